"""Python face of the CPU oracle (test infrastructure, not the product).

Only tests, the smoke check and the benchmark's host-baseline leg may import
this package.  It wraps `snn_oracle.c` (the definition of the sub-bit 3x3
convolution written out as nested loops, Sec. 3 and Sec. 4.4) through ctypes
and adds `conv_bin_shared_order`, the same sum taken in the order the paper's
shared computation takes it (Sec. 4.5, Fig. 6), which tests use as an invariant.

Nothing here imports or calls the CUDA library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_DIR = Path(__file__).resolve().parent
_SRC = _DIR / "snn_oracle.c"
_LIB = _DIR / "libsnn_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the C oracle with gcc (-O3, OpenMP)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.run(
            ["gcc", "-O3", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", str(tmp), str(_SRC), "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_LIB))
        vp, ci = ctypes.c_void_p, ctypes.c_int
        lib.snn_oracle_threads.restype = ci
        lib.snn_oracle_decode.restype = ci
        lib.snn_oracle_decode.argtypes = [vp, ci, vp, ci, ci, vp]
        lib.snn_oracle_conv_bin.restype = ci
        lib.snn_oracle_conv_bin.argtypes = [vp, ci, vp, vp, ci, ci, ci, ci, vp, ci, ci, ci, vp, vp]
        lib.snn_oracle_conv_f16.restype = ci
        lib.snn_oracle_conv_f16.argtypes = [vp, ci, vp, vp, ci, ci, ci, ci, vp, ci, ci, ci, vp]
        lib.snn_oracle_decode1x1.restype = ci
        lib.snn_oracle_decode1x1.argtypes = [vp, ci, vp, ci, ci, vp]
        lib.snn_oracle_conv1x1_bin.restype = ci
        lib.snn_oracle_conv1x1_bin.argtypes = [vp, ci, vp, vp, ci, ci, ci, vp, ci, ci, ci, vp, vp]
        lib.snn_oracle_conv1x1_f16.restype = ci
        lib.snn_oracle_conv1x1_f16.argtypes = [vp, ci, vp, vp, ci, ci, ci, vp, ci, ci, ci, vp]
        _lib = lib
    return _lib


def threads() -> int:
    """Number of host threads the C oracle's parallel loops use."""
    return int(_load().snn_oracle_threads())


def _ptr(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


def _prep(codebook, idx_packed, alpha):
    cb = np.ascontiguousarray(codebook, dtype=np.uint16)
    ip = np.ascontiguousarray(idx_packed, dtype=np.uint8)
    al = np.ascontiguousarray(alpha, dtype=np.float32)
    return cb, ip, al


def out_hw(h: int, w: int, stride: int, pad: int):
    if stride < 1 or pad < 0 or h + 2 * pad < 3 or w + 2 * pad < 3:
        raise ValueError("bad stride / pad / map size")
    return (h + 2 * pad - 3) // stride + 1, (w + 2 * pad - 3) // stride + 1


def decode_weights(codebook, tau: int, idx_packed, c_in: int, c_out: int) -> np.ndarray:
    """+/-1 weights (c_out, c_in, 3, 3) int8 from the stored form (Sec. 4.1, 4.4)."""
    cb = np.ascontiguousarray(codebook, dtype=np.uint16)
    ip = np.ascontiguousarray(idx_packed, dtype=np.uint8)
    assert cb.size == (1 << tau)
    assert ip.size >= (c_out * c_in * tau + 7) // 8
    w = np.empty((c_out, c_in, 3, 3), dtype=np.int8)
    rc = _load().snn_oracle_decode(_ptr(cb), tau, _ptr(ip), c_in, c_out, _ptr(w))
    if rc:
        raise ValueError(f"oracle decode failed rc={rc}")
    return w


def conv_bin(codebook, tau, idx_packed, alpha, c_in, c_out, stride, pad, act_packed):
    """Binary-activation sub-bit conv.  act_packed: uint32 (N, H, W, ceil(c_in/32)).
    Returns (S int32, Y float32), both (N, Ho, Wo, c_out)."""
    cb, ip, al = _prep(codebook, idx_packed, alpha)
    act = np.ascontiguousarray(act_packed, dtype=np.uint32)
    n, h, w, cw = act.shape
    assert cw == (c_in + 31) // 32 and cb.size == (1 << tau) and al.size == c_out
    assert ip.size >= (c_out * c_in * tau + 7) // 8
    ho, wo = out_hw(h, w, stride, pad)
    s = np.empty((n, ho, wo, c_out), dtype=np.int32)
    y = np.empty((n, ho, wo, c_out), dtype=np.float32)
    rc = _load().snn_oracle_conv_bin(_ptr(cb), tau, _ptr(ip), _ptr(al), c_in, c_out, stride, pad,
                                     _ptr(act), n, h, w, _ptr(s), _ptr(y))
    if rc:
        raise ValueError(f"oracle conv_bin failed rc={rc}")
    return s, y


def conv_f16(codebook, tau, idx_packed, alpha, c_in, c_out, stride, pad, act_f16):
    """Weights-only variant: fp16 activations (N, H, W, c_in), double accumulation.
    Returns Y float32 (N, Ho, Wo, c_out)."""
    cb, ip, al = _prep(codebook, idx_packed, alpha)
    act = np.ascontiguousarray(act_f16, dtype=np.float16)
    n, h, w, c = act.shape
    assert c == c_in and cb.size == (1 << tau) and al.size == c_out
    assert ip.size >= (c_out * c_in * tau + 7) // 8
    ho, wo = out_hw(h, w, stride, pad)
    y = np.empty((n, ho, wo, c_out), dtype=np.float32)
    bits = act.view(np.uint16)
    rc = _load().snn_oracle_conv_f16(_ptr(cb), tau, _ptr(ip), _ptr(al), c_in, c_out, stride, pad,
                                     _ptr(bits), n, h, w, _ptr(y))
    if rc:
        raise ValueError(f"oracle conv_f16 failed rc={rc}")
    return y


def conv_bin_shared_order(codebook, tau, idx, c_in, c_out, stride, pad, act_bits):
    """The paper's shared computation (Sec. 4.5, Fig. 6), in its own order:
    first convolve every input channel with each of the 2^tau codebook kernels
    (the per-channel maps P), then for each output channel add, along c_in, the
    map its index selects.  Inputs are *unpacked* here on purpose: idx is the
    (c_out, c_in) integer array and act_bits the (N, H, W, C) 0/1 array.
    Returns S int64 (N, Ho, Wo, c_out)."""
    codebook = np.asarray(codebook, dtype=np.int64)
    idx = np.asarray(idx, dtype=np.int64)
    a = np.asarray(act_bits, dtype=np.int64) * 2 - 1
    n, h, w, c = a.shape
    assert c == c_in and idx.shape == (c_out, c_in)
    ho, wo = out_hw(h, w, stride, pad)
    ap = np.zeros((n, h + 2 * pad, w + 2 * pad, c), dtype=np.int64)
    ap[:, pad:pad + h, pad:pad + w, :] = a
    t = 1 << tau
    # step 1: P[n, y, x, ci, k]
    p = np.zeros((n, ho, wo, c, t), dtype=np.int64)
    for k in range(t):
        code = int(codebook[k])
        for ky in range(3):
            for kx in range(3):
                sgn = 1 if (code >> (8 - (3 * ky + kx))) & 1 else -1
                win = ap[:, ky:ky + (ho - 1) * stride + 1:stride, kx:kx + (wo - 1) * stride + 1:stride, :]
                p[..., k] += sgn * win
    # step 2: lookup + channel-wise addition
    s = np.zeros((n, ho, wo, c_out), dtype=np.int64)
    for co in range(c_out):
        for ci in range(c_in):
            s[..., co] += p[..., ci, idx[co, ci]]
    return s


# ---------------------------------------------------------------------------------------------
# 1x1 extension (appendix "Extending to Bottleneck with 1x1 Kernels"): 8-input-channel +/-1 vectors
# ---------------------------------------------------------------------------------------------

def out_hw1x1(h: int, w: int, stride: int):
    if stride < 1 or h < 1 or w < 1:
        raise ValueError("bad stride / map size")
    return (h - 1) // stride + 1, (w - 1) // stride + 1


def decode_weights1x1(codebook, tau: int, idx_packed, c_in: int, c_out: int) -> np.ndarray:
    """+/-1 weights (c_out, c_in) int8 of a 1x1 layer from its stored form: tau-bit indices of 8-channel vectors."""
    cb = np.ascontiguousarray(codebook, dtype=np.uint16)
    ip = np.ascontiguousarray(idx_packed, dtype=np.uint8)
    assert cb.size == (1 << tau) and c_in % 8 == 0
    assert ip.size >= (c_out * (c_in // 8) * tau + 7) // 8
    w = np.empty((c_out, c_in), dtype=np.int8)
    rc = _load().snn_oracle_decode1x1(_ptr(cb), tau, _ptr(ip), c_in, c_out, _ptr(w))
    if rc:
        raise ValueError(f"oracle decode1x1 failed rc={rc}")
    return w


def conv1x1_bin(codebook, tau, idx_packed, alpha, c_in, c_out, stride, act_packed):
    """Binary-activation sub-bit 1x1 conv.  Returns (S int32, Y float32), both (N, Ho, Wo, c_out)."""
    cb, ip, al = _prep(codebook, idx_packed, alpha)
    act = np.ascontiguousarray(act_packed, dtype=np.uint32)
    n, h, w, cw = act.shape
    assert cw == (c_in + 31) // 32 and cb.size == (1 << tau) and al.size == c_out
    ho, wo = out_hw1x1(h, w, stride)
    s = np.empty((n, ho, wo, c_out), dtype=np.int32)
    y = np.empty((n, ho, wo, c_out), dtype=np.float32)
    rc = _load().snn_oracle_conv1x1_bin(_ptr(cb), tau, _ptr(ip), _ptr(al), c_in, c_out, stride, _ptr(act), n, h, w,
                                        _ptr(s), _ptr(y))
    if rc:
        raise ValueError(f"oracle conv1x1_bin failed rc={rc}")
    return s, y


def conv1x1_f16(codebook, tau, idx_packed, alpha, c_in, c_out, stride, act_f16):
    """Weights-only 1x1 variant: fp16 activations, double accumulation.  Returns Y float32."""
    cb, ip, al = _prep(codebook, idx_packed, alpha)
    act = np.ascontiguousarray(act_f16, dtype=np.float16)
    n, h, w, c = act.shape
    assert c == c_in and cb.size == (1 << tau) and al.size == c_out
    ho, wo = out_hw1x1(h, w, stride)
    y = np.empty((n, ho, wo, c_out), dtype=np.float32)
    rc = _load().snn_oracle_conv1x1_f16(_ptr(cb), tau, _ptr(ip), _ptr(al), c_in, c_out, stride,
                                        _ptr(act.view(np.uint16)), n, h, w, _ptr(y))
    if rc:
        raise ValueError(f"oracle conv1x1_f16 failed rc={rc}")
    return y


def conv1x1_shared_order(codebook, tau, idx, c_in, c_out, stride, act_bits):
    """The shared computation carried over to 1x1 layers (appendix): first the dot product of every group of
    8 input channels with each of the 2^tau codebook vectors (P), then for each output channel the sum, over
    the groups, of the entry its index selects.  idx is the (c_out, c_in/8) integer array, act_bits the
    (N, H, W, C) 0/1 array.  Returns S int64 (N, Ho, Wo, c_out)."""
    codebook = np.asarray(codebook, dtype=np.int64)
    idx = np.asarray(idx, dtype=np.int64)
    a = (np.asarray(act_bits, dtype=np.int64) * 2 - 1)[:, ::stride, ::stride, :]
    n, ho, wo, c = a.shape
    g = c // 8
    assert c == c_in and idx.shape == (c_out, g)
    t = 1 << tau
    vec = np.array([[1 if (int(codebook[k]) >> (7 - e)) & 1 else -1 for e in range(8)] for k in range(t)], dtype=np.int64)
    p = np.einsum("nhwge,ke->nhwgk", a.reshape(n, ho, wo, g, 8), vec)     # step 1
    s = np.zeros((n, ho, wo, c_out), dtype=np.int64)
    for co in range(c_out):                                              # step 2: lookup + addition over groups
        for gi in range(g):
            s[..., co] += p[..., gi, idx[co, gi]]
    return s
