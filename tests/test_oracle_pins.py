"""Pins for the CPU oracle: it is checked here against things other than
itself -- the paper's numbering endpoints (Sec. 4.1), a library convolution in
the tau=9 case where a sub-bit layer is a plain 1-bit BNN layer (Sec. 4.1-4.2),
the XNOR/bitcount identity (Sec. 3), the sharing equivalence (Sec. 4.5, Fig. 6),
closed forms, and symmetry invariants.  No GPU is involved."""
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _ident9():
    """tau=9 codebook whose slot j holds code j."""
    return np.arange(512, dtype=np.uint16)


def _bits_from_pm1(a):
    return ((np.asarray(a) + 1) // 2).astype(np.uint8)


def _run_bin(oracle, shape, params, bits):
    return oracle.conv_bin(params.codebook, params.tau, params.idx_packed, params.alpha, shape.c_in,
                           shape.c_out, shape.stride, shape.pad, wl.pack_activation_bits(bits))


# ---------------------------------------------------------------- numbering
def test_numbering_endpoints_golden(oracle_mod):
    with open(os.path.join(GOLDEN, "kernel_numbering.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    assert len(rows) == 2
    for row in rows:
        paper_index, code = int(row[0]), int(row[1])
        kernel = np.array([int(v) for v in row[2:]], dtype=np.int8).reshape(3, 3)
        assert code == paper_index - 1
        w = oracle_mod.decode_weights(_ident9(), 9, wl.pack_indices(np.array([[code]]), 9), 1, 1)
        assert (w[0, 0] == kernel).all()


def test_decode_single_plus_one_positions(oracle_mod):
    """Code with one set bit: the +1 sits at the row-major position counted from
    the most significant of the 9 bits."""
    for pos in range(9):
        code = 1 << (8 - pos)
        w = oracle_mod.decode_weights(_ident9(), 9, wl.pack_indices(np.array([[code]]), 9), 1, 1)
        expect = -np.ones(9, dtype=np.int8)
        expect[pos] = 1
        assert (w[0, 0].reshape(-1) == expect).all()


def test_decode_goes_through_codebook_and_stream(oracle_mod):
    """Handmade stream (tau=5, bytes 0x41 0x0C = indices 1,2,3) and a codebook
    whose slots 1,2,3 hold codes 511, 0, 256."""
    cb = np.zeros(32, dtype=np.uint16)
    cb[1], cb[2], cb[3] = 511, 0, 256
    w = oracle_mod.decode_weights(cb, 5, np.array([0x41, 0x0C], dtype=np.uint8), 3, 1)
    assert (w[0, 0] == 1).all() and (w[0, 1] == -1).all()
    assert w[0, 2, 0, 0] == 1 and w[0, 2].sum() == -7
    # (c_out, c_in) row-major order of the stream: same bytes as 3 output channels
    w2 = oracle_mod.decode_weights(cb, 5, np.array([0x41, 0x0C], dtype=np.uint8), 1, 3)
    assert (w2[0, 0] == 1).all() and (w2[1, 0] == -1).all() and w2[2, 0, 0, 0] == 1


# ------------------------------------------------------------- brute force
def test_exhaustive_single_window_xnor_bitcount(oracle_mod):
    """All 512 kernels x all 512 3x3 inputs, pad 0: the +/-1 dot product equals
    9 - 2*bitcount(kernel XOR input) (Sec. 3: XNOR + Bitcount)."""
    codes = np.arange(512)
    # image n is the 3x3 input whose row-major bits spell n, MSB first
    bits = ((codes[:, None] >> (8 - np.arange(9))[None, :]) & 1).astype(np.uint8).reshape(512, 3, 3, 1)
    idx = codes.reshape(512, 1)  # output channel co uses kernel code co
    s, y = oracle_mod.conv_bin(_ident9(), 9, wl.pack_indices(idx, 9), np.ones(512, np.float32), 1, 512, 1, 0,
                               wl.pack_activation_bits(bits))
    assert s.shape == (512, 1, 1, 512)
    x = codes[:, None] ^ codes[None, :]
    pop = np.zeros_like(x)
    for b in range(9):
        pop += (x >> b) & 1
    assert (s[:, 0, 0, :] == 9 - 2 * pop).all()
    assert (y[:, 0, 0, :] == (9 - 2 * pop).astype(np.float32)).all()


@pytest.mark.parametrize("h,w,stride,pad", [(3, 3, 1, 1), (4, 5, 1, 1), (4, 5, 2, 1), (4, 5, 1, 0), (5, 4, 2, 0),
                                            (1, 1, 1, 1), (2, 1, 2, 1)])
def test_brute_force_tiny_maps(oracle_mod, h, w, stride, pad):
    """Element-by-element evaluation from a dictionary of coordinates (a
    different traversal from the oracle's loops), random kernels and inputs."""
    rng = np.random.default_rng(h * 100 + w * 10 + stride + 7 * pad)
    c_in, c_out, n = 3, 4, 2
    codes = rng.integers(0, 512, size=(c_out, c_in))
    bits = rng.integers(0, 2, size=(n, h, w, c_in), dtype=np.uint8)
    alpha = rng.uniform(0.5, 1.5, c_out).astype(np.float32)
    s, y = oracle_mod.conv_bin(_ident9(), 9, wl.pack_indices(codes, 9), alpha, c_in, c_out, stride, pad,
                               wl.pack_activation_bits(bits))
    ho, wo = (h + 2 * pad - 3) // stride + 1, (w + 2 * pad - 3) // stride + 1
    assert s.shape == (n, ho, wo, c_out)
    for img in range(n):
        value = {(r, c, ci): 2 * int(bits[img, r, c, ci]) - 1 for r in range(h) for c in range(w) for ci in range(c_in)}
        for co in range(c_out):
            for yo in range(ho):
                for xo in range(wo):
                    tot = 0
                    for ci in range(c_in):
                        kernel = [1 if (int(codes[co, ci]) >> (8 - p)) & 1 else -1 for p in range(9)]
                        for p, kv in enumerate(kernel):
                            r, c = yo * stride + p // 3 - pad, xo * stride + p % 3 - pad
                            tot += kv * value.get((r, c, ci), 0)
                    assert s[img, yo, xo, co] == tot
                    assert y[img, yo, xo, co] == np.float32(tot) * alpha[co]


# ------------------------------------------------- library routine, tau = 9
@pytest.mark.parametrize("c_in,c_out,h,w,stride,pad", [
    (16, 16, 32, 32, 1, 1), (33, 7, 9, 11, 1, 1), (64, 40, 14, 14, 2, 1), (5, 3, 7, 6, 2, 0), (70, 9, 5, 8, 1, 0)])
def test_tau9_is_a_plain_bnn_conv(oracle_mod, c_in, c_out, h, w, stride, pad):
    """With the full 512-kernel codebook the layer is a standard 1-bit conv:
    compare with torch's conv2d in float64 (exact for these magnitudes)."""
    rng = np.random.default_rng(c_in * 1000 + c_out)
    w_pm1 = rng.integers(0, 2, size=(c_out, c_in, 3, 3)) * 2 - 1
    weights = (8 - np.arange(9)).reshape(3, 3)
    codes = (((w_pm1 + 1) // 2) << weights[None, None]).sum(axis=(2, 3))
    perm = rng.permutation(512)            # any arrangement of all 512 kernels
    inv = np.argsort(perm)
    idx = inv[codes]                       # slot that holds each code
    bits = rng.integers(0, 2, size=(2, h, w, c_in), dtype=np.uint8)
    alpha = rng.uniform(0.5, 1.5, c_out).astype(np.float32)
    s, y = oracle_mod.conv_bin(perm.astype(np.uint16), 9, wl.pack_indices(idx, 9), alpha, c_in, c_out, stride, pad,
                               wl.pack_activation_bits(bits))
    a = torch.from_numpy(bits.astype(np.float64) * 2 - 1).permute(0, 3, 1, 2)
    ref = F.conv2d(a, torch.from_numpy(w_pm1.astype(np.float64)), stride=stride, padding=pad)
    ref = ref.permute(0, 2, 3, 1).numpy()
    assert s.shape == ref.shape
    assert (s == ref).all()
    assert (y == (ref.astype(np.float32) * alpha[None, None, None, :])).all()
    # a transposed tap order or a flipped kernel would not pass this pin
    bad = F.conv2d(a, torch.from_numpy(w_pm1.astype(np.float64)).transpose(2, 3), stride=stride, padding=pad)
    assert not (s == bad.permute(0, 2, 3, 1).numpy()).all()


# -------------------------------------------------------- sharing invariant
@pytest.mark.parametrize("tau,stride,pad", [(1, 1, 1), (3, 2, 1), (5, 1, 1), (5, 2, 0), (7, 1, 0)])
def test_shared_computation_equals_direct(oracle_mod, tau, stride, pad):
    """Sec. 4.5 / Fig. 6: convolving once per codebook kernel and then adding the
    maps the indices select gives the same sums as convolving per filter."""
    shape = wl.LayerShape(10, 12, 7, 9, stride, pad)
    p = wl.draw_layer_params(shape, tau, 99 + tau)
    bits = wl.draw_activation_bits(shape, 2, 99 + tau)
    s, _ = _run_bin(oracle_mod, shape, p, bits)
    shared = oracle_mod.conv_bin_shared_order(p.codebook, tau, p.idx, shape.c_in, shape.c_out, stride, pad, bits)
    assert (s == shared).all()


# ------------------------------------------------------------- closed forms
def _nvalid(h, w, stride, pad):
    ho, wo = (h + 2 * pad - 3) // stride + 1, (w + 2 * pad - 3) // stride + 1
    nv = np.zeros((ho, wo, 9), dtype=np.int64)
    for y in range(ho):
        for x in range(wo):
            for t in range(9):
                r, c = y * stride + t // 3 - pad, x * stride + t % 3 - pad
                nv[y, x, t] = 0 <= r < h and 0 <= c < w
    return nv


@pytest.mark.parametrize("stride,pad", [(1, 1), (2, 1), (1, 0)])
def test_closed_forms_constant_input(oracle_mod, stride, pad):
    c_in, c_out, h, w = 37, 5, 6, 7
    shape = wl.LayerShape(c_in, c_out, h, w, stride, pad)
    ones = np.ones((1, h, w, c_in), dtype=np.uint8)
    nv = _nvalid(h, w, stride, pad)
    cb = np.zeros(32, dtype=np.uint16)
    cb[3], cb[4] = 511, 0
    for t in range(9):
        cb[5 + t] = 1 << (8 - t)           # single +1 at tap t
    alpha = np.linspace(0.5, 1.5, c_out).astype(np.float32)
    # every kernel all +1 -> C * (number of taps inside the image)
    s, y = oracle_mod.conv_bin(cb, 5, wl.pack_indices(np.full((c_out, c_in), 3), 5), alpha, c_in, c_out, stride, pad,
                               wl.pack_activation_bits(ones))
    assert (s == (c_in * nv.sum(-1))[None, :, :, None]).all()
    if stride == 1 and pad == 1:
        assert s[0, 2, 3, 0] == 9 * c_in and s[0, 0, 3, 0] == 6 * c_in and s[0, 0, 0, 0] == 4 * c_in
    assert (y == s.astype(np.float32) * alpha).all()
    # all -1 kernels -> the negative
    s2, _ = oracle_mod.conv_bin(cb, 5, wl.pack_indices(np.full((c_out, c_in), 4), 5), alpha, c_in, c_out, stride, pad,
                                wl.pack_activation_bits(ones))
    assert (s2 == -s).all()
    # single +1 at tap t, output channel co uses tap co
    idx = np.repeat((5 + np.arange(c_out))[:, None], c_in, axis=1)
    s3, _ = oracle_mod.conv_bin(cb, 5, wl.pack_indices(idx, 5), alpha, c_in, c_out, stride, pad,
                                wl.pack_activation_bits(ones))
    for co in range(c_out):
        assert (s3[0, :, :, co] == c_in * (2 * nv[:, :, co] - nv.sum(-1))).all()


def test_single_channel_picks_one_input_bit(oracle_mod):
    """Only channel ci0 of a lone pixel is +1 against a -1 background: tells
    channel order inside and across the packed words."""
    c_in, h, w = 70, 3, 3
    for ci0 in (0, 31, 32, 69):
        bits = np.zeros((1, h, w, c_in), dtype=np.uint8)
        bits[0, 1, 1, ci0] = 1
        # kernel for channel ci is all +1 except ci0's, which is all -1
        cb = np.array([511, 0], dtype=np.uint16)
        idx = np.zeros((1, c_in), dtype=np.int64)
        idx[0, ci0] = 1
        s, _ = oracle_mod.conv_bin(cb, 1, wl.pack_indices(idx, 1), np.ones(1, np.float32), c_in, 1, 1, 0,
                                   wl.pack_activation_bits(bits))
        # all-(-1) input gives -(9*(c_in-1)) + 9; flipping that one bit to +1 under a -1 kernel tap subtracts 2
        assert s[0, 0, 0, 0] == -(9 * (c_in - 1)) + 9 - 2


# --------------------------------------------------------------- invariants
def test_invariants_random(oracle_mod):
    shape = wl.LayerShape(45, 11, 9, 8, 1, 1)
    tau = 4
    p = wl.draw_layer_params(shape, tau, 4242)
    bits = wl.draw_activation_bits(shape, 3, 4242)
    s, y = _run_bin(oracle_mod, shape, p, bits)
    nv = _nvalid(shape.h, shape.w, 1, 1).sum(-1)[None, :, :, None]
    assert ((s - shape.c_in * nv) % 2 == 0).all()
    assert (np.abs(s) <= shape.c_in * nv).all()
    # complementing every activation bit negates S
    s_neg, _ = _run_bin(oracle_mod, shape, p, 1 - bits)
    assert (s_neg == -s).all()
    # complementing every code negates S
    s_cb, _ = oracle_mod.conv_bin(511 - p.codebook, tau, p.idx_packed, p.alpha, shape.c_in, shape.c_out, 1, 1,
                                  wl.pack_activation_bits(bits))
    assert (s_cb == -s).all()
    # permuting codebook slots together with the indices changes nothing
    rng = np.random.default_rng(5)
    perm = rng.permutation(1 << tau)
    cb2 = np.empty_like(p.codebook)
    cb2[perm] = p.codebook
    s_perm, _ = oracle_mod.conv_bin(cb2, tau, wl.pack_indices(perm[p.idx], tau), p.alpha, shape.c_in, shape.c_out, 1, 1,
                                    wl.pack_activation_bits(bits))
    assert (s_perm == s).all()
    # permuting input channels together with the index columns changes nothing
    cperm = rng.permutation(shape.c_in)
    s_ch, _ = oracle_mod.conv_bin(p.codebook, tau, wl.pack_indices(p.idx[:, cperm], tau), p.alpha, shape.c_in,
                                  shape.c_out, 1, 1, wl.pack_activation_bits(bits[..., cperm]))
    assert (s_ch == s).all()
    # scale: one fp32 multiply per element
    assert (y == s.astype(np.float32) * p.alpha[None, None, None, :]).all()


def test_interior_statistics(oracle_mod):
    """Bernoulli(1/2) inputs: interior sums have mean 0 and variance 9*C."""
    shape = wl.LayerShape(64, 32, 16, 16, 1, 1)
    p = wl.draw_layer_params(shape, 5, 11)
    bits = wl.draw_activation_bits(shape, 8, 11)
    s, _ = _run_bin(oracle_mod, shape, p, bits)
    inner = s[:, 1:-1, 1:-1, :].astype(np.float64)
    assert abs(inner.mean()) < 5 * np.sqrt(9 * 64 / inner.size) * 3
    assert abs(inner.var() / (9 * 64) - 1.0) < 0.05


# ------------------------------------------------------------ fp16 variant
def test_f16_all_finite_half_patterns(oracle_mod):
    """Every finite binary16 pattern at the window centre under the all +1
    kernel comes back as its exact value."""
    pats = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    vals = pats.view(np.float16)
    keep = np.isfinite(vals)
    vals = vals[keep]
    act = np.zeros((vals.size, 3, 3, 1), dtype=np.float16)
    act[:, 1, 1, 0] = vals
    y = oracle_mod.conv_f16(np.array([511, 0], np.uint16), 1, wl.pack_indices(np.array([[0]]), 1),
                            np.ones(1, np.float32), 1, 1, 1, 0, act)
    assert (y[:, 0, 0, 0] == vals.astype(np.float32)).all()


def test_f16_equals_binary_on_pm1(oracle_mod):
    shape = wl.LayerShape(40, 9, 6, 7, 2, 1)
    p = wl.draw_layer_params(shape, 5, 31)
    bits = wl.draw_activation_bits(shape, 2, 31)
    _, y_bin = _run_bin(oracle_mod, shape, p, bits)
    y16 = oracle_mod.conv_f16(p.codebook, 5, p.idx_packed, p.alpha, shape.c_in, shape.c_out, 2, 1,
                              (bits.astype(np.float16) * 2 - 1))
    assert (y16 == y_bin).all()


@pytest.mark.parametrize("stride,pad", [(1, 1), (2, 1), (1, 0)])
def test_f16_against_library_conv(oracle_mod, stride, pad):
    shape = wl.LayerShape(24, 10, 9, 10, stride, pad)
    p = wl.draw_layer_params(shape, 5, 77)
    act = wl.draw_activation_f16(shape, 2, 77)
    y = oracle_mod.conv_f16(p.codebook, 5, p.idx_packed, p.alpha, shape.c_in, shape.c_out, stride, pad, act)
    w = oracle_mod.decode_weights(p.codebook, 5, p.idx_packed, shape.c_in, shape.c_out).astype(np.float64)
    ref = F.conv2d(torch.from_numpy(act.astype(np.float64)).permute(0, 3, 1, 2), torch.from_numpy(w),
                   stride=stride, padding=pad).permute(0, 2, 3, 1).numpy()
    ref = ref * p.alpha.astype(np.float64)[None, None, None, :]
    assert np.allclose(y, ref, rtol=1e-6, atol=1e-6)


def test_oracle_rejects_bad_arguments(oracle_mod):
    shape = wl.LayerShape(4, 4, 5, 5)
    p = wl.draw_layer_params(shape, 3, 1)
    bits = wl.pack_activation_bits(wl.draw_activation_bits(shape, 1, 1))
    bad_cb = p.codebook.copy()
    bad_cb[0] = 512
    with pytest.raises(ValueError):
        oracle_mod.conv_bin(bad_cb, 3, p.idx_packed, p.alpha, 4, 4, 1, 1, bits)
    with pytest.raises(ValueError):
        oracle_mod.conv_bin(p.codebook, 3, p.idx_packed, p.alpha, 4, 4, 0, 1, bits)
