"""ctypes binding of include/snn_conv.h: argument marshalling only.

The names mirror the C entry points (snn_conv_create -> SnnConv(...),
snn_conv_forward -> SnnConv.forward, ...).  Tensors are torch CUDA tensors
used purely as device memory; streams come from torch.  There is no fallback:
if the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import numpy as np

ACT_BIN, ACT_F16 = 0, 1
OUT_F32, OUT_I32, OUT_BITS = 0, 1, 2
PATH_AUTO, PATH_REUSE, PATH_DECODED, PATH_DECODED_TC = 0, 1, 2, 3
PATH_NAMES = {PATH_AUTO: "auto", PATH_REUSE: "reuse", PATH_DECODED: "decoded", PATH_DECODED_TC: "decoded_tc"}
_STATUS = {0: "OK", 1: "INVALID_ARG", 2: "UNSUPPORTED", 3: "CUDA", 4: "OOM", 5: "TIMEOUT"}

_LIB_PATH = Path(__file__).resolve().parent / "libsnnconv.so"
_lib = None

# every symbol include/snn_conv.h declares
EXPORTED_SYMBOLS = (
    "snn_conv_create", "snn_conv_forward", "snn_conv_forward_host", "snn_conv_tune", "snn_conv_chosen_path",
    "snn_conv_path_supported", "snn_conv_destroy", "snn_last_error", "snn_version", "snn_kernel_launches",
    "snn_microbench", "snn_conv_forward_static",
    "snn_conv_group_create", "snn_conv_group_forward", "snn_conv_group_destroy",
    "snn_conv_stack_create", "snn_conv_stack_forward", "snn_conv_stack_destroy",
)


class SnnError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"snnconv {_STATUS.get(status, status)}: {message}")
        self.status = status
        self.status_name = _STATUS.get(status, str(status))


class _Desc(ctypes.Structure):
    _fields_ = [
        ("c_in", ctypes.c_int32), ("c_out", ctypes.c_int32), ("tau", ctypes.c_int32),
        ("stride", ctypes.c_int32), ("pad", ctypes.c_int32), ("act_type", ctypes.c_int32),
        ("device", ctypes.c_int32),
        ("codebook", ctypes.c_void_p), ("idx_packed", ctypes.c_void_p), ("alpha", ctypes.c_void_p),
        ("shift", ctypes.c_void_p), ("ksize", ctypes.c_int32),
    ]


def library_path() -> Path:
    return _LIB_PATH


def load_library():
    """Loads libsnnconv.so; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not _LIB_PATH.exists():
        raise ImportError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2110_09195_b200.build` "
            "(nvcc, sm_100a).  This package has no CPU or PyTorch fallback.")
    lib = ctypes.CDLL(str(_LIB_PATH))
    i32, vp = ctypes.c_int32, ctypes.c_void_p
    lib.snn_conv_create.restype = i32
    lib.snn_conv_create.argtypes = [ctypes.POINTER(_Desc), ctypes.POINTER(vp)]
    lib.snn_conv_forward.restype = i32
    lib.snn_conv_forward.argtypes = [vp, vp, i32, i32, i32, vp, i32, i32, vp]
    lib.snn_conv_forward_host.restype = i32
    lib.snn_conv_forward_host.argtypes = [vp, vp, i32, i32, i32, vp, i32, i32]
    lib.snn_conv_tune.restype = i32
    lib.snn_conv_tune.argtypes = [vp, i32, i32, i32, ctypes.POINTER(i32), ctypes.POINTER(ctypes.c_float)]
    lib.snn_conv_chosen_path.restype = i32
    lib.snn_conv_chosen_path.argtypes = [vp, i32, i32, i32]
    lib.snn_conv_path_supported.restype = i32
    lib.snn_conv_path_supported.argtypes = [vp, i32, i32, i32, i32]
    lib.snn_conv_destroy.restype = i32
    lib.snn_conv_destroy.argtypes = [vp]
    lib.snn_last_error.restype = ctypes.c_char_p
    lib.snn_last_error.argtypes = []
    lib.snn_version.restype = ctypes.c_char_p
    lib.snn_version.argtypes = []
    lib.snn_kernel_launches.restype = ctypes.c_int64
    lib.snn_kernel_launches.argtypes = []
    lib.snn_conv_forward_static.restype = i32
    lib.snn_conv_forward_static.argtypes = [ctypes.POINTER(_Desc), vp, i32, i32, i32, vp, i32, vp]
    lib.snn_conv_group_create.restype = i32
    lib.snn_conv_group_create.argtypes = [ctypes.POINTER(vp), i32, ctypes.POINTER(i32), ctypes.POINTER(i32),
                                          ctypes.POINTER(i32), ctypes.POINTER(vp)]
    lib.snn_conv_group_forward.restype = i32
    lib.snn_conv_group_forward.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp), i32, vp]
    lib.snn_conv_group_destroy.restype = i32
    lib.snn_conv_group_destroy.argtypes = [vp]
    lib.snn_conv_stack_create.restype = i32
    lib.snn_conv_stack_create.argtypes = [ctypes.POINTER(vp), i32, i32, i32, i32, ctypes.POINTER(vp)]
    lib.snn_conv_stack_forward.restype = i32
    lib.snn_conv_stack_forward.argtypes = [vp, vp, vp, i32, vp]
    lib.snn_conv_stack_destroy.restype = i32
    lib.snn_conv_stack_destroy.argtypes = [vp]
    lib.snn_microbench.restype = i32
    lib.snn_microbench.argtypes = [i32, i32, ctypes.POINTER(ctypes.c_double)]
    _lib = lib
    return lib


def _check(status: int):
    if status != 0:
        raise SnnError(status, load_library().snn_last_error().decode("utf-8", "replace"))


def version() -> str:
    return load_library().snn_version().decode()


def kernel_launches() -> int:
    return int(load_library().snn_kernel_launches())


def microbench(kind: int, device: int = 0) -> float:
    rate = ctypes.c_double(0.0)
    _check(load_library().snn_microbench(kind, device, ctypes.byref(rate)))
    return float(rate.value)


def forward_static(c_in, c_out, tau, codebook, idx_packed, alpha, act, out, stride=1, pad=1, out_type=OUT_F32,
                   device=0, stream=None):
    """snn_conv_forward_static: one forward pass without any device allocation by the library.

    For hosts that cannot let a library allocate (a device handed over to the
    application's own pool, a fixed memory budget, a loop that cannot take an
    allocation's synchronisation).  The layer is given as host arrays each time;
    `act` and `out` are CUDA tensors the caller already owns.  Binary activations
    only, at most 512 channels in and out.  Calls share one fixed scratch array
    per GPU, so do not let two of them overlap on the device."""
    import torch
    cb = np.ascontiguousarray(codebook, dtype=np.uint16)
    ip = np.ascontiguousarray(idx_packed, dtype=np.uint8)
    al = np.ascontiguousarray(alpha, dtype=np.float32)
    if not 1 <= int(tau) <= 9 or cb.size != (1 << int(tau)):
        raise SnnError(1, "tau outside 1..9 or codebook of the wrong size")
    if ip.size < (int(c_out) * int(c_in) * int(tau) + 7) // 8 or al.size != int(c_out):
        raise SnnError(1, "index stream or alpha of the wrong size")
    if not (act.is_cuda and out.is_cuda and act.is_contiguous() and out.is_contiguous()):
        raise SnnError(1, "act and out must be contiguous CUDA tensors")
    # the C entry point cannot see the sizes of the buffers behind its pointers: check them here
    if act.device.index != int(device) or out.device.index != int(device):
        raise SnnError(1, f"act and out must live on cuda:{device}")
    if act.dtype not in (torch.int32, torch.uint32) or act.dim() != 4 or act.shape[3] != (int(c_in) + 31) // 32:
        raise SnnError(1, "binary activations must be int32/uint32 (N, H, W, ceil(c_in/32))")
    if int(stride) not in (1, 2) or int(pad) not in (0, 1):
        raise SnnError(1, "stride must be 1 or 2 and pad 0 or 1")
    n, h, w = int(act.shape[0]), int(act.shape[1]), int(act.shape[2])
    if h + 2 * int(pad) < 3 or w + 2 * int(pad) < 3:
        raise SnnError(1, "the map is smaller than the kernel")
    ho, wo = (h + 2 * int(pad) - 3) // int(stride) + 1, (w + 2 * int(pad) - 3) // int(stride) + 1
    if out_type not in (OUT_F32, OUT_I32):
        raise SnnError(1, "forward_static writes fp32 or int32 outputs")
    want = torch.float32 if out_type == OUT_F32 else torch.int32
    if out.dtype != want or tuple(out.shape) != (n, ho, wo, int(c_out)):
        raise SnnError(1, f"out must be {want} of shape {(n, ho, wo, int(c_out))}")
    d = _Desc(int(c_in), int(c_out), int(tau), int(stride), int(pad), ACT_BIN, int(device),
              cb.ctypes.data, ip.ctypes.data, al.ctypes.data, None, 3)
    if stream is None:
        stream = torch.cuda.current_stream(device)
    _check(load_library().snn_conv_forward_static(ctypes.byref(d), act.data_ptr(), n, h, w, out.data_ptr(),
                                                  int(out_type), ctypes.c_void_p(stream.cuda_stream)))
    return out


class SnnConv:
    """One sub-bit 3x3 layer on one GPU (wraps a snn_conv_t handle)."""

    def __init__(self, c_in, c_out, tau, codebook, idx_packed, alpha, stride=1, pad=1, act_type=ACT_BIN, device=0,
                 shift=None, ksize=3):
        lib = load_library()
        if int(ksize) not in (1, 3):
            raise SnnError(1, f"ksize={ksize} is not 1 or 3")
        one = int(ksize) == 1
        if one and int(c_in) % 8:
            raise SnnError(1, "a 1x1 layer needs c_in divisible by 8")
        cb = np.ascontiguousarray(codebook, dtype=np.uint16)
        ip = np.ascontiguousarray(idx_packed, dtype=np.uint8)
        al = np.ascontiguousarray(alpha, dtype=np.float32)
        if not 1 <= int(tau) <= (8 if one else 9):
            raise SnnError(1, f"tau={tau} outside 1..{8 if one else 9}")
        if cb.size != (1 << int(tau)):
            raise SnnError(1, f"codebook has {cb.size} entries, expected {1 << int(tau)}")
        units = int(c_out) * (int(c_in) // 8 if one else int(c_in))
        if ip.size < (units * int(tau) + 7) // 8:
            raise SnnError(1, "index stream shorter than one tau-bit index per kernel (or per 8-channel vector)")
        if al.size != int(c_out):
            raise SnnError(1, f"alpha has {al.size} entries, expected {c_out}")
        sh = None if shift is None else np.ascontiguousarray(shift, dtype=np.float32)
        if sh is not None and sh.size != int(c_out):
            raise SnnError(1, f"shift has {sh.size} entries, expected {c_out}")
        d = _Desc(int(c_in), int(c_out), int(tau), int(stride), int(pad), int(act_type), int(device),
                  cb.ctypes.data, ip.ctypes.data, al.ctypes.data, None if sh is None else sh.ctypes.data, int(ksize))
        h = ctypes.c_void_p()
        self._h = None
        _check(lib.snn_conv_create(ctypes.byref(d), ctypes.byref(h)))
        self._h = h
        self.c_in, self.c_out, self.tau = int(c_in), int(c_out), int(tau)
        self.stride, self.pad, self.act_type, self.device = int(stride), int(pad), int(act_type), int(device)
        self.ksize = int(ksize)

    # -- helpers ------------------------------------------------------------
    def out_hw(self, h, w):
        k = self.ksize
        return (h + 2 * self.pad - k) // self.stride + 1, (w + 2 * self.pad - k) // self.stride + 1

    def _check_act(self, act):
        import torch
        if self.act_type == ACT_BIN:
            if act.dtype not in (torch.int32, torch.uint32) or act.dim() != 4 or act.shape[3] != (self.c_in + 31) // 32:
                raise SnnError(1, "binary activations must be int32/uint32 (N, H, W, ceil(c_in/32))")
        else:
            if act.dtype != torch.float16 or act.dim() != 4 or act.shape[3] != self.c_in:
                raise SnnError(1, "fp16 activations must be float16 (N, H, W, c_in)")
        if not act.is_contiguous():
            raise SnnError(1, "activations must be contiguous")

    def alloc_out(self, n, h, w, out_type=OUT_F32, device=None, pin=False):
        import torch
        ho, wo = self.out_hw(h, w)
        dt = torch.float32 if out_type == OUT_F32 else torch.int32
        last = (self.c_out + 31) // 32 if out_type == OUT_BITS else self.c_out   # packed signs: 32 channels a word
        if device is None:
            device = f"cuda:{self.device}"
        if pin:
            return torch.empty((n, ho, wo, last), dtype=dt, pin_memory=True)
        return torch.empty((n, ho, wo, last), dtype=dt, device=device)

    # -- the C entry points -------------------------------------------------
    def forward(self, act, out=None, out_type=OUT_F32, path=PATH_AUTO, stream=None):
        """snn_conv_forward: act / out are CUDA tensors; asynchronous on `stream`
        (default: torch's current stream)."""
        import torch
        if not act.is_cuda or act.device.index != self.device:
            raise SnnError(1, f"activations must live on cuda:{self.device}")
        self._check_act(act)
        n, h, w = int(act.shape[0]), int(act.shape[1]), int(act.shape[2])
        if out is None:
            out = self.alloc_out(n, h, w, out_type)
        else:
            ho, wo = self.out_hw(h, w)
            want = torch.float32 if out_type == OUT_F32 else torch.int32
            last = (self.c_out + 31) // 32 if out_type == OUT_BITS else self.c_out
            if (not out.is_cuda or out.device.index != self.device or out.dtype != want or not out.is_contiguous()
                    or tuple(out.shape) != (n, ho, wo, last)):
                raise SnnError(1, "output tensor has the wrong device, dtype, shape or layout")
        if stream is None:
            stream = torch.cuda.current_stream(self.device)
        _check(load_library().snn_conv_forward(self._h, act.data_ptr(), n, h, w, out.data_ptr(), int(out_type),
                                               int(path), ctypes.c_void_p(stream.cuda_stream)))
        return out

    def forward_host(self, act, out=None, out_type=OUT_F32, path=PATH_AUTO):
        """snn_conv_forward_host: act / out are CPU tensors (pinned for speed);
        synchronous, copies included."""
        import torch
        if act.is_cuda:
            raise SnnError(1, "forward_host takes CPU tensors")
        self._check_act(act)
        n, h, w = int(act.shape[0]), int(act.shape[1]), int(act.shape[2])
        if out is None:
            out = self.alloc_out(n, h, w, out_type, pin=True)
        _check(load_library().snn_conv_forward_host(self._h, act.data_ptr(), n, h, w, out.data_ptr(), int(out_type),
                                                    int(path)))
        return out

    def tune(self, n, h, w):
        """snn_conv_tune: returns (best_path, [ms per path], negative = unsupported)."""
        best = ctypes.c_int32(0)
        ms = (ctypes.c_float * 4)()
        _check(load_library().snn_conv_tune(self._h, int(n), int(h), int(w), ctypes.byref(best), ms))
        return int(best.value), [float(v) for v in ms]

    def chosen_path(self, n, h, w) -> int:
        return int(load_library().snn_conv_chosen_path(self._h, int(n), int(h), int(w)))

    def path_supported(self, path, n, h, w) -> bool:
        st = load_library().snn_conv_path_supported(self._h, int(path), int(n), int(h), int(w))
        if st not in (0, 2):
            _check(st)
        return st == 0

    def destroy(self):
        if getattr(self, "_h", None) is not None:
            load_library().snn_conv_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


class SnnConvGroup:
    """Several independent layer problems run as one persistent launch (wraps snn_conv_group_t).

    `layers` are SnnConv objects of one activation type on one device, `shapes` their input
    shapes (N, H, W).  The members must not depend on each other within one call, and the
    SnnConv objects must outlive the group."""

    def __init__(self, layers, shapes):
        lib = load_library()
        n = len(layers)
        if n != len(shapes) or n < 1:
            raise SnnError(1, "a group needs one (N, H, W) per layer")
        self.layers = list(layers)
        self.shapes = [tuple(int(v) for v in s) for s in shapes]
        hs = (ctypes.c_void_p * n)(*[l._h for l in self.layers])
        i32 = ctypes.c_int32
        ns = (i32 * n)(*[s[0] for s in self.shapes])
        hh = (i32 * n)(*[s[1] for s in self.shapes])
        ww = (i32 * n)(*[s[2] for s in self.shapes])
        g = ctypes.c_void_p()
        self._g = None
        _check(lib.snn_conv_group_create(hs, n, ns, hh, ww, ctypes.byref(g)))
        self._g = g
        self.device = self.layers[0].device

    def alloc_outs(self, out_type=OUT_F32):
        import torch
        if out_type == OUT_BITS:   # packed signs: the next layer's binary activation layout
            return [torch.empty((n, *l.out_hw(h, w), (l.c_out + 31) // 32), dtype=torch.int32,
                                device=f"cuda:{self.device}") for l, (n, h, w) in zip(self.layers, self.shapes)]
        return [l.alloc_out(n, h, w, out_type) for l, (n, h, w) in zip(self.layers, self.shapes)]

    def forward(self, acts, outs=None, out_type=OUT_F32, stream=None):
        """snn_conv_group_forward: acts / outs are lists of CUDA tensors, one per member;
        asynchronous on `stream` (default: torch's current stream)."""
        import torch
        n = len(self.layers)
        if len(acts) != n:
            raise SnnError(1, "one activation tensor per member")
        if outs is None:
            outs = self.alloc_outs(out_type)
        want = torch.float32 if out_type == OUT_F32 else torch.int32
        for l, (nb, h, w), a, o in zip(self.layers, self.shapes, acts, outs):
            last = (l.c_out + 31) // 32 if out_type == OUT_BITS else l.c_out
            if not a.is_cuda or a.device.index != self.device:
                raise SnnError(1, f"activations must live on cuda:{self.device}")
            l._check_act(a)
            ho, wo = l.out_hw(h, w)
            if tuple(a.shape[:3]) != (nb, h, w):
                raise SnnError(1, "activation tensor does not have the shape the group was created for")
            if (not o.is_cuda or o.device.index != self.device or o.dtype != want or not o.is_contiguous()
                    or tuple(o.shape) != (nb, ho, wo, last)):
                raise SnnError(1, "output tensor has the wrong device, dtype, shape or layout")
        if stream is None:
            stream = torch.cuda.current_stream(self.device)
        ap = (ctypes.c_void_p * n)(*[a.data_ptr() for a in acts])
        op = (ctypes.c_void_p * n)(*[o.data_ptr() for o in outs])
        _check(load_library().snn_conv_group_forward(self._g, ap, op, int(out_type),
                                                     ctypes.c_void_p(stream.cuda_stream)))
        return outs

    def destroy(self):
        if getattr(self, "_g", None) is not None:
            load_library().snn_conv_group_destroy(self._g)
            self._g = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


class SnnConvStack:
    """Layers that feed one another through their packed thresholded signs, run as one persistent
    launch (wraps snn_conv_stack_t).  `layers` are SnnConv objects with binary activations whose
    shapes chain; (n, h, w) is the input shape of the first.  The SnnConv objects must outlive the stack."""

    def __init__(self, layers, n, h, w):
        lib = load_library()
        cnt = len(layers)
        if cnt < 1:
            raise SnnError(1, "a stack needs at least one layer")
        self.layers = list(layers)
        self.n, self.h, self.w = int(n), int(h), int(w)
        hs = (ctypes.c_void_p * cnt)(*[l._h for l in self.layers])
        st = ctypes.c_void_p()
        self._s = None
        _check(lib.snn_conv_stack_create(hs, cnt, self.n, self.h, self.w, ctypes.byref(st)))
        self._s = st
        self.device = self.layers[0].device
        ho, wo = self.h, self.w
        for l in self.layers:
            ho, wo = l.out_hw(ho, wo)
        self.out_hw = (ho, wo)

    def alloc_out(self, out_type=OUT_F32):
        import torch
        last = self.layers[-1]
        k = (last.c_out + 31) // 32 if out_type == OUT_BITS else last.c_out
        dt = torch.float32 if out_type == OUT_F32 else torch.int32
        return torch.empty((self.n, *self.out_hw, k), dtype=dt, device=f"cuda:{self.device}")

    def forward(self, act, out=None, out_type=OUT_F32, stream=None):
        """snn_conv_stack_forward: act is the first layer's input, out the last layer's output."""
        import torch
        first = self.layers[0]
        if not act.is_cuda or act.device.index != self.device:
            raise SnnError(1, f"activations must live on cuda:{self.device}")
        first._check_act(act)
        if tuple(act.shape[:3]) != (self.n, self.h, self.w):
            raise SnnError(1, "activation tensor does not have the shape the stack was created for")
        if out is None:
            out = self.alloc_out(out_type)
        last = self.layers[-1]
        k = (last.c_out + 31) // 32 if out_type == OUT_BITS else last.c_out
        dt = torch.float32 if out_type == OUT_F32 else torch.int32
        if (not out.is_cuda or out.device.index != self.device or out.dtype != dt or not out.is_contiguous()
                or tuple(out.shape) != (self.n, *self.out_hw, k)):
            raise SnnError(1, "output tensor has the wrong device, dtype, shape or layout")
        if stream is None:
            stream = torch.cuda.current_stream(self.device)
        _check(load_library().snn_conv_stack_forward(self._s, act.data_ptr(), out.data_ptr(), int(out_type),
                                                     ctypes.c_void_p(stream.cuda_stream)))
        return out

    def destroy(self):
        if getattr(self, "_s", None) is not None:
            load_library().snn_conv_stack_destroy(self._s)
            self._s = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
