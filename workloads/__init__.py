"""Seeded synthetic workloads for the sub-bit 3x3 convolution.

This module only *describes* and *draws* inputs: layer shapes, seeded random
codebooks / indices / scales / activations, and the storage packers that put
them in the form the library boundary takes.  It holds none of the method's
arithmetic (no decoding of a code into a kernel, no convolution), so that the
CPU oracle and the CUDA library can both be fed from it without sharing any
computation.

Storage conventions (Sec. 4.1 kernel numbering, Sec. 4.4 storage):
  * codebook entry: 9-bit code, a plain integer in [0, 512);
  * index stream: tau bits per (c_out, c_in) kernel, element e = co*c_in + ci
    occupies bits [e*tau, (e+1)*tau) of an LSB-first byte stream, 0-based;
  * binary activations: uint32 [N][H][W][ceil(c_in/32)], channel ci is bit
    ci % 32 of word ci // 32, bit 1 = +1, bit 0 = -1, unused bits 0;
  * fp16 activations: float16 [N][H][W][c_in].

The layer lists take the shapes of the paper's CIFAR10 / ImageNet ResNets
(Sec. 5, Tables 1-2: first conv, classifier and 1x1 shortcuts excluded); the
datasets themselves are not used.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import List

import numpy as np

BASE_SEED = 20211009


@dataclass(frozen=True)
class LayerShape:
    c_in: int
    c_out: int
    h: int
    w: int
    stride: int = 1
    pad: int = 1
    ksize: int = 3       # 3: the 3x3 layers of the main text; 1: the 1x1 extension of the appendix (pad 0)

    @property
    def h_out(self) -> int:
        return (self.h + 2 * self.pad - self.ksize) // self.stride + 1

    @property
    def w_out(self) -> int:
        return (self.w + 2 * self.pad - self.ksize) // self.stride + 1

    def dense_macs(self, n: int) -> int:
        return n * self.h_out * self.w_out * self.c_out * self.c_in * self.ksize * self.ksize

    def in_bytes_bin(self, n: int) -> int:
        return n * self.h * self.w * ((self.c_in + 31) // 32) * 4

    def in_bytes_f16(self, n: int) -> int:
        return n * self.h * self.w * self.c_in * 2

    def out_bytes(self, n: int) -> int:
        return n * self.h_out * self.w_out * self.c_out * 4


def _stage(c_prev: int, c: int, hw_prev: int, n_convs: int, first_stage: bool) -> List[LayerShape]:
    """Basic-block stage: the first conv of a non-first stage is the stride-2
    channel-doubling conv on the previous stage's map."""
    out: List[LayerShape] = []
    if first_stage:
        out += [LayerShape(c, c, hw_prev, hw_prev, 1)] * n_convs
    else:
        out.append(LayerShape(c_prev, c, hw_prev, hw_prev, 2))
        out += [LayerShape(c, c, hw_prev // 2, hw_prev // 2, 1)] * (n_convs - 1)
    return out


def resnet20_layers() -> List[LayerShape]:
    """18 binary 3x3 layers of the CIFAR ResNet-20 (3 stages x 3 basic blocks)."""
    ls = _stage(16, 16, 32, 6, True)
    ls += _stage(16, 32, 32, 6, False)
    ls += _stage(32, 64, 16, 6, False)
    return ls


def _imagenet_resnet(blocks) -> List[LayerShape]:
    ls = _stage(64, 64, 56, 2 * blocks[0], True)
    ls += _stage(64, 128, 56, 2 * blocks[1], False)
    ls += _stage(128, 256, 28, 2 * blocks[2], False)
    ls += _stage(256, 512, 14, 2 * blocks[3], False)
    return ls


def resnet50_1x1_layers() -> List[LayerShape]:
    """The 32 1x1 layers inside the bottleneck blocks of the ImageNet ResNet-50 (3/4/6/3 blocks; the first 1x1 of a
    block narrows to the block's width, the last widens four-fold; shortcut projections excluded).  The appendix
    applies the 1x1 extension to this architecture."""
    ls: List[LayerShape] = []
    c_prev, hw = 64, 56
    for stage, (width, blocks) in enumerate(((64, 3), (128, 4), (256, 6), (512, 3))):
        for b in range(blocks):
            if stage > 0 and b == 0:
                ls.append(LayerShape(c_prev, width, hw, hw, 1, 0, 1))   # narrows on the previous stage's map
                hw //= 2                                                # the block's 3x3 has stride 2
            else:
                ls.append(LayerShape(c_prev, width, hw, hw, 1, 0, 1))
            ls.append(LayerShape(width, 4 * width, hw, hw, 1, 0, 1))
            c_prev = 4 * width
    return ls


def resnet18_layers() -> List[LayerShape]:
    """16 binary 3x3 layers of the ImageNet ResNet-18 (2/2/2/2 basic blocks)."""
    return _imagenet_resnet((2, 2, 2, 2))


def resnet34_layers() -> List[LayerShape]:
    """32 binary 3x3 layers of the ImageNet ResNet-34 (3/4/6/3 basic blocks)."""
    return _imagenet_resnet((3, 4, 6, 3))


@dataclass(frozen=True)
class Workload:
    name: str
    config: int          # index of the benchmark configuration this stands for
    batch: int
    tau: int
    act: str             # "bin" or "f16"
    layers: tuple

    def dense_macs(self) -> int:
        return sum(l.dense_macs(self.batch) for l in self.layers)

    def algorithmic_bytes(self) -> int:
        """Packed (or fp16) activations in + fp32 outputs out, summed over layers."""
        tot = 0
        for l in self.layers:
            tot += l.in_bytes_bin(self.batch) if self.act == "bin" else l.in_bytes_f16(self.batch)
            tot += l.out_bytes(self.batch)
        return tot

    def with_batch(self, n: int) -> "Workload":
        return replace(self, batch=n)


def get_workload(name: str, tau: int | None = None, batch: int | None = None) -> Workload:
    if name == "single16":
        wl = Workload("single16", 0, 1, 5, "bin", (LayerShape(16, 16, 32, 32, 1),))
    elif name == "resnet20":
        wl = Workload("resnet20", 1, 128, 5, "bin", tuple(resnet20_layers()))
    elif name == "resnet18":
        wl = Workload("resnet18", 2, 64, 5, "bin", tuple(resnet18_layers()))
    elif name == "resnet18_f16":
        wl = Workload("resnet18_f16", 2, 64, 5, "f16", tuple(resnet18_layers()))
    elif name == "resnet34":
        wl = Workload("resnet34", 3, 64, 5, "bin", tuple(resnet34_layers()))
    elif name == "tausweep":
        wl = Workload("tausweep", 4, 64, 5, "bin", (LayerShape(256, 256, 14, 14, 1),))
    elif name == "resnet50_1x1":
        wl = Workload("resnet50_1x1", 5, 64, 5, "bin", tuple(resnet50_1x1_layers()))
    else:
        raise KeyError(name)
    if tau is not None:
        wl = replace(wl, tau=tau)
    if batch is not None:
        wl = replace(wl, batch=batch)
    return wl


WORKLOAD_NAMES = ("single16", "resnet20", "resnet18", "resnet18_f16", "resnet34", "tausweep", "resnet50_1x1")


def layer_seed(config: int, layer_index: int, tau: int | None = None) -> int:
    s = BASE_SEED + 1000 * config + layer_index
    if tau is not None:
        s += 10 * tau
    return s


# ----------------------------------------------------------------------------
# storage packers (formatting only)
# ----------------------------------------------------------------------------

def pack_indices(idx: np.ndarray, tau: int) -> np.ndarray:
    """(c_out, c_in) integers in [0, 2^tau) -> LSB-first tau-bit byte stream."""
    flat = np.ascontiguousarray(idx, dtype=np.uint32).reshape(-1)
    if flat.size and int(flat.max()) >= (1 << tau):
        raise ValueError("index does not fit in tau bits")
    bits = ((flat[:, None] >> np.arange(tau, dtype=np.uint32)[None, :]) & 1).astype(np.uint8)
    return np.packbits(bits.reshape(-1), bitorder="little")


def pack_activation_bits(bits: np.ndarray) -> np.ndarray:
    """(N, H, W, C) array of 0/1 -> uint32 (N, H, W, ceil(C/32)), channel ci at
    bit ci % 32 of word ci // 32."""
    n, h, w, c = bits.shape
    cw = (c + 31) // 32
    padded = np.zeros((n, h, w, cw * 32), dtype=np.uint8)
    padded[..., :c] = bits
    by = np.packbits(padded.reshape(n, h, w, cw * 4, 8), axis=-1, bitorder="little")
    by = np.ascontiguousarray(by.reshape(n, h, w, cw, 4))
    return by.view("<u4").reshape(n, h, w, cw)


# ----------------------------------------------------------------------------
# seeded draws
# ----------------------------------------------------------------------------

@dataclass
class LayerParams:
    tau: int
    codebook: np.ndarray     # (2^tau,) uint16, distinct 9-bit codes
    idx: np.ndarray          # (c_out, c_in) int32 in [0, 2^tau)
    idx_packed: np.ndarray   # uint8 stream
    alpha: np.ndarray        # (c_out,) float32 in [0.5, 1.5)


def draw_layer_params(shape: LayerShape, tau: int, seed: int, index_skew: "IndexSkew | None" = None) -> LayerParams:
    """Random layer-specific subset of the kernel space (Sec. 4.2 sampling distribution; 512 binary 3x3 kernels,
    or the 256 8-channel vectors of a 1x1 layer), indices uniform or, with `index_skew`, concentrated on a few
    codebook entries, and uniform scales."""
    rng = np.random.default_rng(seed)
    t = 1 << tau
    space = 512 if shape.ksize == 3 else 256
    if t > space:
        raise ValueError("codebook larger than the kernel space")
    if t == space:
        codebook = rng.permutation(space).astype(np.uint16)
    else:
        codebook = rng.choice(space, size=t, replace=False).astype(np.uint16)
    cols = shape.c_in if shape.ksize == 3 else shape.c_in // 8
    if shape.ksize == 1 and shape.c_in % 8:
        raise ValueError("a 1x1 layer needs c_in divisible by 8")
    if index_skew is None:
        idx = rng.integers(0, t, size=(shape.c_out, cols), dtype=np.int64).astype(np.int32)
    else:
        idx = draw_skewed_indices(rng, t, (shape.c_out, cols), index_skew)
    alpha = rng.uniform(0.5, 1.5, size=shape.c_out).astype(np.float32)
    return LayerParams(tau, codebook, idx, pack_indices(idx, tau), alpha)


@dataclass(frozen=True)
class IndexSkew:
    """Kernel-frequency profile of a trained layer, as far as Sec. 4.2 states it: the `top` most frequent
    kernels together hold the share `mass` of a layer's kernels (the 64 most frequent of the 512 hold more than
    70 %; in deep layers 8 kernels hold about 60 %); the remaining entries share the rest evenly."""
    top: int
    mass: float


SKEW_TOP64 = IndexSkew(64, 0.70)     # Sec. 4.2: top 64 kernels, > 70 % (meaningful for codebooks larger than 64)
SKEW_DEEP = IndexSkew(8, 0.60)       # Sec. 4.2: 8 kernels, about 60 %, in deep layers


def skewed_probabilities(t: int, skew: IndexSkew) -> np.ndarray:
    """Probability of each of the t codebook entries: the first min(top, t) entries carry `mass` with weights
    falling off harmonically (rank r gets 1/(r+1)), the others share 1 - mass evenly.  With top >= t the whole
    codebook follows the harmonic profile."""
    top = min(skew.top, t)
    head = 1.0 / np.arange(1, top + 1, dtype=np.float64)
    head /= head.sum()
    if top == t:
        return head
    p = np.empty(t, dtype=np.float64)
    p[:top] = head * skew.mass
    p[top:] = (1.0 - skew.mass) / (t - top)
    return p


def draw_skewed_indices(rng, t: int, size, skew: IndexSkew) -> np.ndarray:
    """Indices in [0, t) drawn from skewed_probabilities; the frequent entries sit at a seeded random
    permutation of the codebook slots (a trained layer's frequent kernels are not sorted either)."""
    p = skewed_probabilities(t, skew)
    slots = rng.permutation(t)
    return slots[rng.choice(t, size=size, p=p)].astype(np.int32)


def draw_activation_bits(shape: LayerShape, n: int, seed: int) -> np.ndarray:
    """Bernoulli(1/2) bits, (N, H, W, C) uint8; 1 stands for +1, 0 for -1."""
    rng = np.random.default_rng(seed + 500_000)
    return rng.integers(0, 2, size=(n, shape.h, shape.w, shape.c_in), dtype=np.uint8)


def draw_activation_f16(shape: LayerShape, n: int, seed: int) -> np.ndarray:
    """Standard-normal fp16 activations, (N, H, W, C)."""
    rng = np.random.default_rng(seed + 700_000)
    return rng.standard_normal((n, shape.h, shape.w, shape.c_in), dtype=np.float32).astype(np.float16)


def shard_batch(n: int, rank: int, world: int) -> tuple[int, int]:
    """[start, stop) of the images rank `rank` of `world` owns when a batch of n
    is split as evenly as possible (images are independent, no exchange)."""
    base, rem = divmod(n, world)
    start = rank * base + min(rank, rem)
    return start, start + base + (1 if rank < rem else 0)
