"""Parity of the 1x1 extension (appendix "Extending to Bottleneck with 1x1 Kernels": 8-input-channel vectors,
tau'-bit indices) on the tensor-core path with its CPU oracle: int32 sums bit-exact, fp32 outputs equal,
fp16-activation variant within 2e-2 of max(|ref|, alpha*sqrt(c_in))."""
import numpy as np
import pytest
import torch

import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def snn():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2110_09195_b200 import build
    build.build()
    import paper_2110_09195_b200 as m
    m.load_library()
    return m


def _layer(snn, shape, p, act_type, shift=None):
    return snn.SnnConv(shape.c_in, shape.c_out, p.tau, p.codebook, p.idx_packed, p.alpha, shape.stride, 0, act_type,
                       shift=shift, ksize=1)


@pytest.mark.parametrize("c_in,c_out,h,w,stride,tau,n", [
    (8, 16, 5, 7, 1, 3, 2),          # one group of 8 channels
    (64, 64, 14, 14, 1, 5, 3),
    (64, 256, 28, 28, 1, 5, 4),      # widening layer of a bottleneck, two channel tiles, many tiles
    (256, 64, 28, 28, 1, 5, 4),      # narrowing layer
    (40, 37, 9, 6, 2, 4, 2),         # stride 2, ragged output channels
    (2048, 512, 7, 7, 1, 5, 2),      # deepest bottleneck: eight channel blocks
    (128, 24, 6, 5, 1, 8, 2),        # tau' = 8: the full set of 256 vectors
    (72, 130, 3, 3, 1, 1, 1),        # tau' = 1
])
def test_1x1_binary(snn, oracle_mod, c_in, c_out, h, w, stride, tau, n):
    shape = wl.LayerShape(c_in, c_out, h, w, stride, 0, 1)
    p = wl.draw_layer_params(shape, tau, 400 + c_in + c_out)
    packed = wl.pack_activation_bits(wl.draw_activation_bits(shape, n, 400 + c_in))
    s_ref, y_ref = oracle_mod.conv1x1_bin(p.codebook, tau, p.idx_packed, p.alpha, c_in, c_out, stride, packed)
    layer = _layer(snn, shape, p, snn.ACT_BIN)
    assert layer.path_supported(snn.PATH_DECODED_TC, n, h, w)
    assert not layer.path_supported(snn.PATH_DECODED, n, h, w) and not layer.path_supported(snn.PATH_REUSE, n, h, w)
    act = torch.from_numpy(packed.view(np.int32)).cuda()
    for path in (snn.PATH_DECODED_TC, snn.PATH_AUTO):
        s = layer.forward(act, out_type=snn.OUT_I32, path=path)
        y = layer.forward(act, out_type=snn.OUT_F32, path=path)
        torch.cuda.synchronize()
        assert s.shape == s_ref.shape
        assert (s.cpu().numpy() == s_ref).all()
        assert (y.cpu().numpy() == y_ref).all()
    layer.destroy()


def test_1x1_fp16(snn, oracle_mod):
    for shape, n in [(wl.LayerShape(64, 256, 14, 14, 1, 0, 1), 3), (wl.LayerShape(136, 40, 9, 7, 2, 0, 1), 2)]:
        p = wl.draw_layer_params(shape, 5, 450)
        a = wl.draw_activation_f16(shape, n, 450)
        y_ref = oracle_mod.conv1x1_f16(p.codebook, 5, p.idx_packed, p.alpha, shape.c_in, shape.c_out, shape.stride, a)
        layer = _layer(snn, shape, p, snn.ACT_F16)
        y = layer.forward(torch.from_numpy(a).cuda()).cpu().numpy().astype(np.float64)
        sigma = p.alpha.astype(np.float64) * np.sqrt(float(shape.c_in))
        bound = 2e-2 * np.maximum(np.abs(y_ref.astype(np.float64)), sigma[None, None, None, :])
        assert (np.abs(y - y_ref) <= bound).all()
        layer.destroy()


def _pack_signs(y, shift):
    y = (y.astype(np.float32) + shift.astype(np.float32)[None, None, None, :]).astype(np.float32)
    bits = y >= 0
    n, h, w, k = bits.shape
    kw = (k + 31) // 32
    pad = np.zeros((n, h, w, kw * 32), dtype=np.uint64)
    pad[..., :k] = bits
    weights = np.uint64(1) << np.arange(32, dtype=np.uint64)
    return (pad.reshape(n, h, w, kw, 32) * weights).sum(axis=-1).astype(np.uint32)


def test_bottleneck_as_a_stack(snn, oracle_mod):
    """A ResNet-50 bottleneck (1x1 narrowing, 3x3 with stride 2, 1x1 widening) chained through packed thresholded
    signs in one launch, against the same chain through the oracles."""
    n = 3
    shapes = [wl.LayerShape(256, 128, 28, 28, 1, 0, 1), wl.LayerShape(128, 128, 28, 28, 2, 1, 3),
              wl.LayerShape(128, 512, 14, 14, 1, 0, 1)]
    x = wl.pack_activation_bits(wl.draw_activation_bits(shapes[0], n, 470))
    first, layers = x, []
    for i, shape in enumerate(shapes):
        p = wl.draw_layer_params(shape, 5, 470 + i)
        rng = np.random.default_rng(480 + i)
        shift = (rng.normal(0.0, 1.0, size=shape.c_out) * np.sqrt(shape.c_in * shape.ksize ** 2) * 0.5).astype(np.float32)
        if shape.ksize == 1:
            s_ref, y_ref = oracle_mod.conv1x1_bin(p.codebook, 5, p.idx_packed, p.alpha, shape.c_in, shape.c_out,
                                                  shape.stride, x)
        else:
            s_ref, y_ref = oracle_mod.conv_bin(p.codebook, 5, p.idx_packed, p.alpha, shape.c_in, shape.c_out,
                                               shape.stride, shape.pad, x)
        x = _pack_signs(y_ref, shift)
        layers.append(snn.SnnConv(shape.c_in, shape.c_out, 5, p.codebook, p.idx_packed, p.alpha, shape.stride,
                                  shape.pad, snn.ACT_BIN, shift=shift, ksize=shape.ksize))
    stack = snn.SnnConvStack(layers, n, 28, 28)
    act = torch.from_numpy(first.view(np.int32)).cuda()
    assert (stack.forward(act, out_type=snn.OUT_I32).cpu().numpy() == s_ref).all()
    assert (stack.forward(act, out_type=snn.OUT_BITS).cpu().numpy().view(np.uint32) == x).all()
    stack.destroy()
    for l in layers:
        l.destroy()


def test_1x1_argument_errors(snn):
    shape = wl.LayerShape(16, 8, 4, 4, 1, 0, 1)
    p = wl.draw_layer_params(shape, 3, 1)
    with pytest.raises(snn.SnnError) as ei:      # c_in not divisible by 8
        snn.SnnConv(12, 8, 3, p.codebook, p.idx_packed, p.alpha, 1, 0, ksize=1)
    assert ei.value.status == 1
    with pytest.raises(snn.SnnError) as ei:      # padding
        snn.SnnConv(16, 8, 3, p.codebook, p.idx_packed, p.alpha, 1, 1, ksize=1)
    assert ei.value.status == 1
    bad = p.codebook.copy()
    bad[0] = 300
    with pytest.raises(snn.SnnError) as ei:      # not an 8-bit code
        snn.SnnConv(16, 8, 3, bad, p.idx_packed, p.alpha, 1, 0, ksize=1)
    assert ei.value.status == 1
    with pytest.raises(snn.SnnError) as ei:      # tau' = 9
        snn.SnnConv(16, 8, 9, np.zeros(512, np.uint16), p.idx_packed, p.alpha, 1, 0, ksize=1)
    assert ei.value.status == 1
