"""The dependent stack (snn_conv_stack_*: layers chained through their packed thresholded signs, one
persistent launch with per-tile completion counters) against the same chain through the CPU oracle:
every layer's signs are an integer decision, so the chain is compared bit for bit."""
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


def _pack_signs(y, shift):
    """fl(Y + shift) >= 0 in fp32, packed along c_out into little-endian uint32 words (oracle side)."""
    y = (y.astype(np.float32) + shift.astype(np.float32)[None, None, None, :]).astype(np.float32)
    bits = y >= 0
    n, h, w, k = bits.shape
    kw = (k + 31) // 32
    pad = np.zeros((n, h, w, kw * 32), dtype=np.uint64)
    pad[..., :k] = bits
    weights = np.uint64(1) << np.arange(32, dtype=np.uint64)
    return (pad.reshape(n, h, w, kw, 32) * weights).sum(axis=-1).astype(np.uint32)


def _build_chain(snn, oracle_mod, shapes, tau, n, seed):
    """Draws the layers, runs the chain through the oracle; returns (layers, first input, per-layer packed
    signs, last layer's (S, Y))."""
    layers, mids = [], []
    x = wl.pack_activation_bits(wl.draw_activation_bits(shapes[0], n, seed))
    first = x
    last = None
    for i, shape in enumerate(shapes):
        p = wl.draw_layer_params(shape, tau, seed + i)
        rng = np.random.default_rng(seed + 100 + i)
        alpha = p.alpha.copy()
        alpha[::7] *= -1.0
        # thresholds of the size of the sums' spread keep the signs balanced through the chain
        shift = (rng.normal(0.0, 1.0, size=shape.c_out) * np.sqrt(9.0 * shape.c_in) * 0.5).astype(np.float32)
        s_ref, y_ref = oracle_mod.conv_bin(p.codebook, tau, p.idx_packed, alpha, shape.c_in, shape.c_out, shape.stride,
                                           shape.pad, x)
        last = (s_ref, y_ref)
        x = _pack_signs(y_ref, shift)
        mids.append(x)
        layers.append(snn.SnnConv(shape.c_in, shape.c_out, tau, p.codebook, p.idx_packed, alpha, shape.stride,
                                  shape.pad, snn.ACT_BIN, shift=shift))
    return layers, first, mids, last


def _check_chain(snn, oracle_mod, shapes, tau, n, seed, repeats=2):
    layers, first, mids, (s_ref, y_ref) = _build_chain(snn, oracle_mod, shapes, tau, n, seed)
    stack = snn.SnnConvStack(layers, n, shapes[0].h, shapes[0].w)
    act = torch.from_numpy(first.view(np.int32)).cuda()
    for _ in range(repeats):
        bits = stack.forward(act, out_type=snn.OUT_BITS)
        sums = stack.forward(act, out_type=snn.OUT_I32)
        outs = stack.forward(act, out_type=snn.OUT_F32)
        torch.cuda.synchronize()
        assert (bits.cpu().numpy().view(np.uint32) == mids[-1]).all()
        assert (sums.cpu().numpy() == s_ref).all()
        assert (outs.cpu().numpy() == y_ref).all()
    stack.destroy()
    for l in layers:
        l.destroy()


def test_stack_of_one(snn, oracle_mod):
    _check_chain(snn, oracle_mod, [wl.LayerShape(16, 16, 32, 32, 1, 1)], 5, 1, 301)


def test_stack_small_ragged_chain(snn, oracle_mod):
    shapes = [wl.LayerShape(33, 40, 13, 11, 1, 1), wl.LayerShape(40, 70, 13, 11, 2, 1), wl.LayerShape(70, 24, 7, 6, 1, 0),
              wl.LayerShape(24, 130, 5, 4, 1, 1), wl.LayerShape(130, 9, 5, 4, 2, 1)]
    _check_chain(snn, oracle_mod, shapes, 5, 3, 311)


@pytest.mark.parametrize("n", [2, 64])
def test_stack_resnet18_full_depth(snn, oracle_mod, n):
    """The 16 ResNet-18-shaped layers as one dependent chain, at batch 2 and at the benchmark's batch 64."""
    wk = wl.get_workload("resnet18")
    _check_chain(snn, oracle_mod, list(wk.layers), wk.tau, n, 321, repeats=1 if n == 64 else 2)


def test_stack_resnet20_full_depth(snn, oracle_mod):
    wk = wl.get_workload("resnet20")
    _check_chain(snn, oracle_mod, list(wk.layers), wk.tau, 4, 331)


def test_stack_argument_errors(snn):
    a = wl.draw_layer_params(wl.LayerShape(16, 32, 8, 8), 5, 3)
    b = wl.draw_layer_params(wl.LayerShape(16, 16, 8, 8), 5, 4)
    la = snn.SnnConv(16, 32, 5, a.codebook, a.idx_packed, a.alpha)
    lb = snn.SnnConv(16, 16, 5, b.codebook, b.idx_packed, b.alpha)
    lf = snn.SnnConv(16, 16, 5, b.codebook, b.idx_packed, b.alpha, act_type=snn.ACT_F16)
    with pytest.raises(snn.SnnError) as ei:
        snn.SnnConvStack([la, lb], 1, 8, 8)          # 32 channels out, 16 in
    assert ei.value.status == 1
    with pytest.raises(snn.SnnError) as ei:
        snn.SnnConvStack([lf], 1, 8, 8)              # fp16 activations do not chain
    assert ei.value.status == 1
    st = snn.SnnConvStack([lb, la], 1, 8, 8)
    with pytest.raises(snn.SnnError) as ei:
        st.forward(torch.zeros((2, 8, 8, 1), dtype=torch.int32, device="cuda"))
    assert ei.value.status == 1
    st.destroy()
    for l in (la, lb, lf):
        l.destroy()
