"""Parity of the grouped launch (snn_conv_group_*: several independent layer problems
in one persistent tensor-core kernel) with the CPU oracle, member by member and
element by element.  Bar as for single layers: int32 sums bit-exact, fp32 outputs
equal (1e-6 relative), fp16-activation variant within 2e-2 of max(|ref|, alpha*sqrt(9*c_in))."""
import numpy as np
import pytest
import torch

import workloads as wl

pytestmark = pytest.mark.gpu

REL_F32 = 1e-6
REL_F16 = 2e-2


@pytest.fixture(scope="module")
def snn():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2110_09195_b200 import build
    build.build()
    import paper_2110_09195_b200 as m
    m.load_library()
    return m


def _guarded(shape, dtype, guard=64):
    n = int(np.prod(shape))
    flat = torch.full((n + 2 * guard,), -12345 if dtype == torch.int32 else -12345.0, dtype=dtype, device="cuda:0")
    return flat, flat[guard:guard + n].view(*shape)


def _intact(flat, n, guard=64):
    return bool((flat[:guard] == -12345).all()) and bool((flat[guard + n:] == -12345).all())


def check_bin_group(snn, oracle_mod, members, tau, seed, repeats=1):
    """members: list of (LayerShape, batch).  Every member gets its own parameters and input."""
    layers, acts, refs = [], [], []
    for i, (shape, n) in enumerate(members):
        p = wl.draw_layer_params(shape, tau, seed + i)
        packed = wl.pack_activation_bits(wl.draw_activation_bits(shape, n, seed + i))
        refs.append(oracle_mod.conv_bin(p.codebook, tau, p.idx_packed, p.alpha, shape.c_in, shape.c_out, shape.stride,
                                        shape.pad, packed))
        layers.append(snn.SnnConv(shape.c_in, shape.c_out, tau, p.codebook, p.idx_packed, p.alpha, shape.stride,
                                  shape.pad, snn.ACT_BIN))
        acts.append(torch.from_numpy(packed.view(np.int32)).cuda())
    group = snn.SnnConvGroup(layers, [(n, s.h, s.w) for s, n in members])
    for _ in range(repeats):
        gs = [_guarded(r[0].shape, torch.int32) for r in refs]
        gy = [_guarded(r[1].shape, torch.float32) for r in refs]
        group.forward(acts, [g[1] for g in gs], snn.OUT_I32)
        group.forward(acts, [g[1] for g in gy], snn.OUT_F32)
        torch.cuda.synchronize()
        for i, (s_ref, y_ref) in enumerate(refs):
            s, y = gs[i][1].cpu().numpy(), gy[i][1].cpu().numpy()
            assert _intact(gs[i][0], s_ref.size) and _intact(gy[i][0], y_ref.size), f"member {i}: canary overwritten"
            bad = np.argwhere(s != s_ref)
            assert bad.size == 0, f"member {i} {members[i][0]}: {len(bad)} int32 mismatches, first at {bad[0]}: " \
                                  f"{s[tuple(bad[0])]} vs {s_ref[tuple(bad[0])]}"
            assert (np.abs(y - y_ref) <= REL_F32 * np.abs(y_ref)).all(), f"member {i}"
            assert (y == y_ref).all(), f"member {i}"
    group.destroy()
    for l in layers:
        l.destroy()


def test_group_of_one_small(snn, oracle_mod):
    check_bin_group(snn, oracle_mod, [(wl.LayerShape(16, 16, 32, 32, 1, 1), 1)], 5, 11)


def test_group_ragged_members(snn, oracle_mod):
    """Ragged channels in and out, stride 2 (four parity planes), no padding, one-pixel maps,
    several channel blocks: every member shape the kernel treats differently, in one launch."""
    members = [
        (wl.LayerShape(33, 7, 9, 11, 1, 1), 3),
        (wl.LayerShape(70, 37, 13, 6, 2, 1), 2),
        (wl.LayerShape(5, 3, 7, 6, 2, 0), 2),
        (wl.LayerShape(64, 64, 5, 8, 1, 0), 2),
        (wl.LayerShape(16, 16, 1, 1, 1, 1), 5),
        (wl.LayerShape(96, 130, 3, 17, 1, 1), 1),
        (wl.LayerShape(300, 20, 6, 5, 1, 1), 2),
        (wl.LayerShape(1056, 48, 9, 8, 2, 1), 1),
        (wl.LayerShape(200, 300, 7, 5, 1, 1), 2),
    ]
    check_bin_group(snn, oracle_mod, members, 5, 21)


@pytest.mark.parametrize("net,cfg", [("resnet20", 1), ("resnet18", 2)])
def test_group_stack_small_batch(snn, oracle_mod, net, cfg):
    """The whole stack as one group (all layers, in order), batch 2."""
    wk = wl.get_workload(net)
    check_bin_group(snn, oracle_mod, [(s, 2) for s in wk.layers], wk.tau, 31 + cfg, repeats=2)


def test_group_of_32_members(snn, oracle_mod):
    """The largest group the library takes (SNN_GROUP_MAX): the 32 layers of the ResNet-34-shaped stack, batch 2."""
    wk = wl.get_workload("resnet34")
    assert len(wk.layers) == 32
    check_bin_group(snn, oracle_mod, [(s, 2) for s in wk.layers], wk.tau, 35)


def test_group_benchmark_step_at_full_size(snn, oracle_mod):
    """Exactly what bench.py times: the 16 ResNet-18-shaped layers at batch 64 with the benchmark's seeds, as one
    grouped launch.  fp32 outputs of every member against the oracle, element by element."""
    wk = wl.get_workload("resnet18")
    layers, acts, refs = [], [], []
    for i, shape in enumerate(wk.layers):
        seed = wl.layer_seed(wk.config, i)
        p = wl.draw_layer_params(shape, wk.tau, seed)
        packed = wl.pack_activation_bits(wl.draw_activation_bits(shape, wk.batch, seed))
        refs.append(oracle_mod.conv_bin(p.codebook, wk.tau, p.idx_packed, p.alpha, shape.c_in, shape.c_out, shape.stride,
                                        shape.pad, packed)[1])
        layers.append(snn.SnnConv(shape.c_in, shape.c_out, wk.tau, p.codebook, p.idx_packed, p.alpha, shape.stride,
                                  shape.pad, snn.ACT_BIN))
        acts.append(torch.from_numpy(packed.view(np.int32)).cuda())
    group = snn.SnnConvGroup(layers, [(wk.batch, s.h, s.w) for s in wk.layers])
    outs = group.forward(acts, out_type=snn.OUT_F32)
    torch.cuda.synchronize()
    for i, y_ref in enumerate(refs):
        assert (outs[i].cpu().numpy() == y_ref).all(), f"layer {i}"
    group.destroy()
    for l in layers:
        l.destroy()


def test_group_many_tiles_per_cta(snn, oracle_mod):
    """More tiles than twice the CTAs in several members: every ring (activation units, weight
    stages, accumulator buffers) wraps around many times and carries over between members."""
    members = [
        (wl.LayerShape(64, 64, 56, 56, 1, 1), 24),
        (wl.LayerShape(128, 128, 28, 28, 1, 1), 40),
        (wl.LayerShape(64, 128, 56, 56, 2, 1), 12),
        (wl.LayerShape(256, 256, 14, 14, 1, 1), 48),
        (wl.LayerShape(512, 512, 7, 7, 1, 1), 64),
        (wl.LayerShape(256, 512, 14, 14, 2, 1), 16),
    ]
    check_bin_group(snn, oracle_mod, members, 5, 41)


def test_group_fp16(snn, oracle_mod):
    members = [(wl.LayerShape(64, 64, 14, 14, 1, 1), 3), (wl.LayerShape(136, 72, 9, 7, 2, 1), 2),
               (wl.LayerShape(33, 7, 6, 5, 2, 1), 2), (wl.LayerShape(256, 256, 7, 7, 1, 1), 2),
               (wl.LayerShape(64, 64, 56, 56, 1, 1), 10), (wl.LayerShape(128, 256, 28, 28, 2, 1), 24)]  # many tiles per CTA
    layers, acts, refs, alphas = [], [], [], []
    for i, (shape, n) in enumerate(members):
        p = wl.draw_layer_params(shape, 5, 51 + i)
        a = wl.draw_activation_f16(shape, n, 51 + i)
        refs.append(oracle_mod.conv_f16(p.codebook, 5, p.idx_packed, p.alpha, shape.c_in, shape.c_out, shape.stride,
                                        shape.pad, a))
        alphas.append(p.alpha)
        layers.append(snn.SnnConv(shape.c_in, shape.c_out, 5, p.codebook, p.idx_packed, p.alpha, shape.stride,
                                  shape.pad, snn.ACT_F16))
        acts.append(torch.from_numpy(a).cuda())
    group = snn.SnnConvGroup(layers, [(n, s.h, s.w) for s, n in members])
    outs = group.forward(acts)
    torch.cuda.synchronize()
    for i, ((shape, n), y_ref) in enumerate(zip(members, refs)):
        y = outs[i].cpu().numpy().astype(np.float64)
        sigma = alphas[i].astype(np.float64) * np.sqrt(9.0 * shape.c_in)
        bound = REL_F16 * np.maximum(np.abs(y_ref.astype(np.float64)), sigma[None, None, None, :])
        err = np.abs(y - y_ref.astype(np.float64))
        assert (err <= bound).all(), f"member {i}: max err/bound {np.max(err / bound)}"
        assert np.linalg.norm(err) <= 1e-4 * np.linalg.norm(y_ref)
    group.destroy()
    for l in layers:
        l.destroy()


def test_group_argument_errors(snn):
    shape = wl.LayerShape(16, 16, 8, 8)
    p = wl.draw_layer_params(shape, 5, 3)
    a = snn.SnnConv(16, 16, 5, p.codebook, p.idx_packed, p.alpha)
    b = snn.SnnConv(16, 16, 5, p.codebook, p.idx_packed, p.alpha, act_type=snn.ACT_F16)
    with pytest.raises(snn.SnnError) as ei:
        snn.SnnConvGroup([a, b], [(1, 8, 8), (1, 8, 8)])       # mixed activation types
    assert ei.value.status == 1
    with pytest.raises(snn.SnnError) as ei:
        snn.SnnConvGroup([a], [(0, 8, 8)])                     # empty member
    assert ei.value.status == 1
    with pytest.raises(snn.SnnError) as ei:
        snn.SnnConvGroup([a] * 33, [(1, 8, 8)] * 33)           # more members than a group holds
    assert ei.value.status == 1
    g = snn.SnnConvGroup([a], [(1, 8, 8)])
    with pytest.raises(snn.SnnError) as ei:
        g.forward([torch.zeros((2, 8, 8, 1), dtype=torch.int32, device="cuda")])   # not the group's shape
    assert ei.value.status == 1
    g.destroy()
    a.destroy()
    b.destroy()


def _pack_signs(y, shift=None):
    """Oracle-side packing of the thresholded sign (fl(Y + shift) >= 0 -> bit 1, in fp32) along c_out into
    little-endian uint32 words.  Y is the oracle's fp32 output fl(alpha * S)."""
    if shift is not None:
        y = (y.astype(np.float32) + shift.astype(np.float32)[None, None, None, :]).astype(np.float32)
    bits = (y >= 0)
    n, h, w, k = bits.shape
    kw = (k + 31) // 32
    pad = np.zeros((n, h, w, kw * 32), dtype=np.uint64)
    pad[..., :k] = bits
    weights = (np.uint64(1) << np.arange(32, dtype=np.uint64))
    return (pad.reshape(n, h, w, kw, 32) * weights).sum(axis=-1).astype(np.uint32)


def test_group_packed_sign_outputs(snn, oracle_mod):
    """SNN_OUT_BITS: the signs of alpha*S packed as the next layer's input, bit-exact against the
    oracle's outputs; channel counts that are not multiples of 32 or 16, several channel tiles,
    negative scales and exact zeros (an all-zero... S = 0 must give bit 1)."""
    members = [
        (wl.LayerShape(33, 7, 9, 11, 1, 1), 3),
        (wl.LayerShape(70, 37, 13, 6, 2, 1), 2),
        (wl.LayerShape(64, 48, 5, 8, 1, 0), 2),
        (wl.LayerShape(96, 130, 3, 17, 1, 1), 1),
        (wl.LayerShape(40, 300, 6, 5, 1, 1), 2),
        (wl.LayerShape(64, 64, 20, 20, 1, 1), 4),
        (wl.LayerShape(128, 256, 12, 12, 2, 1), 3),
        (wl.LayerShape(64, 512, 7, 7, 1, 1), 3),
        (wl.LayerShape(2, 40, 6, 6, 1, 1), 2),     # tiny c_in: many sums are exactly 0
        (wl.LayerShape(96, 240, 6, 6, 1, 1), 2),   # the widest single channel tile of the packed-sign plan
        (wl.LayerShape(64, 176, 6, 6, 1, 1), 2),   # one tile here, two under the word-output plan
    ]
    layers, acts, refs = [], [], []
    for i, (shape, n) in enumerate(members):
        p = wl.draw_layer_params(shape, 5, 61 + i)
        alpha = p.alpha.copy()
        alpha[::3] *= -1.0                         # negative scales flip the sign
        packed = wl.pack_activation_bits(wl.draw_activation_bits(shape, n, 61 + i))
        _, y_ref = oracle_mod.conv_bin(p.codebook, 5, p.idx_packed, alpha, shape.c_in, shape.c_out, shape.stride,
                                       shape.pad, packed)
        refs.append(_pack_signs(y_ref))
        layers.append(snn.SnnConv(shape.c_in, shape.c_out, 5, p.codebook, p.idx_packed, alpha, shape.stride,
                                  shape.pad, snn.ACT_BIN))
        acts.append(torch.from_numpy(packed.view(np.int32)).cuda())
    group = snn.SnnConvGroup(layers, [(n, s.h, s.w) for s, n in members])
    guarded = [_guarded(r.shape, torch.int32) for r in refs]
    group.forward(acts, [g[1] for g in guarded], snn.OUT_BITS)
    torch.cuda.synchronize()
    for i, ref in enumerate(refs):
        got = guarded[i][1].cpu().numpy().view(np.uint32)
        assert _intact(guarded[i][0], ref.size), f"member {i}: canary overwritten"
        bad = np.argwhere(got != ref)
        assert bad.size == 0, f"member {i} {members[i][0]}: {len(bad)} words differ, first at {bad[0]}: " \
                              f"{got[tuple(bad[0])]:#x} vs {ref[tuple(bad[0])]:#x}"
    group.destroy()
    for l in layers:
        l.destroy()


def test_group_packed_signs_with_channel_thresholds(snn, oracle_mod):
    """SNN_OUT_BITS with a per-channel shift (the folded batch-normalisation threshold): bit = fl(fl(alpha*S) + shift) >= 0.
    Random shifts, negative scales, and channels whose scale is a power of two with a shift of minus a small
    multiple of it, so that many sums land exactly on zero (which must give bit 1) or one step beside it."""
    members = [
        (wl.LayerShape(33, 7, 9, 11, 1, 1), 3),
        (wl.LayerShape(70, 37, 13, 6, 2, 1), 2),
        (wl.LayerShape(64, 48, 5, 8, 1, 0), 2),
        (wl.LayerShape(96, 130, 3, 17, 1, 1), 1),
        (wl.LayerShape(64, 64, 20, 20, 1, 1), 4),
        (wl.LayerShape(128, 256, 12, 12, 2, 1), 3),
        (wl.LayerShape(2, 40, 6, 6, 1, 1), 2),
        (wl.LayerShape(8, 72, 9, 9, 1, 1), 2),
    ]
    layers, acts, refs, yrefs, zeros = [], [], [], [], 0
    for i, (shape, n) in enumerate(members):
        p = wl.draw_layer_params(shape, 5, 161 + i)
        rng = np.random.default_rng(900 + i)
        alpha = p.alpha.copy()
        alpha[::3] *= -1.0
        shift = rng.normal(0.0, 3.0, size=shape.c_out).astype(np.float32)
        ks = np.array([0, 2, -2, 4, 1, 3, -1, 6], dtype=np.float32)
        sel = np.arange(1, shape.c_out, 5)
        alpha[sel] = np.where(np.arange(sel.size) % 2 == 0, 0.5, -0.25).astype(np.float32)
        shift[sel] = -alpha[sel] * ks[np.arange(sel.size) % ks.size]
        packed = wl.pack_activation_bits(wl.draw_activation_bits(shape, n, 161 + i))
        _, y_ref = oracle_mod.conv_bin(p.codebook, 5, p.idx_packed, alpha, shape.c_in, shape.c_out, shape.stride,
                                       shape.pad, packed)
        zeros += int(((y_ref + shift[None, None, None, :]).astype(np.float32) == 0).sum())
        refs.append(_pack_signs(y_ref, shift))
        yrefs.append(y_ref)
        layers.append(snn.SnnConv(shape.c_in, shape.c_out, 5, p.codebook, p.idx_packed, alpha, shape.stride,
                                  shape.pad, snn.ACT_BIN, shift=shift))
        acts.append(torch.from_numpy(packed.view(np.int32)).cuda())
    assert zeros > 100, "the inputs were meant to land many sums exactly on the threshold"
    group = snn.SnnConvGroup(layers, [(n, s.h, s.w) for s, n in members])
    guarded = [_guarded(r.shape, torch.int32) for r in refs]
    group.forward(acts, [g[1] for g in guarded], snn.OUT_BITS)
    torch.cuda.synchronize()
    for i, ref in enumerate(refs):
        got = guarded[i][1].cpu().numpy().view(np.uint32)
        assert _intact(guarded[i][0], ref.size), f"member {i}: canary overwritten"
        bad = np.argwhere(got != ref)
        assert bad.size == 0, f"member {i} {members[i][0]}: {len(bad)} words differ, first at {bad[0]}"
        # the single-layer entry point gives the same words
        one = layers[i].forward(acts[i], out_type=snn.OUT_BITS)
        assert (one.cpu().numpy().view(np.uint32) == ref).all(), f"member {i} through snn_conv_forward"
    # fp32 outputs ignore the shift
    assert (layers[0].forward(acts[0], out_type=snn.OUT_F32).cpu().numpy() == yrefs[0]).all()
    group.destroy()
    for l in layers:
        l.destroy()


def test_group_packed_signs_many_tiles_and_repeatable(snn, oracle_mod):
    """Packed-sign output with more tiles than CTAs (both accumulator buffers, ring wrap-around),
    twice in a row into fresh buffers: bit-exact against the oracle and identical between runs."""
    members = [(wl.LayerShape(64, 64, 56, 56, 1, 1), 12), (wl.LayerShape(128, 128, 28, 28, 1, 1), 24),
               (wl.LayerShape(256, 512, 14, 14, 2, 1), 16)]
    layers, acts, refs = [], [], []
    for i, (shape, n) in enumerate(members):
        p = wl.draw_layer_params(shape, 5, 81 + i)
        packed = wl.pack_activation_bits(wl.draw_activation_bits(shape, n, 81 + i))
        _, y_ref = oracle_mod.conv_bin(p.codebook, 5, p.idx_packed, p.alpha, shape.c_in, shape.c_out, shape.stride,
                                       shape.pad, packed)
        refs.append(_pack_signs(y_ref))
        layers.append(snn.SnnConv(shape.c_in, shape.c_out, 5, p.codebook, p.idx_packed, p.alpha, shape.stride,
                                  shape.pad, snn.ACT_BIN))
        acts.append(torch.from_numpy(packed.view(np.int32)).cuda())
    group = snn.SnnConvGroup(layers, [(n, s.h, s.w) for s, n in members])
    first = [o.cpu().numpy().view(np.uint32) for o in group.forward(acts, out_type=snn.OUT_BITS)]
    second = [o.cpu().numpy().view(np.uint32) for o in group.forward(acts, out_type=snn.OUT_BITS)]
    for i, ref in enumerate(refs):
        assert (first[i] == ref).all(), f"member {i}"
        assert (second[i] == first[i]).all(), f"member {i}: second run differs"
    group.destroy()
    for l in layers:
        l.destroy()


def test_chained_layers_through_packed_signs(snn, oracle_mod):
    """Two layers chained on the GPU (layer 1 writes packed signs, layer 2 reads them as its binary
    input) against the same chain through the oracle."""
    s1, s2, n = wl.LayerShape(64, 96, 14, 14, 1, 1), wl.LayerShape(96, 128, 14, 14, 2, 1), 3
    p1, p2 = wl.draw_layer_params(s1, 5, 71), wl.draw_layer_params(s2, 5, 72)
    packed = wl.pack_activation_bits(wl.draw_activation_bits(s1, n, 71))
    _, y1 = oracle_mod.conv_bin(p1.codebook, 5, p1.idx_packed, p1.alpha, 64, 96, 1, 1, packed)
    mid_ref = _pack_signs(y1)
    s_ref, y_ref = oracle_mod.conv_bin(p2.codebook, 5, p2.idx_packed, p2.alpha, 96, 128, 2, 1, mid_ref)
    l1 = snn.SnnConv(64, 96, 5, p1.codebook, p1.idx_packed, p1.alpha, 1, 1, snn.ACT_BIN)
    l2 = snn.SnnConv(96, 128, 5, p2.codebook, p2.idx_packed, p2.alpha, 2, 1, snn.ACT_BIN)
    g1 = snn.SnnConvGroup([l1], [(n, 14, 14)])
    mid = g1.forward([torch.from_numpy(packed.view(np.int32)).cuda()], out_type=snn.OUT_BITS)[0]
    out = l2.forward(mid, out_type=snn.OUT_F32)
    torch.cuda.synchronize()
    assert (mid.cpu().numpy().view(np.uint32) == mid_ref).all()
    assert (out.cpu().numpy() == y_ref).all()
    # the same chain through the single-layer entry point
    mid1 = l1.forward(torch.from_numpy(packed.view(np.int32)).cuda(), out_type=snn.OUT_BITS)
    out1 = l2.forward(mid1, out_type=snn.OUT_I32)
    torch.cuda.synchronize()
    assert (mid1.cpu().numpy().view(np.uint32) == mid_ref).all()
    assert (out1.cpu().numpy() == s_ref).all()
    with pytest.raises(snn.SnnError) as ei:       # only the tensor-core path writes packed signs
        l1.forward(torch.from_numpy(packed.view(np.int32)).cuda(), out_type=snn.OUT_BITS, path=snn.PATH_DECODED)
    assert ei.value.status == 2
    g1.destroy()
    l1.destroy()
    l2.destroy()


@pytest.mark.parametrize("c_in,c_out,h,w,stride,pad,n", [
    (33, 7, 9, 11, 1, 1, 3), (70, 37, 13, 6, 2, 1, 2), (64, 48, 5, 8, 1, 0, 2), (96, 130, 3, 17, 1, 1, 1),
    (40, 300, 6, 5, 1, 1, 2), (64, 64, 56, 56, 1, 1, 6), (128, 256, 12, 12, 2, 1, 3), (512, 512, 7, 7, 1, 1, 8),
])
def test_single_layer_packed_sign_outputs(snn, oracle_mod, c_in, c_out, h, w, stride, pad, n):
    """SNN_OUT_BITS through snn_conv_forward, through snn_conv_forward_host, and after tuning (whatever
    path the tuner picked for fp32 outputs, packed signs come from the tensor-core path): bit-exact
    against the oracle's outputs."""
    shape = wl.LayerShape(c_in, c_out, h, w, stride, pad)
    p = wl.draw_layer_params(shape, 5, 91)
    alpha = p.alpha.copy()
    alpha[1::4] *= -1.0
    packed = wl.pack_activation_bits(wl.draw_activation_bits(shape, n, 91))
    _, y_ref = oracle_mod.conv_bin(p.codebook, 5, p.idx_packed, alpha, c_in, c_out, stride, pad, packed)
    ref = _pack_signs(y_ref)
    layer = snn.SnnConv(c_in, c_out, 5, p.codebook, p.idx_packed, alpha, stride, pad, snn.ACT_BIN)
    act = torch.from_numpy(packed.view(np.int32)).cuda()
    flat, out = _guarded(ref.shape, torch.int32)
    layer.forward(act, out, snn.OUT_BITS)
    torch.cuda.synchronize()
    assert _intact(flat, ref.size), "canary overwritten"
    assert (out.cpu().numpy().view(np.uint32) == ref).all()
    host = layer.forward_host(torch.from_numpy(packed.view(np.int32)).pin_memory(), out_type=snn.OUT_BITS)
    assert (host.numpy().view(np.uint32) == ref).all()
    layer.tune(n, h, w)
    assert (layer.forward(act, out_type=snn.OUT_BITS).cpu().numpy().view(np.uint32) == ref).all()
    layer.destroy()
