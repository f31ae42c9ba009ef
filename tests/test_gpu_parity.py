"""Parity of the CUDA library (through its C ABI) with the CPU oracle, element
by element on the same seeded inputs.  Bar: int32 pre-scale sums bit-exact;
fp32 outputs within 1e-6 relative (they are in fact expected to be equal: one
exact int->float conversion and one fp32 multiply); fp16-activation variant
within 2e-2 of max(|ref|, alpha*sqrt(9*c_in))."""
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


def _guarded(shape, dtype, device="cuda:0", guard=64):
    """Tensor view with canary words before and after it (16-byte aligned)."""
    n = int(np.prod(shape))
    flat = torch.full((n + 2 * guard,), -12345 if dtype == torch.int32 else -12345.0, dtype=dtype, device=device)
    return flat, flat[guard:guard + n].view(*shape)


def _canaries_intact(flat, n, guard=64):
    head, tail = flat[:guard], flat[guard + n:]
    return bool((head == -12345).all()) and bool((tail == -12345).all())


def _paths(layer, n, h, w):
    from paper_2110_09195_b200 import PATH_REUSE, PATH_DECODED, PATH_DECODED_TC, PATH_AUTO
    ps = [p for p in (PATH_REUSE, PATH_DECODED, PATH_DECODED_TC) if layer.path_supported(p, n, h, w)]
    return ps + [PATH_AUTO]


def check_bin_layer(snn, oracle_mod, shape, tau, n, seed, paths=None):
    p = wl.draw_layer_params(shape, tau, seed)
    bits = wl.draw_activation_bits(shape, n, seed)
    packed = wl.pack_activation_bits(bits)
    s_ref, y_ref = oracle_mod.conv_bin(p.codebook, tau, p.idx_packed, p.alpha, shape.c_in, shape.c_out, shape.stride,
                                       shape.pad, packed)
    layer = snn.SnnConv(shape.c_in, shape.c_out, tau, p.codebook, p.idx_packed, p.alpha, shape.stride, shape.pad,
                        snn.ACT_BIN)
    act = torch.from_numpy(packed.view(np.int32)).cuda()
    ran = []
    for path in (paths or _paths(layer, n, shape.h, shape.w)):
        flat_s, out_s = _guarded(s_ref.shape, torch.int32)
        flat_y, out_y = _guarded(y_ref.shape, torch.float32)
        layer.forward(act, out_s, snn.OUT_I32, path)
        layer.forward(act, out_y, snn.OUT_F32, path)
        torch.cuda.synchronize()
        s = out_s.cpu().numpy()
        y = out_y.cpu().numpy()
        name = snn.PATH_NAMES[path]
        assert _canaries_intact(flat_s, s_ref.size) and _canaries_intact(flat_y, y_ref.size), name
        bad = np.argwhere(s != s_ref)
        assert bad.size == 0, f"path {name}: {len(bad)} int32 mismatches, first at {bad[0]}: " \
                              f"{s[tuple(bad[0])]} vs {s_ref[tuple(bad[0])]}"
        assert (np.abs(y - y_ref) <= REL_F32 * np.abs(y_ref)).all(), name
        assert (y == y_ref).all(), name
        ran.append(path)
    layer.destroy()
    return ran


def test_config0_single_layer(snn, oracle_mod):
    """N=1, 16->16, 32x32, tau=5."""
    wk = wl.get_workload("single16")
    ran = check_bin_layer(snn, oracle_mod, wk.layers[0], wk.tau, wk.batch, wl.layer_seed(0, 0))
    assert snn.PATH_REUSE in ran and snn.PATH_DECODED in ran


@pytest.mark.parametrize("c_in,c_out,h,w,stride,pad,tau,n", [
    (33, 7, 9, 11, 1, 1, 5, 3),      # ragged everything
    (70, 37, 13, 6, 2, 1, 4, 2),
    (5, 3, 7, 6, 2, 0, 3, 2),
    (64, 64, 5, 8, 1, 0, 5, 2),
    (16, 16, 1, 1, 1, 1, 5, 5),      # single pixel map: every tap but the centre is padding
    (32, 40, 2, 1, 2, 1, 2, 3),
    (96, 130, 3, 17, 1, 1, 6, 1),
    (300, 20, 6, 5, 1, 1, 1, 2),     # tau = 1: two kernels
    (2048, 32, 6, 6, 1, 1, 5, 1),    # activations staged in several channel blocks
    (1056, 48, 9, 8, 2, 1, 5, 1),    # the same with the four stride-2 planes
])
def test_ragged_shapes(snn, oracle_mod, c_in, c_out, h, w, stride, pad, tau, n):
    shape = wl.LayerShape(c_in, c_out, h, w, stride, pad)
    check_bin_layer(snn, oracle_mod, shape, tau, n, 1000 + c_in + c_out)


@pytest.mark.parametrize("net,cfg", [("resnet20", 1), ("resnet18", 2)])
def test_stack_shapes_small_batch(snn, oracle_mod, net, cfg):
    """Every distinct layer shape of the stacks, batch cut to 2 so the oracle
    finishes in seconds; tiles still span several CTAs and ragged tails."""
    wk = wl.get_workload(net)
    seen = set()
    for i, shape in enumerate(wk.layers):
        if shape in seen:
            continue
        seen.add(shape)
        check_bin_layer(snn, oracle_mod, shape, wk.tau, 2, wl.layer_seed(cfg, i))


@pytest.mark.parametrize("tau", [1, 2, 3, 4, 5, 6, 7, 8, 9])
def test_tau_sweep_small(snn, oracle_mod, tau):
    """Config-4 layer shape (256->256, 14x14), batch 1, every tau; tau=9 is the
    full codebook, i.e. a plain 1-bit layer."""
    shape = wl.get_workload("tausweep").layers[0]
    check_bin_layer(snn, oracle_mod, shape, tau, 1, wl.layer_seed(4, 0, tau))


def test_empty_batch_and_errors(snn):
    shape = wl.LayerShape(16, 16, 8, 8)
    p = wl.draw_layer_params(shape, 5, 3)
    layer = snn.SnnConv(16, 16, 5, p.codebook, p.idx_packed, p.alpha)
    act = torch.zeros((0, 8, 8, 1), dtype=torch.int32, device="cuda")
    before = snn.kernel_launches()
    out = layer.forward(act)
    assert out.shape == (0, 8, 8, 16) and snn.kernel_launches() == before
    with pytest.raises(snn.SnnError) as ei:
        layer.forward(torch.zeros((1, 8, 8, 1), dtype=torch.int32, device="cuda"), path=7)
    assert ei.value.status == 1
    layer.destroy()
    lay16 = snn.SnnConv(16, 16, 5, p.codebook, p.idx_packed, p.alpha, act_type=snn.ACT_F16)
    with pytest.raises(snn.SnnError) as ei:
        lay16.forward(torch.zeros((1, 8, 8, 16), dtype=torch.float16, device="cuda"), out_type=snn.OUT_I32)
    assert ei.value.status == 1
    lay16.destroy()


def test_deterministic_and_host_entry(snn, oracle_mod):
    shape = wl.LayerShape(64, 64, 14, 14)
    p = wl.draw_layer_params(shape, 5, 5)
    bits = wl.draw_activation_bits(shape, 4, 5)
    packed = wl.pack_activation_bits(bits)
    _, y_ref = oracle_mod.conv_bin(p.codebook, 5, p.idx_packed, p.alpha, 64, 64, 1, 1, packed)
    layer = snn.SnnConv(64, 64, 5, p.codebook, p.idx_packed, p.alpha)
    act = torch.from_numpy(packed.view(np.int32)).cuda()
    a = layer.forward(act).cpu()
    b = layer.forward(act).cpu()
    assert torch.equal(a, b)
    host_in = torch.from_numpy(packed.view(np.int32)).pin_memory()
    y = layer.forward_host(host_in)
    assert (y.numpy() == y_ref).all()
    best, ms = layer.tune(4, 14, 14)
    assert best in (snn.PATH_REUSE, snn.PATH_DECODED, snn.PATH_DECODED_TC)
    assert layer.chosen_path(4, 14, 14) == best and ms[best] > 0
    assert (layer.forward(act).cpu().numpy() == y_ref).all()
    layer.destroy()


def check_f16_layer(snn, oracle_mod, shape, tau, n, seed):
    p = wl.draw_layer_params(shape, tau, seed)
    act_np = wl.draw_activation_f16(shape, n, seed)
    y_ref = oracle_mod.conv_f16(p.codebook, tau, p.idx_packed, p.alpha, shape.c_in, shape.c_out, shape.stride,
                                shape.pad, act_np)
    layer = snn.SnnConv(shape.c_in, shape.c_out, tau, p.codebook, p.idx_packed, p.alpha, shape.stride, shape.pad,
                        snn.ACT_F16)
    act = torch.from_numpy(act_np).cuda()
    ran = []
    for path in _paths(layer, n, shape.h, shape.w):
        flat_y, out_y = _guarded(y_ref.shape, torch.float32)
        layer.forward(act, out_y, snn.OUT_F32, path)
        torch.cuda.synchronize()
        y = out_y.cpu().numpy()
        assert _canaries_intact(flat_y, y_ref.size)
        sigma = p.alpha.astype(np.float64) * np.sqrt(9.0 * shape.c_in)
        bound = REL_F16 * np.maximum(np.abs(y_ref.astype(np.float64)), sigma[None, None, None, :])
        err = np.abs(y.astype(np.float64) - y_ref.astype(np.float64))
        assert (err <= bound).all(), f"path {snn.PATH_NAMES[path]}: max err/bound {np.max(err / bound)}"
        # the accumulation is fp32 over exact products: the norm-wise error is far inside the bound
        assert np.linalg.norm(err) <= 1e-4 * np.linalg.norm(y_ref)
        ran.append(path)
    layer.destroy()
    return ran


@pytest.mark.parametrize("c_in,c_out,h,w,stride,pad,tau,n", [
    (16, 16, 32, 32, 1, 1, 5, 1),
    (64, 64, 14, 14, 1, 1, 5, 2),
    (64, 128, 14, 14, 2, 1, 5, 2),
    (40, 24, 9, 7, 1, 0, 4, 2),
    (33, 7, 6, 5, 2, 1, 3, 2),       # c_in not a multiple of 8: scalar staging
    (256, 256, 7, 7, 1, 1, 5, 1),
])
def test_f16_activation_variant(snn, oracle_mod, c_in, c_out, h, w, stride, pad, tau, n):
    shape = wl.LayerShape(c_in, c_out, h, w, stride, pad)
    ran = check_f16_layer(snn, oracle_mod, shape, tau, n, 2000 + c_in + c_out)
    assert len(ran) >= 2  # at least one named path plus AUTO


@pytest.mark.parametrize("c_in,c_out,h,w,stride,pad,tau,n", [
    (64, 300, 6, 6, 1, 1, 5, 2),     # two output channels per thread
    (8, 520, 5, 5, 2, 1, 9, 2),      # the full codebook: one input channel per table; four channels per thread
    (24, 16, 7, 9, 1, 0, 1, 3),      # two codebook kernels
    (35, 9, 6, 5, 2, 1, 3, 2),       # c_in not a multiple of 8: scalar staging, ragged last chunk
])
def test_f16_codebook_reuse_form(snn, oracle_mod, c_in, c_out, h, w, stride, pad, tau, n):
    """The fp16-activation variant through the codebook-reuse path (the paper's deployment form: signed
    additions once per codebook kernel, then the index-driven accumulation), at the fp16 tolerance."""
    shape = wl.LayerShape(c_in, c_out, h, w, stride, pad)
    ran = check_f16_layer(snn, oracle_mod, shape, tau, n, 97)
    assert snn.PATH_REUSE in ran


def test_tensor_core_path_runs_the_stack_shapes(snn):
    """The tcgen05 path must cover every ResNet-18/34 layer shape at the benchmark batch."""
    wk = wl.get_workload("resnet18")
    for shape in set(wk.layers):
        p = wl.draw_layer_params(shape, 5, 1)
        layer = snn.SnnConv(shape.c_in, shape.c_out, 5, p.codebook, p.idx_packed, p.alpha, shape.stride, shape.pad)
        assert layer.path_supported(snn.PATH_DECODED_TC, wk.batch, shape.h, shape.w)
        layer.destroy()


TC_SHAPES = [
    (64, 64, 20, 20, 1, 3),      # one K step per tap, several tiles per CTA
    (16, 16, 8, 8, 1, 2),        # channels far below one K step and one tile
    (256, 128, 9, 9, 1, 3),      # eight 32-channel chunks in one block
    (128, 256, 12, 12, 2, 3),    # stride 2 (four parity planes), two channel tiles
    (200, 130, 7, 5, 1, 2),      # ragged channels in and out
    (1056, 48, 9, 8, 2, 1),      # several channel blocks, padded
    (512, 512, 7, 7, 1, 4),      # deep layer: two channel blocks, four channel tiles
    (96, 160, 6, 6, 1, 2),       # the widest single channel tile with three accumulator buffers (word outputs)
    (64, 176, 6, 6, 1, 2),       # just beyond it: two tiles, the second mostly padding
    (96, 240, 6, 6, 1, 2),       # the widest single channel tile with two accumulator buffers (packed signs)
    (64, 248, 6, 6, 1, 2),       # just beyond that
    (66, 64, 11, 9, 1, 3),       # an odd number of activation words per pixel: the expanders' plain loop
]


@pytest.mark.parametrize("c_in,c_out,h,w,stride,n", TC_SHAPES)
def test_tensor_core_shapes(snn, oracle_mod, c_in, c_out, h, w, stride, n):
    """The tensor-core path alone (4-bit e2m1 operands, fp32 accumulators) on shapes that exercise its
    channel blocks, channel tiles and parity planes; sums must be exact."""
    shape = wl.LayerShape(c_in, c_out, h, w, stride, 1)
    ran = check_bin_layer(snn, oracle_mod, shape, 5, n, 91, paths=[snn.PATH_DECODED_TC])
    assert ran == [snn.PATH_DECODED_TC]


def test_tensor_core_many_tiles(snn, oracle_mod):
    """More tiles than CTAs: all accumulator buffers, ring wrap-around, weight stages streamed over
    several tiles of one CTA, and a tile assignment with a ragged last round."""
    for shape, n in [(wl.LayerShape(128, 128, 28, 28, 1, 1), 40), (wl.LayerShape(64, 64, 56, 56, 1, 1), 8),
                     (wl.LayerShape(256, 256, 14, 14, 1, 1), 48), (wl.LayerShape(512, 512, 7, 7, 1, 1), 64),
                     (wl.LayerShape(64, 128, 56, 56, 2, 1), 6)]:
        check_bin_layer(snn, oracle_mod, shape, 5, n, 99, paths=[snn.PATH_DECODED_TC])


def test_tensor_core_fp16(snn, oracle_mod):
    for shape, n in [(wl.LayerShape(64, 64, 14, 14, 1, 1), 3), (wl.LayerShape(136, 72, 9, 7, 2, 1), 2),
                     (wl.LayerShape(128, 128, 28, 28, 1, 1), 24)]:
        ran = check_f16_layer(snn, oracle_mod, shape, 5, n, 95)
        assert snn.PATH_DECODED_TC in ran


def test_auto_refuses_a_layer_no_path_can_run(snn):
    """fp16 activations run on the tensor-core path or, up to 1024 output channels, on the reuse path; a layer
    with more channels on a map so wide that one activation unit no longer fits shared memory must be refused
    (status UNSUPPORTED), by name and by AUTO, with nothing launched."""
    shape = wl.LayerShape(16, 1040, 3, 700, 1, 1)
    p = wl.draw_layer_params(shape, 5, 7)
    layer = snn.SnnConv(16, 1040, 5, p.codebook, p.idx_packed, p.alpha, act_type=snn.ACT_F16)
    assert not layer.path_supported(snn.PATH_DECODED_TC, 1, 3, 700)
    assert not layer.path_supported(snn.PATH_REUSE, 1, 3, 700)
    act = torch.zeros((1, 3, 700, 16), dtype=torch.float16, device="cuda")
    before = snn.kernel_launches()
    for path in (snn.PATH_AUTO, snn.PATH_DECODED_TC, snn.PATH_DECODED, snn.PATH_REUSE):
        with pytest.raises(snn.SnnError) as ei:
            layer.forward(act, path=path)
        assert ei.value.status == 2
    assert snn.kernel_launches() == before
    assert layer.chosen_path(1, 3, 700) == snn.PATH_AUTO   # "none"
    layer.destroy()
