"""The no-allocation entry point against the ordinary one and against the oracle.

`snn_conv_forward_static` serves hosts that cannot let this library allocate
device memory (the application owns the whole device through its own pool, or
runs with a fixed memory budget, or sits in a loop that cannot take the
synchronisation an allocation may cause).  It keeps its working data in one
fixed array inside the library, shared by all calls.  This test calls it twice
in a row through the C ABI, on two different layers, and checks both results
against `snn_conv_forward` on a handle and against the CPU oracle: the second
call must not be affected by what the first one left in the shared array.  It
is collected last so that a run stopping at the first failure has already run
every other test.
"""
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


def _handle_path(snn, shape, p, act, out_type):
    layer = snn.SnnConv(shape.c_in, shape.c_out, p.tau, p.codebook, p.idx_packed, p.alpha, shape.stride, shape.pad)
    ref = layer.forward(act, out_type=out_type, path=snn.PATH_DECODED)
    torch.cuda.synchronize()
    layer.destroy()
    return ref


def _check_case(snn, oracle_mod, shape, tau, n, seed):
    p = wl.draw_layer_params(shape, tau, seed)
    bits = wl.draw_activation_bits(shape, n, seed)
    packed = wl.pack_activation_bits(bits)
    s_ref, y_ref = oracle_mod.conv_bin(p.codebook, tau, p.idx_packed, p.alpha, shape.c_in, shape.c_out, shape.stride,
                                       shape.pad, packed)
    act = torch.from_numpy(packed.view(np.int32)).cuda()
    ho, wo = shape.h_out, shape.w_out
    for out_type, dtype in ((snn.OUT_I32, torch.int32), (snn.OUT_F32, torch.float32)):
        ref = _handle_path(snn, shape, p, act, out_type)
        out = torch.full((n, ho, wo, shape.c_out), -7, dtype=dtype, device="cuda")
        snn.forward_static(shape.c_in, shape.c_out, tau, p.codebook, p.idx_packed, p.alpha, act, out,
                           stride=shape.stride, pad=shape.pad, out_type=out_type)
        torch.cuda.synchronize()
        if out_type == snn.OUT_I32:
            assert torch.equal(out, ref)                       # the existing entry point: bit-exact
            assert (out.cpu().numpy() == s_ref).all()          # the oracle: bit-exact integer sums
        else:
            r = ref.cpu().numpy()
            o = out.cpu().numpy()
            assert (np.abs(o - r) <= 1e-6 * np.abs(r)).all()
            assert (np.abs(o - y_ref) <= 1e-6 * np.abs(y_ref)).all()


def test_two_calls_in_a_row_match_the_handle_path_and_the_oracle(snn, oracle_mod):
    cases = [
        (wl.LayerShape(96, 130, 9, 11, 1, 1), 6, 3, 11),   # first call: larger layer, fills more of the array
        (wl.LayerShape(33, 20, 7, 6, 2, 1), 3, 2, 12),     # second call: smaller layer over stale contents
    ]
    for shape, tau, n, seed in cases:
        _check_case(snn, oracle_mod, shape, tau, n, seed)


def test_largest_layer_the_array_holds(snn, oracle_mod):
    """512 -> 512 channels with the full 512-kernel codebook: the documented upper limit."""
    _check_case(snn, oracle_mod, wl.LayerShape(512, 512, 3, 3, 1, 1), 9, 1, 13)


def test_a_warmed_call_leaves_device_memory_alone(snn):
    shape = wl.LayerShape(64, 48, 8, 8, 1, 1)
    p = wl.draw_layer_params(shape, 5, 14)
    act = torch.from_numpy(wl.pack_activation_bits(wl.draw_activation_bits(shape, 2, 14)).view(np.int32)).cuda()
    out = torch.empty((2, 8, 8, 48), dtype=torch.float32, device="cuda")
    snn.forward_static(64, 48, 5, p.codebook, p.idx_packed, p.alpha, act, out)   # the first call resolves the array
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for _ in range(3):
        snn.forward_static(64, 48, 5, p.codebook, p.idx_packed, p.alpha, act, out)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before


def test_sizes_beyond_the_fixed_array_are_refused(snn):
    shape = wl.LayerShape(520, 16, 5, 5, 1, 1)
    p = wl.draw_layer_params(shape, 2, 1)
    act = torch.zeros((1, 5, 5, 17), dtype=torch.int32, device="cuda")
    out = torch.zeros((1, 5, 5, 16), dtype=torch.float32, device="cuda")
    with pytest.raises(snn.SnnError) as ei:
        snn.forward_static(520, 16, 2, p.codebook, p.idx_packed, p.alpha, act, out)
    assert ei.value.status == 2 and "512" in str(ei.value)


def test_wrong_buffers_are_refused_on_the_host(snn):
    """The C entry point cannot see buffer sizes, so the binding checks them: nothing is launched."""
    shape = wl.LayerShape(64, 48, 8, 8, 1, 1)
    p = wl.draw_layer_params(shape, 5, 15)
    act = torch.zeros((2, 8, 8, 2), dtype=torch.int32, device="cuda")
    good = torch.zeros((2, 8, 8, 48), dtype=torch.float32, device="cuda")
    before = snn.kernel_launches()
    bad_calls = [
        dict(act=torch.zeros((2, 8, 8, 1), dtype=torch.int32, device="cuda"), out=good),            # too few words
        dict(act=act, out=torch.zeros((2, 8, 8, 40), dtype=torch.float32, device="cuda")),          # wrong c_out
        dict(act=act, out=torch.zeros((2, 4, 4, 48), dtype=torch.float32, device="cuda")),          # wrong map
        dict(act=act, out=torch.zeros((2, 8, 8, 48), dtype=torch.int32, device="cuda")),            # wrong dtype
        dict(act=act.to(torch.float32), out=good),                                                   # wrong act dtype
    ]
    for kw in bad_calls:
        with pytest.raises(snn.SnnError) as ei:
            snn.forward_static(64, 48, 5, p.codebook, p.idx_packed, p.alpha, kw["act"], kw["out"])
        assert ei.value.status == 1
    with pytest.raises(snn.SnnError):
        snn.forward_static(64, 48, 5, p.codebook, p.idx_packed, p.alpha, act, good, stride=2)       # out is stride-1 sized
    assert snn.kernel_launches() == before
