"""The no-allocation entry point against the ordinary one.

`snn_conv_forward_static` serves hosts that cannot let this library allocate
device memory (the application owns the whole device through its own pool, or
runs with a fixed memory budget, or sits in a loop that cannot take the
synchronisation an allocation may cause).  It keeps its working data in one
fixed array inside the library, shared by all calls.  This test calls it twice
in a row through the C ABI, on two different layers, and checks both results
against `snn_conv_forward` on a handle: the second call must not be affected by
what the first one left in the shared array.  It is collected last so that a
run stopping at the first failure has already run every other test.
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


def _reference(snn, shape, p, act, out_type):
    layer = snn.SnnConv(shape.c_in, shape.c_out, p.tau, p.codebook, p.idx_packed, p.alpha, shape.stride, shape.pad)
    ref = layer.forward(act, out_type=out_type, path=snn.PATH_DECODED)
    torch.cuda.synchronize()
    layer.destroy()
    return ref


def test_two_calls_in_a_row_match_the_handle_path(snn):
    cases = [
        (wl.LayerShape(96, 130, 9, 11, 1, 1), 6, 3, 11),   # first call: larger layer, fills more of the array
        (wl.LayerShape(33, 20, 7, 6, 2, 1), 3, 2, 12),     # second call: smaller layer over stale contents
    ]
    for shape, tau, n, seed in cases:
        p = wl.draw_layer_params(shape, tau, seed)
        bits = wl.draw_activation_bits(shape, n, seed)
        act = torch.from_numpy(wl.pack_activation_bits(bits).view(np.int32)).cuda()
        ho, wo = shape.h_out, shape.w_out
        for out_type, dtype in ((snn.OUT_I32, torch.int32), (snn.OUT_F32, torch.float32)):
            ref = _reference(snn, shape, p, act, out_type)
            out = torch.full((n, ho, wo, shape.c_out), -7, dtype=dtype, device="cuda")
            snn.forward_static(shape.c_in, shape.c_out, tau, p.codebook, p.idx_packed, p.alpha, act, out,
                               stride=shape.stride, pad=shape.pad, out_type=out_type)
            torch.cuda.synchronize()
            if out_type == snn.OUT_I32:
                assert torch.equal(out, ref)                       # integer sums: bit-exact
            else:
                r = ref.cpu().numpy()
                assert (np.abs(out.cpu().numpy() - r) <= 1e-6 * np.abs(r)).all()


def test_sizes_beyond_the_fixed_array_are_refused(snn):
    shape = wl.LayerShape(520, 16, 5, 5, 1, 1)
    p = wl.draw_layer_params(shape, 2, 1)
    act = torch.zeros((1, 5, 5, 17), dtype=torch.int32, device="cuda")
    out = torch.zeros((1, 5, 5, 16), dtype=torch.float32, device="cuda")
    with pytest.raises(snn.SnnError) as ei:
        snn.forward_static(520, 16, 2, p.codebook, p.idx_packed, p.alpha, act, out)
    assert ei.value.status == 2 and "512" in str(ei.value)
