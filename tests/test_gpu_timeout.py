"""The bounded device-side waits: a wait that can never end must give up at its attempt limit, report
through the status word the host reads (SNN_ERR_TIMEOUT), let its kernel end normally and leave the
device usable.  The library's self-test (snn_microbench kind 9) makes exactly that happen: one thread
waits, with the helper all kernels wait with, on a barrier nothing arrives on.  Nothing faults or hangs:
the wait is a counted loop."""
import numpy as np
import pytest
import torch

import workloads as wl

pytestmark = pytest.mark.gpu

SNN_ERR_TIMEOUT = 5


@pytest.fixture(scope="module")
def snn():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2110_09195_b200 import build
    build.build()
    import paper_2110_09195_b200 as m
    m.load_library()
    return m


def test_a_wait_nothing_ends_gives_up_and_the_device_stays_usable(snn, oracle_mod):
    with pytest.raises(snn.SnnError) as info:
        snn.microbench(9)
    assert info.value.status == SNN_ERR_TIMEOUT, str(info.value)
    assert "gave up" in str(info.value)
    # the kernel ended by itself: no sticky CUDA error, and the next launch of the library is correct
    torch.cuda.synchronize()
    shape = wl.LayerShape(64, 64, 12, 12, 1, 1)
    tau, n, seed = 5, 2, 4242
    p = wl.draw_layer_params(shape, tau, seed)
    packed = wl.pack_activation_bits(wl.draw_activation_bits(shape, n, seed))
    s_ref, _ = oracle_mod.conv_bin(p.codebook, tau, p.idx_packed, p.alpha, shape.c_in, shape.c_out, shape.stride,
                                   shape.pad, packed)
    layer = snn.SnnConv(shape.c_in, shape.c_out, tau, p.codebook, p.idx_packed, p.alpha, shape.stride, shape.pad,
                        snn.ACT_BIN)
    act = torch.from_numpy(packed.view(np.int32)).cuda()
    out = torch.empty(s_ref.shape, dtype=torch.int32, device="cuda:0")
    before = snn.kernel_launches()
    layer.forward(act, out, snn.OUT_I32, snn.PATH_DECODED_TC)
    torch.cuda.synchronize()
    assert snn.kernel_launches() > before
    assert (out.cpu().numpy() == s_ref).all()
    layer.destroy()
