"""Host-side checks of the synthetic workload descriptions and packers."""
import os

import numpy as np
import pytest

import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [l.split() for l in f if l.strip() and not l.startswith("#")]


def test_layer_counts():
    assert len(wl.resnet20_layers()) == 18
    assert len(wl.resnet18_layers()) == 16
    assert len(wl.resnet34_layers()) == 32


def test_layer_lists_reproduce_printed_tables():
    """Tables 1-2: parameter bits and Bit-OPs of the 1-bit rows, and the tau/9
    compressed parameter rows (Sec. 4.4), to the printed precision."""
    lists = {"resnet20": wl.resnet20_layers(), "resnet18": wl.resnet18_layers(), "resnet34": wl.resnet34_layers()}
    for name, p1, ops, p6, p5, p4 in _rows("bitops_tables.txt"):
        ls = lists[name]
        params = sum(9 * l.c_in * l.c_out for l in ls)
        bitops = sum(l.dense_macs(1) for l in ls)

        def printed(v, ref):
            decimals = len(ref.split(".")[1])
            return abs(v - float(ref)) <= 0.5 * 10 ** (-decimals) + 1e-12

        assert printed(params / 1e6, p1), (name, params)
        # the printed Bit-OPs value may carry the "+1" term of Sec. 4.5; it moves only the last digit
        assert abs(bitops / 1e9 - float(ops)) <= 1.5e-3, (name, bitops)
        for tau, ref in ((6, p6), (5, p5), (4, p4)):
            assert printed(params * tau / 9 / 1e6, ref), (name, tau)


def test_storage_sizes():
    for tau, c_in, c_out, ib, cb, bb in _rows("storage_sizes.txt"):
        tau, c_in, c_out = int(tau), int(c_in), int(c_out)
        shape = wl.LayerShape(c_in, c_out, 8, 8)
        p = wl.draw_layer_params(shape, tau, 1)
        assert p.idx_packed.size == (int(ib) + 7) // 8
        assert p.codebook.size * 9 == int(cb)
        assert 9 * c_in * c_out == int(bb)
    # codebook share of a tau=5 ResNet-18/34 layer: 0.01% ~ 0.7% (Sec. 4.4)
    shares = [9 * 32 / (9 * l.c_in * l.c_out) for l in wl.resnet34_layers()]
    assert 0.0001 <= min(shares) < 0.00015 and 0.006 < max(shares) <= 0.008


def test_index_stream_handmade():
    # tau=5, indices 1,2,3 -> LSB-first bits 10000 01000 11000 -> bytes 0x41 0x0C
    packed = wl.pack_indices(np.array([[1, 2, 3]]), 5)
    assert packed.tolist() == [0x41, 0x0C]
    # tau=9 crosses byte borders: 511 then 0 then 256
    packed = wl.pack_indices(np.array([[511, 0, 256]]), 9)
    bits = np.unpackbits(packed, bitorder="little")[:27]
    assert bits[:9].all() and not bits[9:18].any() and bits[18:26].sum() == 0 and bits[26] == 1


def test_pack_indices_rejects_overflow():
    with pytest.raises(ValueError):
        wl.pack_indices(np.array([[32]]), 5)


def test_activation_packing_handmade():
    bits = np.zeros((1, 1, 2, 40), dtype=np.uint8)
    bits[0, 0, 0, 0] = 1
    bits[0, 0, 0, 31] = 1
    bits[0, 0, 0, 32] = 1
    bits[0, 0, 1, 39] = 1
    p = wl.pack_activation_bits(bits)
    assert p.shape == (1, 1, 2, 2) and p.dtype == np.uint32
    assert p[0, 0, 0].tolist() == [0x80000001, 0x1]
    assert p[0, 0, 1].tolist() == [0, 0x80]


def test_draws_are_seeded_and_distinct():
    s = wl.LayerShape(16, 16, 32, 32)
    a = wl.draw_layer_params(s, 5, 7)
    b = wl.draw_layer_params(s, 5, 7)
    assert (a.codebook == b.codebook).all() and (a.idx == b.idx).all() and (a.alpha == b.alpha).all()
    assert len(set(a.codebook.tolist())) == 32 and a.codebook.max() < 512
    assert a.idx.min() >= 0 and a.idx.max() < 32
    assert a.alpha.dtype == np.float32 and a.alpha.min() >= 0.5 and a.alpha.max() < 1.5
    full = wl.draw_layer_params(s, 9, 7)
    assert sorted(full.codebook.tolist()) == list(range(512))
    x = wl.draw_activation_bits(s, 2, 7)
    assert x.shape == (2, 32, 32, 16) and set(np.unique(x)) == {0, 1}
    assert 0.45 < x.mean() < 0.55
    f = wl.draw_activation_f16(s, 2, 7)
    assert f.dtype == np.float16 and abs(float(f.astype(np.float64).std()) - 1.0) < 0.05


def test_workload_totals():
    r18 = wl.get_workload("resnet18")
    assert r18.batch == 64 and r18.tau == 5
    assert abs(r18.dense_macs() / 1e9 - 107.3) < 0.1
    assert abs(r18.algorithmic_bytes() / 1e6 - 398.9) < 0.5
    assert wl.get_workload("tausweep", tau=9).tau == 9
    assert abs(wl.get_workload("resnet34").dense_macs() / 1e9 - 225.7) < 0.1


def test_shard_batch_covers_everything():
    for n in (0, 1, 7, 64, 65):
        for world in (1, 2, 3, 8):
            got = []
            for r in range(world):
                a, b = wl.shard_batch(n, r, world)
                assert 0 <= a <= b <= n
                got += list(range(a, b))
            assert got == list(range(n))


# ------------------------------------------------------- clustered (skewed) indices, Sec. 4.2
def test_skewed_probabilities_follow_the_stated_shares():
    """Sec. 4.2 observation: the 64 most frequent kernels hold more than 70 % of a layer's kernels, and in deep
    layers 8 kernels hold about 60 %.  The generator's probabilities carry exactly these shares."""
    p = wl.skewed_probabilities(512, wl.SKEW_TOP64)
    assert abs(p.sum() - 1) < 1e-12 and abs(np.sort(p)[::-1][:64].sum() - 0.70) < 1e-12
    p = wl.skewed_probabilities(32, wl.SKEW_DEEP)
    assert abs(p.sum() - 1) < 1e-12 and abs(np.sort(p)[::-1][:8].sum() - 0.60) < 1e-12
    assert (np.diff(p[:8]) < 0).all()                        # falling within the frequent entries
    assert np.allclose(p[8:], 0.40 / 24)                     # the rest share the remainder evenly
    q = wl.skewed_probabilities(4, wl.SKEW_DEEP)             # codebook smaller than the frequent set
    assert abs(q.sum() - 1) < 1e-12 and (np.diff(q) < 0).all()


def test_skewed_indices_empirical_frequencies():
    shape = wl.LayerShape(512, 512, 7, 7)
    p = wl.draw_layer_params(shape, 5, 42, index_skew=wl.SKEW_DEEP)
    counts = np.sort(np.bincount(p.idx.reshape(-1), minlength=32))[::-1]
    share = counts[:8].sum() / counts.sum()
    assert abs(share - 0.60) < 0.01
    assert p.idx.min() >= 0 and p.idx.max() < 32
    again = wl.draw_layer_params(shape, 5, 42, index_skew=wl.SKEW_DEEP)
    assert (again.idx == p.idx).all() and (again.codebook == p.codebook).all()      # seeded
    uniform = wl.draw_layer_params(shape, 5, 42)
    assert (uniform.codebook == p.codebook).all()            # same codebook draw, only the indices differ
    # full kernel space (tau = 9): top-64 share
    q = wl.draw_layer_params(wl.LayerShape(256, 256, 14, 14), 9, 43, index_skew=wl.SKEW_TOP64)
    c = np.sort(np.bincount(q.idx.reshape(-1), minlength=512))[::-1]
    assert abs(c[:64].sum() / c.sum() - 0.70) < 0.01


def test_resnet50_1x1_layer_list():
    """32 bottleneck 1x1 layers (3/4/6/3 blocks, two per block), channel counts chaining through the blocks'
    3x3 layers: narrow to the block's width, widen four-fold."""
    ls = wl.resnet50_1x1_layers()
    assert len(ls) == 32 and all(l.ksize == 1 and l.pad == 0 and l.c_in % 8 == 0 for l in ls)
    assert (ls[0].c_in, ls[0].c_out, ls[1].c_in, ls[1].c_out) == (64, 64, 64, 256)
    assert (ls[-2].c_in, ls[-2].c_out, ls[-1].c_in, ls[-1].c_out) == (2048, 512, 512, 2048)
    assert ls[-1].h == 7 and ls[0].h == 56
    p = wl.draw_layer_params(ls[2], 5, 1)
    assert p.idx.shape == (64, 256 // 8) and p.codebook.max() < 256 and len(set(p.codebook.tolist())) == 32
