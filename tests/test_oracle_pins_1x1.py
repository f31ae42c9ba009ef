"""Pins of the 1x1-extension oracle (appendix "Extending to Bottleneck with 1x1 Kernels"): numbering endpoints,
the full-codebook case against a library 1x1 convolution, the XNOR/bitcount identity on every pair of 8-channel
vectors, brute force from a coordinate dictionary, the sharing invariant, closed forms and invariants.  No GPU."""
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _pm1_to_packed(a_pm1):
    return wl.pack_activation_bits(((a_pm1 + 1) // 2).astype(np.uint8))


def test_numbering_endpoints_golden(oracle_mod):
    rows = [l.split() for l in open(os.path.join(GOLDEN, "vector_numbering_1x1.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 2
    for paper_idx, code, *entries in rows:
        assert int(paper_idx) == int(code) + 1
        cb = np.array([int(code), 0], dtype=np.uint16)            # tau = 1, index 0 everywhere
        w = oracle_mod.decode_weights1x1(cb, 1, wl.pack_indices(np.zeros((1, 1), np.int32), 1), 8, 1)
        assert w.reshape(-1).tolist() == [int(e) for e in entries]


def test_single_plus_one_positions(oracle_mod):
    """Code with only bit 7 - j set: +1 at vector element j (first element most significant), -1 elsewhere."""
    for j in range(8):
        cb = np.array([1 << (7 - j), 0], dtype=np.uint16)
        w = oracle_mod.decode_weights1x1(cb, 1, wl.pack_indices(np.zeros((1, 1), np.int32), 1), 8, 1).reshape(-1)
        assert w[j] == 1 and (np.delete(w, j) == -1).all()


def test_decode_goes_through_codebook_stream_and_groups(oracle_mod):
    """Hand-made: two output channels, 16 input channels (two groups), tau = 2; element e = co * 2 + g."""
    cb = np.array([0b00000000, 0b11111111, 0b10000000, 0b00000001], dtype=np.uint16)
    idx = np.array([[2, 1], [3, 0]], dtype=np.int32)
    stream = wl.pack_indices(idx, 2)
    assert stream.tolist() == [0b00110110]            # 2 | 1<<2 | 3<<4 | 0<<6
    w = oracle_mod.decode_weights1x1(cb, 2, stream, 16, 2)
    assert w[0].tolist() == [1, -1, -1, -1, -1, -1, -1, -1] + [1] * 8
    assert w[1].tolist() == [-1] * 7 + [1] + [-1] * 8


def test_exhaustive_vector_pairs_xnor_bitcount(oracle_mod):
    """Every weight vector against every activation vector on one pixel: the +/-1 dot product equals
    8 - 2 * popcount(code_w XOR code_a) with the activation vector coded the same way (Sec. 3: XNOR + bitcount)."""
    codes = np.arange(256)
    a = np.array([[1 if (c >> (7 - e)) & 1 else -1 for e in range(8)] for c in codes], dtype=np.int64)   # (256, 8)
    packed = _pm1_to_packed(a.reshape(256, 1, 1, 8))
    cb = codes.astype(np.uint16)
    idx = np.arange(256, dtype=np.int32).reshape(256, 1)
    s, _ = oracle_mod.conv1x1_bin(cb, 8, wl.pack_indices(idx, 8), np.ones(256, np.float32), 8, 256, 1, packed)
    s = s.reshape(256, 256)                                         # [activation code][weight code]
    x = codes[:, None] ^ codes[None, :]
    pop = np.array([bin(v).count("1") for v in range(256)])[x]
    assert (s == 8 - 2 * pop).all()


@pytest.mark.parametrize("c_in,c_out,h,w,stride", [(8, 3, 3, 4, 1), (24, 5, 5, 4, 2), (16, 2, 1, 1, 1), (40, 7, 6, 7, 3)])
def test_full_codebook_is_a_plain_1x1_conv(oracle_mod, c_in, c_out, h, w, stride):
    """tau' = 8 with all 256 vectors: indices are the codes of arbitrary +/-1 weights, and the layer is an ordinary
    1-bit 1x1 convolution (library routine, float64: exact).  A mutant with the channel order inside the groups
    reversed must differ."""
    rng = np.random.default_rng(5 + c_in + c_out)
    wts = rng.integers(0, 2, size=(c_out, c_in)) * 2 - 1
    perm = rng.permutation(256)
    inv = np.argsort(perm)
    codes = np.zeros((c_out, c_in // 8), dtype=np.int64)
    for e in range(8):
        codes |= ((wts[:, e::8] + 1) // 2) << (7 - e)
    idx = inv[codes].astype(np.int32)                    # slot that holds the code
    n = 2
    a = rng.integers(0, 2, size=(n, h, w, c_in)) * 2 - 1
    alpha = rng.uniform(0.5, 1.5, c_out).astype(np.float32)
    s, y = oracle_mod.conv1x1_bin(perm.astype(np.uint16), 8, wl.pack_indices(idx, 8), alpha, c_in, c_out, stride,
                                  _pm1_to_packed(a))
    ref = F.conv2d(torch.from_numpy(a).double().permute(0, 3, 1, 2), torch.from_numpy(wts).double()[:, :, None, None],
                   stride=stride).permute(0, 2, 3, 1).numpy()
    assert (s == ref).all()
    assert (y == (ref.astype(np.float32) * alpha[None, None, None, :])).all()
    mutant = wts.reshape(c_out, c_in // 8, 8)[:, :, ::-1].reshape(c_out, c_in)
    ref_m = F.conv2d(torch.from_numpy(a).double().permute(0, 3, 1, 2), torch.from_numpy(mutant.copy()).double()[:, :, None, None],
                     stride=stride).permute(0, 2, 3, 1).numpy()
    if c_in > 8 or True:
        assert not (s == ref_m).all()


def test_brute_force_from_a_coordinate_dictionary(oracle_mod):
    rng = np.random.default_rng(77)
    c_in, c_out, h, w, stride, n, tau = 16, 4, 4, 5, 2, 2, 3
    cb = rng.choice(256, size=8, replace=False).astype(np.uint16)
    idx = rng.integers(0, 8, size=(c_out, 2)).astype(np.int32)
    bits = rng.integers(0, 2, size=(n, h, w, c_in)).astype(np.uint8)
    act = {(b, r, c, ci): (1 if bits[b, r, c, ci] else -1) for b in range(n) for r in range(h) for c in range(w)
           for ci in range(c_in)}
    s, _ = oracle_mod.conv1x1_bin(cb, tau, wl.pack_indices(idx, tau), np.ones(c_out, np.float32), c_in, c_out, stride,
                                  wl.pack_activation_bits(bits))
    for b in range(n):
        for y in range((h - 1) // stride + 1):
            for x in range((w - 1) // stride + 1):
                for co in range(c_out):
                    tot = 0
                    for ci in range(c_in):
                        code = int(cb[idx[co, ci // 8]])
                        wv = 1 if (code >> (7 - ci % 8)) & 1 else -1
                        tot += wv * act[(b, y * stride, x * stride, ci)]
                    assert s[b, y, x, co] == tot


@pytest.mark.parametrize("tau,stride", [(1, 1), (3, 2), (5, 1), (7, 1), (8, 2)])
def test_shared_computation_equals_direct(oracle_mod, tau, stride):
    """The appendix carries the computation sharing of Sec. 4.5 over to 1x1 layers: per group of 8 channels one dot
    product per codebook vector, then lookups and additions.  Same sums, exactly."""
    rng = np.random.default_rng(100 + tau)
    shape = wl.LayerShape(40, 9, 5, 6, stride, 0, 1)
    p = wl.draw_layer_params(shape, tau, 200 + tau)
    bits = wl.draw_activation_bits(shape, 2, 300 + tau)
    s, _ = oracle_mod.conv1x1_bin(p.codebook, tau, p.idx_packed, p.alpha, 40, 9, stride, wl.pack_activation_bits(bits))
    shared = oracle_mod.conv1x1_shared_order(p.codebook, tau, p.idx, 40, 9, stride, bits)
    assert (s == shared).all()


def test_closed_forms_and_invariants(oracle_mod):
    shape = wl.LayerShape(32, 6, 4, 4, 1, 0, 1)
    p = wl.draw_layer_params(shape, 4, 9)
    ones = np.ones((1, 4, 4, 32), dtype=np.uint8)
    all_plus = np.full(16, 255, dtype=np.uint16)
    s, _ = oracle_mod.conv1x1_bin(all_plus, 4, p.idx_packed, p.alpha, 32, 6, 1, wl.pack_activation_bits(ones))
    assert (s == 32).all()                                  # all +1 weights, all +1 inputs: S = c_in
    all_minus = np.zeros(16, dtype=np.uint16)
    s, _ = oracle_mod.conv1x1_bin(all_minus, 4, p.idx_packed, p.alpha, 32, 6, 1, wl.pack_activation_bits(ones))
    assert (s == -32).all()
    bits = wl.draw_activation_bits(shape, 3, 10)
    s, y = oracle_mod.conv1x1_bin(p.codebook, 4, p.idx_packed, p.alpha, 32, 6, 1, wl.pack_activation_bits(bits))
    assert (np.abs(s) <= 32).all() and (s % 2 == 0).all()   # parity of c_in
    s_neg, _ = oracle_mod.conv1x1_bin(p.codebook, 4, p.idx_packed, p.alpha, 32, 6, 1, wl.pack_activation_bits(1 - bits))
    assert (s_neg == -s).all()                              # complementing the input negates the sums
    s_cb, _ = oracle_mod.conv1x1_bin((255 - p.codebook).astype(np.uint16), 4, p.idx_packed, p.alpha, 32, 6, 1,
                                     wl.pack_activation_bits(bits))
    assert (s_cb == -s).all()                               # complementing every codebook vector too
    assert (y == s.astype(np.float32) * p.alpha[None, None, None, :]).all()
    # the weights-only variant on +/-1 inputs written as fp16 gives the same sums
    a16 = (bits.astype(np.float32) * 2 - 1).astype(np.float16)
    y16 = oracle_mod.conv1x1_f16(p.codebook, 4, p.idx_packed, p.alpha, 32, 6, 1, a16)
    assert (y16 == y).all()


def test_f16_against_library_conv(oracle_mod):
    shape = wl.LayerShape(24, 5, 6, 5, 2, 0, 1)
    p = wl.draw_layer_params(shape, 5, 21)
    a = wl.draw_activation_f16(shape, 2, 21)
    y = oracle_mod.conv1x1_f16(p.codebook, 5, p.idx_packed, p.alpha, 24, 5, 2, a)
    wts = oracle_mod.decode_weights1x1(p.codebook, 5, p.idx_packed, 24, 5).astype(np.float64)
    ref = F.conv2d(torch.from_numpy(a.astype(np.float64)).permute(0, 3, 1, 2), torch.from_numpy(wts)[:, :, None, None],
                   stride=2).permute(0, 2, 3, 1).numpy() * p.alpha.astype(np.float64)[None, None, None, :]
    assert np.allclose(y, ref, rtol=1e-6, atol=1e-6)


def test_rejects_bad_arguments(oracle_mod):
    p = wl.draw_layer_params(wl.LayerShape(16, 4, 3, 3, 1, 0, 1), 3, 1)
    act = np.zeros((1, 3, 3, 1), dtype=np.uint32)
    with pytest.raises(ValueError):
        oracle_mod.conv1x1_bin(np.array([256] * 8, np.uint16), 3, p.idx_packed, p.alpha, 16, 4, 1, act)   # not an 8-bit code
    with pytest.raises(ValueError):
        oracle_mod.conv1x1_bin(np.zeros(512, np.uint16), 9, p.idx_packed, p.alpha, 16, 4, 1, act)         # tau' > 8
