"""Pins for the 3-bit part of the CPU oracle (packing, W3A4 look-up-table GEMV, export with a learnable centre):
hand-written words, a pure-Python loop, exact-integer identities, reduction to the 2-bit oracle, a hand-worked
fixture and a textbook special case. Nothing here compares the oracle with itself."""
import os

import numpy as np

import oracle
from gen import synth
from helpers import f16_bits, normal_float_table

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- packing
def test_pack3_hand_written_words_and_round_trip():
    codes = np.zeros((1, 64), dtype=np.uint8)
    codes[0, 0] = 5          # low bits 01, top bit 1
    codes[0, 3] = 2          # low bits 10, top bit 0
    codes[0, 17] = 7         # second half of the first plane word: odd bit 2*1+1
    codes[0, 47] = 4         # codes 32..63: plane word 1, i = 15 of the first half -> bit 30; low bits 00
    codes[0, 48] = 6         # i = 0 of the second half -> bit 1; low bits 10 at position 0 of word 3
    w2, w1 = oracle.pack_weights3(codes)
    assert w2.tolist() == [[(1 << 0) | (2 << 6), 3 << 2, 0, 2]]
    assert w1.tolist() == [[(1 << 0) | (1 << 3), (1 << 30) | (1 << 1)]]
    rng = np.random.default_rng(5)
    codes = rng.integers(0, 8, size=(9, 192), dtype=np.uint8)
    w2, w1 = oracle.pack_weights3(codes)
    assert np.array_equal(oracle.unpack_weights3(w2, w1), codes)
    # the low two bits are exactly the 2-bit packing
    assert np.array_equal(w2, oracle.pack_weights(codes & 3))
    # the plane word by the shift recipe: even bits <- codes 0..15, odd bits <- codes 16..31 of each block of 32
    top = (codes >> 2).astype(np.uint64).reshape(9, 6, 2, 16)
    ref = sum((top[:, :, 0, i] << (2 * i)) | (top[:, :, 1, i] << (2 * i + 1)) for i in range(16))
    assert np.array_equal(w1.astype(np.uint64), ref)


# ----------------------------------------------------------------------------- GEMV
def _brute(codes, lut, q, scale, G):
    M, K = q.shape
    N = codes.shape[0]
    NG = K // G
    S = np.zeros((M, N, NG, 8), dtype=np.int64)
    y = np.zeros((M, N))
    for m in range(M):
        for n in range(N):
            acc = 0.0
            for k in range(K):
                S[m, n, k // G, int(codes[n, k])] += int(q[m, k])
            for j in range(NG):
                for c in range(8):
                    acc += float(lut[n, j, c]) * float(S[m, n, j, c])
            y[m, n] = float(scale[m]) * acc
    return S, y


def _small_case(N, K, M, G, seed):
    rng = np.random.default_rng(seed)
    codes = rng.integers(0, 8, size=(N, K), dtype=np.uint8)
    lut = np.sort((rng.standard_normal((N, K // G, 8)) * 0.02).astype(np.float16), axis=2)
    x = synth.make_activations(M, K, seed)
    qa = oracle.quantize_act(f16_bits(x), 32, 1.0)
    return codes, lut, qa


def test_gemv_w3a4_brute_force_small_and_planted_mistakes():
    for (N, K, M, G) in [(8, 32, 1, 32), (16, 64, 2, 64), (5, 128, 3, 32)]:
        codes, lut, qa = _small_case(N, K, M, G, seed=N + K)
        w2, w1 = oracle.pack_weights3(codes)
        ref = oracle.gemv_w3a4(w2, w1, lut.view(np.uint16), qa["xq"], qa["scale"], G)
        S, y = _brute(codes, lut.astype(np.float64), qa["q"], qa["scale"].view(np.float16).astype(np.float64), G)
        assert np.array_equal(ref["S"], S)
        assert np.allclose(ref["y"], y, rtol=1e-13, atol=1e-15)
        # the four sums of a group add up to the group's total of q
        tot = qa["q"].astype(np.int64).reshape(M, K // G, G).sum(axis=2)
        assert np.array_equal(ref["S"].sum(axis=3), np.repeat(tot[:, None, :], N, axis=1))
        # planted mistakes: top bits of the two halves of a plane word swapped; groups reversed
        swapped = codes.reshape(N, K // 32, 2, 16)[:, :, ::-1, :].reshape(N, K)
        bad = np.where(True, (codes & 3) | (swapped & 4), 0).astype(np.uint8)
        S_bad, _ = _brute(bad, lut.astype(np.float64), qa["q"], qa["scale"].view(np.float16).astype(np.float64), G)
        assert not np.array_equal(S_bad, S)
        if K // G > 1:
            S_rev, y_rev = _brute(codes, lut[:, ::-1].astype(np.float64), qa["q"],
                                  qa["scale"].view(np.float16).astype(np.float64), G)
            assert not np.allclose(y_rev, y)


def test_gemv_w3a4_per_code_form_equals_direct_form_as_exact_integers():
    N, K, M, G = 40, 256, 3, 64
    codes, lut, qa = _small_case(N, K, M, G, seed=9)
    w2, w1 = oracle.pack_weights3(codes)
    ref = oracle.gemv_w3a4(w2, w1, lut.view(np.uint16), qa["xq"], qa["scale"], G)
    direct = oracle.gemv_w3a4_direct_int(w2, w1, lut.view(np.uint16), qa["xq"], G)
    Lint = np.round(lut.astype(np.float64) * 2.0 ** 24).astype(np.int64)          # every fp16 level times 2^24 is an integer
    assert np.array_equal(Lint.astype(np.float64) / 2.0 ** 24, lut.astype(np.float64))
    percode = np.einsum("njc,mnjc->mn", Lint, ref["S"].astype(np.int64))
    assert np.array_equal(percode, direct)
    # and the dense product with the dequantized matrix says the same
    Wd = np.take_along_axis(np.repeat(lut.astype(np.float64), G, axis=1).reshape(N, K, 8), codes[:, :, None].astype(np.int64), 2)[:, :, 0]
    dense = qa["q"].astype(np.float64) @ Wd.T * qa["scale"].view(np.float16).astype(np.float64)[:, None]
    assert np.allclose(dense, ref["y"], rtol=1e-12, atol=1e-14)


def test_gemv_w3a4_with_a_grid_that_ignores_the_top_bit_is_the_w2a4_oracle():
    N, K, M = 33, 512, 2
    rng = np.random.default_rng(17)
    codes = rng.integers(0, 8, size=(N, K), dtype=np.uint8)
    lut4 = np.sort((rng.standard_normal((N, 4)) * 0.02).astype(np.float16), axis=1)
    lut8 = np.concatenate([lut4, lut4], axis=1)
    x = synth.make_activations(M, K, 17)
    qa = oracle.quantize_act(f16_bits(x), 128, 1.0)
    w2, w1 = oracle.pack_weights3(codes)
    r3 = oracle.gemv_w3a4(w2, w1, lut8.view(np.uint16), qa["xq"], qa["scale"])
    r2 = oracle.gemv_w2a4(w2, lut4.view(np.uint16), qa["xq"], qa["scale"])
    assert np.array_equal(r3["S"][:, :, 0, :4] + r3["S"][:, :, 0, 4:], r2["S"])
    assert np.allclose(r3["y"], r2["y"], rtol=1e-12, atol=1e-15)
    # one group == one grid per row
    g1 = oracle.gemv_w3a4(w2, w1, lut8.view(np.uint16), qa["xq"], qa["scale"], K)
    assert np.array_equal(g1["S"], r3["S"]) and np.array_equal(g1["y"], r3["y"])
    # equal grids in every group: the group sums add up to the per-row sums
    gg = oracle.gemv_w3a4(w2, w1, np.repeat(lut8[:, None, :], K // 128, axis=1).view(np.uint16), qa["xq"], qa["scale"], 128)
    assert np.array_equal(gg["S"].sum(axis=2), r3["S"][:, :, 0, :])


# ----------------------------------------------------------------------------- export
def _fixture():
    d = {}
    for ln in open(os.path.join(GOLD, "nf3_hand_case.txt")):
        ln = ln.strip()
        if not ln or ln.startswith("#"):
            continue
        k, *v = ln.split()
        d[k] = np.array([float(t) for t in v])
    return d


def test_nf3_export_hand_worked_units_from_fixture():
    d = _fixture()
    table = d["table"].astype(np.float32)
    one = np.ones((1, 1), dtype=np.float32)
    for unit, s1 in (("unitA", 0.5), ("unitB", 0.25)):
        w = d[unit + "_w"].astype(np.float16)[None, :]
        out = oracle.nf3_export(w.view(np.uint16), one, one, np.full((1, 1), s1, np.float32), table, 3, w.shape[1])
        assert out["codes"][0].tolist() == d[unit + "_codes"].astype(int).tolist(), unit
        assert np.array_equal(out["lut"].view(np.float16)[0, 0].astype(np.float64), d[unit + "_levels"]), unit


def test_nf3_export_zero_centred_unit_is_the_absmax_nearest_level_quantizer():
    table, z = normal_float_table(3)
    assert z == 3 and table[0] == -1 and table[-1] == 1 and len(table) == 8
    rng = np.random.default_rng(3)
    N, K, G = 6, 256, 64
    w = (rng.standard_normal((N, K)) * 0.02).astype(np.float16)
    # make every unit symmetric about zero, so that the centre lands on zero and both scales on the absmax
    w[:, 0::64] = np.float16(0.09)
    w[:, 1::64] = np.float16(-0.09)
    one = np.ones((N, K // G), dtype=np.float32)
    out = oracle.nf3_export(w.view(np.uint16), one, one, 0.5 * one, table, z, G)
    v = w.astype(np.float64) / 0.09
    dist = np.abs(v[:, :, None] - table.astype(np.float64)[None, None, :])
    ref = np.argmin(dist, axis=2)          # first minimum: a tie keeps the lower level
    srt = np.sort(dist, axis=2)
    clear = (srt[:, :, 1] - srt[:, :, 0]) > 1e-6   # away from ties the fp32 path cannot differ
    assert clear.mean() > 0.99
    assert np.array_equal(out["codes"][clear], ref[clear])
    lut = out["lut"].view(np.float16).astype(np.float64)
    assert np.allclose(lut, (table.astype(np.float64) * 0.09)[None, None, :], rtol=2 ** -10)


def test_nf3_export_range_ends_centre_monotone_codes_and_degenerate_unit():
    table, z = normal_float_table(3)
    rng = np.random.default_rng(8)
    N, K, G = 10, 384, 128
    w = (rng.laplace(0, 0.02, size=(N, K)) + 0.01).astype(np.float16)     # not zero-centred
    sb = rng.uniform(0.7, 1.0, size=(N, K // G)).astype(np.float32)
    sg = rng.uniform(0.7, 1.0, size=(N, K // G)).astype(np.float32)
    s1 = rng.uniform(0.3, 0.7, size=(N, K // G)).astype(np.float32)
    out = oracle.nf3_export(w.view(np.uint16), sb, sg, s1, table, z, G)
    lut = out["lut"].view(np.float16).astype(np.float64)
    wf = w.astype(np.float64).reshape(N, K // G, G)
    lo = sb * wf.min(axis=2)
    hi = sg * wf.max(axis=2)
    c = lo + (hi - lo) * s1
    assert np.allclose(lut[:, :, 0], lo, rtol=2 ** -10) and np.allclose(lut[:, :, 7], hi, rtol=2 ** -10)
    assert np.allclose(lut[:, :, z], c, rtol=2 ** -9, atol=1e-6)
    assert np.all(np.diff(lut, axis=2) >= 0)
    codes = out["codes"].reshape(N, K // G, G)
    order = np.argsort(wf, axis=2, kind="stable")
    assert np.all(np.diff(np.take_along_axis(codes.astype(int), order, 2), axis=2) >= 0), "codes must not decrease with the weight"
    # sides: weights above the centre never take a negative level and the other way round
    assert np.all(codes[wf > c[:, :, None] + 1e-6] >= z) and np.all(codes[wf < c[:, :, None] - 1e-6] <= z)
    # a constant unit has no range: code zero_index, all levels lo
    wc = np.full((1, 128), 0.25, dtype=np.float16)
    oc = oracle.nf3_export(wc.view(np.uint16), np.ones((1, 1), np.float32), np.ones((1, 1), np.float32),
                           np.full((1, 1), 0.5, np.float32), table, z, 128)
    assert np.all(oc["codes"] == z) and np.all(oc["lut"].view(np.float16) == np.float16(0.25))
