"""Pins for the CPU oracle: every check here compares the oracle with something other than
itself -- a library routine, a closed form, a hand-written fixture or a brute-force loop."""
import fractions
import itertools
import os

import numpy as np
import pytest
import scipy.linalg
import torch

import oracle
from gen import synth
from helpers import f16_bits

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- fp16 <-> fp32
def test_f16_to_f32_all_patterns_match_numpy():
    bits = np.arange(65536, dtype=np.uint16)
    ref = bits.view(np.float16).astype(np.float32)
    got = np.array([oracle.f16_to_f32(int(b)) for b in bits], dtype=np.float32)
    both_nan = np.isnan(ref) & np.isnan(got)
    assert np.array_equal(ref.view(np.uint32)[~both_nan], got.view(np.uint32)[~both_nan])


def test_f32_to_f16_matches_numpy_including_ties_and_subnormals():
    rng = np.random.default_rng(0)
    vals = [rng.standard_normal(20000).astype(np.float32) * s for s in (1e-7, 1e-4, 1.0, 300.0, 7e4)]
    # every exact halfway point between neighbouring fp16 values (ties), and +-1 ulp(fp32) around them
    h = np.arange(0, 0x7C00, dtype=np.uint16).view(np.float16).astype(np.float64)
    mid = ((h[:-1] + h[1:]) / 2).astype(np.float32)
    vals += [mid, np.nextafter(mid, np.float32(np.inf)), np.nextafter(mid, np.float32(-np.inf)), -mid]
    vals += [np.array([0.0, -0.0, 65504.0, 65519.9, 65520.0, 1e9, -1e9, np.inf, -np.inf], dtype=np.float32)]
    v = np.concatenate(vals).astype(np.float32)
    with np.errstate(over="ignore"):
        ref = v.astype(np.float16).view(np.uint16)
    got = np.array([oracle.f32_to_f16(float(x)) for x in v], dtype=np.uint16)
    assert np.array_equal(ref, got)


# ----------------------------------------------------------------------------- Hadamard
def test_hadamard4_matches_handwritten_fixture():
    Hp = np.loadtxt(os.path.join(GOLD, "hadamard4.txt"))
    assert np.array_equal(oracle.hadamard_matrix(4) * 2.0, Hp)


@pytest.mark.parametrize("n", [1, 2, 4, 8, 16, 32, 64])
def test_hadamard_orthogonal_and_matches_library(n):
    H = oracle.hadamard_matrix(n)
    assert np.allclose(H @ H.T, np.eye(n), atol=1e-14)
    assert np.array_equal(np.sign(H), scipy.linalg.hadamard(n).astype(np.float64))
    assert np.allclose(np.abs(H), 1.0 / np.sqrt(n))
    # first row all ones, every other row balanced
    assert np.all(H[0] > 0)
    for i in range(1, n):
        assert (H[i] > 0).sum() == n // 2


@pytest.mark.parametrize("B,K", [(2, 8), (4, 16), (16, 64), (64, 128), (128, 384), (256, 256)])
def test_fwht_equals_matrix_product_bit_exact_on_small_integers(B, K):
    # integer inputs: every butterfly sum is exact in fp32, so the result must equal the dense
    # product with the library's Sylvester matrix, then one fp32 multiply by (float)(1/sqrt(B))
    rng = np.random.default_rng(B)
    xi = rng.integers(-8, 9, size=K)
    x = xi.astype(np.float16).view(np.uint16)
    got = oracle.rotate_f32(x, B)
    Hp = scipy.linalg.hadamard(B).astype(np.int64)
    ref_int = np.concatenate([Hp @ xi[b:b + B] for b in range(0, K, B)])
    ref = ref_int.astype(np.float32) * np.float32(1.0 / np.sqrt(float(B)))
    assert np.array_equal(got.view(np.uint32), ref.view(np.uint32))


def test_fwht_unit_vectors_give_columns():
    B = 32
    Hp = scipy.linalg.hadamard(B)
    for j in (0, 1, 5, 31):
        e = np.zeros(B, dtype=np.float16)
        e[j] = 1.0
        got = oracle.rotate_f32(e.view(np.uint16), B)
        assert np.array_equal(got, Hp[:, j].astype(np.float32) * np.float32(1 / np.sqrt(32.0)))


@pytest.mark.parametrize("B", [4, 16, 64, 256])
def test_rotation_is_involution_when_scale_is_a_power_of_two(B):
    # sqrt(B) is a power of two here and inputs are small integers, so both passes are exact
    rng = np.random.default_rng(1)
    xi = rng.integers(-4, 5, size=B)
    once = oracle.rotate_f32(xi.astype(np.float16).view(np.uint16), B)
    once16 = once.astype(np.float16)
    assert np.array_equal(once16.astype(np.float32), once)  # representable in fp16
    twice = oracle.rotate_f32(once16.view(np.uint16), B)
    assert np.array_equal(twice, xi.astype(np.float32))


@pytest.mark.parametrize("B,K", [(128, 1280), (2048, 2048), (8192, 8192)])
def test_fp32_butterflies_stay_within_rounding_bound_of_exact_rotation(B, K):
    x = synth.make_activations(1, K, seed=11)
    xb = f16_bits(x)[0]
    v32 = oracle.rotate_f32(xb, B).astype(np.float64)
    exact = oracle.rotate_exact_f64(xb.reshape(1, K), B)[0]
    # independent of both: dense product with the library matrix in float64
    Hp = scipy.linalg.hadamard(B).astype(np.float64) if B <= 2048 else None
    if Hp is not None:
        xd = xb.view(np.float16).astype(np.float64)
        lib = np.concatenate([Hp @ xd[b:b + B] for b in range(0, K, B)]) / np.sqrt(B)
        assert np.allclose(exact, lib, rtol=0, atol=1e-9)
    # error of log2(B) fp32 additions + 1 multiply, each <= 2^-24 relative to running magnitude
    l1 = np.abs(xb.view(np.float16).astype(np.float64)).reshape(-1, B).sum(axis=1).repeat(B) / np.sqrt(B)
    bound = (np.log2(B) + 2) * 2.0 ** -24 * l1
    assert np.all(np.abs(v32 - exact) <= bound)
    # Parseval: the rotation preserves the Euclidean norm
    assert np.isclose(np.linalg.norm(exact), np.linalg.norm(xb.view(np.float16).astype(np.float64)), rtol=1e-12)


# ----------------------------------------------------------------------------- quantizer
def _load_hand_cases():
    xs, qs = [], []
    for line in open(os.path.join(GOLD, "quant_hand_cases.txt")):
        if line.startswith("#") or "->" not in line:
            continue
        a, b = line.split("->")
        xs.append(float(a))
        qs.append(int(b))
    return np.array(xs), np.array(qs)


def test_quantizer_hand_cases_from_fixture():
    xs, qs = _load_hand_cases()
    K = 32
    x = np.zeros((1, K), dtype=np.float16)
    x[0, :len(xs)] = xs
    assert np.array_equal(x[0, :len(xs)].astype(np.float64), xs)  # fixture values are exact fp16
    r = oracle.quantize_act(x.view(np.uint16), had_block=1, clip_ratio=1.0)
    assert r["scale"][0] == np.float16(1.0).view(np.uint16)
    assert np.array_equal(r["q"][0, :len(xs)], qs)
    assert np.all(r["q"][0, len(xs):] == 0)


def test_quantizer_scale_matches_library_arithmetic_and_absmax_maps_to_7():
    for seed in range(5):
        x = synth.make_activations(3, 256, seed=seed)
        r = oracle.quantize_act(f16_bits(x), had_block=1, clip_ratio=1.0)
        xf = x.numpy().astype(np.float32)
        amax = np.abs(xf).max(axis=1)
        s16 = (amax / np.float32(7.0)).astype(np.float16)
        assert np.array_equal(r["scale"], s16.view(np.uint16))
        q = r["q"]
        assert np.all(np.abs(q).max(axis=1) == 7)
        idx = np.abs(xf).argmax(axis=1)
        assert np.all(np.abs(q[np.arange(3), idx]) == 7)
        # library restatement: numpy float32 division + rint (round half to even)
        ref = np.clip(np.rint(xf / s16.astype(np.float32)[:, None]), -8, 7).astype(np.int8)
        assert np.array_equal(q, ref)


def test_quantizer_clip_ratio_below_one_reaches_minus8_never_plus8():
    x = np.zeros((2, 16), dtype=np.float16)
    x[0, 0], x[0, 1] = -7.0, 7.0
    x[1, 0], x[1, 1] = 7.0, -6.0
    r = oracle.quantize_act(x.view(np.uint16), had_block=1, clip_ratio=0.9)
    assert r["q"][0, 0] == -8 and r["q"][0, 1] == 7
    assert r["q"][1, 0] == 7 and r["q"][1, 1] == -7  # -6/0.9 = -6.67 -> -7
    assert r["q"].min() >= -8 and r["q"].max() <= 7


def test_quantizer_zero_token_and_nibble_layout():
    x = np.zeros((2, 32), dtype=np.float16)
    x[1, :] = np.arange(32) % 15 - 7
    r = oracle.quantize_act(x.view(np.uint16), had_block=1, clip_ratio=1.0)
    assert r["scale"][0] == 0 and np.all(r["xq"][0] == 0) and np.all(r["q"][0] == 0)
    q = r["q"][1].astype(np.int32)
    assert np.array_equal(q, np.arange(32) % 15 - 7)  # scale is exactly 1
    # low nibble = even index, high nibble = odd index, two's complement
    expect = ((q[0::2] & 0xF) | ((q[1::2] & 0xF) << 4)).astype(np.uint8)
    assert np.array_equal(r["xq"][1], expect)
    # decode with a different formula than the oracle's shift recipe: ((n ^ 8) - 8)
    lo = ((r["xq"][1].astype(np.int32) & 0xF) ^ 8) - 8
    hi = ((r["xq"][1].astype(np.int32) >> 4) ^ 8) - 8
    dec = oracle.unpack_act(r["xq"][1:2])[0]
    assert np.array_equal(dec[0::2], lo) and np.array_equal(dec[1::2], hi)


def test_quantizer_identity_rotation_vs_hadamard_and_exact_rotation_agree_on_codes():
    # with rotation: quantizing the oracle's rotated vector by numpy must give the same codes
    K, B = 512, 128
    x = synth.make_activations(2, K, seed=3)
    r = oracle.quantize_act(f16_bits(x), had_block=B, clip_ratio=1.0)
    v = r["v"]
    amax = np.abs(v).max(axis=1)
    s16 = (amax / np.float32(7.0)).astype(np.float16)
    assert np.array_equal(r["scale"], s16.view(np.uint16))
    ref = np.clip(np.rint(v / s16.astype(np.float32)[:, None]), -8, 7).astype(np.int8)
    assert np.array_equal(r["q"], ref)
    # and the rotated vector is close to the exact one (so codes differ from the exact-rotation
    # codes only where the exact value sits within rounding distance of a decision boundary)
    exact = oracle.rotate_exact_f64(f16_bits(x), B)
    qe = np.clip(np.rint(exact / s16.astype(np.float64)[:, None]), -8, 7)
    frac = np.abs(exact / s16.astype(np.float64)[:, None] - np.floor(exact / s16.astype(np.float64)[:, None]) - 0.5)
    differs = qe != r["q"]
    assert np.all(frac[differs] < 1e-4)
    assert differs.mean() < 1e-3


def test_quantizer_rejects_nonfinite():
    x = np.zeros((1, 16), dtype=np.float16)
    x[0, 3] = np.inf
    with pytest.raises(ValueError):
        oracle.quantize_act(x.view(np.uint16), 1, 1.0)


# ----------------------------------------------------------------------------- packing
def test_pack_single_code_words_and_roundtrip():
    for j in range(16):
        codes = np.zeros((1, 16), dtype=np.uint8)
        codes[0, j] = 3
        assert oracle.pack_weights(codes)[0, 0] == np.uint32(3 << (2 * j))
    rng = np.random.default_rng(5)
    codes = rng.integers(0, 4, size=(7, 96), dtype=np.uint8)
    words = oracle.pack_weights(codes)
    # independent numpy restatement of the layout
    ref = (codes.reshape(7, 6, 16).astype(np.uint64) << (2 * np.arange(16, dtype=np.uint64))).sum(axis=2)
    assert np.array_equal(words, ref.astype(np.uint32))
    assert np.array_equal(oracle.unpack_weights(words), codes)


def test_pack_bytes_decode_with_shift_and_mask_recipe():
    # Appendix A.7 decodes four codes per byte with shifts and the mask 0x03; in this layout the
    # first code sits in the LOW two bits (shifts 0,2,4,6), bytes in little-endian order.
    rng = np.random.default_rng(6)
    codes = rng.integers(0, 4, size=(3, 64), dtype=np.uint8)
    by = oracle.pack_weights(codes).view(np.uint8).reshape(3, 16)
    dec = np.stack([(by >> s) & 0x03 for s in (0, 2, 4, 6)], axis=2).reshape(3, 64)
    assert np.array_equal(dec, codes)


def test_pack_rejects_codes_above_3():
    codes = np.zeros((2, 16), dtype=np.uint8)
    codes[1, 7] = 4
    with pytest.raises(ValueError):
        oracle.pack_weights(codes)


def test_lut_lookup_of_unpacked_codes_reproduces_dequantized_weights():
    codes, lut = synth.make_layer(24, 256, 128, "rotated_laplace", seed=9)
    words = oracle.pack_weights(codes.numpy())
    Wd = oracle.dequant_weights(words, f16_bits(lut))
    ref = np.take_along_axis(lut.numpy().astype(np.float64), codes.numpy().astype(np.int64), axis=1)
    assert np.array_equal(Wd, ref)
    # the generator assigned every weight to a level: all dequantized values are LUT levels
    assert set(np.unique(Wd[0])) <= set(lut.numpy()[0].astype(np.float64))


# ----------------------------------------------------------------------------- GEMV
def _problem(N, K, M, seed, kind="uniform", B=1):
    codes, lut = synth.make_layer(N, K, B, kind, seed)
    x = synth.make_activations(M, K, seed)
    qa = oracle.quantize_act(f16_bits(x), B, 1.0)
    words = oracle.pack_weights(codes.numpy())
    return codes.numpy(), lut, words, qa


def _brute(codes, lut, q, scale_bits):
    """Pure-Python triple loop straight from the definition."""
    M, K = q.shape
    N = codes.shape[0]
    S = np.zeros((M, N, 4), dtype=np.int64)
    y = np.zeros((M, N))
    lutf = lut.numpy().astype(np.float64)
    for m in range(M):
        s = float(scale_bits[m:m + 1].view(np.float16)[0])
        for n in range(N):
            acc = 0.0
            for k in range(K):
                c = int(codes[n, k])
                S[m, n, c] += int(q[m, k])
            for c in range(4):
                acc += lutf[n, c] * float(S[m, n, c])
            y[m, n] = s * acc
    return S, y


@pytest.mark.parametrize("N,K,M,zero_from", [(8, 16, 1, 8), (16, 32, 1, None), (16, 32, 3, None)])
def test_gemv_brute_force_small(N, K, M, zero_from):
    # the 8x8 case is embedded in one packed word: codes beyond k=8 meet zero activations
    codes, lut, words, qa = _problem(N, K, M, seed=N + K)
    xq, q = qa["xq"].copy(), qa["q"].copy()
    if zero_from is not None:
        q[:, zero_from:] = 0
        xq[:, zero_from // 2:] = 0
    r = oracle.gemv_w2a4(words, f16_bits(lut), xq, qa["scale"])
    S, y = _brute(codes, lut, q, qa["scale"])
    assert np.array_equal(r["S"], S)
    assert np.allclose(r["y"], y, rtol=1e-14, atol=0)
    if zero_from is not None:
        S8, y8 = _brute(codes[:, :zero_from], lut, q[:, :zero_from], qa["scale"])
        assert np.array_equal(S[..., 1:], S8[..., 1:]) and np.allclose(y, y8)


def test_gemv_percode_sums_add_up_and_equal_codes_rows():
    codes, lut, words, qa = _problem(32, 256, 2, seed=4)
    codes[5, :] = 2
    codes[6, :] = 0
    words = oracle.pack_weights(codes)
    r = oracle.gemv_w2a4(words, f16_bits(lut), qa["xq"], qa["scale"])
    tot = qa["q"].astype(np.int64).sum(axis=1)
    assert np.array_equal(r["S"].sum(axis=2), np.repeat(tot[:, None], 32, axis=1))
    assert np.array_equal(r["S"][:, 5, 2], tot) and np.all(r["S"][:, 5, [0, 1, 3]] == 0)
    assert np.array_equal(r["S"][:, 6, 0], tot)


@pytest.mark.parametrize("N,K,M,B,kind", [(64, 512, 1, 128, "rotated_laplace"), (40, 2048, 2, 2048, "rotated_laplace"),
                                          (33, 192, 3, 64, "uniform")])
def test_direct_form_equals_percode_form_as_exact_integers(N, K, M, B, kind):
    codes, lut, words, qa = _problem(N, K, M, seed=7, kind=kind, B=B)
    lb = f16_bits(lut)
    r = oracle.gemv_w2a4(words, lb, qa["xq"], qa["scale"])
    d = oracle.gemv_direct(words, lb, qa["xq"], qa["scale"])
    assert np.array_equal(d["acc_int"], oracle.percode_int(lb, r["S"]))
    # numpy restatement of the scaled-integer direct sum (fp16 levels times 2^24 are integers)
    Li = np.round(np.ldexp(lut.numpy().astype(np.float64), 24)).astype(np.int64)
    Wi = np.take_along_axis(Li, codes.astype(np.int64), axis=1)
    assert np.array_equal(d["acc_int"], qa["q"].astype(np.int64) @ Wi.T)
    assert np.allclose(d["y"], r["y"], rtol=1e-12, atol=1e-300)


def test_affine_and_constant_lut_reduce_to_plain_integer_gemv():
    N, K, M = 48, 320, 2
    codes, lut, words, qa = _problem(N, K, M, seed=12, kind="uniform", B=64)
    a, d = 0.125, 0.03125  # exactly representable
    lut_aff = torch.tensor([[a + c * d for c in range(4)]] * N, dtype=torch.float16)
    r = oracle.gemv_w2a4(words, f16_bits(lut_aff), qa["xq"], qa["scale"])
    q = qa["q"].astype(np.int64)
    s = qa["scale"].view(np.float16).astype(np.float64)
    ref = s[:, None] * (a * q.sum(axis=1)[:, None] + d * (q @ codes.astype(np.int64).T))
    assert np.allclose(r["y"], ref, rtol=1e-13, atol=0)
    lut_c = torch.full((N, 4), 0.5, dtype=torch.float16)
    r2 = oracle.gemv_w2a4(words, f16_bits(lut_c), qa["xq"], qa["scale"])
    assert np.allclose(r2["y"], s[:, None] * 0.5 * q.sum(axis=1)[:, None] * np.ones((1, N)), rtol=1e-13)


def test_gemv_equals_dense_matmul_with_dequantized_weights():
    N, K, M = 64, 1024, 3
    codes, lut, words, qa = _problem(N, K, M, seed=21, kind="rotated_laplace", B=128)
    r = oracle.gemv_w2a4(words, f16_bits(lut), qa["xq"], qa["scale"])
    Wd = np.take_along_axis(lut.numpy().astype(np.float64), codes.astype(np.int64), axis=1)  # [N][K]
    s = qa["scale"].view(np.float16).astype(np.float64)
    ref = (qa["q"].astype(np.float64) * s[:, None]) @ Wd.T
    assert np.allclose(r["y"], ref, rtol=1e-11, atol=1e-15)
    mag = s[:, None] * (np.abs(lut.numpy().astype(np.float64))[None] * np.abs(r["S"])).sum(axis=2)
    assert np.allclose(r["tol"], 2e-3 * mag + 1e-5, rtol=1e-12)


def test_planted_mistakes_are_caught_by_the_brute_force_pin():
    # a transposed nibble order or a reversed code order in the inputs changes the result: the pin
    # is sensitive to exactly the mistakes a wrong index would make
    codes, lut, words, qa = _problem(16, 32, 1, seed=3)
    r = oracle.gemv_w2a4(words, f16_bits(lut), qa["xq"], qa["scale"])
    swapped = ((qa["xq"] >> 4) | (qa["xq"] << 4)).astype(np.uint8)
    r_sw = oracle.gemv_w2a4(words, f16_bits(lut), swapped, qa["scale"])
    assert not np.array_equal(r["S"], r_sw["S"])
    rev = oracle.pack_weights(np.ascontiguousarray(codes.reshape(16, 2, 16)[:, :, ::-1].reshape(16, 32)))
    r_rev = oracle.gemv_w2a4(rev, f16_bits(lut), qa["xq"], qa["scale"])
    assert not np.array_equal(r["S"], r_rev["S"])


# ----------------------------------------------------------------------------- GEMV, group-wise grid
def _problem_grouped(N, K, M, G, seed, kind="uniform", B=1):
    codes, lut = synth.make_layer_grouped(N, K, G, B, kind, seed)
    x = synth.make_activations(M, K, seed)
    qa = oracle.quantize_act(f16_bits(x), B, 1.0)
    words = oracle.pack_weights(codes.numpy())
    return codes.numpy(), lut, words, qa


def _brute_grouped(codes, lut, q, scale_bits, G):
    """Pure-Python loops straight from the definition: weight k of row n uses grid k // G of that row."""
    M, K = q.shape
    N = codes.shape[0]
    S = np.zeros((M, N, K // G, 4), dtype=np.int64)
    y = np.zeros((M, N))
    lutf = lut.numpy().astype(np.float64)
    for m in range(M):
        s = float(scale_bits[m:m + 1].view(np.float16)[0])
        for n in range(N):
            acc = 0.0
            for k in range(K):
                S[m, n, k // G, int(codes[n, k])] += int(q[m, k])
                acc += lutf[n, k // G, int(codes[n, k])] * float(q[m, k])
            y[m, n] = s * acc
    return S, y


@pytest.mark.parametrize("N,K,M,G", [(8, 32, 1, 16), (12, 64, 2, 16), (6, 256, 1, 128), (5, 384, 3, 128)])
def test_grouped_gemv_brute_force_small(N, K, M, G):
    codes, lut, words, qa = _problem_grouped(N, K, M, G, seed=N + K)
    r = oracle.gemv_w2a4_grouped(words, f16_bits(lut), qa["xq"], qa["scale"], G)
    S, y = _brute_grouped(codes, lut, qa["q"], qa["scale"], G)
    assert np.array_equal(r["S"], S)
    assert np.allclose(r["y"], y, rtol=1e-12, atol=1e-300)


def test_grouped_gemv_with_one_group_is_the_per_row_gemv():
    N, K, M = 24, 512, 2
    codes, lut, words, qa = _problem(N, K, M, seed=31, kind="rotated_laplace", B=128)
    lb = f16_bits(lut)
    r = oracle.gemv_w2a4(words, lb, qa["xq"], qa["scale"])
    rg = oracle.gemv_w2a4_grouped(words, lb.reshape(N, 1, 4), qa["xq"], qa["scale"], K)
    assert np.array_equal(rg["S"][:, :, 0, :], r["S"])
    assert np.array_equal(rg["y"], r["y"]) and np.array_equal(rg["tol"], r["tol"])


def test_grouped_gemv_with_equal_grids_sums_to_the_per_row_gemv():
    N, K, M, G = 20, 1024, 2, 128
    codes, lut, words, qa = _problem(N, K, M, seed=33, kind="uniform", B=64)
    lb = f16_bits(lut)
    lbg = np.ascontiguousarray(np.repeat(lb[:, None, :], K // G, axis=1))
    r = oracle.gemv_w2a4(words, lb, qa["xq"], qa["scale"])
    rg = oracle.gemv_w2a4_grouped(words, lbg, qa["xq"], qa["scale"], G)
    assert np.array_equal(rg["S"].sum(axis=2), r["S"])
    assert np.allclose(rg["y"], r["y"], rtol=1e-12, atol=1e-300)
    # every group's sums add up to the group's sum of activations
    tot = qa["q"].astype(np.int64).reshape(M, K // G, G).sum(axis=2)
    assert np.array_equal(rg["S"].sum(axis=3), np.repeat(tot[:, None, :], N, axis=1))
    assert np.all(rg["tol"] >= r["tol"] - 1e-18)   # |.| taken per group can only grow the bound


@pytest.mark.parametrize("N,K,M,G,B,kind", [(40, 512, 1, 128, 128, "rotated_laplace"), (17, 2048, 2, 128, 2048, "rotated_laplace"),
                                            (33, 384, 3, 64, 64, "uniform")])
def test_grouped_direct_form_equals_percode_form_as_exact_integers(N, K, M, G, B, kind):
    codes, lut, words, qa = _problem_grouped(N, K, M, G, seed=17, kind=kind, B=B)
    lb = f16_bits(lut)
    r = oracle.gemv_w2a4_grouped(words, lb, qa["xq"], qa["scale"], G)
    d = oracle.gemv_direct_grouped(words, lb, qa["xq"], qa["scale"], G)
    assert np.array_equal(d["acc_int"], oracle.percode_int_grouped(lb, r["S"]))
    # numpy restatement: dequantize with the grid of each weight's group, then one integer matrix product
    Li = np.round(np.ldexp(lut.numpy().astype(np.float64), 24)).astype(np.int64)          # [N][K/G][4]
    Wi = np.take_along_axis(np.repeat(Li, G, axis=1), codes.astype(np.int64)[:, :, None], axis=2)[:, :, 0]
    assert np.array_equal(d["acc_int"], qa["q"].astype(np.int64) @ Wi.T)
    assert np.allclose(d["y"], r["y"], rtol=1e-12, atol=1e-300)


def test_grouped_gemv_equals_dense_matmul_with_groupwise_dequantized_weights():
    N, K, M, G = 48, 1024, 3, 128
    codes, lut, words, qa = _problem_grouped(N, K, M, G, seed=23, kind="rotated_laplace", B=128)
    r = oracle.gemv_w2a4_grouped(words, f16_bits(lut), qa["xq"], qa["scale"], G)
    lutf = lut.numpy().astype(np.float64)
    Wd = np.take_along_axis(np.repeat(lutf, G, axis=1), codes.astype(np.int64)[:, :, None], axis=2)[:, :, 0]
    # the generator put every weight on one of its own group's levels
    assert set(np.unique(Wd[3, G:2 * G])) <= set(lutf[3, 1])
    s = qa["scale"].view(np.float16).astype(np.float64)
    ref = (qa["q"].astype(np.float64) * s[:, None]) @ Wd.T
    assert np.allclose(r["y"], ref, rtol=1e-11, atol=1e-15)
    mag = s[:, None] * (np.abs(lutf)[None] * np.abs(r["S"])).sum(axis=(2, 3))
    assert np.allclose(r["tol"], 2e-3 * mag + 1e-5, rtol=1e-12)


def test_grouped_planted_mistakes_are_caught():
    # a grid looked up by k % G instead of k // G, or the groups taken in reverse, changes the result
    N, K, M, G = 8, 64, 1, 16
    codes, lut, words, qa = _problem_grouped(N, K, M, G, seed=5)
    r = oracle.gemv_w2a4_grouped(words, f16_bits(lut), qa["xq"], qa["scale"], G)
    lut_rev = torch.flip(lut, dims=[1]).contiguous()
    r_rev = oracle.gemv_w2a4_grouped(words, f16_bits(lut_rev), qa["xq"], qa["scale"], G)
    assert not np.allclose(r["y"], r_rev["y"], rtol=1e-6)
    perm = np.arange(K).reshape(K // G, G).T.reshape(-1)   # k -> position under the k % G reading
    r_mod = oracle.gemv_w2a4_grouped(oracle.pack_weights(np.ascontiguousarray(codes[:, perm])), f16_bits(lut),
                                     np.ascontiguousarray(qa["xq"]), qa["scale"], G)
    assert not np.array_equal(r["S"], r_mod["S"])
    with pytest.raises((ValueError, AssertionError)):   # a group size that does not divide K
        oracle.gemv_w2a4_grouped(words, f16_bits(lut)[:, :3].copy(), qa["xq"], qa["scale"], 24)


# ----------------------------------------------------------------------------- partitioning quantizer export
def _ldp_inputs(N, K, G, seed, clip=True):
    rng = np.random.default_rng(seed)
    w = torch.from_numpy(rng.laplace(0.0, 0.02, size=(N, K)).astype(np.float32)).to(torch.float16)
    NG = K // G
    sig = lambda a: (1.0 / (1.0 + np.exp(-a))).astype(np.float32)
    sb = sig(rng.normal(3.0, 1.0, size=(N, NG))) if clip else np.ones((N, NG), np.float32)
    sg = sig(rng.normal(3.0, 1.0, size=(N, NG))) if clip else np.ones((N, NG), np.float32)
    s1 = sig(rng.normal(-0.7, 0.5, size=(N, NG)))
    s2 = sig(rng.normal(0.0, 0.5, size=(N, NG)))
    return w, sb, sg, s1, s2


def test_ldp_hand_case_from_fixture():
    ws, codes, sig, lut = [], [], None, None
    for ln in open(os.path.join(GOLD, "ldp_hand_case.txt")):
        ln = ln.strip()
        if not ln or ln.startswith("#"):
            continue
        if ln.startswith("sig"):
            sig = [float(v) for v in ln.split()[1:]]
        elif ln.startswith("lut"):
            lut = [float(v) for v in ln.split()[1:]]
        else:
            a, b = ln.split("->")
            ws.append(float(a))
            codes.append(int(b))
    G = 16
    w = torch.tensor([ws + [0.5] * (G - len(ws))], dtype=torch.float16)
    one = np.ones((1, 1), np.float32)
    r = oracle.ldp_export(f16_bits(w), one, one, one * sig[0], one * sig[1], G)
    assert list(r["codes"][0, :len(ws)]) == codes
    assert list(r["lut"][0, 0].view(np.float16).astype(np.float64)) == lut


def test_ldp_uniform_initial_point_is_the_textbook_asymmetric_quantizer():
    # fixture: p = t = w at initialisation; then the quantizer is round((w - min) / (h / 3)) with levels min + h i / 3
    fx = {}
    for ln in open(os.path.join(GOLD, "ldp_uniform_init.txt")):
        if ln.strip() and not ln.startswith("#"):
            k, *v = ln.split()
            fx[k] = [float(fractions.Fraction(x)) for x in v]
    assert fx["t"] == [1 / 6, 1 / 2, 5 / 6] and fx["w"] == [0, 1 / 3, 2 / 3, 1]
    N, K, G = 6, 512, 128
    w, _, _, _, _ = _ldp_inputs(N, K, G, 1)
    one = np.ones((N, K // G), np.float32)
    r = oracle.ldp_export(f16_bits(w), one, one, (one / 3).astype(np.float32), (one / 2).astype(np.float32), G)
    wf = w.numpy().astype(np.float64).reshape(N, K // G, G)
    lo, hi = wf.min(axis=2, keepdims=True), wf.max(axis=2, keepdims=True)
    xq = (wf - lo) / ((hi - lo) / 3.0)
    ref = np.clip(np.rint(xq), 0, 3)
    near_tie = np.abs(xq - np.floor(xq) - 0.5) < 1e-5
    got = r["codes"].reshape(N, K // G, G)
    assert near_tie.sum() < 5 and np.array_equal(got[~near_tie], ref[~near_tie].astype(np.uint8))
    levels = lo + (hi - lo) * np.array(fx["w"])[None, None, :]
    assert np.allclose(r["lut"].view(np.float16).astype(np.float64), levels, rtol=2e-3, atol=1e-7)


def test_ldp_range_ends_bin_centres_monotone_codes_and_sum_form():
    N, K, G = 5, 768, 128
    w, sb, sg, s1, s2 = _ldp_inputs(N, K, G, 2)
    r = oracle.ldp_export(f16_bits(w), sb, sg, s1, s2, G)
    wf = w.numpy().astype(np.float64).reshape(N, K // G, G)
    codes = r["codes"].reshape(N, K // G, G)
    lut = r["lut"].view(np.float16).astype(np.float64)
    lo = sb.astype(np.float64) * wf.min(axis=2)
    hi = sg.astype(np.float64) * wf.max(axis=2)
    h = hi - lo
    # the lowest level is the clipped minimum, the highest the clipped maximum (lo + h = hi)
    assert np.allclose(lut[..., 0], lo, rtol=1e-3, atol=1e-7) and np.allclose(lut[..., 3], hi, rtol=1e-3, atol=1e-7)
    # partitions fill the range: the thresholds and the bin centres in exact arithmetic
    p1 = s1.astype(np.float64)
    p2 = (1 - p1) * s2
    p3 = (1 - p1) * (1 - s2.astype(np.float64))
    assert np.allclose(p1 + p2 + p3, 1.0)
    t1 = p1 / 2
    t2 = t1 + (p1 + p2) / 2
    t3 = t2 + (p2 + p3) / 2
    assert np.allclose(t3 + p3 / 2, 1.0)
    assert np.allclose(lut[..., 1], lo + h * (t1 + t2) / 2, rtol=1e-3, atol=1e-7)
    assert np.allclose(lut[..., 2], lo + h * (t2 + t3) / 2, rtol=1e-3, atol=1e-7)
    # codes are monotone in the weight, and each weight sits in the partition its code names
    x = (np.clip(wf, lo[..., None], hi[..., None]) - lo[..., None]) / h[..., None]
    T = np.stack([np.zeros_like(t1) - 1, t1, t2, t3, np.ones_like(t1) * 2], axis=-1)
    lower = np.take_along_axis(T, codes.astype(np.int64), axis=-1)
    upper = np.take_along_axis(T, codes.astype(np.int64) + 1, axis=-1)
    assert np.all(x >= lower - 1e-6) and np.all(x <= upper + 1e-6)
    order = np.argsort(wf, axis=2, kind="stable")
    assert np.all(np.diff(np.take_along_axis(codes.astype(np.int64), order, axis=2), axis=2) >= 0)
    assert len(np.unique(codes)) == 4
    # sum form of the dequantizer (three steps, each adding the gap to the next level) == LUT lookup
    w0, w1, w2, w3 = 0.0, (t1 + t2) / 2, (t2 + t3) / 2, 1.0
    u = lambda z: (z >= -1e-12).astype(np.float64)
    dq = lo[..., None] + h[..., None] * (u(x - t1[..., None]) * (w1 - w0)[..., None] + u(x - t2[..., None]) * (w2 - w1)[..., None]
                                         + u(x - t3[..., None]) * (w3 - w2)[..., None])
    interior = (np.abs(x - t1[..., None]) > 1e-5) & (np.abs(x - t2[..., None]) > 1e-5) & (np.abs(x - t3[..., None]) > 1e-5)
    look = np.take_along_axis(lut, codes.astype(np.int64), axis=-1)
    assert np.allclose(dq[interior], look[interior], rtol=2e-3, atol=1e-6)


def test_ldp_degenerate_unit_and_planted_mistakes():
    G = 32
    w = torch.full((1, 2 * G), 0.25, dtype=torch.float16)
    w[0, G:] = torch.linspace(-1, 1, G).to(torch.float16)
    one = np.ones((1, 2), np.float32)
    r = oracle.ldp_export(f16_bits(w), one, one, one * 0.3, one * 0.6, G)
    assert np.all(r["codes"][0, :G] == 0) and np.all(r["lut"][0, 0].view(np.float16) == np.float16(0.25))
    # swapping the two partition parameters, or the two clipping parameters, changes the second unit
    a = oracle.ldp_export(f16_bits(w), one * 0.9, one * 0.7, one * 0.3, one * 0.6, G)
    b = oracle.ldp_export(f16_bits(w), one * 0.9, one * 0.7, one * 0.6, one * 0.3, G)
    c = oracle.ldp_export(f16_bits(w), one * 0.7, one * 0.9, one * 0.3, one * 0.6, G)
    assert not np.array_equal(a["codes"], b["codes"]) and not np.array_equal(a["lut"], c["lut"])
    with pytest.raises((ValueError, AssertionError)):
        oracle.ldp_export(f16_bits(w), one, one, one, one, 48)


# ----------------------------------------------------------------------------- weight-only variant
def _problem16(N, K, M, seed, kind="uniform"):
    codes, lut = synth.make_layer(N, K, 1, kind, seed)
    x = synth.make_activations(M, K, seed)
    return codes.numpy(), lut, oracle.pack_weights(codes.numpy()), x


def test_w2a16_brute_force_small_and_planted_mistakes():
    codes, lut, words, x = _problem16(16, 32, 2, seed=5)
    r = oracle.gemv_w2a16(words, f16_bits(lut), f16_bits(x))
    lutf, xf = lut.numpy().astype(np.float64), x.numpy().astype(np.float64)
    for m in range(2):
        for n in range(16):
            acc = mag = 0.0
            for k in range(32):
                acc += lutf[n, codes[n, k]] * xf[m, k]
                mag += abs(lutf[n, codes[n, k]]) * abs(xf[m, k])
            assert r["y"][m, n] == pytest.approx(acc, rel=1e-14, abs=0)
            assert r["labsx"][m, n] == pytest.approx(mag, rel=1e-14)
    assert np.allclose(r["labs"], np.abs(np.take_along_axis(lutf, codes.astype(np.int64), axis=1)).sum(axis=1), rtol=1e-14)
    # reversed activations or a reversed code order change the result
    r_rev = oracle.gemv_w2a16(words, f16_bits(lut), f16_bits(x.flip(1).contiguous()))
    assert not np.allclose(r["y"], r_rev["y"], rtol=1e-6)
    rev = oracle.pack_weights(np.ascontiguousarray(codes.reshape(16, 2, 16)[:, :, ::-1].reshape(16, 32)))
    assert not np.allclose(r["y"], oracle.gemv_w2a16(rev, f16_bits(lut), f16_bits(x))["y"], rtol=1e-6)


def test_w2a16_equals_the_w2a4_oracle_on_integer_activations():
    # activations that are int4 values times a power of two: both definitions describe the same product
    N, K, M = 40, 512, 3
    codes, lut, words, qa = _problem(N, K, M, seed=31, kind="rotated_laplace", B=64)
    s = np.array([0.25, 2.0 ** -9, 8.0])
    x = torch.tensor(qa["q"].astype(np.float64) * s[:, None], dtype=torch.float16)
    assert np.array_equal(x.numpy().astype(np.float64), qa["q"] * s[:, None])      # exact in fp16
    r4 = oracle.gemv_w2a4(words, f16_bits(lut), qa["xq"], f16_bits(torch.tensor(s, dtype=torch.float16)))
    r16 = oracle.gemv_w2a16(words, f16_bits(lut), f16_bits(x))
    assert np.allclose(r16["y"], r4["y"], rtol=1e-11, atol=1e-13)
    # and the magnitude sums: sum_k |L||x| >= s * sum_c |L_c||S_c| (no cancellation inside a code's sum)
    assert np.all(r16["labsx"] >= (r4["tol"] - 1e-5) / 2e-3 * (1 - 1e-12))


def test_w2a16_affine_grid_is_a_plain_matrix_product_and_matches_dense_dequantization():
    N, K, M = 48, 320, 2
    codes, lut, words, x = _problem16(N, K, M, seed=12)
    a, d = 0.125, 0.03125
    lut_aff = torch.tensor([[a + c * d for c in range(4)]] * N, dtype=torch.float16)
    xf = x.numpy().astype(np.float64)
    r = oracle.gemv_w2a16(words, f16_bits(lut_aff), f16_bits(x))
    assert np.allclose(r["y"], a * xf.sum(axis=1)[:, None] + d * (xf @ codes.astype(np.float64).T), rtol=1e-11, atol=1e-12)
    Wd = np.take_along_axis(lut.numpy().astype(np.float64), codes.astype(np.int64), axis=1)
    r2 = oracle.gemv_w2a16(words, f16_bits(lut), f16_bits(x))
    assert np.allclose(r2["y"], xf @ Wd.T, rtol=1e-10, atol=1e-12)
    assert np.allclose(r2["labsx"], np.abs(xf) @ np.abs(Wd).T, rtol=1e-12)


def test_split16_hand_cases_from_fixture():
    rows = [ln.split() for ln in open(os.path.join(GOLD, "split16_hand_cases.txt")) if ln.strip() and not ln.startswith("#")]
    x = torch.tensor([[float(r[0]) for r in rows]], dtype=torch.float16)
    assert np.array_equal(x.numpy().astype(np.float64)[0], [float(r[0]) for r in rows])   # the fixture's x are fp16 values
    sp = oracle.split_act16(f16_bits(x))
    want = np.array([[int(v) for v in r[2:6]] for r in rows], dtype=np.int8).T       # [4][K]
    assert np.array_equal(sp["digits"][0], want)
    assert np.array_equal(sp["unit"][0], [2.0 ** -21, 2.0 ** -15, 2.0 ** -9, 2.0 ** -3])


def test_split16_digits_reproduce_the_activations():
    rng = np.random.default_rng(4)
    toks = [synth.make_activations(1, 1024, 9).numpy()[0].astype(np.float64),
            rng.standard_normal(1024) * 1e-3, rng.standard_normal(1024) * 200.0,
            np.concatenate([[65504.0, -65504.0, 2.0 ** -24, -2.0 ** -14], rng.standard_normal(1020)]),
            np.concatenate([[2.0 ** -24 * 3], np.zeros(1023)]),        # a token of subnormals only
            np.zeros(1024)]
    x = torch.tensor(np.stack(toks), dtype=torch.float16)
    xf = x.numpy().astype(np.float64)
    sp = oracle.split_act16(f16_bits(x))
    dg, unit = sp["digits"].astype(np.int64), sp["unit"]
    assert dg[:, :3].min() >= -32 and dg[:, :3].max() <= 31 and np.abs(dg[:, 3]).max() <= 16
    for m in range(x.shape[0]):
        amax = np.abs(xf[m]).max()
        E = int(np.floor(np.log2(amax))) if amax > 0 else 0
        assert np.array_equal(unit[m], 2.0 ** (E - 21 + 6 * np.arange(4)))
        X = dg[m, 0] + 64 * dg[m, 1] + 4096 * dg[m, 2] + 262144 * dg[m, 3]
        rec = X * 2.0 ** (E - 21)
        assert np.all(np.abs(rec - xf[m]) <= 2.0 ** (E - 22))                        # half a unit at most
        big = np.abs(xf[m]) >= 2.0 ** (E - 11)                                       # 11 significant bits fit above the unit
        assert np.array_equal(rec[big], xf[m][big])
        assert np.array_equal(X, np.rint(xf[m] * 2.0 ** (21 - E)).astype(np.int64))   # numpy rounds half to even
    assert not dg[5].any()
    with pytest.raises(ValueError):
        oracle.split_act16(np.array([[0x7C00, 0]], dtype=np.uint16))


# ----------------------------------------------------------------------------- per-code sums of 8-bit planes
def test_percode_sums_i8_brute_force_and_invariants():
    rng = np.random.default_rng(41)
    N, K, C = 7, 64, 3
    codes = rng.integers(0, 4, size=(N, K), dtype=np.uint8)
    planes = rng.integers(-128, 128, size=(C, K)).astype(np.int8)
    S = oracle.percode_sums_i8(oracle.pack_weights(codes), planes)
    ref = np.zeros((C, N, 4), dtype=np.int64)
    for j in range(C):          # the definition as a plain loop
        for n in range(N):
            for k in range(K):
                ref[j, n, int(codes[n, k])] += int(planes[j, k])
    assert np.array_equal(S, ref)
    # the four sums of a row add up to the plane's total, whatever the codes
    assert np.array_equal(S.sum(axis=2), np.repeat(planes.astype(np.int64).sum(axis=1)[:, None], N, axis=1))
    # a planted mistake (codes read in reversed order) is caught
    bad = oracle.percode_sums_i8(oracle.pack_weights(codes[:, ::-1].copy()), planes)
    assert not np.array_equal(bad, ref)


def test_percode_sums_i8_equal_the_w2a4_sums_on_int4_planes():
    N, K, M = 33, 512, 4
    codes, lut = synth.make_layer(N, K, 128, "uniform", 3)
    x = synth.make_activations(M, K, 3)
    qa = oracle.quantize_act(f16_bits(x), 128, 1.0)
    words = oracle.pack_weights(codes.numpy())
    ref = oracle.gemv_w2a4(words, f16_bits(lut), qa["xq"], qa["scale"])
    assert np.array_equal(oracle.percode_sums_i8(words, oracle.unpack_act(qa["xq"]).astype(np.int8)), ref["S"])
