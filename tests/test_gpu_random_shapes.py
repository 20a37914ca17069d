"""Seeded random sweep of shapes through every GEMV entry point against the CPU oracle: row counts around
the tile and phase boundaries of the streaming kernel, K any multiple of 64 (128 with the group-wise grid),
1 to 16 tokens, every kernel variant."""
import numpy as np
import pytest
import torch

import oracle
import paper_2502_15779_b200 as rcp
from gen import synth
from helpers import f16_bits

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _cases(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        # rows: small, around one tile (256), around a round of 148 x 256 rows, and in between
        N = int(rng.choice([rng.integers(1, 40), rng.integers(200, 300), rng.integers(2300, 2450),
                            rng.integers(37800, 38000), rng.integers(1, 6000)]))
        if N > 30000:
            K = 64 * int(rng.integers(1, 9))
        else:
            K = 64 * int(rng.choice([rng.integers(1, 20), rng.integers(20, 180), 128, 172, 224, 448]))
        M = int(rng.choice([1, 1, 2, 3, 5, 8, 9, 16]))
        variant = str(rng.choice(["auto", "dp4a", "mma", "mma_only", "simple"]))
        grouped = bool(rng.integers(0, 2)) and K % 128 == 0
        if grouped and variant == "mma":
            variant = "mma_only"
        out.append(pytest.param(N, K, M, variant, grouped, i, id=f"{i}-N{N}-K{K}-M{M}-{variant}{'-g' if grouped else ''}"))
    return out


@pytest.mark.parametrize("N,K,M,variant,grouped,i", _cases(48, 20250215))
def test_random_shape(N, K, M, variant, grouped, i):
    B = 64 if K % 128 else int(np.random.default_rng(i).choice([1, 64, 128]))
    seed = 5000 + i
    if grouped:
        codes, lut = synth.make_layer_grouped(N, K, 128, B, "uniform", seed, device=DEV)
    else:
        codes, lut = synth.make_layer(N, K, B, "uniform", seed, device=DEV)
    x = synth.make_activations(M, K, seed, device=DEV)
    words = rcp.rcp_pack_weights(codes)
    xq, scale = rcp.rcp_quantize_act(x, B, 1.0)
    ws = rcp.make_workspace(M, N, K, DEV)
    if grouped:
        y = rcp.rcp_gemv_w2a4_grouped(words, lut, xq, scale, group=128, workspace=ws, variant=variant)
    else:
        y = rcp.rcp_gemv_w2a4(words, lut, xq, scale, workspace=ws, variant=variant)
    y_lin = rcp.rcp_linear_w2a4(x, B, 1.0, words, lut, group=128 if grouped else 0, xq=torch.empty_like(xq),
                                scale=torch.empty_like(scale), workspace=ws)
    torch.cuda.synchronize()
    assert int(ws.abs().max()) == 0
    rows = np.arange(N) if N * K * M <= 1 << 24 else np.unique(np.concatenate(
        [np.arange(min(N, 64)), np.arange(max(N - 64, 0), N), np.random.default_rng(i).integers(0, N, size=256)]))
    qa = oracle.quantize_act(f16_bits(x), B, 1.0)
    assert np.array_equal(xq.cpu().numpy(), qa["xq"]) and np.array_equal(f16_bits(scale), qa["scale"])
    w_ref = oracle.pack_weights(codes.cpu().numpy()[rows])
    assert np.array_equal(words.cpu().numpy().view(np.uint32)[rows], w_ref)
    lb = np.ascontiguousarray(f16_bits(lut)[rows])
    ref = (oracle.gemv_w2a4_grouped(w_ref, lb, qa["xq"], qa["scale"], 128) if grouped
           else oracle.gemv_w2a4(w_ref, lb, qa["xq"], qa["scale"]))
    for out in (y, y_lin):
        got = out.float().cpu().numpy().astype(np.float64)[:, rows]
        assert np.all(np.isfinite(got))
        assert np.all(np.abs(got - ref["y"]) <= ref["tol"])
    # the integer sums of the kernel the variant names (auto: the plain kernel) and of the linear call's kernel
    shape = (M, N, K // 128, 4) if grouped else (M, N, 4)
    S1 = torch.full(shape, -12345, dtype=torch.int32, device=DEV)
    S2 = torch.full(shape, -12345, dtype=torch.int32, device=DEV)
    if grouped:
        rcp.rcp_gemv_w2a4_grouped(words, lut, xq, scale, group=128, workspace=ws, variant=variant, S_dbg=S1)
    else:
        rcp.rcp_gemv_w2a4(words, lut, xq, scale, workspace=ws, variant=variant, S_dbg=S1)
    rcp.rcp_linear_w2a4(x, B, 1.0, words, lut, group=128 if grouped else 0, xq=torch.empty_like(xq),
                        scale=torch.empty_like(scale), workspace=ws, S_dbg=S2)
    assert np.array_equal(S1.cpu().numpy()[:, rows], ref["S"])
    assert np.array_equal(S2.cpu().numpy()[:, rows], ref["S"])


@pytest.mark.parametrize("N,K,M,variant,grouped,i", [c for c in _cases(48, 20250215) if not c.values[4]][:20])
def test_random_shape_weight_only(N, K, M, variant, grouped, i):
    """The same sweep through the weight-only form (fp16 activations): digits bit for bit, y within the bound
    its arithmetic gives."""
    seed = 7000 + i
    codes, lut = synth.make_layer(N, K, 64, "uniform", seed, device=DEV)
    x = synth.make_activations(M, K, seed, device=DEV)
    words = rcp.rcp_pack_weights(codes)
    digits = torch.empty((M, 4, K), dtype=torch.int8, device=DEV)
    unit = torch.empty((M, 4), dtype=torch.float32, device=DEV)
    ws = rcp.make_workspace(M, N, K, DEV)
    y = rcp.rcp_gemv_w2a16(words, lut, x, digits=digits, unit=unit, workspace=ws)
    torch.cuda.synchronize()
    assert int(ws.abs().max()) == 0
    sp = oracle.split_act16(f16_bits(x))
    assert np.array_equal(digits.cpu().numpy(), sp["digits"])
    assert np.array_equal(unit.cpu().numpy().astype(np.float64), sp["unit"])
    rows = np.arange(N) if N * K * M <= 1 << 24 else np.unique(np.concatenate(
        [np.arange(min(N, 64)), np.arange(max(N - 64, 0), N), np.random.default_rng(i).integers(0, N, size=256)]))
    ref = oracle.gemv_w2a16(oracle.pack_weights(codes.cpu().numpy()[rows]), np.ascontiguousarray(f16_bits(lut)[rows]),
                            f16_bits(x))
    tol = (0.5 * sp["unit"][:, :1] * ref["labs"][None, :] + 2.0 ** -20 * ref["labsx"]
           + 2.0 ** -11 * np.abs(ref["y"]) + 2.0 ** -24)
    got = y.float().cpu().numpy().astype(np.float64)[:, rows]
    assert np.all(np.isfinite(got)) and np.all(np.abs(got - ref["y"]) <= tol)
    S = torch.full((4 * M, N, 4), -12345, dtype=torch.int32, device=DEV)
    rcp.rcp_gemv_w2a16(words, lut, x, workspace=ws, S_dbg=S)
    w_rows = oracle.pack_weights(codes.cpu().numpy()[rows])
    assert np.array_equal(S.cpu().numpy()[:, rows], oracle.percode_sums_i8(w_rows, sp["digits"].reshape(4 * M, K)))


@pytest.mark.parametrize("N,K,M,grouped", [(70, 65536, 1, False), (40, 65536, 8, False), (33, 65536, 2, True),
                                           (20, 65536, 5, True), (300000, 64, 1, False), (150000, 128, 3, True),
                                           (1, 64, 16, False), (1, 128, 16, True)])
def test_extreme_shapes(N, K, M, grouped):
    """The longest K the library takes, very many short rows, a single row: through the default variant."""
    B = 128 if K >= 128 else 64
    seed = N + K + M
    if grouped:
        codes, lut = synth.make_layer_grouped(N, K, 128, B, "uniform", seed, device=DEV)
    else:
        codes, lut = synth.make_layer(N, K, B, "uniform", seed, device=DEV)
    x = synth.make_activations(M, K, seed, device=DEV)
    words = rcp.rcp_pack_weights(codes)
    xq, scale = rcp.rcp_quantize_act(x, B, 1.0)
    ws = rcp.make_workspace(M, N, K, DEV)
    y = (rcp.rcp_gemv_w2a4_grouped(words, lut, xq, scale, group=128, workspace=ws) if grouped
         else rcp.rcp_gemv_w2a4(words, lut, xq, scale, workspace=ws))
    torch.cuda.synchronize()
    assert int(ws.abs().max()) == 0
    rows = np.arange(N) if N <= 4096 else np.unique(np.concatenate(
        [np.arange(min(N, 64)), np.arange(max(N - 64, 0), N), np.random.default_rng(seed).integers(0, N, size=512)]))
    qa = oracle.quantize_act(f16_bits(x), B, 1.0)
    assert np.array_equal(xq.cpu().numpy(), qa["xq"]) and np.array_equal(f16_bits(scale), qa["scale"])
    w_ref = oracle.pack_weights(codes.cpu().numpy()[rows])
    lb = np.ascontiguousarray(f16_bits(lut)[rows])
    ref = (oracle.gemv_w2a4_grouped(w_ref, lb, qa["xq"], qa["scale"], 128) if grouped
           else oracle.gemv_w2a4(w_ref, lb, qa["xq"], qa["scale"]))
    got = y.float().cpu().numpy().astype(np.float64)[:, rows]
    assert np.all(np.isfinite(got)) and np.all(np.abs(got - ref["y"]) <= ref["tol"])


@pytest.mark.parametrize("N,K,M,variant,grouped", [(4096, 4096, 1, "auto", False), (5000, 2048, 8, "auto", False),
                                                   (3000, 11008, 2, "auto", True), (2600, 8192, 1, "linear", False),
                                                   (2500, 20480, 8, "auto", False), (5000, 4096, 16, "auto", False),
                                                   (3000, 4096, 1, "w2a16", False), (2500, 20480, 2, "w2a16", False)])
def test_many_launches_repeat_bit_for_bit(N, K, M, variant, grouped):
    """A few thousand back-to-back launches (the ring, its barriers and the phases restart every time): the
    status word stays clear and every launch returns the same bits. Covers the forms with shared-memory state of
    their own as well: K in parts, two column tiles, the weight-only form with and without the split inside."""
    B = K if (K & (K - 1)) == 0 else 128
    if grouped:
        codes, lut = synth.make_layer_grouped(N, K, 128, B, "uniform", 77, device=DEV)
    else:
        codes, lut = synth.make_layer(N, K, B, "uniform", 77, device=DEV)
    x = synth.make_activations(M, K, 77, device=DEV)
    words = rcp.rcp_pack_weights(codes)
    xq, scale = rcp.rcp_quantize_act(x, B, 1.0)
    ws = rcp.make_workspace(M, N, K, DEV)
    ys = [torch.empty(M, N, dtype=torch.float16, device=DEV) for _ in range(2)]

    dg = torch.empty(M, 4, K, dtype=torch.int8, device=DEV)
    un = torch.empty(M, 4, dtype=torch.float32, device=DEV)

    def launch(y):
        if variant == "w2a16":
            rcp.rcp_gemv_w2a16(words, lut, x, y=y, digits=dg, unit=un, workspace=ws)
        elif variant == "linear":
            rcp.rcp_linear_w2a4(x, B, 1.0, words, lut, y=y, xq=xq, scale=scale, workspace=ws)
        elif grouped:
            rcp.rcp_gemv_w2a4_grouped(words, lut, xq, scale, group=128, y=y, workspace=ws)
        else:
            rcp.rcp_gemv_w2a4(words, lut, xq, scale, y=y, workspace=ws)

    launch(ys[0])
    ref = ys[0].clone()
    for i in range(3000):
        launch(ys[i & 1])
        if i % 500 == 499:
            torch.cuda.synchronize()
            assert torch.equal(ys[0].view(torch.int16), ref.view(torch.int16))
            assert torch.equal(ys[1].view(torch.int16), ref.view(torch.int16))
    torch.cuda.synchronize()
    assert int(ws.abs().max()) == 0


def test_packed_weights_beyond_four_gibibytes():
    """270 000 rows of 65 536 weights: 17.7 G codes, 4.4 GB of packed words, so every byte offset and element
    index past 2^32 is exercised (packing, the one-token and the eight-token kernel, the plain kernel's integer
    sums, the group-wise grid, the 3-bit kernel), on sampled rows against the oracle."""
    if torch.cuda.get_device_properties(0).total_memory < 60 << 30:
        pytest.skip("needs about 35 GB of device memory")
    N, K, B = 270000, 65536, 128
    g = torch.Generator(device=DEV)
    g.manual_seed(270000)
    codes = torch.randint(0, 4, (N, K), dtype=torch.uint8, device=DEV, generator=g)
    words = rcp.rcp_pack_weights(codes)
    rows = np.unique(np.concatenate([np.arange(24), np.arange(N - 24, N), [65535, 65536, 65537, 131071, 131072],
                                     np.random.default_rng(7).integers(0, N, size=48)]))
    rows_t = torch.from_numpy(rows).to(DEV)
    w_ref = oracle.pack_weights(codes[rows_t].cpu().numpy())
    del codes
    torch.cuda.empty_cache()
    assert np.array_equal(words[rows_t].cpu().numpy().view(np.uint32), w_ref)
    lut = synth.make_lut(N, 11, device=DEV)
    for M, variant in ((1, "auto"), (8, "mma_only"), (1, "simple")):
        x = synth.make_activations(M, K, 3 + M, device=DEV)
        xq, scale = rcp.rcp_quantize_act(x, B, 1.0)
        qa = oracle.quantize_act(f16_bits(x), B, 1.0)
        assert np.array_equal(xq.cpu().numpy(), qa["xq"]) and np.array_equal(f16_bits(scale), qa["scale"])
        ws = rcp.make_workspace(M, N, K, DEV)
        S = torch.zeros(M, N, 4, dtype=torch.int32, device=DEV) if variant == "simple" else None
        y = rcp.rcp_gemv_w2a4(words, lut, xq, scale, workspace=ws, variant=variant, S_dbg=S)
        torch.cuda.synchronize()
        assert int(ws.abs().max()) == 0
        ref = oracle.gemv_w2a4(w_ref, np.ascontiguousarray(f16_bits(lut[rows_t])), qa["xq"], qa["scale"])
        got = y[:, rows_t].float().cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(got)) and np.all(np.abs(got - ref["y"]) <= ref["tol"]), (M, variant)
        if S is not None:
            assert np.array_equal(S[:, rows_t].cpu().numpy(), ref["S"])
    # one token: group-wise grid and the 3-bit kernel on the same words (a random plane of top bits)
    x = synth.make_activations(1, K, 5, device=DEV)
    xq, scale = rcp.rcp_quantize_act(x, B, 1.0)
    qa = oracle.quantize_act(f16_bits(x), B, 1.0)
    ws = rcp.make_workspace(1, N, K, DEV)
    glut = synth.make_lut_grouped(N, K // 128, 13, device=DEV)
    y = rcp.rcp_gemv_w2a4_grouped(words, glut, xq, scale, group=128, workspace=ws)
    torch.cuda.synchronize()
    ref = oracle.gemv_w2a4_grouped(w_ref, np.ascontiguousarray(f16_bits(glut[rows_t])), qa["xq"], qa["scale"], 128)
    got = y[:, rows_t].float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - ref["y"]) <= ref["tol"])
    del glut
    torch.cuda.empty_cache()
    w1 = torch.randint(-2 ** 31, 2 ** 31 - 1, (N, K // 32), dtype=torch.int32, device=DEV, generator=g)
    lut8 = torch.sort(torch.randn(N, 8, device=DEV, generator=g) * 0.02, dim=1).values.half()
    y = rcp.rcp_gemv_w3a4(words, w1, lut8, xq, scale)
    torch.cuda.synchronize()
    ref = oracle.gemv_w3a4(w_ref, w1[rows_t].cpu().numpy().view(np.uint32), np.ascontiguousarray(f16_bits(lut8[rows_t])),
                           qa["xq"], qa["scale"])
    got = y[:, rows_t].float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - ref["y"]) <= ref["tol"])


def test_random_shapes_other_seeds():
    """The sweep above over six more seeds (288 cases) in one test: shapes the fixed list never meets."""
    for seed in (101, 202, 303, 404, 505, 606):
        for c in _cases(48, seed):
            N, K, M, variant, grouped, i = c.values
            test_random_shape(N, K, M, variant, grouped, i)
