"""GPU parity of the 3-bit path (paragraph "Application of LDP on NF3 format": packing and the W3A4
look-up-table GEMV with eight levels per quantization unit), called through the C ABI, against the CPU oracle:
packed words and the per-code sums S_0..S_7 bit for bit, fp16 outputs within
|y - y_ref| <= 2e-3 * (s * sum_j sum_c |LUT[j][c]| * |S_c[j]|) + 1e-5 (y_ref in double); the export with a
learnable centre (Eq. "nf3scales", Eq. "nf3"): packed codes and fp16 levels bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2502_15779_b200 as rcp
from gen import synth
from helpers import f16_bits, normal_float_table

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _layer(N, K, G, seed, kind):
    """codes u8 [N][K] in 0..7 and grids fp16 [N][K/G][8]: uniform codes with sorted normal levels, or a
    Laplace layer exported by the oracle's 3-bit export (learnable centre, normal-float level table)."""
    rng = np.random.default_rng(seed)
    if kind == "uniform":
        codes = rng.integers(0, 8, size=(N, K), dtype=np.uint8)
        lut = np.sort((rng.standard_normal((N, K // G, 8)) * 0.02).astype(np.float16), axis=2)
        return codes, lut
    table, z = normal_float_table(3)
    w = (rng.laplace(0, 0.02, size=(N, K)) + 0.004).astype(np.float16)
    sb = rng.uniform(0.8, 1.0, size=(N, K // G)).astype(np.float32)
    sg = rng.uniform(0.8, 1.0, size=(N, K // G)).astype(np.float32)
    s1 = rng.uniform(0.4, 0.6, size=(N, K // G)).astype(np.float32)
    out = oracle.nf3_export(w.view(np.uint16), sb, sg, s1, table, z, G)
    return out["codes"], out["lut"].view(np.float16)


def _check(N, K, M, group, seed, kind="uniform", rows=None):
    G = group if group else K
    codes, lut = _layer(N, K, G, seed, kind)
    x = synth.make_activations(M, K, seed, device=DEV)
    B = 128 if K % 128 == 0 else 64
    xq, scale = rcp.rcp_quantize_act(x, B, 1.0)
    w2, w1 = rcp.rcp_pack_weights3(torch.from_numpy(codes).to(DEV))
    lut_d = torch.from_numpy(lut.reshape(N, 8) if group == 0 else lut).to(DEV)
    y = rcp.rcp_gemv_w3a4(w2, w1, lut_d, xq, scale, group=group)
    S = torch.full((M, N, K // G, 8), -12345, dtype=torch.int32, device=DEV)
    y2 = rcp.rcp_gemv_w3a4(w2, w1, lut_d, xq, scale, group=group, S_dbg=S)
    torch.cuda.synchronize()
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16)), "checked and production instantiation differ"
    sel = np.arange(N) if rows is None else rows
    r2, r1 = oracle.pack_weights3(codes[sel])
    assert np.array_equal(w2.cpu().numpy().view(np.uint32)[sel], r2)
    assert np.array_equal(w1.cpu().numpy().view(np.uint32)[sel], r1)
    qa = oracle.quantize_act(f16_bits(x), B, 1.0)
    assert np.array_equal(xq.cpu().numpy(), qa["xq"]) and np.array_equal(f16_bits(scale), qa["scale"])
    ref = oracle.gemv_w3a4(r2, r1, np.ascontiguousarray(lut[sel]).view(np.uint16), qa["xq"], qa["scale"], G)
    assert np.array_equal(S.cpu().numpy()[:, sel], ref["S"])
    got = y.float().cpu().numpy().astype(np.float64)[:, sel]
    err = np.abs(got - ref["y"])
    assert np.all(np.isfinite(got))
    assert np.all(err <= ref["tol"]), f"max err/tol {np.max(err / ref['tol'])}"


SMALL = [  # N, K, M
    (1, 64, 1), (8, 128, 1), (17, 192, 3), (100, 320, 2), (129, 512, 1), (127, 1024, 16), (300, 2048, 1), (256, 4096, 4),
    (130, 11008, 1), (64, 28672, 1), (40, 14336, 2), (33, 8192, 8), (2048, 2048, 1), (513, 1088, 5), (1000, 2560, 7),
    (9, 65536, 1), (5000, 64, 2),
    # more rows than resident warps (several rows per warp), odd and even counts of lane steps, ragged last step
    (4000, 4160, 1), (3700, 8256, 2), (3600, 20544, 1),
]


@pytest.mark.parametrize("group", [0, 128])
@pytest.mark.parametrize("N,K,M", SMALL)
def test_w3a4_small_and_ragged(N, K, M, group):
    if group and K % group:
        pytest.skip("group does not divide K")
    _check(N, K, M, group, seed=N + K + M + group, kind="uniform" if K < 512 else "nf3")


@pytest.mark.parametrize("N,K,group", [(22016, 4096, 0), (4096, 11008, 128), (8192, 28672, 0), (57344, 8192, 128)])
def test_w3a4_full_size_sampled_rows(N, K, group):
    rows = np.unique(np.concatenate([np.arange(32), np.arange(N - 32, N), np.random.default_rng(N).integers(0, N, 96)]))
    _check(N, K, 1, group, seed=N + K, kind="uniform", rows=rows)


def test_w3a4_degenerate_inputs_and_argument_errors():
    N, K, M = 70, 1024, 2
    rng = np.random.default_rng(4)
    codes = rng.integers(0, 8, size=(N, K), dtype=np.uint8)
    codes[0] = 7
    codes[1] = 0
    lut = np.sort((rng.standard_normal((N, 8)) * 0.02).astype(np.float16), axis=1)
    lut[3] = np.float16(0.25)                                   # equal levels in a row are legal
    x = synth.make_activations(M, K, 4, device=DEV)
    x[1] = 0                                                    # all-zero token: scale 0, y = 0
    xq, scale = rcp.rcp_quantize_act(x, 128, 1.0)
    w2, w1 = rcp.rcp_pack_weights3(torch.from_numpy(codes).to(DEV))
    y = rcp.rcp_gemv_w3a4(w2, w1, torch.from_numpy(lut).to(DEV), xq, scale)
    r2, r1 = oracle.pack_weights3(codes)
    ref = oracle.gemv_w3a4(r2, r1, lut.view(np.uint16), xq.cpu().numpy(), f16_bits(scale))
    got = y.float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - ref["y"]) <= ref["tol"]) and np.all(got[1] == 0)
    bad = torch.zeros(4, 128, dtype=torch.uint8, device=DEV)
    bad[1, 5] = 8
    with pytest.raises(rcp.RcpError) as e:
        rcp.rcp_pack_weights3(bad)
    assert e.value.status == -4
    L = rcp.lib()
    z = torch.zeros(4096, dtype=torch.int32, device=DEV)
    p = z.data_ptr()
    assert L.rcp_gemv_w3a4(None, p, p, 0, p, p, 1, 16, 64, p, None, None) == -1
    assert L.rcp_gemv_w3a4(p, p, p, 0, p, p, 0, 16, 64, p, None, None) == -2
    assert L.rcp_gemv_w3a4(p, p, p, 64, p, p, 1, 16, 128, p, None, None) == -2     # only groups of 128 (or one grid per row)
    assert L.rcp_gemv_w3a4(p, p, p, 128, p, p, 1, 16, 192, p, None, None) == -2    # 128 does not divide K
    assert L.rcp_gemv_w3a4(p, p + 4, p, 0, p, p, 1, 16, 64, p, None, None) == -3
    assert L.rcp_pack_weights3(None, 4, 128, p, p, None) == -1


# ----------------------------------------------------------------------------- export with a learnable centre
def _export_inputs(N, K, G, seed):
    rng = np.random.default_rng(seed)
    w = (rng.laplace(0, 0.02, size=(N, K)) + 0.004).astype(np.float16)
    NG = K // G
    sb = rng.uniform(0.7, 1.0, size=(N, NG)).astype(np.float32)
    sg = rng.uniform(0.7, 1.0, size=(N, NG)).astype(np.float32)
    s1 = rng.uniform(0.3, 0.7, size=(N, NG)).astype(np.float32)
    return w, sb, sg, s1


def _export_both(w, sb, sg, s1, table, z, G):
    ref = oracle.nf3_export(w.view(np.uint16), sb, sg, s1, table, z, G)
    t = lambda a: torch.from_numpy(a).to(DEV)
    w2, w1, lut = rcp.rcp_nf3_export(t(w), t(sb), t(sg), t(s1), table, z, G)
    torch.cuda.synchronize()
    return ref, w2, w1, lut


@pytest.mark.parametrize("N,K,G", [(1, 64, 32), (5, 128, 128), (33, 1024, 128), (17, 11008, 128), (64, 4096, 4096),
                                   (9, 2048, 64), (300, 512, 256), (3, 28672, 128), (2, 8192, 8192), (40, 384, 96),
                                   (7, 640, 160)])
def test_nf3_export_bit_exact(N, K, G):
    table, z = normal_float_table(3)
    w, sb, sg, s1 = _export_inputs(N, K, G, N + K + G)
    if N > 2:
        w[1, :G] = 0.125                  # a unit without range: code zero_index, eight equal levels
        w[2, :G] = np.abs(w[2, :G])       # a unit whose minimum is positive
        w[0, 5] = w[0, :G].max()          # the maximum twice
    ref, w2, w1, lut = _export_both(w, sb, sg, s1, table, z, G)
    r2, r1 = oracle.pack_weights3(ref["codes"])
    assert np.array_equal(w2.cpu().numpy().view(np.uint32), r2)
    assert np.array_equal(w1.cpu().numpy().view(np.uint32), r1)
    assert np.array_equal(f16_bits(lut), ref["lut"])
    if N * K >= 4096:
        assert len(np.unique(ref["codes"])) == 8


def test_nf3_export_ties_centre_and_range_ends():
    # a symmetric table with levels on a grid of eighths; weights on a grid of sixty-fourths over [-1, 1] with the
    # centre at 0: midpoints between levels are hit exactly (ties take the lower level), 0 goes to the negative side
    table = np.array([-1.0, -0.5, -0.25, 0.0, 0.125, 0.25, 0.5, 1.0], dtype=np.float32)
    G = 192
    w = np.concatenate([np.arange(-64, 65) / 64.0, np.zeros(G - 129)]).astype(np.float16)[None, :].repeat(2, 0)
    one = np.ones((2, 1), dtype=np.float32)
    ref, w2, w1, lut = _export_both(np.ascontiguousarray(w), one, one, 0.5 * one, table, 3, G)
    r2, r1 = oracle.pack_weights3(ref["codes"])
    assert np.array_equal(w2.cpu().numpy().view(np.uint32), r2)
    assert np.array_equal(w1.cpu().numpy().view(np.uint32), r1)
    assert lut[0, 0].tolist() == table.tolist()
    codes = ref["codes"][0]
    assert codes[0] == 0 and codes[128] == 7 and codes[64] == 3          # the ends and the centre
    assert codes[64 - 24] == 1 and codes[64 + 24] == 5                   # -0.375 and 0.375: exact midpoints -> the lower level
    assert codes[64 + 4] == 3 and codes[64 + 5] == 4                     # 0.0625 is the midpoint of 0 and 0.125


def test_nf3_export_rejects_a_bad_table_and_bad_groups():
    table, z = normal_float_table(3)
    w, sb, sg, s1 = _export_inputs(4, 256, 128, 3)
    t = lambda a: torch.from_numpy(a).to(DEV)
    bad = table.copy()
    bad[5] = bad[4]
    with pytest.raises(rcp.RcpError):
        rcp.rcp_nf3_export(t(w), t(sb), t(sg), t(s1), bad, z, 128)
    with pytest.raises(rcp.RcpError):
        rcp.rcp_nf3_export(t(w), t(sb), t(sg), t(s1), table, z + 1, 128)
    w16 = np.ascontiguousarray(w[:, :64])
    s16 = np.ones((4, 4), dtype=np.float32)
    with pytest.raises(rcp.RcpError):
        rcp.rcp_nf3_export(t(w16), t(s16), t(s16), t(s16), table, z, 16)   # groups of 16: below a plane word


@pytest.mark.parametrize("N,K,G,M", [(200, 1024, 128, 1), (150, 2048, 2048, 2), (3000, 4096, 128, 1)])
def test_exported_3bit_layer_through_the_gemv(N, K, G, M):
    table, z = normal_float_table(3)
    w, sb, sg, s1 = _export_inputs(N, K, G, 7 * N + M)
    ref, w2, w1, lut = _export_both(w, sb, sg, s1, table, z, G)
    x = synth.make_activations(M, K, 11, device=DEV)
    B = 128
    xq, scale = rcp.rcp_quantize_act(x, B, 1.0)
    group = 0 if G == K else G
    y = rcp.rcp_gemv_w3a4(w2, w1, lut.reshape(N, 8) if group == 0 else lut, xq, scale, group=group)
    torch.cuda.synchronize()
    qa = oracle.quantize_act(f16_bits(x), B, 1.0)
    r2, r1 = oracle.pack_weights3(ref["codes"])
    out = oracle.gemv_w3a4(r2, r1, ref["lut"], qa["xq"], qa["scale"], G)
    err = np.abs(y.float().cpu().numpy().astype(np.float64) - out["y"])
    assert np.all(err <= out["tol"]), f"max err/tol {np.max(err / out['tol'])}"
