"""Weight-only form of the GEMV (fp16 activations) against the CPU oracle: the fixed-point digits bit for
bit, y within a tolerance derived from the arithmetic of the path."""
import numpy as np
import pytest
import torch

import oracle
import paper_2502_15779_b200 as rcp
from gen import synth
from helpers import f16_bits

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _tolerance(ref, unit0):
    """Fixed point: each activation is off by half a unit 2^(E-21) at most -> 2^(E-22) * sum_k |L|.
    fp32 finish: four fused multiply-adds per digit on exact integers and three additions, a few 2^-24 of
    sum |L||x| (which bounds every partial sum). fp16 result: 2^-11 |y|. Plus the smallest fp16 step."""
    return (0.5 * unit0[:, None] * ref["labs"][None, :] + 2.0 ** -20 * ref["labsx"]
            + 2.0 ** -11 * np.abs(ref["y"]) + 2.0 ** -24)


def _check(N, K, M, seed, kind="rotated_laplace", x=None, rows=None):
    codes, lut = synth.make_layer(N, K, 128 if K % 128 == 0 else 64, kind, seed, device=DEV)
    if x is None:
        x = synth.make_activations(M, K, seed, device=DEV)
    words = rcp.rcp_pack_weights(codes)
    digits = torch.full((M, 4, K), 77, dtype=torch.int8, device=DEV)
    unit = torch.zeros((M, 4), dtype=torch.float32, device=DEV)
    ws = rcp.make_workspace(M, N, K, DEV)
    y = rcp.rcp_gemv_w2a16(words, lut, x, digits=digits, unit=unit, workspace=ws)
    y2 = rcp.rcp_gemv_w2a16(words, lut, x, workspace=ws)
    torch.cuda.synchronize()
    assert int(ws.abs().max()) == 0
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))
    sp = oracle.split_act16(f16_bits(x))
    assert np.array_equal(digits.cpu().numpy(), sp["digits"])
    assert np.array_equal(unit.cpu().numpy().astype(np.float64), sp["unit"])
    sel = np.arange(N) if rows is None else rows
    w_ref = oracle.pack_weights(codes.cpu().numpy()[sel])
    ref = oracle.gemv_w2a16(w_ref, np.ascontiguousarray(f16_bits(lut)[sel]), f16_bits(x))
    got = y.float().cpu().numpy().astype(np.float64)[:, sel]
    tol = _tolerance(ref, sp["unit"][:, 0])
    err = np.abs(got - ref["y"])
    assert np.all(np.isfinite(got))
    assert np.all(err <= tol), f"max err/tol {np.max(err / tol)}"
    # the per-code sums of every digit plane, from the checked instantiation of the same kernels
    S = torch.full((4 * M, N, 4), -12345, dtype=torch.int32, device=DEV)
    y3 = rcp.rcp_gemv_w2a16(words, lut, x, workspace=ws, S_dbg=S)
    assert np.array_equal(S.cpu().numpy()[:, sel], oracle.percode_sums_i8(w_ref, sp["digits"].reshape(4 * M, K)))
    assert torch.equal(y.view(torch.int16), y3.view(torch.int16))
    return err, tol, ref


@pytest.mark.parametrize("N,K,M", [(1, 64, 1), (17, 192, 3), (100, 320, 2), (127, 1024, 4), (300, 2048, 1),
                                   (256, 4096, 4), (130, 11008, 1), (64, 28672, 2), (33, 8192, 5), (40, 32768, 1),
                                   (513, 1088, 16), (2500, 4096, 3), (5000, 2048, 7), (2369, 5120, 4), (37965, 512, 2),
                                   (40, 65536, 2), (300, 28672, 3), (2400, 16448, 2)])
def test_w2a16_small_and_ragged(N, K, M):
    _check(N, K, M, seed=N + K + M, kind="rotated_laplace" if K >= 512 else "uniform")


def test_w2a16_on_llm_like_activations_stays_within_the_w2a4_style_bound():
    # On the synthetic decode activations the derived tolerance is far inside 2e-3 * sum |L||x| + 1e-5.
    err, tol, ref = _check(4096, 4096, 2, seed=3)
    assert np.all(tol <= 2e-3 * ref["labsx"] + 1e-5)
    assert np.max(err / (2e-3 * ref["labsx"] + 1e-5)) < 0.5


def test_w2a16_degenerate_tokens():
    K, N = 1024, 70
    g = torch.Generator().manual_seed(1)
    x = torch.randn(6, K, generator=g)
    x[0] = 0                                        # all-zero token
    x[1] = 0; x[1, 5] = 65504.0                     # one element at the top of the fp16 range
    x[2] *= 1e-6                                    # subnormals and tiny normals
    x[3, ::2] = 0; x[3, 1::2] = 2.0 ** -24          # the smallest subnormal only
    x[4, 0] = 3000.0                                # one outlier over small values
    x[5] = -7.0                                     # constant negative
    x = x.to(torch.float16).to(DEV)
    err, tol, ref = _check(N, K, 6, seed=2, x=x)
    y = rcp.rcp_gemv_w2a16(*_layer(N, K, 2), x)
    assert np.all(y[0].float().cpu().numpy() == 0)


def _layer(N, K, seed):
    codes, lut = synth.make_layer(N, K, 128, "rotated_laplace", seed, device=DEV)
    return rcp.rcp_pack_weights(codes), lut


def test_w2a16_matches_w2a4_on_int4_activations():
    # int4 values times a power of two are both a W2A4 input and exact in the fixed-point form: the integer
    # sums agree, only the fp32 finish differs in order
    N, K, M = 777, 2048, 2
    codes, lut = synth.make_layer(N, K, 128, "rotated_laplace", 8, device=DEV)
    words = rcp.rcp_pack_weights(codes)
    x0 = synth.make_activations(M, K, 8, device=DEV)
    xq, scale = rcp.rcp_quantize_act(x0, 128, 1.0)
    qa = oracle.quantize_act(f16_bits(x0), 128, 1.0)
    s = torch.tensor([0.5, 2.0 ** -7], dtype=torch.float16, device=DEV)
    x = (torch.tensor(qa["q"].astype(np.float32), device=DEV) * s.float()[:, None]).to(torch.float16)
    y4 = rcp.rcp_gemv_w2a4(words, lut, xq, s)
    y16 = rcp.rcp_gemv_w2a16(words, lut, x)
    torch.cuda.synchronize()
    d = np.abs(y4.float().cpu().numpy().astype(np.float64) - y16.float().cpu().numpy().astype(np.float64))
    ref = oracle.gemv_w2a16(oracle.pack_weights(codes.cpu().numpy()), f16_bits(lut), f16_bits(x))
    assert np.all(d <= 2.0 ** -10 * np.abs(ref["y"]) + 2.0 ** -19 * ref["labsx"] + 2.0 ** -23)


def test_w2a16_full_size_sampled_rows():
    N, K = 28672, 4096
    rows = np.unique(np.concatenate([np.arange(min(N, 64)), np.arange(max(N - 64, 0), N), np.random.default_rng(0).integers(0, N, 256)]))
    _check(N, K, 1, seed=11, rows=rows)
    N, K = 8192, 28672
    rows = np.unique(np.concatenate([np.arange(32), np.arange(N - 32, N), np.random.default_rng(1).integers(0, N, 64)]))
    _check(N, K, 2, seed=12, rows=rows)


def test_w2a16_argument_errors():
    L = rcp.lib()
    z = torch.zeros(1 << 16, dtype=torch.int32, device=DEV)
    p = z.data_ptr()
    assert L.rcp_gemv_w2a16(None, p, p, 1, 16, 64, p, p, p, p, None) == -1
    assert L.rcp_gemv_w2a16(p, p, p, 0, 16, 64, p, p, p, p, None) == -2
    assert L.rcp_gemv_w2a16(p, p, p, 17, 16, 64, p, p, p, p, None) == -2
    assert L.rcp_gemv_w2a16(p, p, p, 1, 16, 65600, p, p, p, p, None) == -2   # K above the library's limit
    assert L.rcp_gemv_w2a16(p, p, p + 2, 1, 16, 64, p, p, p, p, None) == -3
