"""GPU parity of rcp_linear_w2a4 (activation quantization and LUT GEMV in one call; one kernel for one
or two tokens) against the CPU oracle: xq and scale bit for bit, y within the GEMV's tolerance."""
import numpy as np
import pytest
import torch

import oracle
import paper_2502_15779_b200 as rcp
from gen import synth
from gen.configs import CONFIGS
from helpers import f16_bits

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _check(N, K, B, M, group, clip, seed, kind="uniform", rows=None, staging=True):
    if group:
        codes, lut = synth.make_layer_grouped(N, K, group, B, kind, seed, device=DEV)
    else:
        codes, lut = synth.make_layer(N, K, B, kind, seed, device=DEV)
    x = synth.make_activations(M, K, seed, device=DEV)
    words = rcp.rcp_pack_weights(codes)
    xq = torch.full((M, K // 2), 0xAB, dtype=torch.uint8, device=DEV) if staging else None
    scale = torch.full((M,), -1.0, dtype=torch.float16, device=DEV) if staging else None
    ws = rcp.make_workspace(M, N, K, DEV)
    y = rcp.rcp_linear_w2a4(x, B, clip, words, lut, group=group, xq=xq, scale=scale, workspace=ws)
    y2 = rcp.rcp_linear_w2a4(x, B, clip, words, lut, group=group, xq=xq, scale=scale, workspace=ws)
    torch.cuda.synchronize()
    assert int(ws.abs().max()) == 0, "a bounded wait gave up"
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))
    qa = oracle.quantize_act(f16_bits(x), B, clip)
    if staging:
        assert np.array_equal(f16_bits(scale), qa["scale"])
        assert np.array_equal(xq.cpu().numpy(), qa["xq"])
    sel = np.arange(N) if rows is None else rows
    w_ref = oracle.pack_weights(codes.cpu().numpy()[sel])
    lb = np.ascontiguousarray(f16_bits(lut)[sel])
    ref = (oracle.gemv_w2a4_grouped(w_ref, lb, qa["xq"], qa["scale"], group) if group
           else oracle.gemv_w2a4(w_ref, lb, qa["xq"], qa["scale"]))
    got = y.float().cpu().numpy().astype(np.float64)[:, sel]
    assert np.all(np.isfinite(got))
    err = np.abs(got - ref["y"])
    assert np.all(err <= ref["tol"]), f"max err/tol {np.max(err / ref['tol'])}"
    # the integer sums of the kernel this call runs (checked instantiation), bit for bit
    S = torch.full((M, N, K // group, 4) if group else (M, N, 4), -12345, dtype=torch.int32, device=DEV)
    y3 = rcp.rcp_linear_w2a4(x, B, clip, words, lut, group=group, xq=xq, scale=scale, workspace=ws, S_dbg=S)
    assert np.array_equal(S.cpu().numpy()[:, sel], ref["S"])
    assert torch.equal(y.view(torch.int16), y3.view(torch.int16))


CASES = [
    # N, K, B, M. One token of 4096 or 8192 under one block takes the single kernel (several row counts:
    # rounds, leftover phases, ragged tail); everything else the two kernels
    (40, 64, 1, 1), (40, 64, 64, 2), (100, 256, 16, 1), (33, 512, 128, 2), (64, 512, 512, 1), (129, 1024, 1024, 1),
    (300, 2048, 2048, 1), (300, 2048, 2048, 2), (256, 4096, 4096, 1), (77, 8192, 8192, 2), (500, 8192, 128, 1),
    (77, 8192, 8192, 1), (2500, 8192, 8192, 1), (4097, 4096, 4096, 1), (1, 4096, 4096, 1), (5000, 8192, 8192, 1),
    (130, 11008, 128, 1), (64, 28672, 128, 2), (40, 14336, 128, 1), (513, 1152, 128, 2), (2500, 4096, 256, 1),
    (4800, 1024, 512, 2), (64, 32768, 512, 1),
    # shapes the single kernel does not take: the two kernels run one after the other
    (100, 2048, 1024, 1), (90, 4096, 128, 3), (50, 16384, 16384 // 2, 1), (64, 2048, 2048, 8),
]


@pytest.mark.parametrize("group", [0, 128])
@pytest.mark.parametrize("N,K,B,M", CASES)
def test_linear_matches_oracle(N, K, B, M, group):
    if group and K % group:
        pytest.skip("group does not divide K")
    _check(N, K, B, M, group, 1.0, seed=N + K + M + group, kind="rotated_laplace" if K >= 512 else "uniform")


def test_linear_clip_ratio_zero_token_and_optional_outputs():
    _check(70, 2048, 2048, 2, 0, 0.9, seed=3)
    _check(70, 4096, 4096, 1, 0, 0.9, seed=5)
    _check(70, 8192, 8192, 1, 128, 0.9, seed=4, staging=False)   # the single kernel needs no staging
    _check(600, 4096, 4096, 1, 0, 1.0, seed=6, staging=False)
    N, K, M = 48, 1024, 2
    codes, lut = synth.make_layer(N, K, 128, "uniform", 9, device=DEV)
    x = synth.make_activations(M, K, 9, device=DEV)
    x[0] = 0
    xq = torch.empty(M, K // 2, dtype=torch.uint8, device=DEV)
    scale = torch.empty(M, dtype=torch.float16, device=DEV)
    y = rcp.rcp_linear_w2a4(x, 128, 1.0, rcp.rcp_pack_weights(codes), lut, xq=xq, scale=scale)
    assert float(scale[0]) == 0 and int(xq[0].max()) == 0 and float(y[0].abs().max()) == 0
    assert float(y[1].abs().max()) > 0


def test_linear_argument_errors():
    L = rcp.lib()
    z = torch.zeros(8192, dtype=torch.int32, device=DEV)
    p = z.data_ptr()
    f = L.rcp_linear_w2a4
    assert f(None, 1, 128, 128, 1.0, p, p, 0, 16, p, p, p, p, None) == -1
    assert f(p, 0, 128, 128, 1.0, p, p, 0, 16, p, p, p, p, None) == -2
    assert f(p, 1, 128, 96, 1.0, p, p, 0, 16, p, p, p, p, None) == -2      # block not a power of two
    assert f(p, 1, 128, 128, 0.0, p, p, 0, 16, p, p, p, p, None) == -2     # clip ratio
    assert f(p, 1, 192, 64, 1.0, p, p, 128, 16, p, p, p, p, None) == -2    # group does not divide K
    assert f(p + 2, 1, 128, 128, 1.0, p, p, 0, 16, p, p, p, p, None) == -3
    assert f(p, 3, 128, 128, 1.0, p, p, 0, 16, p, None, None, p, None) == -1   # two-kernel path without staging


def _full_cases():
    seen, out = set(), []
    for ci, cfg in enumerate(CONFIGS):
        for layer in cfg.layers:
            key = (layer.N, layer.K, layer.had_block)
            if key in seen:
                continue
            seen.add(key)
            out.append(pytest.param(ci, layer.N, layer.K, layer.had_block, id=f"{cfg.key}-{layer.name}"))
    return out


@pytest.mark.parametrize("ci,N,K,B", _full_cases())
def test_linear_full_size_configs_sampled_rows(ci, N, K, B):
    """One token, every layer shape of the five configurations at full size (the call the benchmark's step makes)."""
    rng = np.random.default_rng(N + K)
    rows = np.unique(np.concatenate([np.arange(min(N, 32)), np.arange(max(0, N - 32), N),
                                     rng.integers(0, N, size=min(N, 128))]))
    _check(N, K, B, 1, 0, 1.0, seed=3000 + ci, rows=rows)


@pytest.mark.parametrize("pinned", [True, False])
@pytest.mark.parametrize("N,K,B,M", [(300, 8192, 8192, 1), (200, 4096, 128, 1), (150, 11008, 128, 2), (64, 2048, 2048, 3)])
def test_linear_host_buffers(N, K, B, M, pinned):
    """rcp_linear_w2a4_host: activations from and results to host memory (pinned or pageable), twice with
    different activations in the same buffers (no stale data between calls)."""
    codes, lut = synth.make_layer(N, K, B, "uniform", N + K, device=DEV)
    words = rcp.rcp_pack_weights(codes)
    xh = torch.empty(M, K, dtype=torch.float16)
    yh = torch.empty(M, N, dtype=torch.float16)
    if pinned:
        xh, yh = xh.pin_memory(), yh.pin_memory()
    x_dev = torch.empty(M, K, dtype=torch.float16, device=DEV)
    xq = torch.empty(M, K // 2, dtype=torch.uint8, device=DEV)
    scale = torch.empty(M, dtype=torch.float16, device=DEV)
    y_dev = torch.empty(M, N, dtype=torch.float16, device=DEV)
    ws = rcp.make_workspace(M, N, K, DEV)
    w_ref = oracle.pack_weights(codes.cpu().numpy())
    for rep in range(2):
        xh.copy_(synth.make_activations(M, K, 100 + rep))
        yh.fill_(float("nan"))
        rcp.rcp_linear_w2a4_host(xh, B, 1.0, words, lut, yh, x_dev, xq, scale, y_dev, ws)
        torch.cuda.synchronize()
        qa = oracle.quantize_act(f16_bits(xh), B, 1.0)
        ref = oracle.gemv_w2a4(w_ref, f16_bits(lut), qa["xq"], qa["scale"])
        got = yh.float().numpy().astype(np.float64)
        assert np.all(np.isfinite(got)) and np.all(np.abs(got - ref["y"]) <= ref["tol"])
