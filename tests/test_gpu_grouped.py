"""GPU parity of the group-wise-grid GEMV (one four-entry grid per group of G weights of a row),
called through the C ABI, against the CPU oracle on the same seeded inputs. The per-group per-code
sums S_c are compared bit for bit, the fp16 outputs within
|y - y_ref| <= 2e-3 * (s * sum_j sum_c |LUT[j][c]| * |S_c[j]|) + 1e-5 (y_ref in double)."""
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

VARIANTS = ["simple", "dp4a", "mma_only", "auto"]


def _check(N, K, G, B, M, kind, variant, seed, rows=None, with_S=True):
    codes, lut = synth.make_layer_grouped(N, K, G, B, kind, seed, device=DEV)
    x = synth.make_activations(M, K, seed, device=DEV)
    words = rcp.rcp_pack_weights(codes)
    xq, scale = rcp.rcp_quantize_act(x, B, 1.0)
    ws = rcp.make_workspace(M, N, K, DEV)
    y = rcp.rcp_gemv_w2a4_grouped(words, lut, xq, scale, group=G, workspace=ws, variant=variant)
    y2 = rcp.rcp_gemv_w2a4_grouped(words, lut, xq, scale, group=G, workspace=ws, variant=variant)
    torch.cuda.synchronize()
    assert int(ws.abs().max()) == 0, "a bounded wait gave up"
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16)), "results must repeat bit for bit"

    qa = oracle.quantize_act(f16_bits(x), B, 1.0)
    assert np.array_equal(xq.cpu().numpy(), qa["xq"]) and np.array_equal(f16_bits(scale), qa["scale"])
    sel = np.arange(N) if rows is None else rows
    w_ref = oracle.pack_weights(codes.cpu().numpy()[sel])
    assert np.array_equal(words.cpu().numpy().view(np.uint32)[sel], w_ref)
    ref = oracle.gemv_w2a4_grouped(w_ref, np.ascontiguousarray(f16_bits(lut)[sel]), qa["xq"], qa["scale"], G)
    outs = [y]
    if with_S:
        # the per-group sums from the checked instantiation of the kernel `variant` names; with auto, from the
        # plain kernel and from the streaming kernel auto dispatches to
        todo = [variant]
        if variant == "auto" and G == 128:
            todo.append("dp4a" if M <= 2 else "mma_only")
        for v in todo:
            S = torch.full((M, N, K // G, 4), -12345, dtype=torch.int32, device=DEV)
            outs.append(rcp.rcp_gemv_w2a4_grouped(words, lut, xq, scale, group=G, workspace=ws, S_dbg=S, variant=v))
            assert np.array_equal(S.cpu().numpy()[:, sel], ref["S"]), f"S_c of variant {v}"
            del S
    for out in outs:
        got = out.float().cpu().numpy().astype(np.float64)[:, sel]
        err = np.abs(got - ref["y"])
        assert np.all(np.isfinite(got))
        assert np.all(err <= ref["tol"]), f"max err/tol {np.max(err / ref['tol'])}"


SMALL = [
    # N, K, B, M
    (1, 128, 128, 1), (16, 256, 1, 1), (17, 384, 128, 3), (100, 640, 128, 2), (129, 512, 512, 1),
    (127, 1024, 128, 16), (300, 2048, 2048, 1), (256, 4096, 4096, 4), (130, 11008, 128, 1), (64, 28672, 128, 1),
    (40, 14336, 128, 16), (33, 8192, 8192, 8), (2048, 2048, 2048, 1), (513, 1152, 128, 5), (1000, 2560, 128, 7),
    (4800, 1024, 128, 2), (2500, 512, 128, 8),
    # K so long that eight tokens' expanded activations do not fit: the form with the activations streamed beside
    # the weights (five to eight tokens in one launch, sixteen as two)
    (64, 28672, 128, 8), (200, 20480, 128, 5), (33, 65536, 128, 7), (2400, 16512, 128, 8), (40, 28672, 128, 16),
]


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("N,K,B,M", SMALL)
def test_grouped_gemv_small_and_ragged(N, K, B, M, variant):
    _check(N, K, 128, B, M, "rotated_laplace" if K >= 512 else "uniform", variant, seed=N + K + M)


@pytest.mark.parametrize("N,K,G,M", [(50, 256, 16, 2), (33, 512, 64, 1), (20, 1024, 256, 3), (9, 2048, 2048, 1)])
def test_grouped_gemv_other_group_sizes_take_the_plain_kernel(N, K, G, M):
    _check(N, K, G, 64, M, "uniform", "auto", seed=N + G)
    codes, lut = synth.make_layer_grouped(N, K, G, 1, "uniform", 1, device=DEV)
    xq, scale = rcp.rcp_quantize_act(synth.make_activations(M, K, 1, device=DEV), 1, 1.0)
    with pytest.raises(rcp.RcpError) as e:
        rcp.rcp_gemv_w2a4_grouped(rcp.rcp_pack_weights(codes), lut, xq, scale, group=G, variant="dp4a")
    assert e.value.status == -7


def test_grouped_gemv_with_equal_grids_matches_the_per_row_kernel_within_tolerance_and_degenerate_inputs():
    N, K, M, G = 70, 1024, 2, 128
    lut = synth.make_lut(N, 5, DEV)
    codes = synth.make_codes_uniform(N, K, 5, DEV)
    codes[0] = 3
    codes[1] = 0
    words = rcp.rcp_pack_weights(codes)
    x = synth.make_activations(M, K, 5, DEV)
    x[1] = 0   # all-zero token: scale 0, y = 0
    xq, scale = rcp.rcp_quantize_act(x, 128, 1.0)
    lut_g = lut[:, None, :].repeat(1, K // G, 1).contiguous()
    ref = oracle.gemv_w2a4(oracle.pack_weights(codes.cpu().numpy()), f16_bits(lut), xq.cpu().numpy(), f16_bits(scale))
    for variant in VARIANTS:
        y = rcp.rcp_gemv_w2a4_grouped(words, lut_g, xq, scale, group=G, variant=variant)
        got = y.float().cpu().numpy().astype(np.float64)
        # the per-group bound is at least the per-row bound; the per-row reference is the same number
        refg = oracle.gemv_w2a4_grouped(oracle.pack_weights(codes.cpu().numpy()), f16_bits(lut_g), xq.cpu().numpy(),
                                        f16_bits(scale), G)
        assert np.all(np.abs(got - ref["y"]) <= refg["tol"])
        assert np.all(got[1] == 0)


def test_grouped_gemv_argument_errors():
    L = rcp.lib()
    z = torch.zeros(4096, dtype=torch.int32, device=DEV)
    p = z.data_ptr()
    assert L.rcp_gemv_w2a4_grouped(None, p, 128, p, p, 1, 16, 128, p, p, None, None) == -1
    assert L.rcp_gemv_w2a4_grouped(p, p, 128, p, p, 0, 16, 128, p, p, None, None) == -2
    assert L.rcp_gemv_w2a4_grouped(p, p, 128, p, p, 1, 16, 192, p, p, None, None) == -2   # 128 does not divide K
    assert L.rcp_gemv_w2a4_grouped(p, p, 24, p, p, 1, 16, 192, p, p, None, None) == -2    # not a multiple of 16
    assert L.rcp_gemv_w2a4_grouped(p, p + 4, 128, p, p, 1, 16, 128, p, p, None, None) == -3
    assert L.rcp_gemv_w2a4_grouped_variant(3, p, p, 128, p, p, 1, 16, 128, p, p, None, None) == -7   # no hybrid form


def _full_cases():
    seen, out = set(), []
    for ci, cfg in enumerate(CONFIGS):
        for layer in cfg.layers:
            if layer.K % 128:
                continue
            for M in cfg.Ms:
                key = (layer.N, layer.K, layer.had_block, M)
                if key in seen:
                    continue
                seen.add(key)
                out.append(pytest.param(ci, layer.N, layer.K, layer.had_block, M, id=f"{cfg.key}-{layer.name}-M{M}"))
    return out


@pytest.mark.parametrize("ci,N,K,B,M", _full_cases())
def test_grouped_gemv_full_size_configs_sampled_rows(ci, N, K, B, M):
    """The five configurations at full size with the paper's group size, variant auto; the oracle checks
    the first and last rows plus a random sample. Codes are uniform: the draw is as large as the layer."""
    rng = np.random.default_rng(N + K + M)
    rows = np.unique(np.concatenate([np.arange(min(N, 32)), np.arange(max(0, N - 32), N),
                                     rng.integers(0, N, size=min(N, 128))]))
    _check(N, K, 128, B, M, "uniform", "auto", seed=2000 + ci, rows=rows)
