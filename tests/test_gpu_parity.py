"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs. Bit-exact for packed codes, int4 activations, scales and S_c; fp16 outputs within
|y - y_ref| <= 2e-3 * (s * sum_c |LUT[c]| * |S_c|) + 1e-5 (y_ref in double)."""
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

VARIANTS = ["simple", "dp4a", "mma", "mma_only", "mma_stream", "auto"]


def words_np(words_t):
    return words_t.cpu().numpy().view(np.uint32)


# ------------------------------------------------------------------------------ pack
@pytest.mark.parametrize("N,K", [(1, 64), (3, 192), (17, 2048), (128, 11008), (1000, 4096)])
def test_pack_bit_exact(N, K):
    codes = synth.make_codes_uniform(N, K, seed=N * 7 + K)
    words = rcp.rcp_pack_weights(codes.to(DEV))
    assert np.array_equal(words_np(words), oracle.pack_weights(codes.numpy()))


def test_pack_reports_bad_code_and_bad_arguments():
    codes = torch.zeros(4, 128, dtype=torch.uint8, device=DEV)
    codes[2, 77] = 5
    with pytest.raises(rcp.RcpError) as e:
        rcp.rcp_pack_weights(codes)
    assert e.value.status == -4
    with pytest.raises(rcp.RcpError) as e:
        rcp.rcp_pack_weights(torch.zeros(4, 100, dtype=torch.uint8, device=DEV))  # K % 64 != 0
    assert e.value.status == -2
    L = rcp.lib()
    assert L.rcp_pack_weights(None, 4, 128, None, None) == -1
    buf = torch.zeros(4 * 128 + 64, dtype=torch.uint8, device=DEV)
    assert L.rcp_pack_weights(buf.data_ptr() + 1, 4, 128, buf.data_ptr(), None) == -3
    # the context is still usable
    ok = rcp.rcp_pack_weights(torch.ones(4, 128, dtype=torch.uint8, device=DEV))
    assert int(words_np(ok)[0, 0]) == 0x55555555


# ------------------------------------------------------------------------------ quantize_act
QCASES = [
    (1, 64, 1, 1.0), (1, 64, 64, 1.0), (3, 192, 64, 1.0), (2, 256, 2, 1.0), (2, 256, 4, 0.9),
    (1, 2048, 2048, 1.0), (3, 2048, 128, 0.9), (1, 2048, 256, 1.0), (2, 2048, 512, 1.0), (2, 4096, 1024, 1.0),
    (1, 4096, 4096, 1.0), (16, 4096, 4096, 1.0), (1, 8192, 8192, 1.0), (2, 8192, 2048, 1.0), (2, 8192, 128, 1.0),
    (1, 11008, 128, 1.0), (5, 11008, 128, 0.9), (1, 14336, 128, 1.0), (16, 14336, 128, 1.0),
    (1, 28672, 128, 1.0), (8, 28672, 128, 1.0), (1, 28672, 1, 1.0), (2, 16384, 8192, 1.0), (1, 32768, 4096, 1.0),
    (1, 65536, 128, 1.0),
]


@pytest.mark.parametrize("M,K,B,clip", QCASES)
def test_quantize_act_bit_exact(M, K, B, clip):
    x = synth.make_activations(M, K, seed=M + K + B)
    ref = oracle.quantize_act(f16_bits(x), B, clip)
    xq, scale = rcp.rcp_quantize_act(x.to(DEV), B, clip)
    assert np.array_equal(f16_bits(scale), ref["scale"])
    assert np.array_equal(xq.cpu().numpy(), ref["xq"])


def test_quantize_act_zero_token_and_errors():
    x = synth.make_activations(3, 512, seed=1)
    x[1] = 0
    xq, scale = rcp.rcp_quantize_act(x.to(DEV), 128, 1.0)
    ref = oracle.quantize_act(f16_bits(x), 128, 1.0)
    assert np.array_equal(xq.cpu().numpy(), ref["xq"]) and np.array_equal(f16_bits(scale), ref["scale"])
    assert scale[1].item() == 0 and int(xq[1].max()) == 0
    xd = x.to(DEV)
    for bad_block in (3, 96, 1024, 16384):  # not a power of two / does not divide K / too large
        with pytest.raises(rcp.RcpError) as e:
            rcp.rcp_quantize_act(xd, bad_block, 1.0)
        assert e.value.status == -2
    with pytest.raises(rcp.RcpError):
        rcp.rcp_quantize_act(torch.zeros(1, 100, dtype=torch.float16, device=DEV), 1, 1.0)
    with pytest.raises(rcp.RcpError):
        rcp.rcp_quantize_act(xd, 128, 0.0)


# ------------------------------------------------------------------------------ GEMV
def _check_gemv(N, K, B, M, kind, variant, seed, rows=None):
    codes, lut = synth.make_layer(N, K, B, kind, seed, device=DEV)
    x = synth.make_activations(M, K, seed, device=DEV)
    words = rcp.rcp_pack_weights(codes)
    xq, scale = rcp.rcp_quantize_act(x, B, 1.0)
    ws = rcp.make_workspace(M, N, K, DEV)
    y = rcp.rcp_gemv_w2a4(words, lut, xq, scale, workspace=ws, variant=variant)
    S = torch.full((M, N, 4), -12345, dtype=torch.int32, device=DEV)
    y_dbg = rcp.rcp_gemv_w2a4(words, lut, xq, scale, workspace=ws, S_dbg=S, variant=variant)
    torch.cuda.synchronize()
    assert int(ws.abs().max()) == 0, "workspace must be left zero-filled"
    # a second call on the same workspace must give the same bits (workspace reuse)
    y2 = rcp.rcp_gemv_w2a4(words, lut, xq, scale, workspace=ws, variant=variant)
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))

    # oracle inputs come from the oracle's own quantizer and packer, on the same x and codes
    qa = oracle.quantize_act(f16_bits(x), B, 1.0)
    assert np.array_equal(xq.cpu().numpy(), qa["xq"]) and np.array_equal(f16_bits(scale), qa["scale"])
    sel = np.arange(N) if rows is None else rows
    codes_sel = codes.cpu().numpy()[sel]
    w_ref = oracle.pack_weights(codes_sel)
    assert np.array_equal(words_np(words)[sel], w_ref)
    ref = oracle.gemv_w2a4(w_ref, f16_bits(lut)[sel], qa["xq"], qa["scale"])
    # S comes from the checked instantiation of the very kernel `variant` names (auto: the plain kernel)
    assert np.array_equal(S.cpu().numpy()[:, sel, :], ref["S"])
    assert torch.equal(y.view(torch.int16), y_dbg.view(torch.int16)), "checked and production instantiation differ"
    if variant == "auto":
        # ... and from the streaming kernel that auto dispatches to for this token count
        hot = "dp4a" if M == 1 else "mma_only"
        S_hot = torch.full((M, N, 4), -12345, dtype=torch.int32, device=DEV)
        y_hot = rcp.rcp_gemv_w2a4(words, lut, xq, scale, workspace=ws, S_dbg=S_hot, variant=hot)
        assert np.array_equal(S_hot.cpu().numpy()[:, sel, :], ref["S"]), f"S_c of the {hot} kernel"
        assert torch.equal(y.view(torch.int16), y_hot.view(torch.int16))
    for out in (y, y_dbg):
        got = out.float().cpu().numpy().astype(np.float64)[:, sel]
        err = np.abs(got - ref["y"])
        assert np.all(np.isfinite(got))
        assert np.all(err <= ref["tol"]), f"max err/tol {np.max(err / ref['tol'])}"
    return float(np.max(np.abs(y.float().cpu().numpy().astype(np.float64)[:, sel] - ref["y"]) / ref["tol"]))


SMALL = [
    # N, K, B, M
    (1, 64, 64, 1), (8, 64, 1, 1), (16, 128, 128, 1), (17, 192, 64, 3), (100, 320, 64, 2), (129, 512, 512, 1),
    (127, 1024, 128, 16), (300, 2048, 2048, 1), (256, 4096, 4096, 4), (130, 11008, 128, 1), (64, 28672, 128, 1),
    (40, 14336, 128, 16), (33, 8192, 8192, 8), (2048, 2048, 2048, 1), (513, 1088, 64, 5), (1000, 2560, 128, 7),
    # 9 to 16 tokens in one launch (two column tiles) where they fit, in two launches where they do not
    (2500, 4096, 4096, 9), (5000, 2048, 128, 13), (300, 6144, 128, 13), (70, 5120, 64, 16), (70, 5184, 64, 16),
    (37965, 512, 128, 16), (2369, 1024, 1024, 12),
    # several tokens and a long K: one launch goes through K in parts (the last one shorter, or ending inside a chunk)
    (64, 28672, 128, 8), (1000, 20480, 128, 7), (2400, 16448, 64, 8), (33, 65536, 128, 5), (300, 32768, 8192, 16),
]


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("N,K,B,M", SMALL)
def test_gemv_small_and_ragged(N, K, B, M, variant):
    _check_gemv(N, K, B, M, "rotated_laplace" if K >= 512 else "uniform", variant, seed=N + K + M)


def test_gemv_degenerate_inputs():
    N, K, M = 70, 1024, 2
    lut = synth.make_lut(N, 5, DEV)
    lut[3] = 0.25  # equal levels in a row are legal
    codes = synth.make_codes_uniform(N, K, 5, DEV)
    codes[0] = 3
    codes[1] = 0
    words = rcp.rcp_pack_weights(codes)
    x = synth.make_activations(M, K, 5, DEV)
    x[1] = 0  # all-zero token -> scale 0, y = 0
    xq, scale = rcp.rcp_quantize_act(x, 128, 1.0)
    for variant in VARIANTS:
        ws = rcp.make_workspace(M, N, K, DEV)
        y = rcp.rcp_gemv_w2a4(words, lut, xq, scale, workspace=ws, variant=variant)
        ref = oracle.gemv_w2a4(oracle.pack_weights(codes.cpu().numpy()), f16_bits(lut), xq.cpu().numpy(), f16_bits(scale))
        got = y.float().cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got - ref["y"]) <= ref["tol"])
        assert np.all(got[1] == 0)


def test_bounded_wait_gives_up_reports_and_leaves_the_context_usable():
    """Failure report of the streaming kernels, without a fault or a hang: a thread waits with their bounded
    wait (a short limit) on a barrier nobody arrives at, gives up, writes its code into the workspace and
    returns. A GEMV on the same context afterwards works; a call without a workspace is refused."""
    import ctypes as C
    L = rcp.lib()
    ws = torch.zeros(4, dtype=torch.int32, device=DEV)
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    assert L.rcp_selftest_wait_timeout(C.c_void_p(ws.data_ptr()), 3000, stream) == 0
    torch.cuda.synchronize()
    assert ws.cpu().tolist() == [3, 0, 0, 0]
    ws.zero_()
    _check_gemv(300, 2048, 128, 2, "uniform", "mma_only", seed=5)
    z = torch.zeros(4096, dtype=torch.int32, device=DEV)
    p = z.data_ptr()
    assert L.rcp_gemv_w2a4(p, p, p, p, 1, 16, 64, p, None, None, None) == -5
    assert L.rcp_gemv_w2a4_variant(1, p, p, p, p, 1, 16, 64, p, None, None, None) == 0   # the plain kernel has no waits
    torch.cuda.synchronize()


def test_gemv_argument_errors():
    L = rcp.lib()
    z = torch.zeros(4096, dtype=torch.int32, device=DEV)
    p = z.data_ptr()
    assert L.rcp_gemv_w2a4(None, p, p, p, 1, 16, 64, p, p, None, None) == -1
    assert L.rcp_gemv_w2a4(p, p, p, p, 0, 16, 64, p, p, None, None) == -2
    assert L.rcp_gemv_w2a4(p, p, p, p, 17, 16, 64, p, p, None, None) == -2
    assert L.rcp_gemv_w2a4(p, p, p, p, 1, 16, 96, p, p, None, None) == -2
    assert L.rcp_gemv_w2a4(p + 4, p, p, p, 1, 16, 64, p, p, None, None) == -3
    assert L.rcp_gemv_w2a4_variant(99, p, p, p, p, 1, 16, 64, p, p, None, None) == -7


def _full_cases():
    seen, out = set(), []
    for ci, cfg in enumerate(CONFIGS):
        for layer in cfg.layers:
            for M in cfg.Ms:
                key = (layer.N, layer.K, layer.had_block, M, cfg.codes)
                if key in seen:
                    continue
                seen.add(key)
                out.append(pytest.param(ci, layer.N, layer.K, layer.had_block, M, cfg.codes,
                                        id=f"{cfg.key}-{layer.name}-M{M}"))
    return out


@pytest.mark.parametrize("ci,N,K,B,M,kind", _full_cases())
def test_gemv_full_size_configs_sampled_rows(ci, N, K, B, M, kind):
    """All five configurations at full size, in the launch configuration the benchmark times
    (variant auto); the oracle checks the first and last rows plus a random sample."""
    rng = np.random.default_rng(N + K + M)
    nsamp = min(N, 192)
    rows = np.unique(np.concatenate([np.arange(min(N, 32)), np.arange(max(0, N - 32), N),
                                     rng.integers(0, N, size=nsamp)]))
    _check_gemv(N, K, B, M, kind, "auto", seed=1000 + ci, rows=rows)
