"""GPU parity of rcp_ldp_export (partitioning quantizer -> packed codes and grids) against the CPU oracle:
codes and fp16 levels bit for bit; and the exported layer through the GEMV against the oracle's GEMV."""
import numpy as np
import pytest
import torch

import oracle
import paper_2502_15779_b200 as rcp
from gen import synth
from helpers import f16_bits

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _inputs(N, K, G, seed):
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    u = torch.rand(N, K, generator=g, dtype=torch.float64) - 0.5
    w = (-0.02 * torch.sign(u) * torch.log1p(-2.0 * u.abs())).to(torch.float16)   # Laplace(0, 0.02)
    NG = K // G
    sb = torch.sigmoid(3.0 + torch.randn(N, NG, generator=g)).float()
    sg = torch.sigmoid(3.0 + torch.randn(N, NG, generator=g)).float()
    s1 = torch.sigmoid(-0.7 + 0.5 * torch.randn(N, NG, generator=g)).float()
    s2 = torch.sigmoid(0.5 * torch.randn(N, NG, generator=g)).float()
    return w, sb, sg, s1, s2


@pytest.mark.parametrize("N,K,G", [(1, 64, 16), (5, 128, 128), (33, 1024, 128), (17, 11008, 128), (64, 4096, 4096),
                                   (9, 2048, 64), (300, 512, 256), (3, 28672, 128), (2, 8192, 8192), (40, 384, 48)])
def test_ldp_export_bit_exact(N, K, G):
    w, sb, sg, s1, s2 = _inputs(N, K, G, N + K + G)
    if N > 2:
        w[1, :G] = 0.125            # a unit without range: code 0, four equal levels
        w[2, :G] = w[2, :G].abs()   # a unit whose minimum is positive
    ref = oracle.ldp_export(f16_bits(w), sb.numpy(), sg.numpy(), s1.numpy(), s2.numpy(), G)
    words, lut = rcp.rcp_ldp_export(w.to(DEV), sb.to(DEV), sg.to(DEV), s1.to(DEV), s2.to(DEV), G)
    assert np.array_equal(words.cpu().numpy().view(np.uint32), oracle.pack_weights(ref["codes"]))
    assert np.array_equal(f16_bits(lut), ref["lut"])
    assert len(np.unique(ref["codes"])) == 4


def test_ldp_export_at_the_uniform_initial_point_and_exact_thresholds():
    # weights on a grid of sixteenths over [0, 1], sigmoids 1/2: thresholds 1/4, 5/8, 7/8 are hit exactly
    G = 32
    w = (torch.arange(G, dtype=torch.float32) / 16.0).clamp(max=1.0).to(torch.float16)[None, :].repeat(2, 2).contiguous()
    half = torch.full((2, 2), 0.5, dtype=torch.float32)
    one = torch.ones(2, 2, dtype=torch.float32)
    ref = oracle.ldp_export(f16_bits(w), one.numpy(), one.numpy(), half.numpy(), half.numpy(), G)
    words, lut = rcp.rcp_ldp_export(w.to(DEV), one.to(DEV), one.to(DEV), half.to(DEV), half.to(DEV), G)
    assert np.array_equal(words.cpu().numpy().view(np.uint32), oracle.pack_weights(ref["codes"]))
    assert list(ref["codes"][0, :17]) == [0, 0, 0, 0, 1, 1, 1, 1, 1, 1, 2, 2, 2, 2, 3, 3, 3]
    assert lut[0, 0].tolist() == [0.0, 0.4375, 0.75, 1.0]


@pytest.mark.parametrize("N,K,G,M", [(200, 1024, 128, 1), (300, 4096, 128, 3), (150, 2048, 2048, 2)])
def test_exported_layer_through_the_gemv(N, K, G, M):
    w, sb, sg, s1, s2 = _inputs(N, K, G, 7 * N + M)
    words, lut = rcp.rcp_ldp_export(w.to(DEV), sb.to(DEV), sg.to(DEV), s1.to(DEV), s2.to(DEV), G)
    x = synth.make_activations(M, K, 11, device=DEV)
    B = 128
    xq, scale = rcp.rcp_quantize_act(x, B, 1.0)
    ref_q = oracle.ldp_export(f16_bits(w), sb.numpy(), sg.numpy(), s1.numpy(), s2.numpy(), G)
    qa = oracle.quantize_act(f16_bits(x), B, 1.0)
    w_ref = oracle.pack_weights(ref_q["codes"])
    if G == K:
        y = rcp.rcp_gemv_w2a4(words, lut.reshape(N, 4).contiguous(), xq, scale)
        ref = oracle.gemv_w2a4(w_ref, ref_q["lut"].reshape(N, 4), qa["xq"], qa["scale"])
    else:
        y = rcp.rcp_gemv_w2a4_grouped(words, lut, xq, scale, group=G)
        ref = oracle.gemv_w2a4_grouped(w_ref, ref_q["lut"], qa["xq"], qa["scale"], G)
    got = y.float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - ref["y"]) <= ref["tol"])
    # sanity: the 2-bit layer (untrained partition parameters) still follows the full-precision product
    full = (qa["q"].astype(np.float64) * qa["scale"].view(np.float16).astype(np.float64)[:, None]) @ w.numpy().astype(np.float64).T
    assert np.corrcoef(got.ravel(), full.ravel())[0, 1] > 0.6


@pytest.mark.parametrize("N,K,G,M", [(2500, 8192, 128, 1), (3000, 4096, 4096, 1), (700, 2048, 128, 4)])
def test_export_directly_followed_by_the_linear_call_on_one_stream(N, K, G, M):
    """The export kernel and the linear call back to back on one stream, nothing in between (the GEMV kernels
    start fetching the weights before the kernel in front of them has finished only if that kernel signals an
    early start, which the export kernel never does). Repeated, so that a stale read would show."""
    w, sb, sg, s1, s2 = _inputs(N, K, G, 3 * N + M)
    wd, sbd, sgd, s1d, s2d = (t.to(DEV) for t in (w, sb, sg, s1, s2))
    x = synth.make_activations(M, K, 13, device=DEV)
    B = K if G == K else 128
    ref_q = oracle.ldp_export(f16_bits(w), sb.numpy(), sg.numpy(), s1.numpy(), s2.numpy(), G)
    qa = oracle.quantize_act(f16_bits(x), B, 1.0)
    w_ref = oracle.pack_weights(ref_q["codes"])
    ref = (oracle.gemv_w2a4(w_ref, ref_q["lut"].reshape(N, 4), qa["xq"], qa["scale"]) if G == K
           else oracle.gemv_w2a4_grouped(w_ref, ref_q["lut"], qa["xq"], qa["scale"], G))
    words = torch.empty((N, K // 16), dtype=torch.int32, device=DEV)
    lut = torch.empty((N, K // G, 4), dtype=torch.float16, device=DEV)
    xq = torch.empty(M, K // 2, dtype=torch.uint8, device=DEV)
    scale = torch.empty(M, dtype=torch.float16, device=DEV)
    ws = rcp.make_workspace(M, N, K, DEV)
    L = rcp.lib()
    import ctypes as C
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    for rep in range(5):
        words.fill_(-1)
        lut.fill_(float("nan"))
        torch.cuda.synchronize()
        assert L.rcp_ldp_export(wd.data_ptr(), sbd.data_ptr(), sgd.data_ptr(), s1d.data_ptr(), s2d.data_ptr(), N, K, G,
                                words.data_ptr(), lut.data_ptr(), st) == 0
        y = rcp.rcp_linear_w2a4(x, B, 1.0, words, lut.reshape(N, 4) if G == K else lut, group=0 if G == K else G,
                                xq=xq, scale=scale, workspace=ws)
        torch.cuda.synchronize()
        got = y.float().cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(got)) and np.all(np.abs(got - ref["y"]) <= ref["tol"]), f"repetition {rep}"


def test_ldp_export_argument_errors():
    L = rcp.lib()
    z = torch.zeros(4096, dtype=torch.int32, device=DEV)
    p = z.data_ptr()
    f = L.rcp_ldp_export
    assert f(None, p, p, p, p, 4, 128, 128, p, p, None) == -1
    assert f(p, p, p, p, p, 0, 128, 128, p, p, None) == -2
    assert f(p, p, p, p, p, 4, 128, 48, p, p, None) == -2      # group does not divide K
    assert f(p, p, p, p, p, 4, 128, 8, p, p, None) == -2       # group below 16
    assert f(p + 2, p, p, p, p, 4, 128, 128, p, p, None) == -3
