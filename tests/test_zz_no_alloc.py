"""rcp_gemv_w2a4_static: the LUT GEMV for callers that are not allowed to allocate device memory
(a plug-in in a process whose memory belongs to a pool, a decode loop that cannot take the
synchronization an allocation brings). Its scratch is an array inside the library instead of a
caller buffer, so the checks here are the ones that matter to such a caller: called through the C
ABI with nothing but inputs and outputs, it must give what rcp_gemv_w2a4 gives, also the second
time, when the shared array still holds whatever the first call left behind; and bad arguments must
come back as status codes with nothing put on the stream. A bounded wait that gives up is reported through
the array's status word, which such a caller reads with rcp_gemv_w2a4_static_status; the next call clears it.

This file sorts after the other test files on purpose: a run that stops at the first failure has
then already run everything else."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
import paper_2502_15779_b200 as rcp
from gen import synth
from helpers import f16_bits

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _inputs(N, K, B, M, seed):
    codes, lut = synth.make_layer(N, K, B, "rotated_laplace", seed, device=DEV)
    x = synth.make_activations(M, K, seed, device=DEV)
    words = rcp.rcp_pack_weights(codes)
    xq, scale = rcp.rcp_quantize_act(x, B, 1.0)
    return words, lut, xq, scale


@pytest.mark.parametrize("N,K,B,M", [(300, 2048, 2048, 1), (1000, 2560, 128, 3), (4096, 4096, 4096, 2)])
def test_static_scratch_entry_matches_existing_entry_twice_in_a_row(N, K, B, M):
    words, lut, xq, scale = _inputs(N, K, B, M, seed=N + K + M)
    # the existing entry point, with a caller-provided scratch buffer
    ws = rcp.make_workspace(M, N, K, DEV)
    y_ref = rcp.rcp_gemv_w2a4(words, lut, xq, scale, workspace=ws)
    # tolerance of the GEMV parity tests: |y - y_ref| <= 2e-3 * (s * sum_c |LUT[c]| |S_c|) + 1e-5, from the oracle
    orc = oracle.gemv_w2a4(words.cpu().numpy().view(np.uint32), f16_bits(lut), xq.cpu().numpy(), f16_bits(scale))
    tol = orc["tol"]
    # the new entry point, straight through the C ABI: inputs and outputs only, on the current stream
    L = rcp.lib()
    y = torch.empty(M, N, dtype=torch.float16, device=DEV)
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    args = (C.c_void_p(words.data_ptr()), C.c_void_p(lut.data_ptr()), C.c_void_p(xq.data_ptr()),
            C.c_void_p(scale.data_ptr()), M, N, K, C.c_void_p(y.data_ptr()), stream)
    want = y_ref.float().cpu().numpy().astype(np.float64)
    for call in range(2):  # the second call meets the array as the first one left it
        y.fill_(float("nan"))
        assert L.rcp_gemv_w2a4_static(*args) == 0
        torch.cuda.synchronize()
        got = y.float().cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(got)), f"call {call}"
        assert np.all(np.abs(got - want) <= tol), f"call {call}: max diff/tol {np.max(np.abs(got - want) / tol)}"
        assert np.all(np.abs(got - orc["y"]) <= tol), f"call {call}"


def test_static_scratch_entry_reports_errors_and_wrapper_agrees():
    z = torch.zeros(64, dtype=torch.int32, device=DEV)
    p = C.c_void_p(z.data_ptr())
    L = rcp.lib()
    # every shape the GEMV accepts needs less scratch than the array holds; the size check comes first
    for (M, N, K) in [(1, 57344, 8192), (16, 600000, 64), (8, 8192, 28672)]:
        assert 0 < rcp.rcp_gemv_workspace_bytes(M, N, K) <= rcp.binding.STATIC_SCRATCH_BYTES
    assert L.rcp_status_str(-8) not in (None, b"")       # the text of RCP_ERR_LIMIT
    # bad arguments are reported like the existing entry point reports them, before anything reaches the stream
    assert L.rcp_gemv_w2a4_static(p, p, p, p, 1, 16, 96, p, None) == -2
    assert L.rcp_gemv_w2a4_static(None, p, p, p, 1, 16, 64, p, None) == -1
    assert L.rcp_gemv_w2a4_static(C.c_void_p(z.data_ptr() + 4), p, p, p, 1, 16, 64, p, None) == -3
    # the Python wrapper gives the same bits as the existing entry point
    words, lut, xq, scale = _inputs(64, 256, 128, 1, seed=3)
    y = rcp.rcp_gemv_w2a4_static(words, lut, xq, scale)
    ws = rcp.make_workspace(1, 64, 256, DEV)
    assert torch.equal(y.view(torch.int16), rcp.rcp_gemv_w2a4(words, lut, xq, scale, workspace=ws).view(torch.int16))


def test_static_scratch_status_word_reports_a_wait_that_gave_up_and_the_next_call_clears_it():
    """The built-in array is dirtied the way a real failure would dirty it: a kernel whose bounded wait runs out
    (nobody arrives at its barrier) writes its code into the status word. The caller sees it through the status
    accessor; the next rcp_gemv_w2a4_static call clears the word before its kernel and gives the right answer."""
    L = rcp.lib()
    st = C.c_int32(-1)
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    assert L.rcp_selftest_wait_timeout(None, 2000, stream) == 0
    assert L.rcp_gemv_w2a4_static_status(C.byref(st), stream) == 0
    assert st.value == 3, "the wait must have given up and said so"
    words, lut, xq, scale = _inputs(300, 1024, 128, 2, seed=11)
    y = rcp.rcp_gemv_w2a4_static(words, lut, xq, scale)
    ws = rcp.make_workspace(2, 300, 1024, DEV)
    assert torch.equal(y.view(torch.int16), rcp.rcp_gemv_w2a4(words, lut, xq, scale, workspace=ws).view(torch.int16))
    assert L.rcp_gemv_w2a4_static_status(C.byref(st), stream) == 0
    assert st.value == 0
    assert L.rcp_selftest_wait_timeout(None, 0, stream) == -2
