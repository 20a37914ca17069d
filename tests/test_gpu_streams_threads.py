"""The library on several CUDA streams at once and from several host threads at once: every call gets the bits
it gets when it runs alone (the kernels share nothing but read-only inputs; the host side keeps per-thread
tensor-map caches and sets kernel attributes under a lock)."""
import threading

import numpy as np
import pytest
import torch

import paper_2502_15779_b200 as rcp
from gen import synth
from helpers import f16_bits

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

SHAPES = [(4096, 4096, 4096, 1), (2500, 2048, 128, 8), (6144, 4096, 128, 2), (1000, 11008, 128, 1), (8192, 2048, 2048, 16)]


def _problem(N, K, B, M, seed):
    codes, lut = synth.make_layer(N, K, B, "uniform", seed, device=DEV)
    words = rcp.rcp_pack_weights(codes)
    x = synth.make_activations(M, K, seed, device=DEV)
    return dict(words=words, lut=lut, x=x, B=B, ws=rcp.make_workspace(M, N, K, DEV),
                xq=torch.empty(M, K // 2, dtype=torch.uint8, device=DEV), scale=torch.empty(M, dtype=torch.float16, device=DEV),
                y=torch.empty(M, N, dtype=torch.float16, device=DEV))


def _run(p):
    return rcp.rcp_linear_w2a4(p["x"], p["B"], 1.0, p["words"], p["lut"], y=p["y"], xq=p["xq"], scale=p["scale"],
                               workspace=p["ws"])


def test_interleaved_streams_give_the_serial_bits():
    probs = [_problem(N, K, B, M, 100 + i) for i, (N, K, B, M) in enumerate(SHAPES)]
    want = []
    for p in probs:
        _run(p)
        torch.cuda.synchronize()
        want.append(f16_bits(p["y"]).copy())
        p["y"].zero_()
    streams = [torch.cuda.Stream() for _ in probs]
    for rep in range(20):
        for p, st in zip(probs, streams):
            with torch.cuda.stream(st):
                _run(p)
    torch.cuda.synchronize()
    for p, w in zip(probs, want):
        assert np.array_equal(f16_bits(p["y"]), w)
        assert int(p["ws"].abs().max()) == 0


def test_host_threads_with_their_own_streams():
    probs = [_problem(N, K, B, M, 200 + i) for i, (N, K, B, M) in enumerate(SHAPES)]
    want = []
    for p in probs:
        _run(p)
        torch.cuda.synchronize()
        want.append(f16_bits(p["y"]).copy())
    errors = []

    def worker(i):
        try:
            torch.cuda.set_device(0)
            st = torch.cuda.Stream()
            p = probs[i]
            with torch.cuda.stream(st):
                for rep in range(50):
                    _run(p)
                    if rep % 10 == 9:
                        st.synchronize()
                        if not np.array_equal(f16_bits(p["y"]), want[i]):
                            errors.append((i, rep))
                            return
        except Exception as e:   # noqa: BLE001
            errors.append((i, repr(e)))

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(len(probs))]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    assert not errors, errors
    for p in probs:
        assert int(p["ws"].abs().max()) == 0
