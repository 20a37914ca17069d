"""Host logic of the streaming GEMV: the launch plan (phases of 16-row groups over the CTAs, ring
depth, shared-memory budget, tokens per launch). No GPU needed: rcp_gemv_plan only computes."""
import ctypes as C

import pytest

from paper_2502_15779_b200 import build
from gen.configs import CONFIGS


@pytest.fixture(scope="module")
def L():
    lib = C.CDLL(build.build())
    lib.rcp_gemv_plan.restype = C.c_int
    lib.rcp_gemv_plan.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int), C.c_int]
    return lib


def plan(L, M, N, K, sms=148):
    buf = (C.c_int * 64)()
    n = L.rcp_gemv_plan(M, N, K, sms, buf, 64)
    assert n >= 6, n
    v = list(buf[:n])
    phases = [tuple(v[6 + 5 * i: 11 + 5 * i]) for i in range(v[5])]
    return dict(tokens=v[0], launches=v[1], stages=v[2], smem=v[3], nchunk=v[4], phases=phases, parts=v[6 + 5 * v[5]])


def check(L, M, N, K, sms=148):
    p = plan(L, M, N, K, sms)
    groups = (N + 15) // 16
    # every group is taken exactly once, in order
    nxt = 0
    for gpc, first, total, ncta, reps in p["phases"]:
        assert 1 <= gpc <= 16 and 1 <= ncta <= sms and reps >= 1 and total >= 1
        assert first == nxt
        per_cta_max = -(-total // ncta)
        assert per_cta_max <= gpc, (gpc, total, ncta)
        assert (16 // gpc) * gpc <= 16
        if 16 // gpc > 1:
            assert gpc <= 8          # the shared-memory reduction holds eight groups
        # shares of the CTAs tile [0, total) without gaps: the first total % ncta CTAs take one group more
        q, r = divmod(total, ncta)
        assert sum(q + (1 if b < r else 0) for b in range(ncta)) == total and q + (1 if r else 0) == per_cta_max
        nxt += total * reps
    assert nxt == groups, (nxt, groups)
    assert len(p["phases"]) <= 6
    total_chunks = -(-K // 512)
    assert 1 <= p["parts"] <= 8 and p["nchunk"] == -(-total_chunks // p["parts"])   # chunks per part of K
    assert (p["parts"] - 1) * p["nchunk"] < total_chunks                             # no empty part
    assert p["stages"] >= 2 and p["smem"] <= 232448
    assert 1 <= p["tokens"] <= 16 and p["tokens"] * p["launches"] >= M
    assert p["tokens"] == 1 or p["tokens"] * p["nchunk"] * 512 <= 128 * 1024   # expanded activations of a part fit
    if p["parts"] > 1:
        assert p["tokens"] == min(M, 8) and p["stages"] >= 3
    if p["tokens"] > 8:   # one launch with two column tiles: all the tokens, and a tighter budget
        assert p["tokens"] == M and p["launches"] == 1 and M * K <= 80 * 1024 and p["stages"] >= 3
    return p


def test_plans_of_all_benchmark_shapes(L):
    for cfg in CONFIGS:
        for layer in cfg.layers:
            for M in cfg.Ms:
                check(L, M, layer.N, layer.K)


@pytest.mark.parametrize("N", [1, 15, 16, 17, 255, 256, 257, 2367, 2368, 2369, 4096, 37887, 37888, 37889, 100000])
@pytest.mark.parametrize("K", [64, 512, 4096, 11008, 65536])
def test_plans_cover_every_group_once(L, N, K):
    for M in (1, 2, 8, 16):
        check(L, M, N, K)
    check(L, 1, N, K, sms=1)
    check(L, 1, N, K, sms=132)


def test_plan_examples(L):
    # 57344 rows = 3584 groups = one round of 148 x 16 plus 1216 left over: 8 per CTA, then 32 single groups
    p = check(L, 1, 57344, 8192)
    assert p["phases"][-1] == (16, 1216, 2368, 148, 1)
    assert p["phases"][0][0] == 8 and p["phases"][0][2] == 8 * 148
    assert sum(t * r for _, _, t, _, r in p["phases"][:-1]) == 1216
    # nine to sixteen tokens go in one launch while their expanded activations stay within 80 KB, otherwise
    # in launches of eight at most; long K cuts the tokens per launch further
    assert (check(L, 16, 4096, 4096)["tokens"], check(L, 16, 4096, 4096)["launches"]) == (16, 1)
    assert (check(L, 16, 4096, 5120)["tokens"], check(L, 16, 4096, 5120)["launches"]) == (16, 1)
    assert (check(L, 10, 4096, 8192)["tokens"], check(L, 10, 4096, 8192)["launches"]) == (10, 1)
    assert (check(L, 16, 4096, 5184)["tokens"], check(L, 16, 4096, 5184)["launches"]) == (8, 2)
    assert (check(L, 16, 4096, 11008)["tokens"], check(L, 16, 4096, 11008)["launches"]) == (8, 2)
    # long K: the launch keeps its eight tokens and goes through K in parts
    p = check(L, 8, 8192, 28672)
    assert (p["tokens"], p["launches"], p["parts"]) == (8, 1, 3)
    p = check(L, 16, 64, 65536)
    assert (p["tokens"], p["launches"], p["parts"]) == (8, 2, 6)
    assert check(L, 1, 8192, 28672)["parts"] == 1 and check(L, 2, 64, 65536)["parts"] == 1
    # so many rows per CTA that the parked sums leave no room for the ring: fewer tokens instead
    p = check(L, 8, 300000, 28672)
    assert p["parts"] == 1 and p["tokens"] == 4


def test_plan_rejects_bad_shapes(L):
    buf = (C.c_int * 8)()
    assert L.rcp_gemv_plan(0, 16, 64, 148, buf, 8) == -2
    assert L.rcp_gemv_plan(1, 16, 100, 148, buf, 8) == -2
    assert L.rcp_gemv_plan(17, 16, 64, 148, buf, 8) == -2
    assert L.rcp_gemv_plan(1, 16, 64, 148, None, 8) == -1
