"""The guarded build of the library (-DRCP_CHECKED) stands in for a memory checker: every shared-memory address
the streaming kernel forms and every TMA request is checked against the layout the host planned, and a violation
is reported through the status word instead of faulting. The shape lists below (small and ragged shapes, every
phase form, K in parts, two column tiles, the quantizer inside, group-wise grid, weight-only form, the longest K
and very many rows) must run through it with no guard firing and give the production build's bits."""
import os
import subprocess
import sys

import numpy as np
import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

# N, K, B, M, variant, grouped
CASES = [
    (1, 64, 64, 1, "dp4a", False), (17, 192, 64, 3, "mma", False), (129, 512, 512, 1, "mma_only", False),
    (127, 1024, 128, 16, "mma_only", False), (300, 2048, 2048, 1, "dp4a", False), (2368, 1024, 128, 2, "dp4a", False),
    (2500, 4096, 4096, 9, "mma_only", False), (37965, 512, 128, 16, "mma_only", False), (2369, 1024, 1024, 12, "mma_only", False),
    (64, 28672, 128, 8, "mma_only", False), (2400, 16448, 64, 8, "mma_only", False), (33, 65536, 128, 5, "mma_only", False),
    (300, 32768, 8192, 16, "mma_only", False), (5000, 8192, 8192, 1, "linear", False), (4097, 4096, 4096, 1, "linear", True),
    (130, 11008, 128, 1, "linear", False), (1000, 2560, 128, 7, "mma_only", True), (4800, 1024, 128, 2, "dp4a", True),
    (64, 28672, 128, 1, "dp4a", True), (300, 2048, 128, 1, "w2a16", False), (2369, 5120, 128, 4, "w2a16", False),
    (40, 65536, 128, 2, "w2a16", False), (300000, 64, 64, 1, "dp4a", False), (150000, 128, 128, 3, "mma_only", True),
    (10240, 8192, 8192, 1, "dp4a", False), (8192, 8192, 8192, 8, "mma_only", False),
    (300, 28672, 128, 8, "mma_only", True), (2400, 16512, 128, 6, "mma_only", True),   # group-wise grid, activations streamed
]


def test_guarded_build_runs_the_shape_lists_without_a_guard_firing(tmp_path):
    from paper_2502_15779_b200 import build
    checked = build.build_checked()
    sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
    import checked_build_driver
    want = checked_build_driver.run(CASES)          # production build, this process
    out = str(tmp_path / "checked.npz")
    env = dict(os.environ, RCP_W2A4_LIB=checked, PYTHONPATH=os.pathsep.join([ROOT, os.path.join(ROOT, "tests")]))
    subprocess.run([sys.executable, os.path.join(ROOT, "tests", "checked_build_driver.py"), out], check=True, env=env,
                   cwd=ROOT, timeout=900)
    got = np.load(out)
    for i in range(len(CASES)):
        assert int(got[f"status{i}"][0]) == 0, f"case {CASES[i]}: guard {int(got[f'status{i}'][0]) - 16} fired"
        assert int(want[f"status{i}"][0]) == 0
        assert np.array_equal(got[f"y{i}"], want[f"y{i}"]), f"case {CASES[i]}"
