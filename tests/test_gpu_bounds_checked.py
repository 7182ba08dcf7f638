"""The bounds-checked build of the library (-DBMU_BOUNDS_CHECK): every address a kernel derives
from a feature id, a neuron index or a scanned offset is checked before use; a violation sets
bit 128 of the status word and the access goes to element 0 of the same array instead.  It
stands in for a memory checker: the small planned, tiled, tensor-core, second-best and
half-precision cases run clean under it (status word 0, parity with the oracle), and an id
beyond the vocabulary is reported through the status word without any fault."""
import json
import os
import subprocess
import sys

import pytest
import torch

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def report():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_05138_b200 import build
    lib = build.build_checked_library()
    env = dict(os.environ, BMU_LIBRARY=lib, PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
    out = subprocess.run([sys.executable, "-m", "tests.bounds_child"], cwd=ROOT, env=env,
                         capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stderr[-3000:]
    rec = json.loads([l for l in out.stdout.splitlines() if l.startswith("{")][-1])
    assert rec["library"].endswith("libbmu_checked.so")
    return rec


def test_small_cases_run_clean_under_the_checked_build(report):
    assert len(report["clean"]) == 8
    for case in report["clean"]:
        assert case["status"] == 0 and case["failed"] == 0 and case["docs"] == 1500, case


def test_an_id_beyond_the_vocabulary_is_reported_not_performed(report):
    for case in report["flagged"]:
        assert case["status"] & 128, case
    assert report["after"] == {"status": 0, "failed": 0}
