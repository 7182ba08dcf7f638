"""bmu_search_static: the search for callers that cannot allocate.

Some users of the library sit where cudaMalloc is off limits -- inside a memory
pool that already owns the device, in a loop that must not allocate after
start-up, in a plug-in that only receives its inputs and outputs.  For them the
library carries its scratch in a fixed 8 MiB array of its own image.  The test
calls that entry point through the C ABI twice in a row, with different inputs,
and checks both results against the ordinary entry point (bmu_search_ws, same
kernel, caller-owned workspace) and against the fp64 oracle under the rule of
every other parity test: the second call finds the first call's leftovers in the
shared array and must not be disturbed by them.  Sizes beyond
the array are refused with a message that names them.

Collected last on purpose (file name), so that a failure here cannot hide the
result of any other test in a run that stops at the first failure.
"""
import pytest
import torch

from inputs import synth
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bmu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_05138_b200 as lib
    lib.load()
    return lib


def reference(bmu, W, rp, ci):
    o = bmu.Opts()
    o.kernel = 1
    return bmu.bmu_search_ws(W, rp, ci, opts=o)


def test_two_calls_in_a_row_match_the_workspace_entry_point(bmu):
    dev = torch.device("cuda")
    cfg = synth.CONFIGS["cfg1"]
    cases = [(cfg.M, 6000, 31), (1000, 2500, 32)]        # second call: other sizes, ragged M
    for M, n_docs, seed in cases:
        W = synth.make_codebook(cfg.D, M, seed, device=dev, kind="scaled")
        rp, ci = synth.make_corpus(cfg, n_docs=n_docs, device=dev, seed=seed)
        N = rp.numel() - 1
        ob = torch.full((N,), -7, dtype=torch.int32, device=dev)
        od = torch.full((N,), float("nan"), dtype=torch.float32, device=dev)
        bmu.bmu_search_static(W, rp, ci, ob, od)
        rb, rd = reference(bmu, W, rp, ci)
        torch.cuda.synchronize()
        assert torch.equal(ob, rb)
        # same kernel, same order of additions: the tolerance of the parity tests is ample
        assert bool(((od - rd).abs() <= 1e-5 * rd.abs()).all())
        # and the entry point's own output against the oracle (indices equal except inside a
        # 1e-5 near-tie, distances within 1e-5 relative)
        res = parity.compare(ob.cpu().numpy(), od.cpu().numpy(), W.cpu().numpy(),
                             rp.cpu().numpy(), ci.cpu().numpy())
        assert res["docs"] == N and res["failed"] == 0


def test_sizes_beyond_the_built_in_array_are_refused(bmu):
    dev = torch.device("cuda")
    W = torch.zeros(8, 64, device=dev)
    N = 1_100_000                                          # 8 * N alone exceeds 8 MiB
    rp = torch.zeros(N + 1, dtype=torch.int32, device=dev)
    ci = torch.zeros(0, dtype=torch.int32, device=dev)
    ob = torch.empty(N, dtype=torch.int32, device=dev)
    od = torch.empty(N, dtype=torch.float32, device=dev)
    with pytest.raises(bmu.BmuError, match="built-in array") as e:
        bmu.bmu_search_static(W, rp, ci, ob, od)
    assert e.value.status == 2
