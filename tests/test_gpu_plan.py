"""The reusable tiling plan (bmu_plan_create / bmu_search_planned): the plan is made once for
a frozen corpus and every search that uses it returns exactly what bmu_search_ws returns."""
import pytest
import torch

from inputs import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bmu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_05138_b200 as lib
    lib.load()
    return lib


@pytest.mark.parametrize("kernel", [0, 1, 3, 4, 6])
def test_planned_search_equals_one_shot_search_and_is_reusable(bmu, kernel):
    cfg = synth.CONFIGS["cfg1"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=2300)
    rp, ci = rowptr.cuda(), colidx.cuda()
    o = bmu.Opts()
    o.kernel = kernel
    plan = bmu.Plan(rp, ci, cfg.D, 1024 + 40, o)
    for seed in (3, 4):                                   # two "epochs": two codebooks, one plan
        W = synth.make_codebook(cfg.D, 1024 + 40, seed, kind="scaled").cuda()
        a = plan.search(W)
        b = bmu.bmu_search_ws(W, rp, ci, opts=o)
        torch.cuda.synchronize()
        assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    nrm = bmu.bmu_codebook_norms(W)
    c = plan.search(W, norms=nrm)
    assert torch.equal(c[0], b[0]) and torch.equal(c[1], b[1])
    plan.close()


def test_planned_search_argument_checks(bmu):
    cfg = synth.CONFIGS["cfg1"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=50)
    plan = bmu.Plan(rowptr.cuda(), colidx.cuda(), cfg.D, 256)
    with pytest.raises(ValueError):
        plan.search(torch.zeros(cfg.D, 128, device="cuda"))
    W = torch.zeros(cfg.D * 256 + 1, device="cuda")[1:].view(cfg.D, 256)      # 4-byte aligned only
    with pytest.raises(bmu.BmuError) as e:
        plan.search(W)
    assert e.value.status == 2
    assert bmu.load().bmu_search_planned(None, None, None, None, None, None) == 1


def test_search_with_workspace_can_be_captured_in_a_cuda_graph(bmu):
    """bmu_search_ws allocates nothing and only enqueues work, so a caller can capture it once
    and replay it; the replay gives the bits of the eager call."""
    lib = bmu
    cfg = synth.CONFIGS["cfg1"]
    dev = torch.device("cuda")
    rowptr, colidx = synth.make_corpus(cfg, n_docs=3000, device=dev)
    W = synth.make_codebook(cfg.D, cfg.M, 3, device=dev)
    N = rowptr.numel() - 1
    norms = lib.bmu_codebook_norms(W)
    need = lib.bmu_search_workspace_bytes(cfg.D, cfg.M, N, colidx.numel())
    ws = torch.empty(need + 256, dtype=torch.uint8, device=dev)
    ob = torch.empty(N, dtype=torch.int32, device=dev)
    od = torch.empty(N, dtype=torch.float32, device=dev)

    def call():
        lib.bmu_search_ws(W, rowptr, colidx, norms=norms, workspace=ws, out_bmu=ob, out_dist=od)

    call()
    torch.cuda.synchronize()
    ref_b, ref_d = ob.clone(), od.clone()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):                      # first call on another stream, uncaptured
        call()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        call()
    for _ in range(3):
        ob.zero_()
        od.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(ob, ref_b) and torch.equal(od, ref_d)


@pytest.mark.parametrize("kernel", [0, 3, 6])
def test_calls_on_two_streams_with_their_own_workspaces_do_not_interfere(bmu, kernel):
    """The library keeps no device-side state outside the caller's workspace (the one-shot and
    the static entry points aside): two searches in flight at once give what they give alone."""
    cfg = synth.CONFIGS["cfg3"]
    dev = torch.device("cuda")
    jobs = []
    for k, (n_docs, M) in enumerate(((6000, 2048), (4000, 1536))):
        rowptr, colidx = synth.make_corpus(cfg, batch=k, n_docs=n_docs, device=dev)
        W = synth.make_codebook(cfg.D, M, 70 + k, kind="scaled", device=dev)
        o = bmu.Opts()
        o.kernel = kernel
        alone = bmu.bmu_search_ws(W, rowptr, colidx, opts=o)
        N = rowptr.numel() - 1
        need = bmu.bmu_search_workspace_bytes(cfg.D, M, N, colidx.numel(), o)
        jobs.append(dict(W=W, rp=rowptr, ci=colidx, o=o, alone=alone, s=torch.cuda.Stream(),
                         ws=torch.empty(need + 256, dtype=torch.uint8, device=dev),
                         ob=torch.empty(N, dtype=torch.int32, device=dev),
                         od=torch.empty(N, dtype=torch.float32, device=dev)))
    torch.cuda.synchronize()
    for rep in range(3):
        for j in jobs:
            with torch.cuda.stream(j["s"]):
                bmu.bmu_search_ws(j["W"], j["rp"], j["ci"], opts=j["o"], workspace=j["ws"],
                                  out_bmu=j["ob"], out_dist=j["od"])
    torch.cuda.synchronize()
    for j in jobs:
        assert torch.equal(j["ob"], j["alone"][0]) and torch.equal(j["od"], j["alone"][1])


def test_launch_counter_agrees_with_describe_search(bmu):
    """The library counts its own kernel launches; between two chunk sizes the count differs by
    exactly the sweep launches (and compact copies) bmu_describe_search announces."""
    cfg = synth.CONFIGS["cfg2"]
    dev = torch.device("cuda")
    rowptr, colidx = synth.make_corpus(cfg, n_docs=600, device=dev)
    W = synth.make_codebook(cfg.D, 4096, 2, device=dev)
    N, nnz = rowptr.numel() - 1, colidx.numel()
    counts, descs = [], []
    for chunk in (512, 2048):
        o = bmu.Opts()
        o.kernel, o.chunk_neurons = 6, chunk
        d = bmu.bmu_describe_search(cfg.D, 4096, N, nnz, o)
        n0 = bmu.bmu_kernel_launches()
        bmu.bmu_search_ws(W, rowptr, colidx, opts=o)
        counts.append(bmu.bmu_kernel_launches() - n0)
        descs.append(d)
    torch.cuda.synchronize()
    per = [d.sweep_launches * (1 + d.repack) for d in descs]
    assert [d.sweep_launches for d in descs] == [8, 2]
    assert counts[0] - counts[1] == per[0] - per[1] and counts[1] > per[1]


@pytest.mark.parametrize("kernel,cluster", [(3, 1), (6, 1), (6, 0), (6, 3), (6, 4), (4, 3), (3, 2)])
def test_planned_order_is_a_length_ordered_permutation(bmu, kernel, cluster):
    """bmu_plan_order: every document appears once; unless the corpus order is kept, the lists
    the sweep walks (behind the dense head for the tensor-core sweep) never get longer along
    the planned order -- with or without ordering by content among equally long documents."""
    cfg = synth.CONFIGS["cfg3"]
    dev = torch.device("cuda")
    rowptr, colidx = synth.make_topical_corpus(cfg, n_docs=5000, device=dev, n_topics=64)
    o = bmu.Opts()
    o.kernel, o.cluster, o.relabel = kernel, cluster, 2
    plan = bmu.Plan(rowptr, colidx, cfg.D, 1024, o)
    order = plan.order().to(torch.int64)
    plan.close()
    N = rowptr.numel() - 1
    assert torch.equal(torch.sort(order).values, torch.arange(N, device=dev))
    if cluster == 2:
        assert torch.equal(order, torch.arange(N, device=dev))
        return
    lens = (rowptr[1:] - rowptr[:-1]).to(torch.int64)
    if kernel == 6:                                   # ids below the head (640) are not gathered
        doc = torch.repeat_interleave(torch.arange(N, device=dev), lens)
        lens = torch.zeros(N, dtype=torch.int64, device=dev).index_add_(0, doc, (colidx >= 640).to(torch.int64))
    walked = lens[order]
    assert bool((walked[1:] <= walked[:-1]).all())
    if cluster in (0, 3) and kernel == 6:
        # among equally long documents: ordered by the rarest feature (ids are frequency ranks)
        last = colidx[(rowptr[1:] - 1).to(torch.int64)].to(torch.int64)[order]
        same = walked[1:] == walked[:-1]
        assert bool((last[1:][same] >= last[:-1][same]).all())
