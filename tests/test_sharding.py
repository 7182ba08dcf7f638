"""The N > 1 path on CPU: two gloo ranks shard the documents, each reduces its
own shard (here with the oracle standing in for a GPU), and the gathered
outputs equal the single-process result; throughput is total units over the
slowest rank's time."""
import os

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from inputs import synth
from paper_2609_05138_b200 import sharding


def test_shard_ranges_tile_the_documents():
    for n, w in [(10, 3), (7, 8), (0, 2), (1_000_000, 8), (5, 1)]:
        edges = [sharding.shard_range(n, r, w) for r in range(w)]
        assert edges[0][0] == 0 and edges[-1][1] == n
        assert all(a[1] == b[0] for a, b in zip(edges, edges[1:]))
        sizes = [hi - lo for lo, hi in edges]
        assert max(sizes) - min(sizes) <= 1


def _worker(rank, world, port, tmp):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    cfg = synth.CONFIGS["cfg1"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=301)
    W = synth.make_codebook(cfg.D, 96, 3).numpy()
    rp, ci = sharding.shard_csr(rowptr, colidx, rank, world)
    assert rp[0] == 0 and rp[-1] == ci.numel()
    b, d1, _ = oracle.bmu(W, rp.numpy(), ci.numpy(), threads=1)
    all_b = sharding.gather_outputs(torch.from_numpy(b), 301)
    all_d = sharding.gather_outputs(torch.from_numpy(d1), 301)
    # rank 1 pretends to be twice as slow: the job rate is total / slowest
    rate = sharding.job_throughput(rp.numel() - 1, 1.0 + rank)
    if rank == 0:
        np.save(os.path.join(tmp, "b.npy"), all_b.numpy())
        np.save(os.path.join(tmp, "d.npy"), all_d.numpy())
        np.save(os.path.join(tmp, "rate.npy"), np.array([rate]))
    dist.destroy_process_group()


def test_two_gloo_ranks_match_single_process(tmp_path):
    import oracle
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    cfg = synth.CONFIGS["cfg1"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=301)
    W = synth.make_codebook(cfg.D, 96, 3).numpy()
    b, d1, _ = oracle.bmu(W, rowptr.numpy(), colidx.numpy())
    np.testing.assert_array_equal(np.load(tmp_path / "b.npy"), b)
    np.testing.assert_array_equal(np.load(tmp_path / "d.npy"), d1)
    assert abs(np.load(tmp_path / "rate.npy")[0] - 301 / 2.0) < 1e-9
