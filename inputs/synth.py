"""Seeded synthetic inputs for the BMU search: corpora and codebooks.

This module only *draws inputs*.  It contains none of the method's arithmetic
(no distances, no norms, no argmin) and imports neither the CPU oracle nor the
CUDA library, so both can be fed the very same arrays.

The corpora stand in for the paper's MEDLINE-derived collection of sparse
binary term vectors (Section 1, Section 3), which is not available here.  The
shapes follow the five benchmark configurations:

  cfg1  32x32   map  M=1024    D=4096   N=10,000      nnz ~ max(1,Poisson(64))  Zipf s=1.0
  cfg2  64x64   map  M=4096    D=16384  N=1,000,000   nnz ~ max(1,Poisson(80))  Zipf s=1.0
  cfg3  128x128 map  M=16384   D=16384  N=4,000,000   nnz ~ max(1,Poisson(80))  Zipf s=1.1
  cfg4  512x512 map  M=262144  D=16384  N=2,000,000   nnz ~ max(1,Poisson(80))  Zipf s=1.1
  cfg5  128x128 map  M=16384   D=16384  N=26,900,000  nnz ~ lognormal(median 70, sigma .5)
        clipped to [1,400], Zipf s=1.1, streamed as 1M-document batches

Recipe for one document with target size n: draw feature ids independently from
p_k proportional to (k+1)^-s (k = 0..D-1, feature id = frequency rank), keep the
first occurrence of every id in draw order, and take the first n distinct ids.
That is sampling without replacement with probabilities proportional to p
("successive sampling").  Ids are stored ascending inside a row; indices are
int32; every batch is its own CSR with rowptr[0] == 0.

Everything runs through torch so the same code serves a CPU test (device="cpu")
and a full-size run generated directly in HBM (device="cuda").  The two devices
use different random streams: reproducibility is per (seed, device type).
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch

__all__ = [
    "Config", "CONFIGS", "zipf_cdf", "draw_nnz", "draw_corpus", "make_corpus",
    "make_codebook", "codebook_seed", "corpus_seed", "num_batches", "batch_size",
    "make_topical_corpus",
]


@dataclass(frozen=True)
class Config:
    name: str
    edge: int            # map edge; M = edge * edge neurons
    D: int               # number of features
    N: int               # number of documents
    nnz_kind: str        # "poisson" | "lognormal"
    nnz_param: float     # Poisson mean, or lognormal median
    zipf_s: float
    index: int           # 1-based position in the benchmark list (seeds)
    batch: int = 0       # 0 = one batch; else documents per streamed batch

    @property
    def M(self) -> int:
        return self.edge * self.edge


CONFIGS = {
    "cfg1": Config("cfg1", 32, 4096, 10_000, "poisson", 64.0, 1.0, 1),
    "cfg2": Config("cfg2", 64, 16384, 1_000_000, "poisson", 80.0, 1.0, 2),
    "cfg3": Config("cfg3", 128, 16384, 4_000_000, "poisson", 80.0, 1.1, 3),
    "cfg4": Config("cfg4", 512, 16384, 2_000_000, "poisson", 80.0, 1.1, 4),
    "cfg5": Config("cfg5", 128, 16384, 26_900_000, "lognormal", 70.0, 1.1, 5,
                   batch=1_000_000),
}

LOGNORMAL_SIGMA = 0.5
LOGNORMAL_CLIP = (1, 400)


def codebook_seed(cfg: Config) -> int:
    return 0xC0DE0000 + cfg.index


def corpus_seed(cfg: Config, batch: int = 0) -> int:
    return 0xD0C50000 + cfg.index * 64 + batch


def batch_size(cfg: Config) -> int:
    return cfg.batch if cfg.batch else cfg.N


def num_batches(cfg: Config) -> int:
    b = batch_size(cfg)
    return (cfg.N + b - 1) // b


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def zipf_cdf(D: int, s: float, device="cpu") -> torch.Tensor:
    """Cumulative distribution of p_k ~ (k+1)^-s over k = 0..D-1 (float64)."""
    k = torch.arange(1, D + 1, dtype=torch.float64, device=device)
    p = k.pow(-float(s))
    cdf = torch.cumsum(p, 0)
    return cdf / cdf[-1]


def draw_nnz(kind: str, param: float, N: int, gen: torch.Generator, device) -> torch.Tensor:
    """Target number of active features per document (int64, >= 1)."""
    if kind == "poisson":
        lam = torch.full((N,), float(param), dtype=torch.float32, device=device)
        n = torch.poisson(lam, generator=gen).to(torch.int64)
        return n.clamp_(min=1)
    if kind == "lognormal":
        z = torch.randn(N, generator=gen, device=device, dtype=torch.float32)
        n = torch.round(torch.exp(math.log(param) + LOGNORMAL_SIGMA * z)).to(torch.int64)
        return n.clamp_(LOGNORMAL_CLIP[0], LOGNORMAL_CLIP[1])
    if kind == "const":
        return torch.full((N,), int(param), dtype=torch.int64, device=device)
    raise ValueError(kind)


def _first_distinct(ids: torch.Tensor, want: torch.Tensor):
    """ids [B,K] iid draws; keep, per row, the first `want` distinct values in
    draw order.  Returns (flat ascending-per-row ids, counts per row)."""
    B, K = ids.shape
    pos = torch.arange(K, device=ids.device, dtype=torch.int64)
    key, _ = torch.sort(ids * K + pos, dim=1)            # by (id, draw position)
    sid = key // K
    spos = key - sid * K
    first = torch.ones_like(sid, dtype=torch.bool)
    first[:, 1:] = sid[:, 1:] != sid[:, :-1]            # first draw of each id
    mark = torch.zeros_like(first)
    mark.scatter_(1, spos, first)                        # back to draw order
    rank = torch.cumsum(mark.to(torch.int32), dim=1)    # running distinct count
    keep = mark & (rank <= want.to(torch.int32).unsqueeze(1))
    keep_sorted = torch.gather(keep, 1, spos)
    counts = keep_sorted.sum(dim=1)
    return sid[keep_sorted], counts


def draw_corpus(N: int, D: int, s: float, nnz: torch.Tensor, seed: int, device="cpu",
                block: int = 16384):
    """Binary CSR corpus: (rowptr int32 [N+1], colidx int32 [nnz_total]).

    `nnz` holds the target row sizes (clipped to D).  Rows come out with
    exactly min(nnz_i, D) distinct ascending ids.
    """
    device = torch.device(device)
    gen = _gen(seed, device)
    cdf = zipf_cdf(D, s, device)
    want_all = nnz.to(device=device, dtype=torch.int64).clamp(max=D)
    pieces, counts_all = [], []
    for b0 in range(0, N, block):
        want = want_all[b0:b0 + block]
        B = want.numel()
        # draws per round: a generous multiple of the largest target; rows that
        # still fall short are re-drawn alone with four times as many draws
        cur_K = int(min(max(256, 4 * int(want.max().item())), 1 << 15))
        todo = torch.arange(B, device=device)
        row_chunks = []
        while todo.numel():
            u = torch.rand((todo.numel(), cur_K), generator=gen, device=device,
                           dtype=torch.float64)
            ids = torch.searchsorted(cdf, u).clamp_(max=D - 1)
            w = want[todo]
            sel, cnt = _first_distinct(ids, w)
            ok = cnt == w
            # keep rows that reached their target; re-draw the others
            okrows = torch.nonzero(ok).flatten()
            if okrows.numel():
                row_of = torch.repeat_interleave(
                    torch.arange(todo.numel(), device=device), cnt)
                take = ok[row_of]
                row_chunks.append((todo[okrows], cnt[okrows], sel[take]))
            todo = todo[~ok]
            cur_K = min(cur_K * 4, 1 << 17)
        # stitch the rounds back into row order
        cnt_b = torch.zeros(B, dtype=torch.int64, device=device)
        for r, c, _ in row_chunks:
            cnt_b[r] = c
        off_b = torch.zeros(B + 1, dtype=torch.int64, device=device)
        off_b[1:] = torch.cumsum(cnt_b, 0)
        col_b = torch.empty(int(off_b[-1].item()), dtype=torch.int32, device=device)
        for r, c, v in row_chunks:
            starts = off_b[r]
            within = torch.arange(v.numel(), device=device) - torch.repeat_interleave(
                torch.cumsum(c, 0) - c, c)
            dst = torch.repeat_interleave(starts, c) + within
            col_b[dst] = v.to(torch.int32)
        pieces.append(col_b)
        counts_all.append(cnt_b)
    counts = torch.cat(counts_all) if counts_all else torch.zeros(0, dtype=torch.int64,
                                                                  device=device)
    total = int(counts.sum().item()) if N else 0
    if total >= 2 ** 31:
        raise ValueError("batch has >= 2^31 nonzeros; split it (int32 rowptr)")
    rowptr = torch.zeros(N + 1, dtype=torch.int32, device=device)
    rowptr[1:] = torch.cumsum(counts, 0).to(torch.int32)
    colidx = torch.cat(pieces) if pieces else torch.zeros(0, dtype=torch.int32, device=device)
    return rowptr, colidx


def make_corpus(cfg: Config, batch: int = 0, device="cpu", n_docs: int | None = None,
                seed: int | None = None):
    """One CSR batch of a benchmark configuration.  `n_docs` shrinks the batch
    (same distributions, fewer documents) for tests."""
    bs = batch_size(cfg)
    lo = batch * bs
    n = min(bs, cfg.N - lo)
    if n_docs is not None:
        n = min(n, int(n_docs))
    seed = corpus_seed(cfg, batch) if seed is None else seed
    device = torch.device(device)
    g = _gen(seed ^ 0x5A5A5A5A, device)
    nnz = draw_nnz(cfg.nnz_kind, cfg.nnz_param, n, g, device)
    return draw_corpus(n, cfg.D, cfg.zipf_s, nnz, seed, device)


def make_topical_corpus(cfg: Config, device="cpu", n_docs: int | None = None,
                        seed: int | None = None, n_topics: int = 4096, topic_size: int = 96,
                        topic_share: float = 0.35, first_rare: int = 640):
    """A corpus WITH co-occurrence structure, as an extra test input beside the five
    configurations (whose ids are drawn independently, so that documents share rare features
    only by chance; a real collection has topics).  Every document belongs to one of `n_topics`
    topics; a topic owns `topic_size` rare features (ids >= first_rare, a seeded random set).
    A document takes about `topic_share` of its ids from its topic's features (a uniform sample
    without replacement) and the rest by the configuration's own Zipf recipe; ids that come up
    twice are kept once, so rows are a little shorter than the configuration's.  Same layout as
    make_corpus: (rowptr int32 [N+1], colidx int32 [nnz]), ids ascending in a row."""
    n = cfg.N if n_docs is None else min(cfg.N, int(n_docs))
    seed = corpus_seed(cfg, 50) if seed is None else seed
    device = torch.device(device)
    g = _gen(seed ^ 0x70B1C5, device)
    nnz = draw_nnz(cfg.nnz_kind, cfg.nnz_param, n, g, device)
    k_topic = (nnz.to(torch.float64) * topic_share).round().to(torch.int64).clamp(max=topic_size)
    base_rp, base_ci = draw_corpus(n, cfg.D, cfg.zipf_s, (nnz - k_topic).clamp(min=0), seed, device)
    rare = cfg.D - first_rare
    if rare < topic_size:
        raise ValueError("vocabulary too small for topics of %d rare features" % topic_size)
    # topic t owns the first `topic_size` entries of a random permutation of the rare ids
    feats = torch.rand((n_topics, rare), generator=g, device=device).argsort(dim=1)[:, :topic_size]
    feats = feats + first_rare
    topic = torch.randint(0, n_topics, (n,), generator=g, device=device)
    doc_parts, id_parts = [], []
    for b0 in range(0, n, 1 << 18):                      # bounded scratch
        b1 = min(n, b0 + (1 << 18))
        pick = torch.rand((b1 - b0, topic_size), generator=g, device=device).argsort(dim=1)
        keep = torch.arange(topic_size, device=device)[None, :] < k_topic[b0:b1, None]
        ids = feats[topic[b0:b1]].gather(1, pick)[keep]
        docs = torch.arange(b0, b1, device=device)[:, None].expand(-1, topic_size)[keep]
        doc_parts.append(docs)
        id_parts.append(ids)
    lens = (base_rp[1:] - base_rp[:-1]).to(torch.int64)
    doc_parts.append(torch.repeat_interleave(torch.arange(n, device=device), lens))
    id_parts.append(base_ci.to(torch.int64))
    key = torch.unique(torch.cat(doc_parts) * cfg.D + torch.cat(id_parts))     # sorted, no repeats
    doc = key // cfg.D
    counts = torch.zeros(n, dtype=torch.int64, device=device).index_add_(
        0, doc, torch.ones_like(doc))
    rowptr = torch.zeros(n + 1, dtype=torch.int32, device=device)
    rowptr[1:] = torch.cumsum(counts, 0).to(torch.int32)
    return rowptr, (key - doc * cfg.D).to(torch.int32)


def make_codebook(D: int, M: int, seed: int, device="cpu", kind: str = "uniform",
                  docs=None) -> torch.Tensor:
    """Feature-major fp32 codebook W[f*M + j] (Section 3), shape [D, M].

    kind:
      "uniform"   iid U[0,1)                        -- the benchmark codebooks
      "scaled"    U[0,1) / sqrt(D)                  -- the gathered sum, not the norm, decides
      "sparse"    95 % zeros, the rest U[0,1)
      "signed"    U[-1,1)
      "prototype" every neuron is the indicator of one document of `docs`
                  (rowptr, colidx) blurred with U[0,0.1) noise -- trained-like,
                  small distances, heavy cancellation
      "dupes"     uniform, then every odd neuron copies the neuron before it
      "const"     all entries equal 0.25
    """
    device = torch.device(device)
    g = _gen(seed, device)
    if kind == "const":
        return torch.full((D, M), 0.25, dtype=torch.float32, device=device)
    W = torch.empty((D, M), dtype=torch.float32, device=device)
    W.uniform_(0.0, 1.0, generator=g)
    if kind == "uniform":
        return W
    if kind == "scaled":
        return W.mul_(1.0 / math.sqrt(D))
    if kind == "signed":
        return W.mul_(2.0).sub_(1.0)
    if kind == "sparse":
        keep = torch.rand((D, M), generator=g, device=device) < 0.05
        return W.mul_(keep)
    if kind == "dupes":
        W[:, 1::2] = W[:, 0:(M // 2) * 2:2]
        return W
    if kind == "prototype":
        rowptr, colidx = docs
        N = rowptr.numel() - 1
        W.mul_(0.1)
        pick = torch.randint(0, N, (M,), generator=g, device=device)
        rp = rowptr.to(device=device, dtype=torch.int64)
        ci = colidx.to(device=device, dtype=torch.int64)
        for j in range(M):
            i = int(pick[j])
            W[ci[rp[i]:rp[i + 1]], j] = 1.0 - W[ci[rp[i]:rp[i + 1]], j]
        return W
    raise ValueError(kind)
