"""Pins for the CPU oracle: it is checked against things other than itself.

The oracle evaluates d_ij = |x_i| + ||w_j||^2 - 2 sum_{f in x_i} W[f][j] with a
gather over the CSR row.  Every test below reaches the expected value by another
road: the dense definition sum_f (x_f - w_jf)^2 on densified inputs, closed
forms, a hand-worked fixture, a library matmul, or an invariance of the search
(Section 3: the exact-argmin BMU does not depend on how the codebook is held).
"""
import os

import numpy as np
import pytest

import oracle
from inputs import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng


def random_csr(r, N, D, max_nnz, allow_empty=True, sort=True):
    rows = []
    for _ in range(N):
        k = int(r.integers(0 if allow_empty else 1, min(max_nnz, D) + 1))
        ids = r.choice(D, size=k, replace=False)
        rows.append(np.sort(ids) if sort else ids)
    rowptr = np.zeros(N + 1, dtype=np.int32)
    rowptr[1:] = np.cumsum([len(x) for x in rows])
    colidx = (np.concatenate(rows) if rows else np.zeros(0)).astype(np.int32)
    return rowptr, colidx


def densify(rowptr, colidx, D):
    N = rowptr.size - 1
    X = np.zeros((N, D), dtype=np.float64)
    for i in range(N):
        X[i, colidx[rowptr[i]:rowptr[i + 1]]] = 1.0
    return X


def brute_force(X, W):
    """d[i, j] = sum_f (X[i, f] - W[f, j])^2, the dense definition, in float64."""
    W = W.astype(np.float64)
    N, M = X.shape[0], W.shape[1]
    d = np.empty((N, M))
    for i in range(N):
        for j in range(M):
            diff = X[i] - W[:, j]
            d[i, j] = np.dot(diff, diff)
    return d


def two_smallest(d):
    arg = np.argmin(d, axis=1)                       # numpy: first minimum = lowest index
    d1 = d[np.arange(d.shape[0]), arg]
    if d.shape[1] == 1:
        return arg, d1, np.full_like(d1, np.inf)
    masked = d.copy()
    masked[np.arange(d.shape[0]), arg] = np.inf
    return arg, d1, masked.min(axis=1)


# ---------------------------------------------------------------- 1. brute force
@pytest.mark.parametrize("seed,N,D,M,kind", [
    (0, 60, 17, 9, "uniform"), (1, 200, 64, 32, "uniform"), (2, 50, 33, 7, "signed"),
    (3, 80, 48, 31, "sparse"), (4, 40, 5, 1, "uniform"), (5, 30, 1, 6, "uniform"),
    (6, 64, 40, 25, "scaled"),
])
def test_matches_dense_brute_force(seed, N, D, M, kind):
    r = rng(seed)
    rowptr, colidx = random_csr(r, N, D, D)
    W = synth.make_codebook(D, M, 100 + seed, kind=kind).numpy()
    d = brute_force(densify(rowptr, colidx, D), W)
    arg, e1, e2 = two_smallest(d)
    bmu, d1, d2 = oracle.bmu(W, rowptr, colidx)
    np.testing.assert_allclose(d1, e1, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(d2, e2, rtol=1e-12, atol=1e-12)
    # index must agree wherever the brute-force minimum is not an (fp64-level) tie
    clear = (e2 - e1) > 1e-9
    assert clear.sum() > 0.8 * N
    np.testing.assert_array_equal(bmu[clear], arg[clear])
    # every (i, j) pair, not just the winners
    nrm = oracle.norms(W)
    for i in range(0, N, 7):
        for j in range(M):
            assert abs(oracle.eval_pair(W, rowptr, colidx, nrm, i, j) - d[i, j]) < 1e-11


def test_norms_match_library_and_closed_form():
    W = synth.make_codebook(257, 33, 7, kind="signed").numpy()
    np.testing.assert_allclose(oracle.norms(W), (W.astype(np.float64) ** 2).sum(axis=0),
                               rtol=1e-14)
    # not transposed: a codebook with one non-zero row gives that row squared
    Z = np.zeros((5, 3), dtype=np.float32)
    Z[2] = [1.0, 2.0, 3.0]
    np.testing.assert_array_equal(oracle.norms(Z), [1.0, 4.0, 9.0])
    C = np.full((100, 4), 0.25, dtype=np.float32)
    np.testing.assert_array_equal(oracle.norms(C), [6.25] * 4)


# ---------------------------------------------------------------- 2. hand-worked fixture
def load_fixture(path):
    W, docs, norms, D, M = [], [], None, None, None
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tag, _, rest = line.partition(" ")
        if tag == "D":
            D = int(rest)
        elif tag == "M":
            M = int(rest)
        elif tag == "W":
            W.append([float(v) for v in rest.split()])
        elif tag == "NORMS":
            norms = [float(v) for v in rest.split()]
        elif tag == "DOC":
            ids, dists, res = [p.split() for p in rest.split("|")]
            docs.append(([int(v) for v in ids], [float(v) for v in dists],
                         int(res[0]), float(res[1]), float(res[2])))
    W = np.array(W, dtype=np.float32)
    assert W.shape == (D, M)
    return W, norms, docs


def test_hand_worked_fixture():
    W, norms, docs = load_fixture(os.path.join(GOLDEN, "handworked_bmu.txt"))
    rowptr = np.zeros(len(docs) + 1, dtype=np.int32)
    rowptr[1:] = np.cumsum([len(d[0]) for d in docs])
    colidx = np.array([f for d in docs for f in d[0]], dtype=np.int32)
    nrm = oracle.norms(W)
    np.testing.assert_array_equal(nrm, norms)
    bmu, d1, d2 = oracle.bmu(W, rowptr, colidx)
    for i, (_, dists, eb, e1, e2) in enumerate(docs):
        assert (bmu[i], d1[i], d2[i]) == (eb, e1, e2)
        for j, e in enumerate(dists):
            assert oracle.eval_pair(W, rowptr, colidx, nrm, i, j) == e


# ---------------------------------------------------------------- 3. closed forms
def test_zero_codebook_gives_doc_size_and_lowest_index():
    r = rng(11)
    rowptr, colidx = random_csr(r, 50, 30, 30)
    W = np.zeros((30, 8), dtype=np.float32)
    bmu, d1, d2 = oracle.bmu(W, rowptr, colidx)
    nx = rowptr[1:] - rowptr[:-1]
    np.testing.assert_array_equal(bmu, 0)             # pure tie -> lowest index
    np.testing.assert_array_equal(d1, nx)
    np.testing.assert_array_equal(d2, nx)


def test_ones_codebook_gives_complement_size():
    r = rng(12)
    D = 41
    rowptr, colidx = random_csr(r, 50, D, D)
    W = np.ones((D, 5), dtype=np.float32)
    bmu, d1, _ = oracle.bmu(W, rowptr, colidx)
    np.testing.assert_array_equal(bmu, 0)
    np.testing.assert_array_equal(d1, D - (rowptr[1:] - rowptr[:-1]))


def test_one_hot_codebook_picks_smallest_active_feature():
    r = rng(13)
    D = 37
    rowptr, colidx = random_csr(r, 80, D, 12, allow_empty=False, sort=False)
    W = np.eye(D, dtype=np.float32)                  # neuron j = indicator of feature j
    bmu, d1, d2 = oracle.bmu(W, rowptr, colidx)
    for i in range(80):
        ids = colidx[rowptr[i]:rowptr[i + 1]]
        assert bmu[i] == ids.min()                    # d = |x| + 1 - 2 [j in x]
        assert d1[i] == len(ids) - 1
        assert d2[i] == (len(ids) - 1 if len(ids) > 1 else len(ids) + 1)


def test_constant_per_neuron_codebook_closed_form():
    r = rng(14)
    D, M = 53, 9
    c = np.array([0.0, 0.125, 0.25, 0.375, 0.5, 0.625, 0.75, 0.875, 1.0], dtype=np.float32)
    W = np.tile(c, (D, 1))
    rowptr, colidx = random_csr(r, 60, D, D)
    bmu, d1, _ = oracle.bmu(W, rowptr, colidx)
    nx = (rowptr[1:] - rowptr[:-1]).astype(np.float64)
    d = nx[:, None] + D * c[None, :].astype(np.float64) ** 2 - 2 * nx[:, None] * c[None, :]
    np.testing.assert_array_equal(d1, d.min(axis=1))
    np.testing.assert_array_equal(bmu, d.argmin(axis=1))   # minimiser is c nearest |x|/D


def test_neuron_equal_to_document_has_distance_zero():
    r = rng(15)
    D, N = 64, 20
    rowptr, colidx = random_csr(r, N, D, 20, allow_empty=False)
    X = densify(rowptr, colidx, D)
    W = r.random((D, N + 3)).astype(np.float32)
    W[:, 3:] = X.T                                    # neuron 3+i is document i
    bmu, d1, _ = oracle.bmu(W, rowptr, colidx)
    # identical documents would share a distance-0 neuron: the lowest one wins
    for i in range(N):
        first = min(k for k in range(N) if np.array_equal(X[k], X[i]))
        assert bmu[i] == 3 + first and d1[i] == 0.0


def test_duplicate_neurons_lower_index_wins():
    W = synth.make_codebook(40, 16, 3, kind="dupes").numpy()
    r = rng(16)
    rowptr, colidx = random_csr(r, 200, 40, 10)
    bmu, d1, d2 = oracle.bmu(W, rowptr, colidx)
    assert np.all(bmu % 2 == 0)                      # odd neurons copy the even one before
    np.testing.assert_array_equal(d1, d2)


def test_empty_document_returns_argmin_of_norms():
    W = synth.make_codebook(30, 11, 5).numpy()
    rowptr = np.array([0, 0, 2, 2], dtype=np.int32)
    colidx = np.array([4, 9], dtype=np.int32)
    bmu, d1, _ = oracle.bmu(W, rowptr, colidx)
    n = (W.astype(np.float64) ** 2).sum(axis=0)
    assert bmu[0] == bmu[2] == n.argmin() and d1[0] == d1[2] == n.min()


# ---------------------------------------------------------------- 4. library matmul
def test_matches_blas_matmul_mid_size():
    cfg = synth.CONFIGS["cfg1"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=400)
    rowptr, colidx = rowptr.numpy(), colidx.numpy()
    W = synth.make_codebook(cfg.D, 256, 21).numpy()
    X = densify(rowptr, colidx, cfg.D)
    S = X @ W.astype(np.float64)                      # library routine
    nx = X.sum(axis=1)
    d = nx[:, None] + (W.astype(np.float64) ** 2).sum(axis=0)[None, :] - 2 * S
    arg, e1, e2 = two_smallest(d)
    bmu, d1, d2 = oracle.bmu(W, rowptr, colidx)
    np.testing.assert_allclose(d1, e1, rtol=1e-12)
    np.testing.assert_allclose(d2, e2, rtol=1e-12)
    clear = (e2 - e1) > 1e-9 * e1
    np.testing.assert_array_equal(bmu[clear], arg[clear])


# ---------------------------------------------------------------- 5. invariants
@pytest.fixture(scope="module")
def small_problem():
    r = rng(31)
    D, M, N = 96, 40, 150
    rowptr, colidx = random_csr(r, N, D, 24)
    W = synth.make_codebook(D, M, 32, kind="scaled").numpy()
    return D, M, N, rowptr, colidx, W, oracle.bmu(W, rowptr, colidx)


def test_permuting_neurons_permutes_bmus(small_problem):
    D, M, N, rowptr, colidx, W, (bmu, d1, d2) = small_problem
    perm = rng(1).permutation(M)
    b2, e1, e2 = oracle.bmu(W[:, perm], rowptr, colidx)
    np.testing.assert_array_equal(perm[b2], bmu)     # no exact ties in random data
    np.testing.assert_array_equal(e1, d1)
    np.testing.assert_array_equal(e2, d2)


def test_permuting_documents_permutes_outputs(small_problem):
    D, M, N, rowptr, colidx, W, (bmu, d1, d2) = small_problem
    perm = rng(2).permutation(N)
    rows = [colidx[rowptr[i]:rowptr[i + 1]] for i in perm]
    rp = np.zeros(N + 1, dtype=np.int32)
    rp[1:] = np.cumsum([len(x) for x in rows])
    b2, e1, _ = oracle.bmu(W, rp, np.concatenate(rows).astype(np.int32))
    np.testing.assert_array_equal(b2, bmu[perm])
    np.testing.assert_array_equal(e1, d1[perm])


def test_relabelling_features_changes_nothing(small_problem):
    D, M, N, rowptr, colidx, W, (bmu, d1, _) = small_problem
    perm = rng(3).permutation(D)                     # new id of old feature f is perm[f]
    W2 = np.empty_like(W)
    W2[perm] = W
    b2, e1, _ = oracle.bmu(W2, rowptr, perm[colidx].astype(np.int32))
    np.testing.assert_array_equal(b2, bmu)
    np.testing.assert_allclose(e1, d1, rtol=1e-12)   # rows listed in another order


def test_unused_feature_rows(small_problem):
    D, M, N, rowptr, colidx, W, (bmu, d1, _) = small_problem
    # a zero row no document contains changes nothing
    b2, e1, _ = oracle.bmu(np.vstack([W, np.zeros((1, M), np.float32)]), rowptr, colidx)
    np.testing.assert_array_equal(b2, bmu)
    np.testing.assert_array_equal(e1, d1)
    # a non-zero unused row adds its square to every distance of that neuron
    extra = rng(4).random((1, M)).astype(np.float32)
    W3 = np.vstack([W, extra])
    nrm = oracle.norms(W)
    nrm3 = oracle.norms(W3)
    for i in (0, 17, 99):
        for j in (0, 5, M - 1):
            a = oracle.eval_pair(W, rowptr, colidx, nrm, i, j)
            b = oracle.eval_pair(W3, rowptr, colidx, nrm3, i, j)
            assert abs(b - a - float(extra[0, j]) ** 2) < 1e-12


def test_thread_count_does_not_change_bits(small_problem):
    D, M, N, rowptr, colidx, W, (bmu, d1, d2) = small_problem
    for t in (1, 3):
        b, e1, e2 = oracle.bmu(W, rowptr, colidx, threads=t)
        np.testing.assert_array_equal(b, bmu)
        np.testing.assert_array_equal(e1, d1)
        np.testing.assert_array_equal(e2, d2)


def test_unsorted_rows_give_same_result(small_problem):
    D, M, N, rowptr, colidx, W, (bmu, d1, _) = small_problem
    r = rng(5)
    shuffled = colidx.copy()
    for i in range(N):
        r.shuffle(shuffled[rowptr[i]:rowptr[i + 1]])
    b2, e1, _ = oracle.bmu(W, rowptr, shuffled)
    np.testing.assert_array_equal(b2, bmu)
    np.testing.assert_allclose(e1, d1, rtol=1e-12)


# ---------------------------------------------------------------- second-best unit
@pytest.mark.parametrize("seed,N,D,M", [(0, 80, 23, 11), (1, 50, 40, 2), (2, 30, 9, 1)])
def test_second_best_unit_matches_brute_force(seed, N, D, M):
    r = rng(seed)
    rowptr, colidx = random_csr(r, N, D, D)
    W = synth.make_codebook(D, M, 200 + seed, kind="signed").numpy()
    d = brute_force(densify(rowptr, colidx, D), W)
    b1, d1, b2, d2 = oracle.bmu2(W, rowptr, colidx)
    order = np.argsort(d, axis=1, kind="stable")          # ties -> lower index first
    np.testing.assert_array_equal(b1, order[:, 0])
    if M == 1:
        assert np.all(b2 == -1) and np.all(np.isinf(d2))
        return
    e2 = d[np.arange(N), order[:, 1]]
    np.testing.assert_allclose(d2, e2, rtol=1e-12, atol=1e-12)
    clear = np.ones(N, bool) if M == 2 else (d[np.arange(N), order[:, 2]] - e2) > 1e-9
    np.testing.assert_array_equal(b2[clear], order[:, 1][clear])
    assert np.all(b2 != b1)


def test_second_best_unit_ties_take_the_lower_index():
    W = synth.make_codebook(40, 16, 3, kind="dupes").numpy()   # neuron 2k+1 copies neuron 2k
    rowptr, colidx = random_csr(rng(17), 100, 40, 10)
    b1, d1, b2, d2 = oracle.bmu2(W, rowptr, colidx)
    np.testing.assert_array_equal(b2, b1 + 1)                    # the copy is the runner-up
    np.testing.assert_array_equal(d1, d2)
    Z = np.zeros((5, 4), dtype=np.float32)                       # every neuron ties
    b1, d1, b2, d2 = oracle.bmu2(Z, np.array([0, 2], np.int32), np.array([1, 3], np.int32))
    assert (b1[0], b2[0], d1[0], d2[0]) == (0, 1, 2.0, 2.0)
