"""Pins of the update-step oracle (scatter, blur, write-back; Table 4 of the paper).

The paper times these steps and prints no formula or value for them, so the
oracle is held to the mathematics of the textbook batch update it writes out:
dense brute force with the explicit neighbourhood matrix, closed forms and
invariants.  A dropped term, a transposed plane, a wrong radius, a wrong
boundary rule or a swapped operand fails at least one of these.
"""
import math

import numpy as np
import pytest

import oracle
from inputs import synth


def small_corpus(N=300, D=60, seed=3):
    r = np.random.default_rng(seed)
    rows = [np.sort(r.choice(D, size=int(r.integers(0, 12)), replace=False)) for _ in range(N)]
    rowptr = np.zeros(N + 1, dtype=np.int32)
    rowptr[1:] = np.cumsum([len(x) for x in rows])
    colidx = np.concatenate(rows).astype(np.int32)
    return rowptr, colidx, r


def dense(rowptr, colidx, D):
    X = np.zeros((rowptr.size - 1, D))
    for i in range(rowptr.size - 1):
        for f in colidx[rowptr[i]:rowptr[i + 1]]:
            X[i, f] += 1.0
    return X


def h_matrix(ex, ey, sigma):
    """The neighbourhood written out as an M x M matrix, straight from its definition."""
    M = ex * ey
    R = math.ceil(3 * sigma) if sigma > 0 else 0
    H = np.zeros((M, M))
    for j in range(M):
        for k in range(M):
            dx, dy = abs(j % ex - k % ex), abs(j // ex - k // ex)
            if dx <= R and dy <= R:
                H[j, k] = math.exp(-(dx * dx + dy * dy) / (2 * sigma * sigma)) if sigma > 0 else 1.0
    return H


# ------------------------------------------------------------------ scatter
def test_scatter_is_the_transposed_product_with_the_assignment_matrix():
    rowptr, colidx, r = small_corpus()
    D, M = 60, 12
    bmu = r.integers(0, M, size=rowptr.size - 1).astype(np.int32)
    num, cnt = oracle.scatter(rowptr, colidx, bmu, D, M)
    X = dense(rowptr, colidx, D)
    A = np.zeros((rowptr.size - 1, M))
    A[np.arange(A.shape[0]), bmu] = 1.0
    assert np.array_equal(num, (X.T @ A).astype(np.uint64))
    assert np.array_equal(cnt, A.sum(0).astype(np.uint64))


def test_scatter_invariants_and_repeated_ids():
    rowptr, colidx, r = small_corpus(N=500, D=40, seed=9)
    M = 7
    bmu = r.integers(0, M, size=500).astype(np.int32)
    num, cnt = oracle.scatter(rowptr, colidx, bmu, 40, M)
    assert int(cnt.sum()) == 500
    assert np.array_equal(num.sum(1), np.bincount(colidx, minlength=40).astype(np.uint64))
    lens = (rowptr[1:] - rowptr[:-1]).astype(np.uint64)
    assert np.array_equal(num.sum(0), np.bincount(bmu, weights=lens, minlength=M).astype(np.uint64))
    # a document that lists an id twice adds it twice (multiset rows, as in the search)
    n2, c2 = oracle.scatter(np.array([0, 3], np.int32), np.array([5, 5, 1], np.int32), [2], 8, 4)
    assert n2[5, 2] == 2 and n2[1, 2] == 1 and n2.sum() == 3 and c2[2] == 1
    # an empty document counts for its unit and adds no feature
    n3, c3 = oracle.scatter(np.array([0, 0], np.int32), np.zeros(0, np.int32), [1], 8, 4)
    assert n3.sum() == 0 and c3[1] == 1


# ------------------------------------------------------------------ blur
@pytest.mark.parametrize("ex,ey,sigma", [(7, 5, 0.8), (6, 6, 1.5), (9, 4, 0.34), (5, 8, 2.0)])
def test_blur_equals_the_explicit_neighbourhood_matrix(ex, ey, sigma):
    r = np.random.default_rng(ex * 31 + ey)
    planes = r.integers(0, 50, size=(3, ex * ey)).astype(np.float64)
    got = oracle.blur(planes, ex, ey, sigma)
    np.testing.assert_allclose(got, planes @ h_matrix(ex, ey, sigma).T, rtol=1e-13, atol=0)


def test_blur_closed_forms():
    ex, ey, sigma = 21, 17, 1.2
    R = math.ceil(3 * sigma)
    g = np.array([math.exp(-d * d / (2 * sigma * sigma)) for d in range(-R, R + 1)])
    # impulse in the interior: the response is the separable kernel itself, centred there
    p = np.zeros(ex * ey)
    y0, x0 = 8, 10
    p[y0 * ex + x0] = 3.0
    out = oracle.blur(p, ex, ey, sigma).reshape(ey, ex)
    np.testing.assert_allclose(out[y0 - R:y0 + R + 1, x0 - R:x0 + R + 1], 3.0 * np.outer(g, g), rtol=1e-13)
    assert out[y0, x0 + R + 1] == 0.0 and out[y0 - R - 1, x0] == 0.0       # truncated at R
    np.testing.assert_allclose(out.sum(), 3.0 * g.sum() ** 2, rtol=1e-13)
    # a constant plane: interior values are c * (sum g)^2, a corner sees only a quarter-plane
    c = oracle.blur(np.full(ex * ey, 2.0), ex, ey, sigma).reshape(ey, ex)
    np.testing.assert_allclose(c[R:ey - R, R:ex - R], 2.0 * g.sum() ** 2, rtol=1e-13)
    np.testing.assert_allclose(c[0, 0], 2.0 * g[R:].sum() ** 2, rtol=1e-13)    # no wrap-around
    # sigma = 0 is the identity; the radius is ceil(3 sigma): sigma = 0.34 reaches 2 cells
    q = np.arange(ex * ey, dtype=np.float64)
    assert np.array_equal(oracle.blur(q, ex, ey, 0.0), q)
    o = oracle.blur(p, ex, ey, 0.34).reshape(ey, ex)
    assert o[y0, x0 + 2] > 0.0 and o[y0, x0 + 3] == 0.0
    # rows and columns are not interchangeable: an impulse near the right edge of a wide map
    w = np.zeros(ex * ey)
    w[3 * ex + (ex - 1)] = 1.0
    ow = oracle.blur(w, ex, ey, sigma).reshape(ey, ex)
    assert ow[3, ex - 2] > 0 and ow[4, 0] == 0.0


def test_blur_is_linear_and_symmetric():
    ex, ey, sigma = 8, 6, 1.0
    r = np.random.default_rng(5)
    a, b = r.random(ex * ey), r.random(ex * ey)
    np.testing.assert_allclose(oracle.blur(2 * a + b, ex, ey, sigma),
                               2 * oracle.blur(a, ex, ey, sigma) + oracle.blur(b, ex, ey, sigma), rtol=1e-12)
    # <blur(a), b> = <a, blur(b)>: h(j, k) = h(k, j)
    np.testing.assert_allclose(oracle.blur(a, ex, ey, sigma) @ b, a @ oracle.blur(b, ex, ey, sigma), rtol=1e-12)


# ------------------------------------------------------------------ write-back and the whole update
def test_writeback_divides_where_there_is_weight_and_keeps_the_rest():
    B = np.array([[2.0, 0.0, 9.0], [1.0, 5.0, 3.0]])
    c = np.array([4.0, 0.0, 3.0])
    W = np.full((2, 3), 7.0, dtype=np.float32)
    out = oracle.writeback(B, c, W)
    assert np.array_equal(out, np.array([[0.5, 7.0, 3.0], [0.25, 7.0, 1.0]], dtype=np.float32))
    assert np.all(W == 7.0)                                   # the input is not modified


def test_update_without_neighbourhood_is_the_centroid_of_each_unit():
    rowptr, colidx, r = small_corpus(N=400, D=30, seed=11)
    ex, ey = 4, 3
    M = ex * ey
    bmu = r.integers(0, M - 1, size=400).astype(np.int32)     # the last unit wins nothing
    num, cnt = oracle.scatter(rowptr, colidx, bmu, 30, M)
    W0 = r.random((30, M)).astype(np.float32)
    W1 = oracle.writeback(oracle.blur(num, ex, ey, 0.0), oracle.blur(cnt, ex, ey, 0.0), W0)
    X = dense(rowptr, colidx, 30)
    for j in range(M - 1):
        np.testing.assert_allclose(W1[:, j], X[bmu == j].mean(0), rtol=1e-6)
    assert np.array_equal(W1[:, M - 1], W0[:, M - 1])


def test_update_with_neighbourhood_against_dense_algebra():
    rowptr, colidx, r = small_corpus(N=350, D=25, seed=13)
    ex, ey, sigma = 5, 4, 1.1
    M = ex * ey
    bmu = r.integers(0, M, size=350).astype(np.int32)
    num, cnt = oracle.scatter(rowptr, colidx, bmu, 25, M)
    W1 = oracle.writeback(oracle.blur(num, ex, ey, sigma), oracle.blur(cnt, ex, ey, sigma),
                          np.zeros((25, M), np.float32))
    X = dense(rowptr, colidx, 25)
    A = np.zeros((350, M))
    A[np.arange(350), bmu] = 1.0
    H = h_matrix(ex, ey, sigma)
    ref = (X.T @ A @ H.T) / (A.sum(0) @ H.T)
    np.testing.assert_allclose(W1, ref, rtol=2e-7)
    # a neighbourhood-weighted mean of binary vectors stays inside [0, 1]
    assert W1.min() >= 0.0 and W1.max() <= 1.0


def test_identical_documents_pull_their_unit_onto_the_document():
    ci = np.tile(np.array([1, 4, 6], np.int32), 5)
    rp = np.arange(0, 16, 3, dtype=np.int32)
    num, cnt = oracle.scatter(rp, ci, np.full(5, 2, np.int32), 8, 4)
    W1 = oracle.writeback(oracle.blur(num, 2, 2, 0.0), oracle.blur(cnt, 2, 2, 0.0),
                          np.full((8, 4), 0.5, np.float32))
    want = np.zeros(8, np.float32)
    want[[1, 4, 6]] = 1.0
    assert np.array_equal(W1[:, 2], want) and np.all(W1[:, [0, 1, 3]] == 0.5)


# ------------------------------------------------------------------ stopping metrics
def test_map_errors_hand_computed_case():
    # a 4-column, 3-row map: unit j sits at (x, y) = (j % 4, j // 4)
    #   0  1  2  3
    #   4  5  6  7
    #   8  9 10 11
    bmu = np.array([5, 5, 5, 0, 11, 3], np.int32)
    bmu2 = np.array([6, 10, 7, 4, 7, 4], np.int32)
    #  5-6 share an edge; 5-10 share a corner; 5-7 are two apart; 0-4 share an edge (a row
    #  apart, not neighbours by index); 11-7 share an edge; 3-4 are index neighbours but sit at
    #  opposite ends of two rows
    dist = np.array([4.0, 9.0, 0.25, 16.0, 1.0, 0.0], np.float32)
    e4 = oracle.map_errors(bmu, bmu2, dist, 4, 3, adjacency=4)
    e8 = oracle.map_errors(bmu, bmu2, dist, 4, 3, adjacency=8)
    assert e4[0] == pytest.approx(30.25 / 6, rel=1e-15)            # mean of d
    assert e4[1] == pytest.approx((2 + 3 + 0.5 + 4 + 1 + 0) / 6, rel=1e-15)   # mean of sqrt(d)
    assert e4[2] == pytest.approx(3 / 6, rel=1e-15)                # 5-10, 5-7, 3-4
    assert e8[2] == pytest.approx(2 / 6, rel=1e-15)                # 5-7, 3-4
    assert np.array_equal(e4[:2], e8[:2])


def test_map_errors_edge_cases_and_invariants():
    assert np.array_equal(oracle.map_errors([], [], [], 5, 5), np.zeros(3))
    # a distance rounded below zero counts as zero in the root, as itself in the mean
    e = oracle.map_errors([0, 1], [1, 0], np.array([-1e-6, 4.0], np.float32), 2, 1)
    assert e[0] == pytest.approx((float(np.float32(-1e-6)) + 4.0) / 2, rel=1e-12) and e[1] == 1.0 and e[2] == 0.0
    # no second unit (one-neuron map): not an error
    assert oracle.map_errors([0, 0], [-1, -1], [1.0, 1.0], 1, 1)[2] == 0.0
    # a non-square map: x runs along a row of edge_x units
    assert oracle.map_errors([0], [7], [0.0], 7, 2)[2] == 0.0      # (0,0)-(0,1): an edge
    assert oracle.map_errors([0], [7], [0.0], 2, 7)[2] == 1.0      # (0,0)-(1,3)
    r = np.random.default_rng(17)
    ex, ey, N = 9, 6, 4000
    b1 = r.integers(0, ex * ey, N).astype(np.int32)
    b2 = r.integers(0, ex * ey, N).astype(np.int32)
    d = (r.random(N) * 50).astype(np.float32)
    e4, e8 = oracle.map_errors(b1, b2, d, ex, ey, 4), oracle.map_errors(b1, b2, d, ex, ey, 8)
    assert e8[2] <= e4[2]                                          # corners only ever help
    # the definition written with array operations
    dx, dy = np.abs(b1 % ex - b2 % ex), np.abs(b1 // ex - b2 // ex)
    assert e4[2] == pytest.approx(np.mean(dx + dy != 1), rel=1e-15)
    assert e8[2] == pytest.approx(np.mean(np.maximum(dx, dy) != 1), rel=1e-15)
    assert e4[0] == pytest.approx(d.astype(np.float64).mean(), rel=1e-12)
    assert e4[1] == pytest.approx(np.sqrt(d.astype(np.float64)).mean(), rel=1e-12)
    # swapping best and second-best changes no adjacency; permuting documents changes nothing
    assert oracle.map_errors(b2, b1, d, ex, ey, 4)[2] == e4[2]
    p = r.permutation(N)
    np.testing.assert_allclose(oracle.map_errors(b1[p], b2[p], d[p], ex, ey, 4), e4, rtol=1e-12)
    # by Jensen the mean root is at most the root of the mean
    assert e4[1] <= np.sqrt(e4[0])
