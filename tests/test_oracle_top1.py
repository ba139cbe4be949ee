"""Pins of the oracle's Algorithm-1 (max gradient approximation) path."""
import numpy as np
import pytest

from oracle import oracle

GEOMS = [
    oracle.Shape(3, 4, 6, 6, 5, 3, 3, 1, 1, 1, 1),
    oracle.Shape(2, 3, 8, 8, 4, 3, 3, 2, 2, 1, 1),
    oracle.Shape(4, 2, 6, 5, 3, 5, 5, 1, 1, 2, 2),
    oracle.Shape(2, 2, 4, 4, 2, 3, 3, 1, 1, 0, 0),
]


def _rand(g, seed):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((g.n, g.c, g.h, g.w)), rng.standard_normal((g.n, g.k, g.p, g.q))


@pytest.mark.parametrize("g", GEOMS)
def test_selection_brute_force(g):
    _, dy = _rand(g, 11)
    idx, s, a = oracle.top1_select(dy)
    for n in range(g.n):
        for k in range(g.k):
            flat = dy[n, k].reshape(-1)
            best = 0
            for j in range(len(flat)):
                if abs(flat[j]) > abs(flat[best]):
                    best = j
            assert idx[n, k] == best == int(np.argmax(np.abs(flat)))
            assert abs(s[n, k] - float(np.sum(flat))) < 1e-12
            assert abs(a[n, k] - float(np.sum(np.abs(flat)))) < 1e-12


def test_tie_break_takes_lowest_index_and_sign_is_ignored():
    dy = np.zeros((1, 2, 3, 4))
    dy[0, 0, 1, 2] = -5.0; dy[0, 0, 2, 3] = 5.0; dy[0, 0, 0, 1] = 4.0
    dy[0, 1, 2, 0] = 1.0; dy[0, 1, 0, 3] = -1.0
    idx, s, _ = oracle.top1_select(dy)
    assert idx[0, 0] == 1 * 4 + 2 and idx[0, 1] == 3
    assert s[0, 0] == 4.0 and s[0, 1] == 0.0
    idx0, _, _ = oracle.top1_select(np.zeros((1, 1, 2, 2)))
    assert idx0[0, 0] == 0


@pytest.mark.parametrize("g", GEOMS)
def test_top1_equals_exact_on_sparsified_dy_and_sparse_list(g):
    """Section 2.3: the gradient is 'calculated from this sparse version of the output gradient'."""
    x, dy = _rand(g, 12)
    alpha = 1.0 / 128
    dw, _ = oracle.dw_top1(x, dy, g, alpha)
    idx, s, _ = oracle.top1_select(dy)
    dys = oracle.sparsify(idx, s, g.p * g.q).reshape(dy.shape)
    assert np.count_nonzero(dys) == g.n * g.k                      # sparsity 1 - 1/(PQ)
    assert abs(1 - np.count_nonzero(dys) / dys.size - (1 - 1 / (g.p * g.q))) < 1e-15
    dw_dense, _ = oracle.dw_exact(x, dys, g, alpha)
    np.testing.assert_allclose(dw, dw_dense, rtol=0, atol=1e-13)
    entries = [(n, k, int(idx[n, k]) // g.q, int(idx[n, k]) % g.q, float(s[n, k]))
               for n in range(g.n) for k in range(g.k)]
    np.testing.assert_allclose(dw, oracle.dw_sparse(x, entries, g, alpha), rtol=0, atol=1e-13)


@pytest.mark.parametrize("g", GEOMS)
def test_full_selection_equals_exact(g):
    x, dy = _rand(g, 13)
    entries = [(n, k, p, q, float(dy[n, k, p, q])) for n in range(g.n) for k in range(g.k)
               for p in range(g.p) for q in range(g.q)]
    dw, _ = oracle.dw_exact(x, dy, g)
    np.testing.assert_allclose(oracle.dw_sparse(x, entries, g), dw, rtol=0, atol=1e-12)


@pytest.mark.parametrize("g", GEOMS)
def test_one_hot_dy_makes_top1_exact(g):
    x, _ = _rand(g, 14)
    rng = np.random.default_rng(15)
    dy = np.zeros((g.n, g.k, g.p, g.q))
    for n in range(g.n):
        for k in range(g.k):
            dy[n, k, rng.integers(g.p), rng.integers(g.q)] = rng.standard_normal()
    np.testing.assert_allclose(oracle.dw_top1(x, dy, g)[0], oracle.dw_exact(x, dy, g)[0], rtol=0, atol=1e-13)


def test_single_output_pixel_makes_top1_exact():
    g = oracle.Shape(3, 2, 5, 5, 4, 5, 5)
    x, dy = _rand(g, 16)
    np.testing.assert_allclose(oracle.dw_top1(x, dy, g)[0], oracle.dw_exact(x, dy, g)[0], rtol=0, atol=1e-13)


def test_spatially_constant_x_without_padding_makes_top1_exact():
    """With X constant over each (n,c) map and no padding every patch is that constant, so the
    retained value must be the SIGNED channel sum for Algorithm 1 to reproduce the exact gradient."""
    g = oracle.Shape(3, 4, 7, 7, 5, 3, 3, 2, 2, 0, 0)
    rng = np.random.default_rng(17)
    a = rng.standard_normal((g.n, g.c, 1, 1))
    x = np.broadcast_to(a, (g.n, g.c, g.h, g.w)).copy()
    dy = rng.standard_normal((g.n, g.k, g.p, g.q))
    t1, _ = oracle.dw_top1(x, dy, g)
    ex, _ = oracle.dw_exact(x, dy, g)
    np.testing.assert_allclose(t1, ex, rtol=0, atol=1e-12)
    assert np.max(np.abs(ex)) > 0.1


def test_literal_algorithm_restatement_small():
    """Algorithm 1 on a case small enough to follow by hand: one image, one filter, 2x2 map, pad 0."""
    g = oracle.Shape(1, 1, 3, 3, 1, 2, 2)
    x = np.arange(9, dtype=float).reshape(1, 1, 3, 3)
    dy = np.array([[[[1.0, -4.0], [2.0, 3.0]]]])      # arg max |.| at (0,1); sum = 2
    dw, dn = oracle.dw_top1(x, dy, g)
    np.testing.assert_array_equal(dw[0, 0], 2.0 * x[0, 0, 0:2, 1:3])
    np.testing.assert_array_equal(dn[0, 0], 10.0 * x[0, 0, 0:2, 1:3])


@pytest.mark.parametrize("g", GEOMS[:2])
def test_metamorphic_relations(g):
    x, dy = _rand(g, 18)
    idx, s, _ = oracle.top1_select(dy)
    idx2, s2, _ = oracle.top1_select(-8.0 * dy)
    np.testing.assert_array_equal(idx, idx2)
    np.testing.assert_array_equal(s2, -8.0 * s)
    dw, _ = oracle.dw_top1(x, dy, g)
    np.testing.assert_array_equal(oracle.dw_top1(x, -8.0 * dy, g)[0], -8.0 * dw)
    perm = np.random.default_rng(19).permutation(g.n)
    np.testing.assert_allclose(oracle.dw_top1(x[perm], dy[perm], g)[0], dw, rtol=0, atol=1e-12)
    x2, _ = _rand(g, 20)
    lin = oracle.dw_top1(2.0 * x + x2, dy, g)[0]
    np.testing.assert_allclose(lin, 2.0 * dw + oracle.dw_top1(x2, dy, g)[0], rtol=0, atol=1e-12)
    dy3 = dy.copy(); dy3[1, 2, g.p - 1, g.q - 2] = 100.0
    assert oracle.top1_select(dy3)[0][1, 2] == (g.p - 1) * g.q + g.q - 2


def test_zero_method():
    z = oracle.dw_zero(17)
    assert z.shape == (17,) and np.all(z == 0.0) and not np.any(np.signbit(z))


# ---- the order of magnitudes used by the selection: bit pattern of |v| (any input has a defined position) ----
def test_selection_orders_nan_above_inf_above_finite_and_ignores_the_sign_of_zero():
    dy = np.zeros((1, 6, 2, 3))
    dy[0, 0] = [[1.0, -np.inf, 3.0], [np.inf, 2.0, 0.0]]          # two infinities: the earlier one
    dy[0, 1] = [[1.0, np.inf, 3.0], [np.nan, 2.0, -np.nan]]       # NaN sorts above infinity; equal payloads: the earlier
    dy[0, 2] = [[-0.0, 0.0, -0.0], [0.0, 0.0, 0.0]]               # all zeros of either sign: position 0
    dy[0, 3] = [[-0.0, 0.0, 1e-300], [0.0, -1e-300, 0.0]]         # equal magnitudes of opposite sign: the earlier
    dy[0, 4] = [[5.0, -7.0, 7.0], [1.0, 2.0, 3.0]]
    dy[0, 5] = [[1.0, 2.0, 3.0], [4.0, 5.0, np.float64("nan")]]
    idx, s, _ = oracle.top1_select(dy)
    assert idx[0].tolist() == [1, 3, 0, 2, 1, 5]
    assert np.isnan(s[0, 0]) and np.isnan(s[0, 1]) and s[0, 2] == 0 and s[0, 4] == 11.0      # the sum propagates as IEEE does
    # for finite inputs the order is the order of |v|: same answer as numpy's first arg max of |v|
    rng = np.random.default_rng(77)
    d = rng.standard_normal((3, 4, 5, 6)).astype(np.float32).astype(np.float64)
    want = np.argmax(np.abs(d).reshape(3, 4, -1), axis=2)
    np.testing.assert_array_equal(oracle.top1_select(d)[0], want)


# ---- top-k variant: pinned by k = 1, by the sparse list, by brute force, and by the constant-X case ----
@pytest.mark.parametrize("g", GEOMS)
def test_topk_with_k_one_is_algorithm_1(g):
    x, dy = _rand(g, 30)
    a, an = oracle.dw_topk(x, dy, g, 1, 0.5)
    b, bn = oracle.dw_top1(x, dy, g, 0.5)
    np.testing.assert_array_equal(a, b)
    np.testing.assert_array_equal(an, bn)
    np.testing.assert_array_equal(oracle.topk_select(dy, 1)[0][..., 0], oracle.top1_select(dy)[0])


@pytest.mark.parametrize("topk", [2, 3, 5])
@pytest.mark.parametrize("g", GEOMS[:3])
def test_topk_equals_the_sparse_list_with_sum_over_k(g, topk):
    x, dy = _rand(g, 31)
    t = min(topk, g.p * g.q)
    # brute-force selection: stable sort of positions by descending |v| (numpy), first t of each map
    flat = dy.reshape(g.n, g.k, -1)
    order = np.argsort(-np.abs(flat), axis=2, kind="stable")[..., :t]
    idx, s, _ = oracle.topk_select(dy, topk)
    np.testing.assert_array_equal(idx, order)
    np.testing.assert_allclose(s, flat.sum(axis=2), rtol=0, atol=1e-12)
    entries = [(n, k, int(j) // g.q, int(j) % g.q, float(flat[n, k].sum() / t))
               for n in range(g.n) for k in range(g.k) for j in order[n, k]]
    np.testing.assert_allclose(oracle.dw_topk(x, dy, g, topk, 0.25)[0], oracle.dw_sparse(x, entries, g, 0.25), rtol=0, atol=1e-12)


@pytest.mark.parametrize("topk", [1, 2, 4, 9])
def test_topk_is_exact_for_spatially_constant_x_without_padding(topk):
    """Every patch is the same constant, so any k retained entries that add up to the map's sum give the exact gradient."""
    g = oracle.Shape(3, 4, 7, 7, 5, 3, 3, 2, 2, 0, 0)
    rng = np.random.default_rng(32)
    x = np.broadcast_to(rng.standard_normal((g.n, g.c, 1, 1)), (g.n, g.c, g.h, g.w)).copy()
    dy = rng.standard_normal((g.n, g.k, g.p, g.q))
    np.testing.assert_allclose(oracle.dw_topk(x, dy, g, topk)[0], oracle.dw_exact(x, dy, g)[0], rtol=0, atol=1e-12)


def test_topk_keeping_every_position_of_a_constant_map_is_exact():
    """k = P*Q with a map whose entries are all equal: each keeps sum/k = its own value, so top-k equals exact dW."""
    g = oracle.Shape(2, 3, 6, 6, 4, 3, 3, 1, 1, 1, 1)
    rng = np.random.default_rng(33)
    x = rng.standard_normal((g.n, g.c, g.h, g.w))
    dy = np.broadcast_to(rng.standard_normal((g.n, g.k, 1, 1)), (g.n, g.k, g.p, g.q)).copy()
    np.testing.assert_allclose(oracle.dw_topk(x, dy, g, g.p * g.q)[0], oracle.dw_exact(x, dy, g)[0], rtol=0, atol=1e-12)
