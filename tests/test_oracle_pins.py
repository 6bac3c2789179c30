"""Pins for the fp64 oracle: each part is checked against something that is not
the oracle itself (a library routine, brute force on tiny inputs, a closed
form, or an invariant the paper states)."""
import itertools

import numpy as np
import pytest
import torch

from oracle import sea_oracle as orc


def rng(seed):
    return np.random.default_rng(seed)


# ---------------------------------------------------------------------------
# Sparse attention with every column kept is dense softmax attention
# (Sec. 3.1.1: A* = sigma(rho(Q, K^T, M*)) with M* = 1, then C = A* V).
# The reference here is torch's scaled_dot_product_attention in float64.
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("T,Kc", [(32, 8), (48, 48), (64, 4)])
def test_full_selection_is_dense_attention(causal, T, Kc):
    g = rng(1)
    d = 16
    Q, K, V = (g.standard_normal((T, d)) for _ in range(3))
    scale = 1.0 / np.sqrt(d)
    A_hat = g.standard_normal((T, Kc))
    res = orc.sea_attention_head(Q, K, V, k_hat=Kc, Kc=Kc, causal=causal, scale=scale, A_hat=A_hat)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Q)[None], torch.from_numpy(K)[None], torch.from_numpy(V)[None],
        is_causal=causal, scale=scale)[0].numpy()
    np.testing.assert_allclose(res["O"], ref, rtol=0, atol=1e-12)
    # the CSR probabilities are the dense probabilities read along each row
    logits = torch.from_numpy(Q @ K.T * scale)
    if causal:
        logits = logits.masked_fill(torch.triu(torch.ones(T, T, dtype=torch.bool), 1), float("-inf"))
    dense_p = torch.softmax(logits, dim=-1).numpy()
    for i in range(T):
        lo, hi = res["row_ptr"][i], res["row_ptr"][i + 1]
        np.testing.assert_allclose(res["P"][lo:hi], dense_p[i, res["col_idx"][lo:hi]], atol=1e-13)
        assert hi - lo == (i + 1 if causal else T)


def test_partial_selection_is_masked_dense_attention():
    """With k_hat < Kc the result equals dense attention under the boolean mask M*."""
    g = rng(2)
    T, Kc, d, k_hat = 40, 10, 8, 3
    Q, K, V = (g.standard_normal((T, d)) for _ in range(3))
    A_hat = g.standard_normal((T, Kc))
    for causal in (False, True):
        res = orc.sea_attention_head(Q, K, V, k_hat, Kc, causal, 0.3, A_hat=A_hat)
        mask = torch.zeros(T, T, dtype=torch.bool)
        for i in range(T):
            mask[i, res["col_idx"][res["row_ptr"][i]:res["row_ptr"][i + 1]]] = True
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(Q)[None], torch.from_numpy(K)[None], torch.from_numpy(V)[None],
            attn_mask=mask[None], scale=0.3)[0].numpy()
        nonempty = mask.any(dim=1).numpy()
        np.testing.assert_allclose(res["O"][nonempty], ref[nonempty], atol=1e-12)
        assert np.all(res["O"][~nonempty] == 0.0)  # empty causal rows give exactly zero


# ---------------------------------------------------------------------------
# Top-k: brute force ordering by (value descending, column ascending).
# ---------------------------------------------------------------------------
def brute_topk(row, k_hat):
    order = sorted(range(len(row)), key=lambda c: (-float(row[c]), c))
    return sorted(order[:k_hat])


def test_topk_matches_bruteforce_with_ties_and_zeros():
    g = rng(3)
    rows = [
        g.standard_normal(16),
        np.zeros(16),  # all equal: lowest columns win
        np.array([1.0, 3.0, 3.0, 2.0, 3.0, 0.0, -1.0, 3.0]),  # repeated maximum
        np.array([0.0, -0.0, 0.0, -0.0, 1.0, -1.0, -0.0, 0.0]),  # signed zeros tie
        np.round(g.standard_normal(32) * 2) / 2,  # many duplicates
        -np.abs(g.standard_normal(16)),
    ]
    for row in rows:
        for k_hat in range(1, len(row) + 1):
            got = orc.topk_select(row[None, :], k_hat)[0]
            assert got.tolist() == brute_topk(row, k_hat)


def test_topk_exhaustive_small():
    """All rows over a 3-letter alphabet of length 5: every tie pattern."""
    for vals in itertools.product([-1.0, 0.0, 2.0], repeat=5):
        row = np.array(vals)
        for k_hat in (1, 2, 4):
            assert orc.topk_select(row[None, :], k_hat)[0].tolist() == brute_topk(row, k_hat)


def test_topk_float32_input_keeps_order():
    """The GPU estimate arrives as fp32; widening to fp64 must not change the order."""
    g = rng(4)
    a32 = g.standard_normal((8, 64)).astype(np.float32)
    a32[:, 5] = a32[:, 40]  # plant exact ties
    sel = orc.topk_select(a32, 7)
    for i in range(8):
        assert sel[i].tolist() == brute_topk(a32[i], 7)


# ---------------------------------------------------------------------------
# Mask expansion: nearest-neighbour up-sampling of the dense compressed mask
# by the integer ratio r (App. "Sparse Interpolation"), via a library resize.
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("T,Kc,k_hat", [(32, 8, 3), (64, 64, 5), (48, 4, 2), (16, 16, 16)])
def test_expand_matches_library_nearest_resize(T, Kc, k_hat):
    g = rng(5)
    A_hat = g.standard_normal((T, Kc))
    sel = orc.topk_select(A_hat, k_hat)
    M_hat = np.zeros((T, Kc), dtype=np.float32)
    for i in range(T):
        M_hat[i, sel[i]] = 1
    M_star = torch.nn.functional.interpolate(
        torch.from_numpy(M_hat)[None, None], size=(T, T), mode="nearest")[0, 0].numpy() > 0
    assert np.array_equal(M_star, np.repeat(M_hat, T // Kc, axis=1) > 0)
    row_ptr, col_idx = orc.expand_mask(sel, T, Kc, causal=False)
    # the paper's count: the mask holds a constant T * k non-zeros (k = k_hat * r)
    assert row_ptr[-1] == T * k_hat * (T // Kc)
    for i in range(T):
        cols = col_idx[row_ptr[i]:row_ptr[i + 1]]
        assert cols.tolist() == np.nonzero(M_star[i])[0].tolist()
    # causal: the same rows with keys after the query removed, nothing else
    row_ptr_c, col_idx_c = orc.expand_mask(sel, T, Kc, causal=True)
    for i in range(T):
        cols = col_idx_c[row_ptr_c[i]:row_ptr_c[i + 1]]
        assert cols.tolist() == [j for j in np.nonzero(M_star[i])[0].tolist() if j <= i]
    assert np.all(col_idx_c <= np.repeat(np.arange(T), np.diff(row_ptr_c)))


def test_expand_rejects_ragged_ratio():
    with pytest.raises(ValueError):
        orc.expand_mask(np.zeros((10, 1), dtype=np.int64), 10, 3, False)


# ---------------------------------------------------------------------------
# FAVOR+: the linear form equals the normalised T x T kernel-matrix product,
# and the features are an unbiased estimate of the softmax kernel.
# ---------------------------------------------------------------------------
def kernel_matrix_attention(Q, K, V, omega, causal):
    """D^-1 (Phi_q Phi_k^T [tril]) V with the T x T matrix written out entry by entry."""
    T, d = Q.shape
    m = omega.shape[0]
    A = np.zeros((T, T))
    for i in range(T):
        xq = Q[i] / d ** 0.25
        for j in range(T):
            if causal and j > i:
                continue
            xk = K[j] / d ** 0.25
            acc = 0.0
            for f in range(m):
                acc += (np.exp(omega[f] @ xq - xq @ xq / 2) * np.exp(omega[f] @ xk - xk @ xk / 2)) / m
            A[i, j] = acc
    return (A / A.sum(axis=1, keepdims=True)) @ V, A


@pytest.mark.parametrize("causal", [False, True])
def test_favor_linear_form_equals_kernel_matrix_product(causal):
    g = rng(6)
    T, d, m = 12, 8, 6
    Q, K, V = (g.standard_normal((T, d)) for _ in range(3))
    omega = g.standard_normal((m, d))
    got = orc.favor_attention(Q, K, V, omega, causal)
    ref, _ = kernel_matrix_attention(Q, K, V, omega, causal)
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-13)


def test_favor_with_identity_values_returns_normalised_kernel_matrix():
    """Sec. 3.1: with V = I the Performer output is the attention matrix itself."""
    g = rng(7)
    T, d, m = 10, 4, 5
    Q, K = g.standard_normal((T, d)), g.standard_normal((T, d))
    omega = g.standard_normal((m, d))
    got = orc.favor_attention(Q, K, np.eye(T), omega, causal=False)
    _, A = kernel_matrix_attention(Q, K, np.eye(T), omega, False)
    np.testing.assert_allclose(got, A / A.sum(1, keepdims=True), rtol=1e-12)
    np.testing.assert_allclose(got.sum(1), 1.0, rtol=1e-12)


def test_favor_features_are_unbiased_for_softmax_kernel():
    """E_w[phi(q).phi(k)] = exp(q.k / sqrt(d)): pins the d^(-1/4) scaling, the
    -|x|^2/2 term and the 1/sqrt(m) factor.  Monte Carlo with m = 400k features;
    inputs kept small so the estimator's variance is small."""
    g = rng(8)
    d, m = 8, 400_000
    q = 0.5 * g.standard_normal((3, d))
    k = 0.5 * g.standard_normal((4, d))
    omega = g.standard_normal((m, d))
    est = orc.favor_features(q, omega) @ orc.favor_features(k, omega).T
    exact = np.exp(q @ k.T / np.sqrt(d))
    np.testing.assert_allclose(est, exact, rtol=2e-2)


def test_favor_with_many_features_approaches_softmax_attention():
    g = rng(9)
    T, d, m = 6, 4, 300_000
    Q, K, V = (0.5 * g.standard_normal((T, d)) for _ in range(3))
    omega = g.standard_normal((m, d))
    for causal in (False, True):
        got = orc.favor_attention(Q, K, V, omega, causal)
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(Q)[None], torch.from_numpy(K)[None], torch.from_numpy(V)[None],
            is_causal=causal)[0].numpy()
        np.testing.assert_allclose(got, ref, atol=2e-2)


def test_favor_stabiliser_freedom():
    """Scaling all key features by one constant and each query's features by its
    own constant leaves the normalised output unchanged (so a GPU path may subtract
    maxima inside the exponent)."""
    g = rng(10)
    T, d, m = 9, 4, 7
    Q, K, V = (g.standard_normal((T, d)) for _ in range(3))
    omega = g.standard_normal((m, d))
    base = orc.favor_attention(Q, K, V, omega, True)
    phi_q = orc.favor_features(Q, omega) * np.exp(-g.standard_normal((T, 1)))
    phi_k = orc.favor_features(K, omega) * np.exp(-1.7)
    A = np.tril(phi_q @ phi_k.T)
    np.testing.assert_allclose((A / A.sum(1, keepdims=True)) @ V, base, rtol=1e-11)


def test_decoder_is_plain_matmul():
    g = rng(11)
    C, W = g.standard_normal((5, 3)), g.standard_normal((3, 4))
    ref = np.array([[sum(C[i, t] * W[t, c] for t in range(3)) for c in range(4)] for i in range(5)])
    np.testing.assert_allclose(orc.decode_estimate(C, W), ref, rtol=1e-14)


# ---------------------------------------------------------------------------
# Softmax invariants (Sec. 3.1.1: every row of A* sums to one).
# ---------------------------------------------------------------------------
def test_softmax_rows_sum_to_one_and_shift_invariance():
    g = rng(12)
    T, Kc, d, k_hat = 64, 16, 8, 3
    Q, K, V = (g.standard_normal((T, d)) for _ in range(3))
    sel = orc.topk_select(g.standard_normal((T, Kc)), k_hat)
    row_ptr, col_idx = orc.expand_mask(sel, T, Kc, True)
    O, P = orc.sparse_attention(Q, K, V, row_ptr, col_idx, 0.5)
    for i in range(T):
        if row_ptr[i + 1] > row_ptr[i]:
            assert abs(P[row_ptr[i]:row_ptr[i + 1]].sum() - 1.0) < 1e-14
    # adding a constant vector to every key shifts all of a row's scores equally
    shift = g.standard_normal(d)
    # q.(k + t) = q.k + q.t: a per-row constant, softmax unchanged
    O2, P2 = orc.sparse_attention(Q, K + shift, V, row_ptr, col_idx, 0.5)
    np.testing.assert_allclose(P2, P, atol=1e-13)
    np.testing.assert_allclose(O2, O, atol=1e-13)


def test_single_key_row_copies_value():
    g = rng(13)
    T, d = 8, 4
    Q, K, V = (g.standard_normal((T, d)) for _ in range(3))
    row_ptr = np.arange(T + 1)
    col_idx = g.integers(0, T, size=T)
    O, P = orc.sparse_attention(Q, K, V, row_ptr, col_idx, 1.0)
    np.testing.assert_array_equal(P, np.ones(T))
    np.testing.assert_allclose(O, V[col_idx], rtol=1e-15)


# ---------------------------------------------------------------------------
# Causality end to end: changing tokens after t leaves rows <= t untouched.
# ---------------------------------------------------------------------------
def test_causal_pipeline_ignores_future_tokens():
    g = rng(14)
    T, d, m, Kc, k_hat, t = 32, 8, 6, 8, 3, 13
    Q, K, V = (g.standard_normal((T, d)) for _ in range(3))
    omega, W = g.standard_normal((m, d)), g.standard_normal((d, Kc))
    a = orc.sea_attention_head(Q, K, V, k_hat, Kc, True, 0.35, omega=omega, W_dec=W)
    Q2, K2, V2 = Q.copy(), K.copy(), V.copy()
    for X in (Q2, K2, V2):
        X[t + 1:] = g.standard_normal((T - t - 1, d))
    b = orc.sea_attention_head(Q2, K2, V2, k_hat, Kc, True, 0.35, omega=omega, W_dec=W)
    np.testing.assert_array_equal(a["A_hat"][:t + 1], b["A_hat"][:t + 1])
    np.testing.assert_array_equal(a["sel"][:t + 1], b["sel"][:t + 1])
    np.testing.assert_array_equal(a["row_ptr"][:t + 2], b["row_ptr"][:t + 2])
    n = a["row_ptr"][t + 1]
    np.testing.assert_array_equal(a["col_idx"][:n], b["col_idx"][:n])
    np.testing.assert_array_equal(a["P"][:n], b["P"][:n])
    np.testing.assert_array_equal(a["O"][:t + 1], b["O"][:t + 1])
    assert np.all(a["col_idx"] <= np.repeat(np.arange(T), np.diff(a["row_ptr"])))


# ---------------------------------------------------------------------------
# k -> k_hat (Sec. 3.1), on the paper's own hyper-parameter settings.
# ---------------------------------------------------------------------------
def test_k_hat_from_paper_settings():
    import os

    path = os.path.join(os.path.dirname(__file__), "golden", "k_hat_settings.txt")
    n = 0
    with open(path) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            k, Kc, T, expect = (int(x) for x in line.split())
            assert orc.k_hat_from_k(k, Kc, T) == expect
            n += 1
    assert n >= 6


# ---------------------------------------------------------------------------
# The pins have teeth: plausible mistakes planted in copies of the oracle fail them.
# ---------------------------------------------------------------------------
def test_pins_catch_planted_mistakes(monkeypatch):
    g = rng(15)
    d, m = 8, 200_000
    q, k = 0.5 * g.standard_normal((2, d)), 0.5 * g.standard_normal((2, d))
    omega = g.standard_normal((m, d))
    exact = np.exp(q @ k.T / np.sqrt(d))

    def wrong_scaling(U, om):  # d^(-1/2) instead of d^(-1/4)
        X = np.asarray(U) * U.shape[1] ** (-0.5)
        return np.exp(X @ om.T - 0.5 * np.sum(X * X, 1, keepdims=True)) / np.sqrt(om.shape[0])

    def dropped_norm(U, om):  # missing -|x|^2 / 2
        X = np.asarray(U) * U.shape[1] ** (-0.25)
        return np.exp(X @ om.T) / np.sqrt(om.shape[0])

    for bad in (wrong_scaling, dropped_norm):
        est = bad(q, omega) @ bad(k, omega).T
        assert not np.allclose(est, exact, rtol=2e-2)

    # ties to the higher index, or a descending sort of the wrong sign, fail the brute force
    row = np.array([1.0, 3.0, 3.0, 2.0, 3.0])
    assert np.sort(np.argsort(row, kind="stable")[::-1][:2]).tolist() != brute_topk(row, 2)
    assert np.sort(np.argsort(row, kind="stable")[:2]).tolist() != brute_topk(row, 2)
