"""Pins for the oracle's causal-per-batch selection (Sec. 3.1 "Grouped Top-k Selection"):
brute force over the flattened [H, Kc] slab of every query position, the special cases that
reduce to the per-query form or to a closed form, the invariants the paper states (H * k_hat
columns per query position, no exchange along T), and the chain down to dense attention."""
import numpy as np
import pytest
import torch

from oracle import sea_oracle as orc


def rng(seed):
    return np.random.default_rng(seed)


def brute_grouped(A, k_hat):
    """Pure-Python statement: per t, order (h, c) by (value descending, h, c) and keep H*k_hat."""
    H, T, Kc = A.shape
    out = [[None] * T for _ in range(H)]
    for t in range(T):
        pairs = [(h, c) for h in range(H) for c in range(Kc)]
        pairs.sort(key=lambda hc: (-float(A[hc[0], t, hc[1]]), hc[0], hc[1]))
        keep = set(pairs[: H * k_hat])
        for h in range(H):
            out[h][t] = [c for c in range(Kc) if (h, c) in keep]
    return out


def as_lists(cols):
    return [[list(map(int, c)) for c in per_head] for per_head in cols]


@pytest.mark.parametrize("H,T,Kc,k_hat", [(3, 7, 8, 2), (4, 5, 6, 6), (2, 9, 16, 1), (5, 3, 4, 3)])
def test_grouped_matches_bruteforce(H, T, Kc, k_hat):
    g = rng(21)
    A = g.standard_normal((H, T, Kc))
    assert as_lists(orc.topk_select_grouped(A, k_hat)) == brute_grouped(A, k_hat)


def test_grouped_ties_go_to_lower_flattened_index():
    H, T, Kc, k_hat = 3, 4, 8, 2
    g = rng(22)
    A = np.round(g.standard_normal((H, T, Kc)) * 1.5) / 2  # many equal values, signed zeros among them
    A[1, 0, :] = -0.0
    A[2, 0, :] = 0.0
    assert as_lists(orc.topk_select_grouped(A, k_hat)) == brute_grouped(A, k_hat)
    # an all-equal slab: the first H * k_hat flattened positions, i.e. head 0 first
    Z = np.zeros((H, T, Kc))
    cols = as_lists(orc.topk_select_grouped(Z, k_hat))
    for t in range(T):
        assert cols[0][t] == list(range(H * k_hat)) and cols[1][t] == [] and cols[2][t] == []


def test_grouped_with_one_head_is_per_query():
    g = rng(23)
    A = g.standard_normal((1, 12, 16))
    cols = orc.topk_select_grouped(A, 5)
    sel = orc.topk_select(A[0], 5)
    for t in range(12):
        assert list(cols[0][t]) == list(sel[t])


def test_grouped_keeps_exactly_H_k_hat_columns_per_position_and_no_exchange_along_T():
    g = rng(24)
    H, T, Kc, k_hat = 4, 10, 8, 3
    A = g.standard_normal((H, T, Kc))
    cols = orc.topk_select_grouped(A, k_hat)
    for t in range(T):
        assert sum(len(cols[h][t]) for h in range(H)) == H * k_hat
    # changing the estimate at one position leaves every other position's selection alone
    A2 = A.copy()
    A2[:, 6, :] = g.standard_normal((H, Kc)) * 10
    cols2 = orc.topk_select_grouped(A2, k_hat)
    for t in range(T):
        if t != 6:
            for h in range(H):
                assert list(cols[h][t]) == list(cols2[h][t])
    # the heads of one position do compete: a shift of one head changes what the others keep
    A3 = A.copy()
    A3[0] += 100.0
    cols3 = orc.topk_select_grouped(A3, k_hat)
    for t in range(T):
        assert len(cols3[0][t]) == Kc  # head 0 takes min(Kc, H*k_hat) = 8 of the 12 slots
        assert sum(len(cols3[h][t]) for h in range(1, H)) == H * k_hat - Kc


def test_dominating_head_takes_every_slot_closed_form():
    """H * k_hat <= Kc and one head far above the rest: that head keeps its own top-(H*k_hat)
    (a per-query selection with the larger budget), the others keep nothing and output zero."""
    g = rng(25)
    H, T, Kc, k_hat, d = 3, 16, 16, 2, 8
    A = g.standard_normal((H, T, Kc))
    A[1] += 50.0
    Q, K, V = (g.standard_normal((H, T, d)) for _ in range(3))
    res = orc.sea_attention_grouped_batch(Q, K, V, k_hat, Kc, False, 0.25, A_hat=A)
    alone = orc.sea_attention_head(Q[1], K[1], V[1], H * k_hat, Kc, False, 0.25, A_hat=A[1])
    np.testing.assert_array_equal(res[1]["col_idx"], alone["col_idx"])
    np.testing.assert_array_equal(res[1]["O"], alone["O"])
    for h in (0, 2):
        assert res[h]["row_ptr"][-1] == 0 and np.all(res[h]["O"] == 0.0)


@pytest.mark.parametrize("causal", [False, True])
def test_grouped_full_budget_is_dense_attention(causal):
    """k_hat = Kc keeps every column of every head: dense (causal) softmax attention per head."""
    g = rng(26)
    H, T, Kc, d = 2, 24, 6, 8
    Q, K, V = (g.standard_normal((H, T, d)) for _ in range(3))
    A = g.standard_normal((H, T, Kc))
    res = orc.sea_attention_grouped_batch(Q, K, V, Kc, Kc, causal, 0.3, A_hat=A)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Q)[None], torch.from_numpy(K)[None], torch.from_numpy(V)[None],
        is_causal=causal, scale=0.3)[0].numpy()
    for h in range(H):
        np.testing.assert_allclose(res[h]["O"], ref[h], atol=1e-12)


def test_grouped_partial_selection_is_masked_dense_attention():
    g = rng(27)
    H, T, Kc, d, k_hat = 3, 32, 8, 8, 2
    Q, K, V = (g.standard_normal((H, T, d)) for _ in range(3))
    A = g.standard_normal((H, T, Kc))
    r = T // Kc
    for causal in (False, True):
        res = orc.sea_attention_grouped_batch(Q, K, V, k_hat, Kc, causal, 0.3, A_hat=A)
        want = brute_grouped(A, k_hat)
        for h in range(H):
            mask = torch.zeros(T, T, dtype=torch.bool)
            for i in range(T):
                for c in want[h][i]:
                    for j in range(c * r, c * r + r):
                        if not causal or j <= i:
                            mask[i, j] = True
            rp, ci = res[h]["row_ptr"], res[h]["col_idx"]
            for i in range(T):
                assert list(ci[rp[i]:rp[i + 1]]) == list(torch.nonzero(mask[i]).flatten().numpy())
            ref = torch.nn.functional.scaled_dot_product_attention(
                torch.from_numpy(Q[h])[None], torch.from_numpy(K[h])[None], torch.from_numpy(V[h])[None],
                attn_mask=mask[None], scale=0.3)[0].numpy()
            nonempty = mask.any(dim=1).numpy()
            np.testing.assert_allclose(res[h]["O"][nonempty], ref[nonempty], atol=1e-12)
            assert np.all(res[h]["O"][~nonempty] == 0.0)


def test_grouped_pins_catch_planted_mistakes():
    g = rng(28)
    H, T, Kc, k_hat = 3, 6, 8, 2
    A = g.standard_normal((H, T, Kc))
    want = brute_grouped(A, k_hat)

    def grouped_along_T(A, k_hat):  # the per-head grouping: top T*k_hat of each head's [T, Kc]
        H, T, Kc = A.shape
        out = [[None] * T for _ in range(H)]
        for h in range(H):
            order = np.argsort(-A[h].reshape(T * Kc), kind="stable")[: T * k_hat]
            taken = np.zeros(T * Kc, dtype=bool)
            taken[order] = True
            taken = taken.reshape(T, Kc)
            for t in range(T):
                out[h][t] = list(map(int, np.flatnonzero(taken[t])))
        return out

    def per_query(A, k_hat):
        return [[list(map(int, row)) for row in orc.topk_select(A[h], k_hat)] for h in range(A.shape[0])]

    def smallest(A, k_hat):
        return as_lists(orc.topk_select_grouped(-A, k_hat))

    for bad in (grouped_along_T, per_query, smallest):
        assert bad(A, k_hat) != want


# ---------------------------------------------------------------------------
# Causal-aware per-query selection: only columns that hold a visible key compete.
# ---------------------------------------------------------------------------
def test_causal_aware_selection_bruteforce_and_invariants():
    g = rng(31)
    T, Kc, k_hat = 48, 12, 5
    r = T // Kc
    A = np.round(g.standard_normal((T, Kc)) * 2) / 2  # duplicates: ties go to the lower column
    cols = orc.topk_select_causal_aware(A, k_hat, T)
    for i in range(T):
        visible = i // r + 1
        order = sorted(range(visible), key=lambda c: (-float(A[i, c]), c))
        assert list(cols[i]) == sorted(order[: min(k_hat, visible)])
        assert len(cols[i]) == min(k_hat, visible)
    row_ptr, col_idx = orc.expand_mask(cols, T, Kc, True)
    counts = np.diff(row_ptr)
    assert np.all(counts >= 1), "no causal row is left without keys"
    for i in range(T):
        js = col_idx[row_ptr[i]:row_ptr[i + 1]]
        assert np.all(js <= i) and np.all(np.diff(js) > 0)
    # once every column is visible and the row's k_hat best lie among them, it is the per-query selection
    plain = orc.topk_select(A, k_hat)
    for i in range(T - r, T):
        assert list(cols[i]) == list(plain[i])
    # where the plain selection already avoids invisible columns the two agree, elsewhere they differ
    differ = sum(list(cols[i]) != [c for c in plain[i]] for i in range(T))
    assert differ > 0


def test_causal_aware_first_rows_are_dense_causal_attention():
    """While floor(i / r) + 1 <= k_hat every visible column is kept: rows 0 .. k_hat * r - 1 see
    every key j <= i, i.e. dense causal attention there."""
    g = rng(32)
    T, Kc, k_hat, d = 64, 16, 4, 8
    r = T // Kc
    Q, K, V = (g.standard_normal((T, d)) for _ in range(3))
    A = g.standard_normal((T, Kc))
    cols = orc.topk_select_causal_aware(A, k_hat, T)
    row_ptr, col_idx = orc.expand_mask(cols, T, Kc, True)
    O, P = orc.sparse_attention(Q, K, V, row_ptr, col_idx, 0.3)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Q)[None], torch.from_numpy(K)[None], torch.from_numpy(V)[None], is_causal=True,
        scale=0.3)[0].numpy()
    n_dense = k_hat * r
    np.testing.assert_allclose(O[:n_dense], ref[:n_dense], atol=1e-12)
    assert np.array_equal(np.diff(row_ptr)[:n_dense], np.arange(1, n_dense + 1))


# ---------------------------------------------------------------------------
# Capped replication for long sequences (App. "Sparse Interpolation", k K / T < 1):
# at most k_star uniformly spaced keys per selected column.
# ---------------------------------------------------------------------------
def test_capped_expansion_invariants_and_special_cases():
    g = rng(41)
    T, Kc, k_hat = 96, 8, 2
    r = T // Kc  # 12
    A = g.standard_normal((T, Kc))
    sel = orc.topk_select(A, k_hat)
    full_rp, full_ci = orc.expand_mask(sel, T, Kc, False)
    for k_star in (r, r + 5, None):  # no cap: the whole run
        rp, ci = orc.expand_mask(sel, T, Kc, False, k_star=k_star)
        assert np.array_equal(rp, full_rp) and np.array_equal(ci, full_ci)
    for k_star in (1, 3, 4, 5, 7):
        rp, ci = orc.expand_mask(sel, T, Kc, False, k_star=k_star)
        assert np.all(np.diff(rp) == k_hat * k_star)  # the paper's constant number of non-zeros per row
        for i in range(T):
            js = ci[rp[i]:rp[i + 1]]
            assert np.all(np.diff(js) > 0)
            for n, c in enumerate(sel[i]):
                run = js[n * k_star:(n + 1) * k_star] - c * r
                assert run[0] == 0 and np.all((0 <= run) & (run < r))
                gaps = np.diff(np.append(run, r))  # uniformly spaced: gaps differ by at most one
                assert gaps.max() - gaps.min() <= 1
            assert set(js) <= set(full_ci[full_rp[i]:full_rp[i + 1]])  # a subset of the uncapped mask
        crp, cci = orc.expand_mask(sel, T, Kc, True, k_star=k_star)
        for i in range(T):
            js = ci[rp[i]:rp[i + 1]]
            assert list(cci[crp[i]:crp[i + 1]]) == [j for j in js if j <= i]
    # k_star dividing r: every (r / k_star)-th key of the run
    rp, ci = orc.expand_mask(sel[:1], T, Kc, False, k_star=4)
    c0 = sel[0][0]
    assert list(ci[:4]) == [c0 * r + o for o in (0, 3, 6, 9)]


def test_capped_mask_attention_is_masked_dense_attention():
    g = rng(42)
    T, Kc, d, k_hat, k_star = 64, 4, 8, 1, 5
    r = T // Kc
    Q, K, V = (g.standard_normal((T, d)) for _ in range(3))
    A = g.standard_normal((T, Kc))
    sel = orc.topk_select(A, k_hat)
    for causal in (False, True):
        rp, ci = orc.expand_mask(sel, T, Kc, causal, k_star=k_star)
        O, P = orc.sparse_attention(Q, K, V, rp, ci, 0.3)
        mask = torch.zeros(T, T, dtype=torch.bool)
        for i in range(T):
            for c in sel[i]:
                for u in range(k_star):
                    j = int(c) * r + (u * r) // k_star
                    if not causal or j <= i:
                        mask[i, j] = True
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(Q)[None], torch.from_numpy(K)[None], torch.from_numpy(V)[None],
            attn_mask=mask[None], scale=0.3)[0].numpy()
        nonempty = mask.any(dim=1).numpy()
        np.testing.assert_allclose(O[nonempty], ref[nonempty], atol=1e-12)
        assert np.all(O[~nonempty] == 0.0)
