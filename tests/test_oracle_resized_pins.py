"""Pins of the oracle's nearest-neighbour resize at any ratio (App. "Sparse Interpolation" for T
not a multiple of Kc; App. "Visualization of intermediate buffers": every causal row of the
compressed mask is resized to the row's own width)."""
import numpy as np
import pytest
import torch

from oracle import sea_oracle as orc


def rng(seed):
    return np.random.default_rng(seed)


def dense_rows(row_ptr, col_idx, n, T):
    M = np.zeros((n, T), dtype=bool)
    for i in range(n):
        M[i, col_idx[row_ptr[i]:row_ptr[i + 1]]] = True
    return M


def compressed_mask(sel, Kc):
    M_hat = np.zeros((len(sel), Kc), dtype=np.float64)
    for i, cols in enumerate(sel):
        M_hat[i, cols] = 1
    return M_hat


@pytest.mark.parametrize("T,Kc,k_hat", [(30, 8, 3), (50, 7, 2), (33, 32, 5), (64, 16, 4), (20, 40, 9)])
def test_resize_to_full_width_matches_library_nearest_resize(T, Kc, k_hat):
    """Width T for every row, T and Kc in any ratio (also Kc > T): torch's nearest resize in fp64."""
    sel = orc.topk_select(rng(1).standard_normal((T, Kc)), k_hat)
    M_star = torch.nn.functional.interpolate(torch.from_numpy(compressed_mask(sel, Kc))[None, None], size=(T, T),
                                             mode="nearest")[0, 0].numpy() > 0
    row_ptr, col_idx = orc.expand_mask_resized(sel, T, Kc, causal=False, row_widths=False)
    assert np.array_equal(dense_rows(row_ptr, col_idx, T, T), M_star)
    row_ptr_c, col_idx_c = orc.expand_mask_resized(sel, T, Kc, causal=True, row_widths=False)
    assert np.array_equal(dense_rows(row_ptr_c, col_idx_c, T, T), np.tril(M_star))


@pytest.mark.parametrize("T,Kc,k_hat", [(32, 8, 3), (64, 64, 5), (48, 4, 2)])
def test_integer_ratio_reduces_to_runs_of_r_keys(T, Kc, k_hat):
    sel = orc.topk_select(rng(2).standard_normal((T, Kc)), k_hat)
    for causal in (False, True):
        a = orc.expand_mask(sel, T, Kc, causal)
        b = orc.expand_mask_resized(sel, T, Kc, causal, row_widths=False)
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


@pytest.mark.parametrize("T,Kc,k_hat", [(40, 8, 3), (64, 16, 16), (37, 5, 2)])
def test_causal_rows_resized_to_their_own_width(T, Kc, k_hat):
    """Row i resized to i + 1 pixels: torch's nearest resize of that single row; no key after the
    query; the last row equals the full-width resize; a row at least Kc wide keeps at least k_hat
    keys (every set pixel survives an up-sampling), and k_hat = Kc gives the dense causal mask."""
    sel = orc.topk_select(rng(3).standard_normal((T, Kc)), k_hat)
    M_hat = compressed_mask(sel, Kc)
    row_ptr, col_idx = orc.expand_mask_resized(sel, T, Kc, causal=True, row_widths=True)
    for i in range(T):
        ref = torch.nn.functional.interpolate(torch.from_numpy(M_hat[i])[None, None], size=(i + 1,),
                                              mode="nearest")[0, 0].numpy() > 0
        cols = col_idx[row_ptr[i]:row_ptr[i + 1]]
        assert cols.tolist() == np.nonzero(ref)[0].tolist()
        assert np.all(cols <= i)
        if i + 1 >= Kc:
            assert len(cols) >= k_hat
        if k_hat == Kc:
            assert cols.tolist() == list(range(i + 1))
    full = orc.expand_mask_resized(sel, T, Kc, causal=False, row_widths=False)
    assert col_idx[row_ptr[T - 1]:row_ptr[T]].tolist() == full[1][full[0][T - 1]:full[0][T]].tolist()


def test_a_planted_index_mistake_is_caught():
    """ceil instead of floor in the pixel index, or the ratio turned upside down, changes the mask."""
    T, Kc = 30, 8
    sel = orc.topk_select(rng(4).standard_normal((T, Kc)), 3)
    good = dense_rows(*orc.expand_mask_resized(sel, T, Kc, False, False), T, T)
    for wrong in (lambda j: -((-j * Kc) // T), lambda j: min(Kc - 1, (j * T) // Kc)):
        bad = np.zeros_like(good)
        for i in range(T):
            for j in range(T):
                bad[i, j] = wrong(j) in set(sel[i].tolist())
        assert not np.array_equal(good, bad)


def test_resized_mask_drives_the_sparse_attention_like_a_dense_mask():
    """Attention under the resized mask equals torch's SDPA under the same boolean mask."""
    T, Kc, d = 24, 5, 8
    g = rng(6)
    Q, K, V = (g.standard_normal((T, d)) for _ in range(3))
    sel = orc.topk_select(g.standard_normal((T, Kc)), 2)
    row_ptr, col_idx = orc.expand_mask_resized(sel, T, Kc, causal=True, row_widths=True)
    O, P = orc.sparse_attention(Q, K, V, row_ptr, col_idx, 1.0 / np.sqrt(d))
    M = dense_rows(row_ptr, col_idx, T, T)
    keeps = M.any(axis=1)  # a row narrower than Kc pixels may lose every set pixel: O = 0 there
    assert keeps[Kc - 1:].all() and np.all(O[~keeps] == 0)
    M[~keeps, 0] = True    # (any key, so that the library routine has a row to normalise)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Q)[None], torch.from_numpy(K)[None], torch.from_numpy(V)[None],
        attn_mask=torch.from_numpy(M)[None])[0].numpy()
    assert np.allclose(O[keeps], ref[keeps], atol=1e-12)
