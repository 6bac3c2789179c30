"""fp64 CPU oracle for the SEA attention hot path.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain statement of what the CUDA library computes.  It
is imported by the tests, by the smoke check and by the benchmark's CPU
baseline leg, and by nothing on the product path.  It shares no code with the
CUDA kernels and never imports them.

Every function works on one attention head (2-D arrays) in float64 and follows
the paper's steps in the paper's order:

    favor_features      Sec. 3 "Performer (FAVOR+)": positive random features of
                        the softmax kernel (the paper omits the projection; the
                        benchmark definition fixes it: x = u * d^(-1/4),
                        phi_f(u) = exp(w_f . x - |x|^2 / 2) / sqrt(m)).
    favor_attention     Sec. 3 "Performer (FAVOR+)": phi(Q) (phi(K)^T V), with
                        the row normaliser phi(Q) (phi(K)^T 1); the causal form
                        keeps running prefix sums over phi(k) v^T and phi(k).
    decode_estimate     Sec. 3.1 "CNN Decoder", replaced by one linear head:
                        A_hat = C_perf W_dec.
    topk_select         Sec. 3.1 "Grouped Top-k Selection", per-query grouping:
                        the k_hat largest entries of each row of A_hat; equal
                        values go to the lower column.
    topk_select_grouped Sec. 3.1 "Grouped Top-k Selection", causal-per-batch
                        grouping: A_hat of one batch element is viewed as
                        [T, H, Kc]; for every query position the H * k_hat
                        largest of its H * Kc entries are kept (no exchange along
                        T); equal values go to the lower flattened index
                        h * Kc + c.  Heads then hold different numbers of columns.
    topk_select_causal_aware
                        the per-query selection restricted, for a causal row i,
                        to the compressed columns that hold at least one key
                        j <= i (columns 0 .. floor(i / r)); a row keeps
                        min(k_hat, floor(i / r) + 1) columns, so no row is left
                        without keys.  (The paper resizes every causal row of the
                        estimate to its own width, App. "Visualization of
                        intermediate buffers"; this is the part of that which the
                        fixed-ratio interpolation used here can express.)
    expand_mask         Sec. 3.1 "Linear Sparse Attention Mask Generation" and
                        App. "Sparse Interpolation": nearest-neighbour
                        up-sampling of the compressed mask done on indices; a
                        selected column c covers keys c*r .. c*r+r-1, r = T/Kc;
                        causal rows drop keys j > i.  Output is a flat CSR.
                        With k_star: the appendix's cap for long sequences, at
                        most k_star uniformly spaced keys per selected column.
    expand_mask_resized App. "Sparse Interpolation" at any ratio of T to Kc, and App.
                        "Visualization of intermediate buffers" for causal rows:
                        nearest-neighbour resize of row i of the compressed mask
                        from Kc pixels to a target width W (T; or, with
                        ``row_widths``, the causal row's own width i + 1): key j
                        looks at pixel floor(j * Kc / W).
    sparse_attention    Sec. 3.1.1 "Sparse Attention Mechanism": rho (scores at
                        mask positions), sigma (softmax over a row's non-zeros),
                        then C = A* V.
    sea_attention_head  the four steps chained.
    sea_attention_grouped_batch
                        the same chain for one batch element with the
                        causal-per-batch selection in place of the per-query one.

Pins (tests/test_oracle_*.py): k_hat = Kc reproduces dense (causal) softmax
attention from a library routine; top-k equals a brute-force ordering (the
grouped form too: brute force over the flattened slab, H = 1 reduces to the
per-query form, a head that dominates takes every slot); expansion equals a library nearest-neighbour resize; the feature form equals
the normalised T x T kernel-matrix product and its expectation equals
exp(q.k / sqrt(d)); rows of A* sum to one; causal outputs do not depend on
later tokens.

Parity unpinned: the particular omega / W_dec draws (only their seed is
fixed), and the choice of a linear head in place of the paper's trained
MLP + CNN decoder (a definition of this benchmark, nothing to check against).
"""
from __future__ import annotations

import numpy as np

__all__ = [
    "favor_features",
    "favor_attention",
    "decode_estimate",
    "estimate_head",
    "topk_select",
    "topk_select_grouped",
    "topk_select_causal_aware",
    "sea_attention_grouped_batch",
    "expand_mask",
    "expand_mask_resized",
    "sparse_attention",
    "sea_attention_head",
    "k_hat_from_k",
]


def _f64(a) -> np.ndarray:
    return np.asarray(a, dtype=np.float64)


def k_hat_from_k(k: int, Kc: int, T: int) -> int:
    """Sec. 3.1: k_hat = max(1, round(k * K / T)); halves round to even."""
    return max(1, int(np.rint(k * Kc / T)))


def favor_features(U, omega) -> np.ndarray:
    """Positive softmax-kernel features of the rows of U [T, d] -> [T, m]."""
    U = _f64(U)
    omega = _f64(omega)
    d = U.shape[1]
    m = omega.shape[0]
    X = U * d ** (-0.25)
    proj = X @ omega.T  # [T, m]
    sq = np.sum(X * X, axis=1, keepdims=True)  # [T, 1]
    return np.exp(proj - 0.5 * sq) / np.sqrt(m)


def favor_attention(Q, K, V, omega, causal: bool) -> np.ndarray:
    """Normalised linear attention C_perf [T, d]."""
    V = _f64(V)
    phi_q = favor_features(Q, omega)  # [T, m]
    phi_k = favor_features(K, omega)  # [T, m]
    T, d = V.shape
    if not causal:
        S = phi_k.T @ V  # [m, d]
        z = phi_k.T @ np.ones(T)  # [m]
        return (phi_q @ S) / (phi_q @ z)[:, None]
    m = phi_k.shape[1]
    S = np.zeros((m, d))
    z = np.zeros(m)
    C = np.empty((T, d))
    for i in range(T):
        S += np.outer(phi_k[i], V[i])
        z += phi_k[i]
        C[i] = (phi_q[i] @ S) / (phi_q[i] @ z)
    return C


def decode_estimate(C_perf, W_dec) -> np.ndarray:
    """A_hat [T, Kc] = C_perf [T, d] W_dec [d, Kc]."""
    return _f64(C_perf) @ _f64(W_dec)


def estimate_head(Q, K, V, omega, W_dec, causal: bool) -> np.ndarray:
    return decode_estimate(favor_attention(Q, K, V, omega, causal), W_dec)


def topk_select(A_hat, k_hat: int) -> np.ndarray:
    """Columns of the k_hat largest entries of each row, ascending.  [T, k_hat] int64."""
    A_hat = _f64(A_hat)
    T, Kc = A_hat.shape
    if not 1 <= k_hat <= Kc:
        raise ValueError("k_hat out of range")
    sel = np.empty((T, k_hat), dtype=np.int64)
    for i in range(T):
        # descending by value; a stable sort leaves equal values in column order
        order = np.argsort(-A_hat[i], kind="stable")
        sel[i] = np.sort(order[:k_hat])
    return sel


def topk_select_grouped(A_hat, k_hat: int):
    """Causal-per-batch selection over A_hat [H, T, Kc] of one batch element.

    Returns ``cols[h][t]``: the ascending selected columns of head h at query t.
    Over the heads every query keeps exactly H * k_hat columns.
    """
    A_hat = _f64(A_hat)
    H, T, Kc = A_hat.shape
    if not 1 <= k_hat <= Kc:
        raise ValueError("k_hat out of range")
    cols = [[None] * T for _ in range(H)]
    for t in range(T):
        slab = A_hat[:, t, :].reshape(H * Kc)  # flattened index h * Kc + c
        order = np.argsort(-slab, kind="stable")[: H * k_hat]
        taken = np.zeros(H * Kc, dtype=bool)
        taken[order] = True
        taken = taken.reshape(H, Kc)
        for h in range(H):
            cols[h][t] = np.flatnonzero(taken[h])
    return cols


def topk_select_causal_aware(A_hat, k_hat: int, T: int):
    """Rows of A_hat [T, Kc] are queries 0 .. T-1 of a causal head.  Returns the list of ascending
    column arrays: row i chooses among columns 0 .. floor(i / r), r = T / Kc."""
    A_hat = _f64(A_hat)
    n, Kc = A_hat.shape
    if n != T or T % Kc != 0:
        raise ValueError("one row per query, T a multiple of Kc")
    if not 1 <= k_hat <= Kc:
        raise ValueError("k_hat out of range")
    r = T // Kc
    cols = []
    for i in range(T):
        visible = i // r + 1  # columns that start at or before key i
        order = np.argsort(-A_hat[i, :visible], kind="stable")
        cols.append(np.sort(order[: min(k_hat, visible)]))
    return cols


def expand_mask(sel, T: int, Kc: int, causal: bool, query_index=None, k_star=None):
    """Flat CSR (row_ptr [n+1], col_idx [nnz]) of the up-sampled mask of one head.

    Row t of ``sel`` (an array [n, k_hat], or a list of n column arrays of any
    lengths) belongs to query ``query_index[t]`` (default: t, all T queries).

    ``k_star`` (App. "Sparse Interpolation", the case k K / T < 1): a selected column is
    replicated to at most k_star of its r = T / Kc keys, spaced uniformly over the run:
    keys c*r + floor(u * r / k_star), u = 0 .. k_star-1.  None or k_star >= r: the whole run.
    """
    if T % Kc != 0:
        raise ValueError("T must be a multiple of Kc")
    r = T // Kc
    if k_star is None or k_star >= r:
        offsets = list(range(r))
    else:
        if k_star < 1:
            raise ValueError("k_star must be positive")
        offsets = [(u * r) // k_star for u in range(k_star)]
    n = len(sel)
    if query_index is None:
        query_index = np.arange(n)
    row_ptr = np.zeros(n + 1, dtype=np.int64)
    cols = []
    for t in range(n):
        i = int(query_index[t])
        row = []
        for c in sel[t]:
            for o in offsets:
                j = int(c) * r + o
                if causal and j > i:
                    continue
                row.append(j)
        cols.extend(row)
        row_ptr[t + 1] = row_ptr[t] + len(row)
    return row_ptr, np.asarray(cols, dtype=np.int64)


def expand_mask_resized(sel, T: int, Kc: int, causal: bool, row_widths: bool, query_index=None):
    """Flat CSR of the mask obtained by resizing every row of the compressed mask by nearest
    neighbour, for any T and Kc (T need not be a multiple of Kc).

    Row i of the compressed mask has Kc pixels, those listed in ``sel[i]`` set.  It is resized to
    W pixels, W = T, or W = i + 1 when ``row_widths`` (the paper resizes every causal row to the
    row's own width): key j < W is kept when pixel floor(j * Kc / W) is set.  ``causal`` drops
    keys j > i (with row_widths there are none).
    """
    n = len(sel)
    if query_index is None:
        query_index = np.arange(n)
    row_ptr = np.zeros(n + 1, dtype=np.int64)
    cols = []
    for t in range(n):
        i = int(query_index[t])
        W = i + 1 if row_widths else T
        chosen = set(int(c) for c in sel[t])
        row = []
        for j in range(W):
            if causal and j > i:
                continue
            if (j * Kc) // W in chosen:
                row.append(j)
        cols.extend(row)
        row_ptr[t + 1] = row_ptr[t] + len(row)
    return row_ptr, np.asarray(cols, dtype=np.int64)


def sparse_attention(Q, K, V, row_ptr, col_idx, scale: float):
    """O [T, d] and the CSR probabilities P [nnz] of one head."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    T, d = Q.shape
    O = np.zeros((T, d))
    P = np.zeros(len(col_idx))
    for i in range(T):
        lo, hi = int(row_ptr[i]), int(row_ptr[i + 1])
        if hi == lo:
            continue  # an empty row keeps O_i = 0
        js = col_idx[lo:hi]
        s = (K[js] @ Q[i]) * scale
        e = np.exp(s - np.max(s))
        p = e / np.sum(e)
        P[lo:hi] = p
        O[i] = p @ V[js]
    return O, P


def sea_attention_head(Q, K, V, k_hat: int, Kc: int, causal: bool, scale: float,
                       A_hat=None, omega=None, W_dec=None):
    """All stages for one head.  Returns a dict with A_hat, sel, row_ptr, col_idx, O, P."""
    T = np.asarray(Q).shape[0]
    if A_hat is None:
        A_hat = estimate_head(Q, K, V, omega, W_dec, causal)
    sel = topk_select(A_hat, k_hat)
    row_ptr, col_idx = expand_mask(sel, T, Kc, causal)
    O, P = sparse_attention(Q, K, V, row_ptr, col_idx, scale)
    return dict(A_hat=_f64(A_hat), sel=sel, row_ptr=row_ptr, col_idx=col_idx, O=O, P=P)


def sea_attention_grouped_batch(Q, K, V, k_hat: int, Kc: int, causal: bool, scale: float,
                                A_hat=None, omega=None, W_dec=None):
    """All stages for one batch element (arrays [H, T, .]) with the causal-per-batch selection.

    Returns the list over heads of dicts with A_hat, cols, row_ptr, col_idx, O, P.
    """
    Q, K, V = np.asarray(Q), np.asarray(K), np.asarray(V)
    H, T = Q.shape[0], Q.shape[1]
    if A_hat is None:
        A_hat = np.stack([estimate_head(Q[h], K[h], V[h], omega, W_dec, causal) for h in range(H)])
    cols = topk_select_grouped(A_hat, k_hat)
    out = []
    for h in range(H):
        row_ptr, col_idx = expand_mask(cols[h], T, Kc, causal)
        O, P = sparse_attention(Q[h], K[h], V[h], row_ptr, col_idx, scale)
        out.append(dict(A_hat=_f64(A_hat[h]), cols=cols[h], row_ptr=row_ptr, col_idx=col_idx, O=O, P=P))
    return out
