"""fp64 CPU oracle for the paper's estimator head and output mixing.  TEST INFRASTRUCTURE ONLY.

The plain statement of Sec. 3.1 "Attention Matrix Estimation" / "CNN Decoder", App. "Attention
Estimator CNN" and Sec. 3.1.1 ("Sparse Attention Mechanism": s_prob; "Output Calculation": C_avg,
s_mix) for one batch element (all heads: the CNN treats the heads as channels), with random-init
weights handed in by the caller.  It shares no code with the CUDA kernels, is imported by tests
only, and uses library routines (matmul, torch's conv2d in fp64) as single steps.

Steps, in the paper's order (readings where the paper is silent are marked R):

    v_identity      V_I: nearest-neighbour resize of the identity I_d to T rows: row t is the unit
                    vector e_floor(t d / T).  Causal layers use a positional embedding [T, d] in its
                    place (App. "Attention Estimator CNN").
    performer_cat   C_perf = FAVOR+(Q, K, [V_I ; V]) in R^{T x 2d} (same normalised linear
                    attention as the base estimator, values 2d wide).
    mlp_mu          Z = relu([C_perf ; V] W_mu + b_mu) in R^{T x d'}            (R: one layer, ReLU)
    mlp_nu          Z_hat = relu(Z W_1 + b_1) W_2 + b_2 in R^{T x (K/c_s) c_h}  (R: ReLU between)
    to_image        [H, T, (K/c_s) c_h] -> [H c_h, T, K/c_s]: entry j (K/c_s) + x of head h's vector
                    is channel h c_h + j, width x                               (R: channel-major)
    cnn_decoder     conv 3x3 (C -> C, relu), conv 3x3 (C -> C, relu), nearest resize to [C, T, K],
                    conv 3x3 (C -> H), softmax over K.  Not causal: the first layer has stride c_s
                    along T (padding 1), the resize brings T back.  Causal: no height reduction, and
                    every layer pads two rows at the top and none at the bottom, so that row t sees
                    rows t-2 .. t only; the width is padded by one on both sides in both cases.
    scalers         s_prob = sigmoid(Z w_prob + b_prob), s_mix = sigmoid(Z w_mix + b_mix) in R^T
    pooled_context  not causal: i_hat = mean over rows of A_hat (R^K), resized by nearest neighbour
                    to R^T, C_avg = i^T V in R^d (one vector for all rows); causal: C_avg[t] =
                    mean of V[0 .. t].
    mix_output      C_sea = s_mix * (s_prob * C) + (1 - s_mix) * C_avg, with C the sparse
                    attention's output; the CSR probabilities are s_prob * softmax.

Parity unpinned: the weight draws (only their seed is fixed); the readings marked R are choices
where the paper gives no detail (each is stated in the list of steps above), pinned only in the sense that the
library routines used here are checked against explicit loops.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle.sea_oracle import favor_features

__all__ = ["v_identity", "performer_cat", "mlp_mu", "mlp_nu", "to_image", "cnn_decoder", "decoder_estimate",
           "scalers", "pooled_context", "mix_output"]


def _f64(a):
    return np.asarray(a, dtype=np.float64)


def v_identity(T: int, d: int) -> np.ndarray:
    out = np.zeros((T, d))
    for t in range(T):
        out[t, (t * d) // T] = 1.0
    return out


def performer_cat(Q, K, V, first, omega, causal: bool) -> np.ndarray:
    """C_perf [T, 2d] of one head; ``first`` is V_I (or the positional embedding), [T, d]."""
    Q, K, V, first = _f64(Q), _f64(K), _f64(V), _f64(first)
    pq, pk = favor_features(Q, omega), favor_features(K, omega)
    vcat = np.concatenate([first, V], axis=1)
    T = Q.shape[0]
    if not causal:
        return (pq @ (pk.T @ vcat)) / (pq @ pk.sum(axis=0))[:, None]
    out = np.zeros((T, vcat.shape[1]))
    S = np.zeros((pk.shape[1], vcat.shape[1]))
    z = np.zeros(pk.shape[1])
    for i in range(T):
        S += np.outer(pk[i], vcat[i])
        z += pk[i]
        out[i] = (pq[i] @ S) / (pq[i] @ z)
    return out


def mlp_mu(C_perf, V, W_mu, b_mu) -> np.ndarray:
    x = np.concatenate([_f64(C_perf), _f64(V)], axis=1)
    return np.maximum(x @ _f64(W_mu) + _f64(b_mu), 0.0)


def mlp_nu(Z, W1, b1, W2, b2) -> np.ndarray:
    return np.maximum(_f64(Z) @ _f64(W1) + _f64(b1), 0.0) @ _f64(W2) + _f64(b2)


def to_image(Z_hat, c_h: int) -> np.ndarray:
    """[H, T, Wr * c_h] -> [H * c_h, T, Wr]."""
    H, T, n = Z_hat.shape
    Wr = n // c_h
    return _f64(Z_hat).reshape(H, T, c_h, Wr).transpose(0, 2, 1, 3).reshape(H * c_h, T, Wr)


def _conv3x3(x, w, b, stride_h: int, causal: bool) -> np.ndarray:
    """x [C_in, H, W] -> [C_out, H_out, W]; width padded by 1 on both sides; height padded by 1 on
    both sides, or (causal) by 2 at the top only."""
    xt = torch.from_numpy(_f64(x))[None]
    pad = (1, 1, 2, 0) if causal else (1, 1, 1, 1)  # (left, right, top, bottom)
    xt = torch.nn.functional.pad(xt, pad)
    y = torch.nn.functional.conv2d(xt, torch.from_numpy(_f64(w)), torch.from_numpy(_f64(b)), stride=(stride_h, 1))
    return y[0].numpy()


def cnn_decoder(image, params, T: int, Kc: int, c_s: int, causal: bool) -> np.ndarray:
    """image [C, T, Kc / c_s] -> A_hat [H, T, Kc] (rows softmaxed)."""
    h1 = np.maximum(_conv3x3(image, params["conv1_w"], params["conv1_b"], 1 if causal else c_s, causal), 0.0)
    h2 = np.maximum(_conv3x3(h1, params["conv2_w"], params["conv2_b"], 1, causal), 0.0)
    up = torch.nn.functional.interpolate(torch.from_numpy(h2)[None], size=(T, Kc), mode="nearest")[0].numpy()
    logits = _conv3x3(up, params["conv3_w"], params["conv3_b"], 1, causal)
    e = np.exp(logits - logits.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


def decoder_estimate(Q, K, V, omega, params, Kc: int, c_s: int, c_h: int, causal: bool):
    """One batch element: Q, K, V [H, T, d].  Returns A_hat [H, T, Kc] and Z [H, T, d']."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    H, T, d = Q.shape
    first = _f64(params["pos_emb"]) if causal else v_identity(T, d)
    Z = np.stack([mlp_mu(performer_cat(Q[h], K[h], V[h], first, omega, causal), V[h], params["W_mu"], params["b_mu"])
                  for h in range(H)])
    Z_hat = np.stack([mlp_nu(Z[h], params["W_nu1"], params["b_nu1"], params["W_nu2"], params["b_nu2"]) for h in range(H)])
    A_hat = cnn_decoder(to_image(Z_hat, c_h), params, T, Kc, c_s, causal)
    return A_hat, Z


def scalers(Z, params):
    """s_prob, s_mix [T] of one head from Z [T, d']."""
    sig = lambda x: 1.0 / (1.0 + np.exp(-x))
    Z = _f64(Z)
    return sig(Z @ _f64(params["w_prob"]) + float(np.asarray(params["b_prob"]).reshape(-1)[0])), sig(Z @ _f64(params["w_mix"]) + float(np.asarray(params["b_mix"]).reshape(-1)[0]))


def pooled_context(A_hat, V, causal: bool) -> np.ndarray:
    """C_avg [T, d] of one head (not causal: every row is the same pooled vector)."""
    A_hat, V = _f64(A_hat), _f64(V)
    T, Kc = A_hat.shape
    if causal:
        return np.cumsum(V, axis=0) / np.arange(1, T + 1)[:, None]
    i_hat = A_hat.mean(axis=0)
    i = np.array([i_hat[(j * Kc) // T] for j in range(T)])
    return np.tile(i @ V, (T, 1))


def mix_output(C, P, row_ptr, s_prob, s_mix, C_avg):
    """C_sea [T, d] and the re-scaled CSR probabilities."""
    C, C_avg = _f64(C), _f64(C_avg)
    s_prob, s_mix = _f64(s_prob), _f64(s_mix)
    P2 = _f64(P) * np.repeat(s_prob, np.diff(row_ptr))
    return s_mix[:, None] * (s_prob[:, None] * C) + (1.0 - s_mix[:, None]) * C_avg, P2
