"""Pins of the oracle for the paper's estimator head and output mixing (Sec. 3.1 "Attention Matrix
Estimation", "CNN Decoder"; App. "Attention Estimator CNN"; Sec. 3.1.1 "Output Calculation")."""
import numpy as np
import pytest
import torch

from oracle import sea_decoder_oracle as dec
from oracle import sea_oracle as orc
from paper_2310_01777_b200.inputs import Workload, make_decoder_params, make_inputs


def rng(seed):
    return np.random.default_rng(seed)


def np64(t):
    return t.to(torch.float64).numpy()


def tiny(causal, T=24, H=2, Kc=8, dtype="f32"):
    w = Workload("dec_tiny", 1, H, T, 16, 8, Kc, 2, causal, dtype, seed=4)
    host = make_inputs(w)
    prm = {k: np64(v) for k, v in make_decoder_params(w, d_hidden=12, c_s=2, c_h=3).items()}
    return w, host, prm


def test_v_identity_is_the_library_nearest_resize_of_the_identity():
    for T, d in [(10, 4), (64, 16), (7, 16), (33, 8)]:
        ref = torch.nn.functional.interpolate(torch.eye(d, dtype=torch.float64)[None, None], size=(T, d), mode="nearest")[0, 0]
        assert np.array_equal(dec.v_identity(T, d), ref.numpy())


@pytest.mark.parametrize("causal", [False, True])
def test_performer_cat_is_two_base_estimates_side_by_side(causal):
    """FAVOR+ is linear in V: [V_I ; V] gives the base estimator's output for V_I and for V; and with
    V_I the first half is the (normalised, approximate) attention matrix sampled at d columns."""
    g = rng(2)
    T, d, m = 20, 8, 16
    Q, K, V = (g.standard_normal((T, d)) for _ in range(3))
    om = g.standard_normal((m, d))
    first = dec.v_identity(T, d)
    C = dec.performer_cat(Q, K, V, first, om, causal)
    assert np.allclose(C[:, d:], orc.favor_attention(Q, K, V, om, causal), atol=1e-12)
    assert np.allclose(C[:, :d], orc.favor_attention(Q, K, first, om, causal), atol=1e-12)
    assert np.allclose(C[:, :d].sum(axis=1), 1.0)  # rows of the kernel matrix, pooled into d bins, sum to one


def conv_by_loops(x, w, b, stride_h, causal):
    C_in, H, W = x.shape
    C_out = w.shape[0]
    top = 2 if causal else 1
    H_out = (H + (2 if causal else 2) - 3) // stride_h + 1
    out = np.zeros((C_out, H_out, W))
    for o in range(C_out):
        for y in range(H_out):
            for xx in range(W):
                acc = b[o]
                for c in range(C_in):
                    for ky in range(3):
                        for kx in range(3):
                            yy, xc = y * stride_h + ky - top, xx + kx - 1
                            if 0 <= yy < H and 0 <= xc < W:
                                acc += w[o, c, ky, kx] * x[c, yy, xc]
                out[o, y, xx] = acc
    return out


@pytest.mark.parametrize("causal,stride", [(False, 1), (False, 2), (True, 1)])
def test_convolution_step_against_explicit_loops(causal, stride):
    g = rng(3)
    x, w, b = g.standard_normal((3, 8, 5)), g.standard_normal((4, 3, 3, 3)), g.standard_normal(4)
    assert np.allclose(dec._conv3x3(x, w, b, stride, causal), conv_by_loops(x, w, b, stride, causal), atol=1e-12)


def test_to_image_puts_channel_groups_of_a_head_side_by_side():
    H, T, Wr, c_h = 2, 3, 4, 3
    z = np.arange(H * T * Wr * c_h, dtype=np.float64).reshape(H, T, Wr * c_h)
    img = dec.to_image(z, c_h)
    for h in range(H):
        for j in range(c_h):
            for t in range(T):
                for x in range(Wr):
                    assert img[h * c_h + j, t, x] == z[h, t, j * Wr + x]


@pytest.mark.parametrize("causal", [False, True])
def test_decoder_rows_are_distributions_and_shapes_follow_the_paper(causal):
    w, host, prm = tiny(causal)
    A, Z = dec.decoder_estimate(np64(host["Q"][0]), np64(host["K"][0]), np64(host["V"][0]), np64(host["omega"]), prm, w.Kc, 2, 3,
                                causal)
    assert A.shape == (w.H, w.T, w.Kc) and Z.shape == (w.H, w.T, 12)
    assert np.allclose(A.sum(axis=-1), 1.0) and np.all(A > 0) and np.all(Z >= 0)


def test_causal_decoder_does_not_look_ahead():
    """Changing tokens after t leaves rows <= t of A_hat and Z unchanged (the causal estimator, the
    top-padded convolutions, no height reduction); the non-causal decoder does change."""
    t = 13
    for causal in (True, False):
        w, host, prm = tiny(causal)
        a = dec.decoder_estimate(np64(host["Q"][0]), np64(host["K"][0]), np64(host["V"][0]), np64(host["omega"]), prm, w.Kc, 2, 3,
                                 causal)
        h2 = {k: v.clone() for k, v in host.items()}
        g = torch.Generator().manual_seed(9)
        for k in ("Q", "K", "V"):
            h2[k][:, :, t + 1:] = torch.randn(h2[k][:, :, t + 1:].shape, generator=g)
        b = dec.decoder_estimate(np64(h2["Q"][0]), np64(h2["K"][0]), np64(h2["V"][0]), np64(host["omega"]), prm, w.Kc, 2, 3,
                                 causal)
        same = np.allclose(a[0][:, :t + 1], b[0][:, :t + 1], atol=1e-12) and np.allclose(a[1][:, :t + 1], b[1][:, :t + 1], atol=1e-12)
        assert same == causal


def test_pooled_context_and_mixing():
    g = rng(5)
    T, d, Kc = 12, 4, 3
    V = g.standard_normal((T, d))
    A = g.random((T, Kc))
    # causal: the running mean of V, by brute force
    ca = dec.pooled_context(A, V, True)
    for t in range(T):
        assert np.allclose(ca[t], V[:t + 1].sum(axis=0) / (t + 1))
    # not causal: importance = column means of A_hat, resized by the library's nearest resize, times V
    i_hat = torch.from_numpy(A.mean(axis=0))
    i = torch.nn.functional.interpolate(i_hat[None, None], size=(T,), mode="nearest")[0, 0].numpy()
    assert np.allclose(dec.pooled_context(A, V, False), np.tile(i @ V, (T, 1)))
    # mixing: s_mix = 1 gives s_prob * C, s_mix = 0 gives C_avg; P rows sum to s_prob
    C = g.standard_normal((T, d))
    row_ptr = np.arange(0, 3 * T + 1, 3)
    P = np.full(3 * T, 1.0 / 3.0)
    sp = g.random(T)
    out1, P1 = dec.mix_output(C, P, row_ptr, sp, np.ones(T), ca)
    out0, _ = dec.mix_output(C, P, row_ptr, sp, np.zeros(T), ca)
    assert np.allclose(out1, sp[:, None] * C) and np.allclose(out0, ca)
    assert np.allclose(np.add.reduceat(P1, row_ptr[:-1]), sp)


def test_scalers_are_sigmoids_of_linear_heads():
    g = rng(6)
    Z = g.standard_normal((5, 4))
    prm = dict(w_prob=g.standard_normal(4), b_prob=np.array([0.3]), w_mix=np.zeros(4), b_mix=np.array([0.0]))
    sp, sm = dec.scalers(Z, prm)
    assert np.allclose(sm, 0.5) and np.allclose(np.log(sp / (1 - sp)), Z @ prm["w_prob"] + 0.3)
