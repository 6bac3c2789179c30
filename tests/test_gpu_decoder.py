"""GPU parity of the paper's estimator head (V_cat, MLPs, three-layer CNN, row softmax) and of the
output mixing (s_prob, s_mix, C_avg) against the fp64 oracle, with seeded random-init weights."""
import numpy as np
import pytest
import torch

import paper_2310_01777_b200 as sea
from oracle import sea_decoder_oracle as dec
from oracle import sea_oracle as orc
from paper_2310_01777_b200.inputs import Workload, make_decoder_params, make_inputs, torch_dtype
from tests.helpers import check_a_hat, check_float, np64, scale_of

pytestmark = pytest.mark.gpu


def small(name, **kw):
    base = dict(name=name, B=1, H=2, T=128, d=64, m=32, Kc=16, k_hat=3, causal=True, dtype="bf16", seed=31)
    base.update(kw)
    return Workload(**base)


class Run:
    def __init__(self, w, d_hidden=24, c_s=2, c_h=3, device="cuda:0"):
        self.w, self.dev, self.c_s, self.c_h = w, device, c_s, c_h
        self.host = make_inputs(w)
        self.hp = make_decoder_params(w, d_hidden, c_s, c_h)
        self.d = {k: v.to(device) for k, v in self.host.items()}
        self.p = {k: v.to(device) for k, v in self.hp.items()}
        self.shape = sea.make_shape(w)
        self.dec = sea.make_decoder(self.p, d_hidden, c_s, c_h, w.causal)
        self.ws = torch.empty(sea.sea_workspace_bytes_decoder(self.shape, self.dec), dtype=torch.uint8, device=device)
        self.ws[:256].zero_()
        io = torch_dtype(w.dtype)
        self.O = torch.full((w.B, w.H, w.T, w.d), float("nan"), dtype=io, device=device)
        self.A_hat = torch.full((w.B, w.H, w.T, w.Kc), float("nan"), dtype=torch.float32, device=device)
        self.Z = torch.full((w.B, w.H, w.T, d_hidden), float("nan"), dtype=torch.float32, device=device)
        self.sel = torch.full((w.rows, w.k_hat), -1, dtype=torch.int32, device=device)
        self.row_ptr = torch.full((w.rows + 1,), -1, dtype=torch.int32, device=device)
        self.col_idx = torch.full((w.nnz_cap,), -1, dtype=torch.int32, device=device)
        self.P = torch.full((w.nnz_cap,), float("nan"), dtype=io, device=device)

    def stages(self):
        s, d = self.shape, self.d
        sea.sea_estimate_decoder(s, self.dec, d["Q"], d["K"], d["V"], d["omega"], self.A_hat, self.Z, self.ws)
        sea.sea_topk_mask(s, self.A_hat, self.sel, self.row_ptr, self.col_idx, self.ws)
        sea.sea_sparse_attn(s, d["Q"], d["K"], d["V"], self.row_ptr, self.col_idx, self.sel, self.O, self.P, self.ws)
        sea.sea_mix_output(s, self.dec, self.Z, self.A_hat, d["V"], self.row_ptr, self.O, self.P, self.ws)

    def fused(self):
        d = self.d
        sea.sea_attention_decoder(self.shape, self.dec, d["Q"], d["K"], d["V"], d["omega"], self.O, self.ws, A_hat=self.A_hat,
                                  sel=self.sel, row_ptr=self.row_ptr, col_idx=self.col_idx, P=self.P)

    def done(self):
        torch.cuda.synchronize(self.dev)
        assert sea.sea_device_status(self.ws) == 0


def check_batch(run, b, check_z=True):
    w = run.w
    prm = {k: np64(v) for k, v in run.hp.items()}
    Q, K, V = (np64(run.host[n][b]) for n in ("Q", "K", "V"))
    A_ref, Z_ref = dec.decoder_estimate(Q, K, V, np64(run.host["omega"]), prm, w.Kc, run.c_s, run.c_h, w.causal)
    A = run.A_hat[b].cpu().numpy()
    check_a_hat(A.reshape(-1, w.Kc), A_ref.reshape(-1, w.Kc))
    if check_z:
        check_a_hat(run.Z[b].cpu().numpy().reshape(w.H * w.T, -1), Z_ref.reshape(w.H * w.T, -1))
    for h in range(w.H):
        bh = b * w.H + h
        # mask and attention from the GPU's own estimate, as for the base path
        sel = orc.topk_select(A[h], w.k_hat)
        np.testing.assert_array_equal(run.sel[bh * w.T:(bh + 1) * w.T].cpu().numpy(), sel)
        row_ptr, col_idx = orc.expand_mask(sel, w.T, w.Kc, w.causal)
        C, P = orc.sparse_attention(Q[h], K[h], V[h], row_ptr, col_idx, scale_of(w))
        # scalers from the GPU's Z (checked above), pooled context from the GPU's estimate
        Zg = run.Z[b, h].cpu().numpy() if check_z else Z_ref[h]
        s_prob, s_mix = dec.scalers(Zg, prm)
        C_sea, P2 = dec.mix_output(C, P, row_ptr, s_prob, s_mix, dec.pooled_context(A[h], V[h], w.causal))
        rp = run.row_ptr[bh * w.T:(bh + 1) * w.T + 1].cpu().numpy().astype(np.int64)
        lo, hi = int(rp[0]), int(rp[-1])
        np.testing.assert_array_equal(rp - lo, row_ptr)
        check_float(np64(run.O[b, h]), C_sea, w.dtype, "C_sea")
        check_float(np64(run.P[lo:hi]), P2, w.dtype, "P")


# Images whose width divides 128 (or is a multiple of it) run the tensor-core convolutions with their
# few channels in one block of 64; the others (12 columns) the fp32 ones.
CASES = [
    small("dec_causal"),
    small("dec_nc", causal=False, H=3, T=96, Kc=24, k_hat=5),
    small("dec_f32", dtype="f32", T=64, Kc=8, k_hat=2, m=16),
    small("dec_nc_f32", dtype="f32", causal=False, T=64, Kc=16, k_hat=4, m=16, B=2),
    small("dec_wide", T=256, Kc=128, k_hat=9, H=4, m=64),       # image 64 columns wide: two column tiles, 16 channels
    small("dec_causal_w12", T=96, Kc=24, k_hat=5),              # image 12 columns wide: the fp32 convolutions, causal
]


@pytest.mark.parametrize("w", CASES, ids=lambda w: w.name)
def test_decoder_stages_and_fused_call_match_oracle(w):
    a = Run(w)
    a.stages(); a.done()
    assert bool(torch.isfinite(a.A_hat).all())
    assert torch.allclose(a.A_hat.sum(-1), torch.ones_like(a.A_hat[..., 0]), atol=1e-5)
    for b in range(w.B):
        check_batch(a, b)
    f = Run(w)
    f.fused(); f.done()
    nnz = int(a.row_ptr[-1])
    for name in ("A_hat", "sel", "row_ptr", "O"):
        assert torch.equal(getattr(a, name), getattr(f, name)), name
    view = torch.int16 if w.dtype == "bf16" else torch.int32
    assert torch.equal(a.col_idx[:nnz], f.col_idx[:nnz]) and torch.equal(a.P[:nnz].view(view), f.P[:nnz].view(view))


# Shapes whose convolutions run in the tensor-core form (H c_h a multiple of 64, image width a
# divisor or multiple of 128): one and two blocks of input channels, both paddings, the strided
# first layer, two and four phases of the folded resize, tiles that run past the last row.
TC_CASES = [
    small("dec_tc_causal", H=16, T=256, Kc=32, k_hat=4),
    small("dec_tc_nc", causal=False, H=32, T=192, Kc=64, k_hat=6),
    small("dec_tc_nc_ragged", causal=False, H=16, T=80, Kc=16, k_hat=3),
    small("dec_tc_causal_ragged", H=16, T=80, Kc=16, k_hat=3, B=2),
    small("dec_tc_wide", H=16, T=512, Kc=256, k_hat=8),   # Z_hat 512 wide: two chunks of W_2; image rows of 128 pixels
    small("dec_tc_two_tiles", H=16, T=512, Kc=512, k_hat=8),  # image 256 pixels wide: two column tiles per row, Z_hat in four chunks
    small("dec_tc_h12_nc", causal=False, H=12, T=128, Kc=32, k_hat=4),  # 48 channels in a block of 64, 48 of 64 logit columns
    small("dec_tc_h12", H=12, T=160, Kc=32, k_hat=4, dtype="f32"),      # fp32 I/O; 24 of 32 logit columns; tiles of 4 heads
]


# d' = 64 also takes the MLPs to their tensor-core form (feature map written as bf16 planes: four
# channels at a time when the image is a multiple of 16 wide, else element by element)
@pytest.mark.parametrize("d_hidden", [24, 64])
@pytest.mark.parametrize("w", TC_CASES, ids=lambda w: w.name)
def test_tensor_core_head_matches_oracle(w, d_hidden):
    a = Run(w, d_hidden=d_hidden, c_h=4)
    a.stages(); a.done()
    assert bool(torch.isfinite(a.A_hat).all())
    assert torch.allclose(a.A_hat.sum(-1), torch.ones_like(a.A_hat[..., 0]), atol=1e-5)
    for b in range(w.B):
        check_batch(a, b)


def test_causal_decoder_on_device_does_not_look_ahead():
    w = small("dec_perturb", T=128, Kc=16)
    t = 70
    a = Run(w)
    a.fused(); a.done()
    b = Run(w)
    g = torch.Generator().manual_seed(5)
    for k in ("Q", "K", "V"):
        b.host[k][:, :, t + 1:] = torch.randn(b.host[k][:, :, t + 1:].shape, generator=g).to(b.host[k].dtype)
        b.d[k] = b.host[k].to(b.dev)
    b.fused(); b.done()
    assert torch.equal(a.A_hat[:, :, :t + 1], b.A_hat[:, :, :t + 1])
    assert torch.equal(a.O[:, :, :t + 1], b.O[:, :, :t + 1])


def test_decoder_head_full_size_on_row_windows():
    """The OPT-1.3B-shaped workload with d' = 64, c_s = 2, c_h = 4 (128 channels: the shape the
    benchmark times, both blocks of input channels, two-row pixel tiles): Z for every row of one
    batch element, the estimate on two windows of rows.  A causal layer's row depends on the rows
    above it only, so the oracle's CNN runs on crops: the first rows as they are, later rows with
    six rows of context above them (three layers, two rows each)."""
    from paper_2310_01777_b200.inputs import WORKLOADS
    w = WORKLOADS["opt_1p3b"]
    a = Run(w, d_hidden=64, c_s=2, c_h=4)
    d = a.d
    sea.sea_estimate_decoder(a.shape, a.dec, d["Q"], d["K"], d["V"], d["omega"], a.A_hat, a.Z, a.ws)
    a.done()
    assert bool(torch.isfinite(a.A_hat).all())
    b = w.B - 1
    prm = {k: np64(v) for k, v in a.hp.items()}
    Q, K, V = (np64(a.host[n][b]) for n in ("Q", "K", "V"))
    omega = np64(a.host["omega"])
    Z = np.stack([dec.mlp_mu(dec.performer_cat(Q[h], K[h], V[h], prm["pos_emb"], omega, True), V[h], prm["W_mu"], prm["b_mu"])
                  for h in range(w.H)])
    check_a_hat(a.Z[b].cpu().numpy().reshape(w.H * w.T, -1), Z.reshape(w.H * w.T, -1))
    Z_hat = np.stack([dec.mlp_nu(Z[h], prm["W_nu1"], prm["b_nu1"], prm["W_nu2"], prm["b_nu2"]) for h in range(w.H)])
    image = dec.to_image(Z_hat, a.c_h)
    A = a.A_hat[b].cpu().numpy()
    for lo, hi in ((0, 200), (w.T - 150, w.T)):
        top = max(0, lo - 6)
        ref = dec.cnn_decoder(image[:, top:hi], prm, hi - top, w.Kc, a.c_s, True)[:, lo - top:]
        check_a_hat(A[:, lo:hi].reshape(-1, w.Kc), ref.reshape(-1, w.Kc))


def test_decoder_head_full_size_not_causal():
    """The BERT-base-shaped workload (12 heads: 48 channels in one block of 64; strided first layer,
    four phases of the folded resize): estimate and Z of one batch element, element by element."""
    from paper_2310_01777_b200.inputs import WORKLOADS
    w = WORKLOADS["bert_base"]
    a = Run(w, d_hidden=64, c_s=2, c_h=4)
    d = a.d
    sea.sea_estimate_decoder(a.shape, a.dec, d["Q"], d["K"], d["V"], d["omega"], a.A_hat, a.Z, a.ws)
    a.done()
    b = w.B - 1
    prm = {k: np64(v) for k, v in a.hp.items()}
    Q, K, V = (np64(a.host[n][b]) for n in ("Q", "K", "V"))
    A_ref, Z_ref = dec.decoder_estimate(Q, K, V, np64(a.host["omega"]), prm, w.Kc, a.c_s, a.c_h, False)
    check_a_hat(a.A_hat[b].cpu().numpy().reshape(-1, w.Kc), A_ref.reshape(-1, w.Kc))
    check_a_hat(a.Z[b].cpu().numpy().reshape(w.H * w.T, -1), Z_ref.reshape(w.H * w.T, -1))
