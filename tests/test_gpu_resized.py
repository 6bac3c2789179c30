"""GPU parity of the nearest-neighbour resize at any ratio of T to Kc (App. "Sparse Interpolation")
and of causal rows resized to their own widths (App. "Visualization of intermediate buffers")
against the fp64 oracle."""
import numpy as np
import pytest
import torch

import paper_2310_01777_b200 as sea
from oracle import sea_oracle as orc
from paper_2310_01777_b200 import binding
from paper_2310_01777_b200.inputs import Workload, make_inputs, torch_dtype
from tests.helpers import check_a_hat, check_float, np64, scale_of

pytestmark = pytest.mark.gpu


def small(name, **kw):
    base = dict(name=name, B=1, H=2, T=200, d=64, m=32, Kc=24, k_hat=5, causal=True, dtype="bf16", seed=23)
    base.update(kw)
    return Workload(**base)


class Run:
    def __init__(self, w, device="cuda:0"):
        self.w, self.dev = w, device
        self.host = make_inputs(w)
        self.d = {k: v.to(device) for k, v in self.host.items()}
        self.shape = sea.make_shape(w)
        self.ws = torch.empty(sea.sea_workspace_bytes_resized(self.shape), dtype=torch.uint8, device=device)
        self.ws[:256].zero_()
        io = torch_dtype(w.dtype)
        cap = w.rows * w.k_hat * (-(-w.T // w.Kc))
        self.O = torch.full((w.B, w.H, w.T, w.d), float("nan"), dtype=io, device=device)
        self.A_hat = torch.full((w.B, w.H, w.T, w.Kc), float("nan"), dtype=torch.float32, device=device)
        self.sel = torch.full((w.rows, w.k_hat), -1, dtype=torch.int32, device=device)
        self.row_ptr = torch.full((w.rows + 1,), -1, dtype=torch.int32, device=device)
        self.col_idx = torch.full((cap,), -1, dtype=torch.int32, device=device)
        self.P = torch.full((cap,), float("nan"), dtype=io, device=device)

    def stages(self, row_widths):
        sea.sea_estimate(self.shape, self.d["Q"], self.d["K"], self.d["V"], self.d["omega"], self.d["W_dec"], self.A_hat, self.ws)
        sea.sea_topk_mask_resized(self.shape, row_widths, self.A_hat, self.sel, self.row_ptr, self.col_idx, self.ws)
        sea.sea_sparse_attn(self.shape, self.d["Q"], self.d["K"], self.d["V"], self.row_ptr, self.col_idx, None, self.O, self.P,
                            self.ws[:256])

    def fused(self, row_widths):
        sea.sea_attention_resized(self.shape, row_widths, self.d["Q"], self.d["K"], self.d["V"], self.d["omega"], self.d["W_dec"],
                                  self.O, self.ws, self.col_idx, A_hat=self.A_hat, sel=self.sel, row_ptr=self.row_ptr, P=self.P)

    def done(self):
        torch.cuda.synchronize(self.dev)
        assert sea.sea_device_status(self.ws) == 0


def check_head(run, b, h, row_widths):
    w = run.w
    Q, K, V = (np64(run.host[n][b, h]) for n in ("Q", "K", "V"))
    A = run.A_hat[b, h].cpu().numpy()
    check_a_hat(A, orc.estimate_head(Q, K, V, np64(run.host["omega"]), np64(run.host["W_dec"]), w.causal))
    sel = orc.topk_select(A, w.k_hat)
    bh = b * w.H + h
    np.testing.assert_array_equal(run.sel[bh * w.T:(bh + 1) * w.T].cpu().numpy(), sel)
    row_ptr, col_idx = orc.expand_mask_resized(sel, w.T, w.Kc, w.causal, row_widths)
    O, P = orc.sparse_attention(Q, K, V, row_ptr, col_idx, scale_of(w))
    rp = run.row_ptr[bh * w.T:(bh + 1) * w.T + 1].cpu().numpy().astype(np.int64)
    lo, hi = int(rp[0]), int(rp[-1])
    np.testing.assert_array_equal(rp - lo, row_ptr)
    np.testing.assert_array_equal(run.col_idx[lo:hi].cpu().numpy().astype(np.int64), col_idx)
    check_float(np64(run.O[b, h]), O, w.dtype, "O")
    check_float(np64(run.P[lo:hi]), P, w.dtype, "P")


CASES = [
    (small("rs_ragged"), False),                                         # T / Kc = 8.33: runs of 8 and 9 keys
    (small("rs_ragged_nc", causal=False, T=250, Kc=32, k_hat=7, H=3), False),
    (small("rs_f32", dtype="f32", T=150, Kc=16, k_hat=3, m=16), False),
    (small("rs_exact", T=256, Kc=32, k_hat=6), False),                   # an integer ratio: the plain mask
    (small("rs_rows"), True),                                            # every causal row resized to its own width
    (small("rs_rows_int", T=256, Kc=32, k_hat=6), True),
    (small("rs_rows_many", T=512, Kc=128, k_hat=40, H=1, m=64), True),   # more than 32 selected pixels per row
    (small("rs_rows_f32", dtype="f32", T=130, Kc=16, k_hat=16, m=16), True),  # every pixel selected: dense causal attention
]


@pytest.mark.parametrize("w,row_widths", CASES, ids=[c[0].name for c in CASES])
def test_resized_stages_and_fused_call_match_oracle(w, row_widths):
    a = Run(w)
    a.stages(row_widths); a.done()
    for b in range(w.B):
        for h in range(w.H):
            check_head(a, b, h, row_widths)
    f = Run(w)
    f.fused(row_widths); f.done()
    nnz = int(a.row_ptr[-1])
    for name in ("A_hat", "sel", "row_ptr", "O"):
        assert torch.equal(getattr(a, name), getattr(f, name)), name
    assert torch.equal(a.col_idx[:nnz], f.col_idx[:nnz])
    view = torch.int16 if w.dtype == "bf16" else torch.int32
    assert torch.equal(a.P[:nnz].view(view), f.P[:nnz].view(view))
    if row_widths and w.k_hat == w.Kc:
        assert nnz == w.B * w.H * w.T * (w.T + 1) // 2


def test_integer_ratio_equals_the_plain_mask_bitwise():
    w = small("rs_same", T=256, Kc=32, k_hat=6)
    a = Run(w)
    a.stages(False); a.done()
    sel = torch.empty_like(a.sel); rp = torch.empty_like(a.row_ptr); col = torch.empty_like(a.col_idx)
    ws = sea.new_workspace(a.shape, a.dev)
    sea.sea_topk_mask(a.shape, a.A_hat, sel, rp, col, ws)
    torch.cuda.synchronize()
    nnz = int(rp[-1])
    assert torch.equal(sel, a.sel) and torch.equal(rp, a.row_ptr) and torch.equal(col[:nnz], a.col_idx[:nnz])


def test_resized_argument_checks():
    w = small("rs_bad", causal=False)
    run = Run(w)
    with pytest.raises(sea.SeaError) as e:   # a row's own width is a causal notion
        sea.sea_topk_mask_resized(run.shape, True, run.A_hat, run.sel, run.row_ptr, run.col_idx, run.ws)
    assert e.value.code == binding.SEA_ERR_UNSUPPORTED
    with pytest.raises(sea.SeaError) as e:   # the plain calls still want T % Kc == 0
        sea.sea_workspace_bytes(run.shape)
    assert e.value.code == binding.SEA_ERR_UNSUPPORTED
    with pytest.raises(sea.SeaError) as e:   # a capacity the mask could exceed
        sea.sea_attention_resized(run.shape, False, run.d["Q"], run.d["K"], run.d["V"], run.d["omega"], run.d["W_dec"], run.O,
                                  run.ws, run.col_idx, nnz_cap=run.col_idx.numel() - 1)
    assert e.value.code == binding.SEA_ERR_TOO_LARGE
