"""Shared harness of the GPU parity tests: runs libsea through its C ABI binding and the
oracle on the same seeded host tensors, and holds the tolerances."""
from __future__ import annotations

import numpy as np
import torch

import paper_2310_01777_b200 as sea
from oracle import sea_oracle as orc
from paper_2310_01777_b200.inputs import Workload, make_inputs, torch_dtype

# Tolerances (benchmark definition): A_hat within 1e-3 relative to the reference's scale, both in
# the max norm and in the Frobenius norm; O and P max-abs 1e-5 in fp32, max-abs 1e-2 and mean-abs
# 1e-3 in bf16; probability rows sum to 1 within 1e-5 (fp32) / 1e-2 (bf16, each entry rounded).
A_HAT_REL = 1e-3
TOL = {"f32": dict(max_abs=1e-5, mean_abs=1e-5, row_sum=1e-5),
       "bf16": dict(max_abs=1e-2, mean_abs=1e-3, row_sum=1e-2)}


def np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


def scale_of(w: Workload) -> float:
    return 1.0 / np.sqrt(w.d)


class GpuRun:
    """Device buffers and outputs of one libsea call chain for a workload."""

    def __init__(self, w: Workload, inputs=None, device="cuda:0", want_P=True, want_col=True):
        self.w = w
        self.dev = device
        self.host = inputs if inputs is not None else make_inputs(w)
        self.d = {k: v.to(device) for k, v in self.host.items()}
        self.shape = sea.make_shape(w)
        self.ws = sea.new_workspace(self.shape, device)
        io = torch_dtype(w.dtype)
        self.O = torch.full((w.B, w.H, w.T, w.d), float("nan"), dtype=io, device=device)
        self.A_hat = (self.d["A_hat"] if "A_hat" in self.d
                      else torch.full((w.B, w.H, w.T, w.Kc), float("nan"), dtype=torch.float32, device=device))
        self.sel = torch.full((w.rows, w.k_hat), -1, dtype=torch.int32, device=device)
        self.row_ptr = torch.full((w.rows + 1,), -1, dtype=torch.int32, device=device)
        self.col_idx = torch.full((w.nnz_cap,), -1, dtype=torch.int32, device=device) if want_col else None
        self.P = torch.full((w.nnz_cap,), float("nan"), dtype=io, device=device) if (want_P and want_col) else None

    # stage by stage ------------------------------------------------------------------
    def estimate(self):
        sea.sea_estimate(self.shape, self.d["Q"], self.d["K"], self.d["V"], self.d["omega"],
                         self.d["W_dec"], self.A_hat, self.ws)

    def topk_mask(self):
        sea.sea_topk_mask(self.shape, self.A_hat, self.sel, self.row_ptr, self.col_idx, self.ws)

    def sparse_attn(self, use_sel=True, lean_ws=False):
        """With the full workspace the stage may run its tensor-core tile kernel; with only the
        status word (``lean_ws``) it runs the per-row kernels."""
        sea.sea_sparse_attn(self.shape, self.d["Q"], self.d["K"], self.d["V"], self.row_ptr, self.col_idx,
                            self.sel if use_sel else None, self.O, self.P,
                            self.ws[:256] if lean_ws else self.ws)

    # the fused call ------------------------------------------------------------------
    def attention(self):
        given = "A_hat" in self.d
        sea.sea_attention(self.shape, self.d["Q"], self.d["K"], self.d["V"], self.d.get("omega"),
                          self.d.get("W_dec"), self.O, self.ws,
                          A_hat_in=self.A_hat if given else None, A_hat=None if given else self.A_hat,
                          sel=self.sel, row_ptr=self.row_ptr, col_idx=self.col_idx, P=self.P)

    def status(self) -> int:
        return sea.sea_device_status(self.ws)

    def sync(self):
        torch.cuda.synchronize(self.dev)


def head_slices(run: GpuRun, b: int, h: int):
    """Host fp64 views of one head's inputs and GPU outputs."""
    w = run.w
    bh = b * w.H + h
    rows = slice(bh * w.T, (bh + 1) * w.T)
    rp = run.row_ptr[bh * w.T:(bh + 1) * w.T + 1].cpu().numpy().astype(np.int64)
    lo, hi = int(rp[0]), int(rp[-1])
    out = dict(
        Q=np64(run.host["Q"][b, h]), K=np64(run.host["K"][b, h]), V=np64(run.host["V"][b, h]),
        A_hat=run.A_hat[b, h].cpu().numpy(),  # fp32, as the GPU produced or was given it
        O=np64(run.O[b, h]), sel=run.sel[rows].cpu().numpy().astype(np.int64),
        row_ptr=rp - lo,
        col_idx=run.col_idx[lo:hi].cpu().numpy().astype(np.int64) if run.col_idx is not None else None,
        P=np64(run.P[lo:hi]) if run.P is not None else None, nnz_base=lo)
    return out


def check_a_hat(got: np.ndarray, ref: np.ndarray):
    diff = got.astype(np.float64) - ref
    assert np.max(np.abs(diff)) <= A_HAT_REL * np.max(np.abs(ref)), (
        f"A_hat max err {np.max(np.abs(diff)):.3e} vs scale {np.max(np.abs(ref)):.3e}")
    assert np.linalg.norm(diff) <= A_HAT_REL * np.linalg.norm(ref), (
        f"A_hat Frobenius rel err {np.linalg.norm(diff) / np.linalg.norm(ref):.3e}")


def check_float(got: np.ndarray, ref: np.ndarray, dtype: str, what: str):
    t = TOL[dtype]
    if ref.size == 0:
        assert got.size == 0
        return
    diff = np.abs(got - ref)
    assert np.all(np.isfinite(got)), f"{what}: non-finite values"
    assert diff.max() <= t["max_abs"], f"{what}: max-abs {diff.max():.3e} > {t['max_abs']}"
    assert diff.mean() <= t["mean_abs"], f"{what}: mean-abs {diff.mean():.3e} > {t['mean_abs']}"


def check_head_against_oracle(run: GpuRun, b: int, h: int, check_estimate: bool):
    """Element-by-element parity of one head: A_hat (tolerance), mask (bit-exact given the GPU's
    A_hat), O and P (tolerance, on the oracle's mask, which must equal the GPU's)."""
    w = run.w
    g = head_slices(run, b, h)
    if check_estimate:
        ref_a = orc.estimate_head(g["Q"], g["K"], g["V"], np64(run.host["omega"]), np64(run.host["W_dec"]),
                                  w.causal)
        check_a_hat(g["A_hat"], ref_a)
    ref = orc.sea_attention_head(g["Q"], g["K"], g["V"], w.k_hat, w.Kc, w.causal, scale_of(w),
                                 A_hat=g["A_hat"])
    np.testing.assert_array_equal(g["sel"], ref["sel"])
    np.testing.assert_array_equal(g["row_ptr"], ref["row_ptr"])
    if g["col_idx"] is not None:
        np.testing.assert_array_equal(g["col_idx"], ref["col_idx"])
    check_float(g["O"], ref["O"], w.dtype, "O")
    if g["P"] is not None:
        check_float(g["P"], ref["P"], w.dtype, "P")
        sums = np.add.reduceat(np.append(g["P"], 0.0), ref["row_ptr"][:-1])
        nonempty = np.diff(ref["row_ptr"]) > 0
        assert np.all(np.abs(sums[nonempty] - 1.0) <= TOL[w.dtype]["row_sum"])
    return ref


def global_mask_properties(run: GpuRun):
    """Properties that hold at any size, checked over every row on the device."""
    w = run.w
    r = w.r
    sel = run.sel.long()
    assert int(sel.min()) >= 0 and int(sel.max()) < w.Kc
    if w.k_hat > 1:
        assert bool((sel[:, 1:] > sel[:, :-1]).all()), "sel must be strictly ascending"
    i = torch.arange(w.rows, device=run.dev) % w.T
    if w.causal:
        counts = torch.clamp(i[:, None] + 1 - sel * r, 0, r).sum(1)
    else:
        counts = torch.full((w.rows,), w.k_hat * r, device=run.dev, dtype=torch.long)
    rp = run.row_ptr.long()
    assert int(rp[0]) == 0
    assert bool((rp[1:] - rp[:-1] == counts).all()), "row_ptr differs from the counts implied by sel"
    nnz = int(rp[-1])
    if run.col_idx is not None:
        row_of = torch.repeat_interleave(torch.arange(w.rows, device=run.dev), counts)
        pos = torch.arange(nnz, device=run.dev) - rp[row_of]
        expect = sel[row_of, pos // r] * r + pos % r
        assert bool((run.col_idx[:nnz].long() == expect).all()), "col_idx is not the expansion of sel"
        if w.causal:
            assert bool((run.col_idx[:nnz].long() <= i[row_of]).all()), "a causal row attends a later key"
        if run.P is not None:
            sums = torch.zeros(w.rows, device=run.dev, dtype=torch.float32)
            sums.index_add_(0, row_of, run.P[:nnz].float())
            ok = (sums - 1).abs() <= TOL[w.dtype]["row_sum"]
            assert bool(ok[counts > 0].all()), "a probability row does not sum to 1"
    empty = counts == 0
    if bool(empty.any()):
        assert bool((run.O.reshape(w.rows, w.d)[empty] == 0).all()), "an empty row must give O = 0"
    assert bool(torch.isfinite(run.O.float()).all())
    return nnz
