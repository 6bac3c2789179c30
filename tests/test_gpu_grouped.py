"""GPU parity of the causal-per-batch grouping (Sec. 3.1 "Grouped Top-k Selection"): libsea's
grouped selection, mask expansion and sparse stage against the fp64 oracle on the same inputs."""
import numpy as np
import pytest
import torch

import paper_2310_01777_b200 as sea
from oracle import sea_oracle as orc
from paper_2310_01777_b200 import binding
from paper_2310_01777_b200.inputs import WORKLOADS, Workload, make_inputs, torch_dtype
from tests.helpers import TOL, check_a_hat, check_float, np64, scale_of

pytestmark = pytest.mark.gpu


def small(name, **kw):
    base = dict(name=name, B=1, H=2, T=128, d=64, m=32, Kc=32, k_hat=4, causal=False, dtype="f32", seed=11)
    base.update(kw)
    return Workload(**base)


class GroupedRun:
    def __init__(self, w: Workload, inputs=None, device="cuda:0", want_P=True, want_col=True):
        self.w, self.dev = w, device
        self.host = inputs if inputs is not None else make_inputs(w)
        self.d = {k: v.to(device) for k, v in self.host.items()}
        self.shape = sea.make_shape(w)
        self.ws = sea.new_workspace(self.shape, device)
        io = torch_dtype(w.dtype)
        self.words = (w.Kc + 31) // 32
        self.O = torch.full((w.B, w.H, w.T, w.d), float("nan"), dtype=io, device=device)
        self.A_hat = (self.d["A_hat"] if "A_hat" in self.d
                      else torch.full((w.B, w.H, w.T, w.Kc), float("nan"), dtype=torch.float32, device=device))
        self.bits = torch.full((w.rows, self.words), -1, dtype=torch.int32, device=device)
        self.row_ptr = torch.full((w.rows + 1,), -1, dtype=torch.int32, device=device)
        self.col_idx = torch.full((w.nnz_cap,), -1, dtype=torch.int32, device=device) if want_col else None
        self.P = torch.full((w.nnz_cap,), float("nan"), dtype=io, device=device) if (want_P and want_col) else None

    def estimate(self):
        sea.sea_estimate(self.shape, self.d["Q"], self.d["K"], self.d["V"], self.d["omega"], self.d["W_dec"],
                         self.A_hat, self.ws)

    def topk(self):
        sea.sea_topk_mask_grouped(self.shape, self.A_hat, self.bits, self.row_ptr, self.col_idx, self.ws)

    def sparse(self, lean_ws=False, with_col=True):
        sea.sea_sparse_attn_masked(self.shape, self.d["Q"], self.d["K"], self.d["V"], self.row_ptr,
                                   self.col_idx if with_col else None, self.bits, self.O, self.P,
                                   self.ws[:256] if lean_ws else self.ws)

    def fused(self):
        given = "A_hat" in self.d
        sea.sea_attention_grouped(self.shape, self.d["Q"], self.d["K"], self.d["V"], self.d.get("omega"),
                                  self.d.get("W_dec"), self.O, self.ws,
                                  A_hat_in=self.A_hat if given else None, A_hat=None if given else self.A_hat,
                                  mask_bits=self.bits, row_ptr=self.row_ptr, col_idx=self.col_idx, P=self.P)

    def status(self):
        return sea.sea_device_status(self.ws)

    def sync(self):
        torch.cuda.synchronize(self.dev)

    def cols_of(self, b, h):
        """Selected columns per query of one head, from the bit strings."""
        w = self.w
        bh = b * w.H + h
        words = self.bits[bh * w.T:(bh + 1) * w.T].cpu().numpy().astype(np.uint32)
        unpacked = np.unpackbits(words.view(np.uint8), axis=1, bitorder="little")[:, :w.Kc]
        return [np.flatnonzero(unpacked[t]) for t in range(w.T)]


def check_batch_against_oracle(run: GroupedRun, b: int, check_estimate: bool):
    w = run.w
    Q, K, V = (np64(run.host[n][b]) for n in ("Q", "K", "V"))
    A = run.A_hat[b].cpu().numpy()
    if check_estimate:
        for h in range(w.H):
            check_a_hat(A[h], orc.estimate_head(Q[h], K[h], V[h], np64(run.host["omega"]), np64(run.host["W_dec"]),
                                                w.causal))
    ref = orc.sea_attention_grouped_batch(Q, K, V, w.k_hat, w.Kc, w.causal, scale_of(w), A_hat=A)
    for h in range(w.H):
        bh = b * w.H + h
        got_cols = run.cols_of(b, h)
        for t in range(w.T):
            assert list(got_cols[t]) == list(ref[h]["cols"][t]), f"selection differs at b={b} h={h} t={t}"
        rp = run.row_ptr[bh * w.T:(bh + 1) * w.T + 1].cpu().numpy().astype(np.int64)
        lo, hi = int(rp[0]), int(rp[-1])
        np.testing.assert_array_equal(rp - lo, ref[h]["row_ptr"])
        if run.col_idx is not None:
            np.testing.assert_array_equal(run.col_idx[lo:hi].cpu().numpy().astype(np.int64), ref[h]["col_idx"])
        check_float(np64(run.O[b, h]), ref[h]["O"], w.dtype, "O")
        if run.P is not None:
            got_p = np64(run.P[lo:hi])
            check_float(got_p, ref[h]["P"], w.dtype, "P")
            sums = np.add.reduceat(np.append(got_p, 0.0), ref[h]["row_ptr"][:-1])
            nonempty = np.diff(ref[h]["row_ptr"]) > 0
            assert np.all(np.abs(sums[nonempty] - 1.0) <= TOL[w.dtype]["row_sum"])
    # padding bits beyond Kc stay clear
    if w.Kc % 32:
        last = run.bits[:, -1].cpu().numpy().astype(np.uint32)
        assert np.all(last >> np.uint32(w.Kc % 32) == 0)


def device_properties(run: GroupedRun):
    """Properties that hold at any size, over every row on the device."""
    w = run.w
    r = w.r
    bits = run.bits.long() & 0xFFFFFFFF
    shifts = torch.arange(32, device=run.dev)
    sel = ((bits[:, :, None] >> shifts) & 1).reshape(w.rows, -1)[:, :w.Kc]  # [rows, Kc] 0/1
    per_pos = sel.reshape(w.B, w.H, w.T, w.Kc).sum(dim=(1, 3))
    assert bool((per_pos == w.H * w.k_hat).all()), "every (b, t) keeps exactly H * k_hat columns"
    i = (torch.arange(w.rows, device=run.dev) % w.T)[:, None]
    c = torch.arange(w.Kc, device=run.dev)[None, :]
    per_col = torch.clamp(i + 1 - c * r, 0, r) if w.causal else torch.full_like(sel, r)
    counts = (sel * per_col).sum(1)
    rp = run.row_ptr.long()
    assert int(rp[0]) == 0
    assert bool((rp[1:] - rp[:-1] == counts).all()), "row_ptr differs from the counts the bits imply"
    nnz = int(rp[-1])
    if run.col_idx is not None:
        row_of = torch.repeat_interleave(torch.arange(w.rows, device=run.dev), counts)
        ci = run.col_idx[:nnz].long()
        assert bool((sel[row_of, ci // r] == 1).all()), "col_idx holds a key of an unselected column"
        same_row = row_of[1:] == row_of[:-1]
        assert bool((ci[1:][same_row] > ci[:-1][same_row]).all()), "col_idx must ascend inside a row"
        if w.causal:
            assert bool((ci <= (row_of % w.T)).all()), "a causal row attends a later key"
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


GROUPED_CASES = [
    small("g_nc_f32", H=3),
    small("g_c_f32", H=4, causal=True, T=96, Kc=32, k_hat=5, m=16),                 # r = 3, per-row kernels
    small("g_one_head", H=1, B=2, causal=True),                                       # reduces to per-query
    small("g_c_bf16_r4", dtype="bf16", B=2, H=3, T=384, Kc=96, k_hat=9, causal=True, m=64),   # tile kernel, 32 columns per tile
    small("g_nc_bf16_r8", dtype="bf16", H=5, T=256, Kc=32, k_hat=3, m=64),           # tile kernel, H not a power of two
    small("g_c_bf16_r16", dtype="bf16", B=2, H=8, T=512, Kc=32, k_hat=4, causal=True, m=128),
    small("g_r128", dtype="bf16", H=4, T=1024, Kc=8, k_hat=2, causal=True),          # a column spans a whole tile
    small("g_full", dtype="bf16", H=2, T=256, Kc=16, k_hat=16, causal=True),         # k_hat = Kc: dense causal attention
    small("g_k1", H=6, T=128, Kc=8, k_hat=1, causal=True),                            # many empty rows
    small("g_wide", dtype="bf16", H=4, T=2048, Kc=512, k_hat=24, causal=True, m=64), # 2048 values per position, 16 words per row
    small("g_many_heads", dtype="bf16", H=32, T=256, Kc=64, k_hat=8, causal=True, m=64),      # 2048 values, 4 groups per thread
    small("g_eight_per_thread", dtype="bf16", H=16, T=2048, Kc=512, k_hat=16, causal=True, m=64),  # 8192 values: 1024 threads x 2 groups
    small("g_two_passes", H=36, T=1024, Kc=1024, k_hat=16, causal=True, m=64),  # 36864 values: more than a CTA's registers hold (fp32 I/O: with one key per column, O is as large as V and bf16 rounding alone would pass the absolute bound)
]


@pytest.mark.parametrize("w", GROUPED_CASES, ids=lambda w: w.name)
def test_grouped_stages_match_oracle(w):
    run = GroupedRun(w)
    run.estimate(); run.topk(); run.sparse(); run.sync()
    assert run.status() == 0
    batches = range(w.B) if w.H * w.T <= 8192 else [w.B - 1]
    for b in batches:
        check_batch_against_oracle(run, b, check_estimate=True)
    device_properties(run)


TILE_GROUPED = [w for w in GROUPED_CASES if w.dtype == "bf16" and w.T % 128 == 0 and w.r >= 4 and w.r & (w.r - 1) == 0
                and w.H * w.T <= 8192]


@pytest.mark.parametrize("w", TILE_GROUPED, ids=lambda w: w.name)
def test_grouped_tile_kernel_and_row_kernels_agree_with_oracle(w):
    """With the full workspace the tile kernel runs (col_idx not needed); with only the status
    word the per-row kernels walk the CSR.  Both are checked against the oracle."""
    run = GroupedRun(w)
    run.estimate(); run.topk(); run.sync()
    for lean, with_col in ((False, False), (True, True)):
        run.O.fill_(float("nan")); run.P.fill_(float("nan"))
        run.sparse(lean_ws=lean, with_col=with_col)
        run.sync()
        assert run.status() == 0
        for b in range(w.B):
            check_batch_against_oracle(run, b, check_estimate=False)
        device_properties(run)


def test_grouped_fused_call_equals_stage_calls_bitwise():
    w = small("g_fused", dtype="bf16", B=2, H=4, T=512, Kc=64, k_hat=6, causal=True, m=64)
    a = GroupedRun(w)
    a.estimate(); a.topk(); a.sparse(); a.sync()
    b = GroupedRun(w)
    b.fused(); b.sync()
    assert a.status() == 0 and b.status() == 0
    for name in ("A_hat", "bits", "row_ptr", "O"):
        assert torch.equal(getattr(a, name), getattr(b, name)), name
    nnz = int(a.row_ptr[-1])
    assert torch.equal(a.col_idx[:nnz], b.col_idx[:nnz])
    assert torch.equal(a.P[:nnz].view(torch.int16), b.P[:nnz].view(torch.int16))
    # outputs other than O are optional
    c = GroupedRun(w, want_P=False, want_col=False)
    sea.sea_attention_grouped(c.shape, c.d["Q"], c.d["K"], c.d["V"], c.d["omega"], c.d["W_dec"], c.O, c.ws)
    c.sync()
    assert torch.equal(a.O, c.O)


def test_grouped_ties_zeros_and_dominating_head():
    """Equal values go to the lower flattened index h * Kc + c; signed zeros tie; a head far above
    the others takes every slot and leaves them empty (O = 0)."""
    w = small("g_ties", H=3, T=64, Kc=16, k_hat=2, m=0)
    host = make_inputs(w)
    g = torch.Generator().manual_seed(5)
    A = torch.round(torch.randn((w.B, w.H, w.T, w.Kc), generator=g) * 1.5) / 2  # many duplicates
    A[0, :, 0, :] = 0.0            # an all-equal position: head 0 takes the first H*k_hat columns
    A[0, 1, 1, :] = -0.0
    A[0, 2, 1, :] = 0.0
    A[0, 0, 1, :] = -1.0
    A[0, 1, 2:10, :] += 100.0      # head 1 dominates positions 2..9
    host["A_hat"] = A.contiguous()
    run = GroupedRun(w, inputs=host)
    run.fused(); run.sync()
    assert run.status() == 0
    check_batch_against_oracle(run, 0, check_estimate=False)
    cols0 = run.cols_of(0, 0)
    assert list(cols0[0]) == list(range(w.H * w.k_hat))
    for h in (0, 2):
        assert bool((run.O[0, h, 2:10] == 0).all())


def test_grouped_ties_across_passes():
    """A position with more values than the CTA keeps in registers (two passes over them) and many
    duplicates: equal values still go to the lower flattened index, whichever pass holds them."""
    w = small("g_ties_stream", H=36, T=1024, Kc=1024, k_hat=16, m=0)
    host = make_inputs(w)
    g = torch.Generator().manual_seed(6)
    A = torch.round(torch.randn((w.B, w.H, w.T, w.Kc), generator=g) * 1.5) / 2
    A[0, :, 0, :] = 0.25           # an all-equal position: the first H * k_hat flattened indices win
    A[0, :, 1, :] = -3.0           # ... and one whose k-th largest value sits far below the largest
    A[0, 35, 1, 1000:] = 7.0
    host["A_hat"] = A.contiguous()
    run = GroupedRun(w, inputs=host)
    run.fused(); run.sync()
    assert run.status() == 0
    check_batch_against_oracle(run, 0, check_estimate=False)
    cols0 = run.cols_of(0, 0)
    assert list(cols0[0]) == list(range(w.H * w.k_hat))


def test_grouped_with_one_head_equals_per_query_calls_bitwise():
    w = small("g_h1", H=1, B=3, dtype="bf16", T=256, Kc=64, k_hat=8, causal=True, m=64)
    a = GroupedRun(w)
    a.fused(); a.sync()
    O = torch.empty_like(a.O)
    row_ptr = torch.empty_like(a.row_ptr)
    col_idx = torch.empty_like(a.col_idx)
    P = torch.empty_like(a.P)
    sea.sea_attention(a.shape, a.d["Q"], a.d["K"], a.d["V"], a.d["omega"], a.d["W_dec"], O, a.ws,
                      row_ptr=row_ptr, col_idx=col_idx, P=P)
    a.sync()
    nnz = int(row_ptr[-1])
    assert torch.equal(row_ptr, a.row_ptr) and torch.equal(col_idx[:nnz], a.col_idx[:nnz])
    assert torch.equal(O, a.O) and torch.equal(P[:nnz].view(torch.int16), a.P[:nnz].view(torch.int16))


def test_grouped_rejects_unsupported_shapes_and_reports_overfull_masks():
    w = small("g_bad", H=2, T=128, Kc=32, k_hat=4, dtype="bf16", m=0)
    run = GroupedRun(w, inputs=make_inputs(w, with_a_hat=True))
    bad = sea.make_shape(w.scaled(Kc=6, T=126))  # Kc % 4 != 0
    with pytest.raises(sea.SeaError) as e:
        sea.sea_topk_mask_grouped(bad, run.A_hat, None, run.row_ptr, None, run.ws)
    assert e.value.code == binding.SEA_ERR_UNSUPPORTED
    # without col_idx the per-row kernels cannot run
    run.topk(); run.sync()
    with pytest.raises(sea.SeaError) as e:
        sea.sea_sparse_attn_masked(run.shape, run.d["Q"], run.d["K"], run.d["V"], run.row_ptr, None, run.bits,
                                   run.O, None, run.ws[:256])
    assert e.value.code == binding.SEA_ERR_INVALID_ARG
    # a mask that keeps more than H * k_hat columns at a position: O is still right (it needs no
    # parking area), the rows beyond the budget are reported and their P entries left alone
    full = GroupedRun(w.scaled(k_hat=w.Kc), inputs=run.host)
    full.topk(); full.sync()                      # every column of every head
    run.bits.copy_(full.bits); run.row_ptr.copy_(full.row_ptr)
    col = full.col_idx
    P = torch.full((full.w.nnz_cap,), float("nan"), dtype=torch.bfloat16, device=run.dev)
    sea.sea_sparse_attn_masked(run.shape, run.d["Q"], run.d["K"], run.d["V"], run.row_ptr, col, run.bits,
                               run.O, P, run.ws)
    run.sync()
    assert run.status() & binding.SEA_DEV_ROW_OVERFLOW
    ref = torch.nn.functional.scaled_dot_product_attention(run.d["Q"].float(), run.d["K"].float(), run.d["V"].float())
    assert float((run.O.float() - ref).abs().max()) <= TOL["bf16"]["max_abs"]


@pytest.mark.parametrize("name", ["opt_1p3b", "opt_125m"])
def test_grouped_full_size_sampled_heads_and_global_properties(name):
    """At the benchmark's size, in the fused launch configuration: properties over every row and
    one batch element's worth of sampled query positions against the oracle."""
    w = WORKLOADS[name]
    run = GroupedRun(w)
    run.fused(); run.sync()
    assert run.status() == 0
    nnz = device_properties(run)
    assert 0 < nnz <= w.nnz_cap
    # selection of sampled positions, against the oracle's ordering of the [H, Kc] slab
    b = w.B - 1
    A = run.A_hat[b].cpu().numpy()
    bits = run.bits.reshape(w.B, w.H, w.T, -1)[b].cpu().numpy().astype(np.uint32)
    for t in (0, 1, 17, w.T // 2 + 3, w.T - 1):
        ref = orc.topk_select_grouped(A[:, t:t + 1, :], w.k_hat)
        for h in range(w.H):
            got = np.flatnonzero(np.unpackbits(bits[h, t].view(np.uint8), bitorder="little")[:w.Kc])
            assert list(got) == list(ref[h][0])
    # O and P of sampled rows of one head, given the device's CSR (already shown to be the mask)
    h = w.H // 2
    bh = b * w.H + h
    Q, K, V = (np64(run.host[n][b, h]) for n in ("Q", "K", "V"))
    rp = run.row_ptr[bh * w.T:(bh + 1) * w.T + 1].cpu().numpy().astype(np.int64)
    for t in (5, 100, w.T // 2, w.T - 1):
        lo, hi = int(rp[t]), int(rp[t + 1])
        cols = run.col_idx[lo:hi].cpu().numpy().astype(np.int64)
        o_ref, p_ref = orc.sparse_attention(Q[t:t + 1], K, V, np.array([0, hi - lo]), cols, scale_of(w))
        check_float(np64(run.O[b, h, t]), o_ref[0], w.dtype, "O")
        check_float(np64(run.P[lo:hi]), p_ref, w.dtype, "P")


# ---------------------------------------------------------------------------------------
# Causal-aware per-query selection: a causal row chooses among the columns it can see.
# ---------------------------------------------------------------------------------------
class AwareRun(GroupedRun):
    def topk(self):
        sea.sea_topk_mask_causal_aware(self.shape, self.A_hat, self.bits, self.row_ptr, self.col_idx, self.ws)

    def fused(self):
        given = "A_hat" in self.d
        sea.sea_attention_causal_aware(self.shape, self.d["Q"], self.d["K"], self.d["V"], self.d.get("omega"),
                                       self.d.get("W_dec"), self.O, self.ws,
                                       A_hat_in=self.A_hat if given else None, A_hat=None if given else self.A_hat,
                                       mask_bits=self.bits, row_ptr=self.row_ptr, col_idx=self.col_idx, P=self.P)


def check_aware_head(run: AwareRun, b: int, h: int):
    w = run.w
    Q, K, V = (np64(run.host[n][b, h]) for n in ("Q", "K", "V"))
    A = run.A_hat[b, h].cpu().numpy()
    cols = orc.topk_select_causal_aware(A, w.k_hat, w.T)
    got = run.cols_of(b, h)
    for t in range(w.T):
        assert list(got[t]) == list(cols[t]), f"selection differs at b={b} h={h} t={t}"
    row_ptr, col_idx = orc.expand_mask(cols, w.T, w.Kc, True)
    O, P = orc.sparse_attention(Q, K, V, row_ptr, col_idx, scale_of(w))
    bh = b * w.H + h
    rp = run.row_ptr[bh * w.T:(bh + 1) * w.T + 1].cpu().numpy().astype(np.int64)
    lo, hi = int(rp[0]), int(rp[-1])
    np.testing.assert_array_equal(rp - lo, row_ptr)
    np.testing.assert_array_equal(run.col_idx[lo:hi].cpu().numpy().astype(np.int64), col_idx)
    check_float(np64(run.O[b, h]), O, w.dtype, "O")
    got_p = np64(run.P[lo:hi])
    check_float(got_p, P, w.dtype, "P")
    sums = np.add.reduceat(np.append(got_p, 0.0), row_ptr[:-1])
    assert np.all(np.abs(sums - 1.0) <= TOL[w.dtype]["row_sum"])  # no row is empty


AWARE_CASES = [
    small("a_f32", H=2, causal=True, T=96, Kc=32, k_hat=5, m=16),                       # r = 3, per-row kernels
    small("a_bf16_r4", dtype="bf16", B=2, H=3, T=384, Kc=96, k_hat=9, causal=True, m=64),
    small("a_bf16_r16", dtype="bf16", H=4, T=512, Kc=32, k_hat=4, causal=True, m=128),
    small("a_k1", dtype="bf16", H=2, T=256, Kc=16, k_hat=1, causal=True),                # one column per row, never empty
    small("a_wide", dtype="bf16", H=2, T=2048, Kc=512, k_hat=24, causal=True, m=64),     # 16 values per lane, histogram path
    small("a_full", dtype="bf16", H=2, T=256, Kc=16, k_hat=16, causal=True),             # dense causal attention
]


@pytest.mark.parametrize("w", AWARE_CASES, ids=lambda w: w.name)
def test_causal_aware_stages_and_fused_call_match_oracle(w):
    a = AwareRun(w)
    a.estimate(); a.topk(); a.sparse(); a.sync()
    assert a.status() == 0
    for b in range(w.B):
        for h in range(w.H):
            check_aware_head(a, b, h)
    counts = (a.row_ptr[1:] - a.row_ptr[:-1])
    assert int(counts.min()) >= 1
    f = AwareRun(w)
    f.fused(); f.sync()
    assert f.status() == 0
    nnz = int(a.row_ptr[-1])
    for name in ("A_hat", "bits", "row_ptr", "O"):
        assert torch.equal(getattr(a, name), getattr(f, name)), name
    assert torch.equal(a.col_idx[:nnz], f.col_idx[:nnz])
    assert torch.equal(a.P[:nnz].view(torch.int16 if w.dtype == "bf16" else torch.int32),
                       f.P[:nnz].view(torch.int16 if w.dtype == "bf16" else torch.int32))


def test_causal_aware_needs_a_causal_shape_and_handles_ties():
    w = small("a_nc", H=1, T=128, Kc=32, k_hat=4, m=0)
    run = AwareRun(w, inputs=make_inputs(w, with_a_hat=True))
    with pytest.raises(sea.SeaError) as e:
        run.topk()
    assert e.value.code == binding.SEA_ERR_UNSUPPORTED
    w = small("a_ties", H=1, T=128, Kc=32, k_hat=4, m=0, causal=True)
    host = make_inputs(w, with_a_hat=True)
    host["A_hat"] = (torch.round(host["A_hat"] * 2) / 2).contiguous()
    host["A_hat"][0, 0, 50, :] = 0.0
    host["A_hat"][0, 0, 51, ::2] = -0.0
    run = AwareRun(w, inputs=host)
    run.fused(); run.sync()
    assert run.status() == 0
    check_aware_head(run, 0, 0)


def test_causal_aware_full_size_properties_and_sampled_rows():
    w = WORKLOADS["opt_1p3b"]
    run = AwareRun(w)
    run.fused(); run.sync()
    assert run.status() == 0
    r = w.r
    bits = run.bits.long() & 0xFFFFFFFF
    shifts = torch.arange(32, device=run.dev)
    sel = ((bits[:, :, None] >> shifts) & 1).reshape(w.rows, -1)[:, :w.Kc]
    i = (torch.arange(w.rows, device=run.dev) % w.T)
    visible = i // r + 1
    assert bool((sel.sum(1) == torch.clamp(visible, max=w.k_hat)).all()), "a row keeps min(k_hat, visible) columns"
    c = torch.arange(w.Kc, device=run.dev)[None, :]
    assert bool(((sel == 0) | (c < visible[:, None])).all()), "a selected column holds no visible key"
    counts = (sel * torch.clamp(i[:, None] + 1 - c * r, 0, r)).sum(1)
    rp = run.row_ptr.long()
    assert bool((rp[1:] - rp[:-1] == counts).all()) and int(counts.min()) >= 1
    b, h = w.B - 1, 5
    A = run.A_hat[b, h].cpu().numpy()
    cols = orc.topk_select_causal_aware(A, w.k_hat, w.T)
    got = run.cols_of(b, h)
    for t in (0, 15, 16, 255, 256, 1000, w.T - 1):
        assert list(got[t]) == list(cols[t])
    Q, K, V = (np64(run.host[n][b, h]) for n in ("Q", "K", "V"))
    bh = b * w.H + h
    rph = run.row_ptr[bh * w.T:(bh + 1) * w.T + 1].cpu().numpy().astype(np.int64)
    for t in (0, 3, 100, w.T - 1):
        lo, hi = int(rph[t]), int(rph[t + 1])
        cidx = run.col_idx[lo:hi].cpu().numpy().astype(np.int64)
        o_ref, p_ref = orc.sparse_attention(Q[t:t + 1], K, V, np.array([0, hi - lo]), cidx, scale_of(w))
        check_float(np64(run.O[b, h, t]), o_ref[0], w.dtype, "O")
        check_float(np64(run.P[lo:hi]), p_ref, w.dtype, "P")
