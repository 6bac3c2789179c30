"""GPU parity of the capped replication for long sequences (App. "Sparse Interpolation": at most
k_star uniformly spaced keys per selected column) against the fp64 oracle."""
import numpy as np
import pytest
import torch

import paper_2310_01777_b200 as sea
from oracle import sea_oracle as orc
from paper_2310_01777_b200 import binding
from paper_2310_01777_b200.inputs import Workload, make_inputs, torch_dtype
from tests.helpers import GpuRun, TOL, check_a_hat, check_float, np64, scale_of

pytestmark = pytest.mark.gpu


def small(name, **kw):
    base = dict(name=name, B=1, H=2, T=256, d=64, m=32, Kc=16, k_hat=1, causal=True, dtype="bf16", seed=17)
    base.update(kw)
    return Workload(**base)


def run_capped(w, k_star, fused, device="cuda:0"):
    run = GpuRun(w, device=device)
    if fused:
        sea.sea_attention_capped(run.shape, k_star, run.d["Q"], run.d["K"], run.d["V"], run.d["omega"], run.d["W_dec"],
                                 run.O, run.ws, run.col_idx, A_hat=run.A_hat, sel=run.sel, row_ptr=run.row_ptr, P=run.P)
    else:
        run.estimate()
        sea.sea_topk_mask_capped(run.shape, k_star, run.A_hat, run.sel, run.row_ptr, run.col_idx, run.ws)
        sea.sea_sparse_attn(run.shape, run.d["Q"], run.d["K"], run.d["V"], run.row_ptr, run.col_idx, None, run.O, run.P,
                            run.ws)
    run.sync()
    assert run.status() == 0
    return run


def check_head(run, b, h, k_star):
    w = run.w
    Q, K, V = (np64(run.host[n][b, h]) for n in ("Q", "K", "V"))
    A = run.A_hat[b, h].cpu().numpy()
    check_a_hat(A, orc.estimate_head(Q, K, V, np64(run.host["omega"]), np64(run.host["W_dec"]), w.causal))
    sel = orc.topk_select(A, w.k_hat)
    bh = b * w.H + h
    np.testing.assert_array_equal(run.sel[bh * w.T:(bh + 1) * w.T].cpu().numpy(), sel)
    row_ptr, col_idx = orc.expand_mask(sel, w.T, w.Kc, w.causal, k_star=k_star)
    O, P = orc.sparse_attention(Q, K, V, row_ptr, col_idx, scale_of(w))
    rp = run.row_ptr[bh * w.T:(bh + 1) * w.T + 1].cpu().numpy().astype(np.int64)
    lo, hi = int(rp[0]), int(rp[-1])
    np.testing.assert_array_equal(rp - lo, row_ptr)
    np.testing.assert_array_equal(run.col_idx[lo:hi].cpu().numpy().astype(np.int64), col_idx)
    check_float(np64(run.O[b, h]), O, w.dtype, "O")
    check_float(np64(run.P[lo:hi]), P, w.dtype, "P")


CASES = [
    (small("cap_k1"), 5),                                            # the paper's case: one column, five of 16 keys
    (small("cap_div", T=512, Kc=8, k_hat=1), 16),                    # k_star divides the run of 64
    (small("cap_nc", causal=False, k_hat=2, H=3), 3),
    (small("cap_f32", dtype="f32", T=192, Kc=16, k_hat=2, m=16), 7),  # r = 12, fp32
    (small("cap_one", T=128, Kc=8), 1),                              # a single key per row
    (small("cap_long", H=1, T=8192, Kc=64, k_hat=1, m=64), 24),      # r = 128, a long row
]


@pytest.mark.parametrize("w,k_star", CASES, ids=[c[0].name for c in CASES])
def test_capped_stages_and_fused_call_match_oracle(w, k_star):
    a = run_capped(w, k_star, fused=False)
    for b in range(w.B):
        for h in range(w.H):
            check_head(a, b, h, k_star)
    f = run_capped(w, k_star, fused=True)
    nnz = int(a.row_ptr[-1])
    for name in ("A_hat", "sel", "row_ptr", "O"):
        assert torch.equal(getattr(a, name), getattr(f, name)), name
    assert torch.equal(a.col_idx[:nnz], f.col_idx[:nnz])
    view = torch.int16 if w.dtype == "bf16" else torch.int32
    assert torch.equal(a.P[:nnz].view(view), f.P[:nnz].view(view))
    if not w.causal:
        assert nnz == w.rows * w.k_hat * k_star


def test_cap_at_or_above_the_run_length_is_the_plain_mask_bitwise():
    w = small("cap_none", T=256, Kc=16, k_hat=3)
    plain = GpuRun(w)
    plain.estimate(); plain.topk_mask(); plain.sync()
    for k_star in (16, 40):
        run = GpuRun(w)
        run.estimate()
        sea.sea_topk_mask_capped(run.shape, k_star, run.A_hat, run.sel, run.row_ptr, run.col_idx, run.ws)
        run.sync()
        nnz = int(plain.row_ptr[-1])
        assert torch.equal(run.row_ptr, plain.row_ptr) and torch.equal(run.col_idx[:nnz], plain.col_idx[:nnz])


def test_capped_rejects_bad_arguments():
    w = small("cap_bad")
    run = GpuRun(w)
    with pytest.raises(sea.SeaError) as e:
        sea.sea_topk_mask_capped(run.shape, 0, run.A_hat, run.sel, run.row_ptr, run.col_idx, run.ws)
    assert e.value.code == binding.SEA_ERR_INVALID_ARG


def test_capped_fused_call_refuses_a_capacity_below_the_largest_mask():
    """The per-row sparse kernels walk col_idx by row_ptr alone: a buffer that the mask could
    overrun is refused on the host and nothing is launched."""
    w = small("cap_short", T=256, Kc=16, k_hat=2)
    k_star = 5
    run = GpuRun(w)
    run.col_idx.fill_(0)
    need = w.rows * w.k_hat * k_star
    with pytest.raises(sea.SeaError) as e:
        sea.sea_attention_capped(run.shape, k_star, run.d["Q"], run.d["K"], run.d["V"], run.d["omega"], run.d["W_dec"],
                                 run.O, run.ws, run.col_idx, row_ptr=run.row_ptr, P=run.P, nnz_cap=need - 1)
    assert e.value.code == binding.SEA_ERR_TOO_LARGE
    run.sync()
    assert bool((run.col_idx == 0).all()) and bool((run.row_ptr == -1).all())
    sea.sea_attention_capped(run.shape, k_star, run.d["Q"], run.d["K"], run.d["V"], run.d["omega"], run.d["W_dec"],
                             run.O, run.ws, run.col_idx, row_ptr=run.row_ptr, P=run.P, nnz_cap=need)
    run.sync()
    assert run.status() == 0 and int(run.row_ptr[-1]) <= need


def test_capped_shape_limit_counts_the_capped_mask():
    """T = 131072 with Kc = 128 and 32 heads: the uncapped mask (rows * r = 2^32 entries) is beyond
    int32, the capped one (rows * 64) is not, and only the capped calls accept the shape."""
    w = Workload(name="cap_131k", B=1, H=32, T=131072, d=64, m=128, Kc=128, k_hat=1, causal=True, dtype="bf16", seed=0)
    shape = sea.make_shape(w)
    lib = binding.load_library()
    import ctypes
    n = ctypes.c_size_t(0)
    assert lib.sea_workspace_bytes(ctypes.byref(shape), ctypes.byref(n)) == binding.SEA_ERR_TOO_LARGE
    assert 0 < sea.sea_workspace_bytes_capped(shape, 64) < 8 << 30
    x = torch.zeros(64, dtype=torch.float32, device="cuda:0")
    i = torch.zeros(64, dtype=torch.int32, device="cuda:0")
    # argument checks run in order: the shape passes (no TOO_LARGE), the tiny workspace is what is refused
    with pytest.raises(sea.SeaError) as e:
        sea.sea_topk_mask_capped(shape, 64, x, i, i, i, x.view(torch.uint8), nnz_cap=64)
    assert e.value.code == binding.SEA_ERR_WORKSPACE
    with pytest.raises(sea.SeaError) as e:
        sea.sea_topk_mask_capped(shape, 2048, x, i, i, i, x.view(torch.uint8), nnz_cap=64)
    assert e.value.code == binding.SEA_ERR_TOO_LARGE
