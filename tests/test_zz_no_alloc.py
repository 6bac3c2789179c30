"""sea_topk_mask_static: the mask stage for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not an option - a plugin inside an inference
engine whose memory plan is fixed, a serving loop that may not synchronise the device - and have no
workspace to hand over.  The static variant keeps its scratch in an array inside the library.  It
must give exactly the output of sea_topk_mask, on two calls in a row (the array is shared and keeps
the last call's contents), whether this file runs alone or after the rest of the suite.
"""
import pytest
import torch

import paper_2310_01777_b200 as sea
from paper_2310_01777_b200 import binding
from paper_2310_01777_b200.inputs import Workload

pytestmark = pytest.mark.gpu


def run_both(w: Workload, dev="cuda:0"):
    g = torch.Generator().manual_seed(w.seed)
    a_hat = torch.randn((w.B, w.H, w.T, w.Kc), generator=g, dtype=torch.float32)
    a_hat = (torch.round(a_hat * 4) / 4).to(dev)  # quantised: plenty of ties
    shape = sea.make_shape(w)
    out = []
    for static in (False, True):
        sel = torch.full((w.rows, w.k_hat), -1, dtype=torch.int32, device=dev)
        row_ptr = torch.full((w.rows + 1,), -1, dtype=torch.int32, device=dev)
        col_idx = torch.full((w.nnz_cap,), -1, dtype=torch.int32, device=dev)
        if static:
            sea.sea_topk_mask_static(shape, a_hat, sel, row_ptr, col_idx)
        else:
            ws = sea.new_workspace(shape, dev)
            sea.sea_topk_mask(shape, a_hat, sel, row_ptr, col_idx, ws)
        torch.cuda.synchronize()
        out.append((sel, row_ptr, col_idx))
    return out


def test_static_variant_matches_workspace_variant_on_two_calls_in_a_row():
    # first call: causal, several scan tiles; second call: a smaller, non-causal shape, so stale
    # counts and partial sums of the first call sit in the shared array when it starts
    first = Workload("na1", B=2, H=3, T=2048, d=64, m=0, Kc=128, k_hat=16, causal=True, dtype="bf16", seed=21)
    second = Workload("na2", B=1, H=2, T=512, d=64, m=0, Kc=64, k_hat=5, causal=False, dtype="bf16", seed=22)
    third = Workload("na3", B=1, H=5, T=1024, d=64, m=0, Kc=32, k_hat=3, causal=True, dtype="f32", seed=23)
    for w in (first, second, third):
        (sel_a, rp_a, ci_a), (sel_b, rp_b, ci_b) = run_both(w)
        nnz = int(rp_a[-1])
        assert nnz > 0
        assert torch.equal(sel_a, sel_b)
        assert torch.equal(rp_a, rp_b)
        assert torch.equal(ci_a[:nnz], ci_b[:nnz])


def test_static_variant_rejects_what_it_cannot_hold():
    dev = "cuda:0"
    big = Workload("na_big", B=1, H=33, T=32768, d=64, m=0, Kc=2048, k_hat=1, causal=True, dtype="bf16")
    x = torch.zeros(16, dtype=torch.float32, device=dev)  # never touched: the call fails on the host
    i = torch.zeros(16, dtype=torch.int32, device=dev)
    with pytest.raises(sea.SeaError) as e:
        sea.sea_topk_mask_static(sea.make_shape(big), x, i, i, None)
    assert e.value.code == binding.SEA_ERR_TOO_LARGE  # more than 1 048 576 rows
    small = Workload("na_small", B=1, H=1, T=128, d=64, m=0, Kc=32, k_hat=4, causal=True, dtype="bf16")
    with pytest.raises(sea.SeaError) as e:
        sea.sea_topk_mask_static(sea.make_shape(small), x, i, i, i, nnz_cap=16)
    assert e.value.code == binding.SEA_ERR_TOO_LARGE  # col_idx cannot hold every row in full
    with pytest.raises(sea.SeaError) as e:
        sea.sea_topk_mask_static(sea.make_shape(small), x, None, i, None)
    assert e.value.code == binding.SEA_ERR_INVALID_ARG  # sel is required
