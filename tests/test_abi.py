"""Host-side checks of the C ABI: the library loads, exports every declared symbol, and
rejects bad arguments with status codes before anything is launched (no GPU needed)."""
import ctypes
import os
import re

import pytest

import paper_2310_01777_b200 as sea
from paper_2310_01777_b200 import binding
from paper_2310_01777_b200.build import build_library
from paper_2310_01777_b200.inputs import WORKLOADS

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_library()
    return binding.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "sea.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sea_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert set(binding.EXPORTS) == set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_shape_struct_matches_header():
    assert ctypes.sizeof(binding.SeaShape) == 40


def test_workspace_bytes_and_shape_validation(lib):
    for w in WORKLOADS.values():
        shp = sea.make_shape(w)
        n = sea.sea_workspace_bytes(shp)
        assert n >= 256 + w.rows * 4
    bad = sea.make_shape(WORKLOADS["opt_1p3b"])
    bad.d = 128
    with pytest.raises(sea.SeaError) as e:
        sea.sea_workspace_bytes(bad)
    assert e.value.code == binding.SEA_ERR_UNSUPPORTED
    bad = sea.make_shape(WORKLOADS["opt_1p3b"])
    bad.Kc = 100  # 2048 % 100 != 0
    with pytest.raises(sea.SeaError) as e:
        sea.sea_workspace_bytes(bad)
    assert e.value.code == binding.SEA_ERR_UNSUPPORTED
    bad = sea.make_shape(WORKLOADS["opt_1p3b"])
    bad.k_hat = 129
    with pytest.raises(sea.SeaError) as e:
        sea.sea_workspace_bytes(bad)
    assert e.value.code == binding.SEA_ERR_INVALID_ARG
    bad = sea.make_shape(WORKLOADS["long_32k"])
    bad.B = 64  # rows * k_hat * r exceeds int32
    with pytest.raises(sea.SeaError) as e:
        sea.sea_workspace_bytes(bad)
    assert e.value.code == binding.SEA_ERR_TOO_LARGE


def test_null_and_misaligned_pointers_are_rejected_before_launch(lib):
    shp = sea.make_shape(WORKLOADS["tiny_f32"])
    vp = ctypes.c_void_p
    fake = vp(0x7F0000000000)  # never dereferenced: validation fails first
    odd = vp(0x7F0000000004)
    rc = lib.sea_sparse_attn(ctypes.byref(shp), None, fake, fake, fake, fake, None, fake, None, None, 0, None)
    assert rc == binding.SEA_ERR_INVALID_ARG
    rc = lib.sea_sparse_attn(ctypes.byref(shp), odd, fake, fake, fake, fake, None, fake, None, None, 0, None)
    assert rc == binding.SEA_ERR_INVALID_ARG
    rc = lib.sea_sparse_attn(ctypes.byref(shp), fake, fake, fake, fake, None, None, fake, None, None, 0, None)
    assert rc == binding.SEA_ERR_INVALID_ARG  # neither col_idx nor sel
    rc = lib.sea_topk_mask(ctypes.byref(shp), fake, None, fake, fake, 1024, fake, 16, None)
    assert rc == binding.SEA_ERR_WORKSPACE
    rc = lib.sea_topk_mask(ctypes.byref(shp), fake, None, fake, fake, 2**31, fake, 1 << 40, None)
    assert rc == binding.SEA_ERR_TOO_LARGE
    rc = lib.sea_estimate(ctypes.byref(shp), fake, fake, fake, fake, fake, fake, fake, 1 << 40, None)
    assert rc == binding.SEA_ERR_UNSUPPORTED  # m == 0
    shp2 = sea.make_shape(WORKLOADS["opt_1p3b"])
    rc = lib.sea_attention(ctypes.byref(shp2), fake, fake, fake, None, fake, None, fake, None, None, None,
                           None, 0, None, fake, 1 << 40, None)
    assert rc == binding.SEA_ERR_INVALID_ARG  # estimator needed but omega missing
    rc = lib.sea_attention(ctypes.byref(shp2), fake, fake, fake, fake, fake, None, fake, None, None, None,
                           None, 0, fake, fake, 1 << 40, None)
    assert rc == binding.SEA_ERR_INVALID_ARG  # P without col_idx


def test_grouped_entry_points_reject_bad_arguments_before_launch(lib):
    vp = ctypes.c_void_p
    fake = vp(0x7F0000000000)
    odd = vp(0x7F0000000004)
    shp = sea.make_shape(WORKLOADS["opt_1p3b"])
    rc = lib.sea_topk_mask_grouped(ctypes.byref(shp), fake, None, None, None, 0, fake, 1 << 40, None)
    assert rc == binding.SEA_ERR_INVALID_ARG  # row_ptr is required
    rc = lib.sea_topk_mask_grouped(ctypes.byref(shp), fake, odd, fake, None, 0, fake, 1 << 40, None)
    assert rc == binding.SEA_ERR_INVALID_ARG  # misaligned mask_bits
    rc = lib.sea_topk_mask_grouped(ctypes.byref(shp), fake, None, fake, None, 0, fake, 1024, None)
    assert rc == binding.SEA_ERR_WORKSPACE
    big = sea.make_shape(WORKLOADS["long_32k"].scaled(H=256, T=2048, k_hat=1))  # a position's bit strings: 256 x 65 words > 48 KB
    rc = lib.sea_topk_mask_grouped(ctypes.byref(big), fake, None, fake, None, 0, fake, 1 << 40, None)
    assert rc == binding.SEA_ERR_UNSUPPORTED
    rc = lib.sea_sparse_attn_masked(ctypes.byref(shp), fake, fake, fake, fake, None, None, fake, None, None, 0, None)
    assert rc == binding.SEA_ERR_INVALID_ARG  # no mask
    rc = lib.sea_sparse_attn_masked(ctypes.byref(shp), fake, fake, fake, fake, None, fake, fake, None, None, 0, None)
    assert rc == binding.SEA_ERR_INVALID_ARG  # no workspace, hence per-row kernels, and no col_idx
    rc = lib.sea_attention_grouped(ctypes.byref(shp), fake, fake, fake, fake, fake, None, fake, None, None, None,
                                   None, 0, fake, fake, 1 << 40, None)
    assert rc == binding.SEA_ERR_INVALID_ARG  # P without col_idx
    nc = sea.make_shape(WORKLOADS["bert_base"])  # not causal
    rc = lib.sea_topk_mask_causal_aware(ctypes.byref(nc), fake, None, fake, None, 0, fake, 1 << 40, None)
    assert rc == binding.SEA_ERR_UNSUPPORTED
    rc = lib.sea_topk_mask_causal_aware(ctypes.byref(shp), fake, None, None, None, 0, fake, 1 << 40, None)
    assert rc == binding.SEA_ERR_INVALID_ARG  # row_ptr is required
    rc = lib.sea_attention_causal_aware(ctypes.byref(shp), fake, fake, fake, fake, fake, None, fake, None, None, None,
                                        None, 0, fake, fake, 1 << 40, None)
    assert rc == binding.SEA_ERR_INVALID_ARG  # P without col_idx
    rc = lib.sea_topk_mask_capped(ctypes.byref(shp), 0, fake, None, fake, fake, 1024, fake, 1 << 40, None)
    assert rc == binding.SEA_ERR_INVALID_ARG  # k_star must be positive
    rc = lib.sea_topk_mask_capped(ctypes.byref(shp), 4, fake, None, fake, None, 0, fake, 1 << 40, None)
    assert rc == binding.SEA_ERR_INVALID_ARG  # col_idx is required
    rc = lib.sea_attention_capped(ctypes.byref(shp), 4, fake, fake, fake, fake, fake, None, fake, None, None, None,
                                  None, 0, None, fake, 1 << 40, None)
    assert rc == binding.SEA_ERR_INVALID_ARG  # col_idx is required
    f32 = sea.make_shape(WORKLOADS["tiny_f32"])
    rc = lib.sea_attention_grouped(ctypes.byref(f32), fake, fake, fake, None, None, fake, fake, None, None, None,
                                   None, 0, None, fake, 1 << 40, None)
    assert rc == binding.SEA_ERR_INVALID_ARG  # fp32 runs the per-row kernels, which need col_idx


def test_status_strings(lib):
    assert binding.status_string(0) == "ok"
    assert "workspace" in binding.status_string(binding.SEA_ERR_WORKSPACE)
