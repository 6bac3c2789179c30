"""ctypes binding of libsea.so: the same entry points as include/sea.h, taking torch tensors.

Argument marshalling only: every step of the path runs inside the CUDA library.  There is no
CPU fallback; when the shared library is missing or cannot be loaded every call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from .inputs import Workload

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsea.so")

SEA_OK = 0
SEA_ERR_INVALID_ARG = 1
SEA_ERR_UNSUPPORTED = 2
SEA_ERR_WORKSPACE = 3
SEA_ERR_TOO_LARGE = 4
SEA_ERR_CUDA = 5
SEA_F32 = 0
SEA_BF16 = 1
SEA_DEV_ROW_OVERFLOW = 1
SEA_DEV_NONFINITE = 2
SEA_DEV_TIMEOUT = 4

EXPORTS = (
    "sea_workspace_bytes", "sea_estimate", "sea_topk_mask", "sea_topk_mask_static", "sea_sparse_attn",
    "sea_attention", "sea_topk_mask_grouped", "sea_sparse_attn_masked", "sea_attention_grouped",
    "sea_topk_mask_causal_aware", "sea_attention_causal_aware", "sea_workspace_bytes_capped", "sea_topk_mask_capped",
    "sea_workspace_bytes_decoder", "sea_estimate_decoder", "sea_mix_output", "sea_attention_decoder",
    "sea_attention_capped", "sea_workspace_bytes_resized", "sea_topk_mask_resized", "sea_attention_resized",
    "sea_workspace_host_bytes", "sea_attention_host", "sea_device_status", "sea_last_launch_count",
    "sea_last_sparse_kernel", "sea_last_sparse_flops",
    "sea_status_string",
)


class SeaShape(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("H", ctypes.c_int32), ("T", ctypes.c_int32), ("d", ctypes.c_int32),
        ("m", ctypes.c_int32), ("Kc", ctypes.c_int32), ("k_hat", ctypes.c_int32),
        ("causal", ctypes.c_int32), ("io", ctypes.c_int32), ("scale", ctypes.c_float),
    ]


class SeaDecoder(ctypes.Structure):
    """Mirror of `sea_decoder`: sizes and device pointers of the estimator head's weights."""
    _fields_ = [("d_hidden", ctypes.c_int32), ("c_s", ctypes.c_int32), ("c_h", ctypes.c_int32)] + \
               [(n, ctypes.c_void_p) for n in ("W_mu", "b_mu", "W_nu1", "b_nu1", "W_nu2", "b_nu2", "conv1_w", "conv1_b",
                                               "conv2_w", "conv2_b", "conv3_w", "conv3_b", "pos_emb", "w_prob", "w_mix")] + \
               [("b_prob", ctypes.c_float), ("b_mix", ctypes.c_float)]


class SeaError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (sea_status {code})")


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads libsea.so from the package directory; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2310_01777_b200.build` "
            "(libsea has no CPU fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, sz, i32, i64 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int32, ctypes.c_int64
    shp = ctypes.POINTER(SeaShape)
    lib.sea_workspace_bytes.argtypes = [shp, ctypes.POINTER(sz)]
    lib.sea_workspace_host_bytes.argtypes = [shp, ctypes.POINTER(sz)]
    lib.sea_estimate.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.sea_topk_mask.argtypes = [shp, vp, vp, vp, vp, i64, vp, sz, vp]
    lib.sea_topk_mask_static.argtypes = [shp, vp, vp, vp, vp, i64, vp]
    lib.sea_sparse_attn.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.sea_attention.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i64, vp, vp, sz, vp]
    lib.sea_topk_mask_grouped.argtypes = [shp, vp, vp, vp, vp, i64, vp, sz, vp]
    lib.sea_sparse_attn_masked.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.sea_attention_grouped.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i64, vp, vp, sz, vp]
    lib.sea_topk_mask_causal_aware.argtypes = lib.sea_topk_mask_grouped.argtypes
    lib.sea_attention_causal_aware.argtypes = lib.sea_attention_grouped.argtypes
    lib.sea_workspace_bytes_capped.argtypes = [shp, i32, ctypes.POINTER(sz)]
    lib.sea_topk_mask_capped.argtypes = [shp, i32, vp, vp, vp, vp, i64, vp, sz, vp]
    lib.sea_attention_capped.argtypes = [shp, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i64, vp, vp, sz, vp]
    lib.sea_workspace_bytes_resized.argtypes = [shp, ctypes.POINTER(sz)]
    lib.sea_topk_mask_resized.argtypes = [shp, i32, vp, vp, vp, vp, i64, vp, sz, vp]
    lib.sea_attention_resized.argtypes = [shp, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i64, vp, vp, sz, vp]
    dcp = ctypes.POINTER(SeaDecoder)
    lib.sea_workspace_bytes_decoder.argtypes = [shp, dcp, ctypes.POINTER(sz)]
    lib.sea_estimate_decoder.argtypes = [shp, dcp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.sea_mix_output.argtypes = [shp, dcp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.sea_attention_decoder.argtypes = [shp, dcp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i64, vp, vp, sz, vp]
    lib.sea_attention_host.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.sea_device_status.argtypes = [vp, ctypes.POINTER(i32), i32, vp]
    lib.sea_last_launch_count.argtypes = []
    lib.sea_last_launch_count.restype = i32
    lib.sea_last_sparse_kernel.argtypes = []
    lib.sea_last_sparse_kernel.restype = ctypes.c_char_p
    lib.sea_last_sparse_flops.argtypes = []
    lib.sea_last_sparse_flops.restype = ctypes.c_double
    lib.sea_status_string.argtypes = [ctypes.c_int]
    lib.sea_status_string.restype = ctypes.c_char_p
    for name in EXPORTS:
        fn = getattr(lib, name)
        if name not in ("sea_last_launch_count", "sea_last_sparse_kernel", "sea_last_sparse_flops", "sea_status_string"):
            fn.restype = ctypes.c_int
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().sea_status_string(code).decode()


def make_shape(w: Workload, scale: float = 0.0) -> SeaShape:
    return SeaShape(w.B, w.H, w.T, w.d, w.m, w.Kc, w.k_hat, int(w.causal),
                    SEA_BF16 if w.dtype == "bf16" else SEA_F32, scale)


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("libsea needs contiguous tensors")
    return ctypes.c_void_p(t.data_ptr())


def _stream(device) -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream(device).cuda_stream)


def _check(code: int, where: str):
    if code != SEA_OK:
        raise SeaError(code, where)


def sea_workspace_bytes(shape: SeaShape) -> int:
    out = ctypes.c_size_t(0)
    _check(load_library().sea_workspace_bytes(ctypes.byref(shape), ctypes.byref(out)), "sea_workspace_bytes")
    return out.value


def sea_workspace_bytes_capped(shape: SeaShape, k_star: int) -> int:
    out = ctypes.c_size_t(0)
    _check(load_library().sea_workspace_bytes_capped(ctypes.byref(shape), k_star, ctypes.byref(out)),
           "sea_workspace_bytes_capped")
    return out.value


def sea_workspace_host_bytes(shape: SeaShape) -> int:
    out = ctypes.c_size_t(0)
    _check(load_library().sea_workspace_host_bytes(ctypes.byref(shape), ctypes.byref(out)), "sea_workspace_host_bytes")
    return out.value


def new_workspace(shape: SeaShape, device="cuda:0", host_staging: bool = False) -> torch.Tensor:
    """Device workspace for `shape`, with its status word cleared."""
    n = sea_workspace_host_bytes(shape) if host_staging else sea_workspace_bytes(shape)
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    ws[:256].zero_()
    return ws


def sea_estimate(shape, Q, K, V, omega, W_dec, A_hat, ws):
    _check(load_library().sea_estimate(ctypes.byref(shape), _ptr(Q), _ptr(K), _ptr(V), _ptr(omega),
                                       _ptr(W_dec), _ptr(A_hat), _ptr(ws), ws.numel(), _stream(ws.device)),
           "sea_estimate")


def sea_topk_mask(shape, A_hat, sel, row_ptr, col_idx, ws, nnz_cap: Optional[int] = None):
    if nnz_cap is None:
        nnz_cap = col_idx.numel() if col_idx is not None else 0
    _check(load_library().sea_topk_mask(ctypes.byref(shape), _ptr(A_hat), _ptr(sel), _ptr(row_ptr),
                                        _ptr(col_idx), nnz_cap, _ptr(ws), ws.numel(), _stream(ws.device)),
           "sea_topk_mask")


def sea_topk_mask_static(shape, A_hat, sel, row_ptr, col_idx, nnz_cap: Optional[int] = None):
    """sea_topk_mask for callers without a workspace: scratch lives in a static array of the library."""
    if nnz_cap is None:
        nnz_cap = col_idx.numel() if col_idx is not None else 0
    _check(load_library().sea_topk_mask_static(ctypes.byref(shape), _ptr(A_hat), _ptr(sel), _ptr(row_ptr),
                                               _ptr(col_idx), nnz_cap, _stream(A_hat.device)),
           "sea_topk_mask_static")


def sea_sparse_attn(shape, Q, K, V, row_ptr, col_idx, sel, O, P, ws=None):
    _check(load_library().sea_sparse_attn(ctypes.byref(shape), _ptr(Q), _ptr(K), _ptr(V), _ptr(row_ptr),
                                          _ptr(col_idx), _ptr(sel), _ptr(O), _ptr(P), _ptr(ws),
                                          ws.numel() if ws is not None else 0, _stream(Q.device)),
           "sea_sparse_attn")


def sea_attention(shape, Q, K, V, omega, W_dec, O, ws, A_hat_in=None, A_hat=None, sel=None,
                  row_ptr=None, col_idx=None, P=None, nnz_cap: Optional[int] = None):
    if nnz_cap is None:
        nnz_cap = col_idx.numel() if col_idx is not None else 0
    _check(load_library().sea_attention(ctypes.byref(shape), _ptr(Q), _ptr(K), _ptr(V), _ptr(omega),
                                        _ptr(W_dec), _ptr(A_hat_in), _ptr(O), _ptr(A_hat), _ptr(sel),
                                        _ptr(row_ptr), _ptr(col_idx), nnz_cap, _ptr(P), _ptr(ws),
                                        ws.numel(), _stream(ws.device)),
           "sea_attention")


def sea_topk_mask_grouped(shape, A_hat, mask_bits, row_ptr, col_idx, ws, nnz_cap: Optional[int] = None):
    """Causal-per-batch grouping: mask_bits is an int32 tensor [rows, ceil(Kc/32)] (or None)."""
    if nnz_cap is None:
        nnz_cap = col_idx.numel() if col_idx is not None else 0
    _check(load_library().sea_topk_mask_grouped(ctypes.byref(shape), _ptr(A_hat), _ptr(mask_bits), _ptr(row_ptr),
                                                _ptr(col_idx), nnz_cap, _ptr(ws), ws.numel(), _stream(ws.device)),
           "sea_topk_mask_grouped")


def sea_sparse_attn_masked(shape, Q, K, V, row_ptr, col_idx, mask_bits, O, P, ws=None):
    _check(load_library().sea_sparse_attn_masked(ctypes.byref(shape), _ptr(Q), _ptr(K), _ptr(V), _ptr(row_ptr),
                                                 _ptr(col_idx), _ptr(mask_bits), _ptr(O), _ptr(P), _ptr(ws),
                                                 ws.numel() if ws is not None else 0, _stream(Q.device)),
           "sea_sparse_attn_masked")


def sea_attention_grouped(shape, Q, K, V, omega, W_dec, O, ws, A_hat_in=None, A_hat=None, mask_bits=None,
                          row_ptr=None, col_idx=None, P=None, nnz_cap: Optional[int] = None):
    if nnz_cap is None:
        nnz_cap = col_idx.numel() if col_idx is not None else 0
    _check(load_library().sea_attention_grouped(ctypes.byref(shape), _ptr(Q), _ptr(K), _ptr(V), _ptr(omega),
                                                _ptr(W_dec), _ptr(A_hat_in), _ptr(O), _ptr(A_hat), _ptr(mask_bits),
                                                _ptr(row_ptr), _ptr(col_idx), nnz_cap, _ptr(P), _ptr(ws),
                                                ws.numel(), _stream(ws.device)),
           "sea_attention_grouped")


def sea_topk_mask_causal_aware(shape, A_hat, mask_bits, row_ptr, col_idx, ws, nnz_cap: Optional[int] = None):
    """Per-query selection among the columns a causal row can see; outputs as sea_topk_mask_grouped."""
    if nnz_cap is None:
        nnz_cap = col_idx.numel() if col_idx is not None else 0
    _check(load_library().sea_topk_mask_causal_aware(ctypes.byref(shape), _ptr(A_hat), _ptr(mask_bits), _ptr(row_ptr),
                                                     _ptr(col_idx), nnz_cap, _ptr(ws), ws.numel(), _stream(ws.device)),
           "sea_topk_mask_causal_aware")


def sea_attention_causal_aware(shape, Q, K, V, omega, W_dec, O, ws, A_hat_in=None, A_hat=None, mask_bits=None,
                               row_ptr=None, col_idx=None, P=None, nnz_cap: Optional[int] = None):
    if nnz_cap is None:
        nnz_cap = col_idx.numel() if col_idx is not None else 0
    _check(load_library().sea_attention_causal_aware(ctypes.byref(shape), _ptr(Q), _ptr(K), _ptr(V), _ptr(omega),
                                                     _ptr(W_dec), _ptr(A_hat_in), _ptr(O), _ptr(A_hat),
                                                     _ptr(mask_bits), _ptr(row_ptr), _ptr(col_idx), nnz_cap, _ptr(P),
                                                     _ptr(ws), ws.numel(), _stream(ws.device)),
           "sea_attention_causal_aware")


def sea_topk_mask_capped(shape, k_star: int, A_hat, sel, row_ptr, col_idx, ws, nnz_cap: Optional[int] = None):
    """Per-query selection, each selected column replicated to at most k_star uniformly spaced keys."""
    if nnz_cap is None:
        nnz_cap = col_idx.numel()
    _check(load_library().sea_topk_mask_capped(ctypes.byref(shape), k_star, _ptr(A_hat), _ptr(sel), _ptr(row_ptr),
                                               _ptr(col_idx), nnz_cap, _ptr(ws), ws.numel(), _stream(ws.device)),
           "sea_topk_mask_capped")


def sea_attention_capped(shape, k_star: int, Q, K, V, omega, W_dec, O, ws, col_idx, A_hat_in=None, A_hat=None, sel=None,
                         row_ptr=None, P=None, nnz_cap: Optional[int] = None):
    if nnz_cap is None:
        nnz_cap = col_idx.numel()
    _check(load_library().sea_attention_capped(ctypes.byref(shape), k_star, _ptr(Q), _ptr(K), _ptr(V), _ptr(omega),
                                               _ptr(W_dec), _ptr(A_hat_in), _ptr(O), _ptr(A_hat), _ptr(sel),
                                               _ptr(row_ptr), _ptr(col_idx), nnz_cap, _ptr(P), _ptr(ws), ws.numel(),
                                               _stream(ws.device)),
           "sea_attention_capped")


def sea_workspace_bytes_resized(shape: SeaShape) -> int:
    out = ctypes.c_size_t(0)
    _check(load_library().sea_workspace_bytes_resized(ctypes.byref(shape), ctypes.byref(out)), "sea_workspace_bytes_resized")
    return out.value


def sea_topk_mask_resized(shape, row_widths: bool, A_hat, sel, row_ptr, col_idx, ws, nnz_cap: Optional[int] = None):
    """Nearest-neighbour resize at any ratio of T to Kc; row_widths: causal rows resized to their own width."""
    if nnz_cap is None:
        nnz_cap = col_idx.numel() if col_idx is not None else 0
    _check(load_library().sea_topk_mask_resized(ctypes.byref(shape), int(row_widths), _ptr(A_hat), _ptr(sel), _ptr(row_ptr),
                                                _ptr(col_idx), nnz_cap, _ptr(ws), ws.numel(), _stream(ws.device)),
           "sea_topk_mask_resized")


def sea_attention_resized(shape, row_widths: bool, Q, K, V, omega, W_dec, O, ws, col_idx, A_hat_in=None, A_hat=None,
                          sel=None, row_ptr=None, P=None, nnz_cap: Optional[int] = None):
    if nnz_cap is None:
        nnz_cap = col_idx.numel()
    _check(load_library().sea_attention_resized(ctypes.byref(shape), int(row_widths), _ptr(Q), _ptr(K), _ptr(V),
                                                _ptr(omega), _ptr(W_dec), _ptr(A_hat_in), _ptr(O), _ptr(A_hat), _ptr(sel),
                                                _ptr(row_ptr), _ptr(col_idx), nnz_cap, _ptr(P), _ptr(ws), ws.numel(),
                                                _stream(ws.device)),
           "sea_attention_resized")


def make_decoder(params, d_hidden: int, c_s: int, c_h: int, causal: bool) -> SeaDecoder:
    """`sea_decoder` over the device tensors of `params` (keys as in inputs.make_decoder_params); the
    caller keeps `params` alive while the struct is in use."""
    d = SeaDecoder()
    d.d_hidden, d.c_s, d.c_h = d_hidden, c_s, c_h
    for name in ("W_mu", "b_mu", "W_nu1", "b_nu1", "W_nu2", "b_nu2", "conv1_w", "conv1_b", "conv2_w", "conv2_b", "conv3_w",
                 "conv3_b", "w_prob", "w_mix"):
        t = params[name]
        if not (t.is_cuda and t.is_contiguous() and t.dtype == torch.float32):
            raise ValueError(f"{name}: a contiguous fp32 device tensor is needed")
        setattr(d, name, t.data_ptr())
    d.pos_emb = params["pos_emb"].data_ptr() if causal else None
    d.b_prob, d.b_mix = float(params["b_prob"].reshape(-1)[0]), float(params["b_mix"].reshape(-1)[0])
    return d


def sea_workspace_bytes_decoder(shape: SeaShape, dec: SeaDecoder) -> int:
    out = ctypes.c_size_t(0)
    _check(load_library().sea_workspace_bytes_decoder(ctypes.byref(shape), ctypes.byref(dec), ctypes.byref(out)),
           "sea_workspace_bytes_decoder")
    return out.value


def sea_estimate_decoder(shape, dec, Q, K, V, omega, A_hat, Z, ws):
    _check(load_library().sea_estimate_decoder(ctypes.byref(shape), ctypes.byref(dec), _ptr(Q), _ptr(K), _ptr(V), _ptr(omega),
                                               _ptr(A_hat), _ptr(Z), _ptr(ws), ws.numel(), _stream(ws.device)),
           "sea_estimate_decoder")


def sea_mix_output(shape, dec, Z, A_hat, V, row_ptr, O, P, ws):
    _check(load_library().sea_mix_output(ctypes.byref(shape), ctypes.byref(dec), _ptr(Z), _ptr(A_hat), _ptr(V), _ptr(row_ptr),
                                         _ptr(O), _ptr(P), _ptr(ws), ws.numel(), _stream(ws.device)),
           "sea_mix_output")


def sea_attention_decoder(shape, dec, Q, K, V, omega, O, ws, A_hat=None, sel=None, row_ptr=None, col_idx=None, P=None,
                          nnz_cap: Optional[int] = None):
    if nnz_cap is None:
        nnz_cap = col_idx.numel() if col_idx is not None else 0
    _check(load_library().sea_attention_decoder(ctypes.byref(shape), ctypes.byref(dec), _ptr(Q), _ptr(K), _ptr(V), _ptr(omega),
                                                _ptr(O), _ptr(A_hat), _ptr(sel), _ptr(row_ptr), _ptr(col_idx), nnz_cap, _ptr(P),
                                                _ptr(ws), ws.numel(), _stream(ws.device)),
           "sea_attention_decoder")


def sea_attention_host(shape, hQ, hK, hV, homega, hW_dec, hO, ws):
    """Host tensors in, host O out (copies are part of the call); returns after the stream is idle."""
    for t in (hQ, hK, hV, homega, hW_dec, hO):
        if t.is_cuda:
            raise ValueError("sea_attention_host takes host tensors")
    _check(load_library().sea_attention_host(ctypes.byref(shape), _ptr(hQ), _ptr(hK), _ptr(hV), _ptr(homega),
                                             _ptr(hW_dec), _ptr(hO), _ptr(ws), ws.numel(), _stream(ws.device)),
           "sea_attention_host")


def sea_device_status(ws, clear: bool = True) -> int:
    out = ctypes.c_int32(0)
    _check(load_library().sea_device_status(_ptr(ws), ctypes.byref(out), int(clear), _stream(ws.device)),
           "sea_device_status")
    return out.value


def sea_last_launch_count() -> int:
    return load_library().sea_last_launch_count()


def sea_last_sparse_flops() -> float:
    return load_library().sea_last_sparse_flops()


def sea_last_sparse_kernel() -> str:
    return load_library().sea_last_sparse_kernel().decode()
