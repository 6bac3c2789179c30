"""Seeded synthetic inputs for the SEA attention hot path.

This module only draws random tensors.  It holds none of the method's
arithmetic, so both the CUDA path's tests and the independent CPU oracle's
tests may be fed from it without sharing any computation.

Recipe (one CPU ``torch.Generator`` per workload, seeded, draws in this
order, all in fp32 and then cast once to the I/O dtype):

    Q, K, V   ~ N(0, 1)            [B, H, T, d]
    A_hat     ~ N(0, 1)            [B, H, T, Kc]   (only when the estimate is given)
    omega     ~ N(0, 1)            [m, d]          (FAVOR+ projection, shared by all heads)
    W_dec     ~ N(0, 1/d)          [d, Kc]         (random-init linear decoder head)

The paper's efficiency sweeps are themselves measured on random inputs
(App. Tables A.1/A.2), and its accuracy workloads (GLUE, Wikitext2 with
BERT/OPT weights) are represented here by their layer shapes only.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional

import torch


@dataclass(frozen=True)
class Workload:
    """Shape of one SEA attention call; field names follow the paper's notation.

    ``Kc`` is the paper's compressed width K, ``k_hat`` the number of columns
    kept per row in the compressed space, ``m`` the number of FAVOR+ random
    features (0 when the compressed estimate is supplied by the caller).
    """

    name: str
    B: int
    H: int
    T: int
    d: int
    m: int
    Kc: int
    k_hat: int
    causal: bool
    dtype: str  # "f32" | "bf16"
    seed: int = 0

    @property
    def r(self) -> int:
        return self.T // self.Kc

    @property
    def rows(self) -> int:
        return self.B * self.H * self.T

    @property
    def nnz_cap(self) -> int:
        return self.rows * self.k_hat * self.r

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five workloads named by the benchmark definition.
WORKLOADS: Dict[str, Workload] = {
    "tiny_f32": Workload("tiny_f32", 1, 1, 1024, 64, 0, 128, 16, False, "f32"),
    "bert_base": Workload("bert_base", 32, 12, 512, 64, 64, 128, 32, False, "bf16"),
    "opt_125m": Workload("opt_125m", 8, 12, 2048, 64, 64, 128, 32, True, "bf16"),
    "opt_1p3b": Workload("opt_1p3b", 4, 32, 2048, 64, 128, 128, 16, True, "bf16"),
    "long_8k": Workload("long_8k", 1, 32, 8192, 64, 128, 8192 // 16, 32, True, "bf16"),
    "long_16k": Workload("long_16k", 1, 32, 16384, 64, 128, 16384 // 16, 32, True, "bf16"),
    "long_32k": Workload("long_32k", 1, 32, 32768, 64, 128, 32768 // 16, 32, True, "bf16"),
}


def banded_estimate(w: Workload, width: float = 2.0, sink: bool = True, seed: int = 3) -> torch.Tensor:
    """A compressed estimate [B, H, T, Kc] whose large entries lie in a band of about `width`
    compressed columns around the diagonal (plus, with `sink`, column 0), with a little noise:
    the structure the paper's figures show for trained SEA estimates (diagonal bands, a few
    global columns), which the random-init decoder of the benchmark workloads does not have.
    Only an input recipe: no arithmetic of the method."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    i = torch.arange(w.T, dtype=torch.float32)[:, None] / w.r
    c = torch.arange(w.Kc, dtype=torch.float32)[None, :]
    a = -(c - i).abs() / width + 0.05 * torch.randn((w.B, w.H, w.T, w.Kc), generator=g, dtype=torch.float32)
    if sink:
        a[..., 0] = 10.0
    return a.contiguous()


def make_decoder_params(w: Workload, d_hidden: int = 64, c_s: int = 2, c_h: int = 4, seed: int = 1) -> Dict[str, torch.Tensor]:
    """Random-init weights of the paper's estimator head (MLPs mu and nu, the three convolutions,
    the two scalar heads, and for causal layers the positional embedding that replaces V_I), drawn
    with fan-in scaling so that activations stay of order one.  fp32, except pos_emb which has the
    I/O dtype of V (it is concatenated to V).  Only an input recipe: no arithmetic of the method."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    d, C, Wr = w.d, w.H * c_h, w.Kc // c_s

    def n(shape, std):
        return (torch.randn(shape, generator=g, dtype=torch.float32) * std).contiguous()

    return {
        "W_mu": n((3 * d, d_hidden), (1.0 / (3 * d)) ** 0.5), "b_mu": n((d_hidden,), 0.1),
        "W_nu1": n((d_hidden, d_hidden), (2.0 / d_hidden) ** 0.5), "b_nu1": n((d_hidden,), 0.1),
        "W_nu2": n((d_hidden, Wr * c_h), (2.0 / d_hidden) ** 0.5), "b_nu2": n((Wr * c_h,), 0.1),
        "conv1_w": n((C, C, 3, 3), (2.0 / (9 * C)) ** 0.5), "conv1_b": n((C,), 0.1),
        "conv2_w": n((C, C, 3, 3), (2.0 / (9 * C)) ** 0.5), "conv2_b": n((C,), 0.1),
        "conv3_w": n((w.H, C, 3, 3), (8.0 / (9 * C)) ** 0.5), "conv3_b": n((w.H,), 0.1),
        "pos_emb": torch.randn((w.T, d), generator=g, dtype=torch.float32).to(torch_dtype(w.dtype)).contiguous(),
        "w_prob": n((d_hidden,), (1.0 / d_hidden) ** 0.5), "b_prob": n((1,), 0.5),
        "w_mix": n((d_hidden,), (1.0 / d_hidden) ** 0.5), "b_mix": n((1,), 0.5),
    }


def torch_dtype(name: str) -> torch.dtype:
    if name == "f32":
        return torch.float32
    if name == "bf16":
        return torch.bfloat16
    raise ValueError(f"unknown dtype {name!r}")


def make_inputs(w: Workload, with_a_hat: Optional[bool] = None) -> Dict[str, torch.Tensor]:
    """Draw the host tensors of workload ``w`` (CPU, contiguous).

    ``with_a_hat`` defaults to ``w.m == 0`` (the estimate is an input exactly
    when there is no estimator stage).
    """
    if with_a_hat is None:
        with_a_hat = w.m == 0
    g = torch.Generator(device="cpu")
    g.manual_seed(w.seed)
    io = torch_dtype(w.dtype)
    shape = (w.B, w.H, w.T, w.d)
    out: Dict[str, torch.Tensor] = {}
    for name in ("Q", "K", "V"):
        out[name] = torch.randn(shape, generator=g, dtype=torch.float32).to(io).contiguous()
    if with_a_hat:
        out["A_hat"] = torch.randn((w.B, w.H, w.T, w.Kc), generator=g, dtype=torch.float32)
    if w.m > 0:
        out["omega"] = torch.randn((w.m, w.d), generator=g, dtype=torch.float32)
        out["W_dec"] = torch.randn((w.d, w.Kc), generator=g, dtype=torch.float32) / (w.d ** 0.5)
    return out
