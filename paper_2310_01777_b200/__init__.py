"""libsea: the SEA attention hot path (estimate -> top-k mask -> sparse attention) for B200.

The compute lives in ``libsea.so`` (CUDA, sm_100a; built by ``paper_2310_01777_b200.build``);
``binding`` exposes its C entry points under the same names.
"""
from . import binding, inputs  # noqa: F401
from .binding import (  # noqa: F401
    SeaDecoder, SeaError, SeaShape, make_decoder, sea_attention_decoder, sea_estimate_decoder, sea_mix_output,
    sea_workspace_bytes_decoder, make_shape, new_workspace, sea_attention, sea_attention_host, sea_attention_grouped, sea_attention_causal_aware, sea_topk_mask_causal_aware,
    sea_attention_capped, sea_topk_mask_capped, sea_attention_resized, sea_topk_mask_resized, sea_workspace_bytes_resized,
    sea_sparse_attn_masked, sea_topk_mask_grouped,
    sea_device_status, sea_estimate, sea_last_launch_count, sea_last_sparse_kernel, sea_last_sparse_flops, sea_sparse_attn, sea_topk_mask, sea_topk_mask_static,
    sea_workspace_bytes, sea_workspace_bytes_capped, sea_workspace_host_bytes,
)
from .inputs import WORKLOADS, Workload, make_inputs  # noqa: F401
