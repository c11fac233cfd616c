"""Host-side views of a synthetic layer for the oracle (test infrastructure).

Copies the bf16 bits of a layer's KV buffers to the host and wraps them, with
the layer's strides, in the oracle's descriptor. Works on any object with the
fields of the synthetic LayerKV; holds no arithmetic."""
from __future__ import annotations

import numpy as np
import torch

from . import KV


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 array with the same bits; 8-bit tensors (fp8 codes) -> uint8 (host copy)."""
    if t.element_size() == 1:
        return t.detach().contiguous().view(torch.uint8).cpu().numpy()
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def _host_bits(t: torch.Tensor, keep):
    for buf in keep:
        if buf.untyped_storage().data_ptr() == t.untyped_storage().data_ptr():
            return bits(buf.detach().reshape(-1)), t.storage_offset() - buf.storage_offset()
    return bits(t.detach().contiguous().reshape(-1)), 0


def kv_from_layer(layer) -> KV:
    kb, koff = _host_bits(layer.k, layer.keep)
    if layer.v.untyped_storage().data_ptr() == layer.k.untyped_storage().data_ptr():
        vb, voff = kb, layer.v.storage_offset() - layer.keep[0].storage_offset()
    else:
        vb, voff = _host_bits(layer.v, layer.keep)
    return KV(
        k=kb, v=vb, k_offset=koff, v_offset=voff, batch=layer.batch,
        num_q_heads=layer.num_q_heads, num_kv_heads=layer.num_kv_heads, head_dim=layer.head_dim,
        ctx_lens=layer.ctx_lens.cpu().numpy().astype(np.int32),
        stride_b=layer.stride_b, stride_pos=layer.stride_pos, stride_head=layer.stride_head,
        stride_page=layer.stride_page,
        page_table=None if layer.page_table is None else layer.page_table.cpu().numpy(),
        page_size=layer.page_size, max_pages_per_seq=layer.max_pages_per_seq,
        sm_scale=layer.sm_scale, kv_dtype=getattr(layer, "kv_dtype", 0),
        k_scale=None if getattr(layer, "k_scale", None) is None else layer.k_scale.cpu().numpy(),
        v_scale=None if getattr(layer, "v_scale", None) is None else layer.v_scale.cpu().numpy())
