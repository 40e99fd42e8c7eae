"""Tensor-parallel rebuild: plumbing around kv_tp_bind / kv_tp_plan_host.

The paper's rollout engines run TP = 2 / 4 (Sec. 6.1); each rank then rebuilds
its own KV pool (its share of the kv heads) and the ranks exchange two partial
sums per layer.  The library has no collective of its own: the exchange is a
callback.  This module slices a full weight set for one rank and builds the
callback over torch.distributed (NCCL on GPUs); nothing here computes.
"""
from __future__ import annotations

from typing import Dict

from . import binding as kb


def shard_weights(weights: Dict[str, object], shape, shard) -> Dict[str, object]:
    """The rank's slices of a full weight set as contiguous tensors of the local shape: wq/wk/wv and
    wg/wu by rows, wo/wd by columns, their biases alike; norms, per-head gains and the embedding whole."""
    hd = shape.head_dim
    q0, q1 = shard.q_head0 * hd, (shard.q_head0 + shard.n_q_heads) * hd
    k0, k1 = shard.kv_head0 * hd, (shard.kv_head0 + shard.n_kv_heads) * hd
    f0, f1 = shard.ffn0, shard.ffn0 + shard.ffn
    rows = {"wq": (q0, q1), "wk": (k0, k1), "wv": (k0, k1), "wg": (f0, f1), "wu": (f0, f1),
            "bq": (q0, q1), "bk": (k0, k1), "bv": (k0, k1)}
    cols = {"wo": (q0, q1), "wd": (f0, f1)}
    out: Dict[str, object] = {}
    for name, val in weights.items():
        if name in rows:
            a, b = rows[name]
            out[name] = [t[a:b].contiguous() for t in val]
        elif name in cols:
            a, b = cols[name]
            out[name] = [t[:, a:b].contiguous() for t in val]
        else:
            out[name] = val
    return out


class _DevBuf:
    """Lets torch view `count` fp32 values at a raw device address (no copy)."""

    def __init__(self, ptr: int, count: int):
        self.__cuda_array_interface__ = {"shape": (count,), "typestr": "<f4", "data": (ptr, False), "version": 3}


def dist_allreduce(group=None):
    """Callback for kv_tp_bind that sums over a torch.distributed process group (NCCL when the ranks sit
    on GPUs), enqueued on the stream the library passes."""
    import torch
    import torch.distributed as dist

    def allreduce(buf_ptr, count, stream_ptr, _user):
        try:
            t = torch.as_tensor(_DevBuf(buf_ptr, count), device="cuda")
            with torch.cuda.stream(torch.cuda.ExternalStream(stream_ptr or 0)):
                dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
            return 0
        except Exception:
            return 1
    return allreduce


def local_shape(shape, shard):
    """ModelShape of one rank (per-rank head and ffn counts)."""
    import dataclasses
    return dataclasses.replace(shape, n_q_heads=shard.n_q_heads, n_kv_heads=shard.n_kv_heads, ffn=shard.ffn)
