"""ctypes binding of libkvrebuild.so: argument marshalling only.

Every function has the name and meaning of the C entry point in
include/kvrebuild.h.  Nothing here computes: torch supplies device memory and
streams, numpy the host arrays.  If the shared library is missing the import
of this module fails loudly; there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libkvrebuild.so")

KVR_OK = 0
STATUS = {0: "KVR_OK", -1: "KVR_ERR_INVALID_ARG", -2: "KVR_ERR_NOT_BOUND", -3: "KVR_ERR_UNSUPPORTED",
          -4: "KVR_ERR_BLOCK_OOB", -5: "KVR_ERR_TABLE_TOO_SHORT", -6: "KVR_ERR_ALIAS_CONFLICT",
          -7: "KVR_ERR_TOKEN_OOB", -8: "KVR_ERR_WORKSPACE", -9: "KVR_ERR_CUDA", -10: "KVR_ERR_DEVICE_TIMEOUT"}
KVR_BF16, KVR_FP32 = 0, 1
KINDS = ("rope_table", "embed_rmsnorm", "rmsnorm", "qkv_gemm", "attention", "o_gemm", "gateup_gemm", "down_gemm")

EXPORTS = ("kv_ctx_create", "kv_ctx_destroy", "kv_arena_bind", "kv_weights_bind", "kv_workspace_bytes",
           "kv_workspace_bind", "kv_rebuild", "kv_readback", "kv_readback_dev", "kv_sync_status",
           "kv_check_inputs", "kv_debug_slot_map", "kv_debug_plan", "kv_debug_profile", "kv_set_option", "kv_debug_gemm",
           "kv_status_str", "kv_readback_noalloc", "kv_arena_flush", "kv_health_probe", "kv_resume_logits", "kv_rebuild_from",
           "kv_variant_bind", "kv_plan_host", "kv_tp_bind", "kv_tp_plan_host")


class kv_model_desc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "ffn", "vocab")] \
        + [("rms_eps", C.c_float), ("rope_base", C.c_float), ("dtype", C.c_int32)]


class kv_arena_geometry(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("block_size", "num_blocks", "n_layers", "n_kv_heads", "head_dim", "dtype")]


_PP = C.POINTER(C.c_void_p)


class kv_weights(C.Structure):
    _fields_ = [("embed", C.c_void_p)] + [(n, _PP) for n in ("ln1", "wq", "wk", "wv", "wo", "ln2", "wg", "wu", "wd")]


class kv_proj_variant(C.Structure):
    _fields_ = [(n, _PP) for n in ("bq", "bk", "bv", "q_norm", "k_norm")]


ALLREDUCE_FN = C.CFUNCTYPE(C.c_int, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p)


class kv_tp_config(C.Structure):
    _fields_ = [("tp_world", C.c_int32), ("tp_rank", C.c_int32), ("allreduce", ALLREDUCE_FN), ("user", C.c_void_p)]


class kv_tp_shard(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("q_head0", "n_q_heads", "kv_head0", "n_kv_heads", "ffn0", "ffn")]


class KvrError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: {STATUS.get(status, status)}")
        self.status = status


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2608_14635_b200.build` "
                          "(there is no fallback implementation)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    ip = C.POINTER(C.c_int32)
    sig = {
        "kv_ctx_create": (C.c_int, [C.POINTER(vp), C.c_int]),
        "kv_ctx_destroy": (C.c_int, [vp]),
        "kv_arena_bind": (C.c_int, [vp, vp, sz, C.POINTER(kv_arena_geometry)]),
        "kv_weights_bind": (C.c_int, [vp, C.POINTER(kv_model_desc), C.POINTER(kv_weights)]),
        "kv_variant_bind": (C.c_int, [vp, C.POINTER(kv_proj_variant)]),
        "kv_workspace_bytes": (sz, [vp, i64, i32, i32]),
        "kv_workspace_bind": (C.c_int, [vp, vp, sz, i64, i32, i32]),
        "kv_rebuild": (C.c_int, [vp, C.POINTER(kv_weights), ip, ip, ip, i32, i32, vp]),
        "kv_rebuild_from": (C.c_int, [vp, C.POINTER(kv_weights), ip, ip, ip, ip, i32, i32, vp]),
        "kv_readback": (C.c_int, [vp, i32, ip, i32, vp, vp, vp]),
        "kv_readback_dev": (C.c_int, [vp, i32, ip, i32, vp, vp, vp]),
        "kv_sync_status": (C.c_int, [vp, vp]),
        "kv_check_inputs": (C.c_int, [ip, ip, ip, i32, i32, i32, i32, i32]),
        "kv_plan_host": (C.c_int, [ip, ip, ip, i32, i32, i32, i32, i64, i32, ip, C.POINTER(C.c_int64),
                                   C.POINTER(C.c_int64), C.POINTER(C.c_int64)]),
        "kv_debug_slot_map": (C.c_int, [vp, C.POINTER(C.c_int64), i64]),
        "kv_debug_plan": (C.c_int, [vp, C.POINTER(C.c_int64), C.POINTER(C.c_int64), C.POINTER(C.c_int64)]),
        "kv_debug_profile": (C.c_int, [vp, C.POINTER(C.c_double), C.POINTER(C.c_int64)]),
        "kv_set_option": (C.c_int, [vp, C.c_char_p, i64]),
        "kv_debug_gemm": (C.c_int, [vp, i32, vp, vp, vp, i32, i32, i32, vp]),
        "kv_status_str": (C.c_char_p, [C.c_int]),
        "kv_arena_flush": (C.c_int, [vp, C.c_uint32, vp]),
        "kv_resume_logits": (C.c_int, [vp, vp, vp, vp, vp]),
        "kv_health_probe": (C.c_int, [vp, C.c_uint32, i32, C.POINTER(C.c_uint32), vp]),
        "kv_readback_noalloc": (C.c_int, [vp, C.POINTER(kv_arena_geometry), i32, ip, i32, vp, vp, vp]),
        "kv_tp_bind": (C.c_int, [vp, C.POINTER(kv_tp_config)]),
        "kv_tp_plan_host": (C.c_int, [C.POINTER(kv_model_desc), i32, i32, C.POINTER(kv_model_desc),
                                      C.POINTER(kv_tp_shard)]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    return lib


lib = _load()


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _ip(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_int32))


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream or None
    return getattr(stream, "cuda_stream", stream) or None


def kv_status_str(status: int) -> str:
    return lib.kv_status_str(status).decode()


def kv_check_inputs(tokens, lens, tables, block_size: int, num_blocks: int, vocab: int) -> int:
    tokens, lens, tables = _i32(tokens), _i32(lens), _i32(tables)
    width = tables.shape[1] if tables.ndim == 2 else 0
    return lib.kv_check_inputs(_ip(tokens), _ip(lens), _ip(tables), len(lens), width, block_size, num_blocks, vocab)


def kv_plan_host(lens, tables, block_size: int, chunk_tokens: int, tile_rows: int, valid_lens=None,
                 keep_last_hidden: bool = False):
    """Host-only plan of a rebuild: -> (status, skip[R], computed tokens, chunks, attention tiles)."""
    lens, tables = _i32(lens), _i32(tables)
    width = tables.shape[1] if tables.ndim == 2 else 0
    vl = _i32(valid_lens) if valid_lens is not None else None
    skip = np.zeros(len(lens), dtype=np.int32)
    computed, chunks, tiles = C.c_int64(0), C.c_int64(0), C.c_int64(0)
    st = lib.kv_plan_host(_ip(lens), _ip(vl) if vl is not None else None, _ip(tables), len(lens), width, block_size,
                          int(keep_last_hidden), chunk_tokens, tile_rows, _ip(skip), C.byref(computed),
                          C.byref(chunks), C.byref(tiles))
    return st, skip, computed.value, chunks.value, tiles.value


def kv_tp_plan_host(shape, dtype: int, tp_world: int, tp_rank: int):
    """Host-only partition plan -> (status, local kv_model_desc, kv_tp_shard)."""
    full = make_desc(shape, dtype)
    local, shard = kv_model_desc(), kv_tp_shard()
    st = lib.kv_tp_plan_host(C.byref(full), tp_world, tp_rank, C.byref(local), C.byref(shard))
    return st, local, shard


def kv_readback_noalloc(arena, geom: kv_arena_geometry, layer: int, table, n_tokens: int, stream=None):
    """Allocation-free read-back (no context, no workspace): -> (status, K, V) as host numpy arrays.
    For callers that must not allocate device or pinned memory; at most 2 MiB of K and of V per call."""
    dt = np.float32 if geom.dtype == KVR_FP32 else np.uint16
    k = np.zeros((n_tokens, geom.n_kv_heads, geom.head_dim), dtype=dt)
    v = np.zeros_like(k)
    table = _i32(table)
    st = lib.kv_readback_noalloc(arena.data_ptr(), C.byref(geom), layer, _ip(table), n_tokens, k.ctypes.data,
                                 v.ctypes.data, _stream_ptr(stream))
    return st, k, v


def make_desc(shape, dtype: int) -> kv_model_desc:
    return kv_model_desc(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                         shape.ffn, shape.vocab, shape.rms_eps, shape.rope_base, dtype)


class Context:
    """One kvr_ctx.  Methods are the C calls; tensors passed in are kept alive
    by the object because the library only stores their addresses."""

    def __init__(self, device: int = 0):
        self._h = C.c_void_p()
        self.device = device
        st = lib.kv_ctx_create(C.byref(self._h), device)
        if st != KVR_OK:
            raise KvrError(st, "kv_ctx_create")
        self._keep: Dict[str, object] = {}
        self.geom: Optional[kv_arena_geometry] = None
        self.desc: Optional[kv_model_desc] = None

    def close(self):
        if self._h:
            lib.kv_ctx_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # --- binding calls -------------------------------------------------
    def kv_arena_bind(self, arena, block_size: int, num_blocks: int, n_layers: int, n_kv_heads: int,
                      head_dim: int, dtype: int, nbytes: Optional[int] = None) -> int:
        g = kv_arena_geometry(block_size, num_blocks, n_layers, n_kv_heads, head_dim, dtype)
        nbytes = arena.numel() * arena.element_size() if nbytes is None else nbytes
        st = lib.kv_arena_bind(self._h, arena.data_ptr(), nbytes, C.byref(g))
        if st == KVR_OK:
            self._keep["arena"] = arena
            self.geom = g
        return st

    def kv_weights_bind(self, shape, weights: Dict[str, object], dtype: int) -> int:
        d = make_desc(shape, dtype)
        L = shape.n_layers
        arrs = {}
        w = kv_weights()
        w.embed = weights["embed"].data_ptr()
        for n in ("ln1", "wq", "wk", "wv", "wo", "ln2", "wg", "wu", "wd"):
            arr = (C.c_void_p * L)(*[t.data_ptr() for t in weights[n][:L]])
            arrs[n] = arr
            setattr(w, n, C.cast(arr, _PP))
        st = lib.kv_weights_bind(self._h, C.byref(d), C.byref(w))
        if st == KVR_OK:
            self._keep["weights"] = weights
            self.desc = d
        return st

    def kv_variant_bind(self, weights: Optional[Dict[str, object]]) -> int:
        """Optional projection terms taken from `weights`: 'bq', 'bk', 'bv' and/or
        'qn', 'kn' (lists of per-layer tensors); None or a set without them clears."""
        if weights is None:
            return lib.kv_variant_bind(self._h, None)
        L = self.desc.n_layers
        v = kv_proj_variant()
        arrs = {}
        for field, key in (("bq", "bq"), ("bk", "bk"), ("bv", "bv"), ("q_norm", "qn"), ("k_norm", "kn")):
            if weights.get(key) is not None:
                arr = (C.c_void_p * L)(*[t.data_ptr() for t in weights[key][:L]])
                arrs[field] = arr
                setattr(v, field, C.cast(arr, _PP))
        st = lib.kv_variant_bind(self._h, C.byref(v))
        if st == KVR_OK:
            self._keep["variant"] = weights
        return st

    def kv_tp_bind(self, tp_world: int, tp_rank: int, allreduce) -> int:
        """`allreduce(buf_ptr, count, stream_ptr, user) -> int` is a Python callable (or None with
        tp_world 1): it must enqueue an in-place fp32 sum over the ranks on the given stream."""
        if tp_world <= 1:
            self._keep.pop("tp_cb", None)
            return lib.kv_tp_bind(self._h, None)
        cb = ALLREDUCE_FN(allreduce)
        cfg = kv_tp_config(tp_world, tp_rank, cb, None)
        st = lib.kv_tp_bind(self._h, C.byref(cfg))
        if st == KVR_OK:
            self._keep["tp_cb"] = cb          # the library keeps the function pointer
        return st

    def kv_workspace_bytes(self, max_chunk_tokens: int, max_requests: int, max_blocks_per_req: int) -> int:
        return int(lib.kv_workspace_bytes(self._h, max_chunk_tokens, max_requests, max_blocks_per_req))

    def kv_workspace_bind(self, ws, max_chunk_tokens: int, max_requests: int, max_blocks_per_req: int,
                          nbytes: Optional[int] = None) -> int:
        nbytes = ws.numel() * ws.element_size() if nbytes is None else nbytes
        st = lib.kv_workspace_bind(self._h, ws.data_ptr(), nbytes, max_chunk_tokens, max_requests,
                                   max_blocks_per_req)
        if st == KVR_OK:
            self._keep["ws"] = ws
        return st

    def kv_rebuild(self, tokens, lens, tables, stream=None) -> int:
        tokens, lens, tables = _i32(tokens), _i32(lens), _i32(tables)
        width = tables.shape[1] if tables.ndim == 2 else 0
        return lib.kv_rebuild(self._h, None, _ip(tokens), _ip(lens), _ip(tables), len(lens), width,
                              _stream_ptr(stream))

    def kv_rebuild_from(self, tokens, lens, valid_lens, tables, stream=None) -> int:
        tokens, lens, valid_lens, tables = _i32(tokens), _i32(lens), _i32(valid_lens), _i32(tables)
        width = tables.shape[1] if tables.ndim == 2 else 0
        return lib.kv_rebuild_from(self._h, None, _ip(tokens), _ip(lens), _ip(valid_lens), _ip(tables), len(lens),
                                   width, _stream_ptr(stream))

    def kv_readback(self, layer: int, table, n_tokens: int, stream=None):
        """-> (status, K, V) with K, V host numpy arrays [n, Hkv, hd] (uint16 bf16 patterns or float32)."""
        g = self.geom
        dt = np.float32 if g.dtype == KVR_FP32 else np.uint16
        k = np.zeros((n_tokens, g.n_kv_heads, g.head_dim), dtype=dt)
        v = np.zeros_like(k)
        table = _i32(table)
        st = lib.kv_readback(self._h, layer, _ip(table), n_tokens, k.ctypes.data, v.ctypes.data, _stream_ptr(stream))
        return st, k, v

    def kv_readback_dev(self, layer: int, table, n_tokens: int, k_out, v_out, stream=None) -> int:
        table = _i32(table)
        return lib.kv_readback_dev(self._h, layer, _ip(table), n_tokens, k_out.data_ptr(), v_out.data_ptr(),
                                   _stream_ptr(stream))

    def kv_resume_logits(self, final_gain, lm_head, logits_out, stream=None) -> int:
        return lib.kv_resume_logits(self._h, final_gain.data_ptr(), lm_head.data_ptr(), logits_out.data_ptr(),
                                    _stream_ptr(stream))

    def kv_arena_flush(self, fill_word: int, stream=None) -> int:
        return lib.kv_arena_flush(self._h, fill_word & 0xFFFFFFFF, _stream_ptr(stream))

    def kv_health_probe(self, seed: int, timeout_ms: int, stream=None):
        """-> (status, checksum)"""
        out = C.c_uint32(0)
        st = lib.kv_health_probe(self._h, seed & 0xFFFFFFFF, timeout_ms, C.byref(out), _stream_ptr(stream))
        return st, out.value

    def kv_sync_status(self, stream=None) -> int:
        return lib.kv_sync_status(self._h, _stream_ptr(stream))

    def kv_debug_slot_map(self, n: int):
        out = np.zeros(n, dtype=np.int64)
        st = lib.kv_debug_slot_map(self._h, out.ctypes.data_as(C.POINTER(C.c_int64)), n)
        return st, out

    def kv_debug_plan(self):
        a, b, c = C.c_int64(), C.c_int64(), C.c_int64()
        lib.kv_debug_plan(self._h, C.byref(a), C.byref(b), C.byref(c))
        return a.value, b.value, c.value

    def kv_debug_profile(self):
        """-> (status, {kind name: (ms, launches)}) for the last kv_rebuild (profile option on)."""
        ms = (C.c_double * len(KINDS))()
        cnt = (C.c_int64 * len(KINDS))()
        st = lib.kv_debug_profile(self._h, ms, cnt)
        return st, {k: (ms[i], cnt[i]) for i, k in enumerate(KINDS)}

    def kv_set_option(self, name: str, value: int) -> int:
        return lib.kv_set_option(self._h, name.encode(), value)

    def kv_debug_gemm(self, impl: int, a, w, out, stream=None) -> int:
        M, K = a.shape
        N = w.shape[0]
        return lib.kv_debug_gemm(self._h, impl, a.data_ptr(), w.data_ptr(), out.data_ptr(), M, N, K,
                                 _stream_ptr(stream))
