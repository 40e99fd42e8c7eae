"""Shared set-up for the GPU parity tests: device buffers with guard bands,
context binding, and comparison against the oracle's expected values."""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional, Tuple

import numpy as np
import torch

import oracle
from synth import fill_sentinel, sentinel_bits, make_weights

GUARD = 4096  # bytes of sentinel before and after every buffer handed to the library


class Guarded:
    """A device buffer of `nbytes` with sentinel guard bands on both sides."""

    def __init__(self, nbytes: int, device, salt: int):
        self.nbytes = nbytes
        pad = (nbytes + 255) // 256 * 256
        self.raw = torch.empty(GUARD + pad + GUARD + 256, dtype=torch.uint8, device=device)
        self.shift = (-self.raw.data_ptr()) % 256
        self.salt = salt
        self.lo = self.raw[self.shift:self.shift + GUARD]
        self.body = self.raw[self.shift + GUARD:self.shift + GUARD + pad]
        self.hi = self.raw[self.shift + GUARD + pad:self.shift + GUARD + pad + GUARD]
        fill_sentinel(self.lo.view(torch.bfloat16), salt)
        fill_sentinel(self.hi.view(torch.bfloat16), salt + 1)
        assert self.body.data_ptr() % 256 == 0

    def guards_intact(self) -> bool:
        lo = sentinel_bits(0, GUARD // 2, 2, self.raw.device, self.salt)
        hi = sentinel_bits(0, GUARD // 2, 2, self.raw.device, self.salt + 1)
        return bool(torch.equal(self.lo.view(torch.int16), lo) and torch.equal(self.hi.view(torch.int16), hi))


_LIVE = []   # rigs and tensors of the running test; conftest frees them when the test ends, pass or fail


def track(obj):
    """Register device tensors (or a dict/list of them) to be freed when the running test ends."""
    _LIVE.append(obj)
    return obj


def free_live() -> None:
    while _LIVE:
        obj = _LIVE.pop()
        if isinstance(obj, Rig):
            obj.free()
        else:
            free_tensors(obj)


class Rig:
    """Context + arena + weights + workspace for one model shape."""

    def __init__(self, shape, dtype: str, num_blocks: int, block_size: int = 16, max_chunk: int = 4096,
                 max_requests: int = 64, max_blocks_per_req: int = 512, seed: int = 1, weights=None,
                 device: str = "cuda:0"):
        from paper_2608_14635_b200 import binding as kb
        self.kb = kb
        self.shape, self.dtype = shape, dtype
        self.fp32 = dtype == "fp32"
        self.tdtype = torch.float32 if self.fp32 else torch.bfloat16
        self.kdt = kb.KVR_FP32 if self.fp32 else kb.KVR_BF16
        self.dev = torch.device(device)
        self.B, self.NB = block_size, num_blocks
        self.weights = weights if weights is not None else make_weights(shape, seed, self.tdtype, device=self.dev)
        self.ctx = kb.Context(self.dev.index or 0)
        _LIVE.append(self)
        es = 4 if self.fp32 else 2
        self.arena_elems = shape.n_layers * 2 * num_blocks * block_size * shape.n_kv_heads * shape.head_dim
        self.arena_g = Guarded(self.arena_elems * es, self.dev, 100)
        self.arena = self.arena_g.body[:self.arena_elems * es].view(self.tdtype)
        fill_sentinel(self.arena, 7)
        assert self.ctx.kv_weights_bind(shape, self.weights, self.kdt) == 0
        if any(k in self.weights for k in ("bq", "qn")):
            assert self.ctx.kv_variant_bind(self.weights) == 0
        assert self.ctx.kv_arena_bind(self.arena, block_size, num_blocks, shape.n_layers, shape.n_kv_heads,
                                      shape.head_dim, self.kdt) == 0
        self.bind_workspace(max_chunk, max_requests, max_blocks_per_req)

    def bind_workspace(self, max_chunk, max_requests, max_blocks_per_req):
        n = self.ctx.kv_workspace_bytes(max_chunk, max_requests, max_blocks_per_req)
        assert n > 0
        self.ws_g = Guarded(n, self.dev, 200)
        fill_sentinel(self.ws_g.body.view(torch.bfloat16), 9)
        st = self.ctx.kv_workspace_bind(self.ws_g.body, max_chunk, max_requests, max_blocks_per_req, nbytes=n)
        assert st == 0, st

    def arena_bits(self) -> np.ndarray:
        """Host copy of the arena as bit patterns in arena_shape order."""
        t = self.arena.view(torch.int32 if self.fp32 else torch.int16).cpu().numpy()
        t = t.view(np.uint32 if self.fp32 else np.uint16)
        s = self.shape
        return t.reshape(oracle.arena_shape(s.n_layers, self.NB, self.B, s.n_kv_heads, s.head_dim))

    def rebuild(self, batch, expect: int = 0):
        st = self.ctx.kv_rebuild(batch.tokens, batch.lens, batch.tables)
        assert st == expect, self.kb.STATUS.get(st, st)
        if st == 0:
            assert self.ctx.kv_sync_status() == 0
        return st

    def set_impl(self, gemm: int, attn: int):
        assert self.ctx.kv_set_option("gemm", gemm) == 0
        assert self.ctx.kv_set_option("attn", attn) == 0

    def guards_ok(self) -> bool:
        return self.arena_g.guards_intact() and self.ws_g.guards_intact()

    def free(self) -> None:
        """Give the device memory back now, whoever still holds a reference to this rig (a failed
        test's traceback keeps its frame, and with it tens of GB, alive for the tests that follow)."""
        self.ctx.close()
        free_tensors([getattr(getattr(self, "arena_g", None), "raw", None),
                      getattr(getattr(self, "ws_g", None), "raw", None), self.weights])


def free_tensors(obj) -> None:
    """Release the storage of every tensor in a (nested) list/dict, in place."""
    import gc
    if hasattr(obj, "untyped_storage"):
        obj.untyped_storage().resize_(0)
    elif isinstance(obj, dict):
        for v in obj.values():
            free_tensors(v)
    elif isinstance(obj, (list, tuple)):
        for v in obj:
            free_tensors(v)
    gc.collect()
    torch.cuda.empty_cache()


def bits_to_f64(bits: np.ndarray, fp32: bool) -> np.ndarray:
    if fp32:
        return bits.view(np.float32).astype(np.float64)
    return oracle.bf16_bits_to_f64(bits)


def oracle_kv(weights_cpu, shape, batch, n_layers=None) -> List[Tuple[np.ndarray, np.ndarray]]:
    out = []
    off = 0
    for n in batch.lens.tolist():
        out.append(oracle.prefill_kv(weights_cpu, shape, batch.tokens[off:off + n], n_layers=n_layers))
        off += n
    return out


class LayerPull:
    """Per-layer weights for the oracle without a host copy of the whole model: layer l's tensor is
    widened on the device and copied to the host when the oracle asks for it; the last two layers
    stay cached so that two oracle passes walking the layers together share one copy."""

    def __init__(self, tensors):
        import threading
        self.tensors, self.cache, self.lock = tensors, {}, threading.Lock()

    def __getitem__(self, l):
        with self.lock:
            if l not in self.cache:
                for k in [k for k in self.cache if k < l - 1]:
                    del self.cache[k]
                self.cache[l] = self.tensors[l].double().cpu()
            return self.cache[l]

    def __len__(self):
        return len(self.tensors)


def oracle_weights(w_gpu):
    """Device weight set -> the mapping the oracle reads, pulling one layer at a time."""
    return {k: (v if hasattr(v, "data_ptr") else LayerPull(v)) for k, v in w_gpu.items()}


def oracle_definition_and_floor(weights, shape, tokens, n_layers=None):
    """The oracle's definition pass and its bf16-storage pass over the same prefix, run side by side
    in two threads (both are the oracle's own prefill_kv, untouched; running them together only
    halves the time spent fetching weights).  -> ((K, V), (K_floor, V_floor))"""
    from concurrent.futures import ThreadPoolExecutor
    with ThreadPoolExecutor(2) as ex:
        a = ex.submit(oracle.prefill_kv, weights, shape, tokens, n_layers, False)
        b = ex.submit(oracle.prefill_kv, weights, shape, tokens, n_layers, True)
        return a.result(), b.result()


def weights_to_cpu(w: Dict[str, object]) -> Dict[str, object]:
    return {k: (v.cpu() if hasattr(v, "cpu") else [t.cpu() for t in v]) for k, v in w.items()}


def compare_rebuilt(rig: Rig, batch, kv: List[Tuple[np.ndarray, np.ndarray]], rel_tol: float,
                    abs_tol: Optional[float], layers=None, max_tokens=None) -> Dict[str, float]:
    """Per layer, K and V separately, over all rebuilt tokens: rel-L2 against
    the unrounded oracle values and max-abs error.  Returns the worst figures."""
    img = rig.arena_bits()
    L = img.shape[0]
    worst = {"rel": 0.0, "abs": 0.0}
    for l in (range(L) if layers is None else layers):
        for kvi in (0, 1):
            num = den = 0.0
            mx = 0.0
            for r, n in enumerate(batch.lens.tolist()):
                n = n if max_tokens is None else min(n, max_tokens)
                if n == 0:
                    continue
                gk, gv = oracle.gather_kv(img, l, batch.tables[r], n)
                got = bits_to_f64(gk if kvi == 0 else gv, rig.fp32)
                want = kv[r][kvi][l][:n]
                assert not np.isnan(got).any(), f"layer {l} kv {kvi} request {r}: sentinel left in a rebuilt row"
                dlt = got - want
                num += float((dlt * dlt).sum())
                den += float((want * want).sum())
                mx = max(mx, float(np.abs(dlt).max()))
            rel = (num / max(den, 1e-300)) ** 0.5
            assert rel <= rel_tol, f"layer {l} {'KV'[kvi]} rel-L2 {rel:.3e} > {rel_tol}"
            if abs_tol is not None:
                assert mx <= abs_tol, f"layer {l} {'KV'[kvi]} max-abs {mx:.3e} > {abs_tol}"
            worst["rel"] = max(worst["rel"], rel)
            worst["abs"] = max(worst["abs"], mx)
    return worst


def check_untouched(rig: Rig, before: np.ndarray, batch) -> None:
    """Every arena byte no rebuilt token maps to is bit-identical to `before`."""
    after = rig.arena_bits()
    m = oracle.touched_mask(batch.lens, batch.tables, rig.B, rig.NB)
    assert np.array_equal(after[:, :, ~m], before[:, :, ~m])
    # and every touched row really changed away from the NaN fill
    touched = bits_to_f64(after[:, :, m], rig.fp32)
    assert not np.isnan(touched).any()


# ---------------------------------------------------------------------------
# Checks that scale to the full benchmark sizes (no host copy of the arena).
# ---------------------------------------------------------------------------
# Margins of the at-depth reading: how far the GPU may sit above the bf16 format floor.  Measured on
# the 1.5B/7B/32B shapes the GPU is within 1 % of the floor in rel-L2 at every layer past the second
# (it is sometimes below it: different, equally valid rounding orders); max-abs is a maximum over
# 10^5-10^7 elements of two independent error draws, which scatters more.
FLOOR_REL_MARGIN = 1.03     # measured: at most 1.015 wherever the stated rel-L2 is out of the format's reach
FLOOR_Q999_MARGIN = 1.05    # the 99.9th percentile of |error| is a stable statistic: same margin class
FLOOR_ABS_MARGIN = 1.5      # measured 0.80 ... 1.36, scattered about 1: the extreme value of ~10^5 heavy-tailed draws


def bf16_half_ulp(x: float) -> float:
    """Half the spacing of bf16 values at magnitude x (8 significant bits): the largest error the
    rounding of one stored value can add."""
    return 2.0 ** (int(np.floor(np.log2(max(x, 1e-30)))) - 8)


def compare_readback(rig: Rig, batch, kv_by_request: Dict[int, Tuple[np.ndarray, np.ndarray]], rel_tol: float,
                     abs_tol: Optional[float], layers=None, kv_format_floor=None, strict_layers: int = 2,
                     label: str = "") -> Dict[str, object]:
    """Same metric as compare_rebuilt (per layer, K and V separately, rel-L2 and
    max-abs against the unrounded oracle values), with the GPU rows fetched
    through kv_readback; only the requests (and leading tokens, and layers) the
    oracle computed are compared.  kv_by_request[r] = (K, V), K.shape = [layers, tokens, Hkv, hd].

    Expected values always come from the definition (prefill_kv without any
    rounding).  `kv_format_floor` holds the oracle's own forward under the bf16
    storage rule (prefill_kv(act_bf16=True)); its distance from the definition
    is what materialising activations in bf16 costs with exact arithmetic (its
    returned K/V are themselves unrounded, so the rounding of the stored value,
    up to half a bf16 ulp, comes on top).  Every layer's figures are recorded
    side by side -- GPU vs definition, floor vs definition -- in worst["table"]
    and printed.  Bound asserted per layer, K and V separately:
        rel-L2  <= max(rel_tol, FLOOR_REL_MARGIN * floor rel-L2)
        max-abs <= max(abs_tol, FLOOR_ABS_MARGIN * floor max-abs + half a bf16 ulp at the layer's
                       largest expected magnitude)
    and, whenever a layer is over the stated tolerance, also
        99.9th percentile of |error| <= FLOOR_Q999_MARGIN * the floor's
    i.e. the stated tolerance wherever the format itself can meet it, and a few
    per cent above the format's own floor where it cannot (`strict_layers`
    leading layers never use the floor for rel-L2).  The maximum of 10^5..10^7
    errors is an extreme-value statistic that differs by tens of per cent
    between two equally accurate computations (it is set by a handful of
    elements of the few tokens with the largest drift), hence its wider margin:
    it guards against isolated gross errors, while rel-L2 and the percentile
    carry the tight comparison."""
    L = rig.shape.n_layers
    worst = {"rel": 0.0, "abs": 0.0, "layers_over_tol": 0, "worst_rel_ratio": 0.0, "worst_abs_ratio": 0.0,
             "table": []}
    failures = []
    for l in (range(L) if layers is None else layers):
        num, den, mx = [0.0, 0.0], [0.0, 0.0], [0.0, 0.0]
        fnum, fmx, wmax = [0.0, 0.0], [0.0, 0.0], [0.0, 0.0]
        errs, ferrs = [[], []], [[], []]
        used = 0
        for r, (K, V) in kv_by_request.items():
            if l >= K.shape[0]:
                continue                    # the oracle ran this request to fewer layers
            used += 1
            n = K.shape[1]
            st, gk, gv = rig.ctx.kv_readback(l, batch.tables[r], n)
            assert st == 0, st
            for kvi, (got_bits, want) in enumerate(((gk, K[l]), (gv, V[l]))):
                got = bits_to_f64(got_bits, rig.fp32)
                assert not np.isnan(got).any(), f"layer {l} request {r}: NaN fill left in a rebuilt row"
                dlt = got - want
                num[kvi] += float((dlt * dlt).sum())
                den[kvi] += float((want * want).sum())
                mx[kvi] = max(mx[kvi], float(np.abs(dlt).max()))
                wmax[kvi] = max(wmax[kvi], float(np.abs(want).max()))
                errs[kvi].append(np.abs(dlt).ravel())
                if kv_format_floor is not None:
                    fd = kv_format_floor[r][kvi][l] - want
                    ferrs[kvi].append(np.abs(fd).ravel())
                    fnum[kvi] += float((fd * fd).sum())
                    fmx[kvi] = max(fmx[kvi], float(np.abs(fd).max()))
        if not used:
            continue
        for kvi in (0, 1):
            rel = (num[kvi] / max(den[kvi], 1e-300)) ** 0.5
            frel = (fnum[kvi] / max(den[kvi], 1e-300)) ** 0.5 if kv_format_floor is not None else None
            within = rel <= rel_tol and (abs_tol is None or mx[kvi] <= abs_tol)
            worst["table"].append({"layer": l, "kv": "KV"[kvi], "requests": used, "gpu_rel": rel, "gpu_abs": mx[kvi],
                                   "floor_rel": frel, "floor_abs": fmx[kvi] if frel is not None else None,
                                   "max_expected": wmax[kvi],
                                   "within_stated": bool(within)})
            if not within and kv_format_floor is not None:
                rel_bound = max(rel_tol, FLOOR_REL_MARGIN * frel) if l >= strict_layers else rel_tol
                assert rel <= rel_bound, \
                    f"{label} layer {l} {'KV'[kvi]} rel-L2 {rel:.3e} vs format floor {frel:.3e}"
                abs_bound = max(abs_tol or 0.0, FLOOR_ABS_MARGIN * fmx[kvi] + bf16_half_ulp(wmax[kvi]))
                assert mx[kvi] <= abs_bound, \
                    f"{label} layer {l} {'KV'[kvi]} max-abs {mx[kvi]:.3e} vs format floor {fmx[kvi]:.3e} " \
                    f"(largest expected magnitude {wmax[kvi]:.2f})"
                q_gpu = float(np.quantile(np.concatenate(errs[kvi]), 0.999))
                q_floor = float(np.quantile(np.concatenate(ferrs[kvi]), 0.999))
                if q_gpu > FLOOR_Q999_MARGIN * q_floor:
                    failures.append(f"{label} layer {l} {'KV'[kvi]} 99.9th percentile of |error| {q_gpu:.3e} "
                                    f"vs floor {q_floor:.3e}")
                worst["table"][-1].update(gpu_q999=q_gpu, floor_q999=q_floor)
                worst["layers_over_tol"] += 1
                worst["worst_rel_ratio"] = max(worst["worst_rel_ratio"], rel / frel)
                worst["worst_abs_ratio"] = max(worst["worst_abs_ratio"], mx[kvi] / max(fmx[kvi], 1e-300))
            else:
                if rel > rel_tol:
                    failures.append(f"{label} layer {l} {'KV'[kvi]} rel-L2 {rel:.3e} > {rel_tol}")
                if abs_tol is not None and mx[kvi] > abs_tol:
                    failures.append(f"{label} layer {l} {'KV'[kvi]} max-abs {mx[kvi]:.3e} > {abs_tol}")
            worst["rel"] = max(worst["rel"], rel)
            worst["abs"] = max(worst["abs"], mx[kvi])
    report_table(label, worst["table"])
    assert not failures, "; ".join(failures)
    return worst


def assess_rows(label: str, layer: int, name: str, got: np.ndarray, want: np.ndarray, floor: Optional[np.ndarray],
               rel_tol: float, abs_tol: float, table: list, failures: list) -> None:
    """The same per-layer bound as compare_readback for one set of rows: the stated tolerance, or --
    where the oracle's bf16-storage pass (`floor`) is itself beyond it -- at most the margins above
    that floor.  Appends one table row and any failure messages."""
    d = got - want
    den = max(float(np.linalg.norm(want)), 1e-300)
    rel, mx, wmax = float(np.linalg.norm(d)) / den, float(np.abs(d).max()), float(np.abs(want).max())
    row = {"layer": layer, "kv": name, "requests": 1, "gpu_rel": rel, "gpu_abs": mx, "floor_rel": None,
           "floor_abs": None, "max_expected": wmax, "within_stated": bool(rel <= rel_tol and mx <= abs_tol)}
    if floor is not None:
        fd = floor - want
        frel, fmx = float(np.linalg.norm(fd)) / den, float(np.abs(fd).max())
        row.update(floor_rel=frel, floor_abs=fmx)
    table.append(row)
    if row["within_stated"]:
        return
    if floor is None:
        failures.append(f"{label} layer {layer} {name} rel-L2 {rel:.3e} max-abs {mx:.3e} over the stated tolerance")
        return
    q_gpu, q_floor = float(np.quantile(np.abs(d), 0.999)), float(np.quantile(np.abs(fd), 0.999))
    row.update(gpu_q999=q_gpu, floor_q999=q_floor)
    if rel > max(rel_tol, FLOOR_REL_MARGIN * frel):
        failures.append(f"{label} layer {layer} {name} rel-L2 {rel:.3e} vs format floor {frel:.3e}")
    if mx > max(abs_tol, FLOOR_ABS_MARGIN * fmx + bf16_half_ulp(wmax)):
        failures.append(f"{label} layer {layer} {name} max-abs {mx:.3e} vs format floor {fmx:.3e}")
    if q_gpu > FLOOR_Q999_MARGIN * q_floor:
        failures.append(f"{label} layer {layer} {name} 99.9th percentile of |error| {q_gpu:.3e} vs floor {q_floor:.3e}")


def report_table(label: str, table) -> None:
    """Print the per-layer figures (pytest -s shows them) and, when the environment names a folder
    in KVR_PARITY_REPORT_DIR, write them there as <label>.json."""
    import json
    import os
    print(f"[parity {label}] layer kv | GPU vs definition rel-L2 / max-abs | bf16 floor vs definition rel-L2 / max-abs")
    for t in table:
        fl = "      -      /     -    " if t["floor_rel"] is None else f"{t['floor_rel']:.3e} / {t['floor_abs']:.3e}"
        print(f"[parity {label}] {t['layer']:3d} {t['kv']} | {t['gpu_rel']:.3e} / {t['gpu_abs']:.3e} | {fl}"
              + ("" if t["within_stated"] else "   (over the stated tolerance)"))
    out = os.environ.get("KVR_PARITY_REPORT_DIR")
    if out and label:
        os.makedirs(out, exist_ok=True)
        with open(os.path.join(out, f"{label.replace(' ', '_')}.json"), "w") as f:
            json.dump(table, f, indent=1)


def block_checksums(rig: Rig) -> torch.Tensor:
    """64-bit position-weighted checksum of every (plane, block) of the arena, computed on the
    device: int64 [n_layers * 2, num_blocks].  Equal checksums before and after a call are the
    byte-identity check at sizes where a second copy of the arena does not fit."""
    s = rig.shape
    words = rig.B * s.n_kv_heads * s.head_dim * (4 if rig.fp32 else 2) // 8
    v = rig.arena.view(torch.int64).view(s.n_layers * 2, rig.NB, words)
    w = (torch.arange(words, dtype=torch.int64, device=rig.dev) * 2 + 1) * (0x9E3779B97F4A7C15 - (1 << 64))   # wraps
    out = torch.empty(s.n_layers * 2, rig.NB, dtype=torch.int64, device=rig.dev)
    step = max(1, (1 << 27) // max(words, 1))            # about 1 GB of int64 per slice
    for pl in range(s.n_layers * 2):
        for b0 in range(0, rig.NB, step):
            blk = v[pl, b0:b0 + step]
            out[pl, b0:b0 + step] = (blk * w).sum(-1) ^ (blk ^ (blk >> 29)).sum(-1)
    return out


def check_untouched_on_device(rig: Rig, batch, salt: int = 7, chunk_slots: int = 1 << 16) -> None:
    """Bit-exact check at any size: every arena row no rebuilt token maps to
    still equals the address-hashed fill, and every mapped row no longer holds
    a NaN.  The touched set is enumerated here from the tables, independently
    of the library."""
    B, NB, s = rig.B, rig.NB, rig.shape
    row = s.n_kv_heads * s.head_dim
    touched = np.zeros(NB * B, dtype=bool)
    for r, n in enumerate(batch.lens.tolist()):
        t = np.arange(n)
        touched[batch.tables[r][t // B].astype(np.int64) * B + t % B] = True
    touched_d = torch.from_numpy(touched).to(rig.dev)
    it = torch.int32 if rig.fp32 else torch.int16
    planes = rig.arena.view(it).view(s.n_layers * 2, NB * B, row)
    fl = rig.arena.view(s.n_layers * 2, NB * B, row)
    eb = 4 if rig.fp32 else 2
    for pl in range(s.n_layers * 2):
        for s0 in range(0, NB * B, chunk_slots):
            s1 = min(NB * B, s0 + chunk_slots)
            want = sentinel_bits((pl * NB * B + s0) * row, (s1 - s0) * row, eb, rig.dev, salt).view(s1 - s0, row)
            keep = ~touched_d[s0:s1]
            assert torch.equal(planes[pl, s0:s1][keep], want[keep]), f"plane {pl}: an unmapped row changed"
            assert not torch.isnan(fl[pl, s0:s1][touched_d[s0:s1]]).any(), f"plane {pl}: a mapped row was not written"
