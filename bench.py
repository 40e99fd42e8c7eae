#!/usr/bin/env python
"""Benchmark of the KV-rebuild path: one step = one kv_rebuild of a whole batch
of logged prefixes (all hot-path kernels) into a paged arena.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg3] [--impl reference]

Prints ONE JSON line (rank 0).  `value` is tokens/s with the device time of the
step (CUDA events on the launching stream); `e2e` is tokens/s by host wall
clock through the C-ABI call with host input arrays, including validation,
planning, the host->device copies and a device->host read-back of one request's
last-layer K/V.  With N > 1 every rank rebuilds its own replica of the workload
on its own GPU (the path has no exchange step): weak scaling, no collective on
the data path.  `--impl reference` times the CPU oracle on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "kv_rebuild_prefill_tokens_per_s"
UNIT = "tokens/s"
RESUME_CALLS = 15   # kv_resume_logits calls timed one by one; the median is reported


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clocks and throttle reasons during the timed region."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); pw.append(float(r[2]))
            except ValueError:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


def flops_of(shape, lens_computed_pairs, T):
    """Algorithmic flops of one rebuild: linear layers for T computed tokens
    (last layer: K/V projection only) + causal attention pairs, L-1 layers."""
    d, F = shape.d_model, shape.ffn
    qkv = 2 * d * (shape.q_dim + 2 * shape.kv_dim)
    o = 2 * shape.q_dim * d
    gu = 2 * d * 2 * F
    dn = 2 * F * d
    L = shape.n_layers
    per = {"qkv_gemm": T * (qkv * (L - 1) + 2 * d * 2 * shape.kv_dim), "o_gemm": T * o * (L - 1),
           "gateup_gemm": T * gu * (L - 1), "down_gemm": T * dn * (L - 1),
           "attention": 4 * shape.q_dim * lens_computed_pairs * (L - 1)}
    return per


def attention_pairs(batch, block_size):
    """(query, key) pairs a rebuild of `batch` computes: a request whose leading
    full blocks were already filled by an earlier request of the batch starts
    after them (the library's shared-prefix rule, restated for flop counting)."""
    filled, pairs = set(), 0
    for r, n in enumerate(batch.lens.tolist()):
        need = (n + block_size - 1) // block_size
        lead = 0
        while lead < need and int(batch.tables[r][lead]) in filled:
            lead += 1
        skip = min(n, lead * block_size)
        filled.update(int(x) for x in batch.tables[r][:n // block_size])
        pairs += n * (n + 1) // 2 - skip * (skip + 1) // 2
    return pairs


def run_ours(args):
    import torch
    import __graft_entry__ as ge
    ge.build()
    from paper_2608_14635_b200 import binding as kb
    from paper_2608_14635_b200 import replicas
    from synth import MODEL_SHAPES, WORKLOADS, make_workload, make_weights, fill_sentinel, split_waves

    rank, world, local = replicas.env_world()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    replicas.init("nccl", dev)

    spec = WORKLOADS[args.config]
    shape = MODEL_SHAPES[spec.model]
    reduced = args.layers is not None or args.requests is not None
    if args.layers is not None:        # profiling aid: same layer shapes, fewer layers (not a bench number)
        import dataclasses
        shape = dataclasses.replace(shape, n_layers=args.layers)
    peaks = load_peaks()
    from synth import BENCH_CHUNK_TOKENS
    max_chunk = args.chunk if args.chunk is not None else BENCH_CHUNK_TOKENS

    weights = make_weights(shape, spec.seed, torch.bfloat16, device=dev,
                           qkv_bias=args.variant == "bias", qk_norm=args.variant == "qknorm")
    ctx = kb.Context(local)
    assert ctx.kv_weights_bind(shape, weights, kb.KVR_BF16) == 0
    if args.variant != "none":
        assert ctx.kv_variant_bind(weights) == 0
    if args.gemm is not None:
        assert ctx.kv_set_option("gemm", args.gemm) == 0
    if args.attn is not None:
        assert ctx.kv_set_option("attn", args.attn) == 0
    bytes_per_block = shape.n_layers * 2 * spec.block_size * shape.kv_dim * 2

    if args.config == "cfg5":
        # arena = what is left of HBM after weights and workspace; requests go in waves that fit
        wl = make_workload(spec)
        width = wl.tables.shape[1]
        ws_bytes = ctx.kv_workspace_bytes(max_chunk, len(wl.lens), width)
        free, _ = torch.cuda.mem_get_info(dev)
        num_blocks = int((free - ws_bytes - (4 << 30)) // bytes_per_block)
        waves_ids = split_waves(wl.lens, spec.block_size, num_blocks)
        waves = []
        rng = np.random.default_rng(spec.seed + 7)
        for ids in waves_ids:
            b = wl.subset(ids)
            used = np.unique(b.tables[b.tables >= 0])
            remap = dict(zip(used.tolist(), rng.permutation(num_blocks)[:len(used)].tolist()))
            b.tables = np.vectorize(lambda x: remap.get(int(x), -1), otypes=[np.int32])(b.tables)
            waves.append(b)
        live = None
    else:
        wl = make_workload(spec)
        num_blocks = wl.num_blocks
        batch = wl.rebuild_batch()
        if args.requests is not None:      # profiling aid: the first few requests only
            batch = wl.subset(wl.rebuild_ids[:args.requests])
        waves = [batch]
        # partial recovery: the whole live set is rebuilt once (untimed) before the subset is timed
        live = wl.subset(np.arange(len(wl.lens))) if spec.rebuild_fraction < 1.0 else None
        width = wl.tables.shape[1]
        ws_bytes = ctx.kv_workspace_bytes(max_chunk, len(wl.lens), width)
    T = sum(b.n_tokens for b in waves)
    R = sum(len(b.lens) for b in waves)

    arena = torch.empty(num_blocks * bytes_per_block // 2, dtype=torch.bfloat16, device=dev)
    fill_sentinel(arena, 7)
    assert ctx.kv_arena_bind(arena, spec.block_size, num_blocks, shape.n_layers, shape.n_kv_heads,
                             shape.head_dim, kb.KVR_BF16) == 0
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    assert ctx.kv_workspace_bind(ws, max_chunk, len(wl.lens), width) == 0
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        replicas.barrier()

    plan = {"computed": 0, "chunks": 0, "launches": 0}

    def step(collect=None):
        plan.update(computed=0, chunks=0, launches=0)
        for b in waves:
            st = ctx.kv_rebuild(b.tokens, b.lens, b.tables, stream)
            assert st == 0, kb.STATUS.get(st, st)
            c, ch, la = ctx.kv_debug_plan()
            plan["computed"] += c; plan["chunks"] += ch; plan["launches"] += la
            if collect is not None:
                st, prof = ctx.kv_debug_profile()      # waits for this call's events
                assert st == 0
                for k, (ms, n) in prof.items():
                    collect[k][0] += ms
                    collect[k][1] += n

    if live is not None:
        assert ctx.kv_rebuild(live.tokens, live.lens, live.tables, stream) == 0
        assert ctx.kv_sync_status(stream) == 0
    batch = waves[-1]

    for _ in range(args.warmup):
        step()
    assert ctx.kv_sync_status(stream) == 0
    computed, n_chunks, launches_per_step = plan["computed"], plan["chunks"], plan["launches"]

    # ---- timed region: device time of K steps (per-kernel events off) ----
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    clocks = sampler.stop()
    dev_ms = e0.elapsed_time(e1)
    assert ctx.kv_sync_status(stream) == 0

    # ---- per-kernel breakdown: separate steps with an event pair around every launch ----
    prof_steps = max(1, min(args.steps, args.profile_steps))
    assert ctx.kv_set_option("profile", 1) == 0
    kinds = {k: [0.0, 0] for k in kb.KINDS}
    for _ in range(prof_steps):
        step(kinds)
    assert ctx.kv_sync_status(stream) == 0
    assert ctx.kv_set_option("profile", 0) == 0

    # ---- end to end: host arrays in, wall clock, result read back ----
    r_last = int(np.argmax(batch.lens))
    n_rb = int(min(batch.lens[r_last], 1024))
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
        assert ctx.kv_sync_status(stream) == 0
        st, k_rb, v_rb = ctx.kv_readback(shape.n_layers - 1, batch.tables[r_last], n_rb, stream)
        assert st == 0
    barrier()
    e2e_s = time.perf_counter() - t0
    assert not ((k_rb & 0x7FFF) > 0x7F80).any(), "NaN sentinel left in a rebuilt row"

    dev_s, e2e_s = replicas.max_over_ranks([dev_ms / 1e3, e2e_s], device=dev)

    # ---- handover step 2 on the same arena: flush at HBM speed (the arena is rebuilt above, so it may go) ----
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    assert ctx.kv_arena_flush(0x7FC17FC1, stream) == 0           # warm-up
    f0.record(stream)
    for _ in range(3):
        assert ctx.kv_arena_flush(0x7FC17FC1, stream) == 0
    f1.record(stream)
    torch.cuda.synchronize()
    flush_gbs = 3 * arena.numel() * 2 / (f0.elapsed_time(f1) * 1e-3) / 1e9
    st_probe, _ = ctx.kv_health_probe(1, 200, stream)

    # ---- resume logits of the last wave's requests (after an untimed rebuild that keeps the final hidden rows) ----
    resume_ms = None
    lm_bytes = shape.vocab * shape.d_model * (2 + 4) + len(batch.lens) * shape.vocab * 4   # head (+ fp32 draw), logits
    if torch.cuda.mem_get_info(dev)[0] > lm_bytes + (1 << 30):   # cfg5's arena leaves no room: skipped
        gg = torch.Generator(device=dev).manual_seed(spec.seed + 99)
        final_gain = (1.0 + 0.02 * torch.randn(shape.d_model, generator=gg, device=dev)).to(torch.bfloat16)
        lm_head = (0.02 * torch.randn(shape.vocab, shape.d_model, generator=gg, device=dev)).to(torch.bfloat16)
        logits = torch.empty(len(batch.lens), shape.vocab, dtype=torch.float32, device=dev)
        assert ctx.kv_set_option("keep_last_hidden", 1) == 0
        assert ctx.kv_rebuild(batch.tokens, batch.lens, batch.tables, stream) == 0
        assert ctx.kv_resume_logits(final_gain, lm_head, logits, stream) == 0      # warm-up
        assert ctx.kv_sync_status(stream) == 0
        samples = []
        for _ in range(RESUME_CALLS):            # one call at a time, the device idle before each: what a resume sees
            r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            r0.record(stream)
            assert ctx.kv_resume_logits(final_gain, lm_head, logits, stream) == 0
            r1.record(stream)
            assert ctx.kv_sync_status(stream) == 0
            samples.append(r0.elapsed_time(r1))
        resume_ms = float(np.median(samples))
        assert bool(torch.isfinite(logits).all())
        assert ctx.kv_set_option("keep_last_hidden", 0) == 0

    if rank == 0:
        pairs = sum(attention_pairs(b, spec.block_size) for b in waves)
        fl = flops_of(shape, pairs, computed)
        total_flops = sum(fl.values())
        step_s = dev_s / args.steps
        gemm_kinds = ("qkv_gemm", "o_gemm", "gateup_gemm", "down_gemm")
        gemm_ms = sum(kinds[k][0] for k in gemm_kinds) / prof_steps
        gemm_launches = sum(kinds[k][1] for k in gemm_kinds) // prof_steps
        gemm_tf = sum(fl[k] for k in gemm_kinds) / (gemm_ms * 1e-3) / 1e12 if gemm_ms else None
        peak = peaks["bf16_tflops_sustained"]
        breakdown = {}
        for k, (ms, n) in kinds.items():
            ent = {"ms_per_step": ms / prof_steps, "launches_per_step": n // prof_steps}
            if k in fl and ms:
                ent["tflops"] = fl[k] / (ms / prof_steps * 1e-3) / 1e12
            breakdown[k] = ent
        traffic = None
        tp = os.path.join(ROOT, "profiles", "traffic.json")
        if os.path.exists(tp):
            traffic = json.load(open(tp)).get("gemm_tc_kernel_bytes_per_launch")
        out = {
            "metric": METRIC, "value": replicas.whole_job_value(T, step_s, world), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": step_s * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"{args.config}: {shape.name}-shape decoder bf16, {R} requests, {T} tokens "
                                   f"({computed} computed), block 16, {num_blocks} blocks/layer"
                                   + (f", {len(waves)} waves" if len(waves) > 1 else "")
                                   + (f", subset of {len(wl.lens)} live requests" if live is not None else "")
                                   + (f", projection variant {args.variant}" if args.variant != "none" else ""),
                       "chunk_tokens": max_chunk, "chunks_per_step": n_chunks, "replicas": world,
                       "l2": "inputs larger than L2 (14 GB of weights and >1 GB of activations stream per chunk)",
                       "seed": spec.seed, **({"reduced_for_profiling": True} if reduced else {})},
            "rebuild_latency_ms": step_s * 1e3,
            "achieved_tflops": total_flops / step_s / 1e12,
            "frac_of_peak": {"nominal_2250": total_flops / step_s / 2250e12,
                             "measured_burst": total_flops / step_s / (peaks["bf16_tflops"] * 1e12),
                             "measured_sustained": total_flops / step_s / (peak * 1e12), "peaks": peaks["source"]},
            "e2e": {"value": replicas.whole_job_value(T * args.steps, e2e_s, world), "unit": UNIT,
                    "h2d_bytes_per_step": int(sum(b.tokens.nbytes + b.lens.nbytes + b.tables.nbytes for b in waves)),
                    "d2h_bytes_per_step": int(k_rb.nbytes + v_rb.nbytes + 4)},
            "gpu_launches": int(launches_per_step * args.steps),
            "clocks": clocks,
            "roofline": {"kernel": ("gemm_tc_kernel (single-CTA tcgen05 GEMM" if args.gemm == 1 else
                                    "gemm_tc2_kernel (CTA-pair tcgen05 GEMM") + ", all four GEMM kinds)",
                         "bound": "tensor",
                         "achieved": gemm_tf, "peak": peak, "unit": "TFLOP/s",
                         "frac": gemm_tf / peak if gemm_tf else None, "peak_kind": f"sustained, {peaks['source']}",
                         "launches_per_step": gemm_launches, "traffic": traffic},
            "kernels": breakdown,
            "timing": {"value_steps": args.steps, "value_profile_option": 0,
                       "kernels_steps": prof_steps, "kernels_profile_option": 1,
                       "note": "value/ms_per_step: one event pair around all steps; kernels/roofline: separate steps "
                               "with an event pair around every launch"},
            "aux": {"arena_flush": {"bytes": int(arena.numel() * 2), "gbs": flush_gbs, "peak_gbs": peaks["hbm_gbs"],
                                    "frac": flush_gbs / peaks["hbm_gbs"], "note": "write-only fill; peak is a read+write copy"},
                    "health_probe_status": int(st_probe),
                    "resume_logits_ms": resume_ms, "resume_logits_requests": int(len(batch.lens)),
                    "resume_logits_note": "median of %d calls timed one by one" % RESUME_CALLS},
        }
        if not args.no_cpu_baseline and world == 1:
            out["cpu_baseline"] = cpu_baseline(shape, weights, spec.seed, n_tokens=args.cpu_tokens)
        print(json.dumps(out), flush=True)
    replicas.finish()


def cpu_baseline(shape, weights, seed, n_tokens):
    """The oracle as it stands, timed on the host cores, on one short prefix
    through every layer of the same shape."""
    import torch
    import oracle
    w_cpu = {k: (v.cpu() if hasattr(v, "cpu") else [t.cpu() for t in v]) for k, v in weights.items()}
    toks = np.random.default_rng(seed + 1000).integers(0, shape.vocab, n_tokens)
    t0 = time.perf_counter()
    oracle.prefill_kv(w_cpu, shape, toks)
    dt = time.perf_counter() - t0
    return {"value": n_tokens / dt, "unit": UNIT, "cores": int(torch.get_num_threads()), "kind": "oracle",
            "seconds": dt,
            "sample": f"one {n_tokens}-token prefix through all {shape.n_layers} layers of the {shape.name} shape "
                      "(fp64 numpy, BLAS threads = cores)"}


def run_reference(args):
    """The CPU oracle on host cores, bounded sample per step; rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import torch
    from synth import MODEL_SHAPES, WORKLOADS, make_weights
    spec = WORKLOADS[args.config]
    shape = MODEL_SHAPES[spec.model]
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    w = make_weights(shape, spec.seed, torch.bfloat16, device=dev)      # drawn where it is fastest
    w = {k: (v.cpu() if hasattr(v, "cpu") else [t.cpu() for t in v]) for k, v in w.items()}
    import oracle
    n = args.ref_tokens
    rng = np.random.default_rng(spec.seed + 1000)
    steps = []
    for i in range(args.warmup + args.steps):
        toks = rng.integers(0, shape.vocab, n)
        t0 = time.perf_counter()
        oracle.prefill_kv(w, shape, toks)
        dt = time.perf_counter() - t0
        if i >= args.warmup:
            steps.append(dt)
    total = sum(steps)
    val = n * len(steps) / total
    cores = int(torch.get_num_threads())
    sample = (f"each step: one {n}-token prefix through all {shape.n_layers} layers of the {shape.name} shape "
              "(fp64 numpy oracle)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": total / len(steps) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{args.config}: {shape.name}-shape decoder, bounded sample", "seed": spec.seed},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="cfg3", choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
    ap.add_argument("--chunk", type=int, default=None,
                    help="tokens per workspace chunk (default: synth.BENCH_CHUNK_TOKENS = 18944)")
    ap.add_argument("--profile-steps", type=int, default=2,
                    help="steps of the separate per-kernel timing pass (at most --steps)")
    ap.add_argument("--cpu-tokens", type=int, default=384)
    ap.add_argument("--ref-tokens", type=int, default=64)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--variant", default="none", choices=["none", "bias", "qknorm"],
                    help="optional projection terms: q/k/v biases or per-head q/k RMSNorm (default: the headline model)")
    ap.add_argument("--gemm", type=int, default=None, choices=[1, 2],
                    help="tcgen05 GEMM tiling: 1 = single-CTA 128x256 tiles, 2 = CTA pairs (default: the library's)")
    ap.add_argument("--attn", type=int, default=None, choices=[1, 2],
                    help="attention kernel: 1 = warp MMA, 2 = tcgen05 (default: the library's)")
    ap.add_argument("--layers", type=int, default=None, help="profiling aid: run only this many layers")
    ap.add_argument("--requests", type=int, default=None, help="profiling aid: rebuild only the first N requests")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
