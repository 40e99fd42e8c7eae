"""Parity at the benchmark's own shapes and launch configuration.  The oracle
cannot afford whole batches there, so (as the prefix-consistency argument of
the paper's recovery allows) it computes what is exactly comparable: whole
short requests, leading truncations of long ones (causality makes the first m
rows of a long request independent of the rest), and the first layers of a
long request (layer l's K/V depend only on layers < l).  Everything else is
covered by properties that hold at any size: untouched bytes bit-exact,
idempotence bit-exact, no fill left in a mapped row.

Tolerance at depth.  Expected values always come from the oracle's definition.
rel-L2 <= 1e-2 / max-abs <= 6e-2 is asserted wherever the bf16 format itself can
meet it.  Deeper, the bf16 storage of activations alone (the oracle's own forward
with exact arithmetic but bf16-rounded activation tensors) drifts past it on
these random-init shapes; there the GPU result must stay within a few per cent of
that format floor (margins and the per-layer table: see compare_readback)."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from synth import MODEL_SHAPES, WORKLOADS, BENCH_CHUNK_TOKENS, make_workload
from kvr_harness import (Rig, weights_to_cpu, compare_readback, check_untouched_on_device, oracle_weights,
                         oracle_definition_and_floor)

pytestmark = pytest.mark.gpu
BF16_REL, BF16_ABS = 1e-2, 6e-2


def _layers_cpu(w_gpu, n_layers):
    """Host copy of the first n_layers of a device weight set."""
    return {k: (v.cpu() if hasattr(v, "cpu") else [t.cpu() for t in v[:n_layers]]) for k, v in w_gpu.items()}


def _rig_for(cfg: str, chunk: int = BENCH_CHUNK_TOKENS):
    spec = WORKLOADS[cfg]
    shape = MODEL_SHAPES[spec.model]
    wl = make_workload(spec)
    batch = wl.rebuild_batch()
    rig = Rig(shape, "bf16", wl.num_blocks, max_chunk=chunk, max_requests=len(batch.lens),
              max_blocks_per_req=batch.tables.shape[1], seed=spec.seed)
    return spec, shape, wl, batch, rig


def test_cfg2_full_batch_sampled_parity():
    """1.5B shape, the whole 32-request batch rebuilt as the benchmark does it."""
    spec, shape, wl, batch, rig = _rig_for("cfg2")
    rig.rebuild(batch)
    st, slots = rig.ctx.kv_debug_slot_map(batch.n_tokens)
    assert st == 0
    off = np.concatenate([[0], np.cumsum(batch.lens)])
    for r in (0, 7, 31):                                    # slot mapping, sampled requests, closed form
        t = np.arange(int(batch.lens[r]))
        assert np.array_equal(slots[off[r]:off[r + 1]], batch.tables[r][t // 16].astype(np.int64) * 16 + t % 16)
    check_untouched_on_device(rig, batch)
    # full depth: the two shortest requests whole, 384-token truncations of the longest and one more
    w_cpu = oracle_weights(rig.weights)
    order = np.argsort(batch.lens)
    picks = {int(order[0]): int(batch.lens[order[0]]), int(order[1]): min(int(batch.lens[order[1]]), 640),
             int(order[-1]): 384, int(order[len(order) // 2]): 384}
    kv, floor = {}, {}
    for r, n in picks.items():
        kv[r], floor[r] = oracle_definition_and_floor(w_cpu, shape, batch.tokens[off[r]:off[r] + n])
    worst = compare_readback(rig, batch, kv, BF16_REL, BF16_ABS, kv_format_floor=floor, label="cfg2")
    print("cfg2 full-depth sampled worst", worst, "picks", picks)
    # idempotence at full size, bit for bit (compared on the device)
    snap = rig.arena.clone()
    rig.rebuild(batch)
    assert torch.equal(rig.arena.view(torch.int16), snap.view(torch.int16))
    assert rig.guards_ok()


def test_cfg2_long_request_first_layers():
    """Long range: the longest request (up to 16k tokens, many key steps and
    several chunks) against the oracle's layers 0-1."""
    spec, shape, wl, batch, rig = _rig_for("cfg2", chunk=8192)
    r = int(np.argmax(batch.lens))
    n = int(min(batch.lens[r], 12288))
    off = np.concatenate([[0], np.cumsum(batch.lens)])
    sub = wl.subset([wl.rebuild_ids[r]])
    rig.rebuild(sub)
    assert rig.ctx.kv_debug_plan()[1] >= 2                  # the request is cut into chunks
    K, V = oracle.prefill_kv(_layers_cpu(rig.weights, 2), shape, batch.tokens[off[r]:off[r] + n], n_layers=2)
    worst = compare_readback(rig, sub, {0: (K, V)}, BF16_REL, BF16_ABS, layers=(0, 1))
    print("cfg2 long request layers 0-1 worst", worst, "tokens", n)
    # batch invariance: the same request rebuilt inside the whole batch gives the same rows
    st, k_alone, v_alone = rig.ctx.kv_readback(1, sub.tables[0], 2048)
    rig.rebuild(batch)
    st2, k_batch, v_batch = rig.ctx.kv_readback(1, batch.tables[r], 2048)
    assert st == 0 and st2 == 0
    a = oracle.bf16_bits_to_f64(k_alone)
    b = oracle.bf16_bits_to_f64(k_batch)
    assert np.linalg.norm(a - b) / np.linalg.norm(a) < 2e-3
    print("batch invariance bit-identical:", bool(np.array_equal(k_alone, k_batch) and np.array_equal(v_alone, v_batch)))


def test_cfg3_full_batch_sampled_parity():
    """7B shape (the headline configuration), whole batch, benchmark launch
    configuration; oracle on two 256-token leading truncations at full depth."""
    spec, shape, wl, batch, rig = _rig_for("cfg3")
    rig.rebuild(batch)
    check_untouched_on_device(rig, batch)
    off = np.concatenate([[0], np.cumsum(batch.lens)])
    w_cpu = oracle_weights(rig.weights)
    order = np.argsort(batch.lens)
    kv, floor = {}, {}
    for r in (int(order[0]), int(order[-1])):
        kv[r], floor[r] = oracle_definition_and_floor(w_cpu, shape, batch.tokens[off[r]:off[r] + 256])
    worst = compare_readback(rig, batch, kv, BF16_REL, BF16_ABS, kv_format_floor=floor, label="cfg3")
    print("cfg3 full-depth sampled worst", worst)
    assert rig.guards_ok()


def test_partial_recovery_with_shared_prefixes():
    """The partial-recovery configuration at reduced scale: 32 live requests on
    the 1.5B shape (4 layers), 4 groups of 4 sharing a 256-token prefix; all
    are rebuilt once, then the blocks owned only by a seeded 25 % subset are
    scribbled over and that subset alone is rebuilt.  Blocks of the other
    requests must keep their bytes; rebuilt rows must match the first rebuild."""
    shape = dataclasses.replace(MODEL_SHAPES["1.5B"], n_layers=4, vocab=8192)
    spec = dataclasses.replace(WORKLOADS["cfg4"], n_requests=32, lognormal_median=600.0, clip=(64, 3000),
                               shared_groups=4, shared_group_size=4, shared_prefix_len=256, arena_factor=1.2)
    wl = make_workload(spec, vocab=shape.vocab)
    live = wl.subset(np.arange(32))
    rig = Rig(shape, "bf16", wl.num_blocks, max_chunk=16384, max_requests=32,
              max_blocks_per_req=live.tables.shape[1], seed=4)
    rig.rebuild(live)
    computed, _, _ = rig.ctx.kv_debug_plan()
    assert computed == live.n_tokens - 4 * 3 * 256          # each group's prefix computed once
    check_untouched_on_device(rig, live)
    full = rig.arena.clone()
    sub = wl.rebuild_batch()
    assert len(sub.lens) == 8
    # blocks referenced only by the subset
    others = np.setdiff1d(np.arange(32), wl.rebuild_ids)
    used_by_others = set(wl.tables[others][wl.tables[others] >= 0].tolist())
    own = sorted(set(sub.tables[sub.tables >= 0].tolist()) - used_by_others)
    s = shape
    view = rig.arena.view(s.n_layers * 2, wl.num_blocks, 16 * s.n_kv_heads * s.head_dim)
    view[:, torch.tensor(own, device=rig.dev)] = float("nan")     # the partial-write hazard
    rig.rebuild(sub)
    after = rig.arena.view(torch.int16).view(s.n_layers * 2, wl.num_blocks, -1)
    before = full.view(torch.int16).view(s.n_layers * 2, wl.num_blocks, -1)
    keep = torch.ones(wl.num_blocks, dtype=torch.bool, device=rig.dev)
    touched_blocks = sorted(set(sub.tables[sub.tables >= 0].tolist()))
    keep[torch.tensor(touched_blocks, device=rig.dev)] = False
    assert torch.equal(after[:, keep], before[:, keep])           # byte-identical outside the subset
    # rebuilt rows: same values as the first rebuild (shared blocks rewritten with equal values)
    for i, r in enumerate(wl.rebuild_ids.tolist()):
        n = int(sub.lens[i])
        for layer in (0, 3):
            st, k1, v1 = rig.ctx.kv_readback(layer, sub.tables[i], n)
            assert st == 0 and not ((k1 & 0x7FFF) > 0x7F80).any()
            a = oracle.bf16_bits_to_f64(k1)
            # the first rebuild's rows, gathered from the snapshot
            blk = torch.as_tensor(sub.tables[i][np.arange(n) // 16].astype(np.int64), device=rig.dev)
            rows = full.view(s.n_layers, 2, wl.num_blocks, 16, s.n_kv_heads, s.head_dim)[layer, 0, blk,
                                                                                       torch.arange(n, device=rig.dev) % 16]
            b = rows.double().cpu().numpy()
            assert np.linalg.norm(a - b) / np.linalg.norm(b) < 2e-3
    assert rig.guards_ok()
