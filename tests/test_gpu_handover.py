"""Handover device steps on the GPU: health check (bit-exact against the
oracle; a device wait that runs out is reported, not hung on) and pool flush."""
import time

import numpy as np
import pytest
import torch

import oracle
from synth import MODEL_SHAPES, WORKLOADS, make_workload
from kvr_harness import Rig, oracle_kv, weights_to_cpu, compare_rebuilt

pytestmark = pytest.mark.gpu


def test_health_probe_matches_oracle_and_reports_timeouts():
    from paper_2608_14635_b200 import binding as kb
    ctx = kb.Context(0)
    n_sms = torch.cuda.get_device_properties(0).multi_processor_count
    for seed in (1, 0xDEADBEEF):
        st, got = ctx.kv_health_probe(seed, 200)
        assert st == 0
        assert got == oracle.probe_checksum(seed, n_sms)
    # nothing publishes the flags: every device wait runs out after ~20 ms and is reported
    assert ctx.kv_set_option("probe_mute", 1) == 0
    t0 = time.perf_counter()
    st, _ = ctx.kv_health_probe(5, 20)
    dt = time.perf_counter() - t0
    assert kb.STATUS[st] == "KVR_ERR_DEVICE_TIMEOUT" and dt < 2.0
    # the context stays usable
    assert ctx.kv_set_option("probe_mute", 0) == 0
    st, got = ctx.kv_health_probe(6, 200)
    assert st == 0 and got == oracle.probe_checksum(6, n_sms)
    assert ctx.kv_sync_status() == 0


def test_health_probe_same_seed_twice_cannot_pass_on_stale_flags():
    """A caller that probes with a constant seed: the flags the first call left
    behind must not satisfy the second call's waits.  With publishing muted the
    second call has to run out, exactly as a first call would."""
    from paper_2608_14635_b200 import binding as kb
    ctx = kb.Context(0)
    n_sms = torch.cuda.get_device_properties(0).multi_processor_count
    st, got = ctx.kv_health_probe(1, 200)
    assert st == 0 and got == oracle.probe_checksum(1, n_sms)
    assert ctx.kv_set_option("probe_mute", 1) == 0
    t0 = time.perf_counter()
    st, _ = ctx.kv_health_probe(1, 20)
    dt = time.perf_counter() - t0
    assert kb.STATUS[st] == "KVR_ERR_DEVICE_TIMEOUT" and dt < 2.0
    assert ctx.kv_set_option("probe_mute", 0) == 0
    for _ in range(3):                                   # and the same seed keeps passing unmuted
        st, got = ctx.kv_health_probe(1, 200)
        assert st == 0 and got == oracle.probe_checksum(1, n_sms)
    assert ctx.kv_sync_status() == 0


def test_flush_then_rebuild():
    shape = MODEL_SHAPES["tiny"]
    wl = make_workload(WORKLOADS["cfg1"])
    batch = wl.rebuild_batch()
    rig = Rig(shape, "bf16", wl.num_blocks, max_chunk=512, max_requests=8, max_blocks_per_req=batch.tables.shape[1])
    rig.rebuild(batch)
    word = 0x7FC17FC1                                   # two bf16 NaNs
    assert rig.ctx.kv_arena_flush(word) == 0 and rig.ctx.kv_sync_status() == 0
    got = rig.arena.view(torch.int32).cpu().numpy().view(np.uint32)
    assert np.array_equal(got, oracle.flushed_arena(got.size, word))
    assert rig.guards_ok()                              # not one byte outside the pool
    rig.rebuild(batch)                                  # refill after the flush
    kv = oracle_kv(weights_to_cpu(rig.weights), shape, batch)
    compare_rebuilt(rig, batch, kv, 1e-2, 6e-2)
