"""Bounded waits inside the tensor-core GEMM and attention kernels: a wait that is never satisfied
gives up after the configured limit, the kernel returns, the failure is reported through
kv_sync_status, nothing is written to the arena and the context stays usable.  The wait is made to
run out on the host's terms (the producers are told to issue no loads); no fault, trap or hang is
involved."""
import time

import numpy as np
import pytest

import oracle
from synth import MODEL_SHAPES, WORKLOADS, make_workload
from kvr_harness import Rig, oracle_kv, weights_to_cpu, compare_rebuilt, check_untouched

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("gemm", [1, 2])
def test_kernel_waits_run_out_and_are_reported(gemm):
    shape = MODEL_SHAPES["tiny"]
    wl = make_workload(WORKLOADS["cfg1"])
    batch = wl.rebuild_batch()
    rig = Rig(shape, "bf16", wl.num_blocks, max_chunk=512, max_requests=8, max_blocks_per_req=batch.tables.shape[1])
    rig.set_impl(gemm, 2)
    kb = rig.kb
    before = rig.arena_bits()
    assert rig.ctx.kv_set_option("wait_limit_ms", 20) == 0
    assert rig.ctx.kv_set_option("mute_loads", 1) == 0
    t0 = time.perf_counter()
    assert rig.ctx.kv_rebuild(batch.tokens, batch.lens, batch.tables) == 0          # enqueued as usual
    st = rig.ctx.kv_sync_status()
    dt = time.perf_counter() - t0
    assert kb.STATUS[st] == "KVR_ERR_DEVICE_TIMEOUT"
    n_launches = rig.ctx.kv_debug_plan()[2]
    assert dt < 0.1 * n_launches + 2.0, dt                                           # every kernel gave up within its limit
    assert np.array_equal(rig.arena_bits(), before)                                  # no K/V row was written
    assert rig.guards_ok()
    # the status word is cleared by the read, the context keeps working
    assert rig.ctx.kv_set_option("mute_loads", 0) == 0
    assert rig.ctx.kv_set_option("wait_limit_ms", 0) == 0
    assert rig.ctx.kv_sync_status() == 0
    rig.rebuild(batch)
    kv = oracle_kv(weights_to_cpu(rig.weights), shape, batch)
    compare_rebuilt(rig, batch, kv, 1e-2, 6e-2)
    check_untouched(rig, before, batch)
    assert kb.STATUS[rig.ctx.kv_set_option("wait_limit_ms", 60001)] == "KVR_ERR_INVALID_ARG"
