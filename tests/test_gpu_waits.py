"""Bounded waits inside the tensor-core GEMM and attention kernels: a wait that is never satisfied
gives up after the configured limit, the kernel returns, the failure is reported through
kv_sync_status, nothing is written to the arena and the context stays usable.  The wait is made to
run out on the host's terms (the producers are told to issue no loads); no fault, trap or hang is
involved."""
import time

import numpy as np
import pytest
import torch

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


def test_resume_gemm_waits_run_out_and_are_reported():
    """The weight-streaming GEMM of kv_resume_logits under the same hook: its waits run out, the call
    is reported as timed out, and the same call succeeds once the loads are back."""
    shape = MODEL_SHAPES["tiny"]
    wl = make_workload(WORKLOADS["cfg1"])
    batch = wl.rebuild_batch()
    rig = Rig(shape, "bf16", wl.num_blocks, max_chunk=512, max_requests=8, max_blocks_per_req=batch.tables.shape[1])
    rig.set_impl(2, 2)
    assert rig.ctx.kv_set_option("keep_last_hidden", 1) == 0
    rig.rebuild(batch)
    g = torch.Generator().manual_seed(5)
    gain = (1.0 + 0.02 * torch.randn(shape.d_model, generator=g)).to(rig.tdtype).to(rig.dev)
    lm = (0.02 * torch.randn(shape.vocab, shape.d_model, generator=g)).to(rig.tdtype).to(rig.dev)
    R = len(batch.lens)
    good = torch.zeros(R, shape.vocab, device=rig.dev)
    assert rig.ctx.kv_resume_logits(gain, lm, good) == 0
    assert rig.ctx.kv_sync_status() == 0
    before = rig.arena_bits()
    assert rig.ctx.kv_set_option("wait_limit_ms", 20) == 0
    assert rig.ctx.kv_set_option("mute_loads", 1) == 0
    out = torch.zeros(R, shape.vocab, device=rig.dev)
    t0 = time.perf_counter()
    assert rig.ctx.kv_resume_logits(gain, lm, out) == 0
    st = rig.ctx.kv_sync_status()
    dt = time.perf_counter() - t0
    assert rig.kb.STATUS[st] == "KVR_ERR_DEVICE_TIMEOUT"
    assert dt < 2.0, dt
    assert rig.ctx.kv_set_option("mute_loads", 0) == 0
    assert rig.ctx.kv_set_option("wait_limit_ms", 0) == 0
    assert rig.ctx.kv_sync_status() == 0
    assert rig.ctx.kv_resume_logits(gain, lm, out) == 0
    assert rig.ctx.kv_sync_status() == 0
    assert torch.equal(out, good)
    assert np.array_equal(rig.arena_bits(), before)
    assert rig.guards_ok()
