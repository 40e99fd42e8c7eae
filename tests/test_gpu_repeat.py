"""Repeatability soak: the same rebuild (arena refilled in between) and the same resume-logits call,
many times over, must give the same bits every time.  A race between the kernels' roles (a missing
fence, a buffer reused too early) would show up as a rare difference; none is tolerated."""
import dataclasses

import numpy as np
import pytest
import torch

from synth import WORKLOADS, ModelShape, make_workload, fill_sentinel
from kvr_harness import Rig

pytestmark = pytest.mark.gpu


def test_a_hundred_rebuilds_and_resume_calls_are_bit_identical():
    shape = ModelShape("mid", 4, 1024, 8, 2, 128, 2816, 4096)
    rng = np.random.default_rng(31)
    lens = tuple(int(x) for x in rng.integers(40, 2600, 12))
    spec = dataclasses.replace(WORKLOADS["cfg2"], n_requests=12, fixed_lens=lens, lognormal_median=None, clip=None,
                               seed=31)
    wl = make_workload(spec, vocab=shape.vocab)
    batch = wl.rebuild_batch()
    rig = Rig(shape, "bf16", wl.num_blocks, max_chunk=2048, max_requests=16,
              max_blocks_per_req=batch.tables.shape[1], seed=31)          # chunks of 2048: requests are split
    assert rig.ctx.kv_set_option("keep_last_hidden", 1) == 0
    g = torch.Generator().manual_seed(5)
    gain = (1.0 + 0.02 * torch.randn(shape.d_model, generator=g)).to(rig.tdtype).to(rig.dev)
    lm = (0.02 * torch.randn(shape.vocab, shape.d_model, generator=g)).to(rig.tdtype).to(rig.dev)
    logits = torch.empty(len(batch.lens), shape.vocab, device=rig.dev)
    first_arena = first_logits = None
    for it in range(100):
        fill_sentinel(rig.arena, 11)                                      # the same fill every time
        rig.rebuild(batch)
        bits = rig.arena.view(torch.int16).clone()
        for _ in range(5):
            assert rig.ctx.kv_resume_logits(gain, lm, logits) == 0
            assert rig.ctx.kv_sync_status() == 0
            if first_logits is None:
                first_logits = logits.clone()
            assert torch.equal(first_logits, logits), it
        if first_arena is None:
            first_arena = bits
        assert torch.equal(first_arena, bits), it
    assert rig.guards_ok()
