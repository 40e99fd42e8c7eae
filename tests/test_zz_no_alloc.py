"""kv_readback_noalloc: the read-back for callers that cannot allocate (a probe
running right after a failure on a GPU already filled by weights and KV pool,
a standby process with a fixed footprint).  It must return exactly what
kv_readback returns, on two calls in a row (they share one fixed staging
array), and refuse requests larger than that array."""
import numpy as np
import pytest
import torch

from synth import MODEL_SHAPES, WORKLOADS, make_workload
from kvr_harness import Rig

pytestmark = pytest.mark.gpu


def test_noalloc_readback_matches_readback_twice():
    shape = MODEL_SHAPES["tiny"]
    wl = make_workload(WORKLOADS["cfg1"])
    batch = wl.rebuild_batch()
    rig = Rig(shape, "bf16", wl.num_blocks, max_chunk=512, max_requests=8,
              max_blocks_per_req=batch.tables.shape[1], seed=1)
    rig.rebuild(batch)
    kb = rig.kb
    # two calls in a row, different request / layer / length: the second must not see the first's bytes
    free_after_first = None
    for r, layer in ((3, 0), (1, 1), (3, 1)):
        n = int(batch.lens[r])
        st0, k0, v0 = rig.ctx.kv_readback(layer, batch.tables[r], n)
        st1, k1, v1 = kb.kv_readback_noalloc(rig.arena, rig.ctx.geom, layer, batch.tables[r], n)
        assert st0 == 0 and st1 == 0
        # nothing is allocated on the device: once the first call has run (the runtime may load the
        # library's device image lazily on it), free device memory no longer moves
        torch.cuda.synchronize()
        free_now = torch.cuda.mem_get_info(rig.dev)[0]
        assert free_after_first is None or free_now == free_after_first
        free_after_first = free_now
        assert np.array_equal(k0, k1) and np.array_equal(v0, v1)     # byte work: bit-exact
        assert not ((k1 & 0x7FFF) > 0x7F80).any()                    # rebuilt rows, not the NaN fill
    # limits: more than 2 MiB of K per call, or a bad table, is refused with a clear code
    row_bytes = shape.n_kv_heads * shape.head_dim * 2
    too_many = (2 << 20) // row_bytes + 1
    big_table = np.zeros((too_many + 15) // 16, np.int32)
    st, _, _ = kb.kv_readback_noalloc(rig.arena, rig.ctx.geom, 0, big_table, too_many)
    assert kb.STATUS[st] == "KVR_ERR_WORKSPACE"
    bad = batch.tables[0].copy()
    bad[0] = wl.num_blocks
    assert kb.STATUS[kb.kv_readback_noalloc(rig.arena, rig.ctx.geom, 0, bad, 5)[0]] == "KVR_ERR_BLOCK_OOB"
    assert kb.STATUS[kb.kv_readback_noalloc(rig.arena, rig.ctx.geom, 7, batch.tables[0], 5)[0]] == "KVR_ERR_INVALID_ARG"
    assert kb.kv_readback_noalloc(rig.arena, rig.ctx.geom, 0, batch.tables[0], 0)[0] == 0
    # a geometry that reaches past the allocation holding the arena is refused, not read
    import copy
    wide = copy.copy(rig.ctx.geom)
    wide.num_blocks = 1 << 24
    assert kb.STATUS[kb.kv_readback_noalloc(rig.arena, wide, 1, batch.tables[0], 5)[0]] == "KVR_ERR_INVALID_ARG"
    assert rig.guards_ok()
