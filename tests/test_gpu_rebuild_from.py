"""kv_rebuild_from: rebuild only the tail of each request on top of a verified
prefix that is already in the arena."""
import numpy as np
import pytest
import torch

import oracle
from synth import MODEL_SHAPES, WORKLOADS, make_workload
from kvr_harness import Rig, oracle_kv, weights_to_cpu, compare_rebuilt

pytestmark = pytest.mark.gpu
TINY = MODEL_SHAPES["tiny"]


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_tail_rebuild_on_a_trusted_prefix(dtype):
    wl = make_workload(WORKLOADS["cfg1"])
    batch = wl.rebuild_batch()
    rig = Rig(TINY, dtype, wl.num_blocks, max_chunk=128, max_requests=8, max_blocks_per_req=batch.tables.shape[1])
    rig.rebuild(batch)
    full = rig.arena_bits()
    valid = np.array([16, 0, 100, 200], np.int32)          # block-aligned, none, mid-block, everything
    # wreck every row past the trusted prefix (the partial-write hazard), keep the prefix rows
    s = TINY
    view = rig.arena.view(s.n_layers, 2, wl.num_blocks, 16, s.n_kv_heads * s.head_dim)
    tail_mask = np.zeros((wl.num_blocks, 16), bool)
    for r in range(4):
        for t in range(int(valid[r]), int(batch.lens[r])):
            tail_mask[int(batch.tables[r][t // 16]), t % 16] = True
    view[:, :, torch.from_numpy(tail_mask).to(rig.dev)] = float("nan")
    st = rig.ctx.kv_rebuild_from(batch.tokens, batch.lens, valid, batch.tables)
    assert st == 0 and rig.ctx.kv_sync_status() == 0
    assert rig.ctx.kv_debug_plan()[0] == int((batch.lens - valid).sum())
    after = rig.arena_bits()
    assert np.array_equal(after[:, :, ~tail_mask], full[:, :, ~tail_mask])     # trusted rows and the rest: same bytes
    kv = oracle_kv(weights_to_cpu(rig.weights), TINY, batch)
    compare_rebuilt(rig, batch, kv, 1e-4 if dtype == "fp32" else 1e-2, 1e-3 if dtype == "fp32" else 6e-2)
    print(dtype, "tail rows bit-identical to the full rebuild:", bool(np.array_equal(after, full)))
    bad = valid.copy(); bad[1] = 65
    assert rig.kb.STATUS[rig.ctx.kv_rebuild_from(batch.tokens, batch.lens, bad, batch.tables)] == "KVR_ERR_INVALID_ARG"
    assert rig.guards_ok()


def test_tail_rebuild_hd128_multi_chunk_through_tensor_core_kernels():
    """Head dim 128 through the tcgen05 GEMM and attention kernels, tails that span several chunks and
    start inside a block, inside a 128-key step and on a tile boundary: trusted rows keep their bytes,
    the tail attends to them through the table and matches the oracle's full prefill."""
    from synth import ModelShape
    from synth.workload import RebuildBatch
    shape = ModelShape("from128", n_layers=3, d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=128, ffn=1024,
                       vocab=2048)
    rng = np.random.default_rng(21)
    lens = np.array([1500, 700, 2300, 260], np.int32)
    valid = np.array([1000, 0, 1031, 256], np.int32)        # mid-block, none, mid-step, tile boundary
    nb = [-(-int(n) // 16) for n in lens]
    NB = sum(nb) + 20
    perm = rng.permutation(NB).astype(np.int32)
    tables = np.full((4, max(nb)), -1, np.int32)
    o = 0
    for r, k in enumerate(nb):
        tables[r, :k] = perm[o:o + k]
        o += k
    batch = RebuildBatch(tokens=rng.integers(0, shape.vocab, int(lens.sum())).astype(np.int32), lens=lens,
                         tables=tables, ids=np.arange(4, dtype=np.int32))
    rig = Rig(shape, "bf16", NB, max_chunk=600, max_requests=4, max_blocks_per_req=tables.shape[1], seed=22)
    rig.set_impl(2, 2)
    rig.rebuild(batch)
    full = rig.arena_bits()
    view = rig.arena.view(shape.n_layers, 2, NB, 16, shape.n_kv_heads * shape.head_dim)
    tail_mask = np.zeros((NB, 16), bool)
    for r in range(4):
        t = np.arange(int(valid[r]), int(lens[r]))
        tail_mask[tables[r][t // 16], t % 16] = True
    view[:, :, torch.from_numpy(tail_mask).to(rig.dev)] = float("nan")
    st = rig.ctx.kv_rebuild_from(batch.tokens, batch.lens, valid, batch.tables)
    assert st == 0 and rig.ctx.kv_sync_status() == 0
    computed, n_chunks, _ = rig.ctx.kv_debug_plan()
    assert computed == int((lens - valid).sum()) and n_chunks >= 4
    after = rig.arena_bits()
    assert np.array_equal(after[:, :, ~tail_mask], full[:, :, ~tail_mask])
    kv = oracle_kv(weights_to_cpu(rig.weights), shape, batch)
    worst = compare_rebuilt(rig, batch, kv, 1e-2, 6e-2)
    print("hd128 multi-chunk tail rebuild", worst)
    assert rig.guards_ok()
