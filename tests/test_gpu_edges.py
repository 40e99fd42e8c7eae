"""Edge cases of the rebuild on the GPU: empty inputs, lengths on and around every tile,
block and key-step boundary, chunks of a few tokens, limits of the bound workspace."""
import numpy as np
import pytest
import torch

import oracle
from synth import MODEL_SHAPES, ModelShape, make_weights
from synth.workload import RebuildBatch
from kvr_harness import Rig, oracle_kv, weights_to_cpu, compare_rebuilt, check_untouched

pytestmark = pytest.mark.gpu
TINY = MODEL_SHAPES["tiny"]


def _batch(lens, vocab, num_blocks, seed, width=None):
    rng = np.random.default_rng(seed)
    lens = np.asarray(lens, dtype=np.int32)
    nb = [-(-int(n) // 16) for n in lens]
    assert sum(nb) <= num_blocks
    width = max(nb + [1]) if width is None else width
    perm = rng.permutation(num_blocks).astype(np.int32)
    tables = np.full((len(lens), width), -1, dtype=np.int32)
    o = 0
    for r, k in enumerate(nb):
        tables[r, :k] = perm[o:o + k]
        o += k
    tokens = rng.integers(0, vocab, int(lens.sum())).astype(np.int32)
    return RebuildBatch(tokens=tokens, lens=lens, tables=tables, ids=np.arange(len(lens), dtype=np.int32))


def test_empty_batch_and_empty_requests_are_no_ops():
    rig = Rig(TINY, "bf16", 32, max_chunk=64, max_requests=4, max_blocks_per_req=4)
    before = rig.arena_bits()
    empty = RebuildBatch(tokens=np.zeros(0, np.int32), lens=np.zeros(0, np.int32),
                         tables=np.zeros((0, 4), np.int32), ids=np.zeros(0, np.int32))
    rig.rebuild(empty)
    assert np.array_equal(rig.arena_bits(), before)
    zeros = _batch([0, 0, 0], TINY.vocab, 32, 1, width=4)
    rig.rebuild(zeros)
    assert np.array_equal(rig.arena_bits(), before)
    assert rig.ctx.kv_debug_plan()[0] == 0
    # empty requests between real ones change nothing for the others
    mixed = _batch([0, 33, 0, 5], TINY.vocab, 32, 2, width=4)
    rig.rebuild(mixed)
    kv = oracle_kv(weights_to_cpu(rig.weights), TINY, mixed)
    compare_rebuilt(rig, mixed, kv, 1e-2, 6e-2)
    check_untouched(rig, before, mixed)
    assert rig.guards_ok()


BOUNDARY_LENS = [1, 15, 16, 17, 127, 128, 129, 255, 256, 257, 383, 385]


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_lengths_around_every_boundary_tiny(dtype):
    """Head dim 64 (two heads per GEMM half-tile), lengths around the 16-slot block, the 128-key
    step and the 128/256-row attention tile."""
    batch = _batch(BOUNDARY_LENS, TINY.vocab, 160, 3)
    rig = Rig(TINY, dtype, 160, max_chunk=1024, max_requests=len(BOUNDARY_LENS),
              max_blocks_per_req=batch.tables.shape[1])
    before = rig.arena_bits()
    rig.rebuild(batch)
    kv = oracle_kv(weights_to_cpu(rig.weights), TINY, batch)
    tol = (1e-4, 1e-3) if dtype == "fp32" else (1e-2, 6e-2)
    worst = compare_rebuilt(rig, batch, kv, *tol)
    check_untouched(rig, before, batch)
    assert rig.guards_ok()
    print("boundary lens tiny", dtype, worst)


@pytest.mark.parametrize("attn", [2])
def test_lengths_around_every_boundary_wide_heads(attn):
    """The same with head dim 128 through the tcgen05 attention kernel."""
    shape = ModelShape("edge128", n_layers=2, d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=128, ffn=512, vocab=512)
    lens = BOUNDARY_LENS + [511, 513]
    batch = _batch(lens, shape.vocab, 256, 4)
    rig = Rig(shape, "bf16", 256, max_chunk=700, max_requests=len(lens), max_blocks_per_req=batch.tables.shape[1],
              seed=9)
    rig.set_impl(2, attn)
    before = rig.arena_bits()
    rig.rebuild(batch)
    assert rig.ctx.kv_debug_plan()[1] >= 4          # several chunks, requests cut at arbitrary rows
    kv = oracle_kv(weights_to_cpu(rig.weights), shape, batch)
    worst = compare_rebuilt(rig, batch, kv, 1e-2, 6e-2)
    check_untouched(rig, before, batch)
    first = rig.arena_bits()
    rig.rebuild(batch)
    assert np.array_equal(rig.arena_bits(), first)
    assert rig.guards_ok()
    print("boundary lens hd128 attn", attn, worst)


@pytest.mark.parametrize("heads", [(4, 1), (3, 1), (6, 3)])
def test_head_layouts_that_do_not_fill_128_column_tiles(heads):
    """Head dim 64 with q or k/v widths that are not multiples of 128 (kv_dim 64, q_dim 192): the fused
    projection epilogue cannot split a 128-column half between q, k and v, so these shapes must take
    the separate projection + RoPE/scatter step -- same rows, neighbouring slots and blocks untouched."""
    hq, hkv = heads
    shape = ModelShape("oddheads", n_layers=2, d_model=256, n_q_heads=hq, n_kv_heads=hkv, head_dim=64, ffn=512,
                       vocab=512)
    lens = [1, 16, 17, 130, 300]
    batch = _batch(lens, shape.vocab, 64, 11)
    rig = Rig(shape, "bf16", 64, max_chunk=256, max_requests=len(lens), max_blocks_per_req=batch.tables.shape[1],
              seed=12)
    before = rig.arena_bits()
    rig.rebuild(batch)
    kv = oracle_kv(weights_to_cpu(rig.weights), shape, batch)
    worst = compare_rebuilt(rig, batch, kv, 1e-2, 6e-2)
    check_untouched(rig, before, batch)
    first = rig.arena_bits()
    rig.rebuild(batch)
    assert np.array_equal(rig.arena_bits(), first)
    assert rig.guards_ok()
    print("odd head layout", heads, worst)


@pytest.mark.parametrize("chunk", [1, 7])
def test_chunks_of_a_few_tokens(chunk):
    batch = _batch([5, 40, 18], TINY.vocab, 16, 5)
    rig = Rig(TINY, "bf16", 16, max_chunk=chunk, max_requests=3, max_blocks_per_req=batch.tables.shape[1])
    before = rig.arena_bits()
    rig.rebuild(batch)
    assert rig.ctx.kv_debug_plan()[1] == -(-63 // chunk)
    kv = oracle_kv(weights_to_cpu(rig.weights), TINY, batch)
    compare_rebuilt(rig, batch, kv, 1e-2, 6e-2)
    check_untouched(rig, before, batch)
    assert rig.guards_ok()


def test_workspace_limits_are_enforced():
    batch = _batch([20, 20, 20], TINY.vocab, 16, 6)
    rig = Rig(TINY, "bf16", 16, max_chunk=64, max_requests=2, max_blocks_per_req=2)
    before = rig.arena_bits()
    assert rig.kb.STATUS[rig.ctx.kv_rebuild(batch.tokens, batch.lens, batch.tables)] == "KVR_ERR_WORKSPACE"   # 3 requests > 2
    wide = _batch([20, 20], TINY.vocab, 16, 7, width=3)
    assert rig.kb.STATUS[rig.ctx.kv_rebuild(wide.tokens, wide.lens, wide.tables)] == "KVR_ERR_WORKSPACE"      # width 3 > 2
    assert np.array_equal(rig.arena_bits(), before)
    ok = _batch([20, 32], TINY.vocab, 16, 8, width=2)                                                         # exactly at both limits
    rig.rebuild(ok)
    kv = oracle_kv(weights_to_cpu(rig.weights), TINY, ok)
    compare_rebuilt(rig, ok, kv, 1e-2, 6e-2)
    assert rig.guards_ok()


@pytest.mark.parametrize("attn", [2])
def test_longest_prefix_sampled_rows(attn):
    """One request of 65536 tokens (the longest the workloads draw): 4096 table entries, 512 key
    steps, four benchmark-size chunks.  Layer 0 is compared in full, layer 1 on sampled rows the
    oracle computes one by one (first and last rows, both sides of chunk, tile and step boundaries)."""
    from synth import BENCH_CHUNK_TOKENS
    shape = ModelShape("long128", n_layers=2, d_model=256, n_q_heads=2, n_kv_heads=1, head_dim=128, ffn=512,
                       vocab=1024)
    n = 65536
    batch = _batch([n], shape.vocab, 4200, 11)
    rig = Rig(shape, "bf16", 4200, max_chunk=BENCH_CHUNK_TOKENS, max_requests=1,
              max_blocks_per_req=batch.tables.shape[1], seed=12)
    rig.set_impl(2, attn)
    rig.rebuild(batch)
    assert rig.ctx.kv_debug_plan()[1] == 4
    rng = np.random.default_rng(13)
    rows = sorted(set([0, 1, 127, 128, 255, 256, 257, BENCH_CHUNK_TOKENS - 1, BENCH_CHUNK_TOKENS,
                       2 * BENCH_CHUNK_TOKENS + 255, 32767, 32768, n - 257, n - 2, n - 1]
                      + rng.integers(0, n, 24).tolist()))
    K0, V0, K1, V1 = oracle.prefill_kv_rows(weights_to_cpu(rig.weights), shape, batch.tokens, rows)

    def fetch(layer):
        ks, vs = [], []
        for b0 in range(0, 4096, 512):                      # 8192 rows per call
            st, k, v = rig.ctx.kv_readback(layer, batch.tables[0][b0:], 8192)
            assert st == 0
            ks.append(oracle.bf16_bits_to_f64(k))
            vs.append(oracle.bf16_bits_to_f64(v))
        return np.concatenate(ks), np.concatenate(vs)

    for layer, (wk, wv), sel in ((0, (K0, V0), slice(None)), (1, (K1, V1), rows)):
        gk, gv = fetch(layer)
        assert not np.isnan(gk).any() and not np.isnan(gv).any()
        for got, want in ((gk[sel], wk), (gv[sel], wv)):
            err = float(np.linalg.norm(got - want) / np.linalg.norm(want))
            assert err <= 1e-2 and float(np.abs(got - want).max()) <= 6e-2, (layer, err)
    assert rig.guards_ok()
