"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle
on the same seeded inputs.  Tolerances: slot map and untouched bytes bit-exact;
rebuilt K/V per layer rel-L2 <= 1e-2 and max-abs <= 6e-2 in bf16, rel-L2 <= 1e-4
in the fp32 mode of the tiny configuration."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from synth import MODEL_SHAPES, WORKLOADS, ModelShape, make_workload, make_weights
from synth.workload import RebuildBatch
from kvr_harness import (Rig, oracle_kv, weights_to_cpu, compare_rebuilt, check_untouched, bits_to_f64)

pytestmark = pytest.mark.gpu

TINY = MODEL_SHAPES["tiny"]
BF16_REL, BF16_ABS, FP32_REL = 1e-2, 6e-2, 1e-4


@pytest.fixture(scope="module")
def cfg1():
    wl = make_workload(WORKLOADS["cfg1"])
    return wl, wl.rebuild_batch()


@pytest.fixture(scope="module")
def tiny_oracle(cfg1):
    """Oracle K/V of the four cfg1 requests for fp32 weights and for bf16-rounded weights."""
    _, batch = cfg1
    out = {}
    for name, dt in (("fp32", torch.float32), ("bf16", torch.bfloat16)):
        out[name] = oracle_kv(make_weights(TINY, 1, dt), TINY, batch)
    return out


def _tiny_rig(dtype, wl, batch, max_chunk=512):
    return Rig(TINY, dtype, wl.num_blocks, max_chunk=max_chunk, max_requests=8,
               max_blocks_per_req=batch.tables.shape[1], seed=1)


def test_tiny_fp32_full_parity(cfg1, tiny_oracle):
    wl, batch = cfg1
    rig = _tiny_rig("fp32", wl, batch)
    before = rig.arena_bits()
    rig.rebuild(batch)
    worst = compare_rebuilt(rig, batch, tiny_oracle["fp32"], FP32_REL, 1e-3)
    check_untouched(rig, before, batch)
    st, slots = rig.ctx.kv_debug_slot_map(batch.n_tokens)
    assert st == 0 and np.array_equal(slots, oracle.slot_map(batch.lens, batch.tables, 16))
    first = rig.arena_bits()
    rig.rebuild(batch)                                     # idempotent, bit for bit
    assert np.array_equal(rig.arena_bits(), first)
    # result must not depend on what the rebuilt rows held before (partial-write hazard)
    m = torch.from_numpy(oracle.touched_mask(batch.lens, batch.tables, 16, wl.num_blocks)).to(rig.dev)
    s = TINY
    view = rig.arena.view(s.n_layers, 2, wl.num_blocks, 16, s.n_kv_heads * s.head_dim)
    view[:, :, m] = 12345.0
    rig.rebuild(batch)
    assert np.array_equal(rig.arena_bits(), first)
    assert rig.guards_ok()
    print("tiny fp32 worst", worst)


@pytest.mark.parametrize("gemm,attn", [(0, 0), (1, 0), (0, 1), (1, 1), (0, 2), (1, 2), (2, 0), (2, 2)])
def test_tiny_bf16_parity(cfg1, tiny_oracle, gemm, attn):
    wl, batch = cfg1
    rig = _tiny_rig("bf16", wl, batch)
    rig.set_impl(gemm, attn)
    before = rig.arena_bits()
    rig.rebuild(batch)
    worst = compare_rebuilt(rig, batch, tiny_oracle["bf16"], BF16_REL, BF16_ABS)
    check_untouched(rig, before, batch)
    first = rig.arena_bits()
    rig.rebuild(batch)
    assert np.array_equal(rig.arena_bits(), first)
    assert rig.guards_ok()
    print(f"tiny bf16 gemm={gemm} attn={attn} worst", worst)


@pytest.mark.parametrize("dtype,gemm,attn", [("fp32", 0, 0), ("bf16", 1, 1), ("bf16", 1, 2)])
def test_chunking_invariance(cfg1, tiny_oracle, dtype, gemm, attn):
    """Splitting the token stream into small chunks (requests cut mid-way, later
    chunks attending to K/V written by earlier ones) gives the same arena."""
    wl, batch = cfg1
    big = _tiny_rig(dtype, wl, batch, max_chunk=512)
    small = _tiny_rig(dtype, wl, batch, max_chunk=100)
    for r in (big, small):
        if dtype == "bf16":
            r.set_impl(gemm, attn)
        r.rebuild(batch)
    assert small.ctx.kv_debug_plan()[1] == 5 and big.ctx.kv_debug_plan()[1] == 1
    if dtype == "fp32":
        compare_rebuilt(small, batch, tiny_oracle["fp32"], FP32_REL, 1e-3)
        a, b = bits_to_f64(big.arena_bits(), True), bits_to_f64(small.arena_bits(), True)
        ok = ~np.isnan(a)
        assert np.array_equal(np.isnan(a), np.isnan(b))
        assert np.allclose(a[ok], b[ok], rtol=1e-5, atol=1e-6)
    else:
        compare_rebuilt(small, batch, tiny_oracle["bf16"], BF16_REL, BF16_ABS)
    assert small.guards_ok()


def test_rope_base_is_a_parameter(cfg1):
    wl, batch = cfg1
    shape = dataclasses.replace(TINY, rope_base=1e6)
    rig = Rig(shape, "fp32", wl.num_blocks, max_chunk=512, max_requests=8, max_blocks_per_req=batch.tables.shape[1])
    rig.rebuild(batch)
    kv = oracle_kv(weights_to_cpu(rig.weights), shape, batch)
    compare_rebuilt(rig, batch, kv, FP32_REL, 1e-3)


def test_negative_inputs_leave_arena_untouched(cfg1):
    wl, batch = cfg1
    rig = _tiny_rig("bf16", wl, batch)
    kb = rig.kb
    before = rig.arena_bits()

    def refused(tokens, lens, tables, code):
        st = rig.ctx.kv_rebuild(tokens, lens, tables)
        assert kb.STATUS[st] == code, (kb.STATUS[st], code)
        assert rig.ctx.kv_sync_status() == 0
        assert np.array_equal(rig.arena_bits(), before)

    t, l, tb = batch.tokens, batch.lens, batch.tables
    bad = l.copy(); bad[1] = -3
    refused(t, bad, tb, "KVR_ERR_INVALID_ARG")
    short = tb.copy(); short[3, 12] = -1
    refused(t, l, short, "KVR_ERR_TABLE_TOO_SHORT")
    oob = tb.copy(); oob[2, 0] = wl.num_blocks
    refused(t, l, oob, "KVR_ERR_BLOCK_OOB")
    tok = t.copy(); tok[100] = TINY.vocab
    refused(tok, l, tb, "KVR_ERR_TOKEN_OOB")
    alias = tb.copy(); alias[1, 0] = alias[0, 0]
    refused(t, l, alias, "KVR_ERR_ALIAS_CONFLICT")
    wide = np.full((4, 600), -1, np.int32); wide[:, :tb.shape[1]] = tb
    refused(t, l, wide, "KVR_ERR_WORKSPACE")
    # an all-empty batch and an empty request inside a batch are valid no-ops
    assert rig.ctx.kv_rebuild(np.zeros(0, np.int32), np.zeros(4, np.int32), tb) == 0
    assert np.array_equal(rig.arena_bits(), before)
    l0 = l.copy(); l0[2] = 0
    t0 = np.concatenate([t[:81], t[81 + 129:]])
    assert rig.ctx.kv_rebuild(t0, l0, tb) == 0 and rig.ctx.kv_sync_status() == 0
    b0 = RebuildBatch(t0, l0, tb, batch.ids)
    check_untouched(rig, before, b0)
    # unbound context
    ctx = kb.Context(0)
    assert kb.STATUS[ctx.kv_rebuild(t, l, tb)] == "KVR_ERR_NOT_BOUND"
    assert rig.guards_ok()


def test_readback_matches_arena(cfg1):
    wl, batch = cfg1
    rig = _tiny_rig("bf16", wl, batch)
    rig.rebuild(batch)
    img = rig.arena_bits()
    for r in (0, 3):
        for layer in (0, 1):
            st, k, v = rig.ctx.kv_readback(layer, batch.tables[r], int(batch.lens[r]))
            assert st == 0
            ek, ev = oracle.gather_kv(img, layer, batch.tables[r], int(batch.lens[r]))
            assert np.array_equal(k, ek) and np.array_equal(v, ev)
    n = int(batch.lens[2])
    kd = torch.zeros(n, TINY.n_kv_heads, TINY.head_dim, dtype=torch.bfloat16, device=rig.dev)
    vd = torch.zeros_like(kd)
    assert rig.ctx.kv_readback_dev(1, batch.tables[2], n, kd, vd) == 0
    torch.cuda.synchronize()
    ek, ev = oracle.gather_kv(img, 1, batch.tables[2], n)
    assert np.array_equal(kd.view(torch.int16).cpu().numpy().view(np.uint16), ek)
    assert np.array_equal(vd.view(torch.int16).cpu().numpy().view(np.uint16), ev)
    assert rig.kb.STATUS[rig.ctx.kv_readback(5, batch.tables[0], 4)[0]] == "KVR_ERR_INVALID_ARG"


def test_shared_prefix_is_computed_once():
    """Three requests share their first two blocks (same ids, same tokens); a
    fourth is unrelated.  The shared blocks are computed once and the others
    attend to them through their tables."""
    rng = np.random.default_rng(5)
    B, NB = 16, 40
    lens = np.array([50, 32, 77, 20], np.int32)
    prefix = rng.integers(0, TINY.vocab, 32)
    toks = []
    for r, n in enumerate(lens):
        t = rng.integers(0, TINY.vocab, n)
        if r < 3:
            t[:32] = prefix
        toks.append(t)
    perm = rng.permutation(NB).astype(np.int32)
    tables = np.full((4, 5), -1, np.int32)
    tables[0, :4] = perm[0:4]
    tables[1, :2] = perm[0:2]
    tables[2, :2] = perm[0:2]; tables[2, 2:5] = perm[4:7]
    tables[3, :2] = perm[7:9]
    batch = RebuildBatch(np.concatenate(toks).astype(np.int32), lens, tables, np.arange(4, dtype=np.int32))
    assert oracle.check_inputs(batch.tokens, lens, tables, B, NB, TINY.vocab) == "KVR_OK"
    for dtype, rel, ab in (("fp32", FP32_REL, 1e-3), ("bf16", BF16_REL, BF16_ABS)):
        rig = Rig(TINY, dtype, NB, max_chunk=64, max_requests=4, max_blocks_per_req=5)
        before = rig.arena_bits()
        rig.rebuild(batch)
        computed, chunks, _ = rig.ctx.kv_debug_plan()
        assert computed == 50 + 0 + (77 - 32) + 20 and chunks == 2
        # the host-only planner gives the same answer without a device
        st, skip, h_computed, h_chunks, _ = rig.kb.kv_plan_host(lens, tables, B, 64, 256)
        assert st == 0 and skip.tolist() == [0, 32, 32, 0] and (h_computed, h_chunks) == (computed, chunks)
        kv = oracle_kv(weights_to_cpu(rig.weights), TINY, batch)
        compare_rebuilt(rig, batch, kv, rel, ab)
        check_untouched(rig, before, batch)
        assert rig.guards_ok()


@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (300, 520, 264), (1000, 1376, 256), (77, 256, 688),
                                   (4096, 4608, 3584)])
def test_gemm_kernels_against_fp64(M, N, K):
    """The tcgen05 GEMM and the plain-FMA GEMM against an fp64 product of the
    same bf16 inputs (several tiles, ragged M/N/K tails)."""
    from paper_2608_14635_b200 import binding as kb
    g = torch.Generator().manual_seed(M * 7 + N)
    a = torch.randn(M, K, generator=g).to(torch.bfloat16).cuda()
    w = (torch.randn(N, K, generator=g) * 0.05).to(torch.bfloat16).cuda()
    want = a.double() @ w.double().T
    ctx = kb.Context(0)
    for impl in (0, 1, 2):     # plain FMA, tcgen05 single-CTA tiles, tcgen05 CTA-pair tiles
        out = torch.full((M, N), float("nan"), device="cuda")
        assert ctx.kv_debug_gemm(impl, a, w, out) == 0
        assert ctx.kv_sync_status() == 0
        err = float((out.double() - want).norm() / want.norm())
        tol = (2e-6 * max(1.0, K / 256) ** 0.5 + 1e-6) if impl == 0 else 5e-5
        assert err < tol, (impl, err)


@pytest.mark.parametrize("attn", [1, 2])
def test_mid_shape_bf16_parity(attn):
    """A mid-size decoder (hd 128, GQA group 4, ffn not a multiple of 256) with
    lengths that span several tiles, a ragged tail and a chunk boundary."""
    shape = ModelShape("mid", 4, 1024, 8, 2, 128, 2816, 4096)
    spec = dataclasses.replace(WORKLOADS["cfg2"], n_requests=5, fixed_lens=(300, 1000, 77, 2049, 16),
                               lognormal_median=None, clip=None, seed=21)
    wl = make_workload(spec, vocab=shape.vocab)
    batch = wl.rebuild_batch()
    rig = Rig(shape, "bf16", wl.num_blocks, max_chunk=2048, max_requests=8,
              max_blocks_per_req=batch.tables.shape[1], seed=21)
    rig.set_impl(1, attn)
    before = rig.arena_bits()
    rig.rebuild(batch)
    kv = oracle_kv(weights_to_cpu(rig.weights), shape, batch)
    worst = compare_rebuilt(rig, batch, kv, BF16_REL, BF16_ABS)
    check_untouched(rig, before, batch)
    first = rig.arena_bits()
    rig.rebuild(batch)
    assert np.array_equal(rig.arena_bits(), first)
    assert rig.guards_ok()
    print(f"mid bf16 attn={attn} worst", worst)
