"""kv_resume_logits on the GPU against the oracle: the next-token logits of
every rebuilt request (what a recovered request needs to resume decoding)."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from synth import MODEL_SHAPES, WORKLOADS, ModelShape, make_workload
from synth.workload import RebuildBatch
from kvr_harness import Rig, oracle_kv, weights_to_cpu, compare_rebuilt

pytestmark = pytest.mark.gpu
TINY = MODEL_SHAPES["tiny"]


def _head(shape, dtype, dev, seed=5):
    g = torch.Generator().manual_seed(seed)
    gain = (1.0 + 0.02 * torch.randn(shape.d_model, generator=g)).to(dtype).to(dev)
    lm = (0.02 * torch.randn(shape.vocab, shape.d_model, generator=g)).to(dtype).to(dev)
    return gain, lm


def _check(rig, batch, rel_tol, sample=None):
    """All requests against the oracle, or the `sample` given (indices)."""
    gain, lm = _head(rig.shape, rig.tdtype, rig.dev)
    R = len(batch.lens)
    out = torch.full((R, rig.shape.vocab), float("nan"), device=rig.dev)
    assert rig.ctx.kv_resume_logits(gain, lm, out) == 0
    assert rig.ctx.kv_sync_status() == 0
    got = out.double().cpu().numpy()
    w = weights_to_cpu(rig.weights)
    off = np.concatenate([[0], np.cumsum(batch.lens)])
    worst = 0.0
    for r in (range(R) if sample is None else sample):
        want = oracle.resume_logits(w, rig.shape, batch.tokens[off[r]:off[r + 1]], gain.cpu(), lm.cpu())
        err = float(np.linalg.norm(got[r] - want) / np.linalg.norm(want))
        assert err <= rel_tol, (r, err)
        worst = max(worst, err)
        # the greedy next token agrees whenever the oracle's top-2 margin exceeds the error scale
        top2 = np.sort(want)[-2:]
        if top2[1] - top2[0] > 4 * np.abs(got[r] - want).max():
            assert int(np.argmax(got[r])) == int(np.argmax(want))
    return worst


@pytest.mark.parametrize("dtype,gemm,attn,tol", [("fp32", 0, 0, 1e-4), ("bf16", 0, 0, 2e-2), ("bf16", 1, 1, 2e-2),
                                                 ("bf16", 1, 2, 2e-2)])
def test_tiny_resume_logits(dtype, gemm, attn, tol):
    wl = make_workload(WORKLOADS["cfg1"])
    batch = wl.rebuild_batch()
    rig = Rig(TINY, dtype, wl.num_blocks, max_chunk=100, max_requests=8, max_blocks_per_req=batch.tables.shape[1])
    if dtype == "bf16":
        rig.set_impl(gemm, attn)
    assert rig.kb.STATUS[rig.ctx.kv_resume_logits(*_head(TINY, rig.tdtype, rig.dev),
                                                  torch.zeros(4, TINY.vocab, device=rig.dev))] == "KVR_ERR_NOT_BOUND"
    assert rig.ctx.kv_set_option("keep_last_hidden", 1) == 0
    rig.rebuild(batch)                              # 5 chunks: final tokens sit in different chunks
    worst = _check(rig, batch, tol)
    # keeping the hidden rows changes nothing in the arena
    kv = oracle_kv(weights_to_cpu(rig.weights), TINY, batch)
    gain, lm = _head(TINY, rig.tdtype, rig.dev)
    first = torch.zeros(len(batch.lens), TINY.vocab, device=rig.dev)
    assert rig.ctx.kv_resume_logits(gain, lm, first) == 0
    compare_rebuilt(rig, batch, kv, 1e-4 if dtype == "fp32" else 1e-2, 1e-3 if dtype == "fp32" else 6e-2)
    # the read-backs above put their own tables into the workspace: the next call brings the rebuild's back
    again = torch.zeros_like(first)
    assert rig.ctx.kv_resume_logits(gain, lm, again) == 0
    assert rig.ctx.kv_sync_status() == 0
    assert torch.equal(first, again)
    assert rig.guards_ok()
    print(f"tiny {dtype} gemm={gemm} attn={attn} logits worst rel-L2", worst)


def test_resume_logits_with_fully_shared_request():
    """A request that is a block-aligned prefix of an earlier one computes nothing for its K/V,
    but its final token is still run so that it can resume."""
    rng = np.random.default_rng(3)
    lens = np.array([50, 32, 20], np.int32)
    t0 = rng.integers(0, TINY.vocab, 50)
    toks = [t0, t0[:32].copy(), rng.integers(0, TINY.vocab, 20)]
    perm = rng.permutation(40).astype(np.int32)
    tables = np.full((3, 4), -1, np.int32)
    tables[0, :4] = perm[:4]
    tables[1, :2] = perm[:2]
    tables[2, :2] = perm[4:6]
    batch = RebuildBatch(np.concatenate(toks).astype(np.int32), lens, tables, np.arange(3, dtype=np.int32))
    rig = Rig(TINY, "fp32", 40, max_chunk=64, max_requests=4, max_blocks_per_req=4)
    assert rig.ctx.kv_set_option("keep_last_hidden", 1) == 0
    rig.rebuild(batch)
    assert rig.ctx.kv_debug_plan()[0] == 50 + 1 + 20
    _check(rig, batch, 1e-4)
    kv = oracle_kv(weights_to_cpu(rig.weights), TINY, batch)
    compare_rebuilt(rig, batch, kv, 1e-4, 1e-3)


@pytest.mark.parametrize("resume_gemm", [1, 0])
def test_mid_shape_resume_logits(resume_gemm):
    shape = ModelShape("mid", 4, 1024, 8, 2, 128, 2816, 4096)
    spec = dataclasses.replace(WORKLOADS["cfg2"], n_requests=4, fixed_lens=(300, 1000, 77, 2049),
                               lognormal_median=None, clip=None, seed=21)
    wl = make_workload(spec, vocab=shape.vocab)
    batch = wl.rebuild_batch()
    rig = Rig(shape, "bf16", wl.num_blocks, max_chunk=2048, max_requests=8,
              max_blocks_per_req=batch.tables.shape[1], seed=21)
    assert rig.ctx.kv_set_option("keep_last_hidden", 1) == 0
    assert rig.ctx.kv_set_option("resume_gemm", resume_gemm) == 0
    rig.rebuild(batch)
    print("mid bf16 logits worst rel-L2", _check(rig, batch, 3e-2))
    assert rig.guards_ok()


@pytest.mark.parametrize("resume_gemm,n_req", [(1, 37), (0, 37), (1, 66), (1, 1), (1, 17)])
def test_resume_logits_many_requests_ragged_head_and_repeat(resume_gemm, n_req):
    """1, 17, 37 or 66 requests (the request dimension is padded to 16, 32, 48, 80 on the tensor core; above 64 the
    weight-streaming GEMM stages 128-row activation boxes), a vocabulary that ends inside a 128-row
    weight tile, and the call made twice after one rebuild: the rows the rebuild kept are only read,
    so both calls give the same bits."""
    shape = ModelShape("mid-ragged", 2, 1024, 8, 2, 128, 2816, 4100)
    rng = np.random.default_rng(8)
    lens = tuple(int(x) for x in rng.integers(1, 260, n_req))
    spec = dataclasses.replace(WORKLOADS["cfg2"], n_requests=n_req, fixed_lens=lens, lognormal_median=None, clip=None,
                               seed=23)
    wl = make_workload(spec, vocab=shape.vocab)
    batch = wl.rebuild_batch()
    rig = Rig(shape, "bf16", wl.num_blocks, max_chunk=2048, max_requests=n_req + 3,
              max_blocks_per_req=batch.tables.shape[1], seed=23)
    assert rig.ctx.kv_set_option("keep_last_hidden", 1) == 0
    assert rig.ctx.kv_set_option("resume_gemm", resume_gemm) == 0
    rig.rebuild(batch)
    print(n_req, "requests, logits worst rel-L2", _check(rig, batch, 3e-2))
    gain, lm = _head(shape, rig.tdtype, rig.dev)
    outs = []
    for _ in range(2):
        out = torch.full((n_req, shape.vocab), float("nan"), device=rig.dev)
        assert rig.ctx.kv_resume_logits(gain, lm, out) == 0
        assert rig.ctx.kv_sync_status() == 0
        outs.append(out.cpu())
    assert torch.equal(outs[0], outs[1])
    assert rig.guards_ok()


def test_resume_logits_more_requests_than_the_streaming_gemm_takes():
    """Above 128 requests the projections go through the rebuild's GEMM; the logits still match the oracle
    and the call can still be repeated."""
    rng = np.random.default_rng(9)
    n_req = 131
    lens = tuple(int(x) for x in rng.integers(1, 40, n_req))
    spec = dataclasses.replace(WORKLOADS["cfg1"], n_requests=n_req, fixed_lens=lens, lognormal_median=None, clip=None,
                               num_blocks=600, seed=29)
    wl = make_workload(spec, vocab=TINY.vocab)
    batch = wl.rebuild_batch()
    rig = Rig(TINY, "bf16", wl.num_blocks, max_chunk=1024, max_requests=n_req, max_blocks_per_req=batch.tables.shape[1],
              seed=29)
    assert rig.ctx.kv_set_option("keep_last_hidden", 1) == 0
    rig.rebuild(batch)
    print(n_req, "requests, logits worst rel-L2 (first, last and 22 more)",
          _check(rig, batch, 2e-2, sample=[0, n_req - 1] + sorted(rng.choice(np.arange(1, n_req - 1), 22, replace=False).tolist())))
    gain, lm = _head(TINY, rig.tdtype, rig.dev)
    outs = []
    for _ in range(2):
        out = torch.full((n_req, TINY.vocab), float("nan"), device=rig.dev)
        assert rig.ctx.kv_resume_logits(gain, lm, out) == 0
        assert rig.ctx.kv_sync_status() == 0
        outs.append(out.cpu())
    assert torch.equal(outs[0], outs[1])
    assert rig.guards_ok()
