"""Tensor-parallel rebuild, world size 2, emulated on one device: two contexts (one per rank, each
with its weight slices and its own KV pool of half the kv heads) run in two host threads on two
streams; the all-reduce callback sums the two ranks' partial buffers with stream-ordered copies (no
kernel waits on another kernel).  Each rank's pool must hold the unsharded oracle's K/V of its heads."""
import threading

import numpy as np
import pytest
import torch

import oracle
from synth import ModelShape, make_weights
from synth.workload import RebuildBatch
from kvr_harness import Rig, weights_to_cpu, compare_rebuilt, check_untouched

pytestmark = pytest.mark.gpu


class _DevBuf:
    def __init__(self, ptr, count):
        self.__cuda_array_interface__ = {"shape": (count,), "typestr": "<f4", "data": (ptr, False), "version": 3}


class TwoRankSum:
    """In-place sum of two ranks' buffers on one device.  Host threads meet at barriers; the device
    work is ordered by events: rank 0 adds rank 1's buffer to its own, rank 1 copies the result."""

    def __init__(self):
        self.bar = threading.Barrier(2, timeout=60)
        self.buf = [None, None]
        self.ev = [None, None]
        self.done = None
        self.copied = None
        self.calls = [0, 0]

    def callback(self, rank):
        def allreduce(buf_ptr, count, stream_ptr, _user):
            try:
                stream = torch.cuda.ExternalStream(stream_ptr or 0)
                self.buf[rank] = torch.as_tensor(_DevBuf(buf_ptr, count), device="cuda")
                self.ev[rank] = torch.cuda.Event()
                self.ev[rank].record(stream)                      # my partial is complete at this point
                self.bar.wait()
                if rank == 0:
                    stream.wait_event(self.ev[1])
                    with torch.cuda.stream(stream):
                        self.buf[0].add_(self.buf[1])
                    self.done = torch.cuda.Event()
                    self.done.record(stream)
                self.bar.wait()
                if rank == 1:
                    stream.wait_event(self.done)
                    with torch.cuda.stream(stream):
                        self.buf[1].copy_(self.buf[0])
                    self.copied = torch.cuda.Event()
                    self.copied.record(stream)
                self.bar.wait()
                if rank == 0:
                    stream.wait_event(self.copied)                 # rank 1 has its copy before I reuse the buffer
                self.calls[rank] += 1
                return 0
            except Exception:
                self.bar.abort()
                return 1
        return allreduce


@pytest.mark.parametrize("dtype,gemm,attn", [("fp32", 0, 0), ("bf16", 2, 2)])
def test_tp2_rebuild_matches_unsharded_oracle(dtype, gemm, attn):
    from paper_2608_14635_b200 import binding as kb, tp
    shape = ModelShape("tpmid", n_layers=3, d_model=512, n_q_heads=8, n_kv_heads=4, head_dim=64, ffn=1024, vocab=2048)
    tdt = torch.float32 if dtype == "fp32" else torch.bfloat16
    kdt = kb.KVR_FP32 if dtype == "fp32" else kb.KVR_BF16
    full = make_weights(shape, 41, tdt, device="cuda:0")
    rng = np.random.default_rng(42)
    lens = np.array([300, 77, 513], np.int32)
    nb = [-(-int(n) // 16) for n in lens]
    NB = sum(nb) + 8
    perm = rng.permutation(NB).astype(np.int32)
    tables = np.full((3, max(nb)), -1, np.int32)
    o = 0
    for r, k in enumerate(nb):
        tables[r, :k] = perm[o:o + k]
        o += k
    batch = RebuildBatch(rng.integers(0, shape.vocab, int(lens.sum())).astype(np.int32), lens, tables,
                         np.arange(3, dtype=np.int32))
    summer = TwoRankSum()
    rigs, shards, cbs = [], [], []
    for rank in range(2):
        st, local_desc, shard = kb.kv_tp_plan_host(shape, kdt, 2, rank)
        assert st == 0
        lshape = tp.local_shape(shape, shard)
        rig = Rig(lshape, dtype, NB, max_chunk=256, max_requests=4, max_blocks_per_req=tables.shape[1],
                  weights=tp.shard_weights(full, shape, shard))
        if dtype == "bf16":
            rig.set_impl(gemm, attn)
        assert rig.ctx.kv_tp_bind(2, rank, summer.callback(rank)) == 0
        assert rig.ctx.kv_set_option("keep_last_hidden", 1) == 0
        assert rig.kb.STATUS[rig.ctx.kv_rebuild(batch.tokens, batch.lens, batch.tables)] == "KVR_ERR_NOT_BOUND"
        rig.bind_workspace(256, 4, tables.shape[1])               # the layout gained the partial-sum buffer
        rigs.append(rig)
        shards.append(shard)
    before = [r.arena_bits() for r in rigs]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    status = [None, None]

    def run(rank):
        torch.cuda.set_device(0)
        status[rank] = rigs[rank].ctx.kv_rebuild(batch.tokens, batch.lens, batch.tables, streams[rank])

    for _ in range(2):                                            # twice: idempotent under TP too
        ths = [threading.Thread(target=run, args=(r,)) for r in range(2)]
        [t.start() for t in ths]
        [t.join(120) for t in ths]
        assert status == [0, 0], status
        for r in range(2):
            assert rigs[r].ctx.kv_sync_status(streams[r]) == 0
        if _ == 0:
            first = [r.arena_bits() for r in rigs]
    n_chunks = rigs[0].ctx.kv_debug_plan()[1]
    assert summer.calls[0] == summer.calls[1] == 2 * 2 * n_chunks * (shape.n_layers - 1)   # two per full layer and chunk
    w_cpu = weights_to_cpu(full)
    kv_full = [oracle.prefill_kv(w_cpu, shape, batch.tokens[a:a + n])
               for a, n in zip(np.concatenate([[0], np.cumsum(lens)[:-1]]), lens)]
    tol = (1e-4, 1e-3) if dtype == "fp32" else (1e-2, 6e-2)
    for rank, (rig, sh) in enumerate(zip(rigs, shards)):
        h0, h1 = sh.kv_head0, sh.kv_head0 + sh.n_kv_heads
        kv = [(K[:, :, h0:h1], V[:, :, h0:h1]) for K, V in kv_full]
        worst = compare_rebuilt(rig, batch, kv, *tol)
        check_untouched(rig, before[rank], batch)
        assert np.array_equal(rig.arena_bits(), first[rank])
        assert rig.guards_ok()
        print(f"tp rank {rank} {dtype}: kv heads {h0}..{h1 - 1}, worst", worst)
    # next-token logits under TP: both ranks finish the last layer for the final tokens with their slices, the two
    # row-parallel products are summed through the same callback, the head is whole on every rank
    g = torch.Generator().manual_seed(5)
    gain = (1.0 + 0.02 * torch.randn(shape.d_model, generator=g)).to(tdt).to("cuda:0")
    lm = (0.02 * torch.randn(shape.vocab, shape.d_model, generator=g)).to(tdt).to("cuda:0")
    outs = [torch.full((3, shape.vocab), float("nan"), device="cuda:0") for _ in range(2)]
    calls_before = list(summer.calls)

    def resume(rank):
        torch.cuda.set_device(0)
        status[rank] = rigs[rank].ctx.kv_resume_logits(gain, lm, outs[rank], streams[rank])

    ths = [threading.Thread(target=resume, args=(r,)) for r in range(2)]
    [t.start() for t in ths]
    [t.join(120) for t in ths]
    assert status == [0, 0], status
    for r in range(2):
        assert rigs[r].ctx.kv_sync_status(streams[r]) == 0
    assert [summer.calls[r] - calls_before[r] for r in range(2)] == [2, 2]
    assert torch.equal(outs[0], outs[1])                          # the summed residuals are the same bits on both ranks
    got = outs[0].double().cpu().numpy()
    off = np.concatenate([[0], np.cumsum(lens)])
    for r in range(3):
        want = oracle.resume_logits(w_cpu, shape, batch.tokens[off[r]:off[r + 1]], gain.cpu(), lm.cpu())
        err = float(np.linalg.norm(got[r] - want) / np.linalg.norm(want))
        assert err <= (1e-4 if dtype == "fp32" else 2e-2), (r, err)
    print(f"tp {dtype}: resume logits match the unsharded oracle")
