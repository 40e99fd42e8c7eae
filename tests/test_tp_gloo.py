"""The tensor-parallel partition plan on two CPU processes over gloo: every rank plans its own
shard with the host-only C call, the shards tile the model exactly, and the two row-parallel
products of a layer, computed from each rank's weight slices and summed over the ranks with a real
all-reduce, equal the unsharded products."""
import json
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import numpy as np, torch, torch.distributed as dist
    from paper_2608_14635_b200 import binding as kb, tp
    from synth import ModelShape, make_weights
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo", rank=rank, world_size=world)
    shape = ModelShape("tpcpu", n_layers=1, d_model=64, n_q_heads=6, n_kv_heads=2, head_dim=16, ffn=48, vocab=32)
    st, local, shard = kb.kv_tp_plan_host(shape, kb.KVR_FP32, world, rank)
    assert st == 0
    mine = torch.tensor([shard.q_head0, shard.n_q_heads, shard.kv_head0, shard.n_kv_heads, shard.ffn0, shard.ffn,
                         local.n_q_heads, local.n_kv_heads, local.ffn, local.d_model])
    allsh = [torch.zeros_like(mine) for _ in range(world)]
    dist.all_gather(allsh, mine)
    w = make_weights(shape, 7, torch.float64)
    lw = tp.shard_weights(w, shape, shard)
    rng = np.random.default_rng(3)
    o = torch.from_numpy(rng.standard_normal((5, shape.q_dim)))      # attention output rows, all heads
    m = torch.from_numpy(rng.standard_normal((5, shape.ffn)))        # SwiGLU output rows, all columns
    hd = shape.head_dim
    po = o[:, shard.q_head0 * hd:(shard.q_head0 + shard.n_q_heads) * hd] @ lw["wo"][0].T
    pm = m[:, shard.ffn0:shard.ffn0 + shard.ffn] @ lw["wd"][0].T
    dist.all_reduce(po); dist.all_reduce(pm)
    err_o = float((po - o @ w["wo"][0].T).abs().max()); err_m = float((pm - m @ w["wd"][0].T).abs().max())
    # column-parallel side: the rank's q/k/v/gate rows are rows of the full projections
    a = torch.from_numpy(rng.standard_normal((5, shape.d_model)))
    q_full = a @ w["wq"][0].T
    err_q = float((a @ lw["wq"][0].T - q_full[:, shard.q_head0 * hd:(shard.q_head0 + shard.n_q_heads) * hd]).abs().max())
    bad = kb.kv_tp_plan_host(shape, kb.KVR_FP32, 4, 0)[0]             # 4 does not divide 2 kv heads
    dist.destroy_process_group()
    print(json.dumps({"rank": rank, "shards": [t.tolist() for t in allsh], "err": [err_o, err_m, err_q], "bad": bad}))
""") % ROOT


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_partition_plan_tiles_the_model_and_partial_sums_add_up():
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", LOCAL_RANK=str(r), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        so, se = p.communicate(timeout=180)
        assert p.returncode == 0, se[-2000:]
        outs.append(json.loads(so.strip().splitlines()[-1]))
    for o in outs:
        sh = o["shards"]
        assert sh == outs[0]["shards"]
        # q heads, kv heads and ffn columns: consecutive, disjoint, covering 6 / 2 / 48
        for start, count, total in ((0, 1, 6), (2, 3, 2), (4, 5, 48)):
            pos = 0
            for s in sh:
                assert s[start] == pos
                pos += s[count]
            assert pos == total
        for s in sh:
            assert s[1] == 3 * s[3]                       # whole GQA groups stay on one rank
            assert s[6:10] == [s[1], s[3], s[5], 64]      # the local descriptor carries the per-rank counts
        assert max(o["err"]) < 1e-12
        assert o["bad"] == -3                             # KVR_ERR_UNSUPPORTED
