"""KV-head sharding (one all-reduce of the chunk scores): two CPU processes over gloo check that the
combination of the ranks' local head-means equals the unsharded score block and yields the same
selection on every rank (local blocks come from the oracle here: the library has no CPU path)."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import specext_oracle as orc
        from paper_2505_20776_b200.sharded import combine_scores, head_shard
        rng = np.random.default_rng(11)                     # the same inputs in every process
        Hq, Hkv, D, L, T, C, k = 8, 4, 16, 150, 6, 16, 4
        Q = rng.standard_normal((T, Hq, D))
        Kp, Vp = rng.standard_normal((L, Hkv, D)), rng.standard_normal((L, Hkv, D))
        Kt, Vt = rng.standard_normal((T, Hkv, D)), rng.standard_normal((T, Hkv, D))
        parent = np.array([-1, 0, 0, 1, 2, 2])
        qs, ks = head_shard(Hq, Hkv, rank, world)
        _, _, cs_local = orc.verify_attn(Q[:, qs], Kp[:, ks], Vp[:, ks], Kt[:, ks], Vt[:, ks], parent, C)
        cs = combine_scores(torch.from_numpy(cs_local.copy()))
        _, _, cs_full = orc.verify_attn(Q, Kp, Vp, Kt, Vt, parent, C)
        idx = orc.select_chunks(cs.numpy()[3], L, C, k)
        out.put((rank, float(np.abs(cs.numpy() - cs_full).max()), idx.tolist(),
                 orc.select_chunks(cs_full[3], L, C, k).tolist(), (qs.start, qs.stop, ks.start, ks.stop)))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_reduce_their_head_shards_to_the_unsharded_scores():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() + 777) % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=180)
        assert p.exitcode == 0
    assert [g[4] for g in got] == [(0, 4, 0, 2), (4, 8, 2, 4)]          # consecutive KV heads with their query heads
    for g in got:
        assert g[1] < 1e-14                                              # combined block = unsharded block
        assert g[2] == g[3]                                              # and the same selection
    assert got[0][2] == got[1][2]                                        # on every rank


def test_head_shard_rejects_uneven_splits():
    from paper_2505_20776_b200.sharded import head_shard
    with pytest.raises(ValueError):
        head_shard(32, 8, 0, 3)
    assert head_shard(32, 8, 3, 4) == (slice(24, 32), slice(6, 8))
