"""KV-head sharding on one GPU: the two shards of a c1 layer run one after the other through the ordinary
library calls (no kernel waits for another), their local score blocks are combined the way the all-reduce
combines them, and the result is compared with the oracle on the unsharded layer."""
import numpy as np
import pytest
import torch

from paper_2505_20776_b200.sharded import head_shard
from tests.test_gpu_parity import LSE_ATOL, O_ATOL, SCORE_RTOL, check_retrieval, make_hp, oracle_layer
from tests.guards import GuardedHotPath
from tests.util import f64
from workloads import synth

pytestmark = pytest.mark.gpu


def test_two_head_shards_equal_the_unsharded_layer(cuda_device):
    dev = cuda_device
    w = synth.WORKLOADS["c1"]
    t = synth.make_layer(w)
    parent = synth.make_tree(w)
    par = torch.from_numpy(parent).to(dev)
    L, C, world = w.prefix_len, w.chunk_size, 2
    O_ref, lse_ref, cs_ref = oracle_layer(t, parent, L, C)
    combined = None
    shards = []
    for rank in range(world):
        qs, ks = head_shard(w.n_q_heads, w.n_kv_heads, rank, world)
        hp = GuardedHotPath(w.n_q_heads // world, w.n_kv_heads // world, w.head_dim, w.n_tree, C, w.top_k, L, device=dev)
        tl = {"Q": t["Q"][:, qs].contiguous().to(dev), "K_prefix": t["K_prefix"][:, ks].contiguous().to(dev),
              "V_prefix": t["V_prefix"][:, ks].contiguous().to(dev), "K_tree": t["K_tree"][:, ks].contiguous().to(dev),
              "V_tree": t["V_tree"][:, ks].contiguous().to(dev)}
        hp.verify_attn(tl, par, L, True)
        assert hp.read_status() == 0
        hp.check()
        assert np.abs(f64(hp.O) - O_ref[:, qs]).max() <= O_ATOL
        assert np.abs(f64(hp.lse) - lse_ref[qs]).max() <= LSE_ATOL
        local = hp.chunk_score(L).clone()
        combined = local if combined is None else combined + local          # what the all-reduce sums
        shards.append(hp)
    combined *= 1.0 / world
    rel = np.abs(f64(combined) - cs_ref) / cs_ref
    assert rel.max() <= SCORE_RTOL
    # every rank ranks the same reduced block: selection and gather as in the unsharded case
    hp = shards[0]
    hp.chunk_score(L).copy_(combined)
    wd = synth.Workload("c1-draft-shard", w.n_q_heads // world, w.n_kv_heads // world, w.head_dim, L, w.n_tree, C,
                        w.top_k, w.tree, w.values, seed=w.seed)
    check_retrieval(hp, cs_ref, [0, 37, 59], L, C, w.top_k, synth.make_draft_kv(wd))
