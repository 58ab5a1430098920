"""Draft-model attention on the compact cache (specext_draft_attn): the number of cached tokens lives in
device memory, so select -> gather -> draft attention chain without a host round trip.

Oracle: the same fp64 definition as for verification attention, applied to the first n_tokens rows of
the cache (no new oracle arithmetic).  Rows at and beyond n_tokens are NaN in these tests and must not
influence any output.
"""
import numpy as np
import pytest
import torch

from oracle import specext_oracle as orc
from paper_2505_20776_b200 import api
from tests.guards import GuardedHotPath
from tests.test_gpu_parity import LSE_ATOL, O_ATOL, RECORD
from tests.util import bf16_bits, f64
from workloads import synth

pytestmark = pytest.mark.gpu


class DraftSide:
    """Buffers of one draft-attention shape, guarded."""

    def __init__(self, Hq, Hkv, D, T, capacity, dev):
        self.hp = GuardedHotPath(Hq, Hkv, D, T, 32, 1, max(capacity, 1), device=dev)
        self.dev, self.cap = dev, capacity
        self.status = self.hp.status
        self.n_tokens = self.hp._alloc((1,), torch.int32).zero_()
        self._ws = None

    def run(self, t, parent, K_cache, V_cache, n_tokens_dev=None):
        hp = self.hp
        d = api.make_attn_desc(t["Q"], K_cache, t["K_tree"], hp.O, self.cap, 32, 0.0, False)
        need = api.specext_verify_attn_workspace(d)
        if self._ws is None or self._ws.numel() < need:
            self._ws = hp._alloc((need,), torch.uint8)
        api.specext_draft_attn(d, t["Q"], K_cache, V_cache, self.n_tokens if n_tokens_dev is None else n_tokens_dev,
                               t["K_tree"], t["V_tree"], parent, hp.O, hp.lse, self._ws, hp.status)


def _oracle(t_cpu, Kc, Vc, n, parent):
    return orc.verify_attn(f64(t_cpu["Q"]), f64(Kc[:n]), f64(Vc[:n]), f64(t_cpu["K_tree"]), f64(t_cpu["V_tree"]),
                           parent, 32)


SHAPES = [
    # (Hq, Hkv, D, T, tree, capacity)          draft model class
    (12, 12, 64, 1, "chain", 1024),            # 68M-class heads, plain decode step, 1K working cache
    (12, 12, 64, 8, "uniform", 1024),          # 68M-class, a small tree
    (32, 8, 128, 1, "chain", 2048),            # EAGLE-class single layer (the target's layer shape), decode
    (32, 8, 128, 12, "uniform", 2048),         # EAGLE-class, small tree: 48 stacked rows -> one-CTA kernel
    (32, 8, 128, 60, "levels", 2048),          # EAGLE-class, a full 60-node tree: 240 rows -> paired kernel
    (32, 8, 128, 100, "uniform", 1024),        # a tree of more than 64 nodes: two row blocks
]


@pytest.mark.parametrize("Hq,Hkv,D,T,tree,cap", SHAPES)
def test_draft_attn_lengths_on_device(cuda_device, Hq, Hkv, D, T, tree, cap):
    """Every length class (empty, one token, around a tile boundary, ragged, full capacity) with the same
    descriptor and buffers; only the int32 in device memory changes."""
    dev = cuda_device
    w = synth.Workload("draft", Hq, Hkv, D, cap, T, 32, 1, tree, "normal", seed=31 + T)
    t_cpu = synth.make_layer(w)
    parent = synth.make_tree(w)
    t = {k: v.to(dev) for k, v in t_cpu.items()}
    par = torch.from_numpy(parent).to(dev)
    side = DraftSide(Hq, Hkv, D, T, cap, dev)
    for n in (0, 1, 127, 128, 129, cap // 2 + 37, cap - 1, cap):
        Kc, Vc = t["K_prefix"].clone(), t["V_prefix"].clone()
        Kc[n:] = float("nan")
        Vc[n:] = float("nan")
        side.n_tokens.fill_(n)
        side.hp.O.fill_(float("nan"))
        side.run(t, par, Kc, Vc)
        assert side.hp.read_status() == 0
        side.hp.check()
        O_ref, lse_ref, _ = _oracle(t_cpu, t_cpu["K_prefix"], t_cpu["V_prefix"], n, parent)
        O, lse = f64(side.hp.O), f64(side.hp.lse)
        assert np.isfinite(O).all() and np.isfinite(lse).all(), f"n_tokens={n}"
        o_err, l_err = np.abs(O - O_ref).max(), np.abs(lse - lse_ref).max()
        RECORD.add(f"draft-{Hq}x{D}-T{T}", o_max_abs=o_err, lse_max_abs=l_err)
        assert o_err <= O_ATOL and l_err <= LSE_ATOL, f"n_tokens={n}"
    # a length beyond the capacity is clamped to it
    side.n_tokens.fill_(cap + 1000)
    side.run(t, par, t["K_prefix"], t["V_prefix"])
    assert side.hp.read_status() == 0
    O_ref, _, _ = _oracle(t_cpu, t_cpu["K_prefix"], t_cpu["V_prefix"], cap, parent)
    assert np.abs(f64(side.hp.O) - O_ref).max() <= O_ATOL


def test_select_gather_draft_attn_chain_in_one_graph(cuda_device):
    """Target scores -> SelectChunks + UpdateDraftCache -> draft attention, captured once and replayed with
    different scores: the compact length changes between replays (a short trailing chunk gets selected)
    and only device memory carries it."""
    dev = cuda_device
    L, C, k = 4096 - 20, 32, 32                                  # trailing chunk of 12 tokens
    wt = synth.Workload("chain-target", 32, 8, 128, L, 60, C, k, "levels", "needle", seed=77)
    NC = wt.n_chunks
    dK_cpu, dV_cpu = synth.make_draft_kv(wt)                     # the draft model's full cache [1][L][8][128]
    dK, dV = dK_cpu.to(dev), dV_cpu.to(dev)
    hp = GuardedHotPath(32, 8, 128, 60, C, k, L, device=dev)
    wd = synth.Workload("chain-draft", 32, 8, 128, k * C, 12, C, 1, "uniform", "normal", seed=78)
    td_cpu = synth.make_layer(wd)
    td = {kk: v.to(dev) for kk, v in td_cpu.items()}
    pd_np = synth.make_tree(wd)
    pd = torch.from_numpy(pd_np).to(dev)
    side = DraftSide(32, 8, 128, 12, k * C, dev)
    scores = hp.chunk_score(L)
    rng = np.random.default_rng(3)

    def chain():
        hp.select_gather(5, L, dK, dV)
        side.run(td, pd, hp.K_compact[0], hp.V_compact[0], n_tokens_dev=hp.n_tokens)

    row_a = rng.random(NC).astype(np.float32)
    row_a[NC - 1] = 0.0                                          # trailing chunk not selected: 1024 tokens
    row_b = row_a.copy()
    row_b[NC - 1] = 50.0                                         # trailing chunk selected: 31*32 + 12 tokens
    scores.zero_()
    scores[5] = torch.from_numpy(row_a).to(dev)
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        chain()
        s.synchronize()
        with torch.cuda.graph(g, stream=s):
            chain()
    for row, want_tokens in ((row_a, k * C), (row_b, (k - 1) * C + 12), (row_a, k * C)):
        scores[5] = torch.from_numpy(row).to(dev)
        hp.K_compact.fill_(float("nan"))                         # whatever the gather does not write stays NaN
        hp.V_compact.fill_(float("nan"))
        torch.cuda.synchronize()
        with torch.cuda.stream(s):
            g.replay()
        s.synchronize()
        assert hp.read_status() == 0 and side.hp.read_status() == 0
        hp.check()
        side.hp.check()
        n = int(hp.n_tokens.item())
        assert n == want_tokens
        idx = orc.select_chunks(row, L, C, k, key_dtype=np.float32)
        np.testing.assert_array_equal(hp.idx[: int(hp.n_selected.item())].cpu().numpy(), idx)
        Kr, Vr, n_ref = orc.gather_kv(dK_cpu.view(torch.int16).numpy(), dV_cpu.view(torch.int16).numpy(), idx, L, C)
        assert n_ref == n
        np.testing.assert_array_equal(bf16_bits(hp.K_compact)[:, :n], Kr)
        Kc = torch.from_numpy(Kr[0]).view(torch.bfloat16)
        Vc = torch.from_numpy(Vr[0]).view(torch.bfloat16)
        O_ref, lse_ref, _ = _oracle(td_cpu, Kc, Vc, n, pd_np)
        assert np.abs(f64(side.hp.O) - O_ref).max() <= O_ATOL
        assert np.abs(f64(side.hp.lse) - lse_ref).max() <= LSE_ATOL


def test_draft_attn_host_side_rejection(cuda_device):
    dev = cuda_device
    w = synth.Workload("draft", 8, 2, 128, 256, 4, 32, 1, "chain", "normal", seed=5)
    t = {k: v.to(dev) for k, v in synth.make_layer(w).items()}
    par = torch.from_numpy(synth.make_tree(w)).to(dev)
    side = DraftSide(8, 2, 128, 4, 256, dev)
    hp = side.hp
    d = api.make_attn_desc(t["Q"], t["K_prefix"], t["K_tree"], hp.O, 256, 32, 0.0, True)   # scores are not offered
    ws = torch.empty(api.specext_verify_attn_workspace(d), dtype=torch.uint8, device=dev)
    with pytest.raises(api.SpecextError) as e:
        api.specext_draft_attn(d, t["Q"], t["K_prefix"], t["V_prefix"], side.n_tokens, t["K_tree"], t["V_tree"],
                               par, hp.O, hp.lse, ws, hp.status)
    assert e.value.code == 1
    d.want_chunk_score = 0
    rc = api.lib().specext_draft_attn(d, t["Q"].data_ptr(), t["K_prefix"].data_ptr(), t["V_prefix"].data_ptr(), None,
                                      t["K_tree"].data_ptr(), t["V_tree"].data_ptr(), par.data_ptr(),
                                      hp.O.data_ptr(), hp.lse.data_ptr(), ws.data_ptr(), ws.numel(),
                                      hp.status.data_ptr(), None)
    assert rc == 1                                               # no device-side length given
