"""Pins for the oracle's attention: what the paper and the mathematics fix, not the oracle itself."""
import json
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import specext_oracle as orc
from tests.util import random_forest

HERE = os.path.dirname(os.path.abspath(__file__))


def _rand(rng, *shape):
    return rng.standard_normal(shape)


def _case(rng, Hq, Hkv, D, L, T):
    return (_rand(rng, T, Hq, D), _rand(rng, L, Hkv, D), _rand(rng, L, Hkv, D),
            _rand(rng, T, Hkv, D), _rand(rng, T, Hkv, D))


def _sdpa_masked(Q, Kp, Vp, Kt, Vt, mask_tt, scale):
    """Library routine: torch fp64 scaled_dot_product_attention with an explicit boolean mask."""
    T, Hq, D = Q.shape
    L, Hkv, _ = Kp.shape
    G = Hq // Hkv
    q = torch.from_numpy(Q).permute(1, 0, 2)[None]                         # [1][Hq][T][D]
    k = torch.from_numpy(np.concatenate([Kp, Kt], 0)).permute(1, 0, 2)     # [Hkv][L+T][D]
    v = torch.from_numpy(np.concatenate([Vp, Vt], 0)).permute(1, 0, 2)
    k = k.repeat_interleave(G, dim=0)[None]                                # head h <- kv head h//G
    v = v.repeat_interleave(G, dim=0)[None]
    mask = torch.cat([torch.ones(T, L, dtype=torch.bool), torch.from_numpy(mask_tt)], dim=1)
    o = torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=mask, scale=scale)
    return o[0].permute(1, 0, 2).numpy()                                   # [T][Hq][D]


def test_golden_hand_worked_example():
    g = json.load(open(os.path.join(HERE, "golden", "two_by_two.json")))
    fr = lambda a: np.array([[float(Fraction(n, d)) for n, d in row] for row in a])
    Q = np.array(g["Q"])
    Kp = np.log(np.array(g["K_prefix_log_of"]))
    Kt = np.log(np.array(g["K_tree_log_of"]))
    Vp, Vt = np.array(g["V_prefix"]), np.array(g["V_tree"])
    O, lse, cs1, P = orc.verify_attn(Q, Kp, Vp, Kt, Vt, g["parent"], 1, g["scale"], return_probs=True)
    np.testing.assert_allclose(P[0], fr(g["P_num_den"]), rtol=0, atol=1e-15)
    assert P[0][0, 3] == 0.0
    np.testing.assert_allclose(O[:, 0, :], fr(g["O_num_den"]), rtol=0, atol=1e-15)
    np.testing.assert_allclose(lse[0], np.log(np.array(g["lse_log_of"])), rtol=0, atol=1e-15)
    np.testing.assert_allclose(cs1, fr(g["chunk_score_C1_num_den"]), rtol=0, atol=1e-15)
    _, _, cs2 = orc.verify_attn(Q, Kp, Vp, Kt, Vt, g["parent"], 2, g["scale"])
    np.testing.assert_allclose(cs2, fr(g["chunk_score_C2_num_den"]), rtol=0, atol=1e-15)


def test_rows_sum_to_one_and_masked_entries_are_zero():
    rng = np.random.default_rng(1)
    Hq, Hkv, D, L, T = 4, 2, 16, 37, 7
    parent = random_forest(rng, T)
    anc = orc.ancestor_mask(parent)
    O, lse, cs, P = orc.verify_attn(*_case(rng, Hq, Hkv, D, L, T), parent, 8, return_probs=True)
    np.testing.assert_allclose(P.sum(-1), 1.0, rtol=0, atol=1e-12)
    assert np.all(P[:, :, L:][:, ~anc] == 0.0)
    assert np.all(P[:, :, :L] > 0.0) and np.all(P[:, :, L:][:, anc] > 0.0)
    # chunk masses of a row add up to one minus the probability that went to tree keys
    tree_mass = P[:, :, L:].sum(-1).mean(0)
    np.testing.assert_allclose(cs.sum(-1), 1.0 - tree_mass, rtol=0, atol=1e-12)


def test_single_visible_key_returns_its_value():
    rng = np.random.default_rng(2)
    Q, Kp, Vp, Kt, Vt = _case(rng, 1, 1, 8, 0, 1)
    O, lse, cs = orc.verify_attn(Q, Kp, Vp, Kt, Vt, [-1], 4, scale=0.3)
    np.testing.assert_array_equal(O[0, 0], Vt[0, 0])
    assert lse[0, 0] == pytest.approx(0.3 * Q[0, 0] @ Kt[0, 0], abs=1e-14)
    assert cs.shape == (1, 0)
    # a forest of roots with an empty prefix: every node sees only itself
    Q, Kp, Vp, Kt, Vt = _case(rng, 2, 1, 8, 0, 3)
    O, _, _ = orc.verify_attn(Q, Kp, Vp, Kt, Vt, [-1, -1, -1], 4)
    for t in range(3):
        np.testing.assert_array_equal(O[t, 0], Vt[t, 0])
        np.testing.assert_array_equal(O[t, 1], Vt[t, 0])


def test_two_key_closed_form():
    rng = np.random.default_rng(3)
    Q, Kp, Vp, Kt, Vt = _case(rng, 1, 1, 8, 1, 1)
    sc = 0.7
    O, lse, cs = orc.verify_attn(Q, Kp, Vp, Kt, Vt, [-1], 4, scale=sc)
    s0, s1 = sc * Q[0, 0] @ Kp[0, 0], sc * Q[0, 0] @ Kt[0, 0]
    e0, e1 = np.exp(s0), np.exp(s1)
    np.testing.assert_allclose(O[0, 0], (e0 * Vp[0, 0] + e1 * Vt[0, 0]) / (e0 + e1), rtol=1e-13)
    assert lse[0, 0] == pytest.approx(np.log(e0 + e1), abs=1e-13)
    assert cs[0, 0] == pytest.approx(e0 / (e0 + e1), abs=1e-14)


def test_chain_tree_is_causal_attention():
    rng = np.random.default_rng(4)
    Hq, Hkv, D, L, T = 4, 2, 16, 37, 5
    Q, Kp, Vp, Kt, Vt = _case(rng, Hq, Hkv, D, L, T)
    parent = np.arange(T) - 1
    O, lse, _ = orc.verify_attn(Q, Kp, Vp, Kt, Vt, parent, 8)
    # library routine with is_causal over the whole sequence of L+T tokens: keep the last T rows
    G = Hq // Hkv
    qfull = np.zeros((L + T, Hq, D))
    qfull[L:] = Q
    q = torch.from_numpy(qfull).permute(1, 0, 2)[None]
    k = torch.from_numpy(np.concatenate([Kp, Kt], 0)).permute(1, 0, 2).repeat_interleave(G, 0)[None]
    v = torch.from_numpy(np.concatenate([Vp, Vt], 0)).permute(1, 0, 2).repeat_interleave(G, 0)[None]
    o = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True)
    np.testing.assert_allclose(O, o[0, :, L:].permute(1, 0, 2).numpy(), rtol=0, atol=1e-12)
    # and a separately written plain loop
    sc = 1.0 / np.sqrt(D)
    for h in range(Hq):
        for t in range(T):
            ks = np.concatenate([Kp[:, h // G], Kt[:t + 1, h // G]], 0)
            vs = np.concatenate([Vp[:, h // G], Vt[:t + 1, h // G]], 0)
            logits = np.array([sc * sum(Q[t, h, d] * ks[j, d] for d in range(D)) for j in range(L + t + 1)])
            w = np.exp(logits - logits.max())
            np.testing.assert_allclose(O[t, h], (w[:, None] * vs).sum(0) / w.sum(), rtol=0, atol=1e-12)
            assert lse[h, t] == pytest.approx(logits.max() + np.log(w.sum()), abs=1e-12)


@pytest.mark.parametrize("Hq,Hkv", [(4, 4), (4, 2), (8, 1)])
def test_general_tree_equals_library_masked_attention(Hq, Hkv):
    rng = np.random.default_rng(5 + Hq + Hkv)
    D, L, T = 16, 41, 9
    Q, Kp, Vp, Kt, Vt = _case(rng, Hq, Hkv, D, L, T)
    parent = random_forest(rng, T)
    anc = orc.ancestor_mask(parent)
    sc = 0.31
    O, lse, _ = orc.verify_attn(Q, Kp, Vp, Kt, Vt, parent, 8, scale=sc)
    np.testing.assert_allclose(O, _sdpa_masked(Q, Kp, Vp, Kt, Vt, anc, sc), rtol=0, atol=1e-12)
    G = Hq // Hkv
    for h in range(Hq):
        keys = torch.from_numpy(np.concatenate([Kp[:, h // G], Kt[:, h // G]], 0))
        s = sc * torch.from_numpy(Q[:, h]) @ keys.T
        s[:, L:] = s[:, L:].masked_fill(~torch.from_numpy(anc), float("-inf"))
        np.testing.assert_allclose(lse[h], torch.logsumexp(s, dim=1).numpy(), rtol=0, atol=1e-12)


def test_ancestor_mask_by_walking_up():
    rng = np.random.default_rng(6)
    for T in (1, 2, 13, 64):
        parent = random_forest(rng, T)
        anc = orc.ancestor_mask(parent)
        for t in range(T):
            seen, u = set(), t
            while u >= 0:
                seen.add(u)
                u = parent[u]
            assert set(np.nonzero(anc[t])[0]) == seen
        np.testing.assert_array_equal(orc.depth(parent), [len([1 for u in range(T) if anc[t, u]]) - 1
                                                          for t in range(T)])


@pytest.mark.parametrize("bad", [[0], [-2], [-1, 1], [-1, 2, 0], [-1, -1, 5]])
def test_bad_trees_are_rejected(bad):
    rng = np.random.default_rng(7)
    T = len(bad)
    with pytest.raises(orc.BadTree):
        orc.verify_attn(*_case(rng, 1, 1, 4, 3, T), bad, 2)


@pytest.mark.parametrize("L,C", [(64, 8), (61, 8), (5, 8)])
def test_zero_query_gives_uniform_scores(L, C):
    rng = np.random.default_rng(8)
    Hq, Hkv, D, T = 4, 2, 16, 6
    Q, Kp, Vp, Kt, Vt = _case(rng, Hq, Hkv, D, L, T)
    Q[:] = 0.0
    parent = random_forest(rng, T)
    dep = orc.depth(parent)
    _, lse, cs = orc.verify_attn(Q, Kp, Vp, Kt, Vt, parent, C)
    lens = orc.chunk_lengths(L, C)
    for t in range(T):
        np.testing.assert_allclose(cs[t], lens / (L + dep[t] + 1.0), rtol=1e-13)
        np.testing.assert_allclose(lse[:, t], np.log(L + dep[t] + 1.0), rtol=1e-13)
    # the ranking key (mass / len) is uniform, so ties resolve to the first k chunks
    NC = len(lens)
    row = lens.astype(np.float32)            # mass proportional to length: every key is exactly 1
    np.testing.assert_array_equal(orc.select_chunks(row, L, C, 3), np.arange(min(3, NC)))


def test_rank_one_construction_closed_form():
    """Q = a*e0 and every key of chunk c equal to b_c*e0: logits are a*b_c*scale exactly."""
    Hq, Hkv, D, T, C = 4, 2, 8, 3, 4
    NC = 6
    L = NC * C - 1                        # trailing chunk of 3 tokens
    a, scale = 2.0, 0.5
    z = np.array([0.0, 1.0, -1.0, 2.0, 2.0, 0.5])           # logit of chunk c (chunks 3, 4 tie)
    rng = np.random.default_rng(9)
    Q = np.zeros((T, Hq, D)); Q[:, :, 0] = a
    Kp = np.zeros((L, Hkv, D)); Kp[:, :, 0] = np.repeat(z / (a * scale), C)[:L, None]
    vchunk = rng.standard_normal((NC, Hkv, D))
    Vp = np.repeat(vchunk, C, axis=0)[:L]
    Kt = np.zeros((T, Hkv, D)); Kt[:, :, 0] = -3.0 / (a * scale)           # tree logits = -3
    Vt = rng.standard_normal((T, Hkv, D))
    parent = [-1, 0, 1]
    O, lse, cs = orc.verify_attn(Q, Kp, Vp, Kt, Vt, parent, C, scale=scale)
    lens = orc.chunk_lengths(L, C)
    for t in range(T):
        ntree = t + 1
        Z = (lens * np.exp(z)).sum() + ntree * np.exp(-3.0)
        np.testing.assert_allclose(cs[t], lens * np.exp(z) / Z, rtol=1e-13)
        np.testing.assert_allclose(lse[:, t], np.log(Z), rtol=1e-13)
        for h in range(Hq):
            g = h // 2
            want = ((lens * np.exp(z))[:, None] * vchunk[:, g]).sum(0) + np.exp(-3.0) * Vt[:ntree, g].sum(0)
            np.testing.assert_allclose(O[t, h], want / Z, rtol=1e-12, atol=1e-14)
    # ranking: chunks 3 and 4 tie on their mean and both beat chunk 1; the tie goes to chunk 3
    np.testing.assert_array_equal(orc.select_chunks(cs[0], L, C, 1, key_dtype=np.float64), [3])
    np.testing.assert_array_equal(orc.select_chunks(cs[0], L, C, 3, key_dtype=np.float64), [1, 3, 4])
    # chunk 5 is short (3 tokens) and ranks by its mean e^0.5, ahead of chunks 0 and 2
    np.testing.assert_array_equal(orc.select_chunks(cs[0], L, C, 4, key_dtype=np.float64), [1, 3, 4, 5])


def test_split_merge_identity():
    rng = np.random.default_rng(10)
    Hq, Hkv, D, L, T = 4, 2, 16, 64, 5
    Q, Kp, Vp, Kt, Vt = _case(rng, Hq, Hkv, D, L, T)
    Q *= 3.0                                   # spread the maxima of the parts
    parent = random_forest(rng, T)
    O, lse, _ = orc.verify_attn(Q, Kp, Vp, Kt, Vt, parent, 8)
    for nsplit in (1, 2, 3, 7, 64):
        cuts = sorted(rng.choice(np.arange(1, L), size=nsplit - 1, replace=False).tolist())
        bounds = [0] + cuts + [L]
        O2, lse2 = orc.attn_split_merge(Q, Kp, Vp, Kt, Vt, parent, bounds)
        np.testing.assert_allclose(O2, O, rtol=0, atol=1e-12)
        np.testing.assert_allclose(lse2, lse, rtol=0, atol=1e-12)


def test_gqa_head_mapping():
    """Query head h must read KV head h // G: make KV heads very different and compare per head."""
    rng = np.random.default_rng(11)
    Hq, Hkv, D, L, T = 6, 3, 8, 10, 2
    Q, Kp, Vp, Kt, Vt = _case(rng, Hq, Hkv, D, L, T)
    parent = [-1, 0]
    O, lse, _ = orc.verify_attn(Q, Kp, Vp, Kt, Vt, parent, 4)
    for h in range(Hq):
        g = h // 2
        O1, lse1, _ = orc.verify_attn(Q[:, h:h + 1], Kp[:, g:g + 1], Vp[:, g:g + 1],
                                      Kt[:, g:g + 1], Vt[:, g:g + 1], parent, 4)
        np.testing.assert_allclose(O[:, h], O1[:, 0], rtol=0, atol=1e-14)
        np.testing.assert_allclose(lse[h], lse1[0], rtol=0, atol=1e-14)
