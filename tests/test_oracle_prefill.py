"""Pins of the oracle's prefill (causal self-attention): a library routine, exact special cases and
consistency with the tree-attention oracle, each of which a plausible mistake (an off-by-one in the
causal mask, a wrong GQA map, a transposed operand, a missing scale) would fail."""
import numpy as np
import torch

from oracle import specext_oracle as orc


def _rand(L, Hq, Hkv, D, seed):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((L, Hq, D)), rng.standard_normal((L, Hkv, D)), rng.standard_normal((L, Hkv, D))


def test_equals_torch_causal_sdpa_with_gqa():
    L, Hq, Hkv, D = 37, 6, 3, 16
    Q, K, V = _rand(L, Hq, Hkv, D, 1)
    O, lse = orc.prefill_attn(Q, K, V, scale=0.3)
    G = Hq // Hkv
    q = torch.from_numpy(Q).permute(1, 0, 2)[None]                       # [1][Hq][L][D]
    k = torch.from_numpy(K).permute(1, 0, 2).repeat_interleave(G, dim=0)[None]
    v = torch.from_numpy(V).permute(1, 0, 2).repeat_interleave(G, dim=0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True, scale=0.3)[0]
    np.testing.assert_allclose(O, ref.permute(1, 0, 2).numpy(), rtol=0, atol=1e-12)
    s = 0.3 * torch.einsum("hid,hjd->hij", q[0], k[0])
    s = s.masked_fill(~torch.ones(L, L, dtype=torch.bool).tril(), float("-inf"))
    np.testing.assert_allclose(lse, torch.logsumexp(s, dim=-1).numpy(), rtol=0, atol=1e-12)


def test_first_token_returns_its_own_value_and_default_scale():
    Q, K, V = _rand(9, 4, 2, 8, 2)
    O, lse = orc.prefill_attn(Q, K, V)
    for h in range(4):
        np.testing.assert_array_equal(O[0, h], V[0, h // 2])
        assert lse[h, 0] == np.dot(Q[0, h], K[0, h // 2]) / np.sqrt(8)


def test_block_equals_tree_attention_with_a_chain_tree():
    """Tokens [p, p+T) of the prefill = verification attention with prefix p and a chain of T nodes."""
    L, Hq, Hkv, D, p0, T = 29, 4, 2, 8, 17, 7
    Q, K, V = _rand(L, Hq, Hkv, D, 3)
    rows = list(range(p0, p0 + T))
    O, lse = orc.prefill_attn(Q, K, V, rows=rows)
    O2, lse2, _ = orc.verify_attn(Q[p0:p0 + T], K[:p0], V[:p0], K[p0:p0 + T], V[p0:p0 + T],
                                  np.arange(T) - 1, 4)
    np.testing.assert_allclose(O, O2, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, lse2, rtol=0, atol=1e-12)


def test_rows_subset_matches_full_and_future_keys_do_not_matter():
    Q, K, V = _rand(21, 2, 1, 8, 4)
    O, lse = orc.prefill_attn(Q, K, V)
    rows = [0, 5, 20]
    Os, ls = orc.prefill_attn(Q, K, V, rows=rows)
    np.testing.assert_array_equal(Os, O[rows])
    np.testing.assert_array_equal(ls, lse[:, rows])
    K2, V2 = K.copy(), V.copy()
    K2[6:] = 1e6
    V2[6:] = np.nan
    O5, _ = orc.prefill_attn(Q, K2, V2, rows=[5])
    np.testing.assert_array_equal(O5[0], O[5])
