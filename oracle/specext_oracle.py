"""CPU oracle for the verification hot path of speculative decoding with Cross-model Retrieval.

TEST INFRASTRUCTURE ONLY.  This file is the plain, slow definition that the CUDA library is
checked against.  Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
it; the product never does, and this file imports nothing from the product.

Everything is fp64 numpy on inputs that were converted exactly from bf16.  The paper fixes no
precision.  A matrix product (numpy matmul) is the only library primitive used as a step; there is
no tiling, no online softmax and no fusion: every query row's full masked score vector over
prefix + tree keys is materialised, normalised once, and then reduced.

What the path computes, with the passage each part follows:

* Tree attention over the target model's full prefix KV cache plus the draft tree itself, the
  tree restricted by the ancestor mask (Section 3.1, "Efficient Attention": Hybrid Tree Attention
  makes the split-over-KV decoding kernel usable with tree-structured attention).  Because
  splitting over the KV length and merging by log-sum-exp is an exact re-association, the oracle
  is ordinary softmax attention with a mask.
* The attention scores the retrieval step consumes (Section 3.2.1, "Method Overview": the prefix
  is cut into fixed-size chunks which are ranked by their average attention score; scores come
  from the last layer of the most recent verification pass).
* SelectChunks and UpdateDraftCache of Algorithm 1 (Appendix A): keep the top-k chunks and
  rewrite the draft model's KV cache to hold only those.
* The prefill of the prompt (Section 3.1: FlashAttention for the prefill stage of target and draft
  model): ordinary causal self-attention.

Readings taken where the paper is silent (each one is a stated choice of this build, not a fact of the paper):
a tree node attends to itself and its ancestors; query head h reads KV head h // (Hq/Hkv); the
softmax normaliser covers prefix and visible tree keys together; a chunk's exported score is the
mean over all query heads of its summed probability ("mass"), and chunks are ranked by
mass / chunk length so that a short trailing chunk competes on its average; ties go to the lower
chunk index; selected indices are reported in ascending order; k is clamped to the chunk count.

Pins (tests/test_oracle_*.py): rows of P sum to one and masked entries are exactly zero; a single
visible key returns its V; the two-key closed form; a chain tree equals causal attention and a
general tree equals masked attention as computed by torch's fp64 scaled_dot_product_attention;
lse equals torch.logsumexp; zero queries give mass len_c / (L + depth + 1); a rank-one
construction with exactly representable logits gives closed-form masses and outputs; a hand-worked
rational example (tests/golden); select equals a brute-force sort; gather equals index
arithmetic; the prefill equals torch's fp64 causal scaled_dot_product_attention, its first token
returns V[0], and its block b equals verify_attn with the earlier tokens as prefix and the block as a
chain tree.  No function here is unpinned.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import numpy as np


class BadTree(ValueError):
    """parent[] is not a forest in topological order (parent[i] must lie in [-1, i-1])."""


def ancestor_mask(parent: Sequence[int]) -> np.ndarray:
    """anc[t][u] is True iff u == t or u is a proper ancestor of t (tree attention mask).

    parent[i] == -1 marks a node whose parent is the last prefix token; several such roots are
    allowed.  Section 3.1 (tree-structured attention of the verification step).
    """
    T = len(parent)
    anc = np.zeros((T, T), dtype=bool)
    for t in range(T):
        p = int(parent[t])
        if p < -1 or p >= t:
            raise BadTree(f"parent[{t}] = {p} is outside [-1, {t - 1}]")
        if p >= 0:
            anc[t, :] = anc[p, :]
        anc[t, t] = True
    return anc


def depth(parent: Sequence[int]) -> np.ndarray:
    """Number of proper ancestors of each node inside the tree."""
    return ancestor_mask(parent).sum(axis=1) - 1


def verify_attn(Q: np.ndarray, K_prefix: np.ndarray, V_prefix: np.ndarray,
                K_tree: np.ndarray, V_tree: np.ndarray, parent: Sequence[int],
                chunk_size: int, scale: Optional[float] = None, return_probs: bool = False):
    """Tree attention over prefix + tree and the per-chunk attention mass of the prefix.

    Q [T][Hq][D]; K_prefix, V_prefix [L][Hkv][D]; K_tree, V_tree [T][Hkv][D]; all float64.
    Returns O [T][Hq][D], lse [Hq][T] (natural log, scale included), chunk_score [T][NC] with
    NC = ceil(L / chunk_size), and, if asked, P [Hq][T][L+T].

    Section 3.1 (attention) and Section 3.2.1 (chunk scores from the attention matrix).
    """
    Q = np.asarray(Q, dtype=np.float64)
    Kp = np.asarray(K_prefix, dtype=np.float64)
    Vp = np.asarray(V_prefix, dtype=np.float64)
    Kt = np.asarray(K_tree, dtype=np.float64)
    Vt = np.asarray(V_tree, dtype=np.float64)
    T, Hq, D = Q.shape
    L, Hkv, _ = Kp.shape
    assert Hq % Hkv == 0 and Kt.shape == (T, Hkv, D) and Vt.shape == (T, Hkv, D)
    G = Hq // Hkv
    C = int(chunk_size)
    NC = -(-L // C)
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    anc = ancestor_mask(parent)

    O = np.zeros((T, Hq, D))
    lse = np.zeros((Hq, T))
    mass = np.zeros((Hq, T, NC))
    probs = np.zeros((Hq, T, L + T)) if return_probs else None
    for h in range(Hq):
        g = h // G
        keys = np.concatenate([Kp[:, g, :], Kt[:, g, :]], axis=0)        # [L+T][D]
        vals = np.concatenate([Vp[:, g, :], Vt[:, g, :]], axis=0)
        s = scale * (Q[:, h, :] @ keys.T)                                # [T][L+T]
        s[:, L:] = np.where(anc, s[:, L:], -np.inf)
        m = s.max(axis=1, keepdims=True)
        p = np.exp(s - m)
        Z = p.sum(axis=1, keepdims=True)
        P = p / Z
        lse[h, :] = (m + np.log(Z))[:, 0]
        O[:, h, :] = P @ vals
        for c in range(NC):
            mass[h, :, c] = P[:, c * C:min(L, (c + 1) * C)].sum(axis=1)
        if return_probs:
            probs[h] = P
    chunk_score = mass.mean(axis=0)                                      # [T][NC]
    if return_probs:
        return O, lse, chunk_score, probs
    return O, lse, chunk_score


def attn_split_merge(Q, K_prefix, V_prefix, K_tree, V_tree, parent, bounds: Sequence[int],
                     scale: Optional[float] = None) -> Tuple[np.ndarray, np.ndarray]:
    """The same attention computed the split-over-KV way: one partial per contiguous key range.

    bounds = [0, b1, ..., L] cuts the prefix; the tree is one more part.  Each part keeps its own
    maximum m, sum l and unnormalised output; parts are merged by log-sum-exp (Section 3.1, the
    decoding kernel parallelised over the KV length).  Used only to pin that the re-association
    is exact; returns (O, lse) shaped like verify_attn's.
    """
    Q = np.asarray(Q, dtype=np.float64)
    T, Hq, D = Q.shape
    L, Hkv, _ = K_prefix.shape
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    anc = ancestor_mask(parent)
    O = np.zeros((T, Hq, D))
    lse = np.zeros((Hq, T))
    for h in range(Hq):
        g = h // G
        parts = []
        for lo, hi in zip(bounds[:-1], bounds[1:]):
            if hi > lo:
                s = scale * (Q[:, h, :] @ np.asarray(K_prefix[lo:hi, g, :], dtype=np.float64).T)
                parts.append((s, np.asarray(V_prefix[lo:hi, g, :], dtype=np.float64)))
        st = scale * (Q[:, h, :] @ np.asarray(K_tree[:, g, :], dtype=np.float64).T)
        parts.append((np.where(anc, st, -np.inf), np.asarray(V_tree[:, g, :], dtype=np.float64)))
        ms, ls, os_ = [], [], []
        for s, v in parts:
            m = s.max(axis=1)
            p = np.exp(s - m[:, None])
            ms.append(m)
            ls.append(p.sum(axis=1))
            os_.append(p @ v)
        M = np.max(np.stack(ms), axis=0)
        Z = sum(l * np.exp(m - M) for m, l in zip(ms, ls))
        acc = sum(o * np.exp(m - M)[:, None] for m, o in zip(ms, os_))
        O[:, h, :] = acc / Z[:, None]
        lse[h, :] = M + np.log(Z)
    return O, lse


def prefill_attn(Q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: Optional[float] = None,
                 rows: Optional[Sequence[int]] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Causal self-attention of the prompt (the prefill that Section 3.1 runs with FlashAttention).

    Q [L][Hq][D], K, V [L][Hkv][D].  Token i attends to tokens 0..i (itself included), query head
    h reads KV head h // (Hq/Hkv).  Plain definition, one query row at a time: the masked score
    vector of the row is materialised, normalised once and multiplied with V.  `rows` restricts
    the computation to those token positions (outputs are then indexed by position in `rows`),
    which is how a long prompt is spot-checked.
    Returns (O [n_rows][Hq][D], lse [Hq][n_rows]), natural logarithm, scale included.
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    L, Hq, D = Q.shape
    Hkv = K.shape[1]
    assert K.shape == V.shape == (L, Hkv, D) and Hq % Hkv == 0
    G = Hq // Hkv
    scale = 1.0 / np.sqrt(D) if scale is None else float(scale)
    rows = list(range(L)) if rows is None else [int(r) for r in rows]
    O = np.zeros((len(rows), Hq, D))
    lse = np.zeros((Hq, len(rows)))
    for n, i in enumerate(rows):
        assert 0 <= i < L
        for h in range(Hq):
            g = h // G
            s = scale * (K[: i + 1, g, :] @ Q[i, h, :])          # visible keys only: 0..i
            m = s.max()
            p = np.exp(s - m)
            Z = p.sum()
            O[n, h, :] = (p / Z) @ V[: i + 1, g, :]
            lse[h, n] = m + np.log(Z)
    return O, lse


def chunk_lengths(prefix_len: int, chunk_size: int) -> np.ndarray:
    """len_c = min(C, L - c*C): every chunk is full except possibly the last."""
    NC = -(-prefix_len // chunk_size)
    return np.minimum(chunk_size, prefix_len - np.arange(NC) * chunk_size).astype(np.int64)


def select_chunks(chunk_score_row: np.ndarray, prefix_len: int, chunk_size: int, k: int,
                  key_dtype=np.float64, n_sink: int = 0, n_recent: int = 0) -> np.ndarray:
    """SelectChunks of Algorithm 1: indices of the top-k chunks, ascending.

    chunk_score_row [NC] holds summed probability per chunk; the ranking key is the chunk's
    average score, mass / len_c (Section 3.2.1).  Order: key descending, chunk index ascending
    among equal keys; the first min(k, NC) are kept and returned sorted by index.  n_sink / n_recent
    (an extension, default 0) force the earliest / latest chunks into the selection.  The key is
    formed in `key_dtype`: fp64 by default (the plain definition).  A test that hands the same
    fp32 score row to the oracle and to another implementation may ask for np.float32, so that
    the integer decision is taken in the same arithmetic on both sides.
    """
    score = np.asarray(chunk_score_row)
    NC = score.shape[0]
    assert NC == -(-prefix_len // chunk_size)
    assert n_sink >= 0 and n_recent >= 0
    lens = chunk_lengths(prefix_len, chunk_size)
    key = (score.astype(key_dtype) / lens.astype(key_dtype)).astype(key_dtype)
    # Optional extension (the paper's retrieval forces nothing: n_sink = n_recent = 0): the first n_sink
    # and the last n_recent chunks are kept whatever their score, i.e. they rank above every other chunk
    # (lower index first among themselves); the remaining places go to the best of the rest.
    forced = [c < n_sink or c >= NC - n_recent for c in range(NC)]
    order = sorted(range(NC), key=lambda c: (0 if forced[c] else 1, 0.0 if forced[c] else -float(key[c]), c))
    keep = order[:min(int(k), NC)]
    return np.array(sorted(keep), dtype=np.int32)


def gather_kv(draft_K: np.ndarray, draft_V: np.ndarray, idx: Sequence[int], prefix_len: int,
              chunk_size: int) -> Tuple[np.ndarray, np.ndarray, int]:
    """UpdateDraftCache of Algorithm 1: the compact draft cache holding only the kept chunks.

    draft_K, draft_V [n_layers][L or more][H][D] (any dtype; copied, never converted).  Chunks
    are concatenated in the order of idx; a trailing partial chunk contributes its len_c tokens.
    Returns (K_out, V_out [n_layers][n_tokens][H][D], n_tokens).
    """
    spans: List[Tuple[int, int]] = []
    for c in idx:
        lo = int(c) * chunk_size
        hi = min(prefix_len, lo + chunk_size)
        assert 0 <= lo < hi
        spans.append((lo, hi))
    if not spans:
        z = draft_K[:, :0]
        return z.copy(), draft_V[:, :0].copy(), 0
    K_out = np.concatenate([draft_K[:, lo:hi] for lo, hi in spans], axis=1)
    V_out = np.concatenate([draft_V[:, lo:hi] for lo, hi in spans], axis=1)
    return K_out, V_out, K_out.shape[1]
