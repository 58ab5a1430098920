"""Pins for the oracle's SelectChunks / UpdateDraftCache (Algorithm 1, Section 3.2.1)."""
import itertools

import numpy as np
import pytest

from oracle import specext_oracle as orc


def _brute_force_topk(key, k):
    """Definition by exhaustive comparison: chunk c is kept iff fewer than k chunks beat it,
    where a beats c when key[a] > key[c], or key[a] == key[c] and a < c."""
    NC = len(key)
    keep = []
    for c in range(NC):
        beaten_by = sum(1 for a in range(NC) if key[a] > key[c] or (key[a] == key[c] and a < c))
        if beaten_by < k:
            keep.append(c)
    return np.array(keep, dtype=np.int32)


@pytest.mark.parametrize("NC", [1, 5, 32])
def test_select_equals_brute_force(NC):
    rng = np.random.default_rng(NC)
    C = 4
    for L in (NC * C, NC * C - 3):
        lens = orc.chunk_lengths(L, C)
        assert lens.sum() == L and len(lens) == NC
        for trial in range(4):
            score = rng.random(NC).astype(np.float32)
            if trial >= 2:                                   # force many exact ties
                score = np.round(score * 3).astype(np.float32) * lens.astype(np.float32)
            key = score / lens.astype(np.float32)
            for k in {1, max(1, NC - 1), NC, NC + 3}:
                got = orc.select_chunks(score, L, C, k)
                np.testing.assert_array_equal(got, _brute_force_topk(key, min(k, NC)))
                assert list(got) == sorted(got) and len(got) == min(k, NC)


def test_select_all_equal_and_k_at_least_nc():
    L, C = 40, 8
    score = np.full(5, 0.125, dtype=np.float32)
    np.testing.assert_array_equal(orc.select_chunks(score, L, C, 3), [0, 1, 2])
    np.testing.assert_array_equal(orc.select_chunks(score, L, C, 5), np.arange(5))
    np.testing.assert_array_equal(orc.select_chunks(score, L, C, 99), np.arange(5))


def test_select_ranks_by_mean_not_by_mass():
    # last chunk has 2 of 8 tokens: mass 0.05 means 0.025 per token, above 0.16/8 = 0.02
    score = np.array([0.16, 0.10, 0.05], dtype=np.float32)
    np.testing.assert_array_equal(orc.select_chunks(score, 18, 8, 1), [2])
    np.testing.assert_array_equal(orc.select_chunks(score, 18, 8, 2), [0, 2])


def test_select_tiny_exhaustive():
    """Every assignment of 3 score levels to 4 chunks, every k: compare with a stable full sort."""
    for levels in itertools.product([0.0, 1.0, 2.0], repeat=4):
        score = np.array(levels, dtype=np.float32)
        order = sorted(range(4), key=lambda c: -levels[c])   # Python's sort is stable: ties keep index order
        for k in range(1, 6):
            np.testing.assert_array_equal(orc.select_chunks(score, 16, 4, k), sorted(order[:k]))


def test_planted_needles_are_selected():
    rng = np.random.default_rng(3)
    NC = 64
    score = (rng.random(NC) * 0.001).astype(np.float32)
    needles = [5, 17, 40, 63]
    score[needles] = [0.5, 0.2, 0.1, 0.05]
    got = orc.select_chunks(score, NC * 32, 32, 8)
    assert set(needles) <= set(got.tolist())


def test_gather_equals_index_arithmetic():
    rng = np.random.default_rng(4)
    nl, L, H, D, C = 2, 37, 3, 4, 8
    cap = 48
    dK = rng.integers(-2**15, 2**15, size=(nl, cap, H, D)).astype(np.int16)     # raw 16-bit payload
    dV = rng.integers(-2**15, 2**15, size=(nl, cap, H, D)).astype(np.int16)
    idx = [1, 2, 4]                                                             # chunk 4 has 5 tokens
    K, V, n = orc.gather_kv(dK, dV, idx, L, C)
    assert n == 8 + 8 + 5 and K.shape == (nl, n, H, D) and K.dtype == dK.dtype
    pos = 0
    for c in idx:
        for o in range(min(C, L - c * C)):
            for l in range(nl):
                assert K[l, pos].tobytes() == dK[l, c * C + o].tobytes()
                assert V[l, pos].tobytes() == dV[l, c * C + o].tobytes()
            pos += 1
    assert pos == n
    # selecting every chunk reproduces the first L tokens
    K, V, n = orc.gather_kv(dK, dV, range(5), L, C)
    assert n == L
    np.testing.assert_array_equal(K, dK[:, :L])
    np.testing.assert_array_equal(V, dV[:, :L])
    # nothing selected
    K, V, n = orc.gather_kv(dK, dV, [], L, C)
    assert n == 0 and K.shape[1] == 0


def test_forced_sink_and_recent_chunks_by_set_definition():
    """The extension: forced chunks first, then the best of the rest, against a definition by sets."""
    rng = np.random.default_rng(9)
    NC, C = 12, 4
    L = NC * C - 1
    lens = orc.chunk_lengths(L, C).astype(np.float64)
    for trial in range(20):
        score = rng.random(NC)
        key = score / lens
        for n_sink, n_recent, k in [(0, 0, 3), (1, 0, 3), (0, 2, 3), (2, 2, 6), (2, 2, 4), (3, 2, 4), (1, 1, 1),
                                    (7, 7, 5), (0, 0, 12), (2, 1, 20)]:
            forced = sorted(set(range(min(n_sink, NC))) | set(range(max(0, NC - n_recent), NC)))
            keff = min(k, NC)
            if len(forced) >= keff:
                want = forced[:keff]                                     # sinks first: lowest indices
            else:
                rest = [c for c in range(NC) if c not in forced]
                rest.sort(key=lambda c: (-key[c], c))
                want = sorted(forced + rest[:keff - len(forced)])
            got = orc.select_chunks(score, L, C, k, n_sink=n_sink, n_recent=n_recent)
            assert got.tolist() == want, (n_sink, n_recent, k)
    # nothing forced: exactly the plain selection
    score = rng.random(NC)
    np.testing.assert_array_equal(orc.select_chunks(score, L, C, 5), orc.select_chunks(score, L, C, 5, n_sink=0, n_recent=0))
