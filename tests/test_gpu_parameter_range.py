"""Parity over the retrieval-parameter ranges the paper sweeps (Appendix D: chunk size 1..128, top-k
2..256 on 8K-token inputs) and at the extremely long inputs of Section 4.5 (64K and 128K tokens)."""
import numpy as np
import pytest
import torch

from tests.test_gpu_parity import check_attn, check_retrieval, make_hp
from workloads import synth

pytestmark = pytest.mark.gpu

TOP_KS = (2, 4, 8, 16, 32, 64, 128, 256)


@pytest.mark.parametrize("C", [1, 2, 4, 8, 16, 32, 64, 128])
def test_chunk_size_and_top_k_grid_at_8k(cuda_device, C):
    """One scored attention call per chunk size (every chunk score against the oracle), then select + gather
    for every top-k of the sweep on two rows (k clamps to the number of chunks where it exceeds it)."""
    L = 8192
    w = synth.Workload("grid", 32, 8, 128, L, 60, C, max(TOP_KS), "levels", "needle", seed=4000 + C)
    hp = make_hp(w, cuda_device)
    t = synth.make_layer(w)
    parent = synth.make_tree(w)
    _, _, cs = check_attn(hp, t, parent, L, C, tag=f"grid8k-C{C}")
    draft = synth.make_draft_kv(w)
    for k in TOP_KS:
        hp.k = k                                              # buffers are sized for the largest k
        check_retrieval(hp, cs, [37, 59], L, C, k, draft, tag=f"grid8k-C{C}")


@pytest.mark.parametrize("L", [65536, 131072])
def test_extremely_long_prefix(cuda_device, L):
    """64K and 128K prefixes (Llama-3.1-8B layer shape, 60-node tree, chunk 32, top-k 32): every output
    element and every chunk score against the full oracle layer; retrieval on two rows."""
    w = synth.Workload("long", 32, 8, 128, L, 60, 32, 32, "levels", "needle", needle_span=4096, seed=6000 + L)
    hp = make_hp(w, cuda_device)
    t = synth.make_layer(w)
    parent = synth.make_tree(w)
    _, _, cs = check_attn(hp, t, parent, L, 32, tag=f"long-L{L}")
    check_retrieval(hp, cs, [0, 37], L, 32, 32, synth.make_draft_kv(w), tag=f"long-L{L}")
