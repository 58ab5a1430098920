"""Prefill (specext_prefill_attn, causal self-attention of the prompt) against the oracle's plain
definition: every row at small sizes, sampled rows at the prompt lengths of the paper's tables."""
import numpy as np
import pytest
import torch

from oracle import specext_oracle as orc
from paper_2505_20776_b200 import api
from tests.guards import GuardedAlloc
from tests.test_gpu_parity import LSE_ATOL, O_ATOL, RECORD
from tests.util import f64
from workloads import synth

pytestmark = pytest.mark.gpu


def _inputs(L, Hq, Hkv, seed, values="normal", cap=None):
    w = synth.Workload("prefill", Hq, Hkv, 128, L, 1, 32, 1, "chain", values, seed=seed, capacity=cap)
    t = synth.make_layer(w)
    # queries of all L tokens: generated like the keys (one row per token)
    wq = synth.Workload("prefill-q", Hq, Hq, 128, L, 1, 32, 1, "chain", values, seed=seed + 1)
    Q = synth.make_layer(wq)["K_prefix"][:L].contiguous()
    return Q, t["K_prefix"], t["V_prefix"]


def _run(dev, Q, K, V, scale=0.0):
    L, Hq, D = Q.shape
    ga = GuardedAlloc(dev)
    O = ga.alloc((L, Hq, D), torch.bfloat16).fill_(float("nan"))
    lse = ga.alloc((Hq, L), torch.float32).fill_(float("nan"))
    status = ga.alloc((1,), torch.int32).zero_()
    api.specext_prefill_attn(Q.to(dev), K.to(dev), V.to(dev), O, lse, status, scale)
    assert api.specext_read_status(status) == 0
    ga.check()
    return O, lse


def _compare(O, lse, Q, K, V, rows, tag, scale=None):
    L = Q.shape[0]
    O_ref, lse_ref = orc.prefill_attn(f64(Q), f64(K[:L]), f64(V[:L]), scale, rows=rows)
    Og, lg = f64(O)[rows], f64(lse)[:, rows]
    assert np.isfinite(Og).all() and np.isfinite(lg).all()
    o_err, l_err = np.abs(Og - O_ref).max(), np.abs(lg - lse_ref).max()
    RECORD.add(tag, o_max_abs=o_err, lse_max_abs=l_err)
    assert o_err <= O_ATOL, f"O max abs err {o_err:.3e}"
    assert l_err <= LSE_ATOL, f"lse max abs err {l_err:.3e}"


@pytest.mark.parametrize("Hq,Hkv", [(8, 2), (2, 2), (4, 2), (8, 1), (16, 1)])
@pytest.mark.parametrize("L", [1, 63, 64, 65, 129, 257, 700])
def test_prefill_every_row_small(cuda_device, Hq, Hkv, L):
    """Group sizes 4, 1, 2, 8 and 16 (blocks of 64, 256, 128, 32 and 16 tokens), lengths around the block and
    tile boundaries and a ragged one: every output row against the oracle."""
    Q, K, V = _inputs(L, Hq, Hkv, seed=100 + L + Hq)
    O, lse = _run(cuda_device, Q, K, V)
    _compare(O, lse, Q, K, V, list(range(L)), f"prefill-small-G{Hq // Hkv}")


def test_prefill_explicit_scale_and_memory_beyond_the_prompt(cuda_device):
    """K/V buffers longer than the prompt, NaN beyond it; Q and O views with padded rows; explicit scale."""
    dev = cuda_device
    L, cap = 333, 512
    Q, K, V = _inputs(L, 8, 2, seed=7, cap=cap)
    K, V = K.clone(), V.clone()
    K[L:] = float("nan")
    V[L:] = float("nan")
    Kbig = torch.full((cap, 3, 136), float("nan"), dtype=torch.bfloat16, device=dev)
    Vbig = torch.full((cap, 3, 136), float("nan"), dtype=torch.bfloat16, device=dev)
    Kbig[:, 1:3, :128] = K.to(dev)
    Vbig[:, 1:3, :128] = V.to(dev)
    Qbig = torch.zeros(L, 8, 256, dtype=torch.bfloat16, device=dev)
    Qbig[:, :, :128] = Q.to(dev)
    Obig = torch.full((L, 8, 256), 7.0, dtype=torch.bfloat16, device=dev)
    lse = torch.empty(8, L, dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    api.specext_prefill_attn(Qbig[:, :, :128], Kbig[:, 1:3, :128], Vbig[:, 1:3, :128], Obig[:, :, :128], lse, status,
                             0.07)
    assert api.specext_read_status(status) == 0
    assert (Obig[:, :, 128:] == 7.0).all()                          # the padding of the output view is untouched
    _compare(Obig[:, :, :128], lse, Q, K, V, list(range(L)), "prefill-strided", scale=0.07)


@pytest.mark.parametrize("L", [4096, 16384])
def test_prefill_llama8b_shape_sampled_rows(cuda_device, L):
    """Llama-3.1-8B layer shape with the needle-structured keys of the benchmark configurations: rows at the
    block and tile boundaries plus seeded random ones, all 32 heads each."""
    Q, K, V = _inputs(L, 32, 8, seed=900 + L, values="needle")
    O, lse = _run(cuda_device, Q, K, V)
    rng = np.random.default_rng(L)
    rows = sorted(set([0, 1, 63, 64, 127, 128, 129, 191, 192, L // 2 - 1, L // 2, L - 65, L - 64, L - 1] +
                      rng.integers(0, L, 24).tolist()))
    _compare(O, lse, Q, K, V, rows, f"prefill-llama8b-L{L}")


def test_prefill_host_side_rejection(cuda_device):
    dev = cuda_device
    Q = torch.zeros(16, 4, 64, dtype=torch.bfloat16, device=dev)     # head_dim 64 is not built
    K = torch.zeros(16, 2, 64, dtype=torch.bfloat16, device=dev)
    O = torch.zeros_like(Q)
    lse = torch.zeros(4, 16, dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    with pytest.raises(api.SpecextError) as e:
        api.specext_prefill_attn(Q, K, K, O, lse, status)
    assert e.value.code == 2
