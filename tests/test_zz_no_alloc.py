"""The workspace-free entry point, for callers that are not allowed to allocate device memory
(all memory already handed to a pool they do not own, plug-in sandboxes, out-of-memory recovery).

It must give what the ordinary entry point gives.  The file name sorts last so that a run that stops
at the first failure has already run every other test; the test also passes alone in a fresh process.
"""
import numpy as np
import pytest
import torch

from paper_2505_20776_b200 import api
from workloads import synth

pytestmark = pytest.mark.gpu

O_ATOL = 1e-2
LSE_ATOL = 1e-3
SCORE_RTOL = 1e-3


def _run(entry, w, t, parent, dev, with_workspace, check_no_alloc=False):
    T, Hq, D = t["Q"].shape
    O = torch.full((T, Hq, D), float("nan"), dtype=torch.bfloat16, device=dev)
    lse = torch.full((Hq, T), float("nan"), dtype=torch.float32, device=dev)
    cs = torch.full((T, w.n_chunks), float("nan"), dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    d = api.make_attn_desc(t["Q"], t["K_prefix"], t["K_tree"], O, w.prefix_len, w.chunk_size, 0.0, True)
    args = (d, t["Q"], t["K_prefix"], t["V_prefix"], t["K_tree"], t["V_tree"], parent, O, lse, cs)
    if with_workspace:
        ws = torch.zeros(api.specext_verify_attn_workspace(d), dtype=torch.uint8, device=dev)
        entry(*args, ws, status)
    else:
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info(dev)
        held_before = torch.cuda.memory_allocated(dev)
        entry(*args, status)
        torch.cuda.synchronize()
        if check_no_alloc:
            # neither the driver's free memory nor torch's allocator moved while the call ran
            assert torch.cuda.mem_get_info(dev)[0] == free_before
            assert torch.cuda.memory_allocated(dev) == held_before
    assert api.specext_read_status(status) == 0
    return O.cpu(), lse.cpu(), cs.cpu()


def test_static_scratch_entry_matches_the_ordinary_one(cuda_device):
    dev = cuda_device
    for name, L in (("c1", 4096), ("c0", 1024)):                 # two calls in a row, different shapes
        w = synth.WORKLOADS[name].with_prefix(L)
        t = {k: v.to(dev) for k, v in synth.make_layer(w).items()}
        parent = torch.from_numpy(synth.make_tree(w)).to(dev)
        want = _run(api.specext_verify_attn, w, t, parent, dev, True)
        # within the tolerances of the parity tests ...
        for i in range(2):                                         # and the same shape twice
            # (the first call on a device looks the array's address up, which may load the module)
            got = _run(api.specext_verify_attn_static_scratch, w, t, parent, dev, False, check_no_alloc=i > 0)
            assert (got[0].float() - want[0].float()).abs().max().item() <= O_ATOL
            assert (got[1] - want[1]).abs().max().item() <= LSE_ATOL
            assert ((got[2] - want[2]).abs() / want[2]).max().item() <= SCORE_RTOL
            # ... and, since both entries run the same kernels on the same plan, bit for bit: a scratch
            # address that aliased live data would show up here even if it stayed inside the tolerances
            for a, b in zip(got, want):
                assert torch.equal(a, b)


def test_static_scratch_entry_rejects_what_does_not_fit(cuda_device):
    dev = cuda_device
    w = synth.WORKLOADS["c3"]                                      # 256K prefix with scores: > 32 MiB of scratch
    t = {k: v.to(dev) for k, v in synth.make_layer(w.with_prefix(256), capacity=256).items()}
    O = torch.empty_like(t["Q"])
    d = api.make_attn_desc(t["Q"], t["K_prefix"], t["K_tree"], O, 1 << 18, w.chunk_size, 0.0, True)
    assert api.specext_verify_attn_workspace(d) > api.STATIC_SCRATCH_BYTES
    lse = torch.empty(w.n_q_heads, w.n_tree, dtype=torch.float32, device=dev)
    cs = torch.empty(w.n_tree, 8192, dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    parent = torch.from_numpy(synth.make_tree(w)).to(dev)
    with pytest.raises(api.SpecextError) as e:
        api.specext_verify_attn_static_scratch(d, t["Q"], t["K_prefix"], t["V_prefix"], t["K_tree"], t["V_tree"],
                                               parent, O, lse, cs, status)
    assert e.value.code == 3
