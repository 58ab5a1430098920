"""Seeded synthetic inputs for the verification hot path (test and bench infrastructure).

This module holds no arithmetic of the method itself (no attention, softmax, top-k or gather):
it only produces tensors of the shapes and value structure that the paper's workloads have, so
that the CUDA path and the CPU oracle can be fed exactly the same bytes.

All bulk values come from a counter-based generator written in integer torch ops, which wrap
identically on CPU and CUDA, followed by correctly rounded fp32 elementwise ops and one
round-to-nearest-even conversion to bf16.  The same call therefore yields bit-identical tensors on
either device, which lets a benchmark fill gigabytes of K/V directly in device memory while a
parity test regenerates any layer on the host for the oracle.

Workload shapes follow the paper's setup: Llama-3.1-8B-Instruct / 70B-class GQA layer shapes,
prefixes of 1K..32K tokens (Tables 2 and 6), draft trees of ~50-60 nodes (Appendix C), chunk size
32 and a ~1K-token working draft cache (Appendix D).  They stand in for the GovReport / PG-19 /
BookSum / AIME-24 prompts, none of which is reproduced here.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Optional, Tuple

import numpy as np
import torch

_M64 = (1 << 64) - 1


def _s64(x: int) -> int:
    """Reinterpret an unsigned 64-bit Python int as signed (torch int64 scalar range)."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


_C1 = _s64(0xBF58476D1CE4E5B9)
_C2 = _s64(0x94D049BB133111EB)
_GOLD = 0x9E3779B97F4A7C15


def _lsr(z: torch.Tensor, n: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor (torch's >> is arithmetic)."""
    return (z >> n) & ((1 << (64 - n)) - 1)


def _mix64(z: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser on wrapping int64 tensors."""
    z = (z ^ _lsr(z, 30)) * _C1
    z = (z ^ _lsr(z, 27)) * _C2
    return z ^ _lsr(z, 31)


def _mix64_int(z: int) -> int:
    z &= _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def stream_key(seed: int, *ids: int) -> int:
    """Fold a seed and a tuple of small integers (tensor id, layer, ...) into one 64-bit key."""
    k = _mix64_int(seed * _GOLD + 0x1234567)
    for i in ids:
        k = _mix64_int(k ^ ((int(i) + 1) * _GOLD))
    return k


def std_normal(key: int, start: int, count: int, device) -> torch.Tensor:
    """count fp32 values ~ approximately N(0,1), element i a pure function of (key, start+i).

    Two hashed 64-bit words give eight 16-bit fields; their sum S is Irwin-Hall(8) scaled, with
    mean 262140 and standard deviation 65536*sqrt(8/12) ~= 53510.  x = (S - 262140) / 53510 is an
    exact integer followed by one correctly rounded fp32 division.
    """
    out = torch.empty(count, dtype=torch.float32, device=device)
    step = 1 << 22
    k = _s64(key)
    for lo in range(0, count, step):
        n = min(step, count - lo)
        ctr = torch.arange(start + lo, start + lo + n, dtype=torch.int64, device=device) * 2
        s = torch.zeros(n, dtype=torch.int64, device=device)
        for w in range(2):
            h = _mix64((ctr + w) ^ k)
            for f in range(4):
                s += (h >> (16 * f)) & 0xFFFF
        out[lo:lo + n] = (s - 262140).to(torch.float32) / 53510.0
    return out


def uniform01_int(key: int, n: int) -> np.ndarray:
    """n doubles in [0,1), host side, element i a pure function of (key, i)."""
    return np.array([(_mix64_int(key ^ ((i + 1) * _GOLD)) >> 11) / float(1 << 53) for i in range(n)])


@dataclasses.dataclass(frozen=True)
class Workload:
    """One synthetic configuration (shapes of a single attention layer plus retrieval parameters)."""
    name: str
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    prefix_len: int
    n_tree: int
    chunk_size: int
    top_k: int
    tree: str            # "uniform": parent[i] ~ U{-1..i-1};  "levels": 6 levels x 10 nodes
    values: str          # "normal" or "needle"
    n_layers: int = 1
    capacity: Optional[int] = None     # KV buffer capacity when the cache is appended in place
    draft_kv_heads: Optional[int] = None
    draft_head_dim: Optional[int] = None
    needle_span: Optional[int] = None  # needles fall in the first needle_span tokens (default: all)
    seed: int = 20776

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def n_chunks(self) -> int:
        return -(-self.prefix_len // self.chunk_size)

    def with_prefix(self, prefix_len: int) -> "Workload":
        return dataclasses.replace(self, prefix_len=prefix_len)


WORKLOADS: Dict[str, Workload] = {
    # tiny single layer: 4 query heads on 1 KV head, D=64, 1K prefix, 8-node random tree
    "c0": Workload("c0", 4, 1, 64, 1024, 8, 32, 8, "uniform", "normal", seed=20776),
    # Llama-3.1-8B-shaped layer, 4K prefix, 60-node level tree
    "c1": Workload("c1", 32, 8, 128, 4096, 60, 32, 32, "levels", "needle", seed=20777),
    # same shape, 16K prefix, 32 layers with independent K/V; scores from the last layer
    "c2": Workload("c2", 32, 8, 128, 16384, 60, 32, 32, "levels", "needle", n_layers=32, seed=20778),
    # growth sweep 1K..32K inside one buffer of capacity 32K (prefix_len is set per step)
    "c3": Workload("c3", 32, 8, 128, 32768, 60, 32, 32, "levels", "needle", capacity=32768,
                   needle_span=1024, seed=20779),
    # 70B-class layer: 64 query heads on 8 KV heads (480 stacked rows per KV head), chunk 64
    "c4": Workload("c4", 64, 8, 128, 16384, 60, 64, 32, "levels", "needle", seed=20780),
}
C3_LENGTHS = (1024, 2048, 4096, 8192, 16384, 32768)

_TID = {"q": 1, "kp": 2, "vp": 3, "kt": 4, "vt": 5, "dk": 6, "dv": 7, "u": 8, "delta": 9, "needle": 10,
        "tree": 11}


def make_tree(w: Workload, seed: Optional[int] = None) -> np.ndarray:
    """parent[] (int32, -1 = child of the prefix, parent[i] < i) for the workload's tree recipe."""
    seed = w.seed if seed is None else seed
    key = stream_key(seed, _TID["tree"])
    u = uniform01_int(key, w.n_tree)
    parent = np.empty(w.n_tree, dtype=np.int32)
    if w.tree == "uniform":
        for i in range(w.n_tree):
            parent[i] = int(u[i] * (i + 1)) - 1          # uniform in {-1, .., i-1}
    elif w.tree == "levels":
        width = 10
        for i in range(w.n_tree):
            level = i // width
            if level == 0:
                parent[i] = -1
            else:
                lo = (level - 1) * width
                parent[i] = lo + int(u[i] * width)        # uniform over the previous level
    elif w.tree == "chain":
        parent[:] = np.arange(w.n_tree) - 1
    else:
        raise ValueError(w.tree)
    return parent


def needle_profile(w: Workload, n_chunks: int, background: str, seed: Optional[int] = None
                   ) -> Tuple[np.ndarray, np.ndarray]:
    """Per-chunk logit boosts (float64 [n_chunks]) and the four needle chunk ids.

    Needles get boosts 6, 5, 4, 3.  Elsewhere the boost is 0 ("flat") or U(0,1) per chunk
    ("graded"); chunk c's value depends on (seed, c) only, so a longer prefix reveals more chunks
    without changing the earlier ones.
    """
    seed = w.seed if seed is None else seed
    if background == "flat":
        delta = np.zeros(n_chunks)
    elif background == "graded":
        delta = uniform01_int(stream_key(seed, _TID["delta"]), n_chunks)
    else:
        raise ValueError(background)
    nk = stream_key(seed, _TID["needle"])
    span = n_chunks if w.needle_span is None else max(1, min(n_chunks, w.needle_span // w.chunk_size))
    ids = []
    i = 0
    while len(ids) < min(4, span):
        c = _mix64_int(nk ^ ((i + 1) * _GOLD)) % span
        i += 1
        if c not in ids:
            ids.append(int(c))
    for c, boost in zip(ids, (6.0, 5.0, 4.0, 3.0)):
        delta[c] = boost
    return delta, np.array(ids, dtype=np.int64)


def _unit_vectors(w: Workload, seed: int) -> torch.Tensor:
    """One seeded unit vector per KV head, fp32 [Hkv][D], always computed on the host."""
    z = std_normal(stream_key(seed, _TID["u"]), 0, w.n_kv_heads * w.head_dim, "cpu")
    z = z.view(w.n_kv_heads, w.head_dim).double()
    return (z / z.norm(dim=1, keepdim=True)).float()


def make_layer(w: Workload, layer: int = 0, device="cpu", background: str = "graded",
               seed: Optional[int] = None, capacity: Optional[int] = None
               ) -> Dict[str, torch.Tensor]:
    """Q, prefix K/V and tree K/V of one layer as bf16 tensors on `device`.

    Layouts: Q [T][Hq][D]; K_prefix, V_prefix [capacity or L][Hkv][D]; K_tree, V_tree [T][Hkv][D].
    "normal": every element ~ N(0,1).  "needle": Q = z/sqrt(D) + a*u_g, K = z/sqrt(D) + b_c*u_g
    with a = 8 and b_c = delta_c * sqrt(D) / a, so that the scaled logit of a key in chunk c is
    raised by delta_c; V ~ N(0,1).
    """
    seed = w.seed if seed is None else seed
    T, Hq, Hkv, D, C = w.n_tree, w.n_q_heads, w.n_kv_heads, w.head_dim, w.chunk_size
    cap = capacity or w.capacity or w.prefix_len
    dev = torch.device(device)

    def nrm(tid, n):
        return std_normal(stream_key(seed, _TID[tid], layer), 0, n, dev)

    q = nrm("q", T * Hq * D).view(T, Hq, D)
    kp = nrm("kp", cap * Hkv * D).view(cap, Hkv, D)
    vp = nrm("vp", cap * Hkv * D).view(cap, Hkv, D)
    kt = nrm("kt", T * Hkv * D).view(T, Hkv, D)
    vt = nrm("vt", T * Hkv * D).view(T, Hkv, D)
    if w.values == "needle":
        a = 8.0
        inv = 1.0 / math.sqrt(D)
        u = _unit_vectors(w, seed).to(dev)                               # [Hkv][D]
        nc = -(-cap // C)
        delta, _ = needle_profile(w, nc, background, seed)
        b = torch.tensor(delta * math.sqrt(D) / a, dtype=torch.float32)   # [nc]
        b_tok = b.to(dev).repeat_interleave(C)[:cap].view(cap, 1, 1)
        q = q * inv
        q = q + (a * u).repeat_interleave(w.group, dim=0).view(1, Hq, D)
        kp = kp * inv
        kp = kp + b_tok * u.view(1, Hkv, D)
        kt = kt * inv
    elif w.values != "normal":
        raise ValueError(w.values)
    bf = torch.bfloat16
    return {"Q": q.to(bf).contiguous(), "K_prefix": kp.to(bf).contiguous(),
            "V_prefix": vp.to(bf).contiguous(), "K_tree": kt.to(bf).contiguous(),
            "V_tree": vt.to(bf).contiguous()}


def make_draft_kv(w: Workload, device="cpu", n_layers: int = 1, seed: Optional[int] = None,
                  capacity: Optional[int] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """The draft model's full KV cache, bf16 [n_layers][capacity or L][Hkv_d][D_d], ~ N(0,1)."""
    seed = w.seed if seed is None else seed
    cap = capacity or w.capacity or w.prefix_len
    h = w.draft_kv_heads or w.n_kv_heads
    d = w.draft_head_dim or w.head_dim
    n = n_layers * cap * h * d
    dk = std_normal(stream_key(seed, _TID["dk"]), 0, n, torch.device(device))
    dv = std_normal(stream_key(seed, _TID["dv"]), 0, n, torch.device(device))
    return (dk.view(n_layers, cap, h, d).to(torch.bfloat16).contiguous(),
            dv.view(n_layers, cap, h, d).to(torch.bfloat16).contiguous())
