"""Small helpers shared by the tests (no method arithmetic)."""
import numpy as np
import torch


def f64(t: torch.Tensor) -> np.ndarray:
    """Exact conversion of a (bf16/fp32) torch tensor to a float64 numpy array."""
    return t.detach().to("cpu").to(torch.float64).numpy()


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """The raw 16-bit patterns of a bf16 tensor, for bit-exact comparisons."""
    return t.detach().to("cpu").contiguous().view(torch.int16).numpy()


def random_forest(rng: np.random.Generator, n: int) -> np.ndarray:
    return np.array([int(rng.integers(-1, i)) for i in range(n)], dtype=np.int32)
