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


class ErrorRecord:
    """Collects the errors the parity tests measured, per configuration, and writes them as JSON.

    The file goes to the directory named by SPECEXT_RECORD_DIR (nothing is written when that is not
    set), so that a run can keep the achieved errors next to its other results.
    """

    def __init__(self, filename: str):
        self.filename = filename
        self.data = {}

    def add(self, tag, accumulate: bool = False, **values) -> None:
        import json
        import os
        if tag is None:
            return
        row = self.data.setdefault(tag, {})
        for k, v in values.items():
            v = float(v)
            row[k] = row.get(k, 0.0) + v if accumulate else max(row.get(k, 0.0), v)
        out = os.environ.get("SPECEXT_RECORD_DIR")
        if out:
            os.makedirs(out, exist_ok=True)
            with open(os.path.join(out, self.filename), "w") as f:
                json.dump(self.data, f, indent=1, sort_keys=True)
