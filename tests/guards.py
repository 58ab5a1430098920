"""Guard bands around every device buffer the library writes (test infrastructure).

compute-sanitizer is not available to these tests, so out-of-bounds writes are caught the plain
way: each buffer of a `GuardedHotPath` sits inside a larger allocation with a band of a fixed byte
pattern before and after it, and `check()` verifies after a call that every band is intact.
"""
from __future__ import annotations

from typing import List, Tuple

import torch

from paper_2505_20776_b200.hotpath import HotPath

BAND_BYTES = 4096
PATTERN = 0xA5


class GuardedAlloc:
    """Allocator of guarded device tensors; check() verifies every band handed out so far."""

    def __init__(self, device):
        self.device = torch.device(device)
        self._bands: List[Tuple[str, torch.Tensor]] = []

    _alloc = None           # filled in below (shared with GuardedHotPath)
    check = None


class GuardedHotPath(HotPath):
    """HotPath whose buffers (outputs, status words, indices, compact cache, workspace) are guarded."""

    def _alloc(self, shape, dtype) -> torch.Tensor:
        if not hasattr(self, "_bands"):
            self._bands: List[Tuple[str, torch.Tensor]] = []
        n = 1
        for s in shape:
            n *= int(s)
        item = torch.empty((), dtype=dtype).element_size()
        nbytes = n * item
        body = -(-nbytes // 256) * 256                     # keeps the inner buffer 256-byte aligned
        raw = torch.full((2 * BAND_BYTES + body,), PATTERN, dtype=torch.uint8, device=self.device)
        assert raw.data_ptr() % 256 == 0
        self._bands.append((f"{tuple(shape)}:{dtype}:front", raw[:BAND_BYTES]))
        self._bands.append((f"{tuple(shape)}:{dtype}:back", raw[BAND_BYTES + nbytes:]))
        return raw[BAND_BYTES:BAND_BYTES + nbytes].view(dtype).view(*shape)

    def check(self) -> None:
        """Raises if any byte next to a buffer was overwritten."""
        for name, band in self._bands:
            bad = (band != PATTERN).nonzero()
            assert bad.numel() == 0, f"guard band {name} overwritten at byte offsets {bad[:8].flatten().tolist()}"


GuardedAlloc._alloc = GuardedHotPath._alloc
GuardedAlloc.alloc = GuardedHotPath._alloc
GuardedAlloc.check = GuardedHotPath.check
