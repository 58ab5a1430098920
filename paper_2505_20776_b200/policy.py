"""When to run the retrieval update (host-side policy; Algorithm 1's doRetrieval flag).

Section 3.2.1 notes that, because context is local in long sequences, the draft cache need not be
rewritten after every verification step: updates "can be applied adaptively or less frequently".
Appendix D finds a fixed period of 4 steps (Vicuna-68M) or 8 steps (EAGLE) best.  The paper gives no
rule for "adaptively"; the adaptive rule here is this library's reading: keep the periodic update as a
floor and also update as soon as the draft model's acceptance has dropped, i.e. when the number of
accepted tokens of a verification step falls below a fraction of its running mean since the last update.

The schedule only decides; the caller runs specext_select_gather (or select + gather) when told to.
Nothing here touches the GPU.
"""
from __future__ import annotations

from dataclasses import dataclass, field


@dataclass
class RetrievalSchedule:
    """doRetrieval for decode step 0, 1, 2, ...

    period     : update every `period` steps (>= 1); the first step always updates, since the draft
                 cache starts empty (Algorithm 1 runs SelectChunks / UpdateDraftCache before the first Draft).
    adaptive   : also update when the last step accepted fewer than `drop` x the mean accepted length
                 observed since the previous update (needs at least `min_history` observations).
    """
    period: int = 4
    adaptive: bool = False
    drop: float = 0.5
    min_history: int = 2
    _since: int = field(default=0, init=False)           # verification steps since the last update
    _acc_sum: float = field(default=0.0, init=False)
    _acc_n: int = field(default=0, init=False)
    _started: bool = field(default=False, init=False)
    updates: int = field(default=0, init=False)
    steps: int = field(default=0, init=False)

    def __post_init__(self):
        if self.period < 1:
            raise ValueError("period must be >= 1")
        if not (0.0 < self.drop <= 1.0) or self.min_history < 1:
            raise ValueError("drop must be in (0, 1] and min_history >= 1")

    def observe(self, n_accepted: int) -> None:
        """Reports how many draft tokens the verification step that just finished accepted."""
        if n_accepted < 0:
            raise ValueError("n_accepted must be >= 0")
        self._last = float(n_accepted)
        self._acc_sum += n_accepted
        self._acc_n += 1

    def do_retrieval(self) -> bool:
        """Decision for the step about to start; call once per step, after observe() of the previous one."""
        self.steps += 1
        due = not self._started or self._since + 1 >= self.period
        if not due and self.adaptive and self._acc_n >= self.min_history + 1:
            # the mean excludes the observation being judged
            mean_before = (self._acc_sum - self._last) / (self._acc_n - 1)
            due = self._last < self.drop * mean_before
        if due:
            self._started = True
            self._since = 0
            self._acc_sum, self._acc_n = 0.0, 0
            self.updates += 1
        else:
            self._since += 1
        return due
