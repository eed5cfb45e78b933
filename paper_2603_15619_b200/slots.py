"""Book-keeping for a fixed-size depth slot buffer (the paper's discussion of bounded depth-KV slot caching: a budget of
S slots, and a policy that decides which entries are kept: the most recent ones, the ones of highest utility, or a
hybrid that reserves part of the slots for recency).

Host logic only.  The mechanisms are the library's: ``moda_attn_fwd_append`` may write the next layer's K, V over a slot
that the same call reads (so eviction needs no copy), and ``moda_depth_slot_mass`` gives a utility per slot (the
probability that the queries spent on it).  The operator does not depend on the order of the slots, so a buffer whose
slots hold the layers in any order is attended to correctly.

    buf = SlotBuffer(S, policy="hybrid", n_recent=2)
    for layer in range(n_layers):
        l = buf.filled                                   # slots 0 .. l-1 hold earlier layers
        slot = buf.next_slot(utility)                    # a free slot, else the policy's victim
        O, LSE = moda_attn_fwd_append(Q, K, V, cache, l, scale, cache, slot)
        utility = moda_depth_slot_mass(Q, cache_before, LSE, l, scale).sum((0, 1))   # of the slots that were read
        buf.record(slot, layer)
"""
from __future__ import annotations

from typing import Optional, Sequence


class SlotBuffer:
    POLICIES = ("window", "top", "hybrid")

    def __init__(self, S: int, policy: str = "window", n_recent: int = 0):
        if S < 1:
            raise ValueError("the slot budget S must be at least 1")
        if policy not in self.POLICIES:
            raise ValueError(f"policy must be one of {self.POLICIES}")
        if policy == "hybrid" and not 0 < n_recent < S:
            raise ValueError("a hybrid buffer reserves 0 < n_recent < S slots for the most recent layers")
        self.S, self.policy = int(S), policy
        self.n_recent = int(n_recent) if policy == "hybrid" else 0
        self.owner = [None] * self.S          # layer whose K, V each slot holds

    @property
    def filled(self) -> int:
        """Number of slots in use; they are slots 0 .. filled-1 (free slots are handed out in order)."""
        return sum(o is not None for o in self.owner)

    def layers(self):
        """Layers currently held, in slot order."""
        return [o for o in self.owner if o is not None]

    def next_slot(self, utility: Optional[Sequence[float]] = None) -> int:
        """Slot that the next layer's K, V go to: the first free slot, else the policy's victim.

        ``utility[i]`` (higher = keep) rates slot i; it is needed by "top" and "hybrid" once the buffer is full."""
        for i, o in enumerate(self.owner):
            if o is None:
                return i
        oldest_first = sorted(range(self.S), key=lambda i: self.owner[i])
        if self.policy == "window":
            return oldest_first[0]
        if utility is None or len(utility) != self.S:
            raise ValueError("a full buffer with a utility policy needs one utility value per slot")
        protected = set(oldest_first[self.S - self.n_recent:]) if self.n_recent else set()
        candidates = [i for i in oldest_first if i not in protected]          # ties go to the oldest layer
        return min(candidates, key=lambda i: float(utility[i]))

    def record(self, slot: int, layer: int) -> None:
        if not 0 <= slot < self.S:
            raise ValueError("slot outside the buffer")
        if self.owner[slot] is None and slot != self.filled:
            raise ValueError("free slots are filled in order")
        self.owner[slot] = int(layer)
