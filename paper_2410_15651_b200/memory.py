"""Phase-boundary memory accounting for a PPO step built on this library.

The paper's subject is the memory that PyTorch's caching allocator holds: *reserved* (taken from the
driver) against *allocated* (live tensors), their difference as fragmentation, and the remedy of
releasing the cache after each inference and training phase (Sections 2.2 and 3.3, Appendix A).
This module records those quantities around the phases of the token-level path, so that a caller
can see what the path itself costs: the library allocates nothing (every buffer is the caller's),
the experience phase needs O(B*T) floats, and the loss phase needs one bf16 [B,T,V] gradient -- or
nothing at all when the gradient overwrites the logits in place.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, Dict, List

import torch


@dataclass
class PhaseRecord:
    name: str
    allocated_before: int
    reserved_before: int
    allocated_after: int
    reserved_after: int
    peak_allocated: int
    peak_reserved: int
    driver_used_before: int
    driver_used_after: int

    @property
    def fragmentation_after(self) -> int:
        """Reserved but not allocated bytes when the phase ends (what a later cudaMalloc cannot use)."""
        return self.reserved_after - self.allocated_after


@dataclass
class PhaseMemory:
    """Runs phases and records allocator statistics around each; optionally releases the cache after
    each phase, which is the paper's proposal."""
    device: torch.device
    empty_cache_after_phase: bool = False
    records: List[PhaseRecord] = field(default_factory=list)

    def _driver_used(self) -> int:
        free, total = torch.cuda.mem_get_info(self.device)
        return total - free

    def run(self, name: str, fn: Callable[[], object]):
        torch.cuda.synchronize(self.device)
        torch.cuda.reset_peak_memory_stats(self.device)
        a0, r0, d0 = (torch.cuda.memory_allocated(self.device), torch.cuda.memory_reserved(self.device),
                      self._driver_used())
        out = fn()
        torch.cuda.synchronize(self.device)
        rec = PhaseRecord(name, a0, r0, torch.cuda.memory_allocated(self.device),
                          torch.cuda.memory_reserved(self.device), torch.cuda.max_memory_allocated(self.device),
                          torch.cuda.max_memory_reserved(self.device), d0, self._driver_used())
        self.records.append(rec)
        if self.empty_cache_after_phase:
            torch.cuda.empty_cache()
        return out

    def summary(self) -> Dict[str, Dict[str, int]]:
        return {r.name: {"allocated_delta": r.allocated_after - r.allocated_before,
                         "reserved_delta": r.reserved_after - r.reserved_before,
                         "peak_allocated_over_start": r.peak_allocated - r.allocated_before,
                         "fragmentation_after": r.fragmentation_after,
                         "driver_used_delta": r.driver_used_after - r.driver_used_before}
                for r in self.records}
