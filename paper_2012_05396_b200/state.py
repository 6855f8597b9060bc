"""Device-memory plumbing: allocates the arenas a context works on (torch tensors)."""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch

from . import binding as B


ARENA_ALIGN_BYTES = 4096
GUARD_BYTES = 4096
GUARD_WORD = 0x5AC3A53C          # int32 pattern of the guard words


class ArenaSlab:
    """`count` arenas of n elements carved out of ONE device allocation.

    Every arena starts on a 4 KB boundary: the kernels work with any 16-byte aligned buffers, but
    a block reads 4 KB of every stream per trip, and on B200 arenas that start off a 4 KB boundary
    cost about 3 % of bandwidth (measured on the VGG-16 and ResNet-50 workloads: 6.64 against
    6.85 TB/s).

    A guard page lies before the first arena, between neighbours and after the last one; guard
    pages and the padding behind each arena hold a fixed word.  `guards_intact()` tells whether
    any of them was overwritten, i.e. whether something stored outside an arena (up to 4 KB
    before its start or beyond its end).
    """

    def __init__(self, count: int, n: int, dtype=torch.float32, device="cuda"):
        self.count, self.n = count, n
        esize = torch.empty(0, dtype=dtype).element_size()
        self.arena_bytes = n * esize
        padded = -(-self.arena_bytes // ARENA_ALIGN_BYTES) * ARENA_ALIGN_BYTES
        self.stride = GUARD_BYTES + padded
        self.raw = torch.empty(count * self.stride + GUARD_BYTES, dtype=torch.uint8, device=device)
        words = self.raw.view(torch.int32)
        self.arenas: List[torch.Tensor] = []
        self._gaps: List[torch.Tensor] = []
        end_of_previous = 0
        for i in range(count):
            lo = i * self.stride + GUARD_BYTES
            self._gaps.append(words[end_of_previous // 4: lo // 4])
            self.arenas.append(self.raw[lo: lo + self.arena_bytes].view(dtype))
            end_of_previous = lo + self.arena_bytes
        self._gaps.append(words[end_of_previous // 4:])
        for gap in self._gaps:
            gap.fill_(GUARD_WORD)

    def damaged_gaps(self) -> List[int]:
        """Indices of the gaps that no longer hold the guard word (gap i lies before arena i)."""
        flags = torch.stack([(gap != GUARD_WORD).any() for gap in self._gaps])
        return torch.nonzero(flags).flatten().tolist()

    def guards_intact(self) -> bool:
        return not self.damaged_gaps()


def alloc_arenas(count: int, n: int, dtype=torch.float32, device="cuda") -> List[torch.Tensor]:
    """`count` 4 KB-aligned arenas of n elements out of one allocation (see ArenaSlab)."""
    if count == 0:
        return []
    return ArenaSlab(count, n, dtype, device).arenas


class DeviceState:
    """w, mom and the K workers' w_loc / pre / w_dev arenas on one CUDA device, plus the context.

    Untouched buffers are filled with `fill` (NaN by default) so that a read of something the
    schedule has not written yet shows up in any comparison.

    shared_pre: one pre_weight arena for all workers.  host_pre: pre_weight lives in ONE pinned
    host arena and is streamed through `pre_slots` device slices by ssd_step_host (the other
    delay-stage calls are then not available); `host_chunk` sets the chunk of that pipeline.
    merged_dev: no separate device weights (w_dev[i] is w_loc[i]; K arenas less).
    """

    def __init__(self, numels: Sequence[int], hp: B.ssd_hparams, w0: torch.Tensor,
                 device="cuda", fill: float = float("nan"), worker_state: bool = True,
                 shared_pre: bool = False, host_pre: bool = False, pre_slots: int = 2,
                 host_chunk: int = 0, merged_dev: bool = False):
        self.numels = [int(n) for n in numels]
        self.n = B.ssd_arena_numel(self.numels)
        assert w0.numel() == self.n and w0.dtype == torch.float32
        self.K = hp.K
        self.device = torch.device(device)
        n_pre = 0 if (not worker_state or host_pre) else (1 if shared_pre else self.K)
        self.merged_dev = bool(merged_dev and worker_state)
        n_workers = 0 if not worker_state else (self.K if merged_dev else 2 * self.K)
        self.slab = ArenaSlab(2 + n_workers + n_pre, self.n, torch.float32, self.device)
        arenas = self.slab.arenas
        self.slabs = [self.slab]
        self.w, self.mom = arenas[0], arenas[1]
        self.w.copy_(w0)
        self.mom.zero_()
        if not worker_state:
            # synchronous SGD only (delay_k == 0): the server state is all there is
            assert hp.delay_k == 0
            self.w_loc, self.pre, self.w_dev = [], [], []
            self.ctx = B.Context(self.numels, hp, self.w, self.mom)
            return
        # Algorithm 1 starts with every worker pulling w_0.
        self.w_loc = arenas[2:2 + self.K]
        self.w_dev = self.w_loc if merged_dev else arenas[2 + self.K:2 + 2 * self.K]
        for t in arenas[2 + self.K:]:
            t.fill_(fill)
        for t in self.w_loc:
            t.copy_(self.w)
        if host_pre:
            self.host_pre = torch.full((self.n,), fill, dtype=torch.float32).pin_memory()
            self.pre = [self.host_pre] * self.K
            self.ctx = B.Context(self.numels, hp, self.w, self.mom, self.w_loc, None, self.w_dev)
            if host_chunk:
                self.ctx.ssd_set_host_chunk(host_chunk)
            chunk = min(host_chunk or (1 << 24), self.n)
            slices = ArenaSlab(1, pre_slots * chunk, torch.float32, self.device)
            self.slabs.append(slices)
            self.pre_slices = slices.arenas[0]
            self.ctx.ssd_set_host_pre_weight(self.host_pre, self.pre_slices, pre_slots)
            return
        # shared_pre: one pre_weight buffer for all workers (K references to the same tensor)
        self.pre = arenas[2 + n_workers:] * (self.K if shared_pre else 1)
        self.ctx = B.Context(self.numels, hp, self.w, self.mom, self.w_loc, self.pre, self.w_dev)

    def worker_weights(self, i: int) -> torch.Tensor:
        """The arena worker i computes its next gradient on."""
        _, view = self.ctx.ssd_worker_weights(i)
        return (self.w, self.w_loc[i], self.w_dev[i])[view]

    def guards_intact(self) -> bool:
        """No store landed outside the arenas (see ArenaSlab)."""
        return all(s.guards_intact() for s in self.slabs)

    def bytes(self) -> int:
        """Device bytes of the state arenas (and of the slices of a host-resident pre_weight)."""
        device_pre = {t.data_ptr() for t in self.pre if t.is_cuda}
        total = (2 + len(self.w_loc) + len(device_pre) + (0 if self.merged_dev else len(self.w_dev))) * self.n * 4
        if len(self.slabs) > 1:
            total += self.pre_slices.numel() * 4
        return total
