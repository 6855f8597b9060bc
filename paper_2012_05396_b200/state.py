"""Device-memory plumbing: allocates the arenas a context works on (torch tensors)."""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch

from . import binding as B


ARENA_ALIGN_BYTES = 4096


def alloc_arenas(count: int, n: int, dtype=torch.float32, device="cuda") -> List[torch.Tensor]:
    """`count` arenas of n elements carved out of one device allocation, each starting on a 4 KB
    boundary.  The kernels work with any 16-byte aligned buffers, but a block reads 4 KB of every
    stream per trip, and on B200 arenas that start off a 4 KB boundary cost about 3 % of bandwidth
    (measured on the VGG-16 and ResNet-50 workloads: 6.64 against 6.85 TB/s)."""
    if count == 0:
        return []
    esize = torch.empty(0, dtype=dtype).element_size()
    stride = -(-n * esize // ARENA_ALIGN_BYTES) * ARENA_ALIGN_BYTES // esize
    slab = torch.empty(count * stride, dtype=dtype, device=device)
    return [slab[i * stride: i * stride + n] for i in range(count)]


class DeviceState:
    """w, mom and the K workers' w_loc / pre / w_dev arenas on one CUDA device, plus the context.

    Untouched buffers are filled with `fill` (NaN by default) so that a read of something the
    schedule has not written yet shows up in any comparison.
    """

    def __init__(self, numels: Sequence[int], hp: B.ssd_hparams, w0: torch.Tensor,
                 device="cuda", fill: float = float("nan"), worker_state: bool = True,
                 shared_pre: bool = False):
        self.numels = [int(n) for n in numels]
        self.n = B.ssd_arena_numel(self.numels)
        assert w0.numel() == self.n and w0.dtype == torch.float32
        self.K = hp.K
        self.device = torch.device(device)
        n_pre = 0 if not worker_state else (1 if shared_pre else self.K)
        arenas = alloc_arenas(2 + (2 * self.K if worker_state else 0) + n_pre, self.n, torch.float32, self.device)
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
        self.w_dev = arenas[2 + self.K:2 + 2 * self.K]
        # shared_pre: one pre_weight buffer for all workers (K references to the same tensor)
        self.pre = arenas[2 + 2 * self.K:] * (self.K if shared_pre else 1)
        for t in self.w_loc:
            t.copy_(self.w)
        for t in self.w_dev + arenas[2 + 2 * self.K:]:
            t.fill_(fill)
        self.ctx = B.Context(self.numels, hp, self.w, self.mom, self.w_loc, self.pre, self.w_dev)

    def worker_weights(self, i: int) -> torch.Tensor:
        """The arena worker i computes its next gradient on."""
        _, view = self.ctx.ssd_worker_weights(i)
        return (self.w, self.w_loc[i], self.w_dev[i])[view]

    def bytes(self) -> int:
        return (2 + len(self.w_loc) + len({t.data_ptr() for t in self.pre}) + len(self.w_dev)) * self.n * 4
