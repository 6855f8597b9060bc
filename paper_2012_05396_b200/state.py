"""Device-memory plumbing: allocates the arenas a context works on (torch tensors)."""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch

from . import binding as B


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
        self.w = w0.to(self.device).clone()
        self.mom = torch.zeros(self.n, dtype=torch.float32, device=self.device)
        if not worker_state:
            # synchronous SGD only (delay_k == 0): the server state is all there is
            assert hp.delay_k == 0
            self.w_loc, self.pre, self.w_dev = [], [], []
            self.ctx = B.Context(self.numels, hp, self.w, self.mom)
            return
        # Algorithm 1 starts with every worker pulling w_0.
        self.w_loc = [self.w.clone() for _ in range(self.K)]
        # shared_pre: one pre_weight buffer for all workers (K references to the same tensor)
        self.pre = [torch.full((self.n,), fill, dtype=torch.float32, device=self.device)
                    for _ in range(1 if shared_pre else self.K)] * (self.K if shared_pre else 1)
        self.w_dev = [torch.full((self.n,), fill, dtype=torch.float32, device=self.device)
                      for _ in range(self.K)]
        self.ctx = B.Context(self.numels, hp, self.w, self.mom, self.w_loc, self.pre, self.w_dev)

    def worker_weights(self, i: int) -> torch.Tensor:
        """The arena worker i computes its next gradient on."""
        _, view = self.ctx.ssd_worker_weights(i)
        return (self.w, self.w_loc[i], self.w_dev[i])[view]

    def bytes(self) -> int:
        return (2 + len(self.w_loc) + len({t.data_ptr() for t in self.pre}) + len(self.w_dev)) * self.n * 4
