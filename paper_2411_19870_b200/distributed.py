"""One worker per rank: the deployed form of Algorithm 1 (each accelerator compresses its own momentum,
the fixed-size payloads are exchanged by an all-gather, every rank then runs the same decode + update).

The exchange is the only collective of the method (Section 2.1, "AllGather"): ``chunks * k_eff * 8``
bytes per worker, independent of the model's dense size.  It is issued through ``torch.distributed``
(NCCL over NVLink / NVSwitch on GPUs; any backend that implements ``all_gather_into_tensor``): each
rank's compress kernel writes its records straight into that rank's slice of the gather buffer, the
collective fills the other slices in this GPU's own memory, and the decode kernel reads the W slices
as its W payloads -- no peer memory is touched by a kernel.  Everything else is the single-GPU library.
"""
from __future__ import annotations

from typing import List, Optional

import torch
import torch.distributed as dist

from .binding import DEMO_BF16, DemoTransform


def gather_payloads(slices: List[torch.Tensor], buffer: torch.Tensor, rank: int, group=None) -> None:
    """All-gather in place: ``buffer`` is the [W * payload_bytes] uint8 tensor whose w-th slice is
    ``slices[w]``; on entry slice ``rank`` holds this rank's payload, on return every slice holds the
    payload of the rank with that index (rank order = worker order of the decode's summation)."""
    world = dist.get_world_size(group)
    if len(slices) != world or buffer.numel() != world * slices[0].numel():
        raise ValueError("gather buffer does not match the group size")
    dist.all_gather_into_tensor(buffer, slices[rank], group=group)


class DistributedDemo:
    """DeMo step with one worker per rank of ``group``.  ``shapes`` etc. as for ``DemoTransform``."""

    def __init__(self, shapes, *, chunk: int, topk: int, beta: float, lr: float, weight_decay: float,
                 grad_dtype: int = DEMO_BF16, device: int = 0, group=None):
        self.group = group
        self.rank = dist.get_rank(group)
        self.world = dist.get_world_size(group)
        self.tr = DemoTransform(shapes, chunk=chunk, topk=topk, beta=beta, lr=lr, weight_decay=weight_decay,
                                num_workers=self.world, grad_dtype=grad_dtype, device=device)
        pb = self.tr.payload_bytes
        self.buffer = torch.zeros(self.world * pb, dtype=torch.uint8, device=torch.device("cuda", device))
        self.slices = [self.buffer[w * pb:(w + 1) * pb] for w in range(self.world)]

    def step(self, grads, momentum, params, stream: Optional[torch.cuda.Stream] = None) -> None:
        """grads / momentum: this rank's tensors; params: this rank's replica, updated in place.  All
        three stages are ordered on ``stream`` (default: the current stream)."""
        stream = stream or torch.cuda.current_stream()
        with torch.cuda.stream(stream):
            # worker slot 0 of the context: a rank has one worker, whatever its rank number
            self.tr.compress(0, grads, momentum, self.slices[self.rank], stream=stream)
            gather_payloads(self.slices, self.buffer, self.rank, self.group)
            self.tr.decode_apply(self.slices, params, stream=stream)

    def close(self) -> None:
        self.tr.close()
