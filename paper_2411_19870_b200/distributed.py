"""One worker per rank: the deployed form of Algorithm 1 (each accelerator compresses its own momentum,
the fixed-size payloads are exchanged by an all-gather, every rank then runs the same decode + update).

The exchange is the only collective of the method (Section 2.1, "AllGather"): ``chunks * k_eff * 8``
bytes per worker, independent of the model's dense size.  It is issued through ``torch.distributed``
(NCCL over NVLink / NVSwitch on GPUs; any backend that implements ``all_gather_into_tensor``): each
rank's compress kernel writes its records straight into that rank's slice of the gather buffer, the
collective fills the other slices in this GPU's own memory, and the decode kernel reads the W slices
as its W payloads -- no peer memory is touched by a kernel.  Everything else is the single-GPU library.

``step_server`` is the parameter-server form of Algorithm 1 instead: the payloads are gathered on one
rank only, that rank reconstructs the momentum and broadcasts its sign (one int8 per parameter), and every
rank applies the update itself.  Each rank then receives P bytes per step, whatever the number of
workers, instead of (W - 1) payloads (Section 5: the download volume of the all-gather grows with W).
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


def gather_to_server(slices: List[torch.Tensor], rank: int, server: int, group=None) -> None:
    """Send this rank's slice to ``server``; on the server every slice ends up holding the payload of the
    rank with that index.  The other ranks' buffers are left as they are."""
    dist.gather(slices[rank], gather_list=list(slices) if rank == server else None, dst=server, group=group)


def sign_views(shapes, device):
    """One flat int8 buffer with a view per tensor (each starting on a 16-byte boundary), so that the sign
    tensors of the whole model go out in a single broadcast.  Returns (flat, views)."""
    offsets, total = [], 0
    for s in shapes:
        offsets.append(total)
        n = 1
        for d in s:
            n *= int(d)
        total += (n + 15) // 16 * 16
    flat = torch.zeros(total, dtype=torch.int8, device=device)
    views = []
    for s, off in zip(shapes, offsets):
        n = 1
        for d in s:
            n *= int(d)
        views.append(flat[off:off + n].view(*s))
    return flat, views


def broadcast_signs(flat: torch.Tensor, server: int, group=None) -> None:
    dist.broadcast(flat, src=server, group=group)


class DistributedDemo:
    """DeMo step with one worker per rank of ``group``.  ``shapes`` etc. as for ``DemoTransform``
    (``chunk_shapes``: tensors of any order with rectangular chunks)."""

    def __init__(self, shapes, *, chunk: int = 0, topk: int, beta: float, lr: float, weight_decay: float,
                 grad_dtype: int = DEMO_BF16, device: int = 0, group=None, chunk_shapes=None):
        self.group = group
        self.rank = dist.get_rank(group)
        self.world = dist.get_world_size(group)
        self.tr = DemoTransform(shapes, chunk=chunk, topk=topk, beta=beta, lr=lr, weight_decay=weight_decay,
                                num_workers=self.world, grad_dtype=grad_dtype, device=device,
                                chunk_shapes=chunk_shapes)
        pb = self.tr.payload_bytes
        self.buffer = torch.zeros(self.world * pb, dtype=torch.uint8, device=torch.device("cuda", device))
        self.slices = [self.buffer[w * pb:(w + 1) * pb] for w in range(self.world)]
        self.shapes = [tuple(s) for s in shapes]
        self.sign_flat, self.signs = None, None  # allocated by the first step_server

    def step(self, grads, momentum, params, stream: Optional[torch.cuda.Stream] = None) -> None:
        """grads / momentum: this rank's tensors; params: this rank's replica, updated in place.  All
        three stages are ordered on ``stream`` (default: the current stream)."""
        stream = stream or torch.cuda.current_stream()
        with torch.cuda.stream(stream):
            # worker slot 0 of the context: a rank has one worker, whatever its rank number
            self.tr.compress(0, grads, momentum, self.slices[self.rank], stream=stream)
            gather_payloads(self.slices, self.buffer, self.rank, self.group)
            self.tr.decode_apply(self.slices, params, stream=stream)

    def step_server(self, grads, momentum, params, server: int = 0,
                    stream: Optional[torch.cuda.Stream] = None) -> None:
        """Parameter-server form: compress, gather the payloads on ``server``, decode to signs there,
        broadcast the signs, apply them on every rank."""
        stream = stream or torch.cuda.current_stream()
        with torch.cuda.stream(stream):
            if self.sign_flat is None:
                self.sign_flat, self.signs = sign_views(self.shapes, self.buffer.device)
            self.tr.compress(0, grads, momentum, self.slices[self.rank], stream=stream)
            gather_to_server(self.slices, self.rank, server, self.group)
            if self.rank == server:
                self.tr.decode_signs(self.slices, self.signs, stream=stream)
            broadcast_signs(self.sign_flat, server, self.group)
            self.tr.apply_signs(self.signs, params, stream=stream)

    def close(self) -> None:
        self.tr.close()
