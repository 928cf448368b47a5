"""Algorithm 1's exchange step when every client is one GPU of a node.

The paper's clients upload their encoded update, a server sums the decoded updates,
divides by the number of participants and sends the result back (Algorithm 1, the
server's gather / decode / average / broadcast lines).  Between GPUs of one node there is
no need for a server: every rank receives all N messages with ONE all-gather of
fixed-capacity buffers (capacity = ``sbc_stream_bytes``; the true length is in each
container's header) and every rank decodes and applies the same N messages itself,

    W  <-  W + (1/N) * sum_c decode(message_c)                      (Algorithm 1)

so no broadcast follows.  A single decode launch over all N messages adds the scaled means
at a position in whatever order the hardware adds arrive, so two ranks may differ in the
last bit where several clients sent the same position; ``aggregate(ordered=True)`` decodes
one client per launch in rank order, which makes every rank add in the same order and keeps
the replicas bit-identical.

The gathered messages are in this GPU's own memory before any kernel reads them; the
collective is the process group's (NCCL over NVLink between GPUs, gloo between CPU
ranks), nothing here reads a peer's memory directly.  ``StreamExchange`` only moves
bytes and marshals arguments: encoding and decoding are the CUDA library's.
"""
from __future__ import annotations

from typing import List, Optional

import torch
import torch.distributed as dist


def _round_up(x: int, to: int) -> int:
    return (x + to - 1) // to * to


class StreamExchange:
    """Fixed-capacity all-gather of one message per rank, and the decode of all of them.

    ``capacity`` bytes per rank (rounded up to 16 so that every slot of the receive buffer
    keeps the container's alignment).  ``send`` is this rank's slot to encode into;
    ``gather()`` fills ``slots`` (one view per rank, rank order)."""

    def __init__(self, capacity: int, device: torch.device, group=None):
        if not dist.is_initialized():
            raise RuntimeError("StreamExchange needs an initialised torch.distributed process group")
        if capacity <= 0:
            raise ValueError("capacity must be positive")
        self.group = group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)
        self.capacity = _round_up(int(capacity), 16)
        self.send = torch.zeros(self.capacity, dtype=torch.uint8, device=device)
        self.recv = torch.zeros(self.world * self.capacity, dtype=torch.uint8, device=device)
        self.slots: List[torch.Tensor] = [
            self.recv[r * self.capacity:(r + 1) * self.capacity] for r in range(self.world)
        ]

    @classmethod
    def for_tensor(cls, numel: int, p: float, device: torch.device, group=None) -> "StreamExchange":
        """Capacity from the library's bound for a tensor of ``numel`` elements at sparsity ``p``."""
        from . import binding
        return cls(binding.sbc_stream_bytes(numel, p), device, group)

    def gather(self, async_op: bool = False):
        """All-gather ``send`` of every rank into ``slots``.  On CUDA tensors the collective is
        enqueued on the current stream's dependency chain by the backend; with ``async_op`` the
        work handle is returned and the caller waits on it before reading ``slots``."""
        return dist.all_gather_into_tensor(self.recv, self.send, group=self.group, async_op=async_op)

    def aggregate(self, weights: torch.Tensor, momentum: Optional[torch.Tensor] = None,
                  status: Optional[torch.Tensor] = None, scale: Optional[float] = None,
                  ordered: bool = False, stream=None) -> None:
        """weights += scale * sum_c decode(slot_c) (scale defaults to 1/N, Algorithm 1's average);
        ``momentum`` is zeroed at every transmitted position when given.  ``ordered`` decodes one
        client per launch in rank order, so that every rank adds in the same order."""
        from . import binding
        s = (1.0 / self.world) if scale is None else float(scale)
        # the messages come from other ranks: every header is checked against its slot's capacity
        if ordered:
            for slot in self.slots:
                binding.sbc_decode_apply([slot], s, weights, momentum, status, stream=stream, sizes=[self.capacity])
        else:
            binding.sbc_decode_apply(self.slots, s, weights, momentum, status, stream=stream,
                                     sizes=[self.capacity] * self.world)


def exchange_round(update: torch.Tensor, residual: torch.Tensor, p: float, weights: torch.Tensor,
                   ex: StreamExchange, momentum: Optional[torch.Tensor] = None,
                   status: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                   out_mu: Optional[torch.Tensor] = None, ordered: bool = False) -> None:
    """One communication round of Algorithm 1 on this rank: encode the local update (residual
    carried in place), all-gather the messages, apply the average of all decoded updates."""
    from . import binding
    binding.sbc_encode(update, residual, p, out_stream=ex.send, out_mu=out_mu, workspace=workspace)
    ex.gather()
    ex.aggregate(weights, momentum=momentum, status=status, ordered=ordered)
