"""Exchange of predictions between the model groups (Section 3 of the paper): every device computes one
forward pass and sends its B x C predictions to the devices that train the other models, every T steps;
on the steps in between the distillation term is left out (the loss is called without peers).

Plumbing only: ``torch.distributed`` moves the tensors (NCCL on GPUs: an all-gather that lands every
peer's predictions in local device memory before the loss kernel runs; no kernel of this package ever
reads another GPU's memory), the C library decides which steps exchange (``codistill_is_exchange_step``)
and packs fp32 predictions to bfloat16 when asked to halve the bits sent.  Coordinated sampling (all
groups see the same minibatch on an exchange step) is the caller's business, as in the paper.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import binding as cb


def gather_predictions(logits: torch.Tensor, group=None, compress: bool = False):
    """All-gather of the predictions among the n ranks of `group` (one rank per codistilled model).

    Returns the n-1 peers' predictions in rank order (own rank left out), each shaped like `logits`.
    With compress=True fp32 predictions travel as bfloat16 (half the bits; needs CUDA tensors) and are
    widened again on arrival, so that own logits and peers keep one element type."""
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    payload = logits.contiguous()
    if compress:
        if logits.dtype != torch.float32:
            raise TypeError("compression is for float32 predictions")
        payload = cb.pack_predictions(payload)
    slots = [torch.empty_like(payload) for _ in range(world)]
    dist.all_gather(slots, payload, group=group)
    peers = [slots[r] for r in range(world) if r != rank]
    if compress:
        peers = [cb.unpack_predictions(p) for p in peers]
    return peers


class PredictionExchange:
    """Step counter around gather_predictions: peers on the steps that exchange, none on the others."""

    def __init__(self, period: int = 1, group=None, compress: bool = False):
        if period < 1:
            raise ValueError("the exchange period is at least 1")
        self.period, self.group, self.compress, self.step = int(period), group, bool(compress), 0

    def peers_for_step(self, logits: torch.Tensor):
        """Call once per training step with the step's own predictions.  Returns the peers' predictions on an
        exchange step and an empty list otherwise (the loss then runs with n = 1: no distillation term)."""
        exchange = cb.is_exchange_step(self.step, self.period)
        self.step += 1
        return gather_predictions(logits, self.group, self.compress) if exchange else []

    def bits_sent_per_step(self, classes: int, batch_per_device: int, bits_per_value: int | None = None) -> float:
        """Section 3's cost of this schedule, bits per device and iteration (averaged over a period)."""
        n = dist.get_world_size(self.group)
        bits = bits_per_value if bits_per_value is not None else (16 if self.compress else 32)
        return cb.bits_predictions(n, classes, bits, batch_per_device, self.period)
