"""One SplitLoRA round with the clients sharded over several devices (one process per device).

The clients are independent on the client side and the server loss is a mean over the
concatenated batch, so each rank owns a subset of the clients (and their rows of the cut-layer
activations), holds replicas of the frozen weights and of the server adapters, and runs the three
calls of the round on its own clients.  Two sums over ranks make the result equal to the
single-device round:

  1. the server adapter gradients (and the loss) after the server backward, before Eq. 4-5;
  2. the weighted client adapter sum of Eq. 8-9 at aggregation: one client's worth of parameters per
     rank, so ranks may hold different numbers of clients.

This module only orders the calls and the collectives (torch.distributed: NCCL on GPUs, gloo in
the CPU tests); all arithmetic happens inside the engine.  `engine` is a binding.SplitLoRA or any
object with the same methods.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

SIDE_CLIENT, SIDE_SERVER = 0, 1
KIND_PARAMS, KIND_GRADS = 0, 1


def shard_clients(n_clients_total: int, world_size: int, rank: int):
    """Contiguous block of client indices owned by `rank` (the last ranks get one fewer when the
    division is not exact)."""
    base, extra = divmod(n_clients_total, world_size)
    start = rank * base + min(rank, extra)
    return list(range(start, start + base + (1 if rank < extra else 0)))


class ShardedRound:
    """Runs Algorithm 1 for the local clients of this rank; call `round` on every rank."""

    def __init__(self, engine, group=None, agg_interval: int = 1):
        self.eng = engine
        self.group = group
        self.agg_interval = agg_interval
        self.round_index = 0
        engine.set_deferred_server_update(True)

    def _sum(self, t: torch.Tensor):
        if t.numel() > 0:       # no server adapters when every block is client-side
            dist.all_reduce(t, op=dist.ReduceOp.SUM, group=self.group)

    def round(self, tokens, labels, S, dS, local_counts, total_count: int, n_valid_global: int):
        """tokens, labels: this rank's [K_local, b, T]; S, dS: hand-off buffers [K_local, b, T, d];
        local_counts: |D_i| of the local clients; total_count: |D| over all ranks;
        n_valid_global: number of non-ignored labels over all ranks.  Returns the global loss tensor."""
        eng = self.eng
        eng.set_loss_normalizer(int(n_valid_global))
        eng.client_fwd(tokens, S)                                   # step a1
        eng.server_step(S, labels, dS, want_loss=False)             # step a3 without the update
        grads = eng.adapter_buffer(SIDE_SERVER, KIND_GRADS)
        loss = eng.loss_tensor()
        self._sum(grads)                                            # G_A, G_B over the whole batch
        self._sum(loss)                                             # local sums / global count add up
        eng.server_update()                                         # Eq. 4-5, identical on every rank
        eng.client_bwd(dS)                                          # step a5
        self.round_index += 1
        if self.round_index % self.agg_interval == 0:               # stage b
            part = eng.aggregate_local_sum(local_counts, int(total_count))   # [Pc], whatever K_local is
            self._sum(part)
            eng.aggregate_broadcast()                                        # downlink b3 to the local clients
        return loss
