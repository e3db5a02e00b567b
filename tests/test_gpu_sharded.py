"""Clients spread over ranks, on one GPU: every rank is a context of its own driven by
parallel.ShardedRound.round in a host thread of its own; the all-reduce between them is done by the threads
(each adds the peers' buffers at a barrier).  The result must equal the single-context round on all
clients: with an even split, with an uneven one (two clients and one), and with clients of different
adapter ranks (the cut back to each client's rank has to come after the sum over ranks)."""
import threading

import numpy as np
import pytest
import torch

from paper_2407_00952_b200 import binding as B
from paper_2407_00952_b200 import parallel, runner, synth
import harness as H

pytestmark = pytest.mark.gpu


class ThreadGroupRound(parallel.ShardedRound):
    """ShardedRound whose sum over ranks runs between host threads of this process."""

    def __init__(self, engine, rank, shared, barrier, **kw):
        super().__init__(engine, **kw)
        self.rank, self.shared, self.barrier = rank, shared, barrier

    def _sum(self, t):
        if t.numel() == 0:
            return
        torch.cuda.synchronize()
        self.shared[self.rank] = t
        self.barrier.wait()
        total = sum(x.clone() for x in self.shared)       # every rank reads all buffers before anyone writes
        torch.cuda.synchronize()
        self.barrier.wait()
        t.copy_(total)
        torch.cuda.synchronize()
        self.barrier.wait()


def _run_sharded(w, frozen, cads, sads, tokens, labels, counts, world, rounds, client_ranks=None):
    tok, lab = torch.from_numpy(tokens).cuda(), torch.from_numpy(labels).cuda()
    shared, barrier = [None] * world, threading.Barrier(world)
    n_valid, total = int((labels >= 0).sum()), int(counts.sum())
    out, errors = [None] * world, []

    def work(rank):
        try:
            torch.cuda.set_device(0)
            mine = parallel.shard_clients(w.n_clients, world, rank)
            wl = synth.scaled(w, n_clients=len(mine), counts=tuple(int(counts[i]) for i in mine))
            eng = runner.make_engine(wl, frozen, [cads[i] for i in mine], sads, optimizer="adamw")
            if client_ranks is not None:
                eng.set_client_ranks([client_ranks[i] for i in mine])
            rr = ThreadGroupRound(eng, rank, shared, barrier, agg_interval=w.agg_interval)
            S, dS = eng.new_activation_buffer(), eng.new_activation_buffer()
            losses = []
            for _ in range(rounds):
                loss = rr.round(tok[mine].contiguous(), lab[mine].contiguous(), S, dS,
                                [int(counts[i]) for i in mine], total, n_valid)
                losses.append(float(loss[0]))
            out[rank] = dict(eng=eng, mine=mine, losses=losses)
        except Exception as e:          # a failed rank must not leave the others at the barrier
            errors.append(e)
            barrier.abort()

    threads = [threading.Thread(target=work, args=(r,)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(300)
    assert not errors, errors
    return out


@pytest.mark.parametrize("n_clients,client_ranks", [(4, None), (3, None), (3, (2, 4, 1))])
def test_sharded_round_equals_one_context(n_clients, client_ranks):
    w = synth.scaled(synth.WORKLOADS[1], n_clients=n_clients, counts=(300, 500, 200, 1000)[:n_clients])
    frozen, cads, sads, tokens, labels = H.build_case(w)
    labels = labels.copy()
    labels[0, 1, :9] = -1
    counts = synth.make_counts(w)
    ref = runner.make_engine(w, frozen, cads, sads, optimizer="adamw")
    if client_ranks is not None:
        ref.set_client_ranks(client_ranks)
    tok, lab = torch.from_numpy(tokens).cuda(), torch.from_numpy(labels).cuda()
    ref_losses = [ref.round(tok, lab, counts) for _ in range(2)]
    out = _run_sharded(w, frozen, cads, sads, tokens, labels, counts, 2, 2, client_ranks)
    assert sorted(i for rk in out for i in rk["mine"]) == list(range(n_clients))
    for rk in out:
        for a, b in zip(rk["losses"], ref_losses):
            assert abs(a - b) <= 1e-5 * abs(b)
        for t in w.targets:
            bit = B.TARGET_BITS[t]
            for x, y in zip(rk["eng"].get_adapter(B.SIDE_SERVER, 0, 1, bit), ref.get_adapter(B.SIDE_SERVER, 0, 1, bit)):
                assert H.rel_err(H.tnp(x), H.tnp(y)) <= 1e-4
            for li, gi in enumerate(rk["mine"]):
                for x, y in zip(rk["eng"].get_adapter(B.SIDE_CLIENT, li, 0, bit), ref.get_adapter(B.SIDE_CLIENT, gi, 0, bit)):
                    assert H.rel_err(H.tnp(x), H.tnp(y)) <= 1e-4
                    if client_ranks is not None and client_ranks[gi] < w.lora_r:
                        r = client_ranks[gi]
                        rest = x[r:] if x.shape[0] == w.lora_r else x[:, r:]
                        assert float(rest.abs().max()) == 0.0
        assert rk["eng"].device_status() == 0
