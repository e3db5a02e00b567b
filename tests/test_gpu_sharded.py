"""Sharding hooks of the C ABI on one GPU: two contexts play two ranks (each owns half of the
clients); the two sums over ranks are done by hand between the calls.  The result must equal the
single-context round on all clients."""
import numpy as np
import pytest
import torch

from paper_2407_00952_b200 import binding as B
from paper_2407_00952_b200 import parallel, runner, synth
import harness as H

pytestmark = pytest.mark.gpu


class FakeGroupRound(parallel.ShardedRound):
    """ShardedRound whose all-reduce adds the peer context's buffer (both contexts live in this process)."""
    peers = None

    def _sum(self, t):
        self.pending.append(t)


def test_two_contexts_equal_one():
    w = synth.scaled(synth.WORKLOADS[1], n_clients=4, counts=(300, 500, 200, 1000))
    frozen, cads, sads, tokens, labels = H.build_case(w)
    labels = labels.copy()
    labels[0, 1, :9] = -1
    counts = synth.make_counts(w)
    tok, lab = torch.from_numpy(tokens).cuda(), torch.from_numpy(labels).cuda()
    # reference: one context, all clients
    ref = runner.make_engine(w, frozen, cads, sads, optimizer="adamw")
    ref_losses = [ref.round(tok, lab, counts) for _ in range(2)]
    # two "ranks"
    ranks = []
    for r in range(2):
        mine = parallel.shard_clients(w.n_clients, 2, r)
        wl = synth.scaled(w, n_clients=len(mine), counts=tuple(int(counts[i]) for i in mine))
        eng = runner.make_engine(wl, frozen, [cads[i] for i in mine], sads, optimizer="adamw")
        eng.set_deferred_server_update(True)
        ranks.append(dict(eng=eng, mine=mine, tok=tok[mine].contiguous(), lab=lab[mine].contiguous(),
                          S=eng.new_activation_buffer(), dS=eng.new_activation_buffer()))
    n_valid = int((labels >= 0).sum())
    total = int(counts.sum())

    def allreduce(bufs):
        s = bufs[0] + bufs[1]
        for b in bufs:
            b.copy_(s)

    losses = []
    for _ in range(2):
        for rk in ranks:
            e = rk["eng"]
            e.set_loss_normalizer(n_valid)
            e.client_fwd(rk["tok"], rk["S"])
            e.server_step(rk["S"], rk["lab"], rk["dS"], want_loss=False)
        allreduce([rk["eng"].adapter_buffer(B.SIDE_SERVER, 1) for rk in ranks])
        allreduce([rk["eng"].loss_tensor() for rk in ranks])
        losses.append(float(ranks[0]["eng"].loss_tensor()[0]))
        for rk in ranks:
            rk["eng"].server_update()
            rk["eng"].client_bwd(rk["dS"])
            rk["eng"].aggregate_partial([int(counts[i]) for i in rk["mine"]], total)
        allreduce([rk["eng"].adapter_buffer(B.SIDE_CLIENT, 0) for rk in ranks])
        for rk in ranks:
            rk["eng"].adapters_changed(B.SIDE_CLIENT)
    torch.cuda.synchronize()
    for a, b in zip(losses, ref_losses):
        assert abs(a - b) <= 1e-5 * abs(b)
    for rk in ranks:
        for t in w.targets:
            bit = B.TARGET_BITS[t]
            for x, y in zip(rk["eng"].get_adapter(B.SIDE_SERVER, 0, 1, bit), ref.get_adapter(B.SIDE_SERVER, 0, 1, bit)):
                assert H.rel_err(H.tnp(x), H.tnp(y)) <= 1e-4
            for li, gi in enumerate(rk["mine"]):
                for x, y in zip(rk["eng"].get_adapter(B.SIDE_CLIENT, li, 0, bit), ref.get_adapter(B.SIDE_CLIENT, gi, 0, bit)):
                    assert H.rel_err(H.tnp(x), H.tnp(y)) <= 1e-4
