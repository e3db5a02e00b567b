"""Clients sharded over two ranks (gloo, CPU): the orchestration in paper_2407_00952_b200.parallel
(order of the calls, the two sums over ranks, the global loss normaliser, the aggregation in two halves around one sum)
must reproduce the single-process round.  The engine on each rank is a stand-in with the same
methods as the CUDA binding, backed by the CPU oracle, so this runs without a GPU."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import splitlora_oracle as O
from paper_2407_00952_b200 import parallel, synth


def _workload(n_clients=4):
    counts = (300, 500, 200, 1000)[:n_clients]
    return synth.scaled(synth.WORKLOADS[1], n_layer=3, cut=1, d_model=32, n_head=2, d_ff=64, vocab=96, max_seq=16,
                        seq=16, batch_per_client=2, n_clients=n_clients, lora_r=2, lora_alpha=4.0, counts=counts,
                        agg_interval=1, lr=1e-2)


def _cfg(w, k):
    return O.OracleConfig(n_layer=w.n_layer, cut=w.cut, d_model=w.d_model, n_head=w.n_head, d_ff=w.d_ff, vocab=w.vocab,
                          max_seq=w.max_seq, lora_r=w.lora_r, lora_alpha=w.lora_alpha, targets=w.targets, n_clients=k,
                          batch_per_client=w.batch_per_client, seq=w.seq, optimizer="adamw", lr_client=w.lr,
                          lr_server=w.lr, agg_interval=w.agg_interval)


def _case(w):
    f64 = lambda d: {k: v.astype(np.float64) for k, v in d.items()}
    a64 = lambda a: {k: {"A": v["A"].astype(np.float64), "B": v["B"].astype(np.float64)} for k, v in a.items()}
    params = f64(synth.make_frozen(w, randomize_affine=True))
    cads = [a64(synth.make_adapters(w, range(w.cut), nonzero_b=True, salt=i + 1)) for i in range(w.n_clients)]
    sads = a64(synth.make_adapters(w, range(w.cut, w.n_layer), nonzero_b=True, salt=77))
    tokens, labels = synth.make_tokens(w)
    labels = labels.copy()
    labels[1, 0, :5] = -1           # unequal numbers of valid labels per rank
    return params, cads, sads, tokens, labels


class OracleEngine:
    """Same methods as binding.SplitLoRA (the subset parallel.ShardedRound uses), oracle arithmetic."""

    def __init__(self, cfg, params, client_adapters, server_adapters):
        self.cfg, self.params = cfg, params
        self.state = O.OracleState(client_adapters=client_adapters, server_adapters=server_adapters)
        self.skeys = sorted(server_adapters.keys())
        self.ckeys = sorted(client_adapters[0].keys())
        n_s = sum(server_adapters[k][n].size for k in self.skeys for n in ("A", "B"))
        n_c = sum(client_adapters[0][k][n].size for k in self.ckeys for n in ("A", "B"))
        self.sgrad = torch.zeros(n_s, dtype=torch.float64)
        self.csum = torch.zeros(n_c, dtype=torch.float64)     # one client's worth, whatever the local client count
        self.loss_t = torch.zeros(1, dtype=torch.float64)
        self.norm, self.deferred = 0, False

    def set_loss_normalizer(self, n): self.norm = n
    def set_deferred_server_update(self, on): self.deferred = on
    def loss_tensor(self): return self.loss_t

    def client_fwd(self, tokens, S):
        s, self.caches = O.client_fwd(self.cfg, self.params, self.state.client_adapters, tokens.numpy())
        S.copy_(torch.from_numpy(s))

    def server_step(self, S, labels, dS, want_loss=False):
        lab = labels.numpy()
        loss, ds, grads = O.server_fwd_bwd(self.cfg, self.params, self.state.server_adapters, S.numpy(), lab)
        scale = float((lab >= 0).sum()) / self.norm if self.norm else 1.0
        self.loss_t[0] = loss * scale
        dS.copy_(torch.from_numpy(ds * scale))
        flat = np.concatenate([grads[k][i].ravel() * scale for k in self.skeys for i in (0, 1)])
        self.sgrad.copy_(torch.from_numpy(flat))
        assert self.deferred

    def adapter_buffer(self, side, kind):
        assert side == parallel.SIDE_SERVER
        return self.sgrad

    def server_update(self):
        grads, off, flat = {}, 0, self.sgrad.numpy()
        for k in self.skeys:
            ad = self.state.server_adapters[k]
            dA = flat[off:off + ad["A"].size].reshape(ad["A"].shape); off += ad["A"].size
            dB = flat[off:off + ad["B"].size].reshape(ad["B"].shape); off += ad["B"].size
            grads[k] = (dA.copy(), dB.copy())
        self.state.server_steps += 1
        O.apply_update(self.cfg, self.state.server_adapters, self.state.server_opt, grads, self.cfg.lr_server,
                       self.state.server_steps)

    def client_bwd(self, dS):
        grads = O.client_bwd_grads(self.cfg, self.params, self.state.client_adapters, dS.numpy(), self.caches)
        self.state.client_steps += 1
        for i, g in enumerate(grads):
            O.apply_update(self.cfg, self.state.client_adapters[i], self.state.client_opt[i], g, self.cfg.lr_client,
                           self.state.client_steps)

    def aggregate_local_sum(self, counts, total):
        row = []
        for k in self.ckeys:
            for n in ("A", "B"):
                acc = sum((counts[i] / total) * ca[k][n] for i, ca in enumerate(self.state.client_adapters))
                row.append(acc.ravel())
        self.csum[:] = torch.from_numpy(np.concatenate(row))
        return self.csum

    def aggregate_broadcast(self):
        flat = self.csum.numpy()
        for ca in self.state.client_adapters:
            off = 0
            for k in self.ckeys:
                for n in ("A", "B"):
                    ca[k][n] = flat[off:off + ca[k][n].size].reshape(ca[k][n].shape).copy()
                    off += ca[k][n].size


def _worker(rank, world, port, out, n_clients):
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = _workload(n_clients)
    params, cads, sads, tokens, labels = _case(w)
    mine = parallel.shard_clients(w.n_clients, world, rank)
    counts = synth.make_counts(w)
    eng = OracleEngine(_cfg(w, len(mine)), params, [cads[i] for i in mine], sads)
    runner = parallel.ShardedRound(eng, agg_interval=w.agg_interval)
    tok, lab = torch.from_numpy(tokens[mine]), torch.from_numpy(labels[mine])
    S = torch.zeros(len(mine), w.batch_per_client, w.seq, w.d_model, dtype=torch.float64)
    dS = torch.zeros_like(S)
    n_valid = int((labels >= 0).sum())
    losses = []
    for _ in range(2):
        loss = runner.round(tok, lab, S, dS, [int(counts[i]) for i in mine], int(counts.sum()), n_valid)
        losses.append(float(loss[0]))
    out[rank] = dict(losses=losses, mine=mine, server=eng.state.server_adapters, clients=eng.state.client_adapters)
    dist.destroy_process_group()


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_shard_clients_partition():
    for K, W in ((8, 2), (8, 8), (7, 3), (4, 1)):
        parts = [parallel.shard_clients(K, W, r) for r in range(W)]
        assert sorted(i for p in parts for i in p) == list(range(K))
        assert max(len(p) for p in parts) - min(len(p) for p in parts) <= 1


@pytest.mark.timeout(300)
@pytest.mark.parametrize("n_clients", [4, 3])
def test_two_rank_round_equals_single_process(n_clients):
    """Four clients over two ranks, and three (rank 0 holds two clients, rank 1 one): the messages have the
    same size on both ranks either way, because the aggregation exchanges one client's worth of sums."""
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Manager().dict()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out, n_clients)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(240)
        assert p.exitcode == 0
    # single-process reference: all clients in one oracle state
    w = _workload(n_clients)
    params, cads, sads, tokens, labels = _case(w)
    st = O.OracleState(client_adapters=cads, server_adapters=sads)
    ref_losses = [O.split_round(_cfg(w, w.n_clients), params, st, tokens, labels, synth.make_counts(w))[0] for _ in range(2)]
    assert sorted(i for r in range(world) for i in out[r]["mine"]) == list(range(n_clients))
    for r in range(world):
        # round 1 agrees to rounding; round 2 sees client adapters that the single-process oracle
        # stored as fp32 after aggregation (6e-8 relative), hence the looser bounds below
        assert abs(out[r]["losses"][0] - ref_losses[0]) <= 1e-12 * abs(ref_losses[0])
        assert abs(out[r]["losses"][1] - ref_losses[1]) <= 1e-8 * abs(ref_losses[1])
        for k, ad in st.server_adapters.items():
            for n in ("A", "B"):
                assert np.allclose(out[r]["server"][k][n], ad[n], rtol=1e-7, atol=1e-9)
        for li, gi in enumerate(out[r]["mine"]):
            for k, ad in st.client_adapters[gi].items():
                for n in ("A", "B"):
                    # the single-process oracle stores the average as fp32
                    assert np.allclose(out[r]["clients"][li][k][n], ad[n], rtol=1e-6, atol=1e-9)
    # every client on every rank holds the same aggregated adapters
    a0 = out[0]["clients"][0][(0, "q")]["A"]
    assert np.array_equal(a0, out[1]["clients"][-1][(0, "q")]["A"])
