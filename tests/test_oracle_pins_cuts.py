"""Pins of the oracle's round with clients cut at different depths (oracle/splitlora_oracle.py,
*_cuts functions; Sec. V names per-client cut layers as a direction, the reading is the oracle's).

* equal cuts: the functions are Algorithm 1 as the uniform-cut oracle states it, bit for bit;
* unequal cuts: an autograd model written per client with library routines (client i alone through its
  own blocks with its own adapters, then through the server's blocks with the shared server adapters, one
  cross-entropy over all clients' logits) gives the same loss, hand-off tensors, hand-off gradients and
  adapter gradients; no batching or bookkeeping is shared with the oracle;
* finite differences on a server adapter of a block that only some clients pass on the server side;
* aggregation: per block over its holders (closed forms), a block with one holder is left as it is.
"""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import splitlora_oracle as O
from paper_2407_00952_b200 import synth
from test_oracle_pins import ads64, f64, ocfg, tiny_workload, torch_block

torch.set_default_dtype(torch.float64)


def setup_cuts(cuts, n_layer=4, scale_w=5.0):
    K = len(cuts)
    w = tiny_workload(n_layer=n_layer, cut=max(cuts), n_clients=K, counts=tuple(range(3, 3 + K)))
    params = f64(synth.make_frozen(w, randomize_affine=True))
    for k in params:
        if k.endswith(".w") or k in ("wte", "wpe"):
            params[k] = params[k] * scale_w
    grow = lambda a: {k: {"A": v["A"] * scale_w, "B": v["B"] * scale_w} for k, v in a.items()}
    cads = [grow(ads64(synth.make_adapters(w, range(cuts[i]), nonzero_b=True, salt=i + 1))) for i in range(K)]
    sads = grow(ads64(synth.make_adapters(w, range(min(cuts), w.n_layer), nonzero_b=True, salt=77)))
    tokens, labels = synth.make_tokens(w)
    labels = labels.copy()
    labels[0, 0, :3] = -1
    return w, ocfg(w, optimizer="sgd"), params, cads, sads, tokens, labels


def test_equal_cuts_are_algorithm_1():
    w, cfg, params, cads, sads, tokens, labels = setup_cuts((2, 2, 2))
    cuts = [2, 2, 2]
    S_list, caches = O.client_fwd_cuts(cfg, params, cads, tokens, cuts)
    loss, dS_list, sg = O.server_fwd_bwd_cuts(cfg, params, sads, S_list, labels, cuts)
    cg = O.client_bwd_grads_cuts(cfg, params, cads, dS_list, caches, cuts)
    S, caches0 = O.client_fwd(cfg, params, cads, tokens)
    loss0, dS0, sg0 = O.server_fwd_bwd(cfg, params, sads, S, labels)
    cg0 = O.client_bwd_grads(cfg, params, cads, dS0, caches0)
    assert loss == loss0
    assert np.array_equal(np.stack(S_list), S) and np.array_equal(np.stack(dS_list), dS0)
    for k in sg0:
        assert np.array_equal(sg[k][0], sg0[k][0]) and np.array_equal(sg[k][1], sg0[k][1])
    for i in range(3):
        for k in cg0[i]:
            assert np.array_equal(cg[i][k][0], cg0[i][k][0]) and np.array_equal(cg[i][k][1], cg0[i][k][1])
    # and the whole round, aggregation included
    mk = lambda: O.OracleState(client_adapters=[{k: {n: m.copy() for n, m in a.items()} for k, a in ca.items()}
                                                for ca in cads],
                               server_adapters={k: {n: m.copy() for n, m in a.items()} for k, a in sads.items()})
    a, b = mk(), mk()
    counts = synth.make_counts(w)
    la, _ = O.split_round_cuts(cfg, params, a, tokens, labels, counts, cuts)
    lb, _ = O.split_round(cfg, params, b, tokens, labels, counts)
    assert la == lb
    for i in range(3):
        for k in a.client_adapters[i]:
            assert np.array_equal(a.client_adapters[i][k]["B"], b.client_adapters[i][k]["B"])


def autograd_cuts(cfg, params, cads, sads, tokens, labels, cuts):
    P = {k: torch.from_numpy(v) for k, v in params.items()}
    leaf = lambda a: (torch.from_numpy(a["A"].copy()).requires_grad_(), torch.from_numpy(a["B"].copy()).requires_grad_())
    tc = [{k: leaf(a) for k, a in ca.items()} for ca in cads]
    ts = {k: leaf(a) for k, a in sads.items()}
    tok = torch.from_numpy(tokens.astype(np.int64))
    T, d = tok.shape[-1], cfg.d_model
    S, logits = [], []
    for i in range(tokens.shape[0]):
        x = P["wte"][tok[i]] + P["wpe"][:T]
        for l in range(cuts[i]):
            x = torch_block(cfg, P, l, tc[i], x)
        x.retain_grad()
        S.append(x)
        for l in range(cuts[i], cfg.n_layer):
            x = torch_block(cfg, P, l, ts, x)
        x = F.layer_norm(x, (d,), P["lnf.g"], P["lnf.b"], cfg.norm_eps)
        logits.append(F.linear(x, P["wte"]).reshape(-1, cfg.vocab))
    lab = torch.from_numpy(labels.astype(np.int64)).reshape(-1)
    loss = F.cross_entropy(torch.cat(logits, 0), lab, ignore_index=-1)
    loss.backward()
    return loss.item(), S, tc, ts


@pytest.mark.parametrize("cuts", [(1, 2, 3), (1, 1, 3), (2, 4), (1, 3, 3, 4)])
def test_unequal_cuts_match_autograd(cuts):
    cuts = list(cuts)
    w, cfg, params, cads, sads, tokens, labels = setup_cuts(cuts)
    S_list, caches = O.client_fwd_cuts(cfg, params, cads, tokens, cuts)
    loss, dS_list, sg = O.server_fwd_bwd_cuts(cfg, params, sads, S_list, labels, cuts)
    cg = O.client_bwd_grads_cuts(cfg, params, cads, dS_list, caches, cuts)
    loss_t, S_t, tc, ts = autograd_cuts(cfg, params, cads, sads, tokens, labels, cuts)
    assert abs(loss - loss_t) <= 1e-12 * abs(loss_t)
    rel = lambda a, b: np.abs(a - b).max() / max(np.abs(b).max(), 1e-300)
    for i in range(len(cuts)):
        assert rel(S_list[i], S_t[i].detach().numpy()) <= 1e-12
        assert rel(dS_list[i], S_t[i].grad.numpy()) <= 1e-9
        assert set(cg[i].keys()) == set(tc[i].keys())
        for k, (dA, dB) in cg[i].items():
            assert rel(dA, tc[i][k][0].grad.numpy()) <= 1e-9 and rel(dB, tc[i][k][1].grad.numpy()) <= 1e-9
    assert set(sg.keys()) == set(ts.keys()) and min(k[0] for k in sg) == min(cuts)
    for k, (dA, dB) in sg.items():
        assert rel(dA, ts[k][0].grad.numpy()) <= 1e-9 and rel(dB, ts[k][1].grad.numpy()) <= 1e-9


def test_finite_difference_on_a_partly_shared_server_block():
    """Block 1 (0-based) is passed on the server side by client 0 only; its server adapter gradient must
    be the derivative of the one loss."""
    cuts = [1, 2, 3]
    w, cfg, params, cads, sads, tokens, labels = setup_cuts(cuts)

    def loss_of(sa):
        S_list, _ = O.client_fwd_cuts(cfg, params, cads, tokens, cuts)
        return O.server_fwd_bwd_cuts(cfg, params, sa, S_list, labels, cuts)[0]

    S_list, _ = O.client_fwd_cuts(cfg, params, cads, tokens, cuts)
    _, _, sg = O.server_fwd_bwd_cuts(cfg, params, sads, S_list, labels, cuts)
    rng = np.random.default_rng(0)
    for key in ((1, "q"), (2, "v")):
        for name, part in (("A", 0), ("B", 1)):
            for _ in range(3):
                idx = tuple(rng.integers(0, n) for n in sads[key][name].shape)
                h = 1e-5
                up = {k: {n: m.copy() for n, m in a.items()} for k, a in sads.items()}
                dn = {k: {n: m.copy() for n, m in a.items()} for k, a in sads.items()}
                up[key][name][idx] += h
                dn[key][name][idx] -= h
                fd = (loss_of(up) - loss_of(dn)) / (2 * h)
                assert abs(fd - sg[key][part][idx]) <= 1e-6 * max(1.0, abs(fd)), (key, name, idx)


def test_aggregation_over_the_holders_of_each_block():
    cuts = [1, 2, 3]
    w, cfg, params, cads, sads, tokens, labels = setup_cuts(cuts)
    st = O.OracleState(client_adapters=[{k: {n: m.copy() for n, m in a.items()} for k, a in ca.items()} for ca in cads],
                       server_adapters=sads)
    counts = [3, 5, 8]
    O.aggregate_clients_cuts(st, counts, cuts, store_fp32=False)
    # block 0: all three clients, weights 3/16, 5/16, 8/16 (exact in binary)
    ref0 = (3 * cads[0][(0, "q")]["A"] + 5 * cads[1][(0, "q")]["A"] + 8 * cads[2][(0, "q")]["A"]) / 16
    for i in range(3):
        assert np.allclose(st.client_adapters[i][(0, "q")]["A"], ref0, rtol=1e-15, atol=0)
    # block 1: clients 1 and 2 only, weights 5/13 and 8/13
    ref1 = (5 * cads[1][(1, "v")]["B"] + 8 * cads[2][(1, "v")]["B"]) / 13
    for i in (1, 2):
        assert np.allclose(st.client_adapters[i][(1, "v")]["B"], ref1, rtol=1e-14, atol=0)
    assert (1, "v") not in st.client_adapters[0]
    # block 2: one holder, unchanged
    assert np.array_equal(st.client_adapters[2][(2, "q")]["A"], cads[2][(2, "q")]["A"])
