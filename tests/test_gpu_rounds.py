"""Several rounds of Algorithm 1 in a row on the GPU against the oracle: the loop over t = 1..R with fresh
mini-batches, aggregation every I rounds (I = 1 and I = 2), optimizer steps beyond the first (bias
corrections), and the refresh of the adapters' compute copies after update and aggregation, which is what
feeds the next round's forward.  Also the optimizer kernel alone, on identical inputs, at steps 1, 2 and 7.

Tolerances: fp32 1e-4 (normwise), loss 1e-3 relative, bf16 activations and gradients 2e-2.
"""
import numpy as np
import pytest
import torch

import harness as H
from oracle import splitlora_oracle as O
from paper_2407_00952_b200 import binding as B
from paper_2407_00952_b200 import runner, synth

pytestmark = pytest.mark.gpu

ROUNDS = 4


def _batches(w, rounds):
    return [synth.make_tokens(w, round_index=t) for t in range(rounds)]


def _oracle_state(cads, sads):
    return O.OracleState(client_adapters=[H.ads64(a) for a in cads], server_adapters=H.ads64(sads))


def _adapter_sets(w, eng, st):
    """(label, GPU pair, oracle pair) for every adapter of every client and of the server."""
    for i in range(w.n_clients):
        for (l, t), ad in st.client_adapters[i].items():
            yield ("client", i, l, t), eng.get_adapter(B.SIDE_CLIENT, i, l, B.TARGET_BITS[t]), (ad["A"], ad["B"])
    for (l, t), ad in st.server_adapters.items():
        yield ("server", 0, l, t), eng.get_adapter(B.SIDE_SERVER, 0, l, B.TARGET_BITS[t]), (ad["A"], ad["B"])


@pytest.mark.parametrize("interval", [1, 2])
def test_tiny_fp32_sgd_rounds(interval):
    """Eq. 4-7 as written (SGD): after every one of R rounds every element of every adapter, the loss of
    that round and the round counter equal the oracle's."""
    w = synth.scaled(synth.WORKLOADS[1], agg_interval=interval, n_clients=3, counts=(3, 5, 2), lr=1.0)
    frozen, cads, sads, _, _ = H.build_case(w)
    counts = synth.make_counts(w)
    eng = runner.make_engine(w, frozen, cads, sads, optimizer="sgd")
    start = H.tnp(eng.get_adapter(B.SIDE_SERVER, 0, 1, B.TARGET_V)[1])
    cfg, params, st = H.oracle_config(w, optimizer="sgd"), H.f64(frozen), _oracle_state(cads, sads)
    for t, (tokens, labels) in enumerate(_batches(w, ROUNDS), start=1):
        loss = eng.round(torch.from_numpy(tokens).cuda(), torch.from_numpy(labels).cuda(), counts)
        loss_ref, info = O.split_round(cfg, params, st, tokens, labels, counts)
        assert info["aggregated"] == (t % interval == 0)
        assert abs(loss - loss_ref) <= 1e-3 * abs(loss_ref), (t, loss, loss_ref)
        for key, got, ref in _adapter_sets(w, eng, st):
            for g, r in zip(got, ref):
                assert H.rel_err(H.tnp(g), r) <= 1e-4, (t, key)
        assert eng.get_counters() == (t, t, t)
        same = torch.equal(eng.get_adapter(B.SIDE_CLIENT, 0, 0, B.TARGET_Q)[1],
                           eng.get_adapter(B.SIDE_CLIENT, 2, 0, B.TARGET_Q)[1])
        assert same == (t % interval == 0)        # clients agree exactly after the downlink, and only then
    # the learning rate is large enough for the rounds to matter at the tolerance above
    assert H.rel_err(H.tnp(eng.get_adapter(B.SIDE_SERVER, 0, 1, B.TARGET_V)[1]), start) > 1e-2
    assert eng.device_status() == 0


@pytest.mark.parametrize("interval", [1, 2])
def test_tiny_fp32_adamw_rounds(interval):
    """AdamW over R rounds: the loss series, and the adapters where no gradient so far was tiny (the
    first step is -lr * sign(g), which rounding decides for g near zero)."""
    w = synth.scaled(synth.WORKLOADS[1], agg_interval=interval)
    frozen, cads, sads, _, _ = H.build_case(w)
    counts = synth.make_counts(w)
    eng = runner.make_engine(w, frozen, cads, sads, optimizer="adamw")
    cfg, params, st = H.oracle_config(w, optimizer="adamw"), H.f64(frozen), _oracle_state(cads, sads)
    big = {}      # per adapter matrix: every gradient seen so far (of every client, once averaged) was not tiny
    for t, (tokens, labels) in enumerate(_batches(w, ROUNDS), start=1):
        loss = eng.round(torch.from_numpy(tokens).cuda(), torch.from_numpy(labels).cuda(), counts)
        loss_ref, info = O.split_round(cfg, params, st, tokens, labels, counts)
        assert abs(loss - loss_ref) <= 1e-3 * abs(loss_ref), (t, loss, loss_ref)
        for (l, tg), g in info["server_grads"].items():
            for part in (0, 1):
                m = np.abs(g[part]) > 1e-3 * np.abs(g[part]).max()
                big[("server", 0, l, tg, part)] = big.get(("server", 0, l, tg, part), True) & m
        for (l, tg) in info["client_grads"][0]:
            for part in (0, 1):
                keys = [("client", i, l, tg, part) for i in range(w.n_clients)]
                for i, key in enumerate(keys):
                    g = info["client_grads"][i][(l, tg)][part]
                    big[key] = big.get(key, True) & (np.abs(g) > 1e-3 * np.abs(g).max())
                if info["aggregated"]:               # the average carries every client's ambiguous elements
                    allm = np.logical_and.reduce([big[key] for key in keys])
                    for key in keys:
                        big[key] = allm
        for (side, i, l, tg), got, ref in _adapter_sets(w, eng, st):
            for part in (0, 1):
                mask = big[(side, i, l, tg, part)]
                assert mask.mean() > 0.5
                err = np.abs(H.tnp(got[part]) - ref[part])[mask].max() / np.abs(ref[part]).max()
                assert err <= 1e-4, (t, side, i, l, tg, part, err)
    assert eng.get_counters() == (ROUNDS, ROUNDS, ROUNDS)
    assert eng.device_status() == 0


@pytest.mark.parametrize("interval", [1, 2])
def test_medium_shaped_bf16_rounds(interval):
    """GPT-2-medium-shaped (d 1024, 16 heads, vocabulary 50257) at reduced depth and batch, bf16, AdamW:
    the loss of each of R rounds, then the cut-layer activations and their gradients of one more pass
    computed from the adapters those rounds left behind."""
    w = synth.scaled(synth.WORKLOADS[3], n_layer=3, cut=1, n_clients=2, batch_per_client=1, seq=256, max_seq=256,
                     agg_interval=interval, lr=1e-3)
    frozen, cads, sads, _, _ = H.build_case(w)
    counts = synth.make_counts(w)
    eng = runner.make_engine(w, frozen, cads, sads, optimizer="adamw")
    cfg, params, st = H.oracle_config(w, optimizer="adamw"), H.f64(frozen), _oracle_state(cads, sads)
    batches = _batches(w, ROUNDS + 1)
    for t, (tokens, labels) in enumerate(batches[:ROUNDS], start=1):
        loss = eng.round(torch.from_numpy(tokens).cuda(), torch.from_numpy(labels).cuda(), counts)
        loss_ref, _ = O.split_round(cfg, params, st, tokens, labels, counts)
        assert abs(loss - loss_ref) <= 1e-3 * abs(loss_ref), (t, loss, loss_ref)
    tokens, labels = batches[ROUNDS]
    S, dS = eng.new_activation_buffer(), eng.new_activation_buffer()
    eng.client_fwd(torch.from_numpy(tokens).cuda(), S)
    loss = eng.server_step(S, torch.from_numpy(labels).cuda(), dS)
    S_ref, _ = O.client_fwd(cfg, params, st.client_adapters, tokens)
    loss_ref, dS_ref, _ = O.server_fwd_bwd(cfg, params, st.server_adapters, S_ref, labels)
    assert abs(loss - loss_ref) <= 1e-3 * abs(loss_ref)
    assert H.rel_err(H.tnp(S), S_ref) <= 2e-2
    assert H.rel_err(H.tnp(dS), dS_ref) <= 2e-2
    assert eng.device_status() == 0


@pytest.mark.parametrize("step", [1, 2, 7])
def test_adamw_kernel_on_identical_inputs(step):
    """The optimizer launch alone: moments and step counters are put into the context, one pass runs, and
    the parameters and moments it leaves must equal the AdamW definition applied, in fp64, to the very
    gradients the library holds (bias corrections 1 - beta^step at step 1, 2 and 7)."""
    w = synth.WORKLOADS[1]
    frozen, cads, sads, tokens, labels = H.build_case(w)
    eng = runner.make_engine(w, frozen, cads, sads, optimizer="adamw")
    rng = np.random.default_rng(100 + step)
    dev = lambda a: torch.from_numpy(a.astype(np.float32)).cuda()
    keys = [(B.SIDE_CLIENT, i, l, t) for i in range(w.n_clients) for l in range(w.cut) for t in w.targets] + \
           [(B.SIDE_SERVER, 0, l, t) for l in range(w.cut, w.n_layer) for t in w.targets]
    before = {}
    for key in keys:
        side, i, l, t = key
        bit = B.TARGET_BITS[t]
        shapes = ((w.lora_r, w.d_model), (w.d_model, w.lora_r))
        m = [rng.normal(size=s) * 1e-3 for s in shapes] if step > 1 else [np.zeros(s) for s in shapes]
        v = [rng.uniform(size=s) * 1e-6 for s in shapes] if step > 1 else [np.zeros(s) for s in shapes]
        eng.set_opt_state(side, i, l, bit, dev(m[0]), dev(v[0]), dev(m[1]), dev(v[1]))
        before[key] = dict(p=[H.tnp(x) for x in eng.get_adapter(side, i, l, bit)],
                           m=[H.tnp(x) for x in (dev(m[0]), dev(m[1]))], v=[H.tnp(x) for x in (dev(v[0]), dev(v[1]))])
    eng.set_counters(step - 1, step - 1, step - 1)
    S, dS = eng.new_activation_buffer(), eng.new_activation_buffer()
    eng.client_fwd(torch.from_numpy(tokens).cuda(), S)
    eng.server_step(S, torch.from_numpy(labels).cuda(), dS)
    eng.client_bwd(dS)
    assert eng.get_counters()[1:] == (step, step)
    for key in keys:
        side, i, l, t = key
        bit = B.TARGET_BITS[t]
        g = [H.tnp(x) for x in eng.get_adapter_grad(side, i, l, bit)]
        p = [H.tnp(x) for x in eng.get_adapter(side, i, l, bit)]
        mA, vA, mB, vB = (H.tnp(x) for x in eng.get_opt_state(side, i, l, bit))
        for part, (m_got, v_got) in enumerate(((mA, vA), (mB, vB))):
            b = before[key]
            # the hyper-parameters as the configuration struct holds them (fp32 fields)
            lr, b1, b2, eps, wd = (float(np.float32(x)) for x in (w.lr, 0.9, 0.999, 1e-8, 0.01))
            p_ref, m_ref, v_ref = O.adamw_update(b["p"][part], g[part], b["m"][part], b["v"][part], step, lr,
                                                 b1, b2, eps, wd)
            assert H.rel_err(m_got, m_ref) <= 1e-6, (key, part)
            assert H.rel_err(v_got, v_ref) <= 1e-6, (key, part)
            if step == 1:   # -lr * g / (|g| + eps): the quotient is decided by rounding where g is ~ eps
                sel = np.abs(g[part]) > 1e-5 * np.abs(g[part]).max()
            else:
                sel = np.ones_like(p_ref, dtype=bool)
            assert np.abs(p[part] - p_ref)[sel].max() <= 1e-6 * np.abs(p_ref).max(), (key, part)
