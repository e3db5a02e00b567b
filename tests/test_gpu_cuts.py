"""Clients cut at different depths on the GPU (splitlora_set_client_cuts, configuration field cut_min)
against the oracle's round with per-client cuts: hand-off tensors and their gradients per client at that
client's depth, the one loss, every adapter gradient on both sides, the SGD updates, the aggregation per
block over its holders, and several rounds in a row."""
import numpy as np
import pytest
import torch

import harness as H
from oracle import splitlora_oracle as O
from paper_2407_00952_b200 import binding as B
from paper_2407_00952_b200 import runner, synth

pytestmark = pytest.mark.gpu


def _case(w, cuts):
    frozen = synth.make_frozen(w, randomize_affine=True)
    cads = [synth.make_adapters(w, range(cuts[i]), nonzero_b=True, salt=i + 1) for i in range(w.n_clients)]
    sads = synth.make_adapters(w, range(min(cuts), w.n_layer), nonzero_b=True, salt=77)
    tokens, labels = synth.make_tokens(w)
    labels = labels.copy()
    labels[0, 0, :5] = -1
    return frozen, cads, sads, tokens, labels


def _engine(w, cuts, frozen, cads, sads, optimizer):
    eng = runner.make_engine(w, frozen, cads, sads, optimizer=optimizer, cut_min=min(cuts))
    eng.set_client_cuts(cuts)
    return eng


def _check_three_calls(w, cuts, tol, tol_loss=1e-3, tol_qk=None):
    cuts = list(cuts)
    frozen, cads, sads, tokens, labels = _case(w, cuts)
    eng = _engine(w, cuts, frozen, cads, sads, "sgd")
    tok, lab = torch.from_numpy(tokens).cuda(), torch.from_numpy(labels).cuda()
    S, dS = eng.new_activation_buffer(), eng.new_activation_buffer()
    eng.client_fwd(tok, S)
    loss = eng.server_step(S, lab, dS)
    eng.client_bwd(dS)
    torch.cuda.synchronize()
    assert eng.device_status() == 0
    cfg, params = H.oracle_config(w, optimizer="sgd"), H.f64(frozen)
    c64, s64 = [H.ads64(a) for a in cads], H.ads64(sads)
    S_ref, caches = O.client_fwd_cuts(cfg, params, c64, tokens, cuts)
    loss_ref, dS_ref, sg = O.server_fwd_bwd_cuts(cfg, params, s64, S_ref, labels, cuts)
    cg = O.client_bwd_grads_cuts(cfg, params, c64, dS_ref, caches, cuts)
    assert abs(loss - loss_ref) <= tol_loss * abs(loss_ref)
    for i in range(w.n_clients):
        assert H.rel_err(H.tnp(S[i]), S_ref[i]) <= tol, ("S", i)
        assert H.rel_err(H.tnp(dS[i]), dS_ref[i]) <= tol, ("dS", i)
        assert set(cg[i]) == {(l, t) for l in range(cuts[i]) for t in w.targets}
        for (l, t), (dA, dB) in cg[i].items():
            gA, gB = eng.get_adapter_grad(B.SIDE_CLIENT, i, l, B.TARGET_BITS[t])
            tq = tol_qk if (tol_qk and t in ("q", "k")) else tol
            assert H.rel_err(H.tnp(gA), dA) <= tq and H.rel_err(H.tnp(gB), dB) <= tq, ("client grad", i, l, t)
            A, Bm = eng.get_adapter(B.SIDE_CLIENT, i, l, B.TARGET_BITS[t])
            assert H.rel_err(H.tnp(A), c64[i][(l, t)]["A"] - w.lr * dA) <= 1e-5
        with pytest.raises(B.SplitLoraError):          # a block the client does not hold
            if cuts[i] < w.cut:
                eng.get_adapter(B.SIDE_CLIENT, i, cuts[i], B.TARGET_Q)
            else:
                raise B.SplitLoraError(-1)
    assert set(sg) == {(l, t) for l in range(min(cuts), w.n_layer) for t in w.targets}
    for (l, t), (dA, dB) in sg.items():
        gA, gB = eng.get_adapter_grad(B.SIDE_SERVER, 0, l, B.TARGET_BITS[t])
        tq = tol_qk if (tol_qk and t in ("q", "k")) else tol
        assert H.rel_err(H.tnp(gA), dA) <= tq and H.rel_err(H.tnp(gB), dB) <= tq, ("server grad", l, t)
        A, Bm = eng.get_adapter(B.SIDE_SERVER, 0, l, B.TARGET_BITS[t])
        assert H.rel_err(H.tnp(Bm), s64[(l, t)]["B"] - w.lr * dB) <= 1e-5
    return eng


@pytest.mark.parametrize("cuts", [(1, 2, 3), (1, 1, 3), (2, 4), (1, 3, 3, 4), (2, 2)])
def test_tiny_fp32_three_calls_with_client_cuts(cuts):
    w = synth.scaled(synth.WORKLOADS[1], n_layer=4, cut=max(cuts), n_clients=len(cuts), counts=None, lr=0.5)
    _check_three_calls(w, cuts, 1e-4)


def test_bf16_medium_shaped_with_client_cuts():
    # the q / k adapter gradients take the bound derived in tests/test_storage_noise.py for this case
    w, _, qk_bound = H.qk_case("cuts_medium")
    _check_three_calls(w, H.CUTS_MEDIUM, 2e-2, tol_qk=qk_bound)


@pytest.mark.parametrize("interval", [1, 2])
def test_rounds_with_client_cuts(interval):
    """Three rounds of Algorithm 1 (SGD, fresh tokens) with cuts 1, 2, 2, 3: every adapter after every round,
    the aggregation over each block's holders included."""
    cuts = [1, 2, 2, 3]
    w = synth.scaled(synth.WORKLOADS[1], n_layer=4, cut=3, n_clients=4, counts=(3, 5, 2, 6), lr=1.0, agg_interval=interval)
    frozen, cads, sads, _, _ = _case(w, cuts)
    eng = _engine(w, cuts, frozen, cads, sads, "sgd")
    counts = synth.make_counts(w)
    cfg, params = H.oracle_config(w, optimizer="sgd"), H.f64(frozen)
    st = O.OracleState(client_adapters=[H.ads64(a) for a in cads], server_adapters=H.ads64(sads))
    for t in range(1, 4):
        tokens, labels = synth.make_tokens(w, round_index=t)
        loss = eng.round(torch.from_numpy(tokens).cuda(), torch.from_numpy(labels).cuda(), counts)
        loss_ref, info = O.split_round_cuts(cfg, params, st, tokens, labels, counts, cuts)
        assert info["aggregated"] == (t % interval == 0)
        assert abs(loss - loss_ref) <= 1e-3 * abs(loss_ref), (t, loss, loss_ref)
        for i in range(w.n_clients):
            for (l, tg), ad in st.client_adapters[i].items():
                A, Bm = eng.get_adapter(B.SIDE_CLIENT, i, l, B.TARGET_BITS[tg])
                assert H.rel_err(H.tnp(A), ad["A"]) <= 1e-4 and H.rel_err(H.tnp(Bm), ad["B"]) <= 1e-4, (t, i, l, tg)
        for (l, tg), ad in st.server_adapters.items():
            A, Bm = eng.get_adapter(B.SIDE_SERVER, 0, l, B.TARGET_BITS[tg])
            assert H.rel_err(H.tnp(A), ad["A"]) <= 1e-4 and H.rel_err(H.tnp(Bm), ad["B"]) <= 1e-4, (t, l, tg)
        if t % interval == 0:      # block 1 is held by clients 1, 2, 3: equal after the downlink; client 0 has none
            a1, a3 = (eng.get_adapter(B.SIDE_CLIENT, i, 1, B.TARGET_V)[1] for i in (1, 3))
            assert torch.equal(a1, a3)
    assert eng.device_status() == 0


def test_client_cut_argument_errors():
    w = synth.scaled(synth.WORKLOADS[1], n_layer=4, cut=3, n_clients=3, counts=None)
    frozen, cads, sads, _, _ = _case(w, [1, 2, 3])
    eng = runner.make_engine(w, frozen, cads, sads, optimizer="sgd", cut_min=1)
    for bad in ((2, 1, 3), (0, 1, 3), (1, 2, 4)):
        with pytest.raises(B.SplitLoraError) as e:
            eng.set_client_cuts(bad)
        assert e.value.code == -1
    eng.set_client_cuts((1, 2, 3))
    with pytest.raises(B.SplitLoraError) as e:      # spread over devices: not with per-client cuts
        eng.aggregate_local_sum([3, 5, 8], 16)
    assert e.value.code == -9
    eng.set_client_cuts(None)
    eng2 = runner.make_engine(w, frozen, [synth.make_adapters(w, range(3)) for _ in range(3)],
                              synth.make_adapters(w, range(3, 4)), optimizer="sgd")
    with pytest.raises(B.SplitLoraError):           # a configuration without cut_min takes one cut only
        eng2.set_client_cuts((1, 2, 3))
