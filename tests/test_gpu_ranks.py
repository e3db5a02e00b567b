"""Clients with different adapter ranks on the GPU (zero-padded storage, splitlora_set_client_ranks)
against the oracle, which works with adapters of their true shapes [r_i, d] / [d, r_i]."""
import numpy as np
import pytest
import torch

import harness as H
from oracle import splitlora_oracle as O
from paper_2407_00952_b200 import binding as B
from paper_2407_00952_b200 import runner, synth

pytestmark = pytest.mark.gpu


_cut = H.cut_to_rank


def _check_round(w, ranks, tol, optimizer, tol_qk=None):
    frozen, cads, sads, tokens, labels = H.build_case(w)
    counts = synth.make_counts(w)
    cfg = H.oracle_config(w, optimizer=optimizer)
    params = H.f64(frozen)
    st = O.OracleState(client_adapters=[_cut(H.ads64(cads[i]), ranks[i]) for i in range(w.n_clients)],
                       server_adapters=H.ads64(sads))
    S_ref, caches = O.client_fwd(cfg, params, st.client_adapters, tokens)
    loss_ref, dS_ref, sg = O.server_fwd_bwd(cfg, params, st.server_adapters, S_ref, labels)
    cg = O.client_bwd_grads(cfg, params, st.client_adapters, dS_ref, caches)
    for i, g in enumerate(cg):
        O.apply_update(cfg, st.client_adapters[i], st.client_opt[i], g, cfg.lr_client, 1)

    eng = runner.make_engine(w, frozen, cads, sads, optimizer=optimizer)
    eng.set_client_ranks(ranks)
    tok, lab = torch.from_numpy(tokens).cuda(), torch.from_numpy(labels).cuda()
    S, dS = eng.new_activation_buffer(), eng.new_activation_buffer()
    eng.client_fwd(tok, S)
    loss = eng.server_step(S, lab, dS)
    eng.client_bwd(dS)
    torch.cuda.synchronize()
    assert eng.device_status() == 0
    assert H.rel_err(H.tnp(S), S_ref) <= tol and H.rel_err(H.tnp(dS), dS_ref) <= tol
    assert abs(loss - loss_ref) <= 1e-3 * abs(loss_ref)
    tol_of = lambda t: (tol_qk if (tol_qk and t in ("q", "k")) else tol)
    for i in range(w.n_clients):
        r = ranks[i]
        for (l, t), (dA, dB) in cg[i].items():
            gA, gB = eng.get_adapter_grad(B.SIDE_CLIENT, i, l, B.TARGET_BITS[t])
            assert H.rel_err(H.tnp(gA)[:r], dA) <= tol_of(t) and H.rel_err(H.tnp(gB)[:, :r], dB) <= tol_of(t), (i, l, t)
            # components the client does not have: gradient exactly zero, parameters still exactly zero
            assert float(gA[r:].abs().max() if r < w.lora_r else 0.0) == 0.0
            assert float(gB[:, r:].abs().max() if r < w.lora_r else 0.0) == 0.0
            A, Bm = eng.get_adapter(B.SIDE_CLIENT, i, l, B.TARGET_BITS[t])
            if r < w.lora_r:
                assert float(A[r:].abs().max()) == 0.0 and float(Bm[:, r:].abs().max()) == 0.0
            if optimizer == "sgd":
                assert H.rel_err(H.tnp(A)[:r], st.client_adapters[i][(l, t)]["A"]) <= 1e-5
                assert H.rel_err(H.tnp(Bm)[:, :r], st.client_adapters[i][(l, t)]["B"]) <= 1e-5
    # aggregation: Eq. 8-9 on the padded matrices, every client keeps its own leading components.
    # Parity (SGD): the oracle's own round on true shapes, 1e-4.  Property (any optimizer): what the
    # library wrote back is the weighted mean, in fp64, of what it held before, cut to each rank, and
    # the rest is exactly zero.
    before = {(i, l, t): [H.tnp(x) for x in eng.get_adapter(B.SIDE_CLIENT, i, l, B.TARGET_BITS[t])]
              for i in range(w.n_clients) for (l, t) in cg[i]}
    eng.aggregate(counts)
    if optimizer == "sgd":
        O.aggregate_clients_ranks(st, counts)
    wts = O.aggregation_weights(counts)
    for (l, t) in cg[0]:
        for part, axis in ((0, 0), (1, 1)):
            mean = sum(wts[i] * before[(i, l, t)][part] for i in range(w.n_clients))    # padded, fp64
            for i in range(w.n_clients):
                r = ranks[i]
                got = H.tnp(eng.get_adapter(B.SIDE_CLIENT, i, l, B.TARGET_BITS[t])[part])
                lead = got[:r] if axis == 0 else got[:, :r]
                rest = got[r:] if axis == 0 else got[:, r:]
                want = mean[:r] if axis == 0 else mean[:, :r]
                assert H.rel_err(lead, want) <= 1e-6, (l, t, part, i)
                assert not rest.size or np.abs(rest).max() == 0.0
                if optimizer == "sgd":
                    ref = st.client_adapters[i][(l, t)]["A" if part == 0 else "B"]
                    assert H.rel_err(lead, ref) <= 1e-4, (l, t, part, i)
    return eng


def test_ranks_tiny_fp32_sgd():
    w = synth.scaled(synth.WORKLOADS[1], n_clients=3, counts=(3, 5, 2))
    _check_round(w, (1, 4, 2), 1e-4, "sgd")


def test_ranks_tiny_fp32_adamw_second_round_keeps_zeros():
    w = synth.scaled(synth.WORKLOADS[1], n_clients=3, counts=(3, 5, 2))
    eng = _check_round(w, (3, 1, 4), 1e-4, "adamw")
    _, _, _, tokens, labels = H.build_case(w)
    eng.round(torch.from_numpy(tokens).cuda(), torch.from_numpy(labels).cuda(), synth.make_counts(w))
    for i, r in enumerate((3, 1, 4)):
        for l in range(w.cut):
            for t in w.targets:
                A, Bm = eng.get_adapter(B.SIDE_CLIENT, i, l, B.TARGET_BITS[t])
                mA, vA, mB, vB = eng.get_opt_state(B.SIDE_CLIENT, i, l, B.TARGET_BITS[t])
                if r < w.lora_r:
                    for x in (A[r:], mA[r:], vA[r:], Bm[:, r:], mB[:, r:], vB[:, r:]):
                        assert float(x.abs().max()) == 0.0
                assert float(A[:r].abs().min()) > 0.0


def test_ranks_bf16_medium_shaped():
    w, ranks, qk_bound = H.qk_case("ranks_medium")      # storage noise leaves the general bound in reach here
    _check_round(w, ranks, 2e-2, "sgd", tol_qk=qk_bound)


def test_ranks_argument_errors_and_reset():
    w = synth.scaled(synth.WORKLOADS[1], n_clients=2)
    frozen, cads, sads, tokens, labels = H.build_case(w)
    eng = runner.make_engine(w, frozen, cads, sads, optimizer="sgd")
    for bad in ((0, 4), (4, 5)):
        with pytest.raises(B.SplitLoraError):
            eng.set_client_ranks(bad)
    eng.set_client_ranks(None)
    A, _ = eng.get_adapter(B.SIDE_CLIENT, 0, 0, B.TARGET_Q)
    assert float(A[-1].abs().max()) > 0.0          # untouched: still full rank
