"""Pins for the oracle's per-client-rank aggregation (clients whose adapters have different ranks).

The oracle works with adapters of their true shapes (A_i [r_i, in], B_i [out, r_i]); the CUDA
library stores every client at the configured rank with the missing components zero.  Pinned here:
the padded average in closed form, that equal ranks reduce to Eq. 8-9, and that a zero-padded client
is the same client (same activations, loss, gradients; the padded components get gradient exactly
zero and stay zero through SGD and AdamW), which is what makes the two representations equivalent.
"""
import copy

import numpy as np

from oracle import splitlora_oracle as O
from test_oracle_pins import ads64, ocfg, oracle_grads, setup, tiny_workload


def test_padded_average_closed_form():
    a0 = np.array([[1.0, 2.0, 3.0]])                       # client 0: rank 1
    a1 = np.array([[10.0, 20.0, 30.0], [4.0, 5.0, 6.0]])   # client 1: rank 2
    avg = O.aggregate_ranks([a0, a1], [3, 5], rank_axis=0)
    assert np.allclose(avg[0], 0.375 * a0[0] + 0.625 * a1[0], rtol=1e-15)
    assert np.allclose(avg[1], 0.625 * a1[1], rtol=1e-15)  # client 0 has no second component
    b0, b1 = a0.T.copy(), a1.T.copy()                      # B matrices: rank along axis 1
    assert np.allclose(O.aggregate_ranks([b0, b1], [3, 5], rank_axis=1), avg.T, rtol=1e-15)


def test_equal_ranks_reduce_to_eq_8_9():
    rng = np.random.default_rng(0)
    mats = [rng.normal(size=(4, 7)) for _ in range(3)]
    counts = [200, 1000, 431]
    assert np.array_equal(O.aggregate_ranks(mats, counts, 0), O.aggregate(mats, counts))
    assert np.array_equal(O.aggregate_ranks(mats, counts, 1), O.aggregate(mats, counts))


def _cut(ad, r):
    return {k: {"A": v["A"][:r].copy(), "B": v["B"][:, :r].copy()} for k, v in ad.items()}


def _pad(ad, r_max):
    out = {}
    for k, v in ad.items():
        r = v["A"].shape[0]
        out[k] = {"A": np.pad(v["A"], ((0, r_max - r), (0, 0))), "B": np.pad(v["B"], ((0, 0), (0, r_max - r)))}
    return out


def test_zero_padded_client_is_the_same_client():
    w = tiny_workload(lora_r=4, n_clients=3, counts=(3, 5, 2))
    cfg = ocfg(w)
    params, cads, sads, tokens, labels = setup(w)
    ranks = (1, 4, 2)
    cut = [_cut(cads[i], ranks[i]) for i in range(3)]
    padded = [_pad(c, 4) for c in cut]
    loss_c, S_c, dS_c, sg_c, cg_c = oracle_grads(cfg, params, cut, sads, tokens, labels)
    loss_p, S_p, dS_p, sg_p, cg_p = oracle_grads(cfg, params, padded, sads, tokens, labels)
    assert np.allclose(S_c, S_p, rtol=1e-13, atol=1e-13) and abs(loss_c - loss_p) < 1e-13
    assert np.allclose(dS_c, dS_p, rtol=1e-12, atol=1e-15)
    for i in range(3):
        r = ranks[i]
        for key in cg_c[i]:
            dA_c, dB_c = cg_c[i][key]
            dA_p, dB_p = cg_p[i][key]
            assert dA_c.shape == (r, w.d_model) and dB_c.shape == (w.d_model, r)
            assert np.allclose(dA_p[:r], dA_c, rtol=1e-11, atol=1e-14) and np.allclose(dB_p[:, :r], dB_c, rtol=1e-11, atol=1e-14)
            assert np.all(dA_p[r:] == 0.0) and np.all(dB_p[:, r:] == 0.0)      # exactly zero
    # a rank that is not full changes the function (the cut is not a no-op)
    loss_full, *_ = oracle_grads(cfg, params, cads, sads, tokens, labels)
    assert abs(loss_full - loss_c) > 1e-6


def test_round_with_ranks_padded_equals_true_shapes():
    """One round (update + aggregation) on true shapes equals the same round on zero-padded
    adapters with the padding cut off again after the average, for SGD and for AdamW."""
    for optimizer in ("sgd", "adamw"):
        w = tiny_workload(lora_r=4, n_clients=3, counts=(3, 5, 2))
        cfg = ocfg(w, optimizer=optimizer)
        params, cads, sads, tokens, labels = setup(w)
        ranks = (1, 4, 2)
        cut = [_cut(cads[i], ranks[i]) for i in range(3)]
        st_c = O.OracleState(client_adapters=copy.deepcopy(cut), server_adapters=copy.deepcopy(sads))
        st_p = O.OracleState(client_adapters=[_pad(c, 4) for c in cut], server_adapters=copy.deepcopy(sads))
        for st in (st_c, st_p):
            S, caches = O.client_fwd(cfg, params, st.client_adapters, tokens)
            _, dS, sg = O.server_fwd_bwd(cfg, params, st.server_adapters, S, labels)
            cg = O.client_bwd_grads(cfg, params, st.client_adapters, dS, caches)
            for i, g in enumerate(cg):
                O.apply_update(cfg, st.client_adapters[i], st.client_opt[i], g, cfg.lr_client, 1)
        # the padding is still exactly zero after the update (zero gradient, zero moments)
        for i in range(3):
            for ad in st_p.client_adapters[i].values():
                assert np.all(ad["A"][ranks[i]:] == 0.0) and np.all(ad["B"][:, ranks[i]:] == 0.0)
        O.aggregate_clients_ranks(st_c, w.counts)
        O.aggregate_clients(st_p, w.counts)            # plain Eq. 8-9 on the padded matrices ...
        for i in range(3):
            for key, ad in st_p.client_adapters[i].items():
                r = ranks[i]
                ref = st_c.client_adapters[i][key]
                assert ref["A"].shape[0] == r and ref["B"].shape[1] == r
                assert np.allclose(ad["A"][:r], ref["A"], rtol=1e-12, atol=1e-15)   # ... cut to the client's rank
                assert np.allclose(ad["B"][:, :r], ref["B"], rtol=1e-12, atol=1e-15)
        # the component only client 1 has is scaled by its weight alone
        key = next(iter(st_c.client_adapters[1]))
        assert st_c.client_adapters[1][key]["A"].shape[0] == 4
