"""Pins of the CPU checker (oracle/) against things other than itself: library routines and
autograd in fp64, finite differences, closed forms and the invariants the paper states.
None of these tests touches the CUDA library."""
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import splitlora_oracle as O
from paper_2407_00952_b200 import synth

torch.set_default_dtype(torch.float64)


def tiny_workload(**kw):
    base = dict(n_layer=3, cut=1, d_model=16, n_head=2, d_ff=32, vocab=40, max_seq=8, lora_r=2,
                lora_alpha=6.0, n_clients=2, batch_per_client=2, seq=8, dtype="fp32", counts=(3, 5))
    base.update(kw)
    return synth.scaled(synth.WORKLOADS[1], **base)


def ocfg(w, **kw):
    d = dict(n_layer=w.n_layer, cut=w.cut, d_model=w.d_model, n_head=w.n_head, d_ff=w.d_ff, vocab=w.vocab,
             max_seq=w.max_seq, lora_r=w.lora_r, lora_alpha=w.lora_alpha, targets=w.targets,
             n_clients=w.n_clients, batch_per_client=w.batch_per_client, seq=w.seq,
             bf16_handoff=(w.dtype == "bf16"), lr_client=w.lr, lr_server=w.lr, agg_interval=w.agg_interval)
    d.update(kw)
    return O.OracleConfig(**d)


def f64(d):
    return {k: v.astype(np.float64) for k, v in d.items()}


def ads64(a):
    return {k: {"A": v["A"].astype(np.float64), "B": v["B"].astype(np.float64)} for k, v in a.items()}


def setup(w, nonzero_b=True, distinct_clients=True, scale_w=5.0):
    """Frozen params (scaled up so that every term matters), adapters, tokens."""
    params = f64(synth.make_frozen(w, randomize_affine=True))
    for k in params:
        if k.endswith(".w") or k in ("wte", "wpe"):
            params[k] = params[k] * scale_w
    cads = [ads64(synth.make_adapters(w, range(w.cut), nonzero_b=nonzero_b,
                                      salt=(i + 1 if distinct_clients else 0)))
            for i in range(w.n_clients)]
    for ca in cads:
        for ad in ca.values():
            ad["A"] *= scale_w
            ad["B"] *= scale_w
    sads = ads64(synth.make_adapters(w, range(w.cut, w.n_layer), nonzero_b=nonzero_b, salt=77))
    for ad in sads.values():
        ad["A"] *= scale_w
        ad["B"] *= scale_w
    tokens, labels = synth.make_tokens(w)
    return params, cads, sads, tokens, labels


# ------------------------------------------------------------------ torch restatement
def torch_block(cfg, P, l, ads, x):
    """One block written with library routines only (F.linear, F.layer_norm, SDPA, F.gelu)."""
    d, H = cfg.d_model, cfg.n_head
    u = F.layer_norm(x, (d,), P[f"h.{l}.ln1.g"], P[f"h.{l}.ln1.b"], cfg.norm_eps)
    qkv = F.linear(u, P[f"h.{l}.attn.qkv.w"], P[f"h.{l}.attn.qkv.b"])
    q, k, v = qkv.split(d, dim=-1)
    s = cfg.scale
    parts = {"q": q, "k": k, "v": v}
    for t in cfg.targets:
        if t != "o":
            A, B = ads[(l, t)]
            parts[t] = parts[t] + s * F.linear(F.linear(u, A), B)
    nseq, T, _ = x.shape
    sh = lambda z: z.reshape(nseq, T, H, d // H).transpose(1, 2)
    o = F.scaled_dot_product_attention(sh(parts["q"]), sh(parts["k"]), sh(parts["v"]), is_causal=True)
    o = o.transpose(1, 2).reshape(nseq, T, d)
    Wo = P[f"h.{l}.attn.proj.w"]
    if "o" in cfg.targets:
        A, B = ads[(l, "o")]
        Wo = Wo + s * B @ A            # the update folded into the weight
    x = x + F.linear(o, Wo, P[f"h.{l}.attn.proj.b"])
    u2 = F.layer_norm(x, (d,), P[f"h.{l}.ln2.g"], P[f"h.{l}.ln2.b"], cfg.norm_eps)
    z = F.linear(u2, P[f"h.{l}.mlp.fc1.w"], P[f"h.{l}.mlp.fc1.b"])
    a = F.gelu(z, approximate="tanh" if cfg.gelu_tanh else "none")
    return x + F.linear(a, P[f"h.{l}.mlp.fc2.w"], P[f"h.{l}.mlp.fc2.b"])


def torch_split_model(cfg, params, cads, sads, tokens, labels):
    """Loss, S, dL/dS and all adapter gradients from autograd."""
    P = {k: torch.from_numpy(v) for k, v in params.items()}
    tc = [{k: (torch.from_numpy(a["A"].copy()).requires_grad_(), torch.from_numpy(a["B"].copy()).requires_grad_())
           for k, a in ca.items()} for ca in cads]
    ts = {k: (torch.from_numpy(a["A"].copy()).requires_grad_(), torch.from_numpy(a["B"].copy()).requires_grad_())
          for k, a in sads.items()}
    tok = torch.from_numpy(tokens.astype(np.int64))
    outs = []
    for i in range(tokens.shape[0]):
        T = tok.shape[-1]
        x = P["wte"][tok[i]] + P["wpe"][:T]
        for l in range(cfg.cut):
            x = torch_block(cfg, P, l, tc[i], x)
        outs.append(x)
    S = torch.stack(outs, 0)
    S.retain_grad()
    K, b, T, d = S.shape
    x = S.reshape(K * b, T, d)
    for l in range(cfg.cut, cfg.n_layer):
        x = torch_block(cfg, P, l, ts, x)
    x = F.layer_norm(x, (d,), P["lnf.g"], P["lnf.b"], cfg.norm_eps)
    z = F.linear(x, P["wte"])
    lab = torch.from_numpy(labels.astype(np.int64)).reshape(-1)
    loss = F.cross_entropy(z.reshape(-1, z.shape[-1]), lab, ignore_index=-1)
    loss.backward()
    return loss.item(), S.detach().numpy(), S.grad.numpy(), tc, ts


def oracle_grads(cfg, params, cads, sads, tokens, labels):
    S, caches = O.client_fwd(cfg, params, cads, tokens)
    loss, dS, sg = O.server_fwd_bwd(cfg, params, sads, S, labels)
    cg = O.client_bwd_grads(cfg, params, cads, dS, caches)
    return loss, S, dS, sg, cg


# ------------------------------------------------------------------ primitives vs library
def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(size=4000) * 10.0 ** rng.integers(-6, 6, size=4000),
                        np.array([0.0, 1.0, 1.00390625, 1.01171875, -3.0e-39])])
    ref = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(O.round_to_bf16(x), ref)


def test_layernorm_gelu_attention_ce_match_library():
    rng = np.random.default_rng(1)
    x = rng.normal(size=(6, 16)) * 3 + 1
    g, b = rng.normal(size=16), rng.normal(size=16)
    y, _ = O.layernorm_fwd(x, g, b, 1e-5)
    ref = F.layer_norm(torch.from_numpy(x), (16,), torch.from_numpy(g), torch.from_numpy(b), 1e-5).numpy()
    assert np.allclose(y, ref, rtol=1e-12, atol=1e-12)

    z = rng.normal(size=(5, 7)) * 3
    for tanh_form, mode in ((True, "tanh"), (False, "none")):
        ref = F.gelu(torch.from_numpy(z), approximate=mode).numpy()
        assert np.allclose(O.gelu_fwd(z, tanh_form), ref, rtol=1e-12, atol=1e-14)
        zt = torch.from_numpy(z).requires_grad_()
        F.gelu(zt, approximate=mode).sum().backward()
        assert np.allclose(O.gelu_grad(z, tanh_form), zt.grad.numpy(), rtol=1e-10, atol=1e-12)

    q, k, v = (rng.normal(size=(2, 9, 12)) for _ in range(3))
    o, _ = O.causal_attention_fwd(q, k, v, 3)
    sh = lambda a: torch.from_numpy(a).reshape(2, 9, 3, 4).transpose(1, 2)
    ref = F.scaled_dot_product_attention(sh(q), sh(k), sh(v), is_causal=True).transpose(1, 2).reshape(2, 9, 12)
    assert np.allclose(o, ref.numpy(), rtol=1e-12, atol=1e-12)

    zl = rng.normal(size=(10, 13)) * 2
    lab = rng.integers(0, 13, size=10)
    lab[3] = -1
    loss, dz = O.cross_entropy_fwd_bwd(zl, lab)
    zt = torch.from_numpy(zl).requires_grad_()
    lt = F.cross_entropy(zt, torch.from_numpy(lab), ignore_index=-1)
    lt.backward()
    assert abs(loss - lt.item()) < 1e-12
    assert np.allclose(dz, zt.grad.numpy(), rtol=1e-12, atol=1e-14)


def test_lora_b_zero_is_the_frozen_layer():
    rng = np.random.default_rng(2)
    x, W, bias = rng.normal(size=(7, 10)), rng.normal(size=(6, 10)), rng.normal(size=6)
    A, B = rng.normal(size=(3, 10)), np.zeros((6, 3))
    y, _ = O.lora_linear_fwd(x, W, bias, A, B, 4.0)
    assert np.array_equal(y, x @ W.T + bias)


def test_lora_linear_equals_merged_weight():
    """y must equal x (W + s B A)^T: the layer with the update folded into the weight."""
    rng = np.random.default_rng(3)
    x, W, bias = rng.normal(size=(7, 10)), rng.normal(size=(6, 10)), rng.normal(size=6)
    A, B = rng.normal(size=(3, 10)), rng.normal(size=(6, 3))
    y, _ = O.lora_linear_fwd(x, W, bias, A, B, 1.5)
    ref = F.linear(torch.from_numpy(x), torch.from_numpy(W + 1.5 * B @ A), torch.from_numpy(bias)).numpy()
    assert np.allclose(y, ref, rtol=1e-12, atol=1e-12)
    # gradients against autograd of the merged form
    dy = rng.normal(size=(7, 6))
    xt, At, Bt = (torch.from_numpy(a).requires_grad_() for a in (x, A, B))
    yt = F.linear(xt, torch.from_numpy(W) + 1.5 * Bt @ At, torch.from_numpy(bias))
    (yt * torch.from_numpy(dy)).sum().backward()
    dx, dA, dB = O.lora_linear_bwd(dy, x, W, A, B, 1.5)
    assert np.allclose(dx, xt.grad.numpy(), rtol=1e-11, atol=1e-12)
    assert np.allclose(dA, At.grad.numpy(), rtol=1e-11, atol=1e-12)
    assert np.allclose(dB, Bt.grad.numpy(), rtol=1e-11, atol=1e-12)


# ------------------------------------------------------------------ whole split model
@pytest.mark.parametrize("cut,targets", [(1, ("q", "v")), (2, ("q", "v")), (1, ("q", "k", "v", "o"))])
def test_split_model_matches_autograd(cut, targets):
    w = tiny_workload(cut=cut, targets=targets)
    cfg = ocfg(w)
    params, cads, sads, tokens, labels = setup(w)
    labels = labels.copy()
    labels[0, 0, 2] = -1                     # an ignored position
    loss, S, dS, sg, cg = oracle_grads(cfg, params, cads, sads, tokens, labels)
    tl, tS, tdS, tc, ts = torch_split_model(cfg, params, cads, sads, tokens, labels)
    assert abs(loss - tl) < 1e-11
    assert np.allclose(S, tS, rtol=1e-11, atol=1e-12)
    assert np.allclose(dS, tdS, rtol=1e-9, atol=1e-13)
    for key, (dA, dB) in sg.items():
        assert np.allclose(dA, ts[key][0].grad.numpy(), rtol=1e-9, atol=1e-13), key
        assert np.allclose(dB, ts[key][1].grad.numpy(), rtol=1e-9, atol=1e-13), key
    for i in range(w.n_clients):
        assert set(cg[i].keys()) == set(tc[i].keys())
        for key, (dA, dB) in cg[i].items():
            assert np.allclose(dA, tc[i][key][0].grad.numpy(), rtol=1e-9, atol=1e-13), (i, key)
            assert np.allclose(dB, tc[i][key][1].grad.numpy(), rtol=1e-9, atol=1e-13), (i, key)
    # the gradients are not trivially zero
    assert max(np.abs(g[0]).max() for g in sg.values()) > 1e-6
    assert max(np.abs(g[0]).max() for g in cg[0].values()) > 1e-6


def test_finite_difference_gradients():
    w = tiny_workload(n_layer=2, cut=1, n_clients=2, batch_per_client=1)
    cfg = ocfg(w)
    params, cads, sads, tokens, labels = setup(w)
    loss, S, dS, sg, cg = oracle_grads(cfg, params, cads, sads, tokens, labels)

    def total_loss():
        return oracle_grads(cfg, params, cads, sads, tokens, labels)[0]

    rng = np.random.default_rng(5)
    eps = 1e-5

    def check(mat, grad, n=6):
        for _ in range(n):
            idx = tuple(rng.integers(0, s) for s in mat.shape)
            old = mat[idx]
            mat[idx] = old + eps
            lp = total_loss()
            mat[idx] = old - eps
            lm = total_loss()
            mat[idx] = old
            fd = (lp - lm) / (2 * eps)
            assert abs(fd - grad[idx]) <= 1e-6 * max(1.0, abs(fd)) + 1e-8, (fd, grad[idx])

    for key, (dA, dB) in sg.items():
        check(sads[key]["A"], dA)
        check(sads[key]["B"], dB)
    for i in range(w.n_clients):
        for key, (dA, dB) in cg[i].items():
            check(cads[i][key]["A"], dA)
            check(cads[i][key]["B"], dB)
    # dL/dS: perturb the hand-off buffer itself
    for _ in range(6):
        idx = tuple(rng.integers(0, s) for s in S.shape)
        Sp, Sm = S.copy(), S.copy()
        Sp[idx] += eps
        Sm[idx] -= eps
        fd = (O.server_fwd_bwd(cfg, params, sads, Sp, labels)[0]
              - O.server_fwd_bwd(cfg, params, sads, Sm, labels)[0]) / (2 * eps)
        assert abs(fd - dS[idx]) <= 1e-6 * max(1.0, abs(fd)) + 1e-8


def test_every_cut_gives_the_unsplit_model():
    """Client forward then server forward is the same function of the tokens for every cut
    (Eq. 2 composed with Eq. 3), and so are the per-layer adapter gradients."""
    L = 4
    base = tiny_workload(n_layer=L, cut=1)
    params = f64(synth.make_frozen(base, randomize_affine=True))
    layer_ads = ads64(synth.make_adapters(base, range(L), nonzero_b=True, salt=3))
    tokens, labels = synth.make_tokens(base)
    ref = None
    for cut in range(1, L + 1):          # cut == L: every block on the clients, the server keeps the head
        w = tiny_workload(n_layer=L, cut=cut)
        cfg = ocfg(w)
        cads = [{k: v for k, v in layer_ads.items() if k[0] < cut} for _ in range(w.n_clients)]
        sads = {k: v for k, v in layer_ads.items() if k[0] >= cut}
        loss, S, dS, sg, cg = oracle_grads(cfg, params, cads, sads, tokens, labels)
        per_layer = dict(sg)
        for key in cads[0]:
            per_layer[key] = (sum(cg[i][key][0] for i in range(w.n_clients)),
                              sum(cg[i][key][1] for i in range(w.n_clients)))
        if ref is None:
            ref = (loss, per_layer)
        else:
            assert abs(loss - ref[0]) < 1e-12
            for key in per_layer:
                assert np.allclose(per_layer[key][0], ref[1][key][0], rtol=1e-9, atol=1e-14)
                assert np.allclose(per_layer[key][1], ref[1][key][1], rtol=1e-9, atol=1e-14)


def test_all_blocks_on_clients_is_local_training_per_client():
    """cut == L is the federated baseline of Sec. IV-A: client i's adapter gradients are those of
    training the whole model on client i's data alone, up to the ratio of the loss normalisers
    (the round's loss is one mean over the concatenated batch)."""
    L = 2
    w = tiny_workload(n_layer=L, cut=L)
    cfg = ocfg(w)
    params, cads, _, tokens, labels = setup(w)
    labels = labels.copy()
    labels[1, 0, :3] = -1
    loss, S, dS, sg, cg = oracle_grads(cfg, params, cads, {}, tokens, labels)
    assert sg == {}
    n_all = int((labels >= 0).sum())
    total = 0.0
    for i in range(w.n_clients):
        w1 = tiny_workload(n_layer=L, cut=1, n_clients=1)         # centralised: K = 1, any cut
        ads = cads[i]
        li, _, _, sgi, cgi = oracle_grads(ocfg(w1), params, [{k: v for k, v in ads.items() if k[0] < 1}],
                                          {k: v for k, v in ads.items() if k[0] >= 1}, tokens[i:i + 1], labels[i:i + 1])
        n_i = int((labels[i] >= 0).sum())
        total += li * n_i / n_all
        local = dict(sgi)
        local.update(cgi[0])
        for key, (dA, dB) in cg[i].items():
            assert np.allclose(dA * n_all / n_i, local[key][0], rtol=1e-9, atol=1e-14)
            assert np.allclose(dB * n_all / n_i, local[key][1], rtol=1e-9, atol=1e-14)
    assert abs(total - loss) < 1e-12


def test_initial_loss_is_ln_vocab():
    w = synth.scaled(synth.WORKLOADS[1], batch_per_client=1)
    cfg = ocfg(w)
    params = f64(synth.make_frozen(w))
    cads = [ads64(synth.make_adapters(w, range(w.cut))) for _ in range(w.n_clients)]
    sads = ads64(synth.make_adapters(w, range(w.cut, w.n_layer)))
    tokens, labels = synth.make_tokens(w)
    loss = oracle_grads(cfg, params, cads, sads, tokens, labels)[0]
    assert abs(loss - math.log(w.vocab)) < 0.05      # logits have std ~0.02*sqrt(d): tiny spread


def test_client_independence():
    w = tiny_workload()
    cfg = ocfg(w)
    params, cads, sads, tokens, labels = setup(w)
    _, S, dS, _, _ = oracle_grads(cfg, params, cads, sads, tokens, labels)
    tokens2 = tokens.copy()
    tokens2[1] = (tokens2[1] + 7) % w.vocab
    cads2 = [cads[0], ads64(synth.make_adapters(w, range(w.cut), nonzero_b=True, salt=9))]
    _, S2, dS2, _, _ = oracle_grads(cfg, params, cads2, sads, tokens2, labels)
    assert np.array_equal(S[0], S2[0]) and not np.allclose(S[1], S2[1])
    assert np.allclose(dS[0], dS2[0], rtol=1e-12, atol=1e-15)


# ------------------------------------------------------------------ optimizer
def test_sgd_is_the_literal_rule():
    p, g = np.array([1.0, -2.0]), np.array([0.5, 0.25])
    assert np.array_equal(O.sgd_update(p, g, 0.1), np.array([0.95, -2.025]))


def test_adamw_first_step_closed_form_and_library():
    rng = np.random.default_rng(7)
    p0, g = rng.normal(size=(4, 5)), rng.normal(size=(4, 5))
    lr, wd, eps = 1e-3, 0.01, 1e-8
    p1, m, v = O.adamw_update(p0, g, np.zeros_like(p0), np.zeros_like(p0), 1, lr, 0.9, 0.999, eps, wd)
    assert np.allclose(p1, p0 * (1 - lr * wd) - lr * g / (np.abs(g) + eps), rtol=1e-12, atol=1e-15)
    # zero gradient: pure decay (this is what every A sees in round 1, since B = 0 gives dA = 0)
    pz, _, _ = O.adamw_update(p0, np.zeros_like(p0), np.zeros_like(p0), np.zeros_like(p0), 1, lr, 0.9, 0.999, eps, wd)
    assert np.allclose(pz, p0 * (1 - lr * wd), rtol=0, atol=1e-16)
    # several steps against torch.optim.AdamW
    pt = torch.from_numpy(p0.copy()).requires_grad_()
    opt = torch.optim.AdamW([pt], lr=lr, betas=(0.9, 0.999), eps=eps, weight_decay=wd)
    p, m, v = p0.copy(), np.zeros_like(p0), np.zeros_like(p0)
    for step in range(1, 6):
        gs = rng.normal(size=p0.shape)
        pt.grad = torch.from_numpy(gs.copy())
        opt.step()
        p, m, v = O.adamw_update(p, gs, m, v, step, lr, 0.9, 0.999, eps, wd)
        assert np.allclose(p, pt.detach().numpy(), rtol=1e-12, atol=1e-15)


# ------------------------------------------------------------------ aggregation (Eq. 8-9)
def test_aggregation_pins():
    rng = np.random.default_rng(8)
    mats = [rng.normal(size=(3, 4)) for _ in range(4)]
    assert np.allclose(O.aggregate(mats, [5, 5, 5, 5]), np.mean(mats, axis=0), rtol=1e-15, atol=1e-16)
    assert np.array_equal(O.aggregate(mats[:1], [17]), mats[0])
    same = O.aggregate([mats[0]] * 3, [2, 9, 4])
    assert np.allclose(same, mats[0], rtol=1e-15, atol=1e-16)
    out = O.aggregate(mats, [200, 1000, 431, 777])
    assert np.all(out >= np.min(mats, axis=0) - 1e-15) and np.all(out <= np.max(mats, axis=0) + 1e-15)
    assert abs(O.aggregation_weights([200, 1000, 431, 777]).sum() - 1.0) < 1e-15
    assert np.array_equal(O.aggregate(mats[:2], [3, 5]), 0.375 * mats[0] + 0.625 * mats[1])
    # a bigger dataset pulls the average toward its client
    assert np.array_equal(O.aggregation_weights([1, 3]), np.array([0.25, 0.75]))


def test_round_aggregates_and_writes_back():
    w = tiny_workload(n_layer=2, cut=1)
    cfg = ocfg(w)
    params, cads, sads, tokens, labels = setup(w)
    st = O.OracleState(client_adapters=cads, server_adapters=sads)
    before = [{k: {n: a[n].copy() for n in a} for k, a in ca.items()} for ca in cads]
    loss, info = O.split_round(cfg, params, st, tokens, labels, [3, 5])
    assert info["aggregated"]
    for key in st.client_adapters[0]:
        for n in ("A", "B"):
            assert np.array_equal(st.client_adapters[0][key][n], st.client_adapters[1][key][n])
            assert not np.array_equal(st.client_adapters[0][key][n], before[0][key][n])
    # I = 2: no aggregation in round 1, aggregation in round 2
    params, cads, sads, tokens, labels = setup(w)
    cfg2 = ocfg(w, agg_interval=2)
    st = O.OracleState(client_adapters=cads, server_adapters=sads)
    _, info1 = O.split_round(cfg2, params, st, tokens, labels, [3, 5])
    assert not info1["aggregated"]
    key = next(iter(st.client_adapters[0]))
    assert not np.array_equal(st.client_adapters[0][key]["B"], st.client_adapters[1][key]["B"])
    _, info2 = O.split_round(cfg2, params, st, tokens, labels, [3, 5])
    assert info2["aggregated"]
    assert np.array_equal(st.client_adapters[0][key]["B"], st.client_adapters[1][key]["B"])


def test_single_client_round_is_a_centralised_lora_step():
    """K = 1, I = 1: the round is one ordinary LoRA step of the whole model on that batch
    (the paper's centralised baseline); checked against autograd + torch.optim.AdamW."""
    w = tiny_workload(n_layer=2, cut=1, n_clients=1, counts=(9,))
    cfg = ocfg(w, lr_client=1e-2, lr_server=1e-2)
    params, cads, sads, tokens, labels = setup(w)
    tl, _, _, tc, ts = torch_split_model(cfg, params, cads, sads, tokens, labels)
    leaves = [t for ad in list(tc[0].values()) + list(ts.values()) for t in ad]
    opt = torch.optim.AdamW(leaves, lr=1e-2, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.01)
    opt.step()
    st = O.OracleState(client_adapters=cads, server_adapters=sads)
    loss, _ = O.split_round(cfg, params, st, tokens, labels, [9])
    assert abs(loss - tl) < 1e-11
    for key, (A, B) in tc[0].items():
        got = st.client_adapters[0][key]
        # aggregation with one client stores the fp32-rounded value
        assert np.allclose(got["A"], A.detach().numpy(), rtol=2e-7, atol=1e-12)
        assert np.allclose(got["B"], B.detach().numpy(), rtol=2e-7, atol=1e-12)
    for key, (A, B) in ts.items():
        assert np.allclose(st.server_adapters[key]["A"], A.detach().numpy(), rtol=1e-9, atol=1e-14)
        assert np.allclose(st.server_adapters[key]["B"], B.detach().numpy(), rtol=1e-9, atol=1e-14)


def test_first_round_with_zero_b():
    """B = 0: dA = 0 exactly, so AdamW only decays A; |B_new| <= lr."""
    w = tiny_workload(n_layer=2, cut=1)
    cfg = ocfg(w, agg_interval=5)
    params, cads, sads, tokens, labels = setup(w, nonzero_b=False, distinct_clients=False)
    A0 = {k: a["A"].copy() for k, a in sads.items()}
    st = O.OracleState(client_adapters=cads, server_adapters=sads)
    _, info = O.split_round(cfg, params, st, tokens, labels, [3, 5])
    for key, (dA, dB) in info["server_grads"].items():
        assert np.all(dA == 0.0) and np.abs(dB).max() > 0
        assert np.allclose(st.server_adapters[key]["A"], A0[key] * (1 - cfg.lr_server * cfg.weight_decay),
                           rtol=1e-15, atol=0)
        assert np.abs(st.server_adapters[key]["B"]).max() <= cfg.lr_server * (1 + 1e-12)


# ------------------------------------------------------------------ Table III ratios
def test_table3_ratios():
    path = os.path.join(os.path.dirname(__file__), "golden", "table3_trainable_params.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    shapes = {"GPT2-S": (12, 768), "GPT2-M": (24, 1024)}
    for model, r, full, client in rows:
        L, d = shapes[model]
        r, full, client = int(r), float(full), float(client)
        cfg = O.OracleConfig(n_layer=L, cut=3, d_model=d, n_head=1, d_ff=4 * d, vocab=8, max_seq=8,
                             lora_r=r, lora_alpha=1.0)
        share = O.trainable_parameter_count(cfg, cfg.cut) / O.trainable_parameter_count(cfg, L)
        assert share == 3 / L
        # the table's own ratio agrees up to its 3-decimal rounding
        assert abs(client / full - share) <= (0.0005 / full + 0.0005 * client / full ** 2) * 1.5 + 1e-9
        # linear in r
        cfg1 = O.OracleConfig(n_layer=L, cut=3, d_model=d, n_head=1, d_ff=4 * d, vocab=8, max_seq=8,
                              lora_r=1, lora_alpha=1.0)
        assert O.trainable_parameter_count(cfg, L) == r * O.trainable_parameter_count(cfg1, L)
