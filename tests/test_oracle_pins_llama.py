"""Pins for the Llama-shaped block of the CPU oracle (RMSNorm, rotary q/k, SwiGLU, adapters on
q, k, v and o, separate head).  The paper only cites Llama-2; these pins tie the oracle's definition
to library routines, an independent complex-number statement of the rotation, closed forms and
finite differences.  CPU only."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import splitlora_oracle as O
from paper_2407_00952_b200 import synth

torch.set_default_dtype(torch.float64)


def tiny_llama(**kw):
    base = dict(n_layer=3, cut=1, d_model=16, n_head=2, d_ff=24, vocab=40, max_seq=8, lora_r=2,
                lora_alpha=6.0, n_clients=2, batch_per_client=2, seq=8, dtype="fp32", counts=(3, 5),
                targets=("q", "k", "v", "o"), arch="llama", zipf=False, index=1, name="tiny-llama")
    base.update(kw)
    return synth.scaled(synth.WORKLOADS[5], **base)


def ocfg(w, **kw):
    d = dict(n_layer=w.n_layer, cut=w.cut, d_model=w.d_model, n_head=w.n_head, d_ff=w.d_ff, vocab=w.vocab,
             max_seq=w.max_seq, lora_r=w.lora_r, lora_alpha=w.lora_alpha, targets=w.targets,
             n_clients=w.n_clients, batch_per_client=w.batch_per_client, seq=w.seq,
             lr_client=w.lr, lr_server=w.lr, agg_interval=w.agg_interval, arch=w.arch, rope_theta=w.rope_theta)
    d.update(kw)
    return O.OracleConfig(**d)


def f64(d):
    return {k: v.astype(np.float64) for k, v in d.items()}


def ads64(a, scale=1.0):
    return {k: {"A": v["A"].astype(np.float64) * scale, "B": v["B"].astype(np.float64) * scale} for k, v in a.items()}


def setup(w, scale_w=5.0):
    params = f64(synth.make_frozen(w, randomize_affine=True))
    for k in params:
        if k.endswith(".w") or k == "wte":
            params[k] = params[k] * scale_w
    cads = [ads64(synth.make_adapters(w, range(w.cut), nonzero_b=True, salt=i + 1), scale_w) for i in range(w.n_clients)]
    sads = ads64(synth.make_adapters(w, range(w.cut, w.n_layer), nonzero_b=True, salt=77), scale_w)
    tokens, labels = synth.make_tokens(w)
    return params, cads, sads, tokens, labels


def oracle_grads(cfg, params, cads, sads, tokens, labels):
    S, caches = O.client_fwd(cfg, params, cads, tokens)
    loss, dS, sg = O.server_fwd_bwd(cfg, params, sads, S, labels)
    cg = O.client_bwd_grads(cfg, params, cads, dS, caches)
    return loss, S, dS, sg, cg


# ------------------------------------------------------------------ primitives
def test_rmsnorm_matches_library_and_autograd():
    rng = np.random.default_rng(11)
    x = rng.normal(size=(6, 16)) * 3 + 1
    g = rng.normal(size=16)
    y, cache = O.rmsnorm_fwd(x, g, 1e-5)
    xt = torch.from_numpy(x).requires_grad_()
    ref = F.rms_norm(xt, (16,), torch.from_numpy(g), 1e-5)
    assert np.allclose(y, ref.detach().numpy(), rtol=1e-12, atol=1e-12)
    dy = rng.normal(size=(6, 16))
    (ref * torch.from_numpy(dy)).sum().backward()
    assert np.allclose(O.rmsnorm_bwd(dy, cache), xt.grad.numpy(), rtol=1e-11, atol=1e-13)
    # scaling a row leaves the output unchanged when eps is negligible
    y2, _ = O.rmsnorm_fwd(x * 7.0, g, 1e-30)
    y1, _ = O.rmsnorm_fwd(x, g, 1e-30)
    assert np.allclose(y1, y2, rtol=1e-12)


def test_silu_matches_library():
    z = np.random.default_rng(12).normal(size=(5, 7)) * 3
    zt = torch.from_numpy(z).requires_grad_()
    yt = F.silu(zt)
    assert np.allclose(O.silu(z), yt.detach().numpy(), rtol=1e-13, atol=1e-15)
    yt.sum().backward()
    assert np.allclose(O.silu_grad(z), zt.grad.numpy(), rtol=1e-12, atol=1e-14)


def complex_rope(x, n_head, theta):
    """The rotation stated with complex numbers: (lo + i hi) * exp(i t theta^(-2j/dh))."""
    nseq, T, d = x.shape
    dh = d // n_head
    half = dh // 2
    xh = x.reshape(nseq, T, n_head, dh)
    z = xh[..., :half] + 1j * xh[..., half:]
    out = np.empty_like(xh)
    for t in range(T):
        for j in range(half):
            w = np.exp(1j * t * theta ** (-2.0 * j / dh))
            zz = z[:, t, :, j] * w
            out[:, t, :, j] = zz.real
            out[:, t, :, j + half] = zz.imag
    return out.reshape(nseq, T, d)


def test_rope_properties():
    rng = np.random.default_rng(13)
    H, dh, T = 3, 8, 10
    x = rng.normal(size=(2, T, H * dh))
    y = O.rope_rotate(x, H, 10000.0)
    assert np.allclose(y, complex_rope(x, H, 10000.0), rtol=1e-12, atol=1e-13)
    assert np.array_equal(y[:, 0], x[:, 0])                                  # position 0: no rotation
    assert np.allclose((y.reshape(2, T, H, dh) ** 2).sum(-1), (x.reshape(2, T, H, dh) ** 2).sum(-1), rtol=1e-12)
    assert np.allclose(O.rope_rotate(y, H, 10000.0, sign=-1.0), x, rtol=1e-12, atol=1e-13)
    # closed form with one pair per head: j = 0 has frequency 1, so (1, 0) at position t -> (cos t, sin t)
    e = np.zeros((1, T, 2))
    e[..., 0] = 1.0
    r = O.rope_rotate(e, 1, 123.0)
    assert np.allclose(r[0, :, 0], np.cos(np.arange(T))) and np.allclose(r[0, :, 1], np.sin(np.arange(T)))
    # scores depend on the distance between positions only
    qv, kv = rng.normal(size=dh), rng.normal(size=dh)
    q = O.rope_rotate(np.tile(qv, (1, T, 1)), 1, 10000.0)[0]
    k = O.rope_rotate(np.tile(kv, (1, T, 1)), 1, 10000.0)[0]
    sc = q @ k.T
    for m in range(1, T):
        assert np.allclose(np.diag(sc, -m), sc[m, 0], rtol=1e-11, atol=1e-12)
    # gradient map = inverse rotation: <rope(x), g> = <x, rope^-1(g)>
    g = rng.normal(size=x.shape)
    assert abs((y * g).sum() - (x * O.rope_rotate(g, H, 10000.0, sign=-1.0)).sum()) < 1e-10


# ------------------------------------------------------------------ whole model vs autograd
def torch_rope(z, H, theta):
    nseq, T, d = z.shape
    dh = d // H
    half = dh // 2
    zh = z.reshape(nseq, T, H, dh)
    c = torch.complex(zh[..., :half], zh[..., half:])
    ang = torch.arange(T, dtype=torch.float64)[:, None] * theta ** (-2.0 * torch.arange(half, dtype=torch.float64) / dh)
    c = c * torch.polar(torch.ones_like(ang), ang)[None, :, None, :]
    return torch.cat([c.real, c.imag], dim=-1).reshape(nseq, T, d)


def torch_block(cfg, P, l, ads, x):
    d, H = cfg.d_model, cfg.n_head
    s = cfg.scale
    u = F.rms_norm(x, (d,), P[f"h.{l}.ln1.g"], cfg.norm_eps)
    q, k, v = F.linear(u, P[f"h.{l}.attn.qkv.w"]).split(d, dim=-1)
    parts = {"q": q, "k": k, "v": v}
    for t in cfg.targets:
        if t != "o":
            A, B = ads[(l, t)]
            parts[t] = parts[t] + s * F.linear(F.linear(u, A), B)
    nseq, T, _ = x.shape
    sh = lambda z: z.reshape(nseq, T, H, d // H).transpose(1, 2)
    o = F.scaled_dot_product_attention(sh(torch_rope(parts["q"], H, cfg.rope_theta)),
                                       sh(torch_rope(parts["k"], H, cfg.rope_theta)), sh(parts["v"]), is_causal=True)
    o = o.transpose(1, 2).reshape(nseq, T, d)
    Wo = P[f"h.{l}.attn.proj.w"]
    if "o" in cfg.targets:
        A, B = ads[(l, "o")]
        Wo = Wo + s * B @ A                    # the update folded into the weight
    x = x + F.linear(o, Wo)
    u2 = F.rms_norm(x, (d,), P[f"h.{l}.ln2.g"], cfg.norm_eps)
    a = F.silu(F.linear(u2, P[f"h.{l}.mlp.gate.w"])) * F.linear(u2, P[f"h.{l}.mlp.up.w"])
    return x + F.linear(a, P[f"h.{l}.mlp.down.w"])


def torch_split_model(cfg, params, cads, sads, tokens, labels):
    P = {k: torch.from_numpy(v) for k, v in params.items()}
    leaf = lambda a: torch.from_numpy(a.copy()).requires_grad_()
    tc = [{k: (leaf(a["A"]), leaf(a["B"])) for k, a in ca.items()} for ca in cads]
    ts = {k: (leaf(a["A"]), leaf(a["B"])) for k, a in sads.items()}
    tok = torch.from_numpy(tokens.astype(np.int64))
    outs = []
    for i in range(tokens.shape[0]):
        x = P["wte"][tok[i]]
        for l in range(cfg.cut):
            x = torch_block(cfg, P, l, tc[i], x)
        outs.append(x)
    S = torch.stack(outs, 0)
    S.retain_grad()
    K, b, T, d = S.shape
    x = S.reshape(K * b, T, d)
    for l in range(cfg.cut, cfg.n_layer):
        x = torch_block(cfg, P, l, ts, x)
    x = F.rms_norm(x, (d,), P["lnf.g"], cfg.norm_eps)
    z = F.linear(x, P["head.w"])
    loss = F.cross_entropy(z.reshape(-1, z.shape[-1]), torch.from_numpy(labels.astype(np.int64)).reshape(-1),
                           ignore_index=-1)
    loss.backward()
    return loss.item(), S.detach().numpy(), S.grad.numpy(), tc, ts


@pytest.mark.parametrize("cut,targets", [(1, ("q", "k", "v", "o")), (2, ("q", "k", "v", "o")), (1, ("q", "v"))])
def test_llama_split_model_matches_autograd(cut, targets):
    w = tiny_llama(cut=cut, targets=targets)
    cfg = ocfg(w)
    params, cads, sads, tokens, labels = setup(w)
    labels = labels.copy()
    labels[1, 0, 3] = -1
    loss, S, dS, sg, cg = oracle_grads(cfg, params, cads, sads, tokens, labels)
    tl, tS, tdS, tc, ts = torch_split_model(cfg, params, cads, sads, tokens, labels)
    assert abs(loss - tl) < 1e-11
    assert np.allclose(S, tS, rtol=1e-11, atol=1e-12)
    assert np.allclose(dS, tdS, rtol=1e-9, atol=1e-13)
    assert set(sg.keys()) == set(ts.keys())
    for key, (dA, dB) in sg.items():
        assert np.allclose(dA, ts[key][0].grad.numpy(), rtol=1e-9, atol=1e-13), key
        assert np.allclose(dB, ts[key][1].grad.numpy(), rtol=1e-9, atol=1e-13), key
    for i in range(w.n_clients):
        assert set(cg[i].keys()) == set(tc[i].keys())
        for key, (dA, dB) in cg[i].items():
            assert np.allclose(dA, tc[i][key][0].grad.numpy(), rtol=1e-9, atol=1e-13), (i, key)
            assert np.allclose(dB, tc[i][key][1].grad.numpy(), rtol=1e-9, atol=1e-13), (i, key)
    assert min(np.abs(g[0]).max() for g in sg.values()) > 1e-8      # no target's gradient is trivially zero
    assert min(np.abs(g[1]).max() for g in cg[0].values()) > 1e-8


def test_llama_finite_difference_gradients():
    w = tiny_llama(n_layer=2, cut=1, batch_per_client=1)
    cfg = ocfg(w)
    params, cads, sads, tokens, labels = setup(w)
    loss, S, dS, sg, cg = oracle_grads(cfg, params, cads, sads, tokens, labels)
    rng = np.random.default_rng(15)
    eps = 1e-5

    def check(mat, grad, n=4):
        for _ in range(n):
            idx = tuple(rng.integers(0, s) for s in mat.shape)
            old = mat[idx]
            mat[idx] = old + eps
            lp = oracle_grads(cfg, params, cads, sads, tokens, labels)[0]
            mat[idx] = old - eps
            lm = oracle_grads(cfg, params, cads, sads, tokens, labels)[0]
            mat[idx] = old
            fd = (lp - lm) / (2 * eps)
            assert abs(fd - grad[idx]) <= 1e-6 * max(1.0, abs(fd)) + 1e-8, (fd, grad[idx])

    for key, (dA, dB) in sg.items():
        check(sads[key]["A"], dA)
        check(sads[key]["B"], dB)
    for key, (dA, dB) in cg[1].items():
        check(cads[1][key]["A"], dA)
        check(cads[1][key]["B"], dB)
    for _ in range(6):
        idx = tuple(rng.integers(0, s) for s in S.shape)
        Sp, Sm = S.copy(), S.copy()
        Sp[idx] += eps
        Sm[idx] -= eps
        fd = (O.server_fwd_bwd(cfg, params, sads, Sp, labels)[0]
              - O.server_fwd_bwd(cfg, params, sads, Sm, labels)[0]) / (2 * eps)
        assert abs(fd - dS[idx]) <= 1e-6 * max(1.0, abs(fd)) + 1e-8


def test_llama_zero_b_and_every_cut():
    L = 3
    base = tiny_llama(n_layer=L)
    params = f64(synth.make_frozen(base, randomize_affine=True))
    tokens, labels = synth.make_tokens(base)
    # B = 0: the adapters do not change the function, whatever A is
    zero_b = ads64(synth.make_adapters(base, range(L), nonzero_b=False, salt=3))
    other_a = ads64(synth.make_adapters(base, range(L), nonzero_b=False, salt=4))
    losses = []
    for ads in (zero_b, other_a):
        cfg = ocfg(base)
        cads = [{k: v for k, v in ads.items() if k[0] < 1} for _ in range(base.n_clients)]
        sads = {k: v for k, v in ads.items() if k[0] >= 1}
        losses.append(oracle_grads(cfg, params, cads, sads, tokens, labels)[0])
    assert losses[0] == losses[1]
    # every cut is the same function of the tokens
    layer_ads = ads64(synth.make_adapters(base, range(L), nonzero_b=True, salt=3), 5.0)
    ref = None
    for cut in range(1, L):
        w = tiny_llama(n_layer=L, cut=cut)
        cads = [{k: v for k, v in layer_ads.items() if k[0] < cut} for _ in range(w.n_clients)]
        sads = {k: v for k, v in layer_ads.items() if k[0] >= cut}
        loss, S, dS, sg, cg = oracle_grads(ocfg(w), params, cads, sads, tokens, labels)
        per_layer = dict(sg)
        for key in cads[0]:
            per_layer[key] = tuple(sum(cg[i][key][j] for i in range(w.n_clients)) for j in (0, 1))
        if ref is None:
            ref = (loss, per_layer)
        else:
            assert abs(loss - ref[0]) < 1e-12
            for key in per_layer:
                assert np.allclose(per_layer[key][0], ref[1][key][0], rtol=1e-9, atol=1e-14)
                assert np.allclose(per_layer[key][1], ref[1][key][1], rtol=1e-9, atol=1e-14)


def test_llama_initial_loss_is_ln_vocab():
    w = tiny_llama(vocab=1000, d_model=32, n_head=2, d_ff=64)
    params = f64(synth.make_frozen(w))
    cads = [ads64(synth.make_adapters(w, range(w.cut))) for _ in range(w.n_clients)]
    sads = ads64(synth.make_adapters(w, range(w.cut, w.n_layer)))
    tokens, labels = synth.make_tokens(w)
    loss = oracle_grads(ocfg(w), params, cads, sads, tokens, labels)[0]
    assert abs(loss - math.log(w.vocab)) < 0.05


def test_llama_round_runs_and_aggregates():
    w = tiny_llama()
    cfg = ocfg(w, optimizer="sgd")
    params, cads, sads, tokens, labels = setup(w)
    before = [c[(0, "o")]["B"].copy() for c in cads]
    state = O.OracleState(client_adapters=cads, server_adapters=sads)
    loss, info = O.split_round(cfg, params, state, tokens, labels, [3, 5])
    assert info["aggregated"]
    exp = 0.375 * (before[0] - cfg.lr_client * info["client_grads"][0][(0, "o")][1]) \
        + 0.625 * (before[1] - cfg.lr_client * info["client_grads"][1][(0, "o")][1])
    for c in state.client_adapters:
        assert np.allclose(c[(0, "o")]["B"], exp, rtol=0, atol=1e-7 * np.abs(exp).max())
