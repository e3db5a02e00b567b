"""What bf16 STORAGE alone costs: the split model's three calls in exact fp64 arithmetic, except that every
tensor a bf16 pipeline keeps in memory between two operators is rounded to bf16 once where it is stored.

This is test infrastructure built from the oracle's own primitives (the only arithmetic of its own is
the attention backward written with the row term taken from the stored output, see below).  It answers one question: how far from the exact result can
ANY implementation with bf16 activations land, whatever its kernels do?  The bounds of the GPU parity
tests that exceed the general 2e-2 are derived from it (tests/test_storage_noise.py).

Storage points (the tensors a block writes to memory): the normalised inputs u and u2, the rank-r
projections h, the fused qkv (again after the rotation of q and k in the Llama-shaped block), the
attention output o, the residual stream x_mid and x_out, the MLP pre-activation(s) and activation; the
final normalised x, the logits and their gradient; in the backward every gradient handed from one
operator to the next.  The adapters enter the products as bf16 copies (A, and B scaled by alpha/r); the
adapter gradients themselves are accumulated and kept in fp32 and are not rounded.
"""
import numpy as np

from oracle import splitlora_oracle as O


def _st(x):
    return O.round_to_bf16(np.asarray(x, dtype=np.float64))


def _ident(x):
    return x


def _block_fwd(cfg, params, l, adapters, x, st):
    nseq, T, d = x.shape
    s = cfg.scale
    llama = cfg.arch == "llama"
    P = lambda r: params[f"h.{l}.{r}"]
    x2 = x.reshape(nseq * T, d)
    if llama:
        u, n1 = O.rmsnorm_fwd(x2, P("ln1.g"), cfg.norm_eps)
    else:
        u, n1 = O.layernorm_fwd(x2, P("ln1.g"), P("ln1.b"), cfg.norm_eps)
    u = st(u)
    qkv = u @ P("attn.qkv.w").T + (0.0 if llama else P("attn.qkv.b"))
    h = {}
    for t in cfg.targets:
        if t == "o":
            continue
        ad = adapters[(l, t)]
        j = O.TARGET_SLICE[t]
        h[t] = st(u @ st(ad["A"]).T)
        qkv[:, j * d:(j + 1) * d] += h[t] @ st(s * ad["B"]).T
    qkv = st(qkv)
    q, k, v = (qkv[:, j * d:(j + 1) * d].reshape(nseq, T, d) for j in range(3))
    if llama:
        q = st(O.rope_rotate(q, cfg.n_head, cfg.rope_theta))
        k = st(O.rope_rotate(k, cfg.n_head, cfg.rope_theta))
    o, probs = O.causal_attention_fwd(q, k, v, cfg.n_head)
    o2 = st(o.reshape(nseq * T, d))
    proj = o2 @ P("attn.proj.w").T + (0.0 if llama else P("attn.proj.b"))
    if "o" in cfg.targets:
        ad = adapters[(l, "o")]
        h["o"] = st(o2 @ st(ad["A"]).T)
        proj = proj + h["o"] @ st(s * ad["B"]).T
    x_mid = st(x2 + proj)
    if llama:
        u2, n2 = O.rmsnorm_fwd(x_mid, P("ln2.g"), cfg.norm_eps)
        u2 = st(u2)
        zg, zu = st(u2 @ P("mlp.gate.w").T), st(u2 @ P("mlp.up.w").T)
        a = st(O.silu(zg) * zu)
        y = st(x_mid + a @ P("mlp.down.w").T)
        z = (zg, zu)
    else:
        u2, n2 = O.layernorm_fwd(x_mid, P("ln2.g"), P("ln2.b"), cfg.norm_eps)
        u2 = st(u2)
        z = st(u2 @ P("mlp.fc1.w").T + P("mlp.fc1.b"))
        a = st(O.gelu_fwd(z, cfg.gelu_tanh))
        y = st(x_mid + a @ P("mlp.fc2.w").T + P("mlp.fc2.b"))
    cache = dict(n1=n1, n2=n2, u=u, h=h, q=q, k=k, v=v, probs=probs, o2=o2, z=z, shape=(nseq, T, d))
    return y.reshape(nseq, T, d), cache


def _attention_bwd_from_stored_o(do, q, k, v, probs, o, n_head):
    """The attention gradients with the row term D_i = sum_j P_ij dP_ij taken as sum_c dO_ic O_ic from the
    STORED output (the two are equal in exact arithmetic; a backward pass that does not keep P has only
    the stored O to compute it from, and O carries its bf16 rounding)."""
    nseq, T, d = q.shape
    dh = d // n_head
    dq, dk, dv = np.zeros_like(q), np.zeros_like(k), np.zeros_like(v)
    for b in range(nseq):
        for h in range(n_head):
            sl = slice(h * dh, (h + 1) * dh)
            p = probs[b, h]
            dv[b, :, sl] = p.T @ do[b, :, sl]
            dp = do[b, :, sl] @ v[b, :, sl].T
            D = (do[b, :, sl] * o[b, :, sl]).sum(axis=-1, keepdims=True)
            ds = p * (dp - D) / np.sqrt(dh)
            dq[b, :, sl] = ds @ k[b, :, sl]
            dk[b, :, sl] = ds.T @ q[b, :, sl]
    return dq, dk, dv


def _block_bwd(cfg, params, l, adapters, dy, cache, st):
    nseq, T, d = cache["shape"]
    s = cfg.scale
    llama = cfg.arch == "llama"
    P = lambda r: params[f"h.{l}.{r}"]
    nbwd = O.rmsnorm_bwd if llama else O.layernorm_bwd
    dy2 = dy.reshape(nseq * T, d)
    if llama:
        zg, zu = cache["z"]
        da = st(dy2 @ P("mlp.down.w"))
        dzg, dzu = st(da * zu * O.silu_grad(zg)), st(da * O.silu(zg))
        du2 = st(dzg @ P("mlp.gate.w") + dzu @ P("mlp.up.w"))
    else:
        dz = st((dy2 @ P("mlp.fc2.w")) * O.gelu_grad(cache["z"], cfg.gelu_tanh))
        du2 = st(dz @ P("mlp.fc1.w"))
    dx_mid = st(dy2 + nbwd(du2, cache["n2"]))
    grads = {}
    do2 = dx_mid @ P("attn.proj.w")
    if "o" in cfg.targets:
        ad = adapters[(l, "o")]
        dh = st(dx_mid @ st(s * ad["B"]))
        do2 = do2 + dh @ st(ad["A"])
        grads[(l, "o")] = (dh.T @ cache["o2"], s * (dx_mid.T @ cache["h"]["o"]))
    do2 = st(do2)
    dq, dk, dv = _attention_bwd_from_stored_o(do2.reshape(nseq, T, d), cache["q"], cache["k"], cache["v"],
                                              cache["probs"], cache["o2"].reshape(nseq, T, d), cfg.n_head)
    dq, dk, dv = st(dq), st(dk), st(dv)
    if llama:
        dq = st(O.rope_rotate(dq, cfg.n_head, cfg.rope_theta, sign=-1.0))
        dk = st(O.rope_rotate(dk, cfg.n_head, cfg.rope_theta, sign=-1.0))
    dqkv = np.concatenate([dq.reshape(-1, d), dk.reshape(-1, d), dv.reshape(-1, d)], axis=1)
    u = cache["u"]
    du = dqkv @ P("attn.qkv.w")
    for t in cfg.targets:
        if t == "o":
            continue
        ad = adapters[(l, t)]
        j = O.TARGET_SLICE[t]
        dyt = dqkv[:, j * d:(j + 1) * d]
        dh = st(dyt @ st(s * ad["B"]))
        du = du + dh @ st(ad["A"])
        grads[(l, t)] = (dh.T @ u, s * (dyt.T @ cache["h"][t]))
    dx = st(dx_mid + nbwd(st(du), cache["n1"]))
    return dx.reshape(nseq, T, d), grads


def three_calls(cfg, params, client_adapters, server_adapters, tokens, labels, stored=True, cuts=None):
    """S, dS, loss, server gradients, per-client gradients; stored=False gives the exact model (it must then
    agree with the oracle's own three calls, which the CPU tests check).  cuts: per-client cut depths
    (non-decreasing), None for cfg.cut everywhere; S and dS are stacked [K, b, T, d] either way, row block
    i at client i's depth."""
    st = _st if stored else _ident
    hand = O.round_to_bf16 if cfg.bf16_handoff else _ident
    K = tokens.shape[0]
    cuts = [cfg.cut] * K if cuts is None else list(cuts)
    S, ccaches = [], []
    for i in range(K):
        x = st(O.embed(cfg, params, tokens[i]))
        cl = []
        for l in range(cuts[i]):
            x, c = _block_fwd(cfg, params, l, client_adapters[i], x, st)
            cl.append(c)
        S.append(hand(x))
        ccaches.append(cl)
    b, T, d = S[0].shape
    x = np.zeros((0, T, d))
    order, entered, scaches = [], {}, {}
    for l in range(min(cuts), cfg.n_layer + 1):
        entered[l] = [i for i in range(K) if cuts[i] == l]
        if entered[l]:
            x = np.concatenate([x] + [S[i] for i in entered[l]], axis=0)
            order += entered[l]
        if l < cfg.n_layer:
            x, scaches[l] = _block_fwd(cfg, params, l, server_adapters, x, st)
    if cfg.arch == "llama":
        xf, nf = O.rmsnorm_fwd(x.reshape(-1, d), params["lnf.g"], cfg.norm_eps)
    else:
        xf, nf = O.layernorm_fwd(x.reshape(-1, d), params["lnf.g"], params["lnf.b"], cfg.norm_eps)
    head = params.get("head.w", params["wte"])
    z = st(st(xf) @ head.T)
    loss, dz = O.cross_entropy_fwd_bwd(z, np.concatenate([labels[i].reshape(-1) for i in order]))
    dxf = st(st(dz) @ head)
    dx = st((O.rmsnorm_bwd if cfg.arch == "llama" else O.layernorm_bwd)(dxf, nf)).reshape(-1, T, d)
    sg, dS = {}, [None] * K
    for l in range(cfg.n_layer, min(cuts) - 1, -1):
        if l < cfg.n_layer:
            dx, g = _block_bwd(cfg, params, l, server_adapters, dx, scaches[l], st)
            sg.update(g)
        keep = dx.shape[0] - len(entered[l]) * b
        for j, i in enumerate(entered[l]):
            dS[i] = hand(dx[keep + j * b: keep + (j + 1) * b])
        dx = dx[:keep]
    cg = []
    for i in range(K):
        dx, grads = dS[i], {}
        for l in range(cuts[i] - 1, -1, -1):
            dx, g = _block_bwd(cfg, params, l, client_adapters[i], dx, ccaches[i][l], st)
            grads.update(g)
        cg.append(grads)
    return np.stack(S), np.stack(dS), loss, sg, cg
