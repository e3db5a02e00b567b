"""Plain fp64 CPU statement of one SplitLoRA round (arxiv 2407.00952).

TEST INFRASTRUCTURE ONLY.  This module is the slow, obviously-correct checker
that the CUDA library is compared against.  Nothing in the product path may
import it; it imports nothing from the CUDA package and shares no code,
tables or helpers with it.

Everything is computed in float64 with numpy, one step after another in the
order of the paper's Algorithm 1; no blocking, fusion or reordering.  Each
function names the passage of the paper it restates.

Conventions (the paper fixes none of them, see the readings listed in the
design notes):
  * activations are [rows, features]; a linear layer stores W as [out, in];
  * a LoRA adapter is A [r, in] (Gaussian init) and B [out, r] (zero init) and
    changes the layer to  y = x W^T + bias + s (x A^T) B^T  with s = alpha / r
    (paper Sec. II-C: W + dW with dW a product of two rank-r factors);
  * the model is a pre-LN GPT-style decoder; the fused attention projection
    'attn.qkv.w' is [3d, d] with the q, k, v slices stacked in that order and
    adapters sit on the slices named in cfg.targets;
  * cfg.arch = "llama" selects a second block shape that the paper does not describe (it only
    cites Llama-2 as an LLM): RMSNorm, rotary positions on q and k (pairs (j, j + dh/2)),
    SwiGLU, no biases, no learned positions, a head separate from wte, and "o" (the attention
    output projection) as a fourth possible adapter target.

Parity status: every function below is pinned by tests/test_oracle_*.py
(library routines + autograd in fp64, finite differences, closed forms,
the invariants the paper states).  The paper's accuracy numbers (PPL, BLEU,
...) are "parity unpinned": they need a dataset and weights that are not
available.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64
TARGET_SLICE = {"q": 0, "k": 1, "v": 2}  # position of a target inside the fused qkv weight


# --------------------------------------------------------------------------
# configuration
# --------------------------------------------------------------------------
@dataclass
class OracleConfig:
    n_layer: int
    cut: int                      # blocks 1..cut live on the clients (Sec. III-B, model partition)
    d_model: int
    n_head: int
    d_ff: int
    vocab: int
    max_seq: int
    lora_r: int
    lora_alpha: float
    targets: Tuple[str, ...] = ("q", "v")
    n_clients: int = 2
    batch_per_client: int = 1
    seq: int = 8
    bf16_handoff: bool = False    # round the two hand-off buffers to bf16 once (bf16 configs)
    optimizer: str = "adamw"      # "sgd" is the literal rule of Eq. 4-7
    lr_client: float = 1e-3
    lr_server: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.999
    adam_eps: float = 1e-8
    weight_decay: float = 0.01
    agg_interval: int = 1         # I of Algorithm 1
    norm_eps: float = 1e-5
    gelu_tanh: bool = True
    # "gpt": LayerNorm, learned positions, GELU MLP, biases, head tied to wte (the paper's GPT-2).
    # "llama": RMSNorm, rotary positions on q and k, SwiGLU MLP, no biases, separate head.  The
    # paper only cites Llama-2 as an LLM; this shape is defined by this file (see the notes).
    arch: str = "gpt"
    rope_theta: float = 10000.0

    @property
    def scale(self) -> float:
        return float(self.lora_alpha) / float(self.lora_r)


# --------------------------------------------------------------------------
# bf16 rounding of a hand-off buffer (round to nearest, ties to even)
# --------------------------------------------------------------------------
def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Value of x after storage in a bfloat16 buffer (fp64 -> fp32 -> bf16, RNE), as fp64."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    bits = f.view(np.uint32).astype(np.uint64)
    lsb = (bits >> np.uint64(16)) & np.uint64(1)
    rounded = (bits + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    return rounded.astype(np.uint32).view(np.float32).astype(F64).reshape(x.shape)


# --------------------------------------------------------------------------
# layer primitives: forward and the gradients the round needs
# --------------------------------------------------------------------------
def lora_linear_fwd(x, W, bias, A, B, s):
    """y = x W^T + bias + s (x A^T) B^T      (Sec. II-C, W + dW with rank-r dW).

    x [m, in], W [out, in], bias [out] or None, A [r, in], B [out, r].
    Returns y [m, out] and h = x A^T [m, r].
    """
    y = x @ W.T
    if bias is not None:
        y = y + bias
    h = x @ A.T
    y = y + s * (h @ B.T)
    return y, h


def lora_linear_bwd(dy, x, W, A, B, s):
    """Gradients of lora_linear_fwd w.r.t. x, A and B (W and bias are frozen: no dW).

    dx = dy W + s (dy B) A ;  dA = s (dy B)^T x ;  dB = s dy^T (x A^T).
    These are the G_A, G_B of Eq. 4-7.
    """
    dh = s * (dy @ B)            # [m, r]
    dx = dy @ W + dh @ A
    dA = dh.T @ x                # [r, in]
    dB = s * (dy.T @ (x @ A.T))  # [out, r]
    return dx, dA, dB


def layernorm_fwd(x, g, b, eps):
    """Row-wise LayerNorm: (x - mean) / sqrt(var + eps) * g + b, biased variance."""
    mu = x.mean(axis=-1, keepdims=True)
    xc = x - mu
    var = (xc * xc).mean(axis=-1, keepdims=True)
    rstd = 1.0 / np.sqrt(var + eps)
    xhat = xc * rstd
    return xhat * g + b, (xhat, rstd, g)


def layernorm_bwd(dy, cache):
    """Gradient of layernorm_fwd w.r.t. x only (gain and bias are frozen)."""
    xhat, rstd, g = cache
    dxhat = dy * g
    m1 = dxhat.mean(axis=-1, keepdims=True)
    m2 = (dxhat * xhat).mean(axis=-1, keepdims=True)
    return (dxhat - m1 - xhat * m2) * rstd


_SQRT_2_OVER_PI = math.sqrt(2.0 / math.pi)


def gelu_fwd(z, tanh_form=True):
    """GELU; the tanh form is the GPT-2 definition, the other is the exact erf form."""
    if tanh_form:
        return 0.5 * z * (1.0 + np.tanh(_SQRT_2_OVER_PI * (z + 0.044715 * z ** 3)))
    erf = np.vectorize(math.erf, otypes=[F64])
    return 0.5 * z * (1.0 + erf(z / math.sqrt(2.0)))


def gelu_grad(z, tanh_form=True):
    """d gelu(z) / dz."""
    if tanh_form:
        u = _SQRT_2_OVER_PI * (z + 0.044715 * z ** 3)
        t = np.tanh(u)
        du = _SQRT_2_OVER_PI * (1.0 + 3.0 * 0.044715 * z * z)
        return 0.5 * (1.0 + t) + 0.5 * z * (1.0 - t * t) * du
    erf = np.vectorize(math.erf, otypes=[F64])
    return 0.5 * (1.0 + erf(z / math.sqrt(2.0))) + z * np.exp(-0.5 * z * z) / math.sqrt(2.0 * math.pi)


def rmsnorm_fwd(x, g, eps):
    """Row-wise RMSNorm: x / sqrt(mean(x^2) + eps) * g  (no centring, no bias)."""
    ms = (x * x).mean(axis=-1, keepdims=True)
    rstd = 1.0 / np.sqrt(ms + eps)
    xhat = x * rstd
    return xhat * g, (xhat, rstd, g)


def rmsnorm_bwd(dy, cache):
    """Gradient of rmsnorm_fwd w.r.t. x only (the gain is frozen)."""
    xhat, rstd, g = cache
    dxhat = dy * g
    m2 = (dxhat * xhat).mean(axis=-1, keepdims=True)
    return (dxhat - xhat * m2) * rstd


def rope_rotate(x, n_head, theta, sign=1.0):
    """Rotary position embedding on x [nseq, T, d], heads split d contiguously.

    Inside each head of width dh, element j < dh/2 is paired with element j + dh/2; at position t
    the pair is rotated by the angle sign * t * theta^(-2j/dh).  sign=-1 is the inverse rotation,
    which is also the gradient map (the rotation matrix is orthogonal).
    """
    nseq, T, d = x.shape
    dh = d // n_head
    half = dh // 2
    j = np.arange(half, dtype=F64)
    inv_freq = theta ** (-2.0 * j / dh)
    ang = sign * np.arange(T, dtype=F64)[:, None] * inv_freq[None, :]       # [T, half]
    cos, sin = np.cos(ang)[None, :, None, :], np.sin(ang)[None, :, None, :]
    xh = x.reshape(nseq, T, n_head, dh)
    lo, hi = xh[..., :half], xh[..., half:]
    out = np.concatenate([lo * cos - hi * sin, hi * cos + lo * sin], axis=-1)
    return out.reshape(nseq, T, d)


def silu(z):
    return z / (1.0 + np.exp(-z))


def silu_grad(z):
    sg = 1.0 / (1.0 + np.exp(-z))
    return sg * (1.0 + z * (1.0 - sg))


def causal_attention_fwd(q, k, v, n_head):
    """Multi-head causal softmax attention.  q, k, v [nseq, T, d]; heads split d contiguously.

    For each sequence and head:  P = softmax(q k^T / sqrt(dh) + causal mask),  o = P v.
    """
    nseq, T, d = q.shape
    dh = d // n_head
    o = np.zeros_like(q)
    probs = np.zeros((nseq, n_head, T, T), dtype=F64)
    mask = np.tril(np.ones((T, T), dtype=bool))
    for b in range(nseq):
        for h in range(n_head):
            sl = slice(h * dh, (h + 1) * dh)
            sc = (q[b, :, sl] @ k[b, :, sl].T) / math.sqrt(dh)
            sc = np.where(mask, sc, -np.inf)
            sc = sc - sc.max(axis=-1, keepdims=True)
            p = np.exp(sc)
            p = p / p.sum(axis=-1, keepdims=True)
            probs[b, h] = p
            o[b, :, sl] = p @ v[b, :, sl]
    return o, probs


def causal_attention_bwd(do, q, k, v, probs, n_head):
    """Gradients of causal_attention_fwd w.r.t. q, k, v."""
    nseq, T, d = q.shape
    dh = d // n_head
    dq = np.zeros_like(q)
    dk = np.zeros_like(k)
    dv = np.zeros_like(v)
    for b in range(nseq):
        for h in range(n_head):
            sl = slice(h * dh, (h + 1) * dh)
            p = probs[b, h]
            dv[b, :, sl] = p.T @ do[b, :, sl]
            dp = do[b, :, sl] @ v[b, :, sl].T
            ds = p * (dp - (dp * p).sum(axis=-1, keepdims=True))
            ds = ds / math.sqrt(dh)
            dq[b, :, sl] = ds @ k[b, :, sl]
            dk[b, :, sl] = ds.T @ q[b, :, sl]
    return dq, dk, dv


def cross_entropy_fwd_bwd(z, labels):
    """Mean token-level cross-entropy over the positions whose label is >= 0.

    loss = mean_m [ logsumexp(z_m) - z_m[y_m] ],  dz = (softmax(z) - onehot(y)) / n_valid.
    z [m, V], labels [m] (negative = ignored).  (Sec. III-B step a3: the server computes
    the loss from its predictions and the labels.)
    """
    valid = labels >= 0
    n_valid = int(valid.sum())
    zmax = z.max(axis=-1, keepdims=True)
    e = np.exp(z - zmax)
    ssum = e.sum(axis=-1, keepdims=True)
    lse = (zmax + np.log(ssum))[:, 0]
    rows = np.arange(z.shape[0])
    safe = np.where(valid, labels, 0)
    per_tok = np.where(valid, lse - z[rows, safe], 0.0)
    loss = per_tok.sum() / n_valid
    dz = e / ssum
    dz[rows, safe] -= 1.0
    dz = dz * valid[:, None] / n_valid
    return float(loss), dz


# --------------------------------------------------------------------------
# one decoder block with adapters on the selected attention projections
# --------------------------------------------------------------------------
def _pname(l, rest):
    return f"h.{l}.{rest}"


def block_fwd(cfg: OracleConfig, params, l: int, adapters, x):
    """Pre-LN decoder block l (0-based) on x [nseq, T, d] with adapter set `adapters`.

    adapters[(l, target)] = {"A": [r, d], "B": [d, r]} for each target in cfg.targets.
    """
    if cfg.arch == "llama":
        return llama_block_fwd(cfg, params, l, adapters, x)
    nseq, T, d = x.shape
    s = cfg.scale
    x2 = x.reshape(nseq * T, d)
    u, ln1 = layernorm_fwd(x2, params[_pname(l, "ln1.g")], params[_pname(l, "ln1.b")], cfg.norm_eps)
    Wqkv = params[_pname(l, "attn.qkv.w")]
    bqkv = params[_pname(l, "attn.qkv.b")]
    qkv = u @ Wqkv.T + bqkv
    for t in cfg.targets:
        if t == "o":
            continue
        ad = adapters[(l, t)]
        j = TARGET_SLICE[t]
        # the slice [j*d, (j+1)*d) of the fused projection is a LoRA layer of its own
        qkv[:, j * d:(j + 1) * d] += s * ((u @ ad["A"].T) @ ad["B"].T)
    q = qkv[:, 0:d].reshape(nseq, T, d)
    k = qkv[:, d:2 * d].reshape(nseq, T, d)
    v = qkv[:, 2 * d:3 * d].reshape(nseq, T, d)
    o, probs = causal_attention_fwd(q, k, v, cfg.n_head)
    o2 = o.reshape(nseq * T, d)
    if "o" in cfg.targets:     # the output projection as a LoRA layer
        ad = adapters[(l, "o")]
        proj, _ = lora_linear_fwd(o2, params[_pname(l, "attn.proj.w")], params[_pname(l, "attn.proj.b")],
                                  ad["A"], ad["B"], s)
        x_mid = x2 + proj
    else:
        x_mid = x2 + o2 @ params[_pname(l, "attn.proj.w")].T + params[_pname(l, "attn.proj.b")]
    u2, ln2 = layernorm_fwd(x_mid, params[_pname(l, "ln2.g")], params[_pname(l, "ln2.b")], cfg.norm_eps)
    z = u2 @ params[_pname(l, "mlp.fc1.w")].T + params[_pname(l, "mlp.fc1.b")]
    a = gelu_fwd(z, cfg.gelu_tanh)
    y = x_mid + a @ params[_pname(l, "mlp.fc2.w")].T + params[_pname(l, "mlp.fc2.b")]
    cache = dict(ln1=ln1, u=u, q=q, k=k, v=v, probs=probs, o2=o2, ln2=ln2, z=z, shape=(nseq, T, d))
    return y.reshape(nseq, T, d), cache


def block_bwd(cfg: OracleConfig, params, l: int, adapters, dy, cache):
    """Back-propagate dy [nseq, T, d] through block l.  Returns dx and {(l, target): (dA, dB)}."""
    if cfg.arch == "llama":
        return llama_block_bwd(cfg, params, l, adapters, dy, cache)
    nseq, T, d = cache["shape"]
    s = cfg.scale
    dy2 = dy.reshape(nseq * T, d)
    # MLP branch
    da = dy2 @ params[_pname(l, "mlp.fc2.w")]
    dz = da * gelu_grad(cache["z"], cfg.gelu_tanh)
    du2 = dz @ params[_pname(l, "mlp.fc1.w")]
    dx_mid = dy2 + layernorm_bwd(du2, cache["ln2"])
    # attention branch
    grads = {}
    if "o" in cfg.targets:
        ad = adapters[(l, "o")]
        do2, dAo, dBo = lora_linear_bwd(dx_mid, cache["o2"], params[_pname(l, "attn.proj.w")], ad["A"], ad["B"], s)
        grads[(l, "o")] = (dAo, dBo)
        do = do2.reshape(nseq, T, d)
    else:
        do = (dx_mid @ params[_pname(l, "attn.proj.w")]).reshape(nseq, T, d)
    dq, dk, dv = causal_attention_bwd(do, cache["q"], cache["k"], cache["v"], cache["probs"], cfg.n_head)
    dqkv = np.concatenate([dq.reshape(-1, d), dk.reshape(-1, d), dv.reshape(-1, d)], axis=1)
    u = cache["u"]
    du = dqkv @ params[_pname(l, "attn.qkv.w")]
    for t in cfg.targets:
        if t == "o":
            continue
        ad = adapters[(l, t)]
        j = TARGET_SLICE[t]
        dyt = dqkv[:, j * d:(j + 1) * d]
        dh = s * (dyt @ ad["B"])
        du = du + dh @ ad["A"]
        grads[(l, t)] = (dh.T @ u, s * (dyt.T @ (u @ ad["A"].T)))
    dx = dx_mid + layernorm_bwd(du, cache["ln1"])
    return dx.reshape(nseq, T, d), grads


# --------------------------------------------------------------------------
# the Llama-shaped block (not in the paper: RMSNorm, rotary q/k, SwiGLU, no biases; adapters on
# any of q, k, v and the attention output projection o)
# --------------------------------------------------------------------------
def llama_block_fwd(cfg: OracleConfig, params, l: int, adapters, x):
    nseq, T, d = x.shape
    s = cfg.scale
    x2 = x.reshape(nseq * T, d)
    u, n1 = rmsnorm_fwd(x2, params[_pname(l, "ln1.g")], cfg.norm_eps)
    qkv = u @ params[_pname(l, "attn.qkv.w")].T
    for t in cfg.targets:
        if t == "o":
            continue
        ad = adapters[(l, t)]
        j = TARGET_SLICE[t]
        qkv[:, j * d:(j + 1) * d] += s * ((u @ ad["A"].T) @ ad["B"].T)
    q_pre = qkv[:, 0:d].reshape(nseq, T, d)
    k_pre = qkv[:, d:2 * d].reshape(nseq, T, d)
    v = qkv[:, 2 * d:3 * d].reshape(nseq, T, d)
    q = rope_rotate(q_pre, cfg.n_head, cfg.rope_theta)
    k = rope_rotate(k_pre, cfg.n_head, cfg.rope_theta)
    o, probs = causal_attention_fwd(q, k, v, cfg.n_head)
    o2 = o.reshape(nseq * T, d)
    if "o" in cfg.targets:
        ad = adapters[(l, "o")]
        attn_out, _ = lora_linear_fwd(o2, params[_pname(l, "attn.proj.w")], None, ad["A"], ad["B"], s)
    else:
        attn_out = o2 @ params[_pname(l, "attn.proj.w")].T
    x_mid = x2 + attn_out
    u2, n2 = rmsnorm_fwd(x_mid, params[_pname(l, "ln2.g")], cfg.norm_eps)
    zg = u2 @ params[_pname(l, "mlp.gate.w")].T
    zu = u2 @ params[_pname(l, "mlp.up.w")].T
    a = silu(zg) * zu
    y = x_mid + a @ params[_pname(l, "mlp.down.w")].T
    cache = dict(n1=n1, u=u, q=q, k=k, v=v, probs=probs, o2=o2, n2=n2, zg=zg, zu=zu, shape=(nseq, T, d))
    return y.reshape(nseq, T, d), cache


def llama_block_bwd(cfg: OracleConfig, params, l: int, adapters, dy, cache):
    nseq, T, d = cache["shape"]
    s = cfg.scale
    dy2 = dy.reshape(nseq * T, d)
    grads = {}
    # MLP branch
    da = dy2 @ params[_pname(l, "mlp.down.w")]
    dzu = da * silu(cache["zg"])
    dzg = da * cache["zu"] * silu_grad(cache["zg"])
    du2 = dzg @ params[_pname(l, "mlp.gate.w")] + dzu @ params[_pname(l, "mlp.up.w")]
    dx_mid = dy2 + rmsnorm_bwd(du2, cache["n2"])
    # attention branch
    if "o" in cfg.targets:
        ad = adapters[(l, "o")]
        do2, dA, dB = lora_linear_bwd(dx_mid, cache["o2"], params[_pname(l, "attn.proj.w")], ad["A"], ad["B"], s)
        grads[(l, "o")] = (dA, dB)
    else:
        do2 = dx_mid @ params[_pname(l, "attn.proj.w")]
    dq, dk, dv = causal_attention_bwd(do2.reshape(nseq, T, d), cache["q"], cache["k"], cache["v"],
                                      cache["probs"], cfg.n_head)
    dq = rope_rotate(dq, cfg.n_head, cfg.rope_theta, sign=-1.0)
    dk = rope_rotate(dk, cfg.n_head, cfg.rope_theta, sign=-1.0)
    dqkv = np.concatenate([dq.reshape(-1, d), dk.reshape(-1, d), dv.reshape(-1, d)], axis=1)
    u = cache["u"]
    du = dqkv @ params[_pname(l, "attn.qkv.w")]
    for t in cfg.targets:
        if t == "o":
            continue
        ad = adapters[(l, t)]
        j = TARGET_SLICE[t]
        dyt = dqkv[:, j * d:(j + 1) * d]
        dh = s * (dyt @ ad["B"])
        du = du + dh @ ad["A"]
        grads[(l, t)] = (dh.T @ u, s * (dyt.T @ (u @ ad["A"].T)))
    dx = dx_mid + rmsnorm_bwd(du, cache["n1"])
    return dx.reshape(nseq, T, d), grads


# --------------------------------------------------------------------------
# the three split-fine-tuning calls (Algorithm 1, stage a)
# --------------------------------------------------------------------------
def embed(cfg: OracleConfig, params, tokens):
    """x0[b, t, :] = wte[tokens[b, t], :] + wpe[t, :]  (input side of the client sub-model)."""
    nseq, T = tokens.shape
    if cfg.arch == "llama":        # positions enter through the rotation of q and k instead
        return params["wte"][tokens].astype(F64)
    # stored values (fp32 or bf16-exact) are widened to fp64 before the first addition
    return params["wte"][tokens].astype(F64) + params["wpe"][:T][None, :, :].astype(F64)


def client_fwd(cfg: OracleConfig, params, client_adapters: Sequence[dict], tokens):
    """Step a1, Eq. 2: every client i runs blocks 1..cut with ITS OWN adapters R_{c,i}.

    tokens [K, b, T] int.  Returns S [K, b, T, d] (the cut-layer activations s_i, stacked)
    and the per-client caches needed by client_bwd.
    """
    K = tokens.shape[0]
    outs, caches = [], []
    for i in range(K):
        x = embed(cfg, params, tokens[i])
        cl = []
        for l in range(cfg.cut):
            x, c = block_fwd(cfg, params, l, client_adapters[i], x)
            cl.append(c)
        outs.append(x)
        caches.append(cl)
    S = np.stack(outs, axis=0)
    if cfg.bf16_handoff:
        S = round_to_bf16(S)      # step a2: the hand-off buffer is bf16 in bf16 configs
    return S, caches


def server_fwd_bwd(cfg: OracleConfig, params, server_adapters: dict, S, labels):
    """Step a3, Eq. 3: server forward on the concatenation S^t, loss, and backward.

    S [K, b, T, d], labels [K, b, T].  Returns loss, dS [K, b, T, d] and the server adapter
    gradients {(l, target): (dA, dB)}.  One pass over the concatenated batch, one loss.
    """
    K, b, T, d = S.shape
    x = S.reshape(K * b, T, d)
    caches = []
    for l in range(cfg.cut, cfg.n_layer):
        x, c = block_fwd(cfg, params, l, server_adapters, x)
        caches.append(c)
    if cfg.arch == "llama":
        xf, lnf = rmsnorm_fwd(x.reshape(-1, d), params["lnf.g"], cfg.norm_eps)
    else:
        xf, lnf = layernorm_fwd(x.reshape(-1, d), params["lnf.g"], params["lnf.b"], cfg.norm_eps)
    head = params.get("head.w", params["wte"])   # tied head unless a separate one is given
    z = xf @ head.T
    loss, dz = cross_entropy_fwd_bwd(z, labels.reshape(-1))
    dxf = dz @ head
    dx = (rmsnorm_bwd(dxf, lnf) if cfg.arch == "llama" else layernorm_bwd(dxf, lnf)).reshape(K * b, T, d)
    grads = {}
    for l in range(cfg.n_layer - 1, cfg.cut - 1, -1):
        dx, g = block_bwd(cfg, params, l, server_adapters, dx, caches[l - cfg.cut])
        grads.update(g)
    dS = dx.reshape(K, b, T, d)
    if cfg.bf16_handoff:
        dS = round_to_bf16(dS)    # step a4: gradient hand-off buffer
    return loss, dS, grads


def client_bwd_grads(cfg: OracleConfig, params, client_adapters: Sequence[dict], dS, caches):
    """Step a5: client i back-propagates dL/ds_i through blocks cut..1; returns its G_A, G_B."""
    K = dS.shape[0]
    all_grads = []
    for i in range(K):
        dx = dS[i]
        grads = {}
        for l in range(cfg.cut - 1, -1, -1):
            dx, g = block_bwd(cfg, params, l, client_adapters[i], dx, caches[i][l])
            grads.update(g)
        all_grads.append(grads)
    return all_grads


# --------------------------------------------------------------------------
# parameter updates (Eq. 4-7) and aggregation (Eq. 8-9)
# --------------------------------------------------------------------------
def sgd_update(p, g, lr):
    """Eq. 4-7 literally:  P <- P - gamma * G."""
    return p - lr * g


def adamw_update(p, g, m, v, step, lr, beta1, beta2, eps, wd):
    """One AdamW step (decoupled weight decay, bias correction); step counts from 1."""
    p = p * (1.0 - lr * wd)
    m = beta1 * m + (1.0 - beta1) * g
    v = beta2 * v + (1.0 - beta2) * g * g
    mhat = m / (1.0 - beta1 ** step)
    vhat = v / (1.0 - beta2 ** step)
    p = p - lr * mhat / (np.sqrt(vhat) + eps)
    return p, m, v


def aggregation_weights(counts) -> np.ndarray:
    """w_i = |D_i| / |D|  (Eq. 1, Eq. 8-9)."""
    c = np.asarray(counts, dtype=F64)
    return c / c.sum()


def aggregate(client_mats: Sequence[np.ndarray], counts) -> np.ndarray:
    """Eq. 8-9: P_c = sum_i (|D_i| / |D|) P_{c,i}, summed in client order."""
    w = aggregation_weights(counts)
    acc = np.zeros_like(np.asarray(client_mats[0], dtype=F64))
    for i, p in enumerate(client_mats):
        acc = acc + w[i] * np.asarray(p, dtype=F64)
    return acc


# --------------------------------------------------------------------------
# training state and one full round t of Algorithm 1
# --------------------------------------------------------------------------
def new_opt_state(adapters: dict):
    return {key: {"mA": np.zeros_like(ad["A"]), "vA": np.zeros_like(ad["A"]),
                  "mB": np.zeros_like(ad["B"]), "vB": np.zeros_like(ad["B"])}
            for key, ad in adapters.items()}


@dataclass
class OracleState:
    """R_s, {R_{c,i}}, optimizer moments and the round counter t."""
    client_adapters: List[dict]
    server_adapters: dict
    client_opt: List[dict] = field(default_factory=list)
    server_opt: dict = field(default_factory=dict)
    round_index: int = 0
    server_steps: int = 0
    client_steps: int = 0

    def __post_init__(self):
        if not self.client_opt:
            self.client_opt = [new_opt_state(a) for a in self.client_adapters]
        if not self.server_opt:
            self.server_opt = new_opt_state(self.server_adapters)


def apply_update(cfg: OracleConfig, adapters: dict, opt: dict, grads: dict, lr: float, step: int):
    """Update every A, B of one adapter set from its gradients with the configured rule."""
    for key, (dA, dB) in grads.items():
        ad, st = adapters[key], opt[key]
        if cfg.optimizer == "sgd":
            ad["A"] = sgd_update(ad["A"], dA, lr)
            ad["B"] = sgd_update(ad["B"], dB, lr)
        else:
            ad["A"], st["mA"], st["vA"] = adamw_update(ad["A"], dA, st["mA"], st["vA"], step, lr,
                                                       cfg.beta1, cfg.beta2, cfg.adam_eps, cfg.weight_decay)
            ad["B"], st["mB"], st["vB"] = adamw_update(ad["B"], dB, st["mB"], st["vB"], step, lr,
                                                       cfg.beta1, cfg.beta2, cfg.adam_eps, cfg.weight_decay)


def aggregate_clients(state: OracleState, counts, store_fp32: bool = True):
    """Stage b (b1-b3): average every client A and B separately (Eq. 8-9), then give the
    average back to every client as its adapters for the next round."""
    keys = list(state.client_adapters[0].keys())
    for key in keys:
        for name in ("A", "B"):
            avg = aggregate([ca[key][name] for ca in state.client_adapters], counts)
            if store_fp32:
                avg = avg.astype(np.float32).astype(F64)   # adapters are stored as fp32 masters
            for ca in state.client_adapters:
                ca[key][name] = avg.copy()


def aggregate_ranks(client_mats: Sequence[np.ndarray], counts, rank_axis: int) -> np.ndarray:
    """Clients whose adapters have different ranks r_i (Sec. V, heterogeneous configuration: the
    paper names per-client ranks as a direction and gives no rule for averaging them).  Reading
    taken: every matrix is padded with zeros along its rank axis (0 for A [r_i, in], 1 for
    B [out, r_i]) to the largest rank, and Eq. 8-9 is applied to the padded matrices: rank
    component j of the result is sum_i w_i P_i[j], a client without component j adding nothing.
    Returns the padded average."""
    r_max = max(np.asarray(p).shape[rank_axis] for p in client_mats)
    padded = []
    for p in client_mats:
        p = np.asarray(p, dtype=F64)
        widths = [(0, 0), (0, 0)]
        widths[rank_axis] = (0, r_max - p.shape[rank_axis])
        padded.append(np.pad(p, widths))
    return aggregate(padded, counts)


def aggregate_clients_ranks(state: OracleState, counts, store_fp32: bool = True):
    """Stage b with per-client ranks: the padded average (aggregate_ranks) goes back to every
    client cut to that client's own rank (its leading r_i components)."""
    for key in list(state.client_adapters[0].keys()):
        for name, axis in (("A", 0), ("B", 1)):
            avg = aggregate_ranks([ca[key][name] for ca in state.client_adapters], counts, axis)
            if store_fp32:
                avg = avg.astype(np.float32).astype(F64)
            for ca in state.client_adapters:
                r_i = ca[key][name].shape[axis]
                ca[key][name] = (avg[:r_i, :] if axis == 0 else avg[:, :r_i]).copy()


def split_round(cfg: OracleConfig, params, state: OracleState, tokens, labels, counts):
    """One iteration t of Algorithm 1.  Returns (loss, info) where info holds S, dS and the
    gradients so that tests can compare intermediate quantities."""
    state.round_index += 1
    # a1 + a2
    S, caches = client_fwd(cfg, params, state.client_adapters, tokens)
    # a3 (forward, loss, backward, server update with gamma_s)
    loss, dS, sgrads = server_fwd_bwd(cfg, params, state.server_adapters, S, labels)
    state.server_steps += 1
    apply_update(cfg, state.server_adapters, state.server_opt, sgrads, cfg.lr_server, state.server_steps)
    # a4 + a5 (client backward and update with gamma_c)
    cgrads = client_bwd_grads(cfg, params, state.client_adapters, dS, caches)
    state.client_steps += 1
    for i, g in enumerate(cgrads):
        apply_update(cfg, state.client_adapters[i], state.client_opt[i], g, cfg.lr_client, state.client_steps)
    # b: every I rounds (read "t mod I = 0")
    aggregated = False
    if state.round_index % cfg.agg_interval == 0:
        aggregate_clients(state, counts)
        aggregated = True
    return loss, dict(S=S, dS=dS, server_grads=sgrads, client_grads=cgrads, aggregated=aggregated)


# --------------------------------------------------------------------------
# clients cut at different depths (Sec. V, heterogeneous configuration)
# --------------------------------------------------------------------------
# The paper names the joint choice of cut layers and ranks per client as a direction and gives no rule.
# Reading taken here: client i runs blocks 1..c_i with its own adapters and hands off s_i at depth c_i;
# the server holds adapters on blocks c_min+1..L (c_min = min_i c_i) and takes client i's activations in
# at block c_i+1, so that at block l its batch is the concatenation of everything that has entered so
# far; there is still ONE loss (the mean over all valid positions of all clients) and one server update
# per round; dL/ds_i is handed back at depth c_i; Eq. 8-9 is applied per block to the clients that hold
# that block, w_i = |D_i| / sum over those holders.  With all c_i equal this is Algorithm 1 unchanged.
def client_fwd_cuts(cfg: OracleConfig, params, client_adapters: Sequence[dict], tokens, cuts):
    """Step a1 with per-client depth: returns [s_i] (each [b, T, d], rounded once to bf16 in bf16 configs)
    and the per-client caches."""
    outs, caches = [], []
    for i in range(tokens.shape[0]):
        x = embed(cfg, params, tokens[i])
        cl = []
        for l in range(cuts[i]):
            x, c = block_fwd(cfg, params, l, client_adapters[i], x)
            cl.append(c)
        outs.append(round_to_bf16(x) if cfg.bf16_handoff else x)
        caches.append(cl)
    return outs, caches


def server_fwd_bwd_cuts(cfg: OracleConfig, params, server_adapters: dict, S_list, labels, cuts):
    """Step a3 with per-client depth.  S_list[i] [b, T, d] enters at block cuts[i] (0-based index of the
    first server block it passes); labels [K, b, T].  Returns loss, [dL/ds_i] and the server gradients for
    blocks min(cuts)..L-1."""
    K = len(S_list)
    b, T, d = S_list[0].shape
    order = []                        # clients in the order they entered; rows of x follow this order
    x = np.zeros((0, T, d), dtype=F64)
    caches, entered_at = {}, {}
    for l in range(min(cuts), cfg.n_layer + 1):
        new = [i for i in range(K) if cuts[i] == l]
        if new:
            x = np.concatenate([x] + [S_list[i] for i in new], axis=0)
            order += new
        entered_at[l] = list(new)
        if l < cfg.n_layer:
            x, caches[l] = block_fwd(cfg, params, l, server_adapters, x)
    assert sorted(order) == list(range(K))
    if cfg.arch == "llama":
        xf, lnf = rmsnorm_fwd(x.reshape(-1, d), params["lnf.g"], cfg.norm_eps)
    else:
        xf, lnf = layernorm_fwd(x.reshape(-1, d), params["lnf.g"], params["lnf.b"], cfg.norm_eps)
    head = params.get("head.w", params["wte"])
    z = xf @ head.T
    lab = np.concatenate([labels[i].reshape(-1) for i in order])
    loss, dz = cross_entropy_fwd_bwd(z, lab)
    dxf = dz @ head
    dx = (rmsnorm_bwd(dxf, lnf) if cfg.arch == "llama" else layernorm_bwd(dxf, lnf)).reshape(-1, T, d)
    grads, dS = {}, [None] * K
    for l in range(cfg.n_layer, min(cuts) - 1, -1):
        if l < cfg.n_layer:
            dx, g = block_bwd(cfg, params, l, server_adapters, dx, caches[l])
            grads.update(g)
        n_new = len(entered_at[l])
        if n_new:                     # the last n_new * b sequences entered here: their gradient goes back
            keep = dx.shape[0] - n_new * b
            for j, i in enumerate(entered_at[l]):
                g_i = dx[keep + j * b: keep + (j + 1) * b]
                dS[i] = round_to_bf16(g_i) if cfg.bf16_handoff else g_i
            dx = dx[:keep]
            order = order[:len(order) - n_new]
    return loss, dS, grads


def client_bwd_grads_cuts(cfg: OracleConfig, params, client_adapters: Sequence[dict], dS_list, caches, cuts):
    """Step a5 with per-client depth."""
    all_grads = []
    for i, dx in enumerate(dS_list):
        grads = {}
        for l in range(cuts[i] - 1, -1, -1):
            dx, g = block_bwd(cfg, params, l, client_adapters[i], dx, caches[i][l])
            grads.update(g)
        all_grads.append(grads)
    return all_grads


def aggregate_clients_cuts(state: OracleState, counts, cuts, store_fp32: bool = True):
    """Stage b with per-client depth: Eq. 8-9 per block over the clients that hold the block."""
    for l in range(max(cuts)):
        holders = [i for i in range(len(cuts)) if cuts[i] > l]
        for key in [k for k in state.client_adapters[holders[0]].keys() if k[0] == l]:
            for name in ("A", "B"):
                avg = aggregate([state.client_adapters[i][key][name] for i in holders], [counts[i] for i in holders])
                if store_fp32:
                    avg = avg.astype(np.float32).astype(F64)
                for i in holders:
                    state.client_adapters[i][key][name] = avg.copy()


def split_round_cuts(cfg: OracleConfig, params, state: OracleState, tokens, labels, counts, cuts):
    """One iteration t of Algorithm 1 with client i cut after block cuts[i] (see the reading above).
    state.client_adapters[i] holds blocks 0..cuts[i]-1, state.server_adapters blocks min(cuts)..L-1."""
    state.round_index += 1
    S_list, caches = client_fwd_cuts(cfg, params, state.client_adapters, tokens, cuts)
    loss, dS_list, sgrads = server_fwd_bwd_cuts(cfg, params, state.server_adapters, S_list, labels, cuts)
    state.server_steps += 1
    apply_update(cfg, state.server_adapters, state.server_opt, sgrads, cfg.lr_server, state.server_steps)
    cgrads = client_bwd_grads_cuts(cfg, params, state.client_adapters, dS_list, caches, cuts)
    state.client_steps += 1
    for i, g in enumerate(cgrads):
        apply_update(cfg, state.client_adapters[i], state.client_opt[i], g, cfg.lr_client, state.client_steps)
    aggregated = False
    if state.round_index % cfg.agg_interval == 0:
        aggregate_clients_cuts(state, counts, cuts)
        aggregated = True
    return loss, dict(S=S_list, dS=dS_list, server_grads=sgrads, client_grads=cgrads, aggregated=aggregated)


def trainable_parameter_count(cfg: OracleConfig, n_blocks: int) -> int:
    """Number of LoRA parameters on n_blocks blocks: per block and target r*d (A) + d*r (B)."""
    return n_blocks * len(cfg.targets) * 2 * cfg.lora_r * cfg.d_model
