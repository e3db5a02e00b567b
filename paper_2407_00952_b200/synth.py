"""Seeded synthetic inputs for the split-LoRA round.

This module only draws random numbers and names shapes.  It contains none of the
method's arithmetic and is the one piece that both the CPU checker and the CUDA
harness may use, so that both sides see bit-identical inputs.

The workloads stand in for the paper's setting (pre-trained GPT-2 small/medium
fine-tuned on E2E with sequence length 512 and the first blocks on the clients,
Sec. IV-A), for which neither weights nor data are available: frozen weights and
embeddings ~ N(0, 0.02), adapter A ~ N(0, 0.02), adapter B = 0, the same initial
adapters on every client (Algorithm 1, initialisation), token ids from a bounded
Zipf law, client sample counts uniform in [200, 1000].
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np


@dataclass(frozen=True)
class Workload:
    """Shape and hyper-parameters of one benchmark configuration."""
    index: int
    name: str
    n_layer: int
    cut: int
    d_model: int
    n_head: int
    d_ff: int
    vocab: int
    max_seq: int
    lora_r: int
    lora_alpha: float
    targets: Tuple[str, ...]
    n_clients: int
    batch_per_client: int
    seq: int
    dtype: str            # "fp32" or "bf16"
    lr: float
    zipf: bool
    counts: Optional[Tuple[int, ...]] = None   # fixed sample counts, else drawn in [200, 1000]
    rounds: int = 1
    agg_interval: int = 1
    arch: str = "gpt"     # "gpt": LayerNorm / learned positions / GELU / biases / tied head;
                          # "llama": RMSNorm / rotary q,k / SwiGLU / no biases / separate head
    rope_theta: float = 10000.0

    @property
    def tokens_per_round(self) -> int:
        return self.n_clients * self.batch_per_client * self.seq


WORKLOADS: Dict[int, Workload] = {
    1: Workload(1, "tiny-split-gpt", 2, 1, 128, 4, 512, 1024, 64, 4, 8.0, ("q", "v"),
                2, 4, 64, "fp32", 1e-3, False, (3, 5), 1),
    2: Workload(2, "gpt2-small-shaped", 12, 3, 768, 12, 3072, 50257, 512, 4, 32.0, ("q", "v"),
                4, 8, 512, "bf16", 2e-4, True, None, 10),
    3: Workload(3, "gpt2-medium-shaped", 24, 6, 1024, 16, 4096, 50257, 512, 4, 32.0, ("q", "v"),
                8, 8, 512, "bf16", 2e-4, True, None, 10),
    5: Workload(5, "llama2-7b-shaped", 32, 4, 4096, 32, 11008, 32000, 1024, 16, 32.0, ("q", "k", "v", "o"),
                4, 2, 1024, "bf16", 2e-4, True, None, 1, arch="llama"),
}


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (reduced depth, fewer clients, ...)."""
    d = dict(w.__dict__)
    d.update(kw)
    return Workload(**d)


def _to_bf16_values(a: np.ndarray) -> np.ndarray:
    """fp32 array whose values are exactly representable in bfloat16 (round to nearest even)."""
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16).to(torch.float32).numpy()


def frozen_param_names(w: Workload) -> List[Tuple[str, Tuple[int, ...], str]]:
    """(name, shape, kind) of every frozen tensor, in the order that fixes the seeds."""
    d, F, V = w.d_model, w.d_ff, w.vocab
    if w.arch == "llama":
        out = [("wte", (V, d), "w"), ("head.w", (V, d), "w")]
        for l in range(w.n_layer):
            p = f"h.{l}."
            out += [
                (p + "ln1.g", (d,), "gain"), (p + "attn.qkv.w", (3 * d, d), "w"),
                (p + "attn.proj.w", (d, d), "w"), (p + "ln2.g", (d,), "gain"),
                (p + "mlp.gate.w", (F, d), "w"), (p + "mlp.up.w", (F, d), "w"),
                (p + "mlp.down.w", (d, F), "w"),
            ]
        return out + [("lnf.g", (d,), "gain")]
    out = [("wte", (V, d), "w"), ("wpe", (w.max_seq, d), "w")]
    for l in range(w.n_layer):
        p = f"h.{l}."
        out += [
            (p + "ln1.g", (d,), "gain"), (p + "ln1.b", (d,), "bias"),
            (p + "attn.qkv.w", (3 * d, d), "w"), (p + "attn.qkv.b", (3 * d,), "bias"),
            (p + "attn.proj.w", (d, d), "w"), (p + "attn.proj.b", (d,), "bias"),
            (p + "ln2.g", (d,), "gain"), (p + "ln2.b", (d,), "bias"),
            (p + "mlp.fc1.w", (F, d), "w"), (p + "mlp.fc1.b", (F,), "bias"),
            (p + "mlp.fc2.w", (d, F), "w"), (p + "mlp.fc2.b", (d,), "bias"),
        ]
    out += [("lnf.g", (d,), "gain"), ("lnf.b", (d,), "bias")]
    return out


def make_frozen(w: Workload, randomize_affine: bool = False) -> Dict[str, np.ndarray]:
    """Frozen weights as fp32 arrays (bf16-exact values in bf16 workloads).

    Weights ~ N(0, 0.02); biases 0 and LayerNorm gain 1 / bias 0 unless `randomize_affine`,
    which draws them (used by tests so that no term is hidden by a zero).
    """
    return dict(iter_frozen(w, randomize_affine))


def iter_frozen(w: Workload, randomize_affine: bool = False):
    """The tensors of make_frozen one at a time, as (name, array): a workload whose weights do not
    fit in host memory at once (13.5 GB in bf16 for the Llama-2-7B shape) is uploaded as it is drawn."""
    for idx, (name, shape, kind) in enumerate(frozen_param_names(w)):
        rng = np.random.default_rng(1234 + 1000 * w.index + idx)
        if kind == "w":
            a = rng.normal(0.0, 0.02, size=shape).astype(np.float32)
        elif kind == "gain":
            a = (1.0 + 0.1 * rng.normal(size=shape)).astype(np.float32) if randomize_affine \
                else np.ones(shape, np.float32)
        else:
            a = (0.05 * rng.normal(size=shape)).astype(np.float32) if randomize_affine \
                else np.zeros(shape, np.float32)
        if w.dtype == "bf16":
            a = _to_bf16_values(a)
        yield name, a


def make_adapters(w: Workload, layers, nonzero_b: bool = False, salt: int = 0):
    """{(layer, target): {"A": [r, d], "B": [d, r]}} fp32; A ~ N(0, 0.02), B = 0 (or drawn)."""
    ads = {}
    for l in layers:
        for ti, t in enumerate(w.targets):
            rng = np.random.default_rng(1234 + 1000 * w.index + 500 + 8 * l + ti + 100000 * salt)
            A = rng.normal(0.0, 0.02, size=(w.lora_r, w.d_model)).astype(np.float32)
            B = (rng.normal(0.0, 0.02, size=(w.d_model, w.lora_r)).astype(np.float32)
                 if nonzero_b else np.zeros((w.d_model, w.lora_r), np.float32))
            ads[(l, t)] = {"A": A, "B": B}
    return ads


def make_tokens(w: Workload, round_index: int = 0):
    """tokens, labels [K, b, T] int32: T+1 ids per sequence, labels are the next ids."""
    K, b, T, V = w.n_clients, w.batch_per_client, w.seq, w.vocab
    rng = np.random.default_rng(1234 + 1000 * w.index + 900 + round_index)
    if w.zipf:
        ranks = np.arange(1, V + 1, dtype=np.float64)
        p = ranks ** -1.1
        p /= p.sum()
        perm = np.random.default_rng(1234 + 1000 * w.index + 899).permutation(V)
        draw = rng.choice(V, size=(K, b, T + 1), p=p)
        ids = perm[draw]
    else:
        ids = rng.integers(0, V, size=(K, b, T + 1))
    ids = ids.astype(np.int32)
    return np.ascontiguousarray(ids[..., :T]), np.ascontiguousarray(ids[..., 1:])


def make_counts(w: Workload) -> np.ndarray:
    """|D_i| per client (int64)."""
    if w.counts is not None:
        return np.asarray(w.counts, dtype=np.int64)
    rng = np.random.default_rng(1234 + 1000 * w.index + 898)
    return rng.integers(200, 1001, size=w.n_clients).astype(np.int64)


def make_lora_linear_case(M: int, n_in: int, n_out: int, r: int, G: int, seed: int = 0):
    """Micro-benchmark operands: x [M,in], W [out,in], A [G,r,in], B [G,out,r], dy [M,out],
    all N(0,1)/sqrt(fan_in), bf16-exact fp32 values; G equal contiguous row segments."""
    rng = np.random.default_rng(77000 + seed)
    x = _to_bf16_values(rng.normal(size=(M, n_in)).astype(np.float32))
    W = _to_bf16_values((rng.normal(size=(n_out, n_in)) / np.sqrt(n_in)).astype(np.float32))
    A = _to_bf16_values((rng.normal(size=(G, r, n_in)) / np.sqrt(n_in)).astype(np.float32))
    B = _to_bf16_values((rng.normal(size=(G, n_out, r)) / np.sqrt(r)).astype(np.float32))
    dy = _to_bf16_values((rng.normal(size=(M, n_out)) / np.sqrt(n_out)).astype(np.float32))
    return x, W, A, B, dy
