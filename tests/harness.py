"""Shared helpers of the GPU parity tests: run the oracle and the CUDA library on the same seeded
inputs and compare."""
import numpy as np
import torch

from oracle import splitlora_oracle as O
from paper_2407_00952_b200 import binding as B
from paper_2407_00952_b200 import runner, synth


def oracle_config(w, optimizer="adamw", **kw):
    d = dict(n_layer=w.n_layer, cut=w.cut, d_model=w.d_model, n_head=w.n_head, d_ff=w.d_ff, vocab=w.vocab,
             max_seq=w.max_seq, lora_r=w.lora_r, lora_alpha=w.lora_alpha, targets=w.targets,
             n_clients=w.n_clients, batch_per_client=w.batch_per_client, seq=w.seq,
             bf16_handoff=(w.dtype == "bf16"), optimizer=optimizer, lr_client=w.lr, lr_server=w.lr,
             agg_interval=w.agg_interval, arch=w.arch, rope_theta=w.rope_theta)
    d.update(kw)
    return O.OracleConfig(**d)


def f64(d):
    return {k: v.astype(np.float64) for k, v in d.items()}


def ads64(a):
    return {k: {"A": v["A"].astype(np.float64), "B": v["B"].astype(np.float64)} for k, v in a.items()}


def rel_err(got, ref):
    """Normwise error of a tensor: max |got - ref| / max |ref|."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = np.abs(ref).max()
    return float(np.abs(got - ref).max() / (den if den > 0 else 1.0))


def tnp(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def build_case(w, nonzero_b=True, distinct_clients=True, randomize_affine=True):
    frozen = synth.make_frozen(w, randomize_affine=randomize_affine)
    cads = [synth.make_adapters(w, range(w.cut), nonzero_b=nonzero_b, salt=(i + 1 if distinct_clients else 0))
            for i in range(w.n_clients)]
    sads = synth.make_adapters(w, range(w.cut, w.n_layer), nonzero_b=nonzero_b, salt=77)
    tokens, labels = synth.make_tokens(w)
    return frozen, cads, sads, tokens, labels


def run_three_calls(w, frozen, cads, sads, tokens, labels, optimizer="sgd", use_tensor_cores=True, **over):
    """client_fwd / server_step / client_bwd on the GPU.  Returns engine, S, dS, loss."""
    eng = runner.make_engine(w, frozen, cads, sads, optimizer=optimizer, use_tensor_cores=use_tensor_cores, **over)
    tok = torch.from_numpy(tokens).cuda()
    lab = torch.from_numpy(labels).cuda()
    S = eng.new_activation_buffer()
    dS = eng.new_activation_buffer()
    eng.client_fwd(tok, S)
    loss = eng.server_step(S, lab, dS)
    eng.client_bwd(dS)
    torch.cuda.synchronize()
    assert eng.device_status() == 0
    return eng, S, dS, loss


def oracle_three_calls(w, frozen, cads, sads, tokens, labels, optimizer="sgd", **kw):
    cfg = oracle_config(w, optimizer=optimizer, **kw)
    params = f64(frozen)
    c64 = [ads64(a) for a in cads]
    s64 = ads64(sads)
    S, caches = O.client_fwd(cfg, params, c64, tokens)
    loss, dS, sg = O.server_fwd_bwd(cfg, params, s64, S, labels)
    cg = O.client_bwd_grads(cfg, params, c64, dS, caches)
    return cfg, params, c64, s64, S, dS, loss, sg, cg


# ---- parity cases whose q / k adapter gradients are looser than the general bf16 bound --------------
# The three bf16 cases below have random labels and random non-zero B, and their q / k adapter gradients
# come out of the attention backward, whose row term sum_j P_ij dP_ij is taken from the STORED (bf16)
# attention output.  tests/test_storage_noise.py computes, on the CPU, what bf16 storage alone does to
# these gradients in otherwise exact arithmetic, and fixes the rule: a case keeps the general 2e-2 when
# that noise, with a margin of 1.4 for a different rounding realisation, stays inside it; otherwise its
# q / k bound is QK_BOUND, which must cover the noise with the same margin.
TOL_BF16 = 2e-2
QK_BOUND = 4e-2
NOISE_MARGIN = 1.4


CUTS_MEDIUM = (1, 3, 3)       # per-client cut depths of the "cuts_medium" case


def qk_case(name):
    """(workload, per-client ranks or None, bound for the q / k adapter gradients or None for the general one)"""
    if name == "cuts_medium":
        return (synth.scaled(synth.WORKLOADS[3], n_layer=4, cut=3, n_clients=3, batch_per_client=2, seq=128,
                             max_seq=128), None, QK_BOUND)
    if name == "federated_small":
        return (synth.scaled(synth.WORKLOADS[2], n_layer=2, cut=2, n_clients=2, batch_per_client=2, seq=256,
                             max_seq=256), None, QK_BOUND)
    if name == "llama_full_width":
        return (synth.scaled(synth.WORKLOADS[5], n_layer=2, cut=1, vocab=4096, n_clients=2, batch_per_client=1,
                             seq=256, max_seq=256), None, QK_BOUND)
    if name == "ranks_medium":
        return (synth.scaled(synth.WORKLOADS[3], n_layer=3, cut=2, n_clients=3, batch_per_client=2, seq=128,
                             max_seq=128), (2, 4, 1), None)
    raise KeyError(name)


def cut_to_rank(ad, r):
    return {k: {"A": v["A"][:r].copy(), "B": v["B"][:, :r].copy()} for k, v in ad.items()}
