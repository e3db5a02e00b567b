"""Operator micro-benchmarks through the C ABI: the grouped LoRA linear layer (forward / backward),
the Eq. 8-9 aggregation and causal attention.  Prints one JSON line per case.

  python -m paper_2407_00952_b200.microbench linear --M 32768 --n-in 1024 --n-out 3072 --r 4 --G 8
  python -m paper_2407_00952_b200.microbench linear-sweep [--quick] > sweep.jsonl
  python -m paper_2407_00952_b200.microbench linear-sweep-table --file sweep.jsonl
  python -m paper_2407_00952_b200.microbench aggregate-sweep
  python -m paper_2407_00952_b200.microbench attention --nseq 64 --T 512 --heads 16

Timing: CUDA events on the launching stream, warm-up first; operands are rotated over several
buffer sets when one set would fit in L2.
"""
from __future__ import annotations

import argparse
import json
import os

import torch

from . import binding as B

L2_BYTES = 126 * 2 ** 20


def _peaks():
    path = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return p["hbm_gbs"], p["bf16_tflops"], "measured"
    return 6650.0, 1590.0, "fallback"


def _time(fn, iters, warmup=3):
    for _ in range(warmup):
        fn(0)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(iters):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def _time_graph(fn, iters, warmup=2):
    """Like _time, with the `iters` calls captured in a CUDA graph and replayed: an operator call is half a
    dozen launches from Python, which at small shapes takes the host longer to issue than the device to
    run.  `fn` must allocate nothing."""
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(iters):
            fn(i)
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def bench_linear_shape(M, n_in, n_out, rs, Gs, iters=10, backward=True, tc=True):
    """One (M, in, out) shape of the grouped LoRA linear for every rank in rs and group count in Gs.
    Forward, and the backward in its parts: the rank-r projections, dx, and dA + dB, each timed by itself
    (splitlora_lora_linear_bwd_parts).  Operands rotate over several buffer sets unless one set exceeds
    twice the L2, so every launch reads from HBM.  Yields one dict per (r, G)."""
    hbm, tflops, src = _peaks()
    set_bytes = 2 * (M * n_in + M * n_out + n_in * n_out)
    nset = max(1, min(4, -(-2 * L2_BYTES // set_bytes)))
    g = torch.Generator(device="cuda").manual_seed(1)
    mk = lambda *s, sc=1.0: (torch.randn(*s, device="cuda", generator=g) * sc).bfloat16()
    xs = [mk(M, n_in) for _ in range(nset)]
    dys = [mk(M, n_out, sc=n_out ** -0.5) for _ in range(nset)]
    ys = [torch.empty(M, n_out, device="cuda", dtype=torch.bfloat16) for _ in range(nset)]
    dxs = [torch.empty(M, n_in, device="cuda", dtype=torch.bfloat16) for _ in range(nset)]
    W = mk(n_out, n_in, sc=n_in ** -0.5)
    Wt = B.transpose(W)
    for r in rs:
        for G in Gs:
            if M % G or (G > 1 and (M // G) % 128):
                continue
            A = torch.randn(G, r, n_in, device="cuda", generator=g) * n_in ** -0.5
            Bm = torch.randn(G, n_out, r, device="cuda", generator=g) * r ** -0.5
            ws = B.lora_linear_workspace(B.DTYPE_BF16, M, n_in, n_out, r, G)
            runf = lambda parts: _time_graph(lambda i: B.lora_linear_fwd(xs[i % nset], W, None, A, Bm, 16.0, y=ys[i % nset],
                                                                         workspace=ws, use_tensor_cores=tc, parts=parts), iters)
            f_down = runf(1)                          # compute copies of the adapters and h = x A^T: skinny, HBM-bound
            fwd = runf(3) - f_down                    # y = x W^T + (alpha/r) h B^T on the tensor cores
            flops = 2.0 * M * n_in * n_out + 2.0 * M * r * n_out
            out = {"op": "lora_linear", "M": M, "n_in": n_in, "n_out": n_out, "r": r, "G": G, "buffer_sets": nset,
                   "fwd_down_us": round(f_down * 1e3, 1), "fwd_down_frac_of_hbm": round(2.0 * M * n_in / f_down / 1e6 / hbm, 3),
                   "fwd_us": round(fwd * 1e3, 1), "fwd_tflops": round(flops / fwd / 1e9, 1),
                   "fwd_frac_of_bf16_peak": round(flops / fwd / 1e9 / tflops, 3), "peak_source": src + " burst"}
            if backward:
                dA = torch.empty(G, r, n_in, dtype=torch.float32, device="cuda")
                dB = torch.empty(G, n_out, r, dtype=torch.float32, device="cuda")
                run = lambda parts: _time_graph(lambda i: B.lora_linear_bwd(xs[i % nset], Wt, dys[i % nset], A, Bm, 16.0,
                                                                            workspace=ws, use_tensor_cores=tc, parts=parts,
                                                                            out=(dxs[i % nset], dA, dB)), iters)
                t_down = run(1)                       # h = x A^T and dh = s dy B: skinny, HBM-bound
                t_dx = run(1 | 2) - t_down            # dx = dy W + dh A on the tensor cores
                t_g = run(1 | 4) - t_down             # dA = dh^T x, dB = s dy^T h: skinny reductions over the tokens
                dx_flops = 2.0 * M * n_in * n_out + 2.0 * M * r * n_in
                down_bytes = 2.0 * M * (n_in + n_out)               # x and dy read once
                g_bytes = 2.0 * M * (n_in + n_out)                  # x and dy read once more
                out.update({"down_us": round(t_down * 1e3, 1), "down_GBps": round(down_bytes / t_down / 1e6, 1),
                            "down_frac_of_hbm": round(down_bytes / t_down / 1e6 / hbm, 3),
                            "dx_us": round(t_dx * 1e3, 1), "dx_tflops": round(dx_flops / t_dx / 1e9, 1),
                            "dx_frac_of_bf16_peak": round(dx_flops / t_dx / 1e9 / tflops, 3),
                            "dAdB_us": round(t_g * 1e3, 1), "dAdB_GBps": round(g_bytes / t_g / 1e6, 1),
                            "dAdB_frac_of_hbm": round(g_bytes / t_g / 1e6 / hbm, 3)})
            yield out


def bench_linear(M, n_in, n_out, r, G, iters=20, backward=True, tc=True):
    return next(bench_linear_shape(M, n_in, n_out, [r], [G], iters, backward, tc))


def bench_epilogues(M, d, F, iters=20):
    """The un-adapted linear layers of one block (forward and backward), each with its epilogue."""
    _, tflops, src = _peaks()
    g = torch.Generator(device="cuda").manual_seed(2)
    mk = lambda *s, sc=1.0: (torch.randn(*s, device="cuda", generator=g) * sc).bfloat16()
    xd, xF = mk(M, d), mk(M, F)
    rd, rF = mk(M, d), mk(M, F)
    yd, yF, zF = (torch.empty(M, d, device="cuda", dtype=torch.bfloat16), torch.empty(M, F, device="cuda", dtype=torch.bfloat16),
                  torch.empty(M, F, device="cuda", dtype=torch.bfloat16))
    Wdd, WFd, WdF = mk(d, d, sc=d ** -0.5), mk(F, d, sc=d ** -0.5), mk(d, F, sc=F ** -0.5)
    bd, bF = mk(d), mk(F)
    cases = [
        ("proj fwd  (bias+resid)", lambda i: B.linear(xd, Wdd, bd, B.EPI_BIAS_RESID, r=rd, y=yd), d, d),
        ("fc1 fwd   (bias+gelu)", lambda i: B.linear(xd, WFd, bF, B.EPI_BIAS_GELU, y=yF, z=zF), d, F),
        ("fc2 fwd   (bias+resid)", lambda i: B.linear(xF, WdF, bd, B.EPI_BIAS_RESID, r=rd, y=yd), F, d),
        ("fc2 bwd   (x gelu')", lambda i: B.linear(xd, WFd, None, B.EPI_MUL_GELUGRAD, r=rF, y=yF), d, F),
        ("fc1 bwd   (plain)", lambda i: B.linear(xF, WdF, None, B.EPI_BIAS, y=yd), F, d),
        ("proj bwd  (plain)", lambda i: B.linear(xd, Wdd, None, B.EPI_BIAS, y=yd), d, d),
    ]
    out = []
    for name, fn, k, n in cases:
        ms = _time(fn, iters)
        fl = 2.0 * M * k * n
        out.append({"op": "linear", "case": name, "M": M, "K": k, "N": n, "us": round(ms * 1e3, 1),
                    "tflops": round(fl / ms / 1e9, 1), "frac_of_bf16_peak": round(fl / ms / 1e9 / tflops, 3),
                    "peak_source": src + " burst"})
    return out


def bench_aggregate(K, P, iters=50):
    hbm, _, src = _peaks()
    nset = max(1, min(8, -(-2 * L2_BYTES // (K * P * 4))))
    bufs = [torch.randn(K, P, device="cuda") for _ in range(nset)]
    w = [1.0 / K] * K
    ms = _time(lambda i: B.aggregate_buffers(bufs[i % nset], w), iters)
    gbs = 2.0 * K * P * 4 / ms / 1e6        # read K copies, write K copies
    return {"op": "aggregate", "K": K, "P": P, "us": round(ms * 1e3, 2), "GBps": round(gbs, 1),
            "frac_of_hbm": round(gbs / hbm, 3), "peak_source": src}


def bench_attention(nseq, T, heads, iters=10, head_dim=64):
    _, tflops, src = _peaks()
    d = heads * head_dim
    qkv = torch.randn(nseq * T, 3 * d, device="cuda").bfloat16()
    do = torch.randn(nseq * T, d, device="cuda").bfloat16()
    o, lse = B.attention_fwd(qkv, nseq, T, heads, True)
    f = _time(lambda i: B.attention_fwd(qkv, nseq, T, heads, True), iters)
    b = _time(lambda i: B.attention_bwd(qkv, o, lse, do, nseq, T, heads, True), iters)
    fl = 2.0 * nseq * heads * T * T * head_dim      # causal: half of 4 T^2 dh
    return {"op": "attention", "nseq": nseq, "T": T, "heads": heads, "head_dim": head_dim, "fwd_us": round(f * 1e3, 1),
            "fwd_tflops": round(fl / f / 1e9, 1), "bwd_us": round(b * 1e3, 1),
            "bwd_tflops_algorithmic": round(2.5 * fl / b / 1e9, 1), "peak_source": src}


def bench_split(config: int, cut: int, agg_interval: int, n_clients: int, steps: int):
    """One workload at another split point / aggregation interval / client count: tokens per second of
    whole rounds, the bytes that cross the client-server boundary per round (S and dL/dS, Sec. III-B
    steps a2 and a4, plus labels), the adapter bytes of an aggregation (b1 + b3) and the share of the
    blocks that run on the clients.  cut == n_layer is the federated baseline, n_clients == 1 the
    centralised one (Sec. IV-A)."""
    from . import runner, synth
    w = synth.scaled(synth.WORKLOADS[config], cut=cut, agg_interval=agg_interval, n_clients=n_clients)
    cads = [synth.make_adapters(w, range(w.cut)) for _ in range(w.n_clients)]
    sads = synth.make_adapters(w, range(w.cut, w.n_layer))
    eng = runner.make_engine(w, synth.iter_frozen(w), cads, sads, optimizer="adamw")
    counts = synth.make_counts(w)
    batches = []
    for s in range(2):
        t, l = synth.make_tokens(w, round_index=s)
        batches.append((torch.from_numpy(t).cuda(), torch.from_numpy(l).cuda()))
    ms = _time(lambda i: eng.round(*batches[i % 2], counts, want_loss=False), steps, warmup=3)
    # the same round as its three calls, each timed by itself: what runs on the clients and what on the server
    S, dS = eng.new_activation_buffer(), eng.new_activation_buffer()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    t_client = t_server = 0.0
    for i in range(steps):
        ev[0].record(); eng.client_fwd(batches[i % 2][0], S)
        ev[1].record(); eng.server_step(S, batches[i % 2][1], dS, want_loss=False)
        ev[2].record(); eng.client_bwd(dS)
        ev[3].record(); torch.cuda.synchronize()
        t_client += ev[0].elapsed_time(ev[1]) + ev[2].elapsed_time(ev[3])
        t_server += ev[1].elapsed_time(ev[2])
    assert eng.device_status() == 0
    M, es = w.tokens_per_round, 2 if w.dtype == "bf16" else 4
    per_client = w.cut * len(w.targets) * 2 * w.lora_r * w.d_model * 4
    # algorithmic FLOPs per round (forward + backward without dW): a block's linear layers and its causal
    # attention (forward 2 T d per token, backward 2.5 x that), the head on the server
    d, F, T = w.d_model, w.d_ff, w.seq
    mlp = (6.0 if w.arch == "llama" else 4.0) * d * F
    block = M * (2.0 * (8.0 * d * d + mlp) + 3.5 * 2.0 * T * d)
    head = 2.0 * 2.0 * M * d * w.vocab
    return {"op": "split_round", "config": config, "cut": cut, "n_layer": w.n_layer, "I": agg_interval,
            "K": w.n_clients, "tokens_per_round": M, "ms_per_round": round(ms, 3),
            "tokens_per_s": round(M / ms * 1e3, 1), "client_block_share": round(w.cut / w.n_layer, 4),
            "client_flop_share": round(cut * block / (w.n_layer * block + head), 4),
            "client_time_share": round(t_client / (t_client + t_server), 4),
            "client_ms": round(t_client / steps, 3), "server_ms": round(t_server / steps, 3),
            "handoff_bytes_per_round": 2 * M * w.d_model * es + M * 4,
            "aggregation_bytes_per_client": 2 * per_client, "aggregations_per_round": round(1.0 / agg_interval, 3)}


def bench_handoff(config: int, steps: int):
    """Compressed cut-layer hand-off (E4M3 codes + one scale per token): the two codec kernels against
    the HBM roofline on the workload's [M, d] hand-off tensor (algorithmic bytes: the tensor once in,
    the codes once out, and the reverse), and whole rounds with and without compression with the bytes
    that cross the cut per round."""
    from . import runner, synth
    hbm, _, src = _peaks()
    w = synth.WORKLOADS[config]
    M, d = w.tokens_per_round, w.d_model
    es = 2 if w.dtype == "bf16" else 4
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    nset = max(2, -(-2 * L2_BYTES // (M * d * es)))           # rotate buffers so that nothing stays in L2
    xs = [(torch.randn(M, d, device="cuda") * torch.exp(torch.randn(M, 1, device="cuda"))).to(dt) for _ in range(nset)]
    cs = [torch.empty(M, d, dtype=torch.uint8, device="cuda") for _ in range(nset)]
    sc = torch.empty(M, dtype=torch.float32, device="cuda")
    q = _time(lambda i: B.handoff_quantize(xs[i % nset], cs[i % nset], sc), 20)
    dq = _time(lambda i: B.handoff_dequantize(cs[i % nset], sc, xs[i % nset]), 20)
    by = M * d * (es + 1) + M * 4
    rows = [{"op": "handoff_quantize", "M": M, "d": d, "us": round(q * 1e3, 1), "GBps": round(by / q / 1e6, 1),
             "frac_of_hbm": round(by / q / 1e6 / hbm, 3), "peak_source": src},
            {"op": "handoff_dequantize", "M": M, "d": d, "us": round(dq * 1e3, 1), "GBps": round(by / dq / 1e6, 1),
             "frac_of_hbm": round(by / dq / 1e6 / hbm, 3), "peak_source": src}]
    del xs, cs
    cads = [synth.make_adapters(w, range(w.cut)) for _ in range(w.n_clients)]
    sads = synth.make_adapters(w, range(w.cut, w.n_layer))
    eng = runner.make_engine(w, synth.iter_frozen(w), cads, sads, optimizer="adamw")
    counts = synth.make_counts(w)
    batches = []
    for s in range(2):
        t, l = synth.make_tokens(w, round_index=s)
        batches.append((torch.from_numpy(t).cuda(), torch.from_numpy(l).cuda()))
    codes = torch.empty(2, M, d, dtype=torch.uint8, device="cuda")
    scales = torch.empty(2, M, dtype=torch.float32, device="cuda")
    plain = _time(lambda i: eng.round(*batches[i % 2], counts, want_loss=False), steps)
    comp = _time(lambda i: eng.round_compressed(*batches[i % 2], counts, codes, scales, want_loss=False), steps)
    assert eng.device_status() == 0
    rows.append({"op": "round", "config": config, "handoff": "native", "ms_per_round": round(plain, 3),
                 "tokens_per_s": round(M / plain * 1e3, 1), "handoff_bytes_per_round": 2 * M * d * es + M * 4})
    rows.append({"op": "round", "config": config, "handoff": "e4m3 + scale per token", "ms_per_round": round(comp, 3),
                 "tokens_per_s": round(M / comp * 1e3, 1), "handoff_bytes_per_round": 2 * (M * d + M * 4) + M * 4})
    return rows


def bench_ranks(config: int, steps: int):
    """Per-client adapter ranks (zero-padded storage): whole rounds with one rank for all and with a
    mix of ranks, and the aggregation step (weighted mean + write-back, plus the rank mask) alone."""
    from . import runner, synth
    w = synth.WORKLOADS[config]
    cads = [synth.make_adapters(w, range(w.cut), nonzero_b=True, salt=i + 1) for i in range(w.n_clients)]
    sads = synth.make_adapters(w, range(w.cut, w.n_layer))
    eng = runner.make_engine(w, synth.iter_frozen(w), cads, sads, optimizer="adamw")
    counts = synth.make_counts(w)
    batches = []
    for s in range(2):
        t, l = synth.make_tokens(w, round_index=s)
        batches.append((torch.from_numpy(t).cuda(), torch.from_numpy(l).cuda()))
    M = w.tokens_per_round
    rows = []
    mix = [max(1, w.lora_r >> (i % 3)) for i in range(w.n_clients)]
    for name, ranks in (("one rank", None), ("mixed ranks", mix), ("one rank, measured again", None)):
        eng.set_client_ranks(ranks)
        ms = _time(lambda i: eng.round(*batches[i % 2], counts, want_loss=False), steps)
        agg = _time(lambda i: eng.aggregate(counts), 50)
        rows.append({"op": "round", "config": config, "ranks": name, "client_ranks": ranks or [w.lora_r] * w.n_clients,
                     "ms_per_round": round(ms, 3), "tokens_per_s": round(M / ms * 1e3, 1),
                     "aggregate_us": round(agg * 1e3, 2)})
    assert eng.device_status() == 0
    return rows


def sweep_table(path):
    """Markdown summary of a linear-sweep output file (one JSON line per case): per (M, in, out) shape the
    range over ranks and group counts, and one shape in full."""
    rows = [json.loads(l) for l in open(path) if l.strip().startswith("{")]
    shapes = {}
    for r in rows:
        shapes.setdefault((r["M"], r["n_in"], r["n_out"]), []).append(r)
    rng = lambda rs, k, f=1.0: f"{min(x[k] for x in rs) * f:.0f}-{max(x[k] for x in rs) * f:.0f}"
    out = ["| M | in | out | fwd TF/s | fwd % of burst | dx TF/s | dx % of burst | rank-r projections % of HBM (fwd / bwd) | dA + dB % of HBM |",
           "|---|---|---|---|---|---|---|---|---|"]
    for (M, i, o), rs in sorted(shapes.items()):
        out.append(f"| {M} | {i} | {o} | {rng(rs, 'fwd_tflops')} | {rng(rs, 'fwd_frac_of_bf16_peak', 100)} | "
                   f"{rng(rs, 'dx_tflops')} | {rng(rs, 'dx_frac_of_bf16_peak', 100)} | "
                   f"{rng(rs, 'fwd_down_frac_of_hbm', 100)} / {rng(rs, 'down_frac_of_hbm', 100)} | {rng(rs, 'dAdB_frac_of_hbm', 100)} |")
    out += ["", "One shape in full (M 16384, 1024 -> 3072):", "",
            "| r | G | fwd us | fwd TF/s | dx us | dx TF/s | rank-r fwd us | rank-r bwd us | dA + dB us | dA + dB GB/s |", "|---|---|---|---|---|---|---|---|---|---|"]
    for r in sorted(shapes.get((16384, 1024, 3072), []), key=lambda x: (x["r"], x["G"])):
        out.append(f"| {r['r']} | {r['G']} | {r['fwd_us']} | {r['fwd_tflops']} | {r['dx_us']} | {r['dx_tflops']} | {r['fwd_down_us']} | "
                   f"{r['down_us']} | {r['dAdB_us']} | {r['dAdB_GBps']} |")
    return "\n".join(out)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("what", choices=["linear", "linear-sweep", "linear-sweep-table", "epilogues", "aggregate", "aggregate-sweep",
                                     "attention", "split-sweep", "handoff", "ranks"])
    ap.add_argument("--file", default="", help="linear-sweep-table: the sweep's output file")
    ap.add_argument("--config", type=int, default=3)
    ap.add_argument("--M", type=int, default=32768)
    ap.add_argument("--n-in", type=int, default=1024)
    ap.add_argument("--n-out", type=int, default=3072)
    ap.add_argument("--r", type=int, default=4)
    ap.add_argument("--G", type=int, default=8)
    ap.add_argument("--K", type=int, default=8)
    ap.add_argument("--P", type=int, default=98304)
    ap.add_argument("--nseq", type=int, default=64)
    ap.add_argument("--T", type=int, default=512)
    ap.add_argument("--heads", type=int, default=16)
    ap.add_argument("--head-dim", type=int, default=64)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--no-backward", action="store_true")
    ap.add_argument("--quick", action="store_true")
    a = ap.parse_args()
    if a.what == "linear-sweep-table":
        print(sweep_table(a.file))
        return
    if a.what == "linear":
        print(json.dumps(bench_linear(a.M, a.n_in, a.n_out, a.r, a.G, a.iters, not a.no_backward)))
    elif a.what == "linear-sweep":
        Ms = [4096, 16384, 65536]
        ins = [768, 1024, 4096]
        outs = [768, 3072, 4096, 11008]
        rs = [4, 8, 16, 64]
        Gs = [1, 4, 8, 16]
        if a.quick:
            Ms, rs, Gs = [16384], [4, 64], [1, 8]
        for M in Ms:
            for n_in in ins:
                for n_out in outs:
                    for row in bench_linear_shape(M, n_in, n_out, rs, Gs, a.iters if a.iters < 20 else 8):
                        print(json.dumps(row), flush=True)
                    torch.cuda.empty_cache()
    elif a.what == "epilogues":
        for row in bench_epilogues(a.M, a.n_in, 4 * a.n_in, a.iters):
            print(json.dumps(row), flush=True)
    elif a.what == "aggregate":
        print(json.dumps(bench_aggregate(a.K, a.P, a.iters)))
    elif a.what == "aggregate-sweep":
        for K in (2, 8, 32):
            for lg in range(17, 27 if K == 32 else 29, 2):
                print(json.dumps(bench_aggregate(K, 1 << lg)), flush=True)
        print(json.dumps(dict(bench_aggregate(8, 98304), note="GPT-2-medium-shaped client adapter set")))
    elif a.what == "ranks":
        for row in bench_ranks(a.config, 5):
            print(json.dumps(row), flush=True)
    elif a.what == "handoff":
        for row in bench_handoff(a.config, 5):
            print(json.dumps(row), flush=True)
    elif a.what == "split-sweep":
        from . import synth
        w = synth.WORKLOADS[a.config]
        L = w.n_layer
        cuts = sorted({1, w.cut, L // 4, L // 2, L})
        for cut in cuts:                                   # split point, the paper's aggregation interval I
            for I in (1, 10):
                print(json.dumps(bench_split(a.config, cut, I, w.n_clients, 5)), flush=True)
        print(json.dumps(dict(bench_split(a.config, w.cut, 1, 1, 5), note="one client: centralised baseline")), flush=True)
    else:
        print(json.dumps(bench_attention(a.nseq, a.T, a.heads, a.iters, a.head_dim)))


if __name__ == "__main__":
    main()
