#!/usr/bin/env python
"""Benchmark of the split-LoRA round: training tokens/s on the GPT-2-medium-shaped workload.

  python bench.py --gpus 1 --steps 10 --warmup 3            # the CUDA library
  python bench.py --gpus 4 --scaling strong                 # starts its own 4 ranks (or run it under torchrun)
  python bench.py --impl reference --steps 2 --warmup 1     # the CPU oracle on a bounded sample

A step is one full round of Algorithm 1 (client forward, server step, client backward and the
weighted aggregation) over one batch of synthetic tokens.  Prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2407_00952_b200 import synth  # noqa: E402

METRIC = "split-LoRA training tokens/sec"
UNIT = "tokens/s"


def load_peaks():
    """Measured roofline denominators; falls back to an earlier measurement on the same pool."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], tflops_burst=p["bf16_tflops"], tflops_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, tflops_burst=1590.0, tflops_sustained=1400.0, source="fallback")


def kernel_source_digest():
    """Digest of the sources of the linear-layer kernel, to tell whether counters taken earlier still apply."""
    import hashlib
    h = hashlib.sha256()
    for f in ("gemm_tc.cu", "tc_common.cuh"):
        h.update(open(os.path.join(ROOT, "paper_2407_00952_b200", "csrc", f), "rb").read())
    return h.hexdigest()[:16]


def load_traffic(w):
    """DRAM bytes of one launch of the dominant kernel, from the record written beside its ncu summary
    (profiles/gemm_tc_pair_kernel_traffic.txt: key = value lines).  None when there is no record for this
    workload or when the kernel's sources have changed since the counters were taken."""
    path = os.path.join(ROOT, "profiles", "gemm_tc_pair_kernel_traffic.txt")
    if not os.path.exists(path):
        return None, None
    rec = {}
    for line in open(path):
        if "=" in line and not line.lstrip().startswith("#"):
            k, v = line.split("=", 1)
            rec[k.strip()] = v.strip()
    if rec.get("workload") != f"cfg{w.index}" or rec.get("kernel_source_digest") != kernel_source_digest():
        return None, None
    return int(rec["dram_bytes_per_launch"]), rec.get("launch")


def workload_description(w):
    return {"workload": f"cfg{w.index} {w.name}: L={w.n_layer} cut={w.cut} d={w.d_model} H={w.n_head} F={w.d_ff} "
                        f"V={w.vocab} T={w.seq} r={w.lora_r} alpha={w.lora_alpha:g} targets={''.join(w.targets)} "
                        f"K={w.n_clients} b={w.batch_per_client} I={w.agg_interval} AdamW",
            "tokens_per_step": w.tokens_per_round,
            "l2": "inputs larger than L2 (the activations of one step exceed 126 MB many times over)"}


def gemm_flops_per_round(w):
    """Algorithmic FLOPs of the tensor-core linear layers per round, by launch class (no dW)."""
    M, d, F, V, L = w.tokens_per_round, w.d_model, w.d_ff, w.vocab, w.n_layer
    r = w.lora_r
    nq = len([t for t in w.targets if t != "o"])
    has_o = "o" in w.targets
    mlp = (6.0 if w.arch == "llama" else 4.0) * M * d * F          # gate, up, down / fc1, fc2
    proj = 2.0 * M * d * d + (2.0 * M * r * d if has_o else 0.0)   # output projection (+ its rank-r term)
    qkv = 2.0 * M * d * 3 * d + 2.0 * M * r * d * nq
    return {
        "lora_linear_fwd": L * (qkv + (proj if has_o else 0.0)),
        "linear_fwd": L * (mlp + (0.0 if has_o else proj)),
        "linear_bwd": L * (mlp + (0.0 if has_o else proj)),
        "lora_linear_bwd": (L - 1) * qkv + (L * proj if has_o else 0.0),
        "head_fwd": 2.0 * M * d * V,
        "head_bwd": 2.0 * M * d * V,
    }


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("uuid,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.uuid = uuid
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-lms", "100"], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        self.proc.wait()
        self.tmp.flush()
        rows = [l.strip().split(", ") for l in open(self.tmp.name) if l.strip()]
        os.unlink(self.tmp.name)
        rows = [r for r in rows if len(r) >= 9]
        mine = [r for r in rows if self.uuid and self.uuid in r[0]] or rows
        if not mine:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm = sorted(float(r[1]) for r in mine)
        reasons = set()
        for r in mine:
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if v.strip().lower() == "active":
                    reasons.add(name)
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": float(mine[0][2]), "samples": len(mine),
                "power_w_max": max(float(r[3]) for r in mine), "reasons": sorted(reasons)}


def oracle_sample_workload(w, rounds=1):
    """The bounded sample the CPU oracle is timed on: same model, 2 clients x 1 sequence (1 client when more
    than six rounds are asked for, so that the whole run still ends within a few minutes).  A model whose
    fp64 round would take many minutes even so (width 4096) is cut to one client block and one server
    block on one sequence; time_oracle_rounds scales the time back up to the full depth."""
    if w.d_model >= 2048:
        return synth.scaled(w, n_layer=2, cut=1, n_clients=1, batch_per_client=1, counts=None)
    return synth.scaled(w, n_clients=min(2 if rounds <= 6 else 1, w.n_clients), batch_per_client=1, counts=None)


def time_oracle_rounds(w, steps, warmup):
    """Times oracle rounds (as the oracle stands) on the host cores."""
    from oracle import splitlora_oracle as O
    ws = oracle_sample_workload(w, steps + warmup)
    frozen = synth.make_frozen(ws)          # fp32 arrays holding bf16-exact values; widened on use
    cads = [synth.make_adapters(ws, range(ws.cut)) for _ in range(ws.n_clients)]
    sads = synth.make_adapters(ws, range(ws.cut, ws.n_layer))
    to64 = lambda a: {k: {"A": v["A"].astype(np.float64), "B": v["B"].astype(np.float64)} for k, v in a.items()}
    st = O.OracleState(client_adapters=[to64(a) for a in cads], server_adapters=to64(sads))
    cfg = O.OracleConfig(n_layer=ws.n_layer, cut=ws.cut, d_model=ws.d_model, n_head=ws.n_head, d_ff=ws.d_ff,
                         vocab=ws.vocab, max_seq=ws.max_seq, lora_r=ws.lora_r, lora_alpha=ws.lora_alpha,
                         targets=ws.targets, n_clients=ws.n_clients, batch_per_client=ws.batch_per_client, seq=ws.seq,
                         bf16_handoff=(ws.dtype == "bf16"), optimizer="adamw", lr_client=ws.lr, lr_server=ws.lr,
                         agg_interval=ws.agg_interval, arch=ws.arch, rope_theta=ws.rope_theta)
    counts = synth.make_counts(ws)
    times = []
    for s in range(warmup + steps):
        tokens, labels = synth.make_tokens(ws, round_index=s)
        t0 = time.perf_counter()
        O.split_round(cfg, frozen, st, tokens, labels, counts)
        dt = time.perf_counter() - t0
        if s >= warmup:
            times.append(dt)
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        threads = os.cpu_count() or 1
    sec = float(np.mean(times)) * (w.n_layer / ws.n_layer)     # depth-reduced sample: linear in depth
    return ws.tokens_per_round / sec, sec, threads, ws


def sample_text(ws, sec=None):
    s = (f"one oracle round (numpy fp64) of the same model on {ws.n_clients} clients x {ws.batch_per_client} "
         f"sequence x {ws.seq} tokens = {ws.tokens_per_round} tokens")
    if ws.n_layer == 2 and ws.d_model >= 2048:
        s += (" with one client block and one server block at full width, the time multiplied by (blocks of the "
              "full model / 2): an extrapolation that also multiplies the head's share")
    return s + (f" ({sec:.1f} s)" if sec is not None else "")


def run_reference(args, w):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    tps, sec, threads, ws = time_oracle_rounds(w, args.steps, args.warmup)
    line = {"impl": "reference", "metric": METRIC, "value": tps, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": args.scaling,
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": workload_description(w),
            "cpu_baseline": {"value": tps, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample_text(ws)},
            "e2e": {"value": tps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_gpu(args, w):
    import torch
    import torch.distributed as dist
    from paper_2407_00952_b200 import runner

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    # Clients over ranks.  weak: every rank owns all K clients of the workload (a K*world-client job);
    # strong: the workload's K clients are spread over the ranks (K / world each, contiguous blocks).
    from paper_2407_00952_b200 import parallel
    strong = args.scaling == "strong"
    if strong and world > w.n_clients:
        raise SystemExit(f"strong scaling needs at least one client per rank ({w.n_clients} clients, {world} ranks)")
    mine = parallel.shard_clients(w.n_clients, world, rank) if strong else list(range(w.n_clients))
    all_counts = synth.make_counts(w)
    wl = synth.scaled(w, n_clients=len(mine))
    counts = all_counts[mine]
    cads = [synth.make_adapters(wl, range(wl.cut)) for _ in mine]
    sads = synth.make_adapters(wl, range(wl.cut, wl.n_layer))
    eng = runner.make_engine(wl, synth.iter_frozen(wl), cads, sads, optimizer="adamw")   # uploaded as drawn
    nbatch = 4
    host_tok, host_lab, dev_tok, dev_lab = [], [], [], []
    for s in range(nbatch):
        t, l = synth.make_tokens(w, round_index=s if strong else 1000 * rank + s)
        host_tok.append(torch.from_numpy(np.ascontiguousarray(t[mine])).pin_memory())
        host_lab.append(torch.from_numpy(np.ascontiguousarray(l[mine])).pin_memory())
        dev_tok.append(host_tok[-1].cuda())
        dev_lab.append(host_lab[-1].cuda())
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    if world == 1:
        def step_dev(s):
            eng.round(dev_tok[s % nbatch], dev_lab[s % nbatch], counts, want_loss=False)

        def step_host(s):
            return eng.round_host(host_tok[s % nbatch], host_lab[s % nbatch], counts, want_loss=True)
    else:
        # the server adapter gradients and the aggregation sum are all-reduced (NCCL) inside the round
        sharded = parallel.ShardedRound(eng, agg_interval=w.agg_interval)
        S_buf, dS_buf = eng.new_activation_buffer(), eng.new_activation_buffer()
        total_count = int(all_counts.sum()) * (1 if strong else world)
        n_valid_global = w.tokens_per_round * (1 if strong else world)
        stage_tok, stage_lab = torch.empty_like(dev_tok[0]), torch.empty_like(dev_lab[0])

        def step_dev(s):
            sharded.round(dev_tok[s % nbatch], dev_lab[s % nbatch], S_buf, dS_buf, counts, total_count, n_valid_global)

        def step_host(s):
            stage_tok.copy_(host_tok[s % nbatch], non_blocking=True)
            stage_lab.copy_(host_lab[s % nbatch], non_blocking=True)
            loss = sharded.round(stage_tok, stage_lab, S_buf, dS_buf, counts, total_count, n_valid_global)
            return float(loss.item())

    # ---- device-resident inputs: the headline value ----
    for s in range(args.warmup):
        step_dev(s)
    barrier()
    try:
        uuid = str(torch.cuda.get_device_properties(local).uuid)
    except Exception:
        uuid = None
    sampler = ClockSampler(uuid)
    sampler.start()
    # CUDA events around the tensor-bound linear launches only (the roofline's kernel): events around
    # all 609 launches of a round cost about 3 % of it; the full breakdown is taken after the timed region
    eng.profile_enable(2)
    eng.profile_report()                         # drop anything recorded before
    launches0 = eng.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    t_host = time.perf_counter()
    for s in range(args.steps):
        step_dev(s)
    host_ms = (time.perf_counter() - t_host) * 1e3     # time the host needs to enqueue the steps
    e1.record(stream)
    barrier()
    ms = e0.elapsed_time(e1)
    launches = eng.launch_count() - launches0
    prof = eng.profile_report()
    eng.profile_enable(False)
    clocks = sampler.stop()
    status = eng.device_status()
    if status != 0:
        raise RuntimeError(f"device status {status}: a bounded wait expired")

    # ---- end to end: host tokens in, host loss out, every step ----
    for s in range(2):
        step_host(s)
    barrier()
    e0.record(stream)
    losses = []
    for s in range(args.steps):
        losses.append(step_host(s))
    e1.record(stream)
    barrier()
    ms_e2e = e0.elapsed_time(e1)

    # ---- host cost of enqueueing one round: the stream is empty when the calls start, so nothing in
    # them waits for the device (a round is fewer launches than the launch queue holds) ----
    enq = []
    for s in range(3):
        barrier()
        t0 = time.perf_counter()
        step_dev(s)
        enq.append((time.perf_counter() - t0) * 1e3)
    barrier()
    host_enqueue_empty_ms = min(enq)

    # ---- per-class breakdown (outside the timed regions): events around every launch ----
    eng.profile_enable(1)
    eng.profile_report()
    for s in range(args.steps):
        step_dev(s)
    barrier()
    prof_all = eng.profile_report()
    eng.profile_enable(0)

    if world > 1:
        t = torch.tensor([ms, ms_e2e], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms, ms_e2e = float(t[0]), float(t[1])
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    tokens_total = w.tokens_per_round * args.steps * (1 if strong else world)
    w_local = wl                                   # what one rank runs: the per-launch figures below are its
    value = tokens_total / (ms * 1e-3)
    e2e_value = tokens_total / (ms_e2e * 1e-3)
    peaks = load_peaks()
    fl = gemm_flops_per_round(w_local)
    t_ms = sum(prof[k][1] for k in fl if k in prof)
    n_launch = sum(prof[k][0] for k in fl if k in prof)
    flops = sum(fl[k] for k in fl if k in prof) * args.steps
    achieved = flops / (t_ms * 1e-3) / 1e12 if t_ms > 0 else 0.0
    peak = peaks["tflops_sustained"]
    traffic, traffic_launch = load_traffic(w)
    by_class = {k: {"launches": prof[k][0], "ms_total": round(prof[k][1], 3),
                    "tflops": round(fl[k] * args.steps / (prof[k][1] * 1e-3) / 1e12, 1)}
                for k in fl if k in prof and prof[k][1] > 0}
    roofline = {"bound": "tensor",
                "kernel": "gemm_tc_kernel (tcgen05 linear layers incl. the LoRA-fused projections; skinny rank-r "
                          "down-projections excluded)",
                "achieved": round(achieved, 1), "peak": peak, "unit": "TFLOP/s",
                "frac": round(achieved / peak, 4) if peak else None,
                "peak_source": f"{peaks['source']} sustained bf16 (kernel timed inside a long step)",
                # DRAM bytes of one launch from the ncu capture recorded under profiles/ (None when the
                # kernel has changed since, or for a workload without a capture)
                "traffic": traffic, "traffic_launch": traffic_launch,
                "launches": n_launch, "avg_launch_us": round(t_ms * 1e3 / max(1, n_launch), 2),
                "by_class": by_class, "share_of_step": round(t_ms / ms, 4)}
    breakdown = {k: {"launches": v[0], "ms_per_step": round(v[1] / args.steps, 3)}
                 for k, v in sorted(prof_all.items(), key=lambda kv: -kv[1][1])}

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        tps, sec, threads, ws = time_oracle_rounds(w, 1, 0)
        cpu = {"value": tps, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample_text(ws, sec)}

    M = w_local.tokens_per_round
    if world == 1:
        par = "1 GPU"
    elif strong:
        par = (f"strong: the workload's {w.n_clients} clients spread over {world} GPUs, NCCL all-reduce of the server "
               f"adapter gradients and of one client's worth of aggregation sums")
    else:
        par = (f"weak: {w.n_clients} clients on each of {world} GPUs, NCCL all-reduce of the server adapter gradients "
               f"and of one client's worth of aggregation sums")
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms / args.steps, "host_enqueue_ms_per_step": host_ms / args.steps,
            "host_enqueue_empty_stream_ms": host_enqueue_empty_ms, "higher_is_better": True, "scaling": args.scaling, "vs_baseline": None,
            "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
            "config": workload_description(w), "parallelism": par,
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 2 * M * 4, "d2h_bytes_per_step": 4,
                    "ms_per_step": ms_e2e / args.steps, "last_loss": losses[-1]},
            "gpu_launches": launches, "roofline": roofline, "cpu_baseline": cpu, "kernel_breakdown": breakdown}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=3, help="workload index (3 = GPT-2-medium-shaped, the headline)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="weak: every GPU runs the workload's K clients; strong: the K clients are spread over the GPUs")
    args = ap.parse_args()
    if args.impl == "ours" and args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as a plain command: launch one rank per GPU and let them run this file
        import socket
        sock = socket.socket()
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
        sock.close()
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))
    if args.impl == "ours":
        args.warmup = max(args.warmup, 3)
    w = synth.WORKLOADS[args.config]
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_gpu(args, w)


if __name__ == "__main__":
    main()
