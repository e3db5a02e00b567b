"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element on
the same seeded inputs.

Tolerances (normwise, max|gpu - ref| / max|ref| per tensor):
  fp32 configurations                       1e-4
  bf16 activations / logits / gradients     2e-2   (fp32 accumulation)
  aggregated adapters                       1e-6
  loss after one round                      1e-3 relative
"""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import splitlora_oracle as O
from paper_2407_00952_b200 import binding as B
from paper_2407_00952_b200 import runner, synth
import harness as H

pytestmark = pytest.mark.gpu

TOL_FP32 = 1e-4
TOL_BF16 = 2e-2
TOL_AGG = 1e-6
TOL_LOSS = 1e-3


def check_three_calls(w, tol, use_tc=True, case=None, tol_qk=None):
    """tol_qk: bound for the q and k adapter gradients where it differs from tol (see the caller)."""
    case = case or H.build_case(w)
    tol_of = lambda t: tol_qk if (tol_qk is not None and t in ("q", "k")) else tol
    eng, S, dS, loss = H.run_three_calls(w, *case, optimizer="sgd", use_tensor_cores=use_tc)
    cfg, params, c64, s64, S_ref, dS_ref, loss_ref, sg, cg = H.oracle_three_calls(w, *case, optimizer="sgd")
    assert abs(loss - loss_ref) <= TOL_LOSS * abs(loss_ref)
    assert H.rel_err(H.tnp(S), S_ref) <= tol
    assert H.rel_err(H.tnp(dS), dS_ref) <= tol
    for (l, t), (dA, dB) in sg.items():
        gA, gB = eng.get_adapter_grad(B.SIDE_SERVER, 0, l, B.TARGET_BITS[t])
        assert H.rel_err(H.tnp(gA), dA) <= tol_of(t), ("server dA", l, t)
        assert H.rel_err(H.tnp(gB), dB) <= tol_of(t), ("server dB", l, t)
    for i in range(w.n_clients):
        for (l, t), (dA, dB) in cg[i].items():
            gA, gB = eng.get_adapter_grad(B.SIDE_CLIENT, i, l, B.TARGET_BITS[t])
            assert H.rel_err(H.tnp(gA), dA) <= tol_of(t), ("client dA", i, l, t)
            assert H.rel_err(H.tnp(gB), dB) <= tol_of(t), ("client dB", i, l, t)
    # SGD update is the literal rule of Eq. 4-7: P_new = P - lr * G (on every element)
    for (l, t), (dA, dB) in sg.items():
        A, Bm = eng.get_adapter(B.SIDE_SERVER, 0, l, B.TARGET_BITS[t])
        assert H.rel_err(H.tnp(A), s64[(l, t)]["A"] - w.lr * dA) <= 1e-5
        assert H.rel_err(H.tnp(Bm), s64[(l, t)]["B"] - w.lr * dB) <= 1e-5
    return eng


def test_tiny_fp32_three_calls():
    """Tiny split GPT (fp32): activations, activation gradients, adapter gradients, loss."""
    check_three_calls(synth.WORKLOADS[1], TOL_FP32)


def test_tiny_fp32_zero_b_and_all_targets():
    """B = 0 (the paper-shaped initial state: dA must vanish) and adapters on q, k and v."""
    w = synth.scaled(synth.WORKLOADS[1], targets=("q", "k", "v"))
    case = H.build_case(w, nonzero_b=False, distinct_clients=False)
    eng = check_three_calls(w, TOL_FP32, case=case)
    gA, gB = eng.get_adapter_grad(B.SIDE_SERVER, 0, 1, B.TARGET_Q)
    assert float(gA.abs().max()) == 0.0 and float(gB.abs().max()) > 0.0


@pytest.mark.parametrize("cut", [1, 2])
def test_tiny_fp32_every_cut(cut):
    w = synth.scaled(synth.WORKLOADS[1], n_layer=3, cut=cut)
    check_three_calls(w, TOL_FP32)


def test_degenerate_splits_federated_and_centralised():
    """cut == n_layer (every block client-side and aggregated: the federated baseline of Sec. IV-A) and
    a single client (the centralised baseline) run through the same three calls."""
    check_three_calls(synth.scaled(synth.WORKLOADS[1], n_layer=2, cut=2), TOL_FP32)
    check_three_calls(synth.scaled(synth.WORKLOADS[1], n_clients=1, counts=(7,)), TOL_FP32)
    # bf16 federated case: its q / k adapter gradients take the bound that tests/test_storage_noise.py
    # derives on the CPU from bf16 storage alone; everything else keeps 2e-2
    w, _, qk_bound = H.qk_case("federated_small")
    eng = check_three_calls(w, TOL_BF16, tol_qk=qk_bound)
    # a full round on top: aggregation makes all clients equal on every block
    frozen, cads, sads, tokens, labels = H.build_case(w)
    eng = runner.make_engine(w, frozen, cads, sads, optimizer="sgd")
    eng.round(torch.from_numpy(tokens).cuda(), torch.from_numpy(labels).cuda(), [300, 500])
    for l in range(w.n_layer):
        A0, B0 = eng.get_adapter(B.SIDE_CLIENT, 0, l, B.TARGET_V)
        A1, B1 = eng.get_adapter(B.SIDE_CLIENT, 1, l, B.TARGET_V)
        assert torch.equal(A0, A1) and torch.equal(B0, B1)
    assert eng.adapter_buffer(B.SIDE_SERVER, 0).numel() == 0


def test_tiny_fp32_full_round_adamw_and_aggregation():
    """One full round of Algorithm 1 with AdamW and the 3:5 aggregation, through splitlora_round."""
    w = synth.WORKLOADS[1]
    frozen, cads, sads, tokens, labels = H.build_case(w)
    counts = synth.make_counts(w)
    eng = runner.make_engine(w, frozen, cads, sads, optimizer="adamw")
    loss = eng.round(torch.from_numpy(tokens).cuda(), torch.from_numpy(labels).cuda(), counts)
    cfg = H.oracle_config(w, optimizer="adamw")
    st = O.OracleState(client_adapters=[H.ads64(a) for a in cads], server_adapters=H.ads64(sads))
    loss_ref, info = O.split_round(cfg, H.f64(frozen), st, tokens, labels, counts)
    assert info["aggregated"]
    assert abs(loss - loss_ref) <= TOL_LOSS * abs(loss_ref)
    # AdamW's first step is ~ -lr*sign(g): compare where the gradient is not tiny (elsewhere the
    # sign is decided by rounding); the adapters below went through update + aggregation.
    for i in range(w.n_clients):
        for (l, t), ad in st.client_adapters[i].items():
            A, Bm = eng.get_adapter(B.SIDE_CLIENT, i, l, B.TARGET_BITS[t])
            gs = [info["client_grads"][k][(l, t)] for k in range(w.n_clients)]
            for got, ref, gi in ((A, ad["A"], 0), (Bm, ad["B"], 1)):
                mask = np.ones_like(ref, dtype=bool)
                for g in gs:
                    mask &= np.abs(g[gi]) > 1e-3 * np.abs(g[gi]).max()
                err = np.abs(H.tnp(got) - ref)[mask].max() / np.abs(ref).max()
                assert err <= 1e-4, (i, l, t, gi, err)
    # after aggregation all clients hold the same adapters (downlink b3)
    A0, B0 = eng.get_adapter(B.SIDE_CLIENT, 0, 0, B.TARGET_Q)
    A1, B1 = eng.get_adapter(B.SIDE_CLIENT, 1, 0, B.TARGET_Q)
    assert torch.equal(A0, A1) and torch.equal(B0, B1)
    assert eng.get_counters() == (1, 1, 1)


def test_aggregate_call_matches_oracle():
    """splitlora_aggregate on identical inputs: Eq. 8-9 within 1e-6, with a zero count and random counts."""
    w = synth.scaled(synth.WORKLOADS[1], n_clients=4, counts=None)
    frozen, cads, sads, tokens, labels = H.build_case(w)
    for counts in ([3, 5, 0, 8], synth.make_counts(w)):
        eng = runner.make_engine(w, frozen, cads, sads)
        eng.aggregate(counts)
        for (l, t) in cads[0]:
            for name, idx in (("A", 0), ("B", 1)):
                ref = O.aggregate([ca[(l, t)][name] for ca in cads], counts)
                for i in range(w.n_clients):
                    got = eng.get_adapter(B.SIDE_CLIENT, i, l, B.TARGET_BITS[t])[idx]
                    assert H.rel_err(H.tnp(got), ref) <= TOL_AGG
    # error paths: negative and all-zero counts are rejected before any launch
    with pytest.raises(B.SplitLoraError) as e:
        eng.aggregate([1, -1, 2, 3])
    assert e.value.code == -6
    with pytest.raises(B.SplitLoraError) as e:
        eng.aggregate([0, 0, 0, 0])
    assert e.value.code == -6


@pytest.mark.parametrize("K,P", [(1, 1024), (2, 4100), (8, 98304), (32, 1 << 18)])
def test_aggregate_buffers(K, P):
    rng = np.random.default_rng(K * 7 + P)
    params = rng.normal(size=(K, P)).astype(np.float32)
    counts = rng.integers(200, 1001, size=K)
    wts = O.aggregation_weights(counts)
    ref = O.aggregate(list(params), counts)
    dev = torch.from_numpy(params).cuda()
    B.aggregate_buffers(dev, wts)
    got = H.tnp(dev)
    for i in range(K):
        assert H.rel_err(got[i], ref) <= TOL_AGG
    if K == 1:
        assert np.array_equal(got[0], params[0].astype(np.float64))     # one client: identity


@pytest.mark.parametrize("use_tc", [True, False])
def test_gpt2_small_shaped_reduced_bf16(use_tc):
    """GPT-2-small-shaped model (d 768, 12 heads, vocab 50257) at reduced depth and batch, bf16."""
    w = synth.scaled(synth.WORKLOADS[2], n_layer=4, cut=2, n_clients=2, batch_per_client=1, seq=256, max_seq=256)
    check_three_calls(w, TOL_BF16, use_tc=use_tc)


def test_gpt2_medium_shaped_reduced_bf16():
    """GPT-2-medium-shaped model (d 1024, 16 heads) with 3 clients, two sequences each, ragged labels."""
    w = synth.scaled(synth.WORKLOADS[3], n_layer=3, cut=1, n_clients=3, batch_per_client=2, seq=128, max_seq=128)
    case = list(H.build_case(w))
    labels = case[4].copy()
    labels[0, 0, :17] = -1
    labels[2, 1, 100:] = -1
    case[4] = labels
    check_three_calls(w, TOL_BF16, case=tuple(case))


LINEAR_CASES = [
    # M, in, out, r, G   (several tiles, ragged output tails, every tile width of the kernel)
    (256, 128, 256, 4, 1),
    (512, 256, 512, 4, 2),
    (1024, 1024, 3072, 4, 4),
    (1024, 768, 2304, 16, 1),
    (2048, 1024, 1000, 8, 8),
    (1024, 512, 72, 1, 1),
    (2048, 1024, 4096, 64, 4),
    (4096, 768, 768, 8, 16),
]


def _linear_reference(x, W, bias, A, Bm, dy, alpha, G):
    M, n_in = x.shape
    n_out, r = W.shape[0], A.shape[1]
    rows, s = M // G, alpha / r
    ry, rdx = np.zeros((M, n_out)), np.zeros((M, n_in))
    rdA, rdB = np.zeros(A.shape), np.zeros(Bm.shape)
    b64 = None if bias is None else bias.astype(np.float64)
    for g in range(G):
        sl = slice(g * rows, (g + 1) * rows)
        args = (W.astype(np.float64), A[g].astype(np.float64), Bm[g].astype(np.float64), s)
        ry[sl], _ = O.lora_linear_fwd(x[sl].astype(np.float64), args[0], b64, *args[1:])
        rdx[sl], rdA[g], rdB[g] = O.lora_linear_bwd(dy[sl].astype(np.float64), x[sl].astype(np.float64), *args)
    return ry, rdx, rdA, rdB


@pytest.mark.parametrize("M,n_in,n_out,r,G", LINEAR_CASES)
def test_lora_linear_bf16(M, n_in, n_out, r, G):
    """Grouped LoRA linear forward and backward on tensor cores against the oracle layer."""
    alpha = 16.0
    x, W, A, Bm, dy = synth.make_lora_linear_case(M, n_in, n_out, r, G, seed=M + n_out + r)
    bias = synth._to_bf16_values((np.random.default_rng(5).normal(size=n_out) * 0.1).astype(np.float32))
    dev = lambda a: torch.from_numpy(a).cuda().bfloat16()
    xd, Wd, dyd, bd = dev(x), dev(W), dev(dy), dev(bias)
    Ad, Bd = torch.from_numpy(A).cuda(), torch.from_numpy(Bm).cuda()
    y = B.lora_linear_fwd(xd, Wd, bd, Ad, Bd, alpha)
    dx, dA, dB = B.lora_linear_bwd(xd, B.transpose(Wd), dyd, Ad, Bd, alpha)
    torch.cuda.synchronize()
    ry, rdx, rdA, rdB = _linear_reference(x, W, bias, A, Bm, dy, alpha, G)
    assert H.rel_err(H.tnp(y), ry) <= TOL_BF16
    assert H.rel_err(H.tnp(dx), rdx) <= TOL_BF16
    assert H.rel_err(H.tnp(dA), rdA) <= TOL_BF16
    assert H.rel_err(H.tnp(dB), rdB) <= TOL_BF16
    # the group boundary is respected: rows of group 0 do not depend on the adapters of group 1
    if G > 1:
        A2 = Ad.clone()
        A2[1:] = 0
        y2 = B.lora_linear_fwd(xd, Wd, bd, A2, Bd, alpha)
        assert torch.equal(y2[:M // G], y[:M // G])


def test_lora_linear_fp32():
    M, n_in, n_out, r, G = 512, 96, 200, 3, 2
    x, W, A, Bm, dy = synth.make_lora_linear_case(M, n_in, n_out, r, G, seed=3)
    dev = lambda a: torch.from_numpy(a).cuda()
    y = B.lora_linear_fwd(dev(x), dev(W), None, dev(A), dev(Bm), 6.0)
    dx, dA, dB = B.lora_linear_bwd(dev(x), B.transpose(dev(W)), dev(dy), dev(A), dev(Bm), 6.0)
    ry, rdx, rdA, rdB = _linear_reference(x, W, None, A, Bm, dy, 6.0, G)
    assert H.rel_err(H.tnp(y), ry) <= TOL_FP32
    assert H.rel_err(H.tnp(dx), rdx) <= TOL_FP32
    assert H.rel_err(H.tnp(dA), rdA) <= TOL_FP32
    assert H.rel_err(H.tnp(dB), rdB) <= TOL_FP32


@pytest.mark.parametrize("nseq,T,Hh,d,use_tc", [(2, 64, 2, 128, True), (2, 256, 3, 192, True),
                                                (1, 512, 2, 128, True), (3, 40, 4, 96, False),
                                                (2, 192, 2, 256, True), (1, 1024, 1, 128, True),
                                                (3, 128, 2, 128, True), (2, 384, 4, 256, True),
                                                (40, 128, 8, 512, True), (37, 256, 5, 320, True),
                                                (3, 128, 2, 256, True), (2, 384, 3, 384, True),
                                                (20, 256, 8, 1024, True)])
def test_attention_bf16(nseq, T, Hh, d, use_tc):
    """Causal attention forward/backward: tensor-core kernels (head width 64 and 128) and the plain kernels
    (any head width, ragged length) against the oracle.  Cases 7-10 exercise the persistent tcgen05
    kernels at head width 64: a single query tile, an odd number of tiles (ring and double-buffer
    parities), and more (sequence, head) items than resident CTAs, so that a CTA walks several items
    (320 and 185); the last three do the same at head width 128 (160 items in the last)."""
    torch.manual_seed(T + d)
    qkv = torch.randn(nseq * T, 3 * d, device="cuda").bfloat16()
    do = torch.randn(nseq * T, d, device="cuda").bfloat16()
    o, lse = B.attention_fwd(qkv, nseq, T, Hh, use_tc)
    dqkv = B.attention_bwd(qkv, o, lse, do, nseq, T, Hh, use_tc)
    q64 = H.tnp(qkv)
    q, k, v = (q64[:, i * d:(i + 1) * d].reshape(nseq, T, d) for i in range(3))
    o_ref, probs = O.causal_attention_fwd(q, k, v, Hh)
    dq, dk, dv = O.causal_attention_bwd(H.tnp(do).reshape(nseq, T, d), q, k, v, probs, Hh)
    assert H.rel_err(H.tnp(o), o_ref.reshape(-1, d)) <= TOL_BF16
    got = H.tnp(dqkv)
    for j, ref in enumerate((dq, dk, dv)):
        assert H.rel_err(got[:, j * d:(j + 1) * d], ref.reshape(-1, d)) <= TOL_BF16
    assert B.library_status() == 0          # no bounded wait of the stand-alone kernels expired


@pytest.mark.parametrize("Hh,d,T", [(2, 128, 512), (2, 256, 512), (2, 128, 1024)])
def test_attention_bf16_peaked_scores(Hh, d, T):
    """Scores with a standard deviation of about 6 and a drift along the keys: the row maximum keeps
    moving from key tile to key tile (the running rescale of O and of the row sum does real work, also in
    the kernel that rescales only when the maximum has moved by more than 2^8: with this spread it does so
    several times per row), most probabilities underflow, a few carry the row."""
    nseq = 2
    g = torch.Generator(device="cpu").manual_seed(d)
    dh = d // Hh
    qkv = torch.randn(nseq * T, 3 * d, generator=g)
    qkv[:, :2 * d] *= (6.0 * dh ** 0.5) ** 0.5 / dh ** 0.25          # q.k / sqrt(dh) ~ N(0, 36)
    ramp = torch.linspace(0.0, 3.0, T).repeat(nseq)[:, None]         # later keys score higher
    qkv[:, d:2 * d] += ramp * torch.sign(qkv[:, :d].mean(dim=0, keepdim=True))
    qkv = qkv.bfloat16().cuda()
    do = torch.randn(nseq * T, d, generator=g).bfloat16().cuda()
    o, lse = B.attention_fwd(qkv, nseq, T, Hh, True)
    dqkv = B.attention_bwd(qkv, o, lse, do, nseq, T, Hh, True)
    q64 = H.tnp(qkv)
    q, k, v = (q64[:, i * d:(i + 1) * d].reshape(nseq, T, d) for i in range(3))
    o_ref, probs = O.causal_attention_fwd(q, k, v, Hh)
    dq, dk, dv = O.causal_attention_bwd(H.tnp(do).reshape(nseq, T, d), q, k, v, probs, Hh)
    assert float(probs.max(axis=-1).mean()) > 0.5                    # peaked indeed
    assert H.rel_err(H.tnp(o), o_ref.reshape(-1, d)) <= TOL_BF16
    got = H.tnp(dqkv)
    for j, ref in enumerate((dq, dk, dv)):
        assert H.rel_err(got[:, j * d:(j + 1) * d], ref.reshape(-1, d)) <= TOL_BF16, j


def test_out_of_range_labels_are_ignored():
    """A label outside [0, vocab) is an ignored position for the loss, the gradients and the normaliser
    alike: the round equals the oracle's with those positions marked -1."""
    w = synth.WORKLOADS[1]
    frozen, cads, sads, tokens, labels = H.build_case(w)
    gpu_labels, ref_labels = labels.copy(), labels.copy()
    gpu_labels[0, 1, 5:40] = w.vocab + 3
    gpu_labels[1, 2, :7] = -5
    ref_labels[0, 1, 5:40] = -1
    ref_labels[1, 2, :7] = -1
    eng, S, dS, loss = H.run_three_calls(w, frozen, cads, sads, tokens, gpu_labels)
    _, _, _, _, S_ref, dS_ref, loss_ref, sg, _ = H.oracle_three_calls(w, frozen, cads, sads, tokens, ref_labels)
    assert abs(loss - loss_ref) <= TOL_LOSS * abs(loss_ref)
    assert H.rel_err(H.tnp(dS), dS_ref) <= TOL_FP32
    for (l, t), (dA, dB) in sg.items():
        gA, gB = eng.get_adapter_grad(B.SIDE_SERVER, 0, l, B.TARGET_BITS[t])
        assert H.rel_err(H.tnp(gA), dA) <= TOL_FP32 and H.rel_err(H.tnp(gB), dB) <= TOL_FP32


def test_checkpoint_resume_and_determinism():
    """Two contexts fed the same state produce bit-identical results; state copied out of one
    context and into a fresh one continues identically (adapters, moments, counters)."""
    w = synth.WORKLOADS[1]
    frozen, cads, sads, tokens, labels = H.build_case(w)
    counts = synth.make_counts(w)
    tok, lab = torch.from_numpy(tokens).cuda(), torch.from_numpy(labels).cuda()
    a = runner.make_engine(w, frozen, cads, sads)
    b = runner.make_engine(w, frozen, cads, sads)
    la = [a.round(tok, lab, counts) for _ in range(2)]
    lb = [b.round(tok, lab, counts)]
    c = runner.make_engine(w, frozen, cads, sads)
    for side, clients, layers in ((B.SIDE_CLIENT, range(w.n_clients), range(w.cut)),
                                  (B.SIDE_SERVER, [0], range(w.cut, w.n_layer))):
        for i in clients:
            for l in layers:
                for t in w.targets:
                    bit = B.TARGET_BITS[t]
                    c.set_adapter(side, i, l, bit, *b.get_adapter(side, i, l, bit))
                    c.set_opt_state(side, i, l, bit, *b.get_opt_state(side, i, l, bit))
    c.set_counters(*b.get_counters())
    lb.append(c.round(tok, lab, counts))
    assert la == lb
    for t in w.targets:
        for x, y in zip(a.get_adapter(B.SIDE_SERVER, 0, 1, B.TARGET_BITS[t]),
                        c.get_adapter(B.SIDE_SERVER, 0, 1, B.TARGET_BITS[t])):
            assert torch.equal(x, y)


def test_error_paths():
    w = synth.WORKLOADS[1]
    lib = B.load()
    bad = B.config_from_workload(w)
    bad.cut = w.n_layer + 1
    ctx = C.c_void_p(0)
    assert lib.splitlora_create(C.byref(bad), None, C.byref(ctx)) == -1
    eng = B.SplitLoRA(B.config_from_workload(w))
    S = eng.new_activation_buffer()
    with pytest.raises(B.SplitLoraError) as e:      # frozen tensors not bound yet
        eng.client_fwd(torch.zeros(2, 4, 64, dtype=torch.int32, device="cuda"), S)
    assert e.value.code == -3
    frozen, cads, sads, tokens, labels = H.build_case(w)
    eng = runner.make_engine(w, frozen, cads, sads)
    with pytest.raises(B.SplitLoraError) as e:      # backward without forward
        eng.client_bwd(S)
    assert e.value.code == -3
    with pytest.raises(B.SplitLoraError) as e:      # misaligned buffer
        flat = torch.zeros(S.numel() + 8, dtype=S.dtype, device="cuda")
        eng.client_fwd(torch.from_numpy(tokens).cuda(), flat[1:1 + S.numel()].view_as(S))
    assert e.value.code == -2
    with pytest.raises(B.SplitLoraError) as e:      # wrong size for a frozen tensor
        eng.bind_frozen("wte", torch.zeros(8, dtype=torch.float32, device="cuda"))
    assert e.value.code == -1
    assert eng.device_status() == 0


@pytest.mark.parametrize("M,n_in,n_out", [(256, 128, 512), (1024, 1024, 1000), (512, 256, 64)])
def test_linear_epilogues_bf16(M, n_in, n_out):
    """Frozen linear with each fused epilogue (pair kernel, single-CTA kernel, ragged width)
    against fp64: bias, bias + GELU (pre-activation saved), bias + residual, product with GELU'."""
    rng = np.random.default_rng(M + n_out)
    bfv = lambda a: synth._to_bf16_values(a.astype(np.float32))
    x, W = bfv(rng.normal(size=(M, n_in))), bfv(rng.normal(size=(n_out, n_in)) / np.sqrt(n_in))
    bias, r = bfv(rng.normal(size=n_out) * 0.1), bfv(rng.normal(size=(M, n_out)))
    dev = lambda a: torch.from_numpy(a).cuda().bfloat16()
    xd, Wd, bd, rd = dev(x), dev(W), dev(bias), dev(r)
    acc = x.astype(np.float64) @ W.astype(np.float64).T
    y = B.linear(xd, Wd, bd, B.EPI_BIAS)
    assert H.rel_err(H.tnp(y), acc + bias) <= TOL_BF16
    y, z = B.linear(xd, Wd, bd, B.EPI_BIAS_GELU)
    assert H.rel_err(H.tnp(z), acc + bias) <= TOL_BF16
    assert H.rel_err(H.tnp(y), O.gelu_fwd(acc + bias)) <= TOL_BF16
    y = B.linear(xd, Wd, bd, B.EPI_BIAS_RESID, r=rd)
    assert H.rel_err(H.tnp(y), acc + bias + r) <= TOL_BF16
    y = B.linear(xd, Wd, None, B.EPI_MUL_GELUGRAD, r=rd)
    assert H.rel_err(H.tnp(y), acc * O.gelu_grad(r.astype(np.float64))) <= TOL_BF16
    y2 = B.linear(xd, Wd, None, B.EPI_MUL_GELUGRAD, r=rd, use_tensor_cores=False)
    assert H.rel_err(H.tnp(y2), acc * O.gelu_grad(r.astype(np.float64))) <= TOL_BF16
