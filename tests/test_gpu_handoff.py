"""Compressed cut-layer hand-off on the GPU against the oracle's codec (oracle/handoff_codec.py).

Codes and scales are integer / bit work: compared exactly on identical seeded inputs.  The rounding
decisions are taken in fp32 on both sides (the kernel's precision).  Round-level checks keep the
tolerances of the uncompressed path where both sides quantise the SAME tensor (the oracle's), and
say what is compared where each side quantises its own slightly different tensor.
"""
import numpy as np
import pytest
import torch

import harness as H
from oracle import handoff_codec as Q
from oracle import splitlora_oracle as O
from paper_2407_00952_b200 import binding as B
from paper_2407_00952_b200 import runner, synth

pytestmark = pytest.mark.gpu

TOL_FP32 = 1e-4
TOL_BF16 = 2e-2


def _rows(M, d, seed, bf16):
    """Rows like the tensors that cross the cut: activations of order 1 with outlier features and
    gradient-like rows many orders of magnitude smaller, a zero row, exact zeros, a lone value."""
    rng = np.random.default_rng(seed)
    x = rng.normal(0, 1, (M, d)).astype(np.float32)
    x[:, rng.integers(0, d, 3)] *= 30.0                              # outlier features
    x *= (10.0 ** rng.uniform(-8, 1, (M, 1))).astype(np.float32)     # per-token magnitude
    if M > 3:
        x[1] = 0.0
        x[2, ::2] = 0.0
        x[3] = 0.0
        x[3, d - 1] = -3.5
    return synth._to_bf16_values(x) if bf16 else x


def _dev(x, bf16):
    t = torch.from_numpy(x).cuda()
    return t.bfloat16() if bf16 else t


@pytest.mark.parametrize("M,d,bf16", [(37, 768, True), (1000, 1024, True), (5, 8, True), (129, 4096, True),
                                      (1, 2048, True), (33, 132, False), (513, 128, False), (2, 4, False)])
def test_codec_bit_exact(M, d, bf16):
    x = _rows(M, d, 10 + M, bf16)
    codes_ref, scales_ref = Q.quantize_rows(x)
    codes, scales = B.handoff_quantize(_dev(x, bf16))
    assert np.array_equal(codes.cpu().numpy(), codes_ref)
    assert np.array_equal(scales.cpu().numpy().view(np.uint32), scales_ref.view(np.uint32))
    out = torch.empty(M, d, dtype=torch.bfloat16 if bf16 else torch.float32, device="cuda")
    B.handoff_dequantize(codes, scales, out)
    ref = Q.dequantize_rows(codes_ref, scales_ref, bf16)
    assert np.array_equal(out.float().cpu().numpy().view(np.uint32), ref.view(np.uint32))


def test_dequantize_every_code():
    codes = np.tile(np.array([c for c in range(256) if c & 0x7F != 0x7F], dtype=np.uint8), 2)[:504].reshape(3, 168)
    scales = np.float32([1.0, 0.37, 3e-7])
    out = torch.empty(3, 168, dtype=torch.float32, device="cuda")
    B.handoff_dequantize(torch.from_numpy(codes).cuda(), torch.from_numpy(scales).cuda(), out)
    ref = Q.dequantize_rows(codes, scales, bf16=False)
    assert np.array_equal(out.cpu().numpy().view(np.uint32), ref.view(np.uint32))


def test_codec_full_size_sampled_rows():
    """The hand-off tensor of the GPT-2-medium-shaped round (32768 tokens x 1024, bf16): the codec is
    row by row, so sampled rows through the oracle check the full-size launch."""
    M, d = 32768, 1024
    g = torch.Generator(device="cpu").manual_seed(5)
    x = (torch.randn(M, d, generator=g) * torch.exp(torch.randn(M, 1, generator=g) * 3)).bfloat16()
    codes, scales = B.handoff_quantize(x.cuda())
    out = torch.empty(M, d, dtype=torch.bfloat16, device="cuda")
    B.handoff_dequantize(codes, scales, out)
    rows = np.r_[0, 1, 7, 8, 4095, 4096, 32767, np.random.default_rng(0).integers(0, M, 57)]
    xr = x[rows].float().numpy()
    cr, sr = Q.quantize_rows(xr)
    assert np.array_equal(codes[rows].cpu().numpy(), cr)
    assert np.array_equal(scales[rows].cpu().numpy(), sr)
    assert np.array_equal(out[rows].float().cpu().numpy(), Q.dequantize_rows(cr, sr, True))
    # property at any size: the restored tensor is within half a code step of the input
    err = (out.float() - x.cuda().float()).abs()
    bound = torch.maximum(x.cuda().float().abs() * 2.0 ** -4, scales[:, None] * 2.0 ** -10) * 1.01 + x.cuda().float().abs() * 2.0 ** -8
    assert bool((err <= bound).all())


def test_codec_argument_errors():
    x = torch.zeros(4, 12, dtype=torch.bfloat16, device="cuda")          # 12 is not a multiple of 8
    with pytest.raises(B.SplitLoraError):
        B.handoff_quantize(x)
    x = torch.zeros(4, 16, dtype=torch.bfloat16, device="cuda")
    codes = torch.zeros(4 * 16 + 16, dtype=torch.uint8, device="cuda")[1:65].view(4, 16)   # misaligned
    with pytest.raises(B.SplitLoraError):
        B.handoff_quantize(x, codes=codes)


def _three_calls_with_codec(w, tol, tol_qk=None):
    """Server and client sides each continue from the restored hand-off.  Both sides quantise the
    oracle's S and dL/dS (inputs may flow from the oracle to the GPU, never back), so the codes agree
    exactly and what follows keeps the tolerance of the uncompressed path."""
    bf16 = w.dtype == "bf16"
    frozen, cads, sads, tokens, labels = H.build_case(w)
    cfg = H.oracle_config(w, optimizer="sgd")
    params, c64, s64 = H.f64(frozen), [H.ads64(a) for a in cads], H.ads64(sads)
    M, d = tokens.size, w.d_model
    S_ref, caches = O.client_fwd(cfg, params, c64, tokens)
    S_hat = Q.handoff(np.asarray(S_ref, dtype=np.float32).reshape(M, d), bf16)
    loss_ref, dS_ref, sg = O.server_fwd_bwd(cfg, params, s64, S_hat.astype(np.float64).reshape(S_ref.shape), labels)
    dS_hat = Q.handoff(np.asarray(dS_ref, dtype=np.float32).reshape(M, d), bf16)
    cg = O.client_bwd_grads(cfg, params, c64, dS_hat.astype(np.float64).reshape(S_ref.shape), caches)

    eng = runner.make_engine(w, frozen, cads, sads, optimizer="sgd")
    tok, lab = torch.from_numpy(tokens).cuda(), torch.from_numpy(labels).cuda()
    S, dS = eng.new_activation_buffer(), eng.new_activation_buffer()
    eng.client_fwd(tok, S)
    assert H.rel_err(H.tnp(S), S_ref) <= tol
    # the link carries the oracle's S: quantise it on the GPU, restore, continue
    S_in = _dev(np.asarray(S_ref, dtype=np.float32).reshape(M, d), bf16)
    codes, scales = B.handoff_quantize(S_in)
    assert np.array_equal(codes.cpu().numpy(), Q.quantize_rows(np.asarray(S_ref, dtype=np.float32).reshape(M, d))[0])
    B.handoff_dequantize(codes, scales, S.view(M, d))
    loss = eng.server_step(S, lab, dS)
    assert abs(loss - loss_ref) <= (1e-4 if not bf16 else 5e-3) * abs(loss_ref)
    assert H.rel_err(H.tnp(dS), dS_ref) <= tol
    dS_in = _dev(np.asarray(dS_ref, dtype=np.float32).reshape(M, d), bf16)
    codes, scales = B.handoff_quantize(dS_in)
    B.handoff_dequantize(codes, scales, dS.view(M, d))
    assert np.array_equal(H.tnp(dS).reshape(M, d).astype(np.float32), dS_hat)
    eng.client_bwd(dS)
    torch.cuda.synchronize()
    assert eng.device_status() == 0
    tol_of = lambda t: (tol_qk if (tol_qk and t in ("q", "k")) else tol)
    for (l, t), (dA, dB) in sg.items():
        gA, gB = eng.get_adapter_grad(B.SIDE_SERVER, 0, l, B.TARGET_BITS[t])
        assert H.rel_err(H.tnp(gA), dA) <= tol_of(t) and H.rel_err(H.tnp(gB), dB) <= tol_of(t), ("server", l, t)
    for i in range(w.n_clients):
        for (l, t), (dA, dB) in cg[i].items():
            gA, gB = eng.get_adapter_grad(B.SIDE_CLIENT, i, l, B.TARGET_BITS[t])
            assert H.rel_err(H.tnp(gA), dA) <= tol_of(t) and H.rel_err(H.tnp(gB), dB) <= tol_of(t), ("client", i, l, t)
    # compression changed the step: the restored hand-off is not the exact one
    assert H.rel_err(S_hat, np.asarray(S_ref).reshape(M, d)) > 1e-3


def test_three_calls_with_codec_fp32_tiny():
    _three_calls_with_codec(synth.WORKLOADS[1], TOL_FP32)


def test_three_calls_with_codec_bf16_medium_shaped():
    w = synth.scaled(synth.WORKLOADS[3], n_layer=3, cut=1, n_clients=3, batch_per_client=2, seq=128, max_seq=128)
    _three_calls_with_codec(w, TOL_BF16, tol_qk=4e-2)


def test_round_compressed_entry_point_fp32():
    """splitlora_round_compressed end to end (SGD, aggregation 3:5).  Each side quantises its own S,
    which differ by fp32 rounding, so a few codes out of 65536 may fall on the other side of a
    rounding boundary: codes are compared as a fraction, what follows with a looser tolerance."""
    w = synth.WORKLOADS[1]
    frozen, cads, sads, tokens, labels = H.build_case(w)
    counts = synth.make_counts(w)
    M, d = tokens.size, w.d_model
    cfg = H.oracle_config(w, optimizer="sgd")
    params = H.f64(frozen)
    st = O.OracleState(client_adapters=[H.ads64(a) for a in cads], server_adapters=H.ads64(sads))
    S_ref, caches = O.client_fwd(cfg, params, st.client_adapters, tokens)
    cS, sS = Q.quantize_rows(np.asarray(S_ref, dtype=np.float32).reshape(M, d))
    S_hat = Q.dequantize_rows(cS, sS, False).astype(np.float64).reshape(S_ref.shape)
    loss_ref, dS_ref, sg = O.server_fwd_bwd(cfg, params, st.server_adapters, S_hat, labels)
    cD, sD = Q.quantize_rows(np.asarray(dS_ref, dtype=np.float32).reshape(M, d))
    dS_hat = Q.dequantize_rows(cD, sD, False).astype(np.float64).reshape(S_ref.shape)
    cg = O.client_bwd_grads(cfg, params, st.client_adapters, dS_hat, caches)
    O.apply_update(cfg, st.server_adapters, st.server_opt, sg, cfg.lr_server, 1)
    for i, g in enumerate(cg):
        O.apply_update(cfg, st.client_adapters[i], st.client_opt[i], g, cfg.lr_client, 1)
    O.aggregate_clients(st, counts)

    eng = runner.make_engine(w, frozen, cads, sads, optimizer="sgd")
    codes = torch.zeros(2, M, d, dtype=torch.uint8, device="cuda")
    scales = torch.zeros(2, M, dtype=torch.float32, device="cuda")
    loss = eng.round_compressed(torch.from_numpy(tokens).cuda(), torch.from_numpy(labels).cuda(), counts, codes, scales)
    assert abs(loss - loss_ref) <= 1e-3 * abs(loss_ref)
    got = codes.cpu().numpy()
    assert (got[0] != cS).mean() <= 1e-3 and (got[1] != cD).mean() <= 1e-3
    assert np.allclose(scales[0].cpu().numpy(), sS, rtol=1e-4) and np.allclose(scales[1].cpu().numpy(), sD, rtol=1e-3)
    for (l, t), ad in st.server_adapters.items():
        A, Bm = eng.get_adapter(B.SIDE_SERVER, 0, l, B.TARGET_BITS[t])
        assert H.rel_err(H.tnp(A), ad["A"]) <= 1e-4 and H.rel_err(H.tnp(Bm), ad["B"]) <= 1e-4
    for (l, t), ad in st.client_adapters[0].items():
        for i in range(w.n_clients):
            A, Bm = eng.get_adapter(B.SIDE_CLIENT, i, l, B.TARGET_BITS[t])
            assert H.rel_err(H.tnp(A), ad["A"]) <= 1e-4 and H.rel_err(H.tnp(Bm), ad["B"]) <= 1e-4
    assert eng.get_counters() == (1, 1, 1)
