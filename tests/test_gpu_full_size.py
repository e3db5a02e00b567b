"""The GPT-2-small- and GPT-2-medium-shaped workloads at their full sizes, in the launch configuration
the benchmark times (12 / 24 blocks, 4 / 8 clients x 8 sequences x 512 tokens, vocabulary 50257, bf16).

A full oracle round at this size takes hours, so the check uses what the method itself fixes:
* sequences are independent on the client side (Sec. III-B step a1: clients run in parallel) and on
  the server side up to the common loss normaliser, so the oracle can follow ONE sampled sequence
  through all 24 blocks and the head by itself; its cut-layer activations and, scaled by
  (its valid positions / all valid positions), its activation gradients must equal the rows the GPU
  produced for that sequence inside the full batch;
* the first loss of a model with N(0, 0.02) weights lies just above ln V (closed form);
* Eq. 8-9 on the adapters the full-size round produced, against the weighted mean in fp64;
* the grouped LoRA linear layer alone at the launch shape of the medium-shaped round (32768 rows in 8 groups
  of 4096, 1024 -> 3072, rank 4): groups are independent, so the oracle computes two sampled groups in full
  (output, input gradient, and the adapter gradients G_A, G_B of Eq. 4-7).
"""
import numpy as np
import pytest
import torch

import harness as H
from oracle import splitlora_oracle as O
from paper_2407_00952_b200 import binding as B
from paper_2407_00952_b200 import runner, synth

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2
TOL_AGG = 1e-6


@pytest.mark.parametrize("index", [2, 3])
def test_full_size_sampled_sequences_loss_and_aggregation(index):
    w = synth.WORKLOADS[index]
    frozen = synth.make_frozen(w)
    cads = [synth.make_adapters(w, range(w.cut), nonzero_b=True, salt=i + 1) for i in range(w.n_clients)]
    sads = synth.make_adapters(w, range(w.cut, w.n_layer), nonzero_b=True, salt=77)
    tokens, labels = synth.make_tokens(w)
    counts = synth.make_counts(w)

    eng = runner.make_engine(w, frozen, cads, sads, optimizer="adamw")
    tok, lab = torch.from_numpy(tokens).cuda(), torch.from_numpy(labels).cuda()
    S, dS = eng.new_activation_buffer(), eng.new_activation_buffer()
    eng.client_fwd(tok, S)
    loss = eng.server_step(S, lab, dS)
    eng.client_bwd(dS)
    torch.cuda.synchronize()
    assert eng.device_status() == 0

    # closed form: logits of a random small-weight model have variance d * 0.02^2 (0.31 / 0.41), so
    # the mean cross-entropy is ln V plus about half of that
    assert np.log(w.vocab) < loss < np.log(w.vocab) + 0.6, loss

    # sampled sequences through the oracle, each alone
    params = H.f64(frozen)
    del frozen
    w1 = synth.scaled(w, n_clients=1, batch_per_client=1)
    cfg1 = H.oracle_config(w1, optimizer="adamw")
    n_all = int((labels >= 0).sum())
    Sv = S.view(w.n_clients, w.batch_per_client, w.seq, w.d_model)
    dSv = dS.view(w.n_clients, w.batch_per_client, w.seq, w.d_model)
    for ci, si in ((w.n_clients - 3, 3), (0, 7)):
        tok1, lab1 = tokens[ci:ci + 1, si:si + 1], labels[ci:ci + 1, si:si + 1]
        S_ref, _ = O.client_fwd(cfg1, params, [H.ads64(cads[ci])], tok1)
        loss1, dS_ref, _ = O.server_fwd_bwd(cfg1, params, H.ads64(sads), S_ref, lab1)
        # the oracle normalised by this sequence's valid positions, the round by all of them
        dS_ref = np.asarray(dS_ref) * (int((lab1 >= 0).sum()) / n_all)
        assert H.rel_err(H.tnp(Sv[ci, si]), np.asarray(S_ref).reshape(w.seq, w.d_model)) <= TOL_BF16, (ci, si)
        assert H.rel_err(H.tnp(dSv[ci, si]), dS_ref.reshape(w.seq, w.d_model)) <= TOL_BF16, (ci, si)
    del params

    # Eq. 8-9 at full size, on the adapters this round left behind
    before = [[eng.get_adapter(B.SIDE_CLIENT, i, l, B.TARGET_BITS[t]) for i in range(w.n_clients)]
              for l in range(w.cut) for t in w.targets]
    eng.aggregate(counts)
    wts = O.aggregation_weights(counts)
    k = 0
    for l in range(w.cut):
        for t in w.targets:
            for part in (0, 1):
                ref = sum(wts[i] * H.tnp(before[k][i][part]) for i in range(w.n_clients))
                for i in (0, w.n_clients - 1):
                    got = H.tnp(eng.get_adapter(B.SIDE_CLIENT, i, l, B.TARGET_BITS[t])[part])
                    assert H.rel_err(got, ref) <= TOL_AGG, (l, t, part, i)
            k += 1


def test_full_size_grouped_lora_linear_adapter_gradients():
    """G_A and G_B (and y, dx) of the grouped LoRA linear at M 32768, 8 groups, 1024 -> 3072, rank 4: the
    shape the adapted projection of every client block has in the GPT-2-medium-shaped round."""
    M, n_in, n_out, r, G, alpha = 32768, 1024, 3072, 4, 8, 32.0
    x, W, A, Bm, dy = synth.make_lora_linear_case(M, n_in, n_out, r, G, seed=4242)
    dev = lambda a: torch.from_numpy(a).cuda().bfloat16()
    xd, Wd, dyd = dev(x), dev(W), dev(dy)
    Ad, Bd = torch.from_numpy(A).cuda(), torch.from_numpy(Bm).cuda()
    y = B.lora_linear_fwd(xd, Wd, None, Ad, Bd, alpha)
    dx, dA, dB = B.lora_linear_bwd(xd, B.transpose(Wd), dyd, Ad, Bd, alpha)
    torch.cuda.synchronize()
    rows, s = M // G, alpha / r
    W64 = W.astype(np.float64)
    for g in (2, G - 1):
        sl = slice(g * rows, (g + 1) * rows)
        A64, B64, x64, dy64 = (a.astype(np.float64) for a in (A[g], Bm[g], x[sl], dy[sl]))
        ry, _ = O.lora_linear_fwd(x64, W64, None, A64, B64, s)
        rdx, rdA, rdB = O.lora_linear_bwd(dy64, x64, W64, A64, B64, s)
        assert H.rel_err(H.tnp(y[sl]), ry) <= TOL_BF16, g
        assert H.rel_err(H.tnp(dx[sl]), rdx) <= TOL_BF16, g
        assert H.rel_err(H.tnp(dA[g]), rdA) <= TOL_BF16, g
        assert H.rel_err(H.tnp(dB[g]), rdB) <= TOL_BF16, g
