"""Attention backward for callers that cannot allocate (splitlora_attention_bwd_static).

Some users of the library run where cudaMalloc is off limits once set-up is over: a service with a
device-memory budget fixed at start, or a plug-in whose host application owns the allocator.  For
them the library keeps the small per-row scratch of the attention backward in a fixed internal
array.  This test drives that entry point through the C ABI twice in a row, with different shapes
so that the second call finds the first call's leftovers in the shared array, and requires the
same gradients as the ordinary entry point (which takes caller scratch) and as the CPU reference;
it also checks that a problem larger than the internal array is refused.  It is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from oracle import splitlora_oracle as O
from paper_2407_00952_b200 import binding as B

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2


def _case(nseq, T, heads, d, dtype, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    qkv = torch.randn(nseq * T, 3 * d, device="cuda", generator=g).to(dtype)
    d_o = torch.randn(nseq * T, d, device="cuda", generator=g).to(dtype)
    return qkv, d_o


def _rel(a, b):
    a, b = a.float(), b.float()
    return float((a - b).abs().max() / b.abs().max())


def test_static_scratch_matches_caller_scratch_twice():
    # first call: tensor-core kernels, 2 x 256 x 4 rows; second: plain kernels, fp32, other shape
    for nseq, T, heads, d, dtype, tc, seed in ((2, 256, 4, 256, torch.bfloat16, True, 1),
                                              (3, 96, 2, 48, torch.float32, False, 2),
                                              (1, 128, 2, 128, torch.bfloat16, True, 3)):
        qkv, d_o = _case(nseq, T, heads, d, dtype, seed)
        o, lse = B.attention_fwd(qkv, nseq, T, heads, tc)
        want = B.attention_bwd(qkv, o, lse, d_o, nseq, T, heads, tc)
        out = torch.full_like(qkv, float("nan"))
        got = B.attention_bwd_static(qkv, o, lse, d_o, nseq, T, heads, tc, dqkv=out)
        torch.cuda.synchronize()
        assert torch.isfinite(got).all()
        assert _rel(got, want) <= (TOL_BF16 if dtype == torch.bfloat16 else 1e-4)
        assert torch.equal(got, want)       # same kernels, same order of operations
        # and against the CPU reference of the attention gradients itself
        q64 = qkv.float().cpu().numpy().astype(np.float64)
        q, k, v = (q64[:, j * d:(j + 1) * d].reshape(nseq, T, d) for j in range(3))
        _, probs = O.causal_attention_fwd(q, k, v, heads)
        ref = O.causal_attention_bwd(d_o.float().cpu().numpy().astype(np.float64).reshape(nseq, T, d), q, k, v,
                                     probs, heads)
        got64 = got.float().cpu().numpy().astype(np.float64)
        for j in range(3):
            err = np.abs(got64[:, j * d:(j + 1) * d] - ref[j].reshape(-1, d)).max() / np.abs(ref[j]).max()
            assert err <= (TOL_BF16 if dtype == torch.bfloat16 else 1e-4), (nseq, T, j, err)


    assert B.library_status() == 0


def test_static_scratch_rejects_oversize():
    heads, d, T = 2, 128, 64
    nseq = B.STATIC_ATTENTION_ROWS // (T * heads) + 1
    tiny = torch.zeros(8, 3 * d, device="cuda", dtype=torch.bfloat16)   # never touched: refused before launch
    with pytest.raises(B.SplitLoraError) as e:
        B.attention_bwd_static(tiny, tiny, torch.zeros(8, device="cuda"), tiny, nseq, T, heads, dqkv=tiny)
    assert e.value.code == B.ERR_TOO_LARGE
