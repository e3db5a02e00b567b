"""CPU-only checks: the shared library loads and exports every symbol the header declares, the
Python config struct matches the C struct's field order, and the input generators are seeded."""
import ctypes
import os
import re

import numpy as np

from paper_2407_00952_b200 import binding as B
from paper_2407_00952_b200 import build, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def header_text():
    return open(os.path.join(ROOT, "include", "splitlora.h")).read()


def test_library_exports_every_declared_symbol():
    build.build()
    lib = ctypes.CDLL(build.LIB_PATH)
    declared = set(re.findall(r"\b(splitlora_[a-z_0-9]+)\s*\(", header_text()))
    assert len(declared) >= 30
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(B.EXPORTS)
    for call in ("splitlora_client_fwd", "splitlora_server_step", "splitlora_client_bwd", "splitlora_aggregate",
                 "splitlora_round"):
        assert call in declared


def test_config_struct_matches_header():
    body = re.search(r"typedef struct \{(.*?)\} splitlora_config;", header_text(), re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    names = []
    for decl in body.split(";"):
        decl = decl.strip()
        if not decl:
            continue
        decl = re.sub(r"^(int32_t|uint32_t|float)\s+", "", decl)
        names += [n.strip() for n in decl.split(",")]
    assert names == [f[0] for f in B.Config._fields_]
    assert ctypes.sizeof(B.Config) == 4 * len(names)


def test_calls_without_a_device_fail_cleanly():
    """No GPU here: creation must return an error code, never crash or fall back."""
    import torch
    if torch.cuda.is_available():
        return
    lib = B.load()
    cfg = B.config_from_workload(synth.WORKLOADS[1])
    ctx = ctypes.c_void_p(0)
    rc = lib.splitlora_create(ctypes.byref(cfg), None, ctypes.byref(ctx))
    assert rc < 0 and not ctx.value
    n = ctypes.c_size_t(0)
    assert lib.splitlora_workspace_bytes(ctypes.byref(cfg), ctypes.byref(n)) == 0 and n.value > 0


def test_workspace_plan_scales_with_the_configuration():
    lib = B.load()
    sizes = []
    for idx in (1, 2, 3):
        cfg = B.config_from_workload(synth.WORKLOADS[idx])
        n = ctypes.c_size_t(0)
        assert lib.splitlora_workspace_bytes(ctypes.byref(cfg), ctypes.byref(n)) == 0
        sizes.append(n.value)
    assert sizes[0] < sizes[1] < sizes[2] < 60 * 2 ** 30      # fits one 180 GB device with room to spare
    bad = B.config_from_workload(synth.WORKLOADS[1])
    bad.lora_r = 65
    assert lib.splitlora_workspace_bytes(ctypes.byref(bad), ctypes.byref(ctypes.c_size_t(0))) == -1


def test_generators_are_seeded_and_shaped():
    w = synth.WORKLOADS[1]
    a, b = synth.make_frozen(w), synth.make_frozen(w)
    assert all(np.array_equal(a[k], b[k]) for k in a)
    assert a["h.0.attn.qkv.w"].shape == (3 * w.d_model, w.d_model)
    assert abs(a["wte"].std() - 0.02) < 2e-3 and not a["h.1.mlp.fc1.b"].any() and (a["lnf.g"] == 1).all()
    ads = synth.make_adapters(w, range(w.n_layer))
    assert not ads[(0, "q")]["B"].any() and abs(ads[(0, "q")]["A"].std() - 0.02) < 5e-3
    # Algorithm 1, initialisation: every client starts from the same adapters
    assert np.array_equal(synth.make_adapters(w, range(w.cut))[(0, "v")]["A"], ads[(0, "v")]["A"])
    tok, lab = synth.make_tokens(w)
    assert tok.shape == (2, 4, 64) and tok.dtype == np.int32 and np.array_equal(tok[..., 1:], lab[..., :-1])
    assert list(synth.make_counts(w)) == [3, 5]
    w3 = synth.scaled(synth.WORKLOADS[3], batch_per_client=1)
    tok3, _ = synth.make_tokens(w3)
    assert tok3.min() >= 0 and tok3.max() < w3.vocab
    top = np.bincount(tok3.ravel(), minlength=w3.vocab).max() / tok3.size
    assert 0.05 < top < 0.25                                   # Zipf(1.1): the most frequent id dominates
    c3 = synth.make_counts(synth.WORKLOADS[3])
    assert c3.shape == (8,) and c3.min() >= 200 and c3.max() <= 1000
    # bf16 workloads hand out bf16-exact values
    import torch
    f2 = synth.make_frozen(synth.scaled(synth.WORKLOADS[2], n_layer=2, cut=1, vocab=512))
    wq = torch.from_numpy(f2["h.0.attn.qkv.w"])
    assert torch.equal(wq, wq.to(torch.bfloat16).to(torch.float32))
