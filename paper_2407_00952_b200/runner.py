"""Convenience set-up of a SplitLoRA context from a synth.Workload: uploads frozen tensors and
adapters.  Marshalling only; used by the tests, the benchmark and the smoke entry."""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B


def to_device(a: np.ndarray, dtype: torch.dtype) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).to(device="cuda", dtype=dtype)


def make_engine(w, frozen, client_adapters, server_adapters, optimizer="adamw", use_tensor_cores=True, **over):
    """frozen: {name: fp32 ndarray} or an iterable of (name, array) pairs in which a layer's "mlp.up.w"
    follows its "mlp.gate.w"; client_adapters: list (one per client) of {(layer, target): {"A","B"}};
    server_adapters: {(layer, target): {"A","B"}}."""
    cfg = B.config_from_workload(w, optimizer=optimizer, use_tensor_cores=use_tensor_cores, **over)
    eng = B.SplitLoRA(cfg)
    gate = None
    for name, arr in (frozen.items() if hasattr(frozen, "items") else frozen):
        if name.endswith("mlp.gate.w"):   # the library takes gate and up stacked as one [2F, d] tensor
            gate = to_device(arr, eng.act_dtype)
            continue
        if name.endswith("mlp.up.w"):
            name = name[:-len("up.w")] + "gate_up.w"
            dev = torch.cat([gate, to_device(arr, eng.act_dtype)], dim=0)
            gate = None
        else:
            dev = to_device(arr, eng.act_dtype)
        eng.bind_frozen(name, dev)
    for i, ca in enumerate(client_adapters):
        for (l, t), ad in ca.items():
            eng.set_adapter(B.SIDE_CLIENT, i, l, B.TARGET_BITS[t], to_device(ad["A"], torch.float32),
                            to_device(ad["B"], torch.float32))
    for (l, t), ad in server_adapters.items():
        eng.set_adapter(B.SIDE_SERVER, 0, l, B.TARGET_BITS[t], to_device(ad["A"], torch.float32),
                        to_device(ad["B"], torch.float32))
    torch.cuda.synchronize()
    return eng
