"""Convenience set-up of a SplitLoRA context from a synth.Workload: uploads frozen tensors and
adapters.  Marshalling only; used by the tests, the benchmark and the smoke entry."""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B


def to_device(a: np.ndarray, dtype: torch.dtype) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).to(device="cuda", dtype=dtype)


def make_engine(w, frozen, client_adapters, server_adapters, optimizer="adamw", use_tensor_cores=True, **over):
    """frozen: {name: fp32 ndarray}; client_adapters: list (one per client) of {(layer, target): {"A","B"}};
    server_adapters: {(layer, target): {"A","B"}}."""
    cfg = B.config_from_workload(w, optimizer=optimizer, use_tensor_cores=use_tensor_cores, **over)
    eng = B.SplitLoRA(cfg)
    for name, arr in frozen.items():
        if name.endswith("mlp.up.w"):
            continue                      # bound together with the gate, below
        if name.endswith("mlp.gate.w"):   # the library takes gate and up stacked as one [2F, d] tensor
            up = frozen[name[:-len("gate.w")] + "up.w"]
            name, arr = name[:-len("gate.w")] + "gate_up.w", np.concatenate([arr, up], axis=0)
        eng.bind_frozen(name, to_device(arr, eng.act_dtype))
    for i, ca in enumerate(client_adapters):
        for (l, t), ad in ca.items():
            eng.set_adapter(B.SIDE_CLIENT, i, l, B.TARGET_BITS[t], to_device(ad["A"], torch.float32),
                            to_device(ad["B"], torch.float32))
    for (l, t), ad in server_adapters.items():
        eng.set_adapter(B.SIDE_SERVER, 0, l, B.TARGET_BITS[t], to_device(ad["A"], torch.float32),
                        to_device(ad["B"], torch.float32))
    torch.cuda.synchronize()
    return eng
