"""ctypes binding of libsplitlora.so: same names as the C ABI (include/splitlora.h), argument
marshalling only.  PyTorch supplies device memory and the stream; every step of the round runs in
the library's CUDA kernels.  There is no fallback: a missing library or a failing call raises."""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libsplitlora.so")
_lib = None

DTYPE_FP32, DTYPE_BF16 = 0, 1
OPT_SGD, OPT_ADAMW = 0, 1
TARGET_Q, TARGET_K, TARGET_V = 1, 2, 4
SIDE_CLIENT, SIDE_SERVER = 0, 1
TARGET_O = 8
ARCH_GPT, ARCH_LLAMA = 0, 1
TARGET_BITS = {"q": TARGET_Q, "k": TARGET_K, "v": TARGET_V, "o": TARGET_O}

EXPORTS = [
    "splitlora_create", "splitlora_destroy", "splitlora_workspace_bytes", "splitlora_bind_workspace",
    "splitlora_bind_frozen", "splitlora_set_adapter", "splitlora_get_adapter", "splitlora_get_adapter_grad",
    "splitlora_get_opt_state", "splitlora_set_opt_state", "splitlora_get_counters", "splitlora_set_counters",
    "splitlora_client_fwd", "splitlora_server_step", "splitlora_client_bwd", "splitlora_aggregate",
    "splitlora_round", "splitlora_round_host", "splitlora_loss_device", "splitlora_last_error",
    "splitlora_device_status", "splitlora_launch_count", "splitlora_profile_enable", "splitlora_profile_report",
    "splitlora_lora_linear_workspace_bytes", "splitlora_lora_linear_fwd", "splitlora_lora_linear_bwd",
    "splitlora_transpose", "splitlora_aggregate_buffers", "splitlora_attention_fwd", "splitlora_attention_bwd",
    "splitlora_attention_bwd_static", "splitlora_linear", "splitlora_set_loss_normalizer",
    "splitlora_set_deferred_server_update", "splitlora_server_update", "splitlora_adapter_buffer",
    "splitlora_adapters_changed", "splitlora_aggregate_local_sum", "splitlora_aggregate_broadcast",
    "splitlora_handoff_quantize",
    "splitlora_handoff_dequantize", "splitlora_round_compressed", "splitlora_set_client_ranks",
    "splitlora_library_status", "splitlora_set_client_cuts", "splitlora_lora_linear_bwd_parts",
    "splitlora_lora_linear_fwd_parts",
]


class SplitLoraError(RuntimeError):
    def __init__(self, code: int, msg: str = ""):
        super().__init__(f"splitlora error {code}: {msg}")
        self.code = code


class Config(C.Structure):
    _fields_ = [
        ("n_layer", C.c_int32), ("cut", C.c_int32), ("d_model", C.c_int32), ("n_head", C.c_int32),
        ("d_ff", C.c_int32), ("vocab", C.c_int32), ("max_seq", C.c_int32), ("lora_r", C.c_int32),
        ("lora_alpha", C.c_float), ("lora_targets", C.c_uint32), ("n_clients", C.c_int32),
        ("batch_per_client", C.c_int32), ("seq", C.c_int32), ("dtype", C.c_int32), ("optimizer", C.c_int32),
        ("lr_client", C.c_float), ("lr_server", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float),
        ("adam_eps", C.c_float), ("weight_decay", C.c_float), ("agg_interval", C.c_int32),
        ("norm_eps", C.c_float), ("gelu_tanh", C.c_int32), ("use_tensor_cores", C.c_int32),
        ("arch", C.c_int32), ("rope_theta", C.c_float), ("cut_min", C.c_int32),
    ]


def load():
    """Loads the shared library (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise FileNotFoundError(f"{_LIB_PATH} is missing: run `python -m paper_2407_00952_b200.build`")
        _lib = C.CDLL(_LIB_PATH)
        _lib.splitlora_last_error.restype = C.c_char_p
        for name in EXPORTS:
            getattr(_lib, name)
    return _lib


def config_from_workload(w, optimizer: str = "adamw", use_tensor_cores: bool = True, **over) -> Config:
    """Config for a synth.Workload (AdamW beta1 0.9, beta2 0.999, eps 1e-8, weight decay 0.01)."""
    tb = 0
    for t in w.targets:
        tb |= TARGET_BITS[t]
    cfg = Config(
        n_layer=w.n_layer, cut=w.cut, d_model=w.d_model, n_head=w.n_head, d_ff=w.d_ff, vocab=w.vocab,
        max_seq=w.max_seq, lora_r=w.lora_r, lora_alpha=w.lora_alpha, lora_targets=tb, n_clients=w.n_clients,
        batch_per_client=w.batch_per_client, seq=w.seq, dtype=DTYPE_BF16 if w.dtype == "bf16" else DTYPE_FP32,
        optimizer=OPT_ADAMW if optimizer == "adamw" else OPT_SGD, lr_client=w.lr, lr_server=w.lr, beta1=0.9,
        beta2=0.999, adam_eps=1e-8, weight_decay=0.01, agg_interval=w.agg_interval, norm_eps=1e-5, gelu_tanh=1,
        use_tensor_cores=1 if use_tensor_cores else 0,
        arch=ARCH_LLAMA if getattr(w, "arch", "gpt") == "llama" else ARCH_GPT,
        rope_theta=float(getattr(w, "rope_theta", 10000.0)), cut_min=0)
    for k, v in over.items():
        setattr(cfg, k, v)
    return cfg


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return C.c_void_p(0)
    assert t.is_cuda and t.is_contiguous()
    return C.c_void_p(t.data_ptr())


def _stream_ptr():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


class SplitLoRA:
    """One context: config + workspace + bound frozen weights.  Methods mirror the C calls."""

    def __init__(self, cfg: Config, stream: Optional[torch.cuda.Stream] = None):
        self.lib = load()
        self.cfg = cfg
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        self.ctx = C.c_void_p(0)
        rc = self.lib.splitlora_create(C.byref(cfg), C.c_void_p(self.stream.cuda_stream), C.byref(self.ctx))
        if rc:
            raise SplitLoraError(rc, "splitlora_create")
        nbytes = C.c_size_t(0)
        self._check(self.lib.splitlora_workspace_bytes(C.byref(cfg), C.byref(nbytes)))
        self.workspace_bytes = nbytes.value
        self.workspace = torch.empty(nbytes.value, dtype=torch.uint8, device="cuda")
        self._check(self.lib.splitlora_bind_workspace(self.ctx, _ptr(self.workspace), C.c_size_t(nbytes.value)))
        self.frozen: Dict[str, torch.Tensor] = {}
        self.act_dtype = torch.bfloat16 if cfg.dtype == DTYPE_BF16 else torch.float32

    def _check(self, rc: int):
        if rc:
            msg = self.lib.splitlora_last_error(self.ctx)
            raise SplitLoraError(rc, msg.decode() if msg else "")

    def close(self):
        if self.ctx:
            self.lib.splitlora_destroy(self.ctx)
            self.ctx = C.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- set-up ----
    def bind_frozen(self, name: str, t: torch.Tensor):
        assert t.dtype == self.act_dtype
        self.frozen[name] = t
        self._check(self.lib.splitlora_bind_frozen(self.ctx, name.encode(), _ptr(t), C.c_size_t(t.numel() * t.element_size())))

    def set_adapter(self, side, client, layer, target_bit, A=None, B=None):
        self._check(self.lib.splitlora_set_adapter(self.ctx, side, client, layer, C.c_uint32(target_bit), _ptr(A), _ptr(B)))

    def _get_pair(self, fn, side, client, layer, target_bit):
        r, d = self.cfg.lora_r, self.cfg.d_model
        A = torch.empty(r, d, dtype=torch.float32, device="cuda")
        B = torch.empty(d, r, dtype=torch.float32, device="cuda")
        self._check(fn(self.ctx, side, client, layer, C.c_uint32(target_bit), _ptr(A), _ptr(B)))
        return A, B

    def get_adapter(self, side, client, layer, target_bit):
        return self._get_pair(self.lib.splitlora_get_adapter, side, client, layer, target_bit)

    def get_adapter_grad(self, side, client, layer, target_bit):
        return self._get_pair(self.lib.splitlora_get_adapter_grad, side, client, layer, target_bit)

    def get_opt_state(self, side, client, layer, target_bit):
        r, d = self.cfg.lora_r, self.cfg.d_model
        mA, vA = (torch.empty(r, d, dtype=torch.float32, device="cuda") for _ in range(2))
        mB, vB = (torch.empty(d, r, dtype=torch.float32, device="cuda") for _ in range(2))
        self._check(self.lib.splitlora_get_opt_state(self.ctx, side, client, layer, C.c_uint32(target_bit),
                                                     _ptr(mA), _ptr(vA), _ptr(mB), _ptr(vB)))
        return mA, vA, mB, vB

    def set_opt_state(self, side, client, layer, target_bit, mA, vA, mB, vB):
        self._check(self.lib.splitlora_set_opt_state(self.ctx, side, client, layer, C.c_uint32(target_bit),
                                                     _ptr(mA), _ptr(vA), _ptr(mB), _ptr(vB)))

    def get_counters(self):
        a, b, c = C.c_int64(0), C.c_int64(0), C.c_int64(0)
        self._check(self.lib.splitlora_get_counters(self.ctx, C.byref(a), C.byref(b), C.byref(c)))
        return a.value, b.value, c.value

    def set_counters(self, round_index, server_steps, client_steps):
        self._check(self.lib.splitlora_set_counters(self.ctx, C.c_int64(round_index), C.c_int64(server_steps), C.c_int64(client_steps)))

    # ---- the round ----
    def new_activation_buffer(self):
        c = self.cfg
        return torch.empty(c.n_clients, c.batch_per_client, c.seq, c.d_model, dtype=self.act_dtype, device="cuda")

    def client_fwd(self, tokens: torch.Tensor, act_out: torch.Tensor):
        assert tokens.dtype == torch.int32
        self._check(self.lib.splitlora_client_fwd(self.ctx, _ptr(tokens), _ptr(act_out)))

    def server_step(self, act_in, labels, act_grad_out, want_loss: bool = True):
        assert labels.dtype == torch.int32
        loss = C.c_float(0.0)
        self._check(self.lib.splitlora_server_step(self.ctx, _ptr(act_in), _ptr(labels), _ptr(act_grad_out),
                                                   C.byref(loss) if want_loss else None))
        return loss.value if want_loss else None

    def client_bwd(self, act_grad_in):
        self._check(self.lib.splitlora_client_bwd(self.ctx, _ptr(act_grad_in)))

    def aggregate(self, counts):
        arr = (C.c_int64 * len(counts))(*[int(x) for x in counts])
        self._check(self.lib.splitlora_aggregate(self.ctx, arr))

    def round(self, tokens, labels, counts, want_loss: bool = True):
        arr = (C.c_int64 * len(counts))(*[int(x) for x in counts])
        loss = C.c_float(0.0)
        self._check(self.lib.splitlora_round(self.ctx, _ptr(tokens), _ptr(labels), arr,
                                             C.byref(loss) if want_loss else None))
        return loss.value if want_loss else None

    def set_client_ranks(self, ranks):
        """Per-client adapter ranks (None: one rank for all); see splitlora_set_client_ranks."""
        if ranks is None:
            self._check(self.lib.splitlora_set_client_ranks(self.ctx, None))
            return
        arr = (C.c_int32 * len(ranks))(*[int(x) for x in ranks])
        self._check(self.lib.splitlora_set_client_ranks(self.ctx, arr))

    def set_client_cuts(self, cuts):
        """Per-client cut depths, non-decreasing (None: one cut for all); see splitlora_set_client_cuts."""
        if cuts is None:
            self._check(self.lib.splitlora_set_client_cuts(self.ctx, None))
            return
        arr = (C.c_int32 * len(cuts))(*[int(x) for x in cuts])
        self._check(self.lib.splitlora_set_client_cuts(self.ctx, arr))

    def round_compressed(self, tokens, labels, counts, codes, scales, want_loss: bool = True):
        """codes uint8 [2, M, d], scales fp32 [2, M]: what crosses the cut (S, then dL/dS)."""
        arr = (C.c_int64 * len(counts))(*[int(x) for x in counts])
        loss = C.c_float(0.0)
        self._check(self.lib.splitlora_round_compressed(self.ctx, _ptr(tokens), _ptr(labels), arr, _ptr(codes),
                                                        _ptr(scales), C.byref(loss) if want_loss else None))
        return loss.value if want_loss else None

    def round_host(self, tokens_host: torch.Tensor, labels_host: torch.Tensor, counts, want_loss: bool = True):
        """tokens / labels are (pinned) HOST int32 tensors; the copies happen inside the call."""
        assert not tokens_host.is_cuda and tokens_host.dtype == torch.int32 and tokens_host.is_contiguous()
        assert not labels_host.is_cuda and labels_host.dtype == torch.int32 and labels_host.is_contiguous()
        arr = (C.c_int64 * len(counts))(*[int(x) for x in counts])
        loss = C.c_float(0.0)
        self._check(self.lib.splitlora_round_host(self.ctx, C.c_void_p(tokens_host.data_ptr()),
                                                  C.c_void_p(labels_host.data_ptr()), arr,
                                                  C.byref(loss) if want_loss else None))
        return loss.value if want_loss else None

    # ---- sharding hooks ----
    def set_loss_normalizer(self, n_valid_global: int):
        self._check(self.lib.splitlora_set_loss_normalizer(self.ctx, C.c_int64(n_valid_global)))

    def set_deferred_server_update(self, on: bool):
        self._check(self.lib.splitlora_set_deferred_server_update(self.ctx, 1 if on else 0))

    def server_update(self):
        self._check(self.lib.splitlora_server_update(self.ctx))

    def adapter_buffer(self, side: int, kind: int) -> torch.Tensor:
        """fp32 view (no copy) of an adapter arena inside the workspace: kind 0 parameters, 1 gradients."""
        ptr, n = C.c_void_p(0), C.c_int64(0)
        self._check(self.lib.splitlora_adapter_buffer(self.ctx, side, kind, C.byref(ptr), C.byref(n)))
        off = ptr.value - self.workspace.data_ptr()
        return self.workspace[off:off + 4 * n.value].view(torch.float32)

    def adapters_changed(self, side: int):
        self._check(self.lib.splitlora_adapters_changed(self.ctx, side))

    def aggregate_local_sum(self, counts, total_count: int) -> torch.Tensor:
        """Weighted sum of the local clients' adapters (weights |D_i| / total_count): fp32 view [Pc] of the
        workspace buffer that the caller all-reduces in place before aggregate_broadcast."""
        arr = (C.c_int64 * len(counts))(*[int(x) for x in counts])
        ptr, n = C.c_void_p(0), C.c_int64(0)
        self._check(self.lib.splitlora_aggregate_local_sum(self.ctx, arr, C.c_int64(total_count), C.byref(ptr), C.byref(n)))
        off = ptr.value - self.workspace.data_ptr()
        return self.workspace[off:off + 4 * n.value].view(torch.float32)

    def aggregate_broadcast(self):
        self._check(self.lib.splitlora_aggregate_broadcast(self.ctx))

    def loss_tensor(self) -> torch.Tensor:
        """fp32 view of the device loss scalar of the last server_step."""
        ptr = C.c_void_p(0)
        self._check(self.lib.splitlora_loss_device(self.ctx, C.byref(ptr)))
        off = ptr.value - self.workspace.data_ptr()
        return self.workspace[off:off + 4].view(torch.float32)

    def device_status(self) -> int:
        code = C.c_int32(0)
        self._check(self.lib.splitlora_device_status(self.ctx, C.byref(code)))
        return code.value

    def launch_count(self) -> int:
        n = C.c_int64(0)
        self._check(self.lib.splitlora_launch_count(self.ctx, C.byref(n)))
        return n.value

    def profile_enable(self, on):
        """on: False / 0 off, True / 1 every launch class, 2 the tensor-bound linear layers only."""
        self._check(self.lib.splitlora_profile_enable(self.ctx, int(on)))

    def profile_report(self):
        cap = 64
        names = ((C.c_char * 48) * cap)()
        launches = (C.c_int64 * cap)()
        ms = (C.c_double * cap)()
        n = C.c_int(0)
        self._check(self.lib.splitlora_profile_report(self.ctx, names, launches, ms, cap, C.byref(n)))
        return {names[i].value.decode(): (launches[i], ms[i]) for i in range(min(n.value, cap))}


# ---- stand-alone operators -------------------------------------------------------------------
def _dt(t: torch.Tensor) -> int:
    return DTYPE_BF16 if t.dtype == torch.bfloat16 else DTYPE_FP32


def _rc(rc, what):
    if rc:
        raise SplitLoraError(rc, what)


def lora_linear_workspace(dtype: int, M, n_in, n_out, r, G) -> torch.Tensor:
    lib = load()
    n = C.c_size_t(0)
    _rc(lib.splitlora_lora_linear_workspace_bytes(dtype, M, n_in, n_out, r, G, C.byref(n)), "lora_linear_workspace_bytes")
    return torch.empty(n.value, dtype=torch.uint8, device="cuda")


def lora_linear_fwd(x, W, bias, A, B, alpha, y=None, workspace=None, use_tensor_cores=True, parts=3):
    lib = load()
    M, n_in = x.shape
    n_out = W.shape[0]
    G, r, _ = A.shape
    if y is None:
        y = torch.empty(M, n_out, dtype=x.dtype, device="cuda")
    if workspace is None:
        workspace = lora_linear_workspace(_dt(x), M, n_in, n_out, r, G)
    _rc(lib.splitlora_lora_linear_fwd_parts(_dt(x), 1 if use_tensor_cores else 0, _ptr(x), _ptr(W), _ptr(bias), _ptr(A),
                                            _ptr(B), C.c_float(alpha), M, n_in, n_out, r, G, _ptr(y), _ptr(workspace),
                                            C.c_size_t(workspace.numel()), _stream_ptr(), int(parts)), "lora_linear_fwd")
    return y


def lora_linear_bwd(x, Wt, dy, A, B, alpha, workspace=None, use_tensor_cores=True, parts=7, out=None):
    """parts: sum of 1 (rank-r projections), 2 (dx), 4 (dA, dB), see splitlora_lora_linear_bwd_parts;
    out: (dx, dA, dB) buffers to reuse."""
    lib = load()
    M, n_in = x.shape
    n_out = dy.shape[1]
    G, r, _ = A.shape
    if out is None:
        out = (torch.empty(M, n_in, dtype=x.dtype, device="cuda"),
               torch.empty(G, r, n_in, dtype=torch.float32, device="cuda"),
               torch.empty(G, n_out, r, dtype=torch.float32, device="cuda"))
    dx, dA, dB = out
    if workspace is None:
        workspace = lora_linear_workspace(_dt(x), M, n_in, n_out, r, G)
    _rc(lib.splitlora_lora_linear_bwd_parts(_dt(x), 1 if use_tensor_cores else 0, _ptr(x), _ptr(Wt), _ptr(dy), _ptr(A),
                                            _ptr(B), C.c_float(alpha), M, n_in, n_out, r, G, _ptr(dx), _ptr(dA), _ptr(dB),
                                            _ptr(workspace), C.c_size_t(workspace.numel()), _stream_ptr(), int(parts)),
        "lora_linear_bwd")
    return dx, dA, dB


EPI_BIAS, EPI_BIAS_GELU, EPI_BIAS_RESID, EPI_MUL_GELUGRAD = 0, 1, 2, 3
_status_words = {}


def linear(x, W, bias=None, epilogue=EPI_BIAS, r=None, y=None, z=None, gelu_tanh=True, use_tensor_cores=True):
    """Frozen linear layer with fused epilogue (splitlora_linear).  Returns y, or (y, z) for the GELU epilogue."""
    lib = load()
    M, n_in = x.shape
    n_out = W.shape[0]
    if y is None:
        y = torch.empty(M, n_out, dtype=x.dtype, device="cuda")
    if epilogue == EPI_BIAS_GELU and z is None:
        z = torch.empty(M, n_out, dtype=x.dtype, device="cuda")
    dev = torch.cuda.current_device()
    if dev not in _status_words:
        _status_words[dev] = torch.zeros(64, dtype=torch.int32, device="cuda")
    _rc(lib.splitlora_linear(_dt(x), 1 if use_tensor_cores else 0, _ptr(x), _ptr(W), _ptr(bias), epilogue, _ptr(r),
                             _ptr(z), 1 if gelu_tanh else 0, M, n_in, n_out, _ptr(y), _ptr(_status_words[dev]),
                             _stream_ptr()), "linear")
    return (y, z) if epilogue == EPI_BIAS_GELU else y


def handoff_quantize(x: torch.Tensor, codes: Optional[torch.Tensor] = None, scales: Optional[torch.Tensor] = None):
    """x [M, d] -> (codes uint8 [M, d], scales fp32 [M]) (splitlora_handoff_quantize)."""
    lib = load()
    M, d = x.shape
    if codes is None:
        codes = torch.empty(M, d, dtype=torch.uint8, device="cuda")
    if scales is None:
        scales = torch.empty(M, dtype=torch.float32, device="cuda")
    _rc(lib.splitlora_handoff_quantize(_dt(x), _ptr(x), C.c_int64(M), d, _ptr(codes), _ptr(scales), _stream_ptr()),
        "handoff_quantize")
    return codes, scales


def handoff_dequantize(codes: torch.Tensor, scales: torch.Tensor, out: torch.Tensor) -> torch.Tensor:
    """(codes [M, d], scales [M]) -> out [M, d] in out's dtype (splitlora_handoff_dequantize)."""
    lib = load()
    M, d = codes.shape
    _rc(lib.splitlora_handoff_dequantize(_dt(out), _ptr(codes), _ptr(scales), C.c_int64(M), d, _ptr(out), _stream_ptr()),
        "handoff_dequantize")
    return out


def transpose(t: torch.Tensor) -> torch.Tensor:
    lib = load()
    rows, cols = t.shape
    out = torch.empty(cols, rows, dtype=t.dtype, device="cuda")
    _rc(lib.splitlora_transpose(_dt(t), _ptr(t), rows, cols, _ptr(out), _stream_ptr()), "transpose")
    return out


def aggregate_buffers(params: torch.Tensor, weights):
    lib = load()
    K, P = params.shape
    w = (C.c_double * K)(*[float(x) for x in weights])
    _rc(lib.splitlora_aggregate_buffers(_ptr(params), K, C.c_int64(P), w, _stream_ptr()), "aggregate_buffers")


def attention_fwd(qkv, nseq, T, n_head, use_tensor_cores=True):
    lib = load()
    d = qkv.shape[1] // 3
    o = torch.empty(nseq * T, d, dtype=qkv.dtype, device="cuda")
    lse = torch.empty(nseq, n_head, T, dtype=torch.float32, device="cuda")
    _rc(lib.splitlora_attention_fwd(_dt(qkv), 1 if use_tensor_cores else 0, _ptr(qkv), nseq, T, n_head, d, _ptr(o),
                                    _ptr(lse), _stream_ptr()), "attention_fwd")
    return o, lse


def attention_bwd(qkv, o, lse, d_o, nseq, T, n_head, use_tensor_cores=True):
    lib = load()
    d = qkv.shape[1] // 3
    dqkv = torch.empty_like(qkv)
    rowdot = torch.empty(nseq * n_head * T, dtype=torch.float32, device="cuda")
    _rc(lib.splitlora_attention_bwd(_dt(qkv), 1 if use_tensor_cores else 0, _ptr(qkv), _ptr(o), _ptr(lse), _ptr(d_o),
                                    nseq, T, n_head, d, _ptr(dqkv), _ptr(rowdot), _stream_ptr()), "attention_bwd")
    return dqkv


def library_status() -> int:
    """Status word of the stand-alone operators on the current device (0 = no bounded wait expired);
    synchronises the device."""
    code = C.c_int32(0)
    rc = load().splitlora_library_status(C.byref(code))
    if rc not in (0, -7):
        raise SplitLoraError(rc, "library_status")
    return code.value


STATIC_ATTENTION_ROWS = 1 << 20
ERR_TOO_LARGE = -10


def attention_bwd_static(qkv, o, lse, d_o, nseq, T, n_head, use_tensor_cores=True, dqkv=None):
    """Attention backward through splitlora_attention_bwd_static: the library's built-in scratch is
    used, so the call allocates nothing as long as the caller passes `dqkv`.  Raises SplitLoraError
    (code ERR_TOO_LARGE) when nseq * T * n_head exceeds STATIC_ATTENTION_ROWS."""
    lib = load()
    d = qkv.shape[1] // 3
    if dqkv is None:
        dqkv = torch.empty_like(qkv)
    _rc(lib.splitlora_attention_bwd_static(_dt(qkv), 1 if use_tensor_cores else 0, _ptr(qkv), _ptr(o), _ptr(lse),
                                           _ptr(d_o), nseq, T, n_head, d, _ptr(dqkv), _stream_ptr()),
        "attention_bwd_static")
    return dqkv
