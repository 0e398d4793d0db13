"""ctypes binding of include/zo.h: structure mirrors and argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libzo_b200.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError(
        f"{_LIB_PATH} is missing: build it with `python paper_2409_15520_b200/build.py` "
        "(there is no CPU or PyTorch fallback)")
LIB = C.CDLL(_LIB_PATH)

STATUS_NAMES = ["ZO_OK", "ZO_ERR_INVALID_ARG", "ZO_ERR_UNSUPPORTED", "ZO_ERR_WORKSPACE",
                "ZO_ERR_CUDA", "ZO_ERR_TIMEOUT", "ZO_ERR_NONFINITE", "ZO_ERR_STATE"]
ZO_FP32, ZO_BF16 = 0, 1
ZO_FLAG_SIMT_GEMM, ZO_FLAG_GEMM_PAIR, ZO_FLAG_LORA_EPILOGUE, ZO_FLAG_GEMM_SINGLE = 1, 2, 4, 8
ZO_FLAG_DEQUANT_FUSED = 16
ZO_FLAG_CE_LOGITS = 32
ZO_FLAG_ATTN_WARP_MMA = 64
ZO_FLAG_TEST_EXPIRE_WAIT = 1 << 24


class ZoError(RuntimeError):
    def __init__(self, status, msg=""):
        self.status = int(status)
        name = STATUS_NAMES[self.status] if 0 <= self.status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{name}: {msg}")


class ZoConfig(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("arch", C.c_int32), ("precision", C.c_int32),
                ("loss_kind", C.c_int32), ("n_layers", C.c_int32), ("d_model", C.c_int32),
                ("d_out", C.c_int32), ("n_heads", C.c_int32), ("d_ffn", C.c_int32),
                ("vocab", C.c_int32), ("max_seq", C.c_int32), ("lora_rank", C.c_int32),
                ("lora_scale", C.c_float), ("lora_targets", C.c_uint32),
                ("label_words", C.c_int32 * 2), ("max_q", C.c_int32), ("max_E", C.c_int32),
                ("max_labelled", C.c_int32), ("norm_eps", C.c_float), ("rope_theta", C.c_float),
                ("tie_lm_head", C.c_int32), ("flags", C.c_uint32), ("weight_format", C.c_int32),
                ("max_shard_q", C.c_int32)]


_LAYER_FIELDS = ["norm1_g", "norm1_b", "w_qkv", "b_qkv", "w_o", "b_o", "norm2_g", "norm2_b",
                 "w_fc1", "b_fc1", "w_fc2", "b_fc2"]


class ZoLayerWeights(C.Structure):
    _fields_ = [(f, C.c_void_p) for f in _LAYER_FIELDS] + [(f, C.c_void_p) for f in ("s_qkv", "s_o", "s_fc1", "s_fc2")]


class ZoWeights(C.Structure):
    _fields_ = [("tok_emb", C.c_void_p), ("pos_emb", C.c_void_p), ("lm_head", C.c_void_p),
                ("final_norm_g", C.c_void_p), ("final_norm_b", C.c_void_p),
                ("layers", C.POINTER(ZoLayerWeights)), ("linear_w", C.c_void_p),
                ("linear_bias", C.c_void_p)]


class ZoLora(C.Structure):
    _fields_ = [("A", C.POINTER(C.c_void_p)), ("B", C.POINTER(C.c_void_p))]


class ZoLoraPair(C.Structure):
    _fields_ = [("A", C.POINTER(C.c_void_p)), ("B_pair", C.POINTER(C.c_void_p))]


def _sig(name, res, args):
    f = getattr(LIB, name)
    f.restype, f.argtypes = res, args
    return f


zo_workspace_bytes = _sig("zo_workspace_bytes", C.c_size_t, [C.POINTER(ZoConfig)])
zo_init = _sig("zo_init", C.c_int, [C.POINTER(ZoConfig), C.c_void_p, C.c_size_t, C.c_void_p,
                                    C.POINTER(C.c_void_p)])
_STEP_ARGS = [C.c_void_p, C.POINTER(ZoWeights), C.POINTER(ZoLora), C.c_void_p, C.c_void_p,
              C.c_int32, C.c_int32, C.c_uint64, C.c_int32, C.c_float, C.c_float]
zo_step = _sig("zo_step", C.c_int, _STEP_ARGS)
zo_step_host = _sig("zo_step_host", C.c_int, _STEP_ARGS)
zo_step_varlen = _sig("zo_step_varlen", C.c_int, [
    C.c_void_p, C.POINTER(ZoWeights), C.POINTER(ZoLora), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
    C.c_int32, C.c_int32, C.c_uint64, C.c_int32, C.c_float, C.c_float])
zo_losses = _sig("zo_losses", C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p])
zo_row_losses = _sig("zo_row_losses", C.c_int, [C.c_void_p, C.c_void_p, C.POINTER(C.c_int32)])
zo_launch_count = _sig("zo_launch_count", C.c_int32, [C.c_void_p])
zo_set_schedule = _sig("zo_set_schedule", C.c_int, [C.c_void_p, C.c_int32])
zo_set_query_shard = _sig("zo_set_query_shard", C.c_int, [C.c_void_p, C.c_int32, C.c_int32])
zo_step_pair = _sig("zo_step_pair", C.c_int, [C.c_void_p, C.POINTER(ZoWeights), C.POINTER(ZoLoraPair), C.c_void_p,
                                              C.c_void_p, C.c_int32, C.c_int32, C.c_uint64, C.c_void_p, C.c_float,
                                              C.c_float])
zo_pair_collapse = _sig("zo_pair_collapse", C.c_int, [C.c_void_p, C.POINTER(ZoLoraPair), C.c_void_p, C.c_float,
                                                      C.c_float])
zo_g_buffer = _sig("zo_g_buffer", C.c_int, [C.c_void_p, C.POINTER(C.c_void_p), C.POINTER(C.c_int32)])
zo_mp_lora_linear_pair = _sig("zo_mp_lora_linear_pair", C.c_int, [
    C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
    C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_float, C.c_uint64, C.c_uint32, C.c_float, C.c_float,
    C.c_float, C.c_int32, C.c_void_p, C.c_size_t, C.c_uint32])
zo_test_expire_wait = _sig("zo_test_expire_wait", C.c_int, [C.c_void_p, C.c_uint64])
zo_loss_buffer = _sig("zo_loss_buffer", C.c_int, [C.c_void_p, C.POINTER(C.c_void_p), C.POINTER(C.c_int32)])
zo_apply_update = _sig("zo_apply_update", C.c_int, [C.c_void_p, C.POINTER(ZoLora), C.c_uint64, C.c_int32,
                                                    C.c_float, C.c_float])
SCHEDULES = {"full": 0, "outer_only": 1, "inner_only": 2, "sequential": 3}
zo_free = _sig("zo_free", None, [C.c_void_p])
zo_profile_enable = _sig("zo_profile_enable", C.c_int, [C.c_void_p, C.c_int32])
zo_profile_read = _sig("zo_profile_read", C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p])
PROFILE_CLASSES = ["gemm_tc", "gemm_simt", "attention", "norm", "lora_down", "lora_apply", "rope",
                   "swiglu", "loss", "update", "misc", "gemm_qkv", "gemm_o", "gemm_fc1", "gemm_fc2",
                   "gemm_head", "dequant"]
zo_last_error = _sig("zo_last_error", C.c_char_p, [C.c_void_p])
zo_perturbation = _sig("zo_perturbation", C.c_int, [C.c_void_p, C.c_uint64, C.c_uint32, C.c_uint32,
                                                    C.c_int64, C.c_void_p, C.c_void_p])
zo_dequantize = _sig("zo_dequantize", C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                                C.c_void_p, C.c_int32, C.c_int32])
zo_mp_lora_scratch_bytes = _sig("zo_mp_lora_scratch_bytes", C.c_size_t, [C.c_int32] * 7)
zo_mp_lora_linear = _sig("zo_mp_lora_linear", C.c_int, [
    C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
    C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_float, C.c_uint64, C.c_uint32, C.c_int32,
    C.c_float, C.c_int32, C.c_void_p, C.c_size_t, C.c_uint32])


zo_mp_lora_linear_static = _sig("zo_mp_lora_linear_static", C.c_int, [
    C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
    C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_float, C.c_uint64, C.c_uint32, C.c_int32,
    C.c_float, C.c_int32, C.c_uint32])
zo_mp_lora_linear_static_status = _sig("zo_mp_lora_linear_static_status", C.c_int,
                                       [C.c_void_p, C.POINTER(C.c_uint32)])
STATIC_SCRATCH_BYTES = 16 << 20


WEIGHT_FORMATS = {None: 0, "native": 0, "int8": 1, "nf4": 2}


def make_config(spec, *, max_q=None, max_E=None, max_seq=None, max_labelled=None, flags=0,
                precision=None, weight_format=None, max_shard_q=0) -> ZoConfig:
    """zo_config from a shape record with the attribute names of workloads.ModelSpec."""
    c = ZoConfig()
    c.struct_size = C.sizeof(ZoConfig)
    c.arch, c.loss_kind = spec.arch, spec.loss_kind
    c.precision = (ZO_BF16 if spec.bf16 else ZO_FP32) if precision is None else precision
    c.n_layers, c.d_model, c.d_out = spec.n_layers, spec.d_model, spec.d_out
    c.n_heads, c.d_ffn, c.vocab = spec.n_heads, spec.d_ffn, spec.vocab
    c.max_seq = max_seq or max(spec.max_seq, spec.S)
    c.lora_rank, c.lora_scale, c.lora_targets = spec.lora_rank, spec.lora_scale, spec.lora_targets
    c.label_words[0], c.label_words[1] = spec.label_words
    c.max_q, c.max_E = max_q or spec.q, max_E or spec.E
    c.max_labelled = max_labelled or spec.n_labelled
    c.norm_eps, c.rope_theta = spec.norm_eps, spec.rope_theta
    c.tie_lm_head, c.flags = int(spec.tie_lm_head), flags
    c.weight_format = WEIGHT_FORMATS[weight_format]
    c.max_shard_q = max_shard_q
    return c


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else C.c_void_p(None)


class DeviceProblem:
    """Device copies of a synthetic problem (dict of numpy arrays as produced by the
    workload generators) plus the zo_weights / zo_lora structures pointing at them."""

    def __init__(self, p: dict, bf16: bool, device="cuda", n_layers=None):
        self.dtype = torch.bfloat16 if bf16 else torch.float32
        self.device = device
        self._keep = []
        self.weights = ZoWeights()
        self.lora = ZoLora()
        if "W" in p:  # single linear
            self.linear = True
            self.W, self.bias, self.A = self._up(p["W"]), self._up(p.get("bias")), self._up(p["A"])
            self.B = [torch.tensor(p["B"], dtype=torch.float32, device=device).contiguous()]
            self.weights.linear_w, self.weights.linear_bias = _ptr(self.W), _ptr(self.bias)
            self._A = [self.A]
            self.tokens = self._up(p["X"])
            self.labels = torch.tensor(p["target"], dtype=torch.float32, device=device).contiguous()
            self.host_tokens = self.tokens.cpu().pin_memory()
            self.host_labels = self.labels.cpu().pin_memory()
        else:
            self.linear = False
            for k in ("tok_emb", "pos_emb", "lm_head", "final_norm_g", "final_norm_b"):
                t = self._up(p.get(k))
                setattr(self, k, t)
                setattr(self.weights, k, _ptr(t))
            # p["layers"] may be a generator (one block in host memory at a time)
            n = len(p["layers"]) if n_layers is None else n_layers
            self._layers = (ZoLayerWeights * n)()
            self._A, self.B = [], []
            for l, L in enumerate(p["layers"]):
                for f in _LAYER_FIELDS:
                    v = L.get(f)
                    if isinstance(v, dict):       # quantised record: codes + float32 scales
                        codes = torch.tensor(v["codes"], device=device).contiguous()
                        scale = torch.tensor(v["scale"], dtype=torch.float32, device=device).contiguous()
                        self._keep += [codes, scale]
                        setattr(self._layers[l], f, _ptr(codes))
                        setattr(self._layers[l], "s_" + f[2:], _ptr(scale))
                    else:
                        setattr(self._layers[l], f, _ptr(self._up(v)))
                self._A.append(self._up(L["A"]) if L["A"].size else None)
                self.B.append(torch.tensor(L["B"], dtype=torch.float32, device=device).contiguous()
                              if L["B"].size else None)
            self.weights.layers = self._layers
            self.tokens = torch.tensor(p["tokens"], dtype=torch.int32, device=device).contiguous()
            self.labels = torch.tensor(p["labels"], dtype=torch.int32, device=device).contiguous()
            self.host_tokens = torch.tensor(p["tokens"], dtype=torch.int32).pin_memory()
            self.host_labels = torch.tensor(p["labels"], dtype=torch.int32).pin_memory()
        n = len(self.B)
        self._Aarr = (C.c_void_p * n)(*[(t.data_ptr() if t is not None else None) for t in self._A])
        self._Barr = (C.c_void_p * n)(*[(t.data_ptr() if t is not None else None) for t in self.B])
        self.lora.A = C.cast(self._Aarr, C.POINTER(C.c_void_p))
        self.lora.B = C.cast(self._Barr, C.POINTER(C.c_void_p))

    def _up(self, x):
        if x is None:
            return None
        t = torch.tensor(np.asarray(x, np.float32), device=self.device).to(self.dtype).contiguous()
        self._keep.append(t)
        return t

    def make_pair(self):
        """The trainable tensors in the stored-pair form of Algorithm 2: per layer a float32 tensor
        [2, ...] whose two halves both start as the current B.  Returns the zo_lora_pair structure;
        the tensors are kept in self.B_pair."""
        self.B_pair = [torch.stack([b, b]).contiguous() if b is not None else None for b in self.B]
        self._Parr = (C.c_void_p * len(self.B_pair))(*[(t.data_ptr() if t is not None else None)
                                                       for t in self.B_pair])
        self.pair = ZoLoraPair()
        self.pair.A = C.cast(self._Aarr, C.POINTER(C.c_void_p))
        self.pair.B_pair = C.cast(self._Parr, C.POINTER(C.c_void_p))
        return self.pair

    def pair_numpy(self):
        return [t.detach().cpu().numpy().astype(np.float64) if t is not None else None for t in self.B_pair]

    def B_numpy(self):
        return [b.detach().cpu().numpy().astype(np.float64) if b is not None else None
                for b in self.B]


class Estimator:
    """zo_init / zo_step / zo_losses with a torch-allocated workspace on the current stream."""

    def __init__(self, cfg: ZoConfig, device="cuda"):
        self.cfg = cfg
        nbytes = zo_workspace_bytes(C.byref(cfg))
        if nbytes == 0:
            h = C.c_void_p()
            st = zo_init(C.byref(cfg), None, 0, None, C.byref(h))
            raise ZoError(st, zo_last_error(None).decode())
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        self.stream = torch.cuda.current_stream()
        self._h = C.c_void_p()
        st = zo_init(C.byref(cfg), C.c_void_p(base), nbytes, C.c_void_p(self.stream.cuda_stream),
                     C.byref(self._h))
        if st:
            raise ZoError(st, zo_last_error(None).decode())
        self.q = 0

    def _check(self, st):
        if st:
            raise ZoError(st, zo_last_error(self._h).decode())

    def step(self, prob: DeviceProblem, E, S, seed, q, eps, lr, tokens=None, labels=None):
        tok = prob.tokens if tokens is None else tokens
        lab = prob.labels if labels is None else labels
        self._check(zo_step(self._h, C.byref(prob.weights), C.byref(prob.lora), _ptr(tok), _ptr(lab),
                            E, S, seed, q, eps, lr))
        self.q = q

    def step_varlen(self, prob: DeviceProblem, tokens, labels, cu_seqlens, max_len, seed, q, eps, lr):
        """Packed variable-length batch: int32 device tensors tokens/labels [total], cu_seqlens [E+1]."""
        E, total = cu_seqlens.numel() - 1, tokens.numel()
        self._check(zo_step_varlen(self._h, C.byref(prob.weights), C.byref(prob.lora), _ptr(tokens), _ptr(labels),
                                   _ptr(cu_seqlens), E, total, max_len, seed, q, eps, lr))
        self.q = q

    def step_host(self, prob: DeviceProblem, E, S, seed, q, eps, lr):
        self._check(zo_step_host(self._h, C.byref(prob.weights), C.byref(prob.lora),
                                 C.c_void_p(prob.host_tokens.data_ptr()),
                                 C.c_void_p(prob.host_labels.data_ptr()), E, S, seed, q, eps, lr))
        self.q = q

    def losses(self):
        l = np.zeros(2 * self.q, np.float32)
        g = np.zeros(self.q, np.float32)
        self._check(zo_losses(self._h, l.ctypes.data_as(C.c_void_p), g.ctypes.data_as(C.c_void_p)))
        return l, g

    def row_losses(self):
        n = C.c_int32()
        self._check(zo_row_losses(self._h, None, C.byref(n)))
        out = np.zeros((2 * self.q, n.value), np.float32)
        self._check(zo_row_losses(self._h, out.ctypes.data_as(C.c_void_p), C.byref(n)))
        return out

    def set_schedule(self, name):
        self._check(zo_set_schedule(self._h, SCHEDULES[name]))

    def set_query_shard(self, q_begin, q_count):
        """Later steps run only the queries [q_begin, q_begin + q_count) and stop at their losses
        (q_count = 0: whole steps again)."""
        self._check(zo_set_query_shard(self._h, q_begin, q_count))

    def step_pair(self, prob: DeviceProblem, E, S, seed, g_prev, eps, lr, tokens=None, labels=None):
        """One step in the stored-pair form (Algorithm 2, q = 1) on prob.pair (see make_pair);
        g_prev is a device float tensor holding the previous step's g (e.g. g_buffer()) or None."""
        tok = prob.tokens if tokens is None else tokens
        lab = prob.labels if labels is None else labels
        self._check(zo_step_pair(self._h, C.byref(prob.weights), C.byref(prob.pair), _ptr(tok), _ptr(lab),
                                 E, S, seed, _ptr(g_prev), eps, lr))
        self.q = 1

    def pair_collapse(self, prob: DeviceProblem, g_prev, eps, lr):
        self._check(zo_pair_collapse(self._h, C.byref(prob.pair), _ptr(g_prev), eps, lr))

    def g_buffer(self):
        """The context's projected gradients [max_q] as a float32 tensor aliasing the workspace."""
        ptr, cap = C.c_void_p(), C.c_int32()
        self._check(zo_g_buffer(self._h, C.byref(ptr), C.byref(cap)))
        off = ptr.value - self.workspace.data_ptr()
        assert off % 4 == 0 and 0 <= off and off + 4 * cap.value <= self.workspace.numel()
        return self.workspace[off:off + 4 * cap.value].view(torch.float32)

    def test_expire_wait(self, wait_limit_ns):
        """Failure-detection test aid: bounded waits of the tensor-core GEMM give up after
        wait_limit_ns and one is made to run out (0 = normal operation)."""
        self._check(zo_test_expire_wait(self._h, wait_limit_ns))

    def loss_buffer(self):
        """The step's float64 loss array as a tensor aliasing the workspace: [2 * max_q] losses
        followed by the fault slot of a sharded step."""
        ptr, cap = C.c_void_p(), C.c_int32()
        self._check(zo_loss_buffer(self._h, C.byref(ptr), C.byref(cap)))
        off = ptr.value - self.workspace.data_ptr()
        assert off % 8 == 0 and 0 <= off and off + 8 * cap.value <= self.workspace.numel()
        return self.workspace[off:off + 8 * cap.value].view(torch.float64)

    def apply_update(self, prob: DeviceProblem, seed, q, eps, lr):
        self._check(zo_apply_update(self._h, C.byref(prob.lora), seed, q, eps, lr))

    def profile_enable(self, on=True):
        self._check(zo_profile_enable(self._h, int(on)))

    def profile_read(self):
        """{class: (ms, flops, launches)} since the previous read; synchronises the stream."""
        n = len(PROFILE_CLASSES)
        ms, fl, cnt = np.zeros(n), np.zeros(n), np.zeros(n, np.int32)
        self._check(zo_profile_read(self._h, ms.ctypes.data_as(C.c_void_p),
                                    fl.ctypes.data_as(C.c_void_p), cnt.ctypes.data_as(C.c_void_p)))
        return {k: (float(ms[i]), float(fl[i]), int(cnt[i])) for i, k in enumerate(PROFILE_CLASSES)}

    def launch_count(self):
        return int(zo_launch_count(self._h))

    def close(self):
        if self._h:
            zo_free(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def perturbation(seed, tensor_id, query, n, device="cuda"):
    """(raw 32-bit words, normals) of the perturbation stream, as numpy arrays."""
    u = torch.empty(n, dtype=torch.int32, device=device)
    z = torch.empty(n, dtype=torch.float32, device=device)
    st = zo_perturbation(C.c_void_p(torch.cuda.current_stream().cuda_stream), seed, tensor_id, query,
                         n, _ptr(u), _ptr(z))
    if st:
        raise ZoError(st)
    torch.cuda.synchronize()
    return u.cpu().numpy().view(np.uint32), z.cpu().numpy()


_SCRATCH = {}


def mp_lora_linear(X, W, bias, A, B, T, q, scale, seed, tensor_id, eps, x_replicated, flags=0,
                   out=None, sync=True):
    """Y [2q, T, k_out] = MP-LoRA linear of torch device tensors (float32 or bfloat16).  With
    sync=False the call only enqueues (scratch is cached per size; the device status word is
    not read back)."""
    bf = X.dtype == torch.bfloat16
    k_out, k_in = W.shape
    r = A.shape[0]
    Y = torch.empty((2 * q, T, k_out), dtype=X.dtype, device=X.device) if out is None else out
    nb = zo_mp_lora_scratch_bytes(int(bf), T, k_in, k_out, r, q, int(x_replicated))
    key = (X.device, nb)
    if key not in _SCRATCH:
        _SCRATCH.clear()
        _SCRATCH[key] = torch.empty(nb + 256, dtype=torch.uint8, device=X.device)
    scratch = _SCRATCH[key]
    base = (scratch.data_ptr() + 255) // 256 * 256
    st = zo_mp_lora_linear(C.c_void_p(torch.cuda.current_stream().cuda_stream), int(bf), _ptr(X),
                           _ptr(W), _ptr(bias), _ptr(A), _ptr(B), _ptr(Y), T, k_in, k_out, r, scale,
                           seed, tensor_id, q, eps, int(x_replicated), C.c_void_p(base), nb, flags)
    if st:
        raise ZoError(st)
    if sync:
        torch.cuda.synchronize()
        status = int(scratch.view(torch.int32)[(base - scratch.data_ptr()) // 4].item())
        if status:
            raise ZoError(5, f"device status word {status}")
    return Y


def mp_lora_linear_pair(X, W, bias, A, B_pair, T, scale, seed, tensor_id, g_prev, eps, lr, x_replicated, flags=0):
    """The module of Algorithm 2 on its own: updates the stored pair B_pair [2, r, k_out] in place
    (previous update from g_prev, new perturbation from the seed) and returns Y [2, T, k_out]."""
    bf = X.dtype == torch.bfloat16
    k_out, k_in = W.shape
    r = A.shape[0]
    Y = torch.empty((2, T, k_out), dtype=X.dtype, device=X.device)
    nb = zo_mp_lora_scratch_bytes(int(bf), T, k_in, k_out, r, 1, int(x_replicated))
    scratch = torch.empty(nb + 256, dtype=torch.uint8, device=X.device)
    base = (scratch.data_ptr() + 255) // 256 * 256
    st = zo_mp_lora_linear_pair(C.c_void_p(torch.cuda.current_stream().cuda_stream), int(bf), _ptr(X), _ptr(W),
                                _ptr(bias), _ptr(A), _ptr(B_pair), _ptr(Y), T, k_in, k_out, r, scale, seed,
                                tensor_id, g_prev, eps, lr, int(x_replicated), C.c_void_p(base), nb, flags)
    if st:
        raise ZoError(st, "zo_mp_lora_linear_pair")
    torch.cuda.synchronize()
    status = int(scratch.view(torch.int32)[(base - scratch.data_ptr()) // 4].item())
    if status:
        raise ZoError(5, f"device status word {status}")
    return Y


def mp_lora_linear_static(X, W, bias, A, B, Y, T, q, scale, seed, tensor_id, eps, x_replicated, flags=0):
    """The MP-LoRA linear through the entry point that allocates nothing: the caller passes the
    output tensor Y [2q, T, k_out] as well, and the library's built-in scratch is used.  Raises
    ZoError(ZO_ERR_WORKSPACE) when the problem does not fit STATIC_SCRATCH_BYTES."""
    bf = X.dtype == torch.bfloat16
    k_out, k_in = W.shape
    st = zo_mp_lora_linear_static(C.c_void_p(torch.cuda.current_stream().cuda_stream), int(bf), _ptr(X),
                                  _ptr(W), _ptr(bias), _ptr(A), _ptr(B), _ptr(Y), T, k_in, k_out,
                                  A.shape[0], scale, seed, tensor_id, q, eps, int(x_replicated), flags)
    if st:
        raise ZoError(st, "zo_mp_lora_linear_static")
    return Y


def mp_lora_linear_static_status():
    """Waits for the current stream and returns the device status word of the calls made through
    mp_lora_linear_static on the current device (0 = fine); raises ZoError on a timed-out wait."""
    word = C.c_uint32()
    st = zo_mp_lora_linear_static_status(C.c_void_p(torch.cuda.current_stream().cuda_stream), C.byref(word))
    if st:
        raise ZoError(st, f"device status word {word.value}")
    return int(word.value)
