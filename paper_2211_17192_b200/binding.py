"""Thin Python binding of the C-ABI library (`include/spec_decode.h`).

Argument marshalling only: every function checks tensor device, dtype and
contiguity, passes raw device pointers and the current torch CUDA stream to the
library, and raises `SpecError` on a non-zero status.  No step of the method
runs in Python or in torch ops.  PyTorch is used for device memory and
streams.  If the shared library has not been built this module raises on first
use: there is no fallback of any kind.
"""

import ctypes
import os

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "lib", "libspecdecode.so")
_lib = None

STATUS_NAMES = {
    0: "SPEC_OK", -1: "SPEC_ERR_BAD_ARG", -2: "SPEC_ERR_BAD_CONFIG", -3: "SPEC_ERR_OOM", -4: "SPEC_ERR_CAPACITY",
    -5: "SPEC_ERR_CUDA", -6: "SPEC_ERR_DEVICE_TIMEOUT", -7: "SPEC_ERR_NONFINITE",
}


class SpecError(RuntimeError):
    def __init__(self, status, message):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


def library_path():
    return _LIB_PATH


def lib():
    """The loaded shared library (loads it on first call)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2211_17192_b200.build` "
                "(there is no fallback path)")
        handle = ctypes.CDLL(_LIB_PATH)
        _declare(handle)
        _lib = handle
    return _lib


def _declare(h):
    c = ctypes
    vp, i32, f32, u64, sz = c.c_void_p, c.c_int, c.c_float, c.c_uint64, c.c_size_t
    h.spec_last_error.restype = c.c_char_p
    h.spec_last_error.argtypes = []
    h.spec_verify_sample_workspace_bytes.restype = sz
    h.spec_verify_sample_workspace_bytes.argtypes = [i32, i32, i32]
    h.spec_verify_sample.restype = i32
    h.spec_verify_sample.argtypes = [vp, vp, vp, vp, i32, i32, i32, f32, vp, vp, vp, sz, vp]
    h.spec_verify_sample_static_capacity.restype = sz
    h.spec_verify_sample_static_capacity.argtypes = []
    h.spec_verify_sample_static.restype = i32
    h.spec_verify_sample_static.argtypes = [vp, vp, vp, vp, i32, i32, i32, f32, vp, vp, vp]
    h.spec_sample.restype = i32
    h.spec_sample.argtypes = [vp, vp, i32, i32, f32, vp, vp]
    h.spec_uniforms.restype = i32
    h.spec_uniforms.argtypes = [u64, vp, vp, i32, i32, vp, vp]
    h.spec_linear_workspace_bytes.restype = sz
    h.spec_linear_workspace_bytes.argtypes = [i32, i32, i32]
    h.spec_linear.restype = i32
    h.spec_linear.argtypes = [vp, vp, i32, i32, i32, i32, i32, vp, vp, sz, vp]
    h.spec_packed_weight_bytes.restype = sz
    h.spec_packed_weight_bytes.argtypes = [i32, i32]
    h.spec_pack_weight.restype = i32
    h.spec_pack_weight.argtypes = [vp, i32, i32, vp, vp]
    h.spec_device_error.restype = i32
    h.spec_device_error.argtypes = []


def _check(status):
    if status != 0:
        raise SpecError(status, lib().spec_last_error().decode())


def _ptr(t, dtype, name, optional=False):
    if t is None:
        if optional:
            return None
        raise ValueError(f"{name} is required")
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise ValueError(f"{name} must be {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def spec_verify_sample_workspace_bytes(batch, gamma, vocab):
    return int(lib().spec_verify_sample_workspace_bytes(batch, gamma, vocab))


def spec_verify_sample(target_logits, draft_logits, draft_tokens, uniforms, temperature,
                       n_accepted=None, next_token=None, workspace=None, lenience=1.0, top_k=0, top_p=1.0):
    """Speculative sampling for a batch; see `spec_verify_sample` (and, for
    lenience < 1, `spec_verify_sample_lenient`; for top_k > 0 or top_p < 1,
    `spec_verify_sample_truncated`) in the header.

    target_logits [B, gamma+1, V] fp32, draft_logits [B, gamma, V] fp32,
    draft_tokens [B, gamma] int32, uniforms [B, gamma+1] fp32, all CUDA.
    Returns (n_accepted [B] int32, next_token [B] int32); asynchronous on the
    current stream.  Output and workspace tensors are allocated when not given.
    """
    batch, rows, vocab = target_logits.shape
    gamma = rows - 1
    dev = target_logits.device
    if n_accepted is None:
        n_accepted = torch.empty(batch, dtype=torch.int32, device=dev)
    if next_token is None:
        next_token = torch.empty(batch, dtype=torch.int32, device=dev)
    need = spec_verify_sample_workspace_bytes(batch, gamma, vocab)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=dev)
    if draft_logits is not None and gamma > 0 and tuple(draft_logits.shape) != (batch, gamma, vocab):
        raise ValueError("draft_logits must be [B, gamma, V]")
    if draft_tokens is not None and gamma > 0 and tuple(draft_tokens.shape) != (batch, gamma):
        raise ValueError("draft_tokens must be [B, gamma]")
    if uniforms is not None and tuple(uniforms.shape) != (batch, gamma + 1):
        raise ValueError("uniforms must be [B, gamma+1]")
    pointers = (_ptr(target_logits, torch.float32, "target_logits"),
                _ptr(draft_logits, torch.float32, "draft_logits", optional=True),
                _ptr(draft_tokens, torch.int32, "draft_tokens", optional=True),
                _ptr(uniforms, torch.float32, "uniforms", optional=True))
    outputs = (_ptr(n_accepted, torch.int32, "n_accepted"), _ptr(next_token, torch.int32, "next_token"),
               _ptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream())
    if top_k or top_p != 1.0:
        h = lib()
        h.spec_verify_sample_truncated.restype = ctypes.c_int
        h.spec_verify_sample_truncated.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_int] * 3 + [ctypes.c_float] * 2 + \
            [ctypes.c_int, ctypes.c_float] + [ctypes.c_void_p] * 3 + [ctypes.c_size_t, ctypes.c_void_p]
        _check(h.spec_verify_sample_truncated(*pointers, batch, gamma, vocab, float(temperature), float(lenience),
                                              int(top_k), float(top_p), *outputs))
    elif lenience == 1.0:
        _check(lib().spec_verify_sample(*pointers, batch, gamma, vocab, float(temperature), *outputs))
    else:
        h = lib()
        h.spec_verify_sample_lenient.restype = ctypes.c_int
        h.spec_verify_sample_lenient.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_int] * 3 + [ctypes.c_float] * 2 + \
            [ctypes.c_void_p] * 3 + [ctypes.c_size_t, ctypes.c_void_p]
        _check(h.spec_verify_sample_lenient(*pointers, batch, gamma, vocab, float(temperature), float(lenience), *outputs))
    return n_accepted, next_token


def spec_verify_sample_static(target_logits, draft_logits, draft_tokens, uniforms, temperature, n_accepted, next_token):
    """`spec_verify_sample` for callers that cannot allocate: same inputs and
    results, the scratch lives in a fixed 1 MiB array inside the library, and the
    outputs must be passed in (nothing is allocated here either).  Shapes whose
    statistics do not fit raise SpecError (SPEC_ERR_CAPACITY).  Calls that may
    overlap on the device must not both use this entry point."""
    batch, rows, vocab = target_logits.shape
    _check(lib().spec_verify_sample_static(
        _ptr(target_logits, torch.float32, "target_logits"),
        _ptr(draft_logits, torch.float32, "draft_logits", optional=True),
        _ptr(draft_tokens, torch.int32, "draft_tokens", optional=True),
        _ptr(uniforms, torch.float32, "uniforms", optional=True),
        batch, rows - 1, vocab, float(temperature),
        _ptr(n_accepted, torch.int32, "n_accepted"), _ptr(next_token, torch.int32, "next_token"), _stream()))
    return n_accepted, next_token


def spec_truncation_floors(logits, temperature, top_k=0, top_p=1.0, floors=None):
    """floors[r] = the lowest logit of row r that top-k and then the nucleus keep; logits [R, V] fp32 CUDA."""
    rows, vocab = logits.shape
    if floors is None:
        floors = torch.empty(rows, dtype=torch.float32, device=logits.device)
    h = lib()
    h.spec_truncation_floors.restype = ctypes.c_int
    h.spec_truncation_floors.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_float, ctypes.c_int,
                                         ctypes.c_float, ctypes.c_void_p, ctypes.c_void_p]
    _check(h.spec_truncation_floors(_ptr(logits, torch.float32, "logits"), rows, vocab, float(temperature), int(top_k),
                                    float(top_p), _ptr(floors, torch.float32, "floors"), _stream()))
    return floors


def spec_sample(logits, uniforms, temperature, tokens=None, top_k=0, top_p=1.0):
    """tokens[r] ~ softmax(logits[r] / T) (argmax at T = 0), over what top-k and the
    nucleus keep of each row when top_k > 0 or top_p < 1; logits [R, V] fp32 CUDA."""
    rows, vocab = logits.shape
    if tokens is None:
        tokens = torch.empty(rows, dtype=torch.int32, device=logits.device)
    if top_k or top_p != 1.0:
        floors = torch.empty(max(rows, 1), dtype=torch.float32, device=logits.device)
        h = lib()
        h.spec_sample_truncated.restype = ctypes.c_int
        h.spec_sample_truncated.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_float,
                                            ctypes.c_int, ctypes.c_float, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        _check(h.spec_sample_truncated(_ptr(logits, torch.float32, "logits"),
                                       _ptr(uniforms, torch.float32, "uniforms", optional=True), rows, vocab,
                                       float(temperature), int(top_k), float(top_p), _ptr(tokens, torch.int32, "tokens"),
                                       _ptr(floors, torch.float32, "floors"), _stream()))
        return tokens
    _check(lib().spec_sample(_ptr(logits, torch.float32, "logits"),
                             _ptr(uniforms, torch.float32, "uniforms", optional=True),
                             rows, vocab, float(temperature), _ptr(tokens, torch.int32, "tokens"), _stream()))
    return tokens


def spec_choose_gamma(alpha, base_cost, cost_per_guess, gamma_max):
    """The gamma in [1, gamma_max] maximising (1 + alpha + ... + alpha^gamma) / (base_cost + cost_per_guess * gamma);
    host arithmetic of the library (no GPU needed)."""
    h = lib()
    h.spec_choose_gamma.restype = ctypes.c_int
    h.spec_choose_gamma.argtypes = [ctypes.c_double, ctypes.c_double, ctypes.c_double, ctypes.c_int]
    g = h.spec_choose_gamma(float(alpha), float(base_cost), float(cost_per_guess), int(gamma_max))
    if g < 0:
        raise ValueError("spec_choose_gamma: alpha in [0, 1], base_cost > 0, cost_per_guess >= 0, gamma_max >= 1")
    return g


def spec_uniforms(seed, positions, sequences, purpose, out=None):
    """The method's uniforms for (position, sequence) pairs; int32 CUDA inputs."""
    count = positions.numel()
    if out is None:
        out = torch.empty(count, dtype=torch.float32, device=positions.device)
    _check(lib().spec_uniforms(int(seed) & 0xFFFFFFFFFFFFFFFF, _ptr(positions, torch.int32, "positions"),
                               _ptr(sequences, torch.int32, "sequences"), int(purpose), count,
                               _ptr(out, torch.float32, "out"), _stream()))
    return out


PATHS = {"auto": 0, "alu": 1, "tensor": 2, "tensor_packed": 3}


def spec_pack_weight(w):
    """Tile-major copy of a bf16 CUDA matrix [n_out, k] (see the header); returns a uint8 tensor."""
    n_out, k = w.shape
    out = torch.empty(int(lib().spec_packed_weight_bytes(n_out, k)), dtype=torch.uint8, device=w.device)
    _check(lib().spec_pack_weight(_ptr(w, torch.bfloat16, "w"), n_out, k, out.data_ptr(), _stream()))
    return out


def spec_linear_workspace_bytes(rows, n_out, k):
    return int(lib().spec_linear_workspace_bytes(rows, n_out, k))


def spec_linear(x, w, path="auto", y=None, workspace=None, n_out=None):
    """y = x . W^T; x [rows, k] fp32 CUDA, w [n_out, k] fp32 or bf16 CUDA -> y [rows, n_out] fp32.
    With path "tensor_packed", w is the uint8 tensor from spec_pack_weight and n_out must be given."""
    rows, k = x.shape
    if path == "tensor_packed":
        if n_out is None:
            raise ValueError("n_out is required with packed weights")
    else:
        n_out = w.shape[0]
        if w.shape[1] != k:
            raise ValueError("inner dimensions differ")
        if w.dtype not in (torch.float32, torch.bfloat16):
            raise ValueError("w must be fp32 or bf16")
    if y is None:
        y = torch.empty((rows, n_out), dtype=torch.float32, device=x.device)
    need = spec_linear_workspace_bytes(rows, n_out, k)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=x.device)
    if not w.is_cuda or not w.is_contiguous():
        raise ValueError("w must be a contiguous CUDA tensor")
    _check(lib().spec_linear(_ptr(x, torch.float32, "x"), w.data_ptr(),
                             1 if (w.dtype == torch.bfloat16 or path == "tensor_packed") else 0,
                             rows, n_out, k, PATHS[path], _ptr(y, torch.float32, "y"),
                             _ptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream()))
    return y


def spec_linear_partials(x, w_packed, n_out, workspace, split_input=True, rows=None, k=None):
    """The engine's tensor-core GEMM alone on tile-major weights: returns a view
    [splits, rows, n_out] of the split-K partial sums inside `workspace` (their sum
    over the first axis is x . W^T).  split_input=False reuses the bf16 split of x that
    an earlier call with the same (rows, k, workspace) left there (x may then be None)."""
    h = lib()
    if x is not None:
        rows, k = x.shape
    h.spec_linear_partials.restype = ctypes.c_int
    h.spec_linear_partials.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                       ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t,
                                       ctypes.POINTER(ctypes.c_void_p), ctypes.POINTER(ctypes.c_int), ctypes.c_void_p]
    where, splits = ctypes.c_void_p(), ctypes.c_int()
    _check(h.spec_linear_partials(_ptr(x, torch.float32, "x") if x is not None else None, w_packed.data_ptr(), rows,
                                  n_out, k, 1 if split_input else 0, _ptr(workspace, torch.uint8, "workspace"),
                                  workspace.numel(), ctypes.byref(where), ctypes.byref(splits), _stream()))
    offset = where.value - workspace.data_ptr()
    count = splits.value * rows * n_out
    return workspace[offset:offset + 4 * count].view(torch.float32).view(splits.value, rows, n_out)


def spec_device_error():
    return int(lib().spec_device_error())


# --------------------------------------------------------------------------- #
# models and generation
# --------------------------------------------------------------------------- #
class _ModelCfg(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("arch", "n_layers", "d_model", "n_heads", "n_kv_heads", "d_head", "d_ff",
                                            "ffn", "vocab", "max_positions", "tied_embeddings", "dtype")] + \
               [("rms_eps", ctypes.c_float), ("rope_base", ctypes.c_float)] + \
               [(n, ctypes.c_int) for n in ("n_enc_layers", "rel_buckets", "rel_max_distance", "ngram")]


class _LayerWeights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("ln1", "wqkv", "wo", "ln2", "w_in", "w_out",
                                               "lnx", "wq_x", "wkv_x", "wo_x")]


class _Weights(ctypes.Structure):
    _fields_ = [("tok_emb", ctypes.c_void_p), ("pos_emb", ctypes.c_void_p), ("ln_f", ctypes.c_void_p),
                ("head", ctypes.c_void_p), ("layers", ctypes.POINTER(_LayerWeights)),
                ("enc_layers", ctypes.POINTER(_LayerWeights)), ("enc_ln_f", ctypes.c_void_p),
                ("enc_rel_bias", ctypes.c_void_p), ("rel_bias", ctypes.c_void_p)]


class _RuntimeCfg(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("max_batch", "max_len", "page_size", "max_gamma", "kv_dtype",
                                            "max_src_len", "pass_kernel")]


class _Stats(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in ("iterations", "tokens", "tests_evaluated", "tests_passed",
                                              "target_passes", "draft_passes")] + \
               [("prefill_ms", ctypes.c_double), ("decode_ms", ctypes.c_double), ("accepted_histogram", ctypes.c_int64 * 65)]


def _stats_dict(st):
    d = {name: getattr(st, name) for name, _ in _Stats._fields_}
    d["accepted_histogram"] = list(st.accepted_histogram)
    return d


_ARCH = {"gpt": 0, "llama": 1, "t5": 2, "bigram": 3, "copy": 4}
_FFN = {"gelu": 0, "gated_gelu": 1, "swiglu": 2}
_DTYPE = {"fp32": 0, "bf16": 1, "fp16": 2}
_engine_declared = False


def _declare_engine(h):
    global _engine_declared
    if _engine_declared:
        return
    c = ctypes
    vp = c.c_void_p
    h.spec_init.restype = c.c_int
    h.spec_init.argtypes = [c.POINTER(_ModelCfg), c.POINTER(_ModelCfg), c.POINTER(_Weights), c.POINTER(_Weights),
                            c.POINTER(_RuntimeCfg), c.POINTER(vp)]
    h.spec_free.restype = None
    h.spec_free.argtypes = [vp]
    h.spec_generate.restype = c.c_int
    h.spec_generate.argtypes = [vp, vp, vp, c.c_int, c.c_int, c.c_int, c.c_int, c.c_float, c.c_uint64, vp,
                                c.POINTER(_Stats)]
    h.spec_begin.restype = c.c_int
    h.spec_begin.argtypes = [vp, vp, vp, c.c_int, c.c_int, c.c_int, c.c_int, c.c_float, c.c_uint64]
    h.spec_step.restype = c.c_int
    h.spec_step.argtypes = [vp, c.c_int, c.POINTER(c.c_int), c.POINTER(_Stats)]
    h.spec_read_tokens.restype = c.c_int
    h.spec_read_tokens.argtypes = [vp, vp]
    h.spec_reset.restype = c.c_int
    h.spec_reset.argtypes = [vp]
    h.spec_truncate.restype = c.c_int
    h.spec_truncate.argtypes = [vp, c.c_int, vp, c.c_int]
    h.spec_forward_logits.restype = c.c_int
    h.spec_forward_logits.argtypes = [vp, c.c_int, vp, c.c_int, c.c_int, vp]
    h.spec_set_lenience.restype = c.c_int
    h.spec_set_lenience.argtypes = [vp, c.c_float]
    h.spec_set_truncation.restype = c.c_int
    h.spec_set_truncation.argtypes = [vp, c.c_int, c.c_float]
    h.spec_set_imposed_acceptance.restype = c.c_int
    h.spec_set_imposed_acceptance.argtypes = [vp, c.c_float]
    h.spec_time_forward.restype = c.c_int
    h.spec_time_forward.argtypes = [vp, c.c_int, c.c_int, c.c_int, c.c_int, c.POINTER(c.c_float)]
    h.spec_encode.restype = c.c_int
    h.spec_encode.argtypes = [vp, vp, vp, c.c_int, c.c_int]
    _engine_declared = True


def _cfg_struct(cfg):
    if cfg["arch"] == "bigram":  # only arch, vocab and dtype are read
        return _ModelCfg(_ARCH["bigram"], 0, 0, 0, 0, 0, 0, 0, cfg["vocab"], 0, 0, _DTYPE[cfg["dtype"]], 0.0, 0.0, 0, 0, 0, 0)
    if cfg["arch"] == "copy":  # only arch, vocab and ngram are read
        return _ModelCfg(_ARCH["copy"], 0, 0, 0, 0, 0, 0, 0, cfg["vocab"], 0, 0, 0, 0.0, 0.0, 0, 0, 0, cfg["ngram"])
    return _ModelCfg(_ARCH[cfg["arch"]], cfg["n_layers"], cfg["d_model"], cfg["n_heads"], cfg["n_kv_heads"],
                     cfg["d_head"], cfg["d_ff"], _FFN[cfg["ffn"]], cfg["vocab"], cfg["max_positions"],
                     1 if cfg["tied"] else 0, _DTYPE[cfg["dtype"]], cfg["rms_eps"], cfg["rope_base"],
                     cfg.get("n_enc_layers", 0), cfg.get("rel_buckets", 0), cfg.get("rel_max_distance", 0), 0)


class Engine:
    """A target model, an optional draft model and their KV caches on one GPU.

    `*_cfg` are the dicts of `workloads.model_config`, `*_weights` dicts of
    arrays (numpy or CUDA tensors) by the names of `workloads.tensor_shapes`.
    Weights are uploaded once (bf16 models as bf16) and kept alive here; the
    library borrows the pointers.
    """

    def __init__(self, target_cfg, target_weights, draft_cfg=None, draft_weights=None, max_batch=1, max_len=256,
                 page_size=64, max_gamma=8, kv_dtype=None, device=None, max_src_len=0, pass_kernel=False):
        import numpy as np
        self._np = np
        h = lib()
        _declare_engine(h)
        if kv_dtype is None:  # cached K,V rows: fp16 for bf16 models (inside their logit tolerance), fp32 for fp32 models
            kv_dtype = "fp16" if target_cfg["dtype"] == "bf16" else "fp32"
        self.kv_dtype = kv_dtype
        self.device = torch.device("cuda", torch.cuda.current_device()) if device is None else device
        self.cfgs = [target_cfg, draft_cfg]
        self._keep = []
        structs = []
        for cfg, weights in ((target_cfg, target_weights), (draft_cfg, draft_weights)):
            structs.append(None if cfg is None else self._upload(cfg, weights))
        rt = _RuntimeCfg(max_batch, max_len, page_size, max_gamma, _DTYPE[kv_dtype], max_src_len, 1 if pass_kernel else 0)
        self.max_batch, self.max_len, self.max_gamma = max_batch, max_len, max_gamma
        ctx = ctypes.c_void_p()
        tc = _cfg_struct(target_cfg)
        dc = _cfg_struct(draft_cfg) if draft_cfg is not None else None
        _check(h.spec_init(ctypes.byref(tc), ctypes.byref(dc) if dc is not None else None,
                           ctypes.byref(structs[0]), ctypes.byref(structs[1]) if structs[1] is not None else None,
                           ctypes.byref(rt), ctypes.byref(ctx)))
        self._ctx = ctx

    def _upload(self, cfg, weights):
        bf16 = cfg["dtype"] == "bf16"

        def dev(name, matrix):
            a = weights[name]
            t = a if isinstance(a, torch.Tensor) else torch.from_numpy(self._np.ascontiguousarray(a))
            t = t.to(self.device)
            t = t.to(torch.bfloat16 if (bf16 and matrix) else torch.float32).contiguous()
            self._keep.append(t)
            return t.data_ptr()

        if cfg["arch"] == "bigram":
            return _Weights(dev("table", True), None, None, None, None, None, None, None, None)
        if cfg["arch"] == "copy":
            return _Weights(None, None, None, None, None, None, None, None, None)
        t5 = cfg["arch"] == "t5"

        def block(p, cross):
            extra = (dev(p + "lnx", False), dev(p + "wq_x", True), dev(p + "wkv_x", True), dev(p + "wo_x", True)) \
                if cross else (None, None, None, None)
            return _LayerWeights(dev(p + "ln1", False), dev(p + "wqkv", True), dev(p + "wo", True),
                                 dev(p + "ln2", False), dev(p + "w_in", True), dev(p + "w_out", True), *extra)

        layers = (_LayerWeights * cfg["n_layers"])()
        for l in range(cfg["n_layers"]):
            layers[l] = block(f"l{l}.", t5)
        self._keep.append(layers)
        enc_layers = None
        if t5:
            enc_layers = (_LayerWeights * cfg["n_enc_layers"])()
            for l in range(cfg["n_enc_layers"]):
                enc_layers[l] = block(f"enc.l{l}.", False)
            self._keep.append(enc_layers)
        return _Weights(dev("tok_emb", True), dev("pos_emb", True) if cfg["arch"] == "gpt" else None,
                        dev("ln_f", False), None if cfg["tied"] else dev("head", True), layers,
                        enc_layers, dev("enc.ln_f", False) if t5 else None,
                        dev("enc.rel_bias", False) if t5 else None, dev("rel_bias", False) if t5 else None)

    def close(self):
        if getattr(self, "_ctx", None):
            lib().spec_free(self._ctx)
            self._ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _pack_prompts(self, prompts):
        np = self._np
        stride = max(len(p) for p in prompts)
        flat = np.zeros((len(prompts), stride), dtype=np.int32)
        lens = np.zeros(len(prompts), dtype=np.int32)
        for b, p in enumerate(prompts):
            flat[b, : len(p)] = p
            lens[b] = len(p)
        return flat, lens, stride

    def begin(self, prompts, n_new, gamma, temperature, seed):
        """Prompt pass of a generation that `step` then advances."""
        flat, lens, stride = self._pack_prompts(prompts)
        _check(lib().spec_begin(self._ctx, flat.ctypes.data, lens.ctypes.data, stride, len(prompts), n_new, gamma,
                                float(temperature), int(seed) & 0xFFFFFFFFFFFFFFFF))
        self._session = (len(prompts), n_new)

    def step(self, iterations):
        """`iterations` iterations of Algorithm 1; returns (remaining, stats dict)."""
        left = ctypes.c_int()
        st = _Stats()
        _check(lib().spec_step(self._ctx, iterations, ctypes.byref(left), ctypes.byref(st)))
        return left.value, _stats_dict(st)

    def read_tokens(self):
        batch, n_new = self._session
        out = self._np.zeros((batch, n_new), dtype=self._np.int32)
        _check(lib().spec_read_tokens(self._ctx, out.ctypes.data))
        return out

    def generate(self, prompts, n_new, gamma, temperature, seed):
        """Speculative decoding (gamma = 0: target-only decoding).  `prompts` is a
        list of 1-D int arrays; returns (tokens [B, n_new] int32 numpy, stats dict)."""
        np = self._np
        batch = len(prompts)
        stride = max(len(p) for p in prompts)
        flat = np.zeros((batch, stride), dtype=np.int32)
        lens = np.zeros(batch, dtype=np.int32)
        for b, p in enumerate(prompts):
            flat[b, : len(p)] = p
            lens[b] = len(p)
        out = np.zeros((batch, n_new), dtype=np.int32)
        st = _Stats()
        _check(lib().spec_generate(self._ctx, flat.ctypes.data, lens.ctypes.data, stride, batch, n_new, gamma,
                                   float(temperature), int(seed) & 0xFFFFFFFFFFFFFFFF, out.ctypes.data,
                                   ctypes.byref(st)))
        return out, _stats_dict(st)

    def generate_adaptive(self, prompts, n_new, gamma_max, temperature, seed, burst=4):
        """`generate` with gamma chosen by the library burst by burst (`spec_generate_adaptive`).
        Returns (tokens [B, n_new], stats dict, trace): trace is the list of (gamma, iterations) per burst."""
        np = self._np
        batch = len(prompts)
        lens = np.array([len(p) for p in prompts], dtype=np.int32)
        stride = int(lens.max())
        flat = np.zeros((batch, stride), dtype=np.int32)
        for b, p in enumerate(prompts):
            flat[b, : len(p)] = np.asarray(p, dtype=np.int32)
        out = np.zeros((batch, n_new), dtype=np.int32)
        capacity = 2 * (n_new + 2)  # every burst emits at least one token per unfinished sequence
        trace = np.zeros(capacity, dtype=np.int32)
        n_bursts = ctypes.c_int(0)
        st = _Stats()
        h = lib()
        h.spec_generate_adaptive.restype = ctypes.c_int
        h.spec_generate_adaptive.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int,
                                             ctypes.c_int, ctypes.c_int, ctypes.c_float, ctypes.c_uint64, ctypes.c_int,
                                             ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p]
        _check(h.spec_generate_adaptive(self._ctx, flat.ctypes.data, lens.ctypes.data, stride, batch, n_new, gamma_max,
                                        float(temperature), int(seed) & 0xFFFFFFFFFFFFFFFF, int(burst), out.ctypes.data,
                                        ctypes.byref(st), trace.ctypes.data, capacity, ctypes.byref(n_bursts)))
        pairs = [(int(trace[2 * i]), int(trace[2 * i + 1])) for i in range(min(n_bursts.value, capacity // 2))]
        return out, _stats_dict(st), pairs

    def set_gamma(self, gamma):
        """Number of guesses per iteration for the rest of the generation in progress (`spec_set_gamma`)."""
        h = lib()
        h.spec_set_gamma.restype = ctypes.c_int
        h.spec_set_gamma.argtypes = [ctypes.c_void_p, ctypes.c_int]
        _check(h.spec_set_gamma(self._ctx, int(gamma)))

    def set_lenience(self, lenience):
        """Lenience factor of Appendix A.5 for the generations that follow (1 = Algorithm 1)."""
        _check(lib().spec_set_lenience(self._ctx, float(lenience)))

    def set_truncation(self, top_k=0, top_p=1.0):
        """Top-k and nucleus standardisation (Section 2.2) of both models for the generations
        that follow; top_k = 0 and top_p = 1 switch them off."""
        _check(lib().spec_set_truncation(self._ctx, int(top_k), float(top_p)))

    def set_imposed_acceptance(self, alpha):
        """Timing instrument: accept every drafted token with probability `alpha`
        (i.i.d., from the same uniforms) instead of by Algorithm 1's test; None or a
        negative value restores the algorithm."""
        _check(lib().spec_set_imposed_acceptance(self._ctx, -1.0 if alpha is None else float(alpha)))

    def encode(self, sources):
        """Encoder-decoder models: run the encoders over `sources` (list of 1-D int
        arrays) and keep the cross-attention K,V; clears the decoder caches."""
        flat, lens, stride = self._pack_prompts(sources)
        _check(lib().spec_encode(self._ctx, flat.ctypes.data, lens.ctypes.data, stride, len(sources)))

    def reset(self):
        _check(lib().spec_reset(self._ctx))

    def truncate(self, which, lengths):
        a = self._np.ascontiguousarray(lengths, dtype=self._np.int32)
        _check(lib().spec_truncate(self._ctx, which, a.ctypes.data, a.shape[0]))

    def attention_plan(self, which, batch, rows, cross=False):
        """How the attention of such a pass is launched (`spec_attention_plan`): dict with
        tensor_cores, slices, cluster_merge, in_turn."""
        h = lib()
        h.spec_attention_plan.restype = ctypes.c_int
        h.spec_attention_plan.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                          ctypes.POINTER(ctypes.c_int)]
        plan = (ctypes.c_int * 4)()
        _check(h.spec_attention_plan(self._ctx, which, batch, rows, 1 if cross else 0, plan))
        return dict(tensor_cores=bool(plan[0]), f16=plan[0] == 2, slices=int(plan[1]), cluster_merge=bool(plan[2]),
                    in_turn=bool(plan[3]))

    def pass_trace(self, which, batch, rows, capacity=65536):
        """The CTAs' clocks at the grid barriers of one persistent-kernel pass (`spec_pass_trace`):
        returns (start_ns, arrivals) with arrivals a numpy int64 array [barriers, CTAs]."""
        h = lib()
        h.spec_pass_trace.restype = ctypes.c_int
        h.spec_pass_trace.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_int,
                                      ctypes.POINTER(ctypes.c_int)]
        out = self._np.zeros(capacity, dtype=self._np.uint64)
        count = ctypes.c_int()
        _check(h.spec_pass_trace(self._ctx, which, batch, rows, out.ctypes.data, capacity, ctypes.byref(count)))
        ctas = int(out[0])
        barriers = (count.value - 2) // ctas
        return int(out[1]), out[2:2 + barriers * ctas].astype(self._np.int64).reshape(barriers, ctas)

    def time_forward(self, which, batch, rows, repeats=20):
        """Device time (ms) of one pass of model `which` over `rows` rows per sequence at
        the current cached lengths, graph-replayed `repeats` times; the caches keep their lengths."""
        ms = ctypes.c_float()
        _check(lib().spec_time_forward(self._ctx, which, batch, rows, repeats, ctypes.byref(ms)))
        return ms.value

    def forward_logits(self, which, tokens):
        """Teacher-forced pass: tokens [B, rows] are appended at the cached
        lengths of model `which` (0 target, 1 draft); returns fp32 logits
        [B, rows, vocab] as a CUDA tensor."""
        a = self._np.ascontiguousarray(tokens, dtype=self._np.int32)
        batch, rows = a.shape
        vocab = self.cfgs[which]["vocab"]
        out = torch.empty((batch, rows, vocab), dtype=torch.float32, device=self.device)
        _check(lib().spec_forward_logits(self._ctx, which, a.ctypes.data, batch, rows, out.data_ptr()))
        return out
