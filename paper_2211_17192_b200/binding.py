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
    h.spec_sample.restype = i32
    h.spec_sample.argtypes = [vp, vp, i32, i32, f32, vp, vp]
    h.spec_uniforms.restype = i32
    h.spec_uniforms.argtypes = [u64, vp, vp, i32, i32, vp, vp]


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
                       n_accepted=None, next_token=None, workspace=None):
    """Speculative sampling for a batch; see `spec_verify_sample` in the header.

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
    _check(lib().spec_verify_sample(
        _ptr(target_logits, torch.float32, "target_logits"),
        _ptr(draft_logits, torch.float32, "draft_logits", optional=True),
        _ptr(draft_tokens, torch.int32, "draft_tokens", optional=True),
        _ptr(uniforms, torch.float32, "uniforms", optional=True),
        batch, gamma, vocab, float(temperature),
        _ptr(n_accepted, torch.int32, "n_accepted"), _ptr(next_token, torch.int32, "next_token"),
        _ptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream()))
    return n_accepted, next_token


def spec_sample(logits, uniforms, temperature, tokens=None):
    """tokens[r] ~ softmax(logits[r] / T) (argmax at T = 0); logits [R, V] fp32 CUDA."""
    rows, vocab = logits.shape
    if tokens is None:
        tokens = torch.empty(rows, dtype=torch.int32, device=logits.device)
    _check(lib().spec_sample(_ptr(logits, torch.float32, "logits"),
                             _ptr(uniforms, torch.float32, "uniforms", optional=True),
                             rows, vocab, float(temperature), _ptr(tokens, torch.int32, "tokens"), _stream()))
    return tokens


def spec_uniforms(seed, positions, sequences, purpose, out=None):
    """The method's uniforms for (position, sequence) pairs; int32 CUDA inputs."""
    count = positions.numel()
    if out is None:
        out = torch.empty(count, dtype=torch.float32, device=positions.device)
    _check(lib().spec_uniforms(int(seed) & 0xFFFFFFFFFFFFFFFF, _ptr(positions, torch.int32, "positions"),
                               _ptr(sequences, torch.int32, "sequences"), int(purpose), count,
                               _ptr(out, torch.float32, "out"), _stream()))
    return out
