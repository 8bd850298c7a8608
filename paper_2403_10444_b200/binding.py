"""ctypes binding of libbv_b200.so: argument marshalling only.

Every step of the verification path runs inside the CUDA library; nothing here
computes.  There is no CPU fallback: if the library is missing, or an entry
point reports an error, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libbv_b200.so")

DTYPE_F32 = 0
DTYPE_BF16 = 1

# every symbol include/bv.h declares
EXPORTS = ["bv_verify", "tv_verify", "bv_verify_ex", "tv_verify_ex", "bv_verify_host",
           "tv_verify_host", "bv_verify_noalloc", "bv_verify_lse", "bv_verify_lse_ex", "tv_verify_lse", "tv_verify_lse_ex", "gbv_verify", "gbv_verify_ex", "bv_verify_probs", "tv_verify_probs", "bv_sample_draft", "bv_draft_chain", "bv_stream_status", "bv_set_option", "bv_release", "bv_last_launch_count", "bv_last_kernel", "bv_last_cuda_error",
           "bv_status_string", "bv_version"]


class BVError(RuntimeError):
    """An entry point of libbv_b200.so returned a non-zero status."""

    def __init__(self, status: int, text: str):
        super().__init__("libbv_b200: %s (status %d)" % (text, status))
        self.status = status


_lib = None


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """Load libbv_b200.so (built by ``python -m paper_2403_10444_b200.build``)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or _LIB_PATH
    if not os.path.exists(p):
        raise RuntimeError(
            "CUDA library %s is missing: build it with `python -m paper_2403_10444_b200.build` "
            "(there is no CPU fallback)" % p)
    lib = ctypes.CDLL(p)
    vp, ci, cf = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
    base = [vp, vp, vp, vp, ci, ci, ci, ci, cf, vp, vp]
    for name in ("bv_verify", "tv_verify", "bv_verify_noalloc", "gbv_verify"):
        getattr(lib, name).argtypes = base + [vp]
    for name in ("bv_verify_ex", "tv_verify_ex", "gbv_verify_ex"):
        getattr(lib, name).argtypes = base + [vp, vp, vp, vp, vp, vp]
    for name in ("bv_verify_host", "tv_verify_host"):
        getattr(lib, name).argtypes = base
    lib.bv_sample_draft.argtypes = [vp, vp, ci, ci, ci, cf, vp, vp, vp]
    lib.bv_draft_chain.argtypes = [vp, vp, vp, ci, ci, ci, ci, cf, vp, vp, vp]
    for name in ("bv_verify_probs", "tv_verify_probs"):
        getattr(lib, name).argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, vp, vp, vp, vp, vp, vp]
    for name in ("bv_verify_lse", "tv_verify_lse"):
        getattr(lib, name).argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, cf, vp, vp, vp]
        getattr(lib, name + "_ex").argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, cf, vp, vp, vp, vp, vp, vp, vp, vp]
    for name in EXPORTS:
        getattr(lib, name).restype = ci
    lib.bv_stream_status.argtypes = [vp]
    lib.bv_set_option.argtypes = [ctypes.c_char_p, ci]
    lib.bv_status_string.restype = ctypes.c_char_p
    lib.bv_status_string.argtypes = [ci]
    if path is None:
        _lib = lib
    return lib


def bv_status_string(status: int) -> str:
    return load_library().bv_status_string(int(status)).decode()


def bv_version() -> int:
    return int(load_library().bv_version())


def bv_last_launch_count() -> int:
    return int(load_library().bv_last_launch_count())


def bv_last_kernel() -> int:
    """Code of the kernel the last verification call on this thread launched (1 flow, 2 cluster,
    3 element-wise streaming, 4 small-batch)."""
    return int(load_library().bv_last_kernel())


def bv_release() -> None:
    _check(load_library().bv_release())


def bv_set_option(name: str, value: int) -> None:
    """Process-wide tuning / test option of the library (see include/bv.h); 0 restores the default."""
    _check(load_library().bv_set_option(name.encode(), int(value)))


def bv_stream_status(stream=None) -> int:
    """Waits for the stream and returns 0, or -4 if a device-side wait of a call on it gave up."""
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(load_library().bv_stream_status(ctypes.c_void_p(s.cuda_stream)))


def _check(status: int) -> None:
    if status != 0:
        lib = load_library()
        text = lib.bv_status_string(int(status)).decode()
        if status == -3:
            text += " (cudaError %d)" % lib.bv_last_cuda_error()
        raise BVError(status, text)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return DTYPE_F32
    if t.dtype == torch.bfloat16:
        return DTYPE_BF16
    raise TypeError("logits must be float32 or bfloat16, got %s" % t.dtype)


def _shapes(target, draft, tokens, uniforms, want_cuda: bool):
    if target.dim() != 3 or draft.dim() != 3:
        raise ValueError("target_logits must be [B, gamma+1, V] and draft_logits [B, gamma, V]")
    B, g1, V = target.shape
    gamma = g1 - 1
    if tuple(draft.shape) != (B, gamma, V):
        raise ValueError("draft_logits must be [B, gamma, V]")
    if tuple(tokens.shape) != (B, gamma) or tokens.dtype != torch.int32:
        raise ValueError("draft_tokens must be int32 [B, gamma]")
    if tuple(uniforms.shape) != (B, gamma + 2) or uniforms.dtype != torch.float32:
        raise ValueError("uniforms must be float32 [B, gamma+2]")
    if target.dtype != draft.dtype:
        raise TypeError("target and draft logits must share a dtype")
    for t in (target, draft, tokens, uniforms):
        if not t.is_contiguous():
            raise ValueError("all tensors must be contiguous")
        if t.is_cuda != want_cuda:
            raise ValueError("expected %s tensors" % ("CUDA" if want_cuda else "host"))
    return B, gamma, V


def _device_call(name: str, target, draft, tokens, uniforms, temperature, diagnostics: bool,
                 stream: Optional[torch.cuda.Stream]):
    lib = load_library()
    B, gamma, V = _shapes(target, draft, tokens, uniforms, True)
    dev = target.device
    out_tokens = torch.empty((B, gamma + 1), dtype=torch.int32, device=dev)
    out_len = torch.empty((B,), dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        s = stream if stream is not None else torch.cuda.current_stream(dev)
        args = [target.data_ptr(), draft.data_ptr(), tokens.data_ptr(), uniforms.data_ptr(),
                B, gamma, V, _dtype_code(target), float(temperature),
                out_tokens.data_ptr(), out_len.data_ptr()]
        if diagnostics:
            f = lambda *shape: torch.empty(shape, dtype=torch.float32, device=dev)
            diag = dict(p=f(B, gamma + 1), S=f(B, gamma), h=f(B, gamma + 1),
                        lse_t=f(B, gamma + 1), lse_d=f(B, gamma))
            args += [diag[k].data_ptr() for k in ("p", "S", "h", "lse_t", "lse_d")]
        _check(getattr(lib, name)(*args, s.cuda_stream))
    if diagnostics:
        return out_tokens, out_len, diag
    return out_tokens, out_len


def bv_verify(target_logits, draft_logits, draft_tokens, uniforms, temperature: float = 1.0,
              stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Block Verification (Algorithm 2) on CUDA tensors; returns (out_tokens, out_len)."""
    return _device_call("bv_verify", target_logits, draft_logits, draft_tokens, uniforms,
                        temperature, False, stream)


def tv_verify(target_logits, draft_logits, draft_tokens, uniforms, temperature: float = 1.0,
              stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Token Verification (Algorithm 1) on CUDA tensors; returns (out_tokens, out_len)."""
    return _device_call("tv_verify", target_logits, draft_logits, draft_tokens, uniforms,
                        temperature, False, stream)


def bv_verify_ex(target_logits, draft_logits, draft_tokens, uniforms, temperature: float = 1.0,
                 stream=None):
    """bv_verify plus its intermediates: returns (out_tokens, out_len, dict(p, S, h, lse_t, lse_d))."""
    return _device_call("bv_verify_ex", target_logits, draft_logits, draft_tokens, uniforms,
                        temperature, True, stream)


def tv_verify_ex(target_logits, draft_logits, draft_tokens, uniforms, temperature: float = 1.0,
                 stream=None):
    """tv_verify plus its intermediates (NaN where Algorithm 1 forms none)."""
    return _device_call("tv_verify_ex", target_logits, draft_logits, draft_tokens, uniforms,
                        temperature, True, stream)


def gbv_verify(target_logits, draft_logits, draft_tokens, uniforms, temperature: float = 1.0,
               stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Greedy Block Verification, one iteration (Algorithm 4), on CUDA tensors; returns
    (out_tokens, out_len).  Rows must be whole 16-byte vectors."""
    return _device_call("gbv_verify", target_logits, draft_logits, draft_tokens, uniforms,
                        temperature, False, stream)


def gbv_verify_ex(target_logits, draft_logits, draft_tokens, uniforms, temperature: float = 1.0,
                  stream=None):
    """gbv_verify plus its intermediates: p holds the unclipped products, S the numerator sums of
    the acceptance ratios, h the ratios (above one, or +inf, where the test passes with certainty)."""
    return _device_call("gbv_verify_ex", target_logits, draft_logits, draft_tokens, uniforms,
                        temperature, True, stream)


def _probs_call(name: str, target_probs, draft_probs, tokens, uniforms, diagnostics: bool, stream):
    lib = load_library()
    B, gamma, V = _shapes(target_probs, draft_probs, tokens, uniforms, True)
    dev = target_probs.device
    out_tokens = torch.empty((B, gamma + 1), dtype=torch.int32, device=dev)
    out_len = torch.empty((B,), dtype=torch.int32, device=dev)
    diag, ptrs = None, [None, None, None]
    if diagnostics:
        f = lambda *shape: torch.empty(shape, dtype=torch.float32, device=dev)
        diag = dict(p=f(B, gamma + 1), S=f(B, gamma), h=f(B, gamma + 1))
        ptrs = [diag[k].data_ptr() for k in ("p", "S", "h")]
    with torch.cuda.device(dev):
        s = stream if stream is not None else torch.cuda.current_stream(dev)
        _check(getattr(lib, name)(target_probs.data_ptr(), draft_probs.data_ptr(), tokens.data_ptr(),
                                  uniforms.data_ptr(), B, gamma, V, _dtype_code(target_probs),
                                  out_tokens.data_ptr(), out_len.data_ptr(), *ptrs, s.cuda_stream))
    return (out_tokens, out_len, diag) if diagnostics else (out_tokens, out_len)


def bv_verify_probs(target_probs, draft_probs, draft_tokens, uniforms, diagnostics: bool = False, stream=None):
    """Block Verification (Algorithm 2) on given probabilities [B, gamma+1, V] / [B, gamma, V] (CUDA,
    float32 or bfloat16, used as stored); returns (out_tokens, out_len) and, with ``diagnostics``,
    dict(p, S, h)."""
    return _probs_call("bv_verify_probs", target_probs, draft_probs, draft_tokens, uniforms, diagnostics, stream)


def tv_verify_probs(target_probs, draft_probs, draft_tokens, uniforms, diagnostics: bool = False, stream=None):
    """Token Verification (Algorithm 1) on given probabilities; see bv_verify_probs."""
    return _probs_call("tv_verify_probs", target_probs, draft_probs, draft_tokens, uniforms, diagnostics, stream)


def bv_verify_noalloc(target_logits, draft_logits, draft_tokens, uniforms, out_tokens, out_len,
                      temperature: float = 1.0, stream=None) -> None:
    """Block Verification through the entry point that allocates nothing.

    For embedders that cannot let the library allocate device memory when they call it
    (a memory pool that owns the device, possible stream capture, allocator hooks).  The
    caller supplies the outputs: ``out_tokens`` int32 [B, gamma+1] and ``out_len`` int32 [B],
    CUDA tensors; this wrapper creates no tensor either.  Raises BVError(status -5) when the
    problem needs more than the library's fixed 8 MiB scratch array.
    """
    lib = load_library()
    B, gamma, V = _shapes(target_logits, draft_logits, draft_tokens, uniforms, True)
    if tuple(out_tokens.shape) != (B, gamma + 1) or out_tokens.dtype != torch.int32 or not out_tokens.is_cuda:
        raise ValueError("out_tokens must be a CUDA int32 tensor [B, gamma+1]")
    if tuple(out_len.shape) != (B,) or out_len.dtype != torch.int32 or not out_len.is_cuda:
        raise ValueError("out_len must be a CUDA int32 tensor [B]")
    dev = target_logits.device
    with torch.cuda.device(dev):
        s = stream if stream is not None else torch.cuda.current_stream(dev)
        _check(lib.bv_verify_noalloc(target_logits.data_ptr(), draft_logits.data_ptr(),
                                     draft_tokens.data_ptr(), uniforms.data_ptr(), B, gamma, V,
                                     _dtype_code(target_logits), float(temperature),
                                     out_tokens.data_ptr(), out_len.data_ptr(), s.cuda_stream))


def _host_call(name: str, target, draft, tokens, uniforms, temperature, out_tokens, out_len):
    lib = load_library()
    B, gamma, V = _shapes(target, draft, tokens, uniforms, False)
    if out_tokens is None:
        out_tokens = torch.empty((B, gamma + 1), dtype=torch.int32).pin_memory()
    if out_len is None:
        out_len = torch.empty((B,), dtype=torch.int32).pin_memory()
    _check(getattr(lib, name)(target.data_ptr(), draft.data_ptr(), tokens.data_ptr(),
                              uniforms.data_ptr(), B, gamma, V, _dtype_code(target),
                              float(temperature), out_tokens.data_ptr(), out_len.data_ptr()))
    return out_tokens, out_len


def bv_verify_host(target_logits, draft_logits, draft_tokens, uniforms, temperature: float = 1.0,
                   out_tokens=None, out_len=None):
    """Block Verification on HOST tensors (pinned for speed): copies in, runs, copies out."""
    return _host_call("bv_verify_host", target_logits, draft_logits, draft_tokens, uniforms,
                      temperature, out_tokens, out_len)


def tv_verify_host(target_logits, draft_logits, draft_tokens, uniforms, temperature: float = 1.0,
                   out_tokens=None, out_len=None):
    """Token Verification on HOST tensors (pinned for speed): copies in, runs, copies out."""
    return _host_call("tv_verify_host", target_logits, draft_logits, draft_tokens, uniforms,
                      temperature, out_tokens, out_len)


def bv_sample_draft(logits, uniforms, temperature: float = 1.0, want_lse: bool = True, stream=None):
    """The drafting step of Algorithm 3 on CUDA tensors: logits [rows, V] (float32 or bfloat16),
    uniforms [rows] float32.  Returns (tokens int32 [rows], lse float32 [rows] or None)."""
    if not (logits.is_cuda and uniforms.is_cuda):
        raise ValueError("bv_sample_draft takes CUDA tensors")
    if logits.dim() != 2 or not logits.is_contiguous():
        raise ValueError("logits must be a contiguous [rows, V] tensor")
    rows, V = logits.shape
    if uniforms.shape != (rows,) or uniforms.dtype != torch.float32 or not uniforms.is_contiguous():
        raise ValueError("uniforms must be a contiguous float32 tensor of [rows]")
    lib = load_library()
    tokens = torch.empty((rows,), dtype=torch.int32, device=logits.device)
    lse = torch.empty((rows,), dtype=torch.float32, device=logits.device) if want_lse else None
    st = stream if stream is not None else torch.cuda.current_stream(logits.device)
    with torch.cuda.device(logits.device):
        _check(lib.bv_sample_draft(logits.data_ptr(), uniforms.data_ptr(), rows, V, _dtype_code(logits),
                                   float(temperature), tokens.data_ptr(), lse.data_ptr() if want_lse else None,
                                   st.cuda_stream))
    return tokens, lse


def bv_draft_chain(draft_table, first_tokens, uniforms, temperature: float = 1.0, stream=None):
    """The whole drafting step for a last-token table model: draft_table CUDA [V, V] float32 or bfloat16,
    first_tokens CUDA int32 [B], uniforms CUDA float32 [gamma, B]; returns (tokens int32 [B, gamma],
    lse float32 [B, gamma]) from one launch."""
    lib = load_library()
    V = draft_table.shape[0]
    if draft_table.dim() != 2 or draft_table.shape[1] != V or not draft_table.is_cuda or not draft_table.is_contiguous():
        raise ValueError("draft_table must be a contiguous CUDA tensor [V, V]")
    B = first_tokens.shape[0]
    if first_tokens.dtype != torch.int32 or not first_tokens.is_cuda or not first_tokens.is_contiguous() or first_tokens.dim() != 1:
        raise ValueError("first_tokens must be a contiguous CUDA int32 tensor [B]")
    if (uniforms.dim() != 2 or uniforms.shape[1] != B or uniforms.dtype != torch.float32 or not uniforms.is_cuda
            or not uniforms.is_contiguous()):
        raise ValueError("uniforms must be a contiguous CUDA float32 tensor [gamma, B]")
    gamma = uniforms.shape[0]
    dev = draft_table.device
    tokens = torch.empty((B, gamma), dtype=torch.int32, device=dev)
    lse = torch.empty((B, gamma), dtype=torch.float32, device=dev)
    with torch.cuda.device(dev):
        s = stream if stream is not None else torch.cuda.current_stream(dev)
        _check(lib.bv_draft_chain(draft_table.data_ptr(), first_tokens.data_ptr(), uniforms.data_ptr(), B, gamma, V,
                                  _dtype_code(draft_table), float(temperature), tokens.data_ptr(), lse.data_ptr(),
                                  s.cuda_stream))
    return tokens, lse


def bv_verify_lse(target_logits, draft_logits, draft_tokens, uniforms, draft_lse, temperature: float = 1.0,
                  diagnostics: bool = False, stream=None):
    """Block Verification with the draft rows' log-normalisers supplied (float32 CUDA tensor
    [B, gamma], e.g. the second output of bv_sample_draft reshaped).  Returns (out_tokens, out_len)
    or, with ``diagnostics``, (out_tokens, out_len, dict of p, S, h, lse_t, lse_d)."""
    return _lse_call("bv_verify_lse", target_logits, draft_logits, draft_tokens, uniforms, draft_lse, temperature,
                     diagnostics, stream)


def tv_verify_lse(target_logits, draft_logits, draft_tokens, uniforms, draft_lse, temperature: float = 1.0,
                  diagnostics: bool = False, stream=None):
    """Token Verification with the draft rows' log-normalisers supplied; see bv_verify_lse."""
    return _lse_call("tv_verify_lse", target_logits, draft_logits, draft_tokens, uniforms, draft_lse, temperature,
                     diagnostics, stream)


def _lse_call(name, target_logits, draft_logits, draft_tokens, uniforms, draft_lse, temperature, diagnostics, stream):
    lib = load_library()
    B, gamma, V = _shapes(target_logits, draft_logits, draft_tokens, uniforms, True)
    if (not draft_lse.is_cuda or draft_lse.dtype != torch.float32 or tuple(draft_lse.shape) != (B, gamma)
            or not draft_lse.is_contiguous()):
        raise ValueError("draft_lse must be a contiguous float32 CUDA tensor of [B, gamma]")
    dev = target_logits.device
    out_tokens = torch.empty((B, gamma + 1), dtype=torch.int32, device=dev)
    out_len = torch.empty((B,), dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        s = stream if stream is not None else torch.cuda.current_stream(dev)
        args = [target_logits.data_ptr(), draft_logits.data_ptr(), draft_tokens.data_ptr(), uniforms.data_ptr(),
                draft_lse.data_ptr(), B, gamma, V, _dtype_code(target_logits), float(temperature),
                out_tokens.data_ptr(), out_len.data_ptr()]
        if diagnostics:
            f = lambda *shape: torch.empty(shape, dtype=torch.float32, device=dev)
            diag = dict(p=f(B, gamma + 1), S=f(B, gamma), h=f(B, gamma + 1), lse_t=f(B, gamma + 1), lse_d=f(B, gamma))
            args += [diag[k].data_ptr() for k in ("p", "S", "h", "lse_t", "lse_d")]
            _check(getattr(lib, name + "_ex")(*args, s.cuda_stream))
            return out_tokens, out_len, diag
        _check(getattr(lib, name)(*args, s.cuda_stream))
    return out_tokens, out_len
