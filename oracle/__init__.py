"""TEST INFRASTRUCTURE -- not part of the product path.

Loader for the fp64 CPU oracle of Token Verification (Algorithm 1), Block
Verification (Algorithm 2) and Greedy Block Verification (Algorithm 4, one
iteration) of arXiv 2403.10444, written in plain C in
``verify_oracle.c``.  Only tests, the smoke check and the benchmark's
CPU-baseline leg may import this package; the CUDA library never does, and
this package never imports the CUDA library.

``verify`` marshals numpy arrays into the C entry point ``oracle_verify`` and
returns every output and intermediate as numpy arrays.  No arithmetic of the
method happens in this file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "verify_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

TOKEN_VERIFY = 0
BLOCK_VERIFY = 1
GREEDY_BLOCK_VERIFY = 2

_DTYPE_CODE = {np.dtype(np.float32): 0, np.dtype(np.uint16): 1, np.dtype(np.float64): 2}


def build(force: bool = False) -> str:
    """Compile verify_oracle.c into liboracle.so (gcc, -O2, OpenMP over sequences)."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, ip = ctypes.c_void_p, ctypes.c_int
        lib.oracle_verify.restype = ctypes.c_int
        lib.oracle_verify.argtypes = [ip, vp, vp, vp, vp, ip, ip, ip, ip, ctypes.c_double,
                                      vp, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.oracle_verify_lse.restype = ctypes.c_int
        lib.oracle_verify_lse.argtypes = [ip, vp, vp, vp, vp, vp, ip, ip, ip, ip, ctypes.c_double,
                                          vp, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.oracle_verify_probs.restype = ctypes.c_int
        lib.oracle_verify_probs.argtypes = [ip, vp, vp, vp, vp, ip, ip, ip, ip, vp, vp, vp, vp, vp, vp, vp]
        lib.oracle_threads.restype = ctypes.c_int
        lib.oracle_sample_rows.restype = ctypes.c_int
        lib.oracle_sample_rows.argtypes = [vp, vp, ip, ip, ip, ctypes.c_double, vp, vp, vp]
        _lib = lib
    return _lib


def threads() -> int:
    """Threads the oracle's loop over sequences uses."""
    return int(_load().oracle_threads())


@dataclass
class OracleResult:
    out_tokens: np.ndarray   # [B, gamma+1] int32, X^tau, Y, then -1
    out_len: np.ndarray      # [B] int32, tau+1 or -1
    p: np.ndarray            # [B, gamma+1] f64 (NaN for Token Verification)
    S: np.ndarray            # [B, gamma]   f64
    h: np.ndarray            # [B, gamma+1] f64, h[:,0] = 1
    lse_t: np.ndarray        # [B, gamma+1] f64, natural-log normaliser of logits/T
    lse_d: np.ndarray        # [B, gamma]   f64
    margin_eta: np.ndarray   # [B] f64, min |eta_i - h_i| over deciding comparisons
    margin_smp: np.ndarray   # [B] f64, distance of the sampling uniform to its CDF cell edge


def verify(algo: int, target: np.ndarray, draft: np.ndarray, tokens: np.ndarray,
           uniforms: np.ndarray, temperature: float = 1.0, draft_lse=None) -> OracleResult:
    """Run Algorithm 1 (algo=TOKEN_VERIFY), Algorithm 2 (algo=BLOCK_VERIFY) or
    Algorithm 4 (algo=GREEDY_BLOCK_VERIFY: p holds the unclipped products, S the numerator
    sums and h the printed ratios, which may exceed 1 or be +inf).

    target [B, gamma+1, V] and draft [B, gamma, V] share a dtype: float32,
    float64, or uint16 holding bf16 bit patterns.  tokens [B, gamma] int32,
    uniforms [B, gamma+2] float32.  ``temperature`` is rounded to float32 first
    (the C-ABI of the CUDA library carries it as a float).
    """
    lib = _load()
    target = np.ascontiguousarray(target)
    draft = np.ascontiguousarray(draft)
    if target.dtype != draft.dtype or target.dtype not in _DTYPE_CODE:
        raise TypeError("target/draft must both be float32, float64 or uint16 (bf16 bits)")
    B, g1, V = target.shape
    gamma = g1 - 1
    if draft.shape != (B, gamma, V):
        raise ValueError("draft must be [B, gamma, V]")
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    uniforms = np.ascontiguousarray(uniforms, dtype=np.float32)
    if tokens.shape != (B, gamma) or uniforms.shape != (B, gamma + 2):
        raise ValueError("tokens must be [B, gamma], uniforms [B, gamma+2]")
    res = OracleResult(
        out_tokens=np.empty((B, gamma + 1), np.int32), out_len=np.empty((B,), np.int32),
        p=np.empty((B, gamma + 1)), S=np.empty((B, gamma)), h=np.empty((B, gamma + 1)),
        lse_t=np.empty((B, gamma + 1)), lse_d=np.empty((B, gamma)),
        margin_eta=np.empty((B,)), margin_smp=np.empty((B,)))
    ptr = lambda a: a.ctypes.data_as(ctypes.c_void_p)
    fn, extra = lib.oracle_verify, []
    if draft_lse is not None:
        # the draft rows' log-normalisers are supplied (float32 [B, gamma]) instead of computed
        draft_lse = np.ascontiguousarray(draft_lse, dtype=np.float32)
        if draft_lse.shape != (B, gamma):
            raise ValueError("draft_lse must be [B, gamma]")
        fn, extra = lib.oracle_verify_lse, [ptr(draft_lse)]
    rc = fn(int(algo), ptr(target), ptr(draft), ptr(tokens), ptr(uniforms), *extra,
                           B, gamma, V, _DTYPE_CODE[target.dtype],
                           float(np.float32(temperature)),
                           ptr(res.out_tokens), ptr(res.out_len), ptr(res.p), ptr(res.S),
                           ptr(res.h), ptr(res.lse_t), ptr(res.lse_d),
                           ptr(res.margin_eta), ptr(res.margin_smp))
    if rc != 0:
        raise ValueError("oracle_verify rejected its arguments")
    return res


def verify_probs(algo: int, target_probs: np.ndarray, draft_probs: np.ndarray, tokens: np.ndarray,
                 uniforms: np.ndarray) -> OracleResult:
    """Algorithm 1 or 2 on given probabilities (``oracle_verify_probs``): target_probs
    [B, gamma+1, V], draft_probs [B, gamma, V], float32 / float64 / uint16 bf16 bits, used as
    stored.  ``lse_t`` and ``lse_d`` of the result are NaN."""
    lib = _load()
    target_probs = np.ascontiguousarray(target_probs)
    draft_probs = np.ascontiguousarray(draft_probs)
    if target_probs.dtype != draft_probs.dtype or target_probs.dtype not in _DTYPE_CODE:
        raise TypeError("target/draft must both be float32, float64 or uint16 (bf16 bits)")
    B, g1, V = target_probs.shape
    gamma = g1 - 1
    if draft_probs.shape != (B, gamma, V):
        raise ValueError("draft_probs must be [B, gamma, V]")
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    uniforms = np.ascontiguousarray(uniforms, dtype=np.float32)
    if tokens.shape != (B, gamma) or uniforms.shape != (B, gamma + 2):
        raise ValueError("tokens must be [B, gamma], uniforms [B, gamma+2]")
    res = OracleResult(
        out_tokens=np.empty((B, gamma + 1), np.int32), out_len=np.empty((B,), np.int32),
        p=np.empty((B, gamma + 1)), S=np.empty((B, gamma)), h=np.empty((B, gamma + 1)),
        lse_t=np.full((B, gamma + 1), np.nan), lse_d=np.full((B, gamma), np.nan),
        margin_eta=np.empty((B,)), margin_smp=np.empty((B,)))
    ptr = lambda a: a.ctypes.data_as(ctypes.c_void_p)
    rc = lib.oracle_verify_probs(int(algo), ptr(target_probs), ptr(draft_probs), ptr(tokens), ptr(uniforms),
                                 B, gamma, V, _DTYPE_CODE[target_probs.dtype],
                                 ptr(res.out_tokens), ptr(res.out_len), ptr(res.p), ptr(res.S), ptr(res.h),
                                 ptr(res.margin_eta), ptr(res.margin_smp))
    if rc != 0:
        raise ValueError("oracle_verify_probs rejected its arguments")
    return res


def block_verify(*a, **k) -> OracleResult:
    return verify(BLOCK_VERIFY, *a, **k)


def greedy_block_verify(*a, **k) -> OracleResult:
    return verify(GREEDY_BLOCK_VERIFY, *a, **k)


def token_verify(*a, **k) -> OracleResult:
    return verify(TOKEN_VERIFY, *a, **k)


def sample_rows(logits: np.ndarray, uniforms: np.ndarray, temperature: float = 1.0):
    """The drafting step of Algorithm 3 on rows of logits [rows, V] (float32, float64 or uint16
    bf16 bits) with one float32 uniform per row: returns (tokens int32 [rows], lse f64 [rows],
    margin f64 [rows]); see ``oracle_sample_rows`` in verify_oracle.c."""
    lib = _load()
    logits = np.ascontiguousarray(logits)
    if logits.dtype not in _DTYPE_CODE or logits.ndim != 2:
        raise TypeError("logits must be [rows, V] float32, float64 or uint16 (bf16 bits)")
    rows, V = logits.shape
    uniforms = np.ascontiguousarray(uniforms, dtype=np.float32)
    if uniforms.shape != (rows,):
        raise ValueError("uniforms must be [rows]")
    tok = np.empty((rows,), np.int32)
    lse = np.empty((rows,))
    margin = np.empty((rows,))
    ptr = lambda a: a.ctypes.data_as(ctypes.c_void_p)
    rc = lib.oracle_sample_rows(ptr(logits), ptr(uniforms), rows, V, _DTYPE_CODE[logits.dtype],
                                float(np.float32(temperature)), ptr(tok), ptr(lse), ptr(margin))
    if rc != 0:
        raise ValueError("oracle_sample_rows rejected its arguments")
    return tok, lse, margin
