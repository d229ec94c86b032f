"""ctypes front end of ``rkv_oracle.c`` (TEST INFRASTRUCTURE, not a product path).

Marshals numpy arrays into the C oracle and back; it holds no arithmetic of the
method.  Keys and queries are handed over as float32 (bf16 widens to float32
exactly, and so does an 8-bit E4M3 cache byte, decoded by ``e4m3_to_f32`` below);
the C side computes in double (Eq. 1-7, Algorithm 1).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rkv_oracle.c")
_LIB = os.path.join(_HERE, "librkv_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP over head-problems) if it is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp, fp, ip = (ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_float),
                      ctypes.POINTER(ctypes.c_int32))
        lib.rkv_oracle_head.restype = ctypes.c_int
        lib.rkv_oracle_head.argtypes = [fp, fp] + [ctypes.c_int] * 7 + [ctypes.c_double] * 3 + \
            [ip] + [dp] * 7 + [ctypes.c_int]
        lib.rkv_oracle_batch.restype = ctypes.c_int
        lib.rkv_oracle_batch.argtypes = [fp, fp, ip] + [ctypes.c_int] * 9 + [ctypes.c_double] * 3 + \
            [ip, dp, ip, ctypes.c_int]
        lib.rkv_oracle_gather.restype = None
        lib.rkv_oracle_gather.argtypes = [ctypes.c_void_p, ip, ctypes.c_int, ctypes.c_size_t,
                                          ctypes.c_void_p]
        lib.rkv_oracle_decode_attention.restype = ctypes.c_int
        lib.rkv_oracle_decode_attention.argtypes = [fp, fp, fp, ip] + [ctypes.c_int] * 5 + [dp]
        _lib = lib
    return _lib


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def _ptr(a: Optional[np.ndarray], ctype):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ctype))


@dataclass
class HeadResult:
    compressed: bool
    idx: np.ndarray            # [budget] int32
    A: Optional[np.ndarray]    # [alpha, n]
    I: Optional[np.ndarray]    # [n]
    Sbar: Optional[np.ndarray]
    R: Optional[np.ndarray]
    Z: Optional[np.ndarray]
    S_raw: Optional[np.ndarray]  # [n, n], Eq. 5 with zero diagonal
    S_mod: Optional[np.ndarray]  # [n, n], after the retention rule


def oracle_head(K, Q, *, budget: int, alpha: int, lam: float, W: int, beta: int, T: float,
                eps: float = 1e-8, L: Optional[int] = None, want_S: bool = False,
                mean_then_pool: bool = False, gqa_mean_pool: bool = False) -> HeadResult:
    """One (sequence, KV head): K [>=L, d], Q [G, alpha, d]."""
    lib = _load()
    K = _f32(K)
    Q = _f32(Q)
    L = K.shape[0] if L is None else int(L)
    d = K.shape[1]
    G = Q.shape[0]
    assert Q.shape == (G, alpha, d) and K.shape[0] >= L
    idx = np.empty(budget, dtype=np.int32)
    n = max(L - alpha, 0)
    live = L > budget
    A = np.zeros((alpha, n)) if live else None
    I, Sbar, R, Z = (np.zeros(n) if live else None for _ in range(4))
    S_raw = np.zeros((n, n)) if (live and want_S) else None
    S_mod = np.zeros((n, n)) if (live and want_S) else None
    r = lib.rkv_oracle_head(_ptr(K, ctypes.c_float), _ptr(Q, ctypes.c_float), L, d, G, alpha, budget,
                            W, beta, float(T), float(eps), float(lam), _ptr(idx, ctypes.c_int32),
                            _ptr(A, ctypes.c_double), _ptr(I, ctypes.c_double),
                            _ptr(Sbar, ctypes.c_double), _ptr(R, ctypes.c_double),
                            _ptr(Z, ctypes.c_double), _ptr(S_raw, ctypes.c_double),
                            _ptr(S_mod, ctypes.c_double),
                            (1 if mean_then_pool else 0) | (4 if gqa_mean_pool else 0))
    if r < 0:
        raise ValueError("rkv_oracle_head: bad arguments")
    return HeadResult(bool(r), idx, A, I, Sbar, R, Z, S_raw, S_mod)


@dataclass
class BatchResult:
    idx: np.ndarray         # [B, Hkv, budget] int32
    compressed: np.ndarray  # [B] bool
    I: Optional[np.ndarray]     # [B, Hkv, cap] (first n = L - alpha entries meaningful)
    Sbar: Optional[np.ndarray]
    R: Optional[np.ndarray]
    Z: Optional[np.ndarray]
    threads: int


def oracle_batch(K, Q, seq_lens, *, budget: int, alpha: int, lam: float, W: int, beta: int,
                 T: float, eps: float = 1e-8, want_scores: bool = True,
                 mean_then_pool: bool = False, head_mean: bool = False, gqa_mean_pool: bool = False,
                 budgets=None) -> BatchResult:
    """K [B, Hkv, cap, d], Q [B, Hq, alpha, d], seq_lens [B].
    budgets: optional [B], a budget of its own per sequence (Section 4.2's budget ratios); `budget` is then only
    the row length of idx (entries beyond a sequence's own budget are -1)."""
    if budgets is not None:
        return _oracle_batch_per_sequence(K, Q, seq_lens, budgets, budget=budget, alpha=alpha, lam=lam, W=W, beta=beta,
                                          T=T, eps=eps, want_scores=want_scores, mean_then_pool=mean_then_pool,
                                          head_mean=head_mean, gqa_mean_pool=gqa_mean_pool)
    lib = _load()
    K = _f32(K)
    Q = _f32(Q)
    seq = np.ascontiguousarray(np.asarray(seq_lens, dtype=np.int32))
    B, Hkv, cap, d = K.shape
    Hq = Q.shape[1]
    assert Q.shape == (B, Hq, alpha, d) and seq.shape == (B,)
    idx = np.empty((B, Hkv, budget), dtype=np.int32)
    scores = np.zeros((4, B, Hkv, cap)) if want_scores else None
    comp = np.zeros(B, dtype=np.int32)
    t = lib.rkv_oracle_batch(_ptr(K, ctypes.c_float), _ptr(Q, ctypes.c_float),
                             _ptr(seq, ctypes.c_int32), B, Hkv, Hq, cap, d, alpha, budget, W, beta,
                             float(T), float(eps), float(lam), _ptr(idx, ctypes.c_int32),
                             _ptr(scores, ctypes.c_double), _ptr(comp, ctypes.c_int32),
                             (1 if mean_then_pool else 0) | (2 if head_mean else 0) | (4 if gqa_mean_pool else 0))
    if t < 0:
        raise ValueError("rkv_oracle_batch: bad arguments (seq_len > cap, or sizes)")
    if scores is None:
        return BatchResult(idx, comp.astype(bool), None, None, None, None, t)
    return BatchResult(idx, comp.astype(bool), scores[0], scores[1], scores[2], scores[3], t)


def _oracle_batch_per_sequence(K, Q, seq_lens, budgets, *, budget, want_scores, **kw) -> BatchResult:
    """Every sequence with its own budget: the sequences are independent, so each goes through the C oracle alone
    with its budget, and the results are put side by side (marshalling only)."""
    K = _f32(K)
    Q = _f32(Q)
    B, Hkv, cap, _ = K.shape
    idx = np.full((B, Hkv, budget), -1, dtype=np.int32)
    comp = np.zeros(B, dtype=bool)
    scores = [np.zeros((B, Hkv, cap)) for _ in range(4)] if want_scores else [None] * 4
    threads = 1
    for b in range(B):
        nb = int(budgets[b])
        assert kw["alpha"] < nb <= budget
        r = oracle_batch(K[b:b + 1], Q[b:b + 1], np.asarray(seq_lens)[b:b + 1], budget=nb, want_scores=want_scores, **kw)
        idx[b, :, :nb] = r.idx[0]
        comp[b] = r.compressed[0]
        threads = max(threads, r.threads)
        if want_scores:
            for t, part in enumerate((r.I, r.Sbar, r.R, r.Z)):
                scores[t][b] = part[0]
    return BatchResult(idx, comp, scores[0], scores[1], scores[2], scores[3], threads)


def oracle_decode_attention(K, V, q_new, seq_lens) -> np.ndarray:
    """Section 3.1's decode step: the new query of every query head over the cached keys and values of its KV head
    (Eq. 1 with one query row).  K, V [B, Hkv, cap, d], q_new [B, Hq, d], seq_lens [B] -> [B, Hq, d] float64."""
    lib = _load()
    K, V, q_new = _f32(K), _f32(V), _f32(q_new)
    seq = np.ascontiguousarray(np.asarray(seq_lens, dtype=np.int32))
    B, Hkv, cap, d = K.shape
    Hq = q_new.shape[1]
    assert V.shape == K.shape and q_new.shape == (B, Hq, d) and seq.shape == (B,)
    out = np.zeros((B, Hq, d))
    rc = lib.rkv_oracle_decode_attention(_ptr(K, ctypes.c_float), _ptr(V, ctypes.c_float), _ptr(q_new, ctypes.c_float),
                                         _ptr(seq, ctypes.c_int32), B, Hkv, Hq, cap, d, _ptr(out, ctypes.c_double))
    if rc != 0:
        raise ValueError("rkv_oracle_decode_attention: bad arguments")
    return out


def e4m3_to_f32(codes) -> np.ndarray:
    """Value of every 8-bit E4M3 code (the "fn" variant of the OCP 8-bit floating point format: 1 sign bit, 4 exponent
    bits with bias 7, 3 mantissa bits; no infinities; exponent 15 with mantissa 7 is NaN; largest finite value 448).
    An 8-bit cache holds such codes; the method (Eq. 1-7) is defined on the values they stand for, which float32
    represents exactly.

        exponent field e = 0:   (m / 8) * 2^-6          (subnormal)
        otherwise:              (1 + m / 8) * 2^(e - 7)
    """
    c = np.asarray(codes, dtype=np.uint8)
    sign = np.where(c & 0x80, -1.0, 1.0)
    e = ((c >> 3) & 0xF).astype(np.int32)
    m = (c & 0x7).astype(np.float64)
    val = np.where(e == 0, np.ldexp(m / 8.0, -6), np.ldexp(1.0 + m / 8.0, e - 7))
    val = np.where((e == 15) & (m == 7), np.nan, val)
    return (sign * val).astype(np.float32)


def oracle_gather(rows: np.ndarray, idx: np.ndarray) -> np.ndarray:
    """Algorithm 1's gather for one head: rows [L, ...] of any dtype, idx [count] (-1 = skip).
    Returns out [count, ...] with out[j] = rows[idx[j]], copied byte for byte."""
    lib = _load()
    rows = np.ascontiguousarray(rows)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    out = np.zeros((idx.shape[0],) + rows.shape[1:], dtype=rows.dtype)
    row_bytes = rows.dtype.itemsize * int(np.prod(rows.shape[1:], dtype=np.int64))
    lib.rkv_oracle_gather(rows.ctypes.data, _ptr(idx, ctypes.c_int32), idx.shape[0], row_bytes,
                          out.ctypes.data)
    return out


def oracle_append(k_cache: np.ndarray, v_cache: np.ndarray, k_new: np.ndarray, v_new: np.ndarray,
                  seq_lens: np.ndarray):
    """Section 3.1's decode step on the cache, written out: the new token of sequence b becomes row seq_lens[b] of
    every KV head (k_cache, v_cache [B, H, cap, d] of any dtype; k_new, v_new [B, H, d]); seq_lens[b] grows by one.
    A sequence whose cache is full stays as it is.  Returns new arrays (k, v, seq_lens)."""
    k, v, s = k_cache.copy(), v_cache.copy(), np.array(seq_lens, dtype=np.int32, copy=True)
    cap = k.shape[2]
    for b in range(k.shape[0]):
        L = int(s[b])
        if 0 <= L < cap:
            for h in range(k.shape[1]):
                k[b, h, L] = k_new[b, h]
                v[b, h, L] = v_new[b, h]
            s[b] = L + 1
    return k, v, s


def oracle_push_query(q_window: np.ndarray, q_new: np.ndarray, slot: int) -> np.ndarray:
    """Algorithm 1's observation buffer of the last alpha queries kept as a ring: q_new [B, Hq, d] replaces row `slot`
    of every head's window in q_window [B, Hq, alpha, d].  Returns a new array."""
    q = q_window.copy()
    for b in range(q.shape[0]):
        for h in range(q.shape[1]):
            q[b, h, slot] = q_new[b, h]
    return q
