"""ctypes front end of the CPU oracle (`nsd_oracle.cpp`).

TEST INFRASTRUCTURE, NOT PRODUCT: only `tests/`, the smoke check and the
benchmark's cpu_baseline / reference arm may import this package.  It neither
imports nor is imported by the CUDA package.  Arrays are numpy, on the host;
bf16 tensors travel as uint16 bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "nsd_oracle.cpp")
_SO = os.path.join(_HERE, "libnsd_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no CUDA involved). Returns the .so path."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = ["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-pthread", "-ffp-contract=off",
               "-o", _SO, _SRC]
        subprocess.run(cmd, check=True)
    return _SO


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32, i64, vp = ctypes.c_int, ctypes.c_int64, ctypes.c_void_p
        lib.oracle_hardware_threads.restype = i32
        lib.oracle_kv_prepare.restype = i32
        lib.oracle_kv_prepare.argtypes = [vp, i32, i64, i32, i32, i32, i32, vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, i32, i32, vp]
        lib.oracle_kv_commit.restype = i32
        lib.oracle_kv_commit.argtypes = [vp, i32, i64, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, i32, i32, vp]
        lib.oracle_verify_attn.restype = i32
        lib.oracle_verify_attn.argtypes = [vp, i32, i64, i32, i32, i32, i32, vp, vp, vp, i32, i32, vp, vp, vp, i32, vp, i32, i32, vp]
        lib.oracle_spec_accept.restype = i32
        lib.oracle_spec_accept.argtypes = [vp, vp, vp, vp, vp, i32, i32, i64, vp, vp, vp, vp, i32, vp]
        lib.oracle_spec_accept_logits.restype = i32
        lib.oracle_spec_accept_logits.argtypes = [vp, ctypes.c_double, vp, vp, vp, vp, i32, i32, i64, vp, vp, vp, vp, vp, i32]
        _lib = lib
    return _lib


def hardware_threads() -> int:
    return int(_load().oracle_hardware_threads())


def _ptr(a: Optional[np.ndarray], dtype) -> Optional[int]:
    if a is None:
        return None
    assert isinstance(a, np.ndarray) and a.dtype == dtype and a.flags["C_CONTIGUOUS"], (a.dtype, dtype)
    return a.ctypes.data


def total_rows(batch: int, gamma: int, gamma_r: Optional[np.ndarray]) -> int:
    return batch * (gamma + 1) if gamma_r is None else int(gamma_r.astype(np.int64).sum()) + batch


def kv_prepare(pool, mig_indptr, mig_src, mig_dst, ctx_len, kv_indptr, kv_indices, k_new, v_new,
               gamma: int, layer_begin: int = 0, layer_count: Optional[int] = None,
               gamma_r: Optional[np.ndarray] = None) -> int:
    """In place on `pool` (uint16 [num_slabs][num_blocks][2][Hkv][bs][D]).

    `k_new`/`v_new`: uint16 [num_layers][rows][Hkv][D] or None (no append); rows =
    batch*(gamma+1), or sum(gamma_r+1) when `gamma_r` (int32 [batch], each in [0, gamma]) gives
    per-request draft depths and the rows are ragged.
    """
    S, NB, two, Hkv, bs, D = pool.shape
    assert two == 2
    n_mig = len(mig_indptr) - 1 if mig_indptr is not None else 0
    batch = len(ctx_len)
    if layer_count is None:
        layer_count = (k_new.shape[0] if k_new is not None else S) - layer_begin
    if k_new is not None:
        assert k_new.shape[1:] == (total_rows(batch, gamma, gamma_r), Hkv, D) and v_new.shape == k_new.shape
    return _load().oracle_kv_prepare(
        _ptr(pool, np.uint16), S, NB, Hkv, bs, D, n_mig, _ptr(mig_indptr, np.int64), _ptr(mig_src, np.int32),
        _ptr(mig_dst, np.int32), batch, gamma, _ptr(ctx_len, np.int32), _ptr(kv_indptr, np.int64),
        _ptr(kv_indices, np.int32), _ptr(k_new, np.uint16), _ptr(v_new, np.uint16), layer_begin, layer_count,
        _ptr(gamma_r, np.int32))


def kv_commit(pool, ctx_len, acc_len, kv_indptr, kv_indices, exp_indptr, exp_indices, gamma: int,
              layer_begin: int = 0, layer_count: Optional[int] = None, gamma_r: Optional[np.ndarray] = None):
    """In place on `pool`; returns (rc, new_ctx_len)."""
    S, NB, two, Hkv, bs, D = pool.shape
    batch = len(ctx_len)
    if layer_count is None:
        layer_count = S - layer_begin
    new_ctx = np.empty(batch, dtype=np.int32)
    rc = _load().oracle_kv_commit(_ptr(pool, np.uint16), S, NB, Hkv, bs, D, batch, gamma, _ptr(ctx_len, np.int32),
                                  _ptr(acc_len, np.int32), _ptr(kv_indptr, np.int64), _ptr(kv_indices, np.int32),
                                  _ptr(exp_indptr, np.int64), _ptr(exp_indices, np.int32), _ptr(new_ctx, np.int32),
                                  layer_begin, layer_count, _ptr(gamma_r, np.int32))
    return rc, new_ctx


def verify_attn(pool, q, ctx_len, kv_indptr, kv_indices, gamma: int, layer: int = 0,
                req_list: Optional[np.ndarray] = None, want_lse: bool = False, nthreads: Optional[int] = None,
                gamma_r: Optional[np.ndarray] = None):
    """Returns o fp32 [rows][Hq][D] (and lse [rows][Hq] when asked).  Rows of
    requests outside `req_list` are left as NaN."""
    S, NB, two, Hkv, bs, D = pool.shape
    rows, Hq, D2 = q.shape
    batch = len(ctx_len)
    assert D2 == D and rows == total_rows(batch, gamma, gamma_r)
    o = np.full((rows, Hq, D), np.nan, dtype=np.float32)
    lse = np.full((rows, Hq), np.nan, dtype=np.float32) if want_lse else None
    nt = nthreads or hardware_threads()
    rc = _load().oracle_verify_attn(
        _ptr(pool, np.uint16), S, NB, Hq, Hkv, bs, D, _ptr(q, np.uint16), _ptr(o, np.float32),
        _ptr(lse, np.float32), batch, gamma, _ptr(ctx_len, np.int32), _ptr(kv_indptr, np.int64),
        _ptr(kv_indices, np.int32), layer, _ptr(req_list, np.int32), 0 if req_list is None else len(req_list), nt,
        _ptr(gamma_r, np.int32))
    if rc != 0:
        raise RuntimeError(f"oracle_verify_attn failed: {rc}")
    return (o, lse) if want_lse else o


def spec_accept(p, q, draft_tok, u_acc, u_smp, ctx_len: Optional[np.ndarray] = None, nthreads: Optional[int] = None,
                gamma_r: Optional[np.ndarray] = None, gamma: Optional[int] = None):
    """Returns (acc_len [B], out_tok [B][gamma+1], new_ctx_len [B] or None).

    Ragged form (`gamma_r` int32 [B], `gamma` = its upper bound): p [sum(gamma_r+1)][V],
    q [sum(gamma_r)][V], draft_tok / u_acc [sum(gamma_r)], out_tok [sum(gamma_r+1)]."""
    if gamma_r is None:
        B, g1, V = p.shape
        gamma = g1 - 1
        assert q.shape == (B, gamma, V) and draft_tok.shape == (B, gamma) and u_acc.shape == (B, gamma) and u_smp.shape == (B,)
        out = np.empty((B, gamma + 1), dtype=np.int32)
    else:
        B, V = len(gamma_r), p.shape[-1]
        rows, drafts = total_rows(B, gamma, gamma_r), int(gamma_r.astype(np.int64).sum())
        assert p.shape == (rows, V) and q.shape == (drafts, V) and draft_tok.shape == (drafts,) and u_acc.shape == (drafts,)
        out = np.empty(rows, dtype=np.int32)
    acc = np.empty(B, dtype=np.int32)
    new_ctx = np.empty(B, dtype=np.int32) if ctx_len is not None else None
    nt = nthreads or hardware_threads()
    rc = _load().oracle_spec_accept(
        _ptr(p, np.float32), _ptr(q, np.float32), _ptr(draft_tok, np.int32), _ptr(u_acc, np.float32),
        _ptr(u_smp, np.float32), B, gamma, V, _ptr(ctx_len, np.int32), _ptr(acc, np.int32), _ptr(out, np.int32),
        _ptr(new_ctx, np.int32), nt, _ptr(gamma_r, np.int32))
    if rc != 0:
        raise RuntimeError(f"oracle_spec_accept failed: {rc}")
    return acc, out, new_ctx


def spec_accept_logits(logits, temperature: float, q, draft_tok, u_acc, u_smp, gamma_r: Optional[np.ndarray] = None,
                       ctx_len: Optional[np.ndarray] = None, nthreads: Optional[int] = None):
    """logits fp32 [B][gamma+1][V] (widen bf16 first).  temperature 0 = greedy (q, u_acc, u_smp may be None).
    Returns (acc_len, out_tok, new_ctx_len or None)."""
    B, g1, V = logits.shape
    gamma = g1 - 1
    acc = np.empty(B, dtype=np.int32)
    out = np.empty((B, gamma + 1), dtype=np.int32)
    new_ctx = np.empty(B, dtype=np.int32) if ctx_len is not None else None
    nt = nthreads or hardware_threads()
    rc = _load().oracle_spec_accept_logits(
        _ptr(logits, np.float32), float(temperature), _ptr(q, np.float32), _ptr(draft_tok, np.int32),
        _ptr(u_acc, np.float32), _ptr(u_smp, np.float32), B, gamma, V, _ptr(gamma_r, np.int32), _ptr(ctx_len, np.int32),
        _ptr(acc, np.int32), _ptr(out, np.int32), _ptr(new_ctx, np.int32), nt)
    if rc != 0:
        raise RuntimeError(f"oracle_spec_accept_logits failed: {rc}")
    return acc, out, new_ctx
