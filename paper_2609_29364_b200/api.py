"""ctypes binding of include/nsd.h.  Same names as the C ABI, argument
marshalling only: tensors are torch CUDA tensors (device memory and streams are
torch's), every step runs inside libnsd.so."""
from __future__ import annotations

import ctypes
import os
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libnsd.so")
_lib = None

STATUS = {
    0: "NSD_OK", 1: "NSD_ERR_INVALID_ARG", 2: "NSD_ERR_OUT_OF_RANGE", 3: "NSD_ERR_CAPACITY",
    4: "NSD_ERR_UNSUPPORTED", 5: "NSD_ERR_CUDA", 6: "NSD_ERR_DEVICE_FAULT", 7: "NSD_ERR_NOT_PLANNED",
    8: "NSD_ERR_TIMEOUT",
}


class NsdError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        super().__init__(f"{where}: {STATUS.get(code, code)}" + (f" ({detail})" if detail else ""))


class NsdConfig(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "num_layers", "num_slabs", "num_q_heads", "num_kv_heads", "head_dim", "block_size", "num_blocks",
        "region_b_begin", "max_batch", "max_gamma", "vocab_size", "flags")] + [
        ("max_table_entries", ctypes.c_int64), ("wait_budget", ctypes.c_int32), ("reserved", ctypes.c_int32)]


# nsd_config.flags (include/nsd.h)
NSD_FLAG_ATTN_CP_ASYNC = 1 << 0
NSD_FLAG_ATTN_TCGEN05 = 1 << 1
NSD_FLAG_ATTN_NO_TCGEN05 = 1 << 2
NSD_FLAG_LOGITS_DIRECT = 1 << 3
NSD_FLAG_ROUND_SPLIT_ALWAYS = 1 << 4
NSD_FLAG_ROUND_SPLIT_NEVER = 1 << 5
NSD_FLAG_NO_DEPENDENT_LAUNCH = 1 << 6
NSD_FLAG_TEST_STARVE_GATHER = 1 << 30


_vp = ctypes.c_void_p


class SchedParams(ctypes.Structure):
    _fields_ = [("worker_avail", ctypes.c_double), ("target_interval", ctypes.c_double), ("slack", ctypes.c_double),
                ("max_batch", ctypes.c_int32), ("row_capacity", ctypes.c_int32), ("block_capacity", ctypes.c_int64),
                ("token_limit", ctypes.c_int64)]


class RoundArgs(ctypes.Structure):
    _fields_ = [
        ("kv_pool", _vp), ("n_mig_blocks", ctypes.c_int64), ("mig_src", _vp), ("mig_dst", _vp),
        ("batch", ctypes.c_int32), ("gamma", ctypes.c_int32), ("ctx_len", _vp), ("kv_indptr", _vp),
        ("kv_indices", _vp), ("is_migrated", _vp), ("k_new", _vp), ("v_new", _vp), ("q", _vp), ("o", _vp),
        ("p", _vp), ("q_draft", _vp), ("draft_tok", _vp), ("u_acc", _vp), ("u_smp", _vp), ("acc_len", _vp),
        ("out_tok", _vp), ("new_ctx_len", _vp), ("fuse_gather", ctypes.c_int32), ("reserved", ctypes.c_int32),
        ("q_indptr", _vp),
    ]


def lib_path() -> str:
    return _LIB_PATH


def load_library():
    """Loads libnsd.so; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: run `python -m paper_2609_29364_b200.build` "
                          "(or __graft_entry__.build()); there is no non-CUDA path")
    lib = ctypes.CDLL(_LIB_PATH)
    i32, i64, sz = ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    cfgp = ctypes.POINTER(NsdConfig)
    rap = ctypes.POINTER(RoundArgs)
    lib.nsd_status_string.restype = ctypes.c_char_p
    lib.nsd_status_string.argtypes = [i32]
    lib.nsd_last_error.restype = ctypes.c_char_p
    lib.nsd_last_error.argtypes = [_vp]
    lib.nsd_workspace_bytes.restype = sz
    lib.nsd_workspace_bytes.argtypes = [cfgp]
    lib.nsd_kv_pool_bytes.restype = sz
    lib.nsd_kv_pool_bytes.argtypes = [cfgp]
    lib.nsd_create.restype = i32
    lib.nsd_create.argtypes = [cfgp, _vp, sz, ctypes.POINTER(_vp)]
    lib.nsd_destroy.restype = i32
    lib.nsd_destroy.argtypes = [_vp]
    lib.nsd_verify_plan.restype = i32
    lib.nsd_verify_plan.argtypes = [_vp, i32, i32, _vp, _vp, _vp, _vp, i32, _vp]
    lib.nsd_kv_prepare.restype = i32
    lib.nsd_kv_prepare.argtypes = [_vp, _vp, i64, _vp, _vp, i32, i32, _vp, _vp, _vp, _vp, _vp, _vp, i32, i32, i32, _vp, i64, _vp]
    lib.nsd_kv_commit.restype = i32
    lib.nsd_kv_commit.argtypes = [_vp, _vp, i32, i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, i32, i32, _vp, _vp]
    lib.nsd_verify_attn.restype = i32
    lib.nsd_verify_attn.argtypes = [_vp, _vp, _vp, _vp, _vp, i32, i32, _vp, _vp, _vp, i32, i32, _vp]
    lib.nsd_spec_accept.restype = i32
    lib.nsd_spec_accept.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, i32, i32, i32, _vp, _vp, _vp, _vp, _vp, _vp]
    lib.nsd_spec_accept_logits.restype = i32
    lib.nsd_spec_accept_logits.argtypes = [_vp, _vp, i32, ctypes.c_float, _vp, _vp, _vp, _vp, i32, i32, i32, _vp, _vp, _vp, _vp, _vp, _vp]
    lib.nsd_verify_round.restype = i32
    lib.nsd_verify_round.argtypes = [_vp, rap, _vp]
    lib.nsd_verify_round_host.restype = i32
    lib.nsd_verify_round_host.argtypes = [_vp, rap, rap, i64, _vp, ctypes.POINTER(i64), ctypes.POINTER(i64)]
    lib.nsd_verify_attn_static.restype = i32
    lib.nsd_verify_attn_static.argtypes = [_vp, i32, i32, i32, i32, i32, _vp, _vp, i32, i32, _vp, _vp, _vp, _vp, _vp]
    lib.nsd_schedule_batch.restype = i32
    lib.nsd_schedule_batch.argtypes = [ctypes.POINTER(SchedParams), i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp,
                                       ctypes.POINTER(i32), ctypes.POINTER(ctypes.c_double)]
    lib.nsd_launch_count.restype = i64
    lib.nsd_launch_count.argtypes = [_vp]
    lib.nsd_get_status.restype = i32
    lib.nsd_get_status.argtypes = [_vp, _vp, ctypes.POINTER(i32)]
    _lib = lib
    return lib


def _ptr(t) -> Optional[int]:
    """Address of a torch tensor (CUDA or pinned host), numpy array, int or None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        assert t.is_contiguous()
        return t.data_ptr()
    if hasattr(t, "ctypes"):
        assert t.flags["C_CONTIGUOUS"]
        return t.ctypes.data
    raise TypeError(type(t))


def _stream_handle(stream) -> Optional[int]:
    if stream is None:
        import torch

        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def nsd_verify_attn_static(kv_slab, num_blocks, num_q_heads, num_kv_heads, head_dim, block_size, q, o, batch, gamma,
                           h_ctx_len, ctx_len, kv_indptr, kv_indices, stream=None):
    """Attention without any device allocation: the scratch is a fixed array inside
    libnsd.so (see include/nsd.h for who needs this, the size limits and the rule
    that calls must not overlap on the GPU).  Needs no VerifyContext."""
    rc = load_library().nsd_verify_attn_static(_ptr(kv_slab), num_blocks, num_q_heads, num_kv_heads, head_dim,
                                               block_size, _ptr(q), _ptr(o), batch, gamma, _ptr(h_ctx_len),
                                               _ptr(ctx_len), _ptr(kv_indptr), _ptr(kv_indices),
                                               _stream_handle(stream))
    if rc != 0:
        raise NsdError(rc, "nsd_verify_attn_static")


def nsd_schedule_batch(*, worker_avail, target_interval, slack, max_batch, pred_done, kv_ready, eligible=None,
                       rows=None, blocks=None, tokens=None, row_capacity=2 ** 31 - 1, block_capacity=2 ** 62,
                       token_limit=2 ** 62):
    """Algorithm 1 on the host (numpy arrays in, list of admitted indices and predicted start out)."""
    import numpy as np

    n = len(pred_done)
    prm = SchedParams(worker_avail, target_interval, slack, max_batch, row_capacity, block_capacity, token_limit)
    out = np.empty(max(1, min(n, max(max_batch, 0))), dtype=np.int32)
    m, start = ctypes.c_int32(0), ctypes.c_double(0.0)
    f64 = lambda a: None if a is None else np.ascontiguousarray(a, dtype=np.float64)
    i32a = lambda a: None if a is None else np.ascontiguousarray(a, dtype=np.int32)
    keep = [f64(pred_done), f64(kv_ready), None if eligible is None else np.ascontiguousarray(eligible, dtype=np.uint8),
            i32a(rows), i32a(blocks), i32a(tokens)]
    rc = load_library().nsd_schedule_batch(ctypes.byref(prm), n, _ptr(keep[2]), _ptr(keep[0]), _ptr(keep[1]),
                                           _ptr(keep[3]), _ptr(keep[4]), _ptr(keep[5]), _ptr(out), ctypes.byref(m),
                                           ctypes.byref(start))
    if rc != 0:
        raise NsdError(rc, "nsd_schedule_batch")
    return out[:m.value].tolist(), start.value


class VerifyContext:
    """Owns an nsd_ctx and the torch-allocated workspace it lives on."""

    def __init__(self, *, num_layers, num_q_heads, num_kv_heads, head_dim, block_size, num_blocks, region_b_begin,
                 max_batch, max_gamma, vocab_size, max_table_entries, num_slabs=None, flags=0, wait_budget=0,
                 device="cuda:0"):
        import torch

        self.lib = load_library()
        self.cfg = NsdConfig(num_layers=num_layers, num_slabs=num_slabs or num_layers, num_q_heads=num_q_heads,
                             num_kv_heads=num_kv_heads, head_dim=head_dim, block_size=block_size,
                             num_blocks=num_blocks, region_b_begin=region_b_begin, max_batch=max_batch,
                             max_gamma=max_gamma, vocab_size=vocab_size, flags=flags,
                             max_table_entries=max_table_entries, wait_budget=wait_budget, reserved=0)
        self.device = torch.device(device)
        self._h = _vp()
        nbytes = self.lib.nsd_workspace_bytes(ctypes.byref(self.cfg))
        if nbytes == 0:
            raise NsdError(4, "nsd_workspace_bytes", "invalid or unsupported configuration")
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            rc = self.lib.nsd_create(ctypes.byref(self.cfg), self.workspace.data_ptr(), nbytes, ctypes.byref(self._h))
        if rc != 0:
            raise NsdError(rc, "nsd_create")

    # -- helpers
    def _check(self, rc: int, where: str):
        if rc != 0:
            detail = self.lib.nsd_last_error(self._h).decode() if rc == 5 else ""
            raise NsdError(rc, where, detail)

    def pool_bytes(self) -> int:
        return self.lib.nsd_kv_pool_bytes(ctypes.byref(self.cfg))

    def close(self):
        if self._h:
            self.lib.nsd_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the C ABI, one method per entry point
    def nsd_verify_plan(self, h_ctx_len, h_kv_indptr, h_is_migrated, gamma, chunk_blocks=0, stream=None, h_q_indptr=None):
        batch = len(h_ctx_len)
        self._check(self.lib.nsd_verify_plan(self._h, batch, gamma, _ptr(h_ctx_len), _ptr(h_kv_indptr),
                                             _ptr(h_is_migrated), _ptr(h_q_indptr), chunk_blocks, _stream_handle(stream)),
                    "nsd_verify_plan")

    def nsd_kv_prepare(self, kv_pool, n_mig_blocks, mig_src, mig_dst, batch, gamma, ctx_len, kv_indptr, kv_indices,
                       k_new, v_new, is_migrated=None, append_subset=0, layer_begin=0, layer_count=None, stream=None,
                       q_indptr=None, total_rows=0):
        if layer_count is None:
            layer_count = self.cfg.num_layers - layer_begin
        self._check(self.lib.nsd_kv_prepare(self._h, _ptr(kv_pool), n_mig_blocks, _ptr(mig_src), _ptr(mig_dst), batch,
                                            gamma, _ptr(ctx_len), _ptr(kv_indptr), _ptr(kv_indices), _ptr(k_new),
                                            _ptr(v_new), _ptr(is_migrated), append_subset, layer_begin, layer_count,
                                            _ptr(q_indptr), int(total_rows), _stream_handle(stream)), "nsd_kv_prepare")

    def nsd_kv_commit(self, kv_pool, batch, gamma, ctx_len, acc_len, kv_indptr, kv_indices, exp_indptr, exp_indices,
                      new_ctx_len=None, layer_begin=0, layer_count=None, stream=None, q_indptr=None):
        if layer_count is None:
            layer_count = self.cfg.num_layers - layer_begin
        self._check(self.lib.nsd_kv_commit(self._h, _ptr(kv_pool), batch, gamma, _ptr(ctx_len), _ptr(acc_len),
                                           _ptr(kv_indptr), _ptr(kv_indices), _ptr(exp_indptr), _ptr(exp_indices),
                                           _ptr(new_ctx_len), layer_begin, layer_count, _ptr(q_indptr),
                                           _stream_handle(stream)), "nsd_kv_commit")

    def nsd_verify_attn(self, kv_pool, q, o, lse, batch, gamma, ctx_len, kv_indptr, kv_indices, layer=0, subset=0,
                        stream=None):
        self._check(self.lib.nsd_verify_attn(self._h, _ptr(kv_pool), _ptr(q), _ptr(o), _ptr(lse), batch, gamma,
                                             _ptr(ctx_len), _ptr(kv_indptr), _ptr(kv_indices), layer, subset,
                                             _stream_handle(stream)), "nsd_verify_attn")

    def nsd_spec_accept(self, p, q, draft_tok, u_acc, u_smp, batch, gamma, vocab, ctx_len, acc_len, out_tok,
                        new_ctx_len=None, stream=None, q_indptr=None):
        self._check(self.lib.nsd_spec_accept(self._h, _ptr(p), _ptr(q), _ptr(draft_tok), _ptr(u_acc), _ptr(u_smp),
                                             batch, gamma, vocab, _ptr(ctx_len), _ptr(acc_len), _ptr(out_tok),
                                             _ptr(new_ctx_len), _ptr(q_indptr), _stream_handle(stream)), "nsd_spec_accept")

    def nsd_spec_accept_logits(self, logits, logits_dtype, temperature, q, draft_tok, u_acc, u_smp, batch, gamma, vocab,
                               gamma_r, ctx_len, acc_len, out_tok, new_ctx_len=None, stream=None):
        self._check(self.lib.nsd_spec_accept_logits(self._h, _ptr(logits), logits_dtype, float(temperature), _ptr(q),
                                                    _ptr(draft_tok), _ptr(u_acc), _ptr(u_smp), batch, gamma, vocab,
                                                    _ptr(gamma_r), _ptr(ctx_len), _ptr(acc_len), _ptr(out_tok),
                                                    _ptr(new_ctx_len), _stream_handle(stream)), "nsd_spec_accept_logits")

    @staticmethod
    def round_args(**kw) -> RoundArgs:
        a = RoundArgs()
        a._keepalive = [v for v in kw.values() if hasattr(v, "data_ptr")]    # the struct holds raw addresses only
        for name, _ in RoundArgs._fields_:
            v = kw.pop(name, None)
            if name in ("n_mig_blocks", "batch", "gamma", "fuse_gather", "reserved"):
                setattr(a, name, int(v or 0))
            else:
                setattr(a, name, _ptr(v))
        assert not kw, f"unknown round arguments: {list(kw)}"
        return a

    def nsd_verify_round(self, args: RoundArgs, stream=None):
        self._check(self.lib.nsd_verify_round(self._h, ctypes.byref(args), _stream_handle(stream)), "nsd_verify_round")

    def nsd_verify_round_host(self, h_args: RoundArgs, d_args: RoundArgs, total_table_entries: int, stream=None):
        up, down = ctypes.c_int64(0), ctypes.c_int64(0)
        self._check(self.lib.nsd_verify_round_host(self._h, ctypes.byref(h_args), ctypes.byref(d_args),
                                                   total_table_entries, _stream_handle(stream), ctypes.byref(up),
                                                   ctypes.byref(down)), "nsd_verify_round_host")
        return up.value, down.value

    def nsd_launch_count(self) -> int:
        return int(self.lib.nsd_launch_count(self._h))

    def nsd_get_status(self, stream=None):
        bad = ctypes.c_int32(-1)
        rc = self.lib.nsd_get_status(self._h, _stream_handle(stream), ctypes.byref(bad))
        return rc, bad.value
