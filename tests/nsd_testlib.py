"""Shared plumbing of the GPU parity tests: move generated inputs to the device,
call the C ABI through the binding, fetch results, and compare with the oracle
under the stated tolerances."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import workload as W

ATTN_ATOL, ATTN_RTOL = 1e-2, 2e-2          # bf16 output vs fp32 oracle, elementwise
TOKEN_CDF_TOL = 1e-5                       # a differing token is tolerated only this close to a CDF boundary


def dev(a, device="cuda:0"):
    """numpy -> CUDA tensor; uint16 bf16 patterns travel as int16 (same bytes)."""
    if a is None:
        return None
    if a.dtype == np.uint16:
        a = a.view(np.int16)
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


def host_u16(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint16)


CONTEXT_FLAGS = 0                          # nsd_config.flags of the contexts made here; tests that compare kernels patch it


def make_context(cfg: W.RoundConfig, meta: W.BatchMeta, num_slabs=None, max_gamma=None, flags=None, wait_budget=0):
    import paper_2609_29364_b200 as nsd

    return nsd.VerifyContext(flags=CONTEXT_FLAGS if flags is None else flags, wait_budget=wait_budget,
                             num_layers=cfg.num_layers, num_slabs=num_slabs or cfg.num_layers,
                             num_q_heads=cfg.num_q_heads, num_kv_heads=cfg.num_kv_heads, head_dim=cfg.head_dim,
                             block_size=cfg.block_size, num_blocks=meta.num_blocks,
                             region_b_begin=meta.region_b_begin, max_batch=cfg.batch,
                             max_gamma=max_gamma or cfg.gamma, vocab_size=cfg.vocab,
                             max_table_entries=max(1, int(meta.kv_indptr[-1])))


class DeviceBatch:
    """Device copies of a batch's tables."""

    def __init__(self, meta: W.BatchMeta):
        self.ctx_len = dev(meta.ctx_len)
        self.kv_indptr = dev(meta.kv_indptr)
        self.kv_indices = dev(meta.kv_indices)
        self.is_migrated = dev(meta.is_migrated)
        self.mig_src = dev(meta.mig_src) if len(meta.mig_src) else None
        self.mig_dst = dev(meta.mig_dst) if len(meta.mig_dst) else None
        self.n_mig_blocks = int(len(meta.mig_src))


def guarded_pool(pool_np: np.ndarray, guard_elems: int = 4096):
    """Device pool with canary areas before and after; returns (buffer, pool view)."""
    flat = pool_np.reshape(-1).view(np.int16)
    buf = torch.full((flat.size + 2 * guard_elems,), 0x5A5A, dtype=torch.int16, device="cuda:0")
    view = buf[guard_elems:guard_elems + flat.size]
    view.copy_(torch.from_numpy(flat))
    return buf, view


def guards_intact(buf: torch.Tensor, guard_elems: int = 4096) -> bool:
    return bool((buf[:guard_elems] == 0x5A5A).all() and (buf[-guard_elems:] == 0x5A5A).all())


def stack_layers(cfg, meta, what):
    if what == "kv":
        kv = [W.new_kv(cfg, meta, l) for l in range(cfg.num_layers)]
        return np.stack([a for a, _ in kv]), np.stack([b for _, b in kv])
    return np.stack([W.queries(cfg, meta, l) for l in range(cfg.num_layers)])


def attn_mismatch(o_gpu_bits: np.ndarray, o_ref: np.ndarray, rows=None):
    """Returns (violations, max_abs, max_rel) of the bf16 output against the oracle."""
    got = W.bf16_to_f32(o_gpu_bits)
    if rows is not None:
        got, o_ref = got[rows], o_ref[rows]
    if not np.isfinite(got).all():
        return int((~np.isfinite(got)).sum()), float("inf"), float("inf")
    err = np.abs(got - o_ref)
    bad = err > ATTN_ATOL + ATTN_RTOL * np.abs(o_ref)
    rel = err / np.maximum(np.abs(o_ref), 1e-3)
    return int(bad.sum()), float(err.max()), float(rel.max())


def accept_compare(p, q, tok, u_acc, u_smp, acc_gpu, out_gpu, acc_ref, out_ref):
    """Applies the acceptance parity rule.  Returns a dict with exact-match and
    tolerated counts; raises AssertionError on a real mismatch.

    Accepted lengths must be equal unless the uniform at the position where the
    two sides part lies within 1e-5 of min(1, p/q) (reported).  The drawn token
    must be equal, or else have positive weight and an oracle CDF interval within
    1e-5 (as a fraction of the total) of the draw."""
    B, g1 = out_ref.shape
    g = g1 - 1
    report = dict(requests=B, len_exact=0, len_near_boundary=0, tok_exact=0, tok_tolerated=0)
    for r in range(B):
        if acc_gpu[r] != acc_ref[r]:
            i = int(min(acc_gpu[r], acc_ref[r]))
            x = tok[r, i]
            P, Q = float(p[r, i, x]), float(q[r, i, x])
            ratio = P / Q if Q > 0 else (1.0 if P > 0 else 0.0)
            assert abs(float(u_acc[r, i]) - min(1.0, ratio)) < 1e-5, f"request {r}: accepted length {acc_gpu[r]} != {acc_ref[r]}"
            report["len_near_boundary"] += 1
            continue
        report["len_exact"] += 1
        n = int(acc_ref[r])
        assert (out_gpu[r, :n] == out_ref[r, :n]).all() and (out_gpu[r, n + 1:] == -1).all(), f"request {r}: token layout"
        y_gpu, y_ref = int(out_gpu[r, n]), int(out_ref[r, n])
        if y_gpu == y_ref:
            report["tok_exact"] += 1
            continue
        if n < g:
            w = np.maximum(p[r, n] - q[r, n], np.float32(0)).astype(np.float64)
            if w.sum() == 0:
                w = p[r, n].astype(np.float64)
        else:
            w = p[r, g].astype(np.float64)
        C = np.cumsum(w)
        Z = C[-1]
        t = float(u_smp[r]) * Z
        assert 0 <= y_gpu < len(w) and w[y_gpu] > 0, f"request {r}: token {y_gpu} has no weight"
        lo = (C[y_gpu - 1] if y_gpu > 0 else 0.0) / Z - TOKEN_CDF_TOL
        hi = C[y_gpu] / Z + TOKEN_CDF_TOL
        assert lo <= t / Z <= hi, f"request {r}: token {y_gpu} vs {y_ref} outside the CDF tolerance"
        report["tok_tolerated"] += 1
    return report


def run_accept_gpu(ctx, p, q, tok, u_acc, u_smp, ctx_len=None):
    B, g1, V = p.shape
    acc = torch.full((B,), -7, dtype=torch.int32, device="cuda:0")
    out = torch.full((B, g1), -7, dtype=torch.int32, device="cuda:0")
    new_ctx = torch.full((B,), -7, dtype=torch.int32, device="cuda:0") if ctx_len is not None else None
    ctx.nsd_spec_accept(dev(p), dev(q), dev(tok), dev(u_acc), dev(u_smp), B, g1 - 1, V, dev(ctx_len), acc, out, new_ctx)
    torch.cuda.synchronize()
    return acc.cpu().numpy(), out.cpu().numpy(), (new_ctx.cpu().numpy() if new_ctx is not None else None)
