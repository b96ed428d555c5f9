"""GPU parity of per-request draft depths (ragged rows): one batch mixes depths 0..gamma, nothing is padded.  The whole
round (gather, append, attention in one launch per group of row widths, acceptance), its gather-through variant, the
host-buffer variant and the suffix commit against the oracle: pool bit for bit, attention within tolerance, accepted
lengths and tokens exact."""
import numpy as np
import pytest
import torch

import nsd_testlib
import oracle
import workload as W
from nsd_testlib import (DeviceBatch, accept_compare, attn_mismatch, dev, guarded_pool, guards_intact, host_u16,
                         make_context, stack_layers)

pytestmark = pytest.mark.gpu

MIX = W.RoundConfig("ragged_mix", batch=23, gamma=8, num_layers=3, num_q_heads=32, num_kv_heads=8, head_dim=128,
                    block_size=16, vocab=2000, ctx_dist=("uniform", 1, 1500), frac_reassigned=0.35, seed=9101)
SMALL = W.RoundConfig("ragged_small", batch=7, gamma=5, num_layers=2, num_q_heads=8, num_kv_heads=2, head_dim=64,
                      block_size=16, vocab=400, ctx_dist=("fixed", [0, 15, 16, 17, 100, 31, 64]), frac_reassigned=0.3, seed=9102)


def _ragged_inputs(cfg, meta, gamma_r):
    rows, drafts, q_indptr = W.ragged_index(gamma_r, cfg.gamma)
    k_new, v_new = stack_layers(cfg, meta, "kv")
    q = stack_layers(cfg, meta, "q")
    p, qd, tok, ua, us = W.accept_inputs(cfg)
    V = cfg.vocab
    cut = dict(k_new=np.ascontiguousarray(k_new[:, rows]), v_new=np.ascontiguousarray(v_new[:, rows]), q=np.ascontiguousarray(q[:, rows]),
               p=np.ascontiguousarray(p.reshape(-1, V)[rows]), q_draft=np.ascontiguousarray(qd.reshape(-1, V)[drafts]),
               draft_tok=np.ascontiguousarray(tok.reshape(-1)[drafts]), u_acc=np.ascontiguousarray(ua.reshape(-1)[drafts]), u_smp=us)
    return cut, q_indptr


def _oracle_round(cfg, meta, pool0, x, gamma_r):
    pool = pool0.copy()
    outs = []
    for l in range(cfg.num_layers):
        oracle.kv_prepare(pool, meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr, meta.kv_indices,
                          x["k_new"], x["v_new"], cfg.gamma, layer_begin=l, layer_count=1, gamma_r=gamma_r)
        outs.append(oracle.verify_attn(pool, x["q"][l], meta.ctx_len, meta.kv_indptr, meta.kv_indices, cfg.gamma, layer=l, gamma_r=gamma_r))
    acc, out, new_ctx = oracle.spec_accept(x["p"], x["q_draft"], x["draft_tok"], x["u_acc"], x["u_smp"], meta.ctx_len,
                                           gamma_r=gamma_r, gamma=cfg.gamma)
    return pool, outs, acc, out, new_ctx


def _check_accept(cfg, x, gamma_r, q_indptr, acc_g, out_g, acc_r, out_r):
    """accept_compare works on padded arrays: scatter the ragged ones back (unused entries never take part)."""
    B, g, V = cfg.batch, cfg.gamma, cfg.vocab
    assert np.array_equal(acc_g, acc_r), (acc_g, acc_r)
    for r in range(B):
        a, b = int(q_indptr[r]), int(q_indptr[r + 1])
        assert np.array_equal(out_g[a:b][:acc_r[r]], out_r[a:b][:acc_r[r]]) and (out_g[a + acc_r[r] + 1:b] == -1).all(), r
    # the drawn tokens under the CDF tolerance rule, request by request through the padded checker
    pp = np.zeros((B, g + 1, V), np.float32); qq = np.zeros((B, g, V), np.float32)
    tt = np.zeros((B, g), np.int32); uu = np.zeros((B, g), np.float32)
    og = np.full((B, g + 1), -1, np.int32); orf = np.full((B, g + 1), -1, np.int32)
    for r in range(B):
        a, b = int(q_indptr[r]), int(q_indptr[r + 1])
        d0, n = a - r, b - a - 1
        pp[r, :n + 1] = x["p"][a:b]; qq[r, :n] = x["q_draft"][d0:d0 + n]
        tt[r, :n] = x["draft_tok"][d0:d0 + n]; uu[r, :n] = x["u_acc"][d0:d0 + n]
        og[r, :n + 1] = out_g[a:b]; orf[r, :n + 1] = out_r[a:b]
        if acc_r[r] == n and n < g:                          # bonus row of a shallower request: make the padded checker see it as one
            pp[r, g] = pp[r, n]
    rep = dict(tok_exact=0, tok_tolerated=0)
    for r in range(B):
        n = int(gamma_r[r])
        one = accept_compare(pp[r:r + 1, :n + 1], qq[r:r + 1, :n], tt[r:r + 1, :n], uu[r:r + 1, :n], x["u_smp"][r:r + 1],
                             acc_g[r:r + 1], og[r:r + 1, :n + 1], acc_r[r:r + 1], orf[r:r + 1, :n + 1])
        rep["tok_exact"] += one["tok_exact"]; rep["tok_tolerated"] += one["tok_tolerated"]
    assert rep["tok_exact"] >= B - 1, rep


def _run(cfg, slabs, fuse=False, host_variant=False, chunk_blocks=0, split_flag=0):
    meta = W.make_batch_meta(cfg)
    gamma_r = W.draw_gamma_r(cfg)
    gamma_r[0], gamma_r[1] = 0, cfg.gamma
    x, q_indptr = _ragged_inputs(cfg, meta, gamma_r)
    rows = int(q_indptr[-1])
    pool0 = np.stack([W.pool_layer(cfg, meta, s) for s in range(slabs)])
    ctx = make_context(cfg, meta, num_slabs=slabs, flags=split_flag)
    db = DeviceBatch(meta)
    buf, pool = guarded_pool(pool0)
    B = cfg.batch
    d = dict(kv_pool=pool, n_mig_blocks=db.n_mig_blocks, mig_src=db.mig_src, mig_dst=db.mig_dst, batch=B, gamma=cfg.gamma,
             ctx_len=db.ctx_len, kv_indptr=db.kv_indptr, kv_indices=db.kv_indices, is_migrated=db.is_migrated,
             k_new=dev(x["k_new"]), v_new=dev(x["v_new"]), q=dev(x["q"]),
             o=torch.full(x["q"].shape, 0x7FC0, dtype=torch.int16, device="cuda:0"), p=dev(x["p"]), q_draft=dev(x["q_draft"]),
             draft_tok=dev(x["draft_tok"]), u_acc=dev(x["u_acc"]), u_smp=dev(x["u_smp"]),
             acc_len=torch.full((B,), -7, dtype=torch.int32, device="cuda:0"),
             out_tok=torch.full((rows,), -7, dtype=torch.int32, device="cuda:0"),
             new_ctx_len=torch.full((B,), -7, dtype=torch.int32, device="cuda:0"), fuse_gather=int(fuse), q_indptr=dev(q_indptr))
    stream = torch.cuda.Stream()
    if host_variant:
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a.view(np.int16) if a.dtype == np.uint16 else a)).pin_memory()
        h = dict(kv_pool=None, n_mig_blocks=db.n_mig_blocks, mig_src=pin(meta.mig_src) if db.n_mig_blocks else None,
                 mig_dst=pin(meta.mig_dst) if db.n_mig_blocks else None, batch=B, gamma=cfg.gamma, ctx_len=pin(meta.ctx_len),
                 kv_indptr=pin(meta.kv_indptr), kv_indices=pin(meta.kv_indices), is_migrated=pin(meta.is_migrated),
                 k_new=pin(x["k_new"]), v_new=pin(x["v_new"]), q=pin(x["q"]), o=torch.zeros(x["q"].shape, dtype=torch.int16).pin_memory(),
                 p=pin(x["p"]), q_draft=pin(x["q_draft"]), draft_tok=pin(x["draft_tok"]), u_acc=pin(x["u_acc"]), u_smp=pin(x["u_smp"]),
                 acc_len=torch.zeros(B, dtype=torch.int32).pin_memory(), out_tok=torch.zeros(rows, dtype=torch.int32).pin_memory(),
                 new_ctx_len=torch.zeros(B, dtype=torch.int32).pin_memory(), fuse_gather=int(fuse), q_indptr=pin(q_indptr))
        for k in ("ctx_len", "kv_indptr", "kv_indices", "is_migrated", "k_new", "v_new", "q", "p", "q_draft", "draft_tok", "u_acc",
                  "u_smp", "q_indptr"):
            d[k] = torch.zeros_like(d[k])                    # everything must arrive through the call
        with torch.cuda.stream(stream):
            ctx.nsd_verify_round_host(ctx.round_args(**h), ctx.round_args(**d), int(meta.kv_indptr[-1]), stream=stream)
        o_gpu, acc_g, out_g, new_g = h["o"].numpy().view(np.uint16), h["acc_len"].numpy(), h["out_tok"].numpy(), h["new_ctx_len"].numpy()
    else:
        with torch.cuda.stream(stream):
            ctx.nsd_verify_plan(meta.ctx_len, meta.kv_indptr, meta.is_migrated, cfg.gamma, chunk_blocks=chunk_blocks, stream=stream,
                                h_q_indptr=q_indptr)
            for _ in range(2):
                ctx.nsd_verify_round(ctx.round_args(**d), stream=stream)
        stream.synchronize()
        o_gpu, acc_g, out_g, new_g = host_u16(d["o"]), d["acc_len"].cpu().numpy(), d["out_tok"].cpu().numpy(), d["new_ctx_len"].cpu().numpy()
    rc, bad = ctx.nsd_get_status(stream=stream)
    assert rc == 0, (rc, bad)
    assert guards_intact(buf)
    want_pool, outs, acc_r, out_r, new_r = _oracle_round(cfg, meta, pool0, x, gamma_r)
    assert np.array_equal(host_u16(pool).reshape(want_pool.shape), want_pool)
    for l in range(cfg.num_layers):
        bad, max_abs, max_rel = attn_mismatch(o_gpu[l], outs[l])
        assert bad == 0, (l, bad, max_abs, max_rel)
    _check_accept(cfg, x, gamma_r, q_indptr, acc_g, out_g, acc_r, out_r)
    assert (new_g == new_r).all()
    return ctx, meta, gamma_r, q_indptr, d, want_pool


@pytest.mark.parametrize("split_flag", [1 << 4, 1 << 5], ids=["split_first", "wait_first"])
def test_mixed_depths_round(split_flag):
    """Depths 0..8 at the Qwen3-8B group size: 4..36 stacked rows, the widest on the tcgen05 engine, the rest in one mma.sync launch."""
    _run(MIX, 2, split_flag=split_flag)


def test_mixed_depths_split_kv_and_small_heads():
    _run(MIX, 3, chunk_blocks=6)
    _run(SMALL, 2)
    _run(SMALL, 1, chunk_blocks=2)


def test_mixed_depths_gather_through_and_host_buffers():
    _run(MIX, 2, fuse=True)
    _run(SMALL, 2, fuse=True, chunk_blocks=2)
    _run(MIX, 2, host_variant=True)


def test_mixed_depths_commit():
    """The suffix commit takes each request's own depth as the bound of its accepted length."""
    cfg = SMALL
    ctx, meta, gamma_r, q_indptr, d, pool_after = _run(cfg, 2)
    exp_indptr, exp_indices = W.export_tables(cfg, meta)
    acc = d["acc_len"].cpu().numpy()
    buf, pool = guarded_pool(pool_after)
    new_ctx = torch.full((cfg.batch,), -7, dtype=torch.int32, device="cuda:0")
    ctx.nsd_kv_commit(pool, cfg.batch, cfg.gamma, d["ctx_len"], d["acc_len"], d["kv_indptr"], d["kv_indices"], dev(exp_indptr),
                      dev(exp_indices), new_ctx, q_indptr=d["q_indptr"])
    rc, bad = ctx.nsd_get_status()
    assert rc == 0, (rc, bad)
    want = pool_after.copy()
    rc_o, new_o = oracle.kv_commit(want, meta.ctx_len, acc, meta.kv_indptr, meta.kv_indices, exp_indptr, exp_indices, cfg.gamma, gamma_r=gamma_r)
    assert rc_o == 0 and np.array_equal(host_u16(pool).reshape(want.shape), want) and np.array_equal(new_ctx.cpu().numpy(), new_o)
    # more accepted than drafted is refused on the device
    bad_acc = acc.copy()
    r = int(np.argmin(gamma_r))
    bad_acc[r] = gamma_r[r] + 1
    ctx.nsd_kv_commit(pool, cfg.batch, cfg.gamma, d["ctx_len"], dev(bad_acc), d["kv_indptr"], d["kv_indices"], dev(exp_indptr),
                      dev(exp_indices), None, q_indptr=d["q_indptr"])
    rc, bad = ctx.nsd_get_status()
    assert rc == 6 and bad == r


def test_plan_refuses_impossible_depths():
    import paper_2609_29364_b200 as nsd

    cfg = SMALL
    meta = W.make_batch_meta(cfg)
    ctx = make_context(cfg, meta)
    q_indptr = np.arange(cfg.batch + 1, dtype=np.int64) * (cfg.gamma + 2)            # one row too many per request
    with pytest.raises(nsd.NsdError) as e:
        ctx.nsd_verify_plan(meta.ctx_len, meta.kv_indptr, None, cfg.gamma, h_q_indptr=q_indptr)
    assert e.value.code == 2 and ctx.nsd_launch_count() == 0
