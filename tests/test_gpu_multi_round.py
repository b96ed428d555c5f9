"""Two consecutive verification rounds on one batch, chained the way a worker would chain them:
the first verification round (with reassigned requests) -> suffix commit to the export copy -> context lengths rolled forward
by the accepted lengths -> the second verification round appends over the rejected drafts.  Checked against the oracle run of
the same sequence."""
from dataclasses import replace

import numpy as np
import pytest
import torch

import oracle
import workload as W
from nsd_testlib import DeviceBatch, accept_compare, attn_mismatch, dev, guarded_pool, guards_intact, host_u16, make_context

pytestmark = pytest.mark.gpu


def test_two_rounds_with_commit_and_rolled_context():
    gamma, layers, slabs = 4, 3, 3
    # tables sized for two rounds' worth of appended tokens (gamma 9 -> room for ctx + 10)
    cfg_tab = W.RoundConfig("mr", batch=14, gamma=2 * gamma + 1, num_layers=layers, num_q_heads=32, num_kv_heads=8, head_dim=128,
                            block_size=16, vocab=1500, ctx_dist=("uniform", 1, 900), frac_reassigned=0.35, pool_factor=3.0, seed=190)
    cfg = replace(cfg_tab, gamma=gamma)
    meta = W.make_batch_meta(cfg_tab)                       # block tables with slack; context lengths are shared
    B, g1 = cfg.batch, gamma + 1
    pool0 = np.stack([W.pool_layer(cfg_tab, meta, s) for s in range(slabs)])
    ei, ex = W.export_tables(cfg_tab, meta)
    rounds = []
    for k in range(2):
        c = replace(cfg, seed=cfg.seed + 17 * k)
        kv = [W.new_kv(c, meta, l) for l in range(layers)]
        rounds.append(dict(k_new=np.stack([a for a, _ in kv]), v_new=np.stack([b for _, b in kv]),
                           q=np.stack([W.queries(c, meta, l) for l in range(layers)]), acc_in=W.accept_inputs(c)))

    # ---------------- oracle
    ref_pool = pool0.copy()
    ctx_len = meta.ctx_len.copy()
    ref = []
    for k, rd in enumerate(rounds):
        mig = (meta.mig_indptr, meta.mig_src, meta.mig_dst) if k == 0 else (np.zeros(1, np.int64), np.zeros(0, np.int32), np.zeros(0, np.int32))
        outs = []
        for l in range(layers):
            oracle.kv_prepare(ref_pool, *mig, ctx_len, meta.kv_indptr, meta.kv_indices, rd["k_new"], rd["v_new"], gamma, layer_begin=l, layer_count=1)
            outs.append(oracle.verify_attn(ref_pool, rd["q"][l], ctx_len, meta.kv_indptr, meta.kv_indices, gamma, layer=l))
        acc, out, _ = oracle.spec_accept(*rd["acc_in"])
        if k == 0:
            rc, new_ctx = oracle.kv_commit(ref_pool, ctx_len, acc, meta.kv_indptr, meta.kv_indices, ei, ex, gamma)
            assert rc == 0
        else:
            new_ctx = ctx_len + 1 + acc
        ref.append(dict(outs=outs, acc=acc, out=out, ctx_in=ctx_len.copy()))
        ctx_len = new_ctx.astype(np.int32)

    # ---------------- library
    ctx = make_context(cfg, meta, num_slabs=slabs, max_gamma=gamma)
    db = DeviceBatch(meta)
    buf, pool = guarded_pool(pool0)
    ctx_d = db.ctx_len.clone()
    got = []
    for k, rd in enumerate(rounds):
        p, qd, tok, ua, us = rd["acc_in"]
        o = torch.full(rd["q"].shape, 0x7FC0, dtype=torch.int16, device="cuda:0")
        acc = torch.full((B,), -7, dtype=torch.int32, device="cuda:0")
        out = torch.full((B, g1), -7, dtype=torch.int32, device="cuda:0")
        new_ctx = torch.zeros(B, dtype=torch.int32, device="cuda:0")
        first = k == 0
        h_ctx = ctx_d.cpu().numpy()                          # the scheduler knows the lengths
        ctx.nsd_verify_plan(h_ctx, meta.kv_indptr, meta.is_migrated if first else None, gamma)
        args = ctx.round_args(kv_pool=pool, n_mig_blocks=db.n_mig_blocks if first else 0, mig_src=db.mig_src if first else None,
                              mig_dst=db.mig_dst if first else None, batch=B, gamma=gamma, ctx_len=ctx_d, kv_indptr=db.kv_indptr,
                              kv_indices=db.kv_indices, is_migrated=db.is_migrated if first else None, k_new=dev(rd["k_new"]),
                              v_new=dev(rd["v_new"]), q=dev(rd["q"]), o=o, p=dev(p), q_draft=dev(qd), draft_tok=dev(tok),
                              u_acc=dev(ua), u_smp=dev(us), acc_len=acc, out_tok=out, new_ctx_len=new_ctx)
        ctx.nsd_verify_round(args)
        if first:
            ctx.nsd_kv_commit(pool, B, gamma, ctx_d, acc, db.kv_indptr, db.kv_indices, dev(ei), dev(ex))
        rc, bad = ctx.nsd_get_status()
        assert rc == 0, (k, rc, bad)
        got.append(dict(o=host_u16(o), acc=acc.cpu().numpy(), out=out.cpu().numpy()))
        ctx_d = new_ctx

    assert guards_intact(buf)
    for k in range(2):
        assert np.array_equal(got[k]["acc"], ref[k]["acc"]), k
        rep = accept_compare(*rounds[k]["acc_in"], got[k]["acc"], got[k]["out"], ref[k]["acc"], ref[k]["out"])
        assert rep["len_exact"] == B
        for l in range(layers):
            bad, max_abs, max_rel = attn_mismatch(got[k]["o"][l], ref[k]["outs"][l])
            assert bad == 0, (k, l, bad, max_abs, max_rel)
    assert np.array_equal(ctx_d.cpu().numpy(), ctx_len)
    assert np.array_equal(host_u16(pool).reshape(ref_pool.shape), ref_pool)
    assert (ref[1]["ctx_in"] > ref[0]["ctx_in"]).all()
