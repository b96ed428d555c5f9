"""Pins of the oracle's per-request draft depth (ragged rows): a batch may mix depths (Appendix G.2 runs the draft side at
depths 3, 4 and 5, and the target verifies "anchor plus proposal" tokens of each request).  The ragged forms are tied to
the uniform ones, which have pins of their own: a depth vector that is constant changes nothing, and every request of a
mixed batch gets exactly what it gets when it is run alone at its own depth."""
import numpy as np

import oracle
import workload as W

CFG = W.RoundConfig("ragged", batch=9, gamma=6, num_layers=2, num_q_heads=8, num_kv_heads=2, head_dim=64, block_size=16,
                    vocab=300, ctx_dist=("fixed", [0, 1, 15, 16, 17, 40, 63, 100, 33]), frac_reassigned=0.34, seed=4242)


def _inputs(cfg):
    meta = W.make_batch_meta(cfg)
    pool = np.stack([W.pool_layer(cfg, meta, l) for l in range(cfg.num_layers)])
    kv = [W.new_kv(cfg, meta, l) for l in range(cfg.num_layers)]
    k_new, v_new = np.stack([a for a, _ in kv]), np.stack([b for _, b in kv])
    q = np.stack([W.queries(cfg, meta, l) for l in range(cfg.num_layers)])
    return meta, pool, k_new, v_new, q


def _single(cfg, r, g_r):
    """Request r alone, at uniform depth g_r, keeping its own blocks (tables renumbered to start at zero)."""
    return W.RoundConfig(**{**cfg.__dict__, "batch": 1, "gamma": int(g_r)})


def test_constant_depth_vector_changes_nothing():
    cfg = CFG
    meta, pool, k_new, v_new, q = _inputs(cfg)
    g = np.full(cfg.batch, cfg.gamma, dtype=np.int32)
    a, b = pool.copy(), pool.copy()
    oracle.kv_prepare(a, meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr, meta.kv_indices, k_new, v_new, cfg.gamma)
    oracle.kv_prepare(b, meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr, meta.kv_indices, k_new, v_new, cfg.gamma, gamma_r=g)
    assert np.array_equal(a, b)
    oa = oracle.verify_attn(a, q[1], meta.ctx_len, meta.kv_indptr, meta.kv_indices, cfg.gamma, layer=1)
    ob = oracle.verify_attn(a, q[1], meta.ctx_len, meta.kv_indptr, meta.kv_indices, cfg.gamma, layer=1, gamma_r=g)
    assert np.array_equal(oa, ob)
    p, qd, tok, ua, us = W.accept_inputs(cfg)
    acc_a, out_a, _ = oracle.spec_accept(p, qd, tok, ua, us)
    V = cfg.vocab
    acc_b, out_b, _ = oracle.spec_accept(p.reshape(-1, V), qd.reshape(-1, V), tok.reshape(-1), ua.reshape(-1), us, gamma_r=g, gamma=cfg.gamma)
    assert np.array_equal(acc_a, acc_b) and np.array_equal(out_a.reshape(-1), out_b)


def test_mixed_depths_equal_each_request_run_alone():
    cfg = CFG
    meta, pool, k_new, v_new, q = _inputs(cfg)
    gamma_r = W.draw_gamma_r(cfg)
    gamma_r[0], gamma_r[1] = 0, cfg.gamma                      # both ends of the range are present
    assert len(set(gamma_r.tolist())) >= 4
    rows, drafts, row_indptr = W.ragged_index(gamma_r, cfg.gamma)
    k_r, v_r, q_r = (np.ascontiguousarray(x[:, rows]) for x in (k_new, v_new, q))
    got = pool.copy()
    assert oracle.kv_prepare(got, meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr, meta.kv_indices,
                             k_r, v_r, cfg.gamma, gamma_r=gamma_r) == 0
    o_got = oracle.verify_attn(got, q_r[1], meta.ctx_len, meta.kv_indptr, meta.kv_indices, cfg.gamma, layer=1, gamma_r=gamma_r)
    p, qd, tok, ua, us = W.accept_inputs(cfg)
    V = cfg.vocab
    p_r, qd_r = np.ascontiguousarray(p.reshape(-1, V)[rows]), np.ascontiguousarray(qd.reshape(-1, V)[drafts])
    tok_r, ua_r = np.ascontiguousarray(tok.reshape(-1)[drafts]), np.ascontiguousarray(ua.reshape(-1)[drafts])
    acc_got, out_got, new_got = oracle.spec_accept(p_r, qd_r, tok_r, ua_r, us, ctx_len=meta.ctx_len, gamma_r=gamma_r, gamma=cfg.gamma)

    # the same, one request at a time through the uniform forms
    want = pool.copy()
    mig_of = {int(r): m for m, r in enumerate(meta.mig_req)}
    for r in range(cfg.batch):
        g = int(gamma_r[r])
        sl = slice(int(row_indptr[r]), int(row_indptr[r + 1]))
        one = slice(r, r + 1)
        tbl = meta.kv_indices[meta.kv_indptr[r]:meta.kv_indptr[r + 1]]
        indptr1 = np.array([0, len(tbl)], dtype=np.int64)
        if r in mig_of:
            m = mig_of[r]
            e = slice(int(meta.mig_indptr[m]), int(meta.mig_indptr[m + 1]))
            mi, ms, md = np.array([0, e.stop - e.start], dtype=np.int64), meta.mig_src[e].copy(), meta.mig_dst[e].copy()
        else:
            mi, ms, md = np.zeros(1, dtype=np.int64), np.zeros(0, np.int32), np.zeros(0, np.int32)
        assert oracle.kv_prepare(want, mi, ms, md, meta.ctx_len[one].copy(), indptr1, tbl.copy(),
                                 np.ascontiguousarray(k_r[:, sl]), np.ascontiguousarray(v_r[:, sl]), g) == 0
        o1 = oracle.verify_attn(want, np.ascontiguousarray(q_r[1, sl]), meta.ctx_len[one].copy(), indptr1, tbl.copy(), g, layer=1)
        assert np.array_equal(o1, o_got[sl]), r
        d0 = int(row_indptr[r]) - r
        acc1, out1, new1 = oracle.spec_accept(p_r[sl][None], qd_r[d0:d0 + g][None], tok_r[d0:d0 + g][None], ua_r[d0:d0 + g][None],
                                              us[one].copy(), ctx_len=meta.ctx_len[one].copy())
        assert acc1[0] == acc_got[r] and np.array_equal(out1[0], out_got[sl]) and new1[0] == new_got[r], r
        assert 0 <= acc_got[r] <= g and (out_got[sl][:acc_got[r] + 1] >= 0).all() and (out_got[sl][acc_got[r] + 1:] == -1).all()
    assert np.array_equal(got, want)
    assert acc_got[0] == 0 and out_got[0] >= 0                 # no drafts: the anchor row yields the only token


def test_commit_honours_the_request_depth():
    cfg = CFG
    meta, pool, k_new, v_new, q = _inputs(cfg)
    gamma_r = W.draw_gamma_r(cfg)
    rows, _, _ = W.ragged_index(gamma_r, cfg.gamma)
    work = pool.copy()
    oracle.kv_prepare(work, meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr, meta.kv_indices,
                      np.ascontiguousarray(k_new[:, rows]), np.ascontiguousarray(v_new[:, rows]), cfg.gamma, gamma_r=gamma_r)
    exp_indptr, exp_indices = W.export_tables(cfg, meta)
    acc = np.minimum(gamma_r, np.arange(cfg.batch, dtype=np.int32) % 4).astype(np.int32)
    a, b = work.copy(), work.copy()
    rc_a, new_a = oracle.kv_commit(a, meta.ctx_len, acc, meta.kv_indptr, meta.kv_indices, exp_indptr, exp_indices, cfg.gamma)
    rc_b, new_b = oracle.kv_commit(b, meta.ctx_len, acc, meta.kv_indptr, meta.kv_indices, exp_indptr, exp_indices, cfg.gamma, gamma_r=gamma_r)
    assert rc_a == 0 and rc_b == 0 and np.array_equal(a, b) and np.array_equal(new_a, new_b)
    bad = acc.copy()
    r = int(np.argmin(gamma_r))
    bad[r] = gamma_r[r] + 1                                     # more accepted than were drafted
    if bad[r] <= cfg.gamma:
        rc_c, _ = oracle.kv_commit(work.copy(), meta.ctx_len, bad, meta.kv_indptr, meta.kv_indices, exp_indptr, exp_indices, cfg.gamma, gamma_r=gamma_r)
        assert rc_c != 0
