"""GPU parity: nsd_kv_commit (suffix export after acceptance) against the oracle, whole pool bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import workload as W
from nsd_testlib import DeviceBatch, dev, guarded_pool, guards_intact, host_u16, make_context, stack_layers

pytestmark = pytest.mark.gpu


def _cfg(name, batch, gamma, ctx, layers, d=128, hq=32, hkv=8, seed=70):
    return W.RoundConfig(name, batch=batch, gamma=gamma, num_layers=layers, num_q_heads=hq, num_kv_heads=hkv, head_dim=d,
                         block_size=16, vocab=100, ctx_dist=ctx, frac_reassigned=0.3, pool_factor=3.0, seed=seed)


@pytest.mark.parametrize("cfg,slabs", [(_cfg("c_small", 7, 4, ("fixed", [0, 11, 12, 15, 16, 47, 90]), 3, d=64, hq=8, hkv=2), 3),
                                       (_cfg("c_ragged", 40, 6, ("uniform", 0, 900), 4), 2),
                                       (_cfg("c_g8", 9, 8, ("uniform", 1, 300), 2), 2)], ids=["small", "ragged_alias", "gamma8"])
def test_commit_bit_exact(cfg, slabs):
    meta = W.make_batch_meta(cfg)
    pool0 = np.stack([W.pool_layer(cfg, meta, s) for s in range(slabs)])
    k_new, v_new = stack_layers(cfg, meta, "kv")
    oracle.kv_prepare(pool0, meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr, meta.kv_indices,
                      k_new, v_new, cfg.gamma)
    ei, ex = W.export_tables(cfg, meta)
    acc = np.random.default_rng(cfg.seed).integers(0, cfg.gamma + 1, size=cfg.batch).astype(np.int32)
    acc[0], acc[-1] = 0, cfg.gamma
    want = pool0.copy()
    rc, new_ref = oracle.kv_commit(want, meta.ctx_len, acc, meta.kv_indptr, meta.kv_indices, ei, ex, cfg.gamma,
                                   layer_count=cfg.num_layers)
    assert rc == 0
    ctx = make_context(cfg, meta, num_slabs=slabs)
    db = DeviceBatch(meta)
    buf, pool = guarded_pool(pool0)
    new_ctx = torch.full((cfg.batch,), -7, dtype=torch.int32, device="cuda:0")
    ctx.nsd_kv_commit(pool, cfg.batch, cfg.gamma, db.ctx_len, dev(acc), db.kv_indptr, db.kv_indices, dev(ei), dev(ex), new_ctx)
    rc, bad = ctx.nsd_get_status()
    assert rc == 0, (rc, bad)
    assert guards_intact(buf)
    assert np.array_equal(host_u16(pool).reshape(want.shape), want)
    assert not np.array_equal(want, pool0)
    assert np.array_equal(new_ctx.cpu().numpy(), new_ref)
    assert ctx.nsd_launch_count() == cfg.num_layers


def test_commit_follows_the_round_on_the_stream():
    """Enqueued right behind nsd_verify_round, with the accepted lengths still on the device."""
    cfg = _cfg("c_round", 12, 4, ("uniform", 1, 500), 2, seed=71)
    cfg = W.RoundConfig(**{**cfg.__dict__, "vocab": 2000})
    meta = W.make_batch_meta(cfg)
    pool0 = np.stack([W.pool_layer(cfg, meta, s) for s in range(2)])
    k_new, v_new = stack_layers(cfg, meta, "kv")
    q = stack_layers(cfg, meta, "q")
    p, qd, tok, ua, us = W.accept_inputs(cfg)
    ei, ex = W.export_tables(cfg, meta)
    ctx = make_context(cfg, meta)
    db = DeviceBatch(meta)
    buf, pool = guarded_pool(pool0)
    B, g1 = cfg.batch, cfg.gamma + 1
    acc = torch.zeros(B, dtype=torch.int32, device="cuda:0")
    out = torch.zeros((B, g1), dtype=torch.int32, device="cuda:0")
    new_ctx = torch.zeros(B, dtype=torch.int32, device="cuda:0")
    args = ctx.round_args(kv_pool=pool, n_mig_blocks=db.n_mig_blocks, mig_src=db.mig_src, mig_dst=db.mig_dst, batch=B,
                          gamma=cfg.gamma, ctx_len=db.ctx_len, kv_indptr=db.kv_indptr, kv_indices=db.kv_indices,
                          is_migrated=db.is_migrated, k_new=dev(k_new), v_new=dev(v_new), q=dev(q),
                          o=torch.zeros(q.shape, dtype=torch.int16, device="cuda:0"), p=dev(p), q_draft=dev(qd),
                          draft_tok=dev(tok), u_acc=dev(ua), u_smp=dev(us), acc_len=acc, out_tok=out)
    ctx.nsd_verify_plan(meta.ctx_len, meta.kv_indptr, meta.is_migrated, cfg.gamma)
    ctx.nsd_verify_round(args)
    ctx.nsd_kv_commit(pool, B, cfg.gamma, db.ctx_len, acc, db.kv_indptr, db.kv_indices, dev(ei), dev(ex), new_ctx)
    rc, bad = ctx.nsd_get_status()
    assert rc == 0, (rc, bad)
    want = pool0.copy()
    oracle.kv_prepare(want, meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr, meta.kv_indices,
                      k_new, v_new, cfg.gamma)
    acc_ref, _, _ = oracle.spec_accept(p, qd, tok, ua, us)
    _, new_ref = oracle.kv_commit(want, meta.ctx_len, acc_ref, meta.kv_indptr, meta.kv_indices, ei, ex, cfg.gamma)
    assert np.array_equal(acc.cpu().numpy(), acc_ref)
    assert np.array_equal(host_u16(pool).reshape(want.shape), want)
    assert np.array_equal(new_ctx.cpu().numpy(), new_ref)


def test_commit_bad_arguments_and_bad_lengths():
    import paper_2609_29364_b200 as nsd

    cfg = _cfg("c_bad", 4, 4, ("fixed", [5, 16, 33, 70]), 2, d=64, hq=8, hkv=2)
    meta = W.make_batch_meta(cfg)
    ctx = make_context(cfg, meta)
    db = DeviceBatch(meta)
    pool0 = np.stack([W.pool_layer(cfg, meta, s, poison=False) for s in range(2)])
    buf, pool = guarded_pool(pool0)
    ei, ex = W.export_tables(cfg, meta)
    acc = dev(np.array([1, 9, 0, 2], dtype=np.int32))                  # 9 > gamma
    good = (pool, cfg.batch, cfg.gamma, db.ctx_len, acc, db.kv_indptr, db.kv_indices, dev(ei), dev(ex))
    for args, kw, want in (((None,) + good[1:], {}, 1), (good[:1] + (5,) + good[2:], {}, 2), (good[:2] + (9,) + good[3:], {}, 2),
                           (good, dict(layer_begin=1, layer_count=2), 2), (good[:4] + (None,) + good[5:], {}, 1)):
        with pytest.raises(nsd.NsdError) as e:
            ctx.nsd_kv_commit(*args, **kw)
        assert e.value.code == want
    assert ctx.nsd_launch_count() == 0
    ctx.nsd_kv_commit(*good)
    rc, bad = ctx.nsd_get_status()
    assert rc == 6 and bad == 1                                        # request 1 carries an impossible length
    assert guards_intact(buf)
