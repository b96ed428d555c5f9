"""GPU parity: nsd_kv_prepare against the oracle, whole pool bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import workload as W
from nsd_testlib import DeviceBatch, dev, guarded_pool, guards_intact, host_u16, make_context, stack_layers

pytestmark = pytest.mark.gpu

SMALL = W.RoundConfig("kv_small", batch=6, gamma=4, num_layers=3, num_q_heads=8, num_kv_heads=2, head_dim=64,
                      block_size=16, vocab=100, ctx_dist=("fixed", [1, 15, 16, 17, 47, 64]), frac_reassigned=0.5, seed=41)
RAGGED = W.RoundConfig("kv_ragged", batch=19, gamma=6, num_layers=2, num_q_heads=32, num_kv_heads=8, head_dim=128,
                       block_size=16, vocab=100, ctx_dist=("uniform", 1, 700), frac_reassigned=0.6, seed=42)


def _run(cfg, slabs, append=True, split_calls=False, subsets=False):
    meta = W.make_batch_meta(cfg)
    pool0 = np.stack([W.pool_layer(cfg, meta, s) for s in range(slabs)])
    k_new, v_new = stack_layers(cfg, meta, "kv")
    want = pool0.copy()
    assert oracle.kv_prepare(want, meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr,
                             meta.kv_indices, k_new if append else None, v_new if append else None, cfg.gamma,
                             layer_count=cfg.num_layers) == 0
    ctx = make_context(cfg, meta, num_slabs=slabs)
    db = DeviceBatch(meta)
    buf, pool = guarded_pool(pool0)
    kd, vd = (dev(k_new), dev(v_new)) if append else (None, None)
    common = (pool, db.n_mig_blocks, db.mig_src, db.mig_dst, cfg.batch, cfg.gamma, db.ctx_len, db.kv_indptr,
              db.kv_indices, kd, vd)
    if subsets:
        # gather + reassigned append, then resident append, as the fused round issues them
        for l in range(cfg.num_layers):
            ctx.nsd_kv_prepare(*common, is_migrated=db.is_migrated, append_subset=2, layer_begin=l, layer_count=1)
            ctx.nsd_kv_prepare(pool, 0, None, None, cfg.batch, cfg.gamma, db.ctx_len, db.kv_indptr, db.kv_indices,
                               kd, vd, is_migrated=db.is_migrated, append_subset=1, layer_begin=l, layer_count=1)
    elif split_calls:
        ctx.nsd_kv_prepare(*common, layer_begin=0, layer_count=1)
        ctx.nsd_kv_prepare(*common, layer_begin=1, layer_count=cfg.num_layers - 1)
    else:
        ctx.nsd_kv_prepare(*common)
    rc, bad = ctx.nsd_get_status()
    assert rc == 0, (rc, bad)
    got = host_u16(pool).reshape(want.shape)
    assert guards_intact(buf)
    return meta, pool0, want, got, ctx, (common, db)


@pytest.mark.parametrize("cfg,slabs", [(W.CONFIGS["tiny"], 1), (SMALL, 3), (SMALL, 2), (RAGGED, 2), (RAGGED, 1)],
                         ids=["tiny", "small_3slabs", "small_alias2", "ragged", "ragged_alias1"])
def test_pool_bit_exact(cfg, slabs):
    meta, pool0, want, got, *_ = _run(cfg, slabs)
    assert np.array_equal(got, want)
    assert not np.array_equal(got, pool0)
    assert np.array_equal(got[:, :meta.region_b_begin], pool0[:, :meta.region_b_begin])     # sources untouched


def test_gather_only_and_idempotent():
    meta, pool0, want, got, ctx, (common, db) = _run(SMALL, 3, append=False)
    assert np.array_equal(got, want)
    ctx.nsd_kv_prepare(*common)                          # again on the already-prepared pool
    torch.cuda.synchronize()
    assert np.array_equal(host_u16(common[0]).reshape(want.shape), want)


def test_layer_range_split_and_subset_order_equal_one_call():
    _, _, want, got_split, *_ = _run(SMALL, 2, split_calls=True)
    assert np.array_equal(got_split, want)
    _, _, want2, got_sub, *_ = _run(RAGGED, 2, subsets=True)
    assert np.array_equal(got_sub, want2)


def test_qwen3_b64_config():
    cfg = W.CONFIGS["qwen3_b64"]
    meta, pool0, want, got, *_ = _run(cfg, 1)
    assert np.array_equal(got, want)


def test_empty_batch_and_no_migration_are_noops():
    cfg = W.RoundConfig("nomig", batch=3, gamma=2, num_layers=1, num_q_heads=8, num_kv_heads=2, head_dim=64,
                        block_size=16, vocab=100, ctx_dist=("fixed", [5, 16, 33]), frac_reassigned=0.0, seed=43)
    meta, pool0, want, got, ctx, (common, db) = _run(cfg, 1)
    assert meta.n_mig == 0 and np.array_equal(got, want)
    before = host_u16(common[0]).copy()
    ctx.nsd_kv_prepare(common[0], 0, None, None, 0, cfg.gamma, None, None, None, None, None)
    torch.cuda.synchronize()
    assert np.array_equal(host_u16(common[0]), before)


def test_bad_arguments_return_codes_and_touch_nothing():
    import paper_2609_29364_b200 as nsd

    cfg = SMALL
    meta = W.make_batch_meta(cfg)
    ctx = make_context(cfg, meta, num_slabs=3)
    db = DeviceBatch(meta)
    pool0 = np.stack([W.pool_layer(cfg, meta, s) for s in range(3)])
    buf, pool = guarded_pool(pool0)
    k_new, v_new = stack_layers(cfg, meta, "kv")
    kd, vd = dev(k_new), dev(v_new)
    launches = ctx.nsd_launch_count()

    def code(*a, **k):
        with pytest.raises(nsd.NsdError) as e:
            ctx.nsd_kv_prepare(*a, **k)
        return e.value.code

    base = (pool, db.n_mig_blocks, db.mig_src, db.mig_dst, cfg.batch, cfg.gamma, db.ctx_len, db.kv_indptr, db.kv_indices, kd, vd)
    assert code(None, *base[1:]) == 1                                   # null pool
    assert code(*base, layer_begin=2, layer_count=2) == 2               # layers past the end
    assert code(*base[:5], cfg.gamma + 1, *base[6:]) == 2               # gamma above max_gamma
    assert code(*base[:4], cfg.batch + 1, *base[5:]) == 2               # batch above max_batch
    assert code(*base[:2], None, *base[3:]) == 1                        # pairs without a source list
    assert code(*base[:9], kd, None) == 1                               # K without V
    assert code(*base, append_subset=2) == 1                            # subset without flags
    torch.cuda.synchronize()
    assert ctx.nsd_launch_count() == launches
    assert np.array_equal(host_u16(pool).reshape(pool0.shape), pool0)


def test_out_of_range_block_id_is_reported_not_followed():
    cfg = SMALL
    meta = W.make_batch_meta(cfg)
    ctx = make_context(cfg, meta, num_slabs=1)
    db = DeviceBatch(meta)
    pool0 = W.pool_layer(cfg, meta, 0)[None]
    buf, pool = guarded_pool(pool0)
    bad_dst = meta.mig_dst.copy()
    bad_dst[0] = meta.num_blocks + 5
    ctx.nsd_kv_prepare(pool, db.n_mig_blocks, db.mig_src, dev(bad_dst), 0, cfg.gamma, None, None, None, None, None,
                       layer_count=1)
    rc, _ = ctx.nsd_get_status()
    assert rc == 6                                                      # NSD_ERR_DEVICE_FAULT
    assert guards_intact(buf)
    rc, _ = ctx.nsd_get_status()
    assert rc == 0                                                      # the word is cleared by the read
    got = host_u16(pool).reshape(pool0.shape)
    assert np.array_equal(got[0, meta.mig_dst[1:]], pool0[0, meta.mig_src[1:]])
