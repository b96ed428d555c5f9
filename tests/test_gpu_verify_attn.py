"""GPU parity: nsd_verify_attn (after nsd_kv_prepare) against the fp64 oracle,
elementwise within |err| <= 1e-2 + 2e-2*|ref| on the bf16 output."""
import numpy as np
import pytest
import torch

import oracle
import workload as W
from nsd_testlib import (DeviceBatch, attn_mismatch, dev, guarded_pool, guards_intact, host_u16, make_context,
                         stack_layers)

pytestmark = pytest.mark.gpu


def _cfg(name, batch, gamma, ctx, hq=32, hkv=8, d=128, layers=1, frac=0.3, seed=50):
    return W.RoundConfig(name, batch=batch, gamma=gamma, num_layers=layers, num_q_heads=hq, num_kv_heads=hkv,
                         head_dim=d, block_size=16, vocab=100, ctx_dist=ctx, frac_reassigned=frac, seed=seed)


def _run(cfg, slabs=None, chunk_blocks=0, subset_pair=False, want_lse=False, pool_edit=None):
    slabs = slabs or cfg.num_layers
    meta = W.make_batch_meta(cfg)
    pool0 = np.stack([W.pool_layer(cfg, meta, s) for s in range(slabs)])
    if pool_edit is not None:
        pool_edit(pool0, meta)                                                  # in place, before anybody sees the pool
    k_new, v_new = stack_layers(cfg, meta, "kv")
    q = stack_layers(cfg, meta, "q")
    ctx = make_context(cfg, meta, num_slabs=slabs)
    db = DeviceBatch(meta)
    buf, pool = guarded_pool(pool0)
    kd, vd, qd = dev(k_new), dev(v_new), dev(q)
    o = torch.full(qd.shape, 0x7FC0, dtype=torch.int16, device="cuda:0")         # NaN until written
    lse = torch.full((cfg.num_layers, cfg.rows, cfg.num_q_heads), float("nan"), device="cuda:0") if want_lse else None
    ctx.nsd_verify_plan(meta.ctx_len, meta.kv_indptr, meta.is_migrated, cfg.gamma, chunk_blocks=chunk_blocks)
    ref_pool = pool0.copy()
    results = []
    for l in range(cfg.num_layers):
        ctx.nsd_kv_prepare(pool, db.n_mig_blocks, db.mig_src, db.mig_dst, cfg.batch, cfg.gamma, db.ctx_len,
                           db.kv_indptr, db.kv_indices, kd, vd, layer_begin=l, layer_count=1)
        for subset in ((1, 2) if subset_pair else (0,)):
            ctx.nsd_verify_attn(pool, qd[l], o[l], lse[l] if want_lse else None, cfg.batch, cfg.gamma, db.ctx_len,
                                db.kv_indptr, db.kv_indices, layer=l, subset=subset)
        oracle.kv_prepare(ref_pool, meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr,
                          meta.kv_indices, k_new, v_new, cfg.gamma, layer_begin=l, layer_count=1)
        results.append(oracle.verify_attn(ref_pool, q[l], meta.ctx_len, meta.kv_indptr, meta.kv_indices, cfg.gamma,
                                          layer=l, want_lse=True))
    rc, bad = ctx.nsd_get_status()
    assert rc == 0, (rc, bad)
    assert guards_intact(buf)
    o_gpu = host_u16(o)
    lse_gpu = lse.cpu().numpy() if want_lse else None
    return cfg, meta, o_gpu, lse_gpu, results


def _check(o_gpu, results, lse_gpu=None):
    for l, (o_ref, lse_ref) in enumerate(results):
        bad, max_abs, max_rel = attn_mismatch(o_gpu[l], o_ref)
        assert bad == 0, f"layer {l}: {bad} elements outside tolerance (max abs {max_abs:.3e}, max rel {max_rel:.3e})"
        if lse_gpu is not None:
            np.testing.assert_allclose(lse_gpu[l], lse_ref, rtol=2e-3, atol=2e-3)


def test_tiny_config():
    _, _, o, lse, res = _run(W.CONFIGS["tiny"], want_lse=True)
    _check(o, res, lse)


@pytest.mark.parametrize("gamma", [1, 3, 4, 6, 8, 12, 15])
def test_gamma_sweep_qwen_heads(gamma):
    """M = 4*(gamma+1) rows: 1..4 m-tiles, ragged lengths around block and tile edges."""
    cfg = _cfg(f"g{gamma}", batch=9, gamma=gamma, ctx=("fixed", [0, 1, 15, 16, 17, 31, 33, 200, 517]), seed=60 + gamma)
    _, _, o, lse, res = _run(cfg, want_lse=True)
    _check(o, res, lse)


@pytest.mark.parametrize("hq,hkv,d", [(8, 8, 64), (8, 1, 64), (16, 8, 128), (4, 4, 128)])
def test_group_sizes_and_head_dims(hq, hkv, d):
    cfg = _cfg(f"h{hq}_{hkv}_{d}", batch=5, gamma=4, ctx=("uniform", 1, 300), hq=hq, hkv=hkv, d=d, seed=71)
    _, _, o, _, res = _run(cfg)
    _check(o, res)


@pytest.mark.parametrize("chunk_blocks", [2, 4, 16, 0])
def test_split_kv_does_not_change_the_result(chunk_blocks):
    """Several chunks per request (down to one 32-key tile each) merged by the last
    finisher must agree with the oracle like the single-chunk path does."""
    cfg = _cfg("split", batch=7, gamma=4, ctx=("fixed", [5, 40, 100, 257, 600, 1023, 1500]), seed=72)
    _, _, o, lse, res = _run(cfg, chunk_blocks=chunk_blocks, want_lse=True)
    _check(o, res, lse)


def test_split_counters_reset_between_launches():
    cfg = _cfg("twice", batch=4, gamma=4, ctx=("fixed", [100, 300, 600, 900]), layers=3, seed=73)
    _, _, o, _, res = _run(cfg, slabs=2, chunk_blocks=4)
    _check(o, res)


def test_resident_then_reassigned_subsets_cover_everything():
    cfg = _cfg("subsets", batch=12, gamma=4, ctx=("uniform", 20, 900), layers=2, frac=0.5, seed=74)
    _, _, o, _, res = _run(cfg, subset_pair=True, chunk_blocks=8)
    _check(o, res)


def _grow_keys_along_the_context(steps):
    """Pool edit: the committed K rows of every request are multiplied by a factor that steps up along the context
    (`steps`: (first position, factor) in increasing order), so the largest score of a row rises by far more than
    2^8 several times on the way -- inside a tile's first keys, inside its last keys, several tiles in."""
    def edit(pool0, meta):
        for r in range(len(meta.ctx_len)):
            blocks = meta.kv_indices[meta.kv_indptr[r]:meta.kv_indptr[r + 1]]
            for (p0, f), nxt in zip(steps, list(steps[1:]) + [(1 << 30, 0.0)]):
                for pos in range(p0, min(nxt[0], int(meta.ctx_len[r]))):
                    k = pool0[:, blocks[pos // 16], 0, :, pos % 16, :]
                    pool0[:, blocks[pos // 16], 0, :, pos % 16, :] = W.f32_to_bf16(W.bf16_to_f32(k) * np.float32(f))
    return edit


@pytest.mark.parametrize("gamma", [4, 6, 8, 12])
def test_running_maximum_moves_late_and_often(gamma):
    """Both engines refresh a row's running maximum lazily and rescale what they have accumulated when it moves: with
    keys that grow along the context it moves in the first tile's second half, in a later tile's first and last keys,
    and again far into a long request, for rows that sit in different chunks of a split request too."""
    steps = ((70, 8.0), (200, 48.0), (390, 6.0), (640, 200.0), (1500, 3.0), (1700, 900.0))
    cfg = _cfg(f"late{gamma}", batch=9, gamma=gamma, ctx=("fixed", [50, 75, 130, 210, 400, 650, 1000, 1750, 2100]), frac=0.0, seed=181 + gamma)
    for chunk_blocks in (0, 16):
        _, _, o, lse, res = _run(cfg, chunk_blocks=chunk_blocks, want_lse=True, pool_edit=_grow_keys_along_the_context(steps))
        _check(o, res, lse)


def test_qwen3_b64_config():
    _, _, o, lse, res = _run(W.CONFIGS["qwen3_b64"], want_lse=True)
    _check(o, res, lse)


def test_plan_rejects_bad_tables_and_attn_requires_plan():
    import paper_2609_29364_b200 as nsd

    cfg = _cfg("bad", batch=3, gamma=4, ctx=("fixed", [10, 20, 30]))
    meta = W.make_batch_meta(cfg)
    ctx = make_context(cfg, meta)
    db = DeviceBatch(meta)
    dummy = torch.zeros(cfg.rows * cfg.num_q_heads * cfg.head_dim, dtype=torch.int16, device="cuda:0")
    pool = torch.zeros(ctx.pool_bytes() // 2, dtype=torch.int16, device="cuda:0")

    def code(fn, *a, **k):
        with pytest.raises(nsd.NsdError) as e:
            fn(*a, **k)
        return e.value.code

    attn_args = (pool, dummy, dummy, None, cfg.batch, cfg.gamma, db.ctx_len, db.kv_indptr, db.kv_indices)
    assert code(ctx.nsd_verify_attn, *attn_args) == 7                               # not planned
    neg = meta.ctx_len.copy(); neg[1] = -1
    assert code(ctx.nsd_verify_plan, neg, meta.kv_indptr, None, cfg.gamma) == 1
    short = meta.kv_indptr.copy(); short[1:] -= 1                                    # first table one entry short
    assert code(ctx.nsd_verify_plan, meta.ctx_len, short, None, cfg.gamma) == 1
    assert code(ctx.nsd_verify_plan, meta.ctx_len, meta.kv_indptr, None, cfg.gamma + 1) == 2
    assert code(ctx.nsd_verify_plan, meta.ctx_len, meta.kv_indptr, None, cfg.gamma, chunk_blocks=3) == 1
    big = np.concatenate([meta.ctx_len] * 2)
    assert code(ctx.nsd_verify_plan, big, np.concatenate([meta.kv_indptr, meta.kv_indptr[1:] + meta.kv_indptr[-1]]), None, cfg.gamma) == 2
    assert ctx.nsd_launch_count() == 0
    ctx.nsd_verify_plan(meta.ctx_len, meta.kv_indptr, None, cfg.gamma)
    assert code(ctx.nsd_verify_attn, *attn_args, layer=1) == 2
    assert code(ctx.nsd_verify_attn, *attn_args[:4], cfg.batch - 1, *attn_args[5:]) == 7   # plan is for another batch
    assert code(ctx.nsd_verify_attn, pool, None, *attn_args[2:]) == 1
    assert ctx.nsd_launch_count() == 0
    ctx.nsd_verify_plan(np.zeros(0, np.int32), np.zeros(1, np.int64), None, cfg.gamma)      # empty batch is fine
    ctx.nsd_verify_attn(pool, dummy, dummy, None, 0, cfg.gamma, db.ctx_len, db.kv_indptr, db.kv_indices)
    assert ctx.nsd_launch_count() == 0
