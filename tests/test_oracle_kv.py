"""Pins for the KV-prepare oracle: numpy fancy-index brute force, idempotence,
untouched source region and untouched bystander blocks, gather-before-append
order, and attention equality across the move."""
import numpy as np

import oracle
import workload as W


def _cfg(layers=1, slabs_seed=0, frac=0.5, gamma=4):
    return W.RoundConfig("kvpin", batch=6, gamma=gamma, num_layers=layers, num_q_heads=8, num_kv_heads=2, head_dim=64,
                         block_size=16, vocab=100, ctx_dist=("fixed", [1, 15, 16, 17, 47, 64]),
                         frac_reassigned=frac, seed=31 + slabs_seed)


def _inputs(cfg, slabs=None):
    meta = W.make_batch_meta(cfg)
    S = slabs or cfg.num_layers
    pool = np.stack([W.pool_layer(cfg, meta, s) for s in range(S)])
    kv = [W.new_kv(cfg, meta, l) for l in range(cfg.num_layers)]
    k_new = np.stack([a for a, _ in kv])
    v_new = np.stack([b for _, b in kv])
    return meta, pool, k_new, v_new


def _numpy_prepare(cfg, meta, pool, k_new, v_new):
    """Vectorised restatement: one fancy-index copy per layer, then scatter of the new rows."""
    out = pool.copy()
    S, g1, bs = pool.shape[0], cfg.gamma + 1, cfg.block_size
    for l in range(cfg.num_layers):
        s = l % S
        out[s, meta.mig_dst] = out[s, meta.mig_src]
        r = np.repeat(np.arange(cfg.batch), g1)
        t = np.tile(np.arange(g1), cfg.batch)
        pos = meta.ctx_len[r].astype(np.int64) + t
        blk = meta.kv_indices[meta.kv_indptr[r] + pos // bs]
        out[s, blk, 0, :, pos % bs, :] = k_new[l]
        out[s, blk, 1, :, pos % bs, :] = v_new[l]
    return out


def test_matches_numpy_brute_force_multi_layer():
    cfg = _cfg(layers=3)
    meta, pool, k_new, v_new = _inputs(cfg)
    want = _numpy_prepare(cfg, meta, pool, k_new, v_new)
    got = pool.copy()
    assert oracle.kv_prepare(got, meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr,
                             meta.kv_indices, k_new, v_new, cfg.gamma) == 0
    assert np.array_equal(got, want)
    assert not np.array_equal(got, pool)


def test_layers_alias_slabs_in_order():
    """Five logical layers over two physical slabs: layer l lands in slab l % 2 and
    the later layer's append wins."""
    cfg = _cfg(layers=5)
    meta, pool, k_new, v_new = _inputs(cfg, slabs=2)
    want = _numpy_prepare(cfg, meta, pool, k_new, v_new)
    got = pool.copy()
    oracle.kv_prepare(got, meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr,
                      meta.kv_indices, k_new, v_new, cfg.gamma)
    assert np.array_equal(got, want)
    # layer range split in two calls == one call
    got2 = pool.copy()
    for lb, lc in ((0, 2), (2, 3)):
        oracle.kv_prepare(got2, meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr,
                          meta.kv_indices, k_new, v_new, cfg.gamma, layer_begin=lb, layer_count=lc)
    assert np.array_equal(got2, want)


def test_idempotent_and_source_region_untouched():
    cfg = _cfg()
    meta, pool, k_new, v_new = _inputs(cfg)
    once = pool.copy()
    args = (meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr, meta.kv_indices, k_new, v_new, cfg.gamma)
    oracle.kv_prepare(once, *args)
    twice = once.copy()
    oracle.kv_prepare(twice, *args)
    assert np.array_equal(once, twice)
    assert np.array_equal(once[:, :meta.region_b_begin], pool[:, :meta.region_b_begin])
    # blocks that are neither a destination nor an append target keep their bytes
    g1, bs = cfg.gamma + 1, cfg.block_size
    touched = set(meta.mig_dst.tolist())
    for r in range(cfg.batch):
        for t in range(g1):
            touched.add(int(meta.kv_indices[meta.kv_indptr[r] + (meta.ctx_len[r] + t) // bs]))
    others = np.array(sorted(set(range(meta.num_blocks)) - touched))
    assert np.array_equal(once[:, others], pool[:, others])


def test_gather_without_append_copies_whole_blocks():
    cfg = _cfg()
    meta, pool, _, _ = _inputs(cfg)
    got = pool.copy()
    oracle.kv_prepare(got, meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr,
                      meta.kv_indices, None, None, cfg.gamma)
    assert np.array_equal(got[0, meta.mig_dst], pool[0, meta.mig_src])      # tail slots included, bit for bit
    mask = np.ones(meta.num_blocks, bool)
    mask[meta.mig_dst] = False
    assert np.array_equal(got[0, mask], pool[0, mask])


def test_append_lands_after_gather_in_shared_block():
    """ctx = 17: the append writes slots 1.. of the destination block the gather
    just filled; gathering afterwards would wipe it."""
    cfg = _cfg(frac=1.0)
    meta, pool, k_new, v_new = _inputs(cfg)
    got = pool.copy()
    oracle.kv_prepare(got, meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr,
                      meta.kv_indices, k_new, v_new, cfg.gamma)
    r = 3
    assert meta.ctx_len[r] == 17
    b = meta.kv_indices[meta.kv_indptr[r] + 1]
    row = r * (cfg.gamma + 1)
    assert np.array_equal(got[0, b, 0, :, 1, :], k_new[0, row])
    m = list(meta.mig_req).index(r)
    src = meta.mig_src[meta.mig_indptr[m] + 1]
    assert np.array_equal(got[0, b, :, :, 0, :], pool[0, src, :, :, 0, :])   # slot 0 came from the source block


def test_attention_equal_across_the_move():
    """Attention of a reassigned request over its source blocks before the gather
    equals attention over its destination blocks after it, bit for bit."""
    cfg = _cfg(frac=1.0)
    meta, pool, _, _ = _inputs(cfg)
    q = W.queries(cfg, meta, 0)
    bs, g = cfg.block_size, cfg.gamma
    # rows see keys up to ctx + i; keep only committed keys visible by shortening ctx by gamma + 1
    ctx_short = (meta.ctx_len - (g + 1)).astype(np.int32)
    keep = np.nonzero(ctx_short >= 0)[0].astype(np.int32)
    src_indptr = np.zeros(cfg.batch + 1, dtype=np.int64)
    src_indptr[1:] = np.cumsum((meta.ctx_len + bs - 1) // bs)
    before = oracle.verify_attn(pool, q, ctx_short, src_indptr, meta.mig_src, g, req_list=keep)
    after_pool = pool.copy()
    oracle.kv_prepare(after_pool, meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr,
                      meta.kv_indices, None, None, g)
    after = oracle.verify_attn(after_pool, q, ctx_short, meta.kv_indptr, meta.kv_indices, g, req_list=keep)
    assert len(keep) >= 3
    assert np.array_equal(before, after, equal_nan=True)
    rows = (keep[:, None] * (g + 1) + np.arange(g + 1)[None, :]).ravel()
    assert np.isfinite(after[rows]).all()
