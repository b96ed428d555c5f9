"""Pins for the suffix-commit oracle: numpy restatement, the byte count of the
paper's writeback cost model (Delta_Q tokens x bytes per token), nothing but the
committed slots changes, rejected drafts stay behind."""
import numpy as np

import oracle
import workload as W

CFG = W.RoundConfig("commit", batch=7, gamma=4, num_layers=3, num_q_heads=8, num_kv_heads=2, head_dim=64, block_size=16,
                    vocab=100, ctx_dist=("fixed", [0, 11, 12, 15, 16, 47, 90]), frac_reassigned=0.3, pool_factor=3.0, seed=61)


def _prepared():
    meta = W.make_batch_meta(CFG)
    pool = np.stack([W.pool_layer(CFG, meta, l) for l in range(CFG.num_layers)])
    kv = [W.new_kv(CFG, meta, l) for l in range(CFG.num_layers)]
    oracle.kv_prepare(pool, meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr, meta.kv_indices,
                      np.stack([a for a, _ in kv]), np.stack([b for _, b in kv]), CFG.gamma)
    exp_indptr, exp_indices = W.export_tables(CFG, meta)
    acc = np.array([0, 4, 3, 1, 4, 2, 0], dtype=np.int32)
    return meta, pool, exp_indptr, exp_indices, acc


def test_matches_numpy_and_cost_model_bytes():
    meta, pool, ei, ex, acc = _prepared()
    want = pool.copy()
    bs = CFG.block_size
    for l in range(CFG.num_layers):
        for r in range(CFG.batch):
            pos = meta.ctx_len[r] + np.arange(acc[r] + 1)
            frm = meta.kv_indices[meta.kv_indptr[r] + pos // bs]
            to = ex[ei[r] + pos // bs]
            want[l, to, :, :, pos % bs, :] = pool[l, frm, :, :, pos % bs, :]
    got = pool.copy()
    rc, new_ctx = oracle.kv_commit(got, meta.ctx_len, acc, meta.kv_indptr, meta.kv_indices, ei, ex, CFG.gamma)
    assert rc == 0 and np.array_equal(got, want)
    assert (new_ctx == meta.ctx_len + 1 + acc).all()
    # Eq. (9): Delta_Q tokens x b_KV bytes is everything that may differ (poisoned targets make every byte differ)
    changed = int((got != pool).sum()) * 2
    delta_q = int((acc + 1).sum())
    b_kv = 2 * CFG.num_kv_heads * CFG.head_dim * 2
    assert changed <= delta_q * b_kv * CFG.num_layers
    assert changed > 0.99 * delta_q * b_kv * CFG.num_layers          # NaN-poisoned targets: all of them do differ


def test_rejected_drafts_and_everything_else_stay():
    meta, pool, ei, ex, acc = _prepared()
    got = pool.copy()
    oracle.kv_commit(got, meta.ctx_len, acc, meta.kv_indptr, meta.kv_indices, ei, ex, CFG.gamma)
    bs = CFG.block_size
    for r in range(CFG.batch):
        for t in range(acc[r] + 1, CFG.gamma + 1):                     # rejected drafts were appended but never exported
            pos = int(meta.ctx_len[r]) + t
            to = ex[ei[r] + pos // bs]
            assert np.array_equal(got[:, to, :, :, pos % bs, :], pool[:, to, :, :, pos % bs, :])
    not_export = np.ones(meta.num_blocks, bool)
    not_export[ex[ex >= 0]] = False
    assert np.array_equal(got[:, not_export], pool[:, not_export])    # sources and bystanders untouched
    again = got.copy()
    oracle.kv_commit(again, meta.ctx_len, acc, meta.kv_indptr, meta.kv_indices, ei, ex, CFG.gamma)
    assert np.array_equal(again, got)                                  # idempotent
    part = pool.copy()
    oracle.kv_commit(part, meta.ctx_len, acc, meta.kv_indptr, meta.kv_indices, ei, ex, CFG.gamma, layer_begin=1, layer_count=1)
    assert np.array_equal(part[0], pool[0]) and np.array_equal(part[1], got[1]) and np.array_equal(part[2], pool[2])


def test_committed_suffix_attends_like_the_original():
    """A later round over the export copy sees, for the committed tokens, the same keys and values."""
    meta, pool, ei, ex, acc = _prepared()
    got = pool.copy()
    oracle.kv_commit(got, meta.ctx_len, acc, meta.kv_indptr, meta.kv_indices, ei, ex, CFG.gamma)
    bs = CFG.block_size
    for r in (1, 4, 6):
        for t in range(acc[r] + 1):
            pos = int(meta.ctx_len[r]) + t
            frm = meta.kv_indices[meta.kv_indptr[r] + pos // bs]
            to = ex[ei[r] + pos // bs]
            assert np.array_equal(got[:, to, :, :, pos % bs, :], got[:, frm, :, :, pos % bs, :])
            assert not np.isnan(W.bf16_to_f32(got[:, to, :, :, pos % bs, :])).any()
