"""Pins for the attention oracle: closed forms that fix the visible-key count,
the grouped-query head map and the paging lookup; invariance under physical
block permutation; torch scaled_dot_product_attention in fp64 on gathered KV."""
import numpy as np
import pytest
import torch

import oracle
import workload as W


def _prepared(cfg, layer=0):
    """Pool after gather + append (through the kv oracle), with q for the layer."""
    meta = W.make_batch_meta(cfg)
    pool = W.pool_layer(cfg, meta, layer)[None].copy()
    k_new, v_new = W.new_kv(cfg, meta, layer)
    rc = oracle.kv_prepare(pool, meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr,
                           meta.kv_indices, k_new[None], v_new[None], cfg.gamma)
    assert rc == 0
    return meta, pool, W.queries(cfg, meta, layer)


def _gather_logical(cfg, meta, pool, r, n_keys):
    """K, V of request r as [n_keys][Hkv][D] float64, by direct table lookup."""
    bs = cfg.block_size
    j = np.arange(n_keys)
    blocks = meta.kv_indices[meta.kv_indptr[r] + j // bs]
    k = W.bf16_to_f32(pool[0, blocks, 0, :, j % bs, :]).astype(np.float64)
    v = W.bf16_to_f32(pool[0, blocks, 1, :, j % bs, :]).astype(np.float64)
    return k, v


TINY = W.CONFIGS["tiny"]


def test_zero_keys_give_mean_of_visible_values():
    """K = 0 makes every visible key equally weighted, so row i must be the mean
    of exactly ctx + i + 1 value rows of kv head h div (Hq/Hkv)."""
    cfg = TINY
    meta, pool, q = _prepared(cfg)
    pool[:, :, 0] = 0
    o = oracle.verify_attn(pool, q, meta.ctx_len, meta.kv_indptr, meta.kv_indices, cfg.gamma)
    group = cfg.num_q_heads // cfg.num_kv_heads
    for r in range(cfg.batch):
        for i in range(cfg.gamma + 1):
            n = int(meta.ctx_len[r]) + i + 1
            _, v = _gather_logical(cfg, meta, pool, r, n)
            mean = v.mean(axis=0)                                  # [Hkv][D]
            row = r * (cfg.gamma + 1) + i
            for h in range(cfg.num_q_heads):
                np.testing.assert_allclose(o[row, h], mean[h // group], rtol=1e-6, atol=1e-6)
            # one key more or fewer would be visible as a different mean
            _, v_more = _gather_logical(cfg, meta, pool, r, n - 1)
            assert not np.allclose(o[row, 0], v_more.mean(axis=0)[0], rtol=1e-6, atol=1e-6)


def test_equal_values_pass_through():
    cfg = TINY
    meta, pool, q = _prepared(cfg)
    vrow = W.f32_to_bf16(np.linspace(-2, 2, cfg.head_dim).astype(np.float32))
    pool[:, :, 1] = vrow
    o = oracle.verify_attn(pool, q, meta.ctx_len, meta.kv_indptr, meta.kv_indices, cfg.gamma)
    np.testing.assert_allclose(o, np.broadcast_to(W.bf16_to_f32(vrow), o.shape), rtol=1e-6, atol=1e-6)


def test_dominant_key_selects_its_value_row():
    cfg = TINY
    meta, pool, q = _prepared(cfg)
    r, key = 2, 5
    b = meta.kv_indices[meta.kv_indptr[r] + key // cfg.block_size]
    # every q row of request r gets the same direction; the chosen key is 64x that direction
    d = np.zeros(cfg.head_dim, dtype=np.float32)
    d[0] = 8.0
    rows = slice(r * (cfg.gamma + 1), (r + 1) * (cfg.gamma + 1))
    q[rows] = W.f32_to_bf16(d)
    pool[0, :, 0, :, :, 0] = 0                                   # nobody else has a component along d
    pool[0, b, 0, :, key % cfg.block_size, :] = W.f32_to_bf16(d * 64)
    o = oracle.verify_attn(pool, q, meta.ctx_len, meta.kv_indptr, meta.kv_indices, cfg.gamma)
    group = cfg.num_q_heads // cfg.num_kv_heads
    want = W.bf16_to_f32(pool[0, b, 1, :, key % cfg.block_size, :])
    for h in range(cfg.num_q_heads):
        np.testing.assert_allclose(o[rows, h], np.broadcast_to(want[h // group], (cfg.gamma + 1, cfg.head_dim)),
                                   rtol=1e-5, atol=1e-5)


def test_block_permutation_leaves_output_bit_identical():
    cfg = TINY
    meta, pool, q = _prepared(cfg)
    o1, l1 = oracle.verify_attn(pool, q, meta.ctx_len, meta.kv_indptr, meta.kv_indices, cfg.gamma, want_lse=True)
    perm = np.random.default_rng(0).permutation(meta.num_blocks)          # new id of old block b is perm[b]
    pool2 = np.empty_like(pool)
    pool2[0, perm] = pool[0]
    idx2 = perm[meta.kv_indices].astype(np.int32)
    o2, l2 = oracle.verify_attn(pool2, q, meta.ctx_len, meta.kv_indptr, idx2, cfg.gamma, want_lse=True)
    assert np.array_equal(o1, o2) and np.array_equal(l1, l2)


@pytest.mark.parametrize("name", ["tiny", "gqa_d128"])
def test_matches_torch_sdpa_fp64(name):
    """Library cross-check: gather each request's KV to contiguous, repeat kv
    heads over their group, and call torch's attention with an explicit mask."""
    if name == "tiny":
        cfg = TINY
    else:
        cfg = W.RoundConfig("gqa_d128", batch=3, gamma=6, num_layers=1, num_q_heads=32, num_kv_heads=8, head_dim=128,
                            block_size=16, vocab=100, ctx_dist=("fixed", [1, 16, 75]), frac_reassigned=0.34, seed=7)
    meta, pool, q = _prepared(cfg)
    o, lse = oracle.verify_attn(pool, q, meta.ctx_len, meta.kv_indptr, meta.kv_indices, cfg.gamma, want_lse=True)
    g1, group = cfg.gamma + 1, cfg.num_q_heads // cfg.num_kv_heads
    for r in range(cfg.batch):
        ctx = int(meta.ctx_len[r])
        n = ctx + g1
        k, v = _gather_logical(cfg, meta, pool, r, n)
        kt = torch.from_numpy(k).permute(1, 0, 2).repeat_interleave(group, dim=0)      # [Hq][n][D]
        vt = torch.from_numpy(v).permute(1, 0, 2).repeat_interleave(group, dim=0)
        qt = torch.from_numpy(W.bf16_to_f32(q[r * g1:(r + 1) * g1]).astype(np.float64)).permute(1, 0, 2)
        mask = torch.arange(n)[None, :] <= (ctx + torch.arange(g1))[:, None]
        ref = torch.nn.functional.scaled_dot_product_attention(qt[None], kt[None], vt[None], attn_mask=mask[None, None])
        ref = ref[0].permute(1, 0, 2).numpy()
        np.testing.assert_allclose(o[r * g1:(r + 1) * g1], ref, rtol=2e-6, atol=2e-6)
        s = torch.einsum("hid,hjd->hij", qt, kt) / np.sqrt(cfg.head_dim)
        s = s.masked_fill(~mask[None], float("-inf"))
        np.testing.assert_allclose(lse[r * g1:(r + 1) * g1], torch.logsumexp(s, -1).T.numpy(), rtol=2e-6, atol=2e-6)


def test_poisoned_slots_do_not_leak():
    """Unused blocks and slots past the last visible key hold NaN; none may reach the output."""
    cfg = TINY
    meta, pool, q = _prepared(cfg)
    assert np.isnan(W.bf16_to_f32(pool)).any()
    o = oracle.verify_attn(pool, q, meta.ctx_len, meta.kv_indptr, meta.kv_indices, cfg.gamma)
    assert np.isfinite(o).all()


def test_request_subset_only_touches_listed_requests():
    cfg = TINY
    meta, pool, q = _prepared(cfg)
    full = oracle.verify_attn(pool, q, meta.ctx_len, meta.kv_indptr, meta.kv_indices, cfg.gamma)
    sub = oracle.verify_attn(pool, q, meta.ctx_len, meta.kv_indptr, meta.kv_indices, cfg.gamma,
                             req_list=np.array([2], dtype=np.int32))
    g1 = cfg.gamma + 1
    assert np.array_equal(sub[2 * g1:3 * g1], full[2 * g1:3 * g1])
    assert np.isnan(sub[:2 * g1]).all() and np.isnan(sub[3 * g1:]).all()
