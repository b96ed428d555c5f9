"""nsd_verify_attn_static: attention for hosts that may not allocate device memory
(a plugin inside another runtime's memory budget, a worker whose memory was carved
up at start-up).  Its scratch is a fixed array inside the library, so the checks
that matter are: same output as the workspace-backed nsd_verify_attn and as the
oracle, still the same on a second call that finds the first call's leftovers in
the array, and a clean refusal of batches that exceed the array.

Collected last on purpose (file name): a failure here cannot hide the other tests."""
import numpy as np
import pytest
import torch

import oracle
import workload as W
from nsd_testlib import DeviceBatch, attn_mismatch, dev, host_u16, make_context

pytestmark = pytest.mark.gpu


def _case(seed, ctx):
    """A batch with single-chunk and split (> 1024 keys) requests, pool already holding the new tokens."""
    cfg = W.RoundConfig("static", batch=len(ctx), gamma=4, num_layers=1, num_q_heads=32, num_kv_heads=8, head_dim=128,
                        block_size=16, vocab=100, ctx_dist=("fixed", ctx), frac_reassigned=0.0, seed=seed)
    meta = W.make_batch_meta(cfg)
    pool = W.pool_layer(cfg, meta, 0)
    k_new, v_new = W.new_kv(cfg, meta, 0)
    q = W.queries(cfg, meta, 0)
    ctxh = make_context(cfg, meta)
    db = DeviceBatch(meta)
    pool_d, q_d = dev(pool), dev(q)
    ctxh.nsd_kv_prepare(pool_d, 0, None, None, cfg.batch, cfg.gamma, db.ctx_len, db.kv_indptr, db.kv_indices,
                        dev(k_new[None]), dev(v_new[None]))
    o_ref = torch.full(q_d.shape, 0x7FC0, dtype=torch.int16, device="cuda:0")
    ctxh.nsd_verify_plan(meta.ctx_len, meta.kv_indptr, None, cfg.gamma)
    ctxh.nsd_verify_attn(pool_d, q_d, o_ref, None, cfg.batch, cfg.gamma, db.ctx_len, db.kv_indptr, db.kv_indices)
    torch.cuda.synchronize()
    # the oracle on the same prepared pool
    want = pool[None].copy()
    oracle.kv_prepare(want, None, None, None, meta.ctx_len, meta.kv_indptr, meta.kv_indices, k_new[None], v_new[None], cfg.gamma)
    o_oracle = oracle.verify_attn(want, q, meta.ctx_len, meta.kv_indptr, meta.kv_indices, cfg.gamma)
    return cfg, meta, db, pool_d, q_d, o_ref, o_oracle


def _static(cfg, meta, db, pool_d, q_d):
    import paper_2609_29364_b200 as nsd

    o = torch.full(q_d.shape, 0x7FC0, dtype=torch.int16, device="cuda:0")
    nsd.nsd_verify_attn_static(pool_d, meta.num_blocks, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim,
                               cfg.block_size, q_d, o, cfg.batch, cfg.gamma, meta.ctx_len, db.ctx_len, db.kv_indptr,
                               db.kv_indices)
    torch.cuda.synchronize()
    return o


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    first = _case(91, [3, 200, 1023, 1500, 2500, 40])        # two split requests: 2 and 3 chunks
    second = _case(92, [3000, 17, 1100, 900])                 # other lengths: other chunk counts per slot
    for case in (first, second, first):
        cfg, meta, db, pool_d, q_d, o_ref, o_oracle = case
        o = _static(cfg, meta, db, pool_d, q_d)
        ref = W.bf16_to_f32(host_u16(o_ref))
        bad, max_abs, max_rel = attn_mismatch(host_u16(o), ref)
        assert bad == 0, (bad, max_abs, max_rel)
        bad, max_abs, max_rel = attn_mismatch(host_u16(o), o_oracle)
        assert bad == 0, (bad, max_abs, max_rel)


def test_sizes_beyond_the_static_scratch_are_refused():
    import paper_2609_29364_b200 as nsd

    cfg, meta, db, pool_d, q_d, o_ref, _ = _case(93, [10, 20])
    o = torch.zeros_like(q_d)
    common = (pool_d, meta.num_blocks, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.block_size, q_d, o)
    tables = (db.ctx_len, db.kv_indptr, db.kv_indices)
    with pytest.raises(nsd.NsdError) as e:                    # 65 requests
        nsd.nsd_verify_attn_static(*common, 65, cfg.gamma, np.zeros(65, np.int32), *tables)
    assert e.value.code == 3
    with pytest.raises(nsd.NsdError) as e:                    # 4 * (gamma + 1) = 36 query rows per kv head
        nsd.nsd_verify_attn_static(*common, 2, 8, meta.ctx_len, *tables)
    assert e.value.code == 3
    with pytest.raises(nsd.NsdError) as e:                    # 2 requests x 40 chunks of 1024 keys > 64 partial slots
        nsd.nsd_verify_attn_static(*common, 2, cfg.gamma, np.array([40000, 40000], np.int32), *tables)
    assert e.value.code == 3
    with pytest.raises(nsd.NsdError) as e:
        nsd.nsd_verify_attn_static(*common, 2, cfg.gamma, np.array([10, -1], np.int32), *tables)
    assert e.value.code == 1
    torch.cuda.synchronize()
    assert (o == 0).all()                                     # nothing was launched


def test_a_capturing_stream_is_refused():
    """The call uploads its work list from a buffer that dies with the call, so it cannot become a graph node."""
    import paper_2609_29364_b200 as nsd

    cfg, meta, db, pool_d, q_d, o_ref, _ = _case(94, [10, 20])
    _static(cfg, meta, db, pool_d, q_d)                        # the set-up call, outside any capture
    o = torch.zeros_like(q_d)
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        with pytest.raises(nsd.NsdError) as e:
            nsd.nsd_verify_attn_static(pool_d, meta.num_blocks, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim,
                                       cfg.block_size, q_d, o, cfg.batch, cfg.gamma, meta.ctx_len, db.ctx_len,
                                       db.kv_indptr, db.kv_indices, stream=stream)
        assert e.value.code == 1
