"""The fused round is enqueue-only (no host synchronisation, cross-stream ordering by events), so it can
be captured into a CUDA graph and replayed; the replay must leave the same pool and outputs."""
import numpy as np
import pytest
import torch

import oracle
import workload as W
from nsd_testlib import DeviceBatch, attn_mismatch, dev, guarded_pool, host_u16, make_context, stack_layers
import test_gpu_round as rnd

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("fuse", [False, True], ids=["side_stream", "gather_through"])
def test_round_replayed_from_a_cuda_graph(fuse):
    cfg = rnd.MULTI
    slabs = 2
    meta = W.make_batch_meta(cfg)
    pool0 = np.stack([W.pool_layer(cfg, meta, s) for s in range(slabs)])
    k_new, v_new = stack_layers(cfg, meta, "kv")
    q = stack_layers(cfg, meta, "q")
    acc_in = W.accept_inputs(cfg)
    p, qd, tok, ua, us = acc_in
    ctx = make_context(cfg, meta, num_slabs=slabs)
    db = DeviceBatch(meta)
    buf, pool = guarded_pool(pool0)
    B, g1 = cfg.batch, cfg.gamma + 1
    o = torch.full(q.shape, 0x7FC0, dtype=torch.int16, device="cuda:0")
    acc = torch.full((B,), -7, dtype=torch.int32, device="cuda:0")
    out = torch.full((B, g1), -7, dtype=torch.int32, device="cuda:0")
    args = ctx.round_args(kv_pool=pool, n_mig_blocks=db.n_mig_blocks, mig_src=db.mig_src, mig_dst=db.mig_dst, batch=B,
                          gamma=cfg.gamma, ctx_len=db.ctx_len, kv_indptr=db.kv_indptr, kv_indices=db.kv_indices,
                          is_migrated=db.is_migrated, k_new=dev(k_new), v_new=dev(v_new), q=dev(q), o=o, p=dev(p),
                          q_draft=dev(qd), draft_tok=dev(tok), u_acc=dev(ua), u_smp=dev(us), acc_len=acc, out_tok=out,
                          fuse_gather=int(fuse))
    ctx.nsd_verify_plan(meta.ctx_len, meta.kv_indptr, meta.is_migrated, cfg.gamma)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    stream = torch.cuda.Stream()
    with torch.cuda.graph(graph, stream=stream):
        ctx.nsd_verify_round(args, stream=torch.cuda.current_stream())
    torch.cuda.synchronize()
    assert (acc == -7).all()                    # capture enqueued nothing for real
    for _ in range(2):
        graph.replay()
    torch.cuda.synchronize()
    rc, bad = ctx.nsd_get_status()
    assert rc == 0, (rc, bad)
    want_pool, outs, acc_r, out_r, _ = rnd._oracle_round(cfg, meta, pool0, k_new, v_new, q, acc_in)
    assert np.array_equal(host_u16(pool).reshape(want_pool.shape), want_pool)
    o_gpu = host_u16(o)
    for l in range(cfg.num_layers):
        bad, max_abs, max_rel = attn_mismatch(o_gpu[l], outs[l])
        assert bad == 0, (l, bad, max_abs, max_rel)
    assert np.array_equal(acc.cpu().numpy(), acc_r) and np.array_equal(out.cpu().numpy(), out_r)
