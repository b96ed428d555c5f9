"""GPU parity: the fused nsd_verify_round (side-stream prepare overlapped with
attention, every layer, then acceptance) and its host-buffer variant against the
oracle sequence gather -> append -> attention per layer, then acceptance."""
import numpy as np
import pytest
import torch

import nsd_testlib
import oracle
import workload as W
from nsd_testlib import (DeviceBatch, accept_compare, attn_mismatch, dev, guarded_pool, guards_intact, host_u16,
                         make_context, stack_layers)

pytestmark = pytest.mark.gpu

SPLIT_FLAG = {"always": 1 << 4, "never": 1 << 5}      # NSD_FLAG_ROUND_SPLIT_ALWAYS / _NEVER


def _oracle_round(cfg, meta, pool0, k_new, v_new, q, acc_in):
    pool = pool0.copy()
    outs = []
    for l in range(cfg.num_layers):
        oracle.kv_prepare(pool, meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr,
                          meta.kv_indices, k_new, v_new, cfg.gamma, layer_begin=l, layer_count=1)
        outs.append(oracle.verify_attn(pool, q[l], meta.ctx_len, meta.kv_indptr, meta.kv_indices, cfg.gamma, layer=l))
    acc, out, new_ctx = oracle.spec_accept(*acc_in, meta.ctx_len)
    return pool, outs, acc, out, new_ctx


def _run_round(cfg, slabs, host_variant=False, repeat=1, fuse=False, plan_without_flags=False, pageable_probs=False):
    """The first-layer order is a flag of the context: the tests below set it to cover both orders."""
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
    d = dict(kv_pool=pool, n_mig_blocks=db.n_mig_blocks, mig_src=db.mig_src, mig_dst=db.mig_dst, batch=B,
             gamma=cfg.gamma, ctx_len=db.ctx_len, kv_indptr=db.kv_indptr, kv_indices=db.kv_indices,
             is_migrated=db.is_migrated, k_new=dev(k_new), v_new=dev(v_new), q=dev(q),
             o=torch.full(q.shape, 0x7FC0, dtype=torch.int16, device="cuda:0"), p=dev(p), q_draft=dev(qd),
             draft_tok=dev(tok), u_acc=dev(ua), u_smp=dev(us),
             acc_len=torch.full((B,), -7, dtype=torch.int32, device="cuda:0"),
             out_tok=torch.full((B, g1), -7, dtype=torch.int32, device="cuda:0"),
             new_ctx_len=torch.full((B,), -7, dtype=torch.int32, device="cuda:0"), fuse_gather=int(fuse))
    stream = torch.cuda.Stream()
    if host_variant:
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a.view(np.int16) if a.dtype == np.uint16 else a)).pin_memory()
        # pinned probability tensors are read in place by the acceptance kernel; pageable ones are copied like the rest
        probs = (lambda a: torch.from_numpy(np.ascontiguousarray(a))) if pageable_probs else pin
        h = dict(kv_pool=None, n_mig_blocks=db.n_mig_blocks, mig_src=pin(meta.mig_src) if db.n_mig_blocks else None,
                 mig_dst=pin(meta.mig_dst) if db.n_mig_blocks else None, batch=B, gamma=cfg.gamma,
                 ctx_len=pin(meta.ctx_len), kv_indptr=pin(meta.kv_indptr), kv_indices=pin(meta.kv_indices),
                 is_migrated=pin(meta.is_migrated), k_new=pin(k_new), v_new=pin(v_new), q=pin(q),
                 o=torch.zeros(q.shape, dtype=torch.int16).pin_memory(), p=probs(p), q_draft=probs(qd), draft_tok=pin(tok),
                 u_acc=pin(ua), u_smp=pin(us), acc_len=torch.zeros(B, dtype=torch.int32).pin_memory(),
                 out_tok=torch.zeros((B, g1), dtype=torch.int32).pin_memory(),
                 new_ctx_len=torch.zeros(B, dtype=torch.int32).pin_memory(), fuse_gather=int(fuse))
        # the device copies start as garbage: everything must arrive through the call
        for k in ("ctx_len", "kv_indptr", "kv_indices", "is_migrated", "k_new", "v_new", "q", "p", "q_draft",
                  "draft_tok", "u_acc", "u_smp"):
            d[k] = torch.zeros_like(d[k])
        if db.n_mig_blocks:
            d["mig_src"], d["mig_dst"] = torch.zeros_like(d["mig_src"]), torch.zeros_like(d["mig_dst"])
        with torch.cuda.stream(stream):
            for _ in range(repeat):
                up, down = ctx.nsd_verify_round_host(ctx.round_args(**h), ctx.round_args(**d), int(meta.kv_indptr[-1]),
                                                     stream=stream)
        layers_in = k_new.nbytes + v_new.nbytes + q.nbytes
        assert up > layers_in and down >= q.nbytes
        assert (up > layers_in + p.nbytes + qd.nbytes) == pageable_probs      # copied whole, or read in place row by row
        o_gpu, acc_g, out_g, new_g = h["o"].numpy().view(np.uint16), h["acc_len"].numpy(), h["out_tok"].numpy(), h["new_ctx_len"].numpy()
    else:
        with torch.cuda.stream(stream):
            ctx.nsd_verify_plan(meta.ctx_len, meta.kv_indptr, None if plan_without_flags else meta.is_migrated, cfg.gamma,
                                stream=stream)
            for _ in range(repeat):
                ctx.nsd_verify_round(ctx.round_args(**d), stream=stream)
        stream.synchronize()
        o_gpu, acc_g, out_g, new_g = host_u16(d["o"]), d["acc_len"].cpu().numpy(), d["out_tok"].cpu().numpy(), d["new_ctx_len"].cpu().numpy()
    rc, bad = ctx.nsd_get_status(stream=stream)
    assert rc == 0, (rc, bad)
    assert guards_intact(buf)
    want_pool, outs, acc_r, out_r, new_r = _oracle_round(cfg, meta, pool0, k_new, v_new, q, acc_in)
    assert np.array_equal(host_u16(pool).reshape(want_pool.shape), want_pool)
    for l in range(cfg.num_layers):
        bad, max_abs, max_rel = attn_mismatch(o_gpu[l], outs[l])
        assert bad == 0, (l, bad, max_abs, max_rel)
    rep = accept_compare(p, qd, tok, ua, us, acc_g, out_g, acc_r, out_r)
    assert rep["len_exact"] == cfg.batch
    assert (new_g == new_r).all()
    return ctx


MULTI = W.RoundConfig("round_multi", batch=10, gamma=4, num_layers=5, num_q_heads=32, num_kv_heads=8, head_dim=128,
                      block_size=16, vocab=3000, ctx_dist=("uniform", 1, 1200), frac_reassigned=0.4, seed=81)
NOMIG = W.RoundConfig("round_nomig", batch=6, gamma=6, num_layers=2, num_q_heads=8, num_kv_heads=2, head_dim=64,
                      block_size=16, vocab=500, ctx_dist=("uniform", 1, 300), frac_reassigned=0.0, seed=82)
ALLMIG = W.RoundConfig("round_allmig", batch=6, gamma=8, num_layers=3, num_q_heads=32, num_kv_heads=8, head_dim=128,
                       block_size=16, vocab=500, ctx_dist=("uniform", 1, 500), frac_reassigned=1.0, seed=83)


def test_tiny_config_round():
    _run_round(W.CONFIGS["tiny"], 1)


@pytest.mark.parametrize("split", ["always", "never"])
@pytest.mark.parametrize("cfg,slabs", [(MULTI, 5), (MULTI, 2), (NOMIG, 2), (ALLMIG, 1), (ALLMIG, 3)],
                         ids=["multi", "multi_alias2", "nomig", "allmig_alias1", "allmig"])
def test_multi_layer_round(cfg, slabs, split, monkeypatch):
    """Both orders of the first layer: resident requests attended while the copy runs and the reassigned ones after it
    (what large copies get), or the whole layer after its copy (small copies)."""
    monkeypatch.setattr(nsd_testlib, "CONTEXT_FLAGS", SPLIT_FLAG[split])
    _run_round(cfg, slabs)


@pytest.mark.parametrize("split", ["always", "never"])
@pytest.mark.parametrize("cfg,slabs,fuse", [(MULTI, 2, False), (ALLMIG, 1, False), (ALLMIG, 3, True), (MULTI, 5, True)],
                         ids=["multi_alias2", "allmig_alias1", "allmig_through", "multi_through"])
def test_round_without_dependent_launches(cfg, slabs, fuse, split, monkeypatch):
    """The round's kernels are launched as programmatic dependents of one another by default (every other test here);
    with NSD_FLAG_NO_DEPENDENT_LAUNCH each starts only when the one before it has completed.  Same oracle, same bars."""
    monkeypatch.setattr(nsd_testlib, "CONTEXT_FLAGS", SPLIT_FLAG[split] | (1 << 6))
    _run_round(cfg, slabs, fuse=fuse, repeat=2)


@pytest.mark.parametrize("split", ["always", "never"])
def test_round_twice_gives_the_same_state(split, monkeypatch):
    """The round is idempotent on its inputs (what the benchmark relies on)."""
    monkeypatch.setattr(nsd_testlib, "CONTEXT_FLAGS", SPLIT_FLAG[split])
    _run_round(MULTI, 2, repeat=3)


@pytest.mark.parametrize("split", ["always", "never"])
def test_host_buffer_round(split, monkeypatch):
    monkeypatch.setattr(nsd_testlib, "CONTEXT_FLAGS", SPLIT_FLAG[split])
    _run_round(MULTI, 2, host_variant=True)
    _run_round(MULTI, 2, host_variant=True, pageable_probs=True)
    _run_round(W.CONFIGS["tiny"], 1, host_variant=True, repeat=2)


@pytest.mark.parametrize("cfg,slabs", [(W.CONFIGS["tiny"], 1), (MULTI, 5), (MULTI, 2), (NOMIG, 2), (ALLMIG, 1), (ALLMIG, 3)],
                         ids=["tiny", "multi", "multi_alias2", "nomig", "allmig_alias1", "allmig"])
def test_gather_through_round_gives_the_same_pool_and_outputs(cfg, slabs):
    """fuse_gather = 1: attention moves the reassigned requests' blocks itself; same pool bytes, same outputs."""
    _run_round(cfg, slabs, fuse=True)


def test_gather_through_round_repeated_and_from_host_buffers():
    _run_round(MULTI, 2, fuse=True, repeat=3)
    _run_round(MULTI, 2, fuse=True, host_variant=True)
    ctx = _run_round(MULTI, 5, fuse=True)
    # per layer: one append (resident requests) and one attention launch; one acceptance
    assert ctx.nsd_launch_count() == 5 * 2 + 1


def test_gather_through_needs_a_matching_plan():
    import paper_2609_29364_b200 as nsd
    from nsd_testlib import DeviceBatch, make_context

    meta = W.make_batch_meta(MULTI)
    ctx = make_context(MULTI, meta, num_slabs=2)
    db = DeviceBatch(meta)
    z = torch.zeros(8, dtype=torch.int32, device="cuda:0")
    ctx.nsd_verify_plan(meta.ctx_len, meta.kv_indptr, None, MULTI.gamma)          # planned without the reassignment flags
    args = ctx.round_args(kv_pool=z, n_mig_blocks=db.n_mig_blocks, mig_src=db.mig_src, mig_dst=db.mig_dst, batch=MULTI.batch,
                          gamma=MULTI.gamma, ctx_len=db.ctx_len, kv_indptr=db.kv_indptr, kv_indices=db.kv_indices,
                          is_migrated=db.is_migrated, k_new=z, v_new=z, q=z, o=z, p=z, q_draft=z, draft_tok=z, u_acc=z,
                          u_smp=z, acc_len=z, out_tok=z, fuse_gather=1)
    with pytest.raises(nsd.NsdError) as e:
        ctx.nsd_verify_round(args)
    assert e.value.code == 1 and ctx.nsd_launch_count() == 0


def test_round_with_a_plan_made_without_the_reassignment_flags(monkeypatch):
    """Such a plan has every request on its resident list: the round must not attend that list before the copy has
    finished, even when the context is told to split its first layer."""
    monkeypatch.setattr(nsd_testlib, "CONTEXT_FLAGS", SPLIT_FLAG["always"])
    ctx = _run_round(MULTI, 2, plan_without_flags=True)
    assert ctx.nsd_launch_count() == MULTI.num_layers * 3 + 1            # no second attention launch in the first layer
    _run_round(ALLMIG, 3, plan_without_flags=True, repeat=2)


def test_launch_count_matches_the_choreography(monkeypatch):
    # per layer: the copy (side stream), one append and one attention launch; one acceptance
    assert _run_round(MULTI, 5).nsd_launch_count() == 5 * 3 + 1          # a small copy: the first layer waits for it
    monkeypatch.setattr(nsd_testlib, "CONTEXT_FLAGS", SPLIT_FLAG["always"])
    # the first layer appends and attends its resident and its reassigned requests separately: two launches more
    assert _run_round(MULTI, 5).nsd_launch_count() == 5 * 3 + 2 + 1
