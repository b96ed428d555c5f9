"""Rounds driven by Algorithm 1 on a two-bank worker (schedule -> copy into the standby bank -> run -> export the
accepted suffix), checked round by round against the oracle: the scheduler oracle must pick the same batches from
the same model clock, and the KV / attention / acceptance / commit oracles, applied in the same order to a host
copy of the pool, must leave the same bytes, outputs and context lengths."""
import numpy as np
import pytest
import torch

import oracle
import workload as W
from oracle import schedule as osched
from paper_2609_29364_b200.banks import BankedPool
from nsd_testlib import accept_compare, attn_mismatch, host_u16

pytestmark = pytest.mark.gpu

L, SLABS, HQ, HKV, D, BS, VOCAB, GAMMA = 2, 2, 8, 2, 128, 16, 700, 3
N_REQ, MAX_BATCH, ROUNDS, SEED = 11, 4, 6, 424242


def _round_cfg(k, batch):
    return W.RoundConfig(f"sched{k}", batch=len(batch), gamma=GAMMA, num_layers=L, num_q_heads=HQ, num_kv_heads=HKV,
                         head_dim=D, block_size=BS, vocab=VOCAB, ctx_dist=("uniform", 1, 2), frac_reassigned=0.0,
                         seed=SEED + 31 * k)


def _inputs(k, batch):
    cfg = _round_cfg(k, batch)
    kv = [W.new_kv(cfg, None, l) for l in range(L)]
    p, q_draft, tok, ua, us = W.accept_inputs(cfg)
    return dict(k_new=np.stack([a for a, _ in kv]), v_new=np.stack([b for _, b in kv]),
                q=np.stack([W.queries(cfg, None, l) for l in range(L)]), p=p, q_draft=q_draft, draft_tok=tok, u_acc=ua, u_smp=us)


def test_scheduled_rounds_match_the_oracles():
    import paper_2609_29364_b200 as nsd
    from paper_2609_29364_b200.rounds import ClockModel, ScheduledRounds

    rng = np.random.Generator(np.random.Philox(key=np.array([np.uint64(SEED), np.uint64(5)], dtype=np.uint64)))
    ctx0 = rng.integers(3, 220, size=N_REQ).astype(np.int32)
    max_new = ROUNDS * (GAMMA + 1)
    bank_blocks = MAX_BATCH * ((int(ctx0.max()) + max_new + GAMMA + 1 + BS - 1) // BS) + 4
    mk_banks = lambda: BankedPool(ctx0, GAMMA, BS, max_new, bank_blocks, seed=SEED)
    banks = mk_banks()
    block_elems = 2 * HKV * BS * D
    # the store holds finite data everywhere; the banks start poisoned so that reading an unfilled block shows
    pool0 = W.f32_to_bf16(rng.standard_normal((SLABS, banks.num_blocks * block_elems), dtype=np.float32))
    pool0[:, banks.region_b_begin * block_elems:] = W.BF16_NAN

    ctx = nsd.VerifyContext(num_layers=L, num_slabs=SLABS, num_q_heads=HQ, num_kv_heads=HKV, head_dim=D, block_size=BS,
                            num_blocks=banks.num_blocks, region_b_begin=banks.region_b_begin, max_batch=MAX_BATCH,
                            max_gamma=GAMMA, vocab_size=VOCAB, max_table_entries=MAX_BATCH * bank_blocks)
    pool = torch.from_numpy(pool0.view(np.int16)).cuda()
    clock = ClockModel()
    recs = ScheduledRounds(ctx, pool, banks, ctx0, GAMMA, MAX_BATCH, _inputs, clock).run(ROUNDS)
    assert len(recs) == ROUNDS
    assert len({tuple(r.batch) for r in recs}) > 2                    # the schedule really moves through the pool

    # ---------------- the same rounds through the oracles
    ref_pool, ref_banks = pool0.copy().reshape(SLABS, banks.num_blocks, 2, HKV, BS, D), mk_banks()
    ctx_len = ctx0.copy()
    pred_done = np.arange(N_REQ, dtype=np.float64) * 1.0e-6
    worker_avail, busy = 0.0, []
    copied = 0
    for k, rec in enumerate(recs):
        bank = k % 2
        blocks = [ref_banks.blocks_needed(x) for x in ctx_len]
        kv_ready = [pred_done[r] + (0.0 if r in ref_banks.held[bank] else clock.t_copy_block * blocks[r]) for r in range(N_REQ)]
        eligible = [0 if r in busy else 1 for r in range(N_REQ)]
        batch, start = osched.schedule_batch(worker_avail, clock.target_interval, clock.slack, MAX_BATCH, list(pred_done), kv_ready,
                                             eligible=eligible, rows=[GAMMA + 1] * N_REQ, blocks=blocks, tokens=list(ctx_len),
                                             row_cap=MAX_BATCH * (GAMMA + 1), block_cap=bank_blocks)
        assert batch == rec.batch, (k, batch, rec.batch)
        assert start == pytest.approx(rec.start_pred, abs=1e-12)
        worker_avail = start + clock.t_fixed + clock.t_block * float(sum(blocks[r] for r in batch))
        for r in batch:
            pred_done[r] = worker_avail + clock.t_draft
        busy = batch

        e = ref_banks.enter(bank, batch, ctx_len)
        assert np.array_equal(e.kv_indices, rec.entry.kv_indices) and np.array_equal(e.mig_src, rec.entry.mig_src)
        copied += len(e.mig_src)
        h = _inputs(k, batch)
        bctx = ctx_len[batch].copy()
        mig = (np.array([0, len(e.mig_src)], dtype=np.int64), e.mig_src, e.mig_dst)
        for l in range(L):
            oracle.kv_prepare(ref_pool, *mig, bctx, e.kv_indptr, e.kv_indices, h["k_new"], h["v_new"], GAMMA, layer_begin=l, layer_count=1)
            o_ref = oracle.verify_attn(ref_pool, h["q"][l], bctx, e.kv_indptr, e.kv_indices, GAMMA, layer=l)
            bad, max_abs, max_rel = attn_mismatch(host_u16(rec.o)[l], o_ref)
            assert bad == 0, (k, l, bad, max_abs, max_rel)
        acc, out, _ = oracle.spec_accept(h["p"], h["q_draft"], h["draft_tok"], h["u_acc"], h["u_smp"])
        rep = accept_compare(h["p"], h["q_draft"], h["draft_tok"], h["u_acc"], h["u_smp"], rec.acc_len, rec.out_tok, acc, out)
        assert rep["len_exact"] == len(batch), (k, rep)
        rc, new_ctx = oracle.kv_commit(ref_pool, bctx, acc, e.kv_indptr, e.kv_indices, e.store_indptr, e.store_indices, GAMMA)
        assert rc == 0
        ctx_len[batch] = new_ctx
        assert rec.exposed_wait_ms >= 0.0 and rec.run_ms > 0.0

    assert copied > 0
    assert sum(int(r.entry.resident.sum()) for r in recs) > 0            # some requests came back to a bank that still held them
    assert np.array_equal(host_u16(pool).reshape(ref_pool.shape), ref_pool)      # store and both banks, bit for bit
