"""The bounded waits of the kernels: a wait that runs out ends the kernel with a status the host
reads, and the context stays usable.  Nothing here faults or hangs: the test hook makes the gather
arm its barriers with 16 bytes more than its copies deliver, so each barrier phase can never
complete; with a budget of a few hundred polls the kernel gives up at once, waits for its own
copies, and returns."""
import numpy as np
import pytest
import torch

import oracle
import workload as W
from nsd_testlib import DeviceBatch, dev, guarded_pool, guards_intact, host_u16, make_context

pytestmark = pytest.mark.gpu

NSD_ERR_TIMEOUT = 8
STARVE = 1 << 30            # NSD_FLAG_TEST_STARVE_GATHER


def _tiny():
    cfg = W.RoundConfig("starve", batch=6, gamma=4, num_layers=1, num_q_heads=8, num_kv_heads=2, head_dim=64, block_size=16,
                        vocab=100, ctx_dist=("fixed", [5, 40, 100, 257, 31, 64]), frac_reassigned=0.5, seed=77)
    meta = W.make_batch_meta(cfg)
    return cfg, meta, W.pool_layer(cfg, meta, 0)[None]


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    cfg, meta, pool0 = _tiny()
    db = DeviceBatch(meta)
    assert db.n_mig_blocks > 0
    k_new, v_new = (a[None] for a in W.new_kv(cfg, meta, 0))

    starved = make_context(cfg, meta, flags=STARVE, wait_budget=300)
    buf, pool = guarded_pool(pool0)
    starved.nsd_kv_prepare(pool, db.n_mig_blocks, db.mig_src, db.mig_dst, cfg.batch, cfg.gamma, db.ctx_len, db.kv_indptr,
                           db.kv_indices, None, None)
    rc, _ = starved.nsd_get_status()
    assert rc == NSD_ERR_TIMEOUT
    assert guards_intact(buf)
    rc, _ = starved.nsd_get_status()                       # the word was cleared by the read
    assert rc == 0
    # the source region is untouched, whatever the gather managed to store before it gave up
    got = host_u16(pool).reshape(pool0.shape)
    assert np.array_equal(got[0, :meta.region_b_begin], pool0[0, :meta.region_b_begin])
    starved.close()

    # the same device, a context without the hook: the whole preparation matches the oracle
    ctx = make_context(cfg, meta)
    buf, pool = guarded_pool(pool0)
    ctx.nsd_kv_prepare(pool, db.n_mig_blocks, db.mig_src, db.mig_dst, cfg.batch, cfg.gamma, db.ctx_len, db.kv_indptr,
                       db.kv_indices, dev(k_new), dev(v_new))
    rc, bad = ctx.nsd_get_status()
    assert rc == 0, (rc, bad)
    want = pool0.copy()
    oracle.kv_prepare(want, meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr, meta.kv_indices,
                      k_new, v_new, cfg.gamma)
    assert np.array_equal(host_u16(pool).reshape(want.shape), want) and guards_intact(buf)


def test_a_short_budget_alone_changes_nothing():
    """wait_budget only bounds the polls: with copies that do arrive, a generous budget gives the normal result."""
    cfg, meta, pool0 = _tiny()
    db = DeviceBatch(meta)
    ctx = make_context(cfg, meta, wait_budget=1 << 18)
    buf, pool = guarded_pool(pool0)
    ctx.nsd_kv_prepare(pool, db.n_mig_blocks, db.mig_src, db.mig_dst, cfg.batch, cfg.gamma, db.ctx_len, db.kv_indptr,
                       db.kv_indices, None, None)
    rc, bad = ctx.nsd_get_status()
    assert rc == 0, (rc, bad)
    want = pool0.copy()
    oracle.kv_prepare(want, meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr, meta.kv_indices,
                      None, None, cfg.gamma)
    assert np.array_equal(host_u16(pool).reshape(want.shape), want) and guards_intact(buf)
