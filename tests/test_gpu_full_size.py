"""GPU parity at the benchmark set's full sizes, in the launch configuration the
benchmark times: the whole fused round (36 logical layers over a few physical
slabs, plan chosen by the library), checked against the oracle on the whole pool
bit for bit, on the attention rows of sampled requests in sampled layers, and on
the acceptance of every request.

Every configuration runs at its full batch on any host: a layer slab of the two
largest ones is 11 and 19 GB, so nothing here holds a slab in host memory.  The
slab is generated piece by piece from the seed and uploaded; the check then walks
the batch in groups of consecutive requests, reads the blocks a group can touch
(its committed blocks, its table's blocks) from a pristine device copy of the
input slab, lets the oracle prepare and attend that compact pool with the block
ids renumbered, and compares with the same blocks of the slab the round worked on.
Blocks no request can touch must still hold the fill pattern."""
import numpy as np
import pytest
import torch

import oracle
import workload as W
from nsd_testlib import DeviceBatch, accept_compare, attn_mismatch, dev, host_u16, make_context

pytestmark = pytest.mark.gpu

GROUP_BLOCKS = 16384            # blocks of one compact pool on the host (1 GiB at the Qwen3-8B shape)


def _sample_requests(cfg, meta, n_random=3):
    ctx = meta.ctx_len
    picks = {int(np.argmin(ctx)), int(np.argmax(ctx))}
    if meta.n_mig:
        picks.add(int(meta.mig_req[0]))
        picks.add(int(meta.mig_req[-1]))
    resident = np.nonzero(meta.is_migrated == 0)[0]
    if len(resident):
        picks.add(int(resident[len(resident) // 2]))
    rng = np.random.default_rng(cfg.seed)
    picks.update(int(x) for x in rng.choice(cfg.batch, size=min(n_random, cfg.batch), replace=False))
    return np.array(sorted(picks), dtype=np.int32)


def _upload_slab(cfg, meta):
    """The input slab on the device, [num_blocks][block_elems] int16, generated and uploaded in pieces."""
    slab = torch.full((meta.num_blocks, cfg.block_elems), int(W.BF16_NAN), dtype=torch.int16, device="cuda:0")
    for b0, b1, data in W.pool_layer_chunks(cfg, meta, 0):
        idx = torch.from_numpy(meta.home_blocks[b0:b1].astype(np.int64)).cuda()
        slab.index_copy_(0, idx, torch.from_numpy(data.reshape(b1 - b0, -1).view(np.int16)).cuda())
    return slab


def _groups(meta, batch):
    """Consecutive request ranges whose touchable blocks fit one compact pool."""
    out, r0, n = [], 0, 0
    for r in range(batch):
        need = int(meta.home_indptr[r + 1] - meta.home_indptr[r]) + int(meta.kv_indptr[r + 1] - meta.kv_indptr[r])
        if r > r0 and n + need > GROUP_BLOCKS:
            out.append((r0, r))
            r0, n = r, 0
        n += need
    out.append((r0, batch))
    return out


def _check_against_oracle(cfg, meta, pristine, pool, o, k_new, v_new, q, slabs, layers_to_check, slabs_to_check):
    """Pool slabs `slabs_to_check` bit for bit and the attention rows of sampled requests in `layers_to_check`."""
    L, g1 = cfg.num_layers, cfg.gamma + 1
    Hkv, bs, D = cfg.num_kv_heads, cfg.block_size, cfg.head_dim
    sel = set(int(x) for x in _sample_requests(cfg, meta))
    last_of_slab = {max(l for l in range(L) if l % slabs == s): s for s in slabs_to_check}
    layers = sorted(set(layers_to_check) | set(last_of_slab))
    mig_pos = {int(r): m for m, r in enumerate(meta.mig_req)}
    touched = torch.zeros(meta.num_blocks, dtype=torch.bool, device="cuda:0")
    worst, n_rows = (0.0, 0.0), 0
    for r0, r1 in _groups(meta, cfg.batch):
        home = meta.home_blocks[meta.home_indptr[r0]:meta.home_indptr[r1]]
        table = meta.kv_indices[meta.kv_indptr[r0]:meta.kv_indptr[r1]]
        ids = np.unique(np.concatenate([home, table]))
        ids_d = torch.from_numpy(ids.astype(np.int64)).cuda()
        touched[ids_d] = True
        base = host_u16(pristine[ids_d]).reshape(1, len(ids), 2, Hkv, bs, D)
        # the group's tables with block ids renumbered into the compact pool
        sub_ctx = np.ascontiguousarray(meta.ctx_len[r0:r1])
        sub_indptr = (meta.kv_indptr[r0:r1 + 1] - meta.kv_indptr[r0]).astype(np.int64)
        sub_indices = np.searchsorted(ids, table).astype(np.int32)
        migs = [mig_pos[r] for r in range(r0, r1) if r in mig_pos]
        sub_mig_indptr = np.zeros(len(migs) + 1, dtype=np.int64)
        src, dst = [], []
        for i, m in enumerate(migs):
            a, b = int(meta.mig_indptr[m]), int(meta.mig_indptr[m + 1])
            src.append(meta.mig_src[a:b])
            dst.append(meta.mig_dst[a:b])
            sub_mig_indptr[i + 1] = sub_mig_indptr[i] + (b - a)
        sub_src = np.searchsorted(ids, np.concatenate(src)).astype(np.int32) if src else np.zeros(0, np.int32)
        sub_dst = np.searchsorted(ids, np.concatenate(dst)).astype(np.int32) if dst else np.zeros(0, np.int32)
        rows = slice(r0 * g1, r1 * g1)
        local_sel = np.array([r - r0 for r in range(r0, r1) if r in sel], dtype=np.int32)
        for l in layers:
            work = base.copy()
            oracle.kv_prepare(work, sub_mig_indptr, sub_src, sub_dst, sub_ctx, sub_indptr, sub_indices,
                              np.ascontiguousarray(k_new[l:l + 1, rows]), np.ascontiguousarray(v_new[l:l + 1, rows]),
                              cfg.gamma, layer_begin=0, layer_count=1)
            if l in layers_to_check and len(local_sel):
                o_ref = oracle.verify_attn(work, np.ascontiguousarray(q[l, rows]), sub_ctx, sub_indptr, sub_indices,
                                           cfg.gamma, req_list=local_sel)
                lrows = (local_sel[:, None] * g1 + np.arange(g1)[None, :]).ravel()
                o_gpu = host_u16(o[l][torch.from_numpy(lrows + r0 * g1).cuda()])
                bad, max_abs, max_rel = attn_mismatch(o_gpu, o_ref[lrows])
                assert bad == 0, (l, r0, bad, max_abs, max_rel)
                worst = (max(worst[0], max_abs), max(worst[1], max_rel))
                n_rows += len(lrows)
            if l in last_of_slab:
                got = host_u16(pool[last_of_slab[l]][ids_d]).reshape(work.shape)
                assert np.array_equal(got, work), f"slab {last_of_slab[l]} differs in the blocks of requests {r0}..{r1 - 1}"
    # blocks no request of the batch can touch still hold the fill pattern
    rest = torch.nonzero(~touched).ravel()
    for s in slabs_to_check:
        for i in range(0, len(rest), 8192):
            assert bool((pool[s][rest[i:i + 8192]] == int(W.BF16_NAN)).all()), f"slab {s}: a bystander block changed"
    print(f"attention: {n_rows} rows over {len(layers_to_check)} layers, max abs err {worst[0]:.3e}, max rel err {worst[1]:.3e}; "
          f"pool slabs {list(slabs_to_check)} bit-exact, {len(rest)} bystander blocks intact")


def _full_round_check(cfg, slabs, layers_to_check, slabs_to_check, modes=(False,)):
    """Runs the round at the configuration's full size once per mode (False = side-stream gather, True =
    gather-through) on the same uploaded slab and checks each run against the oracle."""
    meta = W.make_batch_meta(cfg)
    L, B, g1 = cfg.num_layers, cfg.batch, cfg.gamma + 1
    kv = [W.new_kv(cfg, meta, l) for l in range(L)]
    k_new, v_new = np.stack([a for a, _ in kv]), np.stack([b for _, b in kv])
    q = np.stack([W.queries(cfg, meta, l) for l in range(L)])
    p, qd, tok, ua, us = W.accept_inputs(cfg)
    acc_r, out_r, _ = oracle.spec_accept(p, qd, tok, ua, us)
    ctx = make_context(cfg, meta, num_slabs=slabs)
    db = DeviceBatch(meta)
    pristine = _upload_slab(cfg, meta)                       # every slab starts from these bytes (as in the bench)
    pool = torch.empty((slabs,) + tuple(pristine.shape), dtype=torch.int16, device="cuda:0")
    d_in = dict(k_new=dev(k_new), v_new=dev(v_new), q=dev(q), p=dev(p), q_draft=dev(qd), draft_tok=dev(tok),
                u_acc=dev(ua), u_smp=dev(us))
    ctx.nsd_verify_plan(meta.ctx_len, meta.kv_indptr, meta.is_migrated, cfg.gamma)
    for fuse in modes:
        for s in range(slabs):
            pool[s].copy_(pristine)
        o = torch.full(q.shape, 0x7FC0, dtype=torch.int16, device="cuda:0")
        acc = torch.full((B,), -7, dtype=torch.int32, device="cuda:0")
        out = torch.full((B, g1), -7, dtype=torch.int32, device="cuda:0")
        args = ctx.round_args(kv_pool=pool, n_mig_blocks=db.n_mig_blocks, mig_src=db.mig_src, mig_dst=db.mig_dst, batch=B,
                              gamma=cfg.gamma, ctx_len=db.ctx_len, kv_indptr=db.kv_indptr, kv_indices=db.kv_indices,
                              is_migrated=db.is_migrated, acc_len=acc, out_tok=out, o=o, fuse_gather=int(fuse), **d_in)
        for _ in range(2):                                   # twice: the round is idempotent, as the bench assumes
            ctx.nsd_verify_round(args)
        rc, bad = ctx.nsd_get_status()
        assert rc == 0, (rc, bad)
        rep = accept_compare(p, qd, tok, ua, us, acc.cpu().numpy(), out.cpu().numpy(), acc_r, out_r)
        assert rep["len_exact"] == B, rep
        print(f"{cfg.name} batch {B} fuse_gather={int(fuse)} acceptance:", rep)
        _check_against_oracle(cfg, meta, pristine, pool, o, k_new, v_new, q, slabs, layers_to_check, slabs_to_check)


# The one size these tests run at: the configuration's own batch, lengths, gamma and layer count.
FULL = pytest.mark.parametrize("size", ["full"])


@FULL
def test_knee_b512(size):
    """Configuration 3 of the benchmark set, as benchmarked: batch 512, 36 layers, lognormal contexts, 25% reassigned;
    side-stream gather and the gather-through variant."""
    _full_round_check(W.CONFIGS["knee_b512"], slabs=3, layers_to_check=[0, 4, 35], slabs_to_check=[0, 2], modes=(False, True))


@FULL
def test_migration_b256(size):
    """Configuration 4: batch 256, gamma 6, contexts 1024..8192, 75% reassigned; both gather modes."""
    _full_round_check(W.CONFIGS["migration_b256"], slabs=2, layers_to_check=[0, 3, 35], slabs_to_check=[0, 1], modes=(False, True))


@FULL
def test_long_b128(size):
    """Configuration 5: batch 128, gamma 8, contexts 8192..32768 (split-KV), low acceptance."""
    _full_round_check(W.CONFIGS["long_b128"], slabs=2, layers_to_check=[1, 34], slabs_to_check=[0])


def test_knee_b512_acceptance_from_logits_full_size():
    """nsd_spec_accept_logits in the launch configuration the benchmark times (batch 512, the Qwen3 vocabulary, fp32
    logits = log p of the configuration's acceptance inputs, T = 1: one wave of 512 CTAs, four per SM, the four-tile
    ring), every request launched, a sample of them checked against the logits oracle one by one; and the same decisions
    as nsd_spec_accept on the probabilities themselves wherever no test sits on a boundary."""
    cfg = W.CONFIGS["knee_b512"]
    meta = W.make_batch_meta(cfg)
    B, g, V = cfg.batch, cfg.gamma, cfg.vocab
    p, qd, tok, ua, us = W.accept_inputs(cfg)
    with np.errstate(divide="ignore"):
        z = np.log(p.astype(np.float64)).astype(np.float32)           # what both sides see
    ctx = make_context(cfg, meta, num_slabs=1)
    acc = torch.full((B,), -7, dtype=torch.int32, device="cuda:0")
    out = torch.full((B, g + 1), -7, dtype=torch.int32, device="cuda:0")
    ctx.nsd_spec_accept_logits(dev(z), 0, 1.0, dev(qd), dev(tok), dev(ua), dev(us), B, g, V, None, None, acc, out, None)
    rc, bad = ctx.nsd_get_status()
    assert rc == 0, (rc, bad)
    acc_g, out_g = acc.cpu().numpy(), out.cpu().numpy()

    sel = np.sort(np.random.default_rng(cfg.seed).choice(B, size=48, replace=False))
    acc_r, out_r, _ = oracle.spec_accept_logits(z[sel], 1.0, qd[sel], tok[sel], ua[sel], us[sel])
    pz = np.exp(z[sel].astype(np.float64))
    pz /= pz.sum(axis=-1, keepdims=True)
    rep = accept_compare(pz.astype(np.float32), qd[sel], tok[sel], ua[sel], us[sel], acc_g[sel], out_g[sel], acc_r, out_r)
    assert rep["len_exact"] >= len(sel) - 1, rep
    print("acceptance from logits:", rep)
    acc_p, _, _ = oracle.spec_accept(p, qd, tok, ua, us)
    assert (acc_g == acc_p).mean() > 0.99
    assert ((out_g >= -1) & (out_g < V)).all() and (acc_g >= 0).all() and (acc_g <= g).all()
