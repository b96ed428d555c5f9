"""GPU parity: nsd_spec_accept_logits against the fp64 logits oracle.  Greedy mode and
accepted lengths are exact (length mismatches only within 1e-5 of a decision boundary,
reported); sampled tokens exact or within the 1e-5 CDF tolerance (counted)."""
import numpy as np
import pytest
import torch
from scipy.special import softmax

import oracle
import workload as W
import nsd_testlib
from nsd_testlib import TOKEN_CDF_TOL, dev, make_context
from workload.gen import uniforms

pytestmark = pytest.mark.gpu


def _ctx(vocab, batch, gamma):
    cfg = W.RoundConfig("accl", batch=batch, gamma=gamma, num_layers=1, num_q_heads=8, num_kv_heads=2, head_dim=64,
                        block_size=16, vocab=vocab, ctx_dist=("fixed", [1] * batch), frac_reassigned=0.0, seed=1)
    return make_context(cfg, W.make_batch_meta(cfg))


def _gpu(z, dtype, T, q, tok, ua, us, gamma_r=None, ctx_len=None):
    B, g1, V = z.shape
    ctx = _ctx(V, B, g1 - 1)
    if dtype == 1:
        zd = torch.from_numpy(W.f32_to_bf16(z).view(np.int16)).cuda()
    else:
        zd = dev(z)
    acc = torch.full((B,), -7, dtype=torch.int32, device="cuda:0")
    out = torch.full((B, g1), -7, dtype=torch.int32, device="cuda:0")
    new = torch.full((B,), -7, dtype=torch.int32, device="cuda:0") if ctx_len is not None else None
    ctx.nsd_spec_accept_logits(zd, dtype, T, dev(q), dev(tok), dev(ua), dev(us), B, g1 - 1, V, dev(gamma_r), dev(ctx_len),
                               acc, out, new)
    rc, bad = ctx.nsd_get_status()
    assert rc == 0, (rc, bad)
    return acc.cpu().numpy(), out.cpu().numpy(), (new.cpu().numpy() if new is not None else None)


def _compare_sampled(z, T, q, tok, ua, us, acc_g, out_g, acc_r, out_r, gamma_r=None):
    """The acceptance parity rule with p = softmax(z/T) in double."""
    B, g1, V = z.shape
    rep = dict(len_exact=0, len_near=0, tok_exact=0, tok_tol=0)
    for r in range(B):
        g = int(gamma_r[r]) if gamma_r is not None else g1 - 1
        if acc_g[r] != acc_r[r]:
            i = int(min(acc_g[r], acc_r[r]))
            p = softmax(z[r, i].astype(np.float64) / T)
            x = tok[r, i]
            ratio = p[x] / float(q[r, i, x]) if q[r, i, x] > 0 else (1.0 if p[x] > 0 else 0.0)
            assert abs(float(ua[r, i]) - min(1.0, ratio)) < 1e-5, f"request {r}: length {acc_g[r]} vs {acc_r[r]}"
            rep["len_near"] += 1
            continue
        rep["len_exact"] += 1
        n = int(acc_r[r])
        assert (out_g[r, :n] == out_r[r, :n]).all() and (out_g[r, n + 1:] == -1).all()
        if out_g[r, n] == out_r[r, n]:
            rep["tok_exact"] += 1
            continue
        p = softmax(z[r, n].astype(np.float64) / T)
        w = np.maximum(p - q[r, n].astype(np.float64), 0) if n < g else p
        if w.sum() == 0:
            w = p
        C = np.cumsum(w)
        y = int(out_g[r, n])
        frac = float(us[r])
        assert 0 <= y < V and (C[y - 1] if y else 0.0) / C[-1] - TOKEN_CDF_TOL <= frac <= C[y] / C[-1] + TOKEN_CDF_TOL, f"request {r}"
        rep["tok_tol"] += 1
    print("logits accept parity:", rep)
    return rep


def _inputs(rng, B, g, V, T, noise=0.7):
    z = rng.normal(0, 2.0, (B, g + 1, V)).astype(np.float32)
    q = softmax(z[:, :g].astype(np.float64) / T + rng.normal(0, noise, (B, g, V)), axis=-1).astype(np.float32)
    cdf = np.cumsum(q, axis=-1, dtype=np.float64)
    tok = np.array([[min(int(np.searchsorted(cdf[b, i], rng.random() * cdf[b, i, -1], side="right")), V - 1) for i in range(g)]
                    for b in range(B)], dtype=np.int32)
    return z, q, tok, uniforms(rng, (B, g)), uniforms(rng, (B,))


@pytest.mark.parametrize("V,T,dtype", [(1000, 1.0, 0), (1001, 0.7, 0), (4099, 1.5, 0), (1000, 1.0, 1), (130, 0.5, 1), (5, 1.0, 0)])
def test_sampling_matches_the_oracle(V, T, dtype):
    rng = np.random.default_rng(V + dtype)
    B, g = 96, 4
    z, q, tok, ua, us = _inputs(rng, B, g, V, T)
    if dtype == 1:
        z = W.bf16_to_f32(W.f32_to_bf16(z))                          # both sides see the bf16-rounded logits
    ctx_len = np.arange(B, dtype=np.int32)
    acc_g, out_g, new_g = _gpu(z, dtype, T, q, tok, ua, us, ctx_len=ctx_len)
    acc_r, out_r, new_r = oracle.spec_accept_logits(z, T, q, tok, ua, us, ctx_len=ctx_len)
    rep = _compare_sampled(z, T, q, tok, ua, us, acc_g, out_g, acc_r, out_r)
    assert rep["len_exact"] >= B - 1 and rep["tok_exact"] >= B - 3
    same = acc_g == acc_r
    assert (new_g[same] == new_r[same]).all()
    assert len(set(acc_r.tolist())) >= 3


@pytest.mark.parametrize("dtype", [0, 1])
def test_greedy_is_exact(dtype):
    rng = np.random.default_rng(8 + dtype)
    B, g, V = 200, 6, 1003
    z = rng.integers(-4, 5, (B, g + 1, V)).astype(np.float32)          # ties everywhere, exactly representable in bf16
    z[:, :, 77] = np.nan
    am = np.nanargmax(z, axis=-1)
    tok = am[:, :g].astype(np.int32).copy()
    wrong = rng.random((B, g)) < 0.25
    tok[wrong] = (tok[wrong] + 3) % V
    acc_g, out_g, _ = _gpu(z, dtype, 0.0, None, tok, None, None)
    acc_r, out_r, _ = oracle.spec_accept_logits(z, 0.0, None, tok, None, None)
    assert np.array_equal(acc_g, acc_r) and np.array_equal(out_g, out_r)
    assert len(set(acc_r.tolist())) == g + 1


def test_per_request_draft_lengths():
    rng = np.random.default_rng(21)
    B, g, V, T = 80, 5, 512, 1.0
    z, q, tok, ua, us = _inputs(rng, B, g, V, T, noise=0.3)
    gr = rng.integers(0, g + 1, B).astype(np.int32)
    acc_g, out_g, _ = _gpu(z, 0, T, q, tok, ua, us, gamma_r=gr)
    acc_r, out_r, _ = oracle.spec_accept_logits(z, T, q, tok, ua, us, gamma_r=gr)
    rep = _compare_sampled(z, T, q, tok, ua, us, acc_g, out_g, acc_r, out_r, gamma_r=gr)
    assert rep["len_exact"] >= B - 1 and (acc_g <= gr).all()
    acc_g, out_g, _ = _gpu(z, 0, 0.0, None, tok, None, None, gamma_r=gr)
    acc_r, out_r, _ = oracle.spec_accept_logits(z, 0.0, None, tok, None, None, gamma_r=gr)
    assert np.array_equal(acc_g, acc_r) and np.array_equal(out_g, out_r)


def test_qwen3_vocab_bf16_logits():
    rng = np.random.default_rng(33)
    B, g, V, T = 24, 4, 151936, 1.0
    z, q, tok, ua, us = _inputs(rng, B, g, V, T, noise=0.7)
    z = W.bf16_to_f32(W.f32_to_bf16(z))
    acc_g, out_g, _ = _gpu(z, 1, T, q, tok, ua, us)
    acc_r, out_r, _ = oracle.spec_accept_logits(z, T, q, tok, ua, us)
    rep = _compare_sampled(z, T, q, tok, ua, us, acc_g, out_g, acc_r, out_r)
    assert rep["len_exact"] >= B - 1


@pytest.mark.parametrize("B", [200, 320], ids=["deep_ring", "four_per_sm"])
@pytest.mark.parametrize("V,dtype,T", [(4104, 0, 0.8), (20488, 0, 1.0), (8200, 1, 1.0), (12296, 1, 0.0), (2052, 0, 0.0)])
def test_ring_and_direct_feeds_agree_bit_for_bit(V, dtype, T, B, monkeypatch):
    """Rows whose starts are 16-byte aligned travel through the shared-memory ring of bulk copies; NSD_FLAG_LOGITS_DIRECT
    keeps them on direct loads.  Every thread sees the same elements in the same order, so nothing may differ.  The
    vocabularies span several 8 KiB tiles with a ragged last one, both for the row sweep and for the draw."""
    # batch 200: CTAs have an SM (nearly) to themselves and get the 12-tile ring; batch 320: four CTAs per SM, 4 tiles
    rng = np.random.default_rng(V + B)
    g = 5
    z, q, tok, ua, us = _inputs(rng, B, g, V, T if T > 0 else 1.0)
    z[:, :, 5] = 0.25 * np.round(4 * z[:, :, 9])                       # some exact ties for the argmax
    if dtype == 1:
        z = W.bf16_to_f32(W.f32_to_bf16(z))
    if T == 0:                                                         # greedy drafts: the argmax, a quarter of them wrong
        tok = np.argmax(z[:, :g], axis=-1).astype(np.int32)
        wrong = rng.random((B, g)) < 0.25
        tok[wrong] = (tok[wrong] + 3) % V
    res = {}
    for feed in ("ring", "direct"):
        monkeypatch.setattr(nsd_testlib, "CONTEXT_FLAGS", (1 << 3) if feed == "direct" else 0)
        res[feed] = _gpu(z, dtype, T, q, tok, ua, us) if T > 0 else _gpu(z, dtype, 0.0, None, tok, None, None)
    assert np.array_equal(res["ring"][0], res["direct"][0]) and np.array_equal(res["ring"][1], res["direct"][1])
    acc_r, out_r, _ = oracle.spec_accept_logits(z, T, q, tok, ua, us) if T > 0 else oracle.spec_accept_logits(z, 0.0, None, tok, None, None)
    if T > 0:
        rep = _compare_sampled(z, T, q, tok, ua, us, res["ring"][0], res["ring"][1], acc_r, out_r)
        assert rep["len_exact"] >= B - 1 and rep["tok_exact"] >= B - 4
    else:
        assert np.array_equal(res["ring"][0], acc_r) and np.array_equal(res["ring"][1], out_r)
    assert len(set(acc_r.tolist())) >= 3


def test_bad_arguments():
    import paper_2609_29364_b200 as nsd

    ctx = _ctx(100, 4, 2)
    z = torch.zeros(4 * 3 * 100, device="cuda:0")
    zi = torch.zeros(16, dtype=torch.int32, device="cuda:0")
    cases = [((None, 0, 1.0, z, zi, z, z, 4, 2, 100, None, None, zi, zi), 1), ((z, 2, 1.0, z, zi, z, z, 4, 2, 100, None, None, zi, zi), 4),
             ((z, 0, -1.0, z, zi, z, z, 4, 2, 100, None, None, zi, zi), 1), ((z, 0, 1.0, None, zi, z, z, 4, 2, 100, None, None, zi, zi), 1),
             ((z, 0, 1.0, z, zi, z, z, 5, 2, 100, None, None, zi, zi), 2), ((z, 0, 1.0, z, zi, z, z, 4, 2, 100, None, None, zi, zi, zi), 1)]
    for args, want in cases:
        with pytest.raises(nsd.NsdError) as e:
            ctx.nsd_spec_accept_logits(*args)
        assert e.value.code == want
    assert ctx.nsd_launch_count() == 0
    ctx.nsd_spec_accept_logits(z, 0, 0.0, None, zi, None, None, 4, 2, 100, dev(np.array([1, 9, 0, 2], np.int32)), None, zi, zi)
    rc, bad = ctx.nsd_get_status()
    assert rc == 6 and bad == 1
