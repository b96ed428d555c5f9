"""GPU parity: nsd_spec_accept against the oracle: accepted lengths bit-exact,
tokens exact or within the stated CDF tolerance (counted and reported)."""
import numpy as np
import pytest

import oracle
import workload as W
from nsd_testlib import accept_compare, make_context, run_accept_gpu
from test_oracle_accept import _golden_cases
from workload.gen import uniforms

pytestmark = pytest.mark.gpu


def _ctx(vocab, batch, gamma):
    cfg = W.RoundConfig("acc", batch=batch, gamma=gamma, num_layers=1, num_q_heads=8, num_kv_heads=2, head_dim=64,
                        block_size=16, vocab=vocab, ctx_dist=("fixed", [1] * batch), frac_reassigned=0.0, seed=1)
    return make_context(cfg, W.make_batch_meta(cfg))


def _compare(p, q, tok, ua, us, ctx_len=None, expect_all_exact=False):
    B, g1, V = p.shape
    ctx = _ctx(V, B, g1 - 1)
    acc_g, out_g, new_g = run_accept_gpu(ctx, p, q, tok, ua, us, ctx_len)
    rc, bad = ctx.nsd_get_status()
    assert rc == 0, (rc, bad)
    acc_r, out_r, new_r = oracle.spec_accept(p, q, tok, ua, us, ctx_len)
    rep = accept_compare(p, q, tok, ua, us, acc_g, out_g, acc_r, out_r)
    if ctx_len is not None:
        same = acc_g == acc_r
        assert (new_g[same] == new_r[same]).all()
    if expect_all_exact:
        assert rep["len_exact"] == B and rep["tok_exact"] == B, rep
    print("accept parity:", rep)
    return rep, acc_g, out_g


def test_hand_worked_cases_through_the_gpu():
    cases = _golden_cases()
    p = np.array([[c[1], c[3]] for c in cases], dtype=np.float32)
    q = np.array([[c[2]] for c in cases], dtype=np.float32)
    tok = np.array([[c[4]] for c in cases], dtype=np.int32)
    ua = np.array([[c[5]] for c in cases], dtype=np.float32)
    us = np.array([c[6] for c in cases], dtype=np.float32)
    _, acc, out = _compare(p, q, tok, ua, us, expect_all_exact=True)
    assert acc.tolist() == [c[7] for c in cases]
    assert out.tolist() == [[c[8], c[9]] for c in cases]


def test_tiny_config():
    cfg = W.CONFIGS["tiny"]
    meta = W.make_batch_meta(cfg)
    p, q, tok, ua, us = W.accept_inputs(cfg)
    _compare(p, q, tok, ua, us, meta.ctx_len, expect_all_exact=True)
    p, q, tok, ua, us = W.accept_inputs(cfg, batch=300)
    rep, acc, _ = _compare(p, q, tok, ua, us)
    assert rep["len_exact"] == 300 and len(set(acc.tolist())) >= 3


@pytest.mark.parametrize("vocab", [1, 2, 3, 5, 127, 128, 129, 1001, 4099])
def test_odd_vocab_sizes_and_sparse_rows(vocab):
    """Vocabularies that are not a multiple of 4 or of the 128-token segment; rows
    with zeros; draft tokens the draft row gives no mass to."""
    rng = np.random.default_rng(vocab)
    B, g = 64, 3
    p = rng.random((B, g + 1, vocab)) * (rng.random((B, g + 1, vocab)) < 0.6)
    q = rng.random((B, g, vocab)) * (rng.random((B, g, vocab)) < 0.6)
    p[:, :, 0] += 1e-3
    q[:, :, -1] += 1e-3
    p = (p / p.sum(-1, keepdims=True)).astype(np.float32)
    q = (q / q.sum(-1, keepdims=True)).astype(np.float32)
    tok = rng.integers(0, vocab, size=(B, g)).astype(np.int32)
    rep, _, _ = _compare(p, q, tok, uniforms(rng, (B, g)), uniforms(rng, (B,)))
    assert rep["len_exact"] == B


def test_empty_residual_and_all_zero_rows():
    V = 256
    p = np.full((3, 2, V), 0.001, dtype=np.float32)
    q = np.full((3, 1, V), 0.0039, dtype=np.float32)         # p <= q everywhere: the residual is empty
    p[2] = 0.0                                               # nothing to draw from at all -> token -1
    tok = np.array([[5], [9], [1]], dtype=np.int32)
    ua = np.array([[0.9], [0.1], [0.5]], dtype=np.float32)   # ratio = 0.256: reject, accept, reject
    us = np.array([0.5, 0.999, 0.3], dtype=np.float32)
    _, acc, out = _compare(p, q, tok, ua, us, expect_all_exact=True)
    assert acc.tolist() == [0, 1, 0] and out[2].tolist() == [-1, -1]


@pytest.mark.parametrize("batch", [1, 3, 37, 150])
def test_small_batches_share_a_request_among_ctas(batch):
    """Below two CTAs per SM the kernel gives a request to several CTAs (2..8 here, 1 at batch 150 and
    above): same lengths, same tokens as the oracle, twice in a row (the arrival counters must be back
    at zero), including a request whose residual is empty and one whose rows are all zero."""
    V, g = 70000, 3
    cfg = W.RoundConfig("accsplit", batch=batch, gamma=g, num_layers=1, num_q_heads=8, num_kv_heads=2, head_dim=64,
                        block_size=16, vocab=V, ctx_dist=("fixed", [1] * batch), frac_reassigned=0.0, noise_var=1.0, seed=77 + batch)
    p, q, tok, ua, us = W.accept_inputs(cfg)
    q[0, 0] = 1.0 / V
    p[0, 0] = 0.25 / V                                       # p <= q everywhere at the first position of request 0 ...
    ua[0, 0] = 0.9                                           # ... which is rejected: the draw falls back to the target row
    if batch > 2:
        p[2] = 0.0                                           # nothing to draw from at all -> token -1
    ctx = _ctx(V, batch, g)
    acc_r, out_r, _ = oracle.spec_accept(p, q, tok, ua, us)
    for _ in range(2):
        acc_g, out_g, _ = run_accept_gpu(ctx, p, q, tok, ua, us)
        rc, bad = ctx.nsd_get_status()
        assert rc == 0, (rc, bad)
        rep = accept_compare(p, q, tok, ua, us, acc_g, out_g, acc_r, out_r)
        assert rep["len_exact"] == batch, rep
    assert acc_r[0] == 0 and out_g[0, 0] >= 0
    if batch > 2:
        assert out_g[2].tolist().count(-1) >= 1


def test_out_of_vocab_draft_token_is_reported_and_rejected():
    V = 64
    rng = np.random.default_rng(0)
    p = rng.random((2, 3, V)).astype(np.float32)
    q = rng.random((2, 2, V)).astype(np.float32)
    tok = np.array([[3, V + 7], [1, 2]], dtype=np.int32)
    ctx = _ctx(V, 2, 2)
    acc, out, _ = run_accept_gpu(ctx, p, q, tok, np.zeros((2, 2), np.float32), np.array([0.5, 0.5], np.float32))
    rc, bad = ctx.nsd_get_status()
    assert rc == 6 and bad == 0
    assert acc[0] <= 1


def test_qwen3_vocab_high_and_low_acceptance():
    """Vocabulary 151936 at the two divergence settings of the configs (noise
    variance 0.5 -> ~0.72 accepted per position; 1.0 -> ~0.62)."""
    for noise, gamma, seed in ((0.5, 4, 20260930), (1.0, 8, 20260933)):
        cfg = W.RoundConfig("acc_big", batch=48, gamma=gamma, num_layers=1, num_q_heads=32, num_kv_heads=8,
                            head_dim=128, block_size=16, vocab=151936, ctx_dist=("fixed", [1] * 48),
                            frac_reassigned=0.0, noise_var=noise, seed=seed)
        p, q, tok, ua, us = W.accept_inputs(cfg)
        rep, acc, _ = _compare(p, q, tok, ua, us)
        assert rep["len_exact"] == 48
        assert rep["tok_exact"] >= 47


def test_bad_arguments():
    import paper_2609_29364_b200 as nsd
    import torch

    ctx = _ctx(100, 4, 2)
    z = torch.zeros(4 * 3 * 100, device="cuda:0")
    zi = torch.zeros(16, dtype=torch.int32, device="cuda:0")
    for args, want in (((None, z, zi, z, z, 4, 2, 100, None, zi, zi), 1), ((z, z, zi, z, z, 5, 2, 100, None, zi, zi), 2),
                       ((z, z, zi, z, z, 4, 3, 100, None, zi, zi), 2), ((z, z, zi, z, z, 4, 2, 0, None, zi, zi), 2),
                       ((z, z, zi, z, z, 4, 2, 100, None, zi, zi, zi), 1)):
        with pytest.raises(nsd.NsdError) as e:
            ctx.nsd_spec_accept(*args)
        assert e.value.code == want
    assert ctx.nsd_launch_count() == 0
