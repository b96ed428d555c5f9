"""Pins for the acceptance oracle: hand-worked cases, invariants, closed-form
statistics, the exact-distribution rule by chi-square (with a negative control)
and an independent numpy brute force."""
import os

import numpy as np
import pytest

import oracle
import workload as W
from workload.gen import uniforms

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "accept_worked_v4.txt")


def _golden_cases():
    cases = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            tk = line.split()
            vals = [float(x) for x in tk[1:]]
            cases.append((tk[0], vals[0:4], vals[4:8], vals[8:12], int(vals[12]), vals[13], vals[14],
                          int(vals[15]), int(vals[16]), int(vals[17])))
    return cases


@pytest.mark.parametrize("case", _golden_cases(), ids=lambda c: c[0])
def test_worked_example(case):
    _, p0, q0, p1, x, ua, us, want_len, want_t0, want_t1 = case
    p = np.array([[p0, p1]], dtype=np.float32)
    q = np.array([[q0]], dtype=np.float32)
    acc, out, _ = oracle.spec_accept(p, q, np.array([[x]], dtype=np.int32), np.array([[ua]], dtype=np.float32),
                                     np.array([us], dtype=np.float32))
    assert acc[0] == want_len
    assert list(out[0]) == [want_t0, want_t1]


def _fixed_rows(V=16, gamma=4, seed=5):
    """Fixed p, q rows with q>p, p>q, p=0 and tiny-q entries."""
    rng = np.random.default_rng(seed)
    p = rng.gamma(0.6, size=(gamma + 1, V))
    q = rng.gamma(0.6, size=(gamma, V))
    p[:, 3] = 0.0            # target never emits token 3
    q[:, 7] = 1e-6           # draft almost never proposes token 7
    p[:, 11] *= 4.0
    p /= p.sum(-1, keepdims=True)
    q /= q.sum(-1, keepdims=True)
    return p.astype(np.float32), q.astype(np.float32)


def _trials(p_rows, q_rows, n, seed):
    gamma, V = q_rows.shape
    rng = np.random.default_rng(seed)
    cdf = np.cumsum(q_rows.astype(np.float64), axis=-1)
    tok = np.empty((n, gamma), dtype=np.int32)
    for i in range(gamma):
        tok[:, i] = np.minimum(np.searchsorted(cdf[i], rng.random(n) * cdf[i, -1], side="right"), V - 1)
    u_acc = uniforms(rng, (n, gamma))
    u_smp = uniforms(rng, (n,))
    p = np.ascontiguousarray(np.broadcast_to(p_rows, (n, gamma + 1, V)))
    q = np.ascontiguousarray(np.broadcast_to(q_rows, (n, gamma, V)))
    return p, q, tok, u_acc, u_smp


def test_invariants_random():
    cfg = W.CONFIGS["tiny"]
    meta = W.make_batch_meta(cfg)
    p, q, tok, ua, us = W.accept_inputs(cfg, batch=64)
    ctx = np.arange(64, dtype=np.int32) + 17
    acc, out, new_ctx = oracle.spec_accept(p, q, tok, ua, us, ctx)
    g = cfg.gamma
    assert ((acc >= 0) & (acc <= g)).all()
    for r in range(64):
        n = acc[r]
        assert (out[r, :n] == tok[r, :n]).all()
        y = out[r, n]
        assert 0 <= y < cfg.vocab
        assert (out[r, n + 1:] == -1).all()
        if n < g:
            assert p[r, n, y] > q[r, n, y]          # a resampled token has positive residual
            x = tok[r, n]
            assert not (ua[r, n] < min(1.0, float(p[r, n, x]) / float(q[r, n, x])))
        else:
            assert p[r, g, y] > 0
        for i in range(n):
            x = tok[r, i]
            assert ua[r, i] < min(1.0, float(p[r, i, x]) / float(q[r, i, x]))
        assert new_ctx[r] == ctx[r] + 1 + n


def test_closed_form_accept_length_law():
    """P(acc_len = k) = prod_{i<k} a_i * (1 - a_k), a_i = sum_k min(p_i, q_i)."""
    gamma = 4
    p_rows, q_rows = _fixed_rows(gamma=gamma)
    n = 200_000
    acc, out, _ = oracle.spec_accept(*_trials(p_rows, q_rows, n, seed=11))
    a = np.minimum(p_rows[:gamma].astype(np.float64), q_rows.astype(np.float64)).sum(-1)
    want = np.array([np.prod(a[:k]) * (1 - a[k]) for k in range(gamma)] + [np.prod(a)])
    got = np.bincount(acc, minlength=gamma + 1) / n
    sigma = np.sqrt(want * (1 - want) / n)
    assert (np.abs(got - want) < 4.5 * sigma + 1e-9).all(), (got, want)
    mean_tokens = (acc + 1).mean()
    want_mean = float((want * (np.arange(gamma + 1) + 1)).sum())
    assert abs(mean_tokens - want_mean) < 0.02


def _chi2(counts, probs):
    n = counts.sum()
    mask = probs > 0
    assert counts[~mask].sum() == 0, "token with zero target probability was committed"
    e = probs[mask] * n
    return float(((counts[mask] - e) ** 2 / e).sum()), int(mask.sum()) - 1


# chi-square critical values at p = 1e-4 for 14 dof (token 3 has zero mass: 15 cells)
_CRIT_14DOF = 42.58


@pytest.mark.parametrize("gamma", [1, 4])
def test_committed_tokens_follow_target_chi_square(gamma):
    """Exact rule: every committed token at position j is distributed as target row j."""
    V = 16
    p_rows, q_rows = _fixed_rows(V=V, gamma=gamma, seed=5 + gamma)
    total, chunk = 1_000_000, 100_000
    counts = np.zeros((gamma + 1, V), dtype=np.int64)
    for c in range(total // chunk):
        acc, out, _ = oracle.spec_accept(*_trials(p_rows, q_rows, chunk, seed=1000 + c))
        for j in range(gamma + 1):
            t = out[acc >= j, j]
            counts[j] += np.bincount(t, minlength=V)
    for j in range(gamma + 1):
        pj = p_rows[j].astype(np.float64)
        stat, dof = _chi2(counts[j], pj / pj.sum())
        assert dof == 14
        assert stat < _CRIT_14DOF, (j, stat)


def test_chi_square_has_power_negative_control():
    """The same statistic must reject a wrong rule (resampling from p instead of
    the residual), or the test above proves nothing."""
    V, gamma = 16, 1
    p_rows, q_rows = _fixed_rows(V=V, gamma=gamma, seed=6)
    n = 1_000_000
    p, q, tok, ua, us = _trials(p_rows, q_rows, n, seed=77)
    x = tok[:, 0]
    ratio = p_rows[0, x].astype(np.float64) / q_rows[0, x].astype(np.float64)
    accept = ua[:, 0] < np.minimum(1.0, ratio)
    cdf = np.cumsum(p_rows[0].astype(np.float64))
    wrong = np.minimum(np.searchsorted(cdf, us.astype(np.float64) * cdf[-1], side="right"), V - 1)
    first = np.where(accept, x, wrong)
    pj = p_rows[0].astype(np.float64)
    mask = pj > 0
    cnt = np.bincount(first, minlength=V)
    e = pj / pj.sum() * n
    stat = float(((cnt[mask] - e[mask]) ** 2 / e[mask]).sum())
    assert stat > 10 * _CRIT_14DOF


def _numpy_accept(p, q, tok, ua, us):
    """Independent formulation: vector compares, np.cumsum + searchsorted."""
    B, g1, V = p.shape
    g = g1 - 1
    acc = np.empty(B, dtype=np.int32)
    out = np.full((B, g1), -1, dtype=np.int32)
    for r in range(B):
        P = p[r, np.arange(g), tok[r]].astype(np.float64)
        Q = q[r, np.arange(g), tok[r]].astype(np.float64)
        with np.errstate(divide="ignore", invalid="ignore"):
            ratio = np.where(Q > 0, P / Q, np.where(P > 0, 1.0, 0.0))
        ok = ua[r].astype(np.float64) < np.minimum(1.0, ratio)
        n = g if ok.all() else int(np.argmin(ok))
        if n < g:
            w = np.maximum(p[r, n] - q[r, n], np.float32(0)).astype(np.float64)
            if np.cumsum(w)[-1] == 0:
                w = p[r, n].astype(np.float64)
        else:
            w = p[r, g].astype(np.float64)
        C = np.cumsum(w)                       # sequential, double
        k = int(np.searchsorted(C, float(us[r]) * C[-1], side="right"))
        if k >= V:
            k = int(np.nonzero(w > 0)[0][-1])
        acc[r] = n
        out[r, :n] = tok[r, :n]
        out[r, n] = k
    return acc, out


def test_matches_numpy_brute_force_tiny_config():
    cfg = W.CONFIGS["tiny"]
    p, q, tok, ua, us = W.accept_inputs(cfg, batch=256)
    acc, out, _ = oracle.spec_accept(p, q, tok, ua, us)
    acc2, out2 = _numpy_accept(p, q, tok, ua, us)
    assert (acc == acc2).all() and (out == out2).all()


def test_matches_numpy_brute_force_sparse_rows():
    rng = np.random.default_rng(3)
    B, g, V = 500, 3, 37
    p = rng.random((B, g + 1, V)) * (rng.random((B, g + 1, V)) < 0.5)
    q = rng.random((B, g, V)) * (rng.random((B, g, V)) < 0.5)
    p[:, :, 0] += 1e-3
    q[:, :, 1] += 1e-3
    p = (p / p.sum(-1, keepdims=True)).astype(np.float32)
    q = (q / q.sum(-1, keepdims=True)).astype(np.float32)
    tok = rng.integers(0, V, size=(B, g)).astype(np.int32)      # includes tokens with q = 0
    ua, us = uniforms(rng, (B, g)), uniforms(rng, (B,))
    acc, out, _ = oracle.spec_accept(p, q, tok, ua, us)
    acc2, out2 = _numpy_accept(p, q, tok, ua, us)
    assert (acc == acc2).all() and (out == out2).all()
    assert len(set(acc.tolist())) == g + 1                      # every accepted length occurs


def test_synthetic_acceptance_rate_closed_form():
    """q = softmax(z + N(0, s^2)) gives a per-position acceptance rate of
    2*Phi(-s/2) for a large vocabulary: 0.7237 at variance 0.5."""
    from scipy.stats import norm

    cfg = W.RoundConfig("acc_rate", batch=16, gamma=4, num_layers=1, num_q_heads=8, num_kv_heads=2, head_dim=64,
                        block_size=16, vocab=50_000, ctx_dist=("uniform", 17, 100), frac_reassigned=0.0,
                        noise_var=0.5, seed=99)
    p, q, *_ = W.accept_inputs(cfg)
    alpha = np.minimum(p[:, :4], q).sum(-1, dtype=np.float64).mean()
    assert abs(alpha - 2 * norm.cdf(-np.sqrt(0.5) / 2)) < 0.01
