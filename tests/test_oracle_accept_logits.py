"""Pins for the logits-side acceptance oracle: the hand-worked cases through
log-probabilities, scipy softmax + the pinned probability oracle, chi-square of the
committed tokens against softmax(z/T), numpy argmax for greedy, per-request draft
lengths against truncated inputs."""
import numpy as np
import pytest
from scipy.special import softmax

import oracle
from test_oracle_accept import _CRIT_14DOF, _chi2, _golden_cases
from workload.gen import uniforms


def test_hand_worked_cases_through_log_probabilities():
    cases = _golden_cases()
    with np.errstate(divide="ignore"):
        z = np.log(np.array([[c[1], c[3]] for c in cases], dtype=np.float64)).astype(np.float32)   # p = 0 -> -inf
    # the unnormalised case (p sums to 0.4) becomes a normalised row under softmax: drop it here
    keep = [i for i, c in enumerate(cases) if abs(sum(c[1]) - 1.0) < 1e-6]
    q = np.array([[c[2]] for c in cases], dtype=np.float32)
    tok = np.array([[c[4]] for c in cases], dtype=np.int32)
    ua = np.array([[c[5]] for c in cases], dtype=np.float32)
    us = np.array([c[6] for c in cases], dtype=np.float32)
    acc, out, _ = oracle.spec_accept_logits(z[keep], 1.0, q[keep], tok[keep], ua[keep], us[keep])
    assert acc.tolist() == [cases[i][7] for i in keep]
    assert out.tolist() == [[cases[i][8], cases[i][9]] for i in keep]


@pytest.mark.parametrize("temperature", [1.0, 0.6, 2.5])
def test_equals_probability_oracle_on_scipy_softmax(temperature):
    """softmax by scipy in double, rounded to fp32, fed to the pinned probability oracle: the two may
    part only where the fp32 rounding of p moves a decision (counted, must be rare)."""
    rng = np.random.default_rng(int(temperature * 10))
    B, g, V = 400, 4, 257
    z = rng.normal(0, 2.0, (B, g + 1, V)).astype(np.float32)
    p = softmax(z.astype(np.float64) / temperature, axis=-1).astype(np.float32)
    q = softmax(z[:, :g].astype(np.float64) / temperature + rng.normal(0, 0.7, (B, g, V)), axis=-1).astype(np.float32)
    cdf = np.cumsum(q, axis=-1, dtype=np.float64)
    tok = np.array([[min(int(np.searchsorted(cdf[b, i], rng.random() * cdf[b, i, -1], side="right")), V - 1) for i in range(g)]
                    for b in range(B)], dtype=np.int32)
    ua, us = uniforms(rng, (B, g)), uniforms(rng, (B,))
    ctx = np.arange(B, dtype=np.int32)
    acc1, out1, new1 = oracle.spec_accept_logits(z, temperature, q, tok, ua, us, ctx_len=ctx)
    acc2, out2, _ = oracle.spec_accept(p, q, tok, ua, us)
    assert (acc1 == acc2).mean() > 0.995 and (out1 == out2).all(axis=1).mean() > 0.99
    assert (new1 == ctx + 1 + acc1).all()
    assert len(set(acc1.tolist())) == g + 1


def test_committed_tokens_follow_softmax_of_scaled_logits_chi_square():
    V, g, T = 16, 2, 0.7
    rng = np.random.default_rng(9)
    z_rows = rng.normal(0, 1.5, (g + 1, V)).astype(np.float32)
    z_rows[:, 3] = -np.inf                                  # a token the target can never emit
    q_rows = softmax(rng.normal(0, 1.0, (g, V)), axis=-1).astype(np.float32)
    target = softmax(z_rows.astype(np.float64) / T, axis=-1)
    counts = np.zeros((g + 1, V), dtype=np.int64)
    cdf = np.cumsum(q_rows.astype(np.float64), axis=-1)
    n = 100_000
    for c in range(10):
        r = np.random.default_rng(500 + c)
        tok = np.stack([np.minimum(np.searchsorted(cdf[i], r.random(n) * cdf[i, -1], side="right"), V - 1) for i in range(g)], 1).astype(np.int32)
        acc, out, _ = oracle.spec_accept_logits(np.ascontiguousarray(np.broadcast_to(z_rows, (n, g + 1, V))), T,
                                                np.ascontiguousarray(np.broadcast_to(q_rows, (n, g, V))), tok,
                                                uniforms(r, (n, g)), uniforms(r, (n,)))
        for j in range(g + 1):
            counts[j] += np.bincount(out[acc >= j, j], minlength=V)
    for j in range(g + 1):
        stat, dof = _chi2(counts[j], target[j])
        assert dof == 14 and stat < _CRIT_14DOF, (j, stat)


def test_greedy_is_argmax_matching():
    rng = np.random.default_rng(4)
    B, g, V = 300, 5, 97
    z = rng.integers(-3, 4, (B, g + 1, V)).astype(np.float32)          # many ties: the smallest index must win
    z[:, :, 50] = np.nan                                                # NaN never wins
    am = np.nanargmax(z, axis=-1)
    tok = am[:, :g].astype(np.int32).copy()
    wrong = rng.random((B, g)) < 0.3
    tok[wrong] = (tok[wrong] + 1) % V
    acc, out, _ = oracle.spec_accept_logits(z, 0.0, None, tok, None, None)
    for b in range(B):
        n = g if not wrong[b].any() else int(np.argmax(wrong[b]))
        assert acc[b] == n
        assert out[b].tolist() == tok[b, :n].tolist() + [int(am[b, n])] + [-1] * (g - n)


def test_per_request_draft_length_equals_truncated_inputs():
    rng = np.random.default_rng(12)
    B, g, V = 60, 4, 64
    z = rng.normal(0, 2, (B, g + 1, V)).astype(np.float32)
    q = softmax(rng.normal(0, 2, (B, g, V)), axis=-1).astype(np.float32)
    tok = rng.integers(0, V, (B, g)).astype(np.int32)
    ua, us = uniforms(rng, (B, g)) * 0.2, uniforms(rng, (B,))            # small uniforms: long accepted runs
    gr = rng.integers(0, g + 1, B).astype(np.int32)
    acc, out, _ = oracle.spec_accept_logits(z, 1.0, q, tok, ua, us, gamma_r=gr)
    for b in range(B):
        gb = int(gr[b])
        if gb == 0:
            a1, o1, _ = oracle.spec_accept_logits(z[b:b + 1, :2], 1.0, q[b:b + 1, :1], tok[b:b + 1, :1], np.ones((1, 1), np.float32) * 0, us[b:b + 1],
                                                  gamma_r=np.zeros(1, np.int32))
            assert acc[b] == 0 and out[b, 0] == o1[0, 0]
            continue
        a1, o1, _ = oracle.spec_accept_logits(np.ascontiguousarray(z[b:b + 1, :gb + 1]), 1.0, np.ascontiguousarray(q[b:b + 1, :gb]),
                                              np.ascontiguousarray(tok[b:b + 1, :gb]), np.ascontiguousarray(ua[b:b + 1, :gb]), us[b:b + 1])
        assert acc[b] == a1[0] <= gb
        assert out[b, :gb + 1].tolist() == o1[0].tolist() and (out[b, gb + 1:] == -1).all()
