"""Plain-Python oracle of worker-triggered batch reconstruction (Algorithm 1).

TEST INFRASTRUCTURE, NOT PRODUCT.  Written from the paper's statements, step by
step in its notation: Eq. (6) earliest predicted start S(B, w), Eq. (7)
service-admission bound d_r(w), Eq. (8) admissibility, Appendix F.2 physical
fit.  The paper names the ranking criteria (predecessor readiness, waiting time,
temporal compatibility) without a formula; the reading used here is stated in
`rank_key`.  Admissibility is re-evaluated from the definitions for every trial
batch (no incremental state), which is what makes this the slow, obvious version.
"""
from __future__ import annotations


def start_time(batch, a_w, e, k):
    """Eq. (6): S(B, w) = max(a_w, max_r e_r, max_r k_r(w))."""
    return max([a_w] + [e[r] for r in batch] + [k[r] for r in batch])


def admission_bound(r, a_w, e, k, g_s, delta_s):
    """Eq. (7): d_r(w) = max(e_r + g_s, S({r}, w)) + Delta_s."""
    return max(e[r] + g_s, start_time([r], a_w, e, k)) + delta_s


def fits(batch, rows, blocks, tokens, row_cap, block_cap, token_cap):
    """Appendix F.2: batch-row capacity, KV-block capacity, token limit."""
    return (sum(rows[r] for r in batch) <= row_cap and sum(blocks[r] for r in batch) <= block_cap
            and sum(tokens[r] for r in batch) <= token_cap)


def admissible(batch, a_w, e, k, g_s, delta_s, b_max, rows, blocks, tokens, row_cap, block_cap, token_cap):
    """Eq. (8)."""
    if len(batch) > b_max or not fits(batch, rows, blocks, tokens, row_cap, block_cap, token_cap):
        return False
    return start_time(batch, a_w, e, k) <= min(admission_bound(r, a_w, e, k, g_s, delta_s) for r in batch)


def rank_key(r, a_w, e, k, g_s, delta_s):
    """Reading of line 2: most urgent admission bound first, then the older predecessor output
    (waiting time / aging), then the earlier singleton start (temporal compatibility), then index."""
    return (admission_bound(r, a_w, e, k, g_s, delta_s), e[r], start_time([r], a_w, e, k), r)


def schedule_batch(a_w, g_s, delta_s, b_max, e, k, eligible=None, rows=None, blocks=None, tokens=None,
                   row_cap=float("inf"), block_cap=float("inf"), token_cap=float("inf")):
    n = len(e)
    rows = rows if rows is not None else [1] * n
    blocks = blocks if blocks is not None else [0] * n
    tokens = tokens if tokens is not None else [0] * n
    caps = (rows, blocks, tokens, row_cap, block_cap, token_cap)
    # line 1
    cand = [r for r in range(n) if (eligible is None or eligible[r]) and fits([r], *caps)]
    # line 2
    cand.sort(key=lambda r: rank_key(r, a_w, e, k, g_s, delta_s))
    # line 3
    front = cand[:max(b_max, 0)]
    # lines 4-8
    batch = []
    for r in front:
        if admissible(batch + [r], a_w, e, k, g_s, delta_s, b_max, *caps):
            batch.append(r)
    return batch, (start_time(batch, a_w, e, k) if batch else a_w)
