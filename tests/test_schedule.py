"""Algorithm 1 (worker-triggered batch reconstruction): the Python oracle against a
hand-worked instance, Eq. (8) invariants and greedy maximality; the library's host
routine against the oracle on random pools.  No GPU involved."""
import os

import numpy as np
import pytest

from oracle import schedule as osch

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "schedule_worked.txt")


def _golden():
    vals = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        tk = line.split()
        vals[tk[0]] = tk[1:]
    hdr = vals["a_w"]
    prm = dict(a_w=float(hdr[0]), g_s=float(hdr[2]), delta_s=float(hdr[4]), b_max=int(hdr[6]))
    return prm, [float(x) for x in vals["e"]], [float(x) for x in vals["k"]], [int(x) for x in vals["batch"]], float(vals["start"][0])


def test_oracle_reproduces_the_hand_worked_instance():
    prm, e, k, want_batch, want_start = _golden()
    batch, start = osch.schedule_batch(prm["a_w"], prm["g_s"], prm["delta_s"], prm["b_max"], e, k)
    assert batch == want_batch and start == pytest.approx(want_start)


def _random_pool(rng, n):
    e = (1.0 + rng.normal(0, 0.08, n)).round(3)
    k = (e + rng.normal(0.02, 0.06, n)).round(3)
    rows = np.ones(n, dtype=np.int32)
    blocks = rng.integers(4, 200, n).astype(np.int32)
    tokens = (blocks * 16 - rng.integers(0, 16, n)).astype(np.int32)
    eligible = (rng.random(n) < 0.85).astype(np.uint8)
    return e, k, rows, blocks, tokens, eligible


@pytest.mark.parametrize("seed", range(6))
def test_oracle_batches_are_admissible_and_greedily_maximal(seed):
    rng = np.random.default_rng(seed)
    n = 40
    e, k, rows, blocks, tokens, eligible = _random_pool(rng, n)
    a_w, g_s, delta_s, b_max = 1.0, 0.13, 0.03, 12
    caps = dict(row_cap=10, block_cap=900, token_cap=12000)
    batch, start = osch.schedule_batch(a_w, g_s, delta_s, b_max, e, k, eligible, rows, blocks, tokens, **caps)
    args = (a_w, e, k, g_s, delta_s, b_max, rows, blocks, tokens, caps["row_cap"], caps["block_cap"], caps["token_cap"])
    assert len(set(batch)) == len(batch) and all(eligible[r] for r in batch)
    if batch:
        assert osch.admissible(batch, *args)                              # Eq. (8) holds for the result
        assert start == osch.start_time(batch, a_w, e, k)
        for r in batch:                                                   # nobody waits past its own bound
            assert start <= osch.admission_bound(r, a_w, e, k, g_s, delta_s) + 1e-12
    ranked = sorted((r for r in range(n) if eligible[r]), key=lambda r: osch.rank_key(r, a_w, e, k, g_s, delta_s))[:b_max]
    so_far = []
    for r in ranked:                                                      # every skipped candidate really was inadmissible
        if r in batch:
            so_far.append(r)
        else:
            assert not osch.admissible(so_far + [r], *args)


def test_slack_and_interval_only_ever_enlarge_the_batch_front():
    """With unlimited capacity, a larger slack cannot make the first-ranked request inadmissible,
    and zero slack with simultaneous readiness admits everybody up to B_max."""
    e = [1.0] * 6
    k = [1.0] * 6
    batch, start = osch.schedule_batch(1.0, 0.0, 0.0, 4, e, k)
    assert batch == [0, 1, 2, 3] and start == 1.0
    batch, _ = osch.schedule_batch(1.0, 0.0, 0.0, 4, [1.0, 1.0, 1.5], [1.0, 1.0, 1.5])
    assert batch == [0, 1]                                                # waiting for r=2 would delay 0 and 1 by 0.5 s
    batch, _ = osch.schedule_batch(1.0, 0.0, 0.6, 4, [1.0, 1.0, 1.5], [1.0, 1.0, 1.5])
    assert batch == [0, 1, 2]                                             # a slack of 0.6 s allows it


@pytest.mark.parametrize("seed", range(8))
def test_library_matches_the_oracle(seed):
    import paper_2609_29364_b200 as nsd

    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(1, 300))
    e, k, rows, blocks, tokens, eligible = _random_pool(rng, n)
    a_w, g_s, delta_s = 1.0 + float(rng.normal(0, 0.05)), float(rng.choice([0.0, 0.13, 0.16])), float(rng.choice([0.0, 0.03]))
    b_max = int(rng.choice([1, 8, 32, 128]))
    caps = dict(row_capacity=int(rng.choice([4, 32, 1000])), block_capacity=int(rng.choice([300, 3000, 10 ** 9])),
                token_limit=int(rng.choice([4000, 40000, 10 ** 9])))
    got, got_start = nsd.nsd_schedule_batch(worker_avail=a_w, target_interval=g_s, slack=delta_s, max_batch=b_max,
                                            pred_done=e, kv_ready=k, eligible=eligible, rows=rows, blocks=blocks,
                                            tokens=tokens, **caps)
    want, want_start = osch.schedule_batch(a_w, g_s, delta_s, b_max, e.tolist(), k.tolist(), eligible.tolist(),
                                           rows.tolist(), blocks.tolist(), tokens.tolist(), caps["row_capacity"],
                                           caps["block_capacity"], caps["token_limit"])
    assert got == want and got_start == want_start


def test_library_golden_and_edge_cases():
    import paper_2609_29364_b200 as nsd

    prm, e, k, want_batch, want_start = _golden()
    got, start = nsd.nsd_schedule_batch(worker_avail=prm["a_w"], target_interval=prm["g_s"], slack=prm["delta_s"],
                                        max_batch=prm["b_max"], pred_done=e, kv_ready=k)
    assert got == want_batch and start == pytest.approx(want_start)
    assert nsd.nsd_schedule_batch(worker_avail=2.0, target_interval=0.1, slack=0.0, max_batch=4, pred_done=[], kv_ready=[]) == ([], 2.0)
    got, _ = nsd.nsd_schedule_batch(worker_avail=1.0, target_interval=0.1, slack=0.0, max_batch=4, pred_done=[1.0, 1.0],
                                    kv_ready=[1.0, 1.0], eligible=[0, 0])
    assert got == []
    got, _ = nsd.nsd_schedule_batch(worker_avail=1.0, target_interval=0.1, slack=0.0, max_batch=4, pred_done=[1.0, 1.0],
                                    kv_ready=[1.0, 1.0], blocks=[50, 5], block_capacity=10)
    assert got == [1]                                                     # request 0 does not fit the worker alone
    with pytest.raises(nsd.NsdError):
        nsd.nsd_schedule_batch(worker_avail=1.0, target_interval=-1.0, slack=0.0, max_batch=4, pred_done=[1.0], kv_ready=[1.0])
