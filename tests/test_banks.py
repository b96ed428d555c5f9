"""Host bookkeeping of the two-bank worker used by the scheduled-rounds driver and its test."""
import numpy as np
import pytest

from paper_2609_29364_b200.banks import BankedPool


def _pool():
    ctx = np.array([5, 40, 100, 17, 64], dtype=np.int32)
    return ctx, BankedPool(ctx, gamma=3, block_size=16, max_new_tokens=24, bank_blocks=30, seed=3)


def test_store_tables_are_disjoint_and_inside_region_a():
    ctx, b = _pool()
    seen = set()
    for r in range(len(ctx)):
        t = b.store_table(r, b.blocks_needed(ctx[r] + 24))
        assert all(0 <= x < b.region_b_begin for x in t)
        assert not (seen & set(t.tolist()))
        seen |= set(t.tolist())


def test_enter_allocates_copies_and_remembers_residents():
    ctx, b = _pool()
    e = b.enter(0, [0, 2], ctx)
    lo, hi = b.region_b_begin, b.region_b_begin + 30
    assert e.resident.tolist() == [0, 0]
    assert all(lo <= x < hi for x in e.kv_indices)                       # bank 0 range only
    assert len(set(e.kv_indices.tolist())) == len(e.kv_indices)          # nobody shares a block
    assert e.kv_indptr.tolist() == [0, b.blocks_needed(5), b.blocks_needed(5) + b.blocks_needed(100)]
    assert len(e.mig_src) == 1 + 7 and np.array_equal(e.mig_dst, np.concatenate([e.kv_indices[:1], e.kv_indices[1:8]]))
    assert np.array_equal(e.mig_src, np.concatenate([b.store_table(0, 1), b.store_table(2, 7)]))
    # the other bank is untouched by bank 0's occupants and uses its own range
    e1 = b.enter(1, [1], ctx)
    assert all(hi <= x < hi + 30 for x in e1.kv_indices)
    # request 2 comes back to bank 0 (grown by 20 tokens): resident, keeps its blocks, gets more; request 0 left
    ctx2 = ctx.copy()
    ctx2[2] += 20
    old = e.kv_indices[1:].tolist()
    e2 = b.enter(0, [2, 3], ctx2)
    assert e2.resident.tolist() == [1, 0]
    assert e2.kv_indices[:len(old)].tolist() == old and b.blocks_needed(120) == len(old) + 1
    assert len(e2.mig_src) == 2                                           # only request 3's two context blocks are copied
    assert 0 not in b.held[0] and len(b.free[0]) + sum(len(v) for v in b.held[0].values()) == 30


def test_out_of_blocks_is_an_error():
    ctx, b = _pool()
    with pytest.raises(ValueError):
        BankedPool(ctx, 3, 16, 24, bank_blocks=3).enter(0, [2], ctx)
