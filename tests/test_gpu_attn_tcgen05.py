"""GPU parity of the tcgen05 / TMEM / TMA attention kernel (NSD_FLAG_ATTN_TCGEN05 selects it for
every shape it supports), against the same oracle and tolerance as the default kernel."""
import numpy as np
import pytest

import workload as W
import nsd_testlib
import test_gpu_verify_attn as base
import test_gpu_round as rnd

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _tcgen05_path(monkeypatch):
    monkeypatch.setattr(nsd_testlib, "CONTEXT_FLAGS", 1 << 1)


@pytest.mark.parametrize("gamma", [1, 4, 6, 8, 11, 15])
def test_row_counts_32_48_64(gamma):
    """R = 32, 48 and 64 query-row columns; lengths around block, tile (128 keys) and chunk edges."""
    cfg = base._cfg(f"u{gamma}", batch=11, gamma=gamma, ctx=("fixed", [0, 1, 15, 16, 111, 127, 128, 129, 300, 517, 1100]), seed=160 + gamma)
    _, _, o, lse, res = base._run(cfg, want_lse=True)
    base._check(o, res, lse)


@pytest.mark.parametrize("chunk_blocks", [2, 6, 10, 16, 0])
def test_split_kv_with_chunks_that_are_not_whole_tiles(chunk_blocks):
    """Chunks of 2..16 blocks against 8-block tiles: keys past a chunk are zero-filled boxes and must be masked."""
    cfg = base._cfg("usplit", batch=8, gamma=4, ctx=("fixed", [5, 40, 100, 257, 380, 600, 1023, 1500]), seed=172)
    _, _, o, lse, res = base._run(cfg, chunk_blocks=chunk_blocks, want_lse=True)
    base._check(o, res, lse)


def test_many_units_per_cta_and_layers():
    """More (item, head) units than SMs, so the persistent CTAs walk several units each, over aliased slabs."""
    cfg = base._cfg("umany", batch=48, gamma=4, ctx=("uniform", 1, 700), layers=3, seed=173)
    _, _, o, _, res = base._run(cfg, slabs=2, chunk_blocks=8)
    base._check(o, res)


@pytest.mark.parametrize("chunk_blocks", [24, 40, 0])
def test_many_units_of_several_tiles_per_cta(chunk_blocks):
    """Units of three, five and more 128-key tiles, about ten units per persistent CTA: the tile streams change
    parity from unit to unit, and the unit that a stream writes out changes with them."""
    cfg = base._cfg("ulong", batch=40, gamma=8, ctx=("uniform", 500, 2600), seed=175)
    _, _, o, lse, res = base._run(cfg, chunk_blocks=chunk_blocks, want_lse=True)
    base._check(o, res, lse)


@pytest.mark.parametrize("gamma", [4, 8, 15])
def test_running_maximum_moves_late_and_often(gamma):
    base.test_running_maximum_moves_late_and_often(gamma)


def test_fused_round_and_poisoned_tail_slots():
    rnd._run_round(rnd.MULTI, 2)
    rnd._run_round(rnd.ALLMIG, 3)


def test_group_size_one_and_eight():
    for hq, hkv in ((8, 8), (8, 1)):
        cfg = base._cfg(f"ug{hq}_{hkv}", batch=5, gamma=4, ctx=("uniform", 1, 400), hq=hq, hkv=hkv, d=128, seed=174)
        _, _, o, _, res = base._run(cfg)
        base._check(o, res)
