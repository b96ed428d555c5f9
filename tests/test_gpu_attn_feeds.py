"""The mma.sync attention kernel has two ways of fetching K/V tiles: tensor copies (the default where
the shape is bound by HBM) and cp.async (NSD_FLAG_ATTN_CP_ASYNC, and always for the shapes with five or six
row tiles, head_dim 64, gather-through and the allocation-free entry).  Both must match the oracle, and
each other bit for bit: the feed changes where a tile sits in shared memory, not one operation on it."""
import numpy as np
import pytest

import nsd_testlib
import test_gpu_verify_attn as base

pytestmark = pytest.mark.gpu


def _both(monkeypatch, cfg, **kw):
    outs = {}
    for feed in ("tma", "mma"):
        # the tensor-copy feed is the default; neither run may take the tcgen05 engine
        monkeypatch.setattr(nsd_testlib, "CONTEXT_FLAGS", (1 << 2) | ((1 << 0) if feed == "mma" else 0))
        _, _, o, lse, res = base._run(cfg, want_lse=True, **kw)
        base._check(o, res, lse)
        outs[feed] = (o, lse)
    assert np.array_equal(outs["tma"][0], outs["mma"][0])
    assert np.array_equal(outs["tma"][1], outs["mma"][1])


@pytest.mark.parametrize("gamma", [1, 3, 4, 5, 6, 7])
def test_feeds_agree_up_to_four_row_tiles(monkeypatch, gamma):
    """1..4 row tiles (one warp, or two warps of two): lengths around block edges, poisoned tail slots."""
    cfg = base._cfg(f"feed{gamma}", batch=10, gamma=gamma, ctx=("fixed", [0, 1, 15, 16, 17, 31, 33, 200, 517, 1030]), seed=300 + gamma)
    _both(monkeypatch, cfg)


def test_feeds_agree_with_split_kv_and_layers(monkeypatch):
    cfg = base._cfg("feedsplit", batch=12, gamma=4, ctx=("uniform", 1, 900), layers=3, seed=311)
    _both(monkeypatch, cfg, slabs=2, chunk_blocks=6)
