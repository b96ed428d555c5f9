"""Seeded input generators for the target-side verification round.

Every draw comes from a Philox stream keyed by (config seed, purpose, layer),
so any piece can be regenerated alone (one layer slab, one request's rows)
without generating what comes before it.

Recipe (stand-ins for the paper's workload, which uses no public dataset: its
requests "arrive simultaneously" with unspecified prompts, Section 6):

* context lengths: uniform integers or a clipped lognormal;
* `round(frac_reassigned * batch)` requests, picked by a seeded shuffle, are
  "reassigned": their committed KV sits in pool region A (block ids below
  `region_b_begin`) and must be copied into the blocks their table names in
  region B; everybody else already lives in region B (the paper's two banks
  with separate block ranges, Appendix E.2);
* region B is `pool_factor` times the live blocks, and the live block ids are a
  random sample of it, so tables are scattered over the region;
* K, V, Q entries are N(0,1) rounded to bf16; unused blocks, destination
  blocks and the tail slots of a request's last block hold a bf16 NaN;
* probabilities: target row p = softmax(z), z ~ N(0, logit_var); draft row
  q = softmax(z + N(0, noise_var)) (or an independent softmax when
  `noise_var` is None); draft tokens are drawn from q; uniforms are fp32
  multiples of 2^-24 in [0, 1).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional, Tuple

import numpy as np

BF16_NAN = np.uint16(0x7FFF)

_PURPOSE = {
    "ctx": 1, "mig": 2, "blocks_b": 3, "blocks_a": 4, "pool": 5, "new_kv": 6,
    "q": 7, "logits": 8, "noise": 9, "draft": 10, "u_acc": 11, "u_smp": 12,
}


def _rng(seed: int, purpose: str, index: int = 0) -> np.random.Generator:
    key = np.array([np.uint64(seed), np.uint64(_PURPOSE[purpose] * 1_000_003 + index)], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


# --------------------------------------------------------------------------- bf16 helpers
def f32_to_bf16(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern (uint16), round to nearest even; NaN stays NaN."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounded = ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        rounded = np.where(nan, BF16_NAN, rounded)
    return rounded


def bf16_to_f32(u: np.ndarray) -> np.ndarray:
    """bf16 bit pattern (uint16) -> float32, exact."""
    return (np.ascontiguousarray(u, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


_NORMAL_TABLE: Optional[np.ndarray] = None


def _normal_table() -> np.ndarray:
    """65536 equiprobable N(0,1) quantiles, rounded to bf16: an index drawn
    uniformly from it is a bf16 normal sample, at table-lookup cost."""
    global _NORMAL_TABLE
    if _NORMAL_TABLE is None:
        from scipy.special import ndtri

        qs = ndtri((np.arange(65536, dtype=np.float64) + 0.5) / 65536.0)
        _NORMAL_TABLE = f32_to_bf16(qs.astype(np.float32))
    return _NORMAL_TABLE


def _normal_bf16(rng: np.random.Generator, shape) -> np.ndarray:
    n = int(np.prod(shape))
    idx = rng.integers(0, 65536, size=n, dtype=np.uint16)
    return _normal_table()[idx].reshape(shape)


# --------------------------------------------------------------------------- configs
@dataclass(frozen=True)
class RoundConfig:
    name: str
    batch: int
    gamma: int
    num_layers: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    block_size: int
    vocab: int
    ctx_dist: Tuple
    frac_reassigned: float
    pool_factor: float = 1.5
    logit_var: float = 2.0
    noise_var: Optional[float] = 0.5
    seed: int = 20260929

    @property
    def rows(self) -> int:
        return self.batch * (self.gamma + 1)

    @property
    def block_elems(self) -> int:
        """bf16 elements of one (layer, block): K and V, every kv head."""
        return 2 * self.num_kv_heads * self.block_size * self.head_dim


_QWEN = dict(num_q_heads=32, num_kv_heads=8, head_dim=128, block_size=16, vocab=151936)

CONFIGS = {
    # the five configurations of the benchmark set, in order
    "tiny": RoundConfig("tiny", batch=4, gamma=4, num_layers=1, num_q_heads=8, num_kv_heads=2, head_dim=64,
                        block_size=16, vocab=1000, ctx_dist=("uniform", 17, 100), frac_reassigned=0.25,
                        noise_var=None, seed=20260929),
    "qwen3_b64": RoundConfig("qwen3_b64", batch=64, gamma=4, num_layers=1, ctx_dist=("uniform", 512, 2048),
                             frac_reassigned=0.25, seed=20260930, **_QWEN),
    "knee_b512": RoundConfig("knee_b512", batch=512, gamma=4, num_layers=36,
                             ctx_dist=("lognormal", 1024, 0.7, 128, 4096), frac_reassigned=0.25,
                             seed=20260931, **_QWEN),
    "migration_b256": RoundConfig("migration_b256", batch=256, gamma=6, num_layers=36,
                                  ctx_dist=("uniform", 1024, 8192), frac_reassigned=0.75,
                                  seed=20260932, **_QWEN),
    "long_b128": RoundConfig("long_b128", batch=128, gamma=8, num_layers=36,
                             ctx_dist=("uniform", 8192, 32768), frac_reassigned=0.25, noise_var=1.0,
                             seed=20260933, **_QWEN),
}


# --------------------------------------------------------------------------- batch structure
@dataclass
class BatchMeta:
    ctx_len: np.ndarray        # int32 [B]   committed KV entries before the round
    is_migrated: np.ndarray    # uint8 [B]
    kv_indptr: np.ndarray      # int64 [B+1]
    kv_indices: np.ndarray     # int32 [sum ceil((ctx+gamma+1)/bs)]  region-B block ids
    mig_req: np.ndarray        # int32 [n_mig]  request index of each reassigned request
    mig_indptr: np.ndarray     # int64 [n_mig+1]
    mig_src: np.ndarray        # int32 [sum ceil(ctx/bs)]  region-A block ids
    mig_dst: np.ndarray        # int32 same length         region-B block ids (prefix of the request's table)
    num_blocks: int
    region_b_begin: int
    home_blocks: np.ndarray = field(default=None)   # int32: block holding logical block j of request r (src if migrated)
    home_indptr: np.ndarray = field(default=None)   # int64 [B+1] over ceil(ctx/bs)

    @property
    def n_mig(self) -> int:
        return int(self.mig_req.shape[0])


def _draw_ctx(cfg: RoundConfig) -> np.ndarray:
    rng = _rng(cfg.seed, "ctx")
    d = cfg.ctx_dist
    if d[0] == "uniform":
        return rng.integers(d[1], d[2] + 1, size=cfg.batch).astype(np.int32)
    if d[0] == "lognormal":
        _, median, sigma, lo, hi = d
        x = np.exp(np.log(median) + sigma * rng.standard_normal(cfg.batch))
        return np.clip(np.rint(x), lo, hi).astype(np.int32)
    if d[0] == "fixed":
        return np.asarray(d[1], dtype=np.int32).copy()
    raise ValueError(d)


def draw_ctx_len(cfg: RoundConfig) -> np.ndarray:
    """Context lengths of `cfg.batch` requests from the configuration's distribution (int32)."""
    return _draw_ctx(cfg)


def make_batch_meta(cfg: RoundConfig) -> BatchMeta:
    B, bs, g1 = cfg.batch, cfg.block_size, cfg.gamma + 1
    ctx = _draw_ctx(cfg)
    assert ctx.shape[0] == B
    n_mig = int(round(cfg.frac_reassigned * B))
    order = _rng(cfg.seed, "mig").permutation(B)
    mig_req = np.sort(order[:n_mig]).astype(np.int32)
    is_mig = np.zeros(B, dtype=np.uint8)
    is_mig[mig_req] = 1

    nblk = (ctx.astype(np.int64) + g1 + bs - 1) // bs          # table length: room for the appended tokens
    nsrc = (ctx.astype(np.int64) + bs - 1) // bs               # blocks that hold committed KV
    kv_indptr = np.zeros(B + 1, dtype=np.int64)
    np.cumsum(nblk, out=kv_indptr[1:])
    total_live = int(kv_indptr[-1])
    total_src = int(nsrc[mig_req].sum())

    nb_a = total_src
    nb_b = int(np.ceil(cfg.pool_factor * total_live))
    ids_b = _rng(cfg.seed, "blocks_b").permutation(nb_b)[:total_live].astype(np.int32) + np.int32(nb_a)
    ids_a = _rng(cfg.seed, "blocks_a").permutation(nb_a).astype(np.int32)

    mig_indptr = np.zeros(n_mig + 1, dtype=np.int64)
    np.cumsum(nsrc[mig_req], out=mig_indptr[1:])
    mig_src = ids_a
    mig_dst = np.empty(total_src, dtype=np.int32)
    for m, r in enumerate(mig_req):
        n = int(nsrc[r])
        mig_dst[mig_indptr[m]:mig_indptr[m] + n] = ids_b[kv_indptr[r]:kv_indptr[r] + n]

    home_indptr = np.zeros(B + 1, dtype=np.int64)
    np.cumsum(nsrc, out=home_indptr[1:])
    home = np.empty(int(home_indptr[-1]), dtype=np.int32)
    mpos = {int(r): m for m, r in enumerate(mig_req)}
    for r in range(B):
        n = int(nsrc[r])
        if r in mpos:
            m = mpos[r]
            home[home_indptr[r]:home_indptr[r] + n] = mig_src[mig_indptr[m]:mig_indptr[m] + n]
        else:
            home[home_indptr[r]:home_indptr[r] + n] = ids_b[kv_indptr[r]:kv_indptr[r] + n]

    return BatchMeta(ctx_len=ctx, is_migrated=is_mig, kv_indptr=kv_indptr, kv_indices=ids_b,
                     mig_req=mig_req, mig_indptr=mig_indptr, mig_src=mig_src, mig_dst=mig_dst,
                     num_blocks=nb_a + nb_b, region_b_begin=nb_a, home_blocks=home, home_indptr=home_indptr)


# --------------------------------------------------------------------------- per-layer tensors
def pool_layer_chunks(cfg: RoundConfig, meta: BatchMeta, layer: int, poison: bool = True, step: int = 1024):
    """The committed KV of one layer slab, streamed: yields (b0, b1, data) where `data`
    (uint16 [b1-b0][2][num_kv_heads][block_size][head_dim]) is the content of home blocks
    `meta.home_blocks[b0:b1]`, tail slots of a request's last block already filled.  The
    draws are those of `pool_layer` (one stream, `step` home blocks per draw), so a slab far
    larger than host memory can be produced -- or re-read -- piece by piece."""
    Hkv, bs, D = cfg.num_kv_heads, cfg.block_size, cfg.head_dim
    fill = BF16_NAN if poison else np.uint16(0)
    n_home = int(meta.home_indptr[-1])
    rng = _rng(cfg.seed, "pool", layer)
    tail = meta.ctx_len.astype(np.int64) % bs
    last_of = meta.home_indptr[1:] - 1                 # home index of each request's last block
    tailed = np.nonzero(tail)[0]
    assert step == 1024, "the draw size is part of the recipe: it fixes the stream"
    for b0 in range(0, n_home, step):
        b1 = min(n_home, b0 + step)
        data = _normal_bf16(rng, (b1 - b0, 2, Hkv, bs, D))
        for r in tailed[(last_of[tailed] >= b0) & (last_of[tailed] < b1)]:
            data[int(last_of[r]) - b0, :, :, int(tail[r]):, :] = fill
        yield b0, b1, data


def pool_layer(cfg: RoundConfig, meta: BatchMeta, layer: int, poison: bool = True) -> np.ndarray:
    """One layer slab of the paged pool before the round, bf16 bits as uint16,
    shape [num_blocks][2 (K,V)][num_kv_heads][block_size][head_dim].

    Committed KV of request r sits in its home blocks (region A if reassigned,
    else its own table).  With `poison`, everything else -- unused blocks, the
    destination blocks of reassigned requests, the slots past `ctx` in a last
    block -- is a bf16 NaN; without it those bytes are zero.
    """
    Hkv, bs, D = cfg.num_kv_heads, cfg.block_size, cfg.head_dim
    fill = BF16_NAN if poison else np.uint16(0)
    pool = np.full((meta.num_blocks, 2, Hkv, bs, D), fill, dtype=np.uint16)
    for b0, b1, data in pool_layer_chunks(cfg, meta, layer, poison):
        pool[meta.home_blocks[b0:b1]] = data
    return pool


def export_tables(cfg: RoundConfig, meta: BatchMeta):
    """Block table of the export copy (the other region) for the suffix commit: same
    indexing as `kv_indices` (entry j covers positions 16j..16j+15), but only the
    entries that can hold this round's tokens (positions ctx..ctx+gamma) name a block,
    drawn from the free blocks of region B; the persistent prefix is -1."""
    bs = cfg.block_size
    used = np.zeros(meta.num_blocks, dtype=bool)
    used[meta.kv_indices] = True
    used[:meta.region_b_begin] = True
    free = np.nonzero(~used)[0].astype(np.int32)
    free = free[_rng(cfg.seed, "blocks_a", 7).permutation(len(free))]
    exp = np.full(len(meta.kv_indices), -1, dtype=np.int32)
    need = int(((meta.ctx_len.astype(np.int64) + cfg.gamma) // bs - meta.ctx_len.astype(np.int64) // bs + 1).sum())
    if need > len(free):
        raise ValueError(f"export table needs {need} free region-B blocks, the pool has {len(free)} (raise pool_factor)")
    nxt = 0
    for r in range(cfg.batch):
        ctx = int(meta.ctx_len[r])
        for j in range(ctx // bs, (ctx + cfg.gamma) // bs + 1):
            exp[meta.kv_indptr[r] + j] = free[nxt]
            nxt += 1
    return meta.kv_indptr.copy(), exp


def new_kv(cfg: RoundConfig, meta: BatchMeta, layer: int):
    """K and V of the gamma+1 tokens each request verifies this round
    (anchor + drafts), bf16 bits, each [batch*(gamma+1)][num_kv_heads][head_dim]."""
    rng = _rng(cfg.seed, "new_kv", layer)
    shape = (cfg.rows, cfg.num_kv_heads, cfg.head_dim)
    return _normal_bf16(rng, shape), _normal_bf16(rng, shape)


def queries(cfg: RoundConfig, meta: BatchMeta, layer: int) -> np.ndarray:
    """Query rows, bf16 bits, [batch*(gamma+1)][num_q_heads][head_dim]."""
    return _normal_bf16(_rng(cfg.seed, "q", layer), (cfg.rows, cfg.num_q_heads, cfg.head_dim))


# --------------------------------------------------------------------------- acceptance inputs
def _softmax_rows(z: np.ndarray) -> np.ndarray:
    z = z - z.max(axis=-1, keepdims=True)
    e = np.exp(z, dtype=np.float32)
    s = e.sum(axis=-1, keepdims=True, dtype=np.float64)
    return (e / s.astype(np.float32)).astype(np.float32)


def uniforms(rng: np.random.Generator, shape) -> np.ndarray:
    """fp32 uniforms on the 2^-24 grid in [0, 1)."""
    return (rng.integers(0, 1 << 24, size=shape, dtype=np.int64).astype(np.float32) / np.float32(1 << 24)).astype(np.float32)


def accept_inputs(cfg: RoundConfig, batch: Optional[int] = None, chunk: int = 16):
    """Target rows p [B][gamma+1][V], draft rows q [B][gamma][V] (fp32), draft
    tokens [B][gamma] drawn from q, accept uniforms [B][gamma], one sampling
    uniform per request [B]."""
    B = cfg.batch if batch is None else batch
    g, V = cfg.gamma, cfg.vocab
    p = np.empty((B, g + 1, V), dtype=np.float32)
    q = np.empty((B, g, V), dtype=np.float32)
    tok = np.empty((B, g), dtype=np.int32)
    sd = np.float32(np.sqrt(cfg.logit_var))
    for b0 in range(0, B, chunk):
        b1 = min(B, b0 + chunk)
        idx = b0 // chunk
        z = _rng(cfg.seed, "logits", idx).standard_normal((b1 - b0, g + 1, V), dtype=np.float32) * sd
        p[b0:b1] = _softmax_rows(z)
        nz = _rng(cfg.seed, "noise", idx).standard_normal((b1 - b0, g, V), dtype=np.float32)
        if cfg.noise_var is None:
            zq = nz * sd
        else:
            zq = z[:, :g, :] + nz * np.float32(np.sqrt(cfg.noise_var))
        q[b0:b1] = _softmax_rows(zq)
        ud = _rng(cfg.seed, "draft", idx).random((b1 - b0, g))
        cdf = np.cumsum(q[b0:b1], axis=-1, dtype=np.float64)
        for i in range(b1 - b0):
            for j in range(g):
                c = cdf[i, j]
                tok[b0 + i, j] = min(int(np.searchsorted(c, ud[i, j] * c[-1], side="right")), V - 1)
    u_acc = uniforms(_rng(cfg.seed, "u_acc"), (B, g))
    u_smp = uniforms(_rng(cfg.seed, "u_smp"), (B,))
    return p, q, tok, u_acc, u_smp


# --------------------------------------------------------------------------- per-request draft depth
def draw_gamma_r(cfg: RoundConfig, lo: int = 0) -> np.ndarray:
    """Per-request draft depth in [lo, cfg.gamma] (int32 [batch]): a batch that mixes depths, as when requests come from
    draft workers run at different depths."""
    return _rng(cfg.seed, "ctx", 99).integers(lo, cfg.gamma + 1, size=cfg.batch).astype(np.int32)


def ragged_index(gamma_r: np.ndarray, gamma: int):
    """Indices that cut padded per-request tensors down to their ragged form: `rows` picks entries (r, i <= gamma_r[r]) out
    of [batch*(gamma+1)] target rows, `drafts` picks (r, i < gamma_r[r]) out of [batch*gamma] draft rows; `row_indptr`
    (int64 [batch+1]) is the prefix of gamma_r + 1."""
    B = len(gamma_r)
    rows = np.concatenate([r * (gamma + 1) + np.arange(gamma_r[r] + 1) for r in range(B)]).astype(np.int64)
    drafts = np.concatenate([r * gamma + np.arange(gamma_r[r]) for r in range(B)] + [np.zeros(0, np.int64)]).astype(np.int64)
    row_indptr = np.zeros(B + 1, dtype=np.int64)
    np.cumsum(gamma_r.astype(np.int64) + 1, out=row_indptr[1:])
    return rows, drafts, row_indptr
