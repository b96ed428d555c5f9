#!/usr/bin/env python
"""Benchmark of the B200 verification round (metric: verify-round req/s and
tokens/s at the Qwen3-8B shape, HBM GB/s against the B200 peak).

One step = one whole verification round through the C ABI on one batch of
synthetic input: for each of the 36 logical layers the KV-state preparation
(block gather of the reassigned requests + append of the gamma+1 new tokens),
the ragged paged GQA attention, and finally the speculative acceptance.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload knee_b512]
    python bench.py --impl reference ...      # the CPU oracle, on host cores

Prints ONE JSON line (rank 0).  N > 1 (under torchrun) runs one independent
batch per GPU -- the path has no exchange step -- and reports the aggregate.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workload as W  # noqa: E402

NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per algorithmic byte of verify_attn_kernel, from a
# profiler capture of a smaller case of the same kernel (709.4 MB over 698.9 MB for one whole-batch pass); the
# full-size launch is too large to capture under the profiler, and traffic grows with the keys streamed.
ATTN_TRAFFIC_PER_ALGORITHMIC_BYTE = 1.015
# The same for verify_attn_umma_kernel, the engine the library picks from 33 stacked query rows per kv head on
# (2058 MB over 2036 MB for one whole-batch pass of a small long-context case; its merge kernel is timed with it).
UMMA_TRAFFIC_PER_ALGORITHMIC_BYTE = 1.011


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="knee_b512", choices=list(W.CONFIGS))
    ap.add_argument("--slabs", type=int, default=0, help="physical layer slabs (0 = as many as fit in 80%% of free memory)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-scheduled", action="store_true", help="skip the scheduler-driven two-bank rounds leg")
    ap.add_argument("--scheduled-rounds", type=int, default=8)
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="target CPU time of the oracle sample")
    ap.add_argument("--ctx-flags", type=int, default=0, help="comparison runs only: nsd_config.flags of the context (not a bench line)")
    ap.add_argument("--batch", type=int, default=0, help="profiling only: override the batch size (not a bench line)")
    ap.add_argument("--layers", type=int, default=0, help="profiling only: override the layer count (not a bench line)")
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


# ----------------------------------------------------------------------------- algorithmic bytes
def algorithmic_bytes(cfg: W.RoundConfig, meta: W.BatchMeta, acc_len=None):
    """Bytes the method itself must move (per layer unless noted): every KV byte of
    every visible key once, Q read and O written once, each gathered block read
    and written once, each appended row read and written once, and for the
    acceptance the one vocabulary row (pair) the draw needs."""
    kv_tok = 2 * cfg.num_kv_heads * cfg.head_dim * 2
    block_bytes = kv_tok * cfg.block_size
    keys = int((meta.ctx_len.astype(np.int64) + cfg.gamma + 1).sum())
    attn = keys * kv_tok + cfg.rows * cfg.num_q_heads * cfg.head_dim * 2 * 2
    gather = int(len(meta.mig_src)) * block_bytes * 2
    append = cfg.rows * kv_tok * 2
    if acc_len is None:
        accept = cfg.batch * cfg.vocab * 4 * 2
    else:
        accept = int(((acc_len < cfg.gamma) + 1).sum()) * cfg.vocab * 4
    accept += 12 * cfg.batch * cfg.gamma
    per_round = cfg.num_layers * (attn + gather + append) + accept
    return dict(attn_per_layer=attn, gather_per_layer=gather, append_per_layer=append, accept=accept, round=per_round)


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.gpu_id = gpu_id
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(prefix="nsd_clocks_", suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", self.gpu_id, f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        os.unlink(self.path)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), power_w_max=float(max(pw)),
                       reasons=sorted(reasons), samples=len(sm))
        return out


# ----------------------------------------------------------------------------- oracle arm
def oracle_sample(cfg, meta, host, target_seconds):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload and
    extrapolates to one whole round.  Returns (seconds per round, description, cores)."""
    import oracle

    cores = oracle.hardware_threads()
    L, B = cfg.num_layers, cfg.batch
    pool = host["pool_slab"][None].copy()
    t0 = time.perf_counter()
    oracle.kv_prepare(pool, meta.mig_indptr, meta.mig_src, meta.mig_dst, meta.ctx_len, meta.kv_indptr, meta.kv_indices,
                      host["k_new"][:1], host["v_new"][:1], cfg.gamma, layer_begin=0, layer_count=1)
    t_prep = time.perf_counter() - t0
    order = np.random.default_rng(cfg.seed).permutation(B).astype(np.int32)
    n_probe = min(B, cores)
    t0 = time.perf_counter()
    oracle.verify_attn(pool, host["q"][0], meta.ctx_len, meta.kv_indptr, meta.kv_indices, cfg.gamma, layer=0,
                       req_list=np.ascontiguousarray(order[:n_probe]))
    t_probe = time.perf_counter() - t0
    # spend about target_seconds: first more requests of layer 0, then further layers' query rows
    want = n_probe * max(target_seconds, t_probe) / max(t_probe, 1e-3)           # request-layers affordable
    n_attn = int(min(B, max(n_probe, want)))
    sel = np.ascontiguousarray(order[:n_attn])
    keys_all = float((meta.ctx_len.astype(np.int64) + cfg.gamma + 1).sum())
    keys_sel = float((meta.ctx_len[sel].astype(np.int64) + cfg.gamma + 1).sum())
    n_layers = 0
    t0 = time.perf_counter()
    while n_layers < L and (n_layers == 0 or time.perf_counter() - t0 < target_seconds):
        oracle.verify_attn(pool, host["q"][n_layers], meta.ctx_len, meta.kv_indptr, meta.kv_indices, cfg.gamma, layer=0, req_list=sel)
        n_layers += 1
    t_attn = time.perf_counter() - t0
    t_attn_layer = t_attn / n_layers * keys_all / keys_sel   # attention cost is proportional to visible keys
    t0 = time.perf_counter()
    oracle.spec_accept(host["p"], host["q_draft"], host["draft_tok"], host["u_acc"], host["u_smp"], meta.ctx_len)
    t_acc = time.perf_counter() - t0
    t_round = L * (t_prep + t_attn_layer) + t_acc
    desc = (f"kv-prepare: 1 of {L} layers, all {B} requests ({t_prep:.2f}s); attention: {n_layers} layer(s) x {len(sel)} of {B} "
            f"requests ({t_attn:.2f}s, scaled by visible keys); acceptance: all {B} requests ({t_acc:.2f}s); "
            f"round time extrapolated x{L} layers")
    return t_round, desc, cores


def host_inputs(cfg, meta, layers_needed=None, with_pool=True):
    L = cfg.num_layers
    host = {}
    if with_pool:
        host["pool_slab"] = W.pool_layer(cfg, meta, 0, poison=False)
    kv = [W.new_kv(cfg, meta, l) for l in range(L)]
    host["k_new"] = np.stack([a for a, _ in kv])
    host["v_new"] = np.stack([b for _, b in kv])
    host["q"] = np.stack([W.queries(cfg, meta, l) for l in range(L)])
    host["p"], host["q_draft"], host["draft_tok"], host["u_acc"], host["u_smp"] = W.accept_inputs(cfg)
    return host


def run_reference(args):
    """`--impl reference`: the CPU oracle on the host cores, each step a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = pick_config(args)
    meta = W.make_batch_meta(cfg)
    host = host_inputs(cfg, meta)
    per_step = max(2.0, min(args.cpu_seconds, 150.0 / max(1, args.steps + args.warmup)))
    times, walls, desc, cores = [], [], "", 1
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        t, desc, cores = oracle_sample(cfg, meta, host, per_step)
        if i >= args.warmup:
            times.append(t)
            walls.append(time.perf_counter() - t0)
    t_round = float(np.median(times))
    value = cfg.batch / t_round
    line = {
        "impl": "reference", "metric": "verify_round_requests_per_s", "value": value, "unit": "req/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        # a step is a bounded sample of the round (see cpu_baseline.sample): its measured time, and beside it the
        # whole-round time extrapolated from the sample, which is what `value` is computed from
        "ms_per_step": float(np.mean(walls)) * 1e3, "extrapolated_ms_per_round": t_round * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(cfg, meta),
        "cpu_baseline": {"value": value, "unit": "req/s", "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "req/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def pick_config(args) -> W.RoundConfig:
    cfg = W.CONFIGS[args.workload]
    if args.batch or args.layers:
        cfg = W.RoundConfig(**{**cfg.__dict__, "batch": args.batch or cfg.batch, "num_layers": args.layers or cfg.num_layers,
                               "name": cfg.name + "_REDUCED_FOR_PROFILING"})
    return cfg


def workload_config(cfg, meta):
    base = cfg.name.replace("_REDUCED_FOR_PROFILING", "")
    return {
        "workload": f"{cfg.name} (configuration {list(W.CONFIGS).index(base) + 1} of the benchmark set)", "batch": cfg.batch,
        "gamma": cfg.gamma, "layers": cfg.num_layers,
        "heads": f"{cfg.num_q_heads}q/{cfg.num_kv_heads}kv x {cfg.head_dim}", "block_size": cfg.block_size,
        "vocab": cfg.vocab, "ctx": list(cfg.ctx_dist), "mean_ctx": float(meta.ctx_len.mean()),
        "reassigned_requests": int(meta.n_mig), "pool_blocks_per_layer": int(meta.num_blocks),
        "l2_policy": "inputs larger than L2: each layer slab is several GB, consecutive layers use different slabs",
    }


# ----------------------------------------------------------------------------- our arm

def scheduled_rounds_leg(cfg, device, rounds, d_accept):
    """Rounds chosen by Algorithm 1 on a two-bank worker (paper_2609_29364_b200/rounds.py): the copy of batch k+1 into
    the standby bank overlaps the run of batch k, the accepted suffix of batch k-1 is exported beside both.  Reports
    the run time and the exposed KV-ready wait (Appendix G.2) per round.  Timing only: parity of this path is
    tests/test_gpu_scheduled_rounds.py."""
    import torch

    import paper_2609_29364_b200 as nsd
    from paper_2609_29364_b200.rounds import ScheduledRounds
    from paper_2609_29364_b200.banks import BankedPool

    B, g, L = max(4, cfg.batch // 2), cfg.gamma, cfg.num_layers
    n_req = (5 * B) // 2                                     # 2.5 batches in the stage's pool: about half of a batch comes back resident
    ctx0 = W.draw_ctx_len(W.RoundConfig(**{**cfg.__dict__, "batch": n_req, "seed": cfg.seed + 7}))
    max_new = rounds * (g + 1)
    need = np.sort((ctx0.astype(np.int64) + max_new + g + 1 + cfg.block_size - 1) // cfg.block_size)[::-1]
    bank_blocks = int(need[:B].sum()) + 64
    banks = BankedPool(ctx0, g, cfg.block_size, max_new, bank_blocks, seed=cfg.seed)
    slab_bytes = banks.num_blocks * cfg.block_elems * 2
    free, _ = torch.cuda.mem_get_info(device)
    slabs = int(min(L, 4, max(1, (0.6 * free) // slab_bytes)))
    if L > 1 and slabs < 2:
        return {"skipped": "not enough free device memory for two layer slabs"}
    ctx = nsd.VerifyContext(num_layers=L, num_slabs=slabs, num_q_heads=cfg.num_q_heads, num_kv_heads=cfg.num_kv_heads,
                            head_dim=cfg.head_dim, block_size=cfg.block_size, num_blocks=banks.num_blocks,
                            region_b_begin=banks.region_b_begin, max_batch=B, max_gamma=g, vocab_size=cfg.vocab,
                            max_table_entries=bank_blocks, device=str(device))
    pool = torch.empty((slabs, banks.num_blocks * cfg.block_elems), dtype=torch.bfloat16, device=device)
    for s_ in range(slabs):
        pool[s_].normal_()
    pool = pool.view(torch.int16)
    rows = B * (g + 1)
    rnd = lambda *shape: torch.randn(shape, dtype=torch.bfloat16, device=device).view(torch.int16)
    fixed = dict(k_new=rnd(L, rows, cfg.num_kv_heads, cfg.head_dim), v_new=rnd(L, rows, cfg.num_kv_heads, cfg.head_dim),
                 q=rnd(L, rows, cfg.num_q_heads, cfg.head_dim), p=d_accept["p"][:B], q_draft=d_accept["q_draft"][:B],
                 draft_tok=d_accept["draft_tok"][:B], u_acc=d_accept["u_acc"][:B], u_smp=d_accept["u_smp"][:B])

    def inputs(k, batch):
        n = len(batch)
        if n == B:
            return fixed
        cut = {name: fixed[name][:, :n * (g + 1)].contiguous() for name in ("k_new", "v_new", "q")}
        cut.update({name: fixed[name][:n] for name in ("p", "q_draft", "draft_tok", "u_acc", "u_smp")})
        return cut

    recs = ScheduledRounds(ctx, pool, banks, ctx0, g, B, inputs, keep_outputs=False).run(rounds)
    steady = recs[2:] if len(recs) > 3 else recs
    blk_bytes = cfg.block_elems * 2 * L
    out = {
        "what": "Algorithm 1 picks each batch from a pool of %d requests; batch k runs out of bank k %% 2 while batch k+1's "
                "non-resident requests are copied from the store into the other bank and batch k-1's accepted suffix is exported" % n_req,
        "rounds": len(recs), "max_batch": B, "layers": L, "physical_layer_slabs": slabs,
        "batch_sizes": [len(r.batch) for r in recs],
        "resident_fraction": [round(float(r.entry.resident.mean()), 3) for r in recs],
        "copied_GB": [round(r.copied_blocks * blk_bytes / 1e9, 2) for r in recs],
        "run_ms": [round(r.run_ms, 3) for r in recs],
        "exposed_kv_wait_ms": [round(r.exposed_wait_ms, 3) for r in recs],
        "steady_state": {"run_ms_median": float(np.median([r.run_ms for r in steady])),
                         "exposed_kv_wait_ms_median": float(np.median([r.exposed_wait_ms for r in steady])),
                         "req_per_s": float(np.mean([len(r.batch) for r in steady]) / (np.median([r.run_ms for r in steady]) * 1e-3))},
    }
    ctx.close()
    return out


def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2609_29364_b200 as nsd
    from paper_2609_29364_b200 import dist_util

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU path)"
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    n_gpus = world

    base = pick_config(args)
    cfg = dist_util.rank_config(base, rank)          # every rank draws its own batch (weak scaling)
    meta = W.make_batch_meta(cfg)
    host = host_inputs(cfg, meta)
    L, B, g1 = cfg.num_layers, cfg.batch, cfg.gamma + 1
    slab_bytes = meta.num_blocks * cfg.block_elems * 2
    free, _total = torch.cuda.mem_get_info(device)
    other = host["p"].nbytes + host["q_draft"].nbytes + 3 * host["q"].nbytes
    slabs = args.slabs or int(min(L, max(1, (0.8 * free - other) // slab_bytes)))
    if L > 1 and slabs < 2:
        raise SystemExit("not enough device memory for two layer slabs")

    def dev(a):
        return torch.from_numpy(np.ascontiguousarray(a.view(np.int16) if a.dtype == np.uint16 else a)).to(device)

    ctx = nsd.VerifyContext(num_layers=L, num_slabs=slabs, num_q_heads=cfg.num_q_heads, num_kv_heads=cfg.num_kv_heads,
                            head_dim=cfg.head_dim, block_size=cfg.block_size, num_blocks=meta.num_blocks,
                            region_b_begin=meta.region_b_begin, max_batch=B, max_gamma=cfg.gamma, vocab_size=cfg.vocab,
                            max_table_entries=int(meta.kv_indptr[-1]), flags=args.ctx_flags, device=str(device))
    pool = torch.empty((slabs, meta.num_blocks * cfg.block_elems), dtype=torch.int16, device=device)
    pool[0].copy_(torch.from_numpy(host["pool_slab"].reshape(-1).view(np.int16)))
    for s in range(1, slabs):
        pool[s].copy_(pool[0])          # every slab starts from the same bytes; the appends make the layers differ
    d = dict(kv_pool=pool, n_mig_blocks=len(meta.mig_src), mig_src=dev(meta.mig_src), mig_dst=dev(meta.mig_dst),
             batch=B, gamma=cfg.gamma, ctx_len=dev(meta.ctx_len), kv_indptr=dev(meta.kv_indptr),
             kv_indices=dev(meta.kv_indices), is_migrated=dev(meta.is_migrated), k_new=dev(host["k_new"]),
             v_new=dev(host["v_new"]), q=dev(host["q"]), o=torch.zeros(host["q"].shape, dtype=torch.int16, device=device),
             p=dev(host["p"]), q_draft=dev(host["q_draft"]), draft_tok=dev(host["draft_tok"]), u_acc=dev(host["u_acc"]),
             u_smp=dev(host["u_smp"]), acc_len=torch.zeros(B, dtype=torch.int32, device=device),
             out_tok=torch.zeros((B, g1), dtype=torch.int32, device=device),
             new_ctx_len=torch.zeros(B, dtype=torch.int32, device=device))
    d_args = ctx.round_args(**d)
    stream = torch.cuda.Stream(device)

    def barrier():
        torch.cuda.synchronize(device)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(device)

    def max_over_ranks(x: float) -> float:
        return dist_util.combine(x, 0.0, device)[0]

    def timed(fn, steps, warmup):
        """ms per step of fn(), CUDA events on the launching stream, max over ranks."""
        with torch.cuda.stream(stream):
            for _ in range(warmup):
                fn()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            e0.record(stream)
            for _ in range(steps):
                fn()
            e1.record(stream)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1)) / steps

    # ---- headline: whole rounds, inputs resident in HBM
    with torch.cuda.stream(stream):
        ctx.nsd_verify_plan(meta.ctx_len, meta.kv_indptr, meta.is_migrated, cfg.gamma, stream=stream)
    props = torch.cuda.get_device_properties(device)
    sampler = ClockSampler("GPU-" + str(props.uuid) if getattr(props, "uuid", None) else str(local))
    launches0 = None

    def one_round():
        ctx.nsd_verify_round(d_args, stream=stream)

    with torch.cuda.stream(stream):
        for _ in range(args.warmup):
            one_round()
    barrier()
    launches0 = ctx.nsd_launch_count()
    sampler.start()
    time.sleep(0.3)
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    with torch.cuda.stream(stream):
        marks[0].record(stream)
        for i in range(args.steps):
            one_round()
            marks[i + 1].record(stream)
    barrier()
    step_ms = [marks[i].elapsed_time(marks[i + 1]) for i in range(args.steps)]
    ms_round = max_over_ranks(float(np.median(step_ms)))              # median step, the slowest rank's
    ms_round_mean = max_over_ranks(marks[0].elapsed_time(marks[-1])) / args.steps
    gpu_launches = ctx.nsd_launch_count() - launches0
    clocks = sampler.stop()
    rc, bad = ctx.nsd_get_status(stream=stream)
    if rc != 0:
        raise SystemExit(f"device status {rc} (request {bad})")
    acc_len = d["acc_len"].cpu().numpy()
    committed = int((acc_len + 1).sum())
    bytes_ = algorithmic_bytes(cfg, meta, acc_len)

    # ---- the same round replayed from a CUDA graph (the call only enqueues, so it can be captured)
    ms_round_graph = None
    try:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            ctx.nsd_verify_round(d_args, stream=torch.cuda.current_stream())
        ms_round_graph = timed(graph.replay, args.steps, args.warmup)
    except Exception as exc:                                    # reported, never fatal for the bench line
        ms_round_graph = None
        print(f"cuda graph leg skipped: {exc}", file=sys.stderr)

    # ---- dominant kernel alone: attention, one launch per layer, events around the launches
    with torch.cuda.stream(stream):
        ctx.nsd_verify_plan(meta.ctx_len, meta.kv_indptr, None, cfg.gamma, stream=stream)

    def attn_all_layers():
        for l in range(L):
            ctx.nsd_verify_attn(pool, d["q"][l], d["o"][l], None, B, cfg.gamma, d["ctx_len"], d["kv_indptr"],
                                d["kv_indices"], layer=l, subset=0, stream=stream)

    ms_attn_launch = timed(attn_all_layers, args.steps, args.warmup) / L
    peak, peak_kind = measured_peak()
    attn_gbs = bytes_["attn_per_layer"] / (ms_attn_launch * 1e-3) / 1e9
    # which engine the library launches for this batch: the tcgen05 one from 33 stacked query rows per kv head on
    # (unless the context's flags say otherwise), else the mma.sync one
    stacked_rows = (cfg.num_q_heads // cfg.num_kv_heads) * (cfg.gamma + 1)
    use_umma = bool(cfg.head_dim == 128 and cfg.block_size == 16 and stacked_rows <= 64 and
                    ((stacked_rows > 32 and not (args.ctx_flags & 4)) or (args.ctx_flags & 2)))
    attn_kernel_name = "verify_attn_umma_kernel + its merge kernel" if use_umma else "verify_attn_kernel"
    attn_traffic_ratio = UMMA_TRAFFIC_PER_ALGORITHMIC_BYTE if use_umma else ATTN_TRAFFIC_PER_ALGORITHMIC_BYTE

    # ---- the other kernels alone and the round without any reassigned request (exposed prepare time)
    def prepare_all_layers():
        ctx.nsd_kv_prepare(pool, d["n_mig_blocks"], d["mig_src"], d["mig_dst"], B, cfg.gamma, d["ctx_len"], d["kv_indptr"],
                           d["kv_indices"], d["k_new"], d["v_new"], stream=stream)

    def accept_only():
        ctx.nsd_spec_accept(d["p"], d["q_draft"], d["draft_tok"], d["u_acc"], d["u_smp"], B, cfg.gamma, cfg.vocab,
                            d["ctx_len"], d["acc_len"], d["out_tok"], d["new_ctx_len"], stream=stream)

    ms_prepare_layer = timed(prepare_all_layers, max(2, args.steps // 2), 1) / L
    ms_accept = timed(accept_only, max(5, args.steps), 2)

    # ---- acceptance straight from logits (the softmax fused in); logits = log p, so the decisions are the same
    logits = torch.log(d["p"])
    acc2 = torch.zeros_like(d["acc_len"])
    out2 = torch.zeros_like(d["out_tok"])

    def accept_logits_only():
        ctx.nsd_spec_accept_logits(logits, 0, 1.0, d["q_draft"], d["draft_tok"], d["u_acc"], d["u_smp"], B, cfg.gamma, cfg.vocab,
                                   None, d["ctx_len"], acc2, out2, None, stream=stream)

    ms_accept_logits = timed(accept_logits_only, max(5, args.steps), 2)
    acc2_h = acc2.cpu().numpy()
    bytes_accept_logits = int((acc2_h + 1).sum()) * cfg.vocab * 4 + int((acc2_h < cfg.gamma).sum()) * cfg.vocab * 4
    # the same from bf16 logits (what a bf16 model head writes): half the bytes per swept row, its own decisions
    logits16 = logits.to(torch.bfloat16).view(torch.int16)
    del logits

    def accept_logits16_only():
        ctx.nsd_spec_accept_logits(logits16, 1, 1.0, d["q_draft"], d["draft_tok"], d["u_acc"], d["u_smp"], B, cfg.gamma, cfg.vocab,
                                   None, d["ctx_len"], acc2, out2, None, stream=stream)

    ms_accept_logits16 = timed(accept_logits16_only, max(5, args.steps), 2)
    acc3_h = acc2.cpu().numpy()
    bytes_accept_logits16 = int((acc3_h + 1).sum()) * cfg.vocab * 2 + int((acc3_h < cfg.gamma).sum()) * cfg.vocab * 4
    del logits16
    nomig = ctx.round_args(**{**d, "n_mig_blocks": 0, "mig_src": None, "mig_dst": None, "is_migrated": None})
    ms_round_nomig = timed(lambda: ctx.nsd_verify_round(nomig, stream=stream), max(2, args.steps // 2), 1)
    exposed_ms = ms_round - ms_round_nomig
    gather_bar_ms = L * bytes_["gather_per_layer"] / (0.7 * NOMINAL_HBM_GBS * 1e9) * 1e3

    # ---- the gather-through variant of the round (reported beside the headline, never instead of it)
    with torch.cuda.stream(stream):
        ctx.nsd_verify_plan(meta.ctx_len, meta.kv_indptr, meta.is_migrated, cfg.gamma, stream=stream)
    fused_args = ctx.round_args(**{**d, "fuse_gather": 1})
    ms_round_fused = timed(lambda: ctx.nsd_verify_round(fused_args, stream=stream), args.steps, args.warmup)
    assert np.array_equal(d["acc_len"].cpu().numpy(), acc_len)

    # ---- a batch that mixes draft depths (ragged rows) against the same batch padded to the deepest draft
    gamma_r = W.draw_gamma_r(cfg, lo=(cfg.gamma + 1) // 2)
    rows_idx, drafts_idx, q_indptr = W.ragged_index(gamma_r, cfg.gamma)
    ri, di = torch.from_numpy(rows_idx).to(device), torch.from_numpy(drafts_idx).to(device)
    V = cfg.vocab
    rag = dict(d)
    rag.update(k_new=d["k_new"][:, ri].contiguous(), v_new=d["v_new"][:, ri].contiguous(), q=d["q"][:, ri].contiguous(),
               o=torch.zeros((L, len(rows_idx)) + tuple(d["q"].shape[2:]), dtype=torch.int16, device=device),
               p=d["p"].reshape(-1, V)[ri].contiguous(), q_draft=d["q_draft"].reshape(-1, V)[di].contiguous(),
               draft_tok=d["draft_tok"].reshape(-1)[di].contiguous(), u_acc=d["u_acc"].reshape(-1)[di].contiguous(),
               out_tok=torch.zeros(len(rows_idx), dtype=torch.int32, device=device), q_indptr=dev(q_indptr))
    with torch.cuda.stream(stream):
        ctx.nsd_verify_plan(meta.ctx_len, meta.kv_indptr, meta.is_migrated, cfg.gamma, stream=stream, h_q_indptr=q_indptr)
    rag_args = ctx.round_args(**rag)
    ms_round_ragged = timed(lambda: ctx.nsd_verify_round(rag_args, stream=stream), args.steps, args.warmup)
    rc, bad = ctx.nsd_get_status(stream=stream)
    if rc != 0:
        raise SystemExit(f"device status {rc} (request {bad}) in the mixed-depth round")
    del rag, rag_args
    with torch.cuda.stream(stream):
        ctx.nsd_verify_plan(meta.ctx_len, meta.kv_indptr, meta.is_migrated, cfg.gamma, stream=stream)

    # ---- end to end: per-round tensors start in pinned host memory, results read back
    e2e = None
    if not args.no_e2e:
        def pin(a):
            return torch.from_numpy(np.ascontiguousarray(a.view(np.int16) if a.dtype == np.uint16 else a)).pin_memory()

        h = dict(kv_pool=None, n_mig_blocks=len(meta.mig_src), mig_src=pin(meta.mig_src), mig_dst=pin(meta.mig_dst),
                 batch=B, gamma=cfg.gamma, ctx_len=pin(meta.ctx_len), kv_indptr=pin(meta.kv_indptr),
                 kv_indices=pin(meta.kv_indices), is_migrated=pin(meta.is_migrated), k_new=pin(host["k_new"]),
                 v_new=pin(host["v_new"]), q=pin(host["q"]), o=torch.zeros(host["q"].shape, dtype=torch.int16).pin_memory(),
                 p=pin(host["p"]), q_draft=pin(host["q_draft"]), draft_tok=pin(host["draft_tok"]),
                 u_acc=pin(host["u_acc"]), u_smp=pin(host["u_smp"]), acc_len=torch.zeros(B, dtype=torch.int32).pin_memory(),
                 out_tok=torch.zeros((B, g1), dtype=torch.int32).pin_memory(),
                 new_ctx_len=torch.zeros(B, dtype=torch.int32).pin_memory())
        h_args = ctx.round_args(**h)
        moved = {}

        def host_round():
            moved["up"], moved["down"] = ctx.nsd_verify_round_host(h_args, d_args, int(meta.kv_indptr[-1]), stream=stream)

        e2e_steps = max(2, min(args.steps, 5))
        host_round()
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            host_round()                       # synchronises the stream before returning
        barrier()
        ms_e2e = max_over_ranks((time.perf_counter() - t0) * 1e3) / e2e_steps
        assert np.array_equal(h["acc_len"].numpy(), acc_len), "host-buffer round disagrees with the device-buffer round"
        e2e = {"value": n_gpus * B / (ms_e2e * 1e-3), "unit": "req/s", "ms_per_step": ms_e2e, "steps": e2e_steps,
               "h2d_bytes_per_step": int(moved["up"]), "d2h_bytes_per_step": int(moved["down"]),
               "api": "nsd_verify_round_host (pinned host buffers; the KV pool is worker state and stays in HBM)"}

    # ---- rounds driven by the scheduler on a two-bank worker (rank 0, N = 1 only; needs the big pool's memory)
    scheduled = None
    if rank == 0 and world == 1 and not args.no_scheduled:
        d_accept = {k_: d[k_] for k_ in ("p", "q_draft", "draft_tok", "u_acc", "u_smp")}
        barrier()
        ctx.close()
        del pool, d_args, nomig, fused_args                   # everything that pins the big pool
        try:
            del graph
        except NameError:
            pass
        try:
            del h_args, h
        except NameError:
            pass
        d.clear()
        torch.cuda.empty_cache()
        scheduled = scheduled_rounds_leg(cfg, device, args.scheduled_rounds, d_accept)

    # ---- the oracle on the host cores (rank 0, N = 1 only)
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        t_round_cpu, desc, cores = oracle_sample(cfg, meta, host, args.cpu_seconds)
        cpu_baseline = {"value": B / t_round_cpu, "unit": "req/s", "cores": cores, "kind": "oracle", "sample": desc,
                        "seconds_per_round_extrapolated": t_round_cpu}

    if rank == 0:
        round_gbs = bytes_["round"] / (ms_round * 1e-3) / 1e9
        line = {
            "metric": "verify_round_requests_per_s", "value": n_gpus * B / (ms_round * 1e-3), "unit": "req/s",
            "n_gpus": n_gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_round,
            "ms_per_step_mean": ms_round_mean, "timing": "median of per-step CUDA-event pairs on the launching stream, max over ranks",
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": workload_config(cfg, meta), "physical_layer_slabs": slabs,
            "committed_tokens_per_s": n_gpus * committed / (ms_round * 1e-3),
            "verified_rows_per_s": n_gpus * cfg.rows / (ms_round * 1e-3),
            "mean_accepted_len": float(acc_len.mean()),
            "roofline": {"kernel": attn_kernel_name + " (one launch per layer, timed alone)", "bound": "hbm",
                         "achieved": attn_gbs, "peak": peak, "peak_kind": f"{peak_kind} copy bandwidth",
                         "unit": "GB/s", "frac": attn_gbs / peak, "frac_of_nominal_8TBs": attn_gbs / NOMINAL_HBM_GBS,
                         "traffic": int(attn_traffic_ratio * bytes_["attn_per_layer"]),
                         "traffic_source": "profiler capture of a smaller case of the same kernel, scaled by algorithmic bytes",
                         "bytes_per_launch": bytes_["attn_per_layer"], "ms_per_launch": ms_attn_launch},
            "round_roofline": {"bound": "hbm", "achieved": round_gbs, "peak": peak, "unit": "GB/s",
                               "frac": round_gbs / peak, "frac_of_nominal_8TBs": round_gbs / NOMINAL_HBM_GBS,
                               "algorithmic_bytes_per_round": bytes_["round"]},
            "breakdown_ms": {"attn_per_layer_alone": ms_attn_launch, "prepare_per_layer_alone": ms_prepare_layer,
                             "accept_alone": ms_accept, "round_without_reassignment": ms_round_nomig,
                             "exposed_prepare": exposed_ms, "exposed_prepare_bar": gather_bar_ms,
                             "prepare_GBs_alone": (bytes_["gather_per_layer"] + bytes_["append_per_layer"]) / (ms_prepare_layer * 1e-3) / 1e9,
                             "accept_GBs_alone": bytes_["accept"] / (ms_accept * 1e-3) / 1e9,
                             "accept_from_logits_alone": ms_accept_logits,
                             "accept_from_logits_GBs": bytes_accept_logits / (ms_accept_logits * 1e-3) / 1e9,
                             "accept_from_logits_agrees_on": float((acc2_h == acc_len).mean()),
                             "accept_from_bf16_logits_alone": ms_accept_logits16,
                             "accept_from_bf16_logits_GBs": bytes_accept_logits16 / (ms_accept_logits16 * 1e-3) / 1e9},
            "gather_through_round": {
                "what": "nsd_verify_round with fuse_gather=1: attention reads reassigned requests from their source blocks and "
                        "writes the destination blocks itself; no copy kernel, no side stream; same pool bytes and outputs",
                "ms_per_step": ms_round_fused, "value": n_gpus * B / (ms_round_fused * 1e-3), "unit": "req/s",
                "algorithmic_bytes_per_round": bytes_["round"] - L * bytes_["gather_per_layer"] // 2,
                "achieved_GBs": (bytes_["round"] - L * bytes_["gather_per_layer"] // 2) / (ms_round_fused * 1e-3) / 1e9,
                "speedup_over_headline": ms_round / ms_round_fused},
            "mixed_depth_round": {
                "what": "the same batch with per-request draft depths drawn from [%d, %d] (ragged rows) "
                        "against the batch padded to depth %d, which is the headline round" % ((cfg.gamma + 1) // 2, cfg.gamma, cfg.gamma),
                "rows": int(len(rows_idx)), "padded_rows": int(cfg.rows), "ms_per_step": ms_round_ragged,
                "useful_rows_per_s": n_gpus * len(rows_idx) / (ms_round_ragged * 1e-3),
                "useful_rows_per_s_padded": n_gpus * len(rows_idx) / (ms_round * 1e-3),
                "speedup_over_padded": ms_round / ms_round_ragged},
            "round_cuda_graph": None if ms_round_graph is None else {
                "ms_per_step": ms_round_graph, "value": n_gpus * B / (ms_round_graph * 1e-3), "unit": "req/s"},
            "scheduled_rounds": scheduled,
            "e2e": e2e, "gpu_launches": int(gpu_launches), "clocks": clocks, "cpu_baseline": cpu_baseline,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
