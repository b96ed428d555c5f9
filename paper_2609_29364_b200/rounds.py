"""Rounds driven by Algorithm 1: schedule -> prepare the standby bank -> run -> export the suffix.

Host-side sequencing only; every byte is moved and every number computed by the library's kernels.
The worker owns two banks (block ranges) and alternates between them (Appendix E.2); batch k runs out
of bank k % 2 while the copy of batch k+1's non-resident requests from the store into the other bank is
already under way on a second stream (Run(B_k) || Prepare(B_k+1), Section 4) and the accepted suffix of
batch k-1 is exported to the store on a third (Compute_k || D2H_k-1, Appendix E.2).  A bank is refilled
only after the export of its previous occupant has physically completed.

What is measured per batch is the paper's exposed KV-ready wait, E_i = [K_i - max(I_i, W_i)]_+
(Appendix G.2): K_i = the event after the bank's copy, W_i = the event after the previous batch's run;
inputs are on the device before the batch is enqueued, so I_i never binds.

The scheduler's clock is a model, not a measurement, so that a run is reproducible: a batch of n rows
over b blocks is predicted to run for `t_fixed + t_block * b` seconds, a draft step takes `t_draft`,
copying a block from the store takes `t_copy_block` (the profile tables phi_s of Eq. (4) are the
caller's; these four constants stand in for them).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, Dict, List

import numpy as np

from .api import VerifyContext, nsd_schedule_batch


@dataclass
class ClockModel:
    t_fixed: float = 1.0e-3
    t_block: float = 2.0e-7
    t_draft: float = 2.0e-3
    t_copy_block: float = 1.0e-7
    target_interval: float = 4.0e-3
    slack: float = 2.0e-3


@dataclass
class RoundRecord:
    batch: List[int]
    start_pred: float
    entry: object
    ctx_len: np.ndarray
    acc_len: np.ndarray = None
    out_tok: np.ndarray = None
    o: object = None
    exposed_wait_ms: float = 0.0
    run_ms: float = 0.0
    copied_blocks: int = 0
    sched_inputs: Dict[str, object] = field(default_factory=dict)


class ScheduledRounds:
    """`banks` is a BankedPool (banks.py beside this file); `inputs(k, batch)` returns the round's device-side inputs as numpy
    arrays: k_new, v_new, q ([L][rows]...), p, q_draft, draft_tok, u_acc, u_smp."""

    def __init__(self, ctx: VerifyContext, kv_pool, banks, ctx_len0: np.ndarray, gamma: int, max_batch: int,
                 inputs: Callable[[int, List[int]], Dict[str, np.ndarray]], clock: ClockModel = ClockModel(),
                 keep_outputs: bool = True):
        import torch

        self.torch, self.ctx, self.pool, self.banks, self.gamma = torch, ctx, kv_pool, banks, gamma
        self.max_batch, self.inputs, self.clock, self.keep = max_batch, inputs, clock, keep_outputs
        self.ctx_len = np.asarray(ctx_len0, dtype=np.int32).copy()       # per request, as the host knows it
        n = len(self.ctx_len)
        self.pred_done = np.arange(n, dtype=np.float64) * 1.0e-6           # first outputs trickle in by index
        self.worker_avail = 0.0
        self.main, self.prep, self.exp = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
        self.main.wait_stream(torch.cuda.current_stream())                # whatever filled the pool comes first
        self.bank_free = [None, None]                                      # event: the bank's last export has completed
        self.records: List[RoundRecord] = []

    # ---- Algorithm 1 with the model clock
    def _choose(self, busy: List[int], bank: int) -> RoundRecord:
        n, c, bk = len(self.ctx_len), self.clock, self.banks
        eligible = np.ones(n, dtype=np.uint8)
        eligible[busy] = 0
        blocks = np.array([bk.blocks_needed(x) for x in self.ctx_len], dtype=np.int32)
        resident = np.array([1 if r in bk.held[bank] else 0 for r in range(n)], dtype=np.uint8)
        kv_ready = self.pred_done + np.where(resident == 1, 0.0, c.t_copy_block * blocks)
        rows = np.full(n, self.gamma + 1, dtype=np.int32)
        sched = dict(worker_avail=self.worker_avail, target_interval=c.target_interval, slack=c.slack, max_batch=self.max_batch,
                     pred_done=self.pred_done.copy(), kv_ready=kv_ready, eligible=eligible, rows=rows, blocks=blocks,
                     tokens=self.ctx_len.copy(), row_capacity=self.max_batch * (self.gamma + 1), block_capacity=bk.bank_blocks,
                     token_limit=2 ** 62)
        batch, start = nsd_schedule_batch(**sched)
        rec = RoundRecord(batch=batch, start_pred=start, entry=None, ctx_len=self.ctx_len[batch].copy(), sched_inputs=sched)
        if batch:
            run = c.t_fixed + c.t_block * float(blocks[batch].sum())
            self.worker_avail = start + run
            self.pred_done[batch] = self.worker_avail + c.t_draft
        return rec

    def _enqueue_prepare(self, k: int, rec: RoundRecord):
        torch = self.torch
        bank = k % 2
        rec.entry = e = self.banks.enter(bank, rec.batch, self.ctx_len)
        rec.copied_blocks = int(len(e.mig_src))
        dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory().cuda(non_blocking=True)
        rec.ev_k = torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(self.prep):                            # small tables ride the same stream as the copy
            rec.d = dict(ctx_len=dev(rec.ctx_len), kv_indptr=dev(e.kv_indptr), kv_indices=dev(e.kv_indices),
                         store_indptr=dev(e.store_indptr), store_indices=dev(e.store_indices))
            if self.bank_free[bank] is not None:
                self.prep.wait_event(self.bank_free[bank])
            if rec.copied_blocks:
                rec.d["mig_src"], rec.d["mig_dst"] = dev(e.mig_src), dev(e.mig_dst)
                self.ctx.nsd_kv_prepare(self.pool, rec.copied_blocks, rec.d["mig_src"], rec.d["mig_dst"], 0, self.gamma,
                                        None, None, None, None, None, stream=self.prep)
            rec.ev_k.record(self.prep)

    def _enqueue_run(self, k: int, rec: RoundRecord):
        torch, g = self.torch, self.gamma
        B = len(rec.batch)
        h = self.inputs(k, rec.batch)

        def dev(a):                                                   # device tensors pass through, numpy is uploaded
            if isinstance(a, torch.Tensor):
                return a
            return torch.from_numpy(np.ascontiguousarray(a.view(np.int16) if a.dtype == np.uint16 else a)).cuda()

        d = rec.d
        with torch.cuda.stream(self.main):
            self._enqueue_run_on_main(k, rec, h, dev, B, g, d)

    def _enqueue_run_on_main(self, k, rec, h, dev, B, g, d):
        torch = self.torch
        for name in ("k_new", "v_new", "q", "p", "q_draft", "draft_tok", "u_acc", "u_smp"):
            d[name] = dev(h[name])
        d["o"] = torch.zeros_like(d["q"])
        d["acc_len"] = torch.zeros(B, dtype=torch.int32, device="cuda")
        d["out_tok"] = torch.zeros((B, g + 1), dtype=torch.int32, device="cuda")
        d["new_ctx_len"] = torch.zeros(B, dtype=torch.int32, device="cuda")
        rec.ev_w, rec.ev_r = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        rec.ev_done = torch.cuda.Event()
        rec.ev_w.record(self.main)                                   # the worker is free: the previous run has ended
        self.main.wait_event(rec.ev_k)                               # ... and now the bank's state must be there
        self.ctx.nsd_verify_plan(rec.ctx_len, rec.entry.kv_indptr, None, g, stream=self.main)
        args = self.ctx.round_args(kv_pool=self.pool, n_mig_blocks=0, mig_src=None, mig_dst=None, batch=B, gamma=g,
                                   ctx_len=d["ctx_len"], kv_indptr=d["kv_indptr"], kv_indices=d["kv_indices"], is_migrated=None,
                                   k_new=d["k_new"], v_new=d["v_new"], q=d["q"], o=d["o"], p=d["p"], q_draft=d["q_draft"],
                                   draft_tok=d["draft_tok"], u_acc=d["u_acc"], u_smp=d["u_smp"], acc_len=d["acc_len"],
                                   out_tok=d["out_tok"], new_ctx_len=d["new_ctx_len"])
        rec.args = args
        self.ctx.nsd_verify_round(args, stream=self.main)
        rec.ev_r.record(self.main)
        with torch.cuda.stream(self.exp):                             # export the accepted suffix, then the bank may be refilled
            self.exp.wait_event(rec.ev_r)
            self.ctx.nsd_kv_commit(self.pool, B, g, d["ctx_len"], d["acc_len"], d["kv_indptr"], d["kv_indices"],
                                   d["store_indptr"], d["store_indices"], stream=self.exp)
            rec.ev_done.record(self.exp)
        self.bank_free[k % 2] = rec.ev_done

    def _collect(self, rec: RoundRecord):
        rec.ev_done.synchronize()
        rec.acc_len = rec.d["acc_len"].cpu().numpy()
        rec.out_tok = rec.d["out_tok"].cpu().numpy()
        self.ctx_len[rec.batch] = rec.d["new_ctx_len"].cpu().numpy()
        rec.exposed_wait_ms = max(0.0, rec.ev_w.elapsed_time(rec.ev_k))
        rec.run_ms = rec.ev_w.elapsed_time(rec.ev_r)
        if self.keep:
            rec.o = rec.d["o"].cpu()
        keep = {"acc_len", "out_tok"} if not self.keep else set(rec.d)
        rec.d = {k_: v for k_, v in rec.d.items() if k_ in keep}

    def run(self, n_rounds: int) -> List[RoundRecord]:
        recs = self.records
        nxt = self._choose([], 0)
        if nxt.batch:
            self._enqueue_prepare(0, nxt)
        for k in range(n_rounds):
            cur = nxt
            if not cur.batch:
                break
            recs.append(cur)
            self._enqueue_run(k, cur)
            if k >= 1:
                self._collect(recs[k - 1])                           # lengths of the batch before: needed to size the next one
            if k + 1 < n_rounds:
                nxt = self._choose(cur.batch, (k + 1) % 2)
                if nxt.batch:
                    self._enqueue_prepare(k + 1, nxt)
        if recs and recs[-1].acc_len is None:
            self._collect(recs[-1])
        rc, bad = self.ctx.nsd_get_status()
        if rc != 0:
            raise RuntimeError(f"device status {rc} (request {bad})")
        return recs
