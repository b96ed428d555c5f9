"""Block bookkeeping for multi-round runs: a request store and a two-bank worker.

Stand-in for the paper's layout (Section 5, Appendix E.2): every request's
up-to-date KV lives in a store (the paper's pinned HostKV; here pool region A),
and the target worker computes out of two banks with separate block ranges
(here two halves of pool region B), alternating between them from batch to
batch.  A request that was in the batch this bank held last keeps its blocks
("resident"); every other request of the new batch gets blocks from the bank's
free list and has its committed KV copied in from the store.

Only tables are kept here -- which block ids a request owns where.  No KV byte
is touched and none of the method's arithmetic lives in this module, so the
oracle-side test and the CUDA-side driver can both take their tables from it.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List

import numpy as np


@dataclass
class BankEntry:
    """What a batch needs to enter a bank."""
    kv_indptr: np.ndarray      # int64 [B+1]  bank tables of the batch, ceil((ctx+gamma+1)/bs) blocks each
    kv_indices: np.ndarray     # int32
    store_indptr: np.ndarray   # int64 [B+1]  the same requests' store tables (same lengths)
    store_indices: np.ndarray  # int32
    resident: np.ndarray       # uint8 [B]    1 = the bank still holds this request's committed KV
    mig_src: np.ndarray        # int32        store blocks to copy (ceil(ctx/bs) per non-resident request)
    mig_dst: np.ndarray        # int32        bank blocks they go to


class BankedPool:
    def __init__(self, ctx_len: np.ndarray, gamma: int, block_size: int, max_new_tokens: int, bank_blocks: int,
                 seed: int = 0):
        self.bs, self.gamma = block_size, gamma
        n = len(ctx_len)
        # store: room for every token a request can reach, ids scattered over region A
        need = (np.asarray(ctx_len, dtype=np.int64) + max_new_tokens + gamma + 1 + block_size - 1) // block_size
        self.store_indptr = np.zeros(n + 1, dtype=np.int64)
        np.cumsum(need, out=self.store_indptr[1:])
        self.region_b_begin = int(self.store_indptr[-1])
        rng = np.random.Generator(np.random.Philox(key=np.array([np.uint64(seed), np.uint64(77)], dtype=np.uint64)))
        self.store_indices = rng.permutation(self.region_b_begin).astype(np.int32)
        self.bank_blocks = bank_blocks
        self.num_blocks = self.region_b_begin + 2 * bank_blocks
        # banks: free lists (scattered order) and the blocks each request currently holds there
        self.free: List[List[int]] = []
        self.held: List[Dict[int, List[int]]] = [{}, {}]
        for b in range(2):
            ids = self.region_b_begin + b * bank_blocks + rng.permutation(bank_blocks)
            self.free.append([int(x) for x in ids])

    def blocks_needed(self, ctx: int) -> int:
        return (int(ctx) + self.gamma + 1 + self.bs - 1) // self.bs

    def store_table(self, r: int, n_blocks: int) -> np.ndarray:
        lo = int(self.store_indptr[r])
        assert lo + n_blocks <= int(self.store_indptr[r + 1]), "request outgrew its store allocation"
        return self.store_indices[lo:lo + n_blocks]

    def enter(self, bank: int, batch: List[int], ctx_len: np.ndarray) -> BankEntry:
        """Makes `batch` (request ids, with their current context lengths `ctx_len[r]`) the occupant of `bank`."""
        held, free = self.held[bank], self.free[bank]
        for r in [r for r in held if r not in batch]:          # whoever is not coming back gives its blocks up
            free.extend(held.pop(r))
        indptr = np.zeros(len(batch) + 1, dtype=np.int64)
        tables, stores, resident, src, dst = [], [], [], [], []
        for i, r in enumerate(batch):
            nb = self.blocks_needed(ctx_len[r])
            was_here = r in held
            mine = held.setdefault(r, [])
            if len(mine) < nb:
                take = nb - len(mine)
                if take > len(free):
                    raise ValueError("bank is out of blocks")
                mine.extend(free[:take])
                del free[:take]
            tables.append(np.asarray(mine[:nb], dtype=np.int32))
            stores.append(self.store_table(r, nb))
            resident.append(1 if was_here else 0)
            if not was_here:
                n_ctx = (int(ctx_len[r]) + self.bs - 1) // self.bs
                src.append(stores[-1][:n_ctx])
                dst.append(tables[-1][:n_ctx])
            indptr[i + 1] = indptr[i] + nb
        cat = lambda xs: np.concatenate(xs).astype(np.int32) if xs else np.zeros(0, dtype=np.int32)
        return BankEntry(indptr, cat(tables), indptr.copy(), cat(stores), np.asarray(resident, dtype=np.uint8), cat(src), cat(dst))
