"""Glue between the host controller (Algorithm 1) and the transition kernels: the paper's
transition engine in miniature (App. B.2).

  - demotion is synchronous: ekv_downgrade is enqueued, its residual (low byte) slots are copied
    to a pinned host "backing" store, and the released blocks re-enter the free list only after
    the GPU reported completion (an event the host waits for);
  - promotion is asynchronous up to the last step: the residual of every chosen pair travels
    host -> device on a side stream while the main stream keeps executing on the intact BASE
    pair; the main stream then waits for that copy's event and runs ekv_refine, so every launch
    enqueued before it saw BASE and every launch after it sees TARGET (stream order is the
    publication rule); the controller publishes the mapping at that point.
No arithmetic of the method lives here: bytes are moved by the library's kernels."""
from __future__ import annotations

import numpy as np
import torch

from . import binding as b
from .controller import Controller


class ElasticRuntime:
    def __init__(self, pool: b.Pool, max_batch: int, max_blocks: int, resid_slots: int, **ctrl_kw):
        dev = pool.k_pool.device
        self.pool = pool
        self.ctrl = Controller(pool.num_blocks, pool.page_size, resid_slots=resid_slots, **ctrl_kw)
        self.block_table = torch.full((max_batch, max_blocks), -1, dtype=torch.int32, device=dev)
        self.seq_lens = torch.zeros(max_batch, dtype=torch.int32, device=dev)
        self.batch = b.Batch(self.block_table, self.seq_lens, has_base=True)
        self.k_resid, self.v_resid = pool.new_resid(resid_slots), pool.new_resid(resid_slots)
        shape = self.k_resid.shape
        self.k_backing = torch.zeros(shape, dtype=torch.uint8).pin_memory()     # the recoverable host copy
        self.v_backing = torch.zeros(shape, dtype=torch.uint8).pin_memory()
        self.side = torch.cuda.Stream(device=dev)
        self.rows = {}                  # request id -> row of the device table
        self.free_rows = list(range(max_batch - 1, -1, -1))
        self.lens = {}
        self.boundaries = torch.zeros((max_batch, 2), dtype=torch.int32, device=dev)
        self.flags = torch.zeros(4, dtype=torch.int32, device=dev)
        self.stats = {"demoted": 0, "promoted": 0}

    # ---- requests ----
    def lower(self, reqs=None):
        """Bring the device metadata of `reqs` (default: every live request) in line with the
        controller: ONE host-to-device copy of the sparse description (lengths, block lists, BASE
        pair ranges) and ONE library call that writes the table rows, the lengths, the structured
        path's boundaries and the batch flags, and checks the ranges against the tags. Returns the
        flags as a device tensor [any BASE, any irregular, disagreeing pairs, n - first such]."""
        reqs = [r for r in (self.rows if reqs is None else reqs) if self.lens.get(r, 0) > 0]
        lists = [self.ctrl.block_table(r) for r in reqs]
        ranges = []
        for r, t in zip(reqs, lists):
            rr, start = [], None
            for p in range(len(t) // 2 + 1):
                is_base = p < len(t) // 2 and self.ctrl.pair_mode(r, p) == 1
                if is_base and start is None:
                    start = p
                if not is_base and start is not None:
                    rr += [start, p]
                    start = None
            ranges.append(rr)
        parts = [np.array([self.rows[r] for r in reqs], np.int32), np.array([self.lens[r] for r in reqs], np.int32),
                 np.concatenate([[0], np.cumsum([len(t) for t in lists])]).astype(np.int32),
                 np.concatenate(lists).astype(np.int32) if lists else np.zeros(0, np.int32),
                 np.concatenate([[0], np.cumsum([len(x) // 2 for x in ranges])]).astype(np.int32),
                 np.array([v for x in ranges for v in x], np.int32)]
        offs = np.concatenate([[0], np.cumsum([len(x) for x in parts])])
        arena = torch.from_numpy(np.concatenate(parts).astype(np.int32)).to(self.block_table.device)
        v = [arena[offs[k]:offs[k + 1]] for k in range(6)]
        b.ekv_lower_sparse_metadata(self.pool, self.batch, self.seq_lens, v[0], v[1], v[2], v[3], v[4],
                                    v[5] if len(v[5]) else None, self.boundaries, self.flags)
        return self.flags

    def layout(self):
        """(any BASE pair, any irregular request) of the live requests, from the controller's state: a
        request is irregular when a TARGET pair lies between two of its BASE pairs (Sec. 3.2)."""
        any_base = irregular = False
        for r, n in self.lens.items():
            if n <= 0:
                continue
            modes = [self.ctrl.pair_mode(r, p) == 1 for p in range(len(self.ctrl.block_table(r)) // 2)]
            if any(modes):
                any_base = True
                first, last = modes.index(True), len(modes) - 1 - modes[::-1].index(True)
                irregular = irregular or not all(modes[first:last + 1])
        return any_base, irregular

    def decode(self, q, out, num_q_heads, sm_scale, workspace, layer=0):
        """Decode attention with the dispatch of Sec. 3.2, decided on the host (no device read): a batch
        without BASE pairs takes the native path, a batch whose sequences are all regular the structured
        path (boundaries from the sparse lowering), any other the general path. Returns the path's name."""
        any_base, irregular = self.layout()
        msl = max([n for n in self.lens.values()] + [0])
        if any_base and not irregular:
            self.lower()
            b.ekv_attn_decode_structured(self.pool, layer, self.batch, self.boundaries, q, out, num_q_heads, sm_scale, msl,
                                         workspace)
            return "structured"
        self.batch.has_base = any_base
        try:
            b.ekv_attn_decode(self.pool, layer, self.batch, q, out, num_q_heads, sm_scale, msl, workspace)
        finally:
            self.batch.has_base = True
        return "general" if any_base else "native"

    def add_request(self, req, n_tokens):
        self.ctrl.add_request(req, n_tokens)
        self.rows[req] = self.free_rows.pop()
        self.lens[req] = n_tokens
        self.lower([req])

    def grow_request(self, req, n_tokens):
        self.ctrl.grow_request(req, n_tokens)
        self.lens[req] = n_tokens
        self.lower([req])

    def finish_request(self, req):
        """The request leaves: its blocks (and residual slots) return to the controller and its table
        row to the free rows. Blocks that stored a BASE pair are tagged TARGET again (by the
        library), since a released block carries no fidelity."""
        t = self.ctrl.block_table(req)
        base_blocks = [int(t[2 * p]) for p in range(len(t) // 2) if self.ctrl.pair_mode(req, p) == 1]
        self.ctrl.remove_request(req)
        row = self.rows.pop(req)
        if base_blocks:
            b.ekv_reset_tags(self.pool, self._dev(base_blocks))
        self.block_table[row] = -1
        self.seq_lens[row] = 0
        self.boundaries[row] = 0
        del self.lens[req]
        self.free_rows.append(row)
        return base_blocks

    def _dev(self, a):
        return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(self.block_table.device)

    def _rows_of(self, reqs):
        return np.array([self.rows[int(r)] for r in reqs], dtype=np.int32)

    # ---- Algorithm 1, first half: shortage-driven synchronous demotion ----
    def relieve(self, demand_blocks: int):
        """Returns the demotion batch as (table rows, pair indices, slots); empty when no shortage."""
        pr, pi, sl = self.ctrl.plan_demotion(int(demand_blocks))
        if len(pr) == 0:
            return pr, pi, sl
        rows = self._rows_of(pr)
        freed = torch.empty(len(pr), dtype=torch.int32, device=self.block_table.device)
        d_sl = self._dev(sl)
        b.ekv_downgrade(self.pool, self.batch, self._dev(rows), self._dev(pi), self.k_resid, self.v_resid, d_sl, freed)
        done = torch.cuda.Event()
        done.record()
        with torch.cuda.stream(self.side):               # backing copy of the low bytes, off the main stream
            self.side.wait_event(done)
            for s in sl.tolist():
                self.k_backing[s].copy_(self.k_resid[s], non_blocking=True)
                self.v_backing[s].copy_(self.v_resid[s], non_blocking=True)
        done.synchronize()                               # synchronous demotion: commit after GPU completion
        self.ctrl.commit_demotion(freed.cpu().numpy())
        self.stats["demoted"] += len(pr)
        return rows, pi, sl

    # ---- Algorithm 1, second half: reserve-aware asynchronous promotion ----
    def restore(self, transfer_slack: int):
        pr, pi, nb, sl = self.ctrl.plan_promotion(int(transfer_slack))
        if len(pr) == 0:
            return pr, pi, nb, sl
        rows = self._rows_of(pr)
        main = torch.cuda.current_stream()
        arrived = torch.cuda.Event()
        with torch.cuda.stream(self.side):               # residuals travel while the main stream runs on BASE
            for s in sl.tolist():
                self.k_resid[s].copy_(self.k_backing[s], non_blocking=True)
                self.v_resid[s].copy_(self.v_backing[s], non_blocking=True)
            arrived.record()
        main.wait_event(arrived)
        b.ekv_refine(self.pool, self.batch, self._dev(rows), self._dev(pi), self._dev(nb), self.k_resid, self.v_resid,
                     self._dev(sl))
        self.ctrl.commit_promotion(len(pr))              # published in stream order
        self.stats["promoted"] += len(pr)
        return rows, pi, nb, sl
