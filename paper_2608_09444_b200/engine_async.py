"""Pipelined (asynchronous) driver of the CDB hot path, refill mode with the lookahead gate.

What the paper's section 4.3 / Fig. 3 describes: while the GPU runs loop step N, the host already knows
which rows leave after it (the exit flag of step N depends only on the signal stored by step N-1, so the
compaction lists are computed at the START of step N), prepares the descriptor of step N+1 and enqueues
it; the coda + sampling + prelude of the rows that left after step N-1 run on a second stream beside loop
step N, and their tokens rejoin the recurrent batch at step N+1.  The main stream therefore never waits
for the host or for a boundary stage.  While the batch has free rows and the boundary pass is cheap next to a
step (no boundary layers), the boundary stages are instead enqueued before step N, which waits for them on the
device: the tokens rejoin at step N (see eager_refill).  Either way the host never waits for the device
except to read the exit lists of the step it has just enqueued, and everything it sends per step leaves
from pinned memory.

Streams and buffers
  main  H2D descriptor -> cdb_compact (lists) -> [event] -> CUDA graph (loop step, survivor gather to the
        front of h_rec, exit gather to h_exit[parity]) -> refill gather
  side  D2H lists; copy of exited rows into the coda queue; cdb_boundary_coda_lmhead; D2H tokens;
        cdb_boundary_embed / _prelude of the sampled tokens into h_ready
Results (tokens, exit depths) are those of the synchronous engine and of the CPU oracle: scheduling
changes when work runs, never what is computed.
"""
from __future__ import annotations

import time

import numpy as np
import torch

from . import binding as B
from .engine import Engine, _bucket, _static_rows


def boundary_cost_in_steps(dims):
    """Cost of one boundary pass (prelude and coda layers, LM head) in loop steps: twice the FLOP ratio, because small
    steps are bound by latency rather than arithmetic.  ~0.16 for the Ouro shape (no boundary layers), ~2.4 for the
    Huginn shape (2 + 2 boundary layers and a 65536-row LM head against a 4-layer core)."""
    per_layer = 4 * dims.d * dims.d + 3 * dims.d * dims.F
    return 2.0 * ((dims.L_pre + dims.L_coda) * per_layer + dims.V * dims.d) / (dims.L_core * per_layer)


class PipelinedEngine(Engine):
    def __init__(self, *a, background_prefill=True, prefill_priority=0, eager_refill=True, **kw):
        kw.setdefault("mode", "refill")
        kw.setdefault("lookahead", True)
        super().__init__(*a, **kw)
        if self.mode != "refill" or not self.lookahead:
            raise ValueError("the pipelined engine implements refill mode with the lookahead gate")
        # decode work (main and side stream) outranks prompt processing when both have kernels waiting for SMs
        self.main = torch.cuda.Stream(device=self.dev, priority=-1)
        self.side = torch.cuda.Stream(device=self.dev, priority=-1)
        # prompts of newly admitted requests are processed on a stream of their own beside the running decode
        # batch (the library gives prompt calls their own scratch); False = drain the pipeline and process them alone
        self.background_prefill = background_prefill
        # (prefill_priority 0 = below the decode streams, -1 = level with them)
        self.pstream = torch.cuda.Stream(device=self.dev, priority=prefill_priority)
        # While the batch has free rows, the boundary stages of the rows that left after step N-1 can be enqueued
        # BEFORE step N, which then waits for them on the device (no host wait): those tokens rejoin at once instead
        # of sitting out a step, at the price of a bubble of one boundary pass for the surviving rows.  Taken when the
        # rows that rejoin outweigh that bubble, boundary_ratio being the cost of a boundary pass in loop steps
        # (twice the FLOP ratio: small steps are latency-bound): Ouro-like models (no boundary layers) take it at
        # every step with free rows, Huginn-like ones (boundary as heavy as the core) never.  With a full batch
        # (more live sequences than rows) the boundary stages run beside step N as described above.
        self.eager_refill = eager_refill
        self.boundary_ratio = boundary_cost_in_steps(self.dims)
        d = self.dims.d
        self.h_exit2 = [torch.zeros((self.max_rows, d), dtype=torch.float32, device=self.dev) for _ in range(2)]
        self.h_coda_in = torch.zeros((self.cap, d), dtype=torch.float32, device=self.dev)
        # prelude outputs awaiting a batch row: a ring, each boundary call takes a contiguous run of rows (the prelude
        # writes there directly, the refill gather reads by row index).  A sequence has at most one row in it, rows leave
        # in the order they came, so four times the live set cannot wrap onto a row still waiting.
        self.h_ready_ring = torch.zeros((4 * self.cap, d), dtype=torch.float32, device=self.dev)
        self.lists_host = torch.zeros((2 * self.max_rows + 2,), dtype=torch.int32).pin_memory()
        self.lists_dev = torch.zeros((2 * self.max_rows + 2,), dtype=torch.int32, device=self.dev)
        self.pgraphs = {}

    # ---- graph of one step body for (bucket, parity): loop step + gathers; compaction runs before it
    def _body(self, rows, nb, parity):
        c, hx = self.cdb, self.h_rec[:nb]
        c.loop_step(rows, hx, self.gate_val, self.fire)
        c.gather_rows(hx, self.surv_idx, self.counts[0:1], nb, self.h_tmp)
        c.gather_rows(hx, self.exit_idx, self.counts[1:2], nb, self.h_exit2[parity])
        hx.copy_(self.h_tmp[:nb])

    def _capture_all(self):
        """Graphs for every row-count bucket and both parities, captured before any live row exists (the
        warm-up run of a capture scribbles over h_rec)."""
        nb = 32
        while True:
            nb = min(nb, self.max_rows)
            for parity in (0, 1):
                if (nb, parity) in self.pgraphs:
                    continue
                self.desc_dev[5, 0].fill_(0)                      # live count 0, all pads: the warm-up touches no model state
                rows = _static_rows(self, nb)
                self.cdb.compact(rows, self.surv_idx, self.exit_idx, self.counts)
                self._body(rows, nb, parity)
                torch.cuda.synchronize(self.dev)
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    self._body(rows, nb, parity)
                self.pgraphs[(nb, parity)] = (g, rows)
            if nb >= _bucket(self.max_batch, self.max_rows):
                break
            nb += 32
        torch.cuda.synchronize(self.dev)

    # ------------------------------------------------------------------ generation
    def generate(self, prompts, T, forced_depths=None, teacher_tokens=None, arrivals=None):
        """Same contract as Engine.generate.  Sampled tokens stay on the device and feed the prelude directly;
        with teacher_tokens (lock-step replay) the given tokens are fed instead, while the sampled ones are
        still returned.  Gate values are not read back."""
        caller = torch.cuda.current_stream(self.dev)
        self.main.wait_stream(caller)
        with torch.cuda.stream(self.main):
            out = self._generate(prompts, T, forced_depths, teacher_tokens, arrivals)
        caller.wait_stream(self.main)
        return out

    def _generate(self, prompts, T, forced_depths, teacher_tokens, arrivals):
        dims, cdb, dev = self.dims, self.cdb, self.dev
        main, side = torch.cuda.current_stream(dev), self.side
        n = len(prompts)
        Ts = [T] * n if np.isscalar(T) else list(T)
        P = [len(p) for p in prompts]
        tokens = [[None] * Ts[i] for i in range(n)]
        depths = [[] for _ in range(n)]
        gen = [0] * n                                   # tokens sampled so far (values may still be in flight)
        waiting, live_slot = (list(range(n)) if arrivals is None else []), {}
        future = [] if arrivals is None else list(range(n))
        free_slots = list(range(self.max_live - 1, -1, -1))
        ready, ring_head = [], [0]                                    # (sid, row in h_ready_ring, event, iteration)
        coda_q, coda_free = [], list(range(self.cap - 1, -1, -1))     # (sid, depth, slot in h_coda)
        pending_tokens, pending_release = [], []
        ring = [torch.zeros((7, self.max_rows), dtype=torch.int32).pin_memory() for _ in range(4)]
        tok_ring = [torch.zeros(self.cap, dtype=torch.int32).pin_memory() for _ in range(16)]
        tok_dev = torch.zeros(self.cap, dtype=torch.int32, device=dev)
        tokp_dev = torch.zeros(self.cap, dtype=torch.int32, device=dev)      # first tokens of a prompt call
        tokp_host = torch.zeros(self.cap, dtype=torch.int32).pin_memory()
        counts_h = torch.zeros(2, dtype=torch.int32).pin_memory()
        surv_h = torch.zeros(self.max_rows, dtype=torch.int32).pin_memory()
        exit_h = torch.zeros(self.max_rows, dtype=torch.int32).pin_memory()
        i64 = lambda a: torch.tensor(a, dtype=torch.int64, device=dev)
        i32 = lambda a: torch.tensor(np.asarray(a, dtype=np.int32), dtype=torch.int32, device=dev)
        # index arrays of the side stream's boundary calls: one pinned block and one asynchronous copy per call (a
        # copy from pageable memory would hold the host until the side stream has caught up with the running step)
        width = max(self.cap, self.max_rows)
        stage_ring = [(torch.zeros((9, width), dtype=torch.int32).pin_memory(),
                       torch.zeros((9, width), dtype=torch.int32, device=dev), [None]) for _ in range(8)]
        stage_calls = [0]

        def staged(stream, *arrays):
            """device copies of the given integer lists, sent as one block on `stream`"""
            host, devb, ev = stage_ring[stage_calls[0] % len(stage_ring)]
            stage_calls[0] += 1
            if ev[0] is not None:
                ev[0].synchronize()                     # the block's previous copy has left the pinned buffer
            for j, a in enumerate(arrays):
                if len(a):
                    host[j, :len(a)] = torch.as_tensor(np.asarray(a, dtype=np.int32))
            with torch.cuda.stream(stream):
                devb.copy_(host, non_blocking=True)
                ev[0] = torch.cuda.Event()
                ev[0].record(stream)
            return [devb[j, :len(a)] for j, a in enumerate(arrays)]
        self._capture_all()
        self.stats["start"] = time.perf_counter()
        self.stats["first_token_s"], self.stats["finish_s"] = [None] * n, [None] * n
        now = lambda: time.perf_counter() - self.stats["start"]
        x_done = [None, None]                           # h_exit2[parity] copied out (event on the side stream)
        gather_done = None                              # last refill gather on the main stream
        tok_calls = 0

        def forced_for(s):
            if forced_depths is not None and forced_depths[s] is not None:
                return int(forced_depths[s][gen[s] - 1])
            return 0

        def fed_back(sids, sampled):
            """input tokens of the next pass of sequences sids: the sampled ones (device), or the teacher's"""
            if teacher_tokens is None:
                return sampled
            return i32([teacher_tokens[s][gen[s] - 1] for s in sids])

        def drain_tokens(block):
            while pending_tokens and (block or pending_tokens[0][0].query()):
                ev, buf, items = pending_tokens.pop(0)
                ev.synchronize()
                vals = buf.numpy()
                for j, (s, idx) in enumerate(items):
                    tokens[s][idx] = int(vals[j])
                    if idx == Ts[s] - 1:
                        self.stats["finish_s"][s] = now()
            while pending_release and (block or pending_release[0][0].query()):
                ev, s = pending_release.pop(0)
                ev.synchronize()
                self._release_pages(live_slot[s])
                free_slots.append(live_slot.pop(s))

        def enqueue_prelude(sids, tok_t, stream, it, pick=None):
            """prelude of the device-resident input tokens of sequences sids -> h_ready; on `stream`.  The tokens
            are tok_t, or its entries `pick` (indices into it)."""
            sl = [live_slot[s] for s in sids]
            pos = [P[s] + gen[s] - 1 for s in sids]
            n_new = len(sids)
            assert len(ready) + n_new <= self.cap
            if ring_head[0] + n_new > self.h_ready_ring.shape[0]:
                ring_head[0] = 0
            first = ring_head[0]
            ring_head[0] += n_new
            if pick is not None and len(pick) == len(tok_t):
                pick = None                             # everything goes on: no selection needed
            sl_d, pos_d, pick_d = staged(stream, sl, pos, pick if pick is not None else [])
            if pick is not None:
                tok_t = tok_t[pick_d.long()]
            rows = B.Rows(sl_d, pos_d, self.page_table)
            out = self.h_ready_ring[first:first + n_new]
            if gather_done is not None:
                stream.wait_event(gather_done)          # rows of an earlier lap may still be read by the last refill gather
            (cdb.boundary_prelude if dims.L_pre > 0 else cdb.boundary_embed)(tok_t, rows, out, stream=stream)
            ev = torch.cuda.Event()
            ev.record(stream)
            ready.extend((s, first + j, ev, it) for j, s in enumerate(sids))

        prefill_inflight = []                           # at most one: (event, batch, pinned token buffer)

        def admit_background():
            """prompt processing of waiting requests on the prompt stream, beside the running decode batch"""
            if prefill_inflight:
                return
            batch, rows_total = [], 0
            while waiting and free_slots and rows_total + P[waiting[0]] <= self.max_rows:
                s = waiting[0]
                if not self._reserve_pages(free_slots[-1], P[s] + Ts[s]):
                    break
                live_slot[s] = free_slots.pop()
                waiting.pop(0)
                batch.append(s)
                rows_total += P[s]
            if not batch:
                return
            table_ready = torch.cuda.Event()
            table_ready.record(main)                    # the page-table rows were updated on the main stream
            toks = np.concatenate([np.asarray(prompts[s], dtype=np.int32) for s in batch])
            sl = np.concatenate([np.full(P[s], live_slot[s]) for s in batch])
            pos = np.concatenate([np.arange(P[s]) for s in batch])
            ends = np.cumsum([P[s] for s in batch]) - 1
            m = len(batch)
            with torch.cuda.stream(self.pstream):
                self.pstream.wait_event(table_ready)
                cdb.prefill(i32(toks), B.Rows(i32(sl), i32(pos), self.page_table), i32(ends), tokp_dev[:m], stream=self.pstream)
                tokp_host[:m].copy_(tokp_dev[:m], non_blocking=True)
                ev = torch.cuda.Event()
                ev.record(self.pstream)
            prefill_inflight.append((ev, batch))
            self.stats["prefill_calls"] += 1

        def poll_prefill(block):
            """first tokens of a finished prompt call: record them, start the prelude of the sequences that go on"""
            if not prefill_inflight or not (block or prefill_inflight[0][0].query()):
                return
            ev, batch = prefill_inflight.pop(0)
            ev.synchronize()
            vals = tokp_host[:len(batch)].numpy().copy()
            cont = []
            for j, s in enumerate(batch):
                tokens[s][0] = int(vals[j])
                gen[s] = 1
                self.stats["first_token_s"][s] = now()
                if gen[s] >= Ts[s]:
                    self.stats["finish_s"][s] = now()
                    self._release_pages(live_slot[s])
                    free_slots.append(live_slot.pop(s))
                else:
                    cont.append(j)
            if cont:                                     # boundary calls share one scratch lane: all of them on the side stream
                with torch.cuda.stream(side):
                    first = staged(side, vals[cont])[0] if teacher_tokens is None else fed_back([batch[j] for j in cont], None)
                    enqueue_prelude([batch[j] for j in cont], first, side, it)

        def admit():
            """prompt processing of waiting requests while live slots and pages are free (drains the pipeline)"""
            side.synchronize()
            drain_tokens(True)
            while waiting and free_slots:
                batch, rows_total = [], 0
                while waiting and free_slots and rows_total + P[waiting[0]] <= self.max_rows:
                    s = waiting[0]
                    if not self._reserve_pages(free_slots[-1], P[s] + Ts[s]):
                        break
                    live_slot[s] = free_slots.pop()
                    waiting.pop(0)
                    batch.append(s)
                    rows_total += P[s]
                if not batch:
                    break
                toks = np.concatenate([np.asarray(prompts[s], dtype=np.int32) for s in batch])
                sl = np.concatenate([np.full(P[s], live_slot[s]) for s in batch])
                pos = np.concatenate([np.arange(P[s]) for s in batch])
                ends = np.cumsum([P[s] for s in batch]) - 1
                m = len(batch)
                cdb.prefill(i32(toks), B.Rows(i32(sl), i32(pos), self.page_table), i32(ends), tok_dev[:m])
                vals = tok_dev[:m].cpu().numpy()
                self.stats["prefill_calls"] += 1
                cont = []
                for j, s in enumerate(batch):
                    tokens[s][0] = int(vals[j])
                    gen[s] = 1
                    self.stats["first_token_s"][s] = now()
                    if Ts[s] == 1:
                        self.stats["finish_s"][s] = now()
                    if gen[s] >= Ts[s]:
                        self._release_pages(live_slot[s])
                        free_slots.append(live_slot.pop(s))
                    else:
                        cont.append(j)
                if cont:
                    enqueue_prelude([batch[j] for j in cont], fed_back([batch[j] for j in cont], tok_dev[:m][i64(cont)].contiguous()), main, -1)
            torch.cuda.synchronize(dev)

        def boundary_for(prev, it, force):
            """side stream: queue the rows that left after the previous step, run the coda (+ sampling) when
            enough have gathered, and the prelude of the sampled tokens"""
            nonlocal tok_calls
            with torch.cuda.stream(side):
                if prev is not None and prev["ne"]:
                    side.wait_event(prev["G"])
                with self._phase("boundary"):
                    # no minimum coda batch and nothing queued: the rows that left go to the coda where they are
                    direct = prev is not None and prev["ne"] and self.min_coda_batch <= 1 and not coda_q
                    if direct:
                        items = [(s, r, None) for s, r in prev["exits"]]
                    elif prev is not None and prev["ne"]:
                        slots = [coda_free.pop() for _ in range(prev["ne"])]
                        self.h_coda.index_copy_(0, staged(side, slots)[0].long(), self.h_exit2[prev["parity"]][:prev["ne"]])
                        ev = torch.cuda.Event()
                        ev.record(side)
                        x_done[prev["parity"]] = ev
                        coda_q.extend((s, r, slot) for (s, r), slot in zip(prev["exits"], slots))
                    if not direct:
                        if not coda_q or (len(coda_q) < self.min_coda_batch and not force):
                            return
                        items = list(coda_q)
                        coda_q.clear()
                    m = len(items)
                    sids = [it_[0] for it_ in items]
                    from_d, sl_d, pos_d, depth_d = staged(side, [] if direct else [it_[2] for it_ in items], [live_slot[s] for s in sids],
                                                          [P[s] + gen[s] - 1 for s in sids], [it_[1] for it_ in items])
                    if direct:
                        hin = self.h_exit2[prev["parity"]][:m]
                    else:
                        hin = self.h_coda_in[:m]
                        cdb.gather_rows(self.h_coda, from_d, None, m, hin, stream=side)
                    rows = B.Rows(sl_d, pos_d, self.page_table)
                    if self.kv_layout == B.KV_DEPTH_INDEXED:
                        cdb.kv_copy_on_exit(rows, depth_d, stream=side)
                    cdb.boundary_coda_lmhead(rows, hin, tok_dev[:m], stream=side)
                    if direct:                          # the exit buffer of this parity has been consumed
                        x_done[prev["parity"]] = torch.cuda.Event()
                        x_done[prev["parity"]].record(side)
                    buf = tok_ring[tok_calls % len(tok_ring)][:m]
                    tok_calls += 1
                    buf.copy_(tok_dev[:m], non_blocking=True)
                    ev = torch.cuda.Event()
                    ev.record(side)
                    pending_tokens.append((ev, buf, [(s, gen[s]) for s in sids]))
                    self.stats["coda_calls"] += 1
                    cont = []
                    for j, (s, r, slot) in enumerate(items):
                        if slot is not None:
                            coda_free.append(slot)
                        gen[s] += 1
                        if gen[s] >= Ts[s]:
                            pending_release.append((ev, s))
                        else:
                            cont.append(j)
                    if cont and teacher_tokens is None:
                        enqueue_prelude([sids[j] for j in cont], tok_dev[:m], side, it, pick=cont)
                    elif cont:
                        enqueue_prelude([sids[j] for j in cont], fed_back([sids[j] for j in cont], None), side, it)

        rec, prev, it = [], None, 0
        while True:
            drain_tokens(False)
            if future:
                t_now = now()
                while future and arrivals[future[0]] <= t_now:
                    waiting.append(future.pop(0))
            poll_prefill(False)
            if waiting and free_slots and (arrivals is None or len(waiting) >= self.admit_min or not live_slot
                                           or now() - arrivals[waiting[0]] >= self.admit_wait_s):
                if self.background_prefill:
                    admit_background()
                else:
                    admit()
            if "decode_start" not in self.stats and not waiting and not future and not prefill_inflight:
                torch.cuda.synchronize(dev)
                self.stats["decode_start"] = time.perf_counter()
                self._mark_decode_start()
            # ---- free rows in the batch: the rows that left after the previous step pass their boundary stages first
            if (self.eager_refill and prev is not None and len(rec) + len(ready) < self.max_batch
                    and prev["ne"] > self.boundary_ratio * (len(rec) + prev["ne"])):
                boundary_for(prev, it - 1, force=self.min_coda_batch <= 1)
                self.stats["eager_boundaries"] = self.stats.get("eager_boundaries", 0) + 1
                prev = None
            # ---- refills whose prelude was enqueued in an earlier iteration join this step
            take = []
            while ready and len(rec) + len(take) < self.max_batch and ready[0][3] < it:
                take.append(ready.pop(0))
            n_keep = len(rec)
            for s, _, _, _ in take:
                rec.append([s, 1])
            k = len(rec)
            step = None
            if k:
                parity = it & 1
                nb = _bucket(k, self.max_rows)
                dh = ring[it % len(ring)]
                dh[0, :k] = torch.as_tensor(np.asarray([live_slot[s] for s, _ in rec], dtype=np.int32))
                dh[1, :k] = torch.as_tensor(np.asarray([r for _, r in rec], dtype=np.int32))
                dh[2, :k] = torch.as_tensor(np.asarray([P[s] + gen[s] - 1 for s, _ in rec], dtype=np.int32))
                dh[3, :k] = torch.as_tensor(np.asarray([self._slot(r) for _, r in rec], dtype=np.int32))
                dh[4, :k] = torch.as_tensor(np.asarray([forced_for(s) for s, _ in rec], dtype=np.int32))
                dh[5, 0] = k                                # device-side live count: the rows behind it are pads
                if take:
                    dh[6, :len(take)] = torch.as_tensor(np.asarray([t[1] for t in take], dtype=np.int32))
                with self._phase("recurrent"):
                    # one pinned block carries everything the step needs from the host (a pageable copy here would
                    # make the host wait for the previous step and leave the GPU idle while the next one is enqueued)
                    self.desc_dev.copy_(dh, non_blocking=True)
                    if take:
                        for _, _, ev, _ in take:
                            if ev is not None:
                                main.wait_event(ev)
                        cdb.gather_rows(self.h_ready_ring, self.desc_dev[6, :len(take)], None, len(take), self.h_rec[n_keep:n_keep + len(take)])
                        gather_done = torch.cuda.Event()
                        gather_done.record(main)
                    g, rows = self.pgraphs[(nb, parity)]
                    cdb.compact(rows, self.surv_idx, self.exit_idx, self.counts)
                    lists_ready = torch.cuda.Event()
                    lists_ready.record(main)
                    if x_done[parity] is not None:
                        main.wait_event(x_done[parity])     # the exits of two steps ago have left h_exit2[parity]
                    g.replay()
                G = torch.cuda.Event()
                G.record(main)
                with torch.cuda.stream(side):
                    side.wait_event(lists_ready)
                    counts_h.copy_(self.counts, non_blocking=True)
                    surv_h[:nb].copy_(self.surv_idx[:nb], non_blocking=True)
                    exit_h[:nb].copy_(self.exit_idx[:nb], non_blocking=True)
                    lists_copied = torch.cuda.Event()
                    lists_copied.record(side)
                step = (parity, G, lists_copied)
            # ---- boundary stages of the rows that left after the previous step, beside this step
            idle = not k and not ready
            boundary_for(prev, it, force=idle or self.min_coda_batch <= 1)
            prev = None
            if step is not None:
                parity, G, lists_copied = step
                lists_copied.synchronize()
                ns, ne = int(counts_h[0]), int(counts_h[1])
                surv, ex = surv_h[:ns].numpy().copy(), exit_h[:ne].numpy().copy()
                exits = [(rec[int(i)][0], rec[int(i)][1]) for i in ex]
                for s, r in exits:
                    depths[s].append(r)
                self.stats["recurrent_steps"] += 1
                self.stats["row_steps"] += k
                self.stats["rows_hist"][(k - 1) // 32] += 1
                prev = {"parity": parity, "ne": ne, "exits": exits, "G": G}
                rec = [[rec[int(i)][0], rec[int(i)][1] + 1] for i in surv]
            it += 1
            if not rec and prev is None and not ready and not coda_q and prefill_inflight:
                poll_prefill(True)                      # nothing else to run: wait for the prompt call
                continue
            if not rec and prev is None and not ready and not coda_q and not waiting:
                if future and not pending_tokens and not pending_release:
                    time.sleep(min(1e-3, max(0.0, arrivals[future[0]] - now())))
                    continue
                if not future and all(gen[s] >= Ts[s] for s in range(n)):
                    break
                if not pending_tokens and not pending_release:
                    raise RuntimeError("pipelined scheduler stalled")
                drain_tokens(True)
        torch.cuda.synchronize(dev)
        drain_tokens(True)
        self.stats["end"] = time.perf_counter()
        if self.time_device:
            self._collect_device_time()
        return {"tokens": [np.asarray(t, dtype=np.int32) for t in tokens],
                "depths": [np.asarray(d, dtype=np.int32) for d in depths], "gates": None}
