"""Host-side driver of the CDB hot path: the four queues of the paper's section 4.1 (waiting
requests, tokens awaiting the prelude, recurrent items, exited tokens awaiting the coda), the
priority rule (coda > prefill up to the KV budget > recurrent step), refill / no-refill / fixed
depth modes, and page bookkeeping.  It only builds row descriptors and moves index lists; all
model arithmetic, the exit decision and the compaction run in libcdb.so.

The deterministic tick mode implemented here runs one stage per tick and waits for its result, so
that per-tick row lists and page tables are reproducible bit for bit.
"""
from __future__ import annotations

import dataclasses
import time

import numpy as np
import torch

from . import binding as B


@dataclasses.dataclass
class _Seq:
    sid: int
    prompt: np.ndarray
    T: int
    tokens: list
    depths: list
    gates: list
    cur_gates: list
    next_input: int = -1


class Engine:
    def __init__(self, dims, weights, *, max_batch: int, max_live: int, max_len: int, n_pages: int,
                 kv_layout: int = B.KV_SHARED, gate_kind: int = B.GATE_SIGMOID_CDF, q_or_eps: float = 0.5,
                 r_min: int = 1, lookahead: bool = True, mode: str = "refill", min_coda_batch: int = 1,
                 max_prefill_rows: int | None = None, flags: int = 0, record_states: bool = False,
                 record_logits: bool = False, record_ticks: bool = True, use_graphs: bool = True,
                 time_device: bool = False, admit_min: int = 1, admit_wait_s: float = 0.0, device: str = "cuda:0",
                 boundary_pages: int | None = None):
        if mode not in ("refill", "no_refill", "cb"):
            raise ValueError(f"unknown scheduling mode {mode!r}: expected 'refill', 'no_refill' or 'cb'")
        self.dims, self.mode, self.lookahead = dims, mode, lookahead
        self.max_batch, self.max_live, self.min_coda_batch = max_batch, max_live, min_coda_batch
        self.dev = torch.device(device)
        self.max_pages = (max_len + dims.page_size - 1) // dims.page_size
        max_rows = max(max_batch, max_prefill_rows or max_batch)
        self.max_rows = max_rows
        self.cdb = B.Cdb(dims, weights, max_rows=max_rows, max_seqs=max_live, max_position=self.max_pages * dims.page_size,
                         kv_layout=kv_layout, gate_kind=gate_kind, q_or_eps=q_or_eps, r_min=r_min, flags=flags)
        self.n_slots = self.cdb.n_slots
        self.kv_layout = kv_layout
        dt = torch.float32 if dims.dtype == "fp32" else torch.bfloat16
        # A model with prelude / coda layers and more than one depth slot gets a page space of its own for those layers:
        # they cache one k, v per token whatever the layout, so only the core layers' pool pays for the slots (Table 1).
        # boundary_pages: pages of that space (default: the main pool's share of one slot); 0 = one shared page space.
        self.split_kv = self.n_slots > 1 and dims.L_pre + dims.L_coda > 0 and boundary_pages != 0
        if self.split_kv:
            self.n_pages_b = boundary_pages or max(1, n_pages // self.n_slots)
            self.pool_b = torch.zeros((dims.L_pre + dims.L_coda, self.n_pages_b, 2, dims.H, dims.page_size, dims.Dh), dtype=dt, device=self.dev)
            self.free_pages_b = list(range(self.n_pages_b - 1, -1, -1))
            self._page_table_b_pin = torch.full((max_live, self.max_pages), -1, dtype=torch.int32).pin_memory()
            self.page_table_b_host = self._page_table_b_pin.numpy()       # the host's table lives in pinned memory: row updates go out as asynchronous copies
            self.page_table_b = self._page_table_b_pin.to(self.dev)
            self.cdb.kv_bind_boundary(self.pool_b, self.page_table_b)
        self.pool = torch.zeros((dims.L_core if self.split_kv else dims.L, n_pages, 2, dims.H, dims.page_size, dims.Dh), dtype=dt, device=self.dev)
        self.cdb.kv_bind(self.pool)
        self.n_pages = n_pages
        self.free_pages = list(range(n_pages - 1, -1, -1))            # pop() hands out the lowest id first
        self._page_table_pin = torch.full((max_live * self.n_slots, self.max_pages), -1, dtype=torch.int32).pin_memory()
        self.page_table_host = self._page_table_pin.numpy()
        self.page_table = self._page_table_pin.to(self.dev)
        i32 = dict(dtype=torch.int32, device=self.dev)
        f32 = dict(dtype=torch.float32, device=self.dev)
        d = dims.d
        self.h_rec = torch.zeros((max_rows, d), **f32)                # rows of the next recurrent step
        self.h_tmp = torch.zeros((max_rows, d), **f32)
        self.h_exit = torch.zeros((max_rows, d), **f32)               # compaction output: exited rows
        self.cap = max(max_rows, max_live)
        self.h_coda = torch.zeros((self.cap, d), **f32)               # coda queue rows
        self.h_ready = torch.zeros((self.cap, d), **f32)              # prelude output awaiting a batch slot
        self.gate_val = torch.zeros(max_rows, **f32)
        self.fire = torch.zeros(max_rows, dtype=torch.uint8, device=self.dev)
        self.surv_idx = torch.zeros(max_rows, **i32)
        self.exit_idx = torch.zeros(max_rows, **i32)
        self.counts = torch.zeros(2, **i32)
        self.tok_out = torch.zeros(max_rows, **i32)
        self.logits = torch.zeros((max_rows, dims.V), **f32) if record_logits else None
        self.record_states, self.record_logits, self.record_ticks = record_states, record_logits, record_ticks
        self.stats = {"recurrent_steps": 0, "row_steps": 0, "coda_calls": 0, "prefill_calls": 0, "tick_rows": [],
                      "rows_hist": [0] * ((max_batch + 31) // 32)}      # recurrent steps by row count, 32-row bins
        self.trace_states = {}                                        # (sid, token index) -> exit state
        self.trace_step_states = {}                                   # (sid, token index, loop depth) -> state after that loop step
        self.trace_logits = {}
        # Recurrent step as a CUDA graph per row-count bucket (rows padded with seq_id = -1 to a multiple of 32):
        # the descriptor lives in fixed device arrays refreshed by one host-to-device copy per step.
        self.use_graphs = use_graphs
        # five descriptor rows; [5, 0] = live rows; row 6 = h_ready slots of the rows that join (pipelined engine)
        self.desc_host = torch.zeros((7, max_rows), dtype=torch.int32).pin_memory()
        self.desc_dev = torch.zeros((7, max_rows), **i32)
        self.graphs = {}
        # optional accounting of device time: CUDA-event pairs around every GPU phase the engine enqueues
        self.time_device = time_device
        # online serving: hold arrived requests until admit_min of them wait or the oldest has waited admit_wait_s,
        # so that prompts are processed several at a time (one prompt alone re-reads every weight per loop)
        self.admit_min, self.admit_wait_s = admit_min, admit_wait_s
        self._dev_events = []

    class _Phase:
        def __init__(self, eng, name):
            self.eng, self.name = eng, name

        def __enter__(self):
            if self.eng.time_device:
                self.a = torch.cuda.Event(enable_timing=True)
                self.a.record()

        def __exit__(self, *exc):
            if self.eng.time_device:
                b = torch.cuda.Event(enable_timing=True)
                b.record()
                self.eng._dev_events.append((self.name, self.a, b))
            return False

    def _phase(self, name):
        """Brackets the GPU work enqueued inside with an event pair (no-op unless time_device)."""
        return Engine._Phase(self, name)

    def _mark_decode_start(self):
        """Event at the start of the decode phase: brackets recorded before it are left out of the busy time."""
        if self.time_device:
            self._decode_start_ev = torch.cuda.Event(enable_timing=True)
            self._decode_start_ev.record()

    def _collect_device_time(self):
        """stats["device_ms"][phase] = summed event time of that phase's brackets (after a synchronize).
        stats["device_busy_ms"] = length of the UNION of all brackets of the decode phase, whatever stream they were
        recorded on (phases that overlap on two streams count once): wall - busy is the time the GPU had nothing of
        the engine to run, the per-step device idle of the paper's Fig. 3."""
        out = {}
        for name, a, b in self._dev_events:
            out[name] = out.get(name, 0.0) + a.elapsed_time(b)
        self.stats["device_ms"] = out
        spans = []
        if self._dev_events:
            base = self._dev_events[0][1]
            t0 = base.elapsed_time(self._decode_start_ev) if getattr(self, "_decode_start_ev", None) is not None else 0.0
            for name, a, b in self._dev_events:
                s0, s1 = base.elapsed_time(a), base.elapsed_time(b)
                if name != "prefill" and s1 > t0:
                    spans.append((max(s0, t0), s1))
        spans.sort()
        busy, end = 0.0, None
        for s0, s1 in spans:
            if end is None or s0 > end:
                busy += s1 - s0
                end = s1
            elif s1 > end:
                busy += s1 - end
                end = s1
        self.stats["device_busy_ms"] = busy
        self._dev_events = []

    # ------------------------------------------------------------------ descriptor helpers
    def _rows(self, seq_ids, positions, depths=None, slots=None, forced=None):
        t = lambda a: torch.tensor(np.asarray(a, dtype=np.int32), dtype=torch.int32, device=self.dev)
        return B.Rows(t(seq_ids), t(positions), self.page_table,
                      loop_depth=None if depths is None else t(depths),
                      kv_slot=None if slots is None else t(slots),
                      forced_exit=None if forced is None else t(forced))

    def _slot(self, r):
        if self.kv_layout == B.KV_DEPTH_INDEXED:
            return r - 1
        if self.kv_layout == B.KV_FIRST_THEN_SHARED:
            return min(r, 2) - 1
        return 0

    def _reserve_pages(self, slot_id: int, n_tokens: int) -> bool:
        need = (n_tokens + self.dims.page_size - 1) // self.dims.page_size
        if need * self.n_slots > len(self.free_pages) or need > self.max_pages:
            return False
        if self.split_kv:
            if need > len(self.free_pages_b):
                return False
            for j in range(need):
                self.page_table_b_host[slot_id, j] = self.free_pages_b.pop()
            self.page_table_b[slot_id].copy_(self._page_table_b_pin[slot_id], non_blocking=True)
        for s in range(self.n_slots):
            row = slot_id * self.n_slots + s
            for j in range(need):
                self.page_table_host[row, j] = self.free_pages.pop()
        rows = slice(slot_id * self.n_slots, (slot_id + 1) * self.n_slots)
        # (a sequence's rows are next written when it has finished, i.e. after every step that reads this copy)
        self.page_table[rows].copy_(self._page_table_pin[rows], non_blocking=True)
        return True

    def _release_pages(self, slot_id: int):
        if self.split_kv:
            used = self.page_table_b_host[slot_id][self.page_table_b_host[slot_id] >= 0]
            for p in reversed(used):
                self.free_pages_b.append(int(p))
            self.page_table_b_host[slot_id] = -1
        for s in reversed(range(self.n_slots)):
            row = slot_id * self.n_slots + s
            used = self.page_table_host[row][self.page_table_host[row] >= 0]
            for p in reversed(used):
                self.free_pages.append(int(p))
            self.page_table_host[row] = -1

    # ------------------------------------------------------------------ generation
    def generate(self, prompts, T, forced_depths=None, teacher_tokens=None, arrivals=None):
        """prompts: list of int arrays; T: generated tokens per sequence (int or list).  forced_depths[s][j]
        replays the exit depth of adaptive pass j of sequence s (0 / None = decided by the gate);
        teacher_tokens[s][j] replaces the token fed back after generated token j (lock-step replay).
        arrivals[s] (seconds after the call starts, non-decreasing) makes request s visible to the scheduler
        only from that wall-clock time on (online serving); stats["first_token_s"] / ["finish_s"] then hold
        the times at which the host saw each request's first and last token."""
        dims, cdb = self.dims, self.cdb
        n = len(prompts)
        Ts = [T] * n if np.isscalar(T) else list(T)
        seqs = [_Seq(i, np.asarray(prompts[i], dtype=np.int32), Ts[i], [], [], [], []) for i in range(n)]
        waiting = list(range(n)) if arrivals is None else []
        future = [] if arrivals is None else list(range(n))
        self.stats["start"] = time.perf_counter()
        self.stats["first_token_s"], self.stats["finish_s"] = [None] * n, [None] * n
        now = lambda: time.perf_counter() - self.stats["start"]

        def poll_arrivals():
            t = now()
            while future and arrivals[future[0]] <= t:
                waiting.append(future.pop(0))

        live_slot = {}                       # sid -> live slot id (index into gate state / page table)
        free_slots = list(range(self.max_live - 1, -1, -1))
        ready = []                           # [(sid, h row index in h_ready)] awaiting the recurrent batch (FIFO)
        ready_free = list(range(self.cap - 1, -1, -1))
        rec = []                             # current recurrent rows: [sid, depth] in row order (h in h_rec)
        coda_q = []                          # [(sid, depth, row in h_coda)]
        coda_free = list(range(self.cap - 1, -1, -1))
        fixed_depth = self.mode == "cb"

        def forced_for(sq):
            j = len(sq.tokens) - 1           # index of the adaptive pass in flight
            if fixed_depth:
                return dims.R
            if forced_depths is not None and forced_depths[sq.sid] is not None:
                return int(forced_depths[sq.sid][j])
            return 0

        def position_of(sq):
            return len(sq.prompt) + len(sq.tokens) - 1

        def start_tokens(sids):
            """prelude for the next input token of each sequence -> ready queue"""
            if not sids:
                return
            toks, pos, sl = [], [], []
            for s in sids:
                sq = seqs[s]
                toks.append(sq.next_input)
                pos.append(position_of(sq))
                sl.append(live_slot[s])
            rows = self._rows(sl, pos)
            tok_t = torch.tensor(toks, dtype=torch.int32, device=self.dev)
            out = self.h_tmp[:len(sids)]
            slots = [ready_free.pop() for _ in sids]
            with self._phase("prelude"):
                if dims.L_pre > 0:
                    cdb.boundary_prelude(tok_t, rows, out)
                else:
                    cdb.boundary_embed(tok_t, rows, out)
                self.h_ready.index_copy_(0, torch.tensor(slots, dtype=torch.int64, device=self.dev), out)
            ready.extend(zip(sids, slots))

        def finish_or_continue(s, token):
            sq = seqs[s]
            sq.tokens.append(int(token))
            if len(sq.tokens) == 1:
                self.stats["first_token_s"][s] = now()
            if len(sq.tokens) >= sq.T:
                self.stats["finish_s"][s] = now()
                self._release_pages(live_slot[s])
                free_slots.append(live_slot.pop(s))
                return None
            j = len(sq.tokens) - 1
            sq.next_input = int(teacher_tokens[s][j]) if teacher_tokens is not None else int(token)
            return s

        def admission_due():
            if not waiting or not free_slots:
                return False
            if arrivals is None or len(waiting) >= self.admit_min or not live_slot:
                return True
            return now() - arrivals[waiting[0]] >= self.admit_wait_s

        def run_prefill():
            if not admission_due():
                return False
            admitted = []
            rows_total = 0
            while waiting and free_slots:
                s = waiting[0]
                sq = seqs[s]
                P = len(sq.prompt)
                if rows_total + P > self.max_rows:
                    break
                slot = free_slots[-1]
                if not self._reserve_pages(slot, P + sq.T):
                    break
                free_slots.pop()
                waiting.pop(0)
                live_slot[s] = slot
                self.stats.setdefault("admissions", []).append(
                    (s, slot, self.page_table_host[slot * self.n_slots:(slot + 1) * self.n_slots].copy()))
                admitted.append(s)
                rows_total += P
            if not admitted:
                return False
            toks = np.concatenate([seqs[s].prompt for s in admitted])
            sl = np.concatenate([np.full(len(seqs[s].prompt), live_slot[s]) for s in admitted])
            pos = np.concatenate([np.arange(len(seqs[s].prompt)) for s in admitted])
            ends = np.cumsum([len(seqs[s].prompt) for s in admitted]) - 1
            rows = self._rows(sl, pos)
            emit = torch.tensor(ends, dtype=torch.int32, device=self.dev)
            tok_t = torch.tensor(toks, dtype=torch.int32, device=self.dev)
            lg = self.logits[:len(admitted)] if self.record_logits else None
            with self._phase("prefill"):
                cdb.prefill(tok_t, rows, emit, self.tok_out[:len(admitted)], lg)
            out = self.tok_out[:len(admitted)].cpu().numpy()
            self.stats["prefill_calls"] += 1
            cont = []
            for k, s in enumerate(admitted):
                if self.record_logits:
                    self.trace_logits[(s, 0)] = lg[k].cpu().numpy()
                r = finish_or_continue(s, out[k])
                if r is not None:
                    cont.append(r)
            start_tokens(cont)
            return True

        def run_coda():
            items = list(coda_q)
            coda_q.clear()
            k = len(items)
            idx = torch.tensor([it[2] for it in items], dtype=torch.int32, device=self.dev)
            hin = self.h_tmp[:k]
            cdb.gather_rows(self.h_coda, idx, None, k, hin)
            sl = [live_slot[it[0]] for it in items]
            pos = [position_of(seqs[it[0]]) for it in items]
            rows = self._rows(sl, pos)
            if self.record_states:
                states = hin.cpu().numpy()
            if self.kv_layout == B.KV_DEPTH_INDEXED:
                cdb.kv_copy_on_exit(rows, torch.tensor([it[1] for it in items], dtype=torch.int32, device=self.dev))
            lg = self.logits[:k] if self.record_logits else None
            with self._phase("coda"):
                cdb.boundary_coda_lmhead(rows, hin, self.tok_out[:k], lg)
            out = self.tok_out[:k].cpu().numpy()
            self.stats["coda_calls"] += 1
            cont = []
            for j, (s, depth, slot) in enumerate(items):
                coda_free.append(slot)
                sq = seqs[s]
                sq.depths.append(depth)
                sq.gates.append(sq.cur_gates)
                sq.cur_gates = []
                if self.record_states:
                    self.trace_states[(s, len(sq.tokens))] = states[j]
                if self.record_logits:
                    self.trace_logits[(s, len(sq.tokens))] = lg[j].cpu().numpy()
                r = finish_or_continue(s, out[j])
                if r is not None:
                    cont.append(r)
            start_tokens(cont)

        def run_recurrent(allow_refill):
            nonlocal rec
            if "decode_start" not in self.stats and not waiting and not future:   # every prompt processed: decode phase begins
                torch.cuda.synchronize(self.dev)
                self.stats["decode_start"] = time.perf_counter()
                self._mark_decode_start()
            # survivors are already at the front of h_rec in stable order; append refills (FIFO)
            n_keep = len(rec)
            take = []
            while allow_refill and ready and len(rec) < self.max_batch:
                s, slot = ready.pop(0)
                take.append(slot)
                ready_free.append(slot)
                rec.append([s, 1])
            if take:
                cdb.gather_rows(self.h_ready, torch.tensor(take, dtype=torch.int32, device=self.dev), None, len(take),
                                self.h_rec[n_keep:n_keep + len(take)])
            k = len(rec)
            if k == 0:
                return False
            sl = [live_slot[s] for s, _ in rec]
            pos = [position_of(seqs[s]) for s, _ in rec]
            dep = [r for _, r in rec]
            with self._phase("recurrent"):
                _run_step(self, k, sl, dep, pos, [self._slot(r) for r in dep], [forced_for(seqs[s]) for s, _ in rec])
            cnt = self.counts.cpu().numpy()
            ns, ne = int(cnt[0]), int(cnt[1])
            surv = self.surv_idx[:ns].cpu().numpy()
            ex = self.exit_idx[:ne].cpu().numpy()
            gv = self.gate_val[:k].cpu().numpy()
            self.stats["recurrent_steps"] += 1
            self.stats["row_steps"] += k
            self.stats["rows_hist"][(k - 1) // 32] += 1
            if self.record_ticks:
                self.stats["tick_rows"].append([(s, len(seqs[s].tokens), r) for s, r in rec])
            for i, (s, r) in enumerate(rec):
                seqs[s].cur_gates.append(float(gv[i]))
            if self.record_states:                                    # survivors now lead h_rec, exits fill h_exit
                hs, he = self.h_rec[:ns].cpu().numpy(), self.h_exit[:ne].cpu().numpy()
                for j, i in enumerate(surv):
                    self.trace_step_states[(rec[int(i)][0], len(seqs[rec[int(i)][0]].tokens), rec[int(i)][1])] = hs[j]
                for j, i in enumerate(ex):
                    self.trace_step_states[(rec[int(i)][0], len(seqs[rec[int(i)][0]].tokens), rec[int(i)][1])] = he[j]
            if ne:
                slots = [coda_free.pop() for _ in range(ne)]
                self.h_coda.index_copy_(0, torch.tensor(slots, dtype=torch.int64, device=self.dev), self.h_exit[:ne])
                for j, i in enumerate(ex):
                    s, r = rec[int(i)]
                    coda_q.append((s, r, slots[j]))
            rec = [[rec[int(i)][0], rec[int(i)][1] + 1] for i in surv]
            self.last_lists = (surv.copy(), ex.copy())
            return True

        while waiting or live_slot or future:
            if future:
                poll_arrivals()
                if not waiting and not live_slot:
                    time.sleep(min(1e-3, max(0.0, arrivals[future[0]] - now())))
                    continue
            if self.mode == "refill":
                runnable_other = bool(rec) or bool(ready) or (bool(waiting) and bool(free_slots))
                if coda_q and (len(coda_q) >= self.min_coda_batch or not runnable_other):
                    run_coda()
                elif waiting and free_slots and run_prefill():
                    pass
                elif not run_recurrent(True):
                    if coda_q:
                        run_coda()
                    else:
                        raise RuntimeError("scheduler stalled: KV pool too small for any waiting request")
            else:                               # no-refill and fixed-depth: prelude, core until empty, coda
                if not rec and not ready and not coda_q:
                    if not (waiting and free_slots and run_prefill()):
                        if not live_slot:
                            raise RuntimeError("scheduler stalled: KV pool too small for any waiting request")
                elif rec or ready:
                    run_recurrent(allow_refill=not rec)
                    while rec:
                        run_recurrent(False)
                else:
                    run_coda()
                    while waiting and free_slots and run_prefill():
                        pass
        torch.cuda.synchronize(self.dev)
        self.stats["end"] = time.perf_counter()
        if self.time_device:
            self._collect_device_time()
        return {"tokens": [np.asarray(s.tokens, dtype=np.int32) for s in seqs],
                "depths": [np.asarray(s.depths, dtype=np.int32) for s in seqs],
                "gates": [s.gates for s in seqs]}


def kv_footprint(dims, n_slots: int, split_kv: bool = True) -> tuple[int, int]:
    """KV bytes per cached token: (in use, reserved by the engine's page pools).  In use is what the paper's
    Table 1 counts: one K and one V vector per layer, the core layers once per depth slot.  With a page space of
    their own for the prelude and coda layers (the engines' default for more than one slot) exactly that is
    reserved.  With ONE page space shared by all layers every (sequence, slot) pair owns pages in ALL layers, so the
    boundary layers' share of the pages of slots > 0 stays empty: reserved >= in use."""
    eb = 4 if dims.dtype == "fp32" else 2
    per_layer = 2 * dims.H * dims.Dh * eb
    used = (dims.L_pre + dims.L_coda + dims.L_core * n_slots) * per_layer
    reserved = used if split_kv else (dims.L_pre + dims.L_coda + dims.L_core) * n_slots * per_layer
    return used, reserved


def _bucket(k: int, cap: int) -> int:
    return min(cap, (k + 31) // 32 * 32)


def _static_rows(eng: "Engine", nb: int) -> B.Rows:
    d = eng.desc_dev
    # rows beyond the device-side count d[5, 0] are pads: a bucket's graph serves every batch size up to nb
    return B.Rows(d[0, :nb], d[2, :nb], eng.page_table, loop_depth=d[1, :nb], kv_slot=d[3, :nb], forced_exit=d[4, :nb],
                  n_rows_dev=d[5, :1])


def _step_body(eng: "Engine", rows: B.Rows, nb: int):
    """compaction lists, loop step, survivor / exit gathers; survivors end up at the front of h_rec"""
    c, hx = eng.cdb, eng.h_rec[:nb]
    if eng.lookahead:                        # the stored signal is the previous step's: lists before the step
        c.compact(rows, eng.surv_idx, eng.exit_idx, eng.counts)
        c.loop_step(rows, hx, eng.gate_val, eng.fire)
        c.gather_rows(hx, eng.surv_idx, eng.counts[0:1], nb, eng.h_tmp)
        c.gather_rows(hx, eng.exit_idx, eng.counts[1:2], nb, eng.h_exit)
    else:
        c.loop_step(rows, hx, eng.gate_val, eng.fire)
        c.compact(rows, eng.surv_idx, eng.exit_idx, eng.counts, h_src=hx, h_next=eng.h_tmp, h_exit=eng.h_exit)
    hx.copy_(eng.h_tmp[:nb])


def _run_step(eng: "Engine", k: int, seq, depth, pos, slot, forced):
    """One recurrent step over the first k rows of h_rec (descriptor given as host sequences)."""
    nb = _bucket(k, eng.max_rows) if eng.use_graphs else k
    dh = eng.desc_host
    dh[0, :k] = torch.as_tensor(np.asarray(seq, dtype=np.int32))
    dh[1, :k] = torch.as_tensor(np.asarray(depth, dtype=np.int32))
    dh[2, :k] = torch.as_tensor(np.asarray(pos, dtype=np.int32))
    dh[3, :k] = torch.as_tensor(np.asarray(slot, dtype=np.int32))
    dh[4, :k] = torch.as_tensor(np.asarray(forced, dtype=np.int32))
    dh[5, 0] = k
    if not eng.use_graphs:
        eng.desc_dev.copy_(dh, non_blocking=True)
        _step_body(eng, _static_rows(eng, nb), nb)
        return
    if nb not in eng.graphs:
        # Warm-up with a live count of zero (every row a pad), then capture.  Pads touch neither the KV pool nor the
        # gate state, but the body ends by moving the (empty) survivor list to the front of h_rec, which would
        # overwrite the rows waiting there for this very step: keep them aside.
        saved = eng.h_rec[:nb].clone()
        eng.desc_dev[5, 0].fill_(0)
        rows = _static_rows(eng, nb)
        _step_body(eng, rows, nb)
        torch.cuda.synchronize(eng.dev)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            _step_body(eng, rows, nb)
        eng.h_rec[:nb].copy_(saved)
        eng.graphs[nb] = (g, rows)
    eng.desc_dev.copy_(dh, non_blocking=True)
    eng.graphs[nb][0].replay()
