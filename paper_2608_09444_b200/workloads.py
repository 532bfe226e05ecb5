"""Synthetic benchmark workloads for the CDB hot path, built from `synth` on one GPU.

LoopStepWorkload is the Ouro-1.4B-shaped single loop-step microbenchmark: a ragged batch of
(sequence, loop depth) rows with paged KV, and one "step" = exit-flag compaction, the loop step
over all core layers with the exit gate, the survivor / exit row gathers, the LM head + greedy
sampling for the exited rows and the embedding of the sampled tokens.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B
from . import synth


class LoopStepWorkload:
    def __init__(self, dims=synth.OURO_1P4B, n_rows=256, seed=1, ctx_lo=128, ctx_hi=2048, permute=True,
                 p_fire=0.3, device="cuda:0", flags=0, weight_std=None):
        self.dims, self.n_rows, self.dev = dims, n_rows, torch.device(device)
        torch.cuda.set_device(self.dev)
        self.weights = synth.make_weights(dims, seed, device=str(self.dev), std=weight_std or synth.width_scaled_std(dims.d), gate_std=2.0 / np.sqrt(dims.d))
        self.rows_np = synth.make_step_rows(n_rows, dims.R, seed, ctx_lo, ctx_hi, p_fire)
        self.ctx = self.rows_np["position"].astype(np.int64) + 1
        self.table_np, self.n_pages = synth.make_page_table(self.ctx, dims.page_size, seed, permute=permute)
        self.max_position = self.table_np.shape[1] * dims.page_size
        self.cdb = B.Cdb(dims, self.weights, max_rows=n_rows, max_seqs=n_rows, max_position=self.max_position,
                         gate_kind=B.GATE_SIGMOID_CDF, q_or_eps=0.5, flags=flags)
        dt = torch.float32 if dims.dtype == "fp32" else torch.bfloat16
        self.pool = torch.empty(synth.kv_pool_shape(dims, self.n_pages), dtype=dt, device=self.dev)
        synth.fill_kv_pool(self.pool, seed + 1000)
        self.cdb.kv_bind(self.pool)
        gen = torch.Generator(device=self.dev)
        gen.manual_seed(seed + 2000)
        self.h_in = torch.randn((n_rows, dims.d), generator=gen, device=self.dev, dtype=torch.float32)

        # host (pinned) copies of everything a step takes in and gives back
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
        self.host_in = {k: pin(self.rows_np[k]) for k in ("seq_id", "loop_depth", "position", "kv_slot", "forced_exit", "fire_prev")}
        self.host_in["page_table"] = pin(self.table_np)
        self.host_in["h"] = self.h_in.cpu().pin_memory()
        i32 = dict(dtype=torch.int32, device=self.dev)
        self.d_in = {k: torch.empty_like(v, device=self.dev) for k, v in self.host_in.items()}
        for k, v in self.host_in.items():
            self.d_in[k].copy_(v)
        self.rows = B.Rows(self.d_in["seq_id"], self.d_in["position"], self.d_in["page_table"],
                           loop_depth=self.d_in["loop_depth"], kv_slot=self.d_in["kv_slot"],
                           forced_exit=self.d_in["forced_exit"])
        self.h = torch.empty_like(self.h_in)
        self.h_next = torch.empty_like(self.h_in)
        self.h_exit = torch.empty_like(self.h_in)
        self.h_new = torch.empty_like(self.h_in)
        self.surv_idx = torch.zeros(n_rows, **i32)
        self.exit_idx = torch.zeros(n_rows, **i32)
        self.counts = torch.zeros(2, **i32)
        self.gate_val = torch.zeros(n_rows, dtype=torch.float32, device=self.dev)
        self.fire = torch.zeros(n_rows, dtype=torch.uint8, device=self.dev)
        self.tokens = torch.zeros(n_rows, **i32)
        self.host_out = {"surv_idx": torch.zeros(n_rows, dtype=torch.int32).pin_memory(),
                         "exit_idx": torch.zeros(n_rows, dtype=torch.int32).pin_memory(),
                         "counts": torch.zeros(2, dtype=torch.int32).pin_memory(),
                         "gate_val": torch.zeros(n_rows, dtype=torch.float32).pin_memory(),
                         "tokens": torch.zeros(n_rows, dtype=torch.int32).pin_memory()}
        # the exit list depends only on the descriptor and the previous step's signal: compute it once to
        # size the boundary calls (the per-step kernels still recompute it every step)
        self.cdb.compact(self.rows, self.surv_idx, self.exit_idx, self.counts, fire_prev=self.d_in["fire_prev"])
        torch.cuda.synchronize(self.dev)
        self.n_surv, self.n_exit = (int(v) for v in self.counts.cpu())
        ex = self.exit_idx[:self.n_exit].cpu().numpy()
        self.exit_seq = torch.tensor(self.rows_np["seq_id"][ex], **i32)
        self.exit_pos = torch.tensor(self.rows_np["position"][ex], **i32)
        self.exit_rows = B.Rows(self.exit_seq, self.exit_pos, self.d_in["page_table"]) if self.n_exit else None

    # ---- what one step must move (bytes) and compute (flops)
    def algorithmic(self):
        dm = self.dims
        eb = 4 if dm.dtype == "fp32" else 2
        w = dm.L_core * (4 * dm.d * dm.d + 3 * dm.d * dm.F) * eb
        kv_tok = 2 * dm.H * dm.Dh * eb
        kv_read = int(self.ctx.sum()) * dm.L_core * kv_tok
        kv_write = self.n_rows * dm.L_core * kv_tok
        lm = dm.V * dm.d * eb if self.n_exit else 0
        return {"weights": w, "kv_read": kv_read, "kv_write": kv_write, "lm_head": lm,
                "total": w + kv_read + kv_write + lm,
                "attention_per_launch": int(self.ctx.sum()) * kv_tok,
                "gemm_flops": 2 * self.n_rows * dm.L_core * (4 * dm.d * dm.d + 3 * dm.d * dm.F)}

    def step_resident(self, stream=None):
        """One pass of the hot path with every input already in device memory."""
        c = self.cdb
        self.h.copy_(self.h_in)
        c.compact(self.rows, self.surv_idx, self.exit_idx, self.counts, fire_prev=self.d_in["fire_prev"], stream=stream)
        c.loop_step(self.rows, self.h, self.gate_val, self.fire, stream=stream)
        c.gather_rows(self.h, self.surv_idx, self.counts[0:1], self.n_rows, self.h_next, stream=stream)
        c.gather_rows(self.h, self.exit_idx, self.counts[1:2], self.n_rows, self.h_exit, stream=stream)
        if self.n_exit:
            c.boundary_coda_lmhead(self.exit_rows, self.h_exit[:self.n_exit], self.tokens[:self.n_exit], stream=stream)
            c.boundary_embed(self.tokens[:self.n_exit], self.exit_rows, self.h_new[:self.n_exit], stream=stream)

    def step_e2e(self):
        """The same pass through host buffers: descriptor, page table, previous signal and row states
        go host -> device, index lists, counts, gate values and sampled tokens come back."""
        for k, v in self.host_in.items():
            self.d_in[k].copy_(v, non_blocking=True)
        self.h_in.copy_(self.d_in["h"])
        self.step_resident()
        self.host_out["surv_idx"].copy_(self.surv_idx, non_blocking=True)
        self.host_out["exit_idx"].copy_(self.exit_idx, non_blocking=True)
        self.host_out["counts"].copy_(self.counts, non_blocking=True)
        self.host_out["gate_val"].copy_(self.gate_val, non_blocking=True)
        self.host_out["tokens"].copy_(self.tokens, non_blocking=True)
        torch.cuda.current_stream().synchronize()

    def h2d_bytes(self):
        return int(sum(v.numel() * v.element_size() for v in self.host_in.values()))

    def d2h_bytes(self):
        return int(sum(v.numel() * v.element_size() for v in self.host_out.values()))

    # ---- host copies of what the CPU oracle needs for a subset of rows
    def oracle_inputs(self, row_ids):
        """Per row: input state, context length, loop depth and dense per-layer K, V gathered from the
        row's pages (fp32 numpy)."""
        dm = self.dims
        out = []
        for i in row_ids:
            c = int(self.ctx[i])
            n_pages = (c + dm.page_size - 1) // dm.page_size
            ids = torch.from_numpy(self.table_np[i, :n_pages].astype(np.int64)).to(self.dev)
            pages = self.pool[:, ids].float().cpu().numpy()            # [L][n_pages][2][H][16][Dh]
            out.append({"row": int(i), "ctx": c, "depth": int(self.rows_np["loop_depth"][i]),
                        "h": self.h_in[i].cpu().numpy(), "pages": pages,
                        "table": np.arange(n_pages)})
        return out
