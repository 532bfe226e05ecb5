"""Benchmark of the CDB hot path: the Ouro-1.4B-shaped single loop-step microbenchmark (256 ragged
rows, loop depths 1..4, contexts 128..2048, paged KV with 16-token pages, bf16, random init).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl cdb|reference]

Prints one JSON line.  `value` is token-loop-steps/s with inputs resident in HBM; `e2e` is the same
metric through host buffers; `roofline` is the paged-attention kernel (the step's dominant kernel)
against the measured HBM copy bandwidth; `cpu_baseline` is the CPU oracle timed on a bounded sample.
With --impl reference the CPU oracle itself is timed (rank 0 only).  N > 1 runs one replica per
GPU on its own rows (sequences are independent: no data-path collective), weak scaling.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "token_loop_steps_per_s"
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes the attention kernel moved per algorithmic byte in its ncu capture (2.3299 GB read + 7.2 MB written
# for 2.3133 GB of KV, same rows and page tables as the default workload, one core layer).
NCU_TRAFFIC_PER_ALGORITHMIC_BYTE = (2.3299e9 + 7.2e6) / 2.3133e9


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples of one GPU while a region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])), mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def build_oracle(dims, weights_np):
    """The CPU oracle for the core layers alone (the microbenchmark has no prelude or coda)."""
    import numpy as np
    from oracle import cdb_oracle as O
    wn = {k: weights_np[k] for k in ("W_qkv", "W_o", "W_gate", "W_up", "W_down", "g_attn", "g_mlp", "w_gate", "b_gate")}
    wn["g_final"] = np.ones(dims.d, dtype=np.float32)
    return O.Oracle(dims.replace(L_pre=0, L_coda=0), wn, gate_kind=O.GATE_SIGMOID_CDF, q_or_eps=0.5)


def densify(dims, items):
    """Dense per-layer K, V of each sampled row from its pages (untimed set-up)."""
    from oracle import cdb_oracle as O
    for it in items:
        kv = [O.gather_pages(it["pages"][l], it["table"], it["ctx"]) for l in range(dims.L_core)]
        it["K"], it["V"] = [k for k, _ in kv], [v for _, v in kv]
        del it["pages"]
    return items


def oracle_sample(wl, row_ids):
    """The CPU oracle and its inputs for a few rows of the GPU arm's workload (untimed set-up)."""
    from paper_2608_09444_b200 import synth
    dm = wl.dims
    core = {k: v[dm.L_pre:dm.L_pre + dm.L_core] if v.dim() >= 2 and v.shape[0] == dm.L else v for k, v in wl.weights.items()}
    wn = synth.weights_to_numpy({k: core[k] for k in ("W_qkv", "W_o", "W_gate", "W_up", "W_down", "g_attn", "g_mlp", "w_gate", "b_gate")})
    items = [dict(it, pages=it["pages"][dm.L_pre:dm.L_pre + dm.L_core]) for it in wl.oracle_inputs(row_ids)]
    return build_oracle(dm, wn), densify(dm, items)


def host_sample(dims, n_rows, seed, ctx_lo, ctx_hi, row_ids):
    """The reference arm's inputs, made on the host alone from the same recipe as the GPU arm's workload
    (same seeded row descriptor; weights, KV pages and row states are fresh draws of the same distributions,
    since the GPU arm fills those with the device's generator).  Loads nothing of the CUDA library."""
    import numpy as np
    import torch
    from paper_2608_09444_b200 import synth
    gen = torch.Generator().manual_seed(seed)
    grid = (lambda t: t.to(torch.bfloat16).to(torch.float32)) if dims.dtype == "bf16" else (lambda t: t)
    normal = lambda shape, std: grid(torch.empty(shape, dtype=torch.float32).normal_(0.0, std, generator=gen)).numpy()
    d, F, L = dims.d, dims.F, dims.L_core
    wn = {"W_qkv": normal((L, 3 * d, d), 0.02), "W_o": normal((L, d, d), 0.02), "W_gate": normal((L, F, d), 0.02),
          "W_up": normal((L, F, d), 0.02), "W_down": normal((L, d, F), 0.02),
          "g_attn": np.ones((L, d), np.float32), "g_mlp": np.ones((L, d), np.float32),
          "w_gate": normal((d,), 2.0 / np.sqrt(d)), "b_gate": np.zeros(1, np.float32)}
    rows = synth.make_step_rows(n_rows, dims.R, seed, ctx_lo, ctx_hi)
    items = []
    for i in row_ids:
        c = int(rows["position"][i]) + 1
        n_pages = (c + dims.page_size - 1) // dims.page_size
        items.append({"row": int(i), "ctx": c, "depth": int(rows["loop_depth"][i]),
                      "h": torch.empty(d).normal_(0.0, 1.0, generator=gen).numpy(),
                      "pages": normal((L, n_pages, 2, dims.H, dims.page_size, dims.Dh), 1.0),
                      "table": np.arange(n_pages)})
    return build_oracle(dims, wn), densify(dims, items)


def oracle_step(orc, items):
    t0 = time.perf_counter()
    for it in items:
        orc.loop_step_row(it["h"], it["ctx"] - 1, it["depth"], it["K"], it["V"])
    return time.perf_counter() - t0


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        return len(os.sched_getaffinity(0))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cdb", choices=["cdb", "reference"])
    ap.add_argument("--model", default="ouro", choices=["ouro", "huginn"], help="layer shapes of the step (the headline metric is quoted on ouro)")
    ap.add_argument("--rows", type=int, default=256)
    ap.add_argument("--ctx-lo", type=int, default=128)
    ap.add_argument("--ctx-hi", type=int, default=2048)
    ap.add_argument("--layers", type=int, default=0, help="override the core layer count (small ncu captures only)")
    ap.add_argument("--contiguous-pages", action="store_true", help="ascending physical pages instead of a random permutation")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--simt-gemm", action="store_true", help="run projections on the plain-FMA cross-check kernel")
    ap.add_argument("--cta-pairs", action="store_true", help="projections on 128 rows and more as CTA pairs (default: from 512 rows on)")
    ap.add_argument("--two-stream", action="store_true", help="split the step into two half-batches on two streams (experimental)")
    ap.add_argument("--workspace-parts", action="store_true", help="split-K parts through a workspace instead of in-cluster sums (cross-check flow)")
    ap.add_argument("--sm-partition", action="store_true", help="two half-batches with the SMs split between attention and projections (experimental)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "cdb" else args.warmup

    from paper_2608_09444_b200 import dist as D
    rank, local_rank, world = D.env_rank()
    if args.impl == "reference" and rank != 0:
        return 0

    from paper_2608_09444_b200 import synth

    base = synth.OURO_1P4B if args.model == "ouro" else synth.HUGINN_3P5B
    dims = base if args.layers <= 0 else base.replace(L_core=args.layers)
    workload = f"{'ouro-1.4b' if args.model == 'ouro' else 'huginn-3.5b'}-shaped loop step, {args.rows} rows, depth U{{1..{dims.R}}}, context U{{{args.ctx_lo}..{args.ctx_hi}}}, 16-token pages"
    config = {"workload": workload, "rows": args.rows, "core_layers": dims.L_core, "page_table": "contiguous" if args.contiguous_pages else "random permutation",
              "l2": "inputs larger than L2 (each step streams the whole KV pool and all core weights)"}

    if args.impl == "reference":
        # host only: the oracle (NumPy) on inputs drawn on the host; neither the CUDA library nor a GPU is touched
        sample_rows = [0, 1]
        orc, items = host_sample(dims, args.rows, D.rank_seed(1, rank), args.ctx_lo, args.ctx_hi, sample_rows)
        for _ in range(args.warmup):
            oracle_step(orc, items)
        t = sum(oracle_step(orc, items) for _ in range(args.steps))
        value = len(items) * args.steps / t
        print(json.dumps({"impl": "reference", "metric": METRIC, "value": value, "unit": "token-loop-steps/s",
                          "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
                          "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True, "scaling": "weak",
                          "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config,
                          "cpu_baseline": {"value": value, "unit": "token-loop-steps/s", "cores": blas_threads(), "kind": "oracle",
                                           "sample": f"rows {sample_rows} of the workload per step (one loop step each, serial)"},
                          "e2e": {"value": value, "unit": "token-loop-steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                          "gpu_launches": 0}))
        return 0

    import numpy as np
    import torch
    import __graft_entry__
    if local_rank == 0:
        __graft_entry__.build()
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl")
    torch.cuda.set_device(local_rank)
    from paper_2608_09444_b200 import binding as B
    from paper_2608_09444_b200.workloads import LoopStepWorkload
    wl = LoopStepWorkload(dims, n_rows=args.rows, seed=D.rank_seed(1, rank), ctx_lo=args.ctx_lo, ctx_hi=args.ctx_hi,
                          permute=not args.contiguous_pages, device=f"cuda:{local_rank}", flags=(B.FLAG_SIMT_GEMM if args.simt_gemm else 0) | (B.FLAG_TWO_STREAM if args.two_stream else 0) | (B.FLAG_WORKSPACE_PARTS if args.workspace_parts else 0) | (B.FLAG_SM_PARTITION if args.sm_partition else 0) | (B.FLAG_CTA_PAIRS if args.cta_pairs else 0))
    alg = wl.algorithmic()
    cores = len(os.sched_getaffinity(0))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        barrier()
        return D.max_over_ranks(e0.elapsed_time(e1), device=f"cuda:{local_rank}")

    for _ in range(args.warmup):
        wl.step_resident()
    sampler = ClockSampler(local_rank)
    wl.cdb.profile_begin(False)                      # launch counter only: event records between kernels would
    if rank == 0:                                    # break the programmatic launch chain and perturb the timing
        sampler.start()
    ms = timed(wl.step_resident, args.steps)
    clocks = sampler.stop() if rank == 0 else {}
    launches = wl.cdb.profile_read()["launches"]
    # second pass of the same K steps with a CUDA-event pair around every attention / projection launch (on the
    # launching stream): per-kernel durations for the roofline
    wl.cdb.profile_begin(True)
    ms_prof = timed(wl.step_resident, args.steps)
    prof = wl.cdb.profile_read()
    wl.cdb.profile_begin(False)
    assert wl.cdb.poll_status() == 0
    for _ in range(2):
        wl.step_e2e()
    ms_e2e = timed(wl.step_e2e, args.steps)

    if rank != 0:
        return 0
    peak, peak_kind = measured_peak()
    ms_step = ms / args.steps
    att = prof["attention"]
    att_ms = att["ms"] / max(att["count"], 1)
    # a step's attention launches together read the rows' contexts once per layer (one launch per layer, or two
    # half-batch launches): bytes per launch = bytes of all launches / number of launches
    att_bytes_per_launch = alg["attention_per_launch"] * dims.L_core * args.steps / max(att["count"], 1)
    achieved = att_bytes_per_launch / (att_ms * 1e-3) / 1e9 if att_ms > 0 else 0.0
    default_workload = args.model == "ouro" and args.rows == 256 and args.ctx_lo == 128 and args.ctx_hi == 2048 and not args.contiguous_pages
    out = {"metric": METRIC, "value": world * args.rows / (ms_step * 1e-3), "unit": "token-loop-steps/s",
           "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step,
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
           "config": config,
           "hbm_step": {"algorithmic_bytes": alg["total"], "achieved_gbs": alg["total"] / (ms_step * 1e-3) / 1e9,
                        "frac_of_measured_copy_peak": alg["total"] / (ms_step * 1e-3) / 1e9 / peak,
                        "frac_of_nominal_8tbs": alg["total"] / (ms_step * 1e-3) / 1e9 / 8000.0},
           "roofline": {"kernel": "attn_split_kernel (paged decode attention)", "bound": "hbm", "achieved": achieved,
                        "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                        "traffic": NCU_TRAFFIC_PER_ALGORITHMIC_BYTE * att_bytes_per_launch if default_workload else None,
                        "traffic_source": "ncu dram__bytes_read.sum + dram__bytes_write.sum of this kernel on the same rows with one core layer (summary kept under profiles/): 2.3371 GB per launch for 2.3133 GB algorithmic",
                        "launches": att["count"], "avg_launch_ms": att_ms,
                        "algorithmic_bytes_per_launch": att_bytes_per_launch},
           "kernel_time_ms_per_step": {"attention": att["ms"] / args.steps, "projections": prof["linear"]["ms"] / args.steps},
           "e2e": {"value": world * args.rows / (ms_e2e / args.steps * 1e-3), "unit": "token-loop-steps/s",
                   "h2d_bytes_per_step": wl.h2d_bytes(), "d2h_bytes_per_step": wl.d2h_bytes()},
           "gpu_launches": launches, "clocks": clocks,
           "profiled_pass": {"ms_per_step": ms_prof / args.steps, "note": "same K steps repeated with CUDA-event pairs around each attention and projection launch; roofline and kernel_time_ms_per_step come from this pass"}}
    if args.no_cpu_baseline or world > 1:
        out["cpu_baseline"] = None
    else:
        sample_rows = list(range(min(16, args.rows)))
        orc, items = oracle_sample(wl, sample_rows)
        t, passes = 0.0, 0
        while t < 10.0 and passes < 8:                 # about 10-30 s of CPU work in whole passes over the sample
            t += oracle_step(orc, items)
            passes += 1
        out["cpu_baseline"] = {"value": len(items) * passes / t, "unit": "token-loop-steps/s", "cores": blas_threads(), "kind": "oracle",
                               "sample": f"one loop step of rows 0..{len(items) - 1} of the workload, each row alone, {passes} passes, {t:.1f} s",
                               "host_cores": cores}
    print(json.dumps(out))
    return 0


if __name__ == "__main__":
    sys.exit(main())
