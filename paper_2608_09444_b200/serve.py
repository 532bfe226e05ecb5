"""Online serving on synthetic traffic (the config-5 analogue of the paper's section 6 serving experiment).

Requests arrive as a Poisson process; prompt and output lengths are log-normal (median 512 / 256 tokens,
sigma 0.8, clipped to [4, 4096] / [4, 2048]), standing in for the ShareGPT / Alpaca replays the paper
uses.  Each request's normalised latency is (time its last token reached the host - arrival time) /
output length; the report gives its mean, p50 and p99 per arrival rate, next to throughput, for standard
continuous batching (every token loops r_max times) and continuous depth batching with refill.

    python -m paper_2608_09444_b200.serve --model ouro --rates 4,8,16 --requests 300

The engines run against the wall clock, so a run lasts requests / rate seconds plus the drain.

Under torchrun (one rank per GPU) every rank is a full replica with its own page pool and scheduler; a
front-end rule (least reserved KV tokens at arrival, `dist.route_least_loaded`) assigns each request to a
replica, the ranks serve their shares against the same clock, and rank 0 merges the per-request times.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding as B
from . import dist as D
from . import synth
from .engine import Engine
from .engine_async import PipelinedEngine
from .offline import calibrate_gate_bias


def make_requests(n, rate, seed, vocab, prompt_median=512, prompt_cap=4096, out_median=256, out_cap=2048):
    """Seeded request trace: arrival times (s), prompts (token ids), output lengths."""
    arrivals = synth.poisson_arrivals(n, rate, seed)
    p_len = synth.lognormal_lengths(n, seed + 1, prompt_median, prompt_cap)
    t_len = synth.lognormal_lengths(n, seed + 2, out_median, out_cap)
    rng = np.random.default_rng(seed + 3)
    prompts = [rng.integers(0, vocab, size=int(m), dtype=np.int32) for m in p_len]
    return arrivals, prompts, [int(t) for t in t_len]


def summarize(arrivals, out_lens, stats):
    fin = np.asarray(stats["finish_s"], dtype=np.float64)
    first = np.asarray(stats["first_token_s"], dtype=np.float64)
    lat = (fin - arrivals) / np.asarray(out_lens, dtype=np.float64)
    span = float(fin.max() - arrivals[0])
    return {"normalized_latency_s_per_token": {"mean": float(lat.mean()), "p50": float(np.percentile(lat, 50)),
                                               "p99": float(np.percentile(lat, 99))},
            "time_to_first_token_s": {"mean": float((first - arrivals).mean()), "p99": float(np.percentile(first - arrivals, 99))},
            "generated_tokens_per_s": float(np.sum(out_lens) / span), "span_s": span,
            "recurrent_steps": stats["recurrent_steps"], "row_steps": stats["row_steps"],
            "prefill_calls": stats["prefill_calls"], "coda_calls": stats["coda_calls"]}


def merge_replicas(parts, n_requests):
    """Per-request time stamps and summed counters of all replicas, in request order."""
    merged = {"finish_s": [None] * n_requests, "first_token_s": [None] * n_requests,
              "recurrent_steps": 0, "row_steps": 0, "prefill_calls": 0, "coda_calls": 0}
    for p in parts:
        for j, i in enumerate(p["ids"]):
            merged["finish_s"][i], merged["first_token_s"][i] = p["finish_s"][j], p["first_token_s"][j]
        for k, v in p["counters"].items():
            merged[k] += v
    return merged


def run(dims, weights, arrivals, prompts, out_lens, *, mode, pipelined, gate_kind, q_or_eps=0.5, forced_depths=None,
        max_batch=256, max_live=320, pool_tokens=400000, min_coda_batch=1, max_prefill_rows=4096,
        admit_min=1, admit_wait_s=0.0, prefill_priority=0, eager_refill=True, device="cuda:0"):
    max_len = max(len(p) + t for p, t in zip(prompts, out_lens))
    pages = (pool_tokens + dims.page_size - 1) // dims.page_size
    extra = {"prefill_priority": prefill_priority, "eager_refill": eager_refill} if pipelined else {}
    eng = (PipelinedEngine if pipelined else Engine)(
        dims, weights, **extra, max_batch=max_batch, max_live=max_live, max_len=max_len, n_pages=pages, gate_kind=gate_kind,
        q_or_eps=q_or_eps, lookahead=True, mode=mode, min_coda_batch=min_coda_batch,
        max_prefill_rows=max(max_prefill_rows, max(len(p) for p in prompts)), record_ticks=False,
        admit_min=admit_min, admit_wait_s=admit_wait_s, device=device)
    res = eng.generate(prompts, out_lens, forced_depths=forced_depths, arrivals=arrivals)
    out = summarize(arrivals, out_lens, eng.stats)
    out["finish_s"], out["first_token_s"] = list(eng.stats["finish_s"]), list(eng.stats["first_token_s"])
    out["mode"] = mode + ("_pipelined" if pipelined else "")
    out["recurrent_steps_by_rows_32"] = list(eng.stats["rows_hist"])      # this replica's steps by row count, 32-row bins
    out["status"] = eng.cdb.poll_status()
    d = np.concatenate([x for x in res["depths"] if len(x)]) if any(len(x) for x in res["depths"]) else np.zeros(0)
    out["mean_depth"] = float(d.mean()) if d.size else float(dims.R)
    eng.cdb.destroy()
    del eng
    torch.cuda.empty_cache()
    return out, res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--model", default="ouro", choices=["ouro", "huginn"])
    ap.add_argument("--rates", default="4,8,16")
    ap.add_argument("--requests", type=int, default=300)
    ap.add_argument("--max-batch", type=int, default=256)
    ap.add_argument("--max-live", type=int, default=320)
    ap.add_argument("--pool-tokens", type=int, default=400000)
    ap.add_argument("--modes", default="cb_pipelined,refill_pipelined", help="cb, refill, no_refill (synchronous engine); cb_pipelined, refill_pipelined")
    ap.add_argument("--min-coda-batch", type=int, default=0, help="exits gathered before a coda call (0: 1 for ouro, 8 for huginn; the offline runs use 32 for huginn)")
    ap.add_argument("--admit-min", type=int, default=1, help="hold arrived requests until this many wait ...")
    ap.add_argument("--admit-wait-ms", type=float, default=0.0, help="... or the oldest has waited this long")
    ap.add_argument("--prefill-priority", type=int, default=0, choices=[0, -1],
                    help="pipelined engine: CUDA stream priority of prompt processing (0 = below the decode streams, -1 = level with them)")
    ap.add_argument("--no-eager-refill", action="store_true",
                    help="pipelined engine: always run the boundary stages beside the next step (tokens rejoin one step late)")
    ap.add_argument("--first-rate-index", type=int, default=0,
                    help="position of the first of --rates in the sweep it belongs to (the trace seed follows the position): "
                         "--rates 2 --first-rate-index 5 repeats the last trace of --rates 64,32,16,8,4,2")
    args = ap.parse_args()
    known = {"cb", "refill", "no_refill", "cb_pipelined", "refill_pipelined"}
    if not set(args.modes.split(",")) <= known:
        raise SystemExit(f"--modes takes a comma-separated subset of {sorted(known)}")
    rank, local_rank, world = D.env_rank()
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl")
    torch.cuda.set_device(local_rank)
    dims, seed = (synth.OURO_1P4B, 4) if args.model == "ouro" else (synth.HUGINN_3P5B, 5)
    w = synth.make_weights(dims, seed, device=f"cuda:{local_rank}", std=synth.width_scaled_std(dims.d), gate_std=2.0 / np.sqrt(dims.d))
    report = {"model": args.model, "requests": args.requests, "runs": []}
    if args.model == "ouro":
        gate_kind = B.GATE_SIGMOID_CDF
        cal = list(synth.make_prompts(16, 256, dims.V, seed))
        report["b_gate"] = calibrate_gate_bias(dims, w, cal, 24, 2.5)
    else:
        gate_kind = B.GATE_NONE
    for ri, rate in enumerate((float(x) for x in args.rates.split(",")), start=args.first_rate_index):
        arrivals, prompts, out_lens = make_requests(args.requests, rate, seed + 10 * ri, dims.V)
        forced = None
        if args.model == "huginn":       # replayed exit depths: truncated geometric, mean 12
            forced = [list(synth.forced_exit_depths((1, max(t - 1, 1)), seed + 100 + i, 12.0, dims.R)[0]) for i, t in enumerate(out_lens)]
        # this replica's share of the trace (all of it on one GPU)
        owner = D.route_least_loaded(arrivals, [len(p) + t for p, t in zip(prompts, out_lens)], out_lens, world)
        mine = [i for i in range(args.requests) if owner[i] == rank]
        for mode in args.modes.split(","):
            pipelined = mode.endswith("_pipelined")
            m = mode.replace("_pipelined", "")
            fixed = m == "cb" and pipelined                  # continuous batching on the pipelined engine: every token replays depth R
            if fixed:
                m = "refill"
            if world > 1:
                torch.distributed.barrier()           # the replicas start their clocks together
            out, _ = run(dims, w, arrivals[mine], [prompts[i] for i in mine], [out_lens[i] for i in mine], mode=m,
                         pipelined=pipelined, gate_kind=B.GATE_NONE if fixed else gate_kind,
                         forced_depths=[[dims.R] * max(out_lens[i] - 1, 1) for i in mine] if fixed else
                         None if (m == "cb" or forced is None) else [forced[i] for i in mine],
                         max_batch=args.max_batch, max_live=args.max_live,
                         pool_tokens=args.pool_tokens, min_coda_batch=args.min_coda_batch or (1 if args.model == "ouro" else 8),
                         admit_min=args.admit_min, admit_wait_s=args.admit_wait_ms * 1e-3,
                         prefill_priority=args.prefill_priority, eager_refill=not args.no_eager_refill, device=f"cuda:{local_rank}")
            out["mode"] = mode
            parts = D.gather_objects({"ids": mine, "finish_s": out.pop("finish_s"), "first_token_s": out.pop("first_token_s"),
                                      "counters": {k: out[k] for k in ("recurrent_steps", "row_steps", "prefill_calls", "coda_calls")}})
            if rank == 0:
                merged = merge_replicas(parts, args.requests)
                out.update(summarize(arrivals, out_lens, merged))
                out["rate_req_per_s"], out["replicas"] = rate, world
                report["runs"].append(out)
                print(json.dumps(out), flush=True)
    if rank == 0:
        print(json.dumps(report))


if __name__ == "__main__":
    main()
