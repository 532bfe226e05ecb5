"""Offline adaptive decode on synthetic prompts (the paper's offline-throughput setting, section 5.2): all
requests known up front, prompts processed first, then decode under continuous depth batching.  Reports
generated tokens/s of the decode phase, token-loop-steps/s, and the ratio of an adaptive run to the
fixed-depth run (standard continuous batching: every token loops R times) next to the FLOP bound of Eq. 2.

    python -m paper_2608_09444_b200.offline --model ouro --seqs 512 --prompt 256 --tokens 512
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding as B
from . import synth
from .engine import Engine
from .engine_async import PipelinedEngine


def flop_bound(dims, mean_depth):
    """Eq. 2: (F0 + R Fr) / (F0 + dbar Fr), F0 = boundary layers + LM head, Fr = one core application."""
    per_layer = 4 * dims.d * dims.d + 3 * dims.d * dims.F
    f0 = ((dims.L_pre + dims.L_coda) * per_layer + dims.V * dims.d) / (dims.L_core * per_layer)
    return (f0 + dims.R) / (f0 + mean_depth)


def run(dims, weights, prompts, T, *, mode, gate_kind, q_or_eps=0.5, forced_depths=None, max_batch=None, max_live=None,
        min_coda_batch=1, max_prefill_rows=4096, pipelined=False, use_graphs=True, time_device=False, kv_layout=B.KV_SHARED,
        eager_refill=True):
    n, P = len(prompts), max(len(p) for p in prompts)
    live = min(n, max_live or n)
    n_slots = {B.KV_SHARED: 1, B.KV_DEPTH_INDEXED: dims.R, B.KV_FIRST_THEN_SHARED: 2}[kv_layout]
    pages = live * n_slots * ((P + T + dims.page_size - 1) // dims.page_size)
    # all sequences live: prompts first, then the timed decode phase; a queue of waiting sequences: prompts overlap decode
    kw = {"background_prefill": live < n, "eager_refill": eager_refill} if pipelined else {}
    eng = (PipelinedEngine if pipelined else Engine)(dims, weights, max_batch=min(max_batch or n, live), max_live=live, max_len=P + T, n_pages=pages, gate_kind=gate_kind, kv_layout=kv_layout,
                 q_or_eps=q_or_eps, lookahead=True, mode=mode, min_coda_batch=min_coda_batch,
                 max_prefill_rows=max_prefill_rows, record_ticks=False, use_graphs=use_graphs, time_device=time_device, **kw)
    res = eng.generate(prompts, T, forced_depths=forced_depths)
    st = eng.stats
    depths = np.concatenate(res["depths"])
    decode_s = st["end"] - st["decode_start"]
    from .engine import kv_footprint
    out = {"kv_layout": kv_layout, "kv_kib_per_token_in_use": kv_footprint(dims, n_slots)[0] / 1024,
           "mode": mode + ("_pipelined" if pipelined else "") + ("" if use_graphs else "_nographs"), "max_batch": eng.max_batch, "max_live": live, "total_s": st["end"] - st["start"],
           "generated_tokens_per_s_end_to_end": sum(len(t) for t in res["tokens"]) / (st["end"] - st["start"]),
           "decode_s": decode_s, "prefill_s": st["decode_start"] - st["start"],
           "decode_tokens_per_s": len(depths) / decode_s, "token_loop_steps_per_s": st["row_steps"] / decode_s,
           "device_ms": st.get("device_ms"), "device_busy_ms": st.get("device_busy_ms"),
           "device_idle_fraction": (1.0 - st["device_busy_ms"] / (1e3 * decode_s)) if st.get("device_busy_ms") else None,
           "wall_ms_per_recurrent_step": 1e3 * decode_s / max(st["recurrent_steps"], 1),
           "eager_boundaries": st.get("eager_boundaries", 0), "recurrent_steps": st["recurrent_steps"], "row_steps": st["row_steps"], "coda_calls": st["coda_calls"],
           "mean_depth": float(depths.mean()), "depth_histogram": np.bincount(depths, minlength=dims.R + 1)[1:].tolist(),
           "status": eng.cdb.poll_status()}
    eng.cdb.destroy()
    del eng
    torch.cuda.empty_cache()
    return out, res


def calibrate_gate_bias(dims, weights, prompts, T, target, q=0.5, iters=10):
    """Bias of the learned gate for which the mean exit depth of a short adaptive run is about `target`
    (bisection on the product path; mean depth falls as the bias grows)."""
    lo, hi = -8.0, 8.0
    for _ in range(iters):
        mid = 0.5 * (lo + hi)
        weights["b_gate"] = torch.tensor([mid], dtype=torch.float32, device=weights["b_gate"].device)
        out, _ = run(dims, weights, prompts, T, mode="refill", gate_kind=B.GATE_SIGMOID_CDF, q_or_eps=q, max_prefill_rows=2048)
        if out["mean_depth"] > target:
            lo = mid
        else:
            hi = mid
    b = 0.5 * (lo + hi)
    weights["b_gate"] = torch.tensor([b], dtype=torch.float32, device=weights["b_gate"].device)
    return b


def calibrate_convergence_eps(dims, weights, prompts, T, target, iters=14):
    """Threshold of the convergence criterion (appendix C.2: exit once the L2 distance between consecutive
    recurrent states is below eps) for which the mean exit depth of a short adaptive run is closest to
    `target`: bisection on log(eps) on the product path (a larger eps exits earlier).  Returns (eps, mean depth)."""
    lo, hi = np.log(1e-4), np.log(1e6)
    best = None
    for _ in range(iters):
        mid = 0.5 * (lo + hi)
        out, _ = run(dims, weights, prompts, T, mode="refill", gate_kind=B.GATE_L2_CONVERGENCE, q_or_eps=float(np.exp(mid)),
                     max_prefill_rows=2048)
        if best is None or abs(out["mean_depth"] - target) < abs(best[1] - target):
            best = (float(np.exp(mid)), out["mean_depth"])
        if out["mean_depth"] > target:
            lo = mid
        else:
            hi = mid
    return best


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--model", default="ouro", choices=["ouro", "huginn"])
    ap.add_argument("--seqs", type=int, default=512)
    ap.add_argument("--prompt", type=int, default=256)
    ap.add_argument("--tokens", type=int, default=512)
    ap.add_argument("--layers", type=int, default=0, help="override the core layer count (smoke runs)")
    ap.add_argument("--max-batch", type=int, default=0)
    ap.add_argument("--min-coda-batch", type=int, default=0)
    ap.add_argument("--max-live", type=int, default=0, help="sequences resident at once (0 = all); fewer than --seqs queues the rest")
    ap.add_argument("--modes", default="cb,refill,no_refill", help="cb, refill, no_refill, refill_nographs (synchronous engine); cb_pipelined, refill_pipelined")
    ap.add_argument("--kv-layout", default="shared", choices=["shared", "depth_indexed", "first_then_shared"],
                    help="depth_indexed = last-exited cache (copy-on-exit), section 4.2")
    ap.add_argument("--exits", default="forced", choices=["forced", "criterion"],
                    help="huginn: replayed geometric exit depths, or the convergence criterion with a calibrated threshold")
    ap.add_argument("--no-eager-refill", action="store_true",
                    help="pipelined engine: always run the boundary stages beside the next step (tokens rejoin one step late)")
    ap.add_argument("--time-device", action="store_true", help="bracket every GPU phase with CUDA events and report device_ms")
    args = ap.parse_args()
    known = {"cb", "refill", "no_refill", "refill_nographs", "cb_pipelined", "refill_pipelined"}
    if not set(args.modes.split(",")) <= known:
        raise SystemExit(f"--modes takes a comma-separated subset of {sorted(known)}")
    torch.cuda.set_device(0)
    if args.model == "ouro":
        dims, seed = synth.OURO_1P4B, 2
    else:
        dims, seed = synth.HUGINN_3P5B, 3
    if args.layers:
        dims = dims.replace(L_core=args.layers)
    w = synth.make_weights(dims, seed, device="cuda:0", std=synth.width_scaled_std(dims.d), gate_std=2.0 / np.sqrt(dims.d))
    prompts = list(synth.make_prompts(args.seqs, args.prompt, dims.V, seed))
    report = {"model": args.model, "dims": {"d": dims.d, "H": dims.H, "Dh": dims.Dh, "F": dims.F, "V": dims.V,
                                            "layers": [dims.L_pre, dims.L_core, dims.L_coda], "R": dims.R},
              "seqs": args.seqs, "prompt": args.prompt, "tokens": args.tokens, "runs": []}
    forced = None
    q_or_eps = 0.5
    if args.model == "ouro":
        gate_kind = B.GATE_SIGMOID_CDF
        report["b_gate"] = calibrate_gate_bias(dims, w, prompts[:16], min(args.tokens, 24), 2.5)
        min_coda = args.min_coda_batch or 1
    elif args.exits == "forced":            # forced exit depths from a truncated geometric distribution (mean 12, cap 32)
        gate_kind = B.GATE_NONE
        forced = [list(r) for r in synth.forced_exit_depths((args.seqs, args.tokens - 1), seed, 12.0, dims.R)]
        min_coda = args.min_coda_batch or 32
    else:                                   # training-free convergence criterion, threshold calibrated to mean depth ~12
        gate_kind = B.GATE_L2_CONVERGENCE
        q_or_eps, cal_depth = calibrate_convergence_eps(dims, w, prompts[:8], min(args.tokens, 12), 12.0)
        report["eps"], report["calibration_mean_depth"] = q_or_eps, cal_depth
        min_coda = args.min_coda_batch or 32
    for mode in args.modes.split(","):
        pipelined = mode.endswith("_pipelined")
        nographs = mode.endswith("_nographs")
        name = mode
        mode = mode.replace("_pipelined", "").replace("_nographs", "")
        fixed = mode == "cb" and pipelined              # continuous batching on the pipelined engine: every token replays depth R
        out, _ = run(dims, w, prompts, args.tokens, mode="refill" if fixed else mode, pipelined=pipelined, use_graphs=not nographs,
                     time_device=args.time_device, eager_refill=not args.no_eager_refill, gate_kind=B.GATE_NONE if fixed else gate_kind, q_or_eps=q_or_eps,
                     forced_depths=[[dims.R] * (args.tokens - 1)] * args.seqs if fixed else None if mode == "cb" else forced,
                     max_batch=args.max_batch or None, max_live=args.max_live or None, min_coda_batch=min_coda,
                     kv_layout={"shared": B.KV_SHARED, "depth_indexed": B.KV_DEPTH_INDEXED, "first_then_shared": B.KV_FIRST_THEN_SHARED}[args.kv_layout])
        out["mode"] = name
        report["runs"].append(out)
        print(json.dumps(out), flush=True)
    by = {r["mode"]: r for r in report["runs"]}
    if "cb" not in by and "cb_pipelined" in by:
        by["cb"] = by["cb_pipelined"]
    if "cb" in by:
        for m in ("refill", "no_refill", "refill_pipelined"):
            if m in by:
                key = "decode_tokens_per_s" if not args.max_live else "generated_tokens_per_s_end_to_end"
                by[m]["speedup_vs_fixed_depth"] = by[m][key] / by["cb"][key]
                by[m]["flop_bound"] = flop_bound(dims, by[m]["mean_depth"])
                by[m]["fraction_of_flop_bound"] = by[m]["speedup_vs_fixed_depth"] / by[m]["flop_bound"]
    print(json.dumps(report))


if __name__ == "__main__":
    main()
