"""Recurrent-step latency sweep and roofline re-fit (section 5 / appendix A of the paper, on this GPU).

The paper models one loop step of the recurrent core as  t(N_c, N_b) = delta + gamma N_b + alpha N_c
(N_b rows in the batch, N_c cached tokens attended to in total), measures it on batches of B
equal-length requests, and derives the saturation batch  B*(L) = delta / (gamma + alpha L)  below
which a step costs about delta whatever its size.  This module repeats that measurement through the
library's C ABI: `cdb_loop_step` over N_b rows of context L each (distinct sequences, fragmented page
tables, KV pool filled with N(0,1)), CUDA-event time per step, median of `steps` after `warmup`;
then an ordinary least-squares fit of (delta, gamma, alpha).  It also times the boundary stages
(coda + LM head + greedy sampling + embedding / prelude of the sampled token) for the same batches,
the paper's tau_0.

    python -m paper_2608_09444_b200.sweep --model ouro            # prints one JSON document

Combinations whose KV does not fit the pool (`--pool-tokens`) are skipped and listed.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding as B
from . import synth


def _median_ms(fn, warmup, steps, dev):
    for _ in range(warmup):
        fn()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in evs:
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize(dev)
    return float(np.median([a.elapsed_time(b) for a, b in evs]))


def fit(points):
    """Least squares of t = delta + gamma N_b + alpha N_c over (N_b, L, t_ms) points."""
    A = np.array([[1.0, nb, nb * L] for nb, L, _ in points])
    y = np.array([t for _, _, t in points])
    coef, *_ = np.linalg.lstsq(A, y, rcond=None)
    pred = A @ coef
    ss_res, ss_tot = float(((y - pred) ** 2).sum()), float(((y - y.mean()) ** 2).sum())
    return {"delta_ms": float(coef[0]), "gamma_ms_per_row": float(coef[1]), "alpha_ms_per_token": float(coef[2]),
            "r2": 1.0 - ss_res / ss_tot if ss_tot > 0 else 1.0,
            "max_rel_residual": float(np.max(np.abs(pred - y) / y))}


def sweep(dims, batches, lengths, *, pool_tokens, warmup=3, steps=10, seed=7, device="cuda:0", flags=0, graph=False):
    dev = torch.device(device)
    torch.cuda.set_device(dev)
    max_rows, max_len = max(batches), max(lengths)
    width = (max_len + dims.page_size - 1) // dims.page_size
    n_pages = (pool_tokens + dims.page_size - 1) // dims.page_size
    weights = synth.make_weights(dims, seed, device=str(dev), std=synth.width_scaled_std(dims.d), gate_std=2.0 / np.sqrt(dims.d))
    cdb = B.Cdb(dims, weights, max_rows=max_rows, max_seqs=max_rows, max_position=width * dims.page_size,
                gate_kind=B.GATE_SIGMOID_CDF, q_or_eps=0.5, flags=flags)
    dt = torch.float32 if dims.dtype == "fp32" else torch.bfloat16
    pool = torch.empty(synth.kv_pool_shape(dims, n_pages), dtype=dt, device=dev)
    synth.fill_kv_pool(pool, seed + 1000)
    cdb.kv_bind(pool)
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed + 2000)
    h0 = torch.randn((max_rows, dims.d), generator=gen, device=dev, dtype=torch.float32)
    h = torch.empty_like(h0)
    h_new = torch.empty_like(h0)
    tokens = torch.zeros(max_rows, dtype=torch.int32, device=dev)
    i32 = dict(dtype=torch.int32, device=dev)
    rng = np.random.default_rng(seed)
    points, boundary, skipped = [], [], []
    for L in lengths:
        per_row = (L + dims.page_size - 1) // dims.page_size
        for nb in batches:
            if nb * per_row > n_pages:
                skipped.append([nb, L])
                continue
            table = np.full((nb, width), -1, dtype=np.int32)
            table[:, :per_row] = rng.permutation(n_pages)[:nb * per_row].astype(np.int32).reshape(nb, per_row)
            rows = B.Rows(torch.arange(nb, **i32), torch.full((nb,), L - 1, **i32), torch.from_numpy(table).to(dev),
                          loop_depth=torch.full((nb,), 2, **i32), kv_slot=torch.zeros(nb, **i32),
                          forced_exit=torch.full((nb,), -1, **i32))

            def step():
                h[:nb].copy_(h0[:nb])
                cdb.loop_step(rows, h[:nb])

            def bound():
                cdb.boundary_coda_lmhead(rows, h0[:nb], tokens[:nb])
                if dims.L_pre:
                    cdb.boundary_prelude(tokens[:nb], rows, h_new[:nb])
                else:
                    cdb.boundary_embed(tokens[:nb], rows, h_new[:nb])

            if graph:                     # replay the step as one CUDA graph (what the engines do)
                step()
                torch.cuda.synchronize(dev)
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    step()
                t = _median_ms(g.replay, warmup, steps, dev)
            else:
                t = _median_ms(step, warmup, steps, dev)
            points.append([nb, L, t])
            boundary.append([nb, L, _median_ms(bound, warmup, steps, dev)])
            st = cdb.poll_status()
            if st:
                raise RuntimeError(f"library status {st} at N_b={nb}, L={L}")
    out = {"model": {"d": dims.d, "L_core": dims.L_core, "H": dims.H, "Dh": dims.Dh, "F": dims.F, "dtype": dims.dtype},
           "points_nb_L_ms": points, "boundary_nb_L_ms": boundary, "skipped_nb_L": skipped,
           "fit_all": fit(points)}
    small = [p for p in points if p[0] <= 256]
    if len(small) >= 3:
        out["fit_nb_le_256"] = fit(small)
    f = out.get("fit_nb_le_256", out["fit_all"])
    out["b_star"] = {str(L): f["delta_ms"] / (f["gamma_ms_per_row"] + f["alpha_ms_per_token"] * L) for L in lengths}
    eb = 4 if dims.dtype == "fp32" else 2
    w_bytes = dims.L_core * (4 * dims.d * dims.d + 3 * dims.d * dims.F) * eb
    kv_tok = dims.L_core * 2 * dims.H * dims.Dh * eb
    out["implied"] = {"weight_bytes_per_step": w_bytes, "kv_bytes_per_token_step": kv_tok,
                      "weight_stream_GBps_at_delta": w_bytes / f["delta_ms"] / 1e6,
                      "kv_stream_GBps_at_alpha": kv_tok / f["alpha_ms_per_token"] / 1e6}
    cdb.destroy()
    return out


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--model", default="ouro", choices=["ouro", "huginn", "tiny"])
    ap.add_argument("--batches", default="1,2,4,8,16,32,64,128,256,512,1024")
    ap.add_argument("--lengths", default="128,512,2048,8192")
    ap.add_argument("--pool-tokens", type=int, default=524288, help="KV pool size in tokens (Ouro: 192 KiB each)")
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--flags", type=int, default=0, help="library flags (binding.FLAG_*), e.g. 2 = two-stream half-batches")
    ap.add_argument("--graph", action="store_true", help="time CUDA-graph replays of the step instead of direct launches")
    args = ap.parse_args(argv)
    dims = {"ouro": synth.OURO_1P4B, "huginn": synth.HUGINN_3P5B, "tiny": synth.TINY}[args.model]
    out = sweep(dims, [int(x) for x in args.batches.split(",")], [int(x) for x in args.lengths.split(",")],
                pool_tokens=args.pool_tokens, warmup=args.warmup, steps=args.steps, flags=args.flags, graph=args.graph)
    print(json.dumps(out))


if __name__ == "__main__":
    main()
