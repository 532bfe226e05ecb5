"""World-size-2 check of the multi-GPU plumbing on CPU (gloo): sequence sharding is a partition, the
timing reduction returns the slowest rank's value on every rank, and ranks draw different workloads."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    from paper_2608_09444_b200 import dist as D
    from paper_2608_09444_b200 import synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert D.env_rank() == (rank, rank, world)
    mine = D.shard(range(11), world, rank)
    slow = D.max_over_ranks(10.0 + rank)
    rows = synth.make_step_rows(8, 4, D.rank_seed(1, rank))
    dist.barrier()
    out.put((rank, mine, slow, rows["position"].tolist()))
    dist.destroy_process_group()


def test_two_ranks_shard_and_reduce():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    shards = [r[1] for r in res]
    assert sorted(shards[0] + shards[1]) == list(range(11)) and not set(shards[0]) & set(shards[1])
    assert abs(len(shards[0]) - len(shards[1])) <= 1
    assert [r[2] for r in res] == [11.0, 11.0]                 # both ranks see the slowest rank's time
    assert res[0][3] != res[1][3]                              # weak scaling: each rank has its own rows


def test_latency_model_fit_recovers_its_coefficients():
    """The least-squares fit of t = delta + gamma N_b + alpha N_c (section 5) returns the coefficients
    that generated exact synthetic points, and B* follows delta / (gamma + alpha L)."""
    from paper_2608_09444_b200.sweep import fit
    d, g, a = 1.7, 2.5e-3, 3.1e-5
    pts = [[nb, L, d + g * nb + a * nb * L] for nb in (1, 8, 64, 256) for L in (128, 2048, 8192)]
    f = fit(pts)
    assert abs(f["delta_ms"] - d) < 1e-9 and abs(f["gamma_ms_per_row"] - g) < 1e-11 and abs(f["alpha_ms_per_token"] - a) < 1e-13
    assert f["r2"] > 1 - 1e-12 and f["max_rel_residual"] < 1e-9


def test_serving_trace_and_latency_summary():
    """The request trace is seeded and within its clipping bounds; the summary computes per-request
    (finish - arrival) / output length and its percentiles."""
    from paper_2608_09444_b200.serve import make_requests, summarize
    a1, p1, t1 = make_requests(50, 8.0, 3, 1000)
    a2, p2, t2 = make_requests(50, 8.0, 3, 1000)
    assert np.array_equal(a1, a2) and t1 == t2 and all(np.array_equal(x, y) for x, y in zip(p1, p2))
    assert np.all(np.diff(a1) > 0) and 4 <= min(len(p) for p in p1) and max(len(p) for p in p1) <= 4096
    assert 4 <= min(t1) and max(t1) <= 2048 and max(int(p.max()) for p in p1) < 1000
    arr = np.array([0.0, 1.0, 2.0])
    stats = {"finish_s": [2.0, 5.0, 2.5], "first_token_s": [0.5, 1.5, 2.25], "recurrent_steps": 7, "row_steps": 9,
             "prefill_calls": 3, "coda_calls": 4}
    s = summarize(arr, [4, 8, 1], stats)
    lat = np.array([0.5, 0.5, 0.5])
    assert abs(s["normalized_latency_s_per_token"]["mean"] - lat.mean()) < 1e-12
    assert abs(s["normalized_latency_s_per_token"]["p99"] - 0.5) < 1e-12
    assert abs(s["generated_tokens_per_s"] - 13 / 5.0) < 1e-12 and abs(s["time_to_first_token_s"]["mean"] - (0.5 + 0.5 + 0.25) / 3) < 1e-12


def _serve_worker(rank, world, port, out):
    """Two replicas of the serving front end on CPU: same routing on both ranks, each fakes its own requests'
    time stamps, rank 0 merges them."""
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    from paper_2608_09444_b200 import dist as D
    from paper_2608_09444_b200.serve import make_requests, merge_replicas, summarize
    dist.init_process_group("gloo", rank=rank, world_size=world)
    arrivals, prompts, out_lens = make_requests(40, 16.0, 9, 1000)
    owner = D.route_least_loaded(arrivals, [len(p) + t for p, t in zip(prompts, out_lens)], out_lens, world)
    mine = [i for i in range(40) if owner[i] == rank]
    part = {"ids": mine, "finish_s": [float(arrivals[i]) + 0.01 * out_lens[i] for i in mine],
            "first_token_s": [float(arrivals[i]) + 0.005 for i in mine],
            "counters": {"recurrent_steps": 10 + rank, "row_steps": 100, "prefill_calls": len(mine), "coda_calls": 7}}
    parts = D.gather_objects(part)
    merged = merge_replicas(parts, 40)
    summary = summarize(arrivals, out_lens, merged)
    out.put((rank, owner, mine, summary["normalized_latency_s_per_token"]["mean"], merged["recurrent_steps"], merged["prefill_calls"]))
    dist.destroy_process_group()


def test_two_replicas_route_gather_and_merge():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_serve_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][1] == res[1][1]                                           # the same assignment on every rank
    assert sorted(res[0][2] + res[1][2]) == list(range(40))                 # a partition of the requests
    assert min(len(res[0][2]), len(res[1][2])) >= 10                        # both replicas get work
    assert abs(res[0][3] - 0.01) < 1e-9 and abs(res[1][3] - 0.01) < 1e-9    # merged latency = the faked 10 ms/token
    assert res[0][4] == 21 and res[0][5] == 40


def test_router_prefers_the_replica_with_fewer_reserved_tokens():
    from paper_2608_09444_b200.dist import route_least_loaded
    # three requests at the same time: sizes 100, 10, 10 -> ranks 0, 1, 1; after the big one finishes the next goes to 0
    owner = route_least_loaded([0.0, 0.0, 0.0, 5.0], [100, 10, 10, 50], [10, 1000, 1000, 10], 2, est_s_per_token=0.01)
    assert owner == [0, 1, 1, 0]
    assert route_least_loaded([0.0, 1.0], [5, 5], [1, 1], 1) == [0, 0]
