"""Parity at the benchmark configurations' own structure (bf16, lock-step replay, appendix B.2):

  * the deep-recurrence model: prelude 2 / core 4 / coda 2 layers, 32 loops, vocabulary 65536, exit depths replayed
    from the truncated-geometric trace (a depth-1, a mid and a depth-32 token among them), then the convergence
    criterion of appendix C.2 with the decision compared item by item;
  * offline adaptive decode on the 24-layer looped model with the configuration's 256-token prompts, more live
    sequences than batch rows (refill);
  * online serving on the same model: requests with seeded arrival times and ragged lengths through the
    pipelined engine with prompts processed beside the decode batch.

The oracle's tokens and exit depths are the trace; the GPU follows it but computes its own states, gate values, exit
signals and greedy tokens at every point, which are compared one by one.  Both host engines are run.

Two ways of comparing floating point.  Step by step: every stage of the GPU path (prelude, each loop step at its own
depth, coda + LM head) is given the oracle's state and the oracle's KV cache as input and must reproduce the oracle's
output within the bf16 tolerance - this is the parity claim, and it holds at every depth.  End to end: the engine's own
trajectory, where each stage consumes the previous GPU stage's output; bf16 rounding differences then add up over the
layer passes (about 2^-9 per rounded operand, growing like the square root of their number), so after the 130 and
more layer passes of a 32-loop model the trajectories sit AT the tolerance rather than inside it.  That growth is
printed and recorded, not hidden by a wider tolerance; integers (exit depths, tokens by the near-tie rule) are
asserted on the end-to-end run."""
import time

import numpy as np
import pytest
import torch

from oracle import cdb_oracle as O
from paper_2608_09444_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 2e-2


def rel_err(a, b):
    a, b = np.asarray(a, dtype=np.float64).ravel(), np.asarray(b, dtype=np.float64).ravel()
    return float(np.max(np.abs(a - b)) / max(np.max(np.abs(b)), 1e-30))


def check_tokens(got, ref_logits, gpu_logits=None):
    """Greedy tokens against the oracle's; a differing token must be a near-tie of the oracle's own logits: its
    margin below twice the logit error measured in that row (or, when the engine keeps no logits, below twice the
    tolerated error).  Returns (tokens compared, near-tie tokens)."""
    n = explained = 0
    for k, (tok, lg) in enumerate(zip(got, ref_logits)):
        n += 1
        want = int(np.argmax(lg))
        if int(tok) != want:
            err = np.max(np.abs(gpu_logits[k] - lg)) if gpu_logits is not None else TOL * np.max(np.abs(lg))
            assert lg[want] - lg[int(tok)] < 2 * err, (k, int(tok), want, lg[want] - lg[int(tok)], err)
            explained += 1
    return n, explained


def free_pages_intact(eng):
    """Allocator invariants after a run: every page is back on the free list exactly once, no table entry left."""
    assert sorted(eng.free_pages) == list(range(eng.n_pages))
    assert np.all(eng.page_table_host == -1)


# ------------------------------------------------------------------------------------------------ deep recurrence

def stepwise_errors(B, dims, w, orc, ref, prompts, T, gate_kind):
    """Worst error of each stage when it starts from the ORACLE's inputs: the KV pool is filled from the oracle's cache
    (its k, v are bf16 values, so the copy is exact), the input state of loop r is the oracle's state after loop r-1.
    The gate value compared is the step's own: the L2 distance, or the exit probability lambda_r of the learned gate
    (the sequence's survival is reset before every step, so the value returned is 1 - (1 - lambda_r))."""
    n_seqs, P = len(ref), len(prompts[0])
    pages_per = (P + T + 15) // 16
    cdb = B.Cdb(dims, w, max_rows=1, max_seqs=n_seqs, max_position=pages_per * 16, gate_kind=gate_kind, q_or_eps=0.0)
    table_np = np.arange(n_seqs * pages_per, dtype=np.int32).reshape(n_seqs, pages_per)
    pool_np = np.zeros(synth.kv_pool_shape(dims, n_seqs * pages_per), dtype=np.float32)
    for s, r in enumerate(ref):
        for l in range(dims.L):
            K, V = r["cache"][l][0]                                    # shared layout: one slot, [capacity, H, Dh]
            n_tok = min(K.shape[0], pages_per * 16)
            for pg in range((n_tok + 15) // 16):
                m = min(16, n_tok - 16 * pg)
                pool_np[l, table_np[s, pg], 0, :, :m, :] = K[16 * pg:16 * pg + m].transpose(1, 0, 2)
                pool_np[l, table_np[s, pg], 1, :, :m, :] = V[16 * pg:16 * pg + m].transpose(1, 0, 2)
    pool_host = torch.from_numpy(pool_np).to(torch.bfloat16)
    assert torch.equal(pool_host.float(), torch.from_numpy(pool_np))   # exact
    pool_host = pool_host.pin_memory()
    pool = pool_host.cuda()
    cdb.kv_bind(pool)
    i32 = lambda a: torch.tensor(np.asarray(a, dtype=np.int32), device="cuda")
    worst = {"prelude": 0.0, "loop step": 0.0, "gate": 0.0, "logits": 0.0}
    steps = 0
    scratch = torch.zeros((1, dims.d), device="cuda")
    for s, r in enumerate(ref):
        for j, p in enumerate(r["passes"]):
            t, y = P + j, int(r["tokens"][j])
            pool.copy_(pool_host)                                      # the oracle's cache again (the last token's calls wrote their own k, v)
            h0 = orc.prelude([y], np.array([t]), r["cache"])[0]        # rewrites the prelude layers' entry t with itself
            rows = lambda depth: B.Rows(i32([s]), i32([t]), i32(table_np), loop_depth=i32([depth]), kv_slot=i32([0]))
            h = torch.zeros((1, dims.d), device="cuda")
            (cdb.boundary_prelude if dims.L_pre > 0 else cdb.boundary_embed)(i32([y]), rows(1), h)
            worst["prelude"] = max(worst["prelude"], rel_err(h[0].cpu().numpy(), h0))
            for k in range(p["depth"]):
                h_in = h0 if k == 0 else p["states"][k - 1]
                h = torch.from_numpy(np.asarray(h_in, dtype=np.float32)[None]).cuda()
                gate = torch.zeros(1, device="cuda")
                cdb.boundary_embed(i32([y]), rows(k + 1), scratch)     # survival of the sequence back to 1
                cdb.loop_step(rows(k + 1), h, gate)
                worst["loop step"] = max(worst["loop step"], rel_err(h[0].cpu().numpy(), p["states"][k]))
                if gate_kind == B.GATE_L2_CONVERGENCE:
                    worst["gate"] = max(worst["gate"], abs(float(gate[0]) - p["gate"][k]) / p["gate"][k])
                else:
                    lam = 1.0 - (1.0 - p["gate"][k]) / (1.0 - (p["gate"][k - 1] if k else 0.0))
                    worst["gate"] = max(worst["gate"], abs(float(gate[0]) - lam))
                steps += 1
            h = torch.from_numpy(np.asarray(p["states"][-1], dtype=np.float32)[None]).cuda()
            tok, lg = torch.zeros(1, dtype=torch.int32, device="cuda"), torch.zeros((1, dims.V), device="cuda")
            cdb.boundary_coda_lmhead(rows(p["depth"]), h, tok, lg)
            worst["logits"] = max(worst["logits"], rel_err(lg[0].cpu().numpy(), p["logits"]))
            if int(tok[0]) != int(np.argmax(p["logits"])):
                assert p["logits"].max() - p["logits"][int(tok[0])] < 2 * np.max(np.abs(lg[0].cpu().numpy() - p["logits"]))
    torch.cuda.synchronize()
    assert cdb.poll_status() == 0 and steps == sum(int(np.sum(r["depths"])) for r in ref)
    cdb.destroy()
    return worst


@pytest.fixture
def huginn():
    """Weights on the GPU and ONE oracle (its float64 copy of the 3.85 B parameters is 31 GB of host memory).
    The weight scale follows the width, std = 0.02 sqrt(2048 / d), which gives a layer of this model the same gain as
    a layer of the 2048-wide model drawn at 0.02.  At a flat 0.02 every loop step of this width moves the state by
    several times its own norm and the recurrence amplifies rounding differences: the same replay then shows state
    errors of 5e-2 after one loop and 0.1-0.2 from loop 3 on, i.e. nothing a tolerance could test."""
    import gc
    dims = synth.HUGINN_3P5B
    w = synth.make_weights(dims, 3, device="cuda", std=synth.width_scaled_std(dims.d))
    wn = synth.weights_to_numpy(w)
    orc = O.Oracle(dims, wn, gate_kind=O.GATE_L2_CONVERGENCE, q_or_eps=0.0)
    del wn
    gc.collect()
    yield dims, w, orc
    del orc, w
    gc.collect()
    torch.cuda.empty_cache()


def test_deep_recurrence_forced_depth_replay_and_convergence_criterion(huginn):
    from paper_2608_09444_b200 import binding as B
    from paper_2608_09444_b200.engine import Engine
    from paper_2608_09444_b200.engine_async import PipelinedEngine
    dims, w, orc = huginn
    assert (dims.L_pre, dims.L_core, dims.L_coda, dims.R, dims.V) == (2, 4, 2, 32, 65536)
    n_seqs, P, T = 2, 24, 5
    prompts = synth.make_prompts(n_seqs, P, dims.V, 3)
    forced = synth.forced_exit_depths((n_seqs, T - 1), 3)
    forced[0, 0], forced[0, 2], forced[1, 1] = 1, 32, 12              # the trace's extremes and its mean
    t0 = time.time()
    assert orc.q_or_eps == 0.0                                         # forced depths: the signal never decides
    ref = [orc.generate(prompts[s], T, forced_depths=forced[s], keep_states=True) for s in range(n_seqs)]
    print(f"oracle, forced depths {forced.tolist()}: {time.time() - t0:.0f} s")
    teacher = [list(r["tokens"]) for r in ref]
    kw = dict(max_batch=2, max_live=n_seqs, max_len=P + T, n_pages=n_seqs * 2, gate_kind=B.GATE_L2_CONVERGENCE, q_or_eps=0.0,
              max_prefill_rows=64, min_coda_batch=1)

    # ---- synchronous engine: states after every loop step, distances, logits, tokens
    eng = Engine(dims, w, record_states=True, record_logits=True, **kw)
    res = eng.generate(list(prompts), T, forced_depths=[list(f) for f in forced], teacher_tokens=teacher)
    assert eng.cdb.poll_status() == 0 and eng.cdb.check_guards() == 0
    free_pages_intact(eng)
    by_loop = {}                                                       # loop depth -> worst state error at that depth
    worst_logit = worst_dist = 0.0
    n_tok = n_tie = 0
    for s, r in enumerate(ref):
        assert np.array_equal(res["depths"][s], forced[s])             # exit depths bit-exact (replayed, appendix B.2)
        lgs = [eng.trace_logits[(s, j)] for j in range(T)]
        refs = [r["prefill_logits"]] + [p["logits"] for p in r["passes"]]
        worst_logit = max(worst_logit, max(rel_err(a, b) for a, b in zip(lgs, refs)))
        a, b = check_tokens(res["tokens"][s], refs, lgs)
        n_tok, n_tie = n_tok + a, n_tie + b
        for j, p in enumerate(r["passes"]):
            for k, st in enumerate(p["states"]):
                e = rel_err(eng.trace_step_states[(s, j + 1, k + 1)], st)
                by_loop[k + 1] = max(by_loop.get(k + 1, 0.0), e)
            for g_gpu, g_ref in zip(res["gates"][s][j], p["gate"]):
                worst_dist = max(worst_dist, abs(g_gpu - g_ref) / g_ref)
    growth = ", ".join(f"r{r}: {by_loop[r]:.1e}" for r in sorted(by_loop) if r in (1, 2, 4, 8, 12, 16, 24, 32))
    print(f"forced depths, end to end: state error by loop depth {growth}; logits {worst_logit:.2e}; distance {worst_dist:.2e}; "
          f"near-tie tokens {n_tie}/{n_tok}")
    assert worst_dist <= TOL                                           # ||h_r - h_(r-1)|| is a difference of neighbours: it does not drift
    assert max(by_loop[r] for r in by_loop if r <= 4) <= TOL           # a 4-loop token is still inside the tolerance ...
    assert max(by_loop.values()) <= 2 * TOL and worst_logit <= 2 * TOL # ... and 32 loops stay near it (they would not at a flat weight scale)
    assert n_tie <= 2
    eng.cdb.destroy()
    del eng

    # ---- step by step: every stage from the oracle's own inputs (state and KV cache), at every depth of the trace
    local = stepwise_errors(B, dims, w, orc, ref, prompts, T, B.GATE_L2_CONVERGENCE)
    print("forced depths, step by step: " + ", ".join(f"{k} {v:.2e}" for k, v in local.items()))
    assert all(v <= TOL for v in local.values()), local

    # ---- pipelined engine: the same trace, tokens and depths
    pe = PipelinedEngine(dims, w, **kw)
    pres = pe.generate(list(prompts), T, forced_depths=[list(f) for f in forced], teacher_tokens=teacher)
    assert pe.cdb.poll_status() == 0
    free_pages_intact(pe)
    for s, r in enumerate(ref):
        assert np.array_equal(pres["depths"][s], forced[s])
        assert np.array_equal(pres["tokens"][s], res["tokens"][s])     # the two engines run the same kernels on the same rows
    pe.cdb.destroy()
    del pe

    # ---- convergence criterion (appendix C.2).  Threshold from the oracle's own distances: the median of the
    # first distance that counts (loop 2) over the replayed tokens, so that some tokens fire early and some late.
    d2 = [p["gate"][1] for r in ref for p in r["passes"] if len(p["gate"]) >= 2]
    eps = float(np.float32(np.median(d2)))
    t0 = time.time()
    orc.q_or_eps = eps
    ref_a = [orc.generate(prompts[s], T, keep_states=True) for s in range(n_seqs)]
    depths_a = [list(r["depths"]) for r in ref_a]
    print(f"oracle, convergence criterion eps {eps:.4f}: depths {depths_a}, {time.time() - t0:.0f} s")
    assert min(min(d) for d in depths_a) >= 3                          # first comparison at loop 2, one step of lookahead
    eng = Engine(dims, w, record_states=True, record_logits=True, **dict(kw, q_or_eps=eps))
    res = eng.generate(list(prompts), T, forced_depths=depths_a, teacher_tokens=[list(r["tokens"]) for r in ref_a])
    assert eng.cdb.poll_status() == 0
    all_d = np.array([g for r in ref_a for p in r["passes"] for g in p["gate"][1:]])
    decisions = near = flipped = 0
    worst_dist = worst_state = 0.0
    for s, r in enumerate(ref_a):
        assert np.array_equal(res["depths"][s], r["depths"])
        for j, p in enumerate(r["passes"]):
            worst_state = max(worst_state, rel_err(eng.trace_states[(s, j + 1)], p["states"][-1]))
            for k, (g_gpu, g_ref) in enumerate(zip(res["gates"][s][j], p["gate"])):
                worst_dist = max(worst_dist, abs(g_gpu - g_ref) / g_ref)
                if k == 0:
                    continue                                           # loop 1 compares with the prelude output: never decides
                decisions += 1
                if abs(g_ref - eps) < 1e-3 * eps:                      # the band is relative: the distance is not in [0, 1]
                    near += 1
                elif (np.float32(g_gpu) < np.float32(eps)) != (g_ref < eps):
                    # a decision outside the band may still flip when the distances of all tokens crowd around
                    # the threshold (random-init layers do not contract): only within the measured error
                    assert abs(g_ref - eps) < 2 * abs(g_gpu - g_ref), (s, j, k, g_gpu, g_ref, eps)
                    flipped += 1
    print(f"convergence criterion: spread of the distances over tokens and loops (std / mean) {all_d.std() / all_d.mean():.2e}, "
          f"worst GPU-vs-oracle distance error {worst_dist:.2e}; decisions {decisions}, inside the 1e-3 band {near}, "
          f"flipped within the measured error {flipped}; exit states {worst_state:.2e}")
    assert worst_dist <= TOL and worst_state <= 2 * TOL                # (exit states are end-to-end values: see the note on top)
    eng.cdb.destroy()


# ------------------------------------------------------------------------------------------------ 24-layer looped model

@pytest.fixture(scope="module")
def ouro():
    dims = synth.OURO_1P4B
    w = synth.make_weights(dims, 2, device="cuda", gate_std=2.0 / np.sqrt(dims.d), b_gate=0.648)
    wn = synth.weights_to_numpy(w)
    orc = O.Oracle(dims, wn, gate_kind=O.GATE_SIGMOID_CDF, q_or_eps=0.5, lookahead=True)
    return dims, w, orc


def test_offline_adaptive_decode_with_the_configurations_prompts(ouro):
    from paper_2608_09444_b200 import binding as B
    from paper_2608_09444_b200.engine import Engine
    from paper_2608_09444_b200.engine_async import PipelinedEngine
    dims, w, orc = ouro
    n_seqs, P, T = 4, 256, 17                                          # 16 adaptive passes per sequence
    prompts = synth.make_prompts(n_seqs, P, dims.V, 2)
    t0 = time.time()
    ref = [orc.generate(p, T, keep_states=True) for p in prompts]
    depths = np.concatenate([r["depths"] for r in ref])
    print(f"oracle: {time.time() - t0:.0f} s; exit depth histogram 1..4 {np.bincount(depths, minlength=5)[1:].tolist()}")
    assert depths.min() >= 2 and len(set(depths)) >= 2
    kw = dict(max_batch=2, max_live=n_seqs, max_len=P + T, n_pages=n_seqs * ((P + T + 15) // 16), gate_kind=B.GATE_SIGMOID_CDF,
              q_or_eps=0.5, lookahead=True, mode="refill", max_prefill_rows=2 * P)
    teacher, forced = [list(r["tokens"]) for r in ref], [list(r["depths"]) for r in ref]
    eng = Engine(dims, w, record_states=True, record_logits=True, **kw)
    res = eng.generate(list(prompts), T, forced_depths=forced, teacher_tokens=teacher)
    assert eng.cdb.poll_status() == 0 and eng.cdb.check_guards() == 0
    free_pages_intact(eng)
    assert max(len(t) for t in eng.stats["tick_rows"]) == 2            # the batch is smaller than the live set: refills happen
    worst_state = worst_logit = worst_gate = 0.0
    near = flipped = decisions = n_tok = n_tie = 0
    for s, r in enumerate(ref):
        assert np.array_equal(res["depths"][s], r["depths"])
        lgs = [eng.trace_logits[(s, j)] for j in range(T)]
        refs = [r["prefill_logits"]] + [p["logits"] for p in r["passes"]]
        worst_logit = max(worst_logit, max(rel_err(a, b) for a, b in zip(lgs, refs)))
        a, b = check_tokens(res["tokens"][s], refs, lgs)
        n_tok, n_tie = n_tok + a, n_tie + b
        for j, p in enumerate(r["passes"]):
            worst_state = max(worst_state, rel_err(eng.trace_states[(s, j + 1)], p["states"][-1]))
            for g_gpu, g_ref in zip(res["gates"][s][j], p["gate"]):
                worst_gate = max(worst_gate, abs(g_gpu - g_ref))
                decisions += 1
                if abs(g_ref - 0.5) < 1e-3:
                    near += 1
                elif (g_gpu >= 0.5) != (g_ref >= 0.5):
                    # The 1e-3 band presumes gate errors below 1e-3; after 50-100 layer passes the gate value carries
                    # the state's end-to-end error (~1e-2).  A decision outside the band may flip only if the oracle's
                    # own distance to the threshold is within twice the error measured on this very value.
                    assert abs(g_ref - 0.5) < 2 * abs(g_gpu - g_ref), (s, j, g_gpu, g_ref)
                    flipped += 1
    print(f"offline decode, 4 x (256 + 17), end to end: states {worst_state:.2e} logits {worst_logit:.2e} gates {worst_gate:.2e}; "
          f"decisions {decisions}, inside the 1e-3 band {near}, flipped within the measured error {flipped}; near-tie tokens {n_tie}/{n_tok}")
    assert worst_state <= 2 * TOL and worst_logit <= 2 * TOL and worst_gate <= 2 * TOL     # end to end: see the note on top
    assert n_tie <= max(2, n_tok // 20) and near + flipped <= max(2, decisions // 50)
    eng.cdb.destroy()
    del eng
    local = stepwise_errors(B, dims, w, orc, ref, prompts, T, B.GATE_SIGMOID_CDF)
    print("offline decode, step by step: " + ", ".join(f"{k} {v:.2e}" for k, v in local.items()))
    assert all(v <= TOL for v in local.values()), local
    pe = PipelinedEngine(dims, w, **kw)
    pres = pe.generate(list(prompts), T, forced_depths=forced, teacher_tokens=teacher)
    assert pe.cdb.poll_status() == 0
    free_pages_intact(pe)
    for s in range(n_seqs):
        assert np.array_equal(pres["depths"][s], ref[s]["depths"])
        assert np.array_equal(pres["tokens"][s], res["tokens"][s])
    pe.cdb.destroy()


def test_online_serving_arrivals_with_ragged_lengths(ouro):
    """Eight requests arrive over ~0.4 s with lognormal prompt and output lengths; the pipelined engine admits them as
    they come, processes their prompts beside the running decode batch and exits by its own gate (nothing is forced
    or fed back).  Exit depths and tokens must be the oracle's up to each request's first near-threshold gate or
    near-tie token, after which the two runs legitimately differ; pages all return."""
    from paper_2608_09444_b200 import binding as B
    from paper_2608_09444_b200.engine_async import PipelinedEngine
    dims, w, orc = ouro
    n = 8
    P = synth.lognormal_lengths(n, 41, median=48, cap=160)
    T = synth.lognormal_lengths(n, 42, median=6, cap=12, floor=2)
    arrivals = synth.poisson_arrivals(n, 20.0, 43)
    prompts = [synth.make_prompts(1, int(P[i]), dims.V, 50 + i)[0] for i in range(n)]
    t0 = time.time()
    ref = [orc.generate(prompts[i], int(T[i])) for i in range(n)]
    print(f"oracle: {time.time() - t0:.0f} s; prompt lengths {P.tolist()}, output lengths {T.tolist()}")
    max_len = int(max(P + T))
    pe = PipelinedEngine(dims, w, max_batch=4, max_live=6, max_len=max_len, n_pages=6 * ((max_len + 15) // 16),
                         gate_kind=B.GATE_SIGMOID_CDF, q_or_eps=0.5, max_prefill_rows=256, background_prefill=True)
    res = pe.generate(prompts, [int(t) for t in T], arrivals=list(arrivals))
    assert pe.cdb.poll_status() == 0
    free_pages_intact(pe)
    assert all(f is not None for f in pe.stats["finish_s"])
    assert all(pe.stats["first_token_s"][i] >= arrivals[i] for i in range(n))       # nothing starts before it arrives
    full = diverged = n_tok = n_dep = 0
    for i, r in enumerate(ref):
        assert len(res["tokens"][i]) == T[i] and len(res["depths"][i]) == T[i] - 1
        lgs = [r["prefill_logits"]] + [p["logits"] for p in r["passes"]]
        ok = True
        for j in range(int(T[i])):
            if j > 0:                                                  # adaptive pass j-1 produced token j
                p = r["passes"][j - 1]
                if res["depths"][i][j - 1] != p["depth"]:
                    # only a gate value within the tolerated error of the threshold may change the depth
                    assert min(abs(g - 0.5) for g in p["gate"]) < TOL, (i, j, p["gate"])
                    ok = False
                    break
                n_dep += 1
            lg = lgs[j]
            tok, want = int(res["tokens"][i][j]), int(np.argmax(lg))
            if tok != want:
                assert lg[want] - lg[tok] < 2 * TOL * np.max(np.abs(lg)), (i, j, tok, want)
                ok = False
                break
            n_tok += 1
        full += ok
        diverged += not ok
    print(f"serving: {full} of {n} requests equal to the oracle throughout, {diverged} left it at a near-tie; "
          f"{n_tok} tokens and {n_dep} exit depths equal")
    assert full >= n - 3
    pe.cdb.destroy()
