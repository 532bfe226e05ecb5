"""bf16 parity at model level: (1) a Huginn-3.5B-shaped layer stack (d 5280 = 82.5 k-blocks, 55 heads of
96, F 17920: every tile tail of the projection kernel) through prelude, one loop step with the
convergence gate, and coda; (2) lock-step replay of an adaptive decode (the paper's own method of
replaying recorded exits, appendix B.2): the oracle's tokens and exit depths drive the GPU engine,
which still computes its own gate values, exit signals and greedy tokens, compared item by item."""
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


def i32(a):
    return torch.tensor(np.asarray(a, dtype=np.int32), device="cuda")


def test_huginn_shaped_prelude_step_coda():
    from paper_2608_09444_b200 import binding as B
    dims = synth.HUGINN_3P5B.replace(V=4096, L_pre=1, L_core=1, L_coda=1, R=8)
    w = synth.make_weights(dims, 5, device="cuda", std=0.02)
    wn = synth.weights_to_numpy(w)
    ctxs = np.array([1, 16, 33, 250, 257, 90])
    n = len(ctxs)
    table_np, n_pages = synth.make_page_table(ctxs, 16, seed=4, extra_pages=1)
    eps_l2 = 1e30
    cdb = B.Cdb(dims, w, max_rows=n, max_seqs=n, max_position=table_np.shape[1] * 16,
                gate_kind=B.GATE_L2_CONVERGENCE, q_or_eps=eps_l2)
    pool = torch.empty(synth.kv_pool_shape(dims, n_pages), dtype=torch.bfloat16, device="cuda")
    synth.fill_kv_pool(pool, 9)
    pool_np = pool.float().cpu().numpy()
    cdb.kv_bind(pool)
    depth = np.array([1, 2, 3, 1, 2, 8])
    rows = B.Rows(i32(np.arange(n)), i32(ctxs - 1), i32(table_np), loop_depth=i32(depth), kv_slot=i32(np.zeros(n)))
    tok_np = np.array([5, 4095, 17, 0, 300, 9])
    h = torch.zeros((n, dims.d), device="cuda")
    cdb.boundary_prelude(i32(tok_np), rows, h)
    h0 = h.clone()
    gate, fire = torch.zeros(n, device="cuda"), torch.zeros(n, dtype=torch.uint8, device="cuda")
    cdb.loop_step(rows, h, gate, fire)
    h1 = h.clone()
    token, logits = torch.zeros(n, dtype=torch.int32, device="cuda"), torch.zeros((n, dims.V), device="cuda")
    cdb.boundary_coda_lmhead(rows, h, token, logits)
    torch.cuda.synchronize()
    assert cdb.poll_status() == 0
    orc = O.Oracle(dims, wn, gate_kind=O.GATE_L2_CONVERGENCE, q_or_eps=eps_l2)
    worst = {"prelude": 0.0, "step": 0.0, "logits": 0.0, "gate": 0.0}
    for i in range(n):
        c = int(ctxs[i])
        cache = orc.new_cache(c)
        for l in range(dims.L):
            K, V = O.gather_pages(pool_np[l], table_np[i], c)
            cache[l][0][0][:c], cache[l][0][1][:c] = K, V
        pos = np.array([c - 1])
        x0 = orc.prelude([tok_np[i]], pos, cache)
        worst["prelude"] = max(worst["prelude"], rel_err(h0[i].cpu().numpy(), x0[0]))
        x1 = orc.core_step(x0, pos, cache, 1)
        g, f, _ = orc.gate(x1[0], x0[0], 1.0, int(depth[i]))
        worst["step"] = max(worst["step"], rel_err(h1[i].cpu().numpy(), x1[0]))
        worst["gate"] = max(worst["gate"], abs(float(gate[i]) - g) / g)
        assert bool(fire[i]) == f == (depth[i] >= 2)
        lg = orc.coda_logits(x1, pos, cache)[0]
        worst["logits"] = max(worst["logits"], rel_err(logits[i].cpu().numpy(), lg))
        if int(token[i]) != int(np.argmax(lg)):
            assert lg.max() - lg[int(token[i])] < 2 * np.max(np.abs(logits[i].cpu().numpy() - lg))
    print(worst)
    assert all(v <= TOL for v in worst.values()), worst


@pytest.mark.parametrize("case", ["small", "ouro_full_size"])
def test_lockstep_replay_of_adaptive_decode_bf16(case):
    """small: 6 sequences x 12 tokens on a 3-layer model.  ouro_full_size: the offline-decode configuration's model
    (Ouro-1.4B shape: 24 core layers, d 2048, vocabulary 49152, learned gate) on a sample of two sequences, prompt
    processing included - what the oracle can compute token by token in a few seconds."""
    from paper_2608_09444_b200 import binding as B
    from paper_2608_09444_b200.engine import Engine
    if case == "small":
        dims = synth.Dims(V=2048, d=512, H=4, Dh=128, F=1408, L_pre=0, L_core=3, L_coda=0, R=4, dtype="bf16")
        w = synth.make_weights(dims, 6, std=0.03, gate_std=2.0 / np.sqrt(dims.d), b_gate=-0.8)
        n_seqs, T, max_batch = 6, 12, 4
    else:
        dims = synth.OURO_1P4B
        w = synth.make_weights(dims, 2, device="cuda", gate_std=2.0 / np.sqrt(dims.d), b_gate=0.648)
        n_seqs, T, max_batch = 2, 4, 2
    wn = synth.weights_to_numpy(w)
    prompts = synth.make_prompts(n_seqs, 24, dims.V, 3)
    orc = O.Oracle(dims, wn, gate_kind=O.GATE_SIGMOID_CDF, q_or_eps=0.5, lookahead=True)
    ref = [orc.generate(p, T, keep_states=True) for p in prompts]
    depths = np.concatenate([r["depths"] for r in ref])
    assert depths.min() >= 2 and (case != "small" or len(set(depths)) >= 2)
    eng = Engine(dims, {k: v.cuda() for k, v in w.items()}, max_batch=max_batch, max_live=n_seqs, max_len=24 + T, n_pages=n_seqs * 3,
                 gate_kind=B.GATE_SIGMOID_CDF, q_or_eps=0.5, lookahead=True, mode="refill", max_prefill_rows=256,
                 record_states=True, record_logits=True)
    res = eng.generate(list(prompts), T, forced_depths=[list(r["depths"]) for r in ref],
                       teacher_tokens=[list(r["tokens"]) for r in ref])
    assert eng.cdb.poll_status() == 0
    worst_state = worst_logit = worst_gate = 0.0
    near_gate = explained = tokens = decisions = 0
    for s, r in enumerate(ref):
        assert np.array_equal(res["depths"][s], r["depths"])                    # the replayed trace was followed
        logits0 = eng.trace_logits[(s, 0)]
        worst_logit = max(worst_logit, rel_err(logits0, r["prefill_logits"]))
        cands = [(int(res["tokens"][s][0]), r["prefill_logits"], logits0)]
        for j, p in enumerate(r["passes"]):
            worst_state = max(worst_state, rel_err(eng.trace_states[(s, j + 1)], p["states"][-1]))
            lg = eng.trace_logits[(s, j + 1)]
            worst_logit = max(worst_logit, rel_err(lg, p["logits"]))
            cands.append((int(res["tokens"][s][j + 1]), p["logits"], lg))
            for step, (g_gpu, g_ref) in enumerate(zip(res["gates"][s][j], p["gate"])):
                worst_gate = max(worst_gate, abs(g_gpu - g_ref))
                decisions += 1
                if abs(g_ref - 0.5) < 1e-3:
                    near_gate += 1
                else:
                    assert (g_gpu >= 0.5) == (g_ref >= 0.5)                     # the GPU's own exit signal agrees
        for tok, lg_ref, lg_gpu in cands:
            tokens += 1
            want = int(np.argmax(lg_ref))
            if tok != want:
                assert lg_ref[want] - lg_ref[tok] < 2 * np.max(np.abs(lg_gpu - lg_ref)), (s, tok, want)
                explained += 1
    print(f"states {worst_state:.2e} logits {worst_logit:.2e} gates {worst_gate:.2e}; near-threshold {near_gate}/{decisions}, "
          f"near-tie tokens {explained}/{tokens}")
    assert worst_state <= TOL and worst_logit <= TOL and worst_gate <= TOL
    assert explained <= max(2, tokens // 20) and near_gate <= max(2, decisions // 50)


SHORT, LONG = [1, 33, 70, 16, 47], [130, 5, 300, 128, 257]


@pytest.mark.parametrize("H,Dh,dtype,lens,simt", [
    (2, 128, "bf16", SHORT, False), (3, 96, "bf16", SHORT, False), (2, 64, "bf16", SHORT, False), (4, 64, "fp32", SHORT, False),
    (2, 128, "bf16", LONG, False), (3, 96, "bf16", LONG, False), (2, 64, "bf16", LONG, False),
    (2, 128, "bf16", LONG, True), (4, 64, "fp32", LONG, False)])
def test_prefill_matches_oracle(H, Dh, dtype, lens, simt):
    """Lock-step prompt processing (query-tiled causal attention over the pages the call itself writes),
    several prompts of ragged length in one call with a pad row, against the oracle's prefill.  The long
    set spans several query tiles and key tiles of the tensor-core kernel with ragged tails; `simt` runs
    the plain-FMA kernel on the same bf16 input.  The pool starts as NaN: nothing may be read before written."""
    from paper_2608_09444_b200 import binding as B
    dims = synth.Dims(V=300, d=H * Dh, H=H, Dh=Dh, F=192, L_pre=1, L_core=2, L_coda=1, R=3, dtype=dtype)
    w = synth.make_weights(dims, 8, std=0.05, gain_jitter=0.1)
    wn = synth.weights_to_numpy(w)
    prompts = [synth.make_prompts(1, n, dims.V, 20 + i)[0] for i, n in enumerate(lens)]
    table_np, n_pages = synth.make_page_table(np.asarray(lens), 16, seed=2, extra_pages=1)
    n = sum(lens) + 1
    cdb = B.Cdb(dims, {k: v.cuda() for k, v in w.items()}, max_rows=n, max_seqs=len(lens), max_position=table_np.shape[1] * 16,
                gate_kind=B.GATE_NONE, flags=B.FLAG_SIMT_PREFILL if simt else 0)
    tdt = torch.float32 if dtype == "fp32" else torch.bfloat16
    pool = torch.full(synth.kv_pool_shape(dims, n_pages), float("nan"), dtype=tdt, device="cuda")   # nothing is read before written
    cdb.kv_bind(pool)
    seq = np.concatenate([np.full(m, i) for i, m in enumerate(lens)] + [[-1]])
    pos = np.concatenate([np.arange(m) for m in lens] + [[0]])
    tok = np.concatenate(prompts + [[0]])
    ends = np.cumsum(lens) - 1
    rows = B.Rows(i32(seq), i32(pos), i32(table_np))
    token, logits = torch.zeros(len(lens), dtype=torch.int32, device="cuda"), torch.zeros((len(lens), dims.V), device="cuda")
    cdb.prefill(i32(tok), rows, i32(ends), token, logits)
    torch.cuda.synchronize()
    assert cdb.poll_status() == 0
    orc = O.Oracle(dims, wn, gate_kind=O.GATE_NONE)
    tol = 1e-4 if dtype == "fp32" else TOL
    for i, pr in enumerate(prompts):
        cache = orc.new_cache(len(pr))
        ref = orc.prefill(pr, cache)
        assert rel_err(logits[i].cpu().numpy(), ref) <= tol, (i, rel_err(logits[i].cpu().numpy(), ref))
        if int(token[i]) != int(np.argmax(ref)):
            assert ref.max() - ref[int(token[i])] < 2 * np.max(np.abs(logits[i].cpu().numpy() - ref))
        # the KV the prompt left behind (last core layer, shared slot): what decode will attend to
        l = dims.L_pre + dims.L_core - 1
        page, off = table_np[i, (len(pr) - 1) // 16], (len(pr) - 1) % 16
        got = pool[l, page, 0, :, off, :].float().cpu().numpy()
        assert rel_err(got, cache[l][0][0][len(pr) - 1]) <= tol
    assert cdb.check_guards() == 0


@pytest.mark.parametrize("layout", ["depth_indexed", "first_then_shared"])
def test_prefill_and_decode_with_depth_slots_bf16(layout):
    """bf16 prompt processing (tensor-core attention) and a few decode tokens under the depth-aware KV layouts:
    every loop of the prompt writes its own slot, decode reads slot r-1 (or min(r,2)-1) and copy-on-exit fills
    the skipped slots.  Logits of the prompt and the K the last core layer holds in every slot against the oracle."""
    from paper_2608_09444_b200 import binding as B
    dims = synth.Dims(V=300, d=256, H=2, Dh=128, F=192, L_pre=1, L_core=2, L_coda=1, R=3, dtype="bf16")
    w = synth.make_weights(dims, 8, std=0.05, gain_jitter=0.1)
    wn = synth.weights_to_numpy(w)
    o_layout = {"depth_indexed": O.DEPTH_INDEXED, "first_then_shared": O.FIRST_THEN_SHARED}[layout]
    b_layout = {"depth_indexed": B.KV_DEPTH_INDEXED, "first_then_shared": B.KV_FIRST_THEN_SHARED}[layout]
    n_slots = O.n_slots(o_layout, dims.R)
    lens = [150, 40]
    prompts = [synth.make_prompts(1, n, dims.V, 50 + i)[0] for i, n in enumerate(lens)]
    per = (max(lens) + 15) // 16
    table_np = np.arange(len(lens) * n_slots * per, dtype=np.int32).reshape(len(lens) * n_slots, per)
    cdb = B.Cdb(dims, {k: v.cuda() for k, v in w.items()}, max_rows=sum(lens), max_seqs=len(lens), max_position=per * 16,
                gate_kind=B.GATE_NONE, kv_layout=b_layout)
    pool = torch.full(synth.kv_pool_shape(dims, table_np.size), float("nan"), dtype=torch.bfloat16, device="cuda")
    cdb.kv_bind(pool)
    seq = np.concatenate([np.full(m, i) for i, m in enumerate(lens)])
    pos = np.concatenate([np.arange(m) for m in lens])
    rows = B.Rows(i32(seq), i32(pos), i32(table_np))
    token, logits = torch.zeros(len(lens), dtype=torch.int32, device="cuda"), torch.zeros((len(lens), dims.V), device="cuda")
    cdb.prefill(i32(np.concatenate(prompts)), rows, i32(np.cumsum(lens) - 1), token, logits)
    torch.cuda.synchronize()
    assert cdb.poll_status() == 0 and cdb.check_guards() == 0
    orc = O.Oracle(dims, wn, kv_layout=o_layout, gate_kind=O.GATE_NONE)
    l = dims.L_pre + dims.L_core - 1
    for i, pr in enumerate(prompts):
        cache = orc.new_cache(len(pr))
        ref = orc.prefill(pr, cache)
        assert rel_err(logits[i].cpu().numpy(), ref) <= TOL, (i, rel_err(logits[i].cpu().numpy(), ref))
        t = len(pr) - 1
        for slot in range(n_slots):
            page = table_np[i * n_slots + slot, t // 16]
            got = pool[l, page, 0, :, t % 16, :].float().cpu().numpy()
            assert rel_err(got, cache[l][slot][0][t]) <= TOL, (i, slot)
