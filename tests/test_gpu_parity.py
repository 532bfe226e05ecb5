"""Parity of the CUDA path (through the C ABI) against the CPU oracle, stage by stage and for the
whole tiny looped decoder.  Integer outputs must match bit for bit; floating point within the
stated tolerance: max |gpu - oracle| / max |oracle| per compared row <= 1e-4 (fp32 configs) or
2e-2 (bf16 configs)."""
import numpy as np
import pytest
import torch

from oracle import cdb_oracle as O
from paper_2608_09444_b200 import synth

pytestmark = pytest.mark.gpu

TOL = {"fp32": 1e-4, "bf16": 2e-2}


def B():
    from paper_2608_09444_b200 import binding
    return binding


def rel_err(a, b):
    """per-row max abs error over the row's max abs reference value"""
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    a, b = a.reshape(-1, a.shape[-1]), b.reshape(-1, b.shape[-1])
    return float(np.max(np.max(np.abs(a - b), axis=1) / np.maximum(np.max(np.abs(b), axis=1), 1e-30)))


def dev(x, dtype=None):
    t = torch.as_tensor(np.ascontiguousarray(x)).cuda()
    return t if dtype is None else t.to(dtype)


def tdtype(dims):
    return torch.float32 if dims.dtype == "fp32" else torch.bfloat16


def make_model(dims, seed, **kw):
    w = synth.make_weights(dims, seed, std=kw.pop("std", 0.05), gain_jitter=0.1, **kw)
    return {k: v.cuda() for k, v in w.items()}, synth.weights_to_numpy(w)


def rows_of(binding, seq, pos, table, depth=None, slot=None, forced=None):
    i32 = lambda a: None if a is None else dev(np.asarray(a, dtype=np.int32))
    return binding.Rows(i32(seq), i32(pos), table, loop_depth=i32(depth), kv_slot=i32(slot), forced_exit=i32(forced))


# ------------------------------------------------------------------ A3: paged decode attention

ATTN_CASES = [
    ("fp32", 4, 64, [1, 15, 16, 17, 100, 255, 256, 257, 700]),
    ("bf16", 3, 128, [1, 16, 31, 256, 300, 513, 1000, 2048]),
    ("bf16", 5, 96, [2, 17, 250, 256, 600]),
    ("bf16", 2, 64, [3, 64, 257]),
]


@pytest.mark.parametrize("dtype,H,Dh,ctxs", ATTN_CASES)
def test_paged_attention_matches_bruteforce(dtype, H, Dh, ctxs):
    binding = B()
    dims = synth.Dims(V=32, d=H * Dh, H=H, Dh=Dh, F=64, L_pre=0, L_core=2, L_coda=0, R=2, dtype=dtype)
    wd, _ = make_model(dims, 11)
    n = len(ctxs)
    table_np, n_pages = synth.make_page_table(np.asarray(ctxs), 16, seed=5, permute=True, extra_pages=3)
    max_pos = table_np.shape[1] * 16
    cdb = binding.Cdb(dims, wd, max_rows=n + 2, max_seqs=n, max_position=max_pos, gate_kind=binding.GATE_NONE)
    rng = np.random.default_rng(3)
    pool_np = rng.standard_normal(synth.kv_pool_shape(dims, n_pages)).astype(np.float32)
    q_np = rng.standard_normal((n + 2, dims.d)).astype(np.float32)
    if dtype == "bf16":
        pool_np, q_np = synth.to_bf16_grid(pool_np), synth.to_bf16_grid(q_np)
    # slots past each context may hold anything, NaN included: they must not reach the result
    poisoned = pool_np.copy()
    for i, c in enumerate(ctxs):
        if c % 16:
            poisoned[:, table_np[i, (c - 1) // 16], :, :, c % 16:, :] = np.nan
    pool = dev(poisoned, tdtype(dims))
    cdb.kv_bind(pool)
    table = dev(table_np)
    # two pad rows in the middle and at the end
    seq = list(range(n // 2)) + [-1] + list(range(n // 2, n)) + [-1]
    pos = [c - 1 for c in ctxs[:n // 2]] + [0] + [c - 1 for c in ctxs[n // 2:]] + [0]
    rows = rows_of(binding, seq, pos, table, slot=[0] * (n + 2))
    q = dev(q_np, tdtype(dims))
    o = torch.full_like(q, 7.0)
    layer = 1
    cdb.paged_attention(rows, layer, q, o)
    torch.cuda.synchronize()
    assert cdb.poll_status() == 0
    got = o.float().cpu().numpy()
    worst = 0.0
    for r, s in enumerate(seq):
        if s < 0:
            assert np.all(got[r] == 0.0)
            continue
        K, V = O.gather_pages(pool_np[layer], table_np[s], ctxs[s])
        ref = O.attend(q_np[r].reshape(H, Dh).astype(np.float64), K, V).reshape(-1)
        worst = max(worst, rel_err(got[r][None], ref[None]))
    assert worst <= TOL[dtype], worst
    # a row alone gives bit-identical output to the same row inside the batch (splits depend only on the row)
    for r in (0, n):
        if seq[r] < 0:
            continue
        rows1 = rows_of(binding, [seq[r]], [pos[r]], table, slot=[0])
        o1 = torch.zeros((1, dims.d), dtype=q.dtype, device="cuda")
        cdb.paged_attention(rows1, layer, q[r:r + 1].contiguous(), o1)
        torch.cuda.synchronize()
        assert torch.equal(o1[0], o[r])


def test_paged_attention_is_page_permutation_invariant():
    binding = B()
    dims = synth.Dims(V=32, d=256, H=2, Dh=128, F=64, L_pre=0, L_core=1, L_coda=0, R=2, dtype="bf16")
    wd, _ = make_model(dims, 12)
    ctxs = np.array([300, 77])
    rng = np.random.default_rng(4)
    q = dev(rng.standard_normal((2, dims.d)).astype(np.float32), torch.bfloat16)
    outs = []
    dense = synth.to_bf16_grid(rng.standard_normal((2, 2, dims.H, 320, dims.Dh)).astype(np.float32))   # [seq][kv][H][tok][Dh]
    for seed in (1, 2):
        table_np, n_pages = synth.make_page_table(ctxs, 16, seed=seed, permute=True, extra_pages=5)
        pool_np = np.zeros(synth.kv_pool_shape(dims, n_pages), dtype=np.float32)
        for s in range(2):
            for j in range(-(-ctxs[s] // 16)):
                pool_np[0, table_np[s, j]] = dense[s][:, :, j * 16:(j + 1) * 16]
        cdb = binding.Cdb(dims, wd, max_rows=2, max_seqs=2, max_position=table_np.shape[1] * 16, gate_kind=binding.GATE_NONE)
        pool = dev(pool_np, torch.bfloat16)
        cdb.kv_bind(pool)
        rows = rows_of(binding, [0, 1], ctxs - 1, dev(table_np), slot=[0, 0])
        o = torch.zeros_like(q)
        cdb.paged_attention(rows, 0, q, o)
        torch.cuda.synchronize()
        outs.append(o.clone())
        cdb.destroy()
    assert torch.equal(outs[0], outs[1])


# ------------------------------------------------------------------ projections

@pytest.mark.parametrize("dtype,n,N,K", [("fp32", 5, 688, 256), ("fp32", 70, 130, 688), ("bf16", 33, 264, 256),
                                          ("bf16", 256, 512, 2048), ("bf16", 1, 96, 64), ("bf16", 300, 1000, 200),
                                          ("bf16", 100, 6144, 2048), ("bf16", 515, 2048, 5632)])
def test_linear_matches_matmul(dtype, n, N, K):
    binding = B()
    dims = synth.Dims(V=32, d=128, H=2, Dh=64, F=64, L_pre=0, L_core=1, L_coda=0, R=2, dtype=dtype)
    wd, _ = make_model(dims, 13)
    cdb = binding.Cdb(dims, wd, max_rows=8, max_seqs=2, max_position=16, gate_kind=binding.GATE_NONE)
    rng = np.random.default_rng(6)
    x, W = rng.standard_normal((n, K)).astype(np.float32), (rng.standard_normal((N, K)) * 0.05).astype(np.float32)
    if dtype == "bf16":
        x, W = synth.to_bf16_grid(x), synth.to_bf16_grid(W)
    y = torch.zeros((n, N), dtype=torch.float32, device="cuda")
    cdb.linear(dev(x, tdtype(dims)), dev(W, tdtype(dims)), y)
    torch.cuda.synchronize()
    ref = x.astype(np.float64) @ W.astype(np.float64).T
    assert rel_err(y.cpu().numpy(), ref) <= 1e-5


# ------------------------------------------------------------------ A8: exit flag + compaction (bit-exact)

@pytest.mark.parametrize("n", [0, 1, 31, 256, 1000, 1024, 3001])
def test_compaction_bit_exact(n):
    binding = B()
    dims = synth.Dims(V=32, d=128, H=2, Dh=64, F=64, L_pre=0, L_core=1, L_coda=0, R=4, dtype="fp32")
    wd, _ = make_model(dims, 14)
    cap = max(n, 1)
    cdb = binding.Cdb(dims, wd, max_rows=cap, max_seqs=cap, max_position=16, r_min=2)
    rng = np.random.default_rng(n)
    seq = np.arange(cap, dtype=np.int32)[:n]
    rng.shuffle(seq)
    seq[rng.random(n) < 0.1] = -1
    depth = rng.integers(1, 5, n).astype(np.int32)
    forced = np.where(rng.random(n) < 0.2, rng.integers(1, 5, n), 0).astype(np.int32)
    fire = (rng.random(n) < 0.3).astype(np.uint8)
    table = dev(np.zeros((cap, 1), dtype=np.int32))
    if n == 0:
        rows = binding.Rows(dev(np.zeros(1, np.int32)), dev(np.zeros(1, np.int32)), table,
                            loop_depth=dev(np.zeros(1, np.int32)), n_rows=0)
    else:
        rows = rows_of(binding, seq, np.zeros(n), table, depth=depth, forced=forced)
    h_src = torch.randn((cap, dims.d), device="cuda")
    h_next, h_exit = torch.zeros_like(h_src), torch.zeros_like(h_src)
    surv, ex = torch.full((cap,), -7, dtype=torch.int32, device="cuda"), torch.full((cap,), -7, dtype=torch.int32, device="cuda")
    counts = torch.full((2,), -1, dtype=torch.int32, device="cuda")
    cdb.compact(rows, surv, ex, counts, fire_prev=dev(fire) if n else None, h_src=h_src, h_next=h_next, h_exit=h_exit)
    torch.cuda.synchronize()
    flags = [O.exit_now(depth[i], 4, fire[i], forced[i], 2) for i in range(n)]
    want_s, want_e = O.stable_partition(flags, seq >= 0)
    c = counts.cpu().numpy()
    assert (c[0], c[1]) == (len(want_s), len(want_e))
    assert np.array_equal(surv.cpu().numpy()[:c[0]], want_s) and np.array_equal(ex.cpu().numpy()[:c[1]], want_e)
    assert np.all(surv.cpu().numpy()[c[0]:] == -7) and np.all(ex.cpu().numpy()[c[1]:] == -7)
    hs = h_src.cpu().numpy()
    assert np.array_equal(h_next.cpu().numpy()[:c[0]], hs[want_s]) and np.array_equal(h_exit.cpu().numpy()[:c[1]], hs[want_e])


# ------------------------------------------------------------------ one loop step, row by row (A1-A7)

STEP_CASES = [
    (synth.Dims(V=64, d=256, H=4, Dh=64, F=688, L_pre=0, L_core=2, L_coda=0, R=4, dtype="fp32"), 1),
    (synth.Dims(V=64, d=256, H=2, Dh=128, F=320, L_pre=0, L_core=2, L_coda=0, R=4, dtype="bf16"), 1),
    (synth.Dims(V=64, d=192, H=2, Dh=96, F=136, L_pre=0, L_core=1, L_coda=0, R=6, dtype="bf16"), 2),
]


@pytest.mark.parametrize("dims,gate_kind,flags", [c + (0,) for c in STEP_CASES] + [STEP_CASES[1] + (16,), STEP_CASES[2] + (16,)])
def test_loop_step_rows_match_oracle(dims, gate_kind, flags):
    """flags=16: the same step with everything after the attention in one cooperative multi-stage launch."""
    binding = B()
    wd, wn = make_model(dims, 21, gate_std=0.1, b_gate=-0.2)
    ctxs = np.array([1, 16, 17, 40, 255, 256, 257, 300, 33])
    n = len(ctxs)
    table_np, n_pages = synth.make_page_table(ctxs, 16, seed=9, permute=True, extra_pages=2)
    eps_l2 = 1e30 if gate_kind == 2 else 0.5
    cdb = binding.Cdb(dims, wd, max_rows=n + 1, max_seqs=n, max_position=table_np.shape[1] * 16,
                      gate_kind=gate_kind, q_or_eps=0.4 if gate_kind == 1 else eps_l2, flags=flags)
    rng = np.random.default_rng(8)
    pool_np = rng.standard_normal(synth.kv_pool_shape(dims, n_pages)).astype(np.float32)
    h_np = rng.standard_normal((n + 1, dims.d)).astype(np.float32)
    if dims.dtype == "bf16":
        pool_np = synth.to_bf16_grid(pool_np)
    pool = dev(pool_np, tdtype(dims))
    cdb.kv_bind(pool)
    table = dev(table_np)
    depth = rng.integers(1, dims.R + 1, n)
    seq = list(range(n)) + [-1]
    rows = rows_of(binding, seq, list(ctxs - 1) + [0], table, depth=list(depth) + [1], slot=[0] * (n + 1))
    # start every sequence from a fresh gate state (survival 1) through the boundary call
    tok = dev(np.zeros(n + 1, dtype=np.int32))
    scratch = torch.zeros((n + 1, dims.d), device="cuda")
    cdb.boundary_embed(tok, rows, scratch)
    h = dev(h_np)
    gate_val = torch.zeros(n + 1, device="cuda")
    fire = torch.zeros(n + 1, dtype=torch.uint8, device="cuda")
    cdb.loop_step(rows, h, gate_val, fire)
    torch.cuda.synchronize()
    assert cdb.poll_status() == 0
    got_h, got_g, got_f = h.cpu().numpy(), gate_val.cpu().numpy(), fire.cpu().numpy()
    got_pool = pool.float().cpu().numpy()
    assert np.array_equal(got_h[n], h_np[n])                      # the pad row is untouched
    orc = O.Oracle(dims, wn, gate_kind=gate_kind, q_or_eps=0.4 if gate_kind == 1 else eps_l2)
    tol = TOL[dims.dtype]
    near = 0
    for i in range(n):
        Ks, Vs = [], []
        for l in range(dims.L_core):
            K, V = O.gather_pages(pool_np[l], table_np[i], ctxs[i])
            Ks.append(K), Vs.append(V)
        h_ref, g_ref, f_ref, _, new_kv = orc.loop_step_row(h_np[i], ctxs[i] - 1, int(depth[i]), Ks, Vs)
        assert rel_err(got_h[i][None], h_ref[None]) <= tol, (i, rel_err(got_h[i][None], h_ref[None]))
        assert abs(got_g[i] - g_ref) <= tol * max(1.0, abs(g_ref))
        band = 1e-3 if gate_kind == 1 else 1e-3 * eps_l2
        if abs(g_ref - orc.q_or_eps) < band:
            near += 1                                             # too close to the threshold to compare
        else:
            assert bool(got_f[i]) == f_ref, i
        for l in range(dims.L_core):                              # the k, v this step wrote into the row's page
            page, off = table_np[i, (ctxs[i] - 1) // 16], (ctxs[i] - 1) % 16
            k_ref, v_ref = new_kv[l]
            assert rel_err(got_pool[l, page, 0, :, off, :].reshape(1, -1), k_ref.reshape(1, -1)) <= tol
            assert rel_err(got_pool[l, page, 1, :, off, :].reshape(1, -1), v_ref.reshape(1, -1)) <= tol
    # nothing but the rows' own slots was written
    mask = np.ones(pool_np.shape, dtype=bool)
    for i in range(n):
        mask[:, table_np[i, (ctxs[i] - 1) // 16], :, :, (ctxs[i] - 1) % 16, :] = False
    assert np.array_equal(got_pool[mask], pool_np[mask])
    assert near <= 1
    assert cdb.check_guards() == 0                                # no kernel wrote outside its scratch buffer


def test_two_stream_half_batches_equal_the_single_stream_step():
    """With the two-stream flag a loop step of 64+ rows runs as two half-batches on two streams; rows are independent, so the
    result must be bit-identical to the one-batch step (states, gate values, signals, KV pages)."""
    binding = B()
    dims = synth.Dims(V=64, d=256, H=2, Dh=128, F=320, L_pre=0, L_core=3, L_coda=0, R=4, dtype="bf16")
    wd, _ = make_model(dims, 23, gate_std=0.1)
    n = 101
    rng = np.random.default_rng(10)
    ctxs = rng.integers(1, 400, n)
    table_np, n_pages = synth.make_page_table(ctxs, 16, seed=3)
    pool_np = synth.to_bf16_grid(rng.standard_normal(synth.kv_pool_shape(dims, n_pages)).astype(np.float32))
    h_np = rng.standard_normal((n, dims.d)).astype(np.float32)
    outs = []
    for flags in (binding.FLAG_TWO_STREAM, 0):
        cdb = binding.Cdb(dims, wd, max_rows=n, max_seqs=n, max_position=table_np.shape[1] * 16, q_or_eps=0.5, flags=flags)
        pool = dev(pool_np, torch.bfloat16)
        cdb.kv_bind(pool)
        rows = rows_of(binding, np.arange(n), ctxs - 1, dev(table_np), depth=rng.integers(1, 5, n) * 0 + 2, slot=np.zeros(n))
        h, g, f = dev(h_np), torch.zeros(n, device="cuda"), torch.zeros(n, dtype=torch.uint8, device="cuda")
        cdb.boundary_embed(dev(np.zeros(n, dtype=np.int32)), rows, torch.zeros((n, dims.d), device="cuda"))
        cdb.loop_step(rows, h, g, f)
        torch.cuda.synchronize()
        assert cdb.poll_status() == 0
        outs.append((h.clone(), g.clone(), f.clone(), pool.clone()))
        cdb.destroy()
    for a, b in zip(*outs):
        assert torch.equal(a, b)


# ------------------------------------------------------------------ boundary: embedding, coda + LM head + greedy

@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_embed_and_lmhead(dtype):
    binding = B()
    dims = synth.Dims(V=515, d=128, H=2, Dh=64, F=64, L_pre=0, L_core=1, L_coda=0, R=2, dtype=dtype)
    wd, wn = make_model(dims, 31)
    n = 6
    cdb = binding.Cdb(dims, wd, max_rows=n, max_seqs=n, max_position=16)
    table = dev(np.zeros((n, 1), dtype=np.int32))
    rows = rows_of(binding, list(range(n)), [0] * n, table)
    tok = np.array([0, 514, 3, 3, 100, 7], dtype=np.int32)
    h = torch.zeros((n, dims.d), device="cuda")
    cdb.boundary_embed(dev(tok), rows, h)
    torch.cuda.synchronize()
    assert np.array_equal(h.cpu().numpy(), wn["embed"][tok])
    x = np.random.default_rng(2).standard_normal((n, dims.d)).astype(np.float32)
    token = torch.zeros(n, dtype=torch.int32, device="cuda")
    logits = torch.zeros((n, dims.V), device="cuda")
    cdb.boundary_coda_lmhead(rows, dev(x), token, logits)
    torch.cuda.synchronize()
    orc = O.Oracle(dims, wn)
    ref = orc.round(O.rmsnorm(x, wn["g_final"].astype(np.float64), dims.eps)) @ wn["W_lm"].astype(np.float64).T
    assert rel_err(logits.cpu().numpy(), ref) <= TOL[dtype]
    lg = logits.cpu().numpy()
    assert np.array_equal(token.cpu().numpy(), lg.argmax(-1))     # greedy on the kernel's own logits, first maximum


def test_argmax_ties_go_to_the_lowest_id():
    binding = B()
    dims = synth.Dims(V=300, d=128, H=2, Dh=64, F=64, L_pre=0, L_core=1, L_coda=0, R=2, dtype="fp32")
    wd, _ = make_model(dims, 32)
    wd["W_lm"][:] = 0.0
    wd["W_lm"][[17, 250, 299]] = wd["W_lm"].new_ones(dims.d)      # three identical rows -> three equal maxima
    cdb = binding.Cdb(dims, wd, max_rows=2, max_seqs=2, max_position=16)
    rows = rows_of(binding, [0, 1], [0, 0], dev(np.zeros((2, 1), dtype=np.int32)))
    token = torch.zeros(2, dtype=torch.int32, device="cuda")
    cdb.boundary_coda_lmhead(rows, torch.ones((2, dims.d), device="cuda"), token)
    torch.cuda.synchronize()
    assert token.cpu().tolist() == [17, 17]
