"""The allocation-free attention entry point (cdb_paged_attention_static) against the oracle's brute-force
attention and against the handle-based entry point.

It serves callers that cannot allocate device memory when they call the library (their process gave the
GPU's memory to its own pool, or their host framework forbids cudaMalloc): its scratch is an array built
into libcdb.so.  Both entry points run the same kernels, so their outputs must be identical; the check is
made on two calls in a row with different inputs, because the second call finds the first call's
contents in the shared scratch.  This file sorts last so that every other test has run before it."""
import numpy as np
import pytest
import torch

from oracle import cdb_oracle as O
from paper_2608_09444_b200 import synth

pytestmark = pytest.mark.gpu


def i32(a):
    return torch.tensor(np.asarray(a, dtype=np.int32), device="cuda")


def oracle_rows(q_np, pool_np, layer, table_np, ctxs, H, Dh):
    """softmax(q K^T / sqrt(Dh)) V per row, K and V gathered densely from the row's pages."""
    out = []
    for i, c in enumerate(ctxs):
        K, V = O.gather_pages(pool_np[layer], table_np[i], int(c))
        out.append(O.attend(q_np[i].reshape(H, Dh).astype(np.float64), K, V).reshape(-1))
    return np.stack(out)


@pytest.mark.parametrize("dtype,Dh", [("bf16", 128), ("bf16", 96), ("fp32", 64)])
def test_static_attention_matches_oracle_and_handle_based_attention_twice(dtype, Dh):
    from paper_2608_09444_b200 import binding as B
    H = 2
    dims = synth.Dims(V=32, d=H * Dh, H=H, Dh=Dh, F=64, L_pre=0, L_core=2, L_coda=0, R=2, dtype=dtype)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    tol = 2e-2 if dtype == "bf16" else 1e-4                                       # the tolerances of the other parity tests
    grid = synth.to_bf16_grid if dtype == "bf16" else (lambda a: a)
    w = {k: v.cuda() for k, v in synth.make_weights(dims, 3).items()}
    rng = np.random.default_rng(11)
    for call, ctxs in enumerate(([1, 16, 17, 255, 256, 257, 700], [300, 5, 1024, 33])):
        ctxs = np.asarray(ctxs)
        n = len(ctxs)
        table_np, n_pages = synth.make_page_table(ctxs, 16, seed=20 + call, extra_pages=2)
        max_context = table_np.shape[1] * 16
        pool_np = grid(rng.standard_normal(synth.kv_pool_shape(dims, n_pages)).astype(np.float32))
        q_np = grid(rng.standard_normal((n + 1, dims.d)).astype(np.float32))
        pool = torch.from_numpy(pool_np).cuda().to(tdt)
        q = torch.from_numpy(q_np).cuda().to(tdt)
        seq, pos = i32(list(range(n)) + [-1]), i32(list(ctxs - 1) + [0])          # last row is a pad
        table = i32(table_np)
        cdb = B.Cdb(dims, w, max_rows=n + 1, max_seqs=n, max_position=max_context, gate_kind=B.GATE_NONE)
        cdb.kv_bind(pool)
        want = torch.full_like(q, 3.0)
        cdb.paged_attention(B.Rows(seq, pos, table), 1, q, want)
        got = torch.full_like(q, 5.0)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        rc = B.paged_attention_static(q, got, pool, 1, seq, pos, table, max_seqs=n, max_context=max_context)
        assert rc == B.OK
        torch.cuda.synchronize()
        if call > 0:                                                             # (the first call may load the module lazily)
            assert torch.cuda.mem_get_info()[0] == free_before                   # the call took no device memory
        ref = oracle_rows(q_np, pool_np, 1, table_np, ctxs, H, Dh)
        g = got.float().cpu().numpy()
        for i in range(n):
            err = np.max(np.abs(g[i] - ref[i])) / np.max(np.abs(ref[i]))
            assert err <= tol, (call, i, err)
        assert torch.equal(got, want)                                            # same kernels as the handle path: identical
        assert torch.all(got[n] == 0)
        cdb.destroy()


def test_static_attention_zeroes_rows_outside_the_stated_bounds():
    """A row past max_context and a row whose sequence id has no table row come back as zeros (they are skipped,
    not read), the good row beside them is still right, and a bound the page table cannot cover is refused."""
    from paper_2608_09444_b200 import binding as B
    H, Dh = 2, 128
    dims = synth.Dims(V=32, d=H * Dh, H=H, Dh=Dh, F=64, L_pre=0, L_core=1, L_coda=0, R=2, dtype="bf16")
    rng = np.random.default_rng(12)
    ctxs = np.asarray([40, 20, 30])
    table_np, n_pages = synth.make_page_table(ctxs, 16, seed=3)
    pool_np = synth.to_bf16_grid(rng.standard_normal(synth.kv_pool_shape(dims, n_pages)).astype(np.float32))
    q_np = synth.to_bf16_grid(rng.standard_normal((3, dims.d)).astype(np.float32))
    pool, q = torch.from_numpy(pool_np).cuda().bfloat16(), torch.from_numpy(q_np).cuda().bfloat16()
    got = torch.full_like(q, 7.0)
    # row 1 sits at position 36 >= max_context 32 (its table row would cover it: rows are judged by the stated bound);
    # row 2 names sequence 7 of 3
    rc = B.paged_attention_static(q, got, pool, 0, i32([0, 1, 7]), i32([29, 36, 10]), i32(table_np), max_seqs=3, max_context=32)
    assert rc == B.OK
    torch.cuda.synchronize()
    ref = oracle_rows(q_np, pool_np, 0, table_np, [30], H, Dh)
    err = np.max(np.abs(got[0].float().cpu().numpy() - ref[0])) / np.max(np.abs(ref[0]))
    assert err <= 2e-2, err
    assert torch.all(got[1] == 0) and torch.all(got[2] == 0)
    assert B.paged_attention_static(q, got, pool, 0, i32([0, 1, 2]), i32([29, 19, 29]), i32(table_np), max_seqs=3,
                                    max_context=table_np.shape[1] * 16 + 1) == B.ERR_ARG


def test_static_attention_rejects_requests_beyond_its_scratch():
    from paper_2608_09444_b200 import binding as B
    n, H, Dh = 512, 16, 128
    pool = torch.zeros((1, 1, 2, H, 16, Dh), dtype=torch.bfloat16, device="cuda")
    q = torch.zeros((n, H * Dh), dtype=torch.bfloat16, device="cuda")
    z = torch.zeros(n, dtype=torch.int32, device="cuda")
    table = torch.zeros((1, 256), dtype=torch.int32, device="cuda")
    assert B.paged_attention_static(q, torch.empty_like(q), pool, 0, z, z, table, max_seqs=1, max_context=4096) == B.ERR_CAPACITY
