"""The allocation-free attention entry point (cdb_paged_attention_static) against the handle-based one.

It serves callers that cannot allocate device memory when they call the library (their process gave the
GPU's memory to its own pool, or their host framework forbids cudaMalloc): its scratch is an array built
into libcdb.so.  Both entry points run the same kernels, so the outputs must be identical; the check is
made on two calls in a row with different inputs, because the second call finds the first call's
contents in the shared scratch.  This file sorts last so that every other test has run before it."""
import numpy as np
import pytest
import torch

from paper_2608_09444_b200 import synth

pytestmark = pytest.mark.gpu


def test_static_attention_matches_handle_based_attention_twice():
    from paper_2608_09444_b200 import binding as B
    dims = synth.Dims(V=32, d=256, H=2, Dh=128, F=64, L_pre=0, L_core=2, L_coda=0, R=2, dtype="bf16")
    w = {k: v.cuda() for k, v in synth.make_weights(dims, 3).items()}
    i32 = lambda a: torch.tensor(np.asarray(a, dtype=np.int32), device="cuda")
    rng = np.random.default_rng(11)
    for call, ctxs in enumerate(([1, 16, 17, 255, 256, 257, 700], [300, 5, 1024, 33])):
        ctxs = np.asarray(ctxs)
        n = len(ctxs)
        table_np, n_pages = synth.make_page_table(ctxs, 16, seed=20 + call, extra_pages=2)
        max_context = table_np.shape[1] * 16
        pool = torch.from_numpy(synth.to_bf16_grid(rng.standard_normal(synth.kv_pool_shape(dims, n_pages)).astype(np.float32))).cuda().to(torch.bfloat16)
        q = torch.from_numpy(rng.standard_normal((n + 1, dims.d)).astype(np.float32)).cuda().to(torch.bfloat16)
        seq, pos = i32(list(range(n)) + [-1]), i32(list(ctxs - 1) + [0])         # last row is a pad
        table = i32(table_np)
        cdb = B.Cdb(dims, w, max_rows=n + 1, max_seqs=n, max_position=max_context, gate_kind=B.GATE_NONE)
        cdb.kv_bind(pool)
        want = torch.full_like(q, 3.0)
        cdb.paged_attention(B.Rows(seq, pos, table), 1, q, want)
        got = torch.full_like(q, 5.0)
        rc = B.paged_attention_static(q, got, pool, 1, seq, pos, table, max_seqs=n, max_context=max_context)
        assert rc == B.OK
        torch.cuda.synchronize()
        err = float((got.float() - want.float()).abs().max() / want.float().abs().max())
        assert err <= 2e-2, err                                                  # the tolerance of the bf16 tests
        assert torch.equal(got, want)                                            # same kernels: in fact identical
        assert torch.all(got[n] == 0)
        cdb.destroy()


def test_static_attention_rejects_requests_beyond_its_scratch():
    from paper_2608_09444_b200 import binding as B
    n, H, Dh = 512, 16, 128
    pool = torch.zeros((1, 1, 2, H, 16, Dh), dtype=torch.bfloat16, device="cuda")
    q = torch.zeros((n, H * Dh), dtype=torch.bfloat16, device="cuda")
    z = torch.zeros(n, dtype=torch.int32, device="cuda")
    table = torch.zeros((1, 256), dtype=torch.int32, device="cuda")
    assert B.paged_attention_static(q, torch.empty_like(q), pool, 0, z, z, table, max_seqs=1, max_context=4096) == B.ERR_CAPACITY
