"""Edge cases and invariants of the CUDA path through the C ABI: empty and all-pad batches, the largest
position, reported (not faulting) range errors, capacity errors from the host checks, and batch
invariance: a row's loop-step result is the same bit for bit alone or inside any batch, which is what
lets continuous depth batching regroup rows freely without changing predictions (section 3)."""
import numpy as np
import pytest
import torch

from oracle import cdb_oracle as O
from paper_2608_09444_b200 import synth

pytestmark = pytest.mark.gpu


def dev(x, dtype=None):
    t = torch.as_tensor(np.ascontiguousarray(x)).cuda()
    return t if dtype is None else t.to(dtype)


def i32(a):
    return dev(np.asarray(a, dtype=np.int32))


DIMS = synth.Dims(V=64, d=256, H=2, Dh=128, F=320, L_pre=0, L_core=2, L_coda=0, R=4, dtype="bf16")


def setup(ctxs, max_rows, seed=3, dims=DIMS, extra_pages=1, **kw):
    from paper_2608_09444_b200 import binding as B
    w = synth.make_weights(dims, seed, std=0.05, gain_jitter=0.1, gate_std=0.1, b_gate=-0.2)
    wd = {k: v.cuda() for k, v in w.items()}
    table_np, n_pages = synth.make_page_table(np.asarray(ctxs), 16, seed=seed, permute=True, extra_pages=extra_pages)
    cdb = B.Cdb(dims, wd, max_rows=max_rows, max_seqs=len(ctxs), max_position=table_np.shape[1] * 16,
                gate_kind=B.GATE_SIGMOID_CDF, q_or_eps=0.4, **kw)
    rng = np.random.default_rng(seed)
    pool_np = synth.to_bf16_grid(rng.standard_normal(synth.kv_pool_shape(dims, n_pages)).astype(np.float32))
    pool = dev(pool_np, torch.bfloat16)
    cdb.kv_bind(pool)
    return B, cdb, w, table_np, pool, pool_np


def test_empty_and_all_pad_batches_change_nothing():
    B, cdb, _, table_np, pool, pool_np = setup([40, 17], max_rows=4)
    table = dev(table_np)
    h = torch.randn((4, DIMS.d), device="cuda")
    h0 = h.clone()
    rows0 = B.Rows(i32([]), i32([]), table, loop_depth=i32([]), kv_slot=i32([]), n_rows=0)
    cdb.loop_step(rows0, h[:0])
    pads = B.Rows(i32([-1] * 4), i32([0] * 4), table, loop_depth=i32([1] * 4), kv_slot=i32([0] * 4))
    gate, fire = torch.full((4,), 7.0, device="cuda"), torch.zeros(4, dtype=torch.uint8, device="cuda")
    cdb.loop_step(pads, h, gate, fire)
    surv, ex, counts = torch.zeros(4, dtype=torch.int32, device="cuda"), torch.zeros(4, dtype=torch.int32, device="cuda"), torch.full((2,), -1, dtype=torch.int32, device="cuda")
    cdb.compact(pads, surv, ex, counts)
    torch.cuda.synchronize()
    assert cdb.poll_status() == 0
    assert torch.equal(h, h0) and int(fire.sum()) == 0
    assert counts.cpu().tolist() == [0, 0]
    assert np.array_equal(pool.float().cpu().numpy(), pool_np)


def test_last_position_of_the_configured_range():
    """A row at position max_position - 1 (the last token of its last page) against the oracle."""
    ctx = 64
    B, cdb, w, table_np, pool, pool_np = setup([ctx], max_rows=1, extra_pages=0)
    assert table_np.shape[1] * 16 == ctx
    rows = B.Rows(i32([0]), i32([ctx - 1]), dev(table_np), loop_depth=i32([2]), kv_slot=i32([0]))
    scratch = torch.zeros((1, DIMS.d), device="cuda")
    cdb.boundary_embed(i32([0]), rows, scratch)
    h_np = np.random.default_rng(5).standard_normal((1, DIMS.d)).astype(np.float32)
    h = dev(h_np)
    cdb.loop_step(rows, h)
    torch.cuda.synchronize()
    assert cdb.poll_status() == 0
    orc = O.Oracle(DIMS, synth.weights_to_numpy(w), gate_kind=O.GATE_SIGMOID_CDF, q_or_eps=0.4)
    Ks, Vs = zip(*[O.gather_pages(pool_np[l], table_np[0], ctx) for l in range(DIMS.L_core)])
    h_ref = orc.loop_step_row(h_np[0], ctx - 1, 2, list(Ks), list(Vs))[0]
    err = np.max(np.abs(h.cpu().numpy()[0] - h_ref)) / np.max(np.abs(h_ref))
    assert err <= 2e-2, err


def test_range_errors_are_reported_not_faulted():
    """A page id outside the pool, a sequence id outside [0, max_seqs) and a position outside the range
    make the kernels skip the access and latch a status word the host reads; capacity violations are
    refused by the host checks before anything is launched."""
    B, cdb, _, table_np, pool, pool_np = setup([40, 17], max_rows=2)
    bad = table_np.copy()
    bad[0, 1] = 10 ** 6                                    # logical page 1 of sequence 0
    h = torch.randn((2, DIMS.d), device="cuda")
    rows = B.Rows(i32([0, 1]), i32([39, 16]), dev(bad), loop_depth=i32([1, 1]), kv_slot=i32([0, 0]))
    cdb.loop_step(rows, h)
    torch.cuda.synchronize()
    assert cdb.poll_status() == 1                          # page
    assert cdb.poll_status() == 0                          # reading clears it
    rows = B.Rows(i32([0, 5]), i32([39, 16]), dev(table_np), loop_depth=i32([1, 1]), kv_slot=i32([0, 0]))
    cdb.loop_step(rows, h)
    torch.cuda.synchronize()
    assert cdb.poll_status() == 3                          # sequence
    rows = B.Rows(i32([0, 1]), i32([39, 4096]), dev(table_np), loop_depth=i32([1, 1]), kv_slot=i32([0, 0]))
    cdb.loop_step(rows, h)
    torch.cuda.synchronize()
    assert cdb.poll_status() == 2                          # position
    assert bool(torch.isfinite(h[0]).all())                # the good row of the batch was still computed
    big = B.Rows(i32([0, 1, -1]), i32([39, 16, 0]), dev(table_np), loop_depth=i32([1, 1, 1]), kv_slot=i32([0, 0, 0]))
    with pytest.raises(B.CdbError) as e:
        cdb.loop_step(big, torch.zeros((3, DIMS.d), device="cuda"))
    assert e.value.code == -3                              # CDB_ERR_CAPACITY
    assert "max_rows" in str(e.value) or "rows" in str(e.value)


@pytest.mark.parametrize("flags,extra", [(0, 0), (4, 0), (0, 70), (0, 200), (16, 0), (16, 200), (32, 0), (32, 200)])
def test_a_rows_result_does_not_depend_on_its_batch(flags, extra):
    """Run nine rows together, then three of them alone, as a pair in another order and among pads: hidden
    states, gate values, exit signals and the K/V written must be identical bit for bit (shape-only split-K
    with fixed-order sums, attention splits that depend only on the row's own context).  flags=4 repeats the
    check on the unfused layer flow, flags=16 on the multi-stage cooperative layer kernel; `extra` more rows make the full batch wide enough for the projection
    kernel's 128- and 256-row tiles."""
    ctxs = [1, 16, 17, 40, 255, 256, 257, 300, 33] + [int(c) for c in np.random.default_rng(2).integers(1, 90, extra)]
    n = len(ctxs)
    B, cdb, _, table_np, pool, pool_np = setup(ctxs, max_rows=n, flags=flags)
    table = dev(table_np)
    rng = np.random.default_rng(1)
    h_np = rng.standard_normal((n, DIMS.d)).astype(np.float32)
    depth = rng.integers(1, DIMS.R + 1, n)

    def run(idx):
        pool.copy_(dev(pool_np, torch.bfloat16))
        seq = [int(i) if i >= 0 else -1 for i in idx]
        pos = [ctxs[i] - 1 if i >= 0 else 0 for i in idx]
        dep = [int(depth[i]) if i >= 0 else 1 for i in idx]
        rows = B.Rows(i32(seq), i32(pos), table, loop_depth=i32(dep), kv_slot=i32([0] * len(idx)))
        cdb.boundary_embed(i32([0] * len(idx)), rows, torch.zeros((len(idx), DIMS.d), device="cuda"))   # fresh gate state
        h = dev(np.stack([h_np[i] if i >= 0 else np.zeros(DIMS.d, np.float32) for i in idx]))
        gate, fire = torch.zeros(len(idx), device="cuda"), torch.zeros(len(idx), dtype=torch.uint8, device="cuda")
        cdb.loop_step(rows, h, gate, fire)
        torch.cuda.synchronize()
        assert cdb.poll_status() == 0
        out = {}
        pl = pool.view(torch.int16).cpu().numpy()
        for j, i in enumerate(idx):
            if i >= 0:
                page, off = table_np[i, (ctxs[i] - 1) // 16], (ctxs[i] - 1) % 16
                out[i] = (h[j].cpu().numpy().view(np.int32), gate[j].cpu().numpy().view(np.int32), int(fire[j]),
                          pl[:, page, :, :, off, :].copy())
        return out

    full = run(list(range(n)))
    for subset in ([4], [7], [0], [7, 4], [-1, 5, -1, 2], [8, 6, 3, 1]):
        part = run(subset)
        for i, (hh, gg, ff, kv) in part.items():
            assert np.array_equal(hh, full[i][0]), (subset, i)
            assert np.array_equal(gg, full[i][1]) and ff == full[i][2], (subset, i)
            assert np.array_equal(kv, full[i][3]), (subset, i)


def test_device_side_row_count_masks_the_tail_and_serves_one_graph_for_every_batch_size():
    """Static shapes (section 4.3): the call's capacity is fixed on the host, the number of live rows is read from
    device memory.  Rows beyond the count are pads although their descriptor looks like a real row: their state and
    their KV pages stay untouched and they appear in neither compaction list; the live rows get, bit for bit, what a
    call of exactly that many rows gives.  One captured CUDA graph is replayed with three different counts."""
    ctxs = [1, 16, 17, 40, 255, 256, 257, 300, 33, 70, 12, 90]
    cap = len(ctxs)
    B, cdb, _, table_np, pool, pool_np = setup(ctxs, max_rows=cap)
    table = dev(table_np)
    rng = np.random.default_rng(4)
    h_np = rng.standard_normal((cap, DIMS.d)).astype(np.float32)
    depth = rng.integers(1, DIMS.R + 1, cap)
    seq, pos, dep, slot = i32(np.arange(cap)), i32(np.asarray(ctxs) - 1), i32(depth), i32(np.zeros(cap))
    fire_prev = dev((rng.random(cap) < 0.4).astype(np.uint8))

    def fresh():
        pool.copy_(dev(pool_np, torch.bfloat16))
        cdb.boundary_embed(i32([0] * cap), B.Rows(seq, pos, table), torch.zeros((cap, DIMS.d), device="cuda"))   # gate state reset
        return dev(h_np.copy())

    def exact(k):                                            # a call of exactly k rows
        h = fresh()
        rows = B.Rows(seq[:k], pos[:k], table, loop_depth=dep[:k], kv_slot=slot[:k])
        gate = torch.zeros(k, device="cuda")
        surv, ex, cnt = i32(np.zeros(k)), i32(np.zeros(k)), i32(np.zeros(2))
        cdb.compact(rows, surv, ex, cnt, fire_prev=fire_prev[:k])
        cdb.loop_step(rows, h[:k], gate)
        torch.cuda.synchronize()
        c = cnt.cpu().numpy()
        return h.cpu().numpy(), gate.cpu().numpy(), surv.cpu().numpy()[:c[0]], ex.cpu().numpy()[:c[1]], pool.view(torch.int16).cpu().numpy()

    n_live = i32([0])
    rows = B.Rows(seq, pos, table, loop_depth=dep, kv_slot=slot, n_rows_dev=n_live)
    h_g = torch.zeros((cap, DIMS.d), device="cuda")
    gate_g = torch.zeros(cap, device="cuda")
    surv_g, ex_g, cnt_g = i32(np.zeros(cap)), i32(np.zeros(cap)), i32(np.zeros(2))

    def body():
        cdb.compact(rows, surv_g, ex_g, cnt_g, fire_prev=fire_prev)
        cdb.loop_step(rows, h_g, gate_g)

    h_g.copy_(fresh())
    body()                                                   # warm-up with a count of 0: nothing may change
    torch.cuda.synchronize()
    assert np.array_equal(h_g.cpu().numpy(), h_np) and cnt_g.cpu().tolist() == [0, 0]
    assert np.array_equal(pool.float().cpu().numpy(), pool_np)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        body()
    for k in (5, 12, 1):
        want_h, want_gate, want_s, want_e, want_pool = exact(k)
        h_g.copy_(fresh())
        n_live.fill_(k)
        graph.replay()
        torch.cuda.synchronize()
        assert cdb.poll_status() == 0
        c = cnt_g.cpu().numpy()
        assert np.array_equal(surv_g.cpu().numpy()[:c[0]], want_s) and np.array_equal(ex_g.cpu().numpy()[:c[1]], want_e)
        assert np.array_equal(h_g.cpu().numpy().view(np.int32), want_h.view(np.int32))          # live rows equal, dead rows untouched
        assert np.array_equal(gate_g.cpu().numpy()[:k].view(np.int32), want_gate.view(np.int32))
        assert np.array_equal(pool.view(torch.int16).cpu().numpy(), want_pool)                  # dead rows wrote no K/V
    assert cdb.check_guards() == 0


WIDE = synth.Dims(V=64, d=1024, H=8, Dh=128, F=2816, L_pre=0, L_core=2, L_coda=0, R=4, dtype="bf16")


@pytest.mark.parametrize("n_rows", [9, 79, 209, 300, 530])
def test_in_cluster_sums_equal_workspace_sums_and_do_not_depend_on_the_batch(n_rows):
    """A model wide enough for real split-K (4 parts for the QKV and output projections, 8 for the down projection).
    Default flow: the parts are summed inside thread-block clusters, with RoPE and the KV page write in the QKV
    projection's epilogue.  Cross-check flow (flag 32): the parts go through a workspace and row-wise kernels.
    Flags 64 and 96 repeat both flows with the projections of 128 rows and more run by CTA pairs (one MMA over two
    SMs that share the activation tile).  All of them add the same parts in the same order, so states, gate values, exit
    signals and the K/V written must agree bit for bit - between the flows, and between a full batch and subsets.  The
    batch sizes walk through the row-tile widths the projections choose (64 and 128 rows, then any multiple of 16:
    112, 160 and 192-row tiles, ragged last tiles; at 530 rows CTA pairs by default).  Flag 128 runs batches of 64 rows and more as two half-batches with the SMs
    split between an attention and a projection partition (green contexts): the same numbers again."""
    ctxs = [1, 16, 17, 40, 255, 256, 257, 300, 33] + [int(c) for c in np.random.default_rng(2).integers(1, 90, n_rows - 9)]
    n = len(ctxs)
    rng = np.random.default_rng(1)
    h_np = rng.standard_normal((n, WIDE.d)).astype(np.float32)
    depth = rng.integers(1, WIDE.R + 1, n)
    results = {}
    for flags in (0, 32, 64, 96, 128):
        B, cdb, _, table_np, pool, pool_np = setup(ctxs, max_rows=n, dims=WIDE, flags=flags)
        table = dev(table_np)

        def run(idx):
            pool.copy_(dev(pool_np, torch.bfloat16))
            seq = [int(i) if i >= 0 else -1 for i in idx]
            pos = [ctxs[i] - 1 if i >= 0 else 0 for i in idx]
            dep = [int(depth[i]) if i >= 0 else 1 for i in idx]
            rows = B.Rows(i32(seq), i32(pos), table, loop_depth=i32(dep), kv_slot=i32([0] * len(idx)))
            cdb.boundary_embed(i32([0] * len(idx)), rows, torch.zeros((len(idx), WIDE.d), device="cuda"))
            h = dev(np.stack([h_np[i] if i >= 0 else np.zeros(WIDE.d, np.float32) for i in idx]))
            gate, fire = torch.zeros(len(idx), device="cuda"), torch.zeros(len(idx), dtype=torch.uint8, device="cuda")
            cdb.loop_step(rows, h, gate, fire)
            torch.cuda.synchronize()
            assert cdb.poll_status() == 0 and cdb.check_guards() == 0
            out = {}
            pl = pool.view(torch.int16).cpu().numpy()
            for j, i in enumerate(idx):
                if i >= 0:
                    page, off = table_np[i, (ctxs[i] - 1) // 16], (ctxs[i] - 1) % 16
                    out[i] = (h[j].cpu().numpy().view(np.int32), gate[j].cpu().numpy().view(np.int32), int(fire[j]),
                              pl[:, page, :, :, off, :].copy())
            return out

        results[flags] = [run(list(range(n)))] + [run(sub) for sub in ([4], [7, 4], [-1, 5, -1, 2], list(range(8, min(n, 75))))]
        cdb.destroy()
    full = results[0][0]
    assert all(np.isfinite(v[0].view(np.float32)).all() for v in full.values())
    for flags in (0, 32, 64, 96, 128):
        for part in results[flags]:
            for i, (hh, gg, ff, kv) in part.items():
                assert np.array_equal(kv, full[i][3]), (flags, i, "K/V")
                assert np.array_equal(hh, full[i][0]), (flags, i, "state")
                assert np.array_equal(gg, full[i][1]) and ff == full[i][2], (flags, i, "gate")


def test_host_checks_refuse_bad_calls_with_an_error_code():
    """The error behaviour the header promises: inconsistent dims, a missing or undersized KV pool, the wrong
    layout for copy-on-exit and an out-of-range layer come back as negative codes with a message; nothing is
    launched and the handle stays usable."""
    from paper_2608_09444_b200 import binding as B
    w = synth.make_weights(DIMS, 3, std=0.05)
    wd = {k: v.cuda() for k, v in w.items()}
    with pytest.raises(B.CdbError) as e:
        B.Cdb(DIMS.replace(d=DIMS.d + 8), wd, max_rows=4, max_seqs=4, max_position=64)       # d != H * Dh
    assert e.value.code == -1
    cdb = B.Cdb(DIMS, wd, max_rows=4, max_seqs=4, max_position=64)
    table = i32(np.arange(16).reshape(4, 4))
    rows = B.Rows(i32([0, 1]), i32([3, 5]), table, loop_depth=i32([1, 1]), kv_slot=i32([0, 0]))
    h = torch.zeros((2, DIMS.d), device="cuda")
    with pytest.raises(B.CdbError) as e:
        cdb.loop_step(rows, h)                                                                   # no pool bound yet
    assert e.value.code == -5 and "pool" in str(e.value)
    with pytest.raises(B.CdbError) as e:
        cdb.kv_bind(torch.zeros((1, 1000), dtype=torch.bfloat16, device="cuda"))                 # 1000 pages claimed, 2000 bytes given
    assert e.value.code == -1 and "smaller" in str(e.value)
    pool = torch.zeros(synth.kv_pool_shape(DIMS, 16), dtype=torch.bfloat16, device="cuda")
    cdb.kv_bind(pool)
    with pytest.raises(B.CdbError) as e:
        cdb.kv_copy_on_exit(rows, i32([2, 2]))                                                   # shared layout
    assert e.value.code == -5
    with pytest.raises(B.CdbError) as e:
        cdb.paged_attention(rows, 99, torch.zeros((2, DIMS.d), dtype=torch.bfloat16, device="cuda"),
                            torch.zeros((2, DIMS.d), dtype=torch.bfloat16, device="cuda"))
    assert e.value.code == -4
    cdb.loop_step(rows, h)                                                                       # still usable
    torch.cuda.synchronize()
    assert cdb.poll_status() == 0
