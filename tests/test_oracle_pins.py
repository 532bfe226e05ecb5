"""Pins for the CPU oracle: what the paper prints, library special cases, invariants and brute
force.  None of these tests touches the CUDA path."""
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import cdb_oracle as O
from oracle import sched_oracle as SO
from paper_2608_09444_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
SMALL = synth.Dims(V=64, d=64, H=2, Dh=32, F=96, L_pre=1, L_core=2, L_coda=1, R=3, dtype="fp32")


def small_weights(dims=SMALL, seed=7, **kw):
    return synth.weights_to_numpy(synth.make_weights(dims, seed, std=0.08, gain_jitter=0.2, **kw))


# ------------------------------------------------------------------ closed forms printed by the paper

def test_table1_kv_footprint():
    dims = {"ouro": synth.OURO_1P4B, "huginn": synth.HUGINN_3P5B}
    for line in open(os.path.join(GOLDEN, "table1_kv_footprint.txt")):
        if line.startswith("#") or not line.strip():
            continue
        model, slots, kib, gib = line.split()
        b = O.kv_bytes_per_token(dims[model], int(slots))
        assert abs(b / 1024 - float(kib)) <= 0.5, (model, slots, b / 1024)
        assert abs(b * 4096 / 2**30 - float(gib)) <= 0.006, (model, slots)


def test_core_parameter_counts():
    # appendix A: Ouro 1.4B core 1.2 B parameters in 24 layers, Huginn 1.6 B in 4 layers
    assert round(O.core_params(synth.OURO_1P4B) / 1e9, 1) == 1.2
    assert round(O.core_params(synth.HUGINN_3P5B) / 1e9, 1) == 1.6


def test_executed_layers_and_flop_ratios():
    hug = synth.HUGINN_3P5B
    assert O.executed_layers(hug, 4) == 20                      # section 2: 2 + 4*4 + 2
    assert abs(O.boundary_to_core_flops(hug) - 1.2) < 0.05      # section 4: F0 ~ 1.2 Fr
    assert O.boundary_to_core_flops(synth.OURO_1P4B) < 0.1      # F0 << Fr
    # Eq. 2 chain and the "~1.6x for Ouro" figure at mean depth 2.5
    for dims, dbar in ((synth.OURO_1P4B, 2.5), (hug, 12.0)):
        b = O.flop_bound(dims, dbar)
        assert b <= dims.R / dbar <= dims.R / 2
    assert abs(synth.OURO_1P4B.R / 2.5 - 1.6) < 1e-12
    assert 1.5 < O.flop_bound(synth.OURO_1P4B, 2.5) < 1.6


# ------------------------------------------------------------------ elementwise pieces vs library routines

def test_bf16_round_matches_library():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.integers(-6, 6, 20000),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 65504.0]]).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(O.bf16_round(x).astype(np.float32), ref)


def test_rmsnorm_silu_sigmoid_vs_torch():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((5, 48)) * 3
    g = rng.standard_normal(48)
    t = torch.from_numpy(x)
    assert np.allclose(O.rmsnorm(x, g, 1e-6), F.rms_norm(t, (48,), torch.from_numpy(g), 1e-6).numpy(), rtol=1e-12)
    assert np.allclose(O.silu(x), F.silu(t).numpy(), rtol=1e-12)
    assert np.allclose(O.sigmoid(x), torch.sigmoid(t).numpy(), rtol=1e-12)
    # unit RMS without gain, invariance to input scale
    y = O.rmsnorm(x, None, 0.0)
    assert np.allclose(np.sqrt(np.mean(y * y, -1)), 1.0)
    assert np.allclose(O.rmsnorm(7.0 * x, g, 0.0), O.rmsnorm(x, g, 0.0))


def test_attend_vs_sdpa_and_bruteforce():
    rng = np.random.default_rng(2)
    c, H, Dh = 37, 3, 16
    q, K, V = rng.standard_normal((H, Dh)), rng.standard_normal((c, H, Dh)), rng.standard_normal((c, H, Dh))
    out = O.attend(q, K, V)
    ref = F.scaled_dot_product_attention(torch.from_numpy(q)[None, :, None, :],
                                         torch.from_numpy(K).permute(1, 0, 2)[None],
                                         torch.from_numpy(V).permute(1, 0, 2)[None])[0, :, 0].numpy()
    assert np.allclose(out, ref, rtol=1e-10, atol=1e-12)
    # brute force, scalar loops
    for h in range(H):
        s = [sum(q[h, i] * K[j, h, i] for i in range(Dh)) / Dh ** 0.5 for j in range(c)]
        e = [np.exp(v - max(s)) for v in s]
        o = [sum(e[j] * V[j, h, i] for j in range(c)) / sum(e) for i in range(Dh)]
        assert np.allclose(out[h], o, rtol=1e-10)


def test_rope_invariants():
    rng = np.random.default_rng(3)
    H, Dh = 2, 32
    q, k = rng.standard_normal((1, H, Dh)), rng.standard_normal((1, H, Dh))
    assert np.allclose(O.rope(q, [0], 10000.0), q)                                   # position 0 = identity
    for m, n in ((5, 3), (105, 103), (40, 38)):
        qm, kn = O.rope(q, [m], 10000.0), O.rope(k, [n], 10000.0)
        assert np.allclose(np.linalg.norm(qm, axis=-1), np.linalg.norm(q, axis=-1))  # rotation
        d = np.einsum("nhd,nhd->h", qm, kn)
        if (m, n) == (5, 3):
            d0 = d
        assert np.allclose(d, d0)                                                    # depends on m - n only
    # first pair rotates by exactly `pos` radians (frequency theta^0 = 1), pairing (i, i + Dh/2)
    e = np.zeros((1, 1, Dh)); e[0, 0, 0] = 1.0
    r = O.rope(e, [2], 10000.0)[0, 0]
    assert np.allclose([r[0], r[Dh // 2]], [np.cos(2.0), np.sin(2.0)])
    # last pair rotates by pos * theta^(-(Dh-2)/Dh)
    e = np.zeros((1, 1, Dh)); e[0, 0, Dh // 2 - 1] = 1.0
    r = O.rope(e, [7], 10000.0)[0, 0]
    a = 7 * 10000.0 ** (-(Dh - 2) / Dh)
    assert np.allclose([r[Dh // 2 - 1], r[Dh - 1]], [np.cos(a), np.sin(a)])


# ------------------------------------------------------------------ whole model vs a library transformer

def hf_llama(dims, w, layer_ids):
    """A Hugging Face Llama decoder (float64) whose layers are the oracle's layers `layer_ids`."""
    from transformers import LlamaConfig, LlamaForCausalLM
    cfg = LlamaConfig(vocab_size=dims.V, hidden_size=dims.d, intermediate_size=dims.F,
                      num_hidden_layers=len(layer_ids), num_attention_heads=dims.H,
                      num_key_value_heads=dims.H, head_dim=dims.Dh, rms_norm_eps=dims.eps,
                      rope_theta=dims.rope_theta, attention_bias=False, mlp_bias=False,
                      tie_word_embeddings=False, max_position_embeddings=512,
                      attn_implementation="eager")
    m = LlamaForCausalLM(cfg).double().eval()
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).double()
    with torch.no_grad():
        m.model.embed_tokens.weight.copy_(t(w["embed"]))
        m.model.norm.weight.copy_(t(w["g_final"]))
        m.lm_head.weight.copy_(t(w["W_lm"]))
        for i, l in enumerate(layer_ids):
            ly = m.model.layers[i]
            d = dims.d
            ly.self_attn.q_proj.weight.copy_(t(w["W_qkv"][l, :d]))
            ly.self_attn.k_proj.weight.copy_(t(w["W_qkv"][l, d:2 * d]))
            ly.self_attn.v_proj.weight.copy_(t(w["W_qkv"][l, 2 * d:]))
            ly.self_attn.o_proj.weight.copy_(t(w["W_o"][l]))
            ly.mlp.gate_proj.weight.copy_(t(w["W_gate"][l]))
            ly.mlp.up_proj.weight.copy_(t(w["W_up"][l]))
            ly.mlp.down_proj.weight.copy_(t(w["W_down"][l]))
            ly.input_layernorm.weight.copy_(t(w["g_attn"][l]))
            ly.post_attention_layernorm.weight.copy_(t(w["g_mlp"][l]))
    return m


# The library evaluates its rotary cos/sin table in float32, so agreement is to ~1e-7, not 1e-15.
def hf_logits(m, ids):
    with torch.no_grad():
        return m(torch.tensor(ids, dtype=torch.long)[None]).logits[0].numpy()


def unrolled_layer_ids(dims):
    core = list(range(dims.L_pre, dims.L_pre + dims.L_core))
    return list(range(dims.L_pre)) + core * dims.R + list(range(dims.L_pre + dims.L_core, dims.L))


@pytest.mark.parametrize("layout", [O.SHARED, O.DEPTH_INDEXED, O.FIRST_THEN_SHARED])
def test_single_loop_is_an_ordinary_decoder(layout):
    """R = 1: every cache layout reduces to a standard transformer; incremental decode must equal
    the library's full-sequence forward, logits and greedy tokens."""
    dims = SMALL.replace(R=1)
    w = small_weights(dims)
    orc = O.Oracle(dims, w, kv_layout=layout, gate_kind=O.GATE_NONE)
    prompt = synth.make_prompts(1, 9, dims.V, 5)[0]
    out = orc.generate(prompt, 6, keep_states=True)
    m = hf_llama(dims, w, unrolled_layer_ids(dims))
    ids = list(prompt) + list(out["tokens"])
    ref = hf_logits(m, ids[:-1])
    assert np.allclose(out["prefill_logits"], ref[len(prompt) - 1], rtol=1e-5, atol=2e-6)
    for j, p in enumerate(out["passes"]):
        assert np.allclose(p["logits"], ref[len(prompt) + j], rtol=1e-5, atol=2e-6)
    assert list(out["tokens"]) == list(ref[len(prompt) - 1:].argmax(-1))


def test_fixed_depth_depth_indexed_is_the_unrolled_transformer():
    """Section 1: with a fixed loop count the model unrolls into a standard transformer with
    shared weights (true for the depth-indexed cache)."""
    dims = SMALL
    w = small_weights(dims)
    orc = O.Oracle(dims, w, kv_layout=O.DEPTH_INDEXED, gate_kind=O.GATE_NONE)
    prompt = synth.make_prompts(1, 7, dims.V, 6)[0]
    out = orc.generate(prompt, 5)
    assert list(out["depths"]) == [dims.R] * 4
    m = hf_llama(dims, w, unrolled_layer_ids(dims))
    ids = list(prompt) + list(out["tokens"])
    ref = hf_logits(m, ids[:-1])
    assert np.allclose(out["prefill_logits"], ref[len(prompt) - 1], rtol=1e-5, atol=2e-6)
    for j, p in enumerate(out["passes"]):
        assert np.allclose(p["logits"], ref[len(prompt) + j], rtol=1e-5, atol=2e-6)


def test_shared_cache_changes_attention_semantics_but_not_at_prefill_last_layer():
    """Shared layout: decode differs from the unrolled transformer (section 4.2 says it changes
    the attention semantics), but a prompt of length 1 has nothing to attend to but itself, so it
    still matches."""
    dims = SMALL
    w = small_weights(dims)
    m = hf_llama(dims, w, unrolled_layer_ids(dims))
    orc = O.Oracle(dims, w, kv_layout=O.SHARED, gate_kind=O.GATE_NONE)
    one = orc.generate([3], 1)
    assert np.allclose(one["prefill_logits"], hf_logits(m, [3])[0], rtol=1e-5, atol=2e-6)
    out = orc.generate([3, 5, 8, 13], 3)
    ref = hf_logits(m, [3, 5, 8, 13] + list(out["tokens"][:-1]))
    # lock-step prefill under the shared layout still equals the unrolled model ...
    assert np.allclose(out["prefill_logits"], ref[3], rtol=1e-5, atol=2e-6)
    # ... decode does not: loop r of a new token reads the earlier tokens' final (loop R) states
    assert not np.allclose(out["passes"][0]["logits"], ref[4], rtol=1e-6)


# ------------------------------------------------------------------ exit rule

def gated(dims, w, **kw):
    return O.Oracle(dims, w, gate_kind=O.GATE_SIGMOID_CDF, **kw)


def test_exits_disabled_equals_fixed_depth():
    dims = SMALL
    w = small_weights(dims, b_gate=0.3)
    prompt = synth.make_prompts(1, 6, dims.V, 8)[0]
    a = gated(dims, w, q_or_eps=1.5).generate(prompt, 5, keep_states=True)            # threshold never reached
    b = gated(dims, w, q_or_eps=0.5).generate(prompt, 5, forced_depths=[dims.R] * 4, keep_states=True)
    c = O.Oracle(dims, w, gate_kind=O.GATE_NONE).generate(prompt, 5, keep_states=True)
    assert list(a["depths"]) == list(b["depths"]) == list(c["depths"]) == [dims.R] * 4
    assert list(a["tokens"]) == list(b["tokens"]) == list(c["tokens"])
    for pa, pb, pc in zip(a["passes"], b["passes"], c["passes"]):
        assert np.array_equal(pa["states"][-1], pb["states"][-1])
        assert np.array_equal(pa["states"][-1], pc["states"][-1])


def test_lookahead_timing_and_minimum_depth():
    dims = SMALL.replace(R=4)
    prompt = synth.make_prompts(1, 4, dims.V, 9)[0]
    w_fire = small_weights(dims, b_gate=50.0)          # lambda = 1 at every step: fires at step 1
    assert set(gated(dims, w_fire, lookahead=True).generate(prompt, 4)["depths"]) == {2}
    assert set(gated(dims, w_fire, lookahead=False).generate(prompt, 4)["depths"]) == {1}
    assert set(gated(dims, w_fire, lookahead=False, r_min=2).generate(prompt, 4)["depths"]) == {2}
    w_never = small_weights(dims, b_gate=-50.0)
    assert set(gated(dims, w_never).generate(prompt, 4)["depths"]) == {dims.R}
    # convergence gate with a huge threshold: first comparison at r = 2, one more step of delay
    l2 = lambda la: O.Oracle(dims, w_fire, gate_kind=O.GATE_L2_CONVERGENCE, q_or_eps=1e30, lookahead=la)
    assert set(l2(True).generate(prompt, 4)["depths"]) == {3}
    assert set(l2(False).generate(prompt, 4)["depths"]) == {2}
    # forced depths are obeyed and override the signal
    out = gated(dims, w_fire).generate(prompt, 5, forced_depths=[1, 3, 4, 2])
    assert list(out["depths"]) == [1, 3, 4, 2]


def test_gate_cdf_definition_and_threshold_direction():
    dims = SMALL.replace(R=4)
    w = small_weights(dims, gate_std=0.2, b_gate=-0.3)
    prompts = synth.make_prompts(3, 5, dims.V, 10)
    prompt = prompts[0]
    orc = gated(dims, w, q_or_eps=2.0, lookahead=False)
    out = orc.generate(prompt, 4, keep_states=True)
    p = out["passes"][0]
    surv = 1.0
    for r, h in enumerate(p["states"]):
        n = h / np.sqrt(np.mean(h * h) + dims.eps)
        lam = 1.0 / (1.0 + np.exp(-(n @ w["w_gate"].astype(np.float64) + float(w["b_gate"][0]))))
        surv *= 1.0 - lam
        assert abs(p["gate"][r] - (1.0 - surv)) < 1e-12
    assert all(np.diff(p["gate"]) >= 0) and 0 < p["gate"][0] < 1                       # a CDF
    # a higher threshold gives fewer early exits (appendix B.2)
    means = [np.mean([gated(dims, w, q_or_eps=q).generate(p_, 8)["depths"].mean() for p_ in prompts])
             for q in (0.2, 0.5, 0.8, 0.95)]
    assert all(np.diff(means) >= 0) and means[-1] > means[0]


def test_fig2_kv_layouts():
    """Fig. 2 right, exits (2, 1, 3): the shared cache holds each token's last state; the
    last-exited cache holds state min(slot, r_t) with the skipped slots filled by copies."""
    want = {}
    section = None
    for line in open(os.path.join(GOLDEN, "fig2_kv_layout.txt")):
        line = line.split("#")[0].strip()
        if not line:
            continue
        if line.startswith("["):
            section = line.strip("[]")
            continue
        name, *cells = line.split()
        want[(section, int(name[4:]))] = cells
    dims = SMALL.replace(R=3)
    w = small_weights(dims)
    prompt = [1, 2]
    P = len(prompt)
    exits = [2, 1, 3]
    l0 = dims.L_pre                                    # first core layer
    di = O.Oracle(dims, w, kv_layout=O.DEPTH_INDEXED, gate_kind=O.GATE_NONE).generate(prompt, 4, forced_depths=exits)
    assert list(di["depths"]) == exits
    for tok in range(3):
        pos = P + tok
        k_by_slot = [di["cache"][l0][s][0][pos] for s in range(3)]
        for s in range(3):
            cell = want[("last_exited", s + 1)][tok]
            step = int(cell.rstrip("c"))
            assert step == min(s + 1, exits[tok])
            assert np.array_equal(k_by_slot[s], k_by_slot[step - 1])
            if cell.endswith("c"):
                assert s + 1 > exits[tok]
        distinct = {k.tobytes() for k in k_by_slot}
        assert len(distinct) == exits[tok]
    # shared: the single slot holds the state of the token's last executed step
    assert [int(c) for c in want[("shared", 1)]] == exits
    sh = O.Oracle(dims, w, kv_layout=O.SHARED, gate_kind=O.GATE_NONE)
    full = sh.generate(prompt, 4, forced_depths=exits)
    for tok in range(3):
        longer = list(exits)
        longer[tok] = min(3, exits[tok] + 1) if exits[tok] < 3 else 2
        other = sh.generate(prompt, 4, forced_depths=longer, teacher_tokens=full["tokens"][:3])
        pos = P + tok
        changed = not np.array_equal(full["cache"][l0][0][0][pos], other["cache"][l0][0][0][pos])
        assert changed                                  # the slot really is overwritten by the last step
    assert O.n_slots(O.SHARED, 4) == 1 and O.n_slots(O.DEPTH_INDEXED, 4) == 4 and O.n_slots(O.FIRST_THEN_SHARED, 4) == 2
    assert [O.kv_slot(O.FIRST_THEN_SHARED, r) for r in (1, 2, 3, 4)] == [0, 1, 1, 1]


# ------------------------------------------------------------------ paging and compaction

def test_paged_gather_is_permutation_invariant():
    rng = np.random.default_rng(4)
    H, Dh, ps, c = 2, 8, 16, 70
    dense_k, dense_v = rng.standard_normal((c, H, Dh)), rng.standard_normal((c, H, Dh))
    n_pages = -(-c // ps)
    q = rng.standard_normal((H, Dh))
    outs = []
    for seed in (0, 1):
        table = np.random.default_rng(seed).permutation(11)[:n_pages]
        pool = rng.standard_normal((11, 2, H, ps, Dh))
        for j, p in enumerate(table):
            n = min(ps, c - j * ps)
            pool[p, 0, :, :n] = dense_k[j * ps:j * ps + n].transpose(1, 0, 2)
            pool[p, 1, :, :n] = dense_v[j * ps:j * ps + n].transpose(1, 0, 2)
        K, V = O.gather_pages(pool, table, c)
        assert np.array_equal(K, dense_k) and np.array_equal(V, dense_v)
        outs.append(O.attend(q, K, V))
    assert np.array_equal(outs[0], outs[1])


def test_exit_flag_and_stable_partition():
    rng = np.random.default_rng(5)
    R = 4
    n = 200
    depth = rng.integers(1, R + 1, n)
    fire = rng.random(n) < 0.3
    forced = np.where(rng.random(n) < 0.2, rng.integers(1, R + 1, n), 0)
    valid = rng.random(n) < 0.9
    flags = [O.exit_now(depth[i], R, fire[i], forced[i], 2) for i in range(n)]
    for i in range(n):
        if depth[i] == R:
            assert flags[i]
        elif forced[i] > 0:
            assert flags[i] == (forced[i] == depth[i])
        else:
            assert flags[i] == (fire[i] and depth[i] >= 2)
    surv, ex = O.stable_partition(flags, valid)
    assert len(surv) + len(ex) == valid.sum()
    assert not set(surv) & set(ex)
    assert list(surv) == sorted(surv) and list(ex) == sorted(ex)
    assert all(valid[i] and not flags[i] for i in surv) and all(valid[i] and flags[i] for i in ex)


# ------------------------------------------------------------------ scheduler worked example (Fig. 1)

def parse_fig1():
    grids, section = {}, None
    for line in open(os.path.join(GOLDEN, "fig1_slot_grid.txt")):
        line = line.split("#")[0].strip()
        if not line:
            continue
        if line.startswith("["):
            section = line.strip("[]")
            grids[section] = []
            continue
        cells = []
        for c in line.split()[1:]:
            if c == "-":
                cells.append(None)
            else:
                st, dep = c.split(":")
                s, t = st.split(".")
                cells.append((int(s) - 1, int(t) - 1, int(dep)))
        grids[section].append(cells)
    return grids


def test_fig1_slot_grid():
    traces = [[1, 3], [2, 1, 3], [2]]
    want = parse_fig1()
    for mode, passes in (("refill", 6), ("no_refill", 8)):
        grid = SO.simulate(traces, 2, mode)
        assert len(grid) == passes
        for k in range(2):
            assert [row[k] for row in grid] == want[mode][k], (mode, k)
    assert SO.refill_lower_bound(traces, 2) == 6
    # no-refill = sum over rounds of the round's maximum depth
    assert SO.recurrent_passes(traces, 2, "no_refill") == max(1, 2) + max(3, 1) + max(2, 3)


def test_scheduler_conservation_random():
    rng = np.random.default_rng(6)
    for _ in range(20):
        traces = [list(rng.integers(1, 5, rng.integers(1, 6))) for _ in range(rng.integers(1, 9))]
        slots = int(rng.integers(1, 5))
        for mode in ("refill", "no_refill"):
            grid = SO.simulate(traces, slots, mode)
            items = [c for row in grid for c in row if c is not None]
            assert len(items) == len(set(items)) == sum(sum(t) for t in traces)   # every (seq, token, depth) exactly once
            for row in grid:
                seqs = [c[0] for c in row if c is not None]
                assert len(seqs) == len(set(seqs))                                # one token in flight per sequence
        assert SO.recurrent_passes(traces, slots, "refill") >= SO.refill_lower_bound(traces, slots)
        assert SO.recurrent_passes(traces, slots, "refill") <= SO.recurrent_passes(traces, slots, "no_refill")


def test_page_allocator():
    al = SO.PageAllocator(8, 16)
    assert al.ensure(0, 0) == [0]
    assert al.ensure(1, 17) == [1, 2]
    assert al.ensure(0, 16) == [0, 3]
    al.release(1)
    assert al.ensure(2, 40) == [1, 2, 4]
    owned = [p for t in al.table.values() for p in t]
    assert len(owned) == len(set(owned)) and not set(owned) & set(al.free)
    with pytest.raises(MemoryError):
        al.ensure(3, 16 * 4)


# ------------------------------------------------------------------ synthetic input recipes

def test_truncated_geometric_closed_form():
    p = synth.truncated_geometric_p(12.0, 32)
    assert abs(p - 0.076893) < 2e-6
    d = synth.forced_exit_depths((200000,), 3)
    assert d.min() >= 1 and d.max() == 32 and abs(d.mean() - 12.0) < 0.1


# ------------------------------------------------------------------ the step-level entry of the oracle

def _dense_core_kv(orc, cache, r, t):
    """Per core layer, copies of the dense K and V of the slot loop step r uses, positions 0..t."""
    dm = orc.dm
    s = O.kv_slot(orc.layout, r)
    Ks = [cache[l][s][0][:t + 1].copy() for l in range(dm.L_pre, dm.L_pre + dm.L_core)]
    Vs = [cache[l][s][1][:t + 1].copy() for l in range(dm.L_pre, dm.L_pre + dm.L_core)]
    return Ks, Vs


@pytest.mark.parametrize("layout", [O.SHARED, O.DEPTH_INDEXED])
@pytest.mark.parametrize("kind", [O.GATE_SIGMOID_CDF, O.GATE_L2_CONVERGENCE])
def test_loop_step_row_is_the_step_inside_decode(layout, kind):
    """Eq. 1: the single-row loop step used for step-level parity must be the very step that the
    serial decoder (pinned above by the library transformer) takes.  Positions < t of a cache never
    change once their tokens have left, so the finished run's cache is the cache as it stood before
    any step of token t, apart from position t itself, which the step rewrites."""
    dims = SMALL.replace(R=4, L_pre=2)
    w = small_weights(dims, gate_std=0.3, b_gate=-0.4)
    orc = O.Oracle(dims, w, kv_layout=layout, gate_kind=kind, q_or_eps=0.5 if kind == O.GATE_SIGMOID_CDF else 0.0)
    prompt = synth.make_prompts(1, 5, dims.V, 21)[0]
    forced = [4, 2, 3, 1]
    out = orc.generate(prompt, 5, forced_depths=forced, keep_states=True)
    cache = out["cache"]
    core = range(dims.L_pre, dims.L_pre + dims.L_core)
    checked = 0
    for j, rec in enumerate(out["passes"]):
        t = len(prompt) + j
        y = int(out["tokens"][j])
        h = orc.prelude([y], np.array([t]), cache)[0]       # rewrites the prelude layers' entry t with itself
        S = 1.0
        for r in range(1, rec["depth"] + 1):
            Ks, Vs = _dense_core_kv(orc, cache, r, t)
            for a in Ks + Vs:
                a[t] = np.nan                               # the step must write position t before reading it
            h_out, g, fire, S, new_kv = orc.loop_step_row(h, t, r, Ks, Vs, S)
            assert np.array_equal(h_out, rec["states"][r - 1])
            assert g == rec["gate"][r - 1] and fire == rec["fire"][r - 1]
            if layout == O.DEPTH_INDEXED or r == rec["depth"]:
                s = O.kv_slot(layout, r)
                for i, l in enumerate(core):
                    assert np.array_equal(new_kv[i][0], cache[l][s][0][t])
                    assert np.array_equal(new_kv[i][1], cache[l][s][1][t])
            h = h_out
            checked += 1
    assert checked == sum(forced)


def test_convergence_gate_value_and_exit_depths_by_hand():
    """Appendix C.2: the value is the plain L2 distance of consecutive recurrent states (h_0 = the
    prelude output), and a token leaves one step after the first r >= 2 whose distance is below
    the threshold (section 4.3), or after step R."""
    dims = SMALL.replace(R=6, L_pre=1)
    w = small_weights(dims, seed=9)                  # a draw whose distances fall from r = 2 on
    prompt = synth.make_prompts(1, 5, dims.V, 23)[0]
    free = O.Oracle(dims, w, gate_kind=O.GATE_L2_CONVERGENCE, q_or_eps=0.0)         # never fires
    out = free.generate(prompt, 2, keep_states=True)
    rec = out["passes"][0]
    assert rec["depth"] == dims.R
    t = len(prompt)
    h0 = free.prelude([int(out["tokens"][0])], np.array([t]), out["cache"])[0]
    hs = [h0] + rec["states"]
    dist = [float(np.linalg.norm(hs[r] - hs[r - 1])) for r in range(1, dims.R + 1)]
    assert np.allclose(rec["gate"], dist, rtol=1e-13, atol=0)
    assert len(set(np.round(dist[1:], 9))) == len(dist) - 1                          # the thresholds below separate them
    # a threshold just above the r-th distance (r >= 2) and below all earlier ones from r = 2 on
    seen = 0
    for r in range(2, dims.R + 1):
        if any(dist[j - 1] <= dist[r - 1] for j in range(2, r)):
            continue
        eps = dist[r - 1] * (1 + 1e-9)
        for lookahead, want in ((True, min(dims.R, r + 1)), (False, r)):
            orc = O.Oracle(dims, w, gate_kind=O.GATE_L2_CONVERGENCE, q_or_eps=eps, lookahead=lookahead)
            got = orc.generate(prompt, 2)["depths"][0]
            assert got == want, (r, lookahead, got)
        strict = O.Oracle(dims, w, gate_kind=O.GATE_L2_CONVERGENCE, q_or_eps=dist[r - 1], lookahead=False)
        assert r == dims.R or strict.generate(prompt, 2)["depths"][0] > r             # strict "<"
        seen += 1
    assert seen >= 4
    # the first distance (h_1 against the prelude output) never counts, however small the others are
    big = O.Oracle(dims, w, gate_kind=O.GATE_L2_CONVERGENCE, q_or_eps=dist[0] * 1e6, lookahead=False)
    assert big.generate(prompt, 2)["depths"][0] == 2


def test_gate_bias_calibration_finds_a_known_step():
    """The bisection on a stand-in whose mean depth is a known decreasing step function of b."""
    class Stub:
        def __init__(self, b):
            self.b = b

        def generate(self, prompt, T):
            # depth 4 below b = 1.25, depth 3 up to 2.0, depth 2 above
            return {"depths": np.full(T - 1, 4 if self.b < 1.25 else 3 if self.b < 2.0 else 2)}
    b, mean = O.calibrate_gate_bias(Stub, [None, None], 5, 2.5, iters=40, back_off=0.05)
    assert abs(b - 1.95) < 1e-6 or abs(b - 2.05) < 1e-6          # the crossing of 2.5 is at 2.0; either side is 0.5 off
    assert mean in (2.0, 3.0)
    b, mean = O.calibrate_gate_bias(Stub, [None], 5, 3.2, iters=40, back_off=0.05)
    assert abs(b - 1.30) < 1e-6 and mean == 3.0                  # crossing of 3.2 at 1.25; 3.0 is closer than 4.0


def test_golden_gate_bias_reproduces_its_header():
    """The stored bias of the tiny config is data; its header line states what the oracle gets with it."""
    lines = open(os.path.join(GOLDEN, "c1_gate_bias.txt")).read().splitlines()
    b = float(lines[-1])
    import re
    m = re.search(r"sequences 0-1: ([\d.]+); of all 8 sequences: ([\d.]+); histogram depth 1..4: \[([\d, ]+)\]", lines[1])
    mean01, mean_all, hist = float(m.group(1)), float(m.group(2)), [int(x) for x in m.group(3).split(",")]
    dims = synth.TINY
    w = synth.weights_to_numpy(synth.make_weights(dims, seed=0, std=0.02))
    w["b_gate"] = np.array([b], dtype=np.float32)
    prompts = synth.make_prompts(8, 32, dims.V, seed=0)
    orc = O.Oracle(dims, w, gate_kind=O.GATE_SIGMOID_CDF, q_or_eps=0.5, lookahead=True)
    outs = [orc.generate(p, 16, keep_states=False) for p in prompts]
    depths = np.concatenate([o["depths"] for o in outs])
    assert abs(depths[:30].mean() - mean01) < 5e-5 and abs(depths.mean() - mean_all) < 5e-5
    assert np.bincount(depths, minlength=5)[1:].tolist() == hist
    assert depths.min() >= 2                                     # lookahead: no gate-driven exit below depth 2
    # every decision is off the threshold by more than fp32 noise (the calibration's back-off)
    margin = min(abs(g - 0.5) for o in outs for p in o["passes"] for g in p["gate"])
    print("minimum |gate value - q| over the run:", margin)
    assert margin > 1e-4
