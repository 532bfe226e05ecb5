"""CPU oracle for the looped-LM decode path served by continuous depth batching (CDB).

TEST INFRASTRUCTURE.  Plain, slow, float64 NumPy.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may use it; the CUDA product path never does, and this file shares
no code with it.

What it computes (paper section 2, Eq. 1): each sequence alone, token by token,
    h0 = P(x_t);  h_{r+1} = R(h_r, K^{(r)}_{<t});  next token = argmax C(h_{r_t})
with the recurrent core R looped serially to the token's own exit depth r_t.  Section 3 states
that CDB only schedules a given exit rule and leaves the model's outputs as they are, so this
serial definition is the expected result of any batched / refilled / reordered schedule.

Readings of points the paper leaves open (all fixed here, the CUDA path must agree):
  * block: pre-norm Llama-style layer, two RMSNorms (eps 1e-6), no biases, MHA, causal
    attention including the token itself, scale 1/sqrt(Dh), SwiGLU MLP, final RMSNorm before
    the LM head;
  * RoPE: theta 10000, rotate-half pairing (i, i + Dh/2), absolute position, the same at every
    loop depth;
  * learned gate (section 3 related work / appendix C.2 describe only a small gating head and a
    threshold q whose increase gives fewer early exits): lambda_r = sigmoid(w_g . n(h_r) + b)
    with n = RMSNorm without gain, survival S_r = prod_{j<=r}(1 - lambda_j), signal fires when
    1 - S_r >= q;
  * convergence gate (appendix C.2): fires when ||h_r - h_{r-1}||_2 < eps for r >= 2
    (h_0 is the prelude output, not a recurrent state);
  * lookahead (section 4.3): the signal of step r removes the token after step r+1; with
    lookahead off it removes it after step r.  A token always leaves after step R.  A forced
    depth (replayed exit, appendix B.2) overrides the signal;
  * shared KV cache (section 4.2): one slot per layer, overwritten at every loop step; prefill
    runs every prompt position to depth R with all positions of the prompt in lock-step;
  * depth-indexed cache: slot r-1 for loop r, with copy-on-exit of the last state into the
    skipped slots (last-exited cache); first-then-shared: slot min(r,2)-1 (appendix C.1);
  * greedy decoding, ties to the lowest token id; no EOS, output length set by the caller;
  * bf16 mode: weights, KV, GEMM A-operands (normed activations, attention output, SwiGLU
    output) and q/k/v after RoPE are rounded to bf16 (round to nearest even); residual stream,
    accumulators, softmax and gate stay wide.

Parity unpinned: the absolute numeric values of hidden states, logits and gate values (the
paper prints no worked numeric example and its trained weights are not available); they are
pinned by library special cases and invariants only (see tests).  The gate formula itself is a
reading of the paper, not something it prints.
"""
from __future__ import annotations

import numpy as np

SHARED, DEPTH_INDEXED, FIRST_THEN_SHARED = 0, 1, 2
GATE_NONE, GATE_SIGMOID_CDF, GATE_L2_CONVERGENCE = 0, 1, 2


# --------------------------------------------------------------------------- elementwise pieces

def bf16_round(x):
    """Round to the nearest bf16 value (ties to even), via the fp32 bit pattern."""
    a = np.asarray(x, dtype=np.float64).astype(np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(x))


def rmsnorm(x, g, eps):
    """x * rsqrt(mean(x^2) + eps) * g over the last axis; g=None means no gain."""
    x = np.asarray(x, dtype=np.float64)
    y = x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps)
    return y if g is None else y * g


def silu(x):
    return x / (1.0 + np.exp(-x))


def sigmoid(x):
    return 1.0 / (1.0 + np.exp(-x))


def rope(x, pos, theta):
    """Rotary embedding of x [..., n, H, Dh] at integer positions pos [n]: the pair
    (x_i, x_{i+Dh/2}) is rotated by the angle pos * theta^(-2i/Dh)."""
    x = np.asarray(x, dtype=np.float64)
    Dh = x.shape[-1]
    half = Dh // 2
    inv_freq = theta ** (-np.arange(half, dtype=np.float64) * 2.0 / Dh)
    ang = np.asarray(pos, dtype=np.float64)[:, None] * inv_freq[None, :]        # [n, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]                     # [n, 1, half]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def attend(q, K, V):
    """softmax(q K^T / sqrt(Dh)) V for one query per head.  q [H, Dh]; K, V [c, H, Dh]."""
    Dh = q.shape[-1]
    s = np.einsum("hd,chd->hc", q, K) / np.sqrt(Dh)
    s = s - s.max(axis=-1, keepdims=True)
    p = np.exp(s)
    p = p / p.sum(axis=-1, keepdims=True)
    return np.einsum("hc,chd->hd", p, V)


def gather_pages(pool_layer, table_row, n_tokens):
    """Dense [n_tokens, H, Dh] K and V of one sequence from a paged pool.
    pool_layer [phys_page, 2, H, page_size, Dh]; table_row[j] = physical page of logical page j."""
    page_size = pool_layer.shape[3]
    n_pages = (n_tokens + page_size - 1) // page_size
    pages = pool_layer[np.asarray(table_row[:n_pages])]                         # [n_pages, 2, H, ps, Dh]
    kv = np.transpose(pages, (1, 0, 3, 2, 4)).reshape(2, n_pages * page_size, pool_layer.shape[2], -1)
    return kv[0, :n_tokens].astype(np.float64), kv[1, :n_tokens].astype(np.float64)


# --------------------------------------------------------------------------- exit rule pieces

def kv_slot(layout, r):
    """Cache slot used by loop step r (1-based)."""
    if layout == SHARED:
        return 0
    if layout == DEPTH_INDEXED:
        return r - 1
    if layout == FIRST_THEN_SHARED:
        return min(r, 2) - 1
    raise ValueError(layout)


def n_slots(layout, R):
    return {SHARED: 1, DEPTH_INDEXED: R, FIRST_THEN_SHARED: 2}[layout]


def exit_now(loop_depth, R, fire_prev, forced_exit, r_min):
    """Does a row at 1-based loop_depth leave the core after this step?  Always at depth R; at a
    forced (replayed) depth when one is given; otherwise when the exit signal it carries is set
    and the depth has reached r_min."""
    if loop_depth >= R:
        return True
    if forced_exit > 0:
        return loop_depth == forced_exit
    return bool(fire_prev) and loop_depth >= r_min


def stable_partition(exit_flags, valid):
    """Survivor and exit index lists in ascending row order; rows with valid == False (pads)
    appear in neither."""
    surv = [i for i in range(len(exit_flags)) if valid[i] and not exit_flags[i]]
    ex = [i for i in range(len(exit_flags)) if valid[i] and exit_flags[i]]
    return np.asarray(surv, dtype=np.int32), np.asarray(ex, dtype=np.int32)


# --------------------------------------------------------------------------- the model

class Oracle:
    def __init__(self, dims, weights, *, kv_layout=SHARED, gate_kind=GATE_SIGMOID_CDF,
                 q_or_eps=0.5, lookahead=True, r_min=1, copy_on_exit=True):
        """dims: object with V, d, H, Dh, F, L_pre, L_core, L_coda, R, dtype, eps, rope_theta.
        weights: name -> fp32 ndarray, layers stacked in the order prelude, core, coda."""
        self.dm = dims
        self.w = {k: np.asarray(v, dtype=np.float64) for k, v in weights.items()}
        self.b_gate = float(np.asarray(weights.get("b_gate", 0.0)).reshape(-1)[0])
        self.layout = kv_layout
        self.gate_kind = gate_kind
        self.q_or_eps = float(q_or_eps)
        self.lookahead = bool(lookahead)
        self.r_min = int(r_min)
        self.copy_on_exit = copy_on_exit
        self.round = bf16_round if dims.dtype == "bf16" else (lambda x: np.asarray(x, dtype=np.float64))
        self.n_slots = n_slots(kv_layout, dims.R)

    # ---- KV cache of one sequence: [layer][slot] -> (K, V) arrays [capacity, H, Dh]
    def new_cache(self, capacity):
        dm = self.dm
        return [[(np.zeros((capacity, dm.H, dm.Dh)), np.zeros((capacity, dm.H, dm.Dh)))
                 for _ in range(self.n_slots)] for _ in range(dm.L)]

    # ---- one transformer layer over n rows of ONE sequence at the given positions.
    # The rows' k, v are written into (Kc, Vc) first; row i then attends to positions 0..pos[i].
    def layer(self, l, X, pos, Kc, Vc):
        dm, w, rnd = self.dm, self.w, self.round
        n = X.shape[0]
        a_in = rnd(rmsnorm(X, w["g_attn"][l], dm.eps))
        qkv = a_in @ w["W_qkv"][l].T
        q = qkv[:, :dm.d].reshape(n, dm.H, dm.Dh)
        k = qkv[:, dm.d:2 * dm.d].reshape(n, dm.H, dm.Dh)
        v = qkv[:, 2 * dm.d:].reshape(n, dm.H, dm.Dh)
        q = rnd(rope(q, pos, dm.rope_theta))
        k = rnd(rope(k, pos, dm.rope_theta))
        v = rnd(v)
        Kc[pos] = k
        Vc[pos] = v
        att = np.stack([attend(q[i], Kc[:pos[i] + 1], Vc[:pos[i] + 1]) for i in range(n)])
        X = X + rnd(att.reshape(n, dm.d)) @ w["W_o"][l].T
        m_in = rnd(rmsnorm(X, w["g_mlp"][l], dm.eps))
        act = rnd(silu(m_in @ w["W_gate"][l].T) * (m_in @ w["W_up"][l].T))
        return X + act @ w["W_down"][l].T

    def embed(self, tokens):
        return self.w["embed"][np.asarray(tokens)].copy()

    def prelude(self, tokens, pos, cache):
        X = self.embed(tokens)
        for l in range(self.dm.L_pre):
            X = self.layer(l, X, pos, *cache[l][0])
        return X

    def core_step(self, X, pos, cache, r):
        """One application of the recurrent core (loop step r, 1-based) to rows X."""
        dm = self.dm
        s = kv_slot(self.layout, r)
        for l in range(dm.L_pre, dm.L_pre + dm.L_core):
            X = self.layer(l, X, pos, *cache[l][s])
        return X

    def coda_logits(self, X, pos, cache):
        dm = self.dm
        for l in range(dm.L_pre + dm.L_core, dm.L):
            X = self.layer(l, X, pos, *cache[l][0])
        f = self.round(rmsnorm(X, self.w["g_final"], dm.eps))
        return f @ self.w["W_lm"].T

    @staticmethod
    def greedy(logits):
        return np.argmax(logits, axis=-1).astype(np.int32)          # first maximum = lowest id

    # ---- exit signal computed at the end of loop step r from (h_r, h_{r-1})
    def gate(self, h, h_prev, S, r):
        """Returns (gate value, fire, new survival S).  gate value = exit CDF 1 - S for the
        learned gate, the L2 distance for the convergence gate."""
        if self.gate_kind == GATE_SIGMOID_CDF:
            lam = sigmoid(float(rmsnorm(h, None, self.dm.eps) @ self.w["w_gate"]) + self.b_gate)
            S = S * (1.0 - lam)
            return 1.0 - S, (1.0 - S) >= self.q_or_eps, S
        if self.gate_kind == GATE_L2_CONVERGENCE:
            dist = float(np.sqrt(np.sum((h - h_prev) ** 2)))
            return dist, (r >= 2 and dist < self.q_or_eps), S
        return 0.0, False, S

    def copy_last_state(self, cache, pos, r_t):
        """Last-exited cache: fill the slots of the skipped steps with the state of step r_t."""
        dm = self.dm
        if self.layout != DEPTH_INDEXED or not self.copy_on_exit:
            return
        for l in range(dm.L_pre, dm.L_pre + dm.L_core):
            Ks, Vs = cache[l][r_t - 1]
            for s in range(r_t, dm.R):
                cache[l][s][0][pos] = Ks[pos]
                cache[l][s][1][pos] = Vs[pos]

    # ---- prefill: all prompt positions at full depth R in lock-step; returns logits of the last
    def prefill(self, prompt, cache):
        P = len(prompt)
        pos = np.arange(P)
        X = self.prelude(prompt, pos, cache)
        for r in range(1, self.dm.R + 1):
            X = self.core_step(X, pos, cache, r)
        return self.coda_logits(X, pos, cache)[-1]

    # ---- one decode token: input token y at position t; returns a record of the pass
    def decode_token(self, y, t, cache, forced_depth=0, keep_states=False):
        dm = self.dm
        pos = np.array([t])
        h = self.prelude([y], pos, cache)
        S, fire = 1.0, False
        gates, fires, states = [], [], []
        r = 0
        while True:
            r += 1
            h_prev = h
            h = self.core_step(h, pos, cache, r)
            g, fire_new, S = self.gate(h[0], h_prev[0], S, r)
            gates.append(g)
            fires.append(bool(fire_new))
            if keep_states:
                states.append(h[0].copy())
            signal = fire if self.lookahead else fire_new
            fire = fire_new
            if exit_now(r, dm.R, signal, forced_depth, self.r_min):
                break
        self.copy_last_state(cache, t, r)
        logits = self.coda_logits(h, pos, cache)[0]
        return {"depth": r, "gate": gates, "fire": fires, "states": states,
                "logits": logits, "token": int(self.greedy(logits))}

    # ---- whole sequence: prompt -> T generated tokens (token 1 from prefill, then T-1 adaptive passes)
    def generate(self, prompt, T, forced_depths=None, teacher_tokens=None, keep_states=False):
        """forced_depths[j] (0 = free) is the replayed exit depth of adaptive pass j.
        teacher_tokens, when given, replaces the fed-back tokens (lock-step replay)."""
        P = len(prompt)
        cache = self.new_cache(P + T)
        logits0 = self.prefill(np.asarray(prompt), cache)
        tokens = [int(self.greedy(logits0))]
        passes = []
        for j in range(T - 1):
            y = tokens[-1] if teacher_tokens is None else int(teacher_tokens[j])
            fd = 0 if forced_depths is None else int(forced_depths[j])
            rec = self.decode_token(y, P + j, cache, fd, keep_states)
            passes.append(rec)
            tokens.append(rec["token"])
        return {"tokens": np.asarray(tokens, dtype=np.int32),
                "depths": np.asarray([p["depth"] for p in passes], dtype=np.int32),
                "passes": passes, "prefill_logits": logits0, "cache": cache}

    # ---- a single loop step of one batch row on an existing cache (for step-level parity):
    # row state h at loop depth r and position t; dense per-layer caches K[l], V[l] of length >= t+1
    def loop_step_row(self, h, t, r, Ks, Vs, S=1.0):
        """Ks, Vs: lists over core layers of [c, H, Dh] arrays (already holding positions < t;
        position t is overwritten).  Returns (h_out, gate value, fire, S, [(k_t, v_t) per layer])."""
        dm = self.dm
        X = np.asarray(h, dtype=np.float64)[None, :]
        pos = np.array([t])
        new_kv = []
        for i, l in enumerate(range(dm.L_pre, dm.L_pre + dm.L_core)):
            X = self.layer(l, X, pos, Ks[i], Vs[i])
            new_kv.append((Ks[i][t].copy(), Vs[i][t].copy()))
        g, fire, S = self.gate(X[0], np.asarray(h, dtype=np.float64), S, r)
        return X[0], g, bool(fire), S, new_kv


# --------------------------------------------------------------------------- closed forms the paper prints

def kv_bytes_per_token(dims, slots, bytes_per_el=2):
    """Table 1: K and V, H*Dh each, per layer; the core's layers hold `slots` copies."""
    return 2 * dims.H * dims.Dh * bytes_per_el * (dims.L_pre + dims.L_coda + slots * dims.L_core)


def core_params(dims):
    """Appendix A: parameters of the recurrent core (4 d^2 attention + 3 d F MLP per layer)."""
    return dims.L_core * (4 * dims.d * dims.d + 3 * dims.d * dims.F)


def executed_layers(dims, r_t):
    """Section 2: L_pre + L_core * r_t + L_coda."""
    return dims.L_pre + dims.L_core * r_t + dims.L_coda


def boundary_to_core_flops(dims):
    """F0 / Fr of Eq. 2: prelude + coda layers + LM head against one core application."""
    per_layer = 4 * dims.d * dims.d + 3 * dims.d * dims.F
    return ((dims.L_pre + dims.L_coda) * per_layer + dims.V * dims.d) / (dims.L_core * per_layer)


def flop_bound(dims, mean_depth, R=None):
    """Eq. 2: (F0 + R Fr) / (F0 + dbar Fr)."""
    R = dims.R if R is None else R
    f0 = boundary_to_core_flops(dims)
    return (f0 + R) / (f0 + mean_depth)


# --------------------------------------------------------------------------- gate-bias calibration

def calibrate_gate_bias(make_oracle, prompts, T, target_mean_depth, iters=40, lo=-10.0, hi=10.0, back_off=0.05):
    """Bias b of the learned gate for which the free-running mean exit depth of `prompts` is closest
    to the target.  Mean depth falls as b grows, so b is bracketed by bisection (fixed bracket and
    iteration count); the bisection ends on a bias at which some token sits exactly on the
    threshold, so the result backs off by `back_off` to whichever side lands closer to the target.
    make_oracle(b) must return an Oracle whose gate bias is b.  Returns (b, mean depth at b)."""
    def mean_depth(b):
        orc = make_oracle(b)
        return float(np.mean(np.concatenate([orc.generate(p, T)["depths"] for p in prompts])))
    for _ in range(iters):
        mid = 0.5 * (lo + hi)
        if mean_depth(mid) > target_mean_depth:
            lo = mid
        else:
            hi = mid
    b_star = 0.5 * (lo + hi)
    cands = [(abs(mean_depth(b) - target_mean_depth), b) for b in (b_star - back_off, b_star + back_off)]
    b = min(cands)[1]
    return b, mean_depth(b)
