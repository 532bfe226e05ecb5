"""Seeded synthetic inputs for the CDB hot path: shapes, weights, prompts, row descriptors,
page tables, KV fills, forced exit-depth traces and arrival traces.

This module is data only.  It holds none of the method's arithmetic (no norm, projection,
attention, gate or compaction code); both the CPU oracle's tests and the CUDA path's tests and
benchmark draw their inputs from here so that they see identical values.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np
import torch


@dataclasses.dataclass(frozen=True)
class Dims:
    """Shape of a looped decoder: prelude-core-coda split (paper section 2), MHA, SwiGLU."""

    V: int
    d: int
    H: int
    Dh: int
    F: int
    L_pre: int
    L_core: int
    L_coda: int
    R: int
    dtype: str = "bf16"          # storage / GEMM-operand type: "fp32" or "bf16"
    page_size: int = 16
    eps: float = 1e-6
    rope_theta: float = 10000.0

    @property
    def L(self) -> int:
        return self.L_pre + self.L_core + self.L_coda

    def replace(self, **kw) -> "Dims":
        return dataclasses.replace(self, **kw)


# The shapes the benchmark configs name.
TINY = Dims(V=512, d=256, H=4, Dh=64, F=688, L_pre=1, L_core=2, L_coda=1, R=4, dtype="fp32")
OURO_1P4B = Dims(V=49152, d=2048, H=16, Dh=128, F=5632, L_pre=0, L_core=24, L_coda=0, R=4)
HUGINN_3P5B = Dims(V=65536, d=5280, H=55, Dh=96, F=17920, L_pre=2, L_core=4, L_coda=2, R=32)


def to_bf16_grid(x: np.ndarray) -> np.ndarray:
    """Snap fp32 data onto bf16-representable values (round to nearest even); returns fp32."""
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16).to(torch.float32).numpy()


def _torch_dtype(dims: Dims) -> torch.dtype:
    return torch.float32 if dims.dtype == "fp32" else torch.bfloat16


def weight_shapes(dims: Dims) -> dict[str, tuple[int, ...]]:
    L, d, F, V = dims.L, dims.d, dims.F, dims.V
    return {
        "W_qkv": (L, 3 * d, d),     # rows [0,d) Q, [d,2d) K, [2d,3d) V; head-major inside each
        "W_o": (L, d, d),
        "W_gate": (L, F, d),
        "W_up": (L, F, d),
        "W_down": (L, d, F),
        "g_attn": (L, d),
        "g_mlp": (L, d),
        "embed": (V, d),
        "g_final": (d,),
        "W_lm": (V, d),
        "w_gate": (d,),
    }


def make_weights(dims: Dims, seed: int, device: str = "cpu", std: float = 0.02,
                 gate_std: float | None = None, b_gate: float = 0.0,
                 gain_jitter: float = 0.0) -> dict[str, torch.Tensor]:
    """Random-init weights, N(0, std^2); norm gains 1 (+ optional jitter so that a gain that is
    dropped or misplaced shows up); layers ordered prelude, core, coda.  Tensors come back in the
    storage dtype on `device`.  `b_gate` is returned as a 1-element fp32 tensor."""
    shapes = weight_shapes(dims)
    dt = _torch_dtype(dims)
    out: dict[str, torch.Tensor] = {}
    if device == "cpu":
        rng = np.random.default_rng(seed)
        for name, shp in shapes.items():
            if name.startswith("g_"):
                a = 1.0 + gain_jitter * rng.standard_normal(shp)
            elif name == "w_gate":
                a = (gate_std if gate_std is not None else std) * rng.standard_normal(shp)
            else:
                a = std * rng.standard_normal(shp)
            out[name] = torch.from_numpy(a.astype(np.float32)).to(dt)
    else:
        gen = torch.Generator(device=device)
        gen.manual_seed(seed)
        for name, shp in shapes.items():
            t = torch.empty(shp, dtype=dt, device=device)
            if name.startswith("g_"):
                t.normal_(1.0, gain_jitter, generator=gen) if gain_jitter > 0 else t.fill_(1.0)
            elif name == "w_gate":
                t.normal_(0.0, gate_std if gate_std is not None else std, generator=gen)
            else:
                # fill big stacks layer by layer to bound the temporary fp32 memory of normal_()
                if t.dim() == 3:
                    for l in range(t.shape[0]):
                        t[l].normal_(0.0, std, generator=gen)
                else:
                    t.normal_(0.0, std, generator=gen)
            out[name] = t
    # gate weights and bias are always fp32 (the gate reads the fp32 residual stream)
    out["w_gate"] = out["w_gate"].to(torch.float32)
    out["b_gate"] = torch.tensor([b_gate], dtype=torch.float32, device=device)
    return out


def width_scaled_std(d: int, base: float = 0.02, base_width: int = 2048) -> float:
    """Weight scale that keeps the gain of a layer (std * sqrt(d)) at that of a `base_width`-wide layer drawn at
    `base`: random-init stand-in for models wider than the 2048-wide one."""
    return base * math.sqrt(base_width / d)


def weights_to_numpy(w: dict[str, torch.Tensor]) -> dict[str, np.ndarray]:
    """Host fp32 copies (exact for bf16 storage) for the CPU oracle."""
    return {k: v.detach().to("cpu", torch.float32).numpy() for k, v in w.items()}


def make_prompts(n_seqs: int, length: int, V: int, seed: int) -> np.ndarray:
    rng = np.random.default_rng(seed)
    return rng.integers(0, V, size=(n_seqs, length), dtype=np.int64).astype(np.int32)


def make_step_rows(n_rows: int, R: int, seed: int, ctx_lo: int = 128, ctx_hi: int = 2048,
                   p_fire: float = 0.3) -> dict[str, np.ndarray]:
    """Ragged loop-step batch: distinct sequences, loop depth uniform in 1..R, context length
    uniform in ctx_lo..ctx_hi (position = context - 1), a Bernoulli(p_fire) previous-step exit
    signal, no forced exits."""
    rng = np.random.default_rng(seed)
    ctx = rng.integers(ctx_lo, ctx_hi + 1, size=n_rows)
    return {
        "seq_id": np.arange(n_rows, dtype=np.int32),
        "loop_depth": rng.integers(1, R + 1, size=n_rows).astype(np.int32),
        "position": (ctx - 1).astype(np.int32),
        "kv_slot": np.zeros(n_rows, dtype=np.int32),
        "forced_exit": np.zeros(n_rows, dtype=np.int32),
        "fire_prev": (rng.random(n_rows) < p_fire).astype(np.uint8),
    }


def make_page_table(ctx_lens: np.ndarray, page_size: int, seed: int, permute: bool = True,
                    extra_pages: int = 0) -> tuple[np.ndarray, int]:
    """One table row per sequence; entry j is the physical page of logical page j, -1 when
    unused.  Physical ids are a seeded random permutation (fragmented, as in live paged serving)
    or ascending.  Returns (table [n, max_pages] int32, number of physical pages)."""
    n_pages = (np.asarray(ctx_lens) + page_size - 1) // page_size
    total = int(n_pages.sum()) + extra_pages
    ids = np.arange(total, dtype=np.int32)
    if permute:
        ids = np.random.default_rng(seed).permutation(total).astype(np.int32)
    table = np.full((len(ctx_lens), int(n_pages.max())), -1, dtype=np.int32)
    at = 0
    for i, k in enumerate(n_pages):
        table[i, :k] = ids[at:at + k]
        at += int(k)
    return table, total


def kv_pool_shape(dims: Dims, n_phys_pages: int) -> tuple[int, ...]:
    """[layer][physical page][K/V][head][token in page][Dh]; page ids are shared by all layers."""
    return (dims.L, n_phys_pages, 2, dims.H, dims.page_size, dims.Dh)


def fill_kv_pool(pool: torch.Tensor, seed: int, std: float = 1.0) -> None:
    """N(0, std^2) fill of a KV page pool, generated on the pool's own device layer by layer."""
    gen = torch.Generator(device=pool.device)
    gen.manual_seed(seed)
    flat = pool.view(pool.shape[0], -1)
    step = 1 << 28
    for l in range(flat.shape[0]):
        for s in range(0, flat.shape[1], step):
            flat[l, s:s + step].normal_(0.0, std, generator=gen)


def truncated_geometric_p(mean: float = 12.0, cap: int = 32) -> float:
    """Success probability p with E[min(G, cap)] = (1 - (1-p)^cap) / p = mean, by bisection."""
    lo, hi = 1e-6, 1.0
    for _ in range(200):
        mid = 0.5 * (lo + hi)
        if (1.0 - (1.0 - mid) ** cap) / mid > mean:
            lo = mid
        else:
            hi = mid
    return 0.5 * (lo + hi)


def forced_exit_depths(shape: tuple[int, ...], seed: int, mean: float = 12.0, cap: int = 32) -> np.ndarray:
    """Exit depths min(cap, 1 + floor(ln u / ln(1-p))), u uniform(0,1) in float64."""
    p = truncated_geometric_p(mean, cap)
    u = np.random.default_rng(seed).random(shape)
    g = 1 + np.floor(np.log(u) / math.log1p(-p)).astype(np.int64)
    return np.minimum(cap, g).astype(np.int32)


def lognormal_lengths(n: int, seed: int, median: float, cap: int, sigma: float = 0.8, floor: int = 4) -> np.ndarray:
    z = np.random.default_rng(seed).standard_normal(n)
    return np.clip(np.rint(median * np.exp(sigma * z)), floor, cap).astype(np.int32)


def poisson_arrivals(n: int, rate: float, seed: int) -> np.ndarray:
    """Arrival times (seconds) of a Poisson process of the given rate."""
    gaps = np.random.default_rng(seed).exponential(1.0 / rate, size=n)
    return np.cumsum(gaps)
