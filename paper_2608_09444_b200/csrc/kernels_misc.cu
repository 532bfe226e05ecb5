// Row-wise kernels of the loop step: RMSNorm, RoPE + KV page write, SwiGLU, embedding, exit gate,
// exit-flag + block-scan compaction, row gather, greedy argmax, copy-on-exit.
#include "cdb_internal.h"

namespace cdbk {

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

template <typename T> __device__ __forceinline__ void store4(T* p, float a, float b, float c, float d);
template <> __device__ __forceinline__ void store4<float>(float* p, float a, float b, float c, float d) {
    *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d);
}
template <> __device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16* p, float a, float b, float c, float d) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
    uint2 v;
    v.x = *reinterpret_cast<uint32_t*>(&lo);
    v.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(p) = v;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sum over the block in a fixed order (so a row's result does not depend on the batch around it).
template <int NT> __device__ __forceinline__ float block_sum(float v, float* smem /* [NT/32] */) {
    v = warp_sum(v);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) smem[warp] = v;
    __syncthreads();
    float t = 0.f;
#pragma unroll
    for (int i = 0; i < NT / 32; ++i) t += smem[i];
    return t;
}

// ------------------------------------------------------------------------------- RMSNorm
// out[row] = x[row] * rsqrt(mean(x^2) + eps) * gain, rounded to T.  Pad rows get zeros.
template <typename T>
__global__ void __launch_bounds__(256) rmsnorm_kernel(const float* __restrict__ x, const float* __restrict__ gain,
                                                      T* __restrict__ out, RowsDev rows, int d, float eps) {
    pdl_trigger();
    pdl_wait();
    __shared__ float red[8];
    const int row = blockIdx.x;
    const bool pad = rows.seq_of(row) < 0;
    const float* xr = x + (size_t)row * d;
    T* orow = out + (size_t)row * d;
    if (pad) {
        for (int i = threadIdx.x; i < d; i += 256) orow[i] = from_f32<T>(0.f);
        return;
    }
    float ss = 0.f;
    for (int i = threadIdx.x; i < d; i += 256) { float v = xr[i]; ss = fmaf(v, v, ss); }
    ss = block_sum<256>(ss, red);
    const float inv = rsqrtf(ss / (float)d + eps);
    for (int i = threadIdx.x; i < d; i += 256) orow[i] = from_f32<T>(xr[i] * inv * gain[i]);
}

void launch_rmsnorm(const cdb* h, const float* x, const float* gain, void* out, const RowsDev& rows, cudaStream_t st) {
    CDB_LAUNCH(h);
    if (rows.n_rows <= 0) return;
    if (h->cfg.dtype == CDB_FP32)
        launch_pdl(rmsnorm_kernel<float>, dim3(rows.n_rows), dim3(256), 0, st, x, gain, (float*)out, rows, h->cfg.d, h->cfg.eps);
    else
        launch_pdl(rmsnorm_kernel<__nv_bfloat16>, dim3(rows.n_rows), dim3(256), 0, st, x, gain, (__nv_bfloat16*)out, rows, h->cfg.d, h->cfg.eps);
}

// ------------------------------------------------------------------------------- split-K reduce + residual + RMSNorm
// x[row] += ws[0][row] + ws[1][row] + ... (fixed order); when gain != NULL also out[row] = RMSNorm(x[row]) * gain,
// i.e. the normed input of the projection that follows.  d <= 24 * 256.
template <typename T>
__global__ void __launch_bounds__(256) reduce_residual_norm_kernel(const float* __restrict__ ws, int splits, size_t split_stride,
                                                                   float* __restrict__ x, const float* __restrict__ gain,
                                                                   T* __restrict__ out, RowsDev rows, int d, float eps) {
    pdl_trigger();
    pdl_wait();
    __shared__ float red[8];
    constexpr int MAXV = 6;                                    // float4 chunks per thread: d <= 6 * 4 * 256
    const int row = blockIdx.x;
    const int d4 = d / 4;
    if (rows.seq_of(row) < 0) {
        if (gain) for (int i = threadIdx.x; i < d4; i += 256) store4<T>(out + (size_t)row * d + 4 * i, 0.f, 0.f, 0.f, 0.f);
        return;
    }
    float4 v[MAXV];
    float ss = 0.f;
#pragma unroll
    for (int k = 0; k < MAXV; ++k) {
        const int i = threadIdx.x + 256 * k;
        if (i < d4) {
            const size_t at = (size_t)row * d4 + i;
            float4 a = reinterpret_cast<const float4*>(x)[at];
            for (int s = 0; s < splits; ++s) {                 // fixed order: part 0, 1, ...
                const float4 b = __ldcg(reinterpret_cast<const float4*>(ws + (size_t)s * split_stride) + at);
                a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
            }
            if (splits > 0) reinterpret_cast<float4*>(x)[at] = a;
            v[k] = a;
            ss = fmaf(a.x, a.x, fmaf(a.y, a.y, fmaf(a.z, a.z, fmaf(a.w, a.w, ss))));
        }
    }
    if (!gain) return;
    ss = block_sum<256>(ss, red);
    const float inv = rsqrtf(ss / (float)d + eps);
#pragma unroll
    for (int k = 0; k < MAXV; ++k) {
        const int i = threadIdx.x + 256 * k;
        if (i < d4) {
            const float4 g = reinterpret_cast<const float4*>(gain)[i];
            store4<T>(out + (size_t)row * d + 4 * i, v[k].x * inv * g.x, v[k].y * inv * g.y, v[k].z * inv * g.z, v[k].w * inv * g.w);
        }
    }
}

void launch_reduce_residual_norm(const cdb* h, const float* ws, int splits, size_t split_stride, float* x, const float* gain,
                                 void* out, const RowsDev& rows, cudaStream_t st) {
    if (rows.n_rows <= 0) return;
    CDB_LAUNCH(h);
    if (h->cfg.dtype == CDB_FP32)
        launch_pdl(reduce_residual_norm_kernel<float>, dim3(rows.n_rows), dim3(256), 0, st, ws, splits, split_stride, x, gain, (float*)out, rows, h->cfg.d, h->cfg.eps);
    else
        launch_pdl(reduce_residual_norm_kernel<__nv_bfloat16>, dim3(rows.n_rows), dim3(256), 0, st, ws, splits, split_stride, x, gain, (__nv_bfloat16*)out, rows, h->cfg.d, h->cfg.eps);
}

// ------------------------------------------------------------------------------- RoPE + KV write
// Rotates q and k of every row at its position (rotate-half pairing), rounds q, k, v to T, stores
// q to qrot and k, v into the page of (seq, layer, slot) that holds the position.
// qkv arrives as `parts` split-K partial products [part][row][3d] that are summed here in part order.
template <typename T>
__global__ void __launch_bounds__(256) rope_kv_write_kernel(const float* __restrict__ qkv, int parts, size_t part_stride,
                                                            T* __restrict__ qrot, KvPool pool, RowsDev rows, int layer,
                                                            const float* __restrict__ rope_cos,
                                                            const float* __restrict__ rope_sin, int d,
                                                            int max_position, int max_seqs, int32_t* status) {
    pdl_trigger();
    pdl_wait();
    const int row = blockIdx.x;
    // the three descriptor loads go out together, then the page-table load: two memory latencies instead of four
    const int seq = rows.seq_of(row);
    const int pos = rows.position[row];
    const int slot = rows.slot_of(row);
    if (seq < 0) return;
    if (seq >= max_seqs || slot < 0 || slot >= rows.n_slots) { if (threadIdx.x == 0) atomicCAS(status, 0, kStatusSeq); return; }
    if (pos < 0 || pos >= max_position || pos / kPageSize >= rows.page_table_stride) {
        if (threadIdx.x == 0) atomicCAS(status, 0, kStatusPosition);
        return;
    }
    const int page = rows.page_table[((size_t)seq * rows.n_slots + slot) * rows.page_table_stride + pos / kPageSize];
    if (page < 0 || page >= pool.n_phys_pages) { if (threadIdx.x == 0) atomicCAS(status, 0, kStatusPage); return; }
    // four consecutive pair indices per thread: float4 loads of each split-K part, 8- or 16-byte stores
    const int Dh = pool.Dh, half = Dh / 2, q4 = half / 4;
    const float* r = qkv + (size_t)row * 3 * d;
    auto val4 = [&](int i) {
        float4 a = __ldcg(reinterpret_cast<const float4*>(r + i));
        for (int s = 1; s < parts; ++s) {
            const float4 b = __ldcg(reinterpret_cast<const float4*>(r + (size_t)s * part_stride + i));
            a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
        }
        return a;
    };
    T* base = (T*)pool.base;
    for (int idx = threadIdx.x; idx < pool.H * q4; idx += 256) {
        const int hd = idx / q4, i = (idx % q4) * 4;
        const float4 c = *reinterpret_cast<const float4*>(rope_cos + (size_t)pos * half + i);
        const float4 s = *reinterpret_cast<const float4*>(rope_sin + (size_t)pos * half + i);
        const int e = hd * Dh + i;
        const float4 q1 = val4(e), q2 = val4(e + half), k1 = val4(d + e), k2 = val4(d + e + half);
        const float4 v1 = val4(2 * d + e), v2 = val4(2 * d + e + half);
        store4<T>(qrot + (size_t)row * d + e, rope_lo(q1.x, q2.x, c.x, s.x), rope_lo(q1.y, q2.y, c.y, s.y), rope_lo(q1.z, q2.z, c.z, s.z), rope_lo(q1.w, q2.w, c.w, s.w));
        store4<T>(qrot + (size_t)row * d + e + half, rope_hi(q1.x, q2.x, c.x, s.x), rope_hi(q1.y, q2.y, c.y, s.y), rope_hi(q1.z, q2.z, c.z, s.z), rope_hi(q1.w, q2.w, c.w, s.w));
        T* kt = base + pool.tile_offset(layer, page, 0, hd) + (size_t)(pos % kPageSize) * Dh;
        T* vt = base + pool.tile_offset(layer, page, 1, hd) + (size_t)(pos % kPageSize) * Dh;
        store4<T>(kt + i, rope_lo(k1.x, k2.x, c.x, s.x), rope_lo(k1.y, k2.y, c.y, s.y), rope_lo(k1.z, k2.z, c.z, s.z), rope_lo(k1.w, k2.w, c.w, s.w));
        store4<T>(kt + i + half, rope_hi(k1.x, k2.x, c.x, s.x), rope_hi(k1.y, k2.y, c.y, s.y), rope_hi(k1.z, k2.z, c.z, s.z), rope_hi(k1.w, k2.w, c.w, s.w));
        store4<T>(vt + i, v1.x, v1.y, v1.z, v1.w);
        store4<T>(vt + i + half, v2.x, v2.y, v2.z, v2.w);
    }
}

void launch_rope_kv_write(const cdb* h, int ln, int layer, const float* qkv_parts, int parts, size_t part_stride,
                          const RowsDev& rows, cudaStream_t st) {
    CDB_LAUNCH(h);
    if (rows.n_rows <= 0) return;
    const LayerKv kv = layer_kv(h, layer, rows);
    if (h->cfg.dtype == CDB_FP32)
        launch_pdl(rope_kv_write_kernel<float>, dim3(rows.n_rows), dim3(256), 0, st, qkv_parts, parts, part_stride,
                   (float*)h->lane[ln].qrot, kv.pool, kv.rows, kv.layer, h->rope_cos, h->rope_sin, h->cfg.d, h->cfg.max_position,
                   h->cfg.max_seqs, h->status);
    else
        launch_pdl(rope_kv_write_kernel<__nv_bfloat16>, dim3(rows.n_rows), dim3(256), 0, st, qkv_parts, parts, part_stride,
                   (__nv_bfloat16*)h->lane[ln].qrot, kv.pool, kv.rows, kv.layer, h->rope_cos, h->rope_sin, h->cfg.d,
                   h->cfg.max_position, h->cfg.max_seqs, h->status);
}

// ------------------------------------------------------------------------------- SwiGLU
// act = SiLU(g) * u, rounded to T.  g = gu[0], u = gu[1], each [rows_cap][F] fp32.
template <typename T>
__global__ void swiglu_kernel(const float* __restrict__ g, const float* __restrict__ u, T* __restrict__ act, size_t n) {
    pdl_trigger();
    pdl_wait();
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const float a = g[i];
        act[i] = from_f32<T>(a / (1.f + expf(-a)) * u[i]);
    }
}

void launch_swiglu(const cdb* h, int ln, int n_rows, cudaStream_t st) {
    CDB_LAUNCH(h);
    if (n_rows <= 0) return;
    const size_t n = (size_t)n_rows * h->cfg.F;
    const int blocks = (int)((n + 255) / 256 < 148 * 8 ? (n + 255) / 256 : 148 * 8);
    const float* g = h->lane[ln].gu;
    const float* u = h->lane[ln].gu + (size_t)h->lane[ln].rows_cap * h->cfg.F;
    if (h->cfg.dtype == CDB_FP32) launch_pdl(swiglu_kernel<float>, dim3(blocks), dim3(256), 0, st, g, u, (float*)h->lane[ln].act, n);
    else launch_pdl(swiglu_kernel<__nv_bfloat16>, dim3(blocks), dim3(256), 0, st, g, u, (__nv_bfloat16*)h->lane[ln].act, n);
}

// ------------------------------------------------------------------------------- embedding
template <typename T>
__global__ void __launch_bounds__(256) embed_kernel(const T* __restrict__ table, const int32_t* __restrict__ tokens,
                                                    RowsDev rows, float* __restrict__ out, int d,
                                                    int V, int max_seqs, float* gate_S, uint8_t* gate_fire, int reset,
                                                    int32_t* status) {
    pdl_trigger();
    pdl_wait();
    const int row = blockIdx.x;
    const int seq = rows.seq_of(row);
    float* o = out + (size_t)row * d;
    const int tok = tokens[row];
    if (seq < 0 || tok < 0 || tok >= V || seq >= max_seqs) {
        if (seq >= 0 && threadIdx.x == 0) atomicCAS(status, 0, kStatusSeq);
        for (int i = threadIdx.x; i < d; i += 256) o[i] = 0.f;
        return;
    }
    const T* e = table + (size_t)tok * d;
    for (int i = threadIdx.x; i < d; i += 256) o[i] = to_f32<T>(e[i]);
    if (reset && threadIdx.x == 0) { gate_S[seq] = 1.f; gate_fire[seq] = 0; }
}

void launch_embed(const cdb* h, const int32_t* tokens, const RowsDev& rows, float* out, bool reset_gate, cudaStream_t st) {
    CDB_LAUNCH(h);
    if (rows.n_rows <= 0) return;
    if (h->cfg.dtype == CDB_FP32)
        launch_pdl(embed_kernel<float>, dim3(rows.n_rows), dim3(256), 0, st, (const float*)h->w.embed, tokens, rows, out, h->cfg.d,
            h->cfg.V, h->cfg.max_seqs, h->gate_S, h->gate_fire, reset_gate ? 1 : 0, h->status);
    else
        launch_pdl(embed_kernel<__nv_bfloat16>, dim3(rows.n_rows), dim3(256), 0, st, (const __nv_bfloat16*)h->w.embed, tokens, rows, out,
            h->cfg.d, h->cfg.V, h->cfg.max_seqs, h->gate_S, h->gate_fire, reset_gate ? 1 : 0, h->status);
}

// ------------------------------------------------------------------------------- exit gate
// One block per row; fp32 throughout; reductions in a fixed order.
__global__ void __launch_bounds__(256) gate_kernel(const float* __restrict__ x, const float* __restrict__ x_prev,
                                                   const float* __restrict__ w_gate, RowsDev rows, int d, int gate_kind,
                                                   float eps, float b_gate, float q_or_eps, int max_seqs,
                                                   float* gate_S, uint8_t* gate_fire, float* gate_val_out,
                                                   uint8_t* fire_out) {
    pdl_trigger();
    pdl_wait();
    __shared__ float red[8];
    const int row = blockIdx.x;
    const int seq = rows.seq_of(row);
    if (seq < 0 || seq >= max_seqs) {
        if (threadIdx.x == 0) { if (gate_val_out) gate_val_out[row] = 0.f; if (fire_out) fire_out[row] = 0; }
        return;
    }
    const float* xr = x + (size_t)row * d;
    float val = 0.f;
    bool fire = false;
    if (gate_kind == CDB_GATE_SIGMOID_CDF) {
        float ss = 0.f, dot = 0.f;
        for (int i = threadIdx.x; i < d; i += 256) { const float v = xr[i]; ss = fmaf(v, v, ss); dot = fmaf(v, w_gate[i], dot); }
        ss = block_sum<256>(ss, red);
        dot = block_sum<256>(dot, red);
        if (threadIdx.x == 0) {
            const float z = dot * rsqrtf(ss / (float)d + eps) + b_gate;
            const float lam = 1.f / (1.f + expf(-z));
            const float S = gate_S[seq] * (1.f - lam);
            gate_S[seq] = S;
            val = 1.f - S;
            fire = val >= q_or_eps;
        }
    } else if (gate_kind == CDB_GATE_L2_CONVERGENCE) {
        const float* pr = x_prev + (size_t)row * d;
        float ss = 0.f;
        for (int i = threadIdx.x; i < d; i += 256) { const float v = xr[i] - pr[i]; ss = fmaf(v, v, ss); }
        ss = block_sum<256>(ss, red);
        if (threadIdx.x == 0) { val = sqrtf(ss); fire = rows.loop_depth[row] >= 2 && val < q_or_eps; }
    }
    if (threadIdx.x == 0) {
        gate_fire[seq] = fire ? 1 : 0;
        if (gate_val_out) gate_val_out[row] = val;
        if (fire_out) fire_out[row] = fire ? 1 : 0;
    }
}

void launch_gate(const cdb* h, const RowsDev& rows, const float* x, const float* x_prev, float* gate_val_out,
                 uint8_t* fire_out, cudaStream_t st) {
    CDB_LAUNCH(h);
    if (rows.n_rows <= 0) return;
    launch_pdl(gate_kernel, dim3(rows.n_rows), dim3(256), 0, st, x, x_prev, h->w.w_gate, rows, h->cfg.d, h->cfg.gate_kind, h->cfg.eps,
                                             h->cfg.b_gate, h->cfg.q_or_eps, h->cfg.max_seqs, h->gate_S, h->gate_fire,
                                             gate_val_out, fire_out);
}

// ------------------------------------------------------------------------------- exit flag + compaction
// One CTA: per chunk of 1024 rows an exclusive block scan of the survivor and exit flags (warp
// shuffles, then the warp totals), carried across chunks, gives stable ascending index lists.
__global__ void __launch_bounds__(1024) compact_kernel(RowsDev rows, const uint8_t* __restrict__ fire_prev,
                                                       const uint8_t* __restrict__ gate_fire, int R, int r_min,
                                                       int max_seqs, int32_t* __restrict__ survivor_idx,
                                                       int32_t* __restrict__ exit_idx, int32_t* __restrict__ counts,
                                                       uint8_t* __restrict__ exit_flag) {
    pdl_trigger();
    pdl_wait();
    __shared__ int warp_s[32], warp_e[32];
    __shared__ int base_s, base_e;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) { base_s = 0; base_e = 0; }
    __syncthreads();
    for (int start = 0; start < rows.n_rows; start += 1024) {
        const int row = start + threadIdx.x;
        int s = 0, e = 0;
        if (row < rows.n_rows) {
            const int seq = rows.seq_of(row);
            if (seq >= 0 && seq < max_seqs) {
                const int depth = rows.loop_depth[row];
                const int forced = rows.forced_exit ? rows.forced_exit[row] : 0;
                const bool signal = fire_prev ? fire_prev[row] != 0 : gate_fire[seq] != 0;
                const bool ex = depth >= R || (forced > 0 ? forced == depth : (signal && depth >= r_min));
                e = ex ? 1 : 0;
                s = 1 - e;
            }
            exit_flag[row] = (uint8_t)e;
        }
        int ps = s, pe = e;                               // inclusive scan inside the warp
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int ts = __shfl_up_sync(0xffffffffu, ps, o), te = __shfl_up_sync(0xffffffffu, pe, o);
            if (lane >= o) { ps += ts; pe += te; }
        }
        if (lane == 31) { warp_s[warp] = ps; warp_e[warp] = pe; }
        __syncthreads();
        if (warp == 0) {
            int ws = warp_s[lane], we = warp_e[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int ts = __shfl_up_sync(0xffffffffu, ws, o), te = __shfl_up_sync(0xffffffffu, we, o);
                if (lane >= o) { ws += ts; we += te; }
            }
            warp_s[lane] = ws; warp_e[lane] = we;         // inclusive totals of warps 0..lane
        }
        __syncthreads();
        const int off_s = base_s + (warp ? warp_s[warp - 1] : 0) + ps - s;
        const int off_e = base_e + (warp ? warp_e[warp - 1] : 0) + pe - e;
        if (s) survivor_idx[off_s] = row;
        if (e) exit_idx[off_e] = row;
        __syncthreads();
        if (threadIdx.x == 0) { base_s += warp_s[31]; base_e += warp_e[31]; }
        __syncthreads();
    }
    if (threadIdx.x == 0) { counts[0] = base_s; counts[1] = base_e; }
}

void launch_compact(const cdb* h, const RowsDev& rows, const uint8_t* fire_prev, int32_t* survivor_idx,
                    int32_t* exit_idx, int32_t* counts, cudaStream_t st) {
    CDB_LAUNCH(h);
    launch_pdl(compact_kernel, dim3(1), dim3(1024), 0, st, rows, fire_prev, h->gate_fire, h->cfg.R, h->cfg.r_min, h->cfg.max_seqs,
                                       survivor_idx, exit_idx, counts, h->exit_flag);
}

// ------------------------------------------------------------------------------- row gather
__global__ void __launch_bounds__(256) gather_kernel(const float* __restrict__ src, const int32_t* __restrict__ idx,
                                                     const int32_t* __restrict__ count_dev, int max_count,
                                                     float* __restrict__ dst, int d) {
    pdl_trigger();
    pdl_wait();
    const int j = blockIdx.x;
    const int n = count_dev ? *count_dev : max_count;
    if (j >= n) return;
    const float* s = src + (size_t)idx[j] * d;
    float* o = dst + (size_t)j * d;
    for (int i = threadIdx.x; i < d; i += 256) o[i] = s[i];
}

void launch_gather(const cdb* h, const float* src, const int32_t* idx, const int32_t* count_dev, int max_count,
                   float* dst, cudaStream_t st) {
    CDB_LAUNCH(h);
    if (max_count <= 0) return;
    launch_pdl(gather_kernel, dim3(max_count), dim3(256), 0, st, src, idx, count_dev, max_count, dst, h->cfg.d);
}

// ------------------------------------------------------------------------------- greedy argmax
// First maximum (lowest token id on ties) of each row of fp32 logits.
__global__ void __launch_bounds__(256) argmax_kernel(const float* __restrict__ logits, int V, int32_t* __restrict__ out) {
    pdl_trigger();
    pdl_wait();
    __shared__ float bv[256];
    __shared__ int bi[256];
    const float* r = logits + (size_t)blockIdx.x * V;
    float best = -INFINITY;
    int at = 0x7fffffff;
    for (int i = threadIdx.x; i < V; i += 256) {
        const float v = r[i];
        if (v > best) { best = v; at = i; }               // ascending i: keeps the first maximum
    }
    bv[threadIdx.x] = best; bi[threadIdx.x] = at;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) {
            const float v = bv[threadIdx.x + o];
            const int j = bi[threadIdx.x + o];
            if (v > bv[threadIdx.x] || (v == bv[threadIdx.x] && j < bi[threadIdx.x])) { bv[threadIdx.x] = v; bi[threadIdx.x] = j; }
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) out[blockIdx.x] = bi[0] == 0x7fffffff ? 0 : bi[0];
}

void launch_argmax(const cdb* h, const float* logits, int n_rows, int32_t* token_out, cudaStream_t st) {
    CDB_LAUNCH(h);
    if (n_rows <= 0) return;
    launch_pdl(argmax_kernel, dim3(n_rows), dim3(256), 0, st, logits, h->cfg.V, token_out);
}

// ------------------------------------------------------------------------------- copy-on-exit
// Last-exited cache: k, v of the row's position in slot exit_depth-1 -> slots exit_depth..R-1.
template <typename T>
__global__ void __launch_bounds__(256) copy_on_exit_kernel(KvPool pool, RowsDev rows, const int32_t* __restrict__ exit_depth,
                                                           int layer0, int R, int max_seqs, int max_position, int32_t* status) {
    pdl_trigger();
    pdl_wait();
    const int row = blockIdx.x, layer = layer0 + blockIdx.y;
    const int seq = rows.seq_of(row);
    if (seq < 0 || seq >= max_seqs) return;
    const int pos = rows.position[row], rt = exit_depth[row];
    if (rt < 1 || rt >= R) return;
    if (rt > rows.n_slots) { if (threadIdx.x == 0) atomicCAS(status, 0, kStatusSeq); return; }
    if (pos < 0 || pos >= max_position || pos / kPageSize >= rows.page_table_stride) {
        if (threadIdx.x == 0) atomicCAS(status, 0, kStatusPosition);
        return;
    }
    const size_t trow = (size_t)seq * rows.n_slots;
    const int src_page = rows.page_table[(trow + rt - 1) * rows.page_table_stride + pos / kPageSize];
    if (src_page < 0 || src_page >= pool.n_phys_pages) { if (threadIdx.x == 0) atomicCAS(status, 0, kStatusPage); return; }
    T* base = (T*)pool.base;
    const int Dh = pool.Dh;
    for (int s = rt; s < R && s < rows.n_slots; ++s) {
        const int dst_page = rows.page_table[(trow + s) * rows.page_table_stride + pos / kPageSize];
        if (dst_page < 0 || dst_page >= pool.n_phys_pages) { if (threadIdx.x == 0) atomicCAS(status, 0, kStatusPage); continue; }
        for (int idx = threadIdx.x; idx < 2 * pool.H * Dh; idx += 256) {
            const int kv = idx / (pool.H * Dh), rem = idx % (pool.H * Dh), hd = rem / Dh, i = rem % Dh;
            const size_t so = pool.tile_offset(layer, src_page, kv, hd) + (size_t)(pos % kPageSize) * Dh + i;
            const size_t dof = pool.tile_offset(layer, dst_page, kv, hd) + (size_t)(pos % kPageSize) * Dh + i;
            base[dof] = base[so];
        }
    }
}

void launch_copy_on_exit(const cdb* h, const RowsDev& rows, const int32_t* exit_depth, cudaStream_t st) {
    CDB_LAUNCH(h);
    if (rows.n_rows <= 0 || h->cfg.L_core <= 0) return;
    dim3 grid(rows.n_rows, h->cfg.L_core);
    const int layer0 = layer_kv(h, h->cfg.L_pre, rows).layer;          // first core layer's index inside the core layers' pool
    if (h->cfg.dtype == CDB_FP32)
        launch_pdl(copy_on_exit_kernel<float>, dim3(grid), dim3(256), 0, st, h->pool, rows, exit_depth, layer0, h->cfg.R, h->cfg.max_seqs, h->cfg.max_position, h->status);
    else
        launch_pdl(copy_on_exit_kernel<__nv_bfloat16>, dim3(grid), dim3(256), 0, st, h->pool, rows, exit_depth, layer0, h->cfg.R, h->cfg.max_seqs, h->cfg.max_position, h->status);
}

}  // namespace cdbk

CDB_TRACE_SETTER(trace_set_misc)
