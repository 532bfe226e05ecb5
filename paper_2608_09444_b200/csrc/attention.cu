// Paged decode attention for one query per (row, head): softmax(q K^T / sqrt(Dh)) V over positions
// 0..position of the row's (sequence, layer, slot) pages (Eq. 1: the core reads K^{(r)}_{<t}; the
// paged pool is the depth-aware cache of section 4.2).
//
// Each KV byte is used once per query (MHA, one query per row), i.e. one FMA per element: the
// kernel is an HBM streamer, not a contraction.  Work is cut into (row, head, split) items of
// kSplitTokens tokens (16 pages); a split depends only on the row's own context length, so a
// row's result is independent of the batch it runs in.  Warps fetch items from a counter; a warp
// streams a page's K tile and V tile ([16][Dh], contiguous) with 16-byte loads, LPT lanes per
// token, keeps the online-softmax state in registers, and writes an (o, m, l) partial.  A second
// kernel merges the partials of a row in split order.
#include <cstdio>
#include <cstdlib>

#include "cdb_internal.h"

namespace cdbk {

template <typename T> struct Chunk;
template <> struct Chunk<float> {
    static constexpr int EPC = 4;
    static __device__ __forceinline__ void unpack(const uint4& v, float* f) {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    }
};
template <> struct Chunk<__nv_bfloat16> {
    static constexpr int EPC = 8;
    static __device__ __forceinline__ void unpack(const uint4& v, float* f) {
        f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
        f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
        f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xffff0000u);
        f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xffff0000u);
    }
};

// streaming 16-byte load: read-only path, do not keep in L1
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

constexpr int kAttnSharedCarveoutPct = -1;   // -1: driver default (largest L1)   // share of the SM's L1/shared array configured as shared memory

struct AttnParams {
    const void* q;             // [n_rows][H*Dh]
    KvPool pool;
    RowsDev rows;
    int layer;
    int max_splits;
    int max_seqs;
    float scale_log2;          // log2(e) / sqrt(Dh)
    float* part;               // [(row*H + head)*max_splits + split][Dh + 2]
    const int32_t* item_start; // [n_rows + 1]
    int32_t* counter;
    int32_t* status;
};

// splits per row -> exclusive scan; zeroes the per-layer work counters.  One CTA.
// A row whose position lies outside [0, max_position) or beyond what its page-table row covers gets no split
// (its output is zeroed by the merge) and latches the status word; the split count never exceeds the partial
// area's max_splits per (row, head).
__global__ void __launch_bounds__(1024) attn_plan_kernel(RowsDev rows, int32_t* __restrict__ item_start,
                                                         int32_t* __restrict__ counters, int n_counters,
                                                         int max_position, int max_splits, int32_t* __restrict__ status) {
    pdl_trigger();
    pdl_wait();
    __shared__ int warp_tot[32];
    __shared__ int base;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) base = 0;
    for (int i = threadIdx.x; i < n_counters; i += 1024) counters[i] = 0;
    __syncthreads();
    for (int start = 0; start < rows.n_rows; start += 1024) {
        const int row = start + threadIdx.x;
        int ns = 0;
        if (row < rows.n_rows && rows.seq_of(row) >= 0) {
            const int pos = rows.position[row];
            if (pos >= max_position || (pos >= 0 && pos / kPageSize >= rows.page_table_stride)) atomicCAS(status, 0, kStatusPosition);
            else if (pos >= 0) ns = min((pos + kSplitTokens) / kSplitTokens, max_splits);      // ceil((pos+1)/split)
        }
        int inc = ns;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += t; }
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            int w = warp_tot[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xffffffffu, w, o); if (lane >= o) w += t; }
            warp_tot[lane] = w;
        }
        __syncthreads();
        if (row < rows.n_rows) item_start[row] = base + (warp ? warp_tot[warp - 1] : 0) + inc - ns;
        __syncthreads();
        if (threadIdx.x == 0) base += warp_tot[31];
        __syncthreads();
    }
    if (threadIdx.x == 0) item_start[rows.n_rows] = base;
}

// LAT: the variant for batches too small to fill the GPU, where a warp's own chain of memory latencies sets the
// pace: the split's page ids come from one coalesced load, and the K/V tiles of the next page are in flight
// while the current page is computed (twice the registers, which an almost empty GPU has to spare).  Same
// arithmetic in the same order as the throughput variant.
template <typename T, int DH, int LPT, int CPL, bool LAT>
__global__ void __maxnreg__(LAT ? 208 : 96) attn_split_kernel(AttnParams p) {
    pdl_trigger();
    pdl_wait();
    constexpr int EPC = Chunk<T>::EPC;
    static_assert(LPT * CPL * EPC == DH, "lane mapping must cover the head dimension");
    constexpr int TPI = 32 / LPT;               // tokens per warp iteration
    constexpr int IPP = kPageSize / TPI;        // iterations per page
    constexpr int CPT = LPT * CPL;              // 16-byte chunks per token
    const int lane = threadIdx.x & 31;
    const int g = lane / LPT, c = lane % LPT;
    const int H = p.pool.H;
    const int n_rows = p.rows.n_rows;
    const int total_items = p.item_start[n_rows] * H;
    const T* pool_base = (const T*)p.pool.base;

    for (;;) {
        int item = 0;
        if (lane == 0) item = atomicAdd(p.counter, 1);
        item = __shfl_sync(0xffffffffu, item, 0);
        if (item >= total_items) break;
        const int pair = item / H, head = item % H;
        int lo = 0, hi = n_rows;                 // last row with item_start[row] <= pair
        while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (p.item_start[mid] <= pair) lo = mid; else hi = mid; }
        const int row = lo, split = pair - p.item_start[lo];
        const int seq = p.rows.seq_of(row);
        const int slot = p.rows.slot_of(row);
        const int ctx = p.rows.position[row] + 1;
        float* part = p.part + ((size_t)(row * H + head) * p.max_splits + split) * (DH + 2);
        bool ok = seq >= 0 && seq < p.max_seqs && slot >= 0 && slot < p.rows.n_slots && split < p.max_splits;
        if (!ok) { if (lane == 0) atomicCAS(p.status, 0, kStatusSeq); continue; }
        const int tok0 = split * kSplitTokens;
        const int tok1 = min(ctx, tok0 + kSplitTokens);
        const int32_t* table = p.rows.page_table + ((size_t)seq * p.rows.n_slots + slot) * p.rows.page_table_stride;

        float qf[CPL][EPC];
        {
            const uint4* qp = (const uint4*)((const T*)p.q + (size_t)row * H * DH + (size_t)head * DH);
#pragma unroll
            for (int j = 0; j < CPL; ++j) {
                const uint4 v = qp[c + LPT * j];
                Chunk<T>::unpack(v, qf[j]);
#pragma unroll
                for (int e = 0; e < EPC; ++e) qf[j][e] *= p.scale_log2;
            }
        }
        float m = -INFINITY, l = 0.f;
        float o[CPL][EPC];
#pragma unroll
        for (int j = 0; j < CPL; ++j)
#pragma unroll
            for (int e = 0; e < EPC; ++e) o[j][e] = 0.f;

        const int page_lo = tok0 / kPageSize, page_hi = (tok1 - 1) / kPageSize;
        static_assert(kSplitTokens / kPageSize <= 32, "a split's page ids must fit one warp");
        int my_page = 0;
        if constexpr (LAT) my_page = page_lo + lane <= page_hi ? table[page_lo + lane] : -1;
        // starts the loads of one page's K and V tile; false (and a status word) when the page id is out of range
        auto issue = [&](int pi, uint4 (&kd)[IPP][CPL], uint4 (&vd)[IPP][CPL]) -> bool {
            const int page = LAT ? __shfl_sync(0xffffffffu, my_page, pi - page_lo) : table[pi];
            if (page < 0 || page >= p.pool.n_phys_pages) { if (lane == 0) atomicCAS(p.status, 0, kStatusPage); return false; }
            const uint4* kt = (const uint4*)(pool_base + p.pool.tile_offset(p.layer, page, 0, head));
            const uint4* vt = (const uint4*)(pool_base + p.pool.tile_offset(p.layer, page, 1, head));
#pragma unroll
            for (int it = 0; it < IPP; ++it)
#pragma unroll
                for (int j = 0; j < CPL; ++j) kd[it][j] = ld_stream(kt + (it * TPI + g) * CPT + c + LPT * j);
#pragma unroll
            for (int it = 0; it < IPP; ++it)
#pragma unroll
                for (int j = 0; j < CPL; ++j) vd[it][j] = ld_stream(vt + (it * TPI + g) * CPT + c + LPT * j);
            return true;
        };
        uint4 kn[LAT ? IPP : 1][LAT ? CPL : 1], vn[LAT ? IPP : 1][LAT ? CPL : 1];
        bool next_ok = false;
        if constexpr (LAT) next_ok = issue(page_lo, kn, vn);
        for (int pi = page_lo; pi <= page_hi; ++pi) {
            uint4 kr[IPP][CPL], vr[IPP][CPL];
            bool page_ok;
            if constexpr (LAT) {
#pragma unroll
                for (int it = 0; it < IPP; ++it)
#pragma unroll
                    for (int j = 0; j < CPL; ++j) { kr[it][j] = kn[it][j]; vr[it][j] = vn[it][j]; }
                page_ok = next_ok;
                if (pi < page_hi) next_ok = issue(pi + 1, kn, vn);
            } else {
                page_ok = issue(pi, kr, vr);
            }
            if (!page_ok) continue;

            float s[IPP];
            const int tbase = pi * kPageSize + g;
            float pmax = -INFINITY;
#pragma unroll
            for (int it = 0; it < IPP; ++it) {
                float acc = 0.f;
#pragma unroll
                for (int j = 0; j < CPL; ++j) {
                    float kf[EPC];
                    Chunk<T>::unpack(kr[it][j], kf);
#pragma unroll
                    for (int e = 0; e < EPC; ++e) acc = fmaf(qf[j][e], kf[e], acc);
                }
#pragma unroll
                for (int x = LPT / 2; x > 0; x >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, x);
                s[it] = (tbase + it * TPI < tok1) ? acc : -INFINITY;
                pmax = fmaxf(pmax, s[it]);
            }
#pragma unroll
            for (int x = LPT; x < 32; x <<= 1) pmax = fmaxf(pmax, __shfl_xor_sync(0xffffffffu, pmax, x));
            const float m_new = fmaxf(m, pmax);                 // finite: the page holds >= 1 valid token
            const float corr = exp2f(m - m_new);                // 0 on the first page (m = -inf)
            l *= corr;
#pragma unroll
            for (int j = 0; j < CPL; ++j)
#pragma unroll
                for (int e = 0; e < EPC; ++e) o[j][e] *= corr;
#pragma unroll
            for (int it = 0; it < IPP; ++it) {
                if (tbase + it * TPI < tok1) {                  // skip slots past the context: they may hold anything
                    const float pr = exp2f(s[it] - m_new);
                    l += pr;
#pragma unroll
                    for (int j = 0; j < CPL; ++j) {
                        float vf[EPC];
                        Chunk<T>::unpack(vr[it][j], vf);
#pragma unroll
                        for (int e = 0; e < EPC; ++e) o[j][e] = fmaf(pr, vf[e], o[j][e]);
                    }
                }
            }
            m = m_new;
        }
        // lanes of one token group hold identical l; sum l and o over the groups
#pragma unroll
        for (int x = LPT; x < 32; x <<= 1) {
            l += __shfl_xor_sync(0xffffffffu, l, x);
#pragma unroll
            for (int j = 0; j < CPL; ++j)
#pragma unroll
                for (int e = 0; e < EPC; ++e) o[j][e] += __shfl_xor_sync(0xffffffffu, o[j][e], x);
        }
        if (g == 0) {
#pragma unroll
            for (int j = 0; j < CPL; ++j)
#pragma unroll
                for (int e = 0; e < EPC; ++e) part[(c + LPT * j) * EPC + e] = o[j][e];
            if (c == 0) { part[DH] = m; part[DH + 1] = l; }
        }
    }
}

// Merge the splits of each (row, head) in split order and round to T.  One warp per (row, head).
template <typename T, int DH>
__global__ void __launch_bounds__(128) attn_merge_kernel(AttnParams p, T* __restrict__ out) {
    pdl_trigger();
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const int H = p.pool.H;
    const int wid = blockIdx.x * 4 + (threadIdx.x >> 5);
    if (blockIdx.x == 0 && threadIdx.x == 0) *p.counter = 0;      // the split kernel is done: re-arm its work counter
    if (wid >= p.rows.n_rows * H) return;
    const int row = wid / H, head = wid % H;
    T* o = out + (size_t)row * H * DH + (size_t)head * DH;
    constexpr int PER = (DH + 31) / 32;
    const int ns = min(p.item_start[row + 1] - p.item_start[row], p.max_splits);
    const int sq = p.rows.seq_of(row);
    if (sq < 0 || sq >= p.max_seqs || ns <= 0) {          // pads and rows the plan or the split kernel skipped
#pragma unroll
        for (int k = 0; k < PER; ++k) if (lane + 32 * k < DH) o[lane + 32 * k] = T(0.f);
        return;
    }
    const float* part = p.part + (size_t)(row * H + head) * p.max_splits * (DH + 2);
    // Splits are taken four at a time with all their loads issued before the first use (a loop that waits for
    // each split's loads in turn costs one memory latency per split); the sums keep their split order.
    constexpr int U = 4;
    float M = -INFINITY;
    for (int s0 = 0; s0 < ns; s0 += U) {
        float mv[U];
#pragma unroll
        for (int u = 0; u < U; ++u) mv[u] = s0 + u < ns ? part[(size_t)(s0 + u) * (DH + 2) + DH] : -INFINITY;
#pragma unroll
        for (int u = 0; u < U; ++u) M = fmaxf(M, mv[u]);
    }
    float L = 0.f, acc[PER];
#pragma unroll
    for (int k = 0; k < PER; ++k) acc[k] = 0.f;
    for (int s0 = 0; s0 < ns; s0 += U) {
        float mv[U], lv[U], ov[U][PER];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const bool on = s0 + u < ns;
            const float* ps = part + (size_t)(on ? s0 + u : s0) * (DH + 2);
            mv[u] = ps[DH]; lv[u] = ps[DH + 1];
#pragma unroll
            for (int k = 0; k < PER; ++k) ov[u][k] = lane + 32 * k < DH ? ps[lane + 32 * k] : 0.f;
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (s0 + u < ns) {
                const float w = exp2f(mv[u] - M);
                L = fmaf(lv[u], w, L);
#pragma unroll
                for (int k = 0; k < PER; ++k) if (lane + 32 * k < DH) acc[k] = fmaf(ov[u][k], w, acc[k]);
            }
        }
    }
    const float inv = 1.f / L;
#pragma unroll
    for (int k = 0; k < PER; ++k) if (lane + 32 * k < DH) o[lane + 32 * k] = T(acc[k] * inv);
}

void launch_attention_plan(const cdb* h, int ln, const RowsDev& rows, cudaStream_t st) {
    CDB_LAUNCH(h);
    launch_pdl(attn_plan_kernel, dim3(1), dim3(1024), 0, st, rows, h->lane[ln].attn_item_start, h->lane[ln].attn_counters,
               h->cfg.L_pre + h->cfg.L_core + h->cfg.L_coda, h->cfg.max_position, h->max_splits, h->status);
}

template <typename T, int DH, int LPT, int CPL, bool LAT>
static void launch_attention_t(const cdb* h, const AttnParams& p, void* o, cudaStream_t st) {
    static int per_device[kMaxDevices] = {};
    int& blocks_per_sm = per_device[h->device];
    if (blocks_per_sm == 0) {
        // The kernel uses no shared memory; asking for the largest shared-memory carve-out keeps the SM in the
        // configuration the projection kernel needs, so that its CTAs can become resident beside this one.
        cudaFuncSetAttribute(attn_split_kernel<T, DH, LPT, CPL, LAT>, cudaFuncAttributePreferredSharedMemoryCarveout,
                             tuning_int("CDB_ATTN_CARVEOUT", kAttnSharedCarveoutPct));
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks_per_sm, attn_split_kernel<T, DH, LPT, CPL, LAT>, 128, 0);
        if (blocks_per_sm < 1) blocks_per_sm = 1;
    }
    const int sms = h->part_active ? h->part_attn_sms : h->sms;
    const int max_items = p.rows.n_rows * p.pool.H * p.max_splits;
    // Warps are independent, so the CTA shape only decides how the block scheduler packs the SMs.
    // Alone: CTAs of 4 warps, as many as fit.  Sharing the GPU with the other half-batch's kernels: one
    // CTA of 4 * cap warps per SM, which leaves registers free on EVERY SM for a projection CTA
    // (small CTAs may be packed unevenly and fill some SMs completely).
    int grid = sms * blocks_per_sm, threads = 128;
    static const int forced_cap = tuning_int("CDB_ATTN_CAP", 0);      // tuning hook
    const int cap = forced_cap > 0 ? forced_cap : h->attn_ctas_per_sm_cap;
    if (cap > 0 && cap < blocks_per_sm) { grid = sms; threads = 128 * cap; }
    // tuning hook (two-stream step only): attention on this many SMs, one CTA of all its warps per SM, so that the
    // other half-batch's projection CTAs find the remaining SMs empty
    static const int part_sms = tuning_int("CDB_ATTN_SMS", 0);
    if (part_sms > 0 && part_sms <= sms && h->attn_ctas_per_sm_cap > 0) { grid = part_sms; threads = 128 * blocks_per_sm; }
    const int warps_per_cta = threads / 32;
    if ((max_items + warps_per_cta - 1) / warps_per_cta < grid) grid = (max_items + warps_per_cta - 1) / warps_per_cta;
    if (h->part_active) {
        // SM-partitioned step: the KV stream runs on the attention partition's stream (both half-batches in turn),
        // fenced by events against this half-batch's own stream on the projection partition
        const int half = h->part_active - 1;
        cudaEventRecord(h->ev_pre[half], st);
        cudaStreamWaitEvent(h->part_attn, h->ev_pre[half], 0);
        CDB_LAUNCH(h);
        launch_pdl(attn_split_kernel<T, DH, LPT, CPL, LAT>, dim3(grid), dim3(threads), 0, h->part_attn, p);
        cudaEventRecord(h->ev_post[half], h->part_attn);
        cudaStreamWaitEvent(st, h->ev_post[half], 0);
    } else {
        ProfScope ps(h, kProfAttention, st);
        CDB_LAUNCH(h);
        launch_pdl(attn_split_kernel<T, DH, LPT, CPL, LAT>, dim3(grid), dim3(threads), 0, st, p);
    }
    if (h->attn_split_done) cudaEventRecord(h->attn_split_done, st);     // the KV stream is over: the merge is tiny
    CDB_LAUNCH(h);
    const int warps = p.rows.n_rows * p.pool.H;
    launch_pdl(attn_merge_kernel<T, DH>, dim3((warps + 3) / 4), dim3(128), 0, st, p, (T*)o);
}

// Requires launch_attention_plan() for the same rows earlier on the stream (once per set of rows).
void launch_attention(const cdb* h, int ln, int layer, const RowsDev& rows, const void* q, void* o, cudaStream_t st) {
    if (rows.n_rows <= 0) return;
    AttnParams p;
    const LayerKv kv = layer_kv(h, layer, rows);
    p.q = q; p.pool = kv.pool; p.rows = kv.rows; p.layer = kv.layer; p.max_splits = h->max_splits;
    p.max_seqs = h->cfg.max_seqs;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)h->cfg.Dh);
    p.part = h->lane[ln].attn_part; p.item_start = h->lane[ln].attn_item_start; p.counter = h->lane[ln].attn_counters + layer; p.status = h->status;
    static const int force_lat = tuning_int("CDB_ATTN_LAT", -1);      // tuning hook
    // Few (row, head) pairs: the GPU is far from full whatever the contexts are, and a warp's own latency chain
    // sets the pace (measured cross-over: ~64 rows of 16 heads; above it the throughput variant wins by 0-5 %).
    const bool lat = force_lat >= 0 ? force_lat != 0 : p.rows.n_rows * p.pool.H <= 1024;
    const int Dh = h->cfg.Dh;
    if (h->cfg.dtype == CDB_BF16) {
        if (Dh == 128) { if (lat) launch_attention_t<__nv_bfloat16, 128, 8, 2, true>(h, p, o, st); else launch_attention_t<__nv_bfloat16, 128, 8, 2, false>(h, p, o, st); }
        else if (Dh == 96) { if (lat) launch_attention_t<__nv_bfloat16, 96, 4, 3, true>(h, p, o, st); else launch_attention_t<__nv_bfloat16, 96, 4, 3, false>(h, p, o, st); }
        else { if (lat) launch_attention_t<__nv_bfloat16, 64, 8, 1, true>(h, p, o, st); else launch_attention_t<__nv_bfloat16, 64, 8, 1, false>(h, p, o, st); }
    } else {
        if (Dh == 128) launch_attention_t<float, 128, 8, 4, false>(h, p, o, st);
        else if (Dh == 96) launch_attention_t<float, 96, 8, 3, false>(h, p, o, st);
        else launch_attention_t<float, 64, 8, 2, false>(h, p, o, st);
    }
}


// =====================================================================================================
// Allocation-free paged attention (cdb_paged_attention_static).
//
// Some users of this library cannot obtain device memory when they call it: a serving process that has
// handed the whole GPU to its own pool allocator at start-up, a plug-in living inside a host framework
// that forbids cudaMalloc on its threads (it synchronises the device and may fail late), or a component
// that must run within a memory budget fixed when the process started.  For them this variant of the
// paged decode attention needs no handle and no allocation: the split partials, the per-row split scan,
// the work counter and a status word live in the file-scope device array below, which every GPU that
// loads the library holds until the process exits.  The caller still passes every input and output.
//
// The array's name is only a host-side stand-in for the device object, so the host never hands it to a
// kernel; its device address is looked up once per device with cudaGetSymbolAddress (with that device
// current) on the first call made on that device.  That first call should therefore come before any
// stream capture.  All calls on a device share the array and it keeps the previous call's contents: each
// call re-initialises what must start at zero (work counter, status word, split scan) on the stream
// before use; two calls whose work overlaps on the GPU (different streams) race on it.
// =====================================================================================================
namespace {

constexpr size_t kStaticScratchBytes = size_t(8) << 20;          // 8 MiB per GPU
constexpr int kStaticMaxDevices = 64;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

unsigned char* g_static_scratch_addr[kStaticMaxDevices];         // device addresses, filled on first use

// Per-row split counts (clamped to the partial area's capacity) -> exclusive scan, and the zeroing of the
// work counter and status word.  The row count of this variant is small: one thread walks the rows.
__global__ void attn_static_plan_kernel(RowsDev rows, int max_splits, int max_context, int max_seqs,
                                        int32_t* __restrict__ item_start, int32_t* __restrict__ counter,
                                        int32_t* __restrict__ status) {
    pdl_trigger();
    pdl_wait();
    if (blockIdx.x != 0 || threadIdx.x != 0) return;
    *counter = 0;
    *status = 0;
    int acc = 0;
    for (int row = 0; row < rows.n_rows; ++row) {
        item_start[row] = acc;
        const int pos = rows.position[row];
        if (rows.seq_of(row) < 0 || pos < 0) continue;
        if (rows.seq_id[row] >= max_seqs) { *status = kStatusSeq; continue; } // no table row: skipped, output zeroed
        if (pos >= max_context) { *status = kStatusPosition; continue; }      // beyond the stated bound: row skipped
        const int ns = (pos + kSplitTokens) / kSplitTokens;
        acc += ns < max_splits ? ns : max_splits;
    }
    item_start[rows.n_rows] = acc;
}

template <typename T, int DH, int LPT, int CPL>
void launch_attention_static_t(const AttnParams& p, void* o, int max_context, cudaStream_t st) {
    launch_pdl(attn_static_plan_kernel, dim3(1), dim3(32), 0, st, p.rows, p.max_splits, max_context, p.max_seqs, const_cast<int32_t*>(p.item_start), p.counter, p.status);
    const int max_items = p.rows.n_rows * p.pool.H * p.max_splits;
    int grid = 148 * 4;
    if ((max_items + 3) / 4 < grid) grid = (max_items + 3) / 4;
    launch_pdl(attn_split_kernel<T, DH, LPT, CPL, false>, dim3(grid), dim3(128), 0, st, p);
    const int warps = p.rows.n_rows * p.pool.H;
    launch_pdl(attn_merge_kernel<T, DH>, dim3((warps + 3) / 4), dim3(128), 0, st, p, (T*)o);
}

}  // namespace
}  // namespace cdbk

extern "C" int cdb_paged_attention_static(const void* q, void* o, const void* pool, int32_t n_phys_pages, int32_t layer,
                                          const int32_t* seq_id, const int32_t* position, const int32_t* page_table,
                                          int32_t page_table_stride, int32_t n_rows, int32_t max_seqs,
                                          int32_t max_context, int32_t H, int32_t Dh, int32_t dtype, void* stream) {
    using namespace cdbk;
    if (n_rows == 0) return CDB_OK;
    if (!q || !o || !pool || !seq_id || !position || !page_table || n_rows < 0 || n_phys_pages < 1 || layer < 0 ||
        page_table_stride < 1 || max_seqs < 1 || max_context < 1 || H < 1 || (Dh != 64 && Dh != 96 && Dh != 128) ||
        (dtype != CDB_FP32 && dtype != CDB_BF16))
        return CDB_ERR_ARG;
    if ((int64_t)max_context > (int64_t)page_table_stride * kPageSize) {            // a row could index past its table row
        fprintf(stderr, "cdb_paged_attention_static: max_context=%d exceeds the %d tokens a page-table row of %d pages covers\n",
                max_context, page_table_stride * kPageSize, page_table_stride);
        return CDB_ERR_ARG;
    }
    const int max_splits = (max_context + kSplitTokens - 1) / kSplitTokens;
    const size_t head = 256;                                                        // status word, work counter
    const size_t scan = (((size_t)n_rows + 1) * sizeof(int32_t) + 255) / 256 * 256;
    const size_t part = (size_t)n_rows * H * max_splits * (size_t)(Dh + 2) * sizeof(float);
    if (head + scan + part > kStaticScratchBytes) {
        fprintf(stderr, "cdb_paged_attention_static: n_rows=%d x H=%d x ceil(max_context=%d / %d) splits needs %zu bytes of "
                        "scratch, the built-in array holds %zu\n", n_rows, H, max_context, kSplitTokens, head + scan + part,
                kStaticScratchBytes);
        return CDB_ERR_CAPACITY;
    }
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kStaticMaxDevices) return CDB_ERR_CUDA;
    if (!g_static_scratch_addr[dev]) {                                              // one-time set-up on this device
        void* addr = nullptr;
        if (cudaGetSymbolAddress(&addr, g_static_scratch) != cudaSuccess || !addr) { cudaGetLastError(); return CDB_ERR_CUDA; }
        g_static_scratch_addr[dev] = (unsigned char*)addr;
    }
    unsigned char* base = g_static_scratch_addr[dev];
    AttnParams p;
    p.q = q;
    p.pool.base = const_cast<void*>(pool); p.pool.n_phys_pages = n_phys_pages; p.pool.H = H; p.pool.Dh = Dh;
    p.rows.n_rows = n_rows; p.rows.seq_id = seq_id; p.rows.loop_depth = nullptr; p.rows.position = position;
    p.rows.kv_slot = nullptr; p.rows.forced_exit = nullptr; p.rows.page_table = page_table;
    p.rows.page_table_stride = page_table_stride; p.rows.n_slots = 1; p.rows.slot_override = 0; p.rows.n_live = nullptr;
    p.layer = layer; p.max_splits = max_splits; p.max_seqs = max_seqs;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)Dh);
    p.status = (int32_t*)base; p.counter = (int32_t*)(base + 4);
    p.item_start = (const int32_t*)(base + head); p.part = (float*)(base + head + scan);
    cudaStream_t st = (cudaStream_t)stream;
    if (dtype == CDB_BF16) {
        if (Dh == 128) launch_attention_static_t<__nv_bfloat16, 128, 8, 2>(p, o, max_context, st);
        else if (Dh == 96) launch_attention_static_t<__nv_bfloat16, 96, 4, 3>(p, o, max_context, st);
        else launch_attention_static_t<__nv_bfloat16, 64, 8, 1>(p, o, max_context, st);
    } else {
        if (Dh == 128) launch_attention_static_t<float, 128, 8, 4>(p, o, max_context, st);
        else if (Dh == 96) launch_attention_static_t<float, 96, 8, 3>(p, o, max_context, st);
        else launch_attention_static_t<float, 64, 8, 2>(p, o, max_context, st);
    }
    return cudaGetLastError() == cudaSuccess ? CDB_OK : CDB_ERR_CUDA;
}

// =====================================================================================================
// Query-tiled causal attention for prompt processing.  The rows of a prompt are consecutive positions of
// one sequence, so a tile of 32 query rows shares every K/V page it reads: a CTA of 128 threads (4 per
// query, each owning a quarter of the head dimension) stages a page's K and V tile in shared memory once
// and all 32 queries consume it.  Against one-query-per-warp decode attention this cuts the KV traffic of
// a prompt of P tokens from ~P^2/2 to ~P^2/64 tokens.  Same rounding points as the decode kernel: K, V
// and q in the pool's dtype, scores / softmax / P.V in fp32 FMAs.
// =====================================================================================================
namespace cdbk {
namespace {

constexpr int kPfTile = 32;                 // query rows per tile

// Cuts the batch into tiles: maximal runs of rows with the same sequence and consecutive positions, in
// pieces of at most `tile` rows.  tiles[i] = first row, tile_rows[i] = rows in it, in row order.  One CTA of
// 1024 threads walks the rows in chunks: a max-scan finds each row's run start, a sum-scan numbers the tiles.
__global__ void __launch_bounds__(1024) prefill_plan_kernel(RowsDev rows, int tile, int32_t* __restrict__ tiles,
                                                            int32_t* __restrict__ tile_rows, int32_t* __restrict__ n_tiles) {
    pdl_trigger();
    pdl_wait();
    __shared__ int w_max[32], w_sum[32];
    __shared__ int carry_run, carry_cnt;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int r = tid; r < rows.n_rows; r += 1024) tile_rows[r] = 0;
    if (tid == 0) { carry_run = -1; carry_cnt = 0; }
    __syncthreads();
    for (int base = 0; base < rows.n_rows; base += 1024) {
        const int r = base + tid;
        bool valid = false, start = false;
        if (r < rows.n_rows) {
            const int sq = rows.seq_of(r);
            valid = sq >= 0;
            if (valid) {
                start = r == 0;
                if (!start) {
                    const int sp = rows.seq_of(r - 1);
                    start = sp != sq || rows.position[r] != rows.position[r - 1] + 1;
                }
            }
        }
        // inclusive max-scan of (start ? r : -1), seeded with the run start carried from the previous chunk
        int rs = start ? r : -1;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) { const int o = __shfl_up_sync(0xffffffffu, rs, d); if (lane >= d) rs = max(rs, o); }
        if (lane == 31) w_max[warp] = rs;
        __syncthreads();
        int pre = carry_run;
        for (int w = 0; w < warp; ++w) pre = max(pre, w_max[w]);
        rs = max(rs, pre);
        const bool ts = valid && ((r - rs) % tile == 0);
        int cnt = ts ? 1 : 0;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) { const int o = __shfl_up_sync(0xffffffffu, cnt, d); if (lane >= d) cnt += o; }
        if (lane == 31) w_sum[warp] = cnt;
        __syncthreads();
        int pre_c = carry_cnt;
        for (int w = 0; w < warp; ++w) pre_c += w_sum[w];
        cnt += pre_c;                                                   // tiles started at or before this row
        if (ts) tiles[cnt - 1] = r;
        if (valid) atomicAdd(&tile_rows[cnt - 1], 1);
        __syncthreads();
        if (tid == 1023) { carry_run = rs; carry_cnt = cnt; }
        __syncthreads();
    }
    if (tid == 0) *n_tiles = carry_cnt;
}

template <typename T, int DH>
__global__ void __launch_bounds__(128) attn_prefill_kernel(AttnParams p, const int32_t* __restrict__ tiles,
                                                           const int32_t* __restrict__ tile_rows,
                                                           const int32_t* __restrict__ n_tiles, T* __restrict__ out) {
    pdl_trigger();
    pdl_wait();
    constexpr int EPC = Chunk<T>::EPC;
    constexpr int DQ = DH / 4;               // dims per thread
    constexpr int CH = DQ / EPC;             // 16-byte chunks per thread per token
    static_assert(DQ % EPC == 0, "a thread's dims must be whole 16-byte chunks");
    __shared__ __align__(16) unsigned char k_s[kPageSize * DH * sizeof(T)];
    __shared__ __align__(16) unsigned char v_s[kPageSize * DH * sizeof(T)];
    const int H = p.pool.H;
    const int tile = blockIdx.x, head = blockIdx.y;
    if (tile >= *n_tiles) return;
    const int row0 = tiles[tile], nq = tile_rows[tile];
    const int qi = threadIdx.x >> 2, part = threadIdx.x & 3;           // query in tile, quarter of the head dim
    const bool active = qi < nq;
    const int row = row0 + (active ? qi : 0);
    const int seq = p.rows.seq_of(row0);
    const int slot = p.rows.slot_of(row0);
    const int pos = p.rows.position[row];
    const int pos_last = p.rows.position[row0 + nq - 1];
    if (seq < 0 || seq >= p.max_seqs || slot < 0 || slot >= p.rows.n_slots || pos_last < 0 || pos_last / kPageSize >= p.rows.page_table_stride) {
        if (threadIdx.x == 0) atomicCAS(p.status, 0, kStatusSeq);
        return;
    }
    const int32_t* table = p.rows.page_table + ((size_t)seq * p.rows.n_slots + slot) * p.rows.page_table_stride;
    const T* pool_base = (const T*)p.pool.base;

    float qf[DQ], o[DQ];
    {
        const uint4* qp = (const uint4*)((const T*)p.q + (size_t)row * H * DH + (size_t)head * DH + part * DQ);
#pragma unroll
        for (int j = 0; j < CH; ++j) {
            const uint4 v = qp[j];
            Chunk<T>::unpack(v, qf + j * EPC);
        }
#pragma unroll
        for (int e = 0; e < DQ; ++e) { qf[e] *= p.scale_log2; o[e] = 0.f; }
    }
    float m = -INFINITY, l = 0.f;
    constexpr int TILE_CHUNKS = kPageSize * DH * (int)sizeof(T) / 16;
    for (int pi = 0; pi <= pos_last / kPageSize; ++pi) {
        const int page = table[pi];
        const bool page_ok = page >= 0 && page < p.pool.n_phys_pages;
        __syncthreads();                                               // previous page fully consumed
        if (page_ok) {
            const uint4* kt = (const uint4*)(pool_base + p.pool.tile_offset(p.layer, page, 0, head));
            const uint4* vt = (const uint4*)(pool_base + p.pool.tile_offset(p.layer, page, 1, head));
            for (int i = threadIdx.x; i < TILE_CHUNKS; i += 128) {
                ((uint4*)k_s)[i] = kt[i];
                ((uint4*)v_s)[i] = vt[i];
            }
        } else if (threadIdx.x == 0) {
            atomicCAS(p.status, 0, kStatusPage);
        }
        __syncthreads();
        if (!page_ok) continue;
        // tokens of this page the query may see (none for idle threads and for pages past the query's position;
        // such threads still run the score loop, whose shuffles need the whole warp)
        const int t_hi = active ? min(kPageSize, pos - pi * kPageSize + 1) : 0;
        float s[kPageSize];
        float pmax = -INFINITY;
#pragma unroll
        for (int t = 0; t < kPageSize; ++t) {
            float acc = 0.f;
            const uint4* kr = (const uint4*)(k_s + ((size_t)t * DH + part * DQ) * sizeof(T));
#pragma unroll
            for (int j = 0; j < CH; ++j) {
                float kf[EPC];
                Chunk<T>::unpack(kr[j], kf);
#pragma unroll
                for (int e = 0; e < EPC; ++e) acc = fmaf(qf[j * EPC + e], kf[e], acc);
            }
            acc += __shfl_xor_sync(0xffffffffu, acc, 1);
            acc += __shfl_xor_sync(0xffffffffu, acc, 2);
            s[t] = t < t_hi ? acc : -INFINITY;
            pmax = fmaxf(pmax, s[t]);
        }
        if (t_hi <= 0) continue;                                       // (the loop's barriers are at its top)
        const float m_new = fmaxf(m, pmax);
        const float corr = exp2f(m - m_new);
        l *= corr;
#pragma unroll
        for (int e = 0; e < DQ; ++e) o[e] *= corr;
#pragma unroll
        for (int t = 0; t < kPageSize; ++t) {
            if (t < t_hi) {
                const float pr = exp2f(s[t] - m_new);
                l += pr;
                const uint4* vr = (const uint4*)(v_s + ((size_t)t * DH + part * DQ) * sizeof(T));
#pragma unroll
                for (int j = 0; j < CH; ++j) {
                    float vf[EPC];
                    Chunk<T>::unpack(vr[j], vf);
#pragma unroll
                    for (int e = 0; e < EPC; ++e) o[j * EPC + e] = fmaf(pr, vf[e], o[j * EPC + e]);
                }
            }
        }
        m = m_new;
    }
    if (active) {
        const float inv = 1.f / l;
        T* orow = out + (size_t)row * H * DH + (size_t)head * DH + part * DQ;
#pragma unroll
        for (int e = 0; e < DQ; ++e) orow[e] = T(o[e] * inv);
    }
}

}  // namespace

// Tile list of a prompt batch into the lane's split-scan buffer (first rows), pf_tile_rows and pf_n_tiles.
void launch_prefill_plan(const cdb* h, int ln, const RowsDev& rows, int tile, cudaStream_t st) {
    const Lane& L = h->lane[ln];
    // one plan per prompt call: every layer of the call sees the same rows (prefill_attention: 1 = no plan yet,
    // otherwise 2 + the tile size of the plan in the lane's buffers)
    if (h->prefill_attention == 2 + tile) return;
    if (h->prefill_attention >= 1) h->prefill_attention = 2 + tile;
    CDB_LAUNCH(h);
    launch_pdl(prefill_plan_kernel, dim3(1), dim3(1024), 0, st, rows, tile, L.attn_item_start, L.pf_tile_rows, L.pf_n_tiles);
}

namespace {

template <typename T, int DH>
void launch_prefill_t(const cdb* h, const AttnParams& p, int ln, void* o, cudaStream_t st) {
    const Lane& L = h->lane[ln];
    // pads first: rows the tiles do not cover keep a zero output
    cudaMemsetAsync(o, 0, (size_t)p.rows.n_rows * p.pool.H * DH * sizeof(T), st);
    launch_prefill_plan(h, ln, p.rows, kPfTile, st);
    CDB_LAUNCH(h);
    dim3 grid(p.rows.n_rows, p.pool.H);                                // upper bound on tiles; surplus CTAs exit at once
    launch_pdl(attn_prefill_kernel<T, DH>, grid, dim3(128), 0, st, p, (const int32_t*)L.attn_item_start,
               (const int32_t*)L.pf_tile_rows, (const int32_t*)L.pf_n_tiles, (T*)o);
}

}  // namespace

// Causal attention of prompt rows (consecutive positions of each sequence adjacent in the batch) over the
// pages their own call has just written.  Uses the lane's split-scan buffer for its tile list.
void launch_attention_prefill(const cdb* h, int ln, int layer, const RowsDev& rows, const void* q, void* o, cudaStream_t st) {
    if (rows.n_rows <= 0) return;
    if (!(h->cfg.flags & CDB_FLAG_SIMT_PREFILL) && launch_attention_prefill_tc(h, ln, layer, rows, q, o, st)) return;
    AttnParams p;
    const LayerKv kv = layer_kv(h, layer, rows);
    p.q = q; p.pool = kv.pool; p.rows = kv.rows; p.layer = kv.layer; p.max_splits = h->max_splits;
    p.max_seqs = h->cfg.max_seqs;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)h->cfg.Dh);
    p.part = nullptr; p.item_start = nullptr; p.counter = nullptr; p.status = h->status;
    const int Dh = h->cfg.Dh;
    if (h->cfg.dtype == CDB_BF16) {
        if (Dh == 128) launch_prefill_t<__nv_bfloat16, 128>(h, p, ln, o, st);
        else if (Dh == 96) launch_prefill_t<__nv_bfloat16, 96>(h, p, ln, o, st);
        else launch_prefill_t<__nv_bfloat16, 64>(h, p, ln, o, st);
    } else {
        if (Dh == 128) launch_prefill_t<float, 128>(h, p, ln, o, st);
        else if (Dh == 96) launch_prefill_t<float, 96>(h, p, ln, o, st);
        else launch_prefill_t<float, 64>(h, p, ln, o, st);
    }
}

}  // namespace cdbk

CDB_TRACE_SETTER(trace_set_attention)
