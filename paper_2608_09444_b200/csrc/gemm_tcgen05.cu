// bf16 projections on the 5th-generation tensor cores: y[n,N] (fp32) = or += x[n,K] . W[N,K]^T.
//
// At the row counts of a loop step (n <= a few hundred) the projections stream the weights: the
// arithmetic intensity is about n flop per weight byte.  The kernel therefore puts the WEIGHT's
// output features on the MMA's M axis (128 per tile) and the batch rows on its N axis (one MMA
// covers up to 256 rows), so that each weight tile is read exactly once and small batches waste no
// tensor work ("swap-AB").  Per CTA:
//   warp 0 (one lane)  TMA producer: W tile [128][64] and x tile [BN][64] (128-byte swizzle) into a
//                      shared-memory ring, completion on mbarriers;
//   warp 1 (one lane)  issues tcgen05.mma (M=128, N=BN, K=16) into one of two TMEM accumulators,
//                      releases ring stages and publishes accumulators with tcgen05.commit;
//   warps 2-9          epilogue: tcgen05.ld their 32-lane quarter of the accumulator (warps 2-5 the lower
//                      half of its columns, warps 6-9 the upper half) and store / add it to y (lanes =
//                      consecutive features -> coalesced rows of y).
// CTAs are persistent over (feature tile, row tile) pairs.  Every mbarrier wait is bounded: on
// expiry the CTA records a status word, lets its outstanding copies land, frees its TMEM and
// returns.
#include <cstdio>
#include <cstdlib>

#include <cuda.h>
#include <cudaTypedefs.h>

#include "cdb_internal.h"
#include "tc_common.cuh"

namespace cdbk {

namespace {

using namespace tc;

constexpr int BM = 128;            // features per tile (MMA M)
constexpr int BK = 64;             // bf16 elements per k-block = one 128-byte swizzle span
constexpr int UMMA_K = 16;
constexpr int kThreads = 320;          // producer warp, MMA warp, eight epilogue warps
constexpr int kEpiThreads = kThreads - 64;
constexpr int kMaxSmem = 196 * 1024;    // every launch then asks for the same shared-memory carve-out (no SM reconfiguration between projections)

enum { kModeStore = 0, kModeAccumulate = 1, kModeSwiGLU = 2 };

struct GemmParams {
    float* y;                   // store / accumulate: [k_splits][n][N] fp32 (split s at y + s * split_stride)
    __nv_bfloat16* act;         // SwiGLU mode: [n][N] bf16 = SiLU(x.Wg^T) * (x.Wu^T)
    int n, N, K;
    int BN;                     // rows per tile (MMA N): a multiple of 16, 64 to 256
    int n_acc;                  // accumulator sets in TMEM: 2 (the epilogue of a tile runs beside the main loop of the next) or 1
    int stages;
    int mode;
    int k_splits;               // the K range is cut into this many parts, each a tile of its own
    int w_tiled;                // weights come from the tile-major copy: tile (ft, kb) starts at row (ft * n_kb + kb) * 128
    size_t split_stride;
    uint32_t stage_out_off;     // SwiGLU mode: byte offset (from the ring base) of a [BN][128] bf16 output staging tile
    int32_t* status;
    unsigned long long* dbg;    // tuning builds: per-CTA phase time stamps (NULL = off)
};

__device__ __forceinline__ unsigned long long gtime() { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t) :: "memory"); return t; }

// What one CTA needs to know about itself to run a projection: ring base, barrier block, TMEM base.
struct CtaCtx {
    uint32_t ring, bar0, tmem_base;
    volatile int* abortp;
};

// The three roles of one projection over this CTA's share of the tiles (see the header of this file).  The
// mbarriers at cx.bar0 must be freshly initialised (all phases 0) and the ring and TMEM idle.  wait_inputs()
// is called by the producer warp after it has started the weight copies of its first ring fill and before
// its first copy of an activation tile: it must return once the activations (and the output buffers) may
// be touched.
// PAIR: the CTA is one of a pair (cluster of two) that shares every activation tile: tile = 2 x 128 features x BN rows,
// this CTA loads its own 128 features' weights and its own half of the BN activation rows; the even CTA's MMA warp
// issues for both (see tc_common.cuh).  map_x then has a box of BN / 2 rows.  The pair walks the same tile sequence.
template <bool PAIR, typename WaitInputs>
__device__ __forceinline__ void gemm_roles(const CUtensorMap* map_w, const CUtensorMap* map_w2, const CUtensorMap* map_x,
                                           const GemmParams& p, const CtaCtx& cx, WaitInputs wait_inputs) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = p.stages, BN = p.BN;
    const bool dual = p.mode == kModeSwiGLU;                                 // two weight tiles, two accumulators
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
    const int cta = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x, n_cta = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    constexpr int FT = PAIR ? 2 * BM : BM;                                   // features per tile
    const int XR = PAIR ? BN / 2 : BN;                                       // activation rows this CTA loads per tile
    const uint32_t w_bytes = BM * BK * 2, x_bytes = (uint32_t)XR * BK * 2;
    const uint32_t x_off = dual ? 2 * w_bytes : w_bytes, stage_bytes = x_off + x_bytes;
    const uint32_t acc_cols = dual ? 2u * BN : (uint32_t)BN;                 // TMEM columns of one accumulator set
    const uint32_t ring = cx.ring, bar0 = cx.bar0;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (8 + s); };
    auto acc_full_bar = [&](int a) { return bar0 + 8u * (16 + a); };
    auto acc_empty_bar = [&](int a) { return bar0 + 8u * (18 + a); };
    const int n_ftiles = (p.N + FT - 1) / FT, n_rtiles = (p.n + BN - 1) / BN;
    const int n_tiles = n_ftiles * n_rtiles * p.k_splits;                   // tile t = (split, row tile, feature tile)
    // the barrier the loads of a stage report to (a shared::cluster address: in a pair, the even CTA's)
    auto load_bar = [&](int s) { return PAIR ? map_to_cta(full_bar(s), 0u) : full_bar(s); };
    auto load = [&](uint32_t dst, const CUtensorMap* m, int s, int c0, int c1) {
        if (PAIR) tma_load_2d_pair(dst, m, load_bar(s), c0, c1); else tma_load_2d(dst, m, full_bar(s), c0, c1);
    };
    const uint32_t tx_bytes = PAIR ? 2u * stage_bytes : stage_bytes;         // both CTAs' shares arrive on one barrier
    const int n_kb = (p.K + BK - 1) / BK;
    auto kb_begin = [&](int t) { return (int)((long long)(t / (n_ftiles * n_rtiles)) * n_kb / p.k_splits); };
    auto kb_end = [&](int t) { return (int)((long long)(t / (n_ftiles * n_rtiles) + 1) * n_kb / p.k_splits); };

    if (warp == 0) {
        {
            const bool leader = elect_one();
            int s = 0; uint32_t ph = 0;
            bool ok = true;
            // The first fill of the ring runs in two passes over the same (tile, k-block) sequence: pass 0
            // arms the stage barriers and starts the weight copies, then the warp waits for the previous
            // kernel, and pass 1 adds the activation copies.  Later stages take both copies at once.
            int n_pre = 0;                                   // stages filled by pass 0
            int n_filled = 0;                                // stage fills of this CTA
            for (int pass = 0; pass < 2; ++pass) {
                if (pass == 1) wait_inputs();
                int g = 0;                                   // position in this CTA's (tile, k-block) sequence
                for (int t = cta; t < n_tiles && ok; t += n_cta) {
                    const int f0 = (t % n_ftiles) * FT + (int)rank * BM, r0 = (t / n_ftiles % n_rtiles) * BN + (int)rank * XR;
                    // Every CTA walks its k-blocks from a different starting point, so that the CTAs do not all pull
                    // the same activation lines from L2 at once.  The starting point is a function of the 256-feature
                    // group alone: the same in every form of the kernel (alone, in a pair, in a split-K cluster), so
                    // that a part is accumulated in the same order whichever form computes it.
                    const int kb0 = kb_begin(t), nk = kb_end(t) - kb0, rot = (((t % n_ftiles) * FT / (2 * BM)) * 7) % nk;
                    if (pass == 0 && g >= S) break;
                    for (int j = 0; j < nk; ++j, ++g) {
                        if (pass == 0 && g >= S) break;
                        const int kb = kb0 + (j + rot) % nk;
                        const int wc = p.w_tiled ? 0 : kb * BK, wr = p.w_tiled ? ((f0 / BM) * n_kb + kb) * BM : f0;
                        if (pass == 0) {                     // ring is empty: stage g is free
                            const uint32_t dst = ring + (uint32_t)g * stage_bytes;
                            if (leader) {
                                if (rank == 0) mbar_expect_tx(full_bar(g), tx_bytes);
                                load(dst, map_w, g, wc, wr);
                                if (dual) load(dst + w_bytes, map_w2, g, wc, wr);
                            }
                            __syncwarp();
                            n_pre = g + 1;
                            continue;
                        }
                        if (g < n_pre) {
                            if (leader) load(ring + (uint32_t)g * stage_bytes + x_off, map_x, g, kb * BK, r0);
                            __syncwarp();
                            if (++s == S) { s = 0; ph ^= 1u; }
                            continue;
                        }
                        if (!mbar_wait(empty_bar(s), ph ^ 1u, cx.abortp)) { ok = false; break; }
                        const uint32_t dst = ring + (uint32_t)s * stage_bytes;
                        if (leader) {
                            if (rank == 0) mbar_expect_tx(full_bar(s), tx_bytes);
                            load(dst, map_w, s, wc, wr);
                            if (dual) load(dst + w_bytes, map_w2, s, wc, wr);
                            load(dst + x_off, map_x, s, kb * BK, r0);
                        }
                        __syncwarp();
                        if (++s == S) { s = 0; ph ^= 1u; }
                    }
                }
                if (pass == 1) n_filled = g;
            }
            if (!ok || *cx.abortp) {                        // give copies already in flight time to land
                for (int i = 0; i < 64; ++i) __nanosleep(1000);
            } else {
                // Drain: wait until every stage this CTA filled has been released, so that no tcgen05.commit
                // arrival is still on its way when the caller re-arms the barriers for another projection.
                const int n_fill = n_filled;
                for (int j = 0; j < S && j < n_fill; ++j) {
                    const int fills = n_fill / S + (j < n_fill % S ? 1 : 0);
                    if (!mbar_wait(empty_bar(j), (uint32_t)(fills - 1) & 1u, cx.abortp)) break;
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (!PAIR || rank == 0) {
            const bool leader = elect_one();
            // instruction descriptor: fp32 accumulate, bf16 x bf16, both operands K-major, N = BN, M = 128 (256 over a pair)
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(FT >> 4) << 24);
            int s = 0; uint32_t ph = 0;
            int it = 0;
            bool ok = true;
            const long long mma_t0 = clock64();
            for (int t = cta; t < n_tiles && ok; t += n_cta, ++it) {
                const int acc = p.n_acc == 2 ? it & 1 : 0;
                const uint32_t acc_ph = (uint32_t)(p.n_acc == 2 ? it >> 1 : it) & 1u;
                if (!mbar_wait(acc_empty_bar(acc), acc_ph ^ 1u, cx.abortp)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = cx.tmem_base + (uint32_t)acc * acc_cols;
                const int kb0 = kb_begin(t), kb1 = kb_end(t);
                for (int kb = kb0; kb < kb1; ++kb) {        // arrival order of the stages; which k-block is in one does not matter here
                    if (!mbar_wait(full_bar(s), ph, cx.abortp)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_addr = ring + (uint32_t)s * stage_bytes;
                    const uint64_t a_desc = smem_desc_sw128(a_addr), a2_desc = smem_desc_sw128(a_addr + w_bytes);
                    const uint64_t b_desc = smem_desc_sw128(a_addr + x_off);
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) { // advance 32 bytes inside the swizzle span per UMMA_K
                        const uint64_t adv = (uint64_t)(k * UMMA_K * 2 >> 4);
                        const uint32_t accum = (kb > kb0 || k > 0) ? 1u : 0u;
                        if (PAIR) {
                            if (leader) umma_bf16_pair(d_tmem, a_desc + adv, b_desc + adv, idesc, accum);
                            if (leader && dual) umma_bf16_pair(d_tmem + (uint32_t)BN, a2_desc + adv, b_desc + adv, idesc, accum);
                        } else {
                            if (leader) umma_bf16(d_tmem, a_desc + adv, b_desc + adv, idesc, accum);
                            if (leader && dual) umma_bf16(d_tmem + (uint32_t)BN, a2_desc + adv, b_desc + adv, idesc, accum);
                        }
                    }
                    __syncwarp();
                    if (leader) { if (PAIR) umma_commit_pair(empty_bar(s)); else umma_commit(empty_bar(s)); }   // stage is free once these MMAs have read it
                    if (++s == S) { s = 0; ph ^= 1u; }
                }
                if (ok && leader) { if (PAIR) umma_commit_pair(acc_full_bar(acc)); else umma_commit(acc_full_bar(acc)); }   // accumulator complete
            }
            if (kTuningBuild && p.dbg && leader) p.dbg[blockIdx.x * 8 + 2] = clock64() - mma_t0;
        }
        __syncwarp();
    } else {
        const int q = warp & 3;                             // TMEM lane quarter this warp may read
        int it = 0;
        bool ok = true;
        for (int t = cta; t < n_tiles && ok; t += n_cta, ++it) {
            const int acc = p.n_acc == 2 ? it & 1 : 0;
            const uint32_t acc_ph = (uint32_t)(p.n_acc == 2 ? it >> 1 : it) & 1u;
            const int f = (t % n_ftiles) * FT + (int)rank * BM + q * 32 + lane, r0 = (t / n_ftiles % n_rtiles) * BN;
            const int split = t / (n_ftiles * n_rtiles);
            if (!mbar_wait(acc_full_bar(acc), acc_ph, cx.abortp)) { ok = false; break; }
            if (kTuningBuild && p.dbg && it == 0 && warp == 2 && lane == 0) p.dbg[blockIdx.x * 8 + 4] = gtime();
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t t_addr = cx.tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)acc * acc_cols;
            // 16 columns (= 16 batch rows) of this thread's feature per pass: a small register footprint
            const int n_real = min(BN, p.n - r0);               // columns holding real rows (warp-uniform)
            // two warps share a lane quarter: the first takes columns [0, mid), the second [mid, n_real)
            const int mid = min(n_real, ((n_real + 1) / 2 + 15) & ~15);
            const int c_beg = warp < 6 ? 0 : mid, n_cols = warp < 6 ? mid : n_real;
            if (c_beg >= n_cols && !dual) {
                // nothing in this warp's share
            } else if (dual) {
                // gate and up accumulators side by side; loads of the next 16 columns fly while these are finished
                uint32_t v[2][16], u[2][16];
                if (c_beg < n_cols) {
                    tmem_ld16(t_addr + (uint32_t)c_beg, v[0]);
                    tmem_ld16(t_addr + (uint32_t)(BN + c_beg), u[0]);
                }
#pragma unroll 1
                for (int c0 = c_beg; c0 < n_cols; c0 += 32) {
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        const int c = c0 + 16 * hh;
                        if (c >= n_cols) break;
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                        if (c + 16 < n_cols) {
                            tmem_ld16(t_addr + (uint32_t)(c + 16), v[hh ^ 1]);
                            tmem_ld16(t_addr + (uint32_t)(BN + c + 16), u[hh ^ 1]);
                        }
                        // SwiGLU, rounded to bf16, into the staging tile [row][feature of this tile] (2-byte global
                        // stores straight from here cost 7 us per tile; staged rows leave as 16-byte stores)
                        {
                            const uint32_t srow = ring + p.stage_out_off + (uint32_t)c * (BM * 2) + (uint32_t)(q * 32 + lane) * 2;
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                const float g = __uint_as_float(v[hh][j]);
                                const __nv_bfloat16 r = __float2bfloat16_rn(__fdividef(g, 1.f + __expf(-g)) * __uint_as_float(u[hh][j]));
                                asm volatile("st.shared.b16 [%0], %1;" ::"r"(srow + (uint32_t)j * (BM * 2)), "h"(*reinterpret_cast<const uint16_t*>(&r)) : "memory");
                            }
                        }
                    }
                }
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");   // the epilogue warps: tile staged
                {
                    const int et = threadIdx.x - 64;                         // index among the epilogue threads
                    const int f0t = (t % n_ftiles) * FT + (int)rank * BM;
                    for (int idx = et; idx < n_real * 16; idx += kEpiThreads) {   // 16 chunks of 8 features per row
                        const int row = idx >> 4, ch = idx & 15;
                        const int fc = f0t + ch * 8;
                        uint4 val;
                        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w)
                                     : "r"(ring + p.stage_out_off + (uint32_t)row * (BM * 2) + (uint32_t)ch * 16));
                        __nv_bfloat16* dst = p.act + (size_t)(r0 + row) * p.N + fc;
                        if (fc + 8 <= p.N) {
                            *reinterpret_cast<uint4*>(dst) = val;
                        } else {
                            const __nv_bfloat16* e = reinterpret_cast<const __nv_bfloat16*>(&val);
                            for (int k = 0; k < 8; ++k) if (fc + k < p.N) dst[k] = e[k];
                        }
                    }
                }
                asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");   // staging tile free for the next tile
            } else {
                // software pipeline: the TMEM load of the next 16 columns is in flight while these are stored
                uint32_t v[2][16];
                tmem_ld16(t_addr + (uint32_t)c_beg, v[0]);
#pragma unroll 1
                for (int c0 = c_beg; c0 < n_cols; c0 += 32) {
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        const int c = c0 + 16 * hh;
                        if (c >= n_cols) break;
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                        if (c + 16 < n_cols) tmem_ld16(t_addr + (uint32_t)(c + 16), v[hh ^ 1]);
                        if (f < p.N) {
                            float* dst = p.y + (size_t)split * p.split_stride + (size_t)(r0 + c) * p.N + f;
                            if (p.mode == kModeAccumulate) {
                                float prev[16];                  // all residual loads in flight before the first add
#pragma unroll
                                for (int j = 0; j < 16; ++j) prev[j] = (c + j < n_cols) ? __ldcg(dst + (size_t)j * p.N) : 0.f;
#pragma unroll
                                for (int j = 0; j < 16; ++j)
                                    if (c + j < n_cols) dst[(size_t)j * p.N] = prev[j] + __uint_as_float(v[hh][j]);
                            } else {
#pragma unroll
                                for (int j = 0; j < 16; ++j)
                                    if (c + j < n_cols) __stcg(dst + (size_t)j * p.N, __uint_as_float(v[hh][j]));
                            }
                        }
                    }
                }
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (kTuningBuild && p.dbg && warp == 2 && lane == 0) p.dbg[blockIdx.x * 8 + 6] = gtime();
            // the accumulator may be overwritten once BOTH CTAs of a pair have drained their halves: all arrive at the issuing CTA
            if (lane == 0) { if (PAIR && rank != 0) mbar_arrive_cluster(map_to_cta(acc_empty_bar(acc), 0u)); else mbar_arrive(acc_empty_bar(acc)); }
        }
    }

}

template <bool PAIR>
__global__ void __launch_bounds__(kThreads, 1)
gemm_bf16_tcgen05_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_w2,
                         const __grid_constant__ CUtensorMap map_x, GemmParams p) {
    pdl_trigger();
    if (kTuningBuild && p.dbg && threadIdx.x == 0) p.dbg[blockIdx.x * 8 + 0] = gtime();
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[2 * 8 + 4];          // full[stages], empty[stages], acc_full[2], acc_empty[2]
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5;
    const int S = p.stages;
    const uint32_t acc_cols = p.mode == kModeSwiGLU ? 2u * p.BN : (uint32_t)p.BN;   // TMEM columns of one accumulator set (two accumulators for gate/up)
    const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;            // swizzled tiles need 1024-byte alignment
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (8 + s); };
    auto acc_full_bar = [&](int a) { return bar0 + 8u * (16 + a); };
    auto acc_empty_bar = [&](int a) { return bar0 + 8u * (18 + a); };
    uint32_t tmem_cols = 32;                                                // a power of two that holds the accumulator sets
    while (tmem_cols < (uint32_t)p.n_acc * acc_cols) tmem_cols *= 2;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(acc_full_bar(a), 1); mbar_init(acc_empty_bar(a), (PAIR ? 2 : 1) * (kEpiThreads / 32)); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        if (PAIR) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(tmem_cols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(tmem_cols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (PAIR) cluster_sync_all();                 // the peer's barriers exist before anything arrives on them
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_slot;
    volatile int* abortp = &abort_flag;
    if (kTuningBuild && p.dbg && threadIdx.x == 0) p.dbg[blockIdx.x * 8 + 1] = gtime();
    // Set-up above overlaps the previous kernel's tail.  The weights do not depend on that kernel, so the
    // producer warp starts their copies before it waits (below); every other warp waits here.
    if (warp != 0) pdl_wait();

    CtaCtx cx;
    cx.ring = ring; cx.bar0 = bar0; cx.tmem_base = tmem_base; cx.abortp = abortp;
    gemm_roles<PAIR>(&map_w, &map_w2, &map_x, p, cx, [] { pdl_wait(); });

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (PAIR) cluster_sync_all();                 // nothing of the peer reads or signals this CTA's shared memory any more
    if (threadIdx.x == 0 && abort_flag) atomicCAS(p.status, 0, kStatusTimeout);
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (PAIR) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
        else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

// ------------------------------------------------------------------------------------------------------
// Split-K projection whose parts are summed INSIDE a thread-block cluster.  The k_splits CTAs of a cluster
// work on the same [128 features x BN rows] output tile, each on its own share of K (the same shares as the
// split-K launches above, so every part is the same number bit for bit).  Instead of writing fp32 parts to
// a workspace that a row-wise kernel reads back, the CTAs exchange them through distributed shared memory:
// the tile's columns (batch rows) are dealt out in chunks of 16 to the CTAs of the cluster, every CTA stores
// each chunk of its part into the owner's shared memory, and the owner adds the parts in part order.  What
// the owner does with the finished sums is the mode:
//   kClusterResidual  x[row][f] += sum            (output and down projections; x + part 0 + part 1 + ...)
//   kClusterRope      the tile is one head of q, k or v (Dh = 128): q and k are rotated at the row's position,
//                     q goes to the rotated-query buffer, k and v into the row's KV page (RoPE + KV write)
// One tile per CTA (no persistence: the cluster is the scheduling unit).  The cluster barriers are reached
// by every thread on every path (a bounded wait that runs out only skips work), so they cannot hang.
constexpr int kClusterResidual = 0, kClusterRope = 1;

struct ClusterParams {
    float* x;                   // residual mode: [n][N] fp32, updated in place
    int n, N, K, BN, stages, k_splits, w_tiled, mode;
    // RoPE mode
    void* qrot;                 // [n][d] bf16
    KvPool pool;
    RowsDev rows;
    int layer, d, max_position, max_seqs;
    const float* rope_cos;
    const float* rope_sin;
    int32_t* status;
    unsigned long long* dbg;    // tuning builds: per-CTA phase time stamps (NULL = off)
};

__device__ __forceinline__ void st_cluster_f32(uint32_t addr, uint32_t v) {
    asm volatile("st.shared::cluster.b32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ float4 ld_shared_f4(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint2 pack_bf16x4(float a, float b, float c, float d) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
    uint2 v;
    v.x = *reinterpret_cast<const uint32_t*>(&lo);
    v.y = *reinterpret_cast<const uint32_t*>(&hi);
    return v;
}

__global__ void __launch_bounds__(kThreads, 1)
gemm_splitk_cluster_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x, ClusterParams p) {
    pdl_trigger();
    auto stamp = [&](int k) { if (kTuningBuild && p.dbg && threadIdx.x == 64) p.dbg[blockIdx.x * 8 + k] = gtime(); };
    stamp(0);
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[2 * 8 + 1];          // full[stages], empty[stages], acc_full
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = p.stages, BN = p.BN, KS = p.k_splits;
    const uint32_t rank = cluster_ctarank();
    const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (8 + s); };
    const uint32_t acc_full = bar0 + 8u * 16;
    const uint32_t w_bytes = BM * BK * 2, x_bytes = (uint32_t)BN * BK * 2, stage_bytes = w_bytes + x_bytes;
    const uint32_t tmem_cols = (uint32_t)BN;

    const int n_ftiles = (p.N + BM - 1) / BM;
    const int tile = blockIdx.x / KS;
    const int f0 = (tile % n_ftiles) * BM, r0 = (tile / n_ftiles) * BN;
    const int n_kb = (p.K + BK - 1) / BK;
    const int kb0 = (int)((long long)rank * n_kb / KS), nk = (int)((long long)(rank + 1) * n_kb / KS) - kb0;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(acc_full, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_slot;
    volatile int* abortp = &abort_flag;
    if (warp != 0) pdl_wait();
    stamp(1);

    if (warp == 0) {
        // TMA producer: the weight tiles of the first ring fill go out before the wait for the previous kernel
        const bool leader = elect_one();
        const int n_pre = nk < S ? nk : S;
        auto w_coord = [&](int kb, int& wc, int& wr) { wc = p.w_tiled ? 0 : kb * BK; wr = p.w_tiled ? ((f0 / BM) * n_kb + kb) * BM : f0; };
        // the k-blocks of a part are taken in the same rotated order as by the workspace form of this projection
        // (a function of the feature tile only), so that both forms accumulate every part in the same order
        const int rot = (((tile % n_ftiles) / 2) * 7) % nk;
        auto kb_of = [&](int g) { return kb0 + (g + rot) % nk; };
        for (int g = 0; g < n_pre; ++g) {
            int wc, wr; w_coord(kb_of(g), wc, wr);
            if (leader) { mbar_expect_tx(full_bar(g), stage_bytes); tma_load_2d(ring + (uint32_t)g * stage_bytes, &map_w, full_bar(g), wc, wr); }
        }
        __syncwarp();
        pdl_wait();
        for (int g = 0; g < n_pre; ++g)
            if (leader) tma_load_2d(ring + (uint32_t)g * stage_bytes + w_bytes, &map_x, full_bar(g), kb_of(g) * BK, r0);
        __syncwarp();
        int s = n_pre % S; uint32_t ph = n_pre == S ? 1u : 0u;
        for (int g = n_pre; g < nk; ++g) {
            if (!mbar_wait(empty_bar(s), ph ^ 1u, abortp)) break;
            int wc, wr; w_coord(kb_of(g), wc, wr);
            const uint32_t dst = ring + (uint32_t)s * stage_bytes;
            if (leader) {
                mbar_expect_tx(full_bar(s), stage_bytes);
                tma_load_2d(dst, &map_w, full_bar(s), wc, wr);
                tma_load_2d(dst + w_bytes, &map_x, full_bar(s), kb_of(g) * BK, r0);
            }
            __syncwarp();
            if (++s == S) { s = 0; ph ^= 1u; }
        }
        __syncwarp();
    } else if (warp == 1) {
        const bool leader = elect_one();
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
        int s = 0; uint32_t ph = 0;
        bool ok = true;
        for (int g = 0; g < nk; ++g) {
            if (!mbar_wait(full_bar(s), ph, abortp)) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a_addr = ring + (uint32_t)s * stage_bytes;
            const uint64_t a_desc = smem_desc_sw128(a_addr), b_desc = smem_desc_sw128(a_addr + w_bytes);
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k) {
                const uint64_t adv = (uint64_t)(k * UMMA_K * 2 >> 4);
                if (leader) umma_bf16(tmem_base, a_desc + adv, b_desc + adv, idesc, (g > 0 || k > 0) ? 1u : 0u);
            }
            __syncwarp();
            if (leader) umma_commit(empty_bar(s));
            if (++s == S) { s = 0; ph ^= 1u; }
        }
        if (ok && leader) umma_commit(acc_full);
        __syncwarp();
    } else {
        mbar_wait(acc_full, 0u, abortp);                   // this CTA's part is complete in TMEM (or the wait gave up)
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        stamp(2);
    }
    __syncwarp();
    // Every CTA of the cluster has finished reading its ring: the rings now serve as receive buffers.
    cluster_sync_all();
    stamp(3);

    const int n_real = min(BN, p.n - r0);                   // columns of the tile that hold real rows
    const int n_chunks = (n_real + 15) / 16;                // 16-column chunks; chunk i belongs to CTA i % KS
    const bool healthy = *abortp == 0;
    if (warp >= 2 && healthy) {
        const int q = warp & 3, half = (warp - 2) >> 2;     // TMEM lane quarter; even or odd chunks
        const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t f_off = (uint32_t)(q * 32 + lane) * 4u;
        uint32_t v[2][16];                                 // the next chunk's TMEM load flies while this one is sent
        if (half < n_chunks) tmem_ld16(t_addr + (uint32_t)(half * 16), v[0]);
#pragma unroll 1
        for (int i0 = half; i0 < n_chunks; i0 += 4) {
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int i = i0 + 2 * hh;
                if (i >= n_chunks) break;
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (i + 2 < n_chunks) tmem_ld16(t_addr + (uint32_t)((i + 2) * 16), v[hh ^ 1]);
                const uint32_t owner = (uint32_t)(i % KS), li = (uint32_t)(i / KS);
                const uint32_t dst = map_to_cta(ring + ((li * (uint32_t)KS + rank) * 16u) * (BM * 4u) + f_off, owner);
#pragma unroll
                for (int j = 0; j < 16; ++j) st_cluster_f32(dst + (uint32_t)j * (BM * 4u), v[hh][j]);
            }
        }
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
    __syncwarp();
    stamp(4);
    // All parts have arrived in their owners' shared memory.
    cluster_sync_all();
    stamp(5);

    if (warp >= 2 && healthy) {
        const int et = threadIdx.x - 64;                    // 0..255
        for (int i = (int)rank; i < n_chunks; i += KS) {
            const uint32_t li = (uint32_t)(i / KS);
            const uint32_t chunk = ring + (li * (uint32_t)KS * 16u) * (BM * 4u);      // [part][16 columns][128 features]
            if (p.mode == kClusterResidual) {
                for (int idx = et; idx < 16 * (BM / 4); idx += kEpiThreads) {
                    const int j = idx / (BM / 4), f4 = idx % (BM / 4);
                    const int row = r0 + 16 * i + j, f = f0 + 4 * f4;
                    if (row >= p.n || f >= p.N) continue;
                    float4* dst = reinterpret_cast<float4*>(p.x + (size_t)row * p.N + f);
                    float4 a = __ldcg(dst);
                    for (int sp = 0; sp < KS; ++sp) {         // fixed order: x + part 0 + part 1 + ...
                        const float4 b = ld_shared_f4(chunk + (((uint32_t)sp * 16u + (uint32_t)j) * BM + 4u * (uint32_t)f4) * 4u);
                        a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
                    }
                    *dst = a;
                }
            } else {
                // the tile is head `hd` of q (which = 0), k (1) or v (2); pairs (i, i + 64) are rotated
                const int which = f0 / p.d, hd = (f0 % p.d) / BM;
                for (int idx = et; idx < 16 * 16; idx += kEpiThreads) {
                    const int j = idx / 16, i4 = (idx % 16) * 4;
                    const bool reporter = i4 == 0 && hd == 0;
                    const int row = r0 + 16 * i + j;
                    if (row >= p.n) continue;
                    const int seq = p.rows.seq_of(row);
                    if (seq < 0) continue;
                    const int pos = p.rows.position[row], slot = p.rows.slot_of(row);
                    if (seq >= p.max_seqs || slot < 0 || slot >= p.rows.n_slots) { if (reporter && which == 0) atomicCAS(p.status, 0, kStatusSeq); continue; }
                    if (pos < 0 || pos >= p.max_position || pos / kPageSize >= p.rows.page_table_stride) {
                        if (reporter && which == 0) atomicCAS(p.status, 0, kStatusPosition);
                        continue;
                    }
                    const uint32_t at = chunk + ((uint32_t)j * BM + (uint32_t)i4) * 4u;
                    float4 a1 = ld_shared_f4(at), a2 = ld_shared_f4(at + 64u * 4u);
                    for (int sp = 1; sp < KS; ++sp) {         // fixed order: part 0 + part 1 + ...
                        const float4 b1 = ld_shared_f4(at + (uint32_t)sp * 16u * BM * 4u), b2 = ld_shared_f4(at + (uint32_t)sp * 16u * BM * 4u + 64u * 4u);
                        a1.x += b1.x; a1.y += b1.y; a1.z += b1.z; a1.w += b1.w;
                        a2.x += b2.x; a2.y += b2.y; a2.z += b2.z; a2.w += b2.w;
                    }
                    __nv_bfloat16* dst;
                    if (which == 0) {
                        dst = (__nv_bfloat16*)p.qrot + (size_t)row * p.d + (size_t)hd * BM;
                    } else {
                        const int page = p.rows.page_table[((size_t)seq * p.rows.n_slots + slot) * p.rows.page_table_stride + pos / kPageSize];
                        if (page < 0 || page >= p.pool.n_phys_pages) { if (reporter && which == 1) atomicCAS(p.status, 0, kStatusPage); continue; }
                        dst = (__nv_bfloat16*)p.pool.base + p.pool.tile_offset(p.layer, page, which - 1, hd) + (size_t)(pos % kPageSize) * BM;
                    }
                    if (which < 2) {
                        const float4 c = *reinterpret_cast<const float4*>(p.rope_cos + (size_t)pos * 64 + i4);
                        const float4 sv = *reinterpret_cast<const float4*>(p.rope_sin + (size_t)pos * 64 + i4);
                        *reinterpret_cast<uint2*>(dst + i4) = pack_bf16x4(rope_lo(a1.x, a2.x, c.x, sv.x), rope_lo(a1.y, a2.y, c.y, sv.y), rope_lo(a1.z, a2.z, c.z, sv.z), rope_lo(a1.w, a2.w, c.w, sv.w));
                        *reinterpret_cast<uint2*>(dst + 64 + i4) = pack_bf16x4(rope_hi(a1.x, a2.x, c.x, sv.x), rope_hi(a1.y, a2.y, c.y, sv.y), rope_hi(a1.z, a2.z, c.z, sv.z), rope_hi(a1.w, a2.w, c.w, sv.w));
                    } else {
                        *reinterpret_cast<uint2*>(dst + i4) = pack_bf16x4(a1.x, a1.y, a1.z, a1.w);
                        *reinterpret_cast<uint2*>(dst + 64 + i4) = pack_bf16x4(a2.x, a2.y, a2.z, a2.w);
                    }
                }
            }
        }
    }
    stamp(6);
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicCAS(p.status, 0, kStatusTimeout);
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

// ------------------------------------------------------------------------------------------------------
// Several dependent stages of a layer in ONE launch (opt-in, CDB_FLAG_FUSED_STAGES): projections (as above)
// and the row-wise "sum the split-K parts + residual + RMSNorm" step, separated by grid-wide barriers instead
// of kernel boundaries; the producer warp starts the NEXT projection's weight copies before it waits at the
// barrier.  The launch is cooperative (every CTA resident), all waits are bounded.  Measured: a barrier
// among 148 CTAs plus re-arming the pipeline costs MORE (~11.7 us per stage) than a kernel boundary chained
// with programmatic dependent launch (~8 us per stage, set-up already overlapped, weights already
// prefetched), so the separate launches stay the default.
constexpr int kTailMaxPhases = 6;
enum { kPhaseProjection = 0, kPhaseReduceNorm = 1 };

struct TailPhase {
    int kind;
    int map_w, map_w2, map_x;          // projection: indices into TailMaps
    GemmParams g;
    const float* ws;                   // reduce: parts [splits][n_rows][d]
    int splits;
    size_t split_stride;
    float* x;                          // reduce: residual stream, updated in place
    const float* gain;                 // reduce: NULL = no normed output
    __nv_bfloat16* out;
};

struct TailParams {
    int n_phases;
    TailPhase ph[kTailMaxPhases];
    const int32_t* seq_id;             // pads (< 0) are skipped by the row-wise stage
    const int32_t* n_live;             // device count of live rows or NULL
    int n_rows, d;
    float eps;
    unsigned int* sync;                // grid barrier word (top bit flips once per barrier)
    int32_t* status;
};

struct TailMaps { CUtensorMap m[3 * kTailMaxPhases]; };

__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Arrive at the grid barrier (one thread per CTA); returns the ticket to wait on.  CTA 0 adds what is
// missing to carry into the top bit once all gridDim.x CTAs have arrived, so the word needs no reset.
__device__ __forceinline__ unsigned int grid_arrive(unsigned int* word) {
    const unsigned int inc = blockIdx.x == 0 ? 0x80000000u - (gridDim.x - 1) : 1u;
    __threadfence();
    return atomicAdd(word, inc);
}
__device__ __forceinline__ bool grid_wait(const unsigned int* word, unsigned int ticket, volatile int* abort_flag) {
    const long long t0 = clock64();
    for (uint32_t it = 0;; ++it) {
        if (((ticket ^ ld_acquire_u32(word)) & 0x80000000u) != 0) return true;
        if ((it & 63u) == 63u) {
            if (*abort_flag) return false;
            if (clock64() - t0 > kWaitCycles) break;
        }
    }
    *abort_flag = 1;
    return false;
}

__global__ void __launch_bounds__(kThreads, 1)
layer_tail_tcgen05_kernel(const __grid_constant__ TailMaps maps, const __grid_constant__ TailParams P) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[2 * 8 + 4];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ unsigned int ticket;               // of the grid barrier in flight
    __shared__ float red[4];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bar0 = smem_u32(bars);
    constexpr uint32_t tmem_cols = 512;
    auto init_barriers = [&]() {
        for (int s = 0; s < 8; ++s) { mbar_init(bar0 + 8u * s, 1); mbar_init(bar0 + 8u * (8 + s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(bar0 + 8u * (16 + a), 1); mbar_init(bar0 + 8u * (18 + a), kEpiThreads / 32); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    };
    if (threadIdx.x == 0) { abort_flag = 0; init_barriers(); }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    CtaCtx cx;
    cx.ring = ring; cx.bar0 = bar0; cx.tmem_base = tmem_base_slot; cx.abortp = &abort_flag;
    volatile int* abortp = &abort_flag;
    if (warp != 0) pdl_wait();

    for (int pi = 0; pi < P.n_phases; ++pi) {
        const TailPhase& ph = P.ph[pi];
        const bool last_wait = pi + 1 == P.n_phases;        // whoever passes the last barrier lets the next kernel launch
        if (ph.kind == kPhaseProjection) {
            gemm_roles<false>(&maps.m[ph.map_w], &maps.m[ph.map_w2], &maps.m[ph.map_x], ph.g, cx, [&] {
                if (pi == 0) {
                    pdl_wait();
                } else {
                    if (lane == 0) grid_wait(P.sync, ticket, abortp);
                    __syncwarp();
                    asm volatile("fence.proxy.async;" ::: "memory");     // other CTAs' stores, then this warp's TMA reads
                }
                if (last_wait && lane == 0) pdl_trigger();
            });
        } else if (warp >= 2 && warp < 6) {
            const int et = threadIdx.x - 64, q = warp - 2;                // 128 threads share a row
            if (pi > 0) {
                if (et == 0) grid_wait(P.sync, ticket, abortp);
                asm volatile("bar.sync 1, 128;" ::: "memory");
            }
            if (last_wait && et == 0) pdl_trigger();
            constexpr int MAXV = 12;                                      // float4 chunks per thread: d <= 12 * 4 * 128
            const int d4 = P.d / 4;
            for (int row = blockIdx.x; row < P.n_rows; row += gridDim.x) {
                if (P.seq_id != nullptr && (P.seq_id[row] < 0 || (P.n_live != nullptr && row >= *P.n_live))) {
                    if (ph.gain)
                        for (int i = et; i < d4; i += 128) *reinterpret_cast<uint2*>(ph.out + (size_t)row * P.d + 4 * i) = make_uint2(0u, 0u);
                    continue;
                }
                float4 v[MAXV];
                float ss = 0.f;
#pragma unroll
                for (int k = 0; k < MAXV; ++k) {
                    const int i = et + 128 * k;
                    if (i < d4) {
                        const size_t at = (size_t)row * d4 + i;
                        float4 a = __ldcg(reinterpret_cast<const float4*>(ph.x) + at);
                        for (int s = 0; s < ph.splits; ++s) {             // fixed order: part 0, 1, ...
                            const float4 b = __ldcg(reinterpret_cast<const float4*>(ph.ws + (size_t)s * ph.split_stride) + at);
                            a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
                        }
                        reinterpret_cast<float4*>(ph.x)[at] = a;
                        v[k] = a;
                        ss = fmaf(a.x, a.x, fmaf(a.y, a.y, fmaf(a.z, a.z, fmaf(a.w, a.w, ss))));
                    }
                }
                if (!ph.gain) continue;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
                asm volatile("bar.sync 1, 128;" ::: "memory");            // previous row's sums consumed
                if (lane == 0) red[q] = ss;
                asm volatile("bar.sync 1, 128;" ::: "memory");
                const float inv = rsqrtf((red[0] + red[1] + red[2] + red[3]) / (float)P.d + P.eps);
#pragma unroll
                for (int k = 0; k < MAXV; ++k) {
                    const int i = et + 128 * k;
                    if (i < d4) {
                        const float4 g = reinterpret_cast<const float4*>(ph.gain)[i];
                        const __nv_bfloat162 lo = __floats2bfloat162_rn(v[k].x * inv * g.x, v[k].y * inv * g.y);
                        const __nv_bfloat162 hi = __floats2bfloat162_rn(v[k].z * inv * g.z, v[k].w * inv * g.w);
                        uint2 w;
                        w.x = *reinterpret_cast<const uint32_t*>(&lo);
                        w.y = *reinterpret_cast<const uint32_t*>(&hi);
                        *reinterpret_cast<uint2*>(ph.out + (size_t)row * P.d + 4 * i) = w;
                    }
                }
            }
        }
        if (pi + 1 < P.n_phases) {
            // Stage boundary: everything this CTA wrote is made visible (to plain loads and to TMA reads of
            // other CTAs), the pipeline barriers are re-armed, and the CTA arrives at the grid barrier.  The
            // wait happens where the next stage first needs another CTA's data.
            __threadfence();
            asm volatile("fence.proxy.async;" ::: "memory");
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncthreads();
            if (threadIdx.x == 0) {
                for (int b = 0; b < 20; ++b) asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(bar0 + 8u * b) : "memory");
                init_barriers();
                ticket = grid_arrive(P.sync);
            }
            __syncthreads();
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (abort_flag) break;
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicCAS(P.status, 0, kStatusTimeout);
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(cx.tmem_base), "r"(tmem_cols) : "memory");
    }
}

}  // namespace

bool linear_tc_supported(const cdb* h, int n, int N, int K) {
    (void)h;
    return n >= 1 && N >= 1 && K % 8 == 0 && encode_fn() != nullptr;
}

// Tile-major weight copies ----------------------------------------------------------------------------
size_t tiled_weight_bytes(int layers, int N, int K) {
    return (size_t)layers * ((N + BM - 1) / BM) * ((K + BK - 1) / BK) * BM * BK * sizeof(__nv_bfloat16);
}

namespace {
__global__ void repack_tiled_kernel(const __nv_bfloat16* __restrict__ W, __nv_bfloat16* __restrict__ Wt, int layers, int N, int K) {
    const int n_ft = (N + BM - 1) / BM, n_kb = (K + BK - 1) / BK;
    const size_t per_layer = (size_t)n_ft * n_kb * BM * BK, total = per_layer * layers;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const size_t l = i / per_layer, r = i % per_layer;
        const int c = (int)(r % BK), row = (int)(r / BK % BM), kb = (int)(r / (BK * BM) % n_kb), ft = (int)(r / ((size_t)BK * BM * n_kb));
        const int f = ft * BM + row, k = kb * BK + c;
        Wt[i] = (f < N && k < K) ? W[l * (size_t)N * K + (size_t)f * K + k] : __float2bfloat16_rn(0.f);
    }
}

// the tile-major copy of the [N][K] matrix at W, or NULL when W is not (a layer of) a registered stack
const void* find_tiled(const cdb* h, const void* W, int N, int K) {
    for (int i = 0; i < h->n_tiled; ++i) {
        const TiledWeight& t = h->tiled[i];
        if (t.N != N || t.K != K || !t.tiled) continue;
        const size_t layer_bytes = (size_t)N * K * 2;
        const char* w = (const char*)W;
        if (w < t.orig || w >= t.orig + layer_bytes * t.layers || (size_t)(w - t.orig) % layer_bytes) continue;
        return t.tiled + (size_t)(w - t.orig) / layer_bytes * tiled_weight_bytes(1, N, K);
    }
    return nullptr;
}
}  // namespace

void launch_repack_tiled(const void* W, void* Wt, int layers, int N, int K, cudaStream_t st) {
    repack_tiled_kernel<<<148 * 8, 256, 0, st>>>((const __nv_bfloat16*)W, (__nv_bfloat16*)Wt, layers, N, K);
}

static int cluster_fit(const cdb* h, int size);

// Parameters and tensor maps of one projection.  W2 / act only in SwiGLU mode.  k_splits > 1 only with
// kModeStore (y = workspace).  Returns the number of tiles, 0 on failure.
static int setup_gemm(const cdb* h, const void* x, const void* W, const void* W2, float* y, __nv_bfloat16* act, int n,
                      int N, int K, int mode, int k_splits, size_t split_stride, GemmParams& p, CUtensorMap* map_w,
                      CUtensorMap* map_w2, CUtensorMap* map_x, size_t* smem, bool* pair = nullptr) {
    p.y = y; p.act = act; p.n = n; p.N = N; p.K = K; p.mode = mode; p.k_splits = k_splits; p.split_stride = split_stride;
    const int n_ft = (N + BM - 1) / BM;
    static const int forced_bn = tuning_int("CDB_GEMM_BN", 0);       // tuning hook
    const int bn_max = mode == kModeSwiGLU ? 128 : 256;
    // Rows per tile (MMA N): the widest of 64 / 128 / 256 the batch can fill: one tcgen05.mma then does the
    // most work per issue and each weight tile is pulled through L2 the fewest times.
    p.BN = n <= 64 ? 64 : (n <= 128 || bn_max == 128) ? 128 : 256;
    // ... unless that leaves most SMs without a tile (projections without split-K on a few hundred rows, as in
    // prompt processing): narrower row tiles then give more CTAs a share of the weight stream.  The tile
    // width changes which CTA computes an output element, never how it is summed.
    {
        const int sms = h->part_active ? h->part_proj_sms : h->sms;
        auto tiles = [&](int bn) { return n_ft * ((n + bn - 1) / bn) * k_splits; };
        while (p.BN > 64 && tiles(p.BN) * 2 < sms && n > p.BN / 2) p.BN /= 2;
        // ... or when the tiles of the last wave would keep a few CTAs busy while the others idle (192 tiles of 256
        // rows on 148 SMs take two full tile times; 384 tiles of 128 rows take three half ones).  Cost of a width =
        // waves x (rows of a tile + a per-tile overhead worth ~32 rows); the widest of the cheapest widths wins.
        static const int quant = tuning_int("CDB_GEMM_WAVES", 1);     // tuning hook: 0 = off
        if (quant && tiles(p.BN) > sms) {
            auto cost = [&](int bn) { return ((tiles(bn) + sms - 1) / sms) * (bn + 32); };
            int best = p.BN;
            for (int bn = p.BN / 2; bn >= 64; bn /= 2)
                if (cost(bn) * 10 < cost(best) * 9) best = bn;
            p.BN = best;
        }
    }
    // Above 128 rows a row tile need not be a power of two either: any multiple of 16 rows is a valid MMA N, and
    // r row tiles of ceil(n / r) rows can fit the tile count to the SM count where halving cannot.  512 rows of
    // gate/up (44 feature tiles) are 176 tiles of 128 rows - two waves, the second almost empty - or 132 tiles of 176
    // rows: 32 against 24 us measured; the other projections (96 tiles per row tile) like three row tiles too (288
    // tiles, two full waves): 176 rows per tile at 512 rows, 256 at 768.  Cost of a width = waves x (rows of a tile +
    // the weight rows a tile must ingest whatever its width); a width that leaves TMEM no room for a second
    // accumulator set (gate/up above 128 rows) is taken only where every CTA has a single tile, since its epilogue
    // cannot hide under the next tile's main loop (prompt calls: 2.5 % slower with it); fewer row tiles win ties (each
    // one pulls the weights through L2 again).  Measured per stage at 144 ... 1024 rows: never behind the powers of two
    // (2-5 us per layer ahead up to 256 rows, where the rule mostly trims the padding of the last tile; 12-15 us at 448-512).
    static const int chooser = tuning_int("CDB_GEMM_CHOOSER", 1);     // tuning hook: 0 = powers of two only
    static const int chooser_min = tuning_int("CDB_GEMM_CHOOSER_MIN", 128);     // tuning hook
    if (chooser && n > chooser_min) {
        const int sms = h->part_active ? h->part_proj_sms : h->sms;
        const int dual = mode == kModeSwiGLU ? 2 : 1;
        const bool pair_ok = pair != nullptr && !h->part_active && cluster_fit(h, 2) > 0 && ((h->cfg.flags & CDB_FLAG_CTA_PAIRS) || n >= 512);
        long best_cost = 0; int best_bn = 0;
        for (int r = 1; r <= (n + 63) / 64; ++r) {
            const int bn = ((n + r - 1) / r + 15) / 16 * 16;
            if (bn > 256 || bn * dual > 512) continue;
            if (bn < 64) break;
            const int xr = pair_ok && bn >= 128 ? bn / 2 : bn;
            if ((kMaxSmem - 1024 - (dual == 2 ? bn * BM * 2 : 0)) / (dual * BM * BK * 2 + xr * BK * 2) < 2) continue;
            const long tiles = (long)n_ft * ((n + bn - 1) / bn) * k_splits, waves = (tiles + sms - 1) / sms;
            if (2 * dual * bn > 512 && waves > 1) continue;
            const long cost = waves * (bn + BM * dual);
            if (best_bn == 0 || cost * 100 < best_cost * 95) { best_cost = cost; best_bn = bn; }
        }
        if (best_bn) p.BN = best_bn;
    }
    static const int forced_bn_dual = tuning_int("CDB_GEMM_BN_SWIGLU", 0);      // tuning hook
    {
        const int f = mode == kModeSwiGLU ? forced_bn_dual : forced_bn;
        if (f >= 64 && f <= 256 && f % 16 == 0) p.BN = f;
    }
    p.n_acc = (mode == kModeSwiGLU ? 4 : 2) * p.BN <= 512 ? 2 : 1;  // two accumulator sets when TMEM's 512 columns hold them
    // CTA pairs: two CTAs share every activation tile of 128 or 256 rows, each loads half of it.  Same sums in the
    // same order as the single-CTA form.  Measured on the 2048-wide model: prompt calls (thousands of rows, where the
    // projections are bound by the tensor pipe and the L2-to-SM traffic) get 3.5-4.5 % faster and decode steps of 512 and
    // 1024 rows 0.4-0.9 %; at 256 rows the step is 0.2-0.7 % slower (there the main loop waits for the per-k-block
    // hand-shake, not for L2).  So pairs are used from 512 rows on; CDB_FLAG_CTA_PAIRS forces them from 128 rows on.
    static const int pair_mask = tuning_int("CDB_GEMM_PAIR", 7);      // tuning hook: 1 store / split-K, 2 SwiGLU, 4 residual epilogue
    const int pair_bit = mode == kModeSwiGLU ? 2 : mode == kModeAccumulate ? 4 : 1;
    const bool use_pair = pair != nullptr && ((h->cfg.flags & CDB_FLAG_CTA_PAIRS) || n >= 512) && (pair_mask & pair_bit) && p.BN >= 128 &&
                          !h->part_active && cluster_fit(h, 2) > 0;
    if (pair) *pair = use_pair;
    const int x_rows = use_pair ? p.BN / 2 : p.BN;                   // activation rows a CTA loads per k-block
    const int stage_bytes = (mode == kModeSwiGLU ? 2 : 1) * BM * BK * 2 + x_rows * BK * 2;
    static const int smem_cap = tuning_int("CDB_GEMM_SMEM_KB", kMaxSmem / 1024) * 1024;       // tuning hook
    int budget = smem_cap < kMaxSmem ? smem_cap : kMaxSmem;
    if (h->gemm_smem_cap > 0 && h->gemm_smem_cap < budget) budget = h->gemm_smem_cap;
    // Output staging tile of the SwiGLU epilogue.  When every CTA has a single tile (decode batches), the tile is
    // staged in the ring itself - idle by then: all its stages were consumed before the accumulator completed and
    // nothing refills it - which leaves the whole budget to the ring (4 instead of 3 stages of 48 KB).
    const int tiles_now = (use_pair ? (n_ft + 1) / 2 : n_ft) * ((n + p.BN - 1) / p.BN) * k_splits;
    const int ctas_now = (h->part_active ? h->part_proj_sms : h->sms) / (use_pair ? 2 : 1);
    static const int alias_ok = tuning_int("CDB_GEMM_ALIAS", 1);      // tuning hook
    const bool alias_out = mode == kModeSwiGLU && alias_ok && tiles_now <= ctas_now && !(h->cfg.flags & CDB_FLAG_FUSED_STAGES) && p.BN * BM * 2 <= 2 * stage_bytes;
    const int stage_out = mode == kModeSwiGLU && !alias_out ? p.BN * BM * 2 : 0;
    p.stages = (budget - 1024 - stage_out) / stage_bytes;
    if (p.stages < 2) p.stages = 2;
    if (p.stages > 8) p.stages = 8;
    p.stage_out_off = alias_out ? 0u : (uint32_t)(p.stages * stage_bytes);
    p.status = h->status;
    p.dbg = nullptr;
    const int n_kb = (K + BK - 1) / BK;
    const void* Wt = find_tiled(h, W, N, K);
    const void* Wt2 = W2 ? find_tiled(h, W2, N, K) : Wt;
    p.w_tiled = (Wt && Wt2) ? 1 : 0;
    if (p.w_tiled) {
        if (!make_map(map_w, Wt, n_ft * n_kb * BM, BK, BM) || !make_map(map_w2, Wt2, n_ft * n_kb * BM, BK, BM)) return 0;
    } else {
        if (!make_map(map_w, W, N, K, BM) || !make_map(map_w2, W2 ? W2 : W, N, K, BM)) return 0;
    }
    if (!make_map(map_x, x, n, K, x_rows)) return 0;
    *smem = (size_t)p.stages * stage_bytes + stage_out + 1024;
    return (use_pair ? (n_ft + 1) / 2 : n_ft) * ((n + p.BN - 1) / p.BN) * k_splits;      // tiles (of a pair: 256 features)
}

static bool launch_gemm(const cdb* h, const void* x, const void* W, const void* W2, float* y, __nv_bfloat16* act, int n,
                        int N, int K, int mode, int k_splits, size_t split_stride, cudaStream_t st) {
    static bool attr_set_dev[kMaxDevices] = {};
    bool& attr_set = attr_set_dev[h->device];
    if (!attr_set) {
        cudaFuncSetAttribute(gemm_bf16_tcgen05_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
        cudaFuncSetAttribute(gemm_bf16_tcgen05_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
        if (tuning_int("CDB_GEMM_CARVEOUT", -2) > -2)           // tuning hook
            cudaFuncSetAttribute(gemm_bf16_tcgen05_kernel<false>, cudaFuncAttributePreferredSharedMemoryCarveout, tuning_int("CDB_GEMM_CARVEOUT", -2));
        attr_set = true;
    }
    GemmParams p;
    CUtensorMap map_w, map_w2, map_x;
    size_t smem = 0;
    bool pair = false;
    const int n_tiles = setup_gemm(h, x, W, W2, y, act, n, N, K, mode, k_splits, split_stride, p, &map_w, &map_w2, &map_x, &smem, &pair);
    if (!n_tiles) return false;
#ifdef CDB_TUNING
    // tuning hook: device address of a stamp buffer (8 words per CTA), optionally for one launch kind only
    p.dbg = getenv("CDB_GEMM_DBG") && !getenv("CDB_GEMM_DBG_CLUSTER") ? (unsigned long long*)strtoull(getenv("CDB_GEMM_DBG"), nullptr, 0) : nullptr;
    if (getenv("CDB_GEMM_DBG_ONLY") && atoi(getenv("CDB_GEMM_DBG_ONLY")) != mode * 100000 + N) p.dbg = nullptr;
#endif
    static const int part_sms = tuning_int("CDB_GEMM_SMS", 0);      // tuning hook (two-stream step only): CTA count of a projection
    const int sms = h->part_active ? h->part_proj_sms : (part_sms > 0 && part_sms <= h->sms && h->attn_ctas_per_sm_cap > 0) ? part_sms : h->sms;
    if (pair) {
        // one persistent pair per two SMs, launched as clusters of two
        const int pairs = n_tiles < sms / 2 ? n_tiles : sms / 2;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * pairs); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = smem; cfg.stream = st;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr; cfg.numAttrs = 2;
        return cudaLaunchKernelEx(&cfg, gemm_bf16_tcgen05_kernel<true>, map_w, map_w2, map_x, p) == cudaSuccess;
    }
    const int grid = n_tiles < sms ? n_tiles : sms;
    launch_pdl(gemm_bf16_tcgen05_kernel<false>, dim3(grid), dim3(kThreads), smem, st, map_w, map_w2, map_x, p);
    return true;
}

// How many clusters of `size` CTAs of the cluster projection kernel can be resident at once on the handle's device
// (each CTA takes a whole SM, and a cluster must fit inside one GPC); 0 when such clusters cannot be launched.
// Asked once per device and size.
static int cluster_fit(const cdb* h, int size) {
    static int fit[kMaxDevices][kMaxKSplits + 1] = {};          // 0 = not asked yet, -1 = unavailable
    if (size < 1 || size > kMaxKSplits) return 0;
    int& f = fit[h->device][size];
    if (f == 0) {
        f = -1;
        if (cudaFuncSetAttribute(gemm_splitk_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem) == cudaSuccess) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(size * 64); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = kMaxSmem;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = size; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr; cfg.numAttrs = 1;
            int nc = 0;
            if (cudaOccupancyMaxActiveClusters(&nc, gemm_splitk_cluster_kernel, &cfg) == cudaSuccess && nc > 0) f = nc;
            else cudaGetLastError();
            if (kTuningBuild) fprintf(stderr, "cluster projection: %d clusters of %d fit\n", nc, size);
        }
    }
    return f > 0 ? f : 0;
}

// Part count of a split-K projection.  It depends on the weight's shape (and the device) alone, never on the
// number of rows, so that a row's result does not depend on the batch it is computed in: at most one tile per SM
// for a batch that fills one row tile, at least four k-blocks per part, and - so that the parts can be summed
// inside thread-block clusters - no more parts than let one cluster per feature tile be resident at once.
static int splitk_parts(const cdb* h, int N, int K, int max_splits) {
    const int sms = h->sms;
    const int n_ft = (N + BM - 1) / BM, n_kb = (K + BK - 1) / BK;
    int splits = sms / n_ft;                      // rounded down: one tile too many per wave would cost a second wave
    if (splits > n_kb / 4) splits = n_kb / 4;
    if (splits > max_splits) splits = max_splits;
    if (splits < 1) splits = 1;
    static const int fit_aware = tuning_int("CDB_SPLITK_FIT", 1);      // tuning hook: 0 = part counts ignore what clusters fit
    if (fit_aware && !(h->cfg.flags & CDB_FLAG_FUSED_STAGES))
        while (splits > 1 && cluster_fit(h, splits) > 0 && cluster_fit(h, splits) < n_ft) --splits;
    return splits;
}

bool launch_linear_tc(const cdb* h, const void* x, const void* W, float* y, int n, int N, int K, Epilogue ep, cudaStream_t st) {
    return launch_gemm(h, x, W, nullptr, y, nullptr, n, N, K, ep == Epilogue::ResidualAdd ? kModeAccumulate : kModeStore, 1, 0, st);
}

// act[n,F] (bf16) = SiLU(x.Wg^T) * (x.Wu^T): both projections in one launch, SwiGLU in the epilogue.
bool launch_gate_up_swiglu_tc(const cdb* h, const void* x, const void* Wg, const void* Wu, void* act, int n, int F, int K, cudaStream_t st) {
    return launch_gemm(h, x, Wg, Wu, nullptr, (__nv_bfloat16*)act, n, F, K, kModeSwiGLU, 1, 0, st);
}

// Split-K: partial products ws[s][n][N] (fp32), s < returned split count; the caller reduces them in
// split order (deterministic).
int launch_linear_splitk_tc(const cdb* h, const void* x, const void* W, float* ws, int max_splits, int n, int N, int K, cudaStream_t st) {
    const int splits = splitk_parts(h, N, K, max_splits);
    return launch_gemm(h, x, W, nullptr, ws, nullptr, n, N, K, kModeStore, splits, (size_t)n * N, st) ? splits : 0;
}

// ---- split-K projections summed inside thread-block clusters -------------------------------------------
namespace {

// Fills the shape-dependent fields and launches.  false: the cluster form is not available for this shape on
// this device (the caller then takes the workspace path); nothing was launched.
bool launch_cluster_gemm(const cdb* h, const void* xin, const void* W, int n, int N, int K, int max_splits, ClusterParams& p, cudaStream_t st) {
    if (n < 1 || N % 4 != 0) return false;
    const int KS = splitk_parts(h, N, K, max_splits);
    if (KS < 1 || KS > kMaxKSplits) return false;
    p.n = n; p.N = N; p.K = K; p.k_splits = KS;
    p.BN = n <= 64 ? 64 : n <= 128 ? 128 : 256;
    // every cluster of the launch resident at once, or the workspace form (whose CTAs are persistent) does it
    if (((N + BM - 1) / BM) * ((n + p.BN - 1) / p.BN) > cluster_fit(h, KS)) return false;
    const int stage_bytes = BM * BK * 2 + p.BN * BK * 2;
    p.stages = (kMaxSmem - 1024) / stage_bytes;
    if (p.stages > 8) p.stages = 8;
    // the ring doubles as the receive buffer: [chunks owned][parts][16 columns][128 features] fp32
    const int chunks = p.BN / 16, owned = (chunks + KS - 1) / KS;
    if ((size_t)owned * KS * 16 * BM * 4 > (size_t)p.stages * stage_bytes) return false;
    p.status = h->status;
    const int n_ft = (N + BM - 1) / BM, n_kb = (K + BK - 1) / BK;
    const void* Wt = find_tiled(h, W, N, K);
    p.w_tiled = Wt ? 1 : 0;
    CUtensorMap map_w, map_x;
    if (Wt ? !make_map(&map_w, Wt, n_ft * n_kb * BM, BK, BM) : !make_map(&map_w, W, N, K, BM)) return false;
    if (!make_map(&map_x, xin, n, K, p.BN)) return false;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_ft * ((n + p.BN - 1) / p.BN) * KS); cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = (size_t)p.stages * stage_bytes + 1024; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = KS; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 2;
#ifdef CDB_TUNING
    p.dbg = getenv("CDB_GEMM_DBG") ? (unsigned long long*)strtoull(getenv("CDB_GEMM_DBG"), nullptr, 0) : nullptr;
#endif
    return cudaLaunchKernelEx(&cfg, gemm_splitk_cluster_kernel, map_w, map_x, p) == cudaSuccess;
}

}  // namespace

// x[n][N] += xin[n][K] . W[N][K]^T, the split-K parts added in part order on top of x.
bool launch_linear_cluster_residual_tc(const cdb* h, const void* xin, const void* W, float* x, int n, int N, int K, int max_splits, cudaStream_t st) {
    ClusterParams p = {};
    p.mode = kClusterResidual;
    p.x = x;
    return launch_cluster_gemm(h, xin, W, n, N, K, max_splits, p, st);
}

// QKV projection of one layer with RoPE and the KV page write in its epilogue (heads of 128 only).
bool launch_qkv_rope_cluster_tc(const cdb* h, int ln, int layer, const void* xin, const void* W_qkv, const RowsDev& rows, int max_splits, cudaStream_t st) {
    const cdb_config_t& c = h->cfg;
    if (c.Dh != BM || c.d % BM != 0 || c.dtype != CDB_BF16) return false;
    ClusterParams p = {};
    p.mode = kClusterRope;
    const LayerKv kv = layer_kv(h, layer, rows);
    p.qrot = h->lane[ln].qrot; p.pool = kv.pool; p.rows = kv.rows; p.layer = kv.layer; p.d = c.d;
    p.max_position = c.max_position; p.max_seqs = c.max_seqs; p.rope_cos = h->rope_cos; p.rope_sin = h->rope_sin;
    return launch_cluster_gemm(h, xin, W_qkv, rows.n_rows, 3 * c.d, c.d, max_splits, p, st);
}

// Everything of a layer after its attention in one cooperative launch: output projection (split-K) ->
// parts + residual + RMSNorm(g_mlp) -> gate/up projections with SwiGLU -> down projection (split-K) ->
// parts + residual + RMSNorm(next_gain) [-> the next layer's QKV projection (split-K) into qkv_ws].  Same
// arithmetic as the separate launches; returns the part count of the QKV stage (0 when it was not asked
// for), -1 on failure.
int launch_layer_tail_tc(const cdb* h, int ln, const RowsDev& rows, float* x, const void* W_o, const float* g_mlp,
                         const void* W_gate, const void* W_up, const void* W_down, const float* next_gain,
                         const void* W_qkv_next, cudaStream_t st) {
    const Lane& L = h->lane[ln];
    const cdb_config_t& c = h->cfg;
    const int n = rows.n_rows, d = c.d, F = c.F;
    static bool attr_set_dev[kMaxDevices] = {};
    bool& attr_set = attr_set_dev[h->device];
    if (!attr_set) {
        if (cudaFuncSetAttribute(layer_tail_tcgen05_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem) != cudaSuccess) return -1;
        attr_set = true;
    }
    TailMaps maps;
    TailParams P;
    size_t smem = 0, smem_max = 0;
    int np = 0;
    auto projection = [&](const void* xin, const void* W, const void* W2, float* y, __nv_bfloat16* act, int N, int K, int mode, int splits) {
        TailPhase& ph = P.ph[np];
        ph.kind = kPhaseProjection;
        ph.map_w = 3 * np; ph.map_w2 = 3 * np + 1; ph.map_x = 3 * np + 2;
        ph.ws = nullptr; ph.splits = 0; ph.split_stride = 0; ph.x = nullptr; ph.gain = nullptr; ph.out = nullptr;
        const int tiles = setup_gemm(h, xin, W, W2, y, act, n, N, K, mode, splits, (size_t)n * N, ph.g, &maps.m[ph.map_w],
                                     &maps.m[ph.map_w2], &maps.m[ph.map_x], &smem);
        if (smem > smem_max) smem_max = smem;
        ++np;
        return tiles > 0;
    };
    auto reduce = [&](int splits, const float* gain) {
        TailPhase& ph = P.ph[np];
        ph.kind = kPhaseReduceNorm;
        ph.map_w = ph.map_w2 = ph.map_x = 0;
        ph.g = GemmParams();
        ph.ws = L.ws; ph.splits = splits; ph.split_stride = (size_t)n * d; ph.x = x; ph.gain = gain; ph.out = (__nv_bfloat16*)L.xn;
        ++np;
    };
    const int s_o = splitk_parts(h, d, d, kMaxKSplits), s_d = splitk_parts(h, d, F, kMaxKSplits);
    int s_q = 0;
    if (!projection(L.attn_o, W_o, nullptr, L.ws, nullptr, d, d, kModeStore, s_o)) return -1;
    reduce(s_o, g_mlp);
    if (!projection(L.xn, W_gate, W_up, nullptr, (__nv_bfloat16*)L.act, F, d, kModeSwiGLU, 1)) return -1;
    if (!projection(L.act, W_down, nullptr, L.ws, nullptr, d, F, kModeStore, s_d)) return -1;
    reduce(s_d, next_gain);
    if (W_qkv_next) {
        s_q = splitk_parts(h, 3 * d, d, kWsPerRow / 3);
        if (!projection(L.xn, W_qkv_next, nullptr, L.ws, nullptr, 3 * d, d, kModeStore, s_q)) return -1;
    }
    P.n_phases = np;
    P.seq_id = rows.seq_id; P.n_live = rows.n_live; P.n_rows = n; P.d = d; P.eps = c.eps; P.sync = h->grid_sync + ln; P.status = h->status;
    for (int i = 3 * np; i < 3 * kTailMaxPhases; ++i) maps.m[i] = maps.m[0];

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(h->sms); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = smem_max; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    static int with_pdl = tuning_int("CDB_NO_PDL", 0) ? 0 : 1;
    cfg.numAttrs = 1 + with_pdl;
    cudaError_t e = cudaLaunchKernelEx(&cfg, layer_tail_tcgen05_kernel, maps, P);
    if (e != cudaSuccess && with_pdl) {            // this driver does not combine the two attributes: plain cooperative launch
        cudaGetLastError();
        with_pdl = 0;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, layer_tail_tcgen05_kernel, maps, P);
    }
    return e == cudaSuccess ? s_q : -1;
}

}  // namespace cdbk

CDB_TRACE_SETTER(trace_set_gemm)
