// Causal attention of prompt rows on the 5th-generation tensor cores (bf16 pools).
//
// The rows of a prompt are consecutive positions of one sequence, so 128 of them form a query tile that
// shares every K/V page it reads.  Per (query tile, head) a CTA walks the keys in tiles of 128 (8 pages):
//   S = Q K^T     tcgen05.mma, Q [128 x Dh] and K [128 keys x Dh] both K-major in shared memory (TMA,
//                 128-byte swizzle, one 2 KB box per page and 64-wide slice of the head), S in TMEM;
//   softmax       four warps, one query row per thread (= one TMEM lane): running maximum, p = 2^(s - m),
//                 row sum in fp32; p rounded to bf16 and written to shared memory as the next A operand;
//   O_j = P V     tcgen05.mma with V as an MN-major B operand (the pool stores [token][Dh], which is
//                 exactly that), fresh accumulator in TMEM, added by the row's thread to its fp32 output
//                 registers after the usual rescale.
// Roles: warps 0-3 softmax / output, warp 4 TMA producer, warp 5 TMEM owner and MMA issuer.  K/V tiles are
// double buffered; CTAs are persistent over (tile, head) items.  Every mbarrier wait is bounded: on expiry
// the CTA records a status word, frees its TMEM and returns.
// Rounding points: q, K, V bf16 (as in the decode kernel), scores and row sums fp32, p bf16 for P.V.
#include <cstdlib>
#include <cuda_bf16.h>

#include "cdb_internal.h"
#include "tc_common.cuh"

namespace cdbk {

namespace {

using namespace tc;

constexpr int kQT = 128;                // query rows per tile (MMA M, TMEM lanes)
constexpr int kKT = 128;                // keys per tile
constexpr int kPagesPerTile = kKT / kPageSize;
constexpr int kPfThreads = 192;
constexpr uint32_t kChunkBytes = 128 * 128;   // [128 rows][64 bf16]: one swizzled slice of an operand tile

struct PfParams {
    RowsDev rows;
    KvPool pool;
    int layer, max_seqs;
    float scale_log2;
    const int32_t* tiles;
    const int32_t* tile_rows;
    const int32_t* n_tiles;
    __nv_bfloat16* out;
    int32_t* status;
};

// MN-major B operand with 128-byte swizzle: rows (keys) of 64 contiguous head dims = 128 bytes, 8 keys per
// 1024-byte atom; atoms along the keys 1024 bytes apart, the next 64 head dims one slice (16 KB) further.
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(kChunkBytes >> 4) << 16;            // leading-dimension byte offset: next 64 head dims
    d |= (uint64_t)(1024 >> 4) << 32;                   // stride-dimension byte offset: next 8 keys
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

template <int DH>
__global__ void __launch_bounds__(kPfThreads, 1)
attn_prefill_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kv, PfParams p) {
    pdl_trigger();
    constexpr int NCH = (DH + 63) / 64;                  // 64-wide slices of the head dimension
    constexpr uint32_t kQBytes = NCH * kChunkBytes, kKvBytes = NCH * kChunkBytes;       // P takes two chunks (128 keys)
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[16];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t q_s = base, k_s = q_s + kQBytes, v_s = k_s + 2 * kKvBytes, p_s = v_s + 2 * kKvBytes;
    const uint32_t bar0 = smem_u32(bars);
    const uint32_t q_full = bar0, q_empty = bar0 + 8, s_full = bar0 + 16, p_full = bar0 + 24, o_full = bar0 + 32;
    auto k_full = [&](int b) { return bar0 + 40u + 8u * b; };
    auto v_full = [&](int b) { return bar0 + 56u + 8u * b; };
    auto kv_empty = [&](int b) { return bar0 + 72u + 8u * b; };
    constexpr uint32_t kTmemCols = 256;                  // S in columns 0..127, O_j in 128..128+DH

    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(q_full, 1); mbar_init(q_empty, 1); mbar_init(s_full, 1); mbar_init(p_full, 128); mbar_init(o_full, 1);
        for (int b = 0; b < 2; ++b) { mbar_init(k_full(b), 1); mbar_init(v_full(b), 1); mbar_init(kv_empty(b), 1); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 5) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_slot;
    volatile int* abortp = &abort_flag;
    pdl_wait();

    const int H = p.pool.H;
    const int n_items = *p.n_tiles * H;
    // Items in reverse tile order: the last tiles of a prompt have the most keys, so they start first.
    auto item_tile = [&](int it) { return *p.n_tiles - 1 - it / H; };

    if (warp == 4) {
        // ---------------- TMA producer ----------------
        const bool leader = elect_one();
        uint32_t g = 0, item_no = 0;
        bool ok = true;
        for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
            const int tile = item_tile(it), head = it % H;
            const int row0 = p.tiles[tile], nq = p.tile_rows[tile];
            const int seq = p.rows.seq_of(row0), slot = p.rows.slot_of(row0);
            const int pos_last = p.rows.position[row0 + nq - 1];
            if (seq < 0 || seq >= p.max_seqs || slot < 0 || slot >= p.rows.n_slots || pos_last < 0 || pos_last / kPageSize >= p.rows.page_table_stride) continue;   // flagged by the softmax warps
            const int32_t* table = p.rows.page_table + ((size_t)seq * p.rows.n_slots + slot) * p.rows.page_table_stride;
            const int last_page = pos_last / kPageSize;
            const int n_kt = pos_last / kKT + 1;
            if (!mbar_wait(q_empty, (item_no & 1u) ^ 1u, abortp)) { ok = false; break; }
            if (leader) {
                mbar_expect_tx(q_full, kQBytes);
                for (int c = 0; c < NCH; ++c) tma_load_2d(q_s + c * kChunkBytes, &map_q, q_full, head * DH + 64 * c, row0);
            }
            __syncwarp();
            ++item_no;
            for (int j = 0; j < n_kt && ok; ++j, ++g) {
                const int b = g & 1;
                if (!mbar_wait(kv_empty(b), ((g >> 1) & 1u) ^ 1u, abortp)) { ok = false; break; }
                // page ids of this key tile (lanes 0..7); pages past the prompt repeat the last one, so that
                // the tile holds finite values everywhere (their scores are masked, their p is exactly 0)
                int page = 0;
                if (lane < kPagesPerTile) page = table[min(j * kPagesPerTile + lane, last_page)];
                const bool bad = lane < kPagesPerTile && (page < 0 || page >= p.pool.n_phys_pages);
                if (__any_sync(0xffffffffu, bad)) {
                    if (leader) atomicCAS(p.status, 0, kStatusPage);
                    page = bad ? 0 : page;
                }
                if (leader) { mbar_expect_tx(k_full(b), kKvBytes); mbar_expect_tx(v_full(b), kKvBytes); }
                __syncwarp();
#pragma unroll
                for (int kv = 0; kv < 2; ++kv) {
                    for (int i = 0; i < kPagesPerTile; ++i) {
                        const int pg = __shfl_sync(0xffffffffu, page, i);
                        // row of the pool viewed as [layer][page][K/V][head][16 tokens] x [Dh]
                        const long long trow = ((((long long)p.layer * p.pool.n_phys_pages + pg) * 2 + kv) * H + head) * kPageSize;
                        const uint32_t dst = (kv ? v_s : k_s) + (uint32_t)b * kKvBytes + (uint32_t)i * (kPageSize * 128);
                        if (leader)
                            for (int c = 0; c < NCH; ++c)
                                tma_load_2d(dst + c * kChunkBytes, &map_kv, kv ? v_full(b) : k_full(b), 64 * c, (int)trow);
                    }
                }
                __syncwarp();
            }
        }
        if (!ok || *abortp) for (int i = 0; i < 64; ++i) __nanosleep(1000);      // copies in flight may still land
        __syncwarp();
    } else if (warp == 5) {
        // ---------------- MMA issuer ----------------
        const bool leader = elect_one();
        // fp32 accumulate, bf16 x bf16, M = 128; S: N = 128 keys, both K-major; O: N = DH, B MN-major
        const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kKT >> 3) << 17) | ((uint32_t)(kQT >> 4) << 24);
        const uint32_t idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(DH >> 3) << 17) | ((uint32_t)(kQT >> 4) << 24);
        uint32_t g = 0, item_no = 0;
        bool ok = true;
        auto issue_qk = [&](int b) {
#pragma unroll
            for (int k = 0; k < DH / 16; ++k) {
                const uint32_t off = (uint32_t)(k / 4) * kChunkBytes + (uint32_t)(k % 4) * 32u;
                if (leader) umma_bf16(tmem_base, smem_desc_sw128(q_s + off), smem_desc_sw128(k_s + (uint32_t)b * kKvBytes + off), idesc_s, k > 0 ? 1u : 0u);
            }
            __syncwarp();
            if (leader) umma_commit(s_full);
        };
        for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
            const int tile = item_tile(it);
            const int row0 = p.tiles[tile], nq = p.tile_rows[tile];
            const int seq = p.rows.seq_of(row0), slot = p.rows.slot_of(row0);
            const int pos_last = p.rows.position[row0 + nq - 1];
            if (seq < 0 || seq >= p.max_seqs || slot < 0 || slot >= p.rows.n_slots || pos_last < 0 || pos_last / kPageSize >= p.rows.page_table_stride) continue;
            const int n_kt = pos_last / kKT + 1;
            if (!mbar_wait(q_full, item_no & 1u, abortp)) { ok = false; break; }
            ++item_no;
            if (!mbar_wait(k_full(g & 1), (g >> 1) & 1u, abortp)) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            issue_qk(g & 1);
            for (int j = 0; j < n_kt && ok; ++j, ++g) {
                const int b = g & 1;
                if (!mbar_wait(p_full, g & 1u, abortp)) { ok = false; break; }            // P written, S and O_(j-1) consumed
                if (!mbar_wait(v_full(b), (g >> 1) & 1u, abortp)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
                for (int k = 0; k < kKT / 16; ++k) {
                    const uint64_t a_desc = smem_desc_sw128(p_s + (uint32_t)(k / 4) * kChunkBytes + (uint32_t)(k % 4) * 32u);
                    const uint64_t b_desc = smem_desc_mn_sw128(v_s + (uint32_t)b * kKvBytes + (uint32_t)k * (16u * 128u));
                    if (leader) umma_bf16(tmem_base + 128u, a_desc, b_desc, idesc_o, k > 0 ? 1u : 0u);
                }
                __syncwarp();
                if (leader) { umma_commit(o_full); umma_commit(kv_empty(b)); }
                if (j + 1 < n_kt) {
                    const uint32_t g1 = g + 1;
                    if (!mbar_wait(k_full(g1 & 1), (g1 >> 1) & 1u, abortp)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    issue_qk(g1 & 1);
                } else if (leader) {
                    umma_commit(q_empty);
                }
                __syncwarp();
            }
        }
        __syncwarp();
    } else {
        // ---------------- softmax and output: thread = query row = TMEM lane ----------------
        const int r = threadIdx.x;                         // 0..127
        const uint32_t t_lane = tmem_base + ((uint32_t)(warp * 32) << 16);
        uint32_t g = 0;
        bool ok = true;
        for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
            const int tile = item_tile(it), head = it % H;
            const int row0 = p.tiles[tile], nq = p.tile_rows[tile];
            const int seq = p.rows.seq_of(row0), slot = p.rows.slot_of(row0);
            const int pos_last = p.rows.position[row0 + nq - 1];
            if (seq < 0 || seq >= p.max_seqs || slot < 0 || slot >= p.rows.n_slots || pos_last < 0 || pos_last / kPageSize >= p.rows.page_table_stride) {
                if (r == 0) atomicCAS(p.status, 0, kStatusSeq);
                continue;
            }
            const int n_kt = pos_last / kKT + 1;
            const int pos_q = p.rows.position[row0] + r;   // rows of a tile are consecutive positions
            float o_acc[DH];
#pragma unroll
            for (int e = 0; e < DH; ++e) o_acc[e] = 0.f;
            float m = -INFINITY, l = 0.f;
            for (int j = 0; j < n_kt && ok; ++j, ++g) {
                if (!mbar_wait(s_full, g & 1u, abortp)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const int key0 = j * kKT;
                const int n_vis = min(kKT, pos_q - key0 + 1);          // keys of this tile the row may see (<= 0: none)
                // pass 1: row maximum of the visible scores
                float mx = -INFINITY;
#pragma unroll 1
                for (int c = 0; c < kKT; c += 32) {
                    uint32_t v[32];
                    tmem_ld32(t_lane + (uint32_t)c, v);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int i = 0; i < 32; ++i) if (c + i < n_vis) mx = fmaxf(mx, __uint_as_float(v[i]));
                }
                const float m_new = fmaxf(m, mx * p.scale_log2);
                // the previous tile's P.V has landed: add it, then move the running sums to the new maximum
                if (j > 0) {
                    if (!mbar_wait(o_full, (g - 1) & 1u, abortp)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
                    for (int c = 0; c < DH; c += 32) {
                        uint32_t v[32];
                        tmem_ld32(t_lane + 128u + (uint32_t)c, v);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                        for (int i = 0; i < 32; ++i) o_acc[c + i] += __uint_as_float(v[i]);
                    }
                }
                const float corr = (m_new == -INFINITY) ? 1.f : exp2f(m - m_new);
                l *= corr;
#pragma unroll
                for (int e = 0; e < DH; ++e) o_acc[e] *= corr;
                m = m_new;
                // pass 2: p = 2^(s - m), row sum, bf16 P into the swizzled A-operand tile [128 rows][128 keys]
#pragma unroll 1
                for (int c = 0; c < kKT; c += 32) {
                    uint32_t v[32];
                    tmem_ld32(t_lane + (uint32_t)c, v);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        const float p0 = (c + i < n_vis) ? exp2f(__uint_as_float(v[i]) * p.scale_log2 - m) : 0.f;
                        const float p1 = (c + i + 1 < n_vis) ? exp2f(__uint_as_float(v[i + 1]) * p.scale_log2 - m) : 0.f;
                        l += p0 + p1;
                        const __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
                        pk[i >> 1] = *reinterpret_cast<const uint32_t*>(&h2);
                    }
                    // 32 keys = four 16-byte units of this row; unit u of a 64-key slice sits at (u ^ (row & 7))
                    const uint32_t row_base = p_s + (uint32_t)(c / 64) * kChunkBytes + (uint32_t)r * 128u;
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const uint32_t unit = (uint32_t)((c % 64) / 8 + u);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row_base + ((unit ^ (uint32_t)(r & 7)) << 4)),
                                     "r"(pk[4 * u]), "r"(pk[4 * u + 1]), "r"(pk[4 * u + 2]), "r"(pk[4 * u + 3]) : "memory");
                    }
                }
                if (j == n_kt - 1) {
                    // Tokens past the prompt's last position (the tail of its last page, repeated pages) hold
                    // whatever the pool held: their p is 0, but 0 x NaN would still poison P.V, so zero those V rows.
                    const int b = g & 1;
                    if (!mbar_wait(v_full(b), (g >> 1) & 1u, abortp)) { ok = false; break; }
                    if (key0 + r > pos_last) {
#pragma unroll
                        for (int c = 0; c < NCH; ++c)
#pragma unroll
                            for (int u = 0; u < 8; ++u)
                                asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(v_s + (uint32_t)b * kKvBytes + (uint32_t)c * kChunkBytes + (uint32_t)r * 128u + (uint32_t)u * 16u), "r"(0u) : "memory");
                    }
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");       // P (and zeroed V rows) visible to the tensor core's reads
                mbar_arrive(p_full);
            }
            if (!ok) break;
            // last tile's P.V, then normalise and store
            if (!mbar_wait(o_full, (g - 1) & 1u, abortp)) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const float inv = l > 0.f ? 1.f / l : 0.f;
            __nv_bfloat16* orow = p.out + (size_t)(row0 + r) * H * DH + (size_t)head * DH;
#pragma unroll
            for (int c = 0; c < DH; c += 32) {
                uint32_t v[32];
                tmem_ld32(t_lane + 128u + (uint32_t)c, v);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (r < nq) {
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        uint32_t w[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const __nv_bfloat162 h2 = __floats2bfloat162_rn((o_acc[c + i + 2 * k] + __uint_as_float(v[i + 2 * k])) * inv,
                                                                            (o_acc[c + i + 2 * k + 1] + __uint_as_float(v[i + 2 * k + 1])) * inv);
                            w[k] = *reinterpret_cast<const uint32_t*>(&h2);
                        }
                        *reinterpret_cast<uint4*>(orow + c + i) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicCAS(p.status, 0, kStatusTimeout);
    if (warp == 5) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

}  // namespace

// Returns false when the tensor-core path does not apply (fp32 pools, head sizes other than 64 / 96 / 128,
// no tensor-map encoder): the caller then runs the plain-FMA kernel.
bool launch_attention_prefill_tc(const cdb* h, int ln, int layer, const RowsDev& rows, const void* q, void* o, cudaStream_t st) {
    const int Dh = h->cfg.Dh, H = h->cfg.H;
    if (h->cfg.dtype != CDB_BF16 || (Dh != 64 && Dh != 96 && Dh != 128) || encode_fn() == nullptr) return false;
    const LayerKv kv = layer_kv(h, layer, rows);
    const long long kv_rows = (long long)kv.n_layers * kv.pool.n_phys_pages * 2 * H * kPageSize;
    if (kv_rows >= (1LL << 31)) return false;
    CUtensorMap map_q, map_kv;
    if (!make_map(&map_q, q, rows.n_rows, H * Dh, kQT) || !make_map(&map_kv, kv.pool.base, (int)kv_rows, Dh, kPageSize)) return false;
    const Lane& L = h->lane[ln];
    // pads first: rows the tiles do not cover keep a zero output
    cudaMemsetAsync(o, 0, (size_t)rows.n_rows * H * Dh * sizeof(__nv_bfloat16), st);
    launch_prefill_plan(h, ln, rows, kQT, st);
    PfParams p;
    p.rows = kv.rows; p.pool = kv.pool; p.layer = kv.layer; p.max_seqs = h->cfg.max_seqs;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)Dh);
    p.tiles = L.attn_item_start; p.tile_rows = L.pf_tile_rows; p.n_tiles = L.pf_n_tiles;
    p.out = (__nv_bfloat16*)o; p.status = h->status;
    const int nch = (Dh + 63) / 64;
    const size_t smem = 1024 + (size_t)(5 * nch + 2) * kChunkBytes;
    const int sms = h->sms;
    const long long max_items = (long long)rows.n_rows * H;            // at least one row per tile
    const int grid = (int)(max_items < sms ? max_items : sms);
    auto kern = Dh == 128 ? attn_prefill_tc_kernel<128> : Dh == 96 ? attn_prefill_tc_kernel<96> : attn_prefill_tc_kernel<64>;
    static bool attr_set_dev[kMaxDevices][3] = {};
    bool* attr_set = attr_set_dev[h->device];
    const int ki = Dh == 128 ? 0 : Dh == 96 ? 1 : 2;
    if (!attr_set[ki]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return false;
        attr_set[ki] = true;
    }
    ProfScope prof(h, kProfAttention, st);
    CDB_LAUNCH(h);
    return launch_pdl(kern, dim3(grid), dim3(kPfThreads), smem, st, map_q, map_kv, p) == cudaSuccess;
}

}  // namespace cdbk
