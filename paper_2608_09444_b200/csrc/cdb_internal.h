// Internal declarations shared by the translation units of libcdb.so (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>

#include "cdb.h"

namespace cdbk {

constexpr int kPageSize = 16;        // tokens per KV page
constexpr int kSplitTokens = 256;    // attention split length; depends on nothing but the row's own context
constexpr int kMaxKSplits = 8;       // most split-K parts of a projection
constexpr int kWsPerRow = 12;        // workspace floats per row, in units of d: 8 parts of [d] or 3 parts of [3d] fit
constexpr int kStatusPage = 1, kStatusPosition = 2, kStatusSeq = 3;
constexpr int kMaxDevices = 64;      // one-time per-device kernel set-up is remembered per device ordinal

// Tuning hooks: a build made with -DCDB_TUNING reads integer overrides from the environment (once per
// site); the shipped library has none and every hook folds to its default.
#ifdef CDB_TUNING
inline int tuning_int(const char* name, int dflt) { const char* v = getenv(name); return v ? atoi(v) : dflt; }
constexpr bool kTuningBuild = true;
#else
constexpr int tuning_int(const char*, int dflt) { return dflt; }
constexpr bool kTuningBuild = false;
#endif

enum class Epilogue : int { Store = 0, ResidualAdd = 1 };

// Device view of a row descriptor plus the KV pool, passed by value to kernels.
struct RowsDev {
    int32_t n_rows;
    const int32_t* seq_id;
    const int32_t* loop_depth;
    const int32_t* position;
    const int32_t* kv_slot;
    const int32_t* forced_exit;
    const int32_t* page_table;
    int32_t page_table_stride;
    int32_t n_slots;
    int32_t slot_override;   // >= 0: use this KV slot for every row (prelude / coda layers, prefill)
    const int32_t* n_live;   // device count of live rows or NULL: rows at an index >= *n_live are pads
    __device__ __forceinline__ int slot_of(int row) const { return slot_override >= 0 ? slot_override : kv_slot[row]; }
    // sequence id of a row, -1 for pads (0 when the call carries no sequence ids: LM head of gathered rows)
    __device__ __forceinline__ int seq_of(int row) const {
        if (n_live != nullptr && row >= *n_live) return -1;
        return seq_id != nullptr ? seq_id[row] : 0;
    }
};

struct KvPool {
    void* base;              // [layer][page][2][H][16][Dh]
    int32_t n_phys_pages;
    int32_t H, Dh;
    // element offsets (not bytes)
    __host__ __device__ size_t tile_elems() const { return (size_t)kPageSize * Dh; }
    __host__ __device__ size_t tile_offset(int layer, int page, int kv, int head) const {
        return ((((size_t)layer * n_phys_pages + page) * 2 + kv) * H + head) * tile_elems();
    }
};

// Scratch of one half-batch ("lane"): activations between the kernels of a layer, attention partials.
struct Lane {
    int rows_cap;                   // rows this lane's buffers hold
    void* xn;                       // [rows_cap][max(d,F)] normed activations (dtype)
    void* qrot;                     // [rows_cap][d] rotated queries (dtype)
    void* attn_o;                   // [rows_cap][d] attention output (dtype)
    void* act;                      // [rows_cap][F] SwiGLU output (dtype)
    float* qkv;                     // [rows_cap][3d]
    float* gu;                      // [2][rows_cap][F] gate and up projections
    float* ws;                      // [rows_cap * kWsPerRow * d] split-K partial products [part][row][features]
    float* attn_part;               // [rows_cap*H*max_splits][Dh + 2] split partials (o, m, l)
    int32_t* attn_item_start;       // [rows_cap + 1] exclusive scan of splits per row
    int32_t* attn_counters;         // [L] work-fetch counters
    int32_t* pf_tile_rows;          // [rows_cap] rows per prefill tile (tile starts reuse attn_item_start)
    int32_t* pf_n_tiles;            // [1]
};

}  // namespace cdbk

// A weight stack and its tile-major copy: [layer][feature tile][k block][128 rows][64 columns] bf16, zero padded,
// so that the [128 x 64] tile a projection CTA pulls per k-block is 16 KB of contiguous HBM.
struct TiledWeight {
    const char* orig;           // caller's row-major stack [layers][N][K]
    char* tiled;                // library-owned copy
    int layers, N, K;
};

struct cdb {
    cdb_config_t cfg;
    cdb_weights_t w;
    cdbk::KvPool pool;
    cdbk::KvPool pool_b;            // page space of the prelude and coda layers (base NULL: they share `pool`)
    const int32_t* table_b;         // its page table [max_seqs][table_b_stride] (device, caller-owned)
    int32_t table_b_stride;
    size_t elem_size;               // bytes of the configured dtype
    int device;                     // the device that was current in cdb_create: every call on the handle must run there
    int sms;                        // its multiprocessor count
    int max_splits;                 // ceil(max_position / kSplitTokens)

    // library-owned device memory
    float* rope_cos;                // [max_position][Dh/2]
    float* rope_sin;
    float* g_attn;                  // fp32 copies of the gains [L][d]
    float* g_mlp;
    float* g_final;                 // [d]
    float* gate_S;                  // [max_seqs] survival of the cumulative exit probability
    uint8_t* gate_fire;             // [max_seqs] stored exit signal
    TiledWeight tiled[6];           // W_qkv, W_o, W_gate, W_up, W_down, W_lm (bf16 configs)
    int n_tiled;

    // per-lane scratch, max_rows rows each: lane 0 serves the loop step, lane 1 the boundary calls and the second
    // half-batch of a two-stream step, lane 2 prompt processing - so that a boundary call and a prompt call may
    // each overlap a loop step on streams of their own
    cdbk::Lane lane[3];
    float* h_prev;                  // [max_rows][d] state at step entry (convergence gate)
    float* h_work;                  // [max_rows][d] prefill working state
    float* h_emit;                  // [max_rows][d] prefill: rows whose token is emitted
    float* logits;                  // [3][max_rows][V], one per lane
    uint8_t* exit_flag;             // [max_rows]
    int32_t* status;                // [1] first out-of-range access seen (0 = clean)
    unsigned int* grid_sync;        // [3] per lane: barrier word of the multi-stage layer kernel
    int32_t* emit_tmp;              // [max_rows]
    char err[256];
    // every cudaMalloc of the handle: base pointers (guard word, buffer, guard word) and buffer sizes
    static constexpr int kMaxAllocs = 96;
    char* alloc_base[kMaxAllocs];
    size_t alloc_bytes[kMaxAllocs];
    int n_allocs;

    // SM-partitioned execution of a loop step (CDB_FLAG_SM_PARTITION): two green contexts split the GPU's SMs;
    // the attention kernels of both half-batches run on part_attn (in order), everything else of half i on part_proj[i]
    void* green[2];                 // CUgreenCtx of the attention and of the projection partition (NULL: not available)
    cudaStream_t part_attn, part_proj[2];
    int part_attn_sms, part_proj_sms;
    cudaEvent_t ev_pre[2], ev_post[2];
    mutable int part_active;        // != 0 while such a step is being enqueued
    // two-stream execution of a loop step: second half-batch on `side`, joined by events
    cudaStream_t side;
    cudaEvent_t ev_fork, ev_join, ev_attn[2];
    mutable cudaEvent_t attn_split_done; // recorded right after the next attention split kernel when set
    mutable int attn_ctas_per_sm_cap;   // > 0 (two-stream step): attention runs one CTA of this many x 4 warps per SM
    mutable int qkv_parts_ready[3];     // per lane: split-K parts of the next layer's QKV projection already in the workspace
    mutable int prefill_attention;      // != 0 while cdb_prefill runs: layers use the query-tiled causal attention (1: tile list not planned yet)
    mutable int gemm_smem_cap;          // > 0 (two-stream step): projection kernels keep their shared-memory ring below this many bytes

    // instrumentation: kernel launch count, and CUDA-event pairs around the two heavy kernel classes
    mutable uint64_t launches;
    mutable int launch_error;       // a launcher could not set up its kernel (tensor-map encode failed)
    mutable int prof_on, prof_used;
    cudaEvent_t* prof_ev;           // [2 * kProfCap]
    uint8_t* prof_cls;              // [kProfCap]
};

#define CDB_LAUNCH(h) (++(h)->launches)

namespace cdbk {
// Programmatic dependent launch: the kernel may be scheduled while its predecessor on the stream is
// still draining; it runs its set-up, then pdl_wait() blocks until the predecessor has completed and
// its writes are visible.  Every kernel of the library calls pdl_trigger() first (lets ITS successor
// be scheduled early) and pdl_wait() before its first global-memory access.
// Rotation of one rotate-half pair (x_i, x_{i+Dh/2}) by the position's angle, with the roundings spelled out so
// that every kernel that rotates gives the same bits.
__device__ __forceinline__ float rope_lo(float a1, float a2, float c, float s) { return __fmaf_rn(a1, c, -__fmul_rn(a2, s)); }
__device__ __forceinline__ float rope_hi(float a1, float a2, float c, float s) { return __fmaf_rn(a2, c, __fmul_rn(a1, s)); }

__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#ifdef CDB_TUNING
// Tuning builds: every kernel's thread 32 of block 0 records the time at which its wait for the previous kernel ended
// (one shared buffer: word 0 counts, the times follow in launch order).  Each translation unit has its own copy of
// the pointer, set by trace_set_*().
static __device__ unsigned long long* t_trace;
__device__ __forceinline__ void pdl_wait() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (t_trace != nullptr && threadIdx.x == 32 && blockIdx.x == 0 && blockIdx.y == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t) :: "memory");
        const unsigned long long i = atomicAdd(t_trace, 1ULL);
        if (i < (1ULL << 20) - 2) t_trace[1 + i] = t;
    }
}
#define CDB_TRACE_SETTER(name) namespace cdbk { void name(unsigned long long* p) { cudaMemcpyToSymbol(t_trace, &p, sizeof(p)); } }
#else
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#define CDB_TRACE_SETTER(name)
#endif

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    static const bool no_pdl = tuning_int("CDB_NO_PDL", 0) != 0;     // tuning hook: plain stream-ordered launches
    cfg.attrs = attr; cfg.numAttrs = no_pdl ? 0 : 1;
    static const int carve = tuning_int("CDB_MISC_CARVEOUT", -2);    // tuning hook
    if (carve > -2) cudaFuncSetAttribute((const void*)kernel, cudaFuncAttributePreferredSharedMemoryCarveout, carve);
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
}  // namespace cdbk

namespace cdbk {
// What a layer's KV kernels see.  Without a boundary page space every layer lives in `pool` ([L] layers, page ids
// shared by all layers).  With one, the prelude and coda layers live in pool_b ([L_pre + L_coda] layers, one slot per
// sequence, their own page table) and `pool` holds the core layers alone ([L_core] layers): a depth slot then
// reserves pages in the core layers only, which is what the paper's Table 1 counts.
struct LayerKv { KvPool pool; int layer; int n_layers; RowsDev rows; };
inline LayerKv layer_kv(const cdb* h, int layer, const RowsDev& rows) {
    const int Lp = h->cfg.L_pre, Lc = h->cfg.L_core, Lo = h->cfg.L_coda;
    LayerKv k;
    k.pool = h->pool; k.layer = layer; k.n_layers = Lp + Lc + Lo; k.rows = rows;
    if (h->pool_b.base) {
        if (layer < Lp || layer >= Lp + Lc) {
            k.pool = h->pool_b; k.layer = layer < Lp ? layer : layer - Lc; k.n_layers = Lp + Lo;
            k.rows.page_table = h->table_b; k.rows.page_table_stride = h->table_b_stride;
            k.rows.n_slots = 1; k.rows.slot_override = 0;
        } else {
            k.layer = layer - Lp; k.n_layers = Lc;
        }
    }
    return k;
}

constexpr int kProfCap = 8192;
enum { kProfAttention = 0, kProfLinear = 1, kProfClasses = 2 };
// Brackets the kernels launched during its lifetime with an event pair when profiling is on.
struct ProfScope {
    const cdb* h; cudaStream_t st; int slot;
    ProfScope(const cdb* h_, int cls, cudaStream_t st_) : h(h_), st(st_), slot(-1) {
        if (h->prof_on && h->prof_used < kProfCap) {
            slot = h->prof_used++;
            h->prof_cls[slot] = (uint8_t)cls;
            cudaEventRecord(h->prof_ev[2 * slot], st);
        }
    }
    ~ProfScope() { if (slot >= 0) cudaEventRecord(h->prof_ev[2 * slot + 1], st); }
};
}  // namespace cdbk

namespace cdbk {

// ---- launchers (each enqueues on `st`; none synchronises) -----------------------------------
void launch_rmsnorm(const cdb* h, const float* x, const float* gain, void* out, const RowsDev& rows, cudaStream_t st);
void launch_rope_kv_write(const cdb* h, int ln, int layer, const float* qkv_parts, int parts, size_t part_stride, const RowsDev& rows, cudaStream_t st);
void launch_attention(const cdb* h, int ln, int layer, const RowsDev& rows, const void* q, void* o, cudaStream_t st);
void launch_attention_plan(const cdb* h, int ln, const RowsDev& rows, cudaStream_t st);
void launch_attention_prefill(const cdb* h, int ln, int layer, const RowsDev& rows, const void* q, void* o, cudaStream_t st);
void launch_prefill_plan(const cdb* h, int ln, const RowsDev& rows, int tile, cudaStream_t st);
bool launch_attention_prefill_tc(const cdb* h, int ln, int layer, const RowsDev& rows, const void* q, void* o, cudaStream_t st);
void launch_swiglu(const cdb* h, int ln, int n_rows, cudaStream_t st);
void launch_embed(const cdb* h, const int32_t* tokens, const RowsDev& rows, float* out, bool reset_gate, cudaStream_t st);
void launch_gate(const cdb* h, const RowsDev& rows, const float* x, const float* x_prev, float* gate_val_out,
                 uint8_t* fire_out, cudaStream_t st);
void launch_compact(const cdb* h, const RowsDev& rows, const uint8_t* fire_prev, int32_t* survivor_idx,
                    int32_t* exit_idx, int32_t* counts, cudaStream_t st);
void launch_gather(const cdb* h, const float* src, const int32_t* idx, const int32_t* count_dev, int max_count,
                   float* dst, cudaStream_t st);
void launch_argmax(const cdb* h, const float* logits, int n_rows, int32_t* token_out, cudaStream_t st);
void launch_copy_on_exit(const cdb* h, const RowsDev& rows, const int32_t* exit_depth, cudaStream_t st);

// x[row] += sum_s ws[s][row] (fixed order), then out[row] = RMSNorm(x[row]) * gain when gain != NULL.
void launch_reduce_residual_norm(const cdb* h, const float* ws, int splits, size_t split_stride, float* x, const float* gain,
                                 void* out, const RowsDev& rows, cudaStream_t st);
// bf16 tensor-core variants (gemm_tcgen05.cu)
size_t tiled_weight_bytes(int layers, int N, int K);
void launch_repack_tiled(const void* W, void* Wt, int layers, int N, int K, cudaStream_t st);
bool linear_tc_supported(const cdb* h, int n, int N, int K);
bool launch_gate_up_swiglu_tc(const cdb* h, const void* x, const void* Wg, const void* Wu, void* act, int n, int F, int K, cudaStream_t st);
int launch_linear_splitk_tc(const cdb* h, const void* x, const void* W, float* ws, int max_splits, int n, int N, int K, cudaStream_t st);
bool launch_linear_cluster_residual_tc(const cdb* h, const void* xin, const void* W, float* x, int n, int N, int K, int max_splits, cudaStream_t st);
bool launch_qkv_rope_cluster_tc(const cdb* h, int ln, int layer, const void* xin, const void* W_qkv, const RowsDev& rows, int max_splits, cudaStream_t st);
int launch_layer_tail_tc(const cdb* h, int ln, const RowsDev& rows, float* x, const void* W_o, const float* g_mlp,
                         const void* W_gate, const void* W_up, const void* W_down, const float* next_gain,
                         const void* W_qkv_next, cudaStream_t st);

// y[n,N] (fp32) = / += x[n,K] . W[N,K]^T ; x and W of the handle's dtype.
void launch_linear(const cdb* h, const void* x, const void* W, float* y, int n, int N, int K, Epilogue ep, cudaStream_t st);

}  // namespace cdbk
