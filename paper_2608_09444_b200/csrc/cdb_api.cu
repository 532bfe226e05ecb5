// C-ABI entry points of libcdb.so: argument checks, handle life cycle, and the launch sequences of
// the boundary stages, the loop step, the compaction and the prefill.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include <cuda.h>

#include "cdb_internal.h"

using namespace cdbk;

// The boundary stages (embedding / prelude, coda / LM head) use scratch lane 1 and the loop step lane 0, so a
// boundary call on one stream may overlap a loop step on another (the two-stream half-batch mode also uses
// lane 1 and must not be combined with that).
constexpr int kBoundaryLane = 1;
constexpr int kPrefillLane = 2;
constexpr int kMinSplitRows = 64;          // below this a loop step runs as one batch on one stream
constexpr int kSplitGemmSmemBytes = 0;            // no cap: a projection CTA co-resides with attention only when its ring is large
constexpr int kSplitAttnCtasPerSm = 3;     // attention CTAs per SM when two half-batches share the GPU

namespace {

int fail(cdb_t* h, int code, const char* msg) {
    if (h) snprintf(h->err, sizeof(h->err), "%s", msg);
    return code;
}

int fail_cuda(cdb_t* h, cudaError_t e, const char* where) {
    if (h) snprintf(h->err, sizeof(h->err), "%s: %s", where, cudaGetErrorString(e));
    return e == cudaErrorMemoryAllocation ? CDB_ERR_NOMEM : CDB_ERR_CUDA;
}

int check_launch(cdb_t* h, const char* where) {
    if (h->launch_error) { h->launch_error = 0; return fail(h, CDB_ERR_CUDA, "tensor-map encode failed: projection not launched"); }
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? CDB_OK : fail_cuda(h, e, where);
}

// Every scratch buffer sits between two guard words of kGuardBytes filled with a pattern; nothing the library
// launches may write them (cdb_debug_check_guards).  A stand-in for a memory checker on the library's own buffers.
constexpr size_t kGuardBytes = 256;
constexpr int kGuardPattern = 0xA5;

template <typename T> cudaError_t dev_alloc(cdb_t* h, T** p, size_t count) {
    *p = nullptr;
    const size_t bytes = ((count ? count : 1) * sizeof(T) + 15) / 16 * 16;
    char* base = nullptr;
    cudaError_t e = cudaMalloc((void**)&base, bytes + 2 * kGuardBytes);
    if (e != cudaSuccess) return e;
    cudaMemset(base, kGuardPattern, kGuardBytes);
    cudaMemset(base + kGuardBytes + bytes, kGuardPattern, kGuardBytes);
    if (h->n_allocs < cdb::kMaxAllocs) { h->alloc_base[h->n_allocs] = base; h->alloc_bytes[h->n_allocs] = bytes; ++h->n_allocs; }
    *p = (T*)(base + kGuardBytes);
    return cudaSuccess;
}

int slot_of_loop(int layout, int r) {
    if (layout == CDB_KV_DEPTH_INDEXED) return r - 1;
    if (layout == CDB_KV_FIRST_THEN_SHARED) return (r < 2 ? r : 2) - 1;
    return 0;
}

// Host-side descriptor checks; fills the device view.
int make_rows(cdb_t* h, const cdb_rows_t* rows, RowsDev* out, bool need_depth) {
    if (!rows) return fail(h, CDB_ERR_ARG, "rows is NULL");
    if (rows->n_rows < 0 || rows->n_rows > h->cfg.max_rows) return fail(h, CDB_ERR_CAPACITY, "n_rows exceeds max_rows");
    if (rows->n_rows > 0 && (!rows->seq_id || !rows->position || !rows->page_table))
        return fail(h, CDB_ERR_ARG, "rows.seq_id / position / page_table must be device pointers");
    if (need_depth && rows->n_rows > 0 && (!rows->loop_depth || !rows->kv_slot))
        return fail(h, CDB_ERR_ARG, "rows.loop_depth / kv_slot must be device pointers");
    if (rows->page_table_stride * kPageSize < 1) return fail(h, CDB_ERR_ARG, "page_table_stride must be positive");
    out->n_rows = rows->n_rows;
    out->seq_id = rows->seq_id;
    out->loop_depth = rows->loop_depth;
    out->position = rows->position;
    out->kv_slot = rows->kv_slot;
    out->forced_exit = rows->forced_exit;
    out->page_table = rows->page_table;
    out->page_table_stride = rows->page_table_stride;
    out->n_slots = h->cfg.n_slots;
    out->slot_override = -1;
    out->n_live = rows->n_rows_dev;
    return CDB_OK;
}

size_t wstride(const cdb_t* h, size_t elems) { return elems * h->elem_size; }
const void* layer_ptr(const cdb_t* h, const void* base, int layer, size_t elems_per_layer) {
    return (const char*)base + (size_t)layer * wstride(h, elems_per_layer);
}

bool use_tc_layers(const cdb_t* h);
}
#ifdef CDB_TUNING
namespace cdbk { void trace_set_attention(unsigned long long*); void trace_set_misc(unsigned long long*); void trace_set_gemm(unsigned long long*); }
#endif
namespace {

// One transformer layer on `x` (fp32 [n_rows, d], updated in place).  Steps A1-A6 of the loop step:
// RMSNorm + QKV projection, RoPE + KV page write, paged attention, output projection + residual,
// RMSNorm + gate/up projections + SwiGLU, down projection + residual.
void layer_forward(cdb_t* h, int ln, int layer, const RowsDev& rows, float* x, cudaStream_t st,
                   cudaEvent_t attn_after = nullptr, cudaEvent_t attn_done = nullptr) {
    const cdb_config_t& c = h->cfg;
    const Lane& L = h->lane[ln];
    const int n = rows.n_rows;
    const size_t d = c.d, F = c.F;
    launch_rmsnorm(h, x, h->g_attn + (size_t)layer * d, L.xn, rows, st);
    launch_linear(h, L.xn, layer_ptr(h, h->w.W_qkv, layer, 3 * d * d), L.qkv, n, 3 * c.d, c.d, Epilogue::Store, st);
    launch_rope_kv_write(h, ln, layer, L.qkv, 1, 0, rows, st);
    if (attn_after) cudaStreamWaitEvent(st, attn_after, 0);      // the other half-batch's attention goes first
    h->attn_split_done = attn_done;
    if (h->prefill_attention) launch_attention_prefill(h, ln, layer, rows, L.qrot, L.attn_o, st);
    else launch_attention(h, ln, layer, rows, L.qrot, L.attn_o, st);
    h->attn_split_done = nullptr;
    launch_linear(h, L.attn_o, layer_ptr(h, h->w.W_o, layer, d * d), x, n, c.d, c.d, Epilogue::ResidualAdd, st);
    launch_rmsnorm(h, x, h->g_mlp + (size_t)layer * d, L.xn, rows, st);
    bool fused_mlp = false;
    if (use_tc_layers(h)) {                  // bf16 tensor-core path: gate and up in one launch, SwiGLU in its epilogue
        ProfScope ps(h, kProfLinear, st);
        CDB_LAUNCH(h);
        fused_mlp = launch_gate_up_swiglu_tc(h, L.xn, layer_ptr(h, h->w.W_gate, layer, F * d), layer_ptr(h, h->w.W_up, layer, F * d),
                                             L.act, n, c.F, c.d, st);
    }
    if (!fused_mlp) {
        launch_linear(h, L.xn, layer_ptr(h, h->w.W_gate, layer, F * d), L.gu, n, c.F, c.d, Epilogue::Store, st);
        launch_linear(h, L.xn, layer_ptr(h, h->w.W_up, layer, F * d), L.gu + (size_t)L.rows_cap * F, n, c.F, c.d, Epilogue::Store, st);
        launch_swiglu(h, ln, n, st);
    }
    launch_linear(h, L.act, layer_ptr(h, h->w.W_down, layer, d * F), x, n, c.d, c.F, Epilogue::ResidualAdd, st);
}

// The same layer on the bf16 tensor-core path, with fewer and fatter launches: the two residual
// projections run split-K into a workspace and one row-wise kernel reduces the parts in fixed order,
// adds the residual and produces the next projection's normed input; gate and up run as one launch
// with SwiGLU in its epilogue.  xn_ready: L.xn already holds RMSNorm(x; g_attn[layer]).  next_gain:
// gain of the norm that follows this layer on the same rows (NULL: none).
void layer_forward_tc(cdb_t* h, int ln, int layer, const RowsDev& rows, float* x, cudaStream_t st, bool xn_ready,
                      const float* next_gain, int next_layer, cudaEvent_t attn_after = nullptr, cudaEvent_t attn_done = nullptr) {
    const cdb_config_t& c = h->cfg;
    const Lane& L = h->lane[ln];
    const int n = rows.n_rows;
    const size_t d = c.d, F = c.F;
    int& qkv_parts = h->qkv_parts_ready[ln];                    // > 0: the previous layer's launch already left this layer's QKV parts in L.ws
    if (!xn_ready) { launch_rmsnorm(h, x, h->g_attn + (size_t)layer * d, L.xn, rows, st); qkv_parts = 0; }
    // Split-K parts are summed inside thread-block clusters where that is the faster form (CDB_FLAG_WORKSPACE_PARTS:
    // always through a workspace and a row-wise kernel; same sums in the same order either way, so a row's result
    // does not depend on which form its batch took).  Measured on the 2048-wide model: the QKV projection with RoPE
    // and the KV page write in its epilogue wins up to 128 rows (one launch fewer), the in-cluster residual sums up
    // to 64 rows (-4 % step time at 64 rows, -7.5 % at 16); at 256 rows the exchange through distributed shared
    // memory costs as much as the workspace round trip it replaces and the step is 1 % slower.
    const bool in_cluster = !(c.flags & (CDB_FLAG_WORKSPACE_PARTS | CDB_FLAG_FUSED_STAGES)) && !h->part_active;
    static const int cluster_mask = tuning_int("CDB_CLUSTER_MASK", 7);       // tuning hook: 1 QKV, 2 output, 4 down projection
    static const int cluster_rows_qkv = tuning_int("CDB_CLUSTER_ROWS_QKV", 128), cluster_rows_res = tuning_int("CDB_CLUSTER_ROWS_RES", 64);
    {
        ProfScope ps(h, kProfLinear, st);
        int s = qkv_parts;
        bool done = false;
        if (!s && in_cluster && (cluster_mask & 1) && n <= cluster_rows_qkv && !h->prefill_attention) {       // projection, RoPE and KV page write in one launch
            done = launch_qkv_rope_cluster_tc(h, ln, layer, L.xn, layer_ptr(h, h->w.W_qkv, layer, 3 * d * d), rows, kWsPerRow / 3, st);
            if (done) CDB_LAUNCH(h);
        }
        if (!done) {
            if (!s) {
                CDB_LAUNCH(h);
                s = launch_linear_splitk_tc(h, L.xn, layer_ptr(h, h->w.W_qkv, layer, 3 * d * d), L.ws, kWsPerRow / 3, n, 3 * c.d, c.d, st);
                if (!s) h->launch_error = 1;
            }
            launch_rope_kv_write(h, ln, layer, L.ws, s, (size_t)n * 3 * d, rows, st);      // sums the parts
        }
        qkv_parts = 0;
    }
    if (attn_after) cudaStreamWaitEvent(st, attn_after, 0);      // the other half-batch's attention goes first
    h->attn_split_done = attn_done;
    if (h->prefill_attention) launch_attention_prefill(h, ln, layer, rows, L.qrot, L.attn_o, st);
    else launch_attention(h, ln, layer, rows, L.qrot, L.attn_o, st);
    h->attn_split_done = nullptr;
    if (c.flags & CDB_FLAG_FUSED_STAGES) {
        // everything after the attention, and the next layer's QKV projection, in one cooperative launch
        ProfScope ps(h, kProfLinear, st);
        CDB_LAUNCH(h);
        const int s = launch_layer_tail_tc(h, ln, rows, x, layer_ptr(h, h->w.W_o, layer, d * d), h->g_mlp + (size_t)layer * d,
                                           layer_ptr(h, h->w.W_gate, layer, F * d), layer_ptr(h, h->w.W_up, layer, F * d),
                                           layer_ptr(h, h->w.W_down, layer, d * F), next_gain,
                                           next_layer >= 0 ? layer_ptr(h, h->w.W_qkv, next_layer, 3 * d * d) : nullptr, st);
        if (s < 0) h->launch_error = 1;
        qkv_parts = s > 0 ? s : 0;
        return;
    }
    {
        ProfScope ps(h, kProfLinear, st);
        CDB_LAUNCH(h);
        int s = 0;
        if (!(in_cluster && (cluster_mask & 2) && n <= cluster_rows_res && launch_linear_cluster_residual_tc(h, L.attn_o, layer_ptr(h, h->w.W_o, layer, d * d), x, n, c.d, c.d, kMaxKSplits, st))) {
            s = launch_linear_splitk_tc(h, L.attn_o, layer_ptr(h, h->w.W_o, layer, d * d), L.ws, kMaxKSplits, n, c.d, c.d, st);
            if (!s) h->launch_error = 1;
        }
        launch_reduce_residual_norm(h, L.ws, s, (size_t)n * d, x, h->g_mlp + (size_t)layer * d, L.xn, rows, st);   // s == 0: the norm alone
    }
    {
        ProfScope ps(h, kProfLinear, st);
        CDB_LAUNCH(h);
        if (!launch_gate_up_swiglu_tc(h, L.xn, layer_ptr(h, h->w.W_gate, layer, F * d), layer_ptr(h, h->w.W_up, layer, F * d),
                                      L.act, n, c.F, c.d, st))
            h->launch_error = 1;
    }
    {
        ProfScope ps(h, kProfLinear, st);
        CDB_LAUNCH(h);
        int s = 0;
        if (!(in_cluster && (cluster_mask & 4) && n <= cluster_rows_res && launch_linear_cluster_residual_tc(h, L.act, layer_ptr(h, h->w.W_down, layer, d * F), x, n, c.d, c.F, kMaxKSplits, st))) {
            s = launch_linear_splitk_tc(h, L.act, layer_ptr(h, h->w.W_down, layer, d * F), L.ws, kMaxKSplits, n, c.d, c.F, st);
            if (!s) h->launch_error = 1;
        }
        if (s || next_gain) launch_reduce_residual_norm(h, L.ws, s, (size_t)n * d, x, next_gain, L.xn, rows, st);
    }
}

bool use_tc_layers(const cdb_t* h) {
    return h->cfg.dtype == CDB_BF16 && !(h->cfg.flags & (CDB_FLAG_SIMT_GEMM | CDB_FLAG_UNFUSED_LAYER)) && h->cfg.d <= 24 * 256 &&
           linear_tc_supported(h, 1, h->cfg.d, h->cfg.d);
}

// core layers [first, last) on one lane; picks the fused tensor-core flow when available
void core_layers(cdb_t* h, int ln, const RowsDev& rows, float* x, cudaStream_t st, cudaEvent_t attn_after_first,
                 cudaEvent_t attn_after, cudaEvent_t attn_done, int layer) {
    const cdb_config_t& c = h->cfg;
    const int first = c.L_pre, last = c.L_pre + c.L_core;
    cudaEvent_t after = layer == first ? attn_after_first : attn_after;
    if (use_tc_layers(h))
        layer_forward_tc(h, ln, layer, rows, x, st, layer > first, layer + 1 < last ? h->g_attn + (size_t)(layer + 1) * c.d : nullptr,
                         layer + 1 < last ? layer + 1 : -1, after, attn_done);
    else
        layer_forward(h, ln, layer, rows, x, st, after, attn_done);
}

// layers [first, last) of the prelude or coda on a decode batch (one row per sequence): the split-K flow when
// the tensor-core path is available, else the plain sequence
void boundary_layers(cdb_t* h, int ln, int first, int last, const RowsDev& rows, float* x, cudaStream_t st) {
    for (int l = first; l < last; ++l) {
        if (use_tc_layers(h))
            layer_forward_tc(h, ln, l, rows, x, st, l > first, l + 1 < last ? h->g_attn + (size_t)(l + 1) * h->cfg.d : nullptr,
                             l + 1 < last ? l + 1 : -1);
        else
            layer_forward(h, ln, l, rows, x, st);
    }
}

// final RMSNorm + LM head + greedy argmax on n rows of x
void lm_head(cdb_t* h, int ln, const RowsDev& rows, const float* x, int32_t* token_out, float* logits_out, cudaStream_t st) {
    const cdb_config_t& c = h->cfg;
    float* logits = logits_out ? logits_out : h->logits + (size_t)ln * h->cfg.max_rows * h->cfg.V;
    launch_rmsnorm(h, x, h->g_final, h->lane[ln].xn, rows, st);
    launch_linear(h, h->lane[ln].xn, h->w.W_lm, logits, rows.n_rows, c.V, c.d, Epilogue::Store, st);
    launch_argmax(h, logits, rows.n_rows, token_out, st);
}

// ---- SM partition: two green contexts (driver API, looked up at run time like the tensor-map encoder) ------------
constexpr int kPartitionAttnSms = 112;     // SMs of the attention partition (a multiple of 8); the rest run the projections

template <typename F> bool driver_fn(const char* name, F* out) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPointByVersion(name, &p, CUDA_VERSION, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess || !p) return false;
    *out = (F)p;
    return true;
}

void free_sm_partition(cdb_t* h) {
    if (h->part_attn) cudaStreamDestroy(h->part_attn);
    for (cudaStream_t& s : h->part_proj) if (s) cudaStreamDestroy(s);
    h->part_attn = nullptr; h->part_proj[0] = h->part_proj[1] = nullptr;
    for (int i = 0; i < 2; ++i) {
        if (h->ev_pre[i]) cudaEventDestroy(h->ev_pre[i]);
        if (h->ev_post[i]) cudaEventDestroy(h->ev_post[i]);
        h->ev_pre[i] = h->ev_post[i] = nullptr;
    }
    CUresult (*destroy)(CUgreenCtx) = nullptr;
    if ((h->green[0] || h->green[1]) && driver_fn("cuGreenCtxDestroy", &destroy))
        for (void*& g : h->green) { if (g) destroy((CUgreenCtx)g); g = nullptr; }
}

// Leaves h->green[0] == NULL (and the flag without effect) when the driver cannot partition the SMs.
void make_sm_partition(cdb_t* h) {
    CUresult (*get_res)(CUdevice, CUdevResource*, CUdevResourceType) = nullptr;
    CUresult (*split)(CUdevResource*, unsigned int*, const CUdevResource*, CUdevResource*, unsigned int, unsigned int) = nullptr;
    CUresult (*gen_desc)(CUdevResourceDesc*, CUdevResource*, unsigned int) = nullptr;
    CUresult (*create)(CUgreenCtx*, CUdevResourceDesc, CUdevice, unsigned int) = nullptr;
    CUresult (*stream_create)(CUstream*, CUgreenCtx, unsigned int, int) = nullptr;
    CUresult (*dev_get)(CUdevice*, int) = nullptr;
    if (!driver_fn("cuDeviceGetDevResource", &get_res) || !driver_fn("cuDevSmResourceSplitByCount", &split) ||
        !driver_fn("cuDevResourceGenerateDesc", &gen_desc) || !driver_fn("cuGreenCtxCreate", &create) ||
        !driver_fn("cuGreenCtxStreamCreate", &stream_create) || !driver_fn("cuDeviceGet", &dev_get)) {
        if (kTuningBuild) fprintf(stderr, "sm partition: driver entry points missing\n");
        return;
    }
    static const int attn_sms = tuning_int("CDB_PART_ATTN_SMS", kPartitionAttnSms);     // tuning hook
    CUdevice dev;
    CUdevResource all, part[2];
    unsigned int groups = 1;
    if (dev_get(&dev, h->device) != CUDA_SUCCESS || get_res(dev, &all, CU_DEV_RESOURCE_TYPE_SM) != CUDA_SUCCESS ||
        split(&part[0], &groups, &all, &part[1], 0, (unsigned int)attn_sms) != CUDA_SUCCESS || groups != 1 || part[1].sm.smCount < 8) {
        if (kTuningBuild) fprintf(stderr, "sm partition: split failed (groups %u)\n", groups);
        return;
    }
    CUgreenCtx g[2] = {nullptr, nullptr};
    for (int i = 0; i < 2; ++i) {
        CUdevResourceDesc desc;
        if (gen_desc(&desc, &part[i], 1) != CUDA_SUCCESS || create(&g[i], desc, dev, CU_GREEN_CTX_DEFAULT_STREAM) != CUDA_SUCCESS) { g[i] = nullptr; break; }
    }
    CUstream sa = nullptr, sp[2] = {nullptr, nullptr};
    const bool ok = g[0] && g[1] && stream_create(&sa, g[0], CU_STREAM_NON_BLOCKING, 0) == CUDA_SUCCESS &&
                    stream_create(&sp[0], g[1], CU_STREAM_NON_BLOCKING, 0) == CUDA_SUCCESS &&
                    stream_create(&sp[1], g[1], CU_STREAM_NON_BLOCKING, 0) == CUDA_SUCCESS;
    h->green[0] = g[0]; h->green[1] = g[1];
    h->part_attn = (cudaStream_t)sa; h->part_proj[0] = (cudaStream_t)sp[0]; h->part_proj[1] = (cudaStream_t)sp[1];
    h->part_attn_sms = (int)part[0].sm.smCount; h->part_proj_sms = (int)part[1].sm.smCount;
    for (int i = 0; i < 2; ++i) {
        cudaEventCreateWithFlags(&h->ev_pre[i], cudaEventDisableTiming);
        cudaEventCreateWithFlags(&h->ev_post[i], cudaEventDisableTiming);
    }
    if (kTuningBuild) fprintf(stderr, "sm partition: %s, attention %d SMs, projections %d SMs\n", ok ? "ready" : "stream / context creation failed", h->part_attn_sms, h->part_proj_sms);
    if (!ok) free_sm_partition(h);
}

void free_all(cdb_t* h) {
    for (int i = 0; i < h->n_allocs; ++i) cudaFree(h->alloc_base[i]);     // every scratch buffer (with its guards)
    h->n_allocs = 0;
    for (int i = 0; i < h->n_tiled; ++i) if (h->tiled[i].tiled) cudaFree(h->tiled[i].tiled);
    h->n_tiled = 0;
    free_sm_partition(h);
    if (h->side) cudaStreamDestroy(h->side);
    if (h->ev_fork) cudaEventDestroy(h->ev_fork);
    if (h->ev_join) cudaEventDestroy(h->ev_join);
    for (cudaEvent_t e : h->ev_attn) if (e) cudaEventDestroy(e);
    if (h->prof_ev) {
        for (int i = 0; i < 2 * kProfCap; ++i) if (h->prof_ev[i]) cudaEventDestroy(h->prof_ev[i]);
        delete[] h->prof_ev;
        delete[] h->prof_cls;
        h->prof_ev = nullptr;
    }
}

template <typename T> __global__ void to_f32_kernel(const T* in, float* out, size_t n) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        out[i] = (float)in[i];
}

__global__ void init_gate_state_kernel(float* S, uint8_t* fire, int n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) { S[i] = 1.f; fire[i] = 0; }
}

void gains_to_f32(const cdb_t* h, const void* src, float* dst, size_t n) {
    if (h->cfg.dtype == CDB_FP32) to_f32_kernel<float><<<64, 256>>>((const float*)src, dst, n);
    else to_f32_kernel<__nv_bfloat16><<<64, 256>>>((const __nv_bfloat16*)src, dst, n);
}

}  // namespace

extern "C" {

int cdb_create(const cdb_config_t* cfg, const cdb_weights_t* w, cdb_t** out) {
    if (!cfg || !w || !out) return CDB_ERR_ARG;
    *out = nullptr;
    const cdb_config_t& c = *cfg;
    const int L = c.L_pre + c.L_core + c.L_coda;
    const int want_slots = c.kv_layout == CDB_KV_SHARED ? 1 : c.kv_layout == CDB_KV_DEPTH_INDEXED ? c.R : 2;
    if (c.V < 1 || c.d < 1 || c.H < 1 || c.F < 1 || c.d != c.H * c.Dh || (c.Dh != 64 && c.Dh != 96 && c.Dh != 128) ||
        c.L_pre < 0 || c.L_core < 1 || c.L_coda < 0 || c.R < 1 || c.r_min < 1 || c.page_size != kPageSize ||
        (c.dtype != CDB_FP32 && c.dtype != CDB_BF16) || c.max_rows < 1 || c.max_seqs < 1 || c.max_position < 1 ||
        c.kv_layout < 0 || c.kv_layout > 2 || c.n_slots != want_slots || c.gate_kind < 0 || c.gate_kind > 2 ||
        c.d % 8 != 0 || c.F % 8 != 0)
        return CDB_ERR_ARG;
    if (!w->W_qkv || !w->W_o || !w->W_gate || !w->W_up || !w->W_down || !w->g_attn || !w->g_mlp || !w->embed ||
        !w->g_final || !w->W_lm || (c.gate_kind == CDB_GATE_SIGMOID_CDF && !w->w_gate))
        return CDB_ERR_ARG;
    cdb_t* h = new (std::nothrow) cdb_t();
    if (!h) return CDB_ERR_NOMEM;
    memset(h, 0, sizeof(*h));
    h->cfg = c;
    h->w = *w;
    h->elem_size = c.dtype == CDB_FP32 ? 4 : 2;
    h->max_splits = (c.max_position + kSplitTokens - 1) / kSplitTokens;
    {
        int dev = 0;
        h->sms = 148;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices ||
            cudaDeviceGetAttribute(&h->sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || h->sms < 1) {
            delete h;
            return CDB_ERR_CUDA;
        }
        h->device = dev;
    }
    h->pool.H = c.H;
    h->pool.Dh = c.Dh;
    const size_t R_ = c.max_rows, d = c.d, F = c.F, half = c.Dh / 2;
    const size_t wide = d > F ? d : F;
    const int n_layers = L;
    cudaError_t e = cudaSuccess;
#define CDB_ALLOC(ptr, type, count) if (e == cudaSuccess) e = dev_alloc<type>(h, (type**)&(ptr), (count))
    CDB_ALLOC(h->rope_cos, float, (size_t)c.max_position * half);
    CDB_ALLOC(h->rope_sin, float, (size_t)c.max_position * half);
    CDB_ALLOC(h->g_attn, float, (size_t)L * d);
    CDB_ALLOC(h->g_mlp, float, (size_t)L * d);
    CDB_ALLOC(h->g_final, float, d);
    CDB_ALLOC(h->gate_S, float, c.max_seqs);
    CDB_ALLOC(h->gate_fire, uint8_t, c.max_seqs);
    for (int ln = 0; ln < 3; ++ln) {
        Lane& L = h->lane[ln];
        L.rows_cap = c.max_rows;
        const size_t r = L.rows_cap;
        CDB_ALLOC(L.xn, char, r * wide * h->elem_size);
        CDB_ALLOC(L.qrot, char, r * d * h->elem_size);
        CDB_ALLOC(L.attn_o, char, r * d * h->elem_size);
        CDB_ALLOC(L.act, char, r * F * h->elem_size);
        CDB_ALLOC(L.qkv, float, r * 3 * d);
        CDB_ALLOC(L.gu, float, r * 2 * F);
        CDB_ALLOC(L.ws, float, (size_t)kWsPerRow * r * d);
        CDB_ALLOC(L.attn_part, float, r * c.H * h->max_splits * (size_t)(c.Dh + 2));
        CDB_ALLOC(L.attn_item_start, int32_t, r + 1);
        CDB_ALLOC(L.attn_counters, int32_t, n_layers);
        CDB_ALLOC(L.pf_tile_rows, int32_t, r);
        CDB_ALLOC(L.pf_n_tiles, int32_t, 1);
    }
    CDB_ALLOC(h->h_prev, float, R_ * d);
    CDB_ALLOC(h->h_work, float, R_ * d);
    CDB_ALLOC(h->logits, float, 3 * R_ * (size_t)c.V);
    CDB_ALLOC(h->h_emit, float, R_ * d);
    CDB_ALLOC(h->exit_flag, uint8_t, R_);
    CDB_ALLOC(h->status, int32_t, 1);
    CDB_ALLOC(h->grid_sync, unsigned int, 3);
    CDB_ALLOC(h->emit_tmp, int32_t, R_);
#undef CDB_ALLOC
    if (e != cudaSuccess) { free_all(h); delete h; cudaGetLastError(); return e == cudaErrorMemoryAllocation ? CDB_ERR_NOMEM : CDB_ERR_CUDA; }

    // RoPE table: angle = position * theta^(-2i/Dh), evaluated in double, stored as fp32
    {
        std::vector<float> cs((size_t)c.max_position * half), sn((size_t)c.max_position * half);
        for (size_t i = 0; i < half; ++i) {
            const double inv_freq = std::pow((double)c.rope_theta, -2.0 * (double)i / (double)c.Dh);
            for (int p = 0; p < c.max_position; ++p) {
                const double a = (double)p * inv_freq;
                cs[(size_t)p * half + i] = (float)std::cos(a);
                sn[(size_t)p * half + i] = (float)std::sin(a);
            }
        }
        e = cudaMemcpy(h->rope_cos, cs.data(), cs.size() * sizeof(float), cudaMemcpyHostToDevice);
        if (e == cudaSuccess) e = cudaMemcpy(h->rope_sin, sn.data(), sn.size() * sizeof(float), cudaMemcpyHostToDevice);
    }
    if (e == cudaSuccess && c.dtype == CDB_BF16 && !(c.flags & CDB_FLAG_SIMT_GEMM)) {
        // tile-major copies of the projection weights (the caller's row-major tensors stay borrowed)
        struct { const void* p; int layers, N, K; } stacks[6] = {
            {w->W_qkv, L, 3 * c.d, c.d}, {w->W_o, L, c.d, c.d}, {w->W_gate, L, c.F, c.d},
            {w->W_up, L, c.F, c.d}, {w->W_down, L, c.d, c.F}, {w->W_lm, 1, c.V, c.d}};
        for (int i = 0; i < 6 && e == cudaSuccess; ++i) {
            TiledWeight& t = h->tiled[h->n_tiled];
            t.orig = (const char*)stacks[i].p; t.layers = stacks[i].layers; t.N = stacks[i].N; t.K = stacks[i].K;
            e = cudaMalloc((void**)&t.tiled, tiled_weight_bytes(t.layers, t.N, t.K));
            if (e != cudaSuccess) { t.tiled = nullptr; break; }
            ++h->n_tiled;
            launch_repack_tiled(t.orig, t.tiled, t.layers, t.N, t.K, 0);
        }
    }
    if (e == cudaSuccess) {
        gains_to_f32(h, w->g_attn, h->g_attn, (size_t)L * d);
        gains_to_f32(h, w->g_mlp, h->g_mlp, (size_t)L * d);
        gains_to_f32(h, w->g_final, h->g_final, d);
        init_gate_state_kernel<<<(c.max_seqs + 255) / 256, 256>>>(h->gate_S, h->gate_fire, c.max_seqs);
        cudaMemset(h->status, 0, sizeof(int32_t));
        cudaMemset(h->grid_sync, 0, 3 * sizeof(unsigned int));
        for (int ln = 0; ln < 3; ++ln) cudaMemset(h->lane[ln].attn_counters, 0, sizeof(int32_t) * L);
        if (cudaStreamCreateWithFlags(&h->side, cudaStreamNonBlocking) != cudaSuccess) h->side = nullptr;
        if (c.flags & CDB_FLAG_SM_PARTITION) make_sm_partition(h);
        cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming);
        cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming);
        cudaEventCreateWithFlags(&h->ev_attn[0], cudaEventDisableTiming);
        cudaEventCreateWithFlags(&h->ev_attn[1], cudaEventDisableTiming);
        e = cudaDeviceSynchronize();
    }
    if (e != cudaSuccess) { free_all(h); delete h; cudaGetLastError(); return CDB_ERR_CUDA; }
#ifdef CDB_TUNING
    if (const char* t = getenv("CDB_TRACE")) {                   // tuning hook: device buffer for the kernels' start times
        unsigned long long* p = (unsigned long long*)strtoull(t, nullptr, 0);
        trace_set_attention(p); trace_set_misc(p); trace_set_gemm(p);
    }
#endif
    *out = h;
    return CDB_OK;
}

int cdb_destroy(cdb_t* h) {
    if (!h) return CDB_OK;
    cudaDeviceSynchronize();
    free_all(h);
    delete h;
    return CDB_OK;
}

const char* cdb_last_error(const cdb_t* h) { return h ? h->err : "invalid handle"; }

int cdb_kv_bind(cdb_t* h, void* pool_device, size_t bytes, int32_t n_phys_pages) {
    if (!h) return CDB_ERR_ARG;
    if (!pool_device || n_phys_pages < 1) return fail(h, CDB_ERR_ARG, "pool is NULL or has no pages");
    // with a boundary page space bound, this pool holds the core layers alone
    const size_t L = h->pool_b.base ? h->cfg.L_core : h->cfg.L_pre + h->cfg.L_core + h->cfg.L_coda;
    const size_t need = L * n_phys_pages * 2 * h->cfg.H * kPageSize * h->cfg.Dh * h->elem_size;
    if (bytes < need) return fail(h, CDB_ERR_ARG, "pool is smaller than [layers][pages][2][H][16][Dh]");
    if ((uintptr_t)pool_device % 16) return fail(h, CDB_ERR_ARG, "pool must be 16-byte aligned");
    h->pool.base = pool_device;
    h->pool.n_phys_pages = n_phys_pages;
    return CDB_OK;
}

int cdb_kv_bind_boundary(cdb_t* h, void* pool_device, size_t bytes, int32_t n_phys_pages, const int32_t* page_table,
                         int32_t page_table_stride) {
    if (!h) return CDB_ERR_ARG;
    const size_t Lb = h->cfg.L_pre + h->cfg.L_coda;
    if (Lb == 0) return fail(h, CDB_ERR_STATE, "the model has no prelude or coda layers");
    if (h->pool.base) return fail(h, CDB_ERR_STATE, "bind the boundary page space before cdb_kv_bind");
    if (!pool_device || n_phys_pages < 1 || !page_table || page_table_stride < 1) return fail(h, CDB_ERR_ARG, "pool / page table is NULL or empty");
    const size_t need = Lb * n_phys_pages * 2 * h->cfg.H * kPageSize * h->cfg.Dh * h->elem_size;
    if (bytes < need) return fail(h, CDB_ERR_ARG, "boundary pool is smaller than [L_pre + L_coda][pages][2][H][16][Dh]");
    if ((uintptr_t)pool_device % 16) return fail(h, CDB_ERR_ARG, "pool must be 16-byte aligned");
    h->pool_b.base = pool_device;
    h->pool_b.n_phys_pages = n_phys_pages;
    h->pool_b.H = h->cfg.H;
    h->pool_b.Dh = h->cfg.Dh;
    h->table_b = page_table;
    h->table_b_stride = page_table_stride;
    return CDB_OK;
}

int cdb_set_gate(cdb_t* h, float b_gate, float q_or_eps) {
    if (!h) return CDB_ERR_ARG;
    h->cfg.b_gate = b_gate;
    h->cfg.q_or_eps = q_or_eps;
    return CDB_OK;
}

static int boundary_in(cdb_t* h, const int32_t* token_ids, const cdb_rows_t* rows, float* h_out, void* stream, bool prelude) {
    if (!h) return CDB_ERR_ARG;
    RowsDev rd;
    int rc = make_rows(h, rows, &rd, false);
    if (rc) return rc;
    if (rd.n_rows == 0) return CDB_OK;
    if (!token_ids || !h_out) return fail(h, CDB_ERR_ARG, "token_ids / h_out is NULL");
    cudaStream_t st = (cudaStream_t)stream;
    launch_embed(h, token_ids, rd, h_out, true, st);
    if (prelude && h->cfg.L_pre > 0) {
        if (!h->pool.base) return fail(h, CDB_ERR_STATE, "no KV pool bound");
        rd.slot_override = 0;
        launch_attention_plan(h, kBoundaryLane, rd, st);
        boundary_layers(h, kBoundaryLane, 0, h->cfg.L_pre, rd, h_out, st);
    }
    return check_launch(h, "cdb_boundary_embed/prelude");
}

int cdb_boundary_embed(cdb_t* h, const int32_t* token_ids, const cdb_rows_t* rows, float* h_out, void* stream) {
    return boundary_in(h, token_ids, rows, h_out, stream, false);
}

int cdb_boundary_prelude(cdb_t* h, const int32_t* token_ids, const cdb_rows_t* rows, float* h_out, void* stream) {
    return boundary_in(h, token_ids, rows, h_out, stream, true);
}

int cdb_loop_step(cdb_t* h, const cdb_rows_t* rows, float* h_inout, float* gate_val_out, uint8_t* fire_out, void* stream) {
    if (!h) return CDB_ERR_ARG;
    RowsDev rd;
    int rc = make_rows(h, rows, &rd, true);
    if (rc) return rc;
    if (rd.n_rows == 0) return CDB_OK;
    if (!h_inout) return fail(h, CDB_ERR_ARG, "h_inout is NULL");
    if (!h->pool.base) return fail(h, CDB_ERR_STATE, "no KV pool bound");
    cudaStream_t st = (cudaStream_t)stream;
    const cdb_config_t& c = h->cfg;
    if (c.gate_kind == CDB_GATE_L2_CONVERGENCE)
        cudaMemcpyAsync(h->h_prev, h_inout, (size_t)rd.n_rows * c.d * sizeof(float), cudaMemcpyDeviceToDevice, st);
    const int n0 = (rd.n_rows + 1) / 2;
    const bool split = (c.flags & CDB_FLAG_TWO_STREAM) && h->side && rd.n_rows >= kMinSplitRows && !rd.n_live;   // (a half-batch view cannot shift a device-side count)
    const bool partitioned = (c.flags & CDB_FLAG_SM_PARTITION) && h->green[0] && rd.n_rows >= kMinSplitRows && !rd.n_live && use_tc_layers(h);
    if (partitioned) {
        // Two half-batches, the GPU's SMs split between two green contexts: the attention kernels of both halves run
        // one after the other on the attention partition (the KV stream never stops), everything else of a half runs
        // on the projection partition while the OTHER half's KV streams.
        RowsDev half[2] = {rd, rd};
        half[0].n_rows = n0;
        half[1].n_rows = rd.n_rows - n0;
        half[1].seq_id += n0; half[1].loop_depth += n0; half[1].position += n0; half[1].kv_slot += n0;
        if (half[1].forced_exit) half[1].forced_exit += n0;
        float* xs[2] = {h_inout, h_inout + (size_t)n0 * c.d};
        cudaEventRecord(h->ev_fork, st);
        for (int i = 0; i < 2; ++i) cudaStreamWaitEvent(h->part_proj[i], h->ev_fork, 0);
        cudaStreamWaitEvent(h->part_attn, h->ev_fork, 0);
        for (int i = 0; i < 2; ++i) { h->part_active = i + 1; launch_attention_plan(h, i, half[i], h->part_proj[i]); }
        for (int l = c.L_pre; l < c.L_pre + c.L_core; ++l)
            for (int i = 0; i < 2; ++i) {
                h->part_active = i + 1;
                core_layers(h, i, half[i], xs[i], h->part_proj[i], nullptr, nullptr, nullptr, l);
            }
        h->part_active = 0;
        for (int i = 0; i < 2; ++i) { cudaEventRecord(h->ev_post[i], h->part_proj[i]); cudaStreamWaitEvent(st, h->ev_post[i], 0); }
    } else if (!split) {
        h->attn_ctas_per_sm_cap = 0;
        launch_attention_plan(h, 0, rd, st);
        for (int l = c.L_pre; l < c.L_pre + c.L_core; ++l) core_layers(h, 0, rd, h_inout, st, nullptr, nullptr, nullptr, l);
    } else {
        // Two half-batches on two streams: while one half streams its KV pages through the attention
        // kernel (HBM-bound), the other half's projections and row-wise kernels run beside it.  Rows
        // are independent, so the halves never synchronise inside the step.
        RowsDev half[2] = {rd, rd};
        half[0].n_rows = n0;
        half[1].n_rows = rd.n_rows - n0;
        half[1].seq_id += n0; half[1].loop_depth += n0; half[1].position += n0; half[1].kv_slot += n0;
        if (half[1].forced_exit) half[1].forced_exit += n0;
        h->attn_ctas_per_sm_cap = kSplitAttnCtasPerSm;
        h->gemm_smem_cap = kSplitGemmSmemBytes;
        cudaEventRecord(h->ev_fork, st);
        cudaStreamWaitEvent(h->side, h->ev_fork, 0);
        cudaStream_t ss[2] = {st, h->side};
        float* xs[2] = {h_inout, h_inout + (size_t)n0 * c.d};
        for (int ln = 0; ln < 2; ++ln) launch_attention_plan(h, ln, half[ln], ss[ln]);
        // The two attention kernels are chained A(l), B(l), A(l+1), ...: each then streams at full HBM
        // bandwidth, and the other half's projections fill the SMs' spare issue slots meanwhile.
        // Without the chain both halves drift into lock-step (attention together, projections together).
        for (int l = c.L_pre; l < c.L_pre + c.L_core; ++l) {
            core_layers(h, 0, half[0], xs[0], ss[0], nullptr, h->ev_attn[1], h->ev_attn[0], l);
            core_layers(h, 1, half[1], xs[1], ss[1], h->ev_attn[0], h->ev_attn[0], h->ev_attn[1], l);
        }
        cudaEventRecord(h->ev_join, h->side);
        cudaStreamWaitEvent(st, h->ev_join, 0);
        h->attn_ctas_per_sm_cap = 0;
        h->gemm_smem_cap = 0;
    }
    launch_gate(h, rd, h_inout, h->h_prev, gate_val_out, fire_out, st);
    return check_launch(h, "cdb_loop_step");
}

int cdb_compact(cdb_t* h, const cdb_rows_t* rows, const uint8_t* fire_prev, const float* h_src, int32_t* survivor_idx,
                int32_t* exit_idx, int32_t* counts, float* h_next, float* h_exit, void* stream) {
    if (!h) return CDB_ERR_ARG;
    RowsDev rd;
    int rc = make_rows(h, rows, &rd, false);
    if (rc) return rc;
    if (rd.n_rows > 0 && !rows->loop_depth) return fail(h, CDB_ERR_ARG, "rows.loop_depth is NULL");
    if (!survivor_idx || !exit_idx || !counts) return fail(h, CDB_ERR_ARG, "index lists / counts are NULL");
    cudaStream_t st = (cudaStream_t)stream;
    launch_compact(h, rd, fire_prev, survivor_idx, exit_idx, counts, st);
    if (h_src) {
        if (h_next) launch_gather(h, h_src, survivor_idx, counts, rd.n_rows, h_next, st);
        if (h_exit) launch_gather(h, h_src, exit_idx, counts + 1, rd.n_rows, h_exit, st);
    }
    return check_launch(h, "cdb_compact");
}

int cdb_gather_rows(cdb_t* h, const float* h_src, const int32_t* idx, const int32_t* count_device, int32_t max_count,
                    float* h_dst, void* stream) {
    if (!h) return CDB_ERR_ARG;
    if (max_count < 0 || max_count > h->cfg.max_rows) return fail(h, CDB_ERR_CAPACITY, "max_count exceeds max_rows");
    if (max_count == 0) return CDB_OK;
    if (!h_src || !idx || !h_dst) return fail(h, CDB_ERR_ARG, "NULL argument");
    launch_gather(h, h_src, idx, count_device, max_count, h_dst, (cudaStream_t)stream);
    return check_launch(h, "cdb_gather_rows");
}

int cdb_boundary_coda_lmhead(cdb_t* h, const cdb_rows_t* rows, float* h_exit, int32_t* token_out, float* logits_out, void* stream) {
    if (!h) return CDB_ERR_ARG;
    RowsDev rd;
    int rc = make_rows(h, rows, &rd, false);
    if (rc) return rc;
    if (rd.n_rows == 0) return CDB_OK;
    if (!h_exit || !token_out) return fail(h, CDB_ERR_ARG, "h_exit / token_out is NULL");
    cudaStream_t st = (cudaStream_t)stream;
    const cdb_config_t& c = h->cfg;
    if (c.L_coda > 0) {
        if (!h->pool.base) return fail(h, CDB_ERR_STATE, "no KV pool bound");
        rd.slot_override = 0;
        launch_attention_plan(h, kBoundaryLane, rd, st);
        boundary_layers(h, kBoundaryLane, c.L_pre + c.L_core, c.L_pre + c.L_core + c.L_coda, rd, h_exit, st);
    }
    lm_head(h, kBoundaryLane, rd, h_exit, token_out, logits_out, st);
    return check_launch(h, "cdb_boundary_coda_lmhead");
}

int cdb_prefill(cdb_t* h, const int32_t* token_ids, const cdb_rows_t* rows, const int32_t* emit_idx, int32_t n_emit,
                int32_t* token_out, float* logits_out, void* stream) {
    if (!h) return CDB_ERR_ARG;
    RowsDev rd;
    int rc = make_rows(h, rows, &rd, false);
    if (rc) return rc;
    if (rd.n_rows == 0) return CDB_OK;
    if (!token_ids) return fail(h, CDB_ERR_ARG, "token_ids is NULL");
    if (n_emit < 0 || n_emit > rd.n_rows || (n_emit > 0 && (!emit_idx || !token_out))) return fail(h, CDB_ERR_ARG, "bad emit list");
    if (!h->pool.base) return fail(h, CDB_ERR_STATE, "no KV pool bound");
    cudaStream_t st = (cudaStream_t)stream;
    const cdb_config_t& c = h->cfg;
    float* x = h->h_work;
    h->prefill_attention = 1;
    launch_embed(h, token_ids, rd, x, true, st);
    launch_attention_plan(h, kPrefillLane, rd, st);
    rd.slot_override = 0;
    for (int l = 0; l < c.L_pre; ++l) layer_forward(h, kPrefillLane, l, rd, x, st);
    for (int r = 1; r <= c.R; ++r) {
        rd.slot_override = slot_of_loop(c.kv_layout, r);
        for (int l = c.L_pre; l < c.L_pre + c.L_core; ++l) layer_forward(h, kPrefillLane, l, rd, x, st);
    }
    rd.slot_override = 0;
    for (int l = c.L_pre + c.L_core; l < c.L_pre + c.L_core + c.L_coda; ++l) layer_forward(h, kPrefillLane, l, rd, x, st);
    h->prefill_attention = 0;
    if (n_emit > 0) {
        // gather the emitting rows, then LM head on them
        launch_gather(h, x, emit_idx, nullptr, n_emit, h->h_emit, st);
        RowsDev re = rd;
        re.n_rows = n_emit;
        re.seq_id = nullptr;
        re.n_live = nullptr;
        lm_head(h, kPrefillLane, re, h->h_emit, token_out, logits_out, st);
    }
    return check_launch(h, "cdb_prefill");
}

int cdb_kv_copy_on_exit(cdb_t* h, const cdb_rows_t* rows, const int32_t* exit_depth, void* stream) {
    if (!h) return CDB_ERR_ARG;
    if (h->cfg.kv_layout != CDB_KV_DEPTH_INDEXED) return fail(h, CDB_ERR_STATE, "copy-on-exit needs the depth-indexed layout");
    RowsDev rd;
    int rc = make_rows(h, rows, &rd, false);
    if (rc) return rc;
    if (rd.n_rows == 0) return CDB_OK;
    if (!exit_depth) return fail(h, CDB_ERR_ARG, "exit_depth is NULL");
    if (!h->pool.base) return fail(h, CDB_ERR_STATE, "no KV pool bound");
    launch_copy_on_exit(h, rd, exit_depth, (cudaStream_t)stream);
    return check_launch(h, "cdb_kv_copy_on_exit");
}

int cdb_paged_attention(cdb_t* h, const cdb_rows_t* rows, int32_t layer, const void* q, void* o, void* stream) {
    if (!h) return CDB_ERR_ARG;
    RowsDev rd;
    int rc = make_rows(h, rows, &rd, false);
    if (rc) return rc;
    if (rd.n_rows == 0) return CDB_OK;
    if (!q || !o) return fail(h, CDB_ERR_ARG, "q / o is NULL");
    if (layer < 0 || layer >= h->cfg.L_pre + h->cfg.L_core + h->cfg.L_coda) return fail(h, CDB_ERR_RANGE, "layer out of range");
    if (!h->pool.base) return fail(h, CDB_ERR_STATE, "no KV pool bound");
    if (!rows->kv_slot) rd.slot_override = 0;
    launch_attention_plan(h, 0, rd, (cudaStream_t)stream);
    launch_attention(h, 0, layer, rd, q, o, (cudaStream_t)stream);
    return check_launch(h, "cdb_paged_attention");
}

int cdb_linear(cdb_t* h, const void* x, const void* W, float* y, int32_t n, int32_t N, int32_t K, void* stream) {
    if (!h) return CDB_ERR_ARG;
    if (!x || !W || !y || n < 0 || N < 1 || K < 1) return fail(h, CDB_ERR_ARG, "bad argument");
    launch_linear(h, x, W, y, n, N, K, Epilogue::Store, (cudaStream_t)stream);
    return check_launch(h, "cdb_linear");
}

int cdb_poll_status(cdb_t* h, int32_t* status_host) {
    if (!h || !status_host) return CDB_ERR_ARG;
    cudaError_t e = cudaMemcpy(status_host, h->status, sizeof(int32_t), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && *status_host != 0) {                                                 // read and re-arm
        e = cudaMemset(h->status, 0, sizeof(int32_t));
        cudaMemset(h->grid_sync, 0, 3 * sizeof(unsigned int));        // a barrier a timed-out kernel left half way
    }
    return e == cudaSuccess ? CDB_OK : fail_cuda(h, e, "cdb_poll_status");
}

int cdb_debug_check_guards(cdb_t* h, int32_t* n_clobbered) {
    if (!h || !n_clobbered) return CDB_ERR_ARG;
    *n_clobbered = 0;
    unsigned char host[2 * kGuardBytes];
    for (int i = 0; i < h->n_allocs; ++i) {
        cudaError_t e = cudaMemcpy(host, h->alloc_base[i], kGuardBytes, cudaMemcpyDeviceToHost);
        if (e == cudaSuccess) e = cudaMemcpy(host + kGuardBytes, h->alloc_base[i] + kGuardBytes + h->alloc_bytes[i], kGuardBytes, cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) return fail_cuda(h, e, "cdb_debug_check_guards");
        bool bad = false;
        for (size_t k = 0; k < 2 * kGuardBytes; ++k) bad |= host[k] != (unsigned char)kGuardPattern;
        *n_clobbered += bad ? 1 : 0;
    }
    return CDB_OK;
}

int cdb_profile_begin(cdb_t* h, int32_t record_events) {
    if (!h) return CDB_ERR_ARG;
    if (record_events && !h->prof_ev) {
        h->prof_ev = new (std::nothrow) cudaEvent_t[2 * kProfCap]();
        h->prof_cls = new (std::nothrow) uint8_t[kProfCap]();
        if (!h->prof_ev || !h->prof_cls) return fail(h, CDB_ERR_NOMEM, "no memory for profiling events");
        for (int i = 0; i < 2 * kProfCap; ++i)
            if (cudaEventCreate(&h->prof_ev[i]) != cudaSuccess) return fail(h, CDB_ERR_CUDA, "cudaEventCreate failed");
    }
    h->launches = 0;
    h->prof_used = 0;
    h->prof_on = record_events ? 1 : 0;
    return CDB_OK;
}

int cdb_profile_read(cdb_t* h, cdb_profile_t* out) {
    if (!h || !out) return CDB_ERR_ARG;
    const cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return fail_cuda(h, e, "cdb_profile_read");
    memset(out, 0, sizeof(*out));
    out->launches = h->launches;
#ifdef CDB_TUNING
    if (const char* path = getenv("CDB_PROF_DUMP")) {           // tuning hook: (class, start, end) of every bracketed launch
        if (FILE* f = fopen(path, "w")) {
            for (int i = 0; i < h->prof_used; ++i) {
                float a = 0.f, b = 0.f;
                cudaEventElapsedTime(&a, h->prof_ev[0], h->prof_ev[2 * i]);
                cudaEventElapsedTime(&b, h->prof_ev[0], h->prof_ev[2 * i + 1]);
                fprintf(f, "%d,%.4f,%.4f\n", (int)h->prof_cls[i], a, b);
            }
            fclose(f);
        }
    }
#endif
    for (int i = 0; i < h->prof_used; ++i) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, h->prof_ev[2 * i], h->prof_ev[2 * i + 1]) != cudaSuccess) continue;
        const int c = h->prof_cls[i] < kProfClasses ? h->prof_cls[i] : 0;
        out->count[c] += 1;
        out->ms[c] += ms;
    }
    return CDB_OK;
}

}  // extern "C"
