/*
 * cdb.h - C ABI of the continuous-depth-batching (CDB) hot path for looped language models.
 *
 * One loop step of the shared recurrent core over a ragged batch whose rows are
 * (sequence, loop depth) items, the exit decision taken one step ahead, the survivor / exit
 * compaction, and the boundary stages (embedding / prelude, coda / LM head) around it.
 * Notation follows the paper: prelude P, recurrent core R, coda C (section 2, Eq. 1); r is
 * the 1-based loop step, R = r_max the maximum number of loops; d model width, H heads of size
 * Dh, F MLP width, V vocabulary.
 *
 * Conventions
 *  - Every function returns an int: CDB_OK (0) or a negative CDB_ERR_* code.  Nothing throws,
 *    aborts or traps.  cdb_last_error() gives a message for the last failure on that handle.
 *  - "device" pointers are CUDA device memory owned by the CALLER; they must stay valid until
 *    the stream work that uses them has finished.  "host" values are plain C values.
 *  - The library owns only what cdb_create() allocates (scratch buffers, per-sequence gate
 *    state, RoPE table, tile-major copies of bf16 projection weights) and frees it in
 *    cdb_destroy().  The weights are BORROWED: the pointers in cdb_weights_t must outlive the
 *    handle and their contents must not change after cdb_create().
 *  - All work is enqueued on the given stream (a cudaStream_t passed as void*) and no call
 *    synchronises, except cdb_create, cdb_destroy and cdb_poll_status.
 *  - Argument checks that can be made on the host happen before anything is launched.
 *  - Activations (hidden states h) are fp32 row-major [n_rows, d].  Weights, KV pages and the
 *    GEMM A-operands are of the configured dtype (fp32 or bf16); accumulation is fp32.
 *  - A row with seq_id < 0 is a pad: it computes nothing that is visible, writes no KV and
 *    appears in neither compaction list.
 *  - Except in cdb_prefill, a call holds at most one row per sequence (the exit-gate state is kept per
 *    sequence, and a row reads KV that only earlier calls wrote).
 *  - Scratch is per handle: two calls on the same handle must not overlap on the GPU, with two
 *    exceptions, each for rows of sequences the other calls do not touch: a boundary call
 *    (cdb_boundary_embed / _prelude / _coda_lmhead) may run on another stream while cdb_loop_step /
 *    cdb_compact / cdb_gather_rows run (the coda and prelude of exited tokens overlap the next loop
 *    step, Fig. 3 of the paper), and so may one cdb_prefill call on a third stream (prompts are
 *    processed beside the running decode batch).  The three groups have scratch of their own.
 */
#ifndef CDB_H
#define CDB_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct cdb cdb_t;

enum { CDB_OK = 0, CDB_ERR_ARG = -1, CDB_ERR_NOMEM = -2, CDB_ERR_CAPACITY = -3,
       CDB_ERR_RANGE = -4, CDB_ERR_STATE = -5, CDB_ERR_CUDA = -6 };
enum { CDB_FP32 = 0, CDB_BF16 = 1 };
/* KV layouts of section 4.2 / appendix C.1: slot used by loop step r is 0 (shared),
 * r-1 (depth-indexed; with copy-on-exit this is the last-exited cache) or min(r,2)-1. */
enum { CDB_KV_SHARED = 0, CDB_KV_DEPTH_INDEXED = 1, CDB_KV_FIRST_THEN_SHARED = 2 };
/* Exit signals of appendix C.2: a learned head (cumulative exit probability against a
 * threshold q) or the training-free convergence criterion (L2 distance of consecutive
 * recurrent states below eps). */
enum { CDB_GATE_NONE = 0, CDB_GATE_SIGMOID_CDF = 1, CDB_GATE_L2_CONVERGENCE = 2 };

typedef struct {
    int32_t V, d, H, Dh, F;            /* d == H * Dh; Dh in {64, 96, 128} */
    int32_t L_pre, L_core, L_coda;     /* prelude-core-coda layer split (section 2) */
    int32_t R;                         /* r_max */
    int32_t r_min;                     /* a gate-driven exit is honoured only at loop depth >= r_min */
    int32_t dtype;                     /* CDB_FP32 or CDB_BF16: weights, KV pages, GEMM operands */
    int32_t page_size;                 /* tokens per KV page; must be 16 */
    int32_t max_rows;                  /* capacity of one call (rows incl. pads) */
    int32_t max_seqs;                  /* seq_id range [0, max_seqs) */
    int32_t max_position;              /* positions [0, max_position) */
    int32_t kv_layout, n_slots;        /* n_slots: 1 shared, R depth-indexed, 2 first-then-shared */
    int32_t gate_kind;
    float   eps;                       /* RMSNorm epsilon */
    float   rope_theta;
    float   q_or_eps;                  /* threshold q (learned gate) or eps (convergence gate) */
    float   b_gate;                    /* bias of the learned gate */
    int32_t flags;                     /* CDB_FLAG_* */
} cdb_config_t;

enum { CDB_FLAG_SIMT_GEMM = 1,         /* run bf16 projections on the plain-FMA kernel (cross-check) */
       CDB_FLAG_TWO_STREAM = 2,        /* run a loop step of >= 64 rows as two half-batches on two streams (experimental; the second
                                         * half uses the boundary calls' scratch, so no boundary call may overlap such a step) */
       CDB_FLAG_UNFUSED_LAYER = 4,     /* one launch per projection, separate norm and SwiGLU kernels (cross-check) */
       CDB_FLAG_SIMT_PREFILL = 8,      /* prompt attention of bf16 pools on the plain-FMA kernel instead of the tensor cores (cross-check) */
       CDB_FLAG_FUSED_STAGES = 16,     /* everything of a layer after its attention as ONE cooperative launch with grid barriers between
                                         * the stages (experimental: measured slower than the separate, programmatically chained launches) */
       CDB_FLAG_WORKSPACE_PARTS = 32,  /* split-K parts of the decode projections through a workspace and a row-wise kernel instead of being
                                         * summed inside thread-block clusters (cross-check: the sums and their order are the same) */
       CDB_FLAG_CTA_PAIRS = 64,        /* projections on 128 rows and more run as CTA pairs (one 256-feature MMA over two SMs, each CTA loading
                                         * its own weights and half of the activation tile); same results bit for bit.  Without the flag pairs
                                         * are used from 512 rows on (prompt processing, very large batches), where they are faster */
       CDB_FLAG_SM_PARTITION = 128 };  /* a loop step of >= 64 rows runs as two half-batches with the SMs split between two green contexts:
                                         * the attention kernels of both halves back to back on one partition, everything else on the other
                                         * (experimental; same results bit for bit; uses the boundary calls' scratch like the two-stream flag;
                                         * without effect when the driver cannot partition the SMs) */

/* Row-major [out_features, in_features] ("K-major") weights of the configured dtype, layers
 * stacked in the order prelude, core, coda (L = L_pre + L_core + L_coda).  All device pointers. */
typedef struct {
    const void* W_qkv;    /* [L][3d][d]: rows [0,d) Q, [d,2d) K, [2d,3d) V, head-major inside */
    const void* W_o;      /* [L][d][d]  */
    const void* W_gate;   /* [L][F][d]  */
    const void* W_up;     /* [L][F][d]  */
    const void* W_down;   /* [L][d][F]  */
    const void* g_attn;   /* [L][d] RMSNorm gain before attention */
    const void* g_mlp;    /* [L][d] RMSNorm gain before the MLP */
    const void* embed;    /* [V][d] */
    const void* g_final;  /* [d] */
    const void* W_lm;     /* [V][d] */
    const float* w_gate;  /* [d] fp32, learned exit head (may be NULL when gate_kind != SIGMOID_CDF) */
} cdb_weights_t;

/* Row descriptor of one call: rows are (sequence, loop depth) items, i.e. the entries of the
 * recurrent queue of section 4.1.  Arrays are device int32 [n_rows]. */
typedef struct {
    int32_t        n_rows;           /* host: number of rows, pads included; <= max_rows */
    const int32_t* seq_id;           /* -1 = pad */
    const int32_t* loop_depth;       /* 1-based loop step this call executes for the row */
    const int32_t* position;         /* token position; the row attends to positions 0..position */
    const int32_t* kv_slot;          /* depth slot of the KV cache the row reads and writes */
    const int32_t* forced_exit;      /* replayed exit depth, 0 = decided by the gate; may be NULL */
    const int32_t* page_table;       /* device [max_seqs * n_slots][page_table_stride]: physical page
                                        of logical page j of (seq_id, kv_slot), row seq_id*n_slots+kv_slot */
    int32_t        page_table_stride; /* a row whose position needs logical page >= page_table_stride is skipped
                                        (no KV write, zero attention output) and reported as status 2 */
    const int32_t* n_rows_dev;       /* device int32 [1] or NULL.  When given, only the first *n_rows_dev rows are live:
                                        every row at an index >= *n_rows_dev is a pad whatever its seq_id says.  n_rows
                                        stays the host-side capacity of the call (launch shapes follow it), so one
                                        recorded launch sequence - a CUDA graph - serves every batch size up to n_rows
                                        (the static shapes of section 4.3) */
} cdb_rows_t;

/* Creates a handle for one model on the current CUDA device.  Allocates scratch for max_rows
 * rows and gate state for max_seqs sequences.  CDB_ERR_ARG on inconsistent dims, CDB_ERR_NOMEM /
 * CDB_ERR_CUDA when allocation fails.  Synchronises the device.  The handle belongs to that
 * device: every later call on it must be made with the same device current (a process may hold
 * handles on several devices). */
int cdb_create(const cdb_config_t* cfg, const cdb_weights_t* w, cdb_t** out);
int cdb_destroy(cdb_t* h);                       /* NULL is allowed */
const char* cdb_last_error(const cdb_t* h);      /* static / handle-owned string */

/* Binds the paged KV pool (section 4.2; paged attention).  Layout, dtype of the config:
 *   pool[layer][physical page][K=0 / V=1][head][token in page][Dh],  layer in [0, L)
 * Page ids are shared by all layers; which pages a (sequence, slot) owns is the host's policy,
 * expressed through cdb_rows_t.page_table.  CDB_ERR_ARG if `bytes` is too small. */
int cdb_kv_bind(cdb_t* h, void* pool_device, size_t bytes, int32_t n_phys_pages);

/* Optional, before cdb_kv_bind: a page space of their own for the prelude and coda layers.  Those layers cache one
 * k, v per token whatever the depth layout (appendix C.1, Table 1 counts L_pre + L_coda + slots * L_core vectors), so
 * with more than one depth slot they should not share page ids with the core layers, whose every slot owns pages.
 *   pool_device[layer in [0, L_pre + L_coda)][physical page][K / V][head][token in page][Dh]   (prelude layers first)
 *   page_table: device int32 [max_seqs][page_table_stride], row seq_id; caller-owned, must stay valid and may be
 *   updated in place between calls (like cdb_rows_t.page_table).
 * The pool given to cdb_kv_bind afterwards holds the L_core core layers alone, layer index 0 = first core layer.
 * CDB_ERR_STATE for a model without boundary layers or when cdb_kv_bind was already called. */
int cdb_kv_bind_boundary(cdb_t* h, void* pool_device, size_t bytes, int32_t n_phys_pages, const int32_t* page_table,
                         int32_t page_table_stride);

/* Changes the learned gate's bias and the exit threshold (host values). */
int cdb_set_gate(cdb_t* h, float b_gate, float q_or_eps);

/* Boundary, Eq. 1 "h0 = P(x_t)".  embed: h_out[i] = Embed(token_ids[i]) for fully looped models;
 * prelude: embedding followed by the L_pre prelude layers (own KV in slot 0's pages).  Both reset
 * the gate state of the rows' sequences (survival S = 1, no exit signal).
 * token_ids: device int32 [n_rows]; h_out: device fp32 [n_rows, d]. */
int cdb_boundary_embed(cdb_t* h, const int32_t* token_ids, const cdb_rows_t* rows, float* h_out, void* stream);
int cdb_boundary_prelude(cdb_t* h, const int32_t* token_ids, const cdb_rows_t* rows, float* h_out, void* stream);

/* One loop step of the recurrent core, Eq. 1 "h(r+1) = R(h(r), K(r)<t)", for all rows: per core
 * layer RMSNorm + QKV projection, RoPE, KV page write at (seq, layer, slot)[position], paged
 * causal attention over positions 0..position, output projection, RMSNorm + SwiGLU MLP; then the
 * exit signal of this step (section 4.3 lookahead gate; appendix C.2):
 *   learned gate:      lambda = sigmoid(w_gate . n(h) + b), S <- S (1 - lambda), value = 1 - S,
 *                      fire = value >= q         (n = RMSNorm without gain, fp32)
 *   convergence gate:  value = ||h_out - h_in||_2, fire = loop_depth >= 2 && value < eps
 * The signal is stored per sequence for cdb_compact and also written to the optional outputs.
 * h_inout: device fp32 [n_rows, d], updated in place.  gate_val_out: device fp32 [n_rows] or
 * NULL.  fire_out: device uint8 [n_rows] or NULL. */
int cdb_loop_step(cdb_t* h, const cdb_rows_t* rows, float* h_inout, float* gate_val_out,
                  uint8_t* fire_out, void* stream);

/* Exit flag and stable compaction (section 4.1, exit routing: a token either re-enters the
 * recurrent queue or leaves for the coda).  For every non-pad row
 *   exit = loop_depth >= R  ||  (forced_exit > 0 ? forced_exit == loop_depth
 *                                               : signal && loop_depth >= r_min)
 * where signal = fire_prev[row] if fire_prev != NULL, else the sequence's stored signal.  With the
 * lookahead gate the stored signal is the one of the previous step, so this may be called BEFORE
 * cdb_loop_step of the same rows (the host then prepares the next batch while the step runs);
 * called AFTER cdb_loop_step it applies the signal in the same step (no lookahead).
 * Outputs (device): survivor_idx / exit_idx int32 [n_rows], ascending row indices, first
 * counts[0] / counts[1] entries valid; counts int32 [2].  When h_src != NULL the rows are also
 * gathered: h_next[j] = h_src[survivor_idx[j]], h_exit[j] = h_src[exit_idx[j]] (either may be
 * NULL). */
int cdb_compact(cdb_t* h, const cdb_rows_t* rows, const uint8_t* fire_prev, const float* h_src,
                int32_t* survivor_idx, int32_t* exit_idx, int32_t* counts,
                float* h_next, float* h_exit, void* stream);

/* Row gather by a device index list: h_dst[j] = h_src[idx[j]] for j < *count_device (at most
 * max_count rows).  Used after cdb_loop_step when cdb_compact ran before it. */
int cdb_gather_rows(cdb_t* h, const float* h_src, const int32_t* idx, const int32_t* count_device,
                    int32_t max_count, float* h_dst, void* stream);

/* Boundary, Eq. 1 "p = softmax(C(h))" with greedy decoding (appendix C): the L_coda coda layers
 * (own KV), final RMSNorm, LM head, argmax with ties to the lowest id.
 * h_exit: device fp32 [n_rows, d] (clobbered when L_coda > 0); token_out: device int32 [n_rows];
 * logits_out: device fp32 [n_rows, V] or NULL. */
int cdb_boundary_coda_lmhead(cdb_t* h, const cdb_rows_t* rows, float* h_exit, int32_t* token_out,
                             float* logits_out, void* stream);

/* Prompt processing at full depth R with all positions of a prompt in lock-step (one row per
 * prompt position; under the shared layout a position at loop r attends to earlier positions'
 * loop-r states).  Rows of one sequence must all be in the same call.  Runs prelude, R loop
 * steps, coda on every row, and the LM head on the rows listed in emit_idx (device int32
 * [n_emit], typically each prompt's last position): token_out int32 [n_emit],
 * logits_out fp32 [n_emit, V] or NULL.  rows.loop_depth and rows.kv_slot are ignored. */
int cdb_prefill(cdb_t* h, const int32_t* token_ids, const cdb_rows_t* rows, const int32_t* emit_idx,
                int32_t n_emit, int32_t* token_out, float* logits_out, void* stream);

/* Last-exited cache (section 4.2): for each row, copy the k, v the row wrote at its position in
 * slot exit_depth-1 into slots exit_depth..R-1 of every core layer.  exit_depth: device int32
 * [n_rows].  Only for CDB_KV_DEPTH_INDEXED. */
int cdb_kv_copy_on_exit(cdb_t* h, const cdb_rows_t* rows, const int32_t* exit_depth, void* stream);

/* Stage-level entry points (same kernels as inside cdb_loop_step), for tests and microbenchmarks.
 * cdb_paged_attention: q device [n_rows, d] of the configured dtype (already rotated), output o
 * same shape and dtype; reads pool layer `layer`.
 * cdb_linear: y[n, N] = x[n, K] . W[N, K]^T, x and W of the configured dtype, y fp32. */
int cdb_paged_attention(cdb_t* h, const cdb_rows_t* rows, int32_t layer, const void* q, void* o, void* stream);
int cdb_linear(cdb_t* h, const void* x, const void* W, float* y, int32_t n, int32_t N, int32_t K, void* stream);

/* Allocation-free paged decode attention.  The paper has no counterpart: this exists for callers that
 * cannot obtain device memory at call time (a process that gave the whole GPU to its own pool allocator,
 * a plug-in whose host framework forbids cudaMalloc on its threads, a component with a memory budget
 * fixed at start-up).  Same computation and same kernels as cdb_paged_attention for the shared layout
 * (one KV slot), but without a handle: every input and output is passed in, and the scratch (split
 * partials, per-row split scan, work counter, status word) lives in an 8 MiB device array built into
 * the library, which each GPU that loads the library holds until the process exits.  It calls no
 * cudaMalloc / cudaFree and no allocating library routine.
 *   q, o: device [n_rows][H*Dh] of `dtype`;  pool: device [layers][n_phys_pages][2][H][16][Dh];
 *   seq_id, position: device int32 [n_rows] (seq_id < 0 = pad, output row zeroed);
 *   page_table: device int32 [max_seqs][page_table_stride];  max_context: host upper bound on
 *   position + 1, at most 16 * page_table_stride (CDB_ERR_ARG otherwise, so that no row can index past
 *   its table row).
 * Range errors inside the data are NOT reported by this entry point: it has no handle, so there is no
 * status word a caller could poll.  A row with position >= max_context or seq_id >= max_seqs is skipped and
 * its output row zeroed; a page id outside [0, n_phys_pages) is skipped, i.e. the row's output is the
 * attention over its remaining pages.  Callers that need the report use cdb_paged_attention.
 * Limit: 256 + 4*(n_rows+1) rounded up to 256 + n_rows*H*ceil(max_context/256)*(Dh+2)*4 bytes must fit in
 * 8 MiB (e.g. 64 rows x 16 heads x 2048 context at Dh 128); larger requests return CDB_ERR_CAPACITY and
 * print the sizes to stderr.  The first call on a device looks up the array's device address
 * (cudaGetSymbolAddress, with that device current) and should come before any stream capture.  All calls
 * on a device share the array, which keeps the last call's contents; each call re-zeroes what it needs
 * on its stream.  Calls whose GPU work overlaps (different streams) race on it. */
int cdb_paged_attention_static(const void* q, void* o, const void* pool, int32_t n_phys_pages, int32_t layer,
                               const int32_t* seq_id, const int32_t* position, const int32_t* page_table,
                               int32_t page_table_stride, int32_t n_rows, int32_t max_seqs, int32_t max_context,
                               int32_t H, int32_t Dh, int32_t dtype, void* stream);

/* Debug aid: every scratch buffer of the handle lies between two 256-byte guard words that no kernel of the
 * library may touch.  Synchronises the device's default stream order (plain cudaMemcpy) and counts the buffers
 * whose guards were overwritten (0 = clean). */
int cdb_debug_check_guards(cdb_t* h, int32_t* n_clobbered);

/* Synchronises the stream-less status word back to the host: 0 = clean, otherwise the first
 * out-of-range page id (1) / position (2) / sequence id (3) a kernel met since the last poll (the
 * access was skipped), or 4 when a bounded wait inside a tensor-core kernel ran out.  A non-zero
 * word is cleared by the call, so the next poll reports only what happened after this one. */
int cdb_poll_status(cdb_t* h, int32_t* status_host);

/* Instrumentation (not an operation of the paper): how many kernels the handle has launched, and
 * device time of the two heavy kernel classes measured by CUDA events recorded on the launching
 * stream.  cdb_profile_begin(h, 1) resets the counters and turns event recording on (0: counters
 * only); cdb_profile_read synchronises the device and fills `out`.  Index 0 = paged-attention
 * split kernel, 1 = projection kernels. */
typedef struct {
    uint64_t launches;          /* kernels launched since cdb_profile_begin */
    int32_t  count[2];          /* bracketed launches per class */
    float    ms[2];             /* summed device time per class, milliseconds */
} cdb_profile_t;
int cdb_profile_begin(cdb_t* h, int32_t record_events);
int cdb_profile_read(cdb_t* h, cdb_profile_t* out);

#ifdef __cplusplus
}
#endif
#endif /* CDB_H */
