"""ctypes binding of libcdb.so (the C ABI declared in include/cdb.h).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.  PyTorch
tensors provide device memory and streams.  Importing this module raises when the library has not
been built (`python -m paper_2608_09444_b200.build`); there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libcdb.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2608_09444_b200.build`")
lib = C.CDLL(_LIB_PATH)

OK = 0
ERR_ARG, ERR_NOMEM, ERR_CAPACITY, ERR_RANGE, ERR_STATE, ERR_CUDA = -1, -2, -3, -4, -5, -6
FP32, BF16 = 0, 1
KV_SHARED, KV_DEPTH_INDEXED, KV_FIRST_THEN_SHARED = 0, 1, 2
GATE_NONE, GATE_SIGMOID_CDF, GATE_L2_CONVERGENCE = 0, 1, 2
FLAG_SIMT_GEMM = 1
FLAG_TWO_STREAM = 2
FLAG_UNFUSED_LAYER = 4
FLAG_SIMT_PREFILL = 8
FLAG_FUSED_STAGES = 16
FLAG_WORKSPACE_PARTS = 32
FLAG_CTA_PAIRS = 64
FLAG_SM_PARTITION = 128

EXPORTS = ["cdb_create", "cdb_destroy", "cdb_last_error", "cdb_kv_bind", "cdb_set_gate", "cdb_boundary_embed",
           "cdb_boundary_prelude", "cdb_loop_step", "cdb_compact", "cdb_gather_rows", "cdb_boundary_coda_lmhead",
           "cdb_prefill", "cdb_kv_copy_on_exit", "cdb_paged_attention", "cdb_linear", "cdb_poll_status",
           "cdb_profile_begin", "cdb_profile_read", "cdb_paged_attention_static", "cdb_debug_check_guards",
           "cdb_kv_bind_boundary"]


class Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("V", "d", "H", "Dh", "F", "L_pre", "L_core", "L_coda", "R", "r_min", "dtype",
                                         "page_size", "max_rows", "max_seqs", "max_position", "kv_layout", "n_slots",
                                         "gate_kind")] + \
               [("eps", C.c_float), ("rope_theta", C.c_float), ("q_or_eps", C.c_float), ("b_gate", C.c_float),
                ("flags", C.c_int32)]


class Weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("W_qkv", "W_o", "W_gate", "W_up", "W_down", "g_attn", "g_mlp", "embed",
                                          "g_final", "W_lm", "w_gate")]


class RowsStruct(C.Structure):
    _fields_ = [("n_rows", C.c_int32), ("seq_id", C.c_void_p), ("loop_depth", C.c_void_p), ("position", C.c_void_p),
                ("kv_slot", C.c_void_p), ("forced_exit", C.c_void_p), ("page_table", C.c_void_p),
                ("page_table_stride", C.c_int32), ("n_rows_dev", C.c_void_p)]


class Profile(C.Structure):
    _fields_ = [("launches", C.c_uint64), ("count", C.c_int32 * 2), ("ms", C.c_float * 2)]


_P = C.c_void_p
lib.cdb_create.argtypes = [C.POINTER(Config), C.POINTER(Weights), C.POINTER(_P)]
lib.cdb_destroy.argtypes = [_P]
lib.cdb_last_error.argtypes = [_P]
lib.cdb_last_error.restype = C.c_char_p
lib.cdb_kv_bind.argtypes = [_P, _P, C.c_size_t, C.c_int32]
lib.cdb_kv_bind_boundary.argtypes = [_P, _P, C.c_size_t, C.c_int32, _P, C.c_int32]
lib.cdb_set_gate.argtypes = [_P, C.c_float, C.c_float]
lib.cdb_boundary_embed.argtypes = [_P, _P, C.POINTER(RowsStruct), _P, _P]
lib.cdb_boundary_prelude.argtypes = [_P, _P, C.POINTER(RowsStruct), _P, _P]
lib.cdb_loop_step.argtypes = [_P, C.POINTER(RowsStruct), _P, _P, _P, _P]
lib.cdb_compact.argtypes = [_P, C.POINTER(RowsStruct), _P, _P, _P, _P, _P, _P, _P, _P]
lib.cdb_gather_rows.argtypes = [_P, _P, _P, _P, C.c_int32, _P, _P]
lib.cdb_boundary_coda_lmhead.argtypes = [_P, C.POINTER(RowsStruct), _P, _P, _P, _P]
lib.cdb_prefill.argtypes = [_P, _P, C.POINTER(RowsStruct), _P, C.c_int32, _P, _P, _P]
lib.cdb_kv_copy_on_exit.argtypes = [_P, C.POINTER(RowsStruct), _P, _P]
lib.cdb_paged_attention.argtypes = [_P, C.POINTER(RowsStruct), C.c_int32, _P, _P, _P]
lib.cdb_linear.argtypes = [_P, _P, _P, _P, C.c_int32, C.c_int32, C.c_int32, _P]
lib.cdb_poll_status.argtypes = [_P, C.POINTER(C.c_int32)]
lib.cdb_profile_begin.argtypes = [_P, C.c_int32]
lib.cdb_profile_read.argtypes = [_P, C.POINTER(Profile)]
lib.cdb_paged_attention_static.argtypes = [_P, _P, _P, C.c_int32, C.c_int32, _P, _P, _P, C.c_int32, C.c_int32, C.c_int32,
                                           C.c_int32, C.c_int32, C.c_int32, C.c_int32, _P]
for _n in EXPORTS:
    if _n != "cdb_last_error":
        getattr(lib, _n).restype = C.c_int


class CdbError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"cdb error {code}: {msg}")
        self.code = code


def _ptr(t):
    """Device (or pinned host) address of a tensor, None -> NULL."""
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return t.data_ptr()


def _stream(stream):
    return (stream if stream is not None else torch.cuda.current_stream()).cuda_stream


def paged_attention_static(q, o, pool, layer, seq_id, position, page_table, max_seqs, max_context, stream=None) -> int:
    """cdb_paged_attention_static: paged decode attention that allocates nothing (no handle; scratch is an
    array built into the library).  Returns the C return code (OK, or ERR_CAPACITY when the request does
    not fit the built-in scratch)."""
    H, Dh = int(pool.shape[3]), int(pool.shape[5])
    dtype = FP32 if pool.dtype == torch.float32 else BF16
    return lib.cdb_paged_attention_static(_ptr(q), _ptr(o), _ptr(pool), int(pool.shape[1]), int(layer), _ptr(seq_id),
                                          _ptr(position), _ptr(page_table), int(page_table.shape[-1]),
                                          int(seq_id.shape[0]), int(max_seqs), int(max_context), H, Dh, dtype,
                                          _stream(stream))


class Rows:
    """Row descriptor of one call: device int32 tensors (see cdb_rows_t)."""

    def __init__(self, seq_id, position, page_table, loop_depth=None, kv_slot=None, forced_exit=None, n_rows=None,
                 n_rows_dev=None):
        self.seq_id, self.position, self.page_table = seq_id, position, page_table
        self.loop_depth, self.kv_slot, self.forced_exit = loop_depth, kv_slot, forced_exit
        self.n_rows_dev = n_rows_dev                    # device int32 [1]: live rows (the rest are pads), or None
        self.n_rows = int(seq_id.shape[0]) if n_rows is None else int(n_rows)
        for t in (seq_id, position, page_table, loop_depth, kv_slot, forced_exit, n_rows_dev):
            if t is not None and t.dtype != torch.int32:
                raise TypeError("row descriptor tensors must be int32")
        self.struct = RowsStruct(self.n_rows, _ptr(seq_id), _ptr(loop_depth), _ptr(position), _ptr(kv_slot),
                                 _ptr(forced_exit), _ptr(page_table), int(page_table.shape[-1]), _ptr(n_rows_dev))

    @property
    def ref(self):
        return C.byref(self.struct)


class Cdb:
    """Handle of one model (cdb_create / cdb_destroy) with one method per C entry point."""

    def __init__(self, dims, weights: dict, *, max_rows: int, max_seqs: int, max_position: int,
                 kv_layout: int = KV_SHARED, gate_kind: int = GATE_SIGMOID_CDF, q_or_eps: float = 0.5,
                 r_min: int = 1, flags: int = 0):
        n_slots = {KV_SHARED: 1, KV_DEPTH_INDEXED: dims.R, KV_FIRST_THEN_SHARED: 2}[kv_layout]
        b_gate = float(weights["b_gate"].reshape(-1)[0].item()) if "b_gate" in weights else 0.0
        self.cfg = Config(V=dims.V, d=dims.d, H=dims.H, Dh=dims.Dh, F=dims.F, L_pre=dims.L_pre, L_core=dims.L_core,
                          L_coda=dims.L_coda, R=dims.R, r_min=r_min, dtype=FP32 if dims.dtype == "fp32" else BF16,
                          page_size=dims.page_size, max_rows=max_rows, max_seqs=max_seqs, max_position=max_position,
                          kv_layout=kv_layout, n_slots=n_slots, gate_kind=gate_kind, eps=dims.eps,
                          rope_theta=dims.rope_theta, q_or_eps=q_or_eps, b_gate=b_gate, flags=flags)
        self.dims = dims
        self.n_slots = n_slots
        self._weights = weights                          # borrowed by the library: keep alive
        want = torch.float32 if dims.dtype == "fp32" else torch.bfloat16
        names = ("W_qkv", "W_o", "W_gate", "W_up", "W_down", "g_attn", "g_mlp", "embed", "g_final", "W_lm")
        for n in names:
            if weights[n].dtype != want or not weights[n].is_cuda:
                raise TypeError(f"weight {n} must be a CUDA tensor of dtype {want}")
        if weights["w_gate"].dtype != torch.float32:
            raise TypeError("w_gate must be fp32")
        self.w = Weights(**{n: _ptr(weights[n]) for n in names}, w_gate=_ptr(weights["w_gate"]))
        self.h = _P()
        rc = lib.cdb_create(C.byref(self.cfg), C.byref(self.w), C.byref(self.h))
        if rc != OK:
            self.h = _P()
            raise CdbError(rc, "cdb_create failed")
        self._pool = None

    def _check(self, rc):
        if rc != OK:
            raise CdbError(rc, lib.cdb_last_error(self.h).decode())

    def destroy(self):
        if self.h:
            lib.cdb_destroy(self.h)
            self.h = _P()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def kv_bind(self, pool: torch.Tensor):
        self._pool = pool
        self._check(lib.cdb_kv_bind(self.h, _ptr(pool), pool.numel() * pool.element_size(), int(pool.shape[1])))

    def kv_bind_boundary(self, pool: torch.Tensor, page_table: torch.Tensor):
        """Page space of the prelude and coda layers (call before kv_bind; the main pool then holds the core layers)."""
        self._pool_b, self._table_b = pool, page_table
        self._check(lib.cdb_kv_bind_boundary(self.h, _ptr(pool), pool.numel() * pool.element_size(), int(pool.shape[1]),
                                             _ptr(page_table), int(page_table.shape[-1])))

    def set_gate(self, b_gate: float, q_or_eps: float):
        self._check(lib.cdb_set_gate(self.h, b_gate, q_or_eps))

    def boundary_embed(self, token_ids, rows: Rows, h_out, stream=None):
        self._check(lib.cdb_boundary_embed(self.h, _ptr(token_ids), rows.ref, _ptr(h_out), _stream(stream)))

    def boundary_prelude(self, token_ids, rows: Rows, h_out, stream=None):
        self._check(lib.cdb_boundary_prelude(self.h, _ptr(token_ids), rows.ref, _ptr(h_out), _stream(stream)))

    def loop_step(self, rows: Rows, h_inout, gate_val_out=None, fire_out=None, stream=None):
        self._check(lib.cdb_loop_step(self.h, rows.ref, _ptr(h_inout), _ptr(gate_val_out), _ptr(fire_out), _stream(stream)))

    def compact(self, rows: Rows, survivor_idx, exit_idx, counts, fire_prev=None, h_src=None, h_next=None,
                h_exit=None, stream=None):
        self._check(lib.cdb_compact(self.h, rows.ref, _ptr(fire_prev), _ptr(h_src), _ptr(survivor_idx), _ptr(exit_idx),
                                    _ptr(counts), _ptr(h_next), _ptr(h_exit), _stream(stream)))

    def gather_rows(self, h_src, idx, count_device, max_count, h_dst, stream=None):
        self._check(lib.cdb_gather_rows(self.h, _ptr(h_src), _ptr(idx), _ptr(count_device), int(max_count), _ptr(h_dst),
                                        _stream(stream)))

    def boundary_coda_lmhead(self, rows: Rows, h_exit, token_out, logits_out=None, stream=None):
        self._check(lib.cdb_boundary_coda_lmhead(self.h, rows.ref, _ptr(h_exit), _ptr(token_out), _ptr(logits_out),
                                                 _stream(stream)))

    def prefill(self, token_ids, rows: Rows, emit_idx, token_out, logits_out=None, stream=None):
        n_emit = 0 if emit_idx is None else int(emit_idx.shape[0])
        self._check(lib.cdb_prefill(self.h, _ptr(token_ids), rows.ref, _ptr(emit_idx), n_emit, _ptr(token_out),
                                    _ptr(logits_out), _stream(stream)))

    def kv_copy_on_exit(self, rows: Rows, exit_depth, stream=None):
        self._check(lib.cdb_kv_copy_on_exit(self.h, rows.ref, _ptr(exit_depth), _stream(stream)))

    def paged_attention(self, rows: Rows, layer: int, q, o, stream=None):
        self._check(lib.cdb_paged_attention(self.h, rows.ref, int(layer), _ptr(q), _ptr(o), _stream(stream)))

    def linear(self, x, W, y, stream=None):
        n, K = x.shape
        N = W.shape[0]
        self._check(lib.cdb_linear(self.h, _ptr(x), _ptr(W), _ptr(y), n, N, K, _stream(stream)))

    def poll_status(self) -> int:
        v = C.c_int32(0)
        self._check(lib.cdb_poll_status(self.h, C.byref(v)))
        return v.value

    def check_guards(self) -> int:
        """Number of library scratch buffers whose guard words were overwritten (0 = clean)."""
        v = C.c_int32(0)
        self._check(lib.cdb_debug_check_guards(self.h, C.byref(v)))
        return v.value

    def profile_begin(self, record_events: bool = True):
        self._check(lib.cdb_profile_begin(self.h, 1 if record_events else 0))

    def profile_read(self) -> dict:
        p = Profile()
        self._check(lib.cdb_profile_read(self.h, C.byref(p)))
        return {"launches": int(p.launches), "attention": {"count": p.count[0], "ms": p.ms[0]},
                "linear": {"count": p.count[1], "ms": p.ms[1]}}
