"""ctypes binding of libs3scan.so: the same entry points as include/s3.h, taking torch tensors for
device memory and the current torch stream. Argument marshalling only: every step of the path runs
in the library's kernels. There is no fallback: a missing library or a failing call raises."""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libs3scan.so")

S3_OK = 0
S3_ERR_INVALID_ARG, S3_ERR_UNSUPPORTED, S3_ERR_CUDA, S3_ERR_NOMEM = -1, -2, -3, -4
S3_ERR_CAPACITY, S3_ERR_TIMEOUT, S3_ERR_STATE = -5, -6, -7
S3_BF16, S3_F32 = 0, 1
S3_SCORE_MINCOUNT, S3_SCORE_WEIGHTED = 0, 1
S3_WS_HEADER_BYTES = 64
S3_MAX_ENCODE_ITEMS = 8
S3_STATIC_SCRATCH_BYTES = 16 << 20
SCORE_LAUNCHES = 1            # kernels one span-scoring call enqueues

EXPORTS = [
    "s3_last_error", "s3_version", "s3_workspace_status",
    "s3_sae_prepared_bytes", "s3_sae_create", "s3_sae_destroy", "s3_sae_encode_workspace_bytes",
    "s3_sae_encode_topk", "s3_sae_set_schedule", "s3_sae_encode_topk_static",
    "s3_sae_encode_grouped_workspace_bytes", "s3_sae_encode_topk_grouped", "s3_sae_encode_ctas", "s3_encode_schedule_describe",
    "s3_sae_project_encode_workspace_bytes", "s3_sae_project_encode_topk",
    "s3_postings_workspace_bytes", "s3_postings_build", "s3_postings_build_batched",
    "s3_index_create", "s3_index_reserve", "s3_index_append", "s3_index_stream_wait", "s3_index_sync",
    "s3_index_stats", "s3_index_layer_postings", "s3_index_export_csr", "s3_index_destroy",
    "s3_score_workspace_bytes", "s3_coactivation_score_topspans",
    "s3_density_workspace_bytes", "s3_position_density_topcenters",
    "s3_fuse_workspace_bytes", "s3_fuse_index_sets",
    "s3_compact_bound", "s3_compact_workspace_bytes", "s3_compact_build", "s3_coactivation_score_topspans_compact",
    "s3_compact_save", "s3_compact_file_info", "s3_compact_load",
    "s3_sae_decode", "s3_head_aggregate_topk", "s3_compact_expand",
    "s3_sae_backward_workspace_bytes", "s3_sae_backward", "s3_adam_update", "s3_cast_f32_to_bf16", "s3_sae_preact",
]


class S3Error(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"s3 error {code}: {msg}")
        self.code = code


class PostingsItem(C.Structure):
    _fields_ = [("d_ids", C.c_void_p), ("d_vals", C.c_void_p), ("T", C.c_int32), ("k", C.c_int32),
                ("d_sae", C.c_int32), ("reserved", C.c_int32), ("pos_base", C.c_int64),
                ("d_row_ptr", C.c_void_p), ("d_pos", C.c_void_p), ("d_pval", C.c_void_p)]


class EncodeItem(C.Structure):
    _fields_ = [("sae", C.c_void_p), ("d_x", C.c_void_p), ("ldx", C.c_int64), ("T", C.c_int32), ("k", C.c_int32),
                ("d_ids", C.c_void_p), ("d_vals", C.c_void_p)]


class CsrView(C.Structure):
    _fields_ = [("d_row_ptr", C.c_void_p), ("d_pos", C.c_void_p)]


class CompactView(C.Structure):
    _fields_ = [("d_row_ptr", C.c_void_p), ("d_blk_ptr", C.c_void_p), ("d_blk_first", C.c_void_p),
                ("d_blk_desc", C.c_void_p), ("d_payload", C.c_void_p)]


class CompactHostLayer(C.Structure):
    _fields_ = [("h_row_ptr", C.c_void_p), ("h_blk_ptr", C.c_void_p), ("h_blk_first", C.c_void_p),
                ("h_blk_desc", C.c_void_p), ("h_payload", C.c_void_p), ("n_blocks", C.c_uint64), ("n_words", C.c_uint64)]


class AdamParams(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float), ("step", C.c_int32),
                ("reserved", C.c_int32)]


class ScoreParams(C.Structure):
    _fields_ = [("width", C.c_int32), ("stride", C.c_int32), ("mode", C.c_int32), ("s", C.c_int32),
                ("alpha", C.c_float), ("beta", C.c_float), ("stop_freq", C.c_int64)]


class DensityParams(C.Structure):
    _fields_ = [("conv_kernel", C.c_int32), ("nms_radius", C.c_int32), ("n_centers", C.c_int32), ("reserved", C.c_int32),
                ("stop_freq", C.c_int64)]


class IndexStats(C.Structure):
    _fields_ = [("n_chunks", C.c_int64), ("n_postings", C.c_int64), ("host_bytes", C.c_int64),
                ("host_bytes_reserved", C.c_int64), ("max_list_len", C.c_int64), ("n_positions", C.c_int64)]


_lib = None


def lib():
    """Loads the CUDA library; raises if it has not been built (there is no other implementation)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2601_17702_b200.build` "
                              "(there is no CPU or PyTorch fallback)")
        L = C.CDLL(LIB_PATH)
        L.s3_last_error.restype = C.c_char_p
        for name in ("s3_sae_prepared_bytes", "s3_sae_encode_workspace_bytes", "s3_postings_workspace_bytes",
                     "s3_score_workspace_bytes", "s3_density_workspace_bytes", "s3_fuse_workspace_bytes",
                     "s3_compact_workspace_bytes", "s3_sae_backward_workspace_bytes", "s3_sae_encode_grouped_workspace_bytes",
                     "s3_sae_project_encode_workspace_bytes"):
            getattr(L, name).restype = C.c_size_t
        L.s3_sae_prepared_bytes.argtypes = [C.c_int, C.c_int, C.c_int]
        L.s3_sae_create.argtypes = [C.POINTER(C.c_void_p), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                                    C.c_int, C.c_void_p, C.c_size_t, C.c_void_p]
        L.s3_sae_destroy.argtypes = [C.c_void_p]
        L.s3_sae_set_schedule.argtypes = [C.c_void_p, C.c_int, C.c_int]
        L.s3_sae_encode_workspace_bytes.argtypes = [C.c_void_p, C.c_int, C.c_int]
        L.s3_sae_encode_topk.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.c_size_t, C.c_void_p]
        L.s3_sae_encode_topk_static.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_int, C.c_void_p,
                                                C.c_void_p, C.c_void_p, C.c_void_p]
        L.s3_sae_encode_grouped_workspace_bytes.argtypes = [C.POINTER(EncodeItem), C.c_int]
        L.s3_sae_encode_topk_grouped.argtypes = [C.POINTER(EncodeItem), C.c_int, C.c_int, C.c_void_p, C.c_size_t, C.c_void_p]
        L.s3_sae_encode_ctas.argtypes = [C.c_void_p, C.c_int]
        L.s3_encode_schedule_describe.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_int,
                                                  C.c_void_p]
        L.s3_sae_project_encode_workspace_bytes.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int]
        L.s3_sae_project_encode_topk.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_void_p,
                                                 C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.s3_workspace_status.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_uint32)]
        L.s3_postings_workspace_bytes.argtypes = [C.c_int, C.c_int, C.c_int]
        L.s3_postings_build.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int64, C.c_void_p,
                                        C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.s3_postings_build_batched.argtypes = [C.POINTER(PostingsItem), C.c_int, C.c_void_p, C.c_size_t, C.c_void_p]
        L.s3_index_create.argtypes = [C.POINTER(C.c_void_p), C.c_int, C.c_int, C.c_size_t]
        L.s3_index_reserve.argtypes = [C.c_void_p, C.c_size_t]
        L.s3_index_append.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                                      C.c_int64, C.c_void_p, C.POINTER(C.c_void_p)]
        L.s3_index_stream_wait.argtypes = [C.c_void_p, C.c_void_p]
        L.s3_index_sync.argtypes = [C.c_void_p]
        L.s3_index_stats.argtypes = [C.c_void_p, C.POINTER(IndexStats)]
        L.s3_index_layer_postings.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_uint64)]
        L.s3_index_export_csr.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
        L.s3_index_destroy.argtypes = [C.c_void_p]
        L.s3_score_workspace_bytes.argtypes = [C.c_int] * 6
        L.s3_coactivation_score_topspans.argtypes = [C.POINTER(CsrView), C.c_int, C.c_int, C.c_int64, C.c_void_p,
                                                     C.c_void_p, C.c_int, C.c_int, C.c_int, C.POINTER(ScoreParams),
                                                     C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p,
                                                     C.c_void_p, C.c_size_t, C.c_void_p]
        L.s3_density_workspace_bytes.argtypes = [C.c_int, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_int]
        L.s3_position_density_topcenters.argtypes = [C.POINTER(CsrView), C.c_int, C.c_int, C.c_int64, C.c_void_p, C.c_void_p,
                                                     C.c_int, C.c_int, C.c_int, C.POINTER(DensityParams), C.c_void_p,
                                                     C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.s3_fuse_workspace_bytes.argtypes = [C.c_int, C.c_int64]
        L.s3_fuse_index_sets.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int64,
                                         C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.s3_compact_bound.argtypes = [C.c_uint64, C.c_int, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
        L.s3_compact_workspace_bytes.argtypes = [C.c_uint64, C.c_int]
        L.s3_compact_build.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_int, C.c_int64, C.c_void_p, C.c_void_p,
                                       C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p, C.c_uint64, C.c_void_p, C.c_void_p,
                                       C.c_size_t, C.c_void_p]
        L.s3_coactivation_score_topspans_compact.argtypes = [C.POINTER(CompactView)] + L.s3_coactivation_score_topspans.argtypes[1:]
        L.s3_compact_save.argtypes = [C.c_char_p, C.c_int, C.c_int, C.POINTER(CompactHostLayer)]
        L.s3_compact_file_info.argtypes = [C.c_char_p, C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_uint64),
                                           C.POINTER(C.c_uint64), C.c_int]
        L.s3_compact_load.argtypes = [C.c_char_p, C.c_int, C.c_int, C.POINTER(CompactHostLayer)]
        L.s3_sae_decode.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                                    C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]
        L.s3_head_aggregate_topk.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p,
                                             C.c_void_p, C.c_void_p]
        L.s3_compact_expand.argtypes = [C.POINTER(CompactView), C.c_int, C.c_void_p, C.c_uint64, C.c_void_p, C.c_size_t, C.c_void_p]
        L.s3_sae_backward_workspace_bytes.argtypes = [C.c_int]
        L.s3_cast_f32_to_bf16.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.s3_sae_backward.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_int,
                                      C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                      C.c_void_p, C.c_size_t, C.c_void_p]
        L.s3_adam_update.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.POINTER(AdamParams), C.c_void_p]
        L.s3_sae_preact.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_void_p, C.c_int64, C.c_int, C.c_void_p, C.c_size_t,
                                    C.c_void_p]
        _lib = L
    return _lib


def _check(code: int):
    if code != S3_OK:
        raise S3Error(code, lib().s3_last_error().decode())


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def s3_last_error() -> str:
    return lib().s3_last_error().decode()


def s3_version() -> int:
    return int(lib().s3_version())


def new_workspace(n_bytes: int, device="cuda") -> torch.Tensor:
    """A zeroed device workspace (the status block at its start must start at zero)."""
    return torch.zeros(max(int(n_bytes), S3_WS_HEADER_BYTES), dtype=torch.uint8, device=device)


def s3_workspace_status(ws: torch.Tensor, stream=None) -> int:
    code = C.c_uint32(0)
    _check(lib().s3_workspace_status(_ptr(ws), _stream(stream), C.byref(code)))
    return int(code.value)


class Sae:
    """Handle of one SAE encoder (s3_sae_create / s3_sae_destroy). Keeps the tensors it points to alive."""

    def __init__(self, W_enc: torch.Tensor, b_enc: torch.Tensor, b_dec: torch.Tensor, stream=None):
        assert W_enc.is_cuda and W_enc.is_contiguous() and W_enc.dim() == 2
        self.dtype = {torch.bfloat16: S3_BF16, torch.float32: S3_F32}[W_enc.dtype]
        self.d_in, self.d_sae = W_enc.shape
        self.W_enc, self.b_enc, self.b_dec = W_enc, b_enc.contiguous(), b_dec.contiguous()
        assert self.b_enc.dtype == torch.float32 and self.b_dec.dtype == torch.float32
        n = lib().s3_sae_prepared_bytes(self.d_in, self.d_sae, self.dtype)
        self.prepared = torch.empty(n, dtype=torch.uint8, device=W_enc.device)
        h = C.c_void_p()
        _check(lib().s3_sae_create(C.byref(h), _ptr(W_enc), _ptr(self.b_enc), _ptr(self.b_dec), self.d_in, self.d_sae,
                                   self.dtype, _ptr(self.prepared), n, _stream(stream)))
        self.handle = h

    def set_schedule(self, n_slices: int = 0, max_ctas: int = 0):
        _check(lib().s3_sae_set_schedule(self.handle, n_slices, max_ctas))

    def encode_workspace_bytes(self, T_max: int, k: int) -> int:
        return int(lib().s3_sae_encode_workspace_bytes(self.handle, T_max, k))

    def close(self):
        if getattr(self, "handle", None):
            lib().s3_sae_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def s3_sae_encode_topk(sae: Sae, x: torch.Tensor, k: int, ids: torch.Tensor, vals: torch.Tensor, ws: torch.Tensor,
                       stream=None):
    """ids int32 [T,k], vals fp32 [T,k] are written on the stream; x is [T, d_in] with stride(1) == 1."""
    assert x.is_cuda and x.dim() == 2 and x.stride(1) == 1 and x.shape[1] == sae.d_in
    T = x.shape[0]
    assert ids.dtype == torch.int32 and vals.dtype == torch.float32 and ids.is_contiguous() and vals.is_contiguous()
    assert tuple(ids.shape) == (T, k) and tuple(vals.shape) == (T, k)
    _check(lib().s3_sae_encode_topk(sae.handle, _ptr(x), x.stride(0) if T > 1 else max(x.stride(0), sae.d_in), T, k,
                                    _ptr(ids), _ptr(vals), _ptr(ws), ws.numel(), _stream(stream)))


def make_encode_item(sae: Sae, x: torch.Tensor, k: int, ids: torch.Tensor, vals: torch.Tensor) -> EncodeItem:
    assert x.is_cuda and x.dim() == 2 and x.stride(1) == 1 and x.shape[1] == sae.d_in
    T = x.shape[0]
    assert ids.dtype == torch.int32 and vals.dtype == torch.float32 and ids.is_contiguous() and vals.is_contiguous()
    assert tuple(ids.shape) == (T, k) and tuple(vals.shape) == (T, k)
    return EncodeItem(sae.handle, x.data_ptr(), x.stride(0) if T > 1 else max(x.stride(0), sae.d_in), T, k, ids.data_ptr(),
                      vals.data_ptr())


def s3_sae_encode_grouped_workspace_bytes(items: list[EncodeItem]) -> int:
    arr = (EncodeItem * max(len(items), 1))(*items)
    return int(lib().s3_sae_encode_grouped_workspace_bytes(arr, len(items)))


def s3_sae_encode_topk_grouped(items: list[EncodeItem], ws: torch.Tensor, max_ctas: int = 0, stream=None):
    """Several encoder calls (make_encode_item) as one persistent launch plus one selection launch; max_ctas > 0
    limits the launch to that many thread blocks."""
    arr = (EncodeItem * max(len(items), 1))(*items)
    _check(lib().s3_sae_encode_topk_grouped(arr, len(items), max_ctas, _ptr(ws), ws.numel(), _stream(stream)))


def s3_sae_encode_ctas(sae: Sae, T: int) -> int:
    """Thread blocks an s3_sae_encode_topk launch over T tokens occupies."""
    return int(lib().s3_sae_encode_ctas(sae.handle, T))


def s3_encode_schedule_describe(items, n_pairs: int, max_units: int = 4096):
    """items: (T, d_in, d_sae, k) per encoder call. Returns (units int32 [n, 6] = pair, item, row tile, first column tile, one
    past the last, slot; or None when the launch deals uniform slices without a table, slots per row of every item)."""
    import numpy as np
    a = np.ascontiguousarray(np.asarray(items, dtype=np.int32).reshape(-1, 4).T)
    n = a.shape[1]
    units = np.zeros((max_units, 6), dtype=np.int32)
    slots = np.zeros(n, dtype=np.int32)
    rc = int(lib().s3_encode_schedule_describe(a[0].ctypes.data, a[1].ctypes.data, a[2].ctypes.data, a[3].ctypes.data, n, n_pairs,
                                               units.ctypes.data, max_units, slots.ctypes.data))
    if rc == -2:
        raise ValueError("invalid schedule query")
    if rc > max_units:
        raise ValueError(f"{rc} units, room for {max_units}")
    return (units[:rc] if rc >= 0 else None), slots


def s3_sae_project_encode_workspace_bytes(sae: Sae, T_max: int, n_heads: int, k: int) -> int:
    return int(lib().s3_sae_project_encode_workspace_bytes(sae.handle, T_max, n_heads, k))


def s3_sae_project_encode_topk(proj: Sae, sae: Sae, h: torch.Tensor, n_heads: int, k: int, ids: torch.Tensor, vals: torch.Tensor,
                               ws: torch.Tensor, stream=None):
    """h [T, d_model] bf16 -> per (token, head) Top-k codes ids / vals [T, n_heads, k] of x = h W_proj + b read head by head
    through the 128-wide encoder `sae`; `proj` is a Sae handle over W_proj [d_model, n_heads * 128] (b_dec = 0)."""
    assert h.is_cuda and h.dim() == 2 and h.stride(1) == 1 and h.shape[1] == proj.d_in
    T = h.shape[0]
    assert ids.dtype == torch.int32 and vals.dtype == torch.float32 and ids.is_contiguous() and vals.is_contiguous()
    assert tuple(ids.shape) == (T, n_heads, k) and tuple(vals.shape) == (T, n_heads, k)
    _check(lib().s3_sae_project_encode_topk(proj.handle, sae.handle, _ptr(h), h.stride(0) if T > 1 else max(h.stride(0), proj.d_in),
                                            T, n_heads, k, _ptr(ids), _ptr(vals), _ptr(ws), ws.numel(), _stream(stream)))


def s3_sae_encode_topk_static(sae: Sae, x: torch.Tensor, k: int, ids: torch.Tensor, vals: torch.Tensor,
                              status_out: torch.Tensor | None = None, stream=None):
    """The encode for callers that cannot allocate: same outputs as s3_sae_encode_topk, but the scratch
    is the fixed array inside the library (S3_STATIC_SCRATCH_BYTES, one per device, shared by all calls),
    so no workspace is passed. status_out: optional int32/uint32 device tensor (1 element) that receives
    the call's device status word. Raises S3Error(S3_ERR_CAPACITY) when T*k is too large for the array."""
    assert x.is_cuda and x.dim() == 2 and x.stride(1) == 1 and x.shape[1] == sae.d_in
    T = x.shape[0]
    assert ids.dtype == torch.int32 and vals.dtype == torch.float32 and ids.is_contiguous() and vals.is_contiguous()
    assert tuple(ids.shape) == (T, k) and tuple(vals.shape) == (T, k)
    assert status_out is None or (status_out.is_cuda and status_out.element_size() == 4 and status_out.numel() >= 1)
    _check(lib().s3_sae_encode_topk_static(sae.handle, _ptr(x), x.stride(0) if T > 1 else max(x.stride(0), sae.d_in),
                                           T, k, _ptr(ids), _ptr(vals), _ptr(status_out), _stream(stream)))


def s3_postings_workspace_bytes(T_max: int, k: int, d_sae: int) -> int:
    return int(lib().s3_postings_workspace_bytes(T_max, k, d_sae))


def s3_postings_build(ids: torch.Tensor, d_sae: int, pos_base: int, row_ptr: torch.Tensor, pos: torch.Tensor,
                      ws: torch.Tensor, vals: torch.Tensor | None = None, pval: torch.Tensor | None = None, stream=None):
    T, k = ids.shape
    assert ids.dtype == torch.int32 and ids.is_contiguous() and row_ptr.dtype in (torch.uint32, torch.int32)
    assert row_ptr.numel() == d_sae + 1 and pos.dtype == torch.int32 and pos.numel() >= T * k
    _check(lib().s3_postings_build(_ptr(ids), _ptr(vals), T, k, d_sae, pos_base, _ptr(row_ptr), _ptr(pos), _ptr(pval),
                                   _ptr(ws), ws.numel(), _stream(stream)))


def make_postings_item(ids, d_sae, pos_base, row_ptr, pos, vals=None, pval=None) -> PostingsItem:
    T, k = ids.shape
    p = lambda t: None if t is None else t.data_ptr()
    return PostingsItem(p(ids), p(vals), T, k, d_sae, 0, pos_base, p(row_ptr), p(pos), p(pval))


def s3_postings_build_batched(items: list[PostingsItem], ws: torch.Tensor, stream=None):
    arr = (PostingsItem * max(len(items), 1))(*items)
    _check(lib().s3_postings_build_batched(arr, len(items), _ptr(ws), ws.numel(), _stream(stream)))


class Index:
    """Host-resident inverted index (s3_index_*)."""

    def __init__(self, n_layers: int, d_sae: int, pinned_slab_bytes: int = 64 << 20):
        h = C.c_void_p()
        _check(lib().s3_index_create(C.byref(h), n_layers, d_sae, pinned_slab_bytes))
        self.handle, self.n_layers, self.d_sae = h, n_layers, d_sae

    def reserve(self, n_bytes: int):
        _check(lib().s3_index_reserve(self.handle, n_bytes))

    def append(self, layer: int, row_ptr: torch.Tensor, pos: torch.Tensor, T: int, k: int, pos_base: int,
               pval: torch.Tensor | None = None, stream=None):
        _check(lib().s3_index_append(self.handle, layer, _ptr(row_ptr), _ptr(pos), _ptr(pval), T, k, pos_base,
                                     _stream(stream), None))

    def stream_wait(self, stream=None):
        _check(lib().s3_index_stream_wait(self.handle, _stream(stream)))

    def sync(self):
        _check(lib().s3_index_sync(self.handle))

    def stats(self) -> dict:
        st = IndexStats()
        _check(lib().s3_index_stats(self.handle, C.byref(st)))
        return {f: int(getattr(st, f)) for f, _ in IndexStats._fields_}

    def layer_postings(self, layer: int) -> int:
        n = C.c_uint64(0)
        _check(lib().s3_index_layer_postings(self.handle, layer, C.byref(n)))
        return int(n.value)

    def export_csr(self, layer: int, with_values: bool = False):
        """(row_ptr int64-viewed uint64 [d_sae+1], pos int32 [P], pval fp32 [P] or None) as host tensors."""
        n = self.layer_postings(layer)
        row_ptr = torch.empty(self.d_sae + 1, dtype=torch.int64)
        pos = torch.empty(max(n, 1), dtype=torch.int32)
        pval = torch.empty(max(n, 1), dtype=torch.float32) if with_values else None
        _check(lib().s3_index_export_csr(self.handle, layer, _ptr(row_ptr), _ptr(pos), _ptr(pval)))
        return row_ptr, pos[:n], (None if pval is None else pval[:n])

    def close(self):
        if getattr(self, "handle", None):
            lib().s3_index_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def s3_score_workspace_bytes(Q, nq, k, n_layers, n_spans, s) -> int:
    return int(lib().s3_score_workspace_bytes(Q, nq, k, n_layers, n_spans, s))


def s3_coactivation_score_topspans(layers, d_sae: int, L: int, q_ids: torch.Tensor, q_vals: torch.Tensor,
                                   width: int, stride: int, s: int, alpha: float, beta: float, ws: torch.Tensor,
                                   bm25: torch.Tensor | None = None, mode: int = S3_SCORE_MINCOUNT, stop_freq: int = 0,
                                   top_idx: torch.Tensor | None = None, top_score: torch.Tensor | None = None,
                                   all_scores: torch.Tensor | None = None, stream=None):
    """layers: list of (row_ptr int64 [d_sae+1], pos int32) device tensors, one merged CSR per layer.
    q_ids/q_vals: [n_layers, Q, nq, k]. Returns (top_idx [Q,s] int32, top_score [Q,s] fp32)."""
    n_layers, Q, nq, k = q_ids.shape
    assert len(layers) == n_layers and q_ids.dtype == torch.int32 and q_vals.dtype == torch.float32
    assert q_ids.is_contiguous() and q_vals.is_contiguous()
    views = (CsrView * n_layers)(*[CsrView(rp.data_ptr(), ps.data_ptr()) for rp, ps in layers])
    for rp, ps in layers:
        assert rp.dtype == torch.int64 and ps.dtype == torch.int32 and rp.numel() == d_sae + 1
    dev = q_ids.device
    if top_idx is None:
        top_idx = torch.empty((Q, s), dtype=torch.int32, device=dev)
    if top_score is None:
        top_score = torch.empty((Q, s), dtype=torch.float32, device=dev)
    params = ScoreParams(width, stride, mode, s, alpha, beta, stop_freq)
    ld = 0 if bm25 is None else bm25.stride(0)
    _check(lib().s3_coactivation_score_topspans(views, n_layers, d_sae, L, _ptr(q_ids), _ptr(q_vals), Q, nq, k,
                                                C.byref(params), _ptr(bm25), ld, _ptr(top_idx), _ptr(top_score),
                                                _ptr(all_scores), _ptr(ws), ws.numel(), _stream(stream)))
    return top_idx, top_score


def s3_density_workspace_bytes(Q: int, L: int, n_layers: int, d_sae: int, nq: int, k: int) -> int:
    return int(lib().s3_density_workspace_bytes(Q, L, n_layers, d_sae, nq, k))


def s3_position_density_topcenters(layers, d_sae: int, L: int, q_ids: torch.Tensor, q_vals: torch.Tensor, conv_kernel: int,
                                   nms_radius: int, n_centers: int, ws: torch.Tensor, stop_freq: int = 0,
                                   S_out: torch.Tensor | None = None, density_out: torch.Tensor | None = None, stream=None):
    """layers: list of (row_ptr int64 [d_sae+1], pos int32) device tensors; q_ids/q_vals [n_layers, Q, nq, k].
    Returns (centers int32 [Q, n_centers], center_density fp32 [Q, n_centers]); S_out / density_out (optional,
    fp32 [Q, L]) receive the per-position relevance and its smoothed density."""
    n_layers, Q, nq, k = q_ids.shape
    assert len(layers) == n_layers and q_ids.dtype == torch.int32 and q_vals.dtype == torch.float32
    assert q_ids.is_contiguous() and q_vals.is_contiguous()
    views = (CsrView * n_layers)(*[CsrView(rp.data_ptr(), ps.data_ptr()) for rp, ps in layers])
    for rp, ps in layers:
        assert rp.dtype == torch.int64 and ps.dtype == torch.int32 and rp.numel() == d_sae + 1
    dev = q_ids.device
    centers = torch.empty((Q, n_centers), dtype=torch.int32, device=dev)
    dens = torch.empty((Q, n_centers), dtype=torch.float32, device=dev)
    params = DensityParams(conv_kernel, nms_radius, n_centers, 0, stop_freq)
    _check(lib().s3_position_density_topcenters(views, n_layers, d_sae, L, _ptr(q_ids), _ptr(q_vals), Q, nq, k,
                                                C.byref(params), _ptr(centers), _ptr(dens), _ptr(S_out), _ptr(density_out),
                                                _ptr(ws), ws.numel(), _stream(stream)))
    return centers, dens


def s3_fuse_workspace_bytes(Q: int, L: int) -> int:
    return int(lib().s3_fuse_workspace_bytes(Q, L))


def s3_fuse_index_sets(centers: torch.Tensor, span_width: int, lexical: torch.Tensor | None, lead: int, tail: int, L: int,
                       cap: int, ws: torch.Tensor, stream=None):
    """centers int32 [Q, N] (-1 = none), lexical int32 [Q, n_lex] or None. Returns (idx int32 [Q, cap] ascending,
    -1 padded; count int32 [Q])."""
    assert centers.dtype == torch.int32 and centers.is_contiguous() and centers.dim() == 2
    Q, N = centers.shape
    n_lex = 0
    if lexical is not None:
        assert lexical.dtype == torch.int32 and lexical.is_contiguous() and lexical.shape[0] == Q
        n_lex = lexical.shape[1]
    idx = torch.empty((Q, cap), dtype=torch.int32, device=centers.device)
    count = torch.empty((Q,), dtype=torch.int32, device=centers.device)
    _check(lib().s3_fuse_index_sets(_ptr(centers), Q, N, span_width, _ptr(lexical), n_lex, lead, tail, L, _ptr(idx), cap,
                                    _ptr(count), _ptr(ws), ws.numel(), _stream(stream)))
    return idx, count


# ------------------------------------------------------------------------------------------------ compact index
COMPACT_FIELDS = ("row_ptr", "blk_ptr", "blk_first", "blk_desc", "payload")
_COMPACT_DTYPES = dict(row_ptr=torch.int64, blk_ptr=torch.int32, blk_first=torch.int32, blk_desc=torch.int64,
                       payload=torch.int32)


class CompactLayer:
    """The five arrays of one layer's compact index as tensors (unsigned contents in same-width signed dtypes):
    row_ptr int64 [d_sae+1], blk_ptr int32 [d_sae+1], blk_first int32 [n_blocks], blk_desc int64 [n_blocks],
    payload int32 [n_words]."""

    def __init__(self, row_ptr, blk_ptr, blk_first, blk_desc, payload):
        self.row_ptr, self.blk_ptr, self.blk_first, self.blk_desc, self.payload = row_ptr, blk_ptr, blk_first, blk_desc, payload
        for name in COMPACT_FIELDS:
            t = getattr(self, name)
            assert t.dtype == _COMPACT_DTYPES[name] and t.is_contiguous(), name

    def view(self) -> CompactView:
        return CompactView(*[getattr(self, n).data_ptr() for n in COMPACT_FIELDS])

    def host_layer(self) -> CompactHostLayer:
        assert self.row_ptr.device.type == "cpu"
        return CompactHostLayer(*[getattr(self, n).data_ptr() for n in COMPACT_FIELDS], self.blk_first.numel(),
                                self.payload.numel())

    def to(self, device):
        return CompactLayer(*[getattr(self, n).to(device) for n in COMPACT_FIELDS])

    def nbytes(self) -> int:
        return sum(getattr(self, n).numel() * getattr(self, n).element_size() for n in COMPACT_FIELDS)


def s3_compact_bound(n_postings: int, d_sae: int):
    b, w = C.c_uint64(), C.c_uint64()
    _check(lib().s3_compact_bound(n_postings, d_sae, C.byref(b), C.byref(w)))
    return b.value, w.value


def s3_compact_workspace_bytes(n_postings: int, d_sae: int) -> int:
    return int(lib().s3_compact_workspace_bytes(n_postings, d_sae))


def s3_compact_build(row_ptr: torch.Tensor, pos: torch.Tensor, d_sae: int, stop_freq: int = 0, ws: torch.Tensor | None = None,
                     cap_blocks: int | None = None, cap_words: int | None = None, stream=None) -> CompactLayer:
    """row_ptr int64 [d_sae+1], pos int32: one layer's merged CSR on the device. Allocates the outputs at the
    bound (or the given capacities), runs the build, waits for it and returns the arrays cut to their sizes."""
    assert row_ptr.dtype == torch.int64 and pos.dtype == torch.int32 and row_ptr.numel() == d_sae + 1
    dev = row_ptr.device
    n = pos.numel()
    mb, mw = s3_compact_bound(n, d_sae)
    cap_blocks = mb if cap_blocks is None else cap_blocks
    cap_words = mw if cap_words is None else cap_words
    if ws is None:
        ws = torch.zeros(s3_compact_workspace_bytes(n, d_sae), dtype=torch.uint8, device=dev)
    out_rp = torch.empty(d_sae + 1, dtype=torch.int64, device=dev)
    blk_ptr = torch.empty(d_sae + 1, dtype=torch.int32, device=dev)
    blk_first = torch.empty(max(cap_blocks, 1), dtype=torch.int32, device=dev)
    blk_desc = torch.empty(max(cap_blocks, 1), dtype=torch.int64, device=dev)
    payload = torch.empty(max(cap_words, 1), dtype=torch.int32, device=dev)
    sizes = torch.zeros(4, dtype=torch.int64, device=dev)
    _check(lib().s3_compact_build(_ptr(row_ptr), _ptr(pos), n, d_sae, stop_freq, _ptr(out_rp), _ptr(blk_ptr), _ptr(blk_first),
                                  _ptr(blk_desc), cap_blocks, _ptr(payload), cap_words, _ptr(sizes), _ptr(ws), ws.numel(),
                                  _stream(stream)))
    code = C.c_uint32(0)
    _check(lib().s3_workspace_status(_ptr(ws), _stream(stream), C.byref(code)))
    _, n_blocks, n_words, _ = sizes.tolist()
    return CompactLayer(out_rp, blk_ptr, blk_first[:n_blocks].contiguous(), blk_desc[:n_blocks].contiguous(),
                        payload[:n_words].contiguous())


def s3_coactivation_score_topspans_compact(layers, d_sae: int, L: int, q_ids: torch.Tensor, q_vals: torch.Tensor,
                                           width: int, stride: int, s: int, alpha: float, beta: float, ws: torch.Tensor,
                                           bm25: torch.Tensor | None = None, mode: int = S3_SCORE_MINCOUNT, stop_freq: int = 0,
                                           top_idx: torch.Tensor | None = None, top_score: torch.Tensor | None = None,
                                           all_scores: torch.Tensor | None = None, stream=None):
    """As s3_coactivation_score_topspans, with `layers` a list of CompactLayer on the device."""
    n_layers, Q, nq, k = q_ids.shape
    assert len(layers) == n_layers and q_ids.dtype == torch.int32 and q_vals.dtype == torch.float32
    assert q_ids.is_contiguous() and q_vals.is_contiguous()
    for c in layers:
        assert c.row_ptr.numel() == d_sae + 1 and c.payload.numel() >= 1
    views = (CompactView * n_layers)(*[c.view() for c in layers])
    dev = q_ids.device
    if top_idx is None:
        top_idx = torch.empty((Q, s), dtype=torch.int32, device=dev)
    if top_score is None:
        top_score = torch.empty((Q, s), dtype=torch.float32, device=dev)
    params = ScoreParams(width, stride, mode, s, alpha, beta, stop_freq)
    ld = 0 if bm25 is None else bm25.stride(0)
    _check(lib().s3_coactivation_score_topspans_compact(views, n_layers, d_sae, L, _ptr(q_ids), _ptr(q_vals), Q, nq, k,
                                                        C.byref(params), _ptr(bm25), ld, _ptr(top_idx), _ptr(top_score),
                                                        _ptr(all_scores), _ptr(ws), ws.numel(), _stream(stream)))
    return top_idx, top_score


def s3_compact_save(path: str, layers, d_sae: int):
    """layers: list of CompactLayer on the HOST."""
    arr = (CompactHostLayer * len(layers))(*[c.host_layer() for c in layers])
    _check(lib().s3_compact_save(path.encode(), len(layers), d_sae, arr))


def s3_compact_file_info(path: str):
    """Returns (n_layers, d_sae, [n_blocks per layer], [n_words per layer])."""
    n_layers, d_sae = C.c_int(), C.c_int()
    nb = (C.c_uint64 * 16)()
    nw = (C.c_uint64 * 16)()
    _check(lib().s3_compact_file_info(path.encode(), C.byref(n_layers), C.byref(d_sae), nb, nw, 16))
    return n_layers.value, d_sae.value, list(nb[:n_layers.value]), list(nw[:n_layers.value])


def s3_compact_load(path: str):
    """Returns (list of CompactLayer on the host, d_sae)."""
    n_layers, d_sae, nb, nw = s3_compact_file_info(path)
    layers = [CompactLayer(torch.empty(d_sae + 1, dtype=torch.int64), torch.empty(d_sae + 1, dtype=torch.int32),
                           torch.empty(nb[l], dtype=torch.int32), torch.empty(nb[l], dtype=torch.int64),
                           torch.empty(nw[l], dtype=torch.int32)) for l in range(n_layers)]
    arr = (CompactHostLayer * n_layers)(*[c.host_layer() for c in layers])
    _check(lib().s3_compact_load(path.encode(), n_layers, d_sae, arr))
    return layers, d_sae


def s3_sae_decode(W_dec: torch.Tensor, b_dec: torch.Tensor, ids: torch.Tensor, vals: torch.Tensor, x: torch.Tensor | None = None,
                  want_xhat: bool = True, stream=None):
    """W_dec [d_sae, d_in] bf16 or fp32, b_dec fp32 [d_in], ids int32 / vals fp32 [T, k]. Returns (x_hat fp32 [T, d_in] or
    None, sqerr fp32 [T] or None); sqerr is computed when x [T, d_in] (dtype of W_dec) is given."""
    assert W_dec.is_contiguous() and b_dec.dtype == torch.float32 and ids.dtype == torch.int32 and vals.dtype == torch.float32
    assert ids.is_contiguous() and vals.is_contiguous() and ids.shape == vals.shape
    d_sae, d_in = W_dec.shape
    T, k = ids.shape
    dtype = {torch.bfloat16: S3_BF16, torch.float32: S3_F32}[W_dec.dtype]
    dev = W_dec.device
    x_hat = torch.empty((T, d_in), dtype=torch.float32, device=dev) if want_xhat else None
    sqerr = None
    ldx = 0
    if x is not None:
        assert x.dtype == W_dec.dtype and x.shape == (T, d_in) and x.stride(1) == 1
        sqerr = torch.empty((T,), dtype=torch.float32, device=dev)
        ldx = x.stride(0)
    _check(lib().s3_sae_decode(_ptr(W_dec), _ptr(b_dec), d_in, d_sae, dtype, _ptr(ids), _ptr(vals), T, k, _ptr(x_hat), d_in,
                               _ptr(x), ldx, _ptr(sqerr), _stream(stream)))
    return x_hat, sqerr


def s3_head_aggregate_topk(ids: torch.Tensor, vals: torch.Tensor, d_sae: int, k_out: int, stream=None):
    """ids int32 / vals fp32 [T, H, k]: the heads' Top-k codes of every token. Returns (ids int32 [T, k_out],
    vals fp32 [T, k_out]): the features with the largest activation summed over the heads."""
    assert ids.dtype == torch.int32 and vals.dtype == torch.float32 and ids.shape == vals.shape and ids.dim() == 3
    assert ids.is_contiguous() and vals.is_contiguous()
    T, H, k = ids.shape
    out_i = torch.empty((T, k_out), dtype=torch.int32, device=ids.device)
    out_v = torch.empty((T, k_out), dtype=torch.float32, device=ids.device)
    _check(lib().s3_head_aggregate_topk(_ptr(ids), _ptr(vals), T, H, k, d_sae, k_out, _ptr(out_i), _ptr(out_v), _stream(stream)))
    return out_i, out_v


def s3_compact_expand(layer: CompactLayer, d_sae: int, ws: torch.Tensor | None = None, stream=None):
    """The compact layer's kept postings as a raw CSR on the device: (row_ptr int64 [d_sae+1], pos int32)."""
    dev = layer.row_ptr.device
    n = int(layer.row_ptr[-1])
    pos = torch.empty(max(n, 1), dtype=torch.int32, device=dev)
    if ws is None:
        ws = torch.zeros(64, dtype=torch.uint8, device=dev)
    view = layer.view()
    _check(lib().s3_compact_expand(C.byref(view), d_sae, _ptr(pos), n, _ptr(ws), ws.numel(), _stream(stream)))
    code = C.c_uint32(0)
    _check(lib().s3_workspace_status(_ptr(ws), _stream(stream), C.byref(code)))
    return layer.row_ptr, pos[:n]


def s3_sae_backward(W_enc: torch.Tensor, W_dec: torch.Tensor, b_dec: torch.Tensor, x: torch.Tensor, ids: torch.Tensor,
                    vals: torch.Tensor | None, ws: torch.Tensor | None = None, b_enc: torch.Tensor | None = None, stream=None):
    """fp32 tensors: W_enc [d_in, d_sae], W_dec [d_sae, d_in], b_dec [d_in], x [T, d_in]; ids int32 [T, k] and either the
    fp32 vals [T, k] of the same encode or None with b_enc [d_sae] (the code is then recomputed in fp32).
    Returns (loss [1], gW_enc, gb_enc, gW_dec, gb_dec)."""
    for t in (W_enc, W_dec, b_dec, x, vals, b_enc):
        assert t is None or t.dtype == torch.float32
    assert W_enc.is_contiguous() and W_dec.is_contiguous() and ids.is_contiguous() and x.stride(1) == 1
    assert vals is None or vals.is_contiguous()
    d_in, d_sae = W_enc.shape
    T, k = ids.shape
    assert W_dec.shape == (d_sae, d_in) and x.shape == (T, d_in) and ids.dtype == torch.int32
    dev = x.device
    if ws is None:
        ws = torch.zeros(s3_sae_backward_workspace_bytes(T), dtype=torch.uint8, device=dev)
    gW_enc, gW_dec = torch.empty_like(W_enc), torch.empty_like(W_dec)
    gb_enc = torch.empty(d_sae, dtype=torch.float32, device=dev)
    gb_dec = torch.empty(d_in, dtype=torch.float32, device=dev)
    loss = torch.empty(1, dtype=torch.float32, device=dev)
    _check(lib().s3_sae_backward(_ptr(W_enc), _ptr(b_enc), _ptr(W_dec), _ptr(b_dec), _ptr(x), x.stride(0), _ptr(ids), _ptr(vals), T, k, d_in, d_sae,
                                 _ptr(gW_enc), _ptr(gb_enc), _ptr(gW_dec), _ptr(gb_dec), _ptr(loss), _ptr(ws), ws.numel(),
                                 _stream(stream)))
    return loss, gW_enc, gb_enc, gW_dec, gb_dec


def s3_sae_backward_workspace_bytes(T: int) -> int:
    return int(lib().s3_sae_backward_workspace_bytes(T))


def s3_adam_update(param: torch.Tensor, m: torch.Tensor, v: torch.Tensor, grad: torch.Tensor, lr: float, beta1: float, beta2: float,
                   eps: float, step: int, stream=None):
    """In-place Adam step on a contiguous fp32 tensor and its moments."""
    for t in (param, m, v, grad):
        assert t.dtype == torch.float32 and t.is_contiguous() and t.numel() == param.numel()
    params = AdamParams(lr, beta1, beta2, eps, step, 0)
    _check(lib().s3_adam_update(_ptr(param), _ptr(m), _ptr(v), _ptr(grad), param.numel(), C.byref(params), _stream(stream)))


def s3_cast_f32_to_bf16(src: torch.Tensor, dst: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    assert src.dtype == torch.float32 and src.is_contiguous()
    if dst is None:
        dst = torch.empty(src.shape, dtype=torch.bfloat16, device=src.device)
    assert dst.dtype == torch.bfloat16 and dst.is_contiguous() and dst.numel() == src.numel()
    _check(lib().s3_cast_f32_to_bf16(_ptr(src), _ptr(dst), src.numel(), _stream(stream)))
    return dst


def s3_sae_preact(sae: "Sae", x: torch.Tensor, out_dtype: torch.dtype = torch.float32, out: torch.Tensor | None = None,
                  ws: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """Dense pre-activations [T, d_sae] of a bf16 encoder (fp32 or bf16 output)."""
    T = x.shape[0]
    if out is None:
        out = torch.empty((T, sae.d_sae), dtype=out_dtype, device=x.device)
    assert out.dtype == out_dtype and out.stride(1) == 1 and x.stride(1) == 1
    if ws is None:
        ws = torch.zeros(64, dtype=torch.uint8, device=x.device)
    code = {torch.bfloat16: S3_BF16, torch.float32: S3_F32}[out_dtype]
    _check(lib().s3_sae_preact(sae.handle, _ptr(x), x.stride(0) if T > 1 else max(x.stride(0), sae.d_in), T, _ptr(out), out.stride(0),
                               code, _ptr(ws), ws.numel(), _stream(stream)))
    return out
