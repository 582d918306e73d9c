"""ctypes binding of libsparsed.so: same entry points, same names, argument marshalling only.

Torch is used for device memory and the current stream; every step of the attention path
runs inside the CUDA library. There is no CPU or PyTorch fallback: if the shared library is
missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

from . import build as _build

STATUS_BYTES = 256
(OP_ATTN_FULL, OP_SELECT_PATTERN, OP_SELECT_FROM_SCORES, OP_ATTN_SPARSE, OP_PATTERN_VALIDATE, OP_SELECT_POOLED_QK,
 OP_ATTENTION_STEP) = range(7)
MODE_FULL, MODE_FULL_AND_SELECT, MODE_SPARSE = 0, 1, 2
VARIANT_NO_REUSE, VARIANT_NO_ISOLATION = 1, 2

EXPORTED_SYMBOLS = (
    "sparsed_attn_full", "sparsed_select_pattern", "sparsed_select_from_scores", "sparsed_attn_sparse",
    "sparsed_schedule_mode", "sparsed_switch_step", "sparsed_kept_per_row", "sparsed_workspace_bytes",
    "sparsed_workspace_init", "sparsed_pattern_validate", "sparsed_last_device_status",
    "sparsed_status_string", "sparsed_last_cuda_error", "sparsed_select_pattern_static",
    "sparsed_tile_stats_bytes", "sparsed_attn_full_stats", "sparsed_select_from_stats",
    "sparsed_build_window_pattern", "sparsed_selftest_wait_timeout", "sparsed_select_pattern_pooled_qk",
    "sparsed_attention_step", "sparsed_attention_step_variant",
)


class SparsedError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what} failed: status {status} ({status_string(status)})"
                         + (f", cuda error {last_cuda_error()}" if status == 7 else ""))


class Shape(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("heads_q", ctypes.c_int32), ("heads_kv", ctypes.c_int32),
                ("seq_len", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("q_strides", ctypes.c_int64 * 3), ("k_strides", ctypes.c_int64 * 3),
                ("v_strides", ctypes.c_int64 * 3), ("o_strides", ctypes.c_int64 * 3),
                ("softmax_scale", ctypes.c_float)]


class SelectParams(ctypes.Structure):
    _fields_ = [("block_size", ctypes.c_int32), ("prefill_len", ctypes.c_int32),
                ("keep_ratio", ctypes.c_double), ("rounding", ctypes.c_int32)]


class Pattern(ctypes.Structure):
    _fields_ = [("row_ptr", ctypes.c_void_p), ("col_idx", ctypes.c_void_p), ("col_capacity", ctypes.c_int64),
                ("nnz", ctypes.c_int64), ("block_size", ctypes.c_int32), ("num_blocks", ctypes.c_int32),
                ("batch", ctypes.c_int32), ("heads_q", ctypes.c_int32)]


_lib = None


def library_path() -> str:
    return _build.LIB_PATH


def load_library() -> ctypes.CDLL:
    """Loads libsparsed.so (must have been built: ``python -m paper_2509_24014_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_2509_24014_b200.build` "
                           "(there is no CPU fallback)")
    lib = ctypes.CDLL(path)
    vp, sz, i32, f64 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int32, ctypes.c_double
    P = ctypes.POINTER
    lib.sparsed_attn_full.argtypes = [P(Shape), vp, vp, vp, vp, vp, vp, sz, vp]
    lib.sparsed_select_pattern.argtypes = [P(Shape), P(SelectParams), vp, vp, vp, P(Pattern), vp, vp, sz, vp]
    lib.sparsed_select_pattern_pooled_qk.argtypes = [P(Shape), P(SelectParams), vp, vp, P(Pattern), vp, vp, sz, vp]
    lib.sparsed_attention_step.argtypes = [P(Shape), P(SelectParams), i32, i32, ctypes.c_double, vp, vp, vp, vp,
                                           P(Pattern), vp, sz, vp, P(i32)]
    lib.sparsed_attention_step_variant.argtypes = [P(Shape), P(SelectParams), i32, i32, i32, ctypes.c_double, vp, vp, vp,
                                                   vp, P(Pattern), vp, sz, vp, P(i32)]
    lib.sparsed_select_pattern_static.argtypes = [P(Shape), P(SelectParams), vp, vp, vp, P(Pattern), vp]
    lib.sparsed_build_window_pattern.argtypes = [i32, i32, i32, i32, i32, i32, P(Pattern), vp]
    lib.sparsed_selftest_wait_timeout.argtypes = [vp, sz, vp]
    lib.sparsed_tile_stats_bytes.argtypes = [P(Shape), i32, P(sz)]
    lib.sparsed_attn_full_stats.argtypes = [P(Shape), i32, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.sparsed_select_from_stats.argtypes = [P(Shape), P(SelectParams), vp, vp, P(Pattern), vp, vp, sz, vp]
    lib.sparsed_select_from_scores.argtypes = [P(SelectParams), vp, i32, i32, i32, P(Pattern), vp, sz, vp]
    lib.sparsed_attn_sparse.argtypes = [P(Shape), P(Pattern), vp, vp, vp, vp, vp, sz, vp]
    lib.sparsed_schedule_mode.argtypes = [i32, i32, f64]
    lib.sparsed_switch_step.argtypes = [i32, f64]
    lib.sparsed_kept_per_row.argtypes = [P(SelectParams), i32, P(i32), P(i32)]
    lib.sparsed_workspace_bytes.argtypes = [i32, P(Shape), P(SelectParams), P(sz)]
    lib.sparsed_workspace_init.argtypes = [vp, sz, vp]
    lib.sparsed_pattern_validate.argtypes = [P(Pattern), vp, sz, vp]
    lib.sparsed_last_device_status.argtypes = [vp, vp, P(i32), P(i32)]
    lib.sparsed_status_string.argtypes = [i32]
    lib.sparsed_status_string.restype = ctypes.c_char_p
    lib.sparsed_last_cuda_error.argtypes = []
    for name in EXPORTED_SYMBOLS:
        if name not in ("sparsed_status_string",):
            getattr(lib, name).restype = i32
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().sparsed_status_string(int(status)).decode()


def last_cuda_error() -> int:
    return int(load_library().sparsed_last_cuda_error())


def _check(status: int, what: str) -> None:
    if status != 0:
        raise SparsedError(int(status), what)


def _stream(t: torch.Tensor) -> int:
    return int(torch.cuda.current_stream(t.device).cuda_stream)


def _strides3(t: torch.Tensor):
    if t.dim() != 4 or t.stride(3) != 1:
        raise ValueError("tensors must be [batch, heads, seq_len, head_dim] with head_dim contiguous")
    return (ctypes.c_int64 * 3)(t.stride(0), t.stride(1), t.stride(2))


def make_shape(q: torch.Tensor, k: torch.Tensor, v: Optional[torch.Tensor] = None,
               o: Optional[torch.Tensor] = None, softmax_scale: float = 0.0) -> Shape:
    s = Shape()
    s.batch, s.heads_q, s.seq_len, s.head_dim = q.shape
    s.heads_kv = k.shape[1]
    s.q_strides = _strides3(q)
    s.k_strides = _strides3(k)
    s.v_strides = _strides3(v if v is not None else k)
    s.o_strides = _strides3(o if o is not None else q)
    s.softmax_scale = softmax_scale
    return s


def make_params(block_size: int, keep_ratio: float, prefill_len: int = 0, rounding: int = 0) -> SelectParams:
    return SelectParams(int(block_size), int(prefill_len), float(keep_ratio), int(rounding))


# ----------------------------------------------------------------------------- host helpers
def sparsed_schedule_mode(step_1based: int, total_steps: int, skip: float) -> int:
    return int(load_library().sparsed_schedule_mode(step_1based, total_steps, skip))


def sparsed_switch_step(total_steps: int, skip: float) -> int:
    return int(load_library().sparsed_switch_step(total_steps, skip))


def sparsed_kept_per_row(params: SelectParams, seq_len: int) -> Tuple[int, int]:
    a, b = ctypes.c_int32(), ctypes.c_int32()
    _check(load_library().sparsed_kept_per_row(ctypes.byref(params), seq_len, ctypes.byref(a), ctypes.byref(b)),
           "sparsed_kept_per_row")
    return a.value, b.value


def sparsed_workspace_bytes(op: int, shape: Optional[Shape] = None, params: Optional[SelectParams] = None) -> int:
    out = ctypes.c_size_t()
    _check(load_library().sparsed_workspace_bytes(op, ctypes.byref(shape) if shape is not None else None,
                                                  ctypes.byref(params) if params is not None else None,
                                                  ctypes.byref(out)), "sparsed_workspace_bytes")
    return int(out.value)


def new_workspace(nbytes: int, device) -> torch.Tensor:
    """A zeroed workspace of at least ``nbytes`` bytes (torch only provides the memory)."""
    return torch.zeros(max(int(nbytes), STATUS_BYTES), dtype=torch.uint8, device=device)


def sparsed_workspace_init(ws: torch.Tensor) -> None:
    _check(load_library().sparsed_workspace_init(ws.data_ptr(), ws.numel(), _stream(ws)), "sparsed_workspace_init")


def new_pattern(batch: int, heads_q: int, num_blocks: int, kept_per_row: int, device):
    """Caller-owned CSR buffers; returns (Pattern struct, row_ptr tensor, col_idx tensor)."""
    rows = batch * heads_q * num_blocks
    row_ptr = torch.zeros(rows + 1, dtype=torch.int32, device=device)
    col_idx = torch.zeros(max(rows * kept_per_row, 1), dtype=torch.int32, device=device)
    pat = Pattern(row_ptr.data_ptr(), col_idx.data_ptr(), col_idx.numel(), 0, 0, num_blocks, batch, heads_q)
    return pat, row_ptr, col_idx


def pattern_from_csr(row_ptr: torch.Tensor, col_idx: torch.Tensor, block_size: int, num_blocks: int, batch: int,
                     heads_q: int) -> Pattern:
    assert row_ptr.dtype == torch.int32 and col_idx.dtype == torch.int32
    return Pattern(row_ptr.data_ptr(), col_idx.data_ptr(), col_idx.numel(), int(col_idx.numel()), block_size,
                   num_blocks, batch, heads_q)


# ----------------------------------------------------------------------------- device calls
def sparsed_attn_full(q, k, v, o, lse: Optional[torch.Tensor], ws: torch.Tensor, softmax_scale: float = 0.0,
                      shape: Optional[Shape] = None) -> None:
    shape = shape or make_shape(q, k, v, o, softmax_scale)
    _check(load_library().sparsed_attn_full(ctypes.byref(shape), q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                            o.data_ptr(), lse.data_ptr() if lse is not None else None,
                                            ws.data_ptr(), ws.numel(), _stream(q)), "sparsed_attn_full")


def sparsed_select_pattern(q, k, params: SelectParams, pattern: Pattern, ws: torch.Tensor,
                           lse: Optional[torch.Tensor] = None, scores_out: Optional[torch.Tensor] = None,
                           softmax_scale: float = 0.0, shape: Optional[Shape] = None) -> None:
    shape = shape or make_shape(q, k, None, None, softmax_scale)
    _check(load_library().sparsed_select_pattern(
        ctypes.byref(shape), ctypes.byref(params), q.data_ptr(), k.data_ptr(),
        lse.data_ptr() if lse is not None else None, ctypes.byref(pattern),
        scores_out.data_ptr() if scores_out is not None else None, ws.data_ptr(), ws.numel(), _stream(q)),
        "sparsed_select_pattern")


def sparsed_select_pattern_pooled_qk(q, k, params: SelectParams, pattern: Pattern, ws: torch.Tensor,
                                     scores_out: Optional[torch.Tensor] = None, softmax_scale: float = 0.0,
                                     shape: Optional[Shape] = None) -> None:
    """Selection from the block-mean estimate of A' (a contrast scorer, not the paper's)."""
    shape = shape or make_shape(q, k, None, None, softmax_scale)
    _check(load_library().sparsed_select_pattern_pooled_qk(
        ctypes.byref(shape), ctypes.byref(params), q.data_ptr(), k.data_ptr(), ctypes.byref(pattern),
        scores_out.data_ptr() if scores_out is not None else None, ws.data_ptr(), ws.numel(), _stream(q)),
        "sparsed_select_pattern_pooled_qk")


def sparsed_attention_step(q, k, v, o, params: SelectParams, step_1based: int, total_steps: int, skip: float,
                           pattern: Pattern, ws: torch.Tensor, softmax_scale: float = 0.0,
                           shape: Optional[Shape] = None) -> int:
    """Algorithm 1 for one attention call of one denoising step; returns the mode that ran."""
    shape = shape or make_shape(q, k, v, o, softmax_scale)
    mode = ctypes.c_int32(-1)
    _check(load_library().sparsed_attention_step(
        ctypes.byref(shape), ctypes.byref(params), int(step_1based), int(total_steps), float(skip), q.data_ptr(),
        k.data_ptr(), v.data_ptr(), o.data_ptr(), ctypes.byref(pattern), ws.data_ptr(), ws.numel(), _stream(q),
        ctypes.byref(mode)), "sparsed_attention_step")
    return int(mode.value)


def sparsed_attention_step_variant(q, k, v, o, params: SelectParams, variant: int, step_1based: int,
                                   total_steps: int, skip: float, pattern: Pattern, ws: torch.Tensor,
                                   softmax_scale: float = 0.0, shape: Optional[Shape] = None) -> int:
    """sparsed_attention_step with components of the method switched off (VARIANT_* flags)."""
    shape = shape or make_shape(q, k, v, o, softmax_scale)
    mode = ctypes.c_int32(-1)
    _check(load_library().sparsed_attention_step_variant(
        ctypes.byref(shape), ctypes.byref(params), int(variant), int(step_1based), int(total_steps), float(skip),
        q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), ctypes.byref(pattern), ws.data_ptr(), ws.numel(),
        _stream(q), ctypes.byref(mode)), "sparsed_attention_step_variant")
    return int(mode.value)


def sparsed_tile_stats_bytes(shape: Shape, block_size: int) -> int:
    out = ctypes.c_size_t()
    _check(load_library().sparsed_tile_stats_bytes(ctypes.byref(shape), int(block_size), ctypes.byref(out)),
           "sparsed_tile_stats_bytes")
    return int(out.value)


def new_tile_stats(q: torch.Tensor, block_size: int) -> torch.Tensor:
    """Caller-owned buffer for sparsed_attn_full_stats: fp32 [B*Hq, ceil(L/128), L/block_size, 128]."""
    B, Hq, L, _ = q.shape
    return torch.empty(B * Hq, (L + 127) // 128, L // block_size, 128, dtype=torch.float32, device=q.device)


def sparsed_attn_full_stats(q, k, v, o, lse: torch.Tensor, tile_stats: torch.Tensor, ws: torch.Tensor,
                            block_size: int, softmax_scale: float = 0.0, shape: Optional[Shape] = None) -> None:
    """block_size: the pattern block size the statistics are recorded for (one statistic per row and key block)."""
    shape = shape or make_shape(q, k, v, o, softmax_scale)
    assert tile_stats.numel() * 4 >= sparsed_tile_stats_bytes(shape, block_size) and tile_stats.dtype == torch.float32
    _check(load_library().sparsed_attn_full_stats(ctypes.byref(shape), int(block_size), q.data_ptr(), k.data_ptr(),
                                                  v.data_ptr(), o.data_ptr(), lse.data_ptr(), tile_stats.data_ptr(),
                                                  ws.data_ptr(), ws.numel(), _stream(q)), "sparsed_attn_full_stats")


def sparsed_select_from_stats(q, k, params: SelectParams, lse: torch.Tensor, tile_stats: torch.Tensor,
                              pattern: Pattern, ws: torch.Tensor, scores_out: Optional[torch.Tensor] = None,
                              shape: Optional[Shape] = None) -> None:
    """q and k only provide the shape here; the kernels read lse and tile_stats."""
    shape = shape or make_shape(q, k)
    _check(load_library().sparsed_select_from_stats(
        ctypes.byref(shape), ctypes.byref(params), lse.data_ptr(), tile_stats.data_ptr(), ctypes.byref(pattern),
        scores_out.data_ptr() if scores_out is not None else None, ws.data_ptr(), ws.numel(), _stream(lse)),
        "sparsed_select_from_stats")


STATIC_SCRATCH_BYTES = 8 << 20


def sparsed_select_pattern_static(q, k, params: SelectParams, pattern: Pattern, lse: Optional[torch.Tensor] = None,
                                  softmax_scale: float = 0.0, shape: Optional[Shape] = None) -> None:
    """Pattern selection for callers that may not allocate device memory: the scratch is a fixed
    array inside the library (STATIC_SCRATCH_BYTES), shared by every call on the device, so
    calls must not overlap on the GPU. Requests that do not fit raise SparsedError (status 4)."""
    shape = shape or make_shape(q, k, None, None, softmax_scale)
    _check(load_library().sparsed_select_pattern_static(
        ctypes.byref(shape), ctypes.byref(params), q.data_ptr(), k.data_ptr(),
        lse.data_ptr() if lse is not None else None, ctypes.byref(pattern), _stream(q)),
        "sparsed_select_pattern_static")


def sparsed_select_from_scores(scores: torch.Tensor, params: SelectParams, pattern: Pattern,
                               ws: torch.Tensor) -> None:
    assert scores.dtype == torch.float32 and scores.is_contiguous() and scores.dim() == 4
    b, h, nb, nb2 = scores.shape
    assert nb == nb2
    _check(load_library().sparsed_select_from_scores(ctypes.byref(params), scores.data_ptr(), b, h, nb,
                                                     ctypes.byref(pattern), ws.data_ptr(), ws.numel(),
                                                     _stream(scores)), "sparsed_select_from_scores")


def sparsed_attn_sparse(q, k, v, o, pattern: Pattern, ws: torch.Tensor, softmax_scale: float = 0.0,
                        shape: Optional[Shape] = None) -> None:
    shape = shape or make_shape(q, k, v, o, softmax_scale)
    _check(load_library().sparsed_attn_sparse(ctypes.byref(shape), ctypes.byref(pattern), q.data_ptr(),
                                              k.data_ptr(), v.data_ptr(), o.data_ptr(), ws.data_ptr(), ws.numel(),
                                              _stream(q)), "sparsed_attn_sparse")


def sparsed_build_window_pattern(batch: int, heads_q: int, num_blocks: int, block_size: int, sink_blocks: int,
                                 window_blocks: int, device):
    """Sliding-window (+ sink) comparison pattern as CSR; returns (Pattern, row_ptr, col_idx)."""
    half = (window_blocks - 1) // 2
    cap = batch * heads_q * num_blocks * min(num_blocks, 2 * half + 1 + max(sink_blocks, 0))
    row_ptr = torch.zeros(batch * heads_q * num_blocks + 1, dtype=torch.int32, device=device)
    col_idx = torch.zeros(max(cap, 1), dtype=torch.int32, device=device)
    pat = Pattern(row_ptr.data_ptr(), col_idx.data_ptr(), col_idx.numel(), 0, 0, 0, 0, 0)
    _check(load_library().sparsed_build_window_pattern(batch, heads_q, num_blocks, block_size, sink_blocks,
                                                       window_blocks, ctypes.byref(pat), _stream(row_ptr)),
           "sparsed_build_window_pattern")
    return pat, row_ptr, col_idx


def sparsed_pattern_validate(pattern: Pattern, ws: torch.Tensor) -> bool:
    st = load_library().sparsed_pattern_validate(ctypes.byref(pattern), ws.data_ptr(), ws.numel(), _stream(ws))
    if st == 0:
        return True
    if st == 5:
        return False
    raise SparsedError(int(st), "sparsed_pattern_validate")


def sparsed_selftest_wait_timeout(ws: torch.Tensor) -> None:
    _check(load_library().sparsed_selftest_wait_timeout(ws.data_ptr(), ws.numel(), _stream(ws)),
           "sparsed_selftest_wait_timeout")


def save_pattern(path: str, pattern: Pattern, row_ptr: torch.Tensor, col_idx: torch.Tensor, **meta) -> None:
    """Writes a selected pattern to an .npz file: the only state the method carries across denoising
    steps, so a run can resume in its sparse phase without selecting again."""
    import numpy as np
    np.savez(path, row_ptr=row_ptr.cpu().numpy(), col_idx=col_idx.cpu().numpy()[: int(pattern.nnz)],
             block_size=pattern.block_size, num_blocks=pattern.num_blocks, batch=pattern.batch,
             heads_q=pattern.heads_q, **meta)


def load_pattern(path: str, device):
    """Reads a pattern written by save_pattern; returns (Pattern, row_ptr, col_idx, meta dict)."""
    import numpy as np
    z = np.load(path if str(path).endswith(".npz") else str(path) + ".npz")
    row_ptr = torch.from_numpy(z["row_ptr"]).to(device=device, dtype=torch.int32)
    col_idx = torch.from_numpy(z["col_idx"]).to(device=device, dtype=torch.int32)
    pat = pattern_from_csr(row_ptr, col_idx, int(z["block_size"]), int(z["num_blocks"]), int(z["batch"]),
                           int(z["heads_q"]))
    meta = {k: z[k].item() for k in z.files if k not in ("row_ptr", "col_idx", "block_size", "num_blocks", "batch", "heads_q")}
    return pat, row_ptr, col_idx, meta


def sparsed_last_device_status(ws: torch.Tensor) -> Tuple[int, int]:
    code, where = ctypes.c_int32(), ctypes.c_int32()
    st = load_library().sparsed_last_device_status(ws.data_ptr(), _stream(ws), ctypes.byref(code),
                                                   ctypes.byref(where))
    if st not in (0, 8):
        raise SparsedError(int(st), "sparsed_last_device_status")
    return code.value, where.value
