"""Thin ctypes binding over the lw C ABI (``include/lw.h``): argument marshalling only.

Every function has the name and meaning of its C counterpart.  Device buffers are passed as torch
CUDA tensors (or raw integer addresses); PyTorch is used for device memory and streams, nothing
else -- all arithmetic of the path runs in the library's own kernels.  There is no CPU fallback:
if ``liblw.so`` has not been built (``python -m paper_2605_20706_b200.build``) every call raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

F16, Q8_0, Q4_0, Q4_K, Q6_K, Q5_K, Q2_K, Q4_1, Q5_0, Q5_1 = range(10)
FORMATS = {"f16": F16, "q8_0": Q8_0, "q4_0": Q4_0, "q4_K": Q4_K, "q6_K": Q6_K, "q5_K": Q5_K, "q2_K": Q2_K,
           "q4_1": Q4_1, "q5_0": Q5_0, "q5_1": Q5_1}
BITS_PER_WEIGHT = {F16: 16.0, Q8_0: 8.5, Q4_0: 4.5, Q4_K: 4.5, Q6_K: 6.5625, Q5_K: 5.5, Q2_K: 2.625, Q4_1: 5.0,
                   Q5_0: 5.5, Q5_1: 6.0}

VARIANT_AUTO, VARIANT_GENERIC, VARIANT_STREAM, VARIANT_IDOT, VARIANT_TILE, VARIANT_MMA = 0, 1, 2, 3, 4, 5

OK = 0
ERR_FORMAT, ERR_SHAPE, ERR_NULL, ERR_ALIGN, ERR_BATCH, ERR_NONFINITE, ERR_CUDA, ERR_DEVICE = (
    -1, -2, -3, -4, -5, -6, -7, -8)
ERR_WORKSPACE = -9

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "liblw.so")

EXPORTS = ("lw_block_elems", "lw_block_bytes", "lw_row_bytes", "lw_status_string", "lw_quantize",
           "lw_dequant", "lw_matvec", "lw_matvec_group", "lw_matvec_group_batch", "lw_matvec_sequence_batch", "lw_matvec_sequence_batch_host", "lw_matvec_host", "lw_set_variant", "lw_query_variant",
           "lw_set_overlap", "lw_device_status", "lw_set_tuning", "lw_plan_info", "lw_attn_decode",
           "lw_attn_workspace_bytes", "lw_attn_decode_static", "lw_set_attn_variant", "lw_query_attn_variant",
           "lw_debug_drop_copy", "lw_matvec_sequence", "lw_matvec_sequence_workspace_bytes", "lw_probe_read", "lw_set_sequence_mode", "lw_matvec_sequence_host", "lw_set_shape_tuning", "lw_clear_shape_tuning")

_lib = None


class LwError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__("%s: %s (status %d)" % (what, status_string(code), code))
        self.code = code


def lib() -> ctypes.CDLL:
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("liblw.so is missing at %s: build it with "
                           "`python -m paper_2605_20706_b200.build` (needs nvcc)" % LIB_PATH)
    L = ctypes.CDLL(LIB_PATH)
    i64, c_int, vp, sz = ctypes.c_int64, ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t
    L.lw_block_elems.restype, L.lw_block_elems.argtypes = sz, [c_int]
    L.lw_block_bytes.restype, L.lw_block_bytes.argtypes = sz, [c_int]
    L.lw_row_bytes.restype, L.lw_row_bytes.argtypes = sz, [c_int, i64]
    L.lw_status_string.restype, L.lw_status_string.argtypes = ctypes.c_char_p, [c_int]
    L.lw_quantize.restype, L.lw_quantize.argtypes = c_int, [c_int, vp, i64, vp]
    L.lw_dequant.restype, L.lw_dequant.argtypes = c_int, [c_int, vp, i64, vp, vp]
    L.lw_matvec.restype, L.lw_matvec.argtypes = c_int, [c_int, vp, i64, i64, vp, vp, c_int, vp]
    L.lw_matvec_group.restype = c_int
    L.lw_matvec_group.argtypes = [c_int, i64, c_int, vp, vp]
    L.lw_matvec_group_batch.restype = c_int
    L.lw_matvec_group_batch.argtypes = [c_int, i64, c_int, vp, c_int, vp]
    L.lw_matvec_host.restype = c_int
    L.lw_matvec_host.argtypes = [c_int, vp, i64, i64, vp, vp, vp, vp, c_int, vp]
    L.lw_set_variant.restype, L.lw_set_variant.argtypes = c_int, [c_int]
    L.lw_query_variant.restype, L.lw_query_variant.argtypes = c_int, [c_int, i64, i64, c_int]
    L.lw_set_overlap.restype, L.lw_set_overlap.argtypes = c_int, [c_int]
    L.lw_device_status.restype, L.lw_device_status.argtypes = c_int, [vp]
    L.lw_set_tuning.restype, L.lw_set_tuning.argtypes = c_int, [c_int, c_int, c_int]
    L.lw_set_shape_tuning.restype, L.lw_set_shape_tuning.argtypes = c_int, [c_int, i64, i64, c_int, c_int, c_int]
    L.lw_clear_shape_tuning.restype, L.lw_clear_shape_tuning.argtypes = c_int, []
    L.lw_plan_info.restype, L.lw_plan_info.argtypes = c_int, [c_int, i64, i64, vp]
    L.lw_attn_workspace_bytes.restype, L.lw_attn_workspace_bytes.argtypes = i64, [i64, i64, i64, i64]
    L.lw_attn_decode.restype = c_int
    L.lw_attn_decode.argtypes = [c_int, vp, vp, vp, vp, i64, i64, i64, i64, ctypes.c_float, vp, i64, vp]
    L.lw_set_attn_variant.restype, L.lw_set_attn_variant.argtypes = c_int, [c_int]
    L.lw_query_attn_variant.restype, L.lw_query_attn_variant.argtypes = c_int, [c_int, i64, i64, i64, i64]
    L.lw_matvec_sequence_workspace_bytes.restype, L.lw_matvec_sequence_workspace_bytes.argtypes = i64, []
    L.lw_matvec_sequence.restype = c_int
    L.lw_matvec_sequence.argtypes = [c_int, c_int, vp, vp, i64, vp]
    L.lw_set_sequence_mode.restype, L.lw_set_sequence_mode.argtypes = c_int, [c_int]
    L.lw_matvec_sequence_host.restype = c_int
    L.lw_matvec_sequence_host.argtypes = [c_int, c_int, vp, vp, vp, i64, vp, vp, i64, vp, i64, vp]
    L.lw_matvec_sequence_batch.restype = c_int
    L.lw_matvec_sequence_batch.argtypes = [c_int, c_int, vp, c_int, vp]
    L.lw_matvec_sequence_batch_host.restype = c_int
    L.lw_matvec_sequence_batch_host.argtypes = [c_int, c_int, vp, c_int, vp, vp, i64, vp, vp, i64, vp]
    L.lw_probe_read.restype, L.lw_probe_read.argtypes = c_int, [vp, i64, vp]
    L.lw_debug_drop_copy.restype, L.lw_debug_drop_copy.argtypes = c_int, [c_int]
    L.lw_attn_decode_static.restype = c_int
    L.lw_attn_decode_static.argtypes = [c_int, vp, vp, vp, vp, i64, i64, i64, i64, ctypes.c_float, vp]
    _lib = L
    return L


def _addr(buf) -> int:
    """Raw address of a torch tensor, numpy array or integer."""
    if buf is None:
        return 0
    if isinstance(buf, int):
        return buf
    if isinstance(buf, np.ndarray):
        return buf.ctypes.data
    return buf.data_ptr()          # torch.Tensor


def _stream_handle(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(rc: int, what: str) -> None:
    if rc != OK:
        raise LwError(rc, what)


def block_elems(fmt: int) -> int:
    return int(lib().lw_block_elems(fmt))


def block_bytes(fmt: int) -> int:
    return int(lib().lw_block_bytes(fmt))


def row_bytes(fmt: int, cols: int) -> int:
    return int(lib().lw_row_bytes(fmt, cols))


def status_string(code: int) -> str:
    return lib().lw_status_string(code).decode()


def quantize(fmt: int, src: np.ndarray, dst: np.ndarray | None = None) -> np.ndarray:
    """Host quantiser: float32 numpy array (row-major) -> uint8 array of blocks."""
    src = np.ascontiguousarray(src, dtype=np.float32).reshape(-1)
    nbytes = row_bytes(fmt, src.size)
    if dst is None:
        dst = np.empty(nbytes, dtype=np.uint8)
    if block_elems(fmt) and nbytes and (dst.dtype != np.uint8 or dst.size < nbytes or not dst.flags.c_contiguous):
        raise ValueError("dst must be a contiguous uint8 array of at least %d bytes" % nbytes)
    _check(lib().lw_quantize(fmt, _addr(src), src.size, _addr(dst)), "lw_quantize")
    return dst


def dequant(fmt: int, W_blocks, n: int, out, stream=None) -> None:
    _check(lib().lw_dequant(fmt, _addr(W_blocks), n, _addr(out), _stream_handle(stream)), "lw_dequant")


def matvec(fmt: int, W_blocks, rows: int, cols: int, X, Y, batch: int = 1, stream=None) -> None:
    _check(lib().lw_matvec(fmt, _addr(W_blocks), rows, cols, _addr(X), _addr(Y), batch,
                           _stream_handle(stream)), "lw_matvec")


class GroupItem(ctypes.Structure):
    _fields_ = [("W_blocks", ctypes.c_void_p), ("rows", ctypes.c_int64), ("X", ctypes.c_void_p),
                ("Y", ctypes.c_void_p)]


def matvec_group(fmt: int, cols: int, items, stream=None, batch: int = 1) -> None:
    """items: sequence of (W_blocks, rows, X, Y); one launch for all of them where the kernels allow it."""
    arr = (GroupItem * len(items))()
    for j, (w, rows, x, y) in enumerate(items):
        arr[j].W_blocks, arr[j].rows, arr[j].X, arr[j].Y = _addr(w) or None, rows, _addr(x) or None, _addr(y) or None
    if batch == 1:
        _check(lib().lw_matvec_group(fmt, cols, len(items), ctypes.cast(arr, ctypes.c_void_p),
                                     _stream_handle(stream)), "lw_matvec_group")
    else:
        _check(lib().lw_matvec_group_batch(fmt, cols, len(items), ctypes.cast(arr, ctypes.c_void_p), batch,
                                           _stream_handle(stream)), "lw_matvec_group_batch")


class SeqItem(ctypes.Structure):
    _fields_ = [("W_blocks", ctypes.c_void_p), ("rows", ctypes.c_int64), ("cols", ctypes.c_int64),
                ("X", ctypes.c_void_p), ("Y", ctypes.c_void_p), ("flags", ctypes.c_int)]


SEQ_DEPENDENT = 1


def matvec_sequence_workspace_bytes() -> int:
    return int(lib().lw_matvec_sequence_workspace_bytes())


def seq_items(items):
    """Marshals (W_blocks, rows, cols, X, Y, flags) tuples into a C array (reusable across calls)."""
    arr = (SeqItem * len(items))()
    for j, (w, rows, cols, x, y, flags) in enumerate(items):
        arr[j].W_blocks, arr[j].rows, arr[j].cols = _addr(w) or None, rows, cols
        arr[j].X, arr[j].Y, arr[j].flags = _addr(x) or None, _addr(y) or None, flags
    return arr


def matvec_sequence(fmt: int, items, workspace, workspace_bytes: int | None = None, stream=None) -> None:
    """items: sequence of (W_blocks, rows, cols, X, Y, flags) or an array from seq_items(); one persistent
    launch for the whole chain (batch 1)."""
    arr = items if isinstance(items, ctypes.Array) else seq_items(items)
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size() if hasattr(workspace, "numel") else 0
    _check(lib().lw_matvec_sequence(fmt, len(arr), ctypes.cast(arr, ctypes.c_void_p), _addr(workspace),
                                    workspace_bytes, _stream_handle(stream)), "lw_matvec_sequence")


SEQ_AUTO, SEQ_PERSISTENT, SEQ_LAUNCHES = 0, 1, 2


def set_sequence_mode(mode: int) -> None:
    _check(lib().lw_set_sequence_mode(mode), "lw_set_sequence_mode")


def matvec_sequence_host(fmt: int, items, in_host, in_dev, in_bytes: int, out_dev, out_host, out_bytes: int, workspace,
                         workspace_bytes: int | None = None, stream=None) -> None:
    """matvec_sequence with the input block in host memory and the result block returned to host memory (the
    library overlaps the copies with the kernels)."""
    arr = items if isinstance(items, ctypes.Array) else seq_items(items)
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size() if hasattr(workspace, "numel") else 0
    _check(lib().lw_matvec_sequence_host(fmt, len(arr), ctypes.cast(arr, ctypes.c_void_p), _addr(in_host), _addr(in_dev),
                                         in_bytes, _addr(out_dev), _addr(out_host), out_bytes, _addr(workspace),
                                         workspace_bytes, _stream_handle(stream)), "lw_matvec_sequence_host")


def matvec_sequence_batch(fmt: int, items, batch: int, stream=None) -> None:
    """A chain of mat-vecs with `batch` columns each: (W_blocks, rows, cols, X, Y, flags) tuples or seq_items()."""
    arr = items if isinstance(items, ctypes.Array) else seq_items(items)
    _check(lib().lw_matvec_sequence_batch(fmt, len(arr), ctypes.cast(arr, ctypes.c_void_p), batch, _stream_handle(stream)),
           "lw_matvec_sequence_batch")


def matvec_sequence_batch_host(fmt: int, items, batch: int, in_host, in_dev, in_bytes: int, out_dev, out_host,
                               out_bytes: int, stream=None) -> None:
    """matvec_sequence_batch with the input block in host memory and the result block returned to host memory."""
    arr = items if isinstance(items, ctypes.Array) else seq_items(items)
    _check(lib().lw_matvec_sequence_batch_host(fmt, len(arr), ctypes.cast(arr, ctypes.c_void_p), batch, _addr(in_host),
                                               _addr(in_dev), in_bytes, _addr(out_dev), _addr(out_host), out_bytes,
                                               _stream_handle(stream)), "lw_matvec_sequence_batch_host")


def matvec_host(fmt: int, W_blocks, rows: int, cols: int, X_host, Y_host, X_dev, Y_dev,
                batch: int = 1, stream=None) -> None:
    _check(lib().lw_matvec_host(fmt, _addr(W_blocks), rows, cols, _addr(X_host), _addr(Y_host),
                                _addr(X_dev), _addr(Y_dev), batch, _stream_handle(stream)),
           "lw_matvec_host")


ATTN_AUTO, ATTN_GENERAL, ATTN_TENSOR = 0, 1, 2


def set_attn_variant(variant: int) -> None:
    _check(lib().lw_set_attn_variant(variant), "lw_set_attn_variant")


def query_attn_variant(kv_fmt: int, n_head: int, n_kv_head: int, head_dim: int, n_pos: int) -> int:
    rc = lib().lw_query_attn_variant(kv_fmt, n_head, n_kv_head, head_dim, n_pos)
    if rc < 0:
        raise LwError(rc, "lw_query_attn_variant")
    return rc


def attn_workspace_bytes(n_head: int, n_kv_head: int, head_dim: int, n_pos: int) -> int:
    return int(lib().lw_attn_workspace_bytes(n_head, n_kv_head, head_dim, n_pos))


def attn_decode(kv_fmt: int, K_blocks, V_blocks, q, out, n_head: int, n_kv_head: int, head_dim: int, n_pos: int,
                scale: float, workspace, workspace_bytes: int | None = None, stream=None) -> None:
    """out[h] = softmax_t(scale * K[t, g] . q[h]) @ V[:, g] for one query token; device buffers."""
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size() if hasattr(workspace, "numel") else 0
    _check(lib().lw_attn_decode(kv_fmt, _addr(K_blocks), _addr(V_blocks), _addr(q), _addr(out), n_head, n_kv_head,
                                head_dim, n_pos, ctypes.c_float(scale), _addr(workspace), workspace_bytes,
                                _stream_handle(stream)), "lw_attn_decode")


def attn_decode_static(kv_fmt: int, K_blocks, V_blocks, q, out, n_head: int, n_kv_head: int, head_dim: int,
                       n_pos: int, scale: float, stream=None) -> None:
    """attn_decode for callers without a device allocator: partial results go to the library's own fixed
    array (n_head * (head_dim + 2) <= 16384); calls on one device must not overlap."""
    _check(lib().lw_attn_decode_static(kv_fmt, _addr(K_blocks), _addr(V_blocks), _addr(q), _addr(out), n_head,
                                       n_kv_head, head_dim, n_pos, ctypes.c_float(scale), _stream_handle(stream)),
           "lw_attn_decode_static")


def set_variant(variant: int) -> None:
    _check(lib().lw_set_variant(variant), "lw_set_variant")


def query_variant(fmt: int, rows: int, cols: int, batch: int = 1) -> int:
    rc = lib().lw_query_variant(fmt, rows, cols, batch)
    if rc < 0:
        raise LwError(rc, "lw_query_variant")
    return rc


def set_overlap(enabled) -> None:
    """False / 0: ordinary launches; True / 1: programmatic dependent launch; 2: and early weight streaming."""
    _check(lib().lw_set_overlap(int(enabled)), "lw_set_overlap")


def set_tuning(worker_groups: int = 0, stages: int = 0, stage_kb: int = 0) -> None:
    _check(lib().lw_set_tuning(worker_groups, stages, stage_kb), "lw_set_tuning")


def set_shape_tuning(fmt: int, rows: int, cols: int, worker_groups: int = 0, stages: int = 0, stage_kb: int = 0) -> None:
    _check(lib().lw_set_shape_tuning(fmt, rows, cols, worker_groups, stages, stage_kb), "lw_set_shape_tuning")


def clear_shape_tuning() -> None:
    _check(lib().lw_clear_shape_tuning(), "lw_clear_shape_tuning")


def load_tuning_table(path: str) -> int:
    """Installs the per-shape table a sweep wrote (JSON list of {format, rows, cols, worker_groups, stages,
    stage_kb}); returns the number of entries."""
    import json
    with open(path) as fh:
        table = json.load(fh)
    for e in table:
        set_shape_tuning(FORMATS[e["format"]], e["rows"], e["cols"], e.get("worker_groups", 0), e.get("stages", 0),
                         e.get("stage_kb", 0))
    return len(table)


def plan_info(fmt: int, rows: int, cols: int) -> dict:
    out = (ctypes.c_int * 6)()
    _check(lib().lw_plan_info(fmt, rows, cols, ctypes.cast(out, ctypes.c_void_p)), "lw_plan_info")
    keys = ("worker_groups", "stages", "stage_rows", "stage_bytes", "ctas", "smem_bytes")
    return dict(zip(keys, list(out)))


def probe_read(src, nbytes: int, stream=None) -> None:
    """Measurement aid: streams nbytes at src through the streaming kernels' copy pipeline, no arithmetic."""
    _check(lib().lw_probe_read(_addr(src), nbytes, _stream_handle(stream)), "lw_probe_read")


def debug_drop_copy(unit: int) -> None:
    """Testing aid: the next single-matrix streaming mat-vec never requests the copy of pool unit `unit`."""
    _check(lib().lw_debug_drop_copy(unit), "lw_debug_drop_copy")


def device_status() -> int:
    """Reads and clears the device fault word (synchronises the device)."""
    out = ctypes.c_int(0)
    _check(lib().lw_device_status(ctypes.byref(out)), "lw_device_status")
    return out.value
