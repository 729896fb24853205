"""Python binding of libstream (argument marshalling only; every step runs in the CUDA library).

The ``stream_*`` functions mirror the C ABI in ``include/stream.h`` one to one and take torch
CUDA tensors (or raw integer addresses) where the C side takes device pointers. ``build_mask``,
``sparse_attention`` and ``run_host`` are conveniences that allocate outputs with torch and fill
in the problem struct from tensor shapes and strides. PyTorch is used for device memory and
streams only.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libstream.so")

STREAM_OK, STREAM_ERR_INVALID_ARG, STREAM_ERR_UNSUPPORTED, STREAM_ERR_WORKSPACE, STREAM_ERR_CUDA, STREAM_ERR_DEVICE_CHECK = range(6)
STREAM_F32, STREAM_BF16 = 0, 1
IMPL = {"auto": 0, "generic": 1, "tensor": 2}
_STATUS_NAMES = ["OK", "INVALID_ARG", "UNSUPPORTED", "WORKSPACE", "CUDA", "DEVICE_CHECK"]


class StreamProblem(ctypes.Structure):
    """``stream_problem`` of stream.h."""

    _fields_ = [
        ("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
        ("T", ctypes.c_int64),
        ("d", ctypes.c_int32), ("block_q", ctypes.c_int32), ("block_k", ctypes.c_int32), ("k_top", ctypes.c_int32),
        ("causal", ctypes.c_int32), ("dtype", ctypes.c_int32), ("impl", ctypes.c_int32),
        ("q_stride_b", ctypes.c_int64), ("q_stride_h", ctypes.c_int64), ("q_stride_t", ctypes.c_int64),
        ("kv_stride_b", ctypes.c_int64), ("kv_stride_h", ctypes.c_int64), ("kv_stride_t", ctypes.c_int64),
    ]


class StreamStats(ctypes.Structure):
    """``stream_stats`` of stream.h."""

    _fields_ = [("tiles_scored", ctypes.c_uint64), ("rows", ctypes.c_uint64), ("error", ctypes.c_uint32),
                ("error_info", ctypes.c_uint32), ("tile_products", ctypes.c_uint64),
                ("tiles_fetched", ctypes.c_uint64)]


class StreamUnitRates(ctypes.Structure):
    """``stream_unit_rates`` of stream.h."""

    _fields_ = [("tma_bytes_per_clk", ctypes.c_double), ("mma_cycles_m128n64", ctypes.c_double),
                ("error", ctypes.c_uint32), ("reserved", ctypes.c_uint32)]


class StreamError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__(f"libstream: STREAM_ERR_{_STATUS_NAMES[status]}: {text}")
        self.status = status


_lib = None


def library_path() -> str:
    return _LIB_PATH


def _load():
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2510_19875_b200.build` "
            "(there is no fallback path without the CUDA library)")
    lib = ctypes.CDLL(_LIB_PATH)
    P, vp, sz = ctypes.POINTER(StreamProblem), ctypes.c_void_p, ctypes.c_size_t
    lib.stream_version.restype = ctypes.c_int
    lib.stream_version.argtypes = []
    lib.stream_last_error.restype = ctypes.c_char_p
    lib.stream_last_error.argtypes = []
    lib.stream_workspace_bytes.restype = sz
    lib.stream_workspace_bytes.argtypes = [P]
    lib.stream_build_mask.restype = ctypes.c_int
    lib.stream_build_mask.argtypes = [P, vp, vp, vp, vp, vp, sz, vp]
    lib.stream_build_mask_var.restype = ctypes.c_int
    lib.stream_build_mask_var.argtypes = [P, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.stream_workspace_bytes_multi.restype = sz
    lib.stream_workspace_bytes_multi.argtypes = [P, ctypes.c_int32]
    lib.stream_build_mask_multi.restype = ctypes.c_int
    lib.stream_build_mask_multi.argtypes = [P, vp, vp, ctypes.c_int32, vp, vp, vp, vp, sz, vp]
    lib.stream_k_schedule.restype = ctypes.c_int
    lib.stream_k_schedule.argtypes = [P, ctypes.c_double, vp]
    lib.stream_effective_k.restype = ctypes.c_int
    lib.stream_effective_k.argtypes = [ctypes.c_int64, ctypes.c_int32, ctypes.c_double, ctypes.POINTER(ctypes.c_int32)]
    lib.stream_selftest_bounded_wait.restype = ctypes.c_int
    lib.stream_selftest_bounded_wait.argtypes = [ctypes.c_int64, vp, sz, vp]
    lib.stream_probe_scratch_bytes.restype = sz
    lib.stream_probe_scratch_bytes.argtypes = []
    lib.stream_probe_unit_rates.restype = ctypes.c_int
    lib.stream_probe_unit_rates.argtypes = [vp, sz, ctypes.POINTER(StreamUnitRates), vp]
    lib.stream_build_mask_static.restype = ctypes.c_int
    lib.stream_build_mask_static.argtypes = [P, vp, vp, vp, vp, vp]
    lib.stream_sparse_attention.restype = ctypes.c_int
    lib.stream_sparse_attention.argtypes = [P, vp, vp, vp, vp, ctypes.c_float, vp, vp]
    lib.stream_read_stats.restype = ctypes.c_int
    lib.stream_read_stats.argtypes = [vp, ctypes.POINTER(StreamStats), vp]
    lib.stream_vertical_scores.restype = ctypes.c_int
    lib.stream_vertical_scores.argtypes = [P, vp, vp, vp, vp, vp, sz, vp]
    lib.stream_mask_difference.restype = ctypes.c_int
    lib.stream_mask_difference.argtypes = [ctypes.c_int64, ctypes.c_int32, vp, vp, ctypes.c_int32, vp, vp, vp, vp]
    lib.stream_check_device_status.restype = ctypes.c_int
    lib.stream_check_device_status.argtypes = [vp]
    lib.stream_host_staging_bytes.restype = sz
    lib.stream_host_staging_bytes.argtypes = [P]
    lib.stream_run_host.restype = ctypes.c_int
    lib.stream_run_host.argtypes = [P, vp, vp, vp, vp, vp, ctypes.c_float, vp, sz, vp]
    lib.stream_run_host_var.restype = ctypes.c_int
    lib.stream_run_host_var.argtypes = [P, vp, vp, vp, vp, vp, vp, ctypes.c_float, vp, sz, vp]
    _lib = lib
    return lib


def _addr(x):
    if x is None:
        return None
    if isinstance(x, torch.Tensor):
        return x.data_ptr()
    return int(x)


def _stream_handle(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if isinstance(stream, torch.cuda.Stream) else int(stream)


def _raise(status: int):
    if status != STREAM_OK:
        raise StreamError(status, _load().stream_last_error().decode())


# ----------------------------------------------------------------------------------------------
# One-to-one with the C ABI
# ----------------------------------------------------------------------------------------------
def stream_version() -> int:
    return int(_load().stream_version())


def stream_last_error() -> str:
    return _load().stream_last_error().decode()


def stream_workspace_bytes(p: StreamProblem) -> int:
    return int(_load().stream_workspace_bytes(ctypes.byref(p)))


def stream_build_mask(p: StreamProblem, q, k, mask_out, score_out, workspace, workspace_bytes: int, stream=None) -> None:
    _raise(_load().stream_build_mask(ctypes.byref(p), _addr(q), _addr(k), _addr(mask_out), _addr(score_out),
                                     _addr(workspace), workspace_bytes, _stream_handle(stream)))


def stream_build_mask_var(p: StreamProblem, q, k, k_row, mask_out, score_out, workspace, workspace_bytes: int,
                          stream=None) -> None:
    """Mask build with ``k = k_row[query block]`` (device int32 array) instead of one k."""
    _raise(_load().stream_build_mask_var(ctypes.byref(p), _addr(q), _addr(k), _addr(k_row), _addr(mask_out),
                                         _addr(score_out), _addr(workspace), workspace_bytes, _stream_handle(stream)))


def stream_workspace_bytes_multi(p: StreamProblem, n_k: int) -> int:
    """Workspace with which a several-k build scores every (row, block) tile once (0 = invalid)."""
    return int(_load().stream_workspace_bytes_multi(ctypes.byref(p), int(n_k)))


def stream_build_mask_multi(p: StreamProblem, q, k, n_k: int, k_list_host, mask_out, score_out, workspace,
                            workspace_bytes: int, stream=None) -> None:
    """Masks for the ``n_k`` sparsity constants in the HOST int32 array ``k_list_host``, one slab each."""
    _raise(_load().stream_build_mask_multi(ctypes.byref(p), _addr(q), _addr(k), int(n_k), _addr(k_list_host),
                                           _addr(mask_out), _addr(score_out), _addr(workspace), workspace_bytes,
                                           _stream_handle(stream)))


def stream_k_schedule(p: StreamProblem, s: float, k_row_host) -> None:
    """Fills the HOST int32 array ``k_row_host`` ([ceil(T / block_q)]) with the per-row k for sparsity ``s``."""
    _raise(_load().stream_k_schedule(ctypes.byref(p), float(s), _addr(k_row_host)))


def stream_effective_k(T: int, block_q: int, s: float) -> int:
    """k for an effective sparsity ``s`` (the printed formula of Section 4.2, computed by the library)."""
    out = ctypes.c_int32(0)
    _raise(_load().stream_effective_k(int(T), int(block_q), float(s), ctypes.byref(out)))
    return int(out.value)


def stream_selftest_bounded_wait(limit_cycles: int, workspace, workspace_bytes: int, stream=None) -> None:
    """Diagnostic kernel whose bounded wait runs out after ``limit_cycles``; read the outcome with stream_read_stats."""
    _raise(_load().stream_selftest_bounded_wait(int(limit_cycles), _addr(workspace), workspace_bytes, _stream_handle(stream)))


def stream_probe_scratch_bytes() -> int:
    return int(_load().stream_probe_scratch_bytes())


def stream_probe_unit_rates(scratch, scratch_bytes: int, stream=None) -> StreamUnitRates:
    out = StreamUnitRates()
    _raise(_load().stream_probe_unit_rates(_addr(scratch), scratch_bytes, ctypes.byref(out), _stream_handle(stream)))
    return out


def stream_build_mask_static(p: StreamProblem, q, k, mask_out, score_out, stream=None) -> None:
    """Mask build on the library's built-in scratch: no workspace argument, nothing allocated."""
    _raise(_load().stream_build_mask_static(ctypes.byref(p), _addr(q), _addr(k), _addr(mask_out), _addr(score_out),
                                            _stream_handle(stream)))


def stream_sparse_attention(p: StreamProblem, q, k, v, mask, scale: float, out, stream=None) -> None:
    _raise(_load().stream_sparse_attention(ctypes.byref(p), _addr(q), _addr(k), _addr(v), _addr(mask), float(scale),
                                           _addr(out), _stream_handle(stream)))


def stream_read_stats(workspace, stream=None) -> StreamStats:
    st = StreamStats()
    _raise(_load().stream_read_stats(_addr(workspace), ctypes.byref(st), _stream_handle(stream)))
    return st


def stream_vertical_scores(p: StreamProblem, mask, scores, vertical_out, kurtosis_out, workspace, workspace_bytes: int,
                           stream=None) -> None:
    _raise(_load().stream_vertical_scores(ctypes.byref(p), _addr(mask), _addr(scores), _addr(vertical_out),
                                          _addr(kurtosis_out), _addr(workspace), workspace_bytes, _stream_handle(stream)))


def stream_mask_difference(n_rows: int, k_a: int, mask_a, scores_a, k_b: int, mask_b, diff_out, diff_scores_out, stream=None) -> None:
    _raise(_load().stream_mask_difference(n_rows, k_a, _addr(mask_a), _addr(scores_a), k_b, _addr(mask_b), _addr(diff_out),
                                          _addr(diff_scores_out), _stream_handle(stream)))


def stream_check_device_status(stream=None) -> None:
    """Drains the stream; raises if a kernel without a workspace recorded a bounded wait that ran out."""
    _raise(_load().stream_check_device_status(_stream_handle(stream)))


def stream_host_staging_bytes(p: StreamProblem) -> int:
    return int(_load().stream_host_staging_bytes(ctypes.byref(p)))


def stream_run_host(p: StreamProblem, q_host, k_host, v_host, mask_host, out_host, scale: float, staging,
                    staging_bytes: int, stream=None) -> None:
    _raise(_load().stream_run_host(ctypes.byref(p), _addr(q_host), _addr(k_host), _addr(v_host), _addr(mask_host),
                                   _addr(out_host), float(scale), _addr(staging), staging_bytes, _stream_handle(stream)))


def stream_run_host_var(p: StreamProblem, q_host, k_host, v_host, k_row_host, mask_host, out_host, scale: float, staging,
                        staging_bytes: int, stream=None) -> None:
    """The host path with one k per query block (``k_row_host``: HOST int32 array)."""
    _raise(_load().stream_run_host_var(ctypes.byref(p), _addr(q_host), _addr(k_host), _addr(v_host), _addr(k_row_host),
                                       _addr(mask_host), _addr(out_host), float(scale), _addr(staging), staging_bytes,
                                       _stream_handle(stream)))


# ----------------------------------------------------------------------------------------------
# Conveniences: problem struct from tensors, outputs allocated with torch
# ----------------------------------------------------------------------------------------------
def make_problem(q: torch.Tensor, k: torch.Tensor, *, block_q: int, block_k: int, k_top: int, causal: bool = True,
                 impl: str = "auto") -> StreamProblem:
    """Problem struct for q ``[B, H, T, d]`` and k ``[B, G, T, d]`` (any strides with unit innermost)."""
    if q.dim() != 4 or k.dim() != 4 or q.shape[0] != k.shape[0] or q.shape[2:] != k.shape[2:]:
        raise ValueError("q must be [B, H, T, d] and k [B, G, T, d] with matching B, T, d")
    if q.dtype != k.dtype or q.dtype not in (torch.float32, torch.bfloat16):
        raise ValueError("q and k must both be float32 or bfloat16")
    if q.stride(3) != 1 or k.stride(3) != 1:
        raise ValueError("innermost stride must be 1")
    B, H, T, d = q.shape
    return StreamProblem(B, H, k.shape[1], T, d, block_q, block_k, k_top, int(causal),
                         STREAM_F32 if q.dtype == torch.float32 else STREAM_BF16, IMPL[impl],
                         q.stride(0), q.stride(1), q.stride(2), k.stride(0), k.stride(1), k.stride(2))


def n_query_blocks(p: StreamProblem) -> int:
    return -(-p.T // p.block_q)


@dataclass
class MaskResult:
    mask: torch.Tensor            # int32 [B, H, n_query_blocks, k_top]
    scores: torch.Tensor | None   # float32, same shape, if requested
    workspace: torch.Tensor       # holds the counters of this call; see stream_read_stats
    header_bytes: int = 256       # stream_workspace_bytes of the problem: optional per-row counters sit behind it

    def stats(self, stream=None) -> StreamStats:
        return stream_read_stats(self.workspace, stream)

    def row_tiles(self) -> torch.Tensor | None:
        """int32 [B, H, n_query_blocks]: tiles scored per row, if the workspace had room for them."""
        rows = self.mask.shape[0] * self.mask.shape[1] * self.mask.shape[2]
        if self.mask.dim() != 4 or self.workspace.numel() < self.header_bytes + 4 * rows:
            return None
        return self.workspace[self.header_bytes:self.header_bytes + 4 * rows].view(torch.int32).view(self.mask.shape[:3])


def new_workspace(p: StreamProblem, device, row_tiles: bool = False) -> torch.Tensor:
    """Workspace of the size the library asks for; with ``row_tiles`` also room for one counter per row."""
    n = stream_workspace_bytes(p)
    if n == 0:
        raise StreamError(STREAM_ERR_INVALID_ARG, stream_last_error())
    if row_tiles:
        n += 4 * p.batch * p.n_q_heads * n_query_blocks(p)
    return torch.empty(n, dtype=torch.uint8, device=device)


def build_mask(q: torch.Tensor, k: torch.Tensor, *, block_q: int, block_k: int, k_top: int, causal: bool = True,
               impl: str = "auto", want_scores: bool = False, mask_out: torch.Tensor | None = None,
               workspace: torch.Tensor | None = None, k_row: torch.Tensor | None = None, row_tiles: bool = False,
               stream=None) -> MaskResult:
    """Mask of every row. With ``k_row`` (int32 CUDA tensor, one k per query block, see
    :func:`k_schedule`) each row uses its own k and ``k_top`` is the row width. ``row_tiles``
    makes the workspace large enough for the per-row tile counters (``MaskResult.row_tiles()``)."""
    if not q.is_cuda or not k.is_cuda:
        raise ValueError("q and k must be CUDA tensors (there is no CPU path)")
    p = make_problem(q, k, block_q=block_q, block_k=block_k, k_top=k_top, causal=causal, impl=impl)
    shape = (p.batch, p.n_q_heads, n_query_blocks(p), k_top)
    mask = mask_out if mask_out is not None else torch.empty(shape, dtype=torch.int32, device=q.device)
    scores = torch.empty(shape, dtype=torch.float32, device=q.device) if want_scores else None
    ws = workspace if workspace is not None else new_workspace(p, q.device, row_tiles)
    if k_row is None:
        stream_build_mask(p, q, k, mask, scores, ws, ws.numel(), stream)
    else:
        if not k_row.is_cuda or k_row.dtype != torch.int32 or not k_row.is_contiguous() or tuple(k_row.shape) != (shape[2],):
            raise ValueError(f"k_row must be a contiguous int32 CUDA tensor of shape ({shape[2]},)")
        stream_build_mask_var(p, q, k, k_row, mask, scores, ws, ws.numel(), stream)
    return MaskResult(mask, scores, ws, stream_workspace_bytes(p))


def build_masks(q: torch.Tensor, k: torch.Tensor, k_list, *, block_q: int, block_k: int, causal: bool = True,
                impl: str = "auto", want_scores: bool = False, share: bool = True, stream=None) -> MaskResult:
    """Masks for every k in ``k_list`` in one call: ``mask`` is [len(k_list), B, H, rows, max(k_list)].
    ``share=False`` gives the library only the small workspace (the tensor-core kernel then runs
    once per k and does not reuse tile scores between them)."""
    if not q.is_cuda or not k.is_cuda:
        raise ValueError("q and k must be CUDA tensors (there is no CPU path)")
    ks = torch.tensor(list(k_list), dtype=torch.int32)
    p = make_problem(q, k, block_q=block_q, block_k=block_k, k_top=int(ks.max()), causal=causal, impl=impl)
    shape = (len(ks), p.batch, p.n_q_heads, n_query_blocks(p), p.k_top)
    mask = torch.empty(shape, dtype=torch.int32, device=q.device)
    scores = torch.empty(shape, dtype=torch.float32, device=q.device) if want_scores else None
    n_ws = stream_workspace_bytes_multi(p, len(ks)) if share else stream_workspace_bytes(p)
    if n_ws == 0:
        raise StreamError(STREAM_ERR_INVALID_ARG, stream_last_error())
    ws = torch.empty(n_ws, dtype=torch.uint8, device=q.device)
    stream_build_mask_multi(p, q, k, len(ks), ks.data_ptr(), mask, scores, ws, ws.numel(), stream)
    return MaskResult(mask, scores, ws)


def k_schedule(p: StreamProblem, s: float) -> torch.Tensor:
    """Host int32 tensor [ceil(T / block_q)]: k per query block for an effective sparsity ``s``
    (the formula of :func:`effective_k` applied to each row's own number of allowed key blocks,
    clamped to ``1 .. p.k_top``). Move it to the device for :func:`build_mask`."""
    out = torch.empty((n_query_blocks(p),), dtype=torch.int32)
    stream_k_schedule(p, s, out.data_ptr())
    return out


def sparse_attention(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, mask: torch.Tensor, *, block_q: int,
                     block_k: int, causal: bool = True, scale: float = 0.0, impl: str = "auto",
                     out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    if not (q.is_cuda and k.is_cuda and v.is_cuda and mask.is_cuda):
        raise ValueError("q, k, v and mask must be CUDA tensors (there is no CPU path)")
    if v.shape != k.shape or v.stride() != k.stride() or v.dtype != k.dtype:
        raise ValueError("v must have k's shape, strides and dtype")
    if mask.dtype != torch.int32 or not mask.is_contiguous():
        raise ValueError("mask must be a contiguous int32 tensor")
    p = make_problem(q, k, block_q=block_q, block_k=block_k, k_top=mask.shape[-1], causal=causal, impl=impl)
    if tuple(mask.shape) != (p.batch, p.n_q_heads, n_query_blocks(p), mask.shape[-1]):
        raise ValueError("mask must be [B, H, ceil(T / block_q), k_top]")
    if out is None:
        out = torch.empty((p.batch, p.n_q_heads, p.T, p.d), dtype=q.dtype, device=q.device)
    stream_sparse_attention(p, q, k, v, mask, scale, out, stream)
    return out


def run_host(q_host: torch.Tensor, k_host: torch.Tensor, v_host: torch.Tensor, mask_host: torch.Tensor,
             out_host: torch.Tensor, staging: torch.Tensor, *, block_q: int, block_k: int, k_top: int,
             causal: bool = True, scale: float = 0.0, impl: str = "auto", k_row: torch.Tensor | None = None, stream=None) -> None:
    """Whole path from (pinned) host tensors through a caller-provided device staging buffer. With
    ``k_row`` (HOST int32 tensor, one k per query block) the mask is the variable-k build."""
    if q_host.is_cuda or not staging.is_cuda:
        raise ValueError("q/k/v/mask/out live on the host, staging on the device")
    p = make_problem(q_host, k_host, block_q=block_q, block_k=block_k, k_top=k_top, causal=causal, impl=impl)
    if k_row is None:
        stream_run_host(p, q_host, k_host, v_host, mask_host, out_host, scale, staging, staging.numel(), stream)
    else:
        if k_row.is_cuda or k_row.dtype != torch.int32 or not k_row.is_contiguous() or k_row.numel() != n_query_blocks(p):
            raise ValueError("k_row must be a contiguous int32 HOST tensor with one entry per query block")
        stream_run_host_var(p, q_host, k_host, v_host, k_row, mask_host, out_host, scale, staging, staging.numel(), stream)


def vertical_scores(p: StreamProblem, mask: torch.Tensor, scores: torch.Tensor | None = None, stream=None):
    """(vertical [B, H, ceil(T / block_k)], kurtosis [B, H]) of a mask, binary or weighted by ``scores``."""
    if not mask.is_cuda or mask.dtype != torch.int32 or not mask.is_contiguous():
        raise ValueError("mask must be a contiguous int32 CUDA tensor")
    if scores is not None and (scores.shape != mask.shape or scores.dtype != torch.float32 or not scores.is_contiguous()):
        raise ValueError("scores must be a contiguous float32 tensor of the mask's shape")
    n_kb = -(-p.T // p.block_k)
    vert = torch.empty((p.batch, p.n_q_heads, n_kb), dtype=torch.float32, device=mask.device)
    kurt = torch.empty((p.batch, p.n_q_heads), dtype=torch.float32, device=mask.device)
    ws = new_workspace(p, mask.device)
    stream_vertical_scores(p, mask, scores, vert, kurt, ws, ws.numel(), stream)
    stream_read_stats(ws, stream)
    return vert, kurt


def mask_difference(mask_a: torch.Tensor, mask_b: torch.Tensor, scores_a: torch.Tensor | None = None, stream=None):
    """Row-wise ``mask_a`` minus ``mask_b`` (same leading shape, last dims k_a and k_b); returns (diff, scores or None)."""
    if mask_a.shape[:-1] != mask_b.shape[:-1] or mask_a.dtype != torch.int32 or mask_b.dtype != torch.int32:
        raise ValueError("masks must be int32 with the same leading shape")
    if not (mask_a.is_cuda and mask_b.is_cuda and mask_a.is_contiguous() and mask_b.is_contiguous()):
        raise ValueError("masks must be contiguous CUDA tensors")
    if scores_a is not None and (scores_a.shape != mask_a.shape or scores_a.dtype != torch.float32 or not scores_a.is_contiguous()):
        raise ValueError("scores_a must be a contiguous float32 tensor of mask_a's shape")
    diff = torch.empty_like(mask_a)
    dsc = torch.empty_like(scores_a) if scores_a is not None else None
    n = mask_a.numel() // mask_a.shape[-1]
    stream_mask_difference(n, mask_a.shape[-1], mask_a, scores_a, mask_b.shape[-1], mask_b, diff, dsc, stream)
    return diff, dsc


def effective_k(T: int, block_q: int, s: float) -> int:
    """Sparsity constant for an effective sparsity ``s`` in [0, 1] (Section 4.2 of the paper), as
    computed by the library's ``stream_effective_k``."""
    return stream_effective_k(T, block_q, s)


def probe_unit_rates(device="cuda", stream=None) -> StreamUnitRates:
    """TMA gather rate and tensor-core instruction time of the current device (``stream_probe_unit_rates``)."""
    n = stream_probe_scratch_bytes()
    if n == 0:
        raise RuntimeError("no CUDA device to probe")
    scratch = torch.empty(n, dtype=torch.uint8, device=device)
    return stream_probe_unit_rates(scratch, n, stream)
