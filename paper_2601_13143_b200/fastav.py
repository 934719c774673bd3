"""ctypes binding of ``libfastav.so``: the same entry points as ``include/fastav.h``, taking torch
tensors.  Argument marshalling only -- every step of the prune path runs in the library's CUDA
kernels; torch supplies device memory and streams.  If the library cannot be loaded this module
raises: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

from . import build as _build

FASTAV_CAUSAL = 1
FASTAV_PROTECT_QUERY_ROWS = 2
FASTAV_KEEP_IDX_GLOBAL = 4
FASTAV_SELECT_LOWEST = 0x800
FASTAV_CHAIN_CALLS = 0x1000

FASTAV_SCORE_PATH_GENERIC = 0x100
FASTAV_SCORE_PATH_NARROW = 0x200
FASTAV_SCORE_PATH_WIDE = 0x300
FASTAV_COMPACT_PATH_LOADSTORE = 0x400

FASTAV_DEV_K_CLAMPED = 1
FASTAV_DEV_PROTECT_OVERFLOW = 2
FASTAV_DEV_WAIT_EXPIRED = 4
FASTAV_DEV_BAD_INDEX = 8
FASTAV_DEV_SHAPE_MISMATCH = 16
FASTAV_DEV_SLOW_PATH = 32

FASTAV_OK = 0
FASTAV_ERR_INVALID_ARG = -1
FASTAV_ERR_UNSUPPORTED = -2
FASTAV_ERR_WORKSPACE = -3
FASTAV_ERR_CUDA = -4
FASTAV_ERR_TIMEOUT = -5

EXPORTS = ("fastav_version", "fastav_status_string", "fastav_last_cuda_error", "fastav_workspace_bytes",
           "fastav_score", "fastav_lse", "fastav_select", "fastav_compact", "fastav_prune", "fastav_host_arena_bytes",
           "fastav_prune_host", "fastav_kernel_launches", "fastav_select_noalloc", "fastav_select_mask", "fastav_selftest_bounded_wait",
           "fastav_rollout_state_bytes", "fastav_rollout_workspace_bytes", "fastav_rollout_begin", "fastav_rollout_layer",
           "fastav_rollout_read", "fastav_rollout_threshold")


class fastav_params(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32),
        ("total_tokens", ctypes.c_int32), ("max_seqlen", ctypes.c_int32),
        ("total_q", ctypes.c_int32), ("max_qlen", ctypes.c_int32),
        ("total_keep", ctypes.c_int32), ("max_keep", ctypes.c_int32),
        ("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
        ("hidden", ctypes.c_int32),
        ("q_stride_tok", ctypes.c_int64), ("q_stride_head", ctypes.c_int64),
        ("k_stride_tok", ctypes.c_int64), ("k_stride_head", ctypes.c_int64),
        ("v_stride_tok", ctypes.c_int64), ("v_stride_head", ctypes.c_int64),
        ("ko_stride_tok", ctypes.c_int64), ("ko_stride_head", ctypes.c_int64),
        ("vo_stride_tok", ctypes.c_int64), ("vo_stride_head", ctypes.c_int64),
        ("softmax_scale", ctypes.c_float),
        ("flags", ctypes.c_uint32),
    ]


class FastavError(RuntimeError):
    def __init__(self, status: int, where: str):
        lib = library()
        text = lib.fastav_status_string(status).decode()
        if status == FASTAV_ERR_CUDA:
            text += ": " + lib.fastav_last_cuda_error().decode()
        super().__init__(f"{where} failed with status {status} ({text})")
        self.status = status


_lib = None


def library_path() -> str:
    return os.environ.get("FASTAV_LIBRARY", _build.LIB_PATH)


def library() -> ctypes.CDLL:
    """Load the CUDA library (raises OSError if it has not been built)."""
    global _lib
    if _lib is None:
        path = library_path()
        if not os.path.exists(path):
            raise OSError(f"{path} is missing: build it with `python -m paper_2601_13143_b200.build` "
                          "(there is no fallback implementation)")
        lib = ctypes.CDLL(path)
        vp, i32p = ctypes.c_void_p, ctypes.c_void_p
        pp = ctypes.POINTER(fastav_params)
        lib.fastav_version.restype = ctypes.c_int32
        lib.fastav_status_string.restype = ctypes.c_char_p
        lib.fastav_status_string.argtypes = [ctypes.c_int32]
        lib.fastav_last_cuda_error.restype = ctypes.c_char_p
        lib.fastav_workspace_bytes.restype = ctypes.c_int32
        lib.fastav_workspace_bytes.argtypes = [pp, ctypes.POINTER(ctypes.c_size_t)]
        lib.fastav_score.restype = ctypes.c_int32
        lib.fastav_score.argtypes = [pp, vp, i32p, i32p, vp, i32p, vp, vp, vp, ctypes.c_size_t, i32p, vp]
        lib.fastav_lse.restype = ctypes.c_int32
        lib.fastav_lse.argtypes = [pp, vp, i32p, i32p, vp, i32p, vp, vp, ctypes.c_size_t, i32p, vp]
        lib.fastav_select.restype = ctypes.c_int32
        lib.fastav_select.argtypes = [pp, vp, i32p, i32p, vp, i32p, i32p, i32p, i32p, vp, ctypes.c_size_t, i32p, vp]
        lib.fastav_compact.restype = ctypes.c_int32
        lib.fastav_compact.argtypes = [pp, i32p, i32p, i32p, vp, vp, i32p, i32p, vp, vp, vp, vp, i32p, vp]
        lib.fastav_prune.restype = ctypes.c_int32
        lib.fastav_prune.argtypes = [pp, vp, i32p, i32p, vp, vp, i32p, vp, i32p, vp, vp, i32p, vp, i32p, i32p, vp, i32p,
                                     vp, vp, vp, ctypes.c_size_t, i32p, vp]
        lib.fastav_host_arena_bytes.restype = ctypes.c_int32
        lib.fastav_host_arena_bytes.argtypes = [pp, ctypes.POINTER(ctypes.c_size_t)]
        lib.fastav_prune_host.restype = ctypes.c_int32
        lib.fastav_prune_host.argtypes = [pp, vp, i32p, i32p, vp, vp, i32p, vp, i32p, vp, vp, i32p, vp, i32p, i32p, vp, i32p,
                                          vp, vp, i32p, vp, ctypes.c_size_t, vp]
        lib.fastav_kernel_launches.restype = ctypes.c_int64
        lib.fastav_select_mask.restype = ctypes.c_int32
        lib.fastav_select_mask.argtypes = [pp, vp, i32p, i32p, i32p, vp, ctypes.c_size_t, i32p, vp]
        lib.fastav_selftest_bounded_wait.restype = ctypes.c_int32
        lib.fastav_selftest_bounded_wait.argtypes = [ctypes.c_int32, i32p, vp]
        lib.fastav_select_noalloc.restype = ctypes.c_int32
        lib.fastav_select_noalloc.argtypes = [pp, vp, i32p, i32p, vp, i32p, i32p, i32p, i32p, i32p, vp]
        szp = ctypes.POINTER(ctypes.c_size_t)
        lib.fastav_rollout_state_bytes.restype = ctypes.c_int32
        lib.fastav_rollout_state_bytes.argtypes = [ctypes.c_int32, szp]
        lib.fastav_rollout_workspace_bytes.restype = ctypes.c_int32
        lib.fastav_rollout_workspace_bytes.argtypes = [pp, szp]
        lib.fastav_rollout_begin.restype = ctypes.c_int32
        lib.fastav_rollout_begin.argtypes = [ctypes.c_int32, vp, ctypes.c_size_t, vp]
        lib.fastav_rollout_layer.restype = ctypes.c_int32
        lib.fastav_rollout_layer.argtypes = [pp, vp, vp, vp, ctypes.c_float, ctypes.c_int32, vp, ctypes.c_size_t, vp, vp,
                                             ctypes.c_size_t, i32p, vp]
        lib.fastav_rollout_read.restype = ctypes.c_int32
        lib.fastav_rollout_read.argtypes = [ctypes.c_int32, ctypes.c_int32, vp, ctypes.c_size_t, vp, vp, vp]
        lib.fastav_rollout_threshold.restype = ctypes.c_int32
        lib.fastav_rollout_threshold.argtypes = [ctypes.c_int32, vp, ctypes.c_float, vp, vp, i32p, vp]
        _lib = lib
    return _lib


def _p(t: torch.Tensor | None):
    """Device pointer of a tensor (None -> NULL)."""
    if t is None:
        return None
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _strides3(t: torch.Tensor | None, heads: int, dim: int) -> tuple[int, int]:
    if t is None:
        return heads * dim, dim
    if t.dim() != 3 or t.stride(2) != 1:
        raise ValueError("expected a [tokens, heads, head_dim] tensor with a contiguous last dimension")
    return t.stride(0), t.stride(1)


def make_params(*, batch, total_tokens, max_seqlen, total_q, max_qlen, total_keep, max_keep, num_q_heads, num_kv_heads,
                head_dim, hidden, q=None, k=None, v=None, k_out=None, v_out=None, softmax_scale=0.0, flags=0) -> fastav_params:
    """Fill a ``fastav_params`` from host scalars and (optionally) the tensors whose strides it records."""
    p = fastav_params()
    p.batch, p.total_tokens, p.max_seqlen = batch, total_tokens, max_seqlen
    p.total_q, p.max_qlen, p.total_keep, p.max_keep = total_q, max_qlen, total_keep, max_keep
    p.num_q_heads, p.num_kv_heads, p.head_dim, p.hidden = num_q_heads, num_kv_heads, head_dim, hidden
    p.q_stride_tok, p.q_stride_head = _strides3(q, num_q_heads, head_dim)
    p.k_stride_tok, p.k_stride_head = _strides3(k, num_kv_heads, head_dim)
    p.v_stride_tok, p.v_stride_head = _strides3(v, num_kv_heads, head_dim)
    p.ko_stride_tok, p.ko_stride_head = _strides3(k_out, num_kv_heads, head_dim)
    p.vo_stride_tok, p.vo_stride_head = _strides3(v_out, num_kv_heads, head_dim)
    p.softmax_scale, p.flags = float(softmax_scale), int(flags)
    return p


def _check(status: int, where: str) -> None:
    if status != FASTAV_OK:
        raise FastavError(status, where)


def fastav_version() -> int:
    return int(library().fastav_version())


def fastav_status_string(status: int) -> str:
    return library().fastav_status_string(status).decode()


def fastav_workspace_bytes(params: fastav_params) -> int:
    out = ctypes.c_size_t(0)
    _check(library().fastav_workspace_bytes(ctypes.byref(params), ctypes.byref(out)), "fastav_workspace_bytes")
    return int(out.value)


def _ws(workspace: torch.Tensor | None):
    return (_p(workspace), ctypes.c_size_t(0 if workspace is None else workspace.numel() * workspace.element_size()))


def fastav_score(params, q, q_idx, cu_qlens, k, cu_seqlens, scores_out, workspace, device_status=None, stream=None,
                 lse_opt=None) -> None:
    ws, ws_bytes = _ws(workspace)
    _check(library().fastav_score(ctypes.byref(params), _p(q), _p(q_idx), _p(cu_qlens), _p(k), _p(cu_seqlens), _p(lse_opt),
                                  _p(scores_out), ws, ws_bytes, _p(device_status), _stream(stream)), "fastav_score")


def fastav_lse(params, q, q_idx, cu_qlens, k, cu_seqlens, lse_out, workspace, device_status=None, stream=None) -> None:
    """Natural-log log-sum-exp of every scored row's logits per head, [total_q, Hq] (the first sweep alone)."""
    ws, ws_bytes = _ws(workspace)
    _check(library().fastav_lse(ctypes.byref(params), _p(q), _p(q_idx), _p(cu_qlens), _p(k), _p(cu_seqlens), _p(lse_out), ws,
                                ws_bytes, _p(device_status), _stream(stream)), "fastav_lse")


def fastav_select(params, scores, cu_seqlens, keep_counts, protect_opt, q_idx, cu_qlens, keep_idx_out, cu_keep_out, workspace,
                  device_status=None, stream=None) -> None:
    ws, ws_bytes = _ws(workspace)
    _check(library().fastav_select(ctypes.byref(params), _p(scores), _p(cu_seqlens), _p(keep_counts), _p(protect_opt),
                                   _p(q_idx), _p(cu_qlens), _p(keep_idx_out), _p(cu_keep_out), ws, ws_bytes,
                                   _p(device_status), _stream(stream)), "fastav_select")


def fastav_select_mask(params, keep_mask, cu_seqlens, keep_idx_out, cu_keep_out, workspace, device_status=None, stream=None) -> None:
    """Keep list of a rule-given keep mask (the paper's positional global stage)."""
    ws, ws_bytes = _ws(workspace)
    _check(library().fastav_select_mask(ctypes.byref(params), _p(keep_mask), _p(cu_seqlens), _p(keep_idx_out), _p(cu_keep_out),
                                        ws, ws_bytes, _p(device_status), _stream(stream)), "fastav_select_mask")


def fastav_selftest_bounded_wait(limit_ms: int, device_status, stream=None) -> None:
    """Enqueue the bounded-wait self-test (a wait that cannot succeed; it must end with the error bit set)."""
    _check(library().fastav_selftest_bounded_wait(int(limit_ms), _p(device_status), _stream(stream)), "fastav_selftest_bounded_wait")


# ---- attention rollout (Section 2.1, Eq. 2-3): argument marshalling only ------------------------------------

ROLLOUT_MAX_TOKENS = 32768


def fastav_rollout_state_bytes(n: int) -> int:
    out = ctypes.c_size_t(0)
    _check(library().fastav_rollout_state_bytes(int(n), ctypes.byref(out)), "fastav_rollout_state_bytes")
    return int(out.value)


def fastav_rollout_workspace_bytes(params: fastav_params) -> int:
    out = ctypes.c_size_t(0)
    _check(library().fastav_rollout_workspace_bytes(ctypes.byref(params), ctypes.byref(out)), "fastav_rollout_workspace_bytes")
    return int(out.value)


def fastav_rollout_begin(n: int, state, stream=None) -> None:
    """R <- I in the caller's state buffer."""
    st, st_bytes = _ws(state)
    _check(library().fastav_rollout_begin(int(n), st, st_bytes, _stream(stream)), "fastav_rollout_begin")


def fastav_rollout_layer(params, q, k, alpha: float, layer_index: int, state, workspace, lse_opt=None, map_out_opt=None,
                         device_status=None, stream=None) -> None:
    """One layer of Eq. 3: R <- (alpha A^l + (1 - alpha) I) R with A^l the head-mean attention map of (q, k)."""
    st, st_bytes = _ws(state)
    ws, ws_bytes = _ws(workspace)
    _check(library().fastav_rollout_layer(ctypes.byref(params), _p(q), _p(k), _p(lse_opt), float(alpha), int(layer_index), st,
                                          st_bytes, _p(map_out_opt), ws, ws_bytes, _p(device_status), _stream(stream)),
           "fastav_rollout_layer")


def fastav_rollout_read(n: int, layers_applied: int, state, importance_out, rollout_out_opt=None, stream=None) -> None:
    st, st_bytes = _ws(state)
    _check(library().fastav_rollout_read(int(n), int(layers_applied), st, st_bytes, _p(importance_out), _p(rollout_out_opt),
                                         _stream(stream)), "fastav_rollout_read")


def fastav_rollout_threshold(n: int, importance, threshold: float, protect_opt, keep_mask_out, cut_out, stream=None) -> None:
    _check(library().fastav_rollout_threshold(int(n), _p(importance), float(threshold), _p(protect_opt), _p(keep_mask_out),
                                              _p(cut_out), _stream(stream)), "fastav_rollout_threshold")


NOALLOC_MAX_TOKENS = 1 << 20


def fastav_select_noalloc(params, scores, cu_seqlens, keep_counts, protect_opt, q_idx, cu_qlens, keep_idx_out, cu_keep_out,
                          device_status=None, stream=None) -> None:
    """``fastav_select`` for callers that cannot allocate device memory: no workspace argument, the
    keys live in an array inside the library (at most ``NOALLOC_MAX_TOKENS`` tokens per call; calls
    that overlap on the GPU race on it)."""
    _check(library().fastav_select_noalloc(ctypes.byref(params), _p(scores), _p(cu_seqlens), _p(keep_counts), _p(protect_opt),
                                           _p(q_idx), _p(cu_qlens), _p(keep_idx_out), _p(cu_keep_out), _p(device_status),
                                           _stream(stream)), "fastav_select_noalloc")


def fastav_compact(params, keep_idx, cu_keep, cu_seqlens, hidden_in=None, hidden_out=None, pos_in=None, pos_out=None,
                   k_in=None, k_out=None, v_in=None, v_out=None, device_status=None, stream=None) -> None:
    _check(library().fastav_compact(ctypes.byref(params), _p(keep_idx), _p(cu_keep), _p(cu_seqlens), _p(hidden_in),
                                    _p(hidden_out), _p(pos_in), _p(pos_out), _p(k_in), _p(k_out), _p(v_in), _p(v_out),
                                    _p(device_status), _stream(stream)), "fastav_compact")


def fastav_prune(params, q, q_idx, cu_qlens, k, v, cu_seqlens, keep_counts, protect_opt, hidden_in, pos_in, scores_out,
                 keep_idx_out, cu_keep_out, hidden_out, pos_out, k_out, v_out, workspace, device_status=None,
                 stream=None, lse_opt=None) -> None:
    ws, ws_bytes = _ws(workspace)
    _check(library().fastav_prune(ctypes.byref(params), _p(q), _p(q_idx), _p(cu_qlens), _p(k), _p(v), _p(cu_seqlens),
                                  _p(lse_opt), _p(keep_counts), _p(protect_opt), _p(hidden_in), _p(pos_in), _p(scores_out),
                                  _p(keep_idx_out), _p(cu_keep_out), _p(hidden_out), _p(pos_out), _p(k_out), _p(v_out),
                                  ws, ws_bytes, _p(device_status), _stream(stream)), "fastav_prune")


def fastav_kernel_launches() -> int:
    return int(library().fastav_kernel_launches())


def fastav_host_arena_bytes(params: fastav_params) -> int:
    out = ctypes.c_size_t(0)
    _check(library().fastav_host_arena_bytes(ctypes.byref(params), ctypes.byref(out)), "fastav_host_arena_bytes")
    return int(out.value)


def fastav_prune_host(params, q, q_idx, cu_qlens, k, v, cu_seqlens, keep_counts, protect_opt, hidden_in, pos_in, scores_out,
                      keep_idx_out, cu_keep_out, hidden_out, pos_out, k_out, v_out, status_out, device_arena,
                      stream=None, lse_opt=None) -> None:
    """All tensors are HOST tensors (pinned for asynchronous copies) except ``device_arena``."""
    for t in (q, q_idx, cu_qlens, k, v, cu_seqlens, lse_opt, keep_counts, protect_opt, hidden_in, pos_in, scores_out, keep_idx_out,
              cu_keep_out, hidden_out, pos_out, k_out, v_out, status_out):
        if t is not None and (t.is_cuda or not t.is_contiguous()):
            raise ValueError("fastav_prune_host takes contiguous host tensors")
    _check(library().fastav_prune_host(ctypes.byref(params), _p(q), _p(q_idx), _p(cu_qlens), _p(k), _p(v), _p(cu_seqlens),
                                       _p(lse_opt), _p(keep_counts), _p(protect_opt), _p(hidden_in), _p(pos_in), _p(scores_out),
                                       _p(keep_idx_out), _p(cu_keep_out), _p(hidden_out), _p(pos_out), _p(k_out), _p(v_out),
                                       _p(status_out), _p(device_arena),
                                       ctypes.c_size_t(device_arena.numel() * device_arena.element_size()),
                                       _stream(stream)), "fastav_prune_host")


# ---- convenience: buffers for one prune call --------------------------------------------------

@dataclass
class PruneBuffers:
    """Device inputs, outputs and workspace of one prune call (allocated with torch, filled by the
    library)."""
    params: fastav_params
    q: torch.Tensor
    q_idx: torch.Tensor
    cu_qlens: torch.Tensor
    k: torch.Tensor
    v: torch.Tensor | None
    cu_seqlens: torch.Tensor
    keep_counts: torch.Tensor
    hidden: torch.Tensor | None
    pos: torch.Tensor | None
    protect: torch.Tensor | None
    scores: torch.Tensor
    keep_idx: torch.Tensor
    cu_keep: torch.Tensor
    hidden_out: torch.Tensor | None
    pos_out: torch.Tensor | None
    k_out: torch.Tensor | None
    v_out: torch.Tensor | None
    workspace: torch.Tensor
    device_status: torch.Tensor

    def prune(self, stream=None, lse_opt=None) -> None:
        fastav_prune(self.params, self.q, self.q_idx, self.cu_qlens, self.k, self.v, self.cu_seqlens, self.keep_counts,
                     self.protect, self.hidden, self.pos, self.scores, self.keep_idx, self.cu_keep, self.hidden_out,
                     self.pos_out, self.k_out, self.v_out, self.workspace, self.device_status, stream, lse_opt=lse_opt)

    def score(self, stream=None) -> None:
        fastav_score(self.params, self.q, self.q_idx, self.cu_qlens, self.k, self.cu_seqlens, self.scores, self.workspace,
                     self.device_status, stream)

    def select(self, stream=None) -> None:
        fastav_select(self.params, self.scores, self.cu_seqlens, self.keep_counts, self.protect, self.q_idx, self.cu_qlens,
                      self.keep_idx, self.cu_keep, self.workspace, self.device_status, stream)

    def compact(self, stream=None) -> None:
        fastav_compact(self.params, self.keep_idx, self.cu_keep, self.cu_seqlens, self.hidden, self.hidden_out, self.pos,
                       self.pos_out, self.k, self.k_out, self.v, self.v_out, self.device_status, stream)


def make_buffers(*, q, q_idx, cu_qlens, k, v, cu_seqlens, keep_counts, hidden=None, pos=None, protect=None,
                 softmax_scale=0.0, flags=FASTAV_CAUSAL | FASTAV_PROTECT_QUERY_ROWS, lens=None, rows=None,
                 keeps=None) -> PruneBuffers:
    """Allocate outputs and workspace for device inputs.  ``lens``/``rows``/``keeps`` are the host
    copies of the per-sequence token, scored-row and keep counts (taken from the device tensors when
    omitted, which synchronises)."""
    dev = k.device
    if lens is None:
        lens = (cu_seqlens[1:] - cu_seqlens[:-1]).tolist()
    if rows is None:
        rows = (cu_qlens[1:] - cu_qlens[:-1]).tolist()
    if keeps is None:
        keeps = keep_counts.tolist()
    keeps = [min(max(int(c), 0), int(n)) for c, n in zip(keeps, lens)]
    total, total_keep = int(sum(lens)), int(sum(keeps))
    heads_q, dim = q.shape[1], q.shape[2]
    heads_kv = k.shape[1]
    hid = 0 if hidden is None else hidden.shape[1]
    k_out = torch.empty((total_keep, heads_kv, dim), dtype=k.dtype, device=dev)
    v_out = None if v is None else torch.empty((total_keep, heads_kv, dim), dtype=v.dtype, device=dev)
    params = make_params(batch=len(lens), total_tokens=total, max_seqlen=max(lens) if lens else 0, total_q=int(sum(rows)),
                         max_qlen=max(rows) if rows else 0, total_keep=total_keep, max_keep=max(keeps) if keeps else 0,
                         num_q_heads=heads_q, num_kv_heads=heads_kv, head_dim=dim, hidden=hid, q=q, k=k, v=v, k_out=k_out,
                         v_out=v_out, softmax_scale=softmax_scale, flags=flags)
    ws_bytes = fastav_workspace_bytes(params)
    return PruneBuffers(
        params=params, q=q, q_idx=q_idx, cu_qlens=cu_qlens, k=k, v=v, cu_seqlens=cu_seqlens, keep_counts=keep_counts,
        hidden=hidden, pos=pos, protect=protect,
        scores=torch.empty(total, dtype=torch.float32, device=dev),
        keep_idx=torch.empty(max(total_keep, 1), dtype=torch.int32, device=dev),
        cu_keep=torch.empty(len(lens) + 1, dtype=torch.int32, device=dev),
        hidden_out=None if hidden is None else torch.empty((total_keep, hid), dtype=hidden.dtype, device=dev),
        pos_out=None if pos is None else torch.empty(total_keep, dtype=torch.int32, device=dev),
        k_out=k_out, v_out=v_out,
        workspace=torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device=dev),
        device_status=torch.zeros(1, dtype=torch.int32, device=dev))
