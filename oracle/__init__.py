"""CPU oracle for the FastAV prune step.  TEST INFRASTRUCTURE ONLY.

Thin ctypes loader around ``fastav_oracle.c`` (plain C, double precision) plus the
closed-form FLOPs accounting in ``flops.py``.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this package; the CUDA library and its Python
binding never do, and share no code with it.

Arrays are numpy: bf16 tensors travel as ``uint16`` bit patterns, indices as ``int32``.
Every function follows Section 2.2 of the paper ("Fine pruning", Eq. 4) as read in the
C file's header.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fastav_oracle.c")
_LIB = os.path.join(_HERE, "libfastav_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP on).  Building the checker is not using it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        lib.oracle_max_threads.restype = ctypes.c_int
        lib.oracle_score.restype = ctypes.c_int
        lib.oracle_select.restype = ctypes.c_int
        lib.oracle_compact.restype = None
        _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else ctypes.c_void_p(a.ctypes.data)


def _i32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _u16_strided(a, name):
    """Accept a [tokens, heads, dim] uint16 array whose last axis is contiguous."""
    a = np.asarray(a)
    if a.dtype != np.uint16 or a.ndim != 3:
        raise TypeError(f"{name}: expected a 3-d uint16 (bf16 bits) array")
    if a.size == 0:  # numpy reports arbitrary strides for empty arrays
        return a, a.shape[1] * a.shape[2], a.shape[2]
    if a.strides[2] != 2 or a.strides[0] % 2 or a.strides[1] % 2:
        raise ValueError(f"{name}: last axis must be contiguous")
    return a, a.strides[0] // 2, a.strides[1] // 2


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def score(q, k, cu_seqlens, cu_qlens, q_idx, scale, causal, nthreads: int = 0):
    """Eq. 4 importance scores, float64 [N].

    q: [sum R, Hq, d] bf16 bits, k: [N, Hkv, d] bf16 bits; q_idx: sequence-local index of
    each scored row's token.  ``scale`` is the softmax scale (1.0 reproduces Eq. 4 as
    printed, 1/sqrt(d) gives the model's attention weights).
    """
    lib = _load()
    q, qs_t, qs_h = _u16_strided(q, "q")
    k, ks_t, ks_h = _u16_strided(k, "k")
    cu_seqlens, cu_qlens, q_idx = _i32(cu_seqlens), _i32(cu_qlens), _i32(q_idx)
    batch = len(cu_seqlens) - 1
    if q.shape[2] != k.shape[2] or q.shape[1] % k.shape[1]:
        raise ValueError("head shapes do not match")
    out = np.zeros(int(cu_seqlens[-1]), dtype=np.float64)
    rc = lib.oracle_score(
        ctypes.c_int(batch), _ptr(cu_seqlens), _ptr(cu_qlens), _ptr(q_idx),
        _ptr(q), ctypes.c_int64(qs_t), ctypes.c_int64(qs_h),
        _ptr(k), ctypes.c_int64(ks_t), ctypes.c_int64(ks_h),
        ctypes.c_int(q.shape[1]), ctypes.c_int(k.shape[1]), ctypes.c_int(q.shape[2]),
        ctypes.c_double(float(scale)), ctypes.c_int(1 if causal else 0), _ptr(out), ctypes.c_int(nthreads))
    if rc != 0:
        raise MemoryError("oracle_score: allocation failed")
    return out


def select(scores, cu_seqlens, keep_counts, protect_mask=None, protect_rows=False, q_idx=None,
           cu_qlens=None, global_index=False):
    """Keep the k_b best tokens per sequence (score descending, index ascending; protected
    tokens first).  ``scores`` is rounded to float32 before ranking, the precision the CUDA
    selector decides in.  Returns (keep_idx ascending per sequence, cu_keep)."""
    lib = _load()
    scores = np.ascontiguousarray(np.asarray(scores, dtype=np.float32))
    cu_seqlens, keep_counts = _i32(cu_seqlens), _i32(keep_counts)
    batch = len(cu_seqlens) - 1
    lens = np.diff(cu_seqlens)
    total = int(np.clip(keep_counts, 0, lens).sum())
    keep_idx = np.zeros(max(total, 1), dtype=np.int32)
    cu_keep = np.zeros(batch + 1, dtype=np.int32)
    if protect_mask is not None:
        protect_mask = np.ascontiguousarray(np.asarray(protect_mask, dtype=np.uint8))
    if protect_rows:
        q_idx, cu_qlens = _i32(q_idx), _i32(cu_qlens)
    rc = lib.oracle_select(
        ctypes.c_int(batch), _ptr(cu_seqlens), _ptr(scores), _ptr(keep_counts), _ptr(protect_mask),
        ctypes.c_int(1 if protect_rows else 0), _ptr(q_idx) if protect_rows else None,
        _ptr(cu_qlens) if protect_rows else None, ctypes.c_int(1 if global_index else 0),
        _ptr(keep_idx), _ptr(cu_keep))
    if rc != 0:
        raise MemoryError("oracle_select: allocation failed")
    return keep_idx[:total], cu_keep


def select_mask(keep_mask, cu_seqlens, global_index=False):
    """Keep list of a rule-given mask (Section 2.2, "Global pruning": the deployed global stage keeps
    fixed positions): the kept tokens of each sequence in ascending order.  Returns (keep_idx, cu_keep)."""
    keep_mask = np.asarray(keep_mask)
    cu_seqlens = _i32(cu_seqlens)
    parts, cu_keep = [], [0]
    for b in range(len(cu_seqlens) - 1):
        kept = [j for j in range(int(cu_seqlens[b + 1] - cu_seqlens[b])) if keep_mask[cu_seqlens[b] + j] != 0]
        parts.append(np.asarray(kept, dtype=np.int32) + (int(cu_seqlens[b]) if global_index else 0))
        cu_keep.append(cu_keep[-1] + len(kept))
    return (np.concatenate(parts) if parts else np.zeros(0, dtype=np.int32)).astype(np.int32), np.asarray(cu_keep, dtype=np.int32)


def compact(keep_idx, cu_keep, cu_seqlens, hidden=None, pos=None, k=None, v=None, global_index=False):
    """Gather the survivors' rows.  Returns dict(hidden, pos, k, v) of packed outputs (None where
    the input was None)."""
    lib = _load()
    keep_idx, cu_keep, cu_seqlens = _i32(keep_idx), _i32(cu_keep), _i32(cu_seqlens)
    batch = len(cu_seqlens) - 1
    total = int(cu_keep[-1])
    out = {"hidden": None, "pos": None, "k": None, "v": None}
    hid_dim = heads = dim = 0
    if hidden is not None:
        hidden = np.ascontiguousarray(hidden)
        assert hidden.dtype == np.uint16 and hidden.ndim == 2
        hid_dim = hidden.shape[1]
        out["hidden"] = np.zeros((total, hid_dim), dtype=np.uint16)
    if pos is not None:
        pos = _i32(pos)
        out["pos"] = np.zeros(total, dtype=np.int32)
    strides = {}
    for name, t in (("k", k), ("v", v)):
        if t is None:
            strides[name] = (None, 0, 0)
            continue
        t, s_t, s_h = _u16_strided(t, name)
        heads, dim = t.shape[1], t.shape[2]
        strides[name] = (t, s_t, s_h)
        out[name] = np.zeros((total, heads, dim), dtype=np.uint16)
    kin, ks_t, ks_h = strides["k"]
    vin, vs_t, vs_h = strides["v"]
    lib.oracle_compact(
        ctypes.c_int(batch), _ptr(cu_seqlens), _ptr(keep_idx), _ptr(cu_keep), ctypes.c_int(1 if global_index else 0),
        ctypes.c_int(hid_dim), ctypes.c_int(heads), ctypes.c_int(dim),
        _ptr(hidden), _ptr(out["hidden"]), _ptr(pos), _ptr(out["pos"]),
        _ptr(kin), ctypes.c_int64(ks_t), ctypes.c_int64(ks_h),
        _ptr(out["k"]), ctypes.c_int64(heads * dim), ctypes.c_int64(dim),
        _ptr(vin), ctypes.c_int64(vs_t), ctypes.c_int64(vs_h),
        _ptr(out["v"]), ctypes.c_int64(heads * dim), ctypes.c_int64(dim))
    return out


def prune(q, k, v, hidden, pos, cu_seqlens, cu_qlens, q_idx, keep_counts, scale, causal,
          protect_rows=True, protect_mask=None, nthreads: int = 0):
    """score -> select -> compact, the whole prune step of one pruning layer."""
    s = score(q, k, cu_seqlens, cu_qlens, q_idx, scale, causal, nthreads)
    keep_idx, cu_keep = select(s, cu_seqlens, keep_counts, protect_mask, protect_rows, q_idx, cu_qlens)
    packed = compact(keep_idx, cu_keep, cu_seqlens, hidden, pos, k, v)
    packed.update(scores=s, keep_idx=keep_idx, cu_keep=cu_keep)
    return packed
