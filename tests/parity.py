"""Shared helpers of the GPU parity tests: move a generated problem to the device, run the oracle
on the same bits, and compare under the stated rules.

Rules:
  scores      |gpu - ref| <= 2e-3 |ref| + 1e-12      (fp32 accumulation over bf16 inputs)
  keep sets   identical to the oracle's, except tokens whose oracle score lies within 2e-3 relative of
              the oracle's k-th score ("ambiguous"); those are counted and returned
  compaction  bit-exact given the keep set
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from conftest import bf16_bits
from paper_2601_13143_b200 import fastav

SCORE_RTOL = 2e-3
SCORE_ATOL = 1e-12


def flags_of(p) -> int:
    return (fastav.FASTAV_CAUSAL if p.causal else 0) | (fastav.FASTAV_PROTECT_QUERY_ROWS if p.protect_rows else 0)


def to_device(p, hidden=None, pos=None, protect=None, flags=None, device="cuda", extra_flags=0) -> fastav.PruneBuffers:
    """PruneInputs (CPU) -> device buffers + outputs.  ``hidden``/``pos`` override the problem's own
    (used by chained stages)."""
    hidden = p.hidden if hidden is None else hidden
    pos = p.pos if pos is None else pos
    dev = lambda t: None if t is None else t.to(device)
    lens = (p.cu_seqlens[1:] - p.cu_seqlens[:-1]).tolist()
    rows = (p.cu_qlens[1:] - p.cu_qlens[:-1]).tolist()
    return fastav.make_buffers(q=dev(p.q), q_idx=dev(p.q_idx), cu_qlens=dev(p.cu_qlens), k=dev(p.k), v=dev(p.v),
                               cu_seqlens=dev(p.cu_seqlens), keep_counts=dev(p.keep_counts), hidden=dev(hidden), pos=dev(pos),
                               protect=dev(protect), softmax_scale=p.softmax_scale,
                               flags=(flags_of(p) if flags is None else flags) | extra_flags, lens=lens, rows=rows, keeps=p.keep_counts.tolist())


def oracle_scores(p, nthreads=0) -> np.ndarray:
    return oracle.score(bf16_bits(p.q), bf16_bits(p.k), p.cu_seqlens.numpy(), p.cu_qlens.numpy(), p.q_idx.numpy(),
                        p.softmax_scale, p.causal, nthreads)


def oracle_prune(p, hidden=None, pos=None, protect=None):
    hidden = p.hidden if hidden is None else hidden
    pos = p.pos if pos is None else pos
    return oracle.prune(bf16_bits(p.q), bf16_bits(p.k), bf16_bits(p.v), bf16_bits(hidden), pos.numpy(), p.cu_seqlens.numpy(),
                        p.cu_qlens.numpy(), p.q_idx.numpy(), p.keep_counts.numpy(), p.softmax_scale, p.causal,
                        protect_rows=p.protect_rows, protect_mask=None if protect is None else protect.numpy())


def assert_scores_close(gpu_scores: torch.Tensor, ref: np.ndarray, what=""):
    got = gpu_scores.detach().cpu().double().numpy()
    assert got.shape == ref.shape
    assert np.isfinite(got).all(), f"{what}: non-finite scores"
    err = np.abs(got - ref)
    bound = SCORE_RTOL * np.abs(ref) + SCORE_ATOL
    worst = int(np.argmax(err - bound))
    assert (err <= bound).all(), (f"{what}: score mismatch at token {worst}: gpu {got[worst]!r} ref {ref[worst]!r} "
                                  f"rel {err[worst] / max(abs(ref[worst]), 1e-300):.3e}; {(err > bound).sum()} of {len(ref)} off")
    return float((err / np.maximum(np.abs(ref), 1e-300))[np.abs(ref) > 1e-9].max(initial=0.0))


def protected_mask(p, protect=None) -> np.ndarray:
    n = int(p.cu_seqlens[-1])
    m = np.zeros(n, dtype=bool)
    if protect is not None:
        m |= protect.numpy().astype(bool)
    if p.protect_rows:
        cu, cuq, qi = p.cu_seqlens.numpy(), p.cu_qlens.numpy(), p.q_idx.numpy()
        for b in range(len(cu) - 1):
            idx = qi[cuq[b]:cuq[b + 1]]
            idx = idx[(idx >= 0) & (idx < cu[b + 1] - cu[b])]
            m[cu[b] + idx] = True
    return m


def assert_keep_sets_match(p, gpu_keep, gpu_cu_keep, ref_scores, ref_keep, ref_cu_keep, protect=None, what="") -> int:
    """Exact match outside the ambiguous band; returns the number of ambiguous tokens that differed."""
    gpu_keep, gpu_cu_keep = gpu_keep.cpu().numpy(), gpu_cu_keep.cpu().numpy()
    assert gpu_cu_keep.tolist() == ref_cu_keep.tolist(), f"{what}: cu_keep differs"
    cu = p.cu_seqlens.numpy()
    prot = protected_mask(p, protect)
    differing = 0
    for b in range(len(cu) - 1):
        got = gpu_keep[gpu_cu_keep[b]:gpu_cu_keep[b + 1]]
        want = ref_keep[ref_cu_keep[b]:ref_cu_keep[b + 1]]
        assert len(got) == len(want)
        assert (np.diff(got) > 0).all(), f"{what}: keep_idx of sequence {b} not strictly ascending"
        if len(got) and (got.min() < 0 or got.max() >= cu[b + 1] - cu[b]):
            raise AssertionError(f"{what}: keep_idx of sequence {b} out of range")
        if np.array_equal(got, want):
            continue
        s = ref_scores[cu[b]:cu[b + 1]]
        unprot_kept = want[~prot[cu[b] + want]]
        assert len(unprot_kept), f"{what}: sets differ although only protected tokens are kept"
        threshold = s[unprot_kept].min()
        diff = np.setxor1d(got, want)
        off = np.abs(s[diff] - threshold) > SCORE_RTOL * threshold + SCORE_ATOL
        assert not off.any(), (f"{what}: sequence {b}: tokens {diff[off][:8].tolist()} differ from the oracle's keep set but "
                               f"their scores {s[diff[off]][:8]} are not within tolerance of the threshold {threshold}")
        assert not prot[cu[b] + diff].any(), f"{what}: a protected token was dropped"
        differing += len(diff)
    return differing


def gather_rows(p, keep, cu_keep, hidden=None, pos=None):
    """What the survivor layout must hold for a given keep set, by plain indexing (test-side)."""
    hidden = p.hidden if hidden is None else hidden
    pos = p.pos if pos is None else pos
    cu = p.cu_seqlens.numpy()
    src = np.concatenate([cu[b] + keep[cu_keep[b]:cu_keep[b + 1]] for b in range(len(cu) - 1)] + [np.zeros(0, dtype=np.int64)]).astype(np.int64)
    src_t = torch.as_tensor(src)
    return {"hidden": None if hidden is None else hidden[src_t], "pos": None if pos is None else pos[src_t],
            "k": p.k[src_t], "v": None if p.v is None else p.v[src_t]}


def assert_bits_equal(gpu_t: torch.Tensor | None, ref, what=""):
    if gpu_t is None or ref is None:
        assert gpu_t is None and ref is None, what
        return
    got = gpu_t.detach().cpu()
    if isinstance(ref, np.ndarray):
        got_np = bf16_bits(got) if got.dtype == torch.bfloat16 else got.numpy()
        assert got_np.shape == ref.shape, f"{what}: shape {got_np.shape} vs {ref.shape}"
        assert np.array_equal(got_np, ref), f"{what}: {(got_np != ref).sum()} elements differ"
    else:
        assert got.shape == ref.shape, f"{what}: shape {tuple(got.shape)} vs {tuple(ref.shape)}"
        a = got.view(torch.int16) if got.dtype == torch.bfloat16 else got
        r = ref.view(torch.int16) if ref.dtype == torch.bfloat16 else ref
        assert torch.equal(a, r), f"{what}: {(a != r).sum().item()} elements differ"


def check_fused_against_oracle(p, buf: fastav.PruneBuffers, ref: dict, hidden=None, pos=None, protect=None, what="") -> dict:
    """Full comparison of one fused prune call.  Returns statistics."""
    status = int(buf.device_status.cpu())
    max_rel = assert_scores_close(buf.scores, ref["scores"], what)
    total_keep = int(ref["cu_keep"][-1])
    gpu_keep = buf.keep_idx[:total_keep]
    differing = assert_keep_sets_match(p, gpu_keep, buf.cu_keep, ref["scores"], ref["keep_idx"], ref["cu_keep"], protect, what)
    # Band or no band: the keep list must be THE top-k of the scores the GPU itself produced (integer work on
    # fp32 bits, ties to the lower index), i.e. what the oracle's selector makes of those scores.
    own_keep, own_cu = oracle.select(buf.scores.detach().cpu().numpy(), p.cu_seqlens.numpy(), p.keep_counts.numpy(),
                                     None if protect is None else protect.numpy(), p.protect_rows, p.q_idx.numpy(), p.cu_qlens.numpy())
    assert own_cu.tolist() == buf.cu_keep.cpu().tolist(), f"{what}: cu_keep differs from the selection on the GPU's own scores"
    assert np.array_equal(gpu_keep.cpu().numpy(), own_keep), f"{what}: keep list is not the top-k of the GPU's own scores"
    mine = gather_rows(p, gpu_keep.cpu().numpy(), buf.cu_keep.cpu().numpy(), hidden, pos)
    assert_bits_equal(buf.hidden_out, mine["hidden"], what + " hidden (own keep set)")
    assert_bits_equal(buf.pos_out, mine["pos"], what + " pos (own keep set)")
    assert_bits_equal(buf.k_out, mine["k"], what + " k (own keep set)")
    assert_bits_equal(buf.v_out, mine["v"], what + " v (own keep set)")
    if differing == 0:
        assert_bits_equal(buf.hidden_out, ref["hidden"], what + " hidden")
        assert_bits_equal(buf.pos_out, ref["pos"], what + " pos")
        assert_bits_equal(buf.k_out, ref["k"], what + " k")
        assert_bits_equal(buf.v_out, ref["v"], what + " v")
    return {"max_rel_err": max_rel, "ambiguous_differing": differing, "device_status": status}
