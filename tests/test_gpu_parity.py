"""GPU parity: every C-ABI entry point against the CPU oracle on the same seeded bits."""
import numpy as np
import pytest
import torch

import oracle
import parity
from conftest import bf16_bits
from paper_2601_13143_b200 import fastav
from paper_2601_13143_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _sync_status(buf):
    torch.cuda.synchronize()
    return int(buf.device_status.cpu())


# ---- score ------------------------------------------------------------------------------------

SCORE_CASES = [
    # lens, rows, hq, hkv, d
    ([1], [1], 4, 4, 64),
    ([2], [1], 4, 1, 64),
    ([7], [3], 8, 2, 64),
    ([8, 9], [1, 4], 7, 1, 128),
    ([127], [4], 28, 4, 128),
    ([128, 129], [3, 1], 28, 4, 128),
    ([1000], [64], 8, 2, 64),
    ([333, 0, 65], [4, 0, 3], 32, 8, 128),
    ([200], [0], 8, 2, 64),
    ([2500], [5], 4, 2, 128),
    ([3000, 17], [1, 1], 32, 8, 128),
    ([1111], [2], 12, 3, 64),
    ([700, 900], [4, 3], 28, 4, 128),
    ([513], [1], 16, 16, 64),
    ([600], [100], 8, 2, 128),          # 400 query rows per KV head: two row chunks on the tensor-core path
    ([4100, 130], [40, 64], 28, 4, 128),
    ([2100], [33], 8, 1, 64),           # 264 rows: a second row chunk with only 8 rows
]


SCORE_PATHS = {"auto": 0, "generic": fastav.FASTAV_SCORE_PATH_GENERIC, "narrow": fastav.FASTAV_SCORE_PATH_NARROW,
               "wide": fastav.FASTAV_SCORE_PATH_WIDE}


def _path_applies(path, rows, hq, hkv, d):
    if path == "narrow":
        return 1 <= max(rows) <= 4
    if path == "wide":
        return max(rows) >= 1
    return True


@pytest.mark.parametrize("lens,rows,hq,hkv,d", SCORE_CASES)
@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("path", ["auto", "generic", "narrow", "wide"])
def test_score_matches_oracle(lens, rows, hq, hkv, d, causal, path):
    if not _path_applies(path, rows, hq, hkv, d):
        pytest.skip("path does not take these shapes")
    p = W.random_problem(seed=sum(lens) + hq, lens=lens, rows=rows, keeps=[n // 2 for n in lens], num_q_heads=hq,
                         num_kv_heads=hkv, head_dim=d, hidden=64, duplicate_keys=3, trailing_rows=False)
    p.causal = causal
    buf = parity.to_device(p, extra_flags=SCORE_PATHS[path])
    buf.scores.fill_(float("nan"))
    buf.score()
    torch.cuda.synchronize()
    ref = parity.oracle_scores(p)
    parity.assert_scores_close(buf.scores, ref, f"lens={lens} rows={rows}")
    got = buf.scores.cpu().numpy()
    cu = p.cu_seqlens.numpy()
    for b, (n, r) in enumerate(zip(lens, rows)):
        if n and min(r, n):
            assert abs(got[cu[b]:cu[b + 1]].sum() - 1.0) < 1e-4
    # bit-reproducible
    first = buf.scores.clone()
    buf.score()
    torch.cuda.synchronize()
    assert torch.equal(first.view(torch.int32), buf.scores.view(torch.int32))


def _natural_lse(p):
    """log sum_j exp(scale q.k_j) over the keys each scored row may see, per (row, head), in float64 on the CPU
    (what an attention kernel would hand back for these rows)."""
    cu, cuq = p.cu_seqlens.tolist(), p.cu_qlens.tolist()
    hq, hkv = p.q.shape[1], p.k.shape[1]
    out = torch.full((p.q.shape[0], hq), float("-inf"), dtype=torch.float64)
    for b in range(len(cu) - 1):
        k = p.k[cu[b]:cu[b + 1]].double().repeat_interleave(hq // hkv, dim=1)            # [n, Hq, d]
        for r in range(cuq[b], cuq[b + 1]):
            z = torch.einsum("hd,nhd->hn", p.q[r].double(), k) * p.softmax_scale          # [Hq, n]
            if p.causal:
                z = z[:, :int(p.q_idx[r]) + 1]
            if z.shape[1]:
                out[r] = torch.logsumexp(z, dim=1)
    return out.float()


@pytest.mark.parametrize("lens,rows,hq,hkv,d", [([300, 40], [3, 1], 8, 2, 64), ([1000], [64], 8, 2, 128), ([777, 130, 0, 5], [40, 9, 0, 5], 28, 4, 128),
                                                ([5000], [1], 4, 4, 64)])
@pytest.mark.parametrize("path", ["auto", "generic", "narrow", "wide"])
@pytest.mark.parametrize("causal", [True, False])
def test_lse_alone_matches_float64_and_feeds_the_single_sweep_score(lens, rows, hq, hkv, d, path, causal):
    """fastav_lse: the first sweep alone, in the attention kernels' convention; handed back as lse_opt it gives the
    scores of the self-contained call.  |lse - ref| <= 5e-4: fp32 sums of up to a few thousand terms whose
    exponentials are good to 1e-4 relative."""
    if not _path_applies(path, rows, hq, hkv, d):
        pytest.skip("path does not take these shapes")
    p = W.random_problem(seed=17, lens=lens, rows=rows, keeps=[n // 2 for n in lens], num_q_heads=hq, num_kv_heads=hkv,
                         head_dim=d, hidden=64, trailing_rows=False)
    p.causal = causal
    buf = parity.to_device(p, extra_flags=SCORE_PATHS[path])
    lse = torch.full((p.q.shape[0], hq), float("nan"), device="cuda")
    fastav.fastav_lse(buf.params, buf.q, buf.q_idx, buf.cu_qlens, buf.k, buf.cu_seqlens, lse, buf.workspace, buf.device_status)
    torch.cuda.synchronize()
    assert _sync_status(buf) == 0
    ref = _natural_lse(p).double()
    got = lse.cpu().double()
    finite = torch.isfinite(ref)
    assert torch.equal(torch.isfinite(got), finite) and (got[~finite] == float("-inf")).all()
    assert (got[finite] - ref[finite]).abs().max() <= 5e-4 if finite.any() else True
    fastav.fastav_score(buf.params, buf.q, buf.q_idx, buf.cu_qlens, buf.k, buf.cu_seqlens, buf.scores, buf.workspace,
                        buf.device_status, lse_opt=lse)
    torch.cuda.synchronize()
    parity.assert_scores_close(buf.scores, parity.oracle_scores(p), "single sweep from fastav_lse")


@pytest.mark.parametrize("lens,rows,hq,hkv,d", [([300, 40], [3, 1], 8, 2, 64), ([1000], [64], 8, 2, 128), ([777, 130], [40, 9], 28, 4, 128)])
@pytest.mark.parametrize("path", ["auto", "generic"])
def test_score_with_caller_provided_lse(lens, rows, hq, hkv, d, path):
    """The attention kernel's log-sum-exp replaces the first sweep; the scores are the same quantity."""
    p = W.random_problem(seed=11, lens=lens, rows=rows, keeps=[n // 2 for n in lens], num_q_heads=hq, num_kv_heads=hkv,
                         head_dim=d, hidden=64)
    buf = parity.to_device(p, extra_flags=SCORE_PATHS[path])
    lse = _natural_lse(p).cuda()
    fastav.fastav_score(buf.params, buf.q, buf.q_idx, buf.cu_qlens, buf.k, buf.cu_seqlens, buf.scores, buf.workspace,
                        buf.device_status, lse_opt=lse)
    torch.cuda.synchronize()
    parity.assert_scores_close(buf.scores, parity.oracle_scores(p), f"lse given, {path}")


def test_score_many_sequences_and_one_very_long_sequence():
    """More sequences than the tensor-core kernel has threads (its unit table is then walked serially), with empty
    ones in between, and one sequence far longer than a block's share of key chunks."""
    rng = np.random.default_rng(5)
    lens = [int(x) for x in rng.integers(0, 40, size=700)]
    rows = [min(n, int(r)) for n, r in zip(lens, rng.integers(5, 9, size=700))]
    p = W.random_problem(seed=77, lens=lens, rows=rows, keeps=[n // 2 for n in lens], num_q_heads=4, num_kv_heads=2, head_dim=64,
                         hidden=64)
    for path in ("wide", "generic"):
        buf = parity.to_device(p, extra_flags=SCORE_PATHS[path])
        buf.score()
        torch.cuda.synchronize()
        assert int(buf.device_status.cpu()) == 0
        parity.assert_scores_close(buf.scores, parity.oracle_scores(p), f"700 sequences, {path}")
    p = W.random_problem(seed=78, lens=[70_001], rows=[6], keeps=[100], num_q_heads=4, num_kv_heads=1, head_dim=64, hidden=64)
    buf = parity.to_device(p, extra_flags=SCORE_PATHS["wide"])
    buf.score()
    torch.cuda.synchronize()
    assert int(buf.device_status.cpu()) == 0
    parity.assert_scores_close(buf.scores, parity.oracle_scores(p), "one sequence of 70001 keys")


def test_score_softmax_scale_one_is_eq4_as_printed():
    p = W.random_problem(seed=3, lens=[50], rows=[1], keeps=[25], num_q_heads=4, num_kv_heads=2, head_dim=64, hidden=64)
    p.softmax_scale = 1.0
    p.k = (p.k.float() * 0.25).to(torch.bfloat16)
    buf = parity.to_device(p)
    buf.score()
    torch.cuda.synchronize()
    parity.assert_scores_close(buf.scores, parity.oracle_scores(p), "scale 1")


def test_score_strided_qkv_views():
    """q and k as views into one packed [tokens, Hq + 2 Hkv, d] projection output."""
    g = torch.Generator().manual_seed(21)
    n, hq, hkv, d = 300, 8, 2, 64
    packed = torch.randn(n, hq + 2 * hkv, d, generator=g).to(torch.bfloat16)
    p = W.random_problem(seed=1, lens=[n], rows=[4], keeps=[100], num_q_heads=hq, num_kv_heads=hkv, head_dim=d, hidden=64)
    dev = packed.cuda()
    q_view, k_view, v_view = dev[n - 4:, :hq], dev[:, hq:hq + hkv], dev[:, hq + hkv:]
    buf = fastav.make_buffers(q=q_view, q_idx=p.q_idx.cuda(), cu_qlens=p.cu_qlens.cuda(), k=k_view, v=v_view,
                              cu_seqlens=p.cu_seqlens.cuda(), keep_counts=p.keep_counts.cuda(), hidden=p.hidden.cuda(),
                              pos=p.pos.cuda(), softmax_scale=p.softmax_scale, flags=fastav.FASTAV_CAUSAL,
                              lens=[n], rows=[4], keeps=[100])
    buf.prune()
    torch.cuda.synchronize()
    bits = bf16_bits(packed)
    ref = oracle.prune(bits[n - 4:, :hq], bits[:, hq:hq + hkv], bits[:, hq + hkv:], bf16_bits(p.hidden), p.pos.numpy(),
                       p.cu_seqlens.numpy(), p.cu_qlens.numpy(), p.q_idx.numpy(), p.keep_counts.numpy(), p.softmax_scale,
                       True, protect_rows=False)
    parity.assert_scores_close(buf.scores, ref["scores"], "strided")
    if np.array_equal(buf.keep_idx.cpu().numpy()[:100], ref["keep_idx"]):
        parity.assert_bits_equal(buf.k_out, ref["k"], "k")
        parity.assert_bits_equal(buf.v_out, ref["v"], "v")
        parity.assert_bits_equal(buf.hidden_out, ref["hidden"], "hidden")


# ---- select -----------------------------------------------------------------------------------

def _select_case(lens, keeps, scores, protect=None, rows=None, q_idx=None, global_idx=False, protect_rows=False, lowest=False):
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    rows = [0] * len(lens) if rows is None else rows
    cuq = np.concatenate([[0], np.cumsum(rows)]).astype(np.int32)
    q_idx = np.zeros(0, dtype=np.int32) if q_idx is None else np.asarray(q_idx, dtype=np.int32)
    clamped = [min(max(k, 0), n) for k, n in zip(keeps, lens)]
    flags = ((fastav.FASTAV_PROTECT_QUERY_ROWS if protect_rows else 0) | (fastav.FASTAV_KEEP_IDX_GLOBAL if global_idx else 0) |
             (fastav.FASTAV_SELECT_LOWEST if lowest else 0))
    params = fastav.make_params(batch=len(lens), total_tokens=int(cu[-1]), max_seqlen=max(lens), total_q=int(cuq[-1]),
                                max_qlen=max(rows), total_keep=sum(clamped), max_keep=max(clamped), num_q_heads=4,
                                num_kv_heads=2, head_dim=64, hidden=64, flags=flags)
    dev = lambda a, dt: torch.as_tensor(np.asarray(a), dtype=dt).cuda()
    ws = torch.empty(max(fastav.fastav_workspace_bytes(params), 256), dtype=torch.uint8, device="cuda")
    keep_idx = torch.full((max(sum(clamped), 1) + 8,), -7, dtype=torch.int32, device="cuda")
    cu_keep = torch.full((len(lens) + 1,), -7, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    fastav.fastav_select(params, dev(scores, torch.float32), dev(cu, torch.int32), dev(keeps, torch.int32),
                         None if protect is None else dev(protect, torch.uint8), dev(q_idx, torch.int32) if len(q_idx) else None,
                         dev(cuq, torch.int32), keep_idx, cu_keep, ws, status)
    torch.cuda.synchronize()
    # keeping the lowest scores is keeping the highest of the negated scores (same tie rule)
    ref_idx, ref_cu = oracle.select(-np.asarray(scores, dtype=np.float32) if lowest else scores, cu, keeps, protect, protect_rows,
                                    q_idx, cuq, global_idx)
    assert cu_keep.cpu().tolist() == ref_cu.tolist()
    got = keep_idx.cpu().numpy()
    assert got[:len(ref_idx)].tolist() == ref_idx.tolist()
    assert (got[len(ref_idx):] == -7).all()          # nothing written past the end
    return int(status.cpu())


def test_select_matches_oracle_with_ties_protection_and_edge_sizes():
    rng = np.random.default_rng(0)
    lens = [1, 2, 7, 8, 9, 127, 128, 129, 1000, 0, 33, 1025, 4097]
    keeps = [1, 1, 3, 8, 0, 64, 127, 129, 400, 0, 32, 1, 4096]
    n = sum(lens)
    scores = (rng.integers(0, 50, size=n) / 1024.0).astype(np.float32)          # heavy ties
    assert _select_case(lens, keeps, scores) == 0
    protect = (rng.random(n) < 0.05).astype(np.uint8)
    assert _select_case(lens, keeps, scores, protect) & ~fastav.FASTAV_DEV_PROTECT_OVERFLOW == 0
    assert _select_case(lens, keeps, scores, protect, global_idx=True) & ~fastav.FASTAV_DEV_PROTECT_OVERFLOW == 0
    smooth = rng.random(n).astype(np.float32) * 1e-3
    assert _select_case(lens, keeps, smooth) == 0


def test_select_lowest_keeps_the_least_attended_tokens():
    rng = np.random.default_rng(12)
    lens, keeps = [700, 33, 4000], [300, 32, 1]
    scores = (rng.integers(0, 200, size=sum(lens)) / 4096.0).astype(np.float32)
    protect = (rng.random(sum(lens)) < 0.03).astype(np.uint8)
    assert _select_case(lens, keeps, scores, lowest=True) == 0
    assert _select_case(lens, keeps, scores, protect, lowest=True) & ~fastav.FASTAV_DEV_PROTECT_OVERFLOW == 0


def test_the_three_selectors_of_the_ablations_on_one_input():
    """Tables 2-3 compare three ways of choosing what goes: the least attended tokens (the method), the most attended
    ones, and a random subset.  The first two are fastav_select with and without FASTAV_SELECT_LOWEST on the attention
    scores; the random control is fastav_select on one seeded uniform draw per token.  Each is checked against the
    oracle's selection on the same scores, with the text rows protected."""
    rng = np.random.default_rng(21)
    lens, keeps = [2230, 744, 5000], [1115, 595, 1000]
    n = sum(lens)
    attention = rng.dirichlet(np.ones(64), size=(n + 63) // 64).reshape(-1)[:n].astype(np.float32)
    random_scores = W.random_control_scores(seed=2601, total_tokens=n).numpy()
    protect = np.zeros(n, dtype=np.uint8)
    start = 0
    for m in lens:  # the trailing text rows of every sequence survive whatever the selector
        protect[start + m - 16:start + m] = 1
        start += m
    assert _select_case(lens, keeps, attention, protect) == 0
    assert _select_case(lens, keeps, attention, protect, lowest=True) == 0
    assert _select_case(lens, keeps, random_scores, protect) == 0
    assert not np.array_equal(np.argsort(-random_scores[:lens[0]], kind="stable")[:keeps[0]],
                              np.argsort(-attention[:lens[0]], kind="stable")[:keeps[0]])  # the control is a different subset


def test_select_general_floats_negative_zero_and_inf():
    scores = np.array([0.0, -0.0, 1.5, -2.0, np.inf, 3e-39, -3e-39, 1.5, -np.inf, 0.0], dtype=np.float32)
    for k in range(0, 11):
        _select_case([10], [min(k, 10)], scores)


def test_select_clamps_and_reports():
    scores = np.linspace(0, 1, 20).astype(np.float32)
    status = _select_case([10, 10], [12, -3], scores)
    assert status & fastav.FASTAV_DEV_K_CLAMPED
    protect = np.zeros(20, dtype=np.uint8)
    protect[[1, 3, 5, 7]] = 1
    status = _select_case([10, 10], [2, 5], scores, protect)
    assert status & fastav.FASTAV_DEV_PROTECT_OVERFLOW


def test_select_protects_query_rows():
    rng = np.random.default_rng(4)
    lens, rows = [40, 50], [3, 2]
    scores = rng.random(90).astype(np.float32)
    scores[[37, 38, 39, 40 + 48, 40 + 49]] = 0.0          # the scored rows would otherwise be dropped first
    assert _select_case(lens, [10, 10], scores, rows=rows, q_idx=[37, 38, 39, 48, 49], protect_rows=True) == 0


def test_select_sequence_longer_than_shared_memory():
    rng = np.random.default_rng(5)
    n = 70_000
    scores = (rng.integers(0, 5000, size=n) / 65536.0).astype(np.float32)
    assert _select_case([n, 100], [n // 3, 50], scores=np.concatenate([scores, rng.random(100).astype(np.float32)])) == 0


@pytest.mark.parametrize("longest", [2048, 2049, 4097, 8200, 16384, 40_000, 131_072, 131_073])
def test_select_long_sequences_in_ragged_batches(longest):
    """Keep lists of long sequences (keys in shared memory up to about 50k tokens, in the workspace above)
    with short and empty sequences in the same batch: heavy ties, protected tokens and scored rows anywhere,
    a long run of equal scores, nearly everything or nearly nothing kept."""
    rng = np.random.default_rng(longest)
    lens = [longest, 0, 1, 33, longest // 3, 1000]
    keeps = [longest // 2, 0, 1, 20, longest // 3 - 1, 1]
    n = sum(lens)
    scores = (rng.integers(0, 300, size=n) / 8192.0).astype(np.float32)
    assert _select_case(lens, keeps, scores) == 0
    assert _select_case(lens, keeps, scores, lowest=True, global_idx=True) == 0
    protect = (rng.random(n) < 0.02).astype(np.uint8)
    rows = [7, 0, 1, 2, 5, 0]
    q_idx = np.concatenate([np.sort(rng.choice(max(ln, 1), size=r, replace=False)) for ln, r in zip(lens, rows)])
    status = _select_case(lens, keeps, scores, protect, rows=rows, q_idx=q_idx, protect_rows=True)
    assert status & ~fastav.FASTAV_DEV_PROTECT_OVERFLOW == 0
    smooth = rng.random(n).astype(np.float32)
    smooth[: longest // 2] = 0.0        # a long run of zeros: equal keys in whole warps
    assert _select_case(lens, keeps, smooth) == 0
    assert _select_case(lens, [longest - 1, 0, 0, 33, 1, 999], smooth, global_idx=True) == 0


def test_positional_global_prune_keeps_first_audio_tokens():
    """The paper's deployed global stage: a positional rule (here: only the first 10 audio tokens survive,
    everything else is kept) -> keep list -> survivor layout, against the oracle."""
    w = W.WORKLOADS["c2_global_2k"]
    p = W.make_stage(w, 0)
    mask = W.positional_keep_mask(p.modality, p.cu_seqlens, {W.MOD_AUDIO: 10})
    ref_idx, ref_cu = oracle.select_mask(mask.numpy(), p.cu_seqlens.numpy())
    kept = int(ref_cu[-1])
    assert kept == p.total_tokens - (256 - 10)
    ref = oracle.compact(ref_idx, ref_cu, p.cu_seqlens.numpy(), bf16_bits(p.hidden), p.pos.numpy(), bf16_bits(p.k), bf16_bits(p.v))
    p.keep_counts = torch.tensor([kept], dtype=torch.int32)
    buf = parity.to_device(p, flags=0)
    buf.keep_idx.fill_(-7)
    fastav.fastav_select_mask(buf.params, mask.cuda(), buf.cu_seqlens, buf.keep_idx, buf.cu_keep, buf.workspace, buf.device_status)
    buf.compact()
    assert _sync_status(buf) == 0
    assert buf.cu_keep.cpu().tolist() == ref_cu.tolist()
    assert buf.keep_idx.cpu().numpy()[:kept].tolist() == ref_idx.tolist()
    for name in ("hidden", "pos", "k", "v"):
        parity.assert_bits_equal(getattr(buf, name + "_out"), ref[name], name)


def test_select_mask_ragged_global_indices_and_capacity_clamp():
    rng = np.random.default_rng(9)
    lens = [5, 0, 2000, 1, 333]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    mask = (rng.random(cu[-1]) < 0.5).astype(np.uint8)
    for glob in (False, True):
        ref_idx, ref_cu = oracle.select_mask(mask, cu, global_index=glob)
        total = int(ref_cu[-1])
        params = fastav.make_params(batch=len(lens), total_tokens=int(cu[-1]), max_seqlen=max(lens), total_q=0, max_qlen=0,
                                    total_keep=total, max_keep=total, num_q_heads=4, num_kv_heads=2, head_dim=64, hidden=64,
                                    flags=fastav.FASTAV_KEEP_IDX_GLOBAL if glob else 0)
        keep_idx = torch.full((total + 8,), -7, dtype=torch.int32, device="cuda")
        cu_keep = torch.full((len(lens) + 1,), -7, dtype=torch.int32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        ws = torch.empty(256, dtype=torch.uint8, device="cuda")
        fastav.fastav_select_mask(params, torch.as_tensor(mask).cuda(), torch.as_tensor(cu).cuda(), keep_idx, cu_keep, ws, status)
        torch.cuda.synchronize()
        assert cu_keep.cpu().tolist() == ref_cu.tolist() and int(status) == 0
        got = keep_idx.cpu().numpy()
        assert got[:total].tolist() == ref_idx.tolist() and (got[total:] == -7).all()
    # a keep buffer that is too small: nothing written past it, the clamp is reported
    params.total_keep = params.max_keep = total - 50
    keep_idx.fill_(-7)
    status.zero_()
    fastav.fastav_select_mask(params, torch.as_tensor(mask).cuda(), torch.as_tensor(cu).cuda(), keep_idx, cu_keep, ws, status)
    torch.cuda.synchronize()
    assert int(status) & fastav.FASTAV_DEV_K_CLAMPED and int(cu_keep[-1]) == total - 50
    assert (keep_idx.cpu().numpy()[total - 50:] == -7).all()


# ---- compact ----------------------------------------------------------------------------------

@pytest.mark.parametrize("hkv,d,hid", [(2, 64, 64), (4, 128, 3584), (8, 128, 4096), (1, 64, 8)])
@pytest.mark.parametrize("path", [0, fastav.FASTAV_COMPACT_PATH_LOADSTORE])
def test_compact_matches_oracle(hkv, d, hid, path):
    rng = np.random.default_rng(hkv * 100 + d)
    lens = [37, 0, 129, 1]
    keeps = [10, 0, 129, 1]
    p = W.random_problem(seed=hid, lens=lens, rows=[1, 0, 1, 1], keeps=keeps, num_q_heads=hkv * 2, num_kv_heads=hkv,
                         head_dim=d, hidden=hid)
    cu = p.cu_seqlens.numpy()
    keep_idx = np.concatenate([np.sort(rng.choice(n, size=k, replace=False)) for n, k in zip(lens, keeps)]).astype(np.int32)
    cu_keep = np.concatenate([[0], np.cumsum(keeps)]).astype(np.int32)
    ref = oracle.compact(keep_idx, cu_keep, cu, bf16_bits(p.hidden), p.pos.numpy(), bf16_bits(p.k), bf16_bits(p.v))
    buf = parity.to_device(p, flags=path)
    for t in (buf.hidden_out, buf.k_out, buf.v_out):
        t.view(torch.int16).fill_(0x7FC1)
    buf.pos_out.fill_(-1)
    buf.keep_idx[:len(keep_idx)].copy_(torch.as_tensor(keep_idx))
    buf.cu_keep.copy_(torch.as_tensor(cu_keep))
    buf.compact()
    assert _sync_status(buf) == 0
    for name in ("hidden", "pos", "k", "v"):
        parity.assert_bits_equal(getattr(buf, name + "_out"), ref[name], name)
    # global indices, only the K pair
    buf.params.flags = fastav.FASTAV_KEEP_IDX_GLOBAL | path
    global_idx = np.concatenate([cu[b] + keep_idx[cu_keep[b]:cu_keep[b + 1]] for b in range(len(lens))]).astype(np.int32)
    buf.keep_idx[:len(global_idx)].copy_(torch.as_tensor(global_idx))
    buf.k_out.zero_()
    fastav.fastav_compact(buf.params, buf.keep_idx, buf.cu_keep, buf.cu_seqlens, k_in=buf.k, k_out=buf.k_out)
    torch.cuda.synchronize()
    parity.assert_bits_equal(buf.k_out, ref["k"], "k (global indices)")


@pytest.mark.parametrize("path", [0, fastav.FASTAV_COMPACT_PATH_LOADSTORE])
def test_compact_buffers_beyond_4_gib(path):
    """Byte offsets past 2^32: 1.2 M tokens of 2,048 bf16 hidden values (4.9 GB in, 1.6 GB out), three sequences,
    every third token kept through a rule-given mask.  Expected rows by plain indexing on the same tensors."""
    n_seq, per_seq, hid, hkv, d = 3, 400_000, 2048, 1, 64
    n = n_seq * per_seq
    dev = "cuda"
    rows = torch.arange(n, device=dev, dtype=torch.int32)
    hidden = torch.empty(n, hid, dtype=torch.bfloat16, device=dev)
    cols = (torch.arange(hid, device=dev, dtype=torch.int32) % 7).view(1, hid)
    for i in range(0, n, 100_000):                       # row id and column pattern in every element, built in slices
        hidden[i:i + 100_000] = ((rows[i:i + 100_000].view(-1, 1) % 251) + cols).to(torch.bfloat16)
    k = (rows % 509).view(n, 1, 1).expand(n, hkv, d).to(torch.bfloat16).contiguous()
    pos = rows.clone()
    mask = (rows % 3 == 1).to(torch.uint8)
    kept = int(mask.sum())
    cu = torch.tensor([0, per_seq, 2 * per_seq, n], dtype=torch.int32, device=dev)
    p = fastav.make_params(batch=n_seq, total_tokens=n, max_seqlen=per_seq, total_q=0, max_qlen=0, total_keep=kept,
                           max_keep=kept, num_q_heads=hkv, num_kv_heads=hkv, head_dim=d, hidden=hid, k=k, flags=path)
    keep_idx = torch.empty(kept, dtype=torch.int32, device=dev)
    cu_keep = torch.empty(n_seq + 1, dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    ws = torch.empty(max(fastav.fastav_workspace_bytes(p), 256), dtype=torch.uint8, device=dev)
    fastav.fastav_select_mask(p, mask, cu, keep_idx, cu_keep, ws, status)
    hidden_out = torch.empty(kept, hid, dtype=torch.bfloat16, device=dev)
    k_out = torch.empty(kept, hkv, d, dtype=torch.bfloat16, device=dev)
    pos_out = torch.empty(kept, dtype=torch.int32, device=dev)
    fastav.fastav_compact(p, keep_idx, cu_keep, cu, hidden_in=hidden, hidden_out=hidden_out, pos_in=pos, pos_out=pos_out,
                          k_in=k, k_out=k_out, device_status=status)
    torch.cuda.synchronize()
    assert int(status.cpu()) == 0
    src = torch.nonzero(mask).view(-1)                   # survivors in order, as global row numbers
    assert torch.equal(pos_out.long(), src)
    assert cu_keep.cpu().tolist() == [0] + torch.cumsum(mask.view(n_seq, per_seq).sum(dim=1), 0).tolist()
    for i in range(0, kept, 50_000):
        idx = src[i:i + 50_000]
        assert torch.equal(hidden_out[i:i + 50_000].view(torch.int16), hidden[idx].view(torch.int16)), f"hidden rows from {i}"
        assert torch.equal(k_out[i:i + 50_000].view(torch.int16), k[idx].view(torch.int16)), f"k rows from {i}"


def test_compact_many_rows_per_warp_and_bad_rows_in_between():
    """Enough rows that every warp of the bulk-copy kernel cycles its slots many times, with a few
    out-of-range indices sprinkled in (skipped rows must not disturb the rows around them)."""
    rng = np.random.default_rng(77)
    lens, keeps = [9000, 3000], [7000, 3000]
    p = W.random_problem(seed=5, lens=lens, rows=[1, 1], keeps=keeps, num_q_heads=4, num_kv_heads=2, head_dim=64, hidden=256)
    cu = p.cu_seqlens.numpy()
    keep_idx = np.concatenate([np.sort(rng.choice(n, size=k, replace=False)) for n, k in zip(lens, keeps)]).astype(np.int32)
    cu_keep = np.concatenate([[0], np.cumsum(keeps)]).astype(np.int32)
    ref = oracle.compact(keep_idx, cu_keep, cu, bf16_bits(p.hidden), p.pos.numpy(), bf16_bits(p.k), bf16_bits(p.v))
    bad_rows = [5, 1234, 6999, 7000, 9999]
    broken = keep_idx.copy()
    broken[bad_rows] = [-1, 9000, 20000, 3000, -5]
    buf = parity.to_device(p, flags=0)
    for t in (buf.hidden_out, buf.k_out, buf.v_out):
        t.view(torch.int16).fill_(0x7FC1)
    buf.keep_idx[:len(broken)].copy_(torch.as_tensor(broken))
    buf.cu_keep.copy_(torch.as_tensor(cu_keep))
    buf.compact()
    assert _sync_status(buf) == fastav.FASTAV_DEV_BAD_INDEX
    good = np.ones(len(keep_idx), dtype=bool)
    good[bad_rows] = False
    for name in ("hidden", "k", "v"):
        got = getattr(buf, name + "_out").cpu().view(torch.int16).numpy()
        want = ref[name].view(np.int16)
        assert np.array_equal(got[good], want[good]), name
        assert (got[~good] == 0x7FC1).all(), name + ": a skipped row was written"


def test_compact_strided_outputs_and_guard_bands():
    """Outputs are views into a wider cache buffer; bytes outside the views must stay untouched."""
    p = W.random_problem(seed=8, lens=[64], rows=[1], keeps=[20], num_q_heads=4, num_kv_heads=2, head_dim=64, hidden=128)
    keep_idx = np.sort(np.random.default_rng(1).choice(64, 20, replace=False)).astype(np.int32)
    cache = torch.full((20 + 2, 2 * 2 + 1, 64), 7.0, dtype=torch.bfloat16, device="cuda")   # [tokens+guard, k|v|pad heads, d]
    k_out, v_out = cache[1:21, 0:2], cache[1:21, 2:4]
    buf = parity.to_device(p, flags=0)
    buf.k_out, buf.v_out = k_out, v_out
    buf.params.ko_stride_tok, buf.params.ko_stride_head = k_out.stride(0), k_out.stride(1)
    buf.params.vo_stride_tok, buf.params.vo_stride_head = v_out.stride(0), v_out.stride(1)
    buf.keep_idx[:20].copy_(torch.as_tensor(keep_idx))
    buf.cu_keep.copy_(torch.tensor([0, 20], dtype=torch.int32))
    buf.compact()
    assert _sync_status(buf) == 0
    ref = oracle.compact(keep_idx, np.array([0, 20], dtype=np.int32), p.cu_seqlens.numpy(), None, None, bf16_bits(p.k), bf16_bits(p.v))
    parity.assert_bits_equal(k_out.contiguous(), ref["k"], "k view")
    parity.assert_bits_equal(v_out.contiguous(), ref["v"], "v view")
    host = cache.cpu().float()
    assert (host[0] == 7).all() and (host[21] == 7).all() and (host[:, 4] == 7).all()


def test_compact_reports_out_of_range_indices():
    p = W.random_problem(seed=9, lens=[16], rows=[1], keeps=[4], num_q_heads=2, num_kv_heads=1, head_dim=64, hidden=64)
    buf = parity.to_device(p, flags=0)
    buf.keep_idx[:4].copy_(torch.tensor([0, 5, 99, -2], dtype=torch.int32))
    buf.cu_keep.copy_(torch.tensor([0, 4], dtype=torch.int32))
    buf.hidden_out.zero_()
    buf.compact()
    assert _sync_status(buf) & fastav.FASTAV_DEV_BAD_INDEX
    out = buf.hidden_out.cpu()
    assert torch.equal(out[1].view(torch.int16), p.hidden[5].view(torch.int16)) and (out[2:] == 0).all()


# ---- fused prune ------------------------------------------------------------------------------

def test_prune_calls_on_two_streams_at_once_each_match_the_oracle():
    """Two requests pruned at the same time on two streams, each with its own buffers and workspace (how a server
    would run them): the calls share nothing, so each must give the oracle's result whatever the interleaving."""
    shapes = [([3000, 517], [32, 8], [1200, 300], 8, 2, 128, 256), ([900, 2100, 33], [1, 1, 1], [700, 1500, 30], 28, 4, 128, 512)]
    problems = [W.random_problem(seed=400 + i, lens=l, rows=r, keeps=k, num_q_heads=hq, num_kv_heads=hkv, head_dim=d, hidden=hid)
                for i, (l, r, k, hq, hkv, d, hid) in enumerate(shapes)]
    bufs = [parity.to_device(p) for p in problems]
    refs = [parity.oracle_prune(p) for p in problems]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    torch.cuda.synchronize()
    for rep in range(3):
        for buf in bufs:  # poison the outputs, so that a call that did not run cannot pass
            buf.keep_idx.fill_(-3)
            buf.scores.fill_(float("nan"))
        torch.cuda.synchronize()
        for _ in range(4):  # several calls deep on both streams, so that their kernels really interleave
            for buf, st in zip(bufs, streams):
                buf.prune(stream=st)
        torch.cuda.synchronize()
        for p, buf, ref in zip(problems, bufs, refs):
            stats = parity.check_fused_against_oracle(p, buf, ref, what=f"two streams, repetition {rep}")
            assert stats["device_status"] == 0


@pytest.mark.parametrize("lens,rows,keeps,hq,hkv,d,hid", [
    ([9], [1], [4], 4, 2, 64, 64),
    ([129, 0, 64], [4, 0, 1], [64, 0, 64], 8, 2, 64, 128),
    ([1000, 7], [3, 2], [999, 1], 28, 4, 128, 256),
    ([300], [64], [150], 8, 2, 128, 512),
])
@pytest.mark.parametrize("protect_rows", [True, False])
def test_prune_small_problems(lens, rows, keeps, hq, hkv, d, hid, protect_rows):
    p = W.random_problem(seed=len(lens) * 31 + hq, lens=lens, rows=rows, keeps=keeps, num_q_heads=hq, num_kv_heads=hkv,
                         head_dim=d, hidden=hid, duplicate_keys=4)
    p.protect_rows = protect_rows
    buf = parity.to_device(p)
    buf.prune()
    torch.cuda.synchronize()
    ref = parity.oracle_prune(p)
    stats = parity.check_fused_against_oracle(p, buf, ref, what=f"lens={lens}")
    overflow = protect_rows and any(min(r, n) > k for r, n, k in zip(rows, lens, keeps))
    assert stats["device_status"] == (fastav.FASTAV_DEV_PROTECT_OVERFLOW if overflow else 0)
    # twice in a row: bit-identical everything
    first = {k: getattr(buf, k).clone() for k in ("scores", "keep_idx", "hidden_out", "k_out", "v_out", "pos_out")}
    buf.prune()
    torch.cuda.synchronize()
    for k, t in first.items():
        assert torch.equal(t.view(torch.int32) if t.dtype == torch.float32 else t.view(torch.int16) if t.dtype == torch.bfloat16 else t,
                           getattr(buf, k).view(torch.int32) if t.dtype == torch.float32 else getattr(buf, k).view(torch.int16) if t.dtype == torch.bfloat16 else getattr(buf, k)), k


@pytest.mark.parametrize("seed", range(120))
def test_prune_random_shapes(seed):
    """Seeded random problems: batch, ragged lengths (empty ones too), scored rows anywhere in the sequence or
    trailing, head counts, head size, keep counts from 0 to n, duplicate keys (exact ties), a protect mask, the
    causal flag and the score path all drawn at random; the whole fused call against the oracle."""
    rng = np.random.default_rng(1000 + seed)
    batch = int(rng.integers(1, 7))
    lens = [int(rng.choice([0, 1, 2, 31, 64, 127, 128, 129, 300, 515, 1025, 2049])) if rng.random() < 0.5 else int(rng.integers(1, 900))
            for _ in range(batch)]
    if sum(lens) == 0:
        lens[0] = 5
    max_rows = int(rng.choice([1, 2, 4, 5, 17, 64, 130]))
    rows = [int(rng.integers(0, max_rows + 1)) for _ in lens]
    hkv = int(rng.choice([1, 2, 4]))
    hq = hkv * int(rng.choice([1, 2, 4, 7]))
    d = int(rng.choice([64, 128]))
    keeps = [int(rng.integers(0, n + 1)) for n in lens]
    p = W.random_problem(seed=seed, lens=lens, rows=rows, keeps=keeps, num_q_heads=hq, num_kv_heads=hkv, head_dim=d,
                         hidden=int(rng.choice([64, 136, 512])), duplicate_keys=int(rng.integers(0, 5)),
                         trailing_rows=bool(rng.random() < 0.5))
    p.causal = bool(rng.random() < 0.7)
    p.protect_rows = bool(rng.random() < 0.5)
    p.softmax_scale = float(rng.choice([1.0 / np.sqrt(d), 0.05, 0.3]))
    protect = (torch.from_numpy(rng.random(sum(lens))) < 0.04).to(torch.uint8) if rng.random() < 0.5 else None
    path = str(rng.choice(["auto", "auto", "generic", "narrow", "wide"]))
    if not _path_applies(path, [min(r, n) for r, n in zip(rows, lens)], hq, hkv, d):
        path = "auto"
    chain = fastav.FASTAV_CHAIN_CALLS if rng.random() < 0.5 else 0      # inputs are complete either way
    buf = parity.to_device(p, protect=protect, extra_flags=SCORE_PATHS[path] | chain)
    buf.prune()
    torch.cuda.synchronize()
    ref = parity.oracle_prune(p, protect=protect)
    stats = parity.check_fused_against_oracle(p, buf, ref, protect=protect, what=f"seed {seed}: lens={lens} rows={rows} hq={hq} hkv={hkv} d={d} {path}")
    assert stats["device_status"] & ~fastav.FASTAV_DEV_PROTECT_OVERFLOW == 0


@pytest.mark.parametrize("lens,rows,hq,hkv,d", [
    ([364, 2049, 80, 300], [23, 41, 44, 2], 2, 2, 128),      # tensor-core score, register-resident select
    ([900, 512, 33], [1, 2, 1], 8, 2, 64),                   # few rows, short: logits + one fused tail kernel
    ([5000, 3000], [1, 1], 28, 4, 128),                      # few rows, long: logits, statistics, finalize, select
    ([20000, 100], [40, 3], 4, 2, 64),                       # keys in shared memory (longer than the register kernel takes)
    ([70000], [8], 4, 1, 64),                                # keys in the workspace
])
@pytest.mark.parametrize("chain", [0, fastav.FASTAV_CHAIN_CALLS])
def test_prune_never_reads_what_an_earlier_call_left_behind(lens, rows, hq, hkv, d, chain):
    """Kernels of one call start before their predecessors have finished (programmatic launch).  Every buffer a
    kernel of the chain reads from another is overwritten with poison between calls: a read that comes too
    early, or from a line cached during the previous call, changes the result."""
    p = W.random_problem(seed=len(lens) + hq, lens=lens, rows=rows, keeps=[n // 3 + 1 for n in lens], num_q_heads=hq,
                         num_kv_heads=hkv, head_dim=d, hidden=64)
    buf = parity.to_device(p, extra_flags=chain)
    buf.prune()
    torch.cuda.synchronize()
    ref = parity.oracle_prune(p)
    parity.check_fused_against_oracle(p, buf, ref, what=f"lens={lens}")
    names = ("scores", "keep_idx", "cu_keep", "hidden_out", "k_out", "v_out", "pos_out")

    def run(fused):
        if fused:
            buf.prune()
        else:                      # the same three steps as separate calls: they chain on the stream in the same way
            buf.score()
            buf.select()
            buf.compact()
        torch.cuda.synchronize()

    def bits(t):
        return t.view(torch.int32) if t.dtype == torch.float32 else t.view(torch.int16) if t.dtype == torch.bfloat16 else t

    first = {}
    for fused in (True, False):    # the two routes may round the scores differently; each is compared with itself
        run(fused)
        first[fused] = {k: getattr(buf, k).clone() for k in names}
    for rep in range(30):
        buf.scores.fill_(float("nan"))
        buf.workspace.fill_(0xFF)
        buf.keep_idx.fill_(-7)
        buf.cu_keep.fill_(-7)
        for t in (buf.hidden_out, buf.k_out, buf.v_out):
            t.view(torch.int16).fill_(0x7FC1)
        buf.pos_out.fill_(-1)
        fused = rep % 2 == 0
        run(fused)
        for k in names:
            assert torch.equal(bits(first[fused][k]), bits(getattr(buf, k))), f"repetition {rep}: {k} differs from the first call"


@pytest.mark.parametrize("lens,rows1,rows2,hq,hkv,d", [([700, 300, 2049], [40, 8, 16], [1, 1, 1], 8, 2, 64),
                                                        ([900, 512], [1, 1], [1, 1], 28, 4, 128)])
def test_second_call_may_take_its_cu_seqlens_from_the_first(lens, rows1, rows2, hq, hkv, d):
    """Two pruning layers back to back on one stream, the second reading the FIRST call's cu_keep_out as its
    cu_seqlens and its hidden/pos outputs as inputs (no FASTAV_CHAIN_CALLS: those arrays are written by the call
    before).  Outputs of the first call are poisoned before every repetition, so a second call that read them too
    early would see poison."""
    keeps1 = [n // 2 for n in lens]
    keeps2 = [k * 3 // 4 for k in keeps1]
    p1 = W.random_problem(seed=21, lens=lens, rows=rows1, keeps=keeps1, num_q_heads=hq, num_kv_heads=hkv, head_dim=d, hidden=128)
    p1.protect_rows = True
    p2 = W.random_problem(seed=22, lens=keeps1, rows=rows2, keeps=keeps2, num_q_heads=hq, num_kv_heads=hkv, head_dim=d, hidden=128)
    p2.protect_rows = True
    b1 = parity.to_device(p1)
    dev = lambda t: t.cuda()
    b2 = fastav.make_buffers(q=dev(p2.q), q_idx=dev(p2.q_idx), cu_qlens=dev(p2.cu_qlens), k=dev(p2.k), v=dev(p2.v),
                             cu_seqlens=b1.cu_keep, keep_counts=dev(p2.keep_counts), hidden=b1.hidden_out, pos=b1.pos_out,
                             softmax_scale=p2.softmax_scale, flags=parity.flags_of(p2), lens=keeps1,
                             rows=[min(r, n) for r, n in zip(rows2, keeps1)], keeps=keeps2)
    ref1 = parity.oracle_prune(p1)
    ref2 = parity.oracle_prune(p2, hidden=torch.from_numpy(ref1["hidden"].view(np.int16)).view(torch.bfloat16),
                               pos=torch.from_numpy(ref1["pos"]))
    for rep in range(10):
        b1.cu_keep.fill_(-7)
        b1.hidden_out.view(torch.int16).fill_(0x7FC1)
        b1.pos_out.fill_(-1)
        b2.scores.fill_(float("nan"))
        b1.prune()
        b2.prune()
        torch.cuda.synchronize()
        s1 = parity.check_fused_against_oracle(p1, b1, ref1, what=f"first call, repetition {rep}")
        if s1["ambiguous_differing"] == 0:
            s2 = parity.check_fused_against_oracle(p2, b2, ref2, hidden=b1.hidden_out.cpu(), pos=b1.pos_out.cpu(),
                                                   what=f"second call, repetition {rep}")
            assert s2["device_status"] == 0


def test_prune_with_protect_mask_keeps_all_text_tokens():
    w = W.WORKLOADS["c1_tiny"]
    p = W.make_stage(w, 0)
    protect = (p.modality == W.MOD_TEXT).to(torch.uint8)
    buf = parity.to_device(p, protect=protect)
    buf.prune()
    torch.cuda.synchronize()
    ref = parity.oracle_prune(p, protect=protect)
    parity.check_fused_against_oracle(p, buf, ref, protect=protect, what="protect mask")
    kept = set(buf.keep_idx.cpu().tolist())
    assert set(torch.nonzero(protect).flatten().tolist()) <= kept


def _run_workload_chain(name, stats_out=None):
    """All stages of a workload; stage s+1 starts from the ORACLE's survivors of stage s."""
    w = W.WORKLOADS[name]
    hidden = pos = None
    for si in range(len(w.stages)):
        p = W.make_stage(w, si)
        if si == 0:
            hidden, pos = p.hidden, p.pos
        buf = parity.to_device(p, hidden=hidden, pos=pos)
        buf.prune()
        torch.cuda.synchronize()
        ref = parity.oracle_prune(p, hidden=hidden, pos=pos)
        stats = parity.check_fused_against_oracle(p, buf, ref, hidden=hidden, pos=pos, what=f"{name} stage {si}")
        assert stats["device_status"] == 0
        got = buf.scores.cpu().numpy()
        cu = p.cu_seqlens.numpy()
        sums = np.add.reduceat(got, cu[:-1])
        assert np.abs(sums - 1.0).max() < 1e-4
        assert int(buf.cu_keep[-1]) == p.total_keep
        if stats_out is not None:
            stats_out.append(stats)
        hidden = torch.as_tensor(ref["hidden"].view(np.int16)).view(torch.bfloat16)
        pos = torch.as_tensor(ref["pos"])
        del buf
        torch.cuda.empty_cache()


@pytest.mark.parametrize("name", ["c1_tiny", "c2_global_2k", "c3_fine_chain", "n3_fine_chain_13"])
def test_prune_workloads_small(name):
    _run_workload_chain(name)


@pytest.mark.parametrize("name", ["c4_long_av", "c5_ragged"])
def test_prune_workloads_full_size(name):
    stats = []
    _run_workload_chain(name, stats)
    print(name, stats)


def test_prune_host_buffers_match_oracle():
    """The host-buffer entry point computes the same step (copies in, fused prune, copies out)."""
    p = W.make_stage(W.WORKLOADS["c1_tiny"], 0)
    m = p.model
    n, kk = p.total_tokens, p.total_keep
    params = fastav.make_params(batch=1, total_tokens=n, max_seqlen=n, total_q=4, max_qlen=4, total_keep=kk, max_keep=kk,
                                num_q_heads=m.num_q_heads, num_kv_heads=m.num_kv_heads, head_dim=m.head_dim, hidden=m.hidden,
                                softmax_scale=p.softmax_scale, flags=parity.flags_of(p))
    pin = lambda t: t.contiguous().pin_memory()
    out = dict(scores=pin(torch.empty(n)), keep_idx=pin(torch.empty(kk, dtype=torch.int32)), cu_keep=pin(torch.empty(2, dtype=torch.int32)),
               hidden=pin(torch.empty(kk, m.hidden, dtype=torch.bfloat16)), pos=pin(torch.empty(kk, dtype=torch.int32)),
               k=pin(torch.empty(kk, m.num_kv_heads, m.head_dim, dtype=torch.bfloat16)),
               v=pin(torch.empty(kk, m.num_kv_heads, m.head_dim, dtype=torch.bfloat16)), status=pin(torch.full((1,), -1, dtype=torch.int32)))
    arena = torch.empty(fastav.fastav_host_arena_bytes(params), dtype=torch.uint8, device="cuda")
    fastav.fastav_prune_host(params, pin(p.q), pin(p.q_idx), pin(p.cu_qlens), pin(p.k), pin(p.v), pin(p.cu_seqlens),
                             pin(p.keep_counts), None, pin(p.hidden), pin(p.pos), out["scores"], out["keep_idx"], out["cu_keep"],
                             out["hidden"], out["pos"], out["k"], out["v"], out["status"], arena)
    torch.cuda.synchronize()
    ref = parity.oracle_prune(p)
    parity.assert_scores_close(out["scores"], ref["scores"], "host")
    assert int(out["status"]) == 0 and out["cu_keep"].tolist() == [0, kk]
    assert out["keep_idx"].tolist() == ref["keep_idx"].tolist()
    for name in ("hidden", "pos", "k", "v"):
        parity.assert_bits_equal(out[name], ref[name], "host " + name)


def test_a_wait_that_cannot_succeed_ends_with_an_error_bit_and_a_usable_context():
    """Failure detection without a fault: the kernels' waits are bounded; one that nothing satisfies gives up,
    reports FASTAV_DEV_WAIT_EXPIRED, and the next call on the same context works."""
    import time
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    fastav.fastav_selftest_bounded_wait(50, status)
    torch.cuda.synchronize()
    elapsed = time.perf_counter() - t0
    assert int(status) == fastav.FASTAV_DEV_WAIT_EXPIRED
    assert 0.04 < elapsed < 2.0
    p = W.random_problem(seed=1, lens=[200], rows=[8], keeps=[100], num_q_heads=8, num_kv_heads=2, head_dim=64, hidden=64)
    buf = parity.to_device(p)
    buf.prune()
    torch.cuda.synchronize()
    parity.check_fused_against_oracle(p, buf, parity.oracle_prune(p), what="after the expired wait")


def test_bench_per_sequence_host_pipeline_equals_one_batched_call():
    """bench.py's end-to-end leg cuts a batch into one host-buffer call per sequence and stage on two streams;
    every output must equal what the single batched call writes."""
    import os, sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import bench
    w = W.Workload("mini_ragged", 9, 9, W.TINY, 3, (200, 600), None, 4, (W.Stage(2, 5, None), W.Stage(3, 1, 0.8)),
                   keep_range=(0.3, 0.7), description="test only")
    dev = torch.device("cuda", 0)
    chain = bench.host_chain(w, dev)
    bench.run_host_step(chain)
    torch.cuda.synchronize()
    names = ("scores", "keep_idx", "hidden_out", "pos_out", "k_out", "v_out")
    want = [{k: h[k].clone() for k in names} for h in chain]
    calls, streams, chain2 = bench.host_chain_per_sequence(w, dev)
    for h in chain2:
        for k in names:
            h[k].view(torch.uint8).fill_(0xEE)
    bench.run_host_step_per_sequence(calls, streams, torch.cuda.current_stream())
    torch.cuda.synchronize()
    for si, h in enumerate(chain2):
        for k in names:
            assert torch.equal(h[k].view(torch.uint8), want[si][k].view(torch.uint8)), (si, k)
    assert all(int(c["status"]) == 0 for mine in calls for c in mine)


@pytest.mark.parametrize("lens,rows,hq,hkv,d", [([1500, 300], [64, 40], 8, 2, 128), ([900], [2], 28, 4, 128), ([400, 77], [9, 5], 4, 4, 64)])
@pytest.mark.parametrize("path", ["auto", "generic", "narrow"])
def test_workspace_guard_band_and_equal_keys_tie_bit_exactly(lens, rows, hq, hkv, d, path):
    """(1) Nothing is written past fastav_workspace_bytes: a sentinel band after the workspace survives a fused call.
    (2) The per-key arithmetic does not depend on the key's position: with every row seeing every key, tokens that
    carry the same key vector get bit-equal scores."""
    if path == "narrow" and max(rows) > 4:
        pytest.skip("path does not take these shapes")
    p = W.random_problem(seed=3, lens=lens, rows=rows, keeps=[n // 3 for n in lens], num_q_heads=hq, num_kv_heads=hkv, head_dim=d,
                         hidden=64)
    p.causal = False
    cu = p.cu_seqlens.tolist()
    twins = []
    for b in range(len(lens)):            # copy token 5 of each sequence over a few other tokens, far apart
        for j in (17, lens[b] // 2, lens[b] - 1):
            p.k[cu[b] + j] = p.k[cu[b] + 5]
            twins.append((cu[b] + 5, cu[b] + j))
    buf = parity.to_device(p, extra_flags=SCORE_PATHS[path])
    need = fastav.fastav_workspace_bytes(buf.params)
    guard = 4096
    ws = torch.full((need + guard,), 0x5A, dtype=torch.uint8, device="cuda")
    buf.workspace = ws[:need]
    buf.prune()
    torch.cuda.synchronize()
    assert int(buf.device_status.cpu()) == 0
    assert bool((ws[need:] == 0x5A).all()), "the workspace was overrun"
    parity.assert_scores_close(buf.scores, parity.oracle_scores(p), "guarded call")
    bits = buf.scores.view(torch.int32).cpu()
    for a, b in twins:
        assert int(bits[a]) == int(bits[b]), (a, b)


# ---- the fused call with the attention kernel's log-sum-exp -------------------------------------------

@pytest.mark.parametrize("lens,rows,hq,hkv,d,hid", [
    ([2048], [64], 28, 4, 128, 3584),                                   # the 2k global prune's shapes
    ([4100, 1300], [128, 128], 32, 8, 128, 4096),                       # long-clip shapes, cut down to what the oracle does in seconds
    ([1024, 3000, 1500, 2222, 1025], [32] * 5, 28, 4, 128, 3584),       # ragged serving batch shapes
    ([900, 33], [1, 1], 8, 2, 64, 64),                                  # last-token query: the paper's fine stage
])
@pytest.mark.parametrize("host", [False, True])
def test_fused_prune_with_the_attention_kernels_lse(lens, rows, hq, hkv, d, hid, host):
    """fastav_prune / fastav_prune_host given lse_opt (float64 log-sum-exp rounded to fp32, as the layer's attention
    kernel would return it): one sweep over K, same scores, keep set and survivor layout as the oracle."""
    p = W.random_problem(seed=5, lens=lens, rows=rows, keeps=[n * 2 // 5 for n in lens], num_q_heads=hq, num_kv_heads=hkv,
                         head_dim=d, hidden=hid)
    p.protect_rows = True
    lse = _natural_lse(p)
    ref = parity.oracle_prune(p)
    if not host:
        buf = parity.to_device(p)
        launches0 = fastav.fastav_kernel_launches()
        buf.prune(lse_opt=lse.cuda())
        with_lse = fastav.fastav_kernel_launches() - launches0
        torch.cuda.synchronize()
        stats = parity.check_fused_against_oracle(p, buf, ref, what=f"lse given, lens={lens}")
        assert stats["device_status"] == 0
        launches0 = fastav.fastav_kernel_launches()
        buf.prune()
        if max(rows) > 4:          # (short sequences with a last-token query fold their statistics into the select kernel)
            assert with_lse <= fastav.fastav_kernel_launches() - launches0  # never more kernels than the self-contained call
        torch.cuda.synchronize()
        parity.check_fused_against_oracle(p, buf, ref, what=f"self-contained, lens={lens}")
        return
    n, kk, rq = p.total_tokens, p.total_keep, int(p.cu_qlens[-1])
    params = fastav.make_params(batch=len(lens), total_tokens=n, max_seqlen=max(lens), total_q=rq, max_qlen=max(rows), total_keep=kk,
                                max_keep=int(p.keep_counts.max()), num_q_heads=hq, num_kv_heads=hkv, head_dim=d, hidden=hid,
                                softmax_scale=p.softmax_scale, flags=parity.flags_of(p))
    pin = lambda t: t.contiguous().pin_memory()
    out = dict(scores=pin(torch.empty(n)), keep_idx=pin(torch.empty(kk, dtype=torch.int32)), cu_keep=pin(torch.empty(len(lens) + 1, dtype=torch.int32)),
               hidden=pin(torch.empty(kk, hid, dtype=torch.bfloat16)), pos=pin(torch.empty(kk, dtype=torch.int32)),
               k=pin(torch.empty(kk, hkv, d, dtype=torch.bfloat16)), v=pin(torch.empty(kk, hkv, d, dtype=torch.bfloat16)),
               status=pin(torch.full((1,), -1, dtype=torch.int32)))
    arena = torch.empty(fastav.fastav_host_arena_bytes(params), dtype=torch.uint8, device="cuda")
    fastav.fastav_prune_host(params, pin(p.q), pin(p.q_idx), pin(p.cu_qlens), pin(p.k), pin(p.v), pin(p.cu_seqlens),
                             pin(p.keep_counts), None, pin(p.hidden), pin(p.pos), out["scores"], out["keep_idx"], out["cu_keep"],
                             out["hidden"], out["pos"], out["k"], out["v"], out["status"], arena, lse_opt=pin(lse))
    torch.cuda.synchronize()
    parity.assert_scores_close(out["scores"], ref["scores"], "host, lse given")
    assert int(out["status"]) == 0 and out["cu_keep"].tolist() == ref["cu_keep"].tolist()
    own_keep, _ = oracle.select(out["scores"].numpy(), p.cu_seqlens.numpy(), p.keep_counts.numpy(), None, True, p.q_idx.numpy(), p.cu_qlens.numpy())
    assert np.array_equal(out["keep_idx"].numpy(), own_keep)
    if np.array_equal(own_keep, ref["keep_idx"]):
        for name in ("hidden", "pos", "k", "v"):
            parity.assert_bits_equal(out[name], ref[name], "host " + name)


def test_host_entry_point_refuses_before_it_copies_anything():
    """A call the fused entry point would refuse must not have started its uploads: the arena keeps its contents."""
    p = W.make_stage(W.WORKLOADS["c1_tiny"], 0)
    m = p.model
    n, kk = p.total_tokens, p.total_keep
    params = fastav.make_params(batch=1, total_tokens=n, max_seqlen=n, total_q=4, max_qlen=4, total_keep=kk, max_keep=kk,
                                num_q_heads=m.num_q_heads, num_kv_heads=m.num_kv_heads, head_dim=m.head_dim, hidden=m.hidden,
                                softmax_scale=p.softmax_scale, flags=parity.flags_of(p) | fastav.FASTAV_SCORE_PATH_NARROW)
    arena = torch.full((fastav.fastav_host_arena_bytes(params),), 0x3C, dtype=torch.uint8, device="cuda")
    params.max_qlen = params.total_q = 64      # the forced matrix-vector path takes at most 4 scored rows: refused
    pin = lambda t: t.contiguous().pin_memory()
    q = pin(torch.zeros(64, m.num_q_heads, m.head_dim, dtype=torch.bfloat16))
    q_idx = pin(torch.arange(64, dtype=torch.int32))
    outs = [pin(torch.empty(n)), pin(torch.empty(kk, dtype=torch.int32)), pin(torch.empty(2, dtype=torch.int32)),
            pin(torch.empty(kk, m.hidden, dtype=torch.bfloat16)), pin(torch.empty(kk, dtype=torch.int32)),
            pin(torch.empty(kk, m.num_kv_heads, m.head_dim, dtype=torch.bfloat16)),
            pin(torch.empty(kk, m.num_kv_heads, m.head_dim, dtype=torch.bfloat16)), pin(torch.zeros(1, dtype=torch.int32))]
    big = torch.full((max(fastav.fastav_host_arena_bytes(params), arena.numel()),), 0x3C, dtype=torch.uint8, device="cuda")
    with pytest.raises(fastav.FastavError) as err:
        fastav.fastav_prune_host(params, q, q_idx, pin(torch.tensor([0, 64], dtype=torch.int32)), pin(p.k), pin(p.v), pin(p.cu_seqlens),
                                 pin(p.keep_counts), None, pin(p.hidden), pin(p.pos), *outs, big)
    assert err.value.status == fastav.FASTAV_ERR_UNSUPPORTED
    torch.cuda.synchronize()
    assert bool((big == 0x3C).all()), "copies were enqueued although the call was refused"


# ---- chained calls whose tensors (not only index arrays) come from the call before -----------------------

@pytest.mark.parametrize("lens,rows,hq,hkv,d", [([300, 200], [16, 8], 8, 2, 64), ([1500], [40], 4, 1, 128)])
def test_chained_second_call_scores_the_keys_the_first_call_compacted(lens, rows, hq, hkv, d):
    """Under FASTAV_CHAIN_CALLS only the INDEX arrays may be read early.  Here the second call's k and hidden are
    the first call's k_out and hidden_out (a cache compacted in place of the layer's fresh projections), on shapes
    whose tensor-core grids are far smaller than the GPU, so both calls' kernels can be resident together.  The
    first call's outputs are poisoned before every repetition: keys fetched before the gather has finished would
    be poison and change the second call's scores."""
    keeps1 = [n // 2 for n in lens]
    keeps2 = [k // 2 for k in keeps1]
    p1 = W.random_problem(seed=31, lens=lens, rows=rows, keeps=keeps1, num_q_heads=hq, num_kv_heads=hkv, head_dim=d, hidden=128)
    p1.protect_rows = True
    ref1 = parity.oracle_prune(p1)
    p2 = W.random_problem(seed=32, lens=keeps1, rows=rows, keeps=keeps2, num_q_heads=hq, num_kv_heads=hkv, head_dim=d, hidden=128)
    p2.protect_rows = True
    as_bf16 = lambda a: torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16)
    p2.k, p2.v = as_bf16(ref1["k"]), as_bf16(ref1["v"])      # what the first call must produce (checked below)
    ref2 = parity.oracle_prune(p2, hidden=as_bf16(ref1["hidden"]), pos=torch.from_numpy(ref1["pos"]))
    chain = fastav.FASTAV_CHAIN_CALLS | fastav.FASTAV_SCORE_PATH_WIDE
    b1 = parity.to_device(p1, extra_flags=chain)
    dev = lambda t: t.cuda()
    b2 = fastav.make_buffers(q=dev(p2.q), q_idx=dev(p2.q_idx), cu_qlens=dev(p2.cu_qlens), k=b1.k_out, v=b1.v_out,
                             cu_seqlens=dev(p2.cu_seqlens), keep_counts=dev(p2.keep_counts), hidden=b1.hidden_out, pos=b1.pos_out,
                             softmax_scale=p2.softmax_scale, flags=parity.flags_of(p2) | chain, lens=keeps1, rows=rows, keeps=keeps2)
    for rep in range(20):
        for t in (b1.hidden_out, b1.k_out, b1.v_out):
            t.view(torch.int16).fill_(0x7FC1)
        b1.pos_out.fill_(-1)
        b2.scores.fill_(float("nan"))
        b1.prune()
        b2.prune()
        torch.cuda.synchronize()
        s1 = parity.check_fused_against_oracle(p1, b1, ref1, what=f"first call, repetition {rep}")
        assert s1["ambiguous_differing"] == 0
        s2 = parity.check_fused_against_oracle(p2, b2, ref2, hidden=as_bf16(ref1["hidden"]), pos=torch.from_numpy(ref1["pos"]),
                                               what=f"second call, repetition {rep}")
        assert s2["device_status"] == 0


# ---- the paper's fine chain replayed from one CUDA graph --------------------------------------------------

def test_fine_chain_of_13_layers_replayed_from_one_graph_matches_the_oracle():
    """Section 2.2 / 3.1: after the global stage the lowest 20 % go at each of the 13 later layers.  All 13 fused calls
    are captured into ONE CUDA graph (stage s+1 reading stage s's hidden_out / pos_out in place), the graph is
    replayed twice over poisoned outputs, and every stage of each replay is compared with the oracle chain."""
    w = W.WORKLOADS["n3_fine_chain_13"]
    stages, prev = [], None
    for si in range(len(w.stages)):
        p = W.make_stage(w, si)
        lens = (p.cu_seqlens[1:] - p.cu_seqlens[:-1]).tolist()
        rows = (p.cu_qlens[1:] - p.cu_qlens[:-1]).tolist()
        buf = fastav.make_buffers(q=p.q.cuda(), q_idx=p.q_idx.cuda(), cu_qlens=p.cu_qlens.cuda(), k=p.k.cuda(), v=p.v.cuda(),
                                  cu_seqlens=p.cu_seqlens.cuda(), keep_counts=p.keep_counts.cuda(),
                                  hidden=p.hidden.cuda() if si == 0 else prev.hidden_out, pos=p.pos.cuda() if si == 0 else prev.pos_out,
                                  softmax_scale=p.softmax_scale, flags=parity.flags_of(p) | fastav.FASTAV_CHAIN_CALLS, lens=lens, rows=rows,
                                  keeps=p.keep_counts.tolist())
        stages.append((p, buf))
        prev = buf
    refs, hidden, pos = [], stages[0][0].hidden, stages[0][0].pos
    for p, _ in stages:
        ref = parity.oracle_prune(p, hidden=hidden, pos=pos)
        refs.append((ref, hidden, pos))
        hidden = torch.from_numpy(ref["hidden"].view(np.int16).copy()).view(torch.bfloat16)
        pos = torch.from_numpy(ref["pos"].copy())
    for _, buf in stages:                       # one eager pass first: attribute set-up does not belong in a capture
        buf.prune()
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for _, buf in stages:
            buf.prune(side)
    for replay in range(2):
        for _, buf in stages:
            buf.scores.fill_(float("nan"))
            buf.workspace.fill_(0xFF)
            buf.keep_idx.fill_(-7)
            buf.cu_keep.fill_(-7)
            for t in (buf.hidden_out, buf.k_out, buf.v_out):
                t.view(torch.int16).fill_(0x7FC1)
            buf.pos_out.fill_(-1)
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        for si, ((p, buf), (ref, hidden, pos)) in enumerate(zip(stages, refs)):
            stats = parity.check_fused_against_oracle(p, buf, ref, hidden=hidden, pos=pos, what=f"replay {replay}, stage {si}")
            assert stats["device_status"] == 0
            if stats["ambiguous_differing"]:    # a near-threshold token went the other way: later stages see another token set
                break
        else:
            assert int(stages[-1][1].cu_keep[-1]) == stages[-1][0].total_keep


# ---- host scalars that understate what the device arrays describe -----------------------------------------

@pytest.mark.parametrize("true_len,claimed,entry", [(1500, 1000, "select"), (5000, 3000, "select"), (60_000, 52_000, "select"),
                                                    (5000, 3000, "noalloc"), (1500, 1000, "prune_wide"), (1500, 1000, "prune_narrow")])
def test_lengths_beyond_what_params_state_set_the_mismatch_bit(true_len, claimed, entry):
    """Buffers are allocated for the TRUE lengths (so even an unguarded kernel would stay in bounds) while params
    understates max_seqlen: the kernels size shared memory, registers and tables from the host scalars, so they
    must cut the sequence down to what those promise and report FASTAV_DEV_SHAPE_MISMATCH."""
    lens, keeps = [true_len, 200], [claimed // 2, 100]
    rows = [1, 1] if entry == "prune_narrow" else [8, 8]
    p = W.random_problem(seed=9, lens=lens, rows=rows, keeps=keeps, num_q_heads=4, num_kv_heads=2, head_dim=64, hidden=64)
    p.protect_rows = True
    buf = parity.to_device(p)
    buf.params.max_seqlen = claimed
    buf.scores.copy_(torch.rand(sum(lens)))
    if entry == "select":
        buf.select()
    elif entry == "noalloc":
        fastav.fastav_select_noalloc(buf.params, buf.scores, buf.cu_seqlens, buf.keep_counts, None, buf.q_idx, buf.cu_qlens,
                                     buf.keep_idx, buf.cu_keep, buf.device_status)
    else:
        buf.prune()
    torch.cuda.synchronize()
    assert int(buf.device_status.cpu()) & fastav.FASTAV_DEV_SHAPE_MISMATCH
    assert buf.cu_keep.cpu().tolist() == [0, keeps[0], keeps[0] + keeps[1]]
    kept = buf.keep_idx.cpu().numpy()
    assert kept[:keeps[0]].max() < claimed and (np.diff(kept[:keeps[0]]) > 0).all()
