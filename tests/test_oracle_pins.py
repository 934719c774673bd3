"""Pins for the CPU oracle: everything here checks ``oracle/`` against something other than
itself -- hand-worked values (tests/golden), a brute-force full attention map built with torch in
float64, closed forms, invariants, an independent stable sort, and the FLOPs column the paper
prints.  No GPU needed."""
import json
import math
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import flops as oflops
from conftest import bf16_bits, to_bf16_bits

DIM = 4


def _expand(coord0, heads):
    """[tokens][heads] list of coordinate-0 values -> [tokens, heads, DIM] bf16 bits."""
    a = np.zeros((len(coord0), heads, DIM), dtype=np.float32)
    a[:, :, 0] = np.asarray(coord0, dtype=np.float32)
    return to_bf16_bits(a)


def _golden_cases(golden_dir):
    with open(os.path.join(golden_dir, "eq4_hand_worked.json")) as f:
        return json.load(f)["cases"]


def test_hand_worked_scores_and_keep_sets(golden_dir):
    cases = _golden_cases(golden_dir)
    assert len(cases) >= 5
    for c in cases:
        scale = math.log(3.0) if c["scale"] == "ln3" else float(c["scale"])
        n, rows = c["tokens"], len(c["q_idx"])
        q = _expand(c["q"], c["num_q_heads"])
        k = _expand(c["k"], c["num_kv_heads"])
        cu, cuq = [0, n], [0, rows]
        s = oracle.score(q, k, cu, cuq, c["q_idx"], scale, c["causal"])
        want = np.asarray(c["score_num"], dtype=np.float64) / c["score_den"]
        np.testing.assert_allclose(s, want, rtol=0, atol=1e-15, err_msg=c["name"])
        keep, cuk = oracle.select(s, cu, [c["keep"]])
        assert keep.tolist() == c["keep_idx"], c["name"]
        assert cuk.tolist() == [0, c["keep"]]
        keep_p, _ = oracle.select(s, cu, [c["keep"]], None, True, c["q_idx"], cuq)
        assert keep_p.tolist() == c["keep_idx_protect_rows"], c["name"]


def _brute_force_scores(q, k, q_idx, scale, causal):
    """Full n x n attention map per head in float64 (every position gets a query row: positions that
    are not scored get a zero query), then pick the scored rows and average rows and heads."""
    rows, hq, d = q.shape
    n, hkv, _ = k.shape
    g = hq // hkv
    full_q = torch.zeros(n, hq, d, dtype=torch.float64)
    full_q[torch.as_tensor(q_idx, dtype=torch.long)] = q.double()
    kk = k.double().repeat_interleave(g, dim=1)                       # [n, hq, d], head h <- kv head h // g
    logits = torch.einsum("ihd,jhd->hij", full_q, kk) * scale          # [hq, n, n]
    if causal:
        mask = torch.ones(n, n, dtype=torch.bool).tril()
        logits = logits.masked_fill(~mask, float("-inf"))
    attn = torch.softmax(logits, dim=-1)
    picked = attn[:, torch.as_tensor(q_idx, dtype=torch.long), :]      # [hq, rows, n]
    return picked.mean(dim=(0, 1)).numpy()


@pytest.mark.parametrize("hq,hkv,d,n,q_idx,causal", [
    (1, 1, 8, 9, [8], True),
    (4, 2, 8, 16, [13, 14, 15], True),
    (6, 2, 16, 12, [3, 7, 11], True),       # rows in the middle of the sequence: real masking
    (6, 3, 8, 11, [0, 10], True),           # a row that sees exactly one key
    (8, 2, 64, 16, [12, 13, 14, 15], False),
    (7, 1, 8, 5, [4], True),
])
def test_brute_force_full_attention_map(hq, hkv, d, n, q_idx, causal):
    g = torch.Generator().manual_seed(hq * 1000 + n)
    q = torch.randn(len(q_idx), hq, d, generator=g).to(torch.bfloat16)
    k = torch.randn(n, hkv, d, generator=g).to(torch.bfloat16)
    scale = 0.37
    want = _brute_force_scores(q.float(), k.float(), q_idx, scale, causal)
    got = oracle.score(bf16_bits(q), bf16_bits(k), [0, n], [0, len(q_idx)], q_idx, scale, causal)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-15)
    # the same through one thread and through all of them
    got1 = oracle.score(bf16_bits(q), bf16_bits(k), [0, n], [0, len(q_idx)], q_idx, scale, causal, nthreads=1)
    assert np.array_equal(got, got1)


def test_batched_varlen_equals_per_sequence():
    g = torch.Generator().manual_seed(5)
    lens, rows = [7, 0, 12, 1], [2, 0, 3, 1]
    hq, hkv, d = 4, 2, 8
    q = torch.randn(sum(rows), hq, d, generator=g).to(torch.bfloat16)
    k = torch.randn(sum(lens), hkv, d, generator=g).to(torch.bfloat16)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    cuq = np.concatenate([[0], np.cumsum(rows)]).astype(np.int32)
    q_idx = np.concatenate([np.arange(n - r, n) for n, r in zip(lens, rows)]).astype(np.int32)
    s = oracle.score(bf16_bits(q), bf16_bits(k), cu, cuq, q_idx, 0.5, True)
    for b, (n, r) in enumerate(zip(lens, rows)):
        if n == 0:
            continue
        want = _brute_force_scores(q[cuq[b]:cuq[b + 1]].float(), k[cu[b]:cu[b + 1]].float(),
                                   q_idx[cuq[b]:cuq[b + 1]].tolist(), 0.5, True)
        np.testing.assert_allclose(s[cu[b]:cu[b + 1]], want, rtol=1e-12, atol=1e-15)
        assert abs(s[cu[b]:cu[b + 1]].sum() - 1.0) < 1e-12


def test_strided_views_match_contiguous():
    g = torch.Generator().manual_seed(9)
    n, hq, hkv, d = 10, 4, 2, 8
    qkv = torch.randn(n, hq + 2 * hkv, d, generator=g).to(torch.bfloat16)   # packed q|k|v per token
    bits = bf16_bits(qkv)
    q_all, k_view = bits[:, :hq], bits[:, hq:hq + hkv]
    q_rows = q_all[n - 2:]
    s_view = oracle.score(q_rows, k_view, [0, n], [0, 2], [n - 2, n - 1], 0.3, True)
    s_cont = oracle.score(np.ascontiguousarray(q_rows), np.ascontiguousarray(k_view), [0, n], [0, 2], [n - 2, n - 1], 0.3, True)
    assert np.array_equal(s_view, s_cont)


def test_closed_forms():
    g = torch.Generator().manual_seed(11)
    n, hq, hkv, d = 13, 4, 2, 8
    q = torch.randn(1, hq, d, generator=g).to(torch.bfloat16)
    k = torch.randn(n, hkv, d, generator=g).to(torch.bfloat16)
    cu, cuq, qi = [0, n], [0, 1], [n - 1]
    # scale 0: uniform over the visible keys
    s = oracle.score(bf16_bits(q), bf16_bits(k), cu, cuq, qi, 0.0, True)
    np.testing.assert_allclose(s, np.full(n, 1.0 / n), rtol=1e-15)
    # all keys equal: uniform
    k_same = k[:1].expand(n, hkv, d).contiguous()
    s = oracle.score(bf16_bits(q), bf16_bits(k_same), cu, cuq, qi, 1.0, True)
    np.testing.assert_allclose(s, np.full(n, 1.0 / n), rtol=1e-14)
    # one head, one row: the textbook softmax row
    q1 = torch.randn(1, 1, d, generator=g).to(torch.bfloat16)
    k1 = torch.randn(n, 1, d, generator=g).to(torch.bfloat16)
    s = oracle.score(bf16_bits(q1), bf16_bits(k1), cu, cuq, qi, 1.0, True)
    want = torch.softmax((k1[:, 0].double() @ q1[0, 0].double()), dim=0).numpy()
    np.testing.assert_allclose(s, want, rtol=1e-13)
    # a dominating key takes (almost) all the mass in every head
    k_dom = k.clone()
    k_dom[4] = 0
    q_big = torch.zeros(1, hq, d, dtype=torch.bfloat16)
    q_big[..., 0] = 8.0
    k_dom[:, :, 0] = -8.0
    k_dom[4, :, 0] = 8.0
    s = oracle.score(bf16_bits(q_big), bf16_bits(k_dom), cu, cuq, qi, 1.0, True)
    assert s[4] > 1 - 1e-12 and s.sum() == pytest.approx(1.0, abs=1e-12)


def test_invariances_noncausal():
    g = torch.Generator().manual_seed(13)
    n, hq, hkv, d, rows = 17, 6, 3, 8, 3
    q = torch.randn(rows, hq, d, generator=g).to(torch.bfloat16)
    k = torch.randn(n, hkv, d, generator=g).to(torch.bfloat16)
    cu, cuq, qi = [0, n], [0, rows], [n - 3, n - 2, n - 1]
    s = oracle.score(bf16_bits(q), bf16_bits(k), cu, cuq, qi, 0.4, False)
    assert (s >= 0).all() and s.sum() == pytest.approx(1.0, abs=1e-13)
    # permuting the keys permutes the scores
    perm = torch.randperm(n, generator=g)
    s_perm = oracle.score(bf16_bits(q), bf16_bits(k[perm]), cu, cuq, qi, 0.4, False)
    np.testing.assert_allclose(s_perm, s[perm.numpy()], rtol=1e-13)
    # a head whose query is zero contributes a uniform row; doubling scale on +-1 data is not a no-op
    q0 = q.clone()
    q0[:, 0] = 0
    s0 = oracle.score(bf16_bits(q0), bf16_bits(k), cu, cuq, qi, 0.4, False)
    s_rest = oracle.score(bf16_bits(q[:, 1:3]), bf16_bits(k[:, :1]), cu, cuq, qi, 0.4, False)  # heads 1,2 -> kv 0
    assert not np.allclose(s0, s)
    assert s_rest.sum() == pytest.approx(1.0, abs=1e-13)
    # duplicated key rows get bit-equal scores
    k_dup = k.clone()
    k_dup[5] = k_dup[2]
    s_dup = oracle.score(bf16_bits(q), bf16_bits(k_dup), cu, cuq, qi, 0.4, False)
    assert s_dup[5] == s_dup[2]


def test_shift_invariance_via_extra_coordinate():
    """Adding the same constant to every logit of a row leaves the softmax unchanged: append a
    coordinate that is 1 in every key and c in the query."""
    g = torch.Generator().manual_seed(17)
    n, d = 9, 8
    q = torch.randn(1, 2, d, generator=g).to(torch.bfloat16)
    k = torch.randn(n, 1, d, generator=g).to(torch.bfloat16)
    q2 = torch.cat([q, torch.full((1, 2, 1), 2.5, dtype=torch.bfloat16)], dim=2)
    k2 = torch.cat([k, torch.ones(n, 1, 1, dtype=torch.bfloat16)], dim=2)
    s = oracle.score(bf16_bits(q), bf16_bits(k), [0, n], [0, 1], [n - 1], 0.7, True)
    s2 = oracle.score(bf16_bits(q2), bf16_bits(k2), [0, n], [0, 1], [n - 1], 0.7, True)
    np.testing.assert_allclose(s2, s, rtol=1e-12)


def _reference_select(scores32, k, protected):
    """Independent selector: torch's stable descending sort on float64 keys."""
    key = torch.as_tensor(scores32.astype(np.float64)).clone()
    key[torch.as_tensor(protected, dtype=torch.bool)] = float("inf")
    order = torch.sort(key, descending=True, stable=True).indices[:k]
    return np.sort(order.numpy())


def test_select_against_stable_sort_with_ties_and_protection():
    rng = np.random.default_rng(3)
    lens = [1, 2, 7, 8, 9, 127, 128, 129, 1000, 0, 33]
    keeps = [1, 1, 3, 8, 0, 64, 127, 129, 400, 0, 40]           # includes k = n, k = 0 and k > n (clamped)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    scores = rng.integers(0, 12, size=cu[-1]).astype(np.float32) / 64.0       # many exact ties
    protect = (rng.random(cu[-1]) < 0.1).astype(np.uint8)
    for mask in (None, protect):
        keep_idx, cuk = oracle.select(scores, cu, keeps, mask)
        for b, (n, kk) in enumerate(zip(lens, keeps)):
            kk = min(kk, n)
            got = keep_idx[cuk[b]:cuk[b + 1]]
            assert len(got) == kk
            prot = np.zeros(n, dtype=bool) if mask is None else mask[cu[b]:cu[b + 1]].astype(bool)
            want = _reference_select(scores[cu[b]:cu[b + 1]], kk, prot)
            assert got.tolist() == want.tolist()
            assert (np.diff(got) > 0).all()
            if 0 < kk < n and mask is None:
                s = scores[cu[b]:cu[b + 1]]
                dropped = np.setdiff1d(np.arange(n), got)
                assert s[got].min() >= s[dropped].max()
    # global indices are the local ones shifted by the sequence start
    g_idx, g_cu = oracle.select(scores, cu, keeps, protect, global_index=True)
    l_idx, l_cu = oracle.select(scores, cu, keeps, protect)
    assert g_cu.tolist() == l_cu.tolist()
    for b in range(len(lens)):
        assert (g_idx[g_cu[b]:g_cu[b + 1]] - cu[b]).tolist() == l_idx[l_cu[b]:l_cu[b + 1]].tolist()


def test_protected_overflow_keeps_lowest_indices():
    scores = np.linspace(1, 0, 10).astype(np.float32)
    protect = np.zeros(10, dtype=np.uint8)
    protect[[2, 5, 7, 9]] = 1
    keep, _ = oracle.select(scores, [0, 10], [2], protect)
    assert keep.tolist() == [2, 5]
    keep, _ = oracle.select(scores, [0, 10], [6], protect)
    assert keep.tolist() == [0, 1, 2, 5, 7, 9]


def test_compact_is_a_row_gather():
    rng = np.random.default_rng(7)
    lens = [5, 0, 9]
    cu = np.array([0, 5, 5, 14], dtype=np.int32)
    n, hkv, d, hid = 14, 2, 4, 6
    hidden = rng.integers(0, 65536, size=(n, hid)).astype(np.uint16)
    pos = rng.integers(0, 10_000, size=n).astype(np.int32)
    kv = rng.integers(0, 65536, size=(n, 2 * hkv, d)).astype(np.uint16)
    k, v = kv[:, :hkv], kv[:, hkv:]                           # strided views of a packed buffer
    keep_idx = np.array([0, 2, 4, 1, 3, 8], dtype=np.int32)
    cu_keep = np.array([0, 3, 3, 6], dtype=np.int32)
    out = oracle.compact(keep_idx, cu_keep, cu, hidden, pos, k, v)
    src = np.array([0, 2, 4, 6, 8, 13])
    assert np.array_equal(out["hidden"], hidden[src])
    assert np.array_equal(out["pos"], pos[src])
    assert np.array_equal(out["k"], k[src]) and np.array_equal(out["v"], v[src])
    out_g = oracle.compact(src.astype(np.int32), cu_keep, cu, hidden, pos, k, v, global_index=True)
    assert all(np.array_equal(out[x], out_g[x]) for x in ("hidden", "pos", "k", "v"))
    # keep everything: identity
    ident = oracle.compact(np.concatenate([np.arange(5), np.arange(9)]).astype(np.int32), cu, cu, hidden, pos, k, v)
    assert np.array_equal(ident["hidden"], hidden) and np.array_equal(ident["k"], k)
    # optional pairs are skipped
    only_pos = oracle.compact(keep_idx, cu_keep, cu, None, pos, None, None)
    assert only_pos["hidden"] is None and np.array_equal(only_pos["pos"], pos[src])


def test_whole_step_invariants_on_tiny_workload():
    from paper_2601_13143_b200 import workloads as W
    p = W.make_stage(W.WORKLOADS["c1_tiny"], 0)
    out = oracle.prune(bf16_bits(p.q), bf16_bits(p.k), bf16_bits(p.v), bf16_bits(p.hidden), p.pos.numpy(),
                       p.cu_seqlens.numpy(), p.cu_qlens.numpy(), p.q_idx.numpy(), p.keep_counts.numpy(),
                       p.softmax_scale, p.causal, protect_rows=True)
    s, keep = out["scores"], out["keep_idx"]
    assert s.sum() == pytest.approx(1.0, abs=1e-12) and (s >= 0).all()
    assert len(keep) == 256 and (np.diff(keep) > 0).all()
    assert set(p.q_idx.tolist()) <= set(keep.tolist())              # scored rows survive
    assert set(p.anchors[0].tolist()) <= set(keep.tolist())         # anchors dominate the scores
    assert np.array_equal(out["pos"], p.pos.numpy()[keep])          # positions carried, not renumbered
    assert np.array_equal(out["hidden"], bf16_bits(p.hidden)[keep])
    a = p.anchors[0].numpy()
    assert np.all(s[a] == s[a[0]])                                  # identical anchor keys tie exactly


def test_flops_column_of_table_4(golden_dir):
    with open(os.path.join(golden_dir, "table4_flops.json")) as f:
        t = json.load(f)
    a = t["assumed"]
    for p_str, printed in t["printed"].items():
        prunes = oflops.fastav_schedule(a["tokens"], t["num_layers"], t["global_layer"], a["global_keep"], int(p_str) / 100.0)
        rel = oflops.relative_flops(a["tokens"], t["num_layers"], a["hidden"], a["ffn"], prunes)
        assert abs(rel - printed) <= t["tolerance_points"], (p_str, rel, printed)
    # monotone in P, and no pruning is 100
    assert oflops.relative_flops(a["tokens"], 28, a["hidden"], a["ffn"], {}) == pytest.approx(100.0)
    seen = oflops.token_schedule(1000, 6, {3: 500, 4: 400})
    assert seen == [1000, 1000, 1000, 500, 400, 400]
    assert oflops.removed_count(1024, 0.2) == 204 and oflops.removed_count(820, 0.2) == 164


def test_reported_flops_agree_with_the_oracle_count_and_table_4(golden_dir):
    """The benchmark's "prefill FLOPs removed" comes from the product's own restatement of the count; it must
    give the oracle's relative figure (and hence Table 4's column) and the oracle's absolute saving."""
    from paper_2601_13143_b200 import flops as pflops
    from paper_2601_13143_b200 import workloads as W
    with open(os.path.join(golden_dir, "table4_flops.json")) as f:
        t = json.load(f)
    a = t["assumed"]
    for p_str, printed in t["printed"].items():
        prunes = oflops.fastav_schedule(a["tokens"], t["num_layers"], t["global_layer"], a["global_keep"], int(p_str) / 100.0)
        mine = pflops.schedule_flops(a["tokens"], prunes, t["num_layers"], a["hidden"], a["ffn"])
        assert mine["relative"] == pytest.approx(oflops.relative_flops(a["tokens"], t["num_layers"], a["hidden"], a["ffn"], prunes), rel=1e-12)
        assert abs(mine["relative"] - printed) <= t["tolerance_points"]
        assert mine["removed"] == oflops.flops_removed(a["tokens"], t["num_layers"], a["hidden"], a["ffn"], prunes)
    # the long audio-video workload's own schedule, per sequence
    w = W.WORKLOADS["c4_long_av"]
    lens = W.stage_lengths(w)
    m = w.model
    sched = {st.layer: lens[si + 1][0] for si, st in enumerate(w.stages)}
    mine = pflops.schedule_flops(lens[0][0], sched, m.num_layers, m.hidden, m.ffn)
    assert mine["relative"] == pytest.approx(oflops.relative_flops(lens[0][0], m.num_layers, m.hidden, m.ffn, sched), rel=1e-12)
    assert mine["removed"] == oflops.flops_removed(lens[0][0], m.num_layers, m.hidden, m.ffn, sched)
    # flops_removed itself, by hand: 3 layers of 10 tokens, D = 2, m = 3, prune to 4 tokens at layer 1:
    # layer cost(n) = 4 n 4 + 2 n^2 2 + 2 n 6 = 28 n + 4 n^2 -> cost(10) = 680, cost(4) = 176; layers 2 and 3 save 504 each
    assert oflops.flops_removed(10, 3, 2, 3, {1: 4}) == 1008
    assert oflops.relative_flops(10, 3, 2, 3, {1: 4}) == pytest.approx(100.0 * (680 + 176 + 176) / (3 * 680))


def test_mask_selection_equals_score_selection_on_indicator_scores():
    """A keep mask is the special case of the score rule in which kept tokens score 1, dropped ones 0 and
    k is the number of ones: the two oracle routes must agree (ties among the ones go to the lower index,
    which is ascending order)."""
    rng = np.random.default_rng(3)
    lens = [0, 1, 17, 64, 5]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    mask = (rng.random(cu[-1]) < 0.4).astype(np.uint8)
    mask[cu[2]:cu[2] + 3] = 1
    counts = [int(mask[cu[b]:cu[b + 1]].sum()) for b in range(len(lens))]
    by_mask, cu_mask = oracle.select_mask(mask, cu)
    by_score, cu_score = oracle.select(mask.astype(np.float32), cu, counts)
    assert cu_mask.tolist() == cu_score.tolist() == np.concatenate([[0], np.cumsum(counts)]).tolist()
    assert by_mask.tolist() == by_score.tolist()
    glob, _ = oracle.select_mask(mask, cu, global_index=True)
    assert glob.tolist() == np.nonzero(mask)[0].tolist()
