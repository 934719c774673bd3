"""Pins for the attention-rollout oracle (Section 2.1, Eq. 2 and Eq. 3): hand-worked matrices, a closed form,
invariants, and two independent routes to the head-mean attention map (torch.softmax in float64, and the
column means against the plain-C Eq. 4 oracle scoring every row).  No GPU needed."""
import math

import numpy as np
import torch

import oracle
from oracle import rollout as orr
from conftest import to_bf16_bits


def _random_qk(seed, n, hq, hkv, d):
    rng = np.random.default_rng(seed)
    return to_bf16_bits(rng.standard_normal((n, hq, d)).astype(np.float32)), to_bf16_bits(rng.standard_normal((n, hkv, d)).astype(np.float32))


def test_eq3_multiplies_the_newest_layer_from_the_left():
    # two row-stochastic matrices that do not commute
    a1 = np.array([[1.0, 0.0], [0.5, 0.5]])
    a2 = np.array([[0.5, 0.5], [0.0, 1.0]])
    assert np.allclose(orr.rollout([a1, a2], 1.0), [[0.75, 0.25], [0.5, 0.5]], atol=0, rtol=1e-15)       # A2 A1 by hand
    assert not np.allclose(orr.rollout([a2, a1], 1.0), [[0.75, 0.25], [0.5, 0.5]])
    # Eq. 2 with alpha = 1/2: A~1 = [[1,0],[1/4,3/4]], A~2 = [[3/4,1/4],[0,1]]; A~2 A~1 = [[13/16,3/16],[1/4,3/4]]
    assert np.allclose(orr.rollout([a1, a2], 0.5), [[13 / 16, 3 / 16], [0.25, 0.75]], atol=0, rtol=1e-15)


def test_hand_worked_fixture(golden_dir):
    import json
    import os
    with open(os.path.join(golden_dir, "eq23_hand_worked.json")) as f:
        cases = json.load(f)["cases"]
    assert len(cases) >= 3
    for c in cases:
        r = orr.rollout([np.array(m) for m in c["maps"]], c["alpha"])
        assert np.allclose(r, np.array(c["rollout"]), rtol=1e-14, atol=0), c["name"]
        if "importance" in c:
            assert np.allclose(orr.importance(r), c["importance"], rtol=1e-14), c["name"]


def test_eq2_limits():
    rng = np.random.default_rng(0)
    a = rng.random((5, 5))
    a /= a.sum(axis=1, keepdims=True)
    assert np.array_equal(orr.rollout([a, a, a], 0.0), np.eye(5))            # alpha = 0: only the residual
    assert np.allclose(orr.rollout([a], 1.0), a)                              # one layer, alpha = 1: the map itself
    assert np.allclose(orr.with_residual(a, 0.25), 0.25 * a + 0.75 * np.eye(5))


def test_uniform_attention_closed_form():
    """All keys equal, no mask: A = J/n; (alpha J/n + (1-alpha) I)^L = (1 - (1-alpha)^L) J/n + (1-alpha)^L I."""
    n, hq, hkv, d, alpha, layers = 7, 4, 2, 8, 0.3, 5
    q, _ = _random_qk(1, n, hq, hkv, d)
    k = to_bf16_bits(np.ones((n, hkv, d), dtype=np.float32))
    a = orr.attention_map(q, k, 0.7, causal=False)
    assert np.allclose(a, 1.0 / n, rtol=1e-13)
    r = orr.rollout([a] * layers, alpha)
    rest = (1 - alpha) ** layers
    assert np.allclose(r, (1 - rest) / n + rest * np.eye(n), rtol=1e-12)
    assert np.allclose(orr.importance(r), 1.0 / n, rtol=1e-12)


def test_causal_map_of_equal_keys_by_hand():
    q, _ = _random_qk(2, 3, 2, 1, 4)
    k = to_bf16_bits(np.zeros((3, 1, 4), dtype=np.float32))
    a = orr.attention_map(q, k, 1.0, causal=True)
    assert np.allclose(a, [[1, 0, 0], [0.5, 0.5, 0], [1 / 3, 1 / 3, 1 / 3]], rtol=1e-15)
    # rollout of two such layers with alpha = 1: second row [3/4, 1/4, 0], third row [11/18, 5/18, 1/9]
    r = orr.rollout([a, a], 1.0)
    assert np.allclose(r, [[1, 0, 0], [0.75, 0.25, 0], [11 / 18, 5 / 18, 1 / 9]], rtol=1e-14)
    assert np.allclose(orr.importance(r), [(1 + 0.75 + 11 / 18) / 3, (0.25 + 5 / 18) / 3, 1 / 27], rtol=1e-14)


def test_map_against_torch_softmax_and_against_the_eq4_oracle():
    n, hq, hkv, d, scale = 23, 6, 2, 16, 0.31
    q, k = _random_qk(3, n, hq, hkv, d)
    for causal in (True, False):
        a = orr.attention_map(q, k, scale, causal)
        qf = torch.from_numpy((q.astype(np.uint32) << 16).view(np.float32)).double()
        kf = torch.from_numpy((k.astype(np.uint32) << 16).view(np.float32)).double().repeat_interleave(hq // hkv, dim=1)
        z = torch.einsum("ihd,jhd->hij", qf, kf) * scale
        if causal:
            z = z.masked_fill(torch.ones(n, n).triu(1).bool(), float("-inf"))
        ref = torch.softmax(z, dim=-1).mean(dim=0).numpy()
        assert np.allclose(a, ref, rtol=1e-12, atol=1e-15)
        assert np.allclose(a.sum(axis=1), 1.0, rtol=1e-13)
        if causal:
            assert np.array_equal(np.triu(a, 1), np.zeros_like(a))
        # Eq. 4 with every token a scored row is the column mean of the head-mean map (plain-C oracle)
        s = oracle.score(q, k, [0, n], [0, n], np.arange(n), scale, causal)
        assert np.allclose(s, a.mean(axis=0), rtol=1e-12, atol=1e-15)


def test_gqa_mapping_is_contiguous_groups():
    """Hq = 4, Hkv = 2, q = [+1, +1, -1, -1] on coordinate 0, KV head 0 keys [1, 0], KV head 1 keys [0, 1], scale ln 3:
    heads 0, 1 give [3/4, 1/4]; heads 2, 3 (KV head 1, q = -1) give [3/4, 1/4] -> every row [3/4, 1/4].  An
    interleaved mapping would give [1/2, 1/2]."""
    q = np.zeros((2, 4, 4), dtype=np.float32)
    q[:, :, 0] = [1, 1, -1, -1]
    k = np.zeros((2, 2, 4), dtype=np.float32)
    k[0, 0, 0] = 1
    k[1, 1, 0] = 1
    a = orr.attention_map(to_bf16_bits(q), to_bf16_bits(k), math.log(3.0), causal=False)
    assert np.allclose(a, [[0.75, 0.25], [0.75, 0.25]], rtol=1e-13)


def test_rollout_invariants():
    n, hq, hkv, d = 31, 4, 4, 8
    maps = [orr.attention_map(*_random_qk(10 + l, n, hq, hkv, d), 0.4, True) for l in range(4)]
    r = orr.rollout(maps, 0.6)
    assert np.allclose(r.sum(axis=1), 1.0, rtol=1e-12)                 # products of row-stochastic matrices
    assert np.array_equal(np.triu(r, 1), np.zeros_like(r))             # causal maps stay lower triangular
    assert (r >= 0).all()
    assert np.isclose(orr.importance(r).sum(), 1.0, rtol=1e-12)
    assert np.allclose(r[0], np.eye(n)[0])                             # the first token only ever sees itself


def test_threshold_rule_by_hand():
    imp = np.array([0.4, 0.3, 0.02, 0.2, 0.03, 0.05])
    keep, cut = orr.threshold_rule(imp, 0.05)
    assert keep.tolist() == [1, 1, 0, 1, 0, 1] and cut == 6
    keep, cut = orr.threshold_rule(imp, 0.1)
    assert keep.tolist() == [1, 1, 0, 1, 0, 0] and cut == 4
    keep, cut = orr.threshold_rule(imp, 0.1, protect=[0, 0, 0, 0, 0, 1])   # the text suffix always survives
    assert keep.tolist() == [1, 1, 0, 1, 0, 1] and cut == 4
    keep, cut = orr.threshold_rule(imp, 0.9)
    assert keep.tolist() == [0] * 6 and cut == 0
