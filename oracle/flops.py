"""Theoretical prefill FLOPs of a pruned decoder, relative to the unpruned one (= 100).

TEST INFRASTRUCTURE ONLY (part of the CPU oracle).  The paper reports "FLOPs ... relative to
the original theoretical one (set to 100)" following the FastV line of work (Section 3.1,
"Evaluation protocol"; Tables 1, 2 and 4) without printing the formula.  The count used here
is the usual per-layer one for a decoder layer that sees n tokens of width D with an FFN of
width m:

    attention projections 4 n D^2  +  attention map and mix 2 n^2 D  +  FFN 2 n D m

A prune at layer l changes the token count seen by layers l+1, l+2, ...  (the pruning layer
itself still runs on the tokens it was handed).
"""
from __future__ import annotations

import math


def layer_flops(n: int, hidden: int, ffn: int) -> int:
    return 4 * n * hidden * hidden + 2 * n * n * hidden + 2 * n * hidden * ffn


def removed_count(n: int, prune_ratio: float) -> int:
    """Tokens removed by the bottom-P % rule (Section 2.2, "Fine pruning") from n tokens: floor(P n)."""
    return int(math.floor(prune_ratio * n + 1e-6))


def token_schedule(n0: int, num_layers: int, prunes: dict[int, int]) -> list[int]:
    """Tokens seen by layers 1..num_layers when ``prunes[l]`` tokens survive the prune done at
    layer l (1-based)."""
    seen, n = [], n0
    for layer in range(1, num_layers + 1):
        seen.append(n)
        if layer in prunes:
            n = prunes[layer]
    return seen


def relative_flops(n0: int, num_layers: int, hidden: int, ffn: int, prunes: dict[int, int]) -> float:
    """100 * FLOPs(pruned schedule) / FLOPs(no pruning)."""
    seen = token_schedule(n0, num_layers, prunes)
    return 100.0 * sum(layer_flops(n, hidden, ffn) for n in seen) / (num_layers * layer_flops(n0, hidden, ffn))


def fastav_schedule(n0: int, num_layers: int, global_layer: int, global_keep: int, fine_ratio: float) -> dict[int, int]:
    """The paper's two-stage schedule: a global prune at the middle layer, then the bottom P %
    removed at every following layer (Section 2.2; P = 20% in Section 3.1)."""
    prunes = {global_layer: global_keep}
    n = global_keep
    if fine_ratio > 0:
        for layer in range(global_layer + 1, num_layers + 1):
            n = n - removed_count(n, fine_ratio)
            prunes[layer] = n
    return prunes


def flops_removed(n0: int, num_layers: int, hidden: int, ffn: int, prunes: dict[int, int]) -> int:
    """Absolute prefill FLOPs the schedule saves."""
    seen = token_schedule(n0, num_layers, prunes)
    return sum(layer_flops(n0, hidden, ffn) - layer_flops(n, hidden, ffn) for n in seen)
