"""Prefill FLOPs a pruning schedule removes (reporting utility of the benchmark).

The paper reports theoretical FLOPs relative to the unpruned model (= 100), "as in" the FastV line
of work (Section 3.1, Tables 1, 2 and 4).  Per decoder layer that sees n tokens of width D with an
FFN of width m this counts ``4 n D^2 + 2 n^2 D + 2 n D m``; a prune at layer l changes what layers
l+1, l+2, ... see.
"""
from __future__ import annotations


def _layer(n: int, hidden: int, ffn: int) -> int:
    return n * (4 * hidden * hidden + 2 * n * hidden + 2 * hidden * ffn)


def schedule_flops(tokens_in: int, survivors_by_layer: dict[int, int], num_layers: int, hidden: int, ffn: int) -> dict:
    """``survivors_by_layer[l]``: tokens left after the prune done at (1-based) layer l."""
    n, pruned = tokens_in, 0
    for layer in range(1, num_layers + 1):
        pruned += _layer(n, hidden, ffn)
        n = survivors_by_layer.get(layer, n)
    full = num_layers * _layer(tokens_in, hidden, ffn)
    return {"full": full, "pruned": pruned, "removed": full - pruned, "relative": 100.0 * pruned / full}
