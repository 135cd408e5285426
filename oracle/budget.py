"""Bookkeeping formulas the paper states in closed form (TEST INFRASTRUCTURE, see package note).

Pinned by the values the paper prints (tests/golden/).
"""
from __future__ import annotations


def average_retention(r1: float, r2: float, k: int, layers: int) -> float:
    """App. B.1 ("fair comparisons"): layers before the pruning layer k see the Stage-1 set
    (fraction r1 of the tokens), layers from k on see the Stage-2 survivors (r1 * r2); the
    reported rate is the mean over all LLM layers."""
    return (k * r1 + (layers - k) * r1 * r2) / layers


def average_tokens(n_before: int, n_after: int, k: int, layers: int) -> float:
    """Same statement in token counts (App. B.1: 96 before, 32 from layer 16 of 32 on)."""
    return (k * n_before + (layers - k) * n_after) / layers


def prefill_flops(tokens_per_layer, d: int, m: int) -> float:
    """Eq. 6 (App. B.2): sum over layers of 4 n d^2 + 2 n^2 d + 3 n d m."""
    return float(sum(4 * n * d * d + 2 * n * n * d + 3 * n * d * m for n in tokens_per_layer))


def vscan_tokens_per_layer(n_stage1: int, n_stage2: int, k: int, layers: int):
    return [n_stage1] * k + [n_stage2] * (layers - k)
