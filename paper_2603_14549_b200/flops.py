"""Theoretical FLOPs of the LLM backbone attributable to the image tokens (App. A of the paper), and the
key / value cache storage of a pruning schedule (Sec. 5.5, Table 4).

Host-side accounting only; nothing here touches the GPU or the prune step.  One decoder layer
that sees v image tokens costs 4 v d^2 + 2 v^2 d + 3 v d m (attention projections, attention
itself, feed-forward), with d the hidden size and m the feed-forward width (App. A); a schedule
that prunes S times is the sum over its stages of layers * layer_cost(v_n) (Eq. 6), and the
FLOPs ratio divides by the unpruned total L * layer_cost(v_0) (Eq. 7).
"""
from __future__ import annotations

from typing import Sequence, Tuple


def layer_flops(v: int, d: int, m: int) -> int:
    """FLOPs of one decoder layer for v image tokens (App. A)."""
    return 4 * v * d * d + 2 * v * v * d + 3 * v * d * m


def schedule_flops(stages: Sequence[Tuple[int, int]], d: int, m: int) -> int:
    """Eq. 6: `stages` lists (number of layers, image tokens seen by those layers)."""
    return sum(layers * layer_flops(v, d, m) for layers, v in stages)


def flops_ratio(stages: Sequence[Tuple[int, int]], v0: int, d: int, m: int) -> float:
    """Eq. 7: schedule FLOPs over the FLOPs of all its layers at the unpruned token count v0."""
    total_layers = sum(layers for layers, _ in stages)
    return schedule_flops(stages, d, m) / (total_layers * layer_flops(v0, d, m))


def single_prune_stages(total_layers: int, prune_layer: int, v0: int, keep: int):
    """The paper's setting (Sec. 5.1): prune once, after decoder layer index `prune_layer`; layers
    0 .. prune_layer see v0 image tokens, the rest see `keep`."""
    first = prune_layer + 1
    return [(first, v0), (total_layers - first, keep)]


def kv_cache_bytes(stages: Sequence[Tuple[int, int]], d: int, bytes_per_element: int = 2) -> int:
    """Key / value cache storage of a prefill (Sec. 5.5, Table 4, column "Storage"): every layer keeps
    one key row and one value row of width d per token it saw.  `stages` lists (number of layers,
    tokens of the whole sequence seen by those layers), as in schedule_flops."""
    return sum(layers * tokens * 2 * d * bytes_per_element for layers, tokens in stages)


def kv_storage_bytes(rows_before: int, rows_after: int, layers: int, d: int, bytes_per_element: int = 2) -> dict:
    """What compacting the cached keys and values of `layers` layers from rows_before to rows_after
    rows saves (the layers up to the pruning layer, which cached every token before the prune step)."""
    before = kv_cache_bytes([(layers, rows_before)], d, bytes_per_element)
    after = kv_cache_bytes([(layers, rows_after)], d, bytes_per_element)
    return {"layers": layers, "bytes_before": before, "bytes_after": after, "bytes_saved": before - after}
