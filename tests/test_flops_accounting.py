"""App. A's FLOPs accounting against the figures the paper prints (tests/golden/flops_table.json)."""
import json
import os

import pytest

from paper_2603_14549_b200 import flops as F

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "flops_table.json")))


@pytest.mark.parametrize("row", GOLD["rows"], ids=lambda r: f"{r['tokens']} tokens")
def test_printed_flops_are_reproduced(row):
    got = GOLD["layers"] * F.layer_flops(row["tokens"], GOLD["d"], GOLD["m"]) / 1e12
    # the paper prints three decimals, some rounded and some truncated (6.4586 appears as 6.458)
    assert abs(got - row["tflops"]) < 1e-3, (got, row)


@pytest.mark.parametrize("row", GOLD["other_backbones"], ids=lambda r: f"{r['tokens']} tokens, m={r['m']}")
def test_printed_flops_of_the_other_backbone(row):
    got = row["layers"] * F.layer_flops(row["tokens"], row["d"], row["m"]) / 1e12
    assert abs(got - row["tflops"]) < 1e-3, (got, row)


def test_schedule_and_ratio():
    d, m, L = GOLD["d"], GOLD["m"], GOLD["layers"]
    full = F.schedule_flops([(L, 576)], d, m)
    assert full == L * F.layer_flops(576, d, m)
    assert F.flops_ratio([(L, 576)], 576, d, m) == 1.0
    stages = F.single_prune_stages(L, 2, 576, 192)          # prune once after layer index 2 (Sec. 5.1)
    assert stages == [(3, 576), (29, 192)]
    assert F.schedule_flops(stages, d, m) == 3 * F.layer_flops(576, d, m) + 29 * F.layer_flops(192, d, m)
    r = F.flops_ratio(stages, 576, d, m)
    assert F.layer_flops(192, d, m) / F.layer_flops(576, d, m) < r < 1.0
    # the quadratic term: halving the tokens more than halves the attention part
    assert F.layer_flops(288, d, m) * 2 < F.layer_flops(576, d, m)


@pytest.mark.parametrize("row", GOLD["kv_storage"]["rows"], ids=lambda r: f"{r['tokens']} tokens")
def test_printed_kv_storage_is_reproduced(row):
    g = GOLD["kv_storage"]
    got = F.kv_cache_bytes([(g["layers"], row["tokens"])], g["d"], g["bytes_per_element"]) / 1e6
    assert abs(got - row["mb"]) < 5e-3, (got, row)


def test_kv_storage_of_a_schedule_and_of_a_compaction():
    g = GOLD["kv_storage"]
    d, L = g["d"], g["layers"]
    per_token_layer = 2 * d * 2
    stages = [(3, 613), (29, 229)]                      # prune 576 -> 192 image tokens after layer index 2
    assert F.kv_cache_bytes(stages, d) == (3 * 613 + 29 * 229) * per_token_layer
    # no single prune after an integer layer gives the pruned rows the paper prints (see the fixture)
    singles = [F.kv_cache_bytes([(k, 613), (L - k, 229)], d) / 1e6 for k in range(L + 1)]
    assert all(min(abs(s - mb) for s in singles) > 0.5 for mb in g["not_reproduced_mb"][:2])
    s = F.kv_storage_bytes(613, 229, 3, d)
    assert s["bytes_before"] - s["bytes_after"] == s["bytes_saved"] == 3 * (613 - 229) * per_token_layer
