"""Pins for the CPU oracle: hand-worked fixtures, closed forms, invariants and special cases
that reduce to a library routine.  None of these re-types an oracle formula; each is chosen
so that a plausible slip (dropped term, wrong axis, wrong sign, transposed operand, wrong tie
rule) fails at least one of them.  The last block plants such slips and checks they are caught."""
import json
import math
import os
import types

import numpy as np
import pytest
import torch

from oracle import asap_oracle as O
from paper_2603_14549_b200 import workloads as W
from tests.helpers import bits, sample_np

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_worked.json")))


def _ninf(rows):
    return np.array([[-np.inf if v == "ninf" else float(v) for v in r] for r in rows])


def _rand_qk(n, H, d, seed):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((n, H, d)), rng.standard_normal((n, H, d))


# ----------------------------------------------------------------------------- bf16
def test_bf16_widening_matches_torch():
    u = np.arange(0, 65536, dtype=np.uint32).astype(np.uint16)
    t = torch.from_numpy(u.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    o = O.bf16_bits_to_f64(u)
    ok = np.isfinite(t)
    assert np.array_equal(o[ok], t[ok])


def test_bf16_rounding_matches_torch_on_f32_inputs():
    rng = np.random.default_rng(1)
    x32 = np.concatenate([rng.standard_normal(20000).astype(np.float32) * 7.0,
                          np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.0e38, 1e-40], np.float32)])
    want = bits(torch.from_numpy(x32).to(torch.bfloat16))
    got = O.f64_to_bf16_bits(x32.astype(np.float64))
    assert np.array_equal(got, want)


def test_bf16_rounding_is_single_rounding():
    # 1 + 2^-8 + 2^-30 lies just above the midpoint of bf16 neighbours 1.0 and 1.0078125.
    # Rounding first to binary32 (-> exactly the midpoint) and then to bf16 would tie to even (1.0).
    x = np.array([1.0 + 2.0 ** -8 + 2.0 ** -30, -(1.0 + 2.0 ** -8 + 2.0 ** -30), 1.0 + 2.0 ** -8])
    got = O.bf16_bits_to_f64(O.f64_to_bf16_bits(x))
    assert got.tolist() == [1.0078125, -1.0078125, 1.0]


# ----------------------------------------------------------------------------- Eq. 1-3
def check_hand_mass(o):
    g = GOLD["mass_salience_mask"]
    q = np.array(g["Q"], float)[:, None, :]
    k = np.array(g["K"], float)[:, None, :]
    assert np.allclose(o.alignment(q, k, 0), np.array(g["W"]), atol=1e-15)
    s = o.attention_mass(q, k, 0, 3)
    assert np.allclose(s, g["s"], atol=1e-15)
    s_hat = o.salience(s, 1e-6)
    assert np.allclose(s_hat, g["s_hat"], rtol=1e-14, atol=0)
    m = o.mask_log(s_hat, g["lambda_max"], 1e-6)
    assert np.allclose(m, g["m"], rtol=1e-13, atol=0)


def test_hand_mass_salience_mask():
    check_hand_mass(O)


def check_mass_summed_query(o):
    """Closed form: sum_i (q_i . k_j) = (sum_i q_i) . k_j, per head, averaged over heads."""
    n, H, d, v0, nv = 11, 3, 8, 2, 6
    q, k = _rand_qk(n, H, d, 5)
    s = o.attention_mass(q, k, v0, nv)
    qbar = q[v0:v0 + nv].sum(axis=0)                                   # [H, d]
    want = np.einsum("hd,jhd->j", qbar, k[v0:v0 + nv]) / (H * math.sqrt(d))
    assert np.allclose(s, want, rtol=1e-12, atol=1e-12)


def test_mass_summed_query_identity():
    check_mass_summed_query(O)


def test_mass_ignores_tokens_outside_span():
    n, H, d, v0, nv = 9, 2, 4, 3, 4
    q, k = _rand_qk(n, H, d, 6)
    s0 = O.attention_mass(q, k, v0, nv)
    q2, k2 = q.copy(), k.copy()
    q2[:v0] += 100.0; k2[v0 + nv:] -= 50.0; q2[v0 + nv:] *= 3.0; k2[:v0] = 7.0
    assert np.array_equal(O.attention_mass(q2, k2, v0, nv), s0)


def test_salience_range_extremes_affine():
    rng = np.random.default_rng(3)
    s = rng.standard_normal(50) * 40 - 300           # deeply negative logits are expected
    h = O.salience(s, 1e-6)
    assert h.min() == 0.0 and h[np.argmin(s)] == 0.0
    d = s.max() - s.min()
    assert math.isclose(h[np.argmax(s)], d / (d + 1e-6), rel_tol=1e-15)
    assert np.all((h >= 0) & (h < 1))
    assert np.allclose(O.salience(3.0 * s + 11.0, 1e-6), h, rtol=1e-6)   # affine-invariant up to eps
    assert np.array_equal(np.argsort(h, kind="stable"), np.argsort(s, kind="stable"))
    assert np.array_equal(O.salience(np.full(4, 2.5), 1e-6), np.zeros(4))  # flat span -> all zero


def test_mask_log_floor_and_top():
    m = O.mask_log(np.array([0.0, 1e-9, 0.5, 1.0]), 1.0, 1e-6)
    assert m[0] == math.log(1e-6) and m[1] == math.log(1e-6)
    assert m[2] == math.log(0.5) and m[3] == 0.0
    assert np.all(O.mask_log(np.linspace(0, 1, 9), 0.25, 1e-6) <= math.log(0.25))


# ----------------------------------------------------------------------------- Eq. 3-4
def check_hand_mask_matrix(o):
    g = GOLD["mask_matrix"]
    rows = np.arange(g["n"])
    m = np.array(g["m"])
    assert np.array_equal(o.mask_matrix(g["n"], rows, g["v0"], g["nv"], m, True), _ninf(g["M_enabled"]))
    assert np.array_equal(o.mask_matrix(g["n"], rows, g["v0"], g["nv"], m, False), _ninf(g["M_disabled"]))
    sub = np.array([4, 2])
    assert np.array_equal(o.mask_matrix(g["n"], sub, g["v0"], g["nv"], m, True), _ninf(g["M_enabled"])[sub])


def test_hand_mask_matrix():
    check_hand_mask_matrix(O)


def check_rank_zero_logits(o):
    g = GOLD["rank_zero_logits"]
    n, H, d = g["n"], 2, 4
    q = np.zeros((n, H, d))
    k = np.random.default_rng(0).standard_normal((n, H, d))
    m = np.log(np.array(g["lambda"]))
    r = o.rank_scores(q, k, g["v0"], g["nv"], g["r0"], g["nr"], m, True)
    assert np.allclose(r, g["r_enabled"], rtol=1e-14, atol=0)
    r = o.rank_scores(q, k, g["v0"], g["nv"], g["r0"], g["nr"], m, False)
    assert np.allclose(r, g["r_disabled"], rtol=1e-14, atol=0)


def test_rank_zero_logits_closed_form():
    check_rank_zero_logits(O)


def check_causal_matches_library_softmax(o):
    """Mask off: A is the ordinary causal softmax; compare with torch's float64 softmax."""
    n, H, d, v0, nv = 14, 3, 8, 2, 7
    q, k = _rand_qk(n, H, d, 7)
    q *= 2.0
    r0, nr = v0 + nv, n - (v0 + nv)
    r = o.rank_scores(q, k, v0, nv, r0, nr, None, False)
    tq, tk = torch.from_numpy(q), torch.from_numpy(k)
    logits = torch.einsum("ihd,jhd->hij", tq, tk) / math.sqrt(d)
    causal = torch.full((n, n), float("-inf"), dtype=torch.float64).triu(1)
    A = torch.softmax(logits + causal, dim=-1)                     # [H, n, n]
    want = A[:, r0:r0 + nr, v0:v0 + nv].mean(dim=(0, 1)).numpy()
    assert np.allclose(r, want, rtol=1e-12, atol=1e-15)
    # ... and with visual ranking rows too (upper triangle exactly zero)
    r2 = o.rank_scores(q, k, v0, nv, v0, n - v0, None, False)
    want2 = A[:, v0:, v0:v0 + nv].mean(dim=(0, 1)).numpy()
    assert np.allclose(r2, want2, rtol=1e-12, atol=1e-15)


def test_causal_matches_library_softmax():
    check_causal_matches_library_softmax(O)


def check_multiplicative_form(o):
    """Second formulation of Eq. 4: weights lambda_j * exp(W_ij) instead of adding ln lambda_j."""
    n, H, d, v0, nv = 12, 2, 8, 1, 8
    q, k = _rand_qk(n, H, d, 8)
    lam = np.random.default_rng(9).uniform(0.05, 1.0, nv)
    rows = np.arange(v0, n)
    r = o.rank_scores(q, k, v0, nv, v0, n - v0, np.log(lam), True)
    want = np.zeros(nv)
    for h in range(H):
        for i in rows:
            w = np.zeros(n)
            for j in range(n):
                e = math.exp(float(q[i, h] @ k[j, h]) / math.sqrt(d))
                if j <= i:
                    w[j] = e
                elif v0 <= i < v0 + nv and v0 <= j < v0 + nv:
                    w[j] = lam[j - v0] * e
            want += w[v0:v0 + nv] / w.sum()
    want /= H * len(rows)
    assert np.allclose(r, want, rtol=1e-11, atol=1e-15)


def test_multiplicative_form_of_eq4():
    check_multiplicative_form(O)


def test_probability_rows_sum_to_one_and_text_rows_ignore_mask():
    n, H, d, v0, nv = 13, 2, 8, 2, 8
    q, k = _rand_qk(n, H, d, 10)
    m = np.log(np.random.default_rng(2).uniform(0.1, 1.0, nv))
    rows = np.arange(n)
    for h in range(H):
        A = O.attention_probs(q, k, h, rows, v0, nv, m, True)
        assert np.allclose(A.sum(axis=1), 1.0, rtol=1e-13)
        assert np.all(np.triu(A[:v0], 1) == 0.0)                 # system rows stay causal
        # every row: nothing leaks to future TEXT keys
        for i in range(n):
            assert np.all(A[i, max(i + 1, v0 + nv):] == 0.0)
        # visual rows do see later visual keys
        assert np.all(A[v0, v0 + 1:v0 + nv] > 0.0)
        # rows after the span are identical with and without the mask (mask term is 0 there)
        B_ = O.attention_probs(q, k, h, rows, v0, nv, m, False)
        assert np.array_equal(A[v0 + nv:], B_[v0 + nv:])
    r_text_on = O.rank_scores(q, k, v0, nv, v0 + nv, n - v0 - nv, m, True)
    r_text_off = O.rank_scores(q, k, v0, nv, v0 + nv, n - v0 - nv, m, False)
    assert np.array_equal(r_text_on, r_text_off)
    assert r_text_on.sum() <= 1.0


def test_tiny_lambda_approaches_causal():
    n, H, d, v0, nv = 12, 2, 8, 1, 8
    q, k = _rand_qk(n, H, d, 11)
    s_hat = np.random.default_rng(4).uniform(0, 1, nv)
    m = O.mask_log(s_hat, 1e-9, 1e-6)                     # floors at ln(eps) everywhere
    assert np.all(m == math.log(1e-6))
    r_soft = O.rank_scores(q, k, v0, nv, v0, n - v0, m, True)
    r_caus = O.rank_scores(q, k, v0, nv, v0, n - v0, m, False)
    assert np.max(np.abs(r_soft - r_caus)) < 1e-3 and not np.array_equal(r_soft, r_caus)


def test_head_permutation_invariance():
    n, H, d, v0, nv = 12, 4, 8, 2, 6
    q, k = _rand_qk(n, H, d, 12)
    perm = np.array([2, 0, 3, 1])
    s = O.attention_mass(q, k, v0, nv)
    m = O.mask_log(O.salience(s), 0.7)
    r = O.rank_scores(q, k, v0, nv, v0, n - v0, m, True)
    assert np.allclose(O.attention_mass(q[:, perm], k[:, perm], v0, nv), s, rtol=1e-13)
    assert np.allclose(O.rank_scores(q[:, perm], k[:, perm], v0, nv, v0, n - v0, m, True), r, rtol=1e-13)


# ----------------------------------------------------------------------------- top-k
def check_hand_topk(o):
    g = GOLD["topk_ties"]
    r = np.array(g["r"])
    for c in g["cases"]:
        keep, drop = o.select_topk(r, c["k"])
        assert keep.tolist() == c["keep"] and drop.tolist() == c["drop"]


def test_hand_topk_ties():
    check_hand_topk(O)


def test_topk_matches_library_stable_sort():
    rng = np.random.default_rng(13)
    r = np.round(rng.uniform(0, 1, 300), 2)              # many exact ties
    for kk in (1, 17, 150, 299, 300):
        keep, drop = O.select_topk(r, kk)
        order = np.argsort(-r, kind="stable")            # stable: equal keys keep index order
        assert keep.tolist() == sorted(order[:kk].tolist())
        assert sorted(keep.tolist() + drop.tolist()) == list(range(300))
        assert np.all(np.diff(keep) > 0) and np.all(np.diff(drop) > 0)


# ----------------------------------------------------------------------------- cosine / merge
def check_hand_cosine(o):
    g = GOLD["cosine_assign"]
    h = np.array(g["h"], float)
    keep, drop = np.array(g["keep"]), np.array(g["drop"])
    a, best, margin = o.cosine_assign(h, keep, drop, -math.inf)
    assert a.tolist() == g["assign_t_neg_inf"]
    assert np.allclose(best, g["best"], rtol=1e-15, atol=1e-16)
    assert margin[0] == 0.0 and math.isclose(margin[1], 1.0)
    assert o.cosine_assign(h, keep, drop, 0.0)[0].tolist() == g["assign_t_0"]
    assert o.cosine_assign(h, keep, drop, 1.0)[0].tolist() == g["assign_t_1"]


def test_hand_cosine_assign():
    check_hand_cosine(O)


def test_cosine_matches_library():
    rng = np.random.default_rng(14)
    h = rng.standard_normal((40, 32))
    h[5] = 0.0                                            # zero vector: similarity 0 by convention
    keep = np.arange(0, 40, 3); drop = np.setdiff1d(np.arange(40), keep)
    S = O.cosine_matrix(h[drop], h[keep])
    th = torch.from_numpy(h)
    want = torch.nn.functional.cosine_similarity(th[drop][:, None, :], th[keep][None, :, :], dim=-1, eps=1e-300).numpy()
    nz = drop != 5
    assert np.allclose(S[nz], want[nz], rtol=1e-13, atol=1e-15)
    assert np.all(S[~nz] == 0.0)
    a, best, _ = O.cosine_assign(h, keep, drop, -math.inf)
    assert np.array_equal(a[nz], want[nz].argmax(axis=1))
    assert a[~nz][0] == 0                                 # all-zero row: every slot ties at 0 -> slot 0


def check_hand_merge(o):
    g = GOLD["weighted_merge"]
    out = o.weighted_merge(np.array(g["h"], float), np.array(g["s_hat"]), np.array(g["keep"]),
                           np.array(g["drop"]), np.array(g["assign"]), 1e-6)
    assert np.allclose(out, g["merged"], rtol=1e-15, atol=0)


def test_hand_weighted_merge():
    check_hand_merge(O)


def test_merge_convex_and_weight_conserving():
    rng = np.random.default_rng(15)
    nv, D = 60, 16
    h = rng.standard_normal((nv, D))
    s_hat = rng.uniform(0.01, 1, nv)
    keep = np.sort(rng.choice(nv, 12, replace=False)); drop = np.setdiff1d(np.arange(nv), keep)
    assign = rng.integers(-1, 12, len(drop)).astype(np.int32)
    out = O.weighted_merge(h, s_hat, keep, drop, assign, 1e-6)
    total_w, total_wh = 0.0, np.zeros(D)
    for slot, i in enumerate(keep):
        members = np.concatenate([[i], drop[assign == slot]])
        lo, hi = h[members].min(axis=0), h[members].max(axis=0)
        assert np.all(out[slot] >= lo - 1e-12) and np.all(out[slot] <= hi + 1e-12)
        den = s_hat[members].sum()
        total_w += den; total_wh += den * out[slot]
    merged_members = np.concatenate([keep, drop[assign >= 0]])
    assert math.isclose(total_w, s_hat[merged_members].sum(), rel_tol=1e-13)
    assert np.allclose(total_wh, (s_hat[merged_members, None] * h[merged_members]).sum(axis=0), rtol=1e-12)


def test_merge_with_twin_is_unchanged():
    rng = np.random.default_rng(16)
    h = rng.standard_normal((6, 8)); h[4] = h[1]
    s_hat = np.array([0.3, 0.9, 0.1, 0.5, 0.2, 0.7])
    keep, drop = np.array([1, 3]), np.array([0, 2, 4, 5])
    a, best, _ = O.cosine_assign(h, keep, drop, 0.999999)
    assert a.tolist() == [-1, -1, 0, -1] and math.isclose(best[2], 1.0, rel_tol=1e-15)
    out = O.weighted_merge(h, s_hat, keep, drop, a, 1e-6)
    assert np.allclose(out[0], h[1], rtol=1e-15) and np.array_equal(out[1], h[3])


# ----------------------------------------------------------------------------- whole step
@pytest.fixture(scope="module")
def small_batch():
    return W.tiny(B=2, n_vis=[37, 20], text_lens=[5, 9], H=2, keep_k=8, seed=77, head_dim=16)


def _run(batch, b, **kw):
    s = sample_np(batch, b)
    r0 = int(batch.text_start[b]); nr = int(batch.text_len[b])
    kw.setdefault("keep_k", batch.keep_k)
    return O.prune_sample(s["q_bits"], s["k_bits"], s["hidden_bits"], s["pos_ids"], s["v0"], s["nv"],
                          kw.pop("r0", r0), kw.pop("nr", nr), **kw), s


def test_step_keeps_exactly_k_in_order(small_batch):
    for b in range(2):
        out, s = _run(small_batch, b)
        keep = out["keep_idx"]
        assert len(keep) == 8 and np.all(np.diff(keep) > 0)
        assert sorted(keep.tolist() + out["drop_idx"].tolist()) == list(range(s["nv"]))
        n_out = s["v0"] + 8 + int(small_batch.text_len[b])
        assert out["out_hidden_bits"].shape[0] == n_out == len(out["out_pos"]) == len(out["src_row"])
        assert np.array_equal(out["out_pos"], s["pos_ids"][out["src_row"]])     # gathered, not renumbered
        assert np.array_equal(out["out_hidden_bits"][:s["v0"]], s["hidden_bits"][:s["v0"]])
        assert np.array_equal(out["out_hidden_bits"][s["v0"] + 8:], s["hidden_bits"][s["v0"] + s["nv"]:])


def test_step_identity_when_k_equals_visual_count(small_batch):
    out, s = _run(small_batch, 1, keep_k=20)
    assert np.array_equal(out["out_hidden_bits"], s["hidden_bits"])
    assert np.array_equal(out["out_pos"], s["pos_ids"]) and len(out["drop_idx"]) == 0


def test_step_mask_off_merge_off_is_plain_attention_topk(small_batch):
    b = 0
    out, s = _run(small_batch, b, mask_enable=False, merge_enable=False)
    q = torch.from_numpy(O.bf16_bits_to_f64(s["q_bits"])); k = torch.from_numpy(O.bf16_bits_to_f64(s["k_bits"]))
    n, d = q.shape[0], q.shape[-1]
    A = torch.softmax(torch.einsum("ihd,jhd->hij", q, k) / math.sqrt(d)
                      + torch.full((n, n), float("-inf"), dtype=torch.float64).triu(1), dim=-1)
    t0 = s["v0"] + s["nv"]
    col = A[:, t0:, s["v0"]:t0].mean(dim=(0, 1))
    want_keep = torch.sort(torch.topk(col, 8).indices).values.numpy()
    assert np.array_equal(out["keep_idx"], want_keep)
    assert np.array_equal(out["out_hidden_bits"], s["hidden_bits"][out["src_row"]])   # pure gather
    assert np.all(out["assign"] == -1)


def test_step_threshold_one_means_no_merges(small_batch):
    out, s = _run(small_batch, 0, sim_threshold=1.0)
    assert np.all(out["assign"] == -1)
    assert np.array_equal(out["out_hidden_bits"], s["hidden_bits"][out["src_row"]])


def test_step_mask_changes_ranking_only_with_visual_rows(small_batch):
    s = sample_np(small_batch, 0)
    on, _ = _run(small_batch, 0, r0=s["v0"], nr=s["nv"] + 5, lambda_max=1.0)
    off, _ = _run(small_batch, 0, r0=s["v0"], nr=s["nv"] + 5, mask_enable=False)
    assert not np.allclose(on["rank_score"], off["rank_score"])
    # early visual tokens can only gain mass from the relaxed mask's extra admitted keys elsewhere:
    # the LAST visual key is never above any visual row's diagonal beyond itself, so its column only loses
    assert on["rank_score"][-1] > 0


# ----------------------------------------------------------------------------- planted slips
def _mutant():
    """A private copy of the oracle module whose functions can be replaced one at a time."""
    mod = types.ModuleType("mutant")
    src = open(O.__file__).read()
    exec(compile(src, "mutant", "exec"), mod.__dict__)
    return mod


PLANTED = [
    ("mass sums over keys instead of queries",
     lambda mod: dict(attention_mass=lambda q, k, v0, nv: sum(
         mod.alignment(q[v0:v0 + nv], k[v0:v0 + nv], h).sum(axis=1) for h in range(q.shape[1])) / q.shape[1]),
     [check_hand_mass, check_mass_summed_query]),
    ("alignment forgets the 1/sqrt(d)",
     lambda mod: dict(alignment=lambda q, k, h: q[:, h, :] @ k[:, h, :].T),
     [check_hand_mass, check_causal_matches_library_softmax]),
    ("mask admits future text keys for visual rows",
     lambda mod: dict(mask_matrix=lambda n, rows, v0, nv, m, en: np.array(
         [[0.0 if j <= i else (m[min(j - v0, nv - 1)] if en and v0 <= i < v0 + nv and j >= v0 else -np.inf)
           for j in range(n)] for i in rows])),
     [check_hand_mask_matrix, check_rank_zero_logits]),
    ("soft mask applied below the diagonal too",
     lambda mod: dict(mask_matrix=lambda n, rows, v0, nv, m, en: np.array(
         [[(m[j - v0] if en and v0 <= i < v0 + nv and v0 <= j < v0 + nv and j != i else (0.0 if j <= i else -np.inf))
           for j in range(n)] for i in rows])),
     [check_hand_mask_matrix, check_multiplicative_form]),
    ("top-k ties go to the higher index",
     lambda mod: dict(select_topk=lambda r, kk: (
         np.sort(np.lexsort((-np.arange(len(r)), -r))[:kk]).astype(np.int32),
         np.sort(np.lexsort((-np.arange(len(r)), -r))[kk:]).astype(np.int32))),
     [check_hand_topk]),
    ("merge forgets the destination's own weight in the denominator",
     lambda mod: dict(weighted_merge=lambda hv, sh, keep, drop, a, eps=1e-6: np.stack(
         [(sh[i] * hv[i] + sum(sh[j] * hv[j] for j in drop[a == s_])) / max(sum(sh[j] for j in drop[a == s_]), 1e-30)
          for s_, i in enumerate(keep)])),
     [check_hand_merge]),
    ("cosine threshold is not strict",
     lambda mod: dict(cosine_assign=lambda hv, keep, drop, t: (lambda S: (
         np.where(S.max(axis=1) >= t, S.argmax(axis=1), -1).astype(np.int32), S.max(axis=1),
         S.max(axis=1) - np.sort(S, axis=1)[:, -2]))(mod.cosine_matrix(hv[drop], hv[keep]))),
     [check_hand_cosine]),
]


@pytest.mark.parametrize("label,patch,checks", PLANTED, ids=[p[0] for p in PLANTED])
def test_planted_slip_is_caught(label, patch, checks):
    mod = _mutant()
    for name, fn in patch(mod).items():
        setattr(mod, name, fn)
    caught = 0
    for chk in checks:
        try:
            chk(mod)
        except AssertionError:
            caught += 1
    assert caught >= 1, f"no pin noticed: {label}"


# ----------------------------------------------------------------------------- KV-cache compaction
def test_compact_rows_is_a_row_gather():
    rng = np.random.default_rng(11)
    cache = rng.integers(0, 65535, size=(23, 6)).astype(np.uint16)
    src = np.array([0, 1, 2, 7, 9, 15, 21, 22], dtype=np.int32)
    got = O.compact_rows(cache, src)
    assert np.array_equal(got, cache[src])                          # library fancy indexing
    assert np.array_equal(O.compact_rows(cache, np.arange(23)), cache)            # identity map
    assert np.array_equal(O.compact_rows(cache, np.arange(23)[::-1]), cache[::-1])  # reversal
    assert got.dtype == cache.dtype and got.shape == (8, 6)


# ----------------------------------------------------------------------------- Sec. 4.2 inside the kept set
def check_hand_consolidation(o):
    g = GOLD["consolidate_within_kept"]
    h = np.array(g["h"], float)
    s_hat, mass = np.array(g["s_hat"]), np.array(g["mass"], float)
    keep, drop = np.array(g["keep"]), np.array(g["drop"])
    dest, _ = o.route_within_kept(h, s_hat, keep, g["t"])
    assert dest.tolist() == g["dest"]
    assert o.refill_from_pruned(mass, drop, 3).tolist() == g["refill"]
    hb = bits(torch.tensor(h, dtype=torch.float32).to(torch.bfloat16))
    r = o.consolidate_sample(hb, np.arange(10), 0, 10, mass, s_hat, keep, drop, g["t"])
    assert r["final_keep"].tolist() == g["final_keep"] and r["n_absorbed"] == 3
    for slot, row in g["merged_rows"].items():
        assert np.allclose(r["merged"][int(slot)], row, rtol=1e-15)
    assert r["merged_mask"].tolist() == [True, True, False, False, False]
    assert np.array_equal(r["out_hidden_bits"][2:], hb[[4, 6, 7]])          # refilled rows are copies


def test_hand_consolidation_within_kept():
    check_hand_consolidation(O)


def _clustered(n, D, centres, seed, spread=0.25):
    rng = np.random.default_rng(seed)
    c = rng.standard_normal((centres, D))
    h = c[rng.integers(0, centres, n)] + spread * rng.standard_normal((n, D))
    hb = bits(torch.tensor(h, dtype=torch.float32).to(torch.bfloat16))
    return O.bf16_bits_to_f64(hb), hb, rng


def test_refill_matches_library_sort():
    rng = np.random.default_rng(21)
    mass = np.round(rng.uniform(0, 1, 200), 1)                         # many exact ties
    drop = np.sort(rng.choice(200, 120, replace=False))
    for n in (0, 1, 37, 120):
        want = np.sort(drop[np.argsort(-mass[drop], kind="stable")[:n]])
        assert np.array_equal(O.refill_from_pruned(mass, drop, n), want)


def test_routing_invariants_against_library_cosine():
    """What the rules of Sec. 4.2 force, checked with torch's cosine similarity: an absorbed token's
    anchor is itself not absorbed, precedes it in (s_hat desc, index asc), is more similar than t
    and at least as similar as any other anchor that precedes it; two anchors are never more
    similar than t in the direction the order allows."""
    h, hb, rng = _clustered(160, 24, 9, 22)
    s_hat = np.round(rng.uniform(0, 1, 160), 2)                        # ties exercise the index rule
    keep = np.sort(rng.choice(160, 70, replace=False))
    t = 0.8
    dest, _ = O.route_within_kept(h, s_hat, keep, t)
    S = torch.nn.functional.cosine_similarity(torch.from_numpy(h[keep])[:, None], torch.from_numpy(h[keep])[None], dim=-1).numpy()
    before = lambda a, p: (s_hat[keep[a]], -keep[a]) > (s_hat[keep[p]], -keep[p])
    anchors = [p for p in range(70) if dest[p] < 0]
    assert 0 < len(anchors) < 70
    for p in range(70):
        cands = [a for a in anchors if before(a, p)]
        if dest[p] >= 0:
            a = dest[p]
            assert dest[a] < 0 and before(a, p) and S[a, p] > t
            assert all(S[a, p] >= S[c, p] - 1e-12 for c in cands)
        else:
            assert all(S[c, p] <= t + 1e-12 for c in cands)


def test_consolidation_special_cases():
    h, hb, rng = _clustered(120, 16, 5, 23)
    s_hat, mass = rng.uniform(0, 1, 120), rng.uniform(0, 5, 120)
    keep = np.sort(rng.choice(120, 40, replace=False)); drop = np.setdiff1d(np.arange(120), keep)
    pos = np.arange(1000, 1120)
    # t >= 1: nothing can be absorbed; the step is the plain gather of the kept rows
    r = O.consolidate_sample(hb, pos, 0, 120, mass, s_hat, keep, drop, 1.0)
    assert r["n_absorbed"] == 0 and np.array_equal(r["final_keep"], keep)
    assert np.array_equal(r["out_hidden_bits"], hb[keep]) and np.array_equal(r["out_pos"], pos[keep])
    # general t: sizes, disjointness, the refill is the heaviest part of the pool, weights conserved
    r = O.consolidate_sample(hb, pos, 0, 120, mass, s_hat, keep, drop, 0.7)
    a = r["n_absorbed"]
    assert 0 < a < 40 and len(r["final_keep"]) == 40 and np.all(np.diff(r["final_keep"]) > 0)
    assert set(r["refill"]) <= set(drop) and len(r["refill"]) == a
    rest = np.setdiff1d(drop, r["refill"])
    assert mass[r["refill"]].min() >= mass[rest].max()
    anchors = keep[r["dest"] < 0]
    assert set(r["final_keep"]) == set(anchors) | set(r["refill"])
    for slot in np.nonzero(r["merged_mask"])[0]:                      # Eq. 5 is a convex combination
        i = r["final_keep"][slot]
        src = keep[(r["dest"] >= 0) & (keep[np.maximum(r["dest"], 0)] == i)]
        grp = np.concatenate([[i], src])
        lo, hi = h[grp].min(axis=0), h[grp].max(axis=0)
        assert np.all(r["merged"][slot] >= lo - 1e-12) and np.all(r["merged"][slot] <= hi + 1e-12)
        w = s_hat[grp] / s_hat[grp].sum()
        assert np.allclose(r["merged"][slot], w @ h[grp], rtol=1e-12, atol=1e-14)
    # a twin of a kept token (same row, lower salience) is absorbed and leaves its anchor's row unchanged
    h2 = h.copy(); j, i = keep[7], keep[3]
    h2[j] = h2[i]
    hb2 = O.f64_to_bf16_bits(h2)
    s2 = s_hat.copy(); s2[i], s2[j] = 0.99, 0.01
    r2 = O.consolidate_sample(hb2, pos, 0, 120, mass, s2, keep, drop, 0.999)
    assert r2["dest"][7] == 3 or r2["dest"][r2["dest"][7]] < 0
    if r2["dest"][7] == 3 and (r2["dest"] == 3).sum() == 1:
        slot = int(np.nonzero(r2["final_keep"] == i)[0][0])
        assert np.allclose(r2["merged"][slot], h2[i], rtol=1e-12)


PLANTED_42 = [
    ("absorbed tokens may absorb in turn",
     lambda mod: dict(route_within_kept=lambda hv, sh, keep, t: (lambda S, order: (
         np.array([max([(S[a, p], -a) for a in order[:order.index(p)] if S[a, p] > t] or [(0, 1)])[1] * -1
                   for p in range(len(keep))], dtype=np.int32), None))(
         mod.cosine_matrix(hv[keep], hv[keep]), sorted(range(len(keep)), key=lambda p: (-sh[keep[p]], keep[p]))))),
    ("low salience absorbs high salience",
     lambda mod: dict(route_within_kept=lambda hv, sh, keep, t: O.route_within_kept(hv, -sh, keep, t))),
    ("refill ranked by salience instead of attention mass",
     lambda mod: dict(refill_from_pruned=lambda mass, drop, n: np.sort(drop[::-1][:n]).astype(np.int32))),
    ("refill ties go to the higher index",
     lambda mod: dict(refill_from_pruned=lambda mass, drop, n: np.sort(
         drop[np.lexsort((-drop, -mass[drop]))[:n]]).astype(np.int32))),
]


@pytest.mark.parametrize("label,patch", PLANTED_42, ids=[p[0] for p in PLANTED_42])
def test_planted_slip_in_consolidation_is_caught(label, patch):
    mod = _mutant()
    for name, fn in patch(mod).items():
        setattr(mod, name, fn)
    with pytest.raises(AssertionError):
        check_hand_consolidation(mod)


def test_consolidation_never_absorbs_more_than_the_pool_can_refill():
    """Fixed budget: with 40 kept of 46 tokens and everything similar, only six slots can be vacated."""
    rng = np.random.default_rng(24)
    base = rng.standard_normal(16)
    h = base[None, :] + 0.01 * rng.standard_normal((46, 16))              # all mutually similar
    hb = bits(torch.tensor(h, dtype=torch.float32).to(torch.bfloat16))
    s_hat, mass = rng.uniform(0.1, 1, 46), rng.uniform(0, 5, 46)
    keep = np.sort(rng.choice(46, 40, replace=False)); drop = np.setdiff1d(np.arange(46), keep)
    r = O.consolidate_sample(hb, np.arange(46), 0, 46, mass, s_hat, keep, drop, 0.5)
    assert r["n_absorbed"] == 6 and len(r["final_keep"]) == 40 and set(drop) <= set(r["final_keep"])
    order = sorted(range(40), key=lambda p: (-s_hat[keep[p]], keep[p]))
    assert sorted(np.nonzero(r["dest"] >= 0)[0].tolist()) == sorted(order[1:7])   # the first six after the top one
    assert np.all(r["dest"][order[1:7]] == order[0])


# ----------------------------------------------------------------------------- Eq. 4 applied to the values
def _bf16_bits(x):
    return bits(torch.tensor(np.asarray(x), dtype=torch.float32).to(torch.bfloat16))


def test_masked_attention_causal_case_is_library_attention():
    rng = np.random.default_rng(31)
    n, H, d = 23, 3, 16
    qb, kb, vb = (_bf16_bits(rng.standard_normal((n, H, d))) for _ in range(3))
    got = O.masked_attention(qb, kb, vb, 4, 9, None, mask_enable=False)
    tq, tk, tv = (torch.from_numpy(O.bf16_bits_to_f64(x)).permute(1, 0, 2) for x in (qb, kb, vb))
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True).permute(1, 0, 2).numpy()
    assert np.allclose(got, want, rtol=1e-12, atol=1e-14)


def test_masked_attention_hand_worked_three_tokens():
    """One head, d = 1, all tokens visual, q = 0 so every logit is 0: the weights are the mask's alone.
    lambda = (.5, .25, 1): row 0 admits key 0 fully and keys 1, 2 with weights .25 and 1;
    row 1 admits 0, 1 fully and key 2 with weight 1; row 2 is causal.  v = (8, 4, 2)."""
    lam = np.array([0.5, 0.25, 1.0])
    z = _bf16_bits(np.zeros((3, 1, 1)))
    v = _bf16_bits(np.array([8.0, 4.0, 2.0]).reshape(3, 1, 1))
    out = O.masked_attention(z, z, v, 0, 3, np.log(lam))[:, 0, 0]
    want = [(8 + .25 * 4 + 1 * 2) / (1 + .25 + 1), (8 + 4 + 1 * 2) / 3, (8 + 4 + 2) / 3]
    assert np.allclose(out, want, rtol=1e-14)


def test_masked_attention_invariants():
    rng = np.random.default_rng(32)
    n, H, d, v0, nv = 19, 2, 8, 3, 10
    qb, kb = (_bf16_bits(rng.standard_normal((n, H, d))) for _ in range(2))
    m = np.log(rng.uniform(0.05, 1.0, nv))
    # equal value rows: any convex combination returns that row
    row = rng.standard_normal((1, H, d))
    vb = _bf16_bits(np.repeat(row, n, axis=0))
    out = O.masked_attention(qb, kb, vb, v0, nv, m)
    assert np.allclose(out, O.bf16_bits_to_f64(vb), rtol=1e-13, atol=1e-15)
    # one-hot values (d = n): the output IS the probability matrix of Eq. 4
    q2, k2 = (_bf16_bits(rng.standard_normal((n, 1, n))) for _ in range(2))
    eye = _bf16_bits(np.eye(n).reshape(n, 1, n))
    out = O.masked_attention(q2, k2, eye, v0, nv, m)[:, 0, :]
    A = O.attention_probs(O.bf16_bits_to_f64(q2), O.bf16_bits_to_f64(k2), 0, np.arange(n), v0, nv, m, True)
    assert np.allclose(out, A, rtol=1e-13, atol=1e-16) and np.allclose(out.sum(axis=1), 1.0)
    # text and system rows never see the mask; visual rows do
    vb = _bf16_bits(rng.standard_normal((n, H, d)))
    on, off = O.masked_attention(qb, kb, vb, v0, nv, m), O.masked_attention(qb, kb, vb, v0, nv, None, False)
    vis = np.zeros(n, bool); vis[v0:v0 + nv - 1] = True          # the last visual row has no future visual key
    assert np.array_equal(on[~vis], off[~vis]) and np.all(np.abs(on[vis] - off[vis]).max(axis=(1, 2)) > 1e-6)


# ----------------------------------------------------------------------------- per-head variant of Eq. 1-3
def test_per_head_masses_average_to_the_default_mass():
    q, k = _rand_qk(30, 4, 16, 41)
    sh = O.attention_mass_heads(q, k, 5, 20)
    assert sh.shape == (4, 20)
    assert np.allclose(sh.mean(axis=0), O.attention_mass(q, k, 5, 20), rtol=1e-13, atol=1e-13)
    q1, k1 = q[:, :1], k[:, :1]
    assert np.allclose(O.attention_mass_heads(q1, k1, 5, 20)[0], O.attention_mass(q1, k1, 5, 20), rtol=1e-14)


def test_per_head_step_with_identical_heads_is_the_default_step():
    rng = np.random.default_rng(42)
    n, H, d, D, v0, nv = 40, 3, 8, 24, 4, 28
    q1, k1 = rng.standard_normal((n, 1, d)), rng.standard_normal((n, 1, d))
    qb, kb = _bf16_bits(np.repeat(q1, H, axis=1)), _bf16_bits(np.repeat(k1, H, axis=1))
    hb = _bf16_bits(rng.standard_normal((n, D)))
    kw = dict(lambda_max=0.7)
    a = O.prune_sample(qb, kb, hb, np.arange(n), v0, nv, v0, n - v0, 9, per_head=True, **kw)     # ranking rows: image + text
    b = O.prune_sample(qb, kb, hb, np.arange(n), v0, nv, v0, n - v0, 9, per_head=False, **kw)
    for name in ("mass", "salience", "mask_log", "rank_score"):
        assert np.allclose(a[name], b[name], rtol=1e-12, atol=1e-14), name
    assert np.array_equal(a["keep_idx"], b["keep_idx"]) and np.array_equal(a["out_hidden_bits"], b["out_hidden_bits"])
    assert np.allclose(a["mask_log_heads"], np.repeat(b["mask_log"][None], H, axis=0), rtol=1e-12, atol=1e-14)


def check_hand_per_head_merge_weight(o):
    """Two heads whose saliences differ: the Eq. 5 weight of a token is the head mean of the per-head
    saliences -- not one head's salience and not the salience of the head-mean mass."""
    g = GOLD["per_head_merge_weight"]
    qb, kb, hb = _bf16_bits(g["Q"]), _bf16_bits(g["K"]), _bf16_bits(g["hidden"])
    q, k = o.bf16_bits_to_f64(qb), o.bf16_bits_to_f64(kb)
    assert np.allclose(o.attention_mass_heads(q, k, 0, 3), g["s_heads"], atol=1e-15)
    r = o.prune_sample(qb, kb, hb, np.arange(4), 0, 3, 3, 1, 1, per_head=True)
    assert np.allclose(r["salience"], g["salience"], rtol=1e-14, atol=0)
    assert r["keep_idx"].tolist() == g["keep"] and r["assign"].tolist() == g["assign"]
    assert np.allclose(r["merged"], g["merged"], rtol=1e-13, atol=0)


def test_hand_per_head_merge_weight():
    check_hand_per_head_merge_weight(O)


PLANTED_PER_HEAD = [
    ("merge weight taken from head 0", "s_hat = s_hat_heads.mean(axis=0)", "s_hat = s_hat_heads[0]"),
    ("merge weight is the salience of the head-mean mass", "s_hat = s_hat_heads.mean(axis=0)", "s_hat = salience(s, eps)"),
]


@pytest.mark.parametrize("label,old,new", PLANTED_PER_HEAD, ids=[p[0] for p in PLANTED_PER_HEAD])
def test_planted_slip_in_per_head_weight_is_caught(label, old, new):
    src = open(O.__file__).read()
    assert src.count(old) == 1
    mod = types.ModuleType("mutant")
    exec(compile(src.replace(old, new), "mutant", "exec"), mod.__dict__)
    with pytest.raises(AssertionError):
        check_hand_per_head_merge_weight(mod)
    # the permutation test below must notice the first slip as well (head 0 is a different head after it)
    if "heads[0]" in new:
        with pytest.raises(AssertionError):
            check_per_head_permutation(mod)


def check_per_head_permutation(o):
    rng = np.random.default_rng(43)
    n, H, d, v0, nv = 36, 3, 8, 3, 25
    qb, kb = _bf16_bits(rng.standard_normal((n, H, d))), _bf16_bits(rng.standard_normal((n, H, d)))
    hb = _bf16_bits(rng.standard_normal((n, H * d)))
    a = o.prune_sample(qb, kb, hb, np.arange(n), v0, nv, v0, n - v0, 8, per_head=True, lambda_max=0.9)
    perm = [2, 0, 1]
    b = o.prune_sample(qb[:, perm], kb[:, perm], hb, np.arange(n), v0, nv, v0, n - v0, 8, per_head=True, lambda_max=0.9)
    assert np.allclose(b["mask_log_heads"], a["mask_log_heads"][perm], rtol=1e-13, atol=1e-14)
    assert np.allclose(b["rank_score"], a["rank_score"], rtol=1e-12, atol=1e-15)
    # one weight per token, whatever the order of the heads: salience and merged rows do not move
    assert np.allclose(b["salience"], a["salience"], rtol=1e-13, atol=1e-15)
    assert np.array_equal(b["keep_idx"], a["keep_idx"]) and np.array_equal(b["assign"], a["assign"])
    assert np.array_equal(b["out_hidden_bits"], a["out_hidden_bits"])
    return a, qb, kb, hb


def test_per_head_masks_differ_and_follow_a_head_permutation():
    check_per_head_permutation(O)
    rng = np.random.default_rng(43)
    n, H, d, v0, nv = 36, 3, 8, 3, 25
    qb, kb = _bf16_bits(rng.standard_normal((n, H, d))), _bf16_bits(rng.standard_normal((n, H, d)))
    hb = _bf16_bits(rng.standard_normal((n, H * d)))
    a = O.prune_sample(qb, kb, hb, np.arange(n), v0, nv, v0, n - v0, 8, per_head=True, lambda_max=0.9)
    assert np.abs(a["mask_log_heads"][0] - a["mask_log_heads"][1]).max() > 1e-3
    for h in range(H):                                       # every head's salience spans exactly [0, 1)
        lam = np.exp(a["mask_log_heads"][h]) / 0.9
        assert lam.max() > 0.99 and lam.min() <= 1e-6 / 0.9 + 1e-12
    perm = [2, 0, 1]
    b = O.prune_sample(qb[:, perm], kb[:, perm], hb, np.arange(n), v0, nv, v0, n - v0, 8, per_head=True, lambda_max=0.9)
    assert np.allclose(b["mask_log_heads"], a["mask_log_heads"][perm], rtol=1e-13, atol=1e-14)
    assert np.allclose(b["rank_score"], a["rank_score"], rtol=1e-12, atol=1e-15)
    # a per-head mask really is used per head: the default step on the same data ranks differently
    c = O.prune_sample(qb, kb, hb, np.arange(n), v0, nv, v0, n - v0, 8, per_head=False, lambda_max=0.9)
    assert np.abs(c["rank_score"] - a["rank_score"]).max() > 1e-6
