"""Element-by-element comparison of the CUDA prune step with the CPU oracle.

Tolerances (written here so the bar is visible in one place):
  mass, salience, rank_score   |g - o| <= 1e-3 * max(|o|, 1e-3 * max_j |o_j|)      (fp32 vs fp64)
  mask_log                     compared as lambda = exp(m): |exp(g) - exp(o)| <= 1e-4
  keep set                     identical, except that tokens whose oracle score lies within
                               1e-4 (relative) of the k-th / (k+1)-th boundary may swap
  assign                       identical where the oracle's margin between best and runner-up
                               similarity exceeds 1e-4; inside that band the GPU's slot is
                               accepted if its oracle similarity is within 1e-4 of the best
  best_sim                     |g - o| <= 2e-4
  merged hidden (bf16)         |g - o_f64| <= max(2e-2, (2^-8 + 2^-16) * |o|): 2e-2 absolute; for magnitudes
                               above 5.1 the bound of ONE correct bf16 rounding (half a unit in the last
                               place is at most 2^-8 |o|) plus 2^-16 |o| for the fp32 accumulation that
                               precedes it.  How many elements needed the relative term, and their
                               largest error, are recorded in `stats` (merged_wide_*)
  copied rows, position ids, row maps, offsets, index padding      bit-exact
Where the GPU made an allowed in-band choice, the oracle's downstream stages are re-evaluated
with that choice so that later comparisons stay meaningful.
"""
from __future__ import annotations

import math

import numpy as np
import torch

from oracle import asap_oracle as O
from tests.helpers import bits

REL = 1e-3
TIE = 1e-4
MERGED_ABS = 2e-2
MERGED_REL = 2.0 ** -8 + 2.0 ** -16


def merged_tolerance(want):
    """Element-wise bar of a bf16 row computed in fp32 and rounded once, against float64."""
    return np.maximum(MERGED_ABS, np.abs(want) * MERGED_REL)


def check_invariants(batch, b, params, out):
    """What must hold for every sequence whatever the scores are (no oracle involved): exactly k kept
    indices, ascending; the dropped list is the ascending complement; the shortened sequence has the
    right length; its row map is strictly increasing and names prefix rows, kept rows, suffix rows;
    position ids are gathered through it; prefix and suffix rows are bit-identical copies."""
    rows = batch.sample_rows(b)
    v0, nv = int(batch.vis_start[b]), int(batch.vis_len[b])
    n, k = rows.stop - rows.start, params.keep_k
    keep = out.keep_idx[b].cpu().numpy()
    drop = out.drop_idx[b].cpu().numpy()
    assert keep.shape[0] == k and np.all(np.diff(keep) > 0) and keep[0] >= 0 and keep[-1] < nv, f"keep_idx sample {b}"
    assert np.array_equal(drop[:nv - k], np.setdiff1d(np.arange(nv, dtype=np.int32), keep)), f"drop_idx sample {b}"
    assert np.all(drop[nv - k:] == -1)
    ocu = out.out_cu_seqlens.cpu().numpy()
    lo, hi = int(ocu[b]), int(ocu[b + 1])
    assert hi - lo == n - nv + k, f"out_cu_seqlens sample {b}"
    src = out.src_row[lo:hi].cpu().numpy().astype(np.int64)
    assert np.all(np.diff(src) > 0), f"src_row not strictly increasing (sample {b})"
    want_src = np.concatenate([np.arange(v0), v0 + keep, np.arange(v0 + nv, n)]) + rows.start
    assert np.array_equal(src, want_src), f"src_row sample {b}"
    assert np.array_equal(out.out_pos[lo:hi].cpu().numpy(), batch.pos_ids.numpy()[src]), f"out_pos sample {b}"
    oh = out.out_hidden[lo:hi]
    hid = batch.hidden[rows]
    assert torch.equal(oh[:v0].cpu(), hid[:v0]), f"prefix rows sample {b}"
    assert torch.equal(oh[v0 + k:].cpu(), hid[v0 + nv:]), f"suffix rows sample {b}"
    asg = out.assign[b].cpu().numpy()
    assert np.all(asg[nv - k:] == -1) and np.all((asg[:nv - k] >= -1) & (asg[:nv - k] < k)), f"assign sample {b}"


def _rel_err(g, o):
    floor = 1e-3 * np.max(np.abs(o)) if o.size else 0.0
    return np.abs(g - o) / np.maximum(np.maximum(np.abs(o), floor), 1e-300)


def compare_sample(batch, b, params, out, rank_start=None, rank_len=None, stats=None):
    """Checks sample b of a finished prune step.  `out` is binding.Outputs (device tensors)."""
    rows = batch.sample_rows(b)
    v0, nv = int(batch.vis_start[b]), int(batch.vis_len[b])
    r0 = int(batch.text_start[b]) if rank_start is None else int(rank_start[b])
    nr = int(batch.text_len[b]) if rank_len is None else int(rank_len[b])
    k = params.keep_k
    n = rows.stop - rows.start
    qb, kb, hb = bits(batch.q[rows]), bits(batch.k[rows]), bits(batch.hidden[rows])
    pos = batch.pos_ids[rows].numpy()
    okw = dict(lambda_max=params.lambda_max, eps=params.eps, sim_threshold=params.sim_threshold,
               mask_enable=params.mask_enable, merge_enable=params.merge_enable,
               per_head=bool(getattr(params, "per_head_mask", False)))
    ref = O.prune_sample(qb, kb, hb, pos, v0, nv, r0, nr, k, **okw)

    g = lambda t: t[b].detach().cpu().numpy()
    mv = out.mass.shape[1]
    # ---- stage 1 / 2 floats
    for name in ("mass", "salience", "rank_score"):
        gv = g(getattr(out, name)).astype(np.float64)
        err = _rel_err(gv[:nv], ref[name])
        assert err.max() <= REL, f"{name} sample {b}: rel err {err.max():.3e} at {err.argmax()}"
        assert np.all(gv[nv:] == 0.0), f"{name} padding not zero"
        if stats is not None:
            stats[name] = max(stats.get(name, 0.0), float(err.max()))
    lam_g = np.exp(g(out.mask_log).astype(np.float64)[:nv])
    lam_o = np.exp(ref["mask_log"])
    assert np.max(np.abs(lam_g - lam_o)) <= 1e-4, f"mask_log sample {b}: {np.max(np.abs(lam_g - lam_o)):.3e}"
    if okw["per_head"]:                                  # one mask vector per head, same bar
        mh = out.mask_log_heads[b].detach().cpu().numpy().astype(np.float64)      # [H, max_vis]
        err_h = np.abs(np.exp(mh[:, :nv]) - np.exp(ref["mask_log_heads"]))
        assert err_h.max() <= 1e-4, f"mask_log_heads sample {b}: {err_h.max():.3e}"
        assert np.all(mh[:, nv:] == 0.0), "mask_log_heads padding not zero"

    # ---- top-k
    keep_g = g(out.keep_idx)
    drop_g = g(out.drop_idx)
    assert keep_g.shape[0] == k and np.all(np.diff(keep_g) > 0) and keep_g.min() >= 0 and keep_g.max() < nv
    nd = nv - k
    want_drop = np.setdiff1d(np.arange(nv, dtype=np.int32), keep_g)
    assert np.array_equal(drop_g[:nd], want_drop), "drop_idx is not the ascending complement of keep_idx"
    assert np.all(drop_g[nd:] == -1), "drop_idx padding"
    keep_o = ref["keep_idx"]
    swapped = 0
    if not np.array_equal(keep_g, keep_o):
        r = ref["rank_score"]
        srt = np.sort(r)[::-1]
        kth, nxt = srt[k - 1], (srt[k] if k < nv else srt[k - 1])
        diff = np.setxor1d(keep_g, keep_o)
        band = TIE * max(abs(kth), abs(nxt))
        assert abs(kth - nxt) <= band and np.all(np.abs(r[diff] - kth) <= 2 * band), \
            f"kept set differs outside the tie band (sample {b}): {diff.tolist()}"
        swapped = len(diff) // 2
        ref = O.prune_sample(qb, kb, hb, pos, v0, nv, r0, nr, k, keep_override=keep_g, **okw)
    if stats is not None:
        stats["keep_swaps"] = stats.get("keep_swaps", 0) + swapped

    # ---- assignment
    as_g = g(out.assign)
    assert np.all(as_g[nd:] == -1), "assign padding"
    as_g = as_g[:nd]
    if params.merge_enable and nd > 0:
        assert np.all((as_g >= -1) & (as_g < k))
        hv = O.bf16_bits_to_f64(hb[v0:v0 + nv])
        as_o, margin = ref["assign"], ref["margin"]
        mism = np.nonzero(as_g != as_o)[0]
        if len(mism):
            S = O.cosine_matrix(hv[want_drop[mism]], hv[keep_g])
            for row, dp in enumerate(mism):
                best = ref["best_sim"][dp]
                thr = params.sim_threshold
                if as_g[dp] == -1 or as_o[dp] == -1:      # gate decision: only if the similarity sits on the threshold
                    assert abs(best - thr) <= TIE, f"threshold gate differs at dropped {dp} (sample {b})"
                    continue
                assert margin[dp] <= TIE and best - S[row, as_g[dp]] <= TIE, \
                    f"assign differs outside the tie band at dropped {dp} (sample {b}): gpu {as_g[dp]} oracle {as_o[dp]} margin {margin[dp]:.3e}"
            ref = O.prune_sample(qb, kb, hb, pos, v0, nv, r0, nr, k, keep_override=keep_g,
                                 assign_override=as_g, **okw)
        if stats is not None:
            stats["assign_band"] = stats.get("assign_band", 0) + int(len(mism))
        if out.best_sim is not None:
            bs = g(out.best_sim)[:nd].astype(np.float64)
            e = np.abs(bs - ref["best_sim"])
            # a different in-band slot has a similarity within the band as well
            assert e.max() <= 2e-4, f"best_sim sample {b}: {e.max():.3e}"
    else:
        assert np.all(as_g == -1)

    # ---- shortened sequence
    ocu = out.out_cu_seqlens.detach().cpu().numpy()
    n_out = n - nv + k
    assert ocu[b + 1] - ocu[b] == n_out, "out_cu_seqlens"
    o_rows = slice(int(ocu[b]), int(ocu[b + 1]))
    oh = bits(out.out_hidden[o_rows].detach().cpu())
    assert np.array_equal(out.out_pos[o_rows].cpu().numpy(), ref["out_pos"]), "out_pos"
    assert np.array_equal(out.src_row[o_rows].cpu().numpy(), ref["src_row"] + rows.start), "src_row"
    assert np.array_equal(oh[:v0], hb[:v0]), "prefix rows must be bit-identical"
    assert np.array_equal(oh[v0 + k:], hb[v0 + nv:]), "suffix rows must be bit-identical"
    gh = O.bf16_bits_to_f64(oh[v0:v0 + k])
    want = ref["merged"]
    tol = merged_tolerance(want)
    err = np.abs(gh - want)
    assert np.all(err <= tol), f"merged hidden sample {b}: max err {err.max():.4e} (tol {tol.flat[err.argmax()]:.3e})"
    if stats is not None:
        stats["merged_abs"] = max(stats.get("merged_abs", 0.0), float(err.max()))
        wide = err > MERGED_ABS                     # passed only because of the relative term
        stats["merged_wide_count"] = stats.get("merged_wide_count", 0) + int(wide.sum())
        if wide.any():
            stats["merged_wide_max_abs"] = max(stats.get("merged_wide_max_abs", 0.0), float(err[wide].max()))
            stats["merged_wide_max_rel"] = max(stats.get("merged_wide_max_rel", 0.0),
                                               float((err[wide] / np.abs(want[wide])).max()))
    # rows that received nothing must be exact copies
    if params.merge_enable and nd > 0:
        untouched = np.setdiff1d(np.arange(k), as_g[as_g >= 0])
    else:
        untouched = np.arange(k)
    assert np.array_equal(oh[v0 + untouched], hb[v0 + keep_g[untouched]]), "unmerged kept rows must be copies"
    return ref
