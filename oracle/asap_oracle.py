"""CPU oracle for the ASAP visual-token prune step  --  TEST INFRASTRUCTURE ONLY.

Plain numpy in float64, written from the paper's method section (Sec. 4.1 Eq. 1-4,
Sec. 4.2 Eq. 5) equation by equation, with no blocking, fusion or reordering.  It is
slow on purpose.  Only the tests, the smoke check and the benchmark's CPU-baseline
leg may import it; the CUDA library never does and shares no code with it.

Inputs are the bf16 bit patterns (numpy uint16) the CUDA path receives; they are
widened exactly to float64 before any arithmetic.

Parity status of each function (what pins it, see tests/test_oracle_pins.py):
  attention_mass        pinned  (closed form via the summed query; hand-worked fixture)
  attention_mass_heads  pinned  (its head mean is attention_mass; one head = attention_mass; the
                                 per-head step with identical heads equals the default step; a hand-worked
                                 two-head case fixes the per-head masses and the Eq. 5 weight of the
                                 per-head step -- the head mean of the per-head saliences)
  salience / mask_log   pinned  (hand-worked fixture; extremes; affine invariance)
  mask_matrix           pinned  (hand-enumerated 5x5 fixture; causal limit)
  attention_probs /
  rank_scores           pinned  (library float64 softmax in the causal case; the
                                 multiplicative form of Eq. 4; closed form for W = 0)
  select_topk           pinned  (hand-enumerated ties; library stable sort)
  cosine_assign         pinned  (library cosine similarity; hand-worked vectors)
  weighted_merge        pinned  (hand-worked fixture; convexity; weight conservation)
  compact_rows          pinned  (library fancy indexing; identity and reversal maps)
  route_within_kept /
  refill_from_pruned /
  consolidate_sample    pinned  (hand-worked fixture; t >= 1 -> nothing merges and the output is the
                                 plain top-k gather; twins; anchors are never absorbed; set sizes;
                                 Eq. 5 weight conservation; library sort for the refill).  Not pinned
                                 by the paper: the reading of which anchor absorbs a token.
  masked_attention      pinned  (library float64 scaled-dot-product attention in the causal case; value
                                 rows all equal -> output equals that row; one-hot values recover the
                                 Eq. 4 probabilities, themselves pinned above; hand-worked 3-token case)
  compact / prune_step  pinned  (invariants: k kept ascending; identity at k = N_v;
                                 plain attention top-k with mask and merge off; twins)
  Not pinned by anything the paper prints: that the ranking rule (mean of the Eq. 4
  probabilities over heads and ranking rows) and the drop->keep merge topology are
  what the authors ran.  The paper gives no worked numeric example of a prune step.
"""
from __future__ import annotations

import math
from typing import Dict, Optional

import numpy as np

EPS_DEFAULT = 1e-6


# ----------------------------------------------------------------------------------
# bf16 <-> float64
# ----------------------------------------------------------------------------------
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening: a bf16 value is the upper half of an IEEE binary32."""
    u32 = bits.astype(np.uint32) << np.uint32(16)
    return u32.view(np.float32).astype(np.float64)


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float64 to the nearest bf16 (ties to even) in ONE rounding.

    The two bf16 neighbours of x are found by truncating the binary32 image of x to its
    upper 16 bits (one neighbour) and stepping one bf16 ulp away from zero (the other);
    the nearer one in float64 wins, an exact tie goes to the even mantissa."""
    x = np.asarray(x, dtype=np.float64)
    f32 = x.astype(np.float32)
    u = f32.view(np.uint32)
    lo_bits = (u >> np.uint32(16)).astype(np.uint32)
    # binary32 rounding may have moved |f32| above |x|; step the truncated candidate down if so
    lo_val = bf16_bits_to_f64(lo_bits.astype(np.uint16))
    too_big = np.abs(lo_val) > np.abs(x)
    lo_bits = np.where(too_big, lo_bits - np.uint32(1), lo_bits)
    lo_val = bf16_bits_to_f64(lo_bits.astype(np.uint16))
    hi_bits = lo_bits + np.uint32(1)
    hi_val = bf16_bits_to_f64(hi_bits.astype(np.uint16))
    d_lo = np.abs(x - lo_val)
    d_hi = np.abs(hi_val - x)
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & ((lo_bits & np.uint32(1)) == 1))
    out = np.where(pick_hi, hi_bits, lo_bits).astype(np.uint16)
    # zeros, infinities and NaN pass through the truncated image
    special = ~np.isfinite(x) | (x == 0.0)
    return np.where(special, (u >> np.uint32(16)).astype(np.uint16), out)


# ----------------------------------------------------------------------------------
# Stage 1: salience-guided bidirectional mask (Sec. 4.1)
# ----------------------------------------------------------------------------------
def alignment(q: np.ndarray, k: np.ndarray, h: int) -> np.ndarray:
    """W = Q K^T / sqrt(d) for one head (Sec. 4.1, definition above Eq. 1).
    q: [n_q, H, d], k: [n_k, H, d] float64 -> [n_q, n_k]."""
    d = q.shape[-1]
    return (q[:, h, :] @ k[:, h, :].T) / math.sqrt(d)


def attention_mass(q: np.ndarray, k: np.ndarray, v0: int, nv: int) -> np.ndarray:
    """Eq. 1: s_j = sum over visual queries i of W[i, j], for visual keys j.
    The sum uses the raw, unmasked, pre-softmax W (all i in the image span, before and
    after j).  Heads are combined by their mean (one salience per token)."""
    H = q.shape[1]
    qv, kv = q[v0:v0 + nv], k[v0:v0 + nv]
    s = np.zeros(nv, dtype=np.float64)
    for h in range(H):
        W = alignment(qv, kv, h)          # [i, j]
        s += W.sum(axis=0)                # sum over queries i
    return s / H


def attention_mass_heads(q: np.ndarray, k: np.ndarray, v0: int, nv: int) -> np.ndarray:
    """Eq. 1 kept per head: s^h_j = sum over visual queries i of W^h[i, j].  [H, nv].  (The variant in
    which every head has its own salience and mask; the default combines the heads by their mean.)"""
    H = q.shape[1]
    qv, kv = q[v0:v0 + nv], k[v0:v0 + nv]
    return np.stack([alignment(qv, kv, h).sum(axis=0) for h in range(H)])


def salience(s: np.ndarray, eps: float = EPS_DEFAULT) -> np.ndarray:
    """Eq. 2: min-max normalisation over the image span."""
    s_min, s_max = s.min(), s.max()
    return (s - s_min) / (s_max - s_min + eps)


def mask_log(s_hat: np.ndarray, lambda_max: float, eps: float = EPS_DEFAULT) -> np.ndarray:
    """Eq. 3, the value written above the diagonal: ln(max(lambda_j, eps)),
    lambda_j = lambda_max * s_hat_j."""
    lam = lambda_max * s_hat
    return np.log(np.maximum(lam, eps))


def mask_matrix(n: int, rows: np.ndarray, v0: int, nv: int, m: Optional[np.ndarray],
                mask_enable: bool) -> np.ndarray:
    """Additive mask for query positions `rows` against keys 0..n-1.

    Eq. 3: 0 on and below the diagonal.  Above the diagonal the causal -inf stays,
    except inside the image span (query AND key visual) where it is overwritten by
    m_j.  With the mask disabled this is the causal mask of Sec. 3.2."""
    i = np.asarray(rows)[:, None]                 # query position
    j = np.arange(n)[None, :]                     # key position
    M = np.where(j <= i, 0.0, -np.inf)
    if mask_enable:
        m_of_key = np.full(n, -np.inf)
        m_of_key[v0:v0 + nv] = m
        in_span = (i >= v0) & (i < v0 + nv) & (j >= v0) & (j < v0 + nv)
        M = np.where(in_span & (i < j), m_of_key[None, :], M)
    return M


def attention_probs(q: np.ndarray, k: np.ndarray, h: int, rows: np.ndarray, v0: int, nv: int,
                    m: Optional[np.ndarray], mask_enable: bool, M: Optional[np.ndarray] = None) -> np.ndarray:
    """Eq. 4: A = Softmax(W + M_bidir), rows `rows` of one head, over all keys.
    (M may be passed in when several heads share it; it is the same for every head.)"""
    W = alignment(q[rows], k, h)
    if M is None:
        M = mask_matrix(k.shape[0], rows, v0, nv, m, mask_enable)
    Z = W + M
    Z = Z - Z.max(axis=1, keepdims=True)
    E = np.exp(Z)
    return E / E.sum(axis=1, keepdims=True)


def rank_scores(q: np.ndarray, k: np.ndarray, v0: int, nv: int, r0: int, nr: int,
                m: Optional[np.ndarray], mask_enable: bool) -> np.ndarray:
    """Ranking score of visual key j: the mean, over heads and over the ranking query rows
    r0 .. r0+nr-1, of the Eq. 4 attention probability A[i, j].  `m` is Eq. 3's vector [nv], or
    one vector per head [H, nv] in the per-head variant."""
    H = q.shape[1]
    rows = np.arange(r0, r0 + nr)
    r = np.zeros(nv, dtype=np.float64)
    per_head = m is not None and np.ndim(m) == 2
    M = None if per_head else mask_matrix(k.shape[0], rows, v0, nv, m, mask_enable)
    for h in range(H):
        if per_head:
            A = attention_probs(q, k, h, rows, v0, nv, m[h], mask_enable)
            r += A[:, v0:v0 + nv].sum(axis=0)
            continue
        A = attention_probs(q, k, h, rows, v0, nv, m, mask_enable, M)
        r += A[:, v0:v0 + nv].sum(axis=0)
    return r / (H * nr)


def select_topk(r: np.ndarray, keep_k: int):
    """The keep_k visual tokens of largest score, equal scores resolved toward the lower
    index; both the kept and the dropped list come back in ascending index order."""
    idx = np.arange(len(r))
    order = np.lexsort((idx, -r))         # primary: descending score, secondary: ascending index
    keep = np.sort(order[:keep_k]).astype(np.int32)
    drop = np.sort(order[keep_k:]).astype(np.int32)
    return keep, drop


# ----------------------------------------------------------------------------------
# Stage 2: salience-weighted consolidation (Sec. 4.2)
# ----------------------------------------------------------------------------------
def cosine_matrix(hd: np.ndarray, hk: np.ndarray) -> np.ndarray:
    """Pairwise cosine similarity S[j, i] between rows of hd and rows of hk.  A row whose
    norm is below 1e-12 has similarity 0 to everything."""
    nd = np.sqrt((hd * hd).sum(axis=1))
    nk = np.sqrt((hk * hk).sum(axis=1))
    dots = hd @ hk.T
    den = nd[:, None] * nk[None, :]
    ok = (nd[:, None] >= 1e-12) & (nk[None, :] >= 1e-12)
    return np.where(ok, dots / np.where(ok, den, 1.0), 0.0)


def cosine_assign(hv: np.ndarray, keep: np.ndarray, drop: np.ndarray, threshold: float):
    """Each dropped token j goes to the kept slot a(j) of highest cosine similarity (lowest
    slot among equals) and is merged only if that similarity is strictly above `threshold`.
    Returns (assign [n_drop] slot or -1, best_sim, margin to the runner-up slot)."""
    n_drop, n_keep = len(drop), len(keep)
    assign = np.full(n_drop, -1, dtype=np.int32)
    best = np.zeros(n_drop, dtype=np.float64)
    margin = np.full(n_drop, np.inf, dtype=np.float64)
    if n_drop == 0 or n_keep == 0:
        return assign, best, margin
    S = cosine_matrix(hv[drop], hv[keep])
    a = S.argmax(axis=1)                  # numpy returns the first maximiser
    best = S[np.arange(n_drop), a]
    if n_keep > 1:
        S2 = S.copy()
        S2[np.arange(n_drop), a] = -np.inf
        margin = best - S2.max(axis=1)
    assign = np.where(best > threshold, a, -1).astype(np.int32)
    return assign, best, margin


def weighted_merge(hv: np.ndarray, s_hat: np.ndarray, keep: np.ndarray, drop: np.ndarray,
                   assign: np.ndarray, eps: float = EPS_DEFAULT) -> np.ndarray:
    """Eq. 5 for every kept token: the salience-weighted convex combination of the token and
    the dropped tokens assigned to it.  A total weight of at most eps leaves the token as is."""
    out = np.empty((len(keep), hv.shape[1]), dtype=np.float64)
    for slot, i in enumerate(keep):
        src = drop[assign == slot]
        num = s_hat[i] * hv[i]
        den = s_hat[i]
        for j in src:
            num = num + s_hat[j] * hv[j]
            den = den + s_hat[j]
        out[slot] = hv[i] if den <= eps else num / den
    return out


# ----------------------------------------------------------------------------------
# One sample, whole step
# ----------------------------------------------------------------------------------
def prune_sample(q_bits, k_bits, hidden_bits, pos_ids, v0: int, nv: int, r0: int, nr: int,
                 keep_k: int, lambda_max: float = 1.0, eps: float = EPS_DEFAULT,
                 sim_threshold: float = -math.inf, mask_enable: bool = True,
                 merge_enable: bool = True, assign_override: Optional[np.ndarray] = None,
                 keep_override: Optional[np.ndarray] = None, per_head: bool = False) -> Dict[str, np.ndarray]:
    """The prune step for one sequence [prefix | visual span | suffix].

    q_bits, k_bits: uint16 [n, H, d]; hidden_bits: uint16 [n, D]; pos_ids: int32 [n].
    keep_override / assign_override replace the oracle's own top-k / assignment (used by
    the tests when a decision falls inside the stated tie band).
    per_head: Eq. 1-3 separately for every head (s^h, s_hat^h, m^h); head h's logits get head h's
    mask; one token has one merge weight, the mean over heads of s_hat^h."""
    q = bf16_bits_to_f64(q_bits)
    k = bf16_bits_to_f64(k_bits)
    hid = bf16_bits_to_f64(hidden_bits)
    n = q.shape[0]

    m_heads = None
    if per_head:
        s_heads = attention_mass_heads(q, k, v0, nv)
        s_hat_heads = np.stack([salience(sh, eps) for sh in s_heads])
        m_heads = np.stack([mask_log(x, lambda_max, eps) for x in s_hat_heads])
        s = s_heads.mean(axis=0)
        s_hat = s_hat_heads.mean(axis=0)
        m = mask_log(s_hat, lambda_max, eps)
        r = rank_scores(q, k, v0, nv, r0, nr, m_heads, mask_enable)
    else:
        s = attention_mass(q, k, v0, nv)
        s_hat = salience(s, eps)
        m = mask_log(s_hat, lambda_max, eps)
        r = rank_scores(q, k, v0, nv, r0, nr, m, mask_enable)

    keep, drop = select_topk(r, keep_k)
    if keep_override is not None:
        keep = np.asarray(keep_override, dtype=np.int32)
        drop = np.setdiff1d(np.arange(nv, dtype=np.int32), keep).astype(np.int32)

    hv = hid[v0:v0 + nv]
    if merge_enable:
        assign, best, margin = cosine_assign(hv, keep, drop, sim_threshold)
        if assign_override is not None:
            assign = np.asarray(assign_override, dtype=np.int32)
        merged = weighted_merge(hv, s_hat, keep, drop, assign, eps)
    else:
        assign = np.full(len(drop), -1, dtype=np.int32)
        best = np.zeros(len(drop))
        margin = np.full(len(drop), np.inf)
        merged = hv[keep].copy()

    # hand-off: prefix rows, kept visual rows in ascending order, suffix rows; position ids gathered
    src_row = np.concatenate([np.arange(0, v0), v0 + keep, np.arange(v0 + nv, n)]).astype(np.int32)
    out_hidden = np.concatenate([hid[:v0], merged, hid[v0 + nv:]], axis=0)
    out_bits = f64_to_bf16_bits(out_hidden)
    # rows that are pure copies must keep their exact bit pattern
    out_bits[:v0] = hidden_bits[:v0]
    out_bits[v0 + len(keep):] = hidden_bits[v0 + nv:]
    return dict(mass=s, salience=s_hat, mask_log=m, mask_log_heads=m_heads, rank_score=r, keep_idx=keep, drop_idx=drop,
                assign=assign, best_sim=best, margin=margin, merged=merged,
                out_hidden=out_hidden, out_hidden_bits=out_bits,
                out_pos=np.asarray(pos_ids)[src_row].astype(np.int32), src_row=src_row)


# ----------------------------------------------------------------------------------
# Stage 2 as Sec. 4.2 states it: consolidation INSIDE the kept set, then budget reallocation
# ----------------------------------------------------------------------------------
def route_within_kept(hv: np.ndarray, s_hat: np.ndarray, keep: np.ndarray, threshold: float,
                      max_absorb=None):
    """Salience-anchored routing of Sec. 4.2 among the kept tokens.

    A token j may be absorbed by a token i only if S_ij > t and i comes before j in the order
    (s_hat descending, sequence index ascending) -- the paper's "s_hat_i >= s_hat_j, ties by
    sequence index".  Reading taken for what the paper leaves open (which i, and whether an
    absorbed token can absorb): the kept tokens are visited in that order; a token joins the
    most similar token among those that were NOT absorbed before it (the anchors), lowest
    sequence index among equally similar ones, provided that similarity exceeds t; otherwise it
    becomes an anchor itself.  Source sets are therefore disjoint and end at anchors.
    A vacated slot must be refilled from the pruned pool (the budget is fixed), so at most
    `max_absorb` tokens (the size of that pool) are absorbed: once that many have been, every
    later token stays an anchor.

    Returns (dest [k]: slot of the absorbing anchor, -1 for anchors; margin [k]: how far the
    decision of each token was from flipping: distance of its best similarity from t, and from
    the runner-up anchor's)."""
    k = len(keep)
    S = cosine_matrix(hv[keep], hv[keep])
    order = sorted(range(k), key=lambda p: (-s_hat[keep[p]], int(keep[p])))
    dest = np.full(k, -1, dtype=np.int32)
    margin = np.full(k, np.inf)
    anchors = []
    n_absorbed = 0
    for p in order:
        best, best_a, second = -np.inf, -1, -np.inf
        for a in sorted(anchors):                 # ascending slot = ascending sequence index
            v = S[a, p]
            if v > best:
                second, best, best_a = best, v, a
            elif v > second:
                second = v
        if best_a >= 0:
            margin[p] = min(abs(best - threshold), best - second)
        if best_a >= 0 and best > threshold and (max_absorb is None or n_absorbed < max_absorb):
            dest[p] = best_a
            n_absorbed += 1
        else:
            anchors.append(p)
    return dest, margin


def refill_from_pruned(mass: np.ndarray, drop: np.ndarray, n: int) -> np.ndarray:
    """Budget reallocation of Sec. 4.2: the n pruned tokens of largest attention mass s_j (Eq. 1),
    lower index first among equals; returned in ascending index order."""
    if n == 0:
        return np.zeros(0, dtype=np.int32)
    order = np.lexsort((drop, -mass[drop]))
    return np.sort(drop[order[:n]]).astype(np.int32)


def consolidate_sample(hidden_bits, pos_ids, v0: int, nv: int, mass, s_hat, keep, drop, threshold: float,
                       eps: float = EPS_DEFAULT, dest_override=None, refill_override=None):
    """Sec. 4.2 on one sequence, given stage 1's outputs (mass s, salience s_hat, kept / pruned
    lists): routing inside the kept set, Eq. 5 at every anchor (sources added in ascending
    sequence index), refill of the vacated slots from the pruned pool by s_j, hand-off."""
    hid = bf16_bits_to_f64(hidden_bits)
    hv = hid[v0:v0 + nv]
    n = hid.shape[0]
    dest, margin = route_within_kept(hv, s_hat, keep, threshold, max_absorb=len(drop))
    if dest_override is not None:
        dest = np.asarray(dest_override, dtype=np.int32)
    absorbed = np.nonzero(dest >= 0)[0]
    anchors = np.nonzero(dest < 0)[0]
    refill = refill_from_pruned(mass, drop, len(absorbed))
    if refill_override is not None:
        refill = np.asarray(refill_override, dtype=np.int32)
    final = np.sort(np.concatenate([keep[anchors], refill])).astype(np.int32)
    rows = np.empty((len(final), hv.shape[1]))
    merged_mask = np.zeros(len(final), dtype=bool)
    slot_of = {int(v): i for i, v in enumerate(final)}
    for i, v in enumerate(final):
        rows[i] = hv[v]
    for a in anchors:
        src = [int(keep[p]) for p in absorbed if dest[p] == a]          # ascending: keep is ascending
        if not src:
            continue
        i = int(keep[a])
        num = s_hat[i] * hv[i]
        den = s_hat[i]
        for j in src:
            num = num + s_hat[j] * hv[j]
            den = den + s_hat[j]
        if den > eps:
            rows[slot_of[i]] = num / den
            merged_mask[slot_of[i]] = True
    src_row = np.concatenate([np.arange(0, v0), v0 + final, np.arange(v0 + nv, n)]).astype(np.int32)
    out_hidden = np.concatenate([hid[:v0], rows, hid[v0 + nv:]], axis=0)
    out_bits = f64_to_bf16_bits(out_hidden)
    out_bits[:v0] = hidden_bits[:v0]
    out_bits[v0 + len(final):] = hidden_bits[v0 + nv:]
    unmerged = np.nonzero(~merged_mask)[0]
    out_bits[v0 + unmerged] = hidden_bits[v0 + final[unmerged]]        # pure copies keep their bits
    return dict(dest=dest, margin=margin, n_absorbed=len(absorbed), refill=refill, final_keep=final,
                merged=rows, merged_mask=merged_mask, out_hidden=out_hidden, out_hidden_bits=out_bits,
                out_pos=np.asarray(pos_ids)[src_row].astype(np.int32), src_row=src_row)


# ----------------------------------------------------------------------------------
# The layer's attention under the SG-BiMask (Eq. 4 applied to the values)
# ----------------------------------------------------------------------------------
def masked_attention(q_bits, k_bits, v_bits, v0: int, nv: int, m: Optional[np.ndarray],
                     mask_enable: bool = True, rows: Optional[np.ndarray] = None) -> np.ndarray:
    """Eq. 4: O^h = Softmax(W^h + M_bidir) V^h for every query row of one sequence and every head.
    q, k, v: bf16 bit patterns [n, H, d]; m: Eq. 3's vector over the image span (ignored with the
    mask off, which gives the causal attention of Sec. 3.2).  `rows`: the query rows wanted (default
    all).  Returns float64 [len(rows), H, d]."""
    q, k, v = bf16_bits_to_f64(q_bits), bf16_bits_to_f64(k_bits), bf16_bits_to_f64(v_bits)
    n, H, d = q.shape
    rows = np.arange(n) if rows is None else np.asarray(rows)
    per_head = m is not None and np.ndim(m) == 2            # one mask vector per head
    M = None if per_head else mask_matrix(n, rows, v0, nv, m, mask_enable)
    out = np.empty((len(rows), H, d))
    for h in range(H):
        A = attention_probs(q, k, h, rows, v0, nv, m[h] if per_head else m, mask_enable, M)
        out[:, h, :] = A @ v[:, h, :]
    return out


def compact_rows(cache: np.ndarray, src_row: np.ndarray) -> np.ndarray:
    """KV-cache compaction after the hand-off: the cached key / value row of every surviving token,
    in the order of the shortened sequence (row r of the result is row src_row[r] of the cache)."""
    out = np.empty((len(src_row),) + cache.shape[1:], dtype=cache.dtype)
    for r, sr in enumerate(src_row):
        out[r] = cache[int(sr)]
    return out


def prune_batch(q_bits, k_bits, hidden_bits, pos_ids, cu_seqlens, vis_start, vis_len,
                rank_start, rank_len, keep_k: int, samples=None, **params):
    """Packed batch: run prune_sample on each requested sample (all by default)."""
    B = len(cu_seqlens) - 1
    out = {}
    for b in (range(B) if samples is None else samples):
        lo, hi = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        out[b] = prune_sample(q_bits[lo:hi], k_bits[lo:hi], hidden_bits[lo:hi], pos_ids[lo:hi],
                              int(vis_start[b]), int(vis_len[b]), int(rank_start[b]),
                              int(rank_len[b]), keep_k, **params)
    return out
