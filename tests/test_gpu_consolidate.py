"""asap_consolidate (Sec. 4.2 as worded: routing inside the kept set, Eq. 5 at the anchors, refill
by attention mass) against the CPU oracle, through the C ABI.

Stage 1's results are taken from the oracle, rounded to fp32, and given to both sides, so the
comparison isolates stage 2.  Integer results (who is absorbed by whom, the refill, the final
kept list, position ids, row maps) must be identical; if they are not, the oracle must have had
a decision closer than 1e-4 to flipping (similarity against t, or best against runner-up anchor),
the GPU's routing must pass the structural checks, and the oracle is re-evaluated with it."""
import math

import numpy as np
import pytest
import torch

from oracle import asap_oracle as O
from paper_2603_14549_b200 import binding as A
from paper_2603_14549_b200 import workloads as W
from tests.helpers import bits
from tests.parity import merged_tolerance

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TIE = 1e-4


@pytest.fixture(scope="module")
def ctx():
    c = A.asap_init(0, max_total_tokens=40000, max_B=16, max_H=8, max_D=1024, max_keep_rows=20000)
    yield c
    A.asap_free(c)


def _stage1(batch, b, k):
    rows = batch.sample_rows(b)
    ref = O.prune_sample(bits(batch.q[rows]), bits(batch.k[rows]), bits(batch.hidden[rows]),
                         batch.pos_ids[rows].numpy(), int(batch.vis_start[b]), int(batch.vis_len[b]),
                         int(batch.text_start[b]), int(batch.text_len[b]), k)
    f32 = lambda x: x.astype(np.float32)
    return f32(ref["mass"]), f32(ref["salience"]), ref["keep_idx"], ref["drop_idx"]


def _run(ctx, batch, k, t, salience_override=None, stage1=None):
    B = batch.B
    p = A.Params(keep_k=k, sim_threshold=t)
    inp = A.make_inputs(batch, DEV)
    mv = inp.max_vis
    mass = torch.zeros(B, mv); sal = torch.zeros(B, mv)
    keep = torch.zeros(B, k, dtype=torch.int32); drop = torch.full((B, mv - k), -1, dtype=torch.int32)
    st1 = []
    for b in range(B):
        m, s, kp, dp = (stage1 or _stage1)(batch, b, k)
        if salience_override is not None:
            s = salience_override(b, s)
        nv = int(batch.vis_len[b])
        mass[b, :nv] = torch.from_numpy(m); sal[b, :nv] = torch.from_numpy(s)
        keep[b] = torch.from_numpy(kp); drop[b, :nv - k] = torch.from_numpy(dp)
        st1.append((m.astype(np.float64), s.astype(np.float64), kp, dp))
    out = A.alloc_outputs(inp, k, fill=True)
    scratch = torch.empty(A.asap_consolidate_scratch_bytes(B, k), dtype=torch.uint8, device=DEV)
    n_abs = torch.full((B,), -7, dtype=torch.int32, device=DEV)
    A.asap_consolidate(ctx, inp, p, mass.to(DEV), sal.to(DEV), keep.to(DEV), drop.to(DEV), scratch, out, n_abs)
    torch.cuda.synchronize(); A.asap_check(ctx)
    return out, n_abs.cpu().numpy(), st1


def _check(batch, k, t, out, n_abs, st1, samples=None):
    ocu = out.out_cu_seqlens.cpu().numpy()
    total_abs = 0
    for b in (range(batch.B) if samples is None else samples):
        rows = batch.sample_rows(b)
        v0, nv = int(batch.vis_start[b]), int(batch.vis_len[b])
        m, s, kp, dp = st1[b]
        hb = bits(batch.hidden[rows]); pos = batch.pos_ids[rows].numpy()
        ref = O.consolidate_sample(hb, pos, v0, nv, m, s, kp, dp, t)
        a = int(n_abs[b]); nd = nv - k
        fk = out.keep_idx[b].cpu().numpy()
        src = out.drop_idx[b].cpu().numpy(); asg = out.assign[b].cpu().numpy()
        assert np.all(src[a:] == -1) and np.all(asg[a:] == -1) and 0 <= a <= nd
        assert np.all(np.diff(fk) > 0) and fk.min() >= 0 and fk.max() < nv
        # the GPU's routing in the oracle's terms: dest[slot of stage-1 keep] = slot of the anchor or -1
        slot_of = {int(v): i for i, v in enumerate(kp)}
        dest = np.full(k, -1, dtype=np.int32)
        for i in range(a):
            assert asg[i] >= 0
            dest[slot_of[int(src[i])]] = slot_of[int(fk[asg[i]])]
        if not np.array_equal(dest, ref["dest"]):
            finite = ref["margin"][np.isfinite(ref["margin"])]
            assert finite.size and finite.min() <= TIE, (b, "routing differs although no oracle decision was close")
            hv = O.bf16_bits_to_f64(hb)[v0:v0 + nv]
            S = O.cosine_matrix(hv[kp], hv[kp])
            for pslot in np.nonzero(dest >= 0)[0]:
                an = dest[pslot]
                assert dest[an] < 0 and S[an, pslot] > t - TIE
                assert (s[kp[an]], -kp[an]) > (s[kp[pslot]], -kp[pslot])
            ref = O.consolidate_sample(hb, pos, v0, nv, m, s, kp, dp, t, dest_override=dest)
        assert a == ref["n_absorbed"]
        if not np.array_equal(fk, ref["final_keep"]):       # refill: only equal-mass-within-rounding swaps
            extra, missing = np.setdiff1d(fk, ref["final_keep"]), np.setdiff1d(ref["final_keep"], fk)
            assert len(extra) == len(missing) and set(extra) <= set(dp)
            assert np.all(np.abs(m[extra] - m[missing].mean()) <= TIE * np.abs(m).max())
            ref = O.consolidate_sample(hb, pos, v0, nv, m, s, kp, dp, t, dest_override=dest,
                                       refill_override=np.setdiff1d(fk, kp))
        assert np.array_equal(fk, ref["final_keep"])
        lo, hi = int(ocu[b]), int(ocu[b + 1])
        assert hi - lo == (rows.stop - rows.start) - nv + k
        assert np.array_equal(out.out_pos[lo:hi].cpu().numpy(), ref["out_pos"])
        assert np.array_equal(out.src_row[lo:hi].cpu().numpy() - int(rows.start), ref["src_row"])
        gbits = bits(out.out_hidden[lo:hi].cpu())
        gh = O.bf16_bits_to_f64(gbits)
        err = np.abs(gh - ref["out_hidden"])
        assert np.all(err <= merged_tolerance(ref["out_hidden"])), (b, err.max())
        copies = np.ones(hi - lo, dtype=bool)
        copies[v0 + np.nonzero(ref["merged_mask"])[0]] = False
        assert np.array_equal(gbits[copies], ref["out_hidden_bits"][copies])            # copies: bit-exact
        if out.best_sim is not None and a:
            hv = O.bf16_bits_to_f64(hb)[v0:v0 + nv]
            S = O.cosine_matrix(hv[src[:a]], hv[fk[asg[:a]]]).diagonal()
            assert np.all(np.abs(out.best_sim[b, :a].cpu().numpy() - S) <= 2e-4)
        total_abs += a
    return total_abs


@pytest.mark.parametrize("nvs,texts,k,t,centres", [
    ([300, 170, 520], [9, 30, 4], 96, 0.8, 12),          # one row tile, ragged
    ([450, 260], [5, 5], 200, 0.85, 20),                 # two row tiles with a ragged second one
    ([700], [12], 300, 0.8, 25),                         # two accumulators of kept slots
    ([130, 600], [3, 3], 129, 0.7, 6),                   # 129: a one-row second tile; sample 0 has a pool of one
], ids=["k96", "k200", "k300", "k129"])
def test_consolidate_matches_oracle(ctx, nvs, texts, k, t, centres):
    batch = W.tiny(B=len(nvs), n_vis=nvs, text_lens=texts, H=2, keep_k=k, seed=500 + k, centres=centres)
    out, n_abs, st1 = _run(ctx, batch, k, t)
    total = _check(batch, k, t, out, n_abs, st1)
    assert total > 0, "the case was meant to exercise merging"


def test_refill_treats_signed_zero_masses_as_equal(ctx):
    """Attention masses of -0.0 and +0.0 are one value: the refill takes the lower index among them,
    exactly as the oracle's (mass descending, index ascending) order does.  Most of the pruned pool
    carries a zero of alternating sign, so the vacated slots are refilled across such ties."""
    nvs, k, t = [300, 170, 520], 96, 0.8
    batch = W.tiny(B=3, n_vis=nvs, text_lens=[9, 30, 4], H=2, keep_k=k, seed=500 + k, centres=12)

    def stage1(bt, b, kk):
        m, s, kp, dp = _stage1(bt, b, kk)
        m = m.copy()
        m[dp[0::2]] = -0.0
        m[dp[1::2]] = 0.0
        m[dp[5::17]] = -1.5                     # a few pruned tokens rank below the zeros
        m[dp[3::29]] = 2.0                      # ... and a few above
        return m, s, kp, dp

    out, n_abs, st1 = _run(ctx, batch, k, t, stage1=stage1)
    assert n_abs.sum() > 0
    for b in range(3):
        rows = batch.sample_rows(b)
        m, s, kp, dp = st1[b]
        ref = O.consolidate_sample(bits(batch.hidden[rows]), batch.pos_ids[rows].numpy(), int(batch.vis_start[b]),
                                   nvs[b], m, s, kp, dp, t)
        if int(n_abs[b]) == ref["n_absorbed"]:   # same routing (it does not depend on the masses): same refill, bit for bit
            want = np.setdiff1d(ref["final_keep"], kp)
            got = np.setdiff1d(out.keep_idx[b].cpu().numpy(), kp)
            assert np.array_equal(got, want), b
    _check(batch, k, t, out, n_abs, st1)


def test_threshold_one_is_a_plain_gather(ctx):
    batch = W.tiny(B=2, n_vis=[200, 90], text_lens=[4, 4], H=2, keep_k=40, seed=510, centres=5)
    out, n_abs, st1 = _run(ctx, batch, 40, 1.0)
    assert np.all(n_abs == 0)
    _check(batch, 40, 1.0, out, n_abs, st1)
    for b in range(2):
        assert np.array_equal(out.keep_idx[b].cpu().numpy(), st1[b][2])


def test_absorption_stops_when_the_pool_is_empty(ctx):
    """One cluster, tiny pool: every kept token is similar to the first, only nv - k can go."""
    batch = W.tiny(B=2, n_vis=[64, 100], text_lens=[4, 4], H=2, keep_k=60, seed=511, centres=1)
    out, n_abs, st1 = _run(ctx, batch, 60, 0.5)
    assert n_abs.tolist() == [4, 40]
    _check(batch, 60, 0.5, out, n_abs, st1)
    for b in range(2):                                     # the whole pool was refilled
        assert set(st1[b][3]) <= set(out.keep_idx[b].cpu().numpy().tolist())


def test_equal_salience_is_ordered_by_sequence_index(ctx):
    batch = W.tiny(B=1, n_vis=[260], text_lens=[6], H=2, keep_k=80, seed=512, centres=8)
    out, n_abs, st1 = _run(ctx, batch, 80, 0.8, salience_override=lambda b, s: np.round(s * 4) / 4)
    assert _check(batch, 80, 0.8, out, n_abs, st1) > 0


def test_consolidate_argument_errors(ctx):
    batch = W.tiny(B=1, n_vis=[100], text_lens=[4], H=2, keep_k=20, seed=513)
    inp = A.make_inputs(batch, DEV)
    out = A.alloc_outputs(inp, 20, fill=True)
    z = torch.zeros(1, 100, device=DEV)
    keep = torch.arange(20, dtype=torch.int32, device=DEV)[None]
    drop = torch.arange(20, 100, dtype=torch.int32, device=DEV)[None]
    small = torch.empty(16, dtype=torch.uint8, device=DEV)
    big = torch.empty(A.asap_consolidate_scratch_bytes(1, 20), dtype=torch.uint8, device=DEV)
    n0 = A.asap_launch_count(ctx)
    with pytest.raises(A.AsapError) as e:
        A.asap_consolidate(ctx, inp, A.Params(keep_k=20), z, z, keep, drop, small, out)
    assert e.value.status == -3
    with pytest.raises(A.AsapError) as e:
        A.asap_consolidate(ctx, inp, A.Params(keep_k=20, merge_enable=0), z, z, keep, drop, big, out)
    assert e.value.status == -1
    with pytest.raises(A.AsapError) as e:
        A.asap_consolidate(ctx, inp, A.Params(keep_k=20), z, z, out.keep_idx, drop, big, out)
    assert e.value.status == -1
    assert A.asap_launch_count(ctx) == n0
    assert A.asap_consolidate_scratch_bytes(1, 20) >= 20 * 20 * 4 and A.asap_consolidate_scratch_bytes(0, 20) == 0


def test_bit_matrix_in_global_memory_for_large_keep(ctx):
    """keep_k = 1400: the bit matrix (1400 x 44 words) no longer fits in shared memory and lives in the
    caller's scratch; six row tiles, six accumulators."""
    batch = W.tiny(B=1, n_vis=[3000], text_lens=[8], H=2, keep_k=1400, seed=514, centres=90)
    out, n_abs, st1 = _run(ctx, batch, 1400, 0.85)
    assert _check(batch, 1400, 0.85, out, n_abs, st1) > 0


@pytest.fixture(scope="module")
def big_ctx():
    c = A.asap_init(0, max_total_tokens=32 * (35 + 2304 + 128) + 2304, max_B=32, max_H=40, max_D=5120,
                    max_keep_rows=32 * 1152)
    yield c
    A.asap_free(c)


@pytest.mark.parametrize("name,t,samples", [("c2", 0.8, None), ("c3", 0.8, [0, 7]), ("c5", 0.85, [31])])
def test_consolidate_at_benchmark_sizes(big_ctx, name, t, samples):
    """Full batches of the benchmark shapes (hidden sizes 4096 / 5120, keep_k 64 / 320 / 1152) with
    seeded stand-ins for stage 1's results; the oracle checks the listed sequences."""
    batch = W.config(name)
    k = batch.keep_k
    out, n_abs, st1 = _run(big_ctx, batch, k, t, stage1=lambda bt, b, kk: W.random_stage1(bt, b, kk, 900))
    assert np.all(n_abs >= 0) and np.all(n_abs <= np.asarray(batch.vis_len) - k)
    assert _check(batch, k, t, out, n_abs, st1, samples=samples) > 0


def test_a_bad_sequence_is_skipped_and_flagged(ctx):
    """Device-side validation: a sequence whose span does not fit its length is skipped (outputs -1 / 0
    rows untouched), the status word says so, the other sequence is processed normally."""
    batch = W.tiny(B=2, n_vis=[200, 150], text_lens=[4, 4], H=2, keep_k=40, seed=515, centres=5)
    good_out, good_abs, st1 = _run(ctx, batch, 40, 0.8)
    inp = A.make_inputs(batch, DEV)
    bad_len = batch.vis_len.clone(); bad_len[0] = 9999
    inp.vis_len = bad_len.to(DEV)
    mv = inp.max_vis
    mass = torch.zeros(2, mv); sal = torch.zeros(2, mv)
    keep = torch.zeros(2, 40, dtype=torch.int32); drop = torch.full((2, mv - 40), -1, dtype=torch.int32)
    for b in range(2):
        m, s, kp, dp = st1[b]
        nv = int(batch.vis_len[b])
        mass[b, :nv] = torch.from_numpy(m).float(); sal[b, :nv] = torch.from_numpy(s).float()
        keep[b] = torch.from_numpy(kp); drop[b, :nv - 40] = torch.from_numpy(dp)
    out = A.alloc_outputs(inp, 40, fill=True)
    scratch = torch.empty(A.asap_consolidate_scratch_bytes(2, 40), dtype=torch.uint8, device=DEV)
    n_abs = torch.full((2,), -7, dtype=torch.int32, device=DEV)
    A.asap_consolidate(ctx, inp, A.Params(keep_k=40, sim_threshold=0.8), mass.to(DEV), sal.to(DEV), keep.to(DEV),
                       drop.to(DEV), scratch, out, n_abs)
    torch.cuda.synchronize()
    with pytest.raises(A.AsapError) as e:
        A.asap_check(ctx)
    assert e.value.status == -6 and "validation" in str(e.value)
    assert torch.all(out.keep_idx[0] == -1) and int(n_abs[0]) == 0
    assert torch.equal(out.keep_idx[1], good_out.keep_idx[1]) and int(n_abs[1]) == int(good_abs[1])


def test_threshold_minus_infinity_absorbs_until_the_pool_is_empty(ctx):
    """t = -inf: every token after the first is similar enough to some anchor, so the walk absorbs until
    the pruned pool cannot refill another slot (here nv - k = 30 and 50 of the 59 candidates)."""
    batch = W.tiny(B=2, n_vis=[90, 110], text_lens=[4, 4], H=2, keep_k=60, seed=516, centres=7)
    out, n_abs, st1 = _run(ctx, batch, 60, -math.inf)
    assert n_abs.tolist() == [30, 50]
    _check(batch, 60, -math.inf, out, n_abs, st1)
