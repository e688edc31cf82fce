"""The similarity launch picks one of several kernel forms from the problem size.  The large-batch form
(two row tiles per block, kept slots in groups, Sec. 4.2's assignment) is forced here onto small ragged
inputs, so that its edges are compared with the oracle element by element: a second row tile that is
empty, one that is partly filled, several slot groups with a ragged last group, nothing dropped.  The
small-problem form whose slices of the hidden dimension are a thread-block cluster (2, 4 or 8 blocks adding
their partial products through distributed shared memory) is reached with wider hidden states."""
import os

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


@pytest.fixture(scope="module")
def ctx_pair_form():
    old = os.environ.get("ASAP_SIM_PAIR_MIN_BLOCKS")
    os.environ["ASAP_SIM_PAIR_MIN_BLOCKS"] = "1"          # read once, when the context is made
    try:
        c = A.asap_init(0, max_total_tokens=40000, max_B=8, max_H=8, max_D=1024, max_keep_rows=8000)
    finally:
        if old is None:
            del os.environ["ASAP_SIM_PAIR_MIN_BLOCKS"]
        else:
            os.environ["ASAP_SIM_PAIR_MIN_BLOCKS"] = old
    yield c
    A.asap_free(c)


def _merge_matches_oracle(ctx, n_vis, k, H, seed):
    B = len(n_vis)
    batch = W.tiny(B=B, n_vis=n_vis, text_lens=[5 + 3 * b for b in range(B)], H=H, keep_k=k, seed=seed, centres=9)
    p = A.Params(keep_k=k)
    inp = A.make_inputs(batch, DEV)
    mv = inp.max_vis
    sal = torch.zeros(B, mv)
    keep = torch.zeros(B, k, dtype=torch.int32)
    drop = torch.full((B, max(mv - k, 1)), -1, dtype=torch.int32)[:, :mv - k]
    refs = []
    for b in range(B):
        rows = batch.sample_rows(b)
        ref = O.prune_sample(bits(batch.q[rows]), bits(batch.k[rows]), bits(batch.hidden[rows]),
                             batch.pos_ids[rows].numpy(), int(batch.vis_start[b]), int(batch.vis_len[b]),
                             int(batch.text_start[b]), int(batch.text_len[b]), k)
        nv = int(batch.vis_len[b])
        sal[b, :nv] = torch.from_numpy(ref["salience"]).float()
        keep[b] = torch.from_numpy(ref["keep_idx"])
        drop[b, :nv - k] = torch.from_numpy(ref["drop_idx"])
        refs.append(ref)
    out = A.alloc_outputs(inp, k, fill=True)
    A.asap_merge(ctx, inp, p, sal.to(DEV), keep.to(DEV), drop.to(DEV), out)
    torch.cuda.synchronize()
    A.asap_check(ctx)
    ocu = out.out_cu_seqlens.cpu().numpy()
    for b in range(B):
        ref = refs[b]
        nv, v0 = int(batch.vis_len[b]), int(batch.vis_start[b])
        nd = nv - k
        ag = out.assign[b, :nd].cpu().numpy()
        mism = np.nonzero(ag != ref["assign"])[0]
        assert np.all(ref["margin"][mism] <= 1e-4), (b, mism[:8])     # only near-ties may go to another slot
        if nd:
            sim = out.best_sim[b, :nd].cpu().numpy()
            assert np.all(np.abs(sim - ref["best_sim"]) <= 2e-4), b
        rows = batch.sample_rows(b)
        ref2 = O.prune_sample(bits(batch.q[rows]), bits(batch.k[rows]), bits(batch.hidden[rows]),
                              batch.pos_ids[rows].numpy(), v0, nv, int(batch.text_start[b]),
                              int(batch.text_len[b]), k, assign_override=ag)
        gh = O.bf16_bits_to_f64(bits(out.out_hidden[int(ocu[b]):int(ocu[b + 1])].cpu()))
        assert np.all(np.abs(gh - ref2["out_hidden"]) <= merged_tolerance(ref2["out_hidden"])), b
        assert np.array_equal(out.out_pos[int(ocu[b]):int(ocu[b + 1])].cpu().numpy(), ref2["out_pos"])


@pytest.fixture(scope="module")
def ctx_default():
    c = A.asap_init(0, max_total_tokens=40000, max_B=8, max_H=8, max_D=1024, max_keep_rows=8000)
    yield c
    A.asap_free(c)


@pytest.mark.parametrize("n_vis,k,H", [
    ([300, 129], 100, 8),        # hidden size 1024: eight slices per row tile, ragged last row tiles
    ([640], 256, 8),             # the widest single slot tile, 384 dropped rows
    ([200, 130, 131], 16, 4),    # hidden size 512: four slices, one narrow slot tile
    ([129, 129, 129, 129, 129, 129, 129, 129], 33, 8),   # sixteen row tiles: fewer slices per tile
])
def test_cluster_form_matches_the_oracle(ctx_default, n_vis, k, H):
    _merge_matches_oracle(ctx_default, n_vis, k, H, seed=933)


@pytest.mark.parametrize("n_vis,k", [
    ([520, 300, 257], 40),      # three / two / two row tiles: pairs with a full, a partial and an empty second tile
    ([600, 513], 257),          # two groups of 144 slots, the second ragged (113 slots)
    ([256, 300], 256),          # sample 0 drops nothing
    ([129, 1000], 17),          # one group narrower than an MMA's smallest useful width
])
def test_pair_form_matches_the_oracle(ctx_pair_form, n_vis, k):
    _merge_matches_oracle(ctx_pair_form, n_vis, k, H=2, seed=911)


def test_pair_form_gives_up_and_the_context_recovers(ctx_pair_form):
    """The bounded waits of this form, in the harmless way: the wait limit of one call is a single clock
    cycle, the call returns, the status names the kernel, and the next call is a fresh one bit for bit."""
    ctx = ctx_pair_form
    batch = W.tiny(B=2, n_vis=[400, 330], text_lens=[9, 12], H=2, keep_k=150, seed=602, centres=9)
    inp = A.make_inputs(batch, DEV)
    p = A.Params(keep_k=150)
    good = A.alloc_outputs(inp, 150, fill=True)
    A.asap_prune_step(ctx, inp, p, good)
    torch.cuda.synchronize(); A.asap_check(ctx)
    args = (good.salience.clone(), good.keep_idx.clone(), good.drop_idx.clone())

    ref = A.alloc_outputs(inp, 150, fill=True)
    A.asap_merge(ctx, inp, p, *args, ref)
    torch.cuda.synchronize(); A.asap_check(ctx)

    bad = A.alloc_outputs(inp, 150, fill=True)
    A.asap_debug_wait_limit(ctx, 1)
    A.asap_merge(ctx, inp, p, *args, bad)
    torch.cuda.synchronize()
    with pytest.raises(A.AsapError) as e:
        A.asap_check(ctx)
    assert e.value.status == -6 and "timed out in the similarity kernel" in str(e.value)

    again = A.alloc_outputs(inp, 150, fill=True)
    A.asap_merge(ctx, inp, p, *args, again)
    torch.cuda.synchronize(); A.asap_check(ctx)
    for n in ("assign", "best_sim", "out_hidden", "out_pos", "src_row", "out_cu_seqlens"):
        assert torch.equal(getattr(ref, n), getattr(again, n)), n
