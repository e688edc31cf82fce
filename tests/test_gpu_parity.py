"""GPU parity: the CUDA prune step, called through the C ABI, against the CPU oracle on the
same seeded inputs.  Sizes span several 128-wide tiles with ragged tails; the benchmark shapes
run at full size with the oracle evaluated on a sample of the sequences."""
import math

import numpy as np
import pytest
import torch

from paper_2603_14549_b200 import binding as A
from paper_2603_14549_b200 import workloads as W
from tests.parity import check_invariants, compare_sample

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    c = A.asap_init(0, max_total_tokens=80000, max_B=32, max_H=40, max_D=5120, max_keep_rows=40000)
    yield c
    A.asap_free(c)


def run_step(ctx, batch, params, rank_start=None, rank_len=None, samples=None, stats=None):
    inp = A.make_inputs(batch, DEV, rank_start, rank_len)
    out = A.alloc_outputs(inp, params.keep_k, fill=True, per_head=params.per_head_mask)
    A.asap_prune_step(ctx, inp, params, out)
    torch.cuda.synchronize()
    A.asap_check(ctx)
    for b in (range(batch.B) if samples is None else samples):
        compare_sample(batch, b, params, out, rank_start, rank_len, stats)
    if samples is not None:          # the oracle saw a sample of the batch: every sequence still has to be well formed
        for b in range(batch.B):
            check_invariants(batch, b, params, out)
    return inp, out


def test_ragged_multi_tile(ctx):
    batch = W.tiny(B=3, n_vis=[130, 257, 64], text_lens=[5, 17, 33], H=2, keep_k=16, seed=101, centres=6)
    run_step(ctx, batch, A.Params(keep_k=16))


@pytest.mark.parametrize("k", [300, 512, 257])
def test_two_slot_tiles_in_one_pass(ctx, k):
    """257 .. 512 kept slots: two slot tiles whose accumulators share tensor memory, one pass over the
    hidden dimension (300 and 257 leave a ragged second slot tile, 512 fills every column)."""
    batch = W.tiny(B=2, n_vis=[700, 650], text_lens=[12, 40], H=2, keep_k=k, seed=107, centres=30)
    run_step(ctx, batch, A.Params(keep_k=k))


def test_many_row_tiles_and_three_slot_tiles(ctx):
    """A batch large enough that the similarity kernel runs unsliced with more blocks than SMs
    (15 sequences x 19 row tiles) and three slot tiles (600 kept slots).  Odd and even numbers of row
    tiles, a ragged last tile of one row; the oracle checks three sequences."""
    nvs = [2350 if b % 2 else 2432 for b in range(15)]
    nvs[0] = 2305                                               # 19 row tiles, one row in the last
    batch = W.tiny(B=15, n_vis=nvs, text_lens=[6 + b for b in range(15)], H=2, keep_k=600, seed=108, centres=40)
    run_step(ctx, batch, A.Params(keep_k=600), samples=[0, 1, 14])


def test_a_late_dominant_key_moves_the_softmax_reference(ctx):
    """One visual key far into the sequence is scaled so that its logits exceed every earlier logit of a
    ranking row by hundreds of nats (or fall that far below, for rows whose dot product is negative).  A
    running sum kept relative to an early maximum would overflow there: the row's reference has to move,
    and the probabilities of all other keys have to come out as (correctly) vanishing."""
    batch = W.tiny(B=2, n_vis=[400, 330], text_lens=[40, 150], H=2, keep_k=50, seed=110, centres=8)
    for b, where in ((0, 300), (1, 200)):
        row = int(batch.cu_seqlens[b]) + int(batch.vis_start[b]) + where
        batch.k[row] = (batch.k[row].float() * 300.0).to(torch.bfloat16)
    run_step(ctx, batch, A.Params(keep_k=50))


def test_text_longer_than_one_row_tile(ctx):
    batch = W.tiny(B=2, n_vis=[200, 140], text_lens=[150, 129], H=2, keep_k=40, seed=102, centres=8)
    run_step(ctx, batch, A.Params(keep_k=40))


@pytest.mark.parametrize("lambda_max", [1.0, 0.5, 0.1])
def test_visual_ranking_rows_use_the_soft_mask(ctx, lambda_max):
    batch = W.tiny(B=2, n_vis=[300, 129], text_lens=[20, 7], H=2, keep_k=32, seed=103, centres=8)
    rs = batch.vis_start.clone()
    rl = batch.vis_len + batch.text_len            # ranking rows = image span + text span
    run_step(ctx, batch, A.Params(keep_k=32, lambda_max=lambda_max), rs, rl)


@pytest.mark.parametrize("lambda_max", [1.0, 0.3])
def test_per_head_masks_with_visual_ranking_rows(ctx, lambda_max):
    """Eq. 1-3 per head: four heads with their own salience and mask vector; the ranking rows include
    the image span, so every head's logits are really shifted by that head's mask."""
    batch = W.tiny(B=2, n_vis=[300, 129], text_lens=[20, 7], H=4, keep_k=32, seed=105, centres=8)
    rs = batch.vis_start.clone()
    rl = batch.vis_len + batch.text_len
    inp, out = run_step(ctx, batch, A.Params(keep_k=32, lambda_max=lambda_max, per_head_mask=True), rs, rl)
    mh = out.mask_log_heads.cpu()
    assert float((mh[0, 0, :300] - mh[0, 1, :300]).abs().max()) > 1e-3      # the heads' masks do differ


def test_per_head_masks_with_text_ranking_rows(ctx):
    batch = W.tiny(B=3, n_vis=[130, 257, 64], text_lens=[5, 17, 33], H=2, keep_k=16, seed=106, centres=6)
    run_step(ctx, batch, A.Params(keep_k=16, per_head_mask=True))


def test_ranking_rows_partly_visual_and_mask_off(ctx):
    batch = W.tiny(B=2, n_vis=[260, 131], text_lens=[9, 30], H=1, keep_k=20, seed=104)
    rs = batch.vis_start + 100
    rl = batch.vis_len - 100 + batch.text_len
    run_step(ctx, batch, A.Params(keep_k=20, lambda_max=0.7), rs, rl)
    run_step(ctx, batch, A.Params(keep_k=20, mask_enable=False), rs, rl)


def test_identity_when_k_equals_visual_count(ctx):
    batch = W.tiny(B=2, n_vis=[150, 150], text_lens=[4, 40], H=2, keep_k=150, seed=105)
    inp, out = run_step(ctx, batch, A.Params(keep_k=150))
    assert torch.equal(out.out_hidden.cpu(), batch.hidden)
    assert torch.equal(out.out_pos.cpu(), batch.pos_ids)


def test_one_sequence_keeps_everything_while_another_merges(ctx):
    """keep_k equals the first sequence's visual count (nothing dropped there, its rows are copies) while
    the second one drops and merges 80 tokens."""
    batch = W.tiny(B=2, n_vis=[150, 230], text_lens=[9, 21], H=2, keep_k=150, seed=109, centres=9)
    inp, out = run_step(ctx, batch, A.Params(keep_k=150))
    n0 = int(batch.cu_seqlens[1])
    assert torch.equal(out.out_hidden[:n0].cpu(), batch.hidden[:n0])
    assert int((out.assign[0] >= 0).sum()) == 0 and int((out.assign[1] >= 0).sum()) == 80


def test_mask_off_merge_off_is_plain_topk_gather(ctx):
    batch = W.tiny(B=2, n_vis=[190, 133], text_lens=[12, 31], H=2, keep_k=24, seed=106)
    inp, out = run_step(ctx, batch, A.Params(keep_k=24, mask_enable=False, merge_enable=False))
    n_out = int(out.out_cu_seqlens[-1])                 # the buffers are sized for the worst case
    src = out.src_row[:n_out].cpu().long()
    assert torch.equal(out.out_hidden[:n_out].cpu(), batch.hidden[src])


@pytest.mark.parametrize("t", [0.8, 0.95, 1.0])
def test_similarity_threshold(ctx, t):
    batch = W.tiny(B=2, n_vis=[180, 140], text_lens=[10, 20], H=2, keep_k=30, seed=107, centres=5)
    inp, out = run_step(ctx, batch, A.Params(keep_k=30, sim_threshold=t))
    if t >= 1.0:
        assert int((out.assign >= 0).sum()) == 0


@pytest.mark.parametrize("nv", [1, 2, 3, 5, 8, 127, 128, 129])
@pytest.mark.parametrize("tl", [1, 16, 17])
def test_edge_sizes(ctx, nv, tl):
    ks = sorted({1, max(1, nv - 1), nv})
    for k in ks:
        batch = W.tiny(B=2, n_vis=[nv, nv], text_lens=[tl, tl + 1], H=1, keep_k=k, seed=200 + nv, centres=2)
        run_step(ctx, batch, A.Params(keep_k=k))


def test_duplicate_token_merges_into_its_twin(ctx):
    """Ranking reads only Q and K, so overwriting a dropped token's hidden row does not change the kept
    set: the token stays dropped, and as a copy of a kept row it must land on that row's slot with
    similarity 1 (no other kept row equals it: the rows are noisy draws)."""
    batch = W.tiny(B=1, n_vis=[140], text_lens=[8], H=2, keep_k=20, seed=108, centres=50)
    inp = A.make_inputs(batch, DEV)
    out = A.alloc_outputs(inp, 20, fill=True)
    p = A.Params(keep_k=20)
    A.asap_prune_step(ctx, inp, p, out)
    torch.cuda.synchronize()
    keep = out.keep_idx[0].cpu()
    drop = out.drop_idx[0].cpu()
    v0 = int(batch.vis_start[0])
    victim = int(drop[5])
    batch.hidden[v0 + victim] = batch.hidden[v0 + int(keep[3])]
    inp2, out2 = run_step(ctx, batch, p)
    assert torch.equal(out2.keep_idx[0].cpu(), keep)          # same Q / K, same ranking
    pos = (out2.drop_idx[0] == victim).nonzero()
    assert len(pos) == 1
    dp = int(pos[0])
    assert int(out2.assign[0, dp]) == 3
    assert abs(float(out2.best_sim[0, dp]) - 1.0) < 1e-5


def test_c1_full(ctx):
    stats = {}
    batch = W.config("c1")
    run_step(ctx, batch, A.Params(keep_k=batch.keep_k), stats=stats)
    print("c1 parity maxima", stats)


def test_c2_full_size_sampled(ctx):
    stats = {}
    batch = W.config("c2")
    run_step(ctx, batch, A.Params(keep_k=batch.keep_k), samples=[0, 7, 15], stats=stats)
    print("c2 parity maxima", stats)


@pytest.mark.parametrize("k", [320, 160])
def test_c3_prefix_with_outliers(ctx, k):
    stats = {}
    batch = W.config("c3", B=2, keep_k=k)
    run_step(ctx, batch, A.Params(keep_k=k), samples=[1], stats=stats)
    print("c3 parity maxima", stats)


def test_c4_prefix_sampled(ctx):
    stats = {}
    batch = W.config("c4", B=6)
    run_step(ctx, batch, A.Params(keep_k=batch.keep_k), samples=[5], stats=stats)
    print("c4 parity maxima", stats)


@pytest.fixture(scope="module")
def big_ctx():
    """Capacity of the largest benchmark shape (64 sequences of 35 + 2880 + up to 256 tokens)."""
    c = A.asap_init(0, max_total_tokens=64 * (35 + 2880 + 256), max_B=64, max_H=40, max_D=5120,
                    max_keep_rows=64 * 1152)
    yield c
    A.asap_free(c)


@pytest.mark.parametrize("k", [320, 160])
def test_c3_full_size_sampled(big_ctx, k):
    """The whole LLaVA-NeXT batch of 8 as bench.py runs it; the oracle checks two sequences."""
    stats = {}
    batch = W.config("c3", keep_k=k)
    run_step(big_ctx, batch, A.Params(keep_k=k), samples=[0, 7], stats=stats)
    print("c3 full parity maxima", stats)


@pytest.mark.parametrize("k", [510, 340])
def test_c6_internvl_shape_full_size_sampled(big_ctx, k):
    """InternVL-2.5-8B-shaped batch (1536 visual tokens in six tiles of 256) at the two budgets of
    Sec. 5.4 (~510 and ~340 tokens); neither is a multiple of 16, so the similarity kernel's kept-slot
    tiles are ragged.  The oracle checks two sequences."""
    stats = {}
    batch = W.config("c6", keep_k=k)
    run_step(big_ctx, batch, A.Params(keep_k=k), samples=[0, 7], stats=stats)
    print("c6 full parity maxima", stats)


def test_c4_full_size_sampled(big_ctx):
    """The AnyRes throughput shape at full size (64 sequences, 2880 visual tokens, ragged text up
    to 256 rows = two ranking-row tiles); the oracle checks the first and the last sequence."""
    stats = {}
    batch = W.config("c4")
    run_step(big_ctx, batch, A.Params(keep_k=batch.keep_k), samples=[0, 63], stats=stats)
    print("c4 full parity maxima", stats)


def test_c5_full_size_first_step_sampled(big_ctx):
    """13B-shaped batch of 32 (D = 5120, 40 heads), first step 2304 -> 1152, at full size."""
    stats = {}
    batch = W.config("c5")
    run_step(big_ctx, batch, A.Params(keep_k=batch.keep_k), samples=[31], stats=stats)
    print("c5 full parity maxima", stats)


def _c5_schedule(ctx, B, samples):
    batch = W.config("c5", B=B)
    cur = batch
    for step, k in enumerate(W.C5_SCHEDULE):
        p = A.Params(keep_k=k)
        cur.keep_k = k
        stats = {}
        inp, out = run_step(ctx, cur, p, samples=samples, stats=stats)
        print(f"c5 step {step + 1} (B = {B}) parity maxima", stats)
        ocu = out.out_cu_seqlens.cpu()
        hidden = out.out_hidden[: int(ocu[-1])].cpu()
        pos = out.out_pos[: int(ocu[-1])].cpu()
        q, kk = W.redraw_qk(pos, ocu, cur.H, cur.head_dim, cur.seed, step + 1)
        cur = W.Batch(name="c5", B=cur.B, H=cur.H, head_dim=cur.head_dim, D=cur.D, keep_k=k, cu_seqlens=ocu,
                      vis_start=cur.vis_start, vis_len=torch.full_like(cur.vis_len, k),
                      text_start=cur.vis_start + k, text_len=cur.text_len, q=q, k=kk, hidden=hidden,
                      pos_ids=pos, seed=cur.seed)


def test_c5_progressive_three_steps(ctx):
    """13B-shaped schedule 2304 -> 1152 -> 576 -> 288: every step consumes the previous step's
    hidden states and gathered position ids, with Q/K re-drawn at those positions."""
    _c5_schedule(ctx, 2, [1])


def test_c5_progressive_three_steps_full_batch(big_ctx):
    """The same schedule on the whole batch of 32 (the sizes the benchmark times): the oracle checks one
    sequence per step, every other sequence is checked for the properties that need no oracle."""
    _c5_schedule(big_ctx, 32, [17])
