"""GPU tests of the individual entry points, of the integer paths (bit-exact), and of the
boundary's error handling."""
import math

import numpy as np
import pytest
import torch

from oracle import asap_oracle as O
from paper_2603_14549_b200 import binding as A
from paper_2603_14549_b200 import workloads as W
from tests.helpers import bits
from tests.parity import compare_sample, merged_tolerance

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    c = A.asap_init(0, max_total_tokens=40000, max_B=64, max_H=8, max_D=1024, max_keep_rows=20000)
    yield c
    A.asap_free(c)


def _oracle_scores(batch, b, params):
    rows = batch.sample_rows(b)
    return O.prune_sample(bits(batch.q[rows]), bits(batch.k[rows]), bits(batch.hidden[rows]),
                          batch.pos_ids[rows].numpy(), int(batch.vis_start[b]), int(batch.vis_len[b]),
                          int(batch.text_start[b]), int(batch.text_len[b]), params.keep_k,
                          lambda_max=params.lambda_max)


def test_score_entry_point_alone(ctx):
    batch = W.tiny(B=3, n_vis=[140, 70, 260], text_lens=[9, 40, 3], H=2, keep_k=10, seed=301)
    p = A.Params(keep_k=10, lambda_max=0.6)
    inp = A.make_inputs(batch, DEV)
    out = A.alloc_outputs(inp, 10, fill=True)
    A.asap_score(ctx, inp, p, out)
    torch.cuda.synchronize(); A.asap_check(ctx)
    for b in range(3):
        ref = _oracle_scores(batch, b, p)
        nv = int(batch.vis_len[b])
        for name in ("mass", "salience", "rank_score"):
            g = getattr(out, name)[b, :nv].cpu().numpy().astype(np.float64)
            o = ref[name]
            err = np.abs(g - o) / np.maximum(np.abs(o), 1e-3 * np.abs(o).max())
            assert err.max() <= 1e-3, (name, b, err.max())
    assert int(out.keep_idx.min()) == -7          # untouched by asap_score


def test_score_entry_point_per_head(ctx):
    batch = W.tiny(B=2, n_vis=[140, 260], text_lens=[9, 3], H=4, keep_k=10, seed=305)
    p = A.Params(keep_k=10, lambda_max=0.6, per_head_mask=True)
    inp = A.make_inputs(batch, DEV)
    out = A.alloc_outputs(inp, 10, fill=True, per_head=True)
    A.asap_score(ctx, inp, p, out)
    torch.cuda.synchronize(); A.asap_check(ctx)
    for b in range(2):
        rows = batch.sample_rows(b)
        ref = O.prune_sample(bits(batch.q[rows]), bits(batch.k[rows]), bits(batch.hidden[rows]),
                             batch.pos_ids[rows].numpy(), int(batch.vis_start[b]), int(batch.vis_len[b]),
                             int(batch.text_start[b]), int(batch.text_len[b]), 10, lambda_max=0.6, per_head=True)
        nv = int(batch.vis_len[b])
        for name in ("mass", "salience", "rank_score"):
            g = getattr(out, name)[b, :nv].cpu().numpy().astype(np.float64)
            o = ref[name]
            err = np.abs(g - o) / np.maximum(np.abs(o), 1e-3 * np.abs(o).max())
            assert err.max() <= 1e-3, (name, b, err.max())
        mh = out.mask_log_heads[b, :, :nv].cpu().numpy().astype(np.float64)
        assert np.abs(np.exp(mh) - np.exp(ref["mask_log_heads"])).max() <= 1e-4
    with pytest.raises(A.AsapError) as e:                      # the per-head array is required in this mode
        A.asap_score(ctx, inp, p, A.alloc_outputs(inp, 10))
    assert e.value.status == -1


def test_select_is_bit_exact_with_ties(ctx):
    """asap_select on given fp32 scores must reproduce the stable top-k exactly, ties included."""
    g = torch.Generator().manual_seed(5)
    B, mv = 5, 700
    nvs = [700, 699, 513, 512, 64]
    ks = [64]
    batch = W.tiny(B=B, n_vis=nvs, text_lens=[2] * B, H=1, keep_k=64, seed=302)
    inp = A.make_inputs(batch, DEV)
    for trial, k in enumerate([1, 63, 64]):
        scores = torch.zeros(B, mv)
        for b in range(B):
            base = torch.randn(nvs[b], generator=g)
            if trial % 2 == 0:
                base = torch.round(base * 4) / 4          # heavy ties, negative and positive values
            scores[b, :nvs[b]] = base
        scores[0, 10] = float("inf"); scores[1, 11] = float("-inf"); scores[2, :5] = -0.0; scores[2, 5:9] = 0.0
        out = A.alloc_outputs(inp, k, fill=True)
        p = A.Params(keep_k=k)
        A.asap_select(ctx, inp, p, scores.to(DEV), out)
        torch.cuda.synchronize(); A.asap_check(ctx)
        for b in range(B):
            r = scores[b, :nvs[b]].numpy().astype(np.float64)
            keep, drop = O.select_topk(r, k)
            # sample 2 holds -0.0 and +0.0: one score, so the lower index wins among them
            assert np.array_equal(out.keep_idx[b].cpu().numpy(), keep), (trial, b)
            assert np.array_equal(out.drop_idx[b, :nvs[b] - k].cpu().numpy(), drop), (trial, b)
            assert torch.all(out.drop_idx[b, nvs[b] - k:] == -1)


def test_merge_entry_point_with_given_indices(ctx):
    batch = W.tiny(B=2, n_vis=[210, 150], text_lens=[6, 11], H=2, keep_k=25, seed=303, centres=7)
    p = A.Params(keep_k=25)
    inp = A.make_inputs(batch, DEV)
    mv = inp.max_vis
    sal = torch.zeros(2, mv); keep = torch.zeros(2, 25, dtype=torch.int32)
    drop = torch.full((2, mv - 25), -1, dtype=torch.int32)
    refs = []
    for b in range(2):
        ref = _oracle_scores(batch, b, p)
        nv = int(batch.vis_len[b])
        sal[b, :nv] = torch.from_numpy(ref["salience"]).float()
        keep[b] = torch.from_numpy(ref["keep_idx"]); drop[b, :nv - 25] = torch.from_numpy(ref["drop_idx"])
        refs.append(ref)
    out = A.alloc_outputs(inp, 25, fill=True)
    A.asap_merge(ctx, inp, p, sal.to(DEV), keep.to(DEV), drop.to(DEV), out)
    torch.cuda.synchronize(); A.asap_check(ctx)
    ocu = out.out_cu_seqlens.cpu().numpy()
    for b in range(2):
        ref = refs[b]
        nv, v0 = int(batch.vis_len[b]), int(batch.vis_start[b])
        nd = nv - 25
        ag = out.assign[b, :nd].cpu().numpy()
        mism = np.nonzero(ag != ref["assign"])[0]
        assert np.all(ref["margin"][mism] <= 1e-4)
        rows = batch.sample_rows(b)
        ref2 = O.prune_sample(bits(batch.q[rows]), bits(batch.k[rows]), bits(batch.hidden[rows]),
                              batch.pos_ids[rows].numpy(), v0, nv, int(batch.text_start[b]),
                              int(batch.text_len[b]), 25, assign_override=ag)
        gh = O.bf16_bits_to_f64(bits(out.out_hidden[int(ocu[b]):int(ocu[b + 1])].cpu()))
        err = np.abs(gh - ref2["out_hidden"])
        assert np.all(err <= merged_tolerance(ref2["out_hidden"]))
        assert np.array_equal(out.out_pos[int(ocu[b]):int(ocu[b + 1])].cpu().numpy(), ref2["out_pos"])


def test_host_side_argument_errors_launch_nothing(ctx):
    batch = W.tiny(B=2, n_vis=[40, 40], text_lens=[4, 4], H=1, keep_k=8, seed=304)
    inp = A.make_inputs(batch, DEV)
    out = A.alloc_outputs(inp, 8, fill=True)
    n0 = A.asap_launch_count(ctx)

    def expect(status, **changes):
        import dataclasses
        bad_inp = dataclasses.replace(inp, **{k: v for k, v in changes.items() if hasattr(inp, k)})
        pk = {k: v for k, v in changes.items() if not hasattr(inp, k)}
        p = A.Params(**{"keep_k": 8, **pk})
        with pytest.raises(A.AsapError) as e:
            A.asap_prune_step(ctx, bad_inp, p, out)
        assert e.value.status == status, (changes, e.value)
        assert A.asap_last_error(ctx) != ""

    expect(-5, head_dim=64)
    expect(-1, D=inp.D + 8)
    expect(-1, keep_k=0)
    expect(-1, keep_k=41)
    expect(-1, lambda_max=0.0)
    expect(-1, lambda_max=1.5)
    expect(-1, eps=0.0)
    expect(-1, q=None)
    expect(-1, cu_seqlens=None)
    expect(-1, rank_start=inp.vis_start)                     # rank_len missing
    expect(-3, B=65)
    expect(-3, total_tokens=50000)
    expect(-2, q=inp.q.view(-1)[1:-7].view(-1))              # 2 bytes off a 16-byte boundary
    assert A.asap_launch_count(ctx) == n0
    torch.cuda.synchronize()
    assert int(out.keep_idx.min()) == -7                     # outputs untouched


def test_device_side_bad_sample_is_skipped_and_reported(ctx):
    batch = W.tiny(B=3, n_vis=[60, 60, 60], text_lens=[5, 5, 5], H=1, keep_k=12, seed=305)
    bad = batch.vis_len.clone(); bad[1] = 5000                # span leaves its sequence
    inp = A.make_inputs(batch, DEV)
    inp.vis_len = bad.to(DEV)
    inp.max_vis = 60
    out = A.alloc_outputs(inp, 12, fill=True)
    p = A.Params(keep_k=12)
    A.asap_prune_step(ctx, inp, p, out)
    torch.cuda.synchronize()
    with pytest.raises(A.AsapError) as e:
        A.asap_check(ctx)
    assert e.value.status == -6 and "span" in str(e.value)
    A.asap_check(ctx)                                         # the word was cleared
    assert torch.all(out.keep_idx[1] == -1) and torch.all(out.rank_score[1] == 0)
    ocu = out.out_cu_seqlens.cpu()
    assert int(ocu[2] - ocu[1]) == 0
    # the good samples are still right; sample 2's rows start where sample 0's end
    compare_sample(batch, 0, p, out)
    compare_sample_shifted = int(ocu[3] - ocu[2])
    assert compare_sample_shifted == 3 + 12 + 5


def test_output_capacity_overflow_is_reported(ctx):
    batch = W.tiny(B=2, n_vis=[50, 50], text_lens=[5, 5], H=1, keep_k=10, seed=306)
    inp = A.make_inputs(batch, DEV)
    out = A.alloc_outputs(inp, 10, fill=True)
    out.out_hidden = out.out_hidden[:20]                      # too few rows
    A.asap_prune_step(ctx, inp, A.Params(keep_k=10), out)
    torch.cuda.synchronize()
    with pytest.raises(A.AsapError) as e:
        A.asap_check(ctx)
    assert e.value.status == -6 and "capacity" in str(e.value)
    assert float(out.out_hidden.float().abs().sum()) == 0.0   # nothing was written


def test_repeated_calls_are_deterministic(ctx):
    batch = W.tiny(B=2, n_vis=[300, 170], text_lens=[33, 8], H=2, keep_k=40, seed=307, centres=5)
    inp = A.make_inputs(batch, DEV)
    p = A.Params(keep_k=40)
    outs = []
    for _ in range(3):
        out = A.alloc_outputs(inp, 40, fill=True)
        A.asap_prune_step(ctx, inp, p, out)
        torch.cuda.synchronize()
        outs.append(out)
    for o in outs[1:]:
        for name in ("mass", "salience", "rank_score", "keep_idx", "assign", "out_pos"):
            assert torch.equal(getattr(o, name), getattr(outs[0], name)), name
        assert torch.equal(o.out_hidden.view(torch.int16), outs[0].out_hidden.view(torch.int16))


def test_kv_cache_compaction_follows_the_row_map(ctx):
    """asap_compact_kv gathers cached K / V rows with the step's own row map: bit-exact against the
    oracle's row gather, rows past the shortened batch untouched, several tensors per call."""
    batch = W.tiny(B=3, n_vis=[90, 140, 64], text_lens=[5, 9, 2], H=2, keep_k=20, seed=308)
    inp = A.make_inputs(batch, DEV)
    p = A.Params(keep_k=20)
    out = A.alloc_outputs(inp, 20, fill=True)
    A.asap_prune_step(ctx, inp, p, out)
    g = torch.Generator().manual_seed(9)
    kv_dim = 2 * 128
    caches = [torch.randint(-30000, 30000, (batch.total, kv_dim), generator=g, dtype=torch.int16).view(torch.bfloat16)
              for _ in range(6)]                                   # K and V of three layers
    src = [c.to(DEV) for c in caches]
    rows_cap = out.out_hidden.shape[0]
    dst = [torch.full((rows_cap, kv_dim), 7.0, dtype=torch.bfloat16, device=DEV) for _ in range(6)]
    A.asap_compact_kv(ctx, out.src_row, out.out_cu_seqlens[batch.B:], src, dst)
    torch.cuda.synchronize(); A.asap_check(ctx)
    n_out = int(out.out_cu_seqlens[-1])
    rowmap = out.src_row[:n_out].cpu().numpy()
    for c, d in zip(caches, dst):
        want = O.compact_rows(bits(c), rowmap)
        assert np.array_equal(bits(d[:n_out].cpu()), want)
        assert torch.all(d[n_out:] == 7.0)                          # capacity tail untouched
    with pytest.raises(A.AsapError):                                # 65 tensors: refused before any launch
        A.asap_compact_kv(ctx, out.src_row, out.out_cu_seqlens[batch.B:], src * 11, dst * 11)


def test_prune_step_can_be_captured_into_a_cuda_graph(ctx):
    """The step allocates nothing, never synchronises, and its side stream forks from and joins back
    into the caller's stream inside the call, so a stream capture records it whole; a replay on new
    input contents (same buffers) gives what a direct call gives, bit for bit."""
    batch = W.tiny(B=3, n_vis=[300, 170, 520], text_lens=[9, 30, 4], H=2, keep_k=48, seed=306, centres=8)
    other = W.tiny(B=3, n_vis=[300, 170, 520], text_lens=[9, 30, 4], H=2, keep_k=48, seed=307, centres=8)
    inp = A.make_inputs(batch, DEV)
    p = A.Params(keep_k=48)
    out = A.alloc_outputs(inp, 48, fill=True)
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        A.asap_prune_step(ctx, inp, p, out, s)
        s.synchronize()
        g.capture_begin()
        A.asap_prune_step(ctx, inp, p, out, s)
        g.capture_end()
    for src in (other, batch):
        for name in ("q", "k", "hidden"):                       # new contents, same device buffers
            getattr(inp, name).copy_(getattr(src, name).to(DEV))
        ref = A.alloc_outputs(inp, 48, fill=True)
        A.asap_prune_step(ctx, inp, p, ref)
        torch.cuda.synchronize()
        for t in (out.out_hidden, out.keep_idx, out.rank_score, out.out_pos):
            t.zero_()
        g.replay()
        torch.cuda.synchronize(); A.asap_check(ctx)
        n_out = int(ref.out_cu_seqlens[-1])                  # rows past it are untouched capacity
        for name in ("keep_idx", "drop_idx", "assign", "rank_score", "salience", "out_cu_seqlens"):
            assert torch.equal(getattr(out, name), getattr(ref, name)), name
        for name in ("out_hidden", "out_pos", "src_row"):
            assert torch.equal(getattr(out, name)[:n_out], getattr(ref, name)[:n_out]), name


def test_per_head_mask_needs_an_even_number_of_heads(ctx):
    batch = W.tiny(B=1, n_vis=[100], text_lens=[4], H=3, keep_k=8, seed=308)
    inp = A.make_inputs(batch, DEV)
    out = A.alloc_outputs(inp, 8, per_head=True)
    n0 = A.asap_launch_count(ctx)
    with pytest.raises(A.AsapError) as e:
        A.asap_prune_step(ctx, inp, A.Params(keep_k=8, per_head_mask=True), out)
    assert e.value.status == -5 and A.asap_launch_count(ctx) == n0
