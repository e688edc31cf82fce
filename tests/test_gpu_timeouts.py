"""The give-up path of the bounded waits in the three tensor-core kernels, exercised in the harmless
form: the wait limit of ONE call is set to a single clock cycle, so a healthy run gives up at its
first wait that is not satisfied at once.  The call must return, asap_check must name the kernel's
time-out bit, and the next ordinary call on the same context must give the results of a fresh one
bit for bit.  Nothing is made to hang and nothing is expected to fault: the blocks leave through
the same teardown as always, after draining the copies and MMAs they have in flight."""
import pytest
import torch

from paper_2603_14549_b200 import binding as A
from paper_2603_14549_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    c = A.asap_init(0, max_total_tokens=20000, max_B=8, max_H=4, max_D=512, max_keep_rows=8000)
    yield c
    A.asap_free(c)


def _same(a, b, names):
    for n in names:
        x, y = getattr(a, n), getattr(b, n)
        assert torch.equal(x, y), n


def test_score_kernel_gives_up_and_the_context_recovers(ctx):
    batch = W.tiny(B=3, n_vis=[300, 260, 140], text_lens=[20, 150, 7], H=2, keep_k=40, seed=601, centres=6)
    inp = A.make_inputs(batch, DEV)
    p = A.Params(keep_k=40)
    good = A.alloc_outputs(inp, 40, fill=True)
    A.asap_prune_step(ctx, inp, p, good)
    torch.cuda.synchronize(); A.asap_check(ctx)

    bad = A.alloc_outputs(inp, 40, fill=True)
    A.asap_debug_wait_limit(ctx, 1)
    A.asap_prune_step(ctx, inp, p, bad)              # returns normally; its results are void
    torch.cuda.synchronize()
    with pytest.raises(A.AsapError) as e:
        A.asap_check(ctx)
    assert e.value.status == -6 and "timed out in the score kernel" in str(e.value)

    again = A.alloc_outputs(inp, 40, fill=True)       # the limit held for one call only
    A.asap_prune_step(ctx, inp, p, again)
    torch.cuda.synchronize(); A.asap_check(ctx)
    _same(good, again, ("rank_score", "keep_idx", "drop_idx", "assign", "out_hidden", "out_pos", "src_row", "out_cu_seqlens"))


def test_similarity_kernel_gives_up_and_the_context_recovers(ctx):
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
    _same(ref, again, ("assign", "best_sim", "out_hidden", "out_pos", "src_row", "out_cu_seqlens"))


def test_attention_kernel_gives_up_and_the_context_recovers(ctx):
    batch = W.tiny(B=2, n_vis=[300, 200], text_lens=[30, 11], H=2, keep_k=40, seed=603, centres=6)
    inp = A.make_inputs(batch, DEV)
    p = A.Params(keep_k=40)
    out = A.alloc_outputs(inp, 40, fill=True)
    A.asap_score(ctx, inp, p, out)
    v = W.draw_values(batch, 77).to(DEV)
    scratch = torch.empty(A.asap_attention_scratch_bytes(batch.total, batch.D), dtype=torch.uint8, device=DEV)
    good = torch.zeros_like(v)
    A.asap_attention(ctx, inp, p, out.mask_log, v, scratch, good)
    torch.cuda.synchronize(); A.asap_check(ctx)

    bad = torch.zeros_like(v)
    A.asap_debug_wait_limit(ctx, 1)
    A.asap_attention(ctx, inp, p, out.mask_log, v, scratch, bad)
    torch.cuda.synchronize()
    with pytest.raises(A.AsapError) as e:
        A.asap_check(ctx)
    assert e.value.status == -6 and "timed out in the attention kernel" in str(e.value)

    again = torch.zeros_like(v)
    A.asap_attention(ctx, inp, p, out.mask_log, v, scratch, again)
    torch.cuda.synchronize(); A.asap_check(ctx)
    assert torch.equal(good, again)
