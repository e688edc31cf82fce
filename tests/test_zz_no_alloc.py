"""asap_select_static: the top-k selection for callers that may not allocate device memory
(code running inside someone else's memory budget or real-time loop, with no chance to call
asap_init, whose scratch comes from cudaMalloc).  Its scratch is a fixed array inside the
library, so the test checks the one thing that matters to such a caller: called through the C
ABI, twice in a row on the shared array, it returns exactly what asap_select returns.

Collected last on purpose (file name), so a run that stops at the first failure has already
been through every other test.  It passes alone in a fresh process as well: it needs no state
from the other tests."""
import pytest
import torch

from paper_2603_14549_b200 import binding as A
from paper_2603_14549_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _scores(B, nvs, mv, seed, ties):
    g = torch.Generator().manual_seed(seed)
    s = torch.zeros(B, mv)
    for b in range(B):
        r = torch.randn(nvs[b], generator=g)
        s[b, :nvs[b]] = torch.round(r * 3) / 3 if ties else r     # ties exercise the lower-index rule
    if ties:                      # -0.0 and +0.0 are one score: among them the lower index wins too
        s[1, 0:40:2] = -0.0
        s[1, 1:40:2] = 0.0
    return s.to(DEV)


def test_static_select_matches_select_on_two_calls_in_a_row():
    torch.cuda.set_device(0)
    nvs = [700, 333, 512, 64]
    B, mv = len(nvs), max(nvs)
    batch = W.tiny(B=B, n_vis=nvs, text_lens=[3, 9, 1, 20], H=1, keep_k=64, seed=401)
    inp = A.make_inputs(batch, DEV)
    ctx = A.asap_init(0, max_total_tokens=batch.total + B * mv, max_B=B, max_H=1, max_D=128)
    try:
        # two different problems back to back: the second call finds the first one's leftovers
        for call, (k, ties) in enumerate([(64, True), (17, False)]):
            p = A.Params(keep_k=k)
            scores = _scores(B, nvs, mv, 50 + call, ties)
            want = A.alloc_outputs(inp, k, fill=True)
            A.asap_select(ctx, inp, p, scores, want)
            keep = torch.full((B, k), -7, dtype=torch.int32, device=DEV)
            drop = torch.full((B, mv - k), -7, dtype=torch.int32, device=DEV)
            status = torch.full((1,), 99, dtype=torch.int32, device=DEV)
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info(0)[0]
            A.asap_select_static(inp, p, scores, keep, drop, status)
            torch.cuda.synchronize()
            if call > 0:       # (the first call on a device may load the library's device code)
                assert torch.cuda.mem_get_info(0)[0] == free_before, "the call changed the device's free memory"
            A.asap_check(ctx)
            assert int(status.item()) == 0
            assert torch.equal(keep, want.keep_idx), f"call {call}: keep_idx differs"      # indices: bit-exact
            assert torch.equal(drop, want.drop_idx), f"call {call}: drop_idx differs"
    finally:
        A.asap_free(ctx)


def test_static_select_rejects_sizes_beyond_its_array():
    torch.cuda.set_device(0)
    batch = W.tiny(B=2, n_vis=[40, 40], text_lens=[2, 2], H=1, keep_k=8, seed=402)
    inp = A.make_inputs(batch, DEV)
    keep = torch.full((2, 8), -7, dtype=torch.int32, device=DEV)
    drop = torch.full((2, 32), -7, dtype=torch.int32, device=DEV)
    scores = torch.zeros(2, 40, device=DEV)
    import dataclasses
    for bad in (dataclasses.replace(inp, B=65), dataclasses.replace(inp, B=64, max_vis=4097, max_seq=5000)):
        with pytest.raises(A.AsapError) as e:
            A.asap_select_static(bad, A.Params(keep_k=8), scores, keep, drop)
        assert e.value.status == -3 and "exceed the fixed scratch" in str(e.value)
    torch.cuda.synchronize()
    assert int(keep.min()) == -7 and int(drop.min()) == -7          # nothing ran


def test_static_select_flags_a_bad_sequence_in_the_callers_status_word():
    torch.cuda.set_device(0)
    batch = W.tiny(B=2, n_vis=[50, 50], text_lens=[2, 2], H=1, keep_k=5, seed=403)
    inp = A.make_inputs(batch, DEV)
    bad = batch.vis_len.clone(); bad[0] = 9999
    inp.vis_len = bad.to(DEV)
    keep = torch.full((2, 5), -7, dtype=torch.int32, device=DEV)
    drop = torch.full((2, 45), -7, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    A.asap_select_static(inp, A.Params(keep_k=5), torch.randn(2, 50, device=DEV), keep, drop, status)
    torch.cuda.synchronize()
    assert int(status.item()) & 1
    assert torch.all(keep[0] == -1) and torch.all(keep[1] >= 0)
