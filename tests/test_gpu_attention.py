"""asap_attention (Eq. 4 applied to the values: the layer's attention under the SG-BiMask) against
the CPU oracle, through the C ABI, every output element.

The mask vector m_j given to both sides is the oracle's (Eq. 1-3), rounded to fp32.
Tolerance: |g - o| <= max(2e-2, 2^-7 |o|) -- the bar of the merged rows: probabilities enter the
second contraction as bf16 (relative error 2^-9 each, averaged over a row), the output is rounded to
bf16 once (2^-9 relative)."""
import numpy as np
import pytest
import torch

from oracle import asap_oracle as O
from paper_2603_14549_b200 import binding as A
from paper_2603_14549_b200 import workloads as W
from tests.helpers import bits

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    c = A.asap_init(0, max_total_tokens=40000, max_B=16, max_H=8, max_D=1024)
    yield c
    A.asap_free(c)


def _mask_vectors(batch, lambda_max):
    mv = int(batch.vis_len.max())
    m = torch.zeros(batch.B, mv)
    ms = []
    for b in range(batch.B):
        rows = batch.sample_rows(b)
        q, k = O.bf16_bits_to_f64(bits(batch.q[rows])), O.bf16_bits_to_f64(bits(batch.k[rows]))
        v0, nv = int(batch.vis_start[b]), int(batch.vis_len[b])
        mb = O.mask_log(O.salience(O.attention_mass(q, k, v0, nv)), lambda_max).astype(np.float32)
        m[b, :nv] = torch.from_numpy(mb)
        ms.append(mb.astype(np.float64))
    return m, ms


def _run(ctx, batch, v, m, mask_enable=True):
    inp = A.make_inputs(batch, DEV)
    out = torch.full((batch.total, batch.H, batch.head_dim), 7.0, dtype=torch.bfloat16, device=DEV)
    scratch = torch.empty(A.asap_attention_scratch_bytes(batch.total, batch.D), dtype=torch.uint8, device=DEV)
    p = A.Params(keep_k=int(batch.vis_len.min()), mask_enable=mask_enable)
    A.asap_attention(ctx, inp, p, None if m is None else m.to(DEV), v.to(DEV), scratch, out)
    torch.cuda.synchronize(); A.asap_check(ctx)
    return out.cpu()


def _compare(batch, v, out, ms, mask_enable=True):
    worst = 0.0
    for b in range(batch.B):
        rows = batch.sample_rows(b)
        ref = O.masked_attention(bits(batch.q[rows]), bits(batch.k[rows]), bits(v[rows]), int(batch.vis_start[b]),
                                 int(batch.vis_len[b]), ms[b] if mask_enable else None, mask_enable)
        g = O.bf16_bits_to_f64(bits(out[rows]))
        err = np.abs(g - ref)
        assert np.all(err <= np.maximum(2e-2, np.abs(ref) * 2.0 ** -7)), (b, err.max(), np.unravel_index(err.argmax(), err.shape))
        worst = max(worst, err.max())
    return worst


@pytest.mark.parametrize("nvs,texts,lam", [
    ([300, 170, 520], [9, 30, 4], 1.0),          # ragged; sequence starts off the 8-row grid
    ([130, 257], [1, 140], 0.3),                 # text longer than a tile; image span ends one past a tile edge
    ([64], [3], 1.0),                            # a single, partly filled tile
], ids=["ragged3", "longtext", "single"])
def test_attention_matches_oracle(ctx, nvs, texts, lam):
    batch = W.tiny(B=len(nvs), n_vis=nvs, text_lens=texts, H=2, keep_k=8, seed=600 + len(nvs))
    v = W.draw_values(batch, 77)
    m, ms = _mask_vectors(batch, lam)
    out = _run(ctx, batch, v, m)
    print("attention max abs err", _compare(batch, v, out, ms))


def test_mask_off_is_causal_attention_and_only_visual_rows_differ(ctx):
    batch = W.tiny(B=2, n_vis=[200, 333], text_lens=[17, 5], H=2, keep_k=8, seed=610)
    v = W.draw_values(batch, 78)
    m, ms = _mask_vectors(batch, 1.0)
    off = _run(ctx, batch, v, None, mask_enable=False)
    _compare(batch, v, off, ms, mask_enable=False)
    on = _run(ctx, batch, v, m)
    for b in range(2):
        rows = batch.sample_rows(b)
        v0, nv = int(batch.vis_start[b]), int(batch.vis_len[b])
        a, c = bits(on[rows]), bits(off[rows])
        vis = np.zeros(rows.stop - rows.start, bool); vis[v0:v0 + nv - 1] = True
        assert np.array_equal(a[~vis], c[~vis])             # system, text and the last visual row: bit-identical
        assert np.any(a[vis] != c[vis])


def test_attention_argument_errors(ctx):
    batch = W.tiny(B=1, n_vis=[100], text_lens=[4], H=2, keep_k=8, seed=611)
    inp = A.make_inputs(batch, DEV)
    v = W.draw_values(batch, 79).to(DEV)
    out = torch.empty_like(v)
    big = torch.empty(A.asap_attention_scratch_bytes(batch.total, batch.D), dtype=torch.uint8, device=DEV)
    n0 = A.asap_launch_count(ctx)
    with pytest.raises(A.AsapError) as e:
        A.asap_attention(ctx, inp, A.Params(keep_k=8), None, v, big, out)          # mask on, no vector
    assert e.value.status == -1
    with pytest.raises(A.AsapError) as e:
        A.asap_attention(ctx, inp, A.Params(keep_k=8, mask_enable=False), None, v, big[:64], out)
    assert e.value.status == -3
    assert A.asap_launch_count(ctx) == n0
    assert A.asap_attention_scratch_bytes(13, 256) == 16 * 256 * 2


@pytest.fixture(scope="module")
def big_ctx():
    c = A.asap_init(0, max_total_tokens=64 * (35 + 2880 + 256), max_B=64, max_H=40, max_D=5120)
    yield c
    A.asap_free(c)


@pytest.mark.parametrize("name,B,samples", [("c2", None, [0, 15]), ("c4", 4, [3]), ("c5", 2, [1])])
def test_attention_at_benchmark_sizes_sampled_rows(big_ctx, name, B, samples):
    """Benchmark shapes at full width (32 / 40 heads); the oracle checks 48 sampled query rows of the
    listed sequences (system, image-span and text rows, the span's first and last rows among them)."""
    batch = W.config(name, B=B)
    v = W.draw_values(batch, 80)
    mv = int(batch.vis_len.max())
    m = torch.zeros(batch.B, mv)
    ms = {}
    for b in range(batch.B):
        rows = batch.sample_rows(b)
        nv = int(batch.vis_len[b])
        if b in samples:
            q, k = O.bf16_bits_to_f64(bits(batch.q[rows])), O.bf16_bits_to_f64(bits(batch.k[rows]))
            mb = O.mask_log(O.salience(O.attention_mass(q, k, int(batch.vis_start[b]), nv)), 1.0).astype(np.float32)
        else:                                                         # unchecked sequences: any valid vector
            mb = np.log(np.linspace(0.01, 1.0, nv)).astype(np.float32)
        m[b, :nv] = torch.from_numpy(mb)
        ms[b] = mb.astype(np.float64)
    out = _run(big_ctx, batch, v, m)
    rng = np.random.default_rng(81)
    for b in samples:
        rows = batch.sample_rows(b)
        n, v0, nv = rows.stop - rows.start, int(batch.vis_start[b]), int(batch.vis_len[b])
        pick = np.unique(np.concatenate([[0, v0 - 1, v0, v0 + nv - 1, v0 + nv, n - 1], rng.integers(0, n, 42)]))
        ref = O.masked_attention(bits(batch.q[rows]), bits(batch.k[rows]), bits(v[rows]), v0, nv, ms[b], True, rows=pick)
        g = O.bf16_bits_to_f64(bits(out[rows][pick]))
        err = np.abs(g - ref)
        assert np.all(err <= np.maximum(2e-2, np.abs(ref) * 2.0 ** -7)), (b, err.max())


def test_attention_with_a_mask_per_head(ctx):
    """per_head_mask: head h adds its own Eq. 3 vector (asap_outputs::mask_log_heads layout [B, H, max_vis])."""
    batch = W.tiny(B=2, n_vis=[200, 333], text_lens=[17, 5], H=2, keep_k=8, seed=612)
    v = W.draw_values(batch, 83)
    mv = int(batch.vis_len.max())
    m = torch.zeros(batch.B, batch.H, mv)
    ms = []
    for b in range(batch.B):
        rows = batch.sample_rows(b)
        q, k = O.bf16_bits_to_f64(bits(batch.q[rows])), O.bf16_bits_to_f64(bits(batch.k[rows]))
        v0, nv = int(batch.vis_start[b]), int(batch.vis_len[b])
        mh = np.stack([O.mask_log(O.salience(sh), 0.8) for sh in O.attention_mass_heads(q, k, v0, nv)]).astype(np.float32)
        m[b, :, :nv] = torch.from_numpy(mh)
        ms.append(mh.astype(np.float64))
    inp = A.make_inputs(batch, DEV)
    out = torch.full((batch.total, batch.H, batch.head_dim), 7.0, dtype=torch.bfloat16, device=DEV)
    scratch = torch.empty(A.asap_attention_scratch_bytes(batch.total, batch.D), dtype=torch.uint8, device=DEV)
    A.asap_attention(ctx, inp, A.Params(keep_k=8, per_head_mask=True), m.to(DEV), v.to(DEV), scratch, out)
    torch.cuda.synchronize(); A.asap_check(ctx)
    _compare(batch, v, out.cpu(), ms)
    assert float((m[0, 0] - m[0, 1]).abs().max()) > 1e-3


def test_attention_skips_a_bad_sequence(ctx):
    batch = W.tiny(B=2, n_vis=[200, 150], text_lens=[4, 4], H=2, keep_k=8, seed=613)
    v = W.draw_values(batch, 84)
    good = _run(ctx, batch, v, None, mask_enable=False)
    inp = A.make_inputs(batch, DEV)
    bad = batch.vis_len.clone(); bad[0] = 9999
    inp.vis_len = bad.to(DEV)
    out = torch.full((batch.total, batch.H, batch.head_dim), 7.0, dtype=torch.bfloat16, device=DEV)
    scratch = torch.empty(A.asap_attention_scratch_bytes(batch.total, batch.D), dtype=torch.uint8, device=DEV)
    A.asap_attention(ctx, inp, A.Params(keep_k=8, mask_enable=False), None, v.to(DEV), scratch, out)
    torch.cuda.synchronize()
    with pytest.raises(A.AsapError) as e:
        A.asap_check(ctx)
    assert e.value.status == -6
    r0, r1 = batch.sample_rows(0), batch.sample_rows(1)
    assert torch.all(out[r0].float() == 7.0)                    # skipped: untouched
    assert torch.equal(out[r1].cpu(), good[r1])


def test_attention_and_consolidation_can_be_captured_into_a_cuda_graph(ctx):
    """Both calls allocate nothing and do not synchronise: a stream capture records them, and a replay
    reproduces the directly launched results bit for bit."""
    batch = W.tiny(B=2, n_vis=[200, 150], text_lens=[4, 9], H=2, keep_k=40, seed=614, centres=5)
    inp = A.make_inputs(batch, DEV)
    p = A.Params(keep_k=40, sim_threshold=0.8)
    step_out = A.alloc_outputs(inp, 40, fill=True)
    A.asap_prune_step(ctx, inp, p, step_out)                           # stage-1 results to feed both calls
    torch.cuda.synchronize()
    v = W.draw_values(batch, 85).to(DEV)
    st1 = [t.clone() for t in (step_out.mass, step_out.salience, step_out.keep_idx, step_out.drop_idx, step_out.mask_log)]
    a_scr = torch.empty(A.asap_attention_scratch_bytes(batch.total, batch.D), dtype=torch.uint8, device=DEV)
    c_scr = torch.empty(A.asap_consolidate_scratch_bytes(batch.B, 40), dtype=torch.uint8, device=DEV)

    def run(att_out, cons_out, n_abs, stream=None):
        A.asap_attention(ctx, inp, p, st1[4], v, a_scr, att_out, stream)
        A.asap_consolidate(ctx, inp, p, st1[0], st1[1], st1[2], st1[3], c_scr, cons_out, n_abs, stream)

    ref_att = torch.zeros_like(v); ref_cons = A.alloc_outputs(inp, 40, fill=True)
    ref_abs = torch.zeros(batch.B, dtype=torch.int32, device=DEV)
    run(ref_att, ref_cons, ref_abs)
    torch.cuda.synchronize(); A.asap_check(ctx)
    att = torch.zeros_like(v); cons = A.alloc_outputs(inp, 40, fill=True)
    n_abs = torch.zeros(batch.B, dtype=torch.int32, device=DEV)
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        run(att, cons, n_abs, s)
        s.synchronize()
        g.capture_begin()
        run(att, cons, n_abs, s)
        g.capture_end()
    att.zero_(); cons.out_hidden.zero_(); cons.keep_idx.zero_(); n_abs.zero_()
    g.replay()
    torch.cuda.synchronize(); A.asap_check(ctx)
    n_out = int(ref_cons.out_cu_seqlens[-1])
    assert torch.equal(att, ref_att) and torch.equal(n_abs, ref_abs) and int(ref_abs.sum()) > 0
    assert torch.equal(cons.keep_idx, ref_cons.keep_idx) and torch.equal(cons.assign, ref_cons.assign)
    assert torch.equal(cons.out_hidden[:n_out], ref_cons.out_hidden[:n_out])
