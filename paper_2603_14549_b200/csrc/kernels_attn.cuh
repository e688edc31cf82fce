// The layer's attention under the salience-guided bidirectional mask (Eq. 4 applied to the
// values):  O^h = Softmax(W^h + M_bidir) V^h,  W^h = Q^h K^h^T / sqrt(d).
//
//   transpose_v_kernel  V [tokens, D] -> V^T [D, tokens] (row pitch padded to 8 tokens), so that
//                       a value tile can be loaded as a K-major MMA operand like every other tile.
//   attn_kernel         one block per (two tiles of 128 query rows, head, sequence); the two row
//                       tiles share every key / value tile and take turns on the tensor pipe.
//                       For every tile of 128 keys:  S = Q K^T on tcgen05 into tensor memory; the
//                       row tile's eight softmax warps read S once (two threads per row, 64 keys
//                       each, exchanging their maxima through shared memory), add Eq. 3's
//                       m_j for the future keys of the image span on rows of the image span (nothing
//                       else above the diagonal is admitted), turn the logits into probabilities
//                       relative to a reference maximum and store them as bf16 over S's own columns;
//                       O += P V then runs with P read from tensor memory and O accumulated in
//                       tensor memory.  The reference maximum only moves (and O is only rescaled)
//                       when a row's maximum has grown by more than 2^8; the final division by the
//                       row sum makes the result independent of the reference.  M_bidir is never
//                       materialised: it is the vector m_j plus position tests.
//
// Key tiles start at the sequence's first packed row rounded DOWN to a multiple of 8, because the
// token coordinate is the contiguous one of V^T and a TMA copy must start on a 16-byte boundary;
// the up to seven foreign keys in front are masked like any other inadmissible key.
#pragma once

#include "common.cuh"

namespace asap {

enum : uint32_t { STATUS_ATTN_TIMEOUT = 16u };   // a bounded wait ran out in the attention kernel

// ---------------------------------------------------------------------------------------
constexpr int TR_TILE = 64;
constexpr int TR_THREADS = 256;

__global__ void __launch_bounds__(TR_THREADS)
transpose_v_kernel(const __nv_bfloat16 *__restrict__ v, __nv_bfloat16 *__restrict__ vt, int total,
                   int total_pad, int D) {
  pdl_enter();
  __shared__ uint16_t tile[TR_TILE][TR_TILE + 2];
  const int t0 = blockIdx.x * TR_TILE, d0 = blockIdx.y * TR_TILE;
  const uint16_t *src = reinterpret_cast<const uint16_t *>(v);
  uint16_t *dst = reinterpret_cast<uint16_t *>(vt);
  for (int i = threadIdx.x; i < TR_TILE * (TR_TILE / 8); i += TR_THREADS) {
    const int r = i / (TR_TILE / 8), c8 = i % (TR_TILE / 8);
    uint4 x = make_uint4(0u, 0u, 0u, 0u);
    if (t0 + r < total && d0 + c8 * 8 < D)
      x = __ldg(reinterpret_cast<const uint4 *>(src + (size_t)(t0 + r) * D + d0 + c8 * 8));
    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      tile[c8 * 8 + 2 * e][r] = (uint16_t)(w[e] & 0xffffu);
      tile[c8 * 8 + 2 * e + 1][r] = (uint16_t)(w[e] >> 16);
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < TR_TILE * (TR_TILE / 8); i += TR_THREADS) {
    const int dd = i / (TR_TILE / 8), c8 = i % (TR_TILE / 8);
    if (d0 + dd >= D || t0 + c8 * 8 >= total_pad) continue;
    uint32_t w[4];
#pragma unroll
    for (int e = 0; e < 4; ++e)
      w[e] = (uint32_t)tile[dd][c8 * 8 + 2 * e] | ((uint32_t)tile[dd][c8 * 8 + 2 * e + 1] << 16);
    *reinterpret_cast<uint4 *>(dst + (size_t)(d0 + dd) * total_pad + t0 + c8 * 8) = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

// ---------------------------------------------------------------------------------------
constexpr int AT_THREADS = 576;                 // warp 0: copies, warp 1: MMA issue, warps 2-17: two softmax groups of eight
constexpr int AT_TILE_BYTES = 128 * 128 * 2;    // 128 rows x 128 bf16 as two 64-column blocks of 16 KB
constexpr int AT_BLOCK_BYTES = AT_TILE_BYTES / 2;
constexpr int AT_STAGES = 2;                    // a stage = one key tile + one value tile
constexpr int AT_MAIN_BYTES = 2 * AT_TILE_BYTES + AT_STAGES * 2 * AT_TILE_BYTES;
constexpr int AT_BOOK_BYTES = 3072;
constexpr int AT_SMEM_BYTES = AT_MAIN_BYTES + AT_BOOK_BYTES;
constexpr uint32_t AT_TMEM_COLS = 512;          // per row tile: S / P (128 columns) and O (128 columns)
constexpr long long AT_WAIT_LIMIT = 2000000000LL;
constexpr float AT_RESCALE_STEP = 8.0f;         // log2 units the row maximum may outgrow the reference
static_assert(AT_SMEM_BYTES <= 195 * 1024, "the attention block must stay inside the 196 KB carve-out");

struct AttnArgs {
  const SampleDesc *desc;
  int H, D, max_vis, mask_enable;
  float scale_log2;            // log2(e) / sqrt(head_dim)
  const float *mask_log;       // [B, max_vis] m_j (natural log) or [B, H, max_vis]; may be null with the mask off
  int mask_b_stride, mask_h_stride;   // max_vis, 0   or   H * max_vis, max_vis
  __nv_bfloat16 *out;          // [tokens, H, 128]
  uint32_t *status;
  long long wait_limit;        // clock cycles a wait may take before the block gives up
};

struct AttnBook {
  uint64_t full[AT_STAGES], empty[AT_STAGES], q_full, s_full[2], p_ready[2], pv_done[2], mma_done;
  uint32_t tmem_base;
  int abort_flag;
  alignas(16) float m_tile[2][128];   // [row tile][key]: Eq. 3's addend for the keys of the current tile
  uint32_t row_max[2][128];    // [row tile][row]: running row maximum as an order-preserving integer
};
static_assert(sizeof(AttnBook) <= AT_BOOK_BYTES, "attention kernel bookkeeping exceeds its shared-memory slot");

// order-preserving integer image of a float (no NaN here) and its inverse, for atomicMax
__device__ __forceinline__ uint32_t attn_key(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float attn_unkey(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// keys a tile of query rows [q_lo, q_lo + 128) can see: up to its last row (causal), and to the end
// of the image span if one of its rows lies inside the span and the mask is on
__device__ __forceinline__ int attn_key_end(const SampleDesc &d, int q_lo, int mask_enable, bool &sees_span) {
  const int q_hi = min(q_lo + 128, d.n);
  sees_span = mask_enable && q_lo < d.v0 + d.nv && q_hi > d.v0;
  return min(d.n, sees_span ? max(q_hi, d.v0 + d.nv) : q_hi);
}

__global__ void __launch_bounds__(AT_THREADS, 1)
attn_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
            const __grid_constant__ CUtensorMap tmap_vt, AttnArgs a) {
  pdl_enter();
  extern __shared__ __align__(1024) uint8_t at_smem[];
  const int pair = (int)gridDim.x - 1 - (int)blockIdx.x;     // long rows first
  const int h = blockIdx.y, b = blockIdx.z;
  const SampleDesc d = a.desc[b];
  const int q_base = pair * 256;
  if (!d.valid || q_base >= d.n) return;
  if (*reinterpret_cast<volatile uint32_t *>(a.status) & STATUS_ATTN_TIMEOUT) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t base = smem_u32(at_smem);
  const uint32_t q_smem = base, ring = base + 2 * AT_TILE_BYTES;
  AttnBook *bk = reinterpret_cast<AttnBook *>(at_smem + AT_MAIN_BYTES);

  const int delta = d.row0 & 7;
  const int kbase = d.row0 - delta;
  bool sees0 = false, sees1 = false;
  const int n_kt0 = (attn_key_end(d, q_base, a.mask_enable, sees0) + delta + 127) / 128;
  const int n_kt1 = q_base + 128 < d.n ? (attn_key_end(d, q_base + 128, a.mask_enable, sees1) + delta + 127) / 128 : 0;
  const int n_max = max(n_kt0, n_kt1);

  if (threadIdx.x == 0) {
    for (int s = 0; s < AT_STAGES; ++s) {
      mbar_init(smem_u32(&bk->full[s]), 1);
      mbar_init(smem_u32(&bk->empty[s]), 1);
    }
    mbar_init(smem_u32(&bk->q_full), 1);
    for (int g = 0; g < 2; ++g) {
      mbar_init(smem_u32(&bk->s_full[g]), 1);
      mbar_init(smem_u32(&bk->p_ready[g]), 256);
      mbar_init(smem_u32(&bk->pv_done[g]), 1);
      if (g == 0) mbar_init(smem_u32(&bk->mma_done), 1);
    }
    bk->abort_flag = 0;
    fence_barrier_init();
    // the query tiles and the first key / value tiles are requested right away, while the other
    // warps are still setting up (this thread is the copy thread)
    tma_prefetch_desc(&tmap_q);
    tma_prefetch_desc(&tmap_k);
    tma_prefetch_desc(&tmap_vt);
    const int n_q = n_kt1 > 0 ? 2 : 1;
    mbar_expect_tx(smem_u32(&bk->q_full), n_q * AT_TILE_BYTES);
    for (int g = 0; g < n_q; ++g) {
      tma_load_2d(q_smem + g * AT_TILE_BYTES, &tmap_q, smem_u32(&bk->q_full), h * 128, d.row0 + q_base + g * 128);
      tma_load_2d(q_smem + g * AT_TILE_BYTES + AT_BLOCK_BYTES, &tmap_q, smem_u32(&bk->q_full), h * 128 + 64,
                  d.row0 + q_base + g * 128);
    }
    for (int kt = 0; kt < min(n_max, AT_STAGES); ++kt) {
      const uint32_t dst = ring + kt * 2 * AT_TILE_BYTES;
      const uint32_t bar = smem_u32(&bk->full[kt]);
      const int key0 = kbase + kt * 128;
      mbar_expect_tx(bar, 2 * AT_TILE_BYTES);
      tma_load_2d(dst, &tmap_k, bar, h * 128, key0);
      tma_load_2d(dst + AT_BLOCK_BYTES, &tmap_k, bar, h * 128 + 64, key0);
      tma_load_2d(dst + AT_TILE_BYTES, &tmap_vt, bar, key0, h * 128);
      tma_load_2d(dst + AT_TILE_BYTES + AT_BLOCK_BYTES, &tmap_vt, bar, key0 + 64, h * 128);
    }
  }
  if (threadIdx.x < 256) (&bk->row_max[0][0])[threadIdx.x] = 0u;      // below every encoded float
  if (warp == 1) {
    tmem_alloc(smem_u32(&bk->tmem_base), AT_TMEM_COLS);
    tmem_relinquish();
    tc_fence_before();
  }
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bk->tmem_base;
  WaitCtx wc{&bk->abort_flag, a.status, STATUS_ATTN_TIMEOUT, a.wait_limit};

  if (warp == 0) {
    if (lane == 0) {
      int issued = min(n_max, AT_STAGES);          // the first tiles were requested during set-up
      for (int kt = issued; kt < n_max; ++kt) {
        const int s = kt % AT_STAGES;
        if (kt >= AT_STAGES) mbar_wait(smem_u32(&bk->empty[s]), ((kt / AT_STAGES) - 1) & 1, wc);
        if (bk->abort_flag) break;
        const uint32_t dst = ring + s * 2 * AT_TILE_BYTES;
        const uint32_t bar = smem_u32(&bk->full[s]);
        const int key0 = kbase + kt * 128;
        mbar_expect_tx(bar, 2 * AT_TILE_BYTES);
        tma_load_2d(dst, &tmap_k, bar, h * 128, key0);
        tma_load_2d(dst + AT_BLOCK_BYTES, &tmap_k, bar, h * 128 + 64, key0);
        tma_load_2d(dst + AT_TILE_BYTES, &tmap_vt, bar, key0, h * 128);
        tma_load_2d(dst + AT_TILE_BYTES + AT_BLOCK_BYTES, &tmap_vt, bar, key0 + 64, h * 128);
        issued = kt + 1;
      }
      // drain: every copy issued must have landed before the block leaves
      mbar_wait_drain(smem_u32(&bk->q_full), 0, AT_WAIT_LIMIT);
      for (int s = 0; s < AT_STAGES; ++s) {
        if (issued > s) {
          const int last = ((issued - 1 - s) / AT_STAGES) * AT_STAGES + s;
          mbar_wait_drain(smem_u32(&bk->full[s]), (last / AT_STAGES) & 1, AT_WAIT_LIMIT);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(128, 128);
      // S of row tile g for key tile kt.  Issued after the P V of key tile kt - 1 of the same row tile,
      // whose P it overwrites; the tensor pipe runs one thread's MMAs in issue order.
      auto issue_s = [&](int g, int kt) {
        const int s = kt % AT_STAGES;
        mbar_wait(smem_u32(&bk->full[s]), (kt / AT_STAGES) & 1, wc);
        tc_fence_after();
        if (bk->abort_flag) return;
        const uint32_t qa = q_smem + g * AT_TILE_BYTES, kb = ring + s * 2 * AT_TILE_BYTES;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
          tc_mma_bf16(tmem_base + g * 256, umma_desc_sw128(qa + (kk >> 2) * AT_BLOCK_BYTES + (kk & 3) * 32),
                      umma_desc_sw128(kb + (kk >> 2) * AT_BLOCK_BYTES + (kk & 3) * 32), idesc, kk > 0 ? 1u : 0u);
        tc_commit(smem_u32(&bk->s_full[g]));
      };
      mbar_wait(smem_u32(&bk->q_full), 0, wc);
      issue_s(0, 0);
      if (n_kt1 > 0) issue_s(1, 0);
      for (int kt = 0; kt < n_max; ++kt) {
        const int s = kt % AT_STAGES;
#pragma unroll
        for (int g = 0; g < 2; ++g) {
          const int n_g = g == 0 ? n_kt0 : n_kt1;
          if (kt >= n_g) continue;
          mbar_wait(smem_u32(&bk->p_ready[g]), kt & 1, wc);
          tc_fence_after();
          if (!bk->abort_flag) {
            const uint32_t vb = ring + s * 2 * AT_TILE_BYTES + AT_TILE_BYTES;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
              tc_mma_bf16_ta(tmem_base + g * 256 + 128, tmem_base + g * 256 + kk * 8,
                             umma_desc_sw128(vb + (kk >> 2) * AT_BLOCK_BYTES + (kk & 3) * 32), idesc,
                             (kt > 0 || kk > 0) ? 1u : 0u);
            tc_commit(smem_u32(&bk->pv_done[g]));
          }
          if (kt + 1 < n_g) issue_s(g, kt + 1);
        }
        if (!bk->abort_flag) tc_commit(smem_u32(&bk->empty[s]));
      }
      // every MMA this thread issued has completed before tensor memory is given back: after an abort the
      // softmax warps no longer wait for S or P V, so nothing else would hold the block until then
      tc_commit(smem_u32(&bk->mma_done));
      mbar_wait_drain(smem_u32(&bk->mma_done), 0, AT_WAIT_LIMIT);
    }
  } else {
    // Two threads per query row: warps w and w + 4 of a group own the same 32 rows (tensor-memory
    // lanes) and one half of the tile's 128 key columns each.
    const int sw = warp - 2;
    const int g = sw >> 3;                        // row tile of this softmax group
    const int hf = (sw >> 2) & 1;                 // column half
    const int quarter = warp & 3;                 // the TMEM lanes this warp may read
    const int lrow = quarter * 32 + lane;
    const int q_lo = q_base + g * 128;
    const int i = q_lo + lrow;                    // sequence-relative query row
    const bool vis_row = a.mask_enable && i >= d.v0 && i < d.v0 + d.nv;
    const int hi_adm = min(d.n - 1, vis_row ? max(i, d.v0 + d.nv - 1) : i);   // last admitted key
    const uint32_t s_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + g * 256;
    const uint32_t s_addr = s_row + hf * 64;      // this thread's 64 logits
    const uint32_t p_addr = s_row + hf * 32;      // its 64 probabilities, packed in 32 columns
    const uint32_t o_addr = s_row + 128 + hf * 64;   // its 64 columns of O
    const float *mlog_b = a.mask_log ? a.mask_log + (size_t)b * a.mask_b_stride + (size_t)h * a.mask_h_stride : nullptr;
    const int st = (threadIdx.x - 64) & 255;      // 0..255 inside the group
    const int my_kt = g == 0 ? n_kt0 : n_kt1;
    const bool my_sees = g == 0 ? sees0 : sees1;
    const int pair_bar = 1 + g * 4 + quarter;     // named barrier of the two warps that share these rows
    const int group_bar = 9 + g;

    // Logits stay in the units the MMA produced (q.k); the scale log2(e)/sqrt(d) enters inside the
    // exponential's multiply-add.  m_ref is the reference maximum in those units.
    const float step_raw = AT_RESCALE_STEP / a.scale_log2;
    const float m_to_raw = 1.4426950408889634f / a.scale_log2;
    float m_ref = -INFINITY, l_run = 0.f;
    for (int kt = 0; kt < my_kt; ++kt) {
      const int j0 = kt * 128 - delta;            // sequence-relative key of column 0
      // a tile strictly below the diagonal for every row of the row tile needs no mask at all
      const bool plain = j0 >= 0 && j0 + 127 <= q_lo && j0 + 127 < d.n;
      const bool soft = !plain && my_sees && j0 + 127 > q_lo;      // may hold future keys of the span
      const float *mt = bk->m_tile[g] + hf * 64;
      // addend of key j for a query row of the span that lies before it: m_j inside the
      // span, -infinity outside (such a key is never admitted above the diagonal)
      float mv = -INFINITY;
      if (soft && st < 128) {
        const int j = j0 + st;
        if (mlog_b && j >= d.v0 && j < d.v0 + d.nv) mv = __ldg(mlog_b + (j - d.v0)) * m_to_raw;
      }
      mbar_wait(smem_u32(&bk->s_full[g]), kt & 1, wc);
      tc_fence_after();
      if (soft) {
        // every thread of the group has finished the previous tile (its arrival was needed for
        // the S just waited for), so the addends can be replaced
        if (st < 128) bk->m_tile[g][st] = mv;
        asm volatile("bar.sync %0, 256;" ::"r"(group_bar) : "memory");
      }
      // ---- this thread's 64 logits, once
      uint32_t xr[64];
      tmem_ld32p(s_addr, xr);
      tmem_ld32p(s_addr + 32, xr + 32);
      tmem_wait_ld();
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};     // four independent chains
      if (plain) {
#pragma unroll
        for (int c = 0; c < 64; ++c) mx4[c & 3] = fmaxf(mx4[c & 3], __uint_as_float(xr[c]));
      } else {
        // columns relative to this half: the diagonal, the first and the last admitted column
        const int di = i - j0 - hf * 64, lo = -j0 - hf * 64, hi = hi_adm - j0 - hf * 64;
        if (soft && j0 > q_lo + 127) {
          // the whole tile lies above the diagonal of every row of the row tile: a row of the span
          // admits exactly the keys of the span (finite addend), any other row admits nothing.  Two
          // additions per logit on the FMA pipe instead of compares and selects on the half-rate one.
          const float rowoff = vis_row ? 0.f : -INFINITY;
#pragma unroll
          for (int c4 = 0; c4 < 64; c4 += 4) {
            const float4 m4 = *reinterpret_cast<const float4 *>(mt + c4);
            const float add[4] = {m4.x, m4.y, m4.z, m4.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float v = __uint_as_float(xr[c4 + e]) + (add[e] + rowoff);
              xr[c4 + e] = __float_as_uint(v);
              mx4[e] = fmaxf(mx4[e], v);
            }
          }
        } else if (soft) {
          // the addends are loaded unconditionally (four per load) and selected, so the loop has no branch
#pragma unroll
          for (int c4 = 0; c4 < 64; c4 += 4) {
            const float4 m4 = *reinterpret_cast<const float4 *>(mt + c4);
            const float add[4] = {m4.x, m4.y, m4.z, m4.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int c = c4 + e;
              float v = __uint_as_float(xr[c]) + (c > di ? add[e] : 0.f);
              v = (c < lo || c > hi) ? -INFINITY : v;
              xr[c] = __float_as_uint(v);
              mx4[e] = fmaxf(mx4[e], v);
            }
          }
        } else {
#pragma unroll
          for (int c = 0; c < 64; ++c) {
            const float v = (c < lo || c > hi) ? -INFINITY : __uint_as_float(xr[c]);
            xr[c] = __float_as_uint(v);
            mx4[c & 3] = fmaxf(mx4[c & 3], v);
          }
        }
      }
      float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      // ---- the running row maximum over both halves and all tiles so far.  (The partner has read
      // its logits by the time it passes this barrier, so the probabilities may overwrite them.)
      atomicMax(&bk->row_max[g][lrow], attn_key(mx));
      asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
      mx = attn_unkey(bk->row_max[g][lrow]);
      // ---- move the reference (and rescale O) only when some row of the warp outgrew it
      if (kt == 0) {
        m_ref = mx;
      } else {
        const bool need = mx > m_ref + step_raw;
        if (__any_sync(0xffffffffu, need)) {
          // O holds every earlier P V: the S just waited for was committed after them
          const float f = need ? fast_exp2((m_ref - mx) * a.scale_log2) : 1.0f;
#pragma unroll
          for (int c0 = 0; c0 < 64; c0 += 16) {
            uint32_t r[16];
            tmem_ld16(o_addr + c0, r);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 16; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * f);
            tmem_st16(o_addr + c0, r);
          }
          l_run *= f;
          if (need) m_ref = mx;
        }
      }
      // ---- probabilities relative to the reference, stored as bf16 over S's first 64 columns
      const float neg_ref = -m_ref * a.scale_log2;
      float l0 = 0.f, l1 = 0.f;
#pragma unroll
      for (int c0 = 0; c0 < 64; c0 += 32) {
        uint32_t w[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const float p0 = fast_exp2(fmaf(__uint_as_float(xr[c0 + 2 * e]), a.scale_log2, neg_ref));
          const float p1 = fast_exp2(fmaf(__uint_as_float(xr[c0 + 2 * e + 1]), a.scale_log2, neg_ref));
          l0 += p0;
          l1 += p1;
          w[e] = pack2_rn(p0, p1);
        }
        tmem_st16(p_addr + (c0 >> 1), w);
      }
      l_run += l0 + l1;
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(smem_u32(&bk->p_ready[g]));
    }
    // ---- normalisation and store: the two halves of a row add their sums first
    if (my_kt > 0) {
      // the row's slot of maxima is free once both threads have read the last one
      asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
      if (hf == 0) bk->row_max[g][lrow] = __float_as_uint(l_run);
      asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
      if (hf == 1) {
        l_run += __uint_as_float(bk->row_max[g][lrow]);
        bk->row_max[g][lrow] = __float_as_uint(l_run);
      }
      asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
      if (hf == 0) l_run = __uint_as_float(bk->row_max[g][lrow]);
      mbar_wait(smem_u32(&bk->pv_done[g]), (my_kt - 1) & 1, wc);
      tc_fence_after();
      const float inv_l = l_run > 0.f ? 1.0f / l_run : 0.f;
      const bool store = i < d.n && !bk->abort_flag;
      uint4 *orow = reinterpret_cast<uint4 *>(a.out + ((size_t)(d.row0 + i) * a.H + h) * 128 + hf * 64);
#pragma unroll
      for (int c0 = 0; c0 < 64; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(o_addr + c0, r);
        tmem_wait_ld();
        if (store) {
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            uint4 w;
            w.x = pack2_rn(__uint_as_float(r[8 * q4 + 0]) * inv_l, __uint_as_float(r[8 * q4 + 1]) * inv_l);
            w.y = pack2_rn(__uint_as_float(r[8 * q4 + 2]) * inv_l, __uint_as_float(r[8 * q4 + 3]) * inv_l);
            w.z = pack2_rn(__uint_as_float(r[8 * q4 + 4]) * inv_l, __uint_as_float(r[8 * q4 + 5]) * inv_l);
            w.w = pack2_rn(__uint_as_float(r[8 * q4 + 6]) * inv_l, __uint_as_float(r[8 * q4 + 7]) * inv_l);
            orow[(c0 >> 3) + q4] = w;
          }
        }
      }
    }
    tc_fence_before();
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, AT_TMEM_COLS);
  }
}

}  // namespace asap
