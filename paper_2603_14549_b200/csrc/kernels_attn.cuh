// The layer's attention under the salience-guided bidirectional mask (Eq. 4 applied to the
// values):  O^h = Softmax(W^h + M_bidir) V^h,  W^h = Q^h K^h^T / sqrt(d).
//
//   transpose_v_kernel  V [tokens, D] -> V^T [D, tokens] (row pitch padded to 8 tokens), so that
//                       a value tile can be loaded as a K-major MMA operand like every other tile.
//   attn_kernel         one block per (128 query rows, head, sequence).  For every tile of 128
//                       keys:  S = Q K^T on tcgen05 into tensor memory, the softmax warps turn S
//                       into probabilities relative to the running row maximum (Eq. 3's m_j is
//                       added for the future keys of the image span on rows of the image span,
//                       nothing else above the diagonal is admitted), write them as a bf16
//                       operand tile into shared memory, and  O_tile = P V  runs on tcgen05 again;
//                       the softmax warps fold O_tile into their fp32 running output with the
//                       usual rescaling.  M_bidir is never materialised: it is the vector m_j
//                       plus position tests.
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
constexpr int AT_THREADS = 192;                 // warp 0: copies, warp 1: MMA issue, warps 2-5: softmax
constexpr int AT_TILE_BYTES = 128 * 128 * 2;    // 128 rows x 128 bf16 as two 64-column blocks of 16 KB
constexpr int AT_BLOCK_BYTES = AT_TILE_BYTES / 2;
constexpr int AT_STAGES = 2;                    // a stage = one key tile + one value tile
constexpr int AT_MAIN_BYTES = 2 * AT_TILE_BYTES + AT_STAGES * 2 * AT_TILE_BYTES;
constexpr int AT_BOOK_BYTES = 2048;
constexpr int AT_SMEM_BYTES = AT_MAIN_BYTES + AT_BOOK_BYTES;
constexpr uint32_t AT_TMEM_COLS = 512;          // S (two buffers of 128 columns) and O_tile (128 columns)
constexpr long long AT_WAIT_LIMIT = 2000000000LL;
static_assert(AT_SMEM_BYTES <= 195 * 1024, "the attention block must stay inside the 196 KB carve-out");

struct AttnArgs {
  const SampleDesc *desc;
  int H, D, max_vis, mask_enable;
  float scale_log2;            // log2(e) / sqrt(head_dim)
  const float *mask_log;       // [B, max_vis] m_j (natural log), may be null with the mask off
  __nv_bfloat16 *out;          // [tokens, H, 128]
  uint32_t *status;
};

struct AttnBook {
  uint64_t full[AT_STAGES], empty[AT_STAGES], q_full, s_full[2], s_free[2], p_ready, pv_done, o_free;
  uint32_t tmem_base;
  int abort_flag;
  float m_tile[2][128];
};
static_assert(sizeof(AttnBook) <= AT_BOOK_BYTES, "attention kernel bookkeeping exceeds its shared-memory slot");

__global__ void __launch_bounds__(AT_THREADS, 1)
attn_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
            const __grid_constant__ CUtensorMap tmap_vt, AttnArgs a) {
  pdl_enter();
  extern __shared__ __align__(1024) uint8_t at_smem[];
  const int qt = (int)gridDim.x - 1 - (int)blockIdx.x;     // long rows first
  const int h = blockIdx.y, b = blockIdx.z;
  const SampleDesc d = a.desc[b];
  const int q_lo = qt * 128;
  if (!d.valid || q_lo >= d.n) return;
  if (*reinterpret_cast<volatile uint32_t *>(a.status) & STATUS_ATTN_TIMEOUT) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t base = smem_u32(at_smem);
  const uint32_t q_smem = base, p_smem = base + AT_TILE_BYTES, ring = base + 2 * AT_TILE_BYTES;
  AttnBook *bk = reinterpret_cast<AttnBook *>(at_smem + AT_MAIN_BYTES);

  // keys this row tile can see: up to its last row (causal), and to the end of the image span
  // if one of its rows lies inside the span and the mask is on
  const int q_hi = min(q_lo + 128, d.n);
  const bool sees_span = a.mask_enable && q_lo < d.v0 + d.nv && q_hi > d.v0;
  const int j_end = min(d.n, sees_span ? max(q_hi, d.v0 + d.nv) : q_hi);
  const int delta = d.row0 & 7;
  const int kbase = d.row0 - delta;
  const int n_kt = (j_end + delta + 127) / 128;

  if (threadIdx.x == 0) {
    for (int s = 0; s < AT_STAGES; ++s) {
      mbar_init(smem_u32(&bk->full[s]), 1);
      mbar_init(smem_u32(&bk->empty[s]), 1);
    }
    mbar_init(smem_u32(&bk->q_full), 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&bk->s_full[i]), 1);
      mbar_init(smem_u32(&bk->s_free[i]), 128);
    }
    mbar_init(smem_u32(&bk->p_ready), 128);
    mbar_init(smem_u32(&bk->pv_done), 1);
    mbar_init(smem_u32(&bk->o_free), 128);
    bk->abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&bk->tmem_base), AT_TMEM_COLS);
    tmem_relinquish();
    tc_fence_before();
  }
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bk->tmem_base;
  WaitCtx wc{&bk->abort_flag, a.status, STATUS_ATTN_TIMEOUT, AT_WAIT_LIMIT};

  if (warp == 0) {
    if (lane == 0) {
      tma_prefetch_desc(&tmap_q);
      tma_prefetch_desc(&tmap_k);
      tma_prefetch_desc(&tmap_vt);
      mbar_expect_tx(smem_u32(&bk->q_full), AT_TILE_BYTES);
      tma_load_2d(q_smem, &tmap_q, smem_u32(&bk->q_full), h * 128, d.row0 + q_lo);
      tma_load_2d(q_smem + AT_BLOCK_BYTES, &tmap_q, smem_u32(&bk->q_full), h * 128 + 64, d.row0 + q_lo);
      int issued = 0;
      for (int kt = 0; kt < n_kt; ++kt) {
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
      const uint32_t o_tmem = tmem_base + 256;
      auto issue_s = [&](int kt) {
        const int s = kt % AT_STAGES, buf = kt & 1;
        mbar_wait(smem_u32(&bk->full[s]), (kt / AT_STAGES) & 1, wc);
        if (kt >= 2) mbar_wait(smem_u32(&bk->s_free[buf]), ((kt >> 1) - 1) & 1, wc);
        tc_fence_after();
        if (bk->abort_flag) return;
        const uint32_t kb = ring + s * 2 * AT_TILE_BYTES;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
          tc_mma_bf16(tmem_base + buf * 128, umma_desc_sw128(q_smem + (kk >> 2) * AT_BLOCK_BYTES + (kk & 3) * 32),
                      umma_desc_sw128(kb + (kk >> 2) * AT_BLOCK_BYTES + (kk & 3) * 32), idesc, kk > 0 ? 1u : 0u);
        tc_commit(smem_u32(&bk->s_full[buf]));
      };
      mbar_wait(smem_u32(&bk->q_full), 0, wc);
      issue_s(0);
      for (int kt = 0; kt < n_kt; ++kt) {
        if (kt + 1 < n_kt) issue_s(kt + 1);
        const int s = kt % AT_STAGES;
        mbar_wait(smem_u32(&bk->p_ready), kt & 1, wc);
        if (kt >= 1) mbar_wait(smem_u32(&bk->o_free), (kt - 1) & 1, wc);
        tc_fence_after();
        if (!bk->abort_flag) {
          const uint32_t vb = ring + s * 2 * AT_TILE_BYTES + AT_TILE_BYTES;
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            tc_mma_bf16(o_tmem, umma_desc_sw128(p_smem + (kk >> 2) * AT_BLOCK_BYTES + (kk & 3) * 32),
                        umma_desc_sw128(vb + (kk >> 2) * AT_BLOCK_BYTES + (kk & 3) * 32), idesc, kk > 0 ? 1u : 0u);
          tc_commit(smem_u32(&bk->pv_done));
          tc_commit(smem_u32(&bk->empty[s]));
        }
      }
    }
  } else {
    const int quarter = warp & 3;                 // the TMEM lanes this warp may read
    const int lrow = quarter * 32 + lane;
    const int i = q_lo + lrow;                    // sequence-relative query row
    const bool vis_row = a.mask_enable && i >= d.v0 && i < d.v0 + d.nv;
    const int hi_adm = min(d.n - 1, vis_row ? max(i, d.v0 + d.nv - 1) : i);   // last admitted key
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const float *mlog_b = a.mask_log ? a.mask_log + (size_t)b * a.max_vis : nullptr;
    uint8_t *p_row = at_smem + AT_TILE_BYTES + lrow * 128;
    const int st = threadIdx.x - 64;              // 0..127 among the softmax threads

    float o_acc[128];
#pragma unroll
    for (int c = 0; c < 128; ++c) o_acc[c] = 0.f;
    float m_run = -INFINITY, l_run = 0.f, alpha_prev = 0.f;

    for (int kt = 0; kt < n_kt; ++kt) {
      const int buf = kt & 1;
      const int j0 = kt * 128 - delta;            // sequence-relative key of column 0
      // a tile strictly below the diagonal for every row of the block needs no mask at all
      const bool plain = j0 >= 0 && j0 + 127 <= q_lo && j0 + 127 < d.n;
      const bool soft = !plain && sees_span && j0 + 127 > q_lo;    // may hold future keys of the span
      if (soft) {
        const int j = j0 + st;
        float mv = 0.f;
        if (mlog_b && j >= d.v0 && j < d.v0 + d.nv) mv = __ldg(mlog_b + (j - d.v0)) * 1.4426950408889634f;
        bk->m_tile[buf][st] = mv;
        asm volatile("bar.sync 1, 128;" ::: "memory");
      }
      const float *mt = bk->m_tile[buf];
      mbar_wait(smem_u32(&bk->s_full[buf]), (kt >> 1) & 1, wc);
      tc_fence_after();
      const uint32_t s_addr = lane_addr + buf * 128;
      // ---- pass 1: row maximum of the admitted logits
      float mx = m_run;
#pragma unroll 1
      for (int c0 = 0; c0 < 128; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(s_addr + c0, r);
        tmem_wait_ld();
        if (plain) {
#pragma unroll
          for (int e = 0; e < 32; ++e) mx = fmaxf(mx, __uint_as_float(r[e]) * a.scale_log2);
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const int j = j0 + c0 + e;
            float x = __uint_as_float(r[e]) * a.scale_log2;
            if (soft && j > i) x += mt[c0 + e];
            if (j >= 0 && j <= hi_adm) mx = fmaxf(mx, x);
          }
        }
      }
      const float alpha = fast_exp2(m_run - mx);           // first tile: exp2(-inf) = 0
      // ---- fold the previous tile's P V into the running output
      if (kt > 0) {
        mbar_wait(smem_u32(&bk->pv_done), (kt - 1) & 1, wc);
        tc_fence_after();
#pragma unroll
        for (int c0 = 0; c0 < 128; c0 += 32) {
          uint32_t r[32];
          tmem_ld32(lane_addr + 256 + c0, r);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) o_acc[c0 + e] = fmaf(o_acc[c0 + e], alpha_prev, __uint_as_float(r[e]));
        }
        tc_fence_before();
        mbar_arrive(smem_u32(&bk->o_free));
      }
      // ---- pass 2: probabilities relative to the new maximum, as a bf16 operand tile
      float l_tile = 0.f;
#pragma unroll 1
      for (int c0 = 0; c0 < 128; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(s_addr + c0, r);
        tmem_wait_ld();
        float pv[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          const int j = j0 + c0 + e;
          float x = __uint_as_float(r[e]) * a.scale_log2;
          if (!plain) {
            if (soft && j > i) x += mt[c0 + e];
            if (!(j >= 0 && j <= hi_adm)) x = -INFINITY;
          }
          pv[e] = fast_exp2(x - mx);
        }
#pragma unroll
        for (int g = 0; g < 4; ++g) {                       // four 16-byte chunks of eight keys
          uint4 w;
          w.x = pack2_rn(pv[8 * g + 0], pv[8 * g + 1]);
          w.y = pack2_rn(pv[8 * g + 2], pv[8 * g + 3]);
          w.z = pack2_rn(pv[8 * g + 4], pv[8 * g + 5]);
          w.w = pack2_rn(pv[8 * g + 6], pv[8 * g + 7]);
          // the row sum uses the rounded values the MMA will see
          l_tile += (bf16_lo(w.x) + bf16_hi(w.x)) + (bf16_lo(w.y) + bf16_hi(w.y)) +
                    (bf16_lo(w.z) + bf16_hi(w.z)) + (bf16_lo(w.w) + bf16_hi(w.w));
          const int col = c0 + 8 * g;                       // first key of the chunk
          const int blk = col >> 6, chunk = (col & 63) >> 3;
          *reinterpret_cast<uint4 *>(p_row + blk * AT_BLOCK_BYTES + ((chunk ^ (lrow & 7)) << 4)) = w;
        }
      }
      l_run = l_run * alpha + l_tile;
      m_run = mx;
      alpha_prev = alpha;
      tc_fence_before();
      fence_proxy_async();                                  // the MMA reads P through the async proxy
      mbar_arrive(smem_u32(&bk->s_free[buf]));
      mbar_arrive(smem_u32(&bk->p_ready));
    }
    // ---- last tile's P V, normalisation, store
    mbar_wait(smem_u32(&bk->pv_done), (n_kt - 1) & 1, wc);
    tc_fence_after();
    const float inv_l = l_run > 0.f ? 1.0f / l_run : 0.f;
    const bool store = i < d.n && !bk->abort_flag;
    uint4 *orow = reinterpret_cast<uint4 *>(a.out + ((size_t)(d.row0 + i) * a.H + h) * 128);
#pragma unroll
    for (int c0 = 0; c0 < 128; c0 += 32) {
      uint32_t r[32];
      tmem_ld32(lane_addr + 256 + c0, r);
      tmem_wait_ld();
      // the last fold needs no rescaling: O_tile is already relative to the final maximum
#pragma unroll
      for (int e = 0; e < 32; ++e) o_acc[c0 + e] = fmaf(o_acc[c0 + e], alpha_prev, __uint_as_float(r[e])) * inv_l;
      if (store) {
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          uint4 w;
          w.x = pack2_rn(o_acc[c0 + 8 * g + 0], o_acc[c0 + 8 * g + 1]);
          w.y = pack2_rn(o_acc[c0 + 8 * g + 2], o_acc[c0 + 8 * g + 3]);
          w.z = pack2_rn(o_acc[c0 + 8 * g + 4], o_acc[c0 + 8 * g + 5]);
          w.w = pack2_rn(o_acc[c0 + 8 * g + 6], o_acc[c0 + 8 * g + 7]);
          orow[(c0 >> 3) + g] = w;
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
