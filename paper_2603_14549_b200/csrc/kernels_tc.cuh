// The two dense contractions of the ASAP prune step on the sm_100a tensor cores
// (tcgen05.mma, operands staged by TMA into 128-byte-swizzled shared memory, fp32
// accumulators in tensor memory):
//
//   score_kernel  Eq. 3 / Eq. 4: masked softmax of the ranking rows' logits, reduced over
//                 ranking rows; the logits never leave the SM.
//   sim_kernel    Sec. 4.2: cosine similarity of every visual row against the kept rows with
//                 the arg-max over kept slots taken in the epilogue.
//
// Both use one TMA-producer warp, one MMA-issuer warp (a single elected lane) and four
// epilogue warps that read tensor memory (warp w may touch lanes 32*(w%4) .. 32*(w%4)+31).
// Every mbarrier wait is bounded (see WaitCtx); after an abort the block keeps walking its
// uniform control flow so that every named barrier and the final teardown are still reached.
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "kernels_stream.cuh"

namespace asap {

constexpr long long TC_WAIT_LIMIT = 1500000000LL;   // clock cycles, roughly one second
constexpr float LOG2E_F = 1.4426950408889634f;

// named barriers of the score kernel: 2 = all eight epilogue
// warps; 3 / 4 = one of its two epilogue groups
__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 2, 256;" ::: "memory"); }
__device__ __forceinline__ void group_bar_sync(int group) {
  asm volatile("bar.sync %0, 128;" ::"r"(3 + group) : "memory");
}

// =======================================================================================
// score_kernel
//
// Persistent blocks; a work item is one (sample b, head h); blocks draw items from a global
// counter (the ranking rows per sample differ by up to 8x, so a fixed deal leaves blocks idle).
// The ranking rows of an item are taken 256 at a time (a row pair: two row tiles of 128).  For
// each row pair, every key tile is brought to shared memory once per pass and serves both row tiles:
//   pass 1  D = Q_rows K_tile^T   (M = 128 rows, N = 128 keys, one accumulator per row tile):
//           thread-per-row running max / sum over all admitted keys -> off_i = max_i + log2(sum_i)
//   pass 2  D = K_tile Q_rows^T   (M = 128 keys, N = all rows of the pair, up to 256): thread-per-key
//           sum over rows of exp2(logit + mask - off_i), i.e. of the Eq. 4 probabilities A[i, j]
// Key tiles stream through a shared-memory ring in one linear order (pass 1 ascending, pass 2
// over the tiles that hold visual keys, coming back from L2); tensor memory holds two halves of 256
// columns that alternate between consecutive operations, so the MMA issuer runs one operation ahead
// of the epilogue warps.
// Epilogue: two groups of four warps.  Pass 1 with two row tiles: group g owns row tile g of every
// key tile.  Pass 1 with one row tile, and pass 2: the groups take alternate operations.  Every
// epilogue warp passes every operation's barriers (waits for the accumulator, releases it), whether
// it has work on it or not, so the barrier counts never depend on the shape of the item.
// Additive mask (Eq. 3), logits in log2 units: 0 for key j <= row position p; m_j*log2(e) for
// j > p when both are in the image span (mask enabled); -inf otherwise.
// The per-head sums over ranking rows go to `partial`; head_sum_kernel adds them in head order.
// Attention mass on the way (a.qbar given; ranking rows after the image span): Eq. 1 with the sum over
// the queries taken first is qbar^h . k_j^h, and pass 2 already multiplies every visual key tile by the
// row pair's queries.  The summed query rides along as three more "query rows" (its bf16 value, the bf16
// value of what that rounding lost, and again: 24 bits of mantissa together, all that fp32 holds),
// written behind the pair's rows in shared memory, so the first row pair's pass-2 accumulators get three
// more columns whose sum is the key's mass for this head.  Row pairs then hold at most 240 rows (the
// accumulator grows by the 16 columns an MMA's width moves in).
// =======================================================================================
constexpr int SC_THREADS = 320;          // producer warp, MMA warp, 2 x 4 epilogue warps
constexpr int SC_EPI_THREADS = 256;
constexpr int SC_STAGES = 4;
constexpr int SC_HALF_BYTES = 128 * 128;        // 128 rows x 64 bf16
constexpr int SC_TILE_BYTES = 2 * SC_HALF_BYTES;
constexpr int SC_Q_HALF_BYTES = 256 * 128;      // 256 rows x 64 bf16: one 64-column half of a row pair
constexpr int SC_Q_BYTES = 2 * SC_Q_HALF_BYTES;
constexpr int SC_SMEM_MAIN = SC_Q_BYTES + SC_STAGES * SC_TILE_BYTES;
// Total dynamic shared memory stays at 195 KB: with the 1 KB the system reserves per block that
// is the 196 KB carve-out, which leaves the SM 32 KB of L1 for the memory-bound kernels that run
// beside this one; one byte more selects the 228 KB carve-out and costs them about 10 us.
constexpr int SC_BOOK_BYTES = 3072;
constexpr int SC_SMEM_BYTES = SC_SMEM_MAIN + SC_BOOK_BYTES;
constexpr uint32_t SC_TMEM_COLS = 512;     // two halves of 256 columns
constexpr int SC_ITEM_SLOTS = 4;

struct ScoreArgs {
  PrepareArgs pa;             // every block derives its descriptors itself: the kernel does not wait
                              // for the validation kernel (it writes nothing but scratch)
  int B, H, max_vis, mask_enable;
  float scale_log2;           // log2(e) / sqrt(head_dim)
  const float *mask_log;      // [B, max_vis] m_j (natural log), or [B, H, max_vis] with a mask per head
  int mask_b_stride, mask_h_stride;   // max_vis, 0   or   H * max_vis, max_vis
  float *partial;             // [B, H, max_vis] per-head sums over ranking rows
  const float *qbar;          // [B, D] sum of the visual queries (Eq. 1, queries first), or nullptr.  Given: the
                              // kernel also writes mass_heads (the attention mass per head), see below
  float *mass_heads;          // [B, H, max_vis] qbar^h . k_j^h for every visual key j (unscaled)
  int D;
  unsigned int *work;         // [2] next item / blocks that have finished; both zero between launches
  uint32_t *status;
  long long wait_limit;       // clock cycles a wait may take before the block gives up
};

struct ScoreBook {             // bookkeeping block placed after the tiles in shared memory
  uint64_t full[SC_STAGES], empty[SC_STAGES], q_full, q_empty, acc_full[2], acc_empty[2];
  uint64_t item_full[SC_ITEM_SLOTS], item_empty[SC_ITEM_SLOTS], mma_done, qbar_ready;
  int item_q[SC_ITEM_SLOTS];   // items drawn by the producer, -1 = no more
  alignas(16) float off[256];  // per ranking row of the pair: max + log2(sum), +inf for rows past its end
                               // (with one row tile, off[128..255] carries group 1's partial sums)
  alignas(16) float soft[2][128];   // per epilogue group, per key of its current tile: m_j*log2(e) or -inf
                               // (soft[1] also carries group 1's partial maxima at the end of pass 1)
  uint32_t tmem_base;
  int abort_flag;
};

static_assert(sizeof(ScoreBook) <= SC_BOOK_BYTES, "score kernel bookkeeping exceeds its shared-memory slot");

struct RowPair {
  int R0, nrows, nrt, n2, n_kt, t_lo, t_hi, n_p2;
  bool use_soft;
};

// Row pair rp of a sample's ranking rows: rows R0 .. R0 + nrows - 1 (sequence-relative positions).
__device__ __forceinline__ RowPair score_row_pair(const SampleDesc &d, int rp, int mask_enable, int pair_rows) {
  RowPair r;
  r.R0 = d.r0 + rp * pair_rows;
  r.nrows = min(pair_rows, d.nr - rp * pair_rows);
  r.nrt = (r.nrows + 127) >> 7;
  r.n2 = (r.nrows + 15) & ~15;
  const int p_max = r.R0 + r.nrows - 1;
  r.use_soft = mask_enable && (r.R0 < d.v0 + d.nv) && (p_max >= d.v0);
  int jmax = p_max;
  if (r.use_soft) jmax = max(jmax, d.v0 + d.nv - 1);
  r.n_kt = jmax / 128 + 1;
  r.t_lo = d.v0 / 128;
  r.t_hi = min((d.v0 + d.nv - 1) / 128, r.n_kt - 1);
  r.n_p2 = r.t_hi >= r.t_lo ? r.t_hi - r.t_lo + 1 : 0;
  return r;
}

__global__ void __launch_bounds__(SC_THREADS, 1)
score_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
             ScoreArgs a) {
  // (the wait for the preceding kernel comes after the block's set-up, which reads nothing that kernel writes)
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_items = a.B * a.H;
  const bool with_mass = a.qbar != nullptr;
  const int pair_rows = with_mass ? 240 : 256;           // ranking rows per row pair

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
  if ((base - smem_u32(smem_raw)) + SC_SMEM_MAIN + sizeof(ScoreBook) > (uint32_t)SC_SMEM_BYTES) {
    // the tiles need a 1024-byte aligned start; the window is expected to provide it
    if (threadIdx.x == 0) atomicOr(a.status, STATUS_SCORE_TIMEOUT);
    return;
  }
  const uint32_t q_smem = base;                          // the row pair's queries
  const uint32_t k_smem = base + SC_Q_BYTES;             // ring of key tiles
  ScoreBook *bk = reinterpret_cast<ScoreBook *>(base_ptr + SC_SMEM_MAIN);

  if (threadIdx.x == 0) {
    for (int s = 0; s < SC_STAGES; ++s) {
      mbar_init(smem_u32(&bk->full[s]), 1);
      mbar_init(smem_u32(&bk->empty[s]), 1);
    }
    mbar_init(smem_u32(&bk->q_full), 1);
    mbar_init(smem_u32(&bk->q_empty), 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&bk->acc_full[i]), 1);
      mbar_init(smem_u32(&bk->acc_empty[i]), 8);          // every epilogue warp
    }
    for (int i = 0; i < SC_ITEM_SLOTS; ++i) {
      mbar_init(smem_u32(&bk->item_full[i]), 1);
      mbar_init(smem_u32(&bk->item_empty[i]), 9);         // the MMA issuer + every epilogue warp
    }
    mbar_init(smem_u32(&bk->mma_done), 1);
    mbar_init(smem_u32(&bk->qbar_ready), 1);
    bk->abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&bk->tmem_base), SC_TMEM_COLS);
    tmem_relinquish();
    tc_fence_before();
  }
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bk->tmem_base;
  WaitCtx wc{&bk->abort_flag, a.status, STATUS_SCORE_TIMEOUT, a.wait_limit};
  if (*reinterpret_cast<volatile uint32_t *>(a.status) & STATUS_SCORE_TIMEOUT) bk->abort_flag = 1;   // benign race: same value
  __syncthreads();
  pdl_enter();

  if (warp == 0) {
    // ------------------------------------------------------------------ producer: items, queries, key tiles
    if (lane == 0) {
      tma_prefetch_desc(&tmap_q);
      tma_prefetch_desc(&tmap_k);
      int kc = 0, qc = 0, ic = 0;               // key tiles / row pairs / items so far
      int k_issued = 0, q_issued = 0;           // copies actually issued (an abort is sticky, so
                                                // these are prefixes of the two sequences)
      while (true) {
        const int slot = ic % SC_ITEM_SLOTS;
        // The item queue keeps working after an abort (its waits ignore the flag and are bounded on their
        // own): every consumer must see the same sequence of items, ending with -1, or the epilogue warps'
        // named barriers would no longer match.  After an abort that sequence ends at once.
        if (ic >= SC_ITEM_SLOTS &&
            !mbar_wait_drain(smem_u32(&bk->item_empty[slot]), ((ic / SC_ITEM_SLOTS) - 1) & 1, TC_WAIT_LIMIT))
          break;
        int item = bk->abort_flag ? n_items : (int)atomicAdd(a.work, 1u);
        if (item >= n_items) item = -1;
        bk->item_q[slot] = item;
        mbar_arrive(smem_u32(&bk->item_full[slot]));      // release: the slot's content is visible to the waiters
        ++ic;
        if (item < 0) break;
        const int b = item / a.H, h = item - b * a.H;
        const SampleDesc d = make_desc(a.pa, b);
        if (!d.valid) continue;
        const int n_rp = (d.nr + pair_rows - 1) / pair_rows;
        for (int rp = 0; rp < n_rp; ++rp, ++qc) {
          const RowPair T = score_row_pair(d, rp, a.mask_enable, pair_rows);
          if (qc >= 1) mbar_wait(smem_u32(&bk->q_empty), (qc - 1) & 1, wc);
          if (!bk->abort_flag) {
            mbar_expect_tx(smem_u32(&bk->q_full), T.nrt * SC_TILE_BYTES);
            for (int hf = 0; hf < 2; ++hf)
              for (int rt = 0; rt < T.nrt; ++rt)
                tma_load_2d(q_smem + hf * SC_Q_HALF_BYTES + rt * SC_HALF_BYTES, &tmap_q, smem_u32(&bk->q_full),
                            h * 128 + hf * 64, d.row0 + T.R0 + rt * 128);
            q_issued = qc + 1;
          }
          for (int u = 0; u < T.n_kt + T.n_p2; ++u, ++kc) {
            const int t = u < T.n_kt ? u : T.t_hi - (u - T.n_kt);
            const int s = kc % SC_STAGES;
            if (kc >= SC_STAGES) mbar_wait(smem_u32(&bk->empty[s]), ((kc / SC_STAGES) - 1) & 1, wc);
            if (!bk->abort_flag) {
              const uint32_t dst = k_smem + s * SC_TILE_BYTES;
              mbar_expect_tx(smem_u32(&bk->full[s]), SC_TILE_BYTES);
              tma_load_2d(dst, &tmap_k, smem_u32(&bk->full[s]), h * 128, d.row0 + t * 128);
              tma_load_2d(dst + SC_HALF_BYTES, &tmap_k, smem_u32(&bk->full[s]), h * 128 + 64, d.row0 + t * 128);
              k_issued = kc + 1;
            }
          }
        }
      }
      // every copy this thread issued must have landed before the block may leave
      for (int s = 0; s < SC_STAGES; ++s) {
        const int fills = k_issued > s ? (k_issued - s + SC_STAGES - 1) / SC_STAGES : 0;
        if (fills > 0) mbar_wait_drain(smem_u32(&bk->full[s]), (fills - 1) & 1, TC_WAIT_LIMIT);
      }
      if (q_issued > 0) mbar_wait_drain(smem_u32(&bk->q_full), (q_issued - 1) & 1, TC_WAIT_LIMIT);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int kc = 0, qc = 0, g = 0, ic = 0, mc = 0;      // mc: items whose summed-query rows were waited for
      bool issued_any = false;
      const uint32_t idesc1 = umma_idesc_bf16(128, 128);
      const uint64_t qdesc = umma_desc_sw128(q_smem);          // (every tile lies below 256 KB: offsets never carry out of the address field)
      while (true) {
        const int slot = ic % SC_ITEM_SLOTS;
        const bool got = mbar_wait_drain(smem_u32(&bk->item_full[slot]), (ic / SC_ITEM_SLOTS) & 1, TC_WAIT_LIMIT);
        const int item = got ? bk->item_q[slot] : -1;
        mbar_arrive(smem_u32(&bk->item_empty[slot]));
        ++ic;
        if (item < 0) break;
        const int b = item / a.H;
        const SampleDesc d = make_desc(a.pa, b);
        if (!d.valid) continue;
        const int n_rp = (d.nr + pair_rows - 1) / pair_rows;
        for (int rp = 0; rp < n_rp; ++rp, ++qc) {
          const RowPair T = score_row_pair(d, rp, a.mask_enable, pair_rows);
          const bool mass_here = with_mass && rp == 0;       // three more columns (16 with padding): the summed query
          const uint32_t idesc2 = umma_idesc_bf16(128, T.n2 + (mass_here ? 16 : 0));
          mbar_wait(smem_u32(&bk->q_full), qc & 1, wc);
          for (int u = 0; u < T.n_kt + T.n_p2; ++u, ++kc, ++g) {
            const bool pass1 = u < T.n_kt;
            if (mass_here && u == T.n_kt) {                  // an epilogue warp has written the summed-query rows
              mbar_wait(smem_u32(&bk->qbar_ready), mc & 1, wc);
              ++mc;
            }
            const int s = kc % SC_STAGES, hh = g & 1;
            if (g >= 2) mbar_wait(smem_u32(&bk->acc_empty[hh]), ((g >> 1) - 1) & 1, wc);
            mbar_wait(smem_u32(&bk->full[s]), (kc / SC_STAGES) & 1, wc);
            tc_fence_after();
            if (!bk->abort_flag) {
              const uint32_t ks = k_smem + s * SC_TILE_BYTES;
              const uint32_t dcol = tmem_base + hh * 256;
              const uint64_t kdesc = umma_desc_sw128(ks);
              if (pass1) {
                tc_mma_bf16_k128<SC_Q_HALF_BYTES, SC_HALF_BYTES>(dcol, qdesc, kdesc, idesc1);
                if (T.nrt == 2)
                  tc_mma_bf16_k128<SC_Q_HALF_BYTES, SC_HALF_BYTES>(dcol + 128, qdesc + (SC_HALF_BYTES >> 4), kdesc, idesc1);
              } else {
                tc_mma_bf16_k128<SC_HALF_BYTES, SC_Q_HALF_BYTES>(dcol, kdesc, qdesc, idesc2);
              }
              tc_commit(smem_u32(&bk->empty[s]));
              tc_commit(smem_u32(&bk->acc_full[hh]));
              issued_any = true;
            }
          }
          if (mass_here && T.n_p2 == 0) {                    // (no visual key tile: keep the barrier's phases in step)
            mbar_wait(smem_u32(&bk->qbar_ready), mc & 1, wc);
            ++mc;
          }
          if (!bk->abort_flag) tc_commit(smem_u32(&bk->q_empty));
        }
      }
      // every MMA this thread issued has completed before tensor memory is given back: after an abort the
      // epilogue warps no longer wait for the accumulators, so nothing else would hold the block until then
      if (issued_any) {
        tc_commit(smem_u32(&bk->mma_done));
        mbar_wait_drain(smem_u32(&bk->mma_done), 0, TC_WAIT_LIMIT);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (2 groups x 4 warps)
    // Warp q of a group reads tensor-memory lanes 32q .. 32q+31.
    const int group = (warp - 2) >> 2;
    const int quarter = warp & 3;
    const int lrow = quarter * 32 + lane;          // tensor-memory lane owned by this thread
    const int et = (warp - 2) * 32 + lane;         // 0..255 among the epilogue threads
    const float scale = a.scale_log2;
    const uint32_t tlane0 = tmem_base + ((uint32_t)(quarter * 32) << 16);
    float *soft = bk->soft[group];
    float *pm = bk->soft[1], *pl = bk->off + 128;  // group 1's (max, sum) when both groups share one row tile
    int g = 0, ic = 0, qc = 0;
    while (true) {
      const int slot = ic % SC_ITEM_SLOTS;
      const bool got = mbar_wait_drain(smem_u32(&bk->item_full[slot]), (ic / SC_ITEM_SLOTS) & 1, TC_WAIT_LIMIT);
      const int item = got ? bk->item_q[slot] : -1;
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bk->item_empty[slot]));
      ++ic;
      if (item < 0) break;
      const int b = item / a.H, h = item - b * a.H;
      const SampleDesc d = make_desc(a.pa, b);
      if (!d.valid) continue;
      const int n_rp = (d.nr + pair_rows - 1) / pair_rows;
      float *part = a.partial + ((size_t)b * a.H + h) * a.max_vis;
      const float *mlog = a.mask_log + (size_t)b * a.mask_b_stride + (size_t)h * a.mask_h_stride;
      const int v_end = d.v0 + d.nv;
      {
        // visual keys beyond the tiles the first row pair visits in pass 2 (possible only when
        // ranking rows lie before the end of the image span) start from zero; the epilogue-wide
        // barrier that ends every pass 1 orders these stores before any later add
        const RowPair T0 = score_row_pair(d, 0, a.mask_enable, pair_rows);
        const int first = T0.n_p2 > 0 ? max((T0.t_hi + 1) * 128 - d.v0, 0) : 0;
        for (int j = first + et; j < d.nv; j += SC_EPI_THREADS) part[j] = 0.f;
      }
      for (int rp = 0; rp < n_rp; ++rp, ++qc) {
        const RowPair T = score_row_pair(d, rp, a.mask_enable, pair_rows);
        if (with_mass && rp == 0 && warp == 2) {
          // The summed query of this head as rows n2 .. n2 + 2 of the pair's query tile: 3 rows x 16 chunks
          // of 16 bytes at their swizzled places (row r of a 64-column half is 128 bytes at
          // r * 128, chunk c at c ^ (r & 7)), once the tiled copy of the queries has landed.
          mbar_wait(smem_u32(&bk->q_full), qc & 1, wc);
          const int c16 = lane & 15;
          const float *src = a.qbar + (size_t)b * a.D + h * 128 + c16 * 8;
          uint32_t w[3][4];                                 // the value as three bf16 pieces: 24 bits of mantissa, all of fp32's
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float x[2] = {__ldcg(src + 2 * e), __ldcg(src + 2 * e + 1)}, piece[3][2];
#pragma unroll
            for (int t = 0; t < 2; ++t) {
              float rest = x[t];
#pragma unroll
              for (int k = 0; k < 3; ++k) {
                piece[k][t] = __bfloat162float(__float2bfloat16_rn(rest));
                rest -= piece[k][t];
              }
            }
#pragma unroll
            for (int k = 0; k < 3; ++k) w[k][e] = pack2_rn(piece[k][0], piece[k][1]);
          }
          // lanes 0-15 write the first piece's row and the third's, lanes 16-31 the second's
#pragma unroll
          for (int k = 0; k < 3; ++k) {
            if ((k == 1) == (lane >= 16)) {
              const int row = T.n2 + k;
              uint8_t *dst = base_ptr + (c16 >> 3) * SC_Q_HALF_BYTES + row * 128 + (((c16 & 7) ^ (row & 7)) << 4);
              *reinterpret_cast<uint4 *>(dst) = make_uint4(w[k][0], w[k][1], w[k][2], w[k][3]);
            }
          }
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&bk->qbar_ready));
        }
        // ---------------- pass 1: thread = ranking row.  Two row tiles: group g owns tile g of every key
        // tile; one row tile: the groups take alternate key tiles
        const bool two = T.nrt == 2;
        const int my_row = (two ? group * 128 : 0) + lrow;             // row of the pair
        const bool row_ok = my_row < T.nrows;
        const bool warp_rows = (two ? group * 128 : 0) + quarter * 32 < T.nrows;
        const int p_i = T.R0 + my_row;
        const bool row_vis = T.use_soft && p_i >= d.v0 && p_i < v_end;
        float m = -INFINITY, l = 0.f;
        for (int t = 0; t < T.n_kt; ++t, ++g) {
          const int hh = g & 1;
          const bool mine = two || hh == group;
          const int j0 = t * 128;
          const bool fast = (j0 + 127 <= T.R0 + (two ? group * 128 : 0));
          const bool stage_soft = mine && T.use_soft && !fast;
          if (stage_soft) {
            const int j = j0 + lrow;
            soft[lrow] = (j >= d.v0 && j < v_end) ? __ldg(mlog + (j - d.v0)) * LOG2E_F : -INFINITY;
            group_bar_sync(group);
          }
          const uint32_t tlane = tlane0 + hh * 256 + (two ? group * 128 : 0);
          mbar_wait(smem_u32(&bk->acc_full[hh]), (g >> 1) & 1, wc);
          tc_fence_after();
          if (mine && warp_rows && !bk->abort_flag) {
#pragma unroll 1
            for (int c = 0; c < 128; c += 64) {
              uint32_t r[64];
              tmem_ld32p(tlane + c, r);
              tmem_ld32p(tlane + c + 32, r + 32);
              tmem_wait_ld();
              bool summed = false;
              if (fast && m > -INFINITY) {
                // every key admitted, no mask, and the row already has a reference maximum: add
                // exp2(dot * scale - m) without looking for a new maximum (a stale reference only scales
                // the sum; off_i = m + log2(l) comes out the same).  Should a term outgrow fp32's range
                // the chunk is done again below, with its true maximum as the new reference.
                float sm[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int e = 0; e < 64; ++e) sm[e & 7] += fast_exp2(fmaf(__uint_as_float(r[e]), scale, -m));
                const float cs = ((sm[0] + sm[1]) + (sm[2] + sm[3])) + ((sm[4] + sm[5]) + (sm[6] + sm[7]));
                if (cs < 1e30f) {
                  if (row_ok) l += cs;
                  summed = true;
                }
              }
              if (summed) {
              } else if (fast) {
                // every key admitted, no mask: max on the raw dot products (scale > 0), then
                // exp2(dot * scale - max) into eight independent partial sums
                float mx[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) mx[e] = __uint_as_float(r[e]);
#pragma unroll
                for (int e = 8; e < 64; ++e) mx[e & 7] = fmaxf(mx[e & 7], __uint_as_float(r[e]));
                const float cmax = fmaxf(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])),
                                         fmaxf(fmaxf(mx[4], mx[5]), fmaxf(mx[6], mx[7])));
                const float m_new = fmaxf(m, cmax * scale);
                if (row_ok) {
                  float sm[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
                  for (int e = 0; e < 64; ++e) sm[e & 7] += fast_exp2(fmaf(__uint_as_float(r[e]), scale, -m_new));
                  l = l * fast_exp2(m - m_new) +
                      (((sm[0] + sm[1]) + (sm[2] + sm[3])) + ((sm[4] + sm[5]) + (sm[6] + sm[7])));
                  m = m_new;
                }
              } else {
                // tile that crosses a row's own position: selects only, no branches.  `lim` =
                // last column of this chunk the row may attend to without the soft mask
                const int lim = p_i - (j0 + c);
                float mx[8] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY, -INFINITY, -INFINITY, -INFINITY, -INFINITY};
                if (!stage_soft) {
#pragma unroll
                  for (int e = 0; e < 64; ++e) {
                    const float x = (e <= lim) ? __uint_as_float(r[e]) * scale : -INFINITY;
                    r[e] = __float_as_uint(x);
                    mx[e & 7] = fmaxf(mx[e & 7], x);
                  }
                } else {
#pragma unroll
                  for (int e = 0; e < 64; ++e) {
                    const float sv = row_vis ? soft[c + e] : -INFINITY;
                    const float x = fmaf(__uint_as_float(r[e]), scale, (e <= lim) ? 0.f : sv);
                    r[e] = __float_as_uint(x);
                    mx[e & 7] = fmaxf(mx[e & 7], x);
                  }
                }
                const float cmax = fmaxf(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])),
                                         fmaxf(fmaxf(mx[4], mx[5]), fmaxf(mx[6], mx[7])));
                const float m_new = fmaxf(m, cmax);
                if (row_ok && m_new > -INFINITY) {
                  float sm[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
                  for (int e = 0; e < 64; ++e) sm[e & 7] += fast_exp2(__uint_as_float(r[e]) - m_new);
                  l = l * fast_exp2(m - m_new) +
                      (((sm[0] + sm[1]) + (sm[2] + sm[3])) + ((sm[4] + sm[5]) + (sm[6] + sm[7])));
                  m = m_new;
                }
              }
            }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&bk->acc_empty[hh]));
          if (stage_soft) group_bar_sync(group);   // soft[] is rewritten by this group's next masked tile
        }
        // off_i = max_i + log2(sum_i), so that exp2(x - off_i) = exp2(x - max_i) / sum_i.  With one row
        // tile the two groups saw disjoint key tiles: their (max, sum) per row are merged first
        if (two) {
          bk->off[my_row] = row_ok ? (m + __log2f(l)) : INFINITY;
          epi_bar_sync();
        } else {
          epi_bar_sync();                           // group 0 is past its last use of soft[1] and off[128..]
          if (group == 1) { pm[lrow] = m; pl[lrow] = l; }
          epi_bar_sync();
          if (group == 0) {
            const float m1 = pm[lrow], l1 = pl[lrow];
            const float mm = fmaxf(m, m1);
            float ll = 0.f;
            if (m > -INFINITY) ll += l * fast_exp2(m - mm);
            if (m1 > -INFINITY) ll += l1 * fast_exp2(m1 - mm);
            bk->off[lrow] = row_ok ? (mm + __log2f(ll)) : INFINITY;
          }
          epi_bar_sync();
        }
        // ---------------- pass 2: thread = key; the groups take alternate visual key tiles
        for (int u = 0; u < T.n_p2; ++u, ++g) {
          const int hh = g & 1;
          const bool mine = hh == group;
          const int t = T.t_hi - u, j0 = t * 128;
          const int j = j0 + lrow;
          const bool key_ok = j >= d.v0 && j < v_end;
          const bool fast = (j0 + 127 <= T.R0);
          const bool warp_keys = (j0 + quarter * 32 + 31 >= d.v0) && (j0 + quarter * 32 < v_end);
          const float soft_j = (mine && T.use_soft && key_ok) ? __ldg(mlog + (j - d.v0)) * LOG2E_F : -INFINITY;
          const uint32_t tlane = tlane0 + hh * 256;
          mbar_wait(smem_u32(&bk->acc_full[hh]), (g >> 1) & 1, wc);
          tc_fence_after();
          if (mine && warp_keys && !bk->abort_flag) {
            float sm[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
            for (int c = 0; c < T.n2; c += 32) {
              uint32_t r[32];
              const bool full = c + 32 <= T.n2;       // n2 is a multiple of 16: the last chunk may be half
              if (full) tmem_ld32p(tlane + c, r);
              else {
                tmem_ld16p(tlane + c, r);
#pragma unroll
                for (int e = 16; e < 32; ++e) r[e] = 0u;
              }
              tmem_wait_ld();
              // rows past the pair's end have off = +inf (every entry up to the next multiple of 128 is
              // written), so their terms vanish; four offsets per shared-memory load
              float o32[32];
#pragma unroll
              for (int e = 0; e < 32; e += 4)
                *reinterpret_cast<float4 *>(o32 + e) = *reinterpret_cast<const float4 *>(bk->off + c + e);
              if (fast) {
#pragma unroll
                for (int e = 0; e < 32; ++e) sm[e & 7] += fast_exp2(fmaf(__uint_as_float(r[e]), scale, -o32[e]));
              } else {
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                  const int p = T.R0 + c + e;
                  const float o = o32[e];
                  const float above = (p >= d.v0 && p < v_end) ? soft_j : -INFINITY;
                  const float add = (j <= p) ? 0.f : above;
                  sm[e & 7] += fast_exp2(fmaf(__uint_as_float(r[e]), scale, add) - o);
                }
              }
            }
            if (key_ok) {
              const float sum = ((sm[0] + sm[1]) + (sm[2] + sm[3])) + ((sm[4] + sm[5]) + (sm[6] + sm[7]));
              // the first row pair initialises the slots it covers; later row pairs add
              if (rp == 0) part[j - d.v0] = sum;
              else part[j - d.v0] += sum;
            }
            if (with_mass && rp == 0) {
              // columns n2 .. n2 + 2: the three pieces of the summed query against this key
              uint32_t r[16];
              tmem_ld16(tlane + T.n2, r);
              tmem_wait_ld();
              if (key_ok)
                a.mass_heads[((size_t)b * a.H + h) * a.max_vis + (j - d.v0)] =
                    (__uint_as_float(r[0]) + __uint_as_float(r[1])) + __uint_as_float(r[2]);
            }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&bk->acc_empty[hh]));
        }
        epi_bar_sync();   // off[] is rewritten by the next row pair; its sums are visible to the next pair's adds
      }
    }
    __threadfence();
  }

  // ---------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, SC_TMEM_COLS);
  }
  // the block that leaves last puts the work counters back to zero for the next launch (every block
  // has drawn its last item by then: a block only gets here after a draw past the end)
  if (threadIdx.x == 0) {
    const unsigned int done = atomicAdd(a.work + 1, 1u);
    if (done == gridDim.x - 1) {
      a.work[0] = 0u;
      a.work[1] = 0u;
      __threadfence();
    }
  }
}

// r_j = (1 / (H |R|)) sum_h partial[b, h, j]: the mean over heads and ranking rows of the Eq. 4
// probabilities, heads added in ascending order.  grid (ceil(max_vis / 256), B).
__global__ void __launch_bounds__(256)
head_sum_kernel(const SampleDesc *__restrict__ desc, int H, int max_vis,
                const float *__restrict__ partial, float *__restrict__ rank_score) {
  pdl_enter();
  const int b = blockIdx.y;
  const SampleDesc d = desc[b];
  const int j = blockIdx.x * 256 + threadIdx.x;
  if (j >= max_vis) return;
  float tot = 0.f;
  if (d.valid && j < d.nv) {
    const float *p = partial + (size_t)b * H * max_vis + j;
    int hh = 0;
    for (; hh + 8 <= H; hh += 8) {
      float v[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] = __ldcg(p + (size_t)(hh + e) * max_vis);
#pragma unroll
      for (int e = 0; e < 8; ++e) tot += v[e];
    }
    for (; hh < H; ++hh) tot += __ldcg(p + (size_t)hh * max_vis);
    tot *= 1.0f / ((float)H * (float)d.nr);
  }
  rank_score[(size_t)b * max_vis + j] = tot;
}

// =======================================================================================
// sim_kernel
//
// One block per (128 rows, sample, slice of the hidden dimension).  D = Row_tile Kept^T
// with M = 128 rows (see "row operand" below), N = n_tile kept slots per accumulator, K = this block's slice of
// the hidden size in steps of 64.
//   row operand:    either the dropped rows alone, fetched where they lie in `hidden` by the gather
//                   warps (16-byte asynchronous copies, written in the 128-byte-swizzled layout the
//                   tiled copies produce), so that only rows whose result is used are multiplied; or
//                   every visual row by plain tiled copies, the kept rows' results being thrown away.
//                   The gather path moves at most ~23 bytes per clock and SM (the load/store unit's
//                   requests in flight; a gather copy of four rows per instruction through the
//                   tensor-map unit managed a third of that), the tiled path twice as much, so the host
//                   gathers only when the kept rows are a large share of the span (two fifths or more).
// While the first
// accumulator is being built the epilogue warps also read every row tile from shared memory and
// add up the squares (the row norms of Sec. 4.2's cosine similarity).
//   one slice:      the epilogue scales column s by 1/||kept_s||, keeps the running maximum
//                   and the first slot attaining it, and writes, for rows that were dropped,
//                   the slot (or -1 if the cosine similarity is not above the threshold) and
//                   the similarity.
//   several slices: (small problems, to fill the machine) every block stores its partial dot
//                   products and partial squared norms; the block that finishes last for the
//                   row tile adds the slices in slice order and does the same epilogue.
// Rows past the last dropped token (the ragged tail of the last tile) repeat that token and are
// not written.  The block that finishes a sample's last row tile groups the dropped tokens by
// destination.
//   one pass:       (a.wide, when all kept slots fit the 512 tensor-memory columns) the accumulators of
//                   all slot tiles are live at once and a stage is one 64-column block of the rows
//                   plus the matching block of EVERY slot tile, so the visual rows are read from
//                   memory once instead of once per slot tile.
//   slot groups:    (a.groups > 1, one-pass layout, blockIdx.x = row tile * groups + group) more kept slots than tensor memory
//                   holds at once: every block takes one group of slot tiles in ONE pass over the hidden
//                   dimension and publishes its rows' best (value, slot); the block that finishes a row
//                   tile last takes the maximum over the groups (lowest slot among equals).  The blocks
//                   of a row tile are neighbours in launch order and stream the same rows at the same
//                   time, so the rows come from memory once and from L2 afterwards -- several passes in
//                   one block read them from memory every time, because the rows of all resident
//                   blocks together do not fit L2.
//   matrix mode:    (a.smat set) the row operand is the dense kept-row array too, and
//                   the epilogue writes the whole keep_k x keep_k cosine matrix of the sample,
//                   S[p][q] = <h_p, h_q> * (1/||h_p|| * 1/||h_q||), for the routing inside the
//                   kept set; `tmap_h` is then a map of the kept rows with a 128-row box (plain
//                   tiled copies, no gather).
// =======================================================================================
#ifndef SIM_GWARPS_N
#define SIM_GWARPS_N 4
#endif
constexpr int SIM_GWARPS = SIM_GWARPS_N;                // gather warps
constexpr int SIM_THREADS = 192 + 32 * SIM_GWARPS;      // copy warp, MMA warp, four epilogue warps, the gather warps
constexpr int SIM_A_BYTES = 128 * 128;           // 128 rows x 64 bf16
constexpr int SIM_BOOK_BYTES = 2048;
constexpr uint32_t SIM_TMEM_COLS = 512;
constexpr int SIM_MAX_STAGES = 8;

struct SimArgs {
  const SampleDesc *desc;
  int D, max_vis, keep_k, n_tile, n_nt, stages, splits, max_mt;
  int wide;                  // 1: one pass, all slot tiles' accumulators live at once
  int groups;                // > 1: slot tiles dealt to `groups` blocks per row tile (n_nt counts one group's tiles)
  int cluster;               // 1: the `splits` slices of a row tile form a thread-block cluster (grid z) and add their
                             // partial products through distributed shared memory instead of `part`
  uint32_t tmem_cols;        // power of two >= 2 * n_tile: two accumulators
  float threshold;
  const int32_t *drop_idx;   // [B, max_vis-keep_k] dropped tokens, ascending: the row operand is gathered from them;
                             // nullptr: the row operand is every visual row (tiled copies), kept rows' results unused
  const int32_t *role;       // [B, max_vis] kept slot / -(dropped position + 1) of every visual token (all-rows form)
  const int32_t *drop_all;   // [B, max_vis-keep_k] the dropped tokens whatever the form (for member_meta), or nullptr
  const __nv_bfloat16 *hidden;   // [tokens, D] (the gather warps read the dropped rows from here)
  const float *kept_inv;     // [B*keep_k]   1/||kept row||, 0 for a zero row
  int32_t *assign;           // [B, max_vis-keep_k]
  float *best_sim;           // [B, max_vis-keep_k] or nullptr
  int32_t *seg;              // [B, keep_k+1]       CSR of assign, built by the last block of a sample
  int32_t *members;          // [B, max_vis-keep_k]
  unsigned int *counters;    // [B]            finished row tiles per sample
  unsigned int *tile_counters;  // [B, max_mt] finished slices per row tile
  float *part;               // [B, max_mt, splits, keep_k, 128] partial dot products (several slices only)
  float *ss_part;            // [B, max_mt, splits, 128]         partial squared norms
  float *smat;               // [B, keep_k, keep_k] or nullptr: matrix mode
  const float *salience;     // [B, max_vis] or nullptr: with member_meta, the merge weights the grouping copies
  int2 *member_meta;         // [B, max_vis-keep_k] or nullptr (see csr_block)
  uint32_t *status;
  long long wait_limit;      // clock cycles a wait may take before the block gives up
};

struct SimBook {
  uint64_t full[SIM_MAX_STAGES], empty[SIM_MAX_STAGES], acc_full[2], acc_empty[2], mma_done;
  uint32_t tmem_base;
  int abort_flag;
  int is_last;
  int skip;                  // cluster form: an earlier similarity kernel of this call gave up
  int scan[33];
  int rows[128];             // packed row of each of the tile's dropped tokens (main mode)
};

static_assert(sizeof(SimBook) <= SIM_BOOK_BYTES, "similarity kernel bookkeeping exceeds its shared-memory slot");

__device__ __forceinline__ void mbar_arrive_n(uint32_t bar, uint32_t n) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(n) : "memory");
}

constexpr int SIM_THREADS_TILED = 192;                  // without gather warps: two such blocks fit an SM

template <bool GATHER>
__global__ void __launch_bounds__(GATHER ? SIM_THREADS : SIM_THREADS_TILED, 1)
sim_kernel(const __grid_constant__ CUtensorMap tmap_h, const __grid_constant__ CUtensorMap tmap_kept,
           SimArgs a) {
  // (the wait for the preceding kernel comes after this block's set-up, which reads nothing that kernel
  // writes: descriptors and status word are older; barriers, tensor memory and the cluster's first barrier
  // are then ready when the kept rows are)
  extern __shared__ uint8_t smem_raw[];
  // the groups of a row tile are neighbours in launch order (blockIdx.x = row tile * groups + group)
  const int mt = blockIdx.x / a.groups, b = blockIdx.y;
  const int z = blockIdx.z;                              // slice of the hidden dimension
  const int gz = blockIdx.x - mt * a.groups;             // group of slot tiles
  const int tile0 = gz * a.n_nt;                         // first slot tile of this block
  const SampleDesc d = a.desc[b];
  if (!d.valid) return;
  const int nd = d.nv - a.keep_k;                        // dropped tokens of this sample
  constexpr bool gather = GATHER;                        // a.drop_idx given, not matrix mode
  const int n_rows = a.smat ? a.keep_k : (gather ? nd : d.nv);   // rows of the row operand
  if (mt * 128 >= max(n_rows, 1)) return;
  // (in the cluster form the blocks of a cluster must leave together: decided below, by the cluster's first block)
  if (!a.cluster && (*reinterpret_cast<volatile uint32_t *>(a.status) & STATUS_SIM_TIMEOUT)) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
  // a stage holds two adjacent 64-column blocks (256 contiguous bytes of every row):
  // [ rows, block 0 | rows, block 1 | kept, block 0 | kept, block 1 ]
  const int b_bytes = a.n_tile * 128;
  const int stage_bytes = a.wide ? SIM_A_BYTES + a.n_nt * b_bytes : 2 * (SIM_A_BYTES + b_bytes);
  SimBook *bk = reinterpret_cast<SimBook *>(base_ptr + (size_t)a.stages * stage_bytes);
  if (n_rows <= 0) {
    // nothing was dropped in this sample: only the (empty) grouping has to be written
    pdl_enter();
    if (z == 0 && gz == 0) csr_block(d, b, a.max_vis, a.keep_k, a.assign, a.seg, a.members, reinterpret_cast<int *>(base_ptr), bk->scan, a.drop_all, a.salience, a.member_meta);
    return;
  }

  if (threadIdx.x == 0) {
    for (int s = 0; s < a.stages; ++s) {
      mbar_init(smem_u32(&bk->full[s]), GATHER ? 1 + 32 * SIM_GWARPS : 1);  // the copy warp's announcement (+ every gather thread)
      mbar_init(smem_u32(&bk->empty[s]), 5);      // the MMAs that read the stage + four epilogue warps
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&bk->acc_full[i]), 1);
      mbar_init(smem_u32(&bk->acc_empty[i]), 4);
    }
    mbar_init(smem_u32(&bk->mma_done), 1);
    bk->abort_flag = 0;
    bk->is_last = 0;
    bk->skip = (*reinterpret_cast<volatile uint32_t *>(a.status) & STATUS_SIM_TIMEOUT) ? 1 : 0;
    fence_barrier_init();
  }
  if (a.cluster) {
    cluster_sync_all();
    if (ld_cluster_s32(cluster_map(smem_u32(&bk->skip), 0))) {
      cluster_sync_all();                                // the first block's shared memory has been read by all
      return;
    }
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&bk->tmem_base), a.tmem_cols);
    tmem_relinquish();
    tc_fence_before();
  }
  __syncthreads();
  tc_fence_after();
  pdl_enter();
  const uint32_t tmem_base = bk->tmem_base;
  WaitCtx wc{&bk->abort_flag, a.status, STATUS_SIM_TIMEOUT, a.wait_limit};
  // cluster form, in the tile ring once it is free: this slice's partial products [keep_k][128]; per quarter
  // of this block's share of the slots the rows' best (value [4][128], slot [4][128]); and, filled by all
  // blocks in the cluster's first block, every slice's partial squared norms and every block's best
  // (value, slot) ([splits][128] each)
  const int cl_per = (a.keep_k + a.splits - 1) / a.splits;
  float *cl_p = reinterpret_cast<float *>(base_ptr);
  float *cl_wv = cl_p + (size_t)a.keep_k * 128;
  int *cl_ws = reinterpret_cast<int *>(cl_wv + 4 * 128);
  float *cl_ss = reinterpret_cast<float *>(cl_ws + 4 * 128);
  float *cl_bv = cl_ss + a.splits * 128;
  int *cl_bs = reinterpret_cast<int *>(cl_bv + a.splits * 128);
  // steps of this slice: 128 columns each, or 64 in the one-pass layout
  const int n_kb = a.wide ? (a.D / 64) / a.splits : (a.D / 128) / a.splits;
  const int kb0 = z * n_kb;
  const int total_it = a.wide ? n_kb : a.n_nt * n_kb;

  if (warp == 0) {
    // ---- copy warp: the kept-row tiles (and, in matrix mode, the row operand) by tiled copies
    if (lane == 0) {
      tma_prefetch_desc(&tmap_h);
      tma_prefetch_desc(&tmap_kept);
      const int row_b = b * a.keep_k;
      // tiled row operand: rows of the dense kept array (matrix mode) or of the image span
      const int row_a = a.smat ? row_b + mt * 128 : d.row0 + d.v0 + mt * 128;
      const int tx_bytes = gather ? stage_bytes - (a.wide ? 1 : 2) * SIM_A_BYTES : stage_bytes;
      const int rot = (mt * 5 + b * 3) % n_kb;
      int issued = 0;
      for (int it = 0; it < total_it; ++it) {
        // every block walks its k-blocks from a different starting point, so that at any moment
        // the blocks read different 128-byte columns of the rows and spread over the memory channels
        const int s = it % a.stages, nt = it / n_kb, kb = kb0 + (it - nt * n_kb + rot) % n_kb;
        const uint32_t full = smem_u32(&bk->full[s]);
        if (it >= a.stages) mbar_wait(smem_u32(&bk->empty[s]), ((it / a.stages) - 1) & 1, wc);
        if (bk->abort_flag) break;
        const uint32_t dst = base + s * stage_bytes;
        mbar_expect_tx(full, tx_bytes);
        if (a.wide) {
          if (!gather) tma_load_2d(dst, &tmap_h, full, kb * 64, row_a);
          for (int t = 0; t < a.n_nt; ++t)
            tma_load_2d(dst + SIM_A_BYTES + t * b_bytes, &tmap_kept, full, kb * 64, row_b + (tile0 + t) * a.n_tile);
        } else {
          if (!gather) {
            tma_load_2d(dst, &tmap_h, full, kb * 128, row_a);
            tma_load_2d(dst + SIM_A_BYTES, &tmap_h, full, kb * 128 + 64, row_a);
          }
          tma_load_2d(dst + 2 * SIM_A_BYTES, &tmap_kept, full, kb * 128, row_b + nt * a.n_tile);
          tma_load_2d(dst + 2 * SIM_A_BYTES + b_bytes, &tmap_kept, full, kb * 128 + 64, row_b + nt * a.n_tile);
        }
        issued = it + 1;
      }
      // drain: the last fill of every stage must have landed before the block leaves
      for (int s = 0; s < a.stages; ++s) {
        if (issued > s) {
          const int last = ((issued - 1 - s) / a.stages) * a.stages + s;
          // after an abort the gather warps may not have handed their part of the stage over, so the
          // barrier may never complete: the tiled copies themselves land within microseconds
          mbar_wait_drain(smem_u32(&bk->full[s]), (last / a.stages) & 1, bk->abort_flag ? 400000LL : TC_WAIT_LIMIT);
        }
      }
    }
    __syncwarp();
    if (a.cluster) { cluster_sync_all(); cluster_sync_all(); }   // the two barriers of the epilogue warps' reduction
  } else if (warp >= 6) {
    // ---- gather warps (main mode): warp g fetches its share of the tile's rows (128 / SIM_GWARPS hidden rows
    // of dropped tokens), one stage's columns at a time.  A warp instruction covers whole rows
    // (2 rows x 256 bytes, or 4 rows x 128 bytes in the one-pass layout), each lane one 16-byte chunk,
    // written where the tiled copies would put it: row r of a 64-column block is 128 bytes at
    // r * 128, its chunk c at position c ^ (r & 7).  Every lane's copies of a stage arrive on the stage's
    // barrier by themselves when they have landed, so the warps only ever wait for a free stage.  Few
    // threads with many copies each: every thread costs the barrier one arrival per stage, and 128
    // arrivals per stage were measured to hold the whole pipeline back.
    if (gather) {
      const int g = warp - 6;
      constexpr int RW = 128 / SIM_GWARPS;                // rows of the tile per gather warp
      const int cpr = a.wide ? 8 : 16;                   // 16-byte chunks per row and stage
      const int c = lane & (cpr - 1), rsub = lane / cpr, rpi = 32 / cpr, n_i = RW / rpi;
      const int32_t *drop_b = a.drop_idx + (size_t)b * (a.max_vis - a.keep_k);
      for (int r = g * RW + lane; r < (g + 1) * RW; r += 32) {
        const int dp = min(mt * 128 + r, nd - 1);        // the ragged tail repeats the last dropped token
        bk->rows[r] = d.row0 + d.v0 + min(max(__ldg(drop_b + dp), 0), d.nv - 1);
      }
      __syncwarp();
      const uint8_t *hid = reinterpret_cast<const uint8_t *>(a.hidden) + (size_t)c * 16;
      const size_t pitch = (size_t)a.D * 2;
      const uint32_t dst_c = (uint32_t)((c >> 3) * SIM_A_BYTES);
      const int stage_cols_bytes = a.wide ? 128 : 256;
      const int rot = (mt * 5 + b * 3) % n_kb;
      for (int it = 0; it < total_it; ++it) {
        const int s = it % a.stages, nt = it / n_kb, kb = kb0 + (it - nt * n_kb + rot) % n_kb;
        int go = 1;
        if (lane == 0) {
          if (it >= a.stages) mbar_wait(smem_u32(&bk->empty[s]), ((it / a.stages) - 1) & 1, wc);
          go = bk->abort_flag ? 0 : 1;
        }
        go = __shfl_sync(0xffffffffu, go, 0);
        if (!go) break;
        const uint32_t dst = base + s * stage_bytes + dst_c;
        const uint8_t *src = hid + (size_t)kb * stage_cols_bytes;
#pragma unroll 8
        for (int i = 0; i < n_i; ++i) {
          const int r = g * RW + i * rpi + rsub;
          cp_async16(dst + r * 128 + (((c & 7) ^ (r & 7)) << 4), src + (size_t)bk->rows[r] * pitch);
        }
        cp_async_arrive_on(smem_u32(&bk->full[s]));       // this lane's share of the stage, once it has landed
      }
      cp_async_commit();
      cp_async_wait<0>();                                 // nothing of this thread's is in flight when the block leaves
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(128, a.n_tile);
      int it = 0;
      if (a.wide) {
        for (int kb = 0; kb < n_kb; ++kb) {
          const int s = kb % a.stages;
          mbar_wait(smem_u32(&bk->full[s]), (kb / a.stages) & 1, wc);
          fence_proxy_async();       // the gathered rows were written by ordinary asynchronous copies
          tc_fence_after();
          if (!bk->abort_flag) {
            const uint32_t sa = base + s * stage_bytes, sb = sa + SIM_A_BYTES;
            for (int t = 0; t < a.n_nt; ++t)
#pragma unroll
              for (int kk = 0; kk < 4; ++kk)
                tc_mma_bf16(tmem_base + t * a.n_tile, umma_desc_sw128(sa + kk * 32),
                            umma_desc_sw128(sb + t * b_bytes + kk * 32), idesc, (kb > 0 || kk > 0) ? 1u : 0u);
            tc_commit(smem_u32(&bk->empty[s]));
            if (a.smat) mbar_arrive_n(smem_u32(&bk->empty[s]), 4);
          }
        }
        if (!bk->abort_flag) tc_commit(smem_u32(&bk->acc_full[0]));
      }
      for (int nt = 0; nt < (a.wide ? 0 : a.n_nt); ++nt) {
        const int buf = nt & 1;
        if (nt >= 2) mbar_wait(smem_u32(&bk->acc_empty[buf]), ((nt >> 1) - 1) & 1, wc);
        const uint32_t dcol = tmem_base + buf * (a.tmem_cols >> 1);
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const int s = it % a.stages;
          mbar_wait(smem_u32(&bk->full[s]), (it / a.stages) & 1, wc);
          fence_proxy_async();
          tc_fence_after();
          if (!bk->abort_flag) {
            const uint32_t sa = base + s * stage_bytes, sb = sa + 2 * SIM_A_BYTES;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
              tc_mma_bf16(dcol, umma_desc_sw128(sa + (kk >> 2) * SIM_A_BYTES + (kk & 3) * 32),
                          umma_desc_sw128(sb + (kk >> 2) * b_bytes + (kk & 3) * 32), idesc,
                          (kb > 0 || kk > 0) ? 1u : 0u);
            tc_commit(smem_u32(&bk->empty[s]));
            // after the first accumulator the epilogue warps no longer read the stages
            if (nt > 0 || a.smat) mbar_arrive_n(smem_u32(&bk->empty[s]), 4);
          }
        }
        if (!bk->abort_flag) tc_commit(smem_u32(&bk->acc_full[buf]));
      }
      // every MMA this thread issued has completed before tensor memory is given back: after an abort the
      // epilogue warps no longer wait for the accumulators, so nothing else would hold the block until then
      tc_commit(smem_u32(&bk->mma_done));
      mbar_wait_drain(smem_u32(&bk->mma_done), 0, TC_WAIT_LIMIT);
    }
    __syncwarp();
    if (a.cluster) { cluster_sync_all(); cluster_sync_all(); }
  } else {
    const int quarter = warp & 3;
    const int lrow = quarter * 32 + lane;
    const int v = mt * 128 + lrow;                       // this thread's row: dropped position (kept slot in matrix mode)
    const float *kinv = a.kept_inv + (size_t)b * a.keep_k;
    // ---- squared norm of this thread's row, from the row tiles of the first accumulator's pass.
    // Row r of a tile is 128 bytes; its 16-byte chunk c sits at chunk position c ^ (r & 7).
    float ssq[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int it = 0; it < (a.smat ? 0 : n_kb); ++it) {
      const int s = it % a.stages;
      mbar_wait(smem_u32(&bk->full[s]), (it / a.stages) & 1, wc);
      if (!bk->abort_flag) {
#pragma unroll
        for (int hb = 0; hb < 2; ++hb) {
          if (hb == 1 && a.wide) break;                  // one 64-column block of the rows per stage
          const uint4 *row = reinterpret_cast<const uint4 *>(base_ptr + (size_t)s * stage_bytes +
                                                             hb * SIM_A_BYTES + lrow * 128);
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            const uint4 x = row[c ^ (lrow & 7)];
            float f[8];
            unpack8(x, f);
#pragma unroll
            for (int e = 0; e < 8; ++e) ssq[c] = fmaf(f[e], f[e], ssq[c]);
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bk->empty[s]));
    }
    const float ss = ((ssq[0] + ssq[1]) + (ssq[2] + ssq[3])) + ((ssq[4] + ssq[5]) + (ssq[6] + ssq[7]));

    float best = -INFINITY;
    int best_slot = 0;
    float *part = nullptr;
    if (a.cluster) {
      // the four epilogue warps are done reading the row tiles for the norms: from here on the ring only
      // holds stages the MMAs still read, and those are complete once acc_full has been passed
      asm volatile("bar.sync 1, 128;" ::: "memory");
      part = cl_p;
    } else if (a.splits > 1) {
      const size_t tile = ((size_t)b * a.max_mt + mt) * a.splits + z;
      part = a.part + tile * (size_t)a.keep_k * 128;
      a.ss_part[tile * 128 + lrow] = ss;
    }
    for (int nt = 0; nt < a.n_nt; ++nt) {
      const int buf = a.wide ? 0 : (nt & 1);
      mbar_wait(smem_u32(&bk->acc_full[buf]), a.wide ? 0 : ((nt >> 1) & 1), wc);
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) +
                             (a.wide ? nt * a.n_tile : buf * (a.tmem_cols >> 1));
      const int slot0 = (tile0 + nt) * a.n_tile;
      const int ncol = min(a.n_tile, a.keep_k - slot0);   // kept slots in this accumulator (none in a group's ragged end)
      int c0 = 0;
      if (!a.smat || part) {
        // 32 columns per tensor-memory wait while they last (see sim_pair_kernel)
#pragma unroll 1
        for (; c0 + 32 <= ncol; c0 += 32) {
          uint32_t r[32];
          tmem_ld32(taddr + c0, r);
          tmem_wait_ld();
          if (part) {
#pragma unroll
            for (int e = 0; e < 32; ++e) part[(size_t)(slot0 + c0 + e) * 128 + lrow] = __uint_as_float(r[e]);
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              const int slot = slot0 + c0 + e;
              const float val = __uint_as_float(r[e]) * __ldg(kinv + slot);
              if (val > best) { best = val; best_slot = slot; }
            }
          }
        }
      }
#pragma unroll 1
      for (int c = c0; c < ncol; c += 16) {
        uint32_t r[16];
        tmem_ld16(taddr + c, r);
        tmem_wait_ld();
        if (a.smat && !part) {
          if (v < a.keep_k && !bk->abort_flag) {
            const float inv_p = __ldg(kinv + v);
            float *srow = a.smat + ((size_t)b * a.keep_k + v) * a.keep_k + slot0 + c;
#pragma unroll
            for (int e = 0; e < 16; ++e)
              if (c + e < ncol) srow[e] = __uint_as_float(r[e]) * (inv_p * __ldg(kinv + slot0 + c + e));
          }
        } else if (part) {
#pragma unroll
          for (int e = 0; e < 16; ++e)
            if (c + e < ncol) part[(size_t)(slot0 + c + e) * 128 + lrow] = __uint_as_float(r[e]);
        } else {
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const int slot = slot0 + c + e;
            if (c + e < ncol) {
              const float val = __uint_as_float(r[e]) * __ldg(kinv + slot);
              if (val > best) { best = val; best_slot = slot; }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bk->acc_empty[buf]));
    }
    float ss_tot = ss;
    bool finalize = true;
    if (a.cluster) {
      // ---- the slices of this row tile are the blocks of one cluster.  Block r adds, in slice order, the
      // partial products of ITS share of the kept slots, read from every block's shared memory: warp q takes
      // every fourth slot of the share, a lane four neighbouring rows (one 16-byte load per slice).  The
      // warps' bests per row are merged (larger value, lower slot among equals), handed to the cluster's
      // first block, and that block takes the maximum over the blocks in ascending slots.
      const int rank = (int)cluster_cta_rank(), S = a.splits;
      st_cluster_f32(cluster_map(smem_u32(cl_ss), 0) + (uint32_t)(rank * 128 + lrow) * 4u, ss);
      cluster_sync_all();
      const int s_lo = min(a.keep_k, rank * cl_per), n_mine = min(a.keep_k, s_lo + cl_per) - s_lo;
      uint32_t pz[8];
#pragma unroll
      for (int zz = 0; zz < 8; ++zz)
        pz[zz] = cluster_map(smem_u32(cl_p), (uint32_t)min(zz, S - 1)) + (uint32_t)lane * 16u;
      float wb[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
      int wsl[4] = {0, 0, 0, 0};
      for (int i = quarter; i < n_mine; i += 4) {
        const int slot = s_lo + i;
        float4 x[8];
#pragma unroll
        for (int zz = 0; zz < 8; ++zz)
          if (zz < S) x[zz] = ld_cluster_v4f32(pz[zz] + (uint32_t)slot * 512u);
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int zz = 0; zz < 8; ++zz)
          if (zz < S) { acc[0] += x[zz].x; acc[1] += x[zz].y; acc[2] += x[zz].z; acc[3] += x[zz].w; }
        const float ks = __ldg(kinv + slot);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (a.smat) {
            const int vr = mt * 128 + lane * 4 + j;
            if (vr < a.keep_k && !bk->abort_flag)
              a.smat[((size_t)b * a.keep_k + vr) * a.keep_k + slot] = acc[j] * (__ldg(kinv + vr) * ks);
          } else {
            const float val = acc[j] * ks;
            if (val > wb[j]) { wb[j] = val; wsl[j] = slot; }
          }
        }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        cl_wv[quarter * 128 + lane * 4 + j] = wb[j];
        cl_ws[quarter * 128 + lane * 4 + j] = wsl[j];
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      for (int q2 = 0; q2 < 4; ++q2) {
        const float val = cl_wv[q2 * 128 + lrow];
        const int sl = cl_ws[q2 * 128 + lrow];
        if (val > best || (val == best && val > -INFINITY && sl < best_slot)) { best = val; best_slot = sl; }
      }
      st_cluster_f32(cluster_map(smem_u32(cl_bv), 0) + (uint32_t)(rank * 128 + lrow) * 4u, best);
      st_cluster_s32(cluster_map(smem_u32(cl_bs), 0) + (uint32_t)(rank * 128 + lrow) * 4u, best_slot);
      cluster_sync_all();
      finalize = rank == 0;
      if (finalize) {
        ss_tot = 0.f;
        for (int r2 = 0; r2 < S; ++r2) ss_tot += cl_ss[r2 * 128 + lrow];
        best = -INFINITY;
        best_slot = 0;
        for (int r2 = 0; r2 < S; ++r2) {                    // ascending slots: the first maximum stays
          const float val = cl_bv[r2 * 128 + lrow];
          if (val > best) { best = val; best_slot = cl_bs[r2 * 128 + lrow]; }
        }
      }
    } else if (a.splits > 1) {
      // publish this slice; the last slice to arrive for the row tile reduces all of them
      __threadfence();
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (warp == 2 && lane == 0) {
        unsigned int *cnt = a.tile_counters + (size_t)b * a.max_mt + mt;
        const unsigned int old = atomicAdd(cnt, 1u);
        bk->is_last = (old == (unsigned int)(a.splits - 1));
        if (bk->is_last) *cnt = 0u;
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      finalize = bk->is_last != 0;
      if (finalize) {
        __threadfence();
        const size_t tile0 = ((size_t)b * a.max_mt + mt) * a.splits;
        ss_tot = 0.f;
        for (int zz = 0; zz < a.splits; ++zz) ss_tot += __ldcg(a.ss_part + (tile0 + zz) * 128 + lrow);
        const float *p0 = a.part + tile0 * (size_t)a.keep_k * 128 + lrow;
        const size_t zstride = (size_t)a.keep_k * 128;
        for (int s0 = 0; s0 < a.keep_k; s0 += 16) {     // 16 slots x all slices in flight per thread
          float acc[16];
#pragma unroll
          for (int e = 0; e < 16; ++e) acc[e] = 0.f;
          for (int zz = 0; zz < a.splits; zz += 4) {    // 64 loads in flight per thread
            float x[4][16];
#pragma unroll
            for (int t = 0; t < 4; ++t)
#pragma unroll
              for (int e = 0; e < 16; ++e)
                x[t][e] = (zz + t < a.splits && s0 + e < a.keep_k)
                              ? __ldcg(p0 + (zz + t) * zstride + (size_t)(s0 + e) * 128) : 0.f;
#pragma unroll
            for (int t = 0; t < 4; ++t)
#pragma unroll
              for (int e = 0; e < 16; ++e) acc[e] += x[t][e];
          }
          if (a.smat) {
            if (v < a.keep_k && !bk->abort_flag) {
              const float inv_p = __ldg(kinv + v);
              float *srow = a.smat + ((size_t)b * a.keep_k + v) * a.keep_k + s0;
#pragma unroll
              for (int e = 0; e < 16; ++e)
                if (s0 + e < a.keep_k) srow[e] = acc[e] * (inv_p * __ldg(kinv + s0 + e));
            }
            continue;
          }
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const int slot = s0 + e;
            if (slot < a.keep_k) {
              const float val = acc[e] * __ldg(kinv + slot);
              if (val > best) { best = val; best_slot = slot; }
            }
          }
        }
      }
    }
    if (a.groups > 1) {
      // publish this group's best (value, slot); the last group to arrive for the row tile combines them
      const size_t tile = ((size_t)b * a.max_mt + mt) * a.groups;
      a.part[(tile + gz) * 256 + lrow] = best;
      reinterpret_cast<int *>(a.part)[(tile + gz) * 256 + 128 + lrow] = best_slot;
      __threadfence();
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (warp == 2 && lane == 0) {
        unsigned int *cnt = a.tile_counters + (size_t)b * a.max_mt + mt;
        const unsigned int old = atomicAdd(cnt, 1u);
        bk->is_last = (old == (unsigned int)(a.groups - 1));
        if (bk->is_last) *cnt = 0u;
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      finalize = bk->is_last != 0;
      if (finalize) {
        __threadfence();
        best = -INFINITY;
        best_slot = 0;
        for (int g2 = 0; g2 < a.groups; ++g2) {           // ascending slots: the first maximum stays
          const float val = __ldcg(a.part + (tile + g2) * 256 + lrow);
          const int slot = __ldcg(reinterpret_cast<const int *>(a.part) + (tile + g2) * 256 + 128 + lrow);
          if (val > best) { best = val; best_slot = slot; }
        }
      }
    }
    if (a.smat) finalize = false;
    // the dropped position of this thread's row: the row index itself, or looked up for a visual row
    int dp = -1;
    if (finalize && v < n_rows) {
      if (gather) dp = v;
      else { const int role = a.role[(size_t)b * a.max_vis + v]; dp = role < 0 ? -role - 1 : -1; }
    }
    if (dp >= 0 && dp < nd && !bk->abort_flag) {
      const bool zero_row = !(ss_tot >= 1e-24f);        // ||h|| < 1e-12: similarity 0 to every slot
      const float sim = zero_row ? 0.f : best * rsqrtf(ss_tot);
      const int slot = zero_row ? 0 : best_slot;
      const size_t o = (size_t)b * (a.max_vis - a.keep_k) + dp;
      a.assign[o] = (sim > a.threshold) ? slot : -1;
      if (a.best_sim) a.best_sim[o] = sim;
    }
    if (warp == 2 && lane == 0) bk->is_last = finalize ? 1 : 0;
    __threadfence();
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, a.tmem_cols);
  }
  if (a.smat) return;
  if (!bk->is_last && (a.splits > 1 || a.groups > 1)) return;     // a slice / group that did not finalize its row tile
  __syncthreads();
  // the block that finishes the sample's last row tile groups the dropped tokens by destination
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned int n_mt = (unsigned int)((n_rows + 127) / 128);
    const unsigned int old = atomicAdd(a.counters + b, 1u);
    bk->is_last = (old == n_mt - 1u);
    if (bk->is_last) a.counters[b] = 0u;
  }
  __syncthreads();
  if (!bk->is_last) return;
  __threadfence();
  // the tile ring is free: every copy has landed and every MMA that read it has completed
  csr_block(d, b, a.max_vis, a.keep_k, a.assign, a.seg, a.members, reinterpret_cast<int *>(base_ptr),
            bk->scan, a.drop_all, a.salience, a.member_meta);
}

// =======================================================================================
// sim_pair_kernel
//
// The all-rows form of sim_kernel for batches large enough to fill the machine without slicing the
// hidden dimension.  There the similarity kernel is bound by the bytes an SM can take in, not by the
// tensor pipe: measured, the tiled copies of a block deliver about 34 bytes per clock whatever the
// stage size or count (9.6 TB/s over 148 SMs), and a block of sim_kernel streams 128 rows and
// n_tile kept rows per 64 columns, (128 + n_tile) * 128 bytes for 128 * n_tile * 64 products.  This
// kernel multiplies TWO row tiles against each stage's kept rows -- (256 + n_tile) * 128 bytes for
// twice the products, 30 % fewer bytes per product at n_tile = 192; tensor memory (512 columns =
// 2 tiles x n_tile <= 256) allows no larger block.  (MMAs spanning a pair of CTAs, each CTA loading half
// of the kept rows, were built and measured: the half an SM reads from its partner's shared memory
// arrives through the same 34 bytes per clock, once per row tile, and the kernel ran 30 % slower.)
// It makes a single pass over the hidden dimension: the kept slots are dealt in groups of n_tile <= 256 to `groups` blocks per
// pair of row tiles (blockIdx.x = pair * groups + group).  The blocks of a pair are neighbours in
// launch order and stream the same rows at the same pace, so the rows come from memory once and
// from L2 for the other groups.  Accumulators: row tile t at tensor-memory column t * n_tile.
// Every block adds up its rows' squares from shared memory only if it is group 0, and publishes
// its rows' best (value, slot); the block that finishes a pair last takes the maximum over the
// groups (lowest slot among equals), looks up which rows were dropped and writes their assignment.
// The block that finishes a sample's last pair groups the dropped tokens by destination.
// Matrix mode (a.smat set): the row operand is the dense kept-row array too (`tmap_h` maps it with a 128-row box)
// and every block writes its 256 x n_tile piece of the sample's keep_k x keep_k cosine matrix; nothing else.
// =======================================================================================
constexpr int SIMP_THREADS = 320;                // copy warp, MMA warp, two groups of four epilogue warps

struct SimPairBook {
  uint64_t full[SIM_MAX_STAGES], empty[SIM_MAX_STAGES], acc_full, mma_done;
  uint32_t tmem_base;
  int abort_flag;
  int is_last;
  int scan[33];
};

static_assert(sizeof(SimPairBook) <= SIM_BOOK_BYTES, "pair kernel bookkeeping exceeds its shared-memory slot");

__global__ void __launch_bounds__(SIMP_THREADS, 1)
sim_pair_kernel(const __grid_constant__ CUtensorMap tmap_h, const __grid_constant__ CUtensorMap tmap_kept,
                SimArgs a) {
  // (the wait for the preceding kernel comes after the block's set-up, which reads nothing that kernel writes)
  extern __shared__ uint8_t smem_raw[];
  const int pr = blockIdx.x / a.groups, b = blockIdx.y;
  const int gz = blockIdx.x - pr * a.groups;             // group of kept slots
  const SampleDesc d = a.desc[b];
  if (!d.valid) return;
  const int nd = d.nv - a.keep_k;
  const int n_rows = a.smat ? a.keep_k : d.nv;           // matrix mode: the row operand is the dense kept-row array
  if (pr * 256 >= n_rows) return;
  if (*reinterpret_cast<volatile uint32_t *>(a.status) & STATUS_SIM_TIMEOUT) return;
  const bool two = pr * 256 + 128 < n_rows;              // the pair's second row tile holds visual rows
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
  // a stage: [ row tile 0 | row tile 1 | kept rows ] of one 64-column block
  const int b_bytes = a.n_tile * 128;
  const int stage_bytes = 2 * SIM_A_BYTES + b_bytes;
  SimPairBook *bk = reinterpret_cast<SimPairBook *>(base_ptr + (size_t)a.stages * stage_bytes);

  // the epilogue warps of group 0 read their row tile from the stages (for the row norms)
  const int n_readers = (gz == 0 && !a.smat) ? (two ? 8 : 4) : 0;   // (matrix mode takes the norms from kept_inv)
  if (threadIdx.x == 0) {
    for (int s = 0; s < a.stages; ++s) {
      mbar_init(smem_u32(&bk->full[s]), 1);
      mbar_init(smem_u32(&bk->empty[s]), 1 + n_readers);   // the MMAs that read the stage + the warps that do
    }
    mbar_init(smem_u32(&bk->acc_full), 1);
    mbar_init(smem_u32(&bk->mma_done), 1);
    bk->abort_flag = 0;
    bk->is_last = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&bk->tmem_base), a.tmem_cols);
    tmem_relinquish();
    tc_fence_before();
  }
  __syncthreads();
  tc_fence_after();
  pdl_enter();
  const uint32_t tmem_base = bk->tmem_base;
  WaitCtx wc{&bk->abort_flag, a.status, STATUS_SIM_TIMEOUT, a.wait_limit};
  const int n_kb = a.D / 64;
  // the groups of a pair walk the 64-column blocks from the same starting point (they share the rows
  // through L2); different pairs start elsewhere and spread over the memory channels
  const int rot = (pr * 5 + b * 3) % n_kb;

  if (warp == 0) {
    if (lane == 0) {
      tma_prefetch_desc(&tmap_h);
      tma_prefetch_desc(&tmap_kept);
      const int row_a = a.smat ? b * a.keep_k + pr * 256 : d.row0 + d.v0 + pr * 256;
      const int row_b = b * a.keep_k + gz * a.n_tile;
      const int tx_bytes = two ? stage_bytes : stage_bytes - SIM_A_BYTES;
      int issued = 0;
      for (int it = 0; it < n_kb; ++it) {
        const int s = it % a.stages, kb = (it + rot) % n_kb;
        const uint32_t full = smem_u32(&bk->full[s]);
        if (it >= a.stages) mbar_wait(smem_u32(&bk->empty[s]), ((it / a.stages) - 1) & 1, wc);
        if (bk->abort_flag) break;
        const uint32_t dst = base + s * stage_bytes;
        mbar_expect_tx(full, tx_bytes);
        tma_load_2d(dst, &tmap_h, full, kb * 64, row_a);
        if (two) tma_load_2d(dst + SIM_A_BYTES, &tmap_h, full, kb * 64, row_a + 128);
        tma_load_2d(dst + 2 * SIM_A_BYTES, &tmap_kept, full, kb * 64, row_b);
        issued = it + 1;
      }
      // drain: the last fill of every stage must have landed before the block leaves
      for (int s = 0; s < a.stages; ++s) {
        if (issued > s) {
          const int last = ((issued - 1 - s) / a.stages) * a.stages + s;
          mbar_wait_drain(smem_u32(&bk->full[s]), (last / a.stages) & 1, TC_WAIT_LIMIT);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(128, a.n_tile);
      const int n_t = two ? 2 : 1;
      for (int it = 0; it < n_kb; ++it) {
        const int s = it % a.stages;
        mbar_wait(smem_u32(&bk->full[s]), (it / a.stages) & 1, wc);
        tc_fence_after();
        if (!bk->abort_flag) {
          const uint32_t sa = base + s * stage_bytes, sb = sa + 2 * SIM_A_BYTES;
          for (int t = 0; t < n_t; ++t)
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              tc_mma_bf16(tmem_base + t * a.n_tile, umma_desc_sw128(sa + t * SIM_A_BYTES + kk * 32),
                          umma_desc_sw128(sb + kk * 32), idesc, (it > 0 || kk > 0) ? 1u : 0u);
          tc_commit(smem_u32(&bk->empty[s]));
        }
      }
      if (!bk->abort_flag) tc_commit(smem_u32(&bk->acc_full));
      // every MMA this thread issued has completed before tensor memory is given back
      tc_commit(smem_u32(&bk->mma_done));
      mbar_wait_drain(smem_u32(&bk->mma_done), 0, TC_WAIT_LIMIT);
    }
  } else {
    const int grp = (warp - 2) >> 2;                     // row tile of the pair
    const int quarter = warp & 3;                        // the tensor-memory lanes a warp may read
    const int lrow = quarter * 32 + lane;
    const int prow = grp * 128 + lrow;                   // row inside the pair
    const int v = pr * 256 + prow;                       // visual token
    const bool active = grp == 0 || two;
    const float *kinv = a.kept_inv + (size_t)b * a.keep_k;
    // ---- squared norm of this thread's row (group 0 only; the other groups just free the stages)
    float ssq[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    const bool norms = gz == 0 && active && !a.smat;
    for (int it = 0; it < (norms ? n_kb : 0); ++it) {
      const int s = it % a.stages;
      mbar_wait(smem_u32(&bk->full[s]), (it / a.stages) & 1, wc);
      if (!bk->abort_flag) {
        const uint4 *row = reinterpret_cast<const uint4 *>(base_ptr + (size_t)s * stage_bytes +
                                                           grp * SIM_A_BYTES + lrow * 128);
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const uint4 x = row[c ^ (lrow & 7)];
          float f[8];
          unpack8(x, f);
#pragma unroll
          for (int e = 0; e < 8; ++e) ssq[c] = fmaf(f[e], f[e], ssq[c]);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bk->empty[s]));
    }
    float ss = ((ssq[0] + ssq[1]) + (ssq[2] + ssq[3])) + ((ssq[4] + ssq[5]) + (ssq[6] + ssq[7]));

    float best = -INFINITY;
    int best_slot = 0;
    mbar_wait(smem_u32(&bk->acc_full), 0, wc);
    tc_fence_after();
    const int slot0 = gz * a.n_tile;
    const int ncol = max(0, min(a.n_tile, a.keep_k - slot0));
    if (active && !bk->abort_flag) {
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + grp * a.n_tile;
      const float inv_p = (a.smat && v < a.keep_k) ? __ldg(kinv + v) : 0.f;
      int c0 = 0;
      if (!a.smat) {
        // 32 columns per tensor-memory wait while they last: half as many waits on the path every block goes
        // through after its last MMA, which nothing overlaps (c4 881 -> 833 us; 64 columns per wait: the same)
#pragma unroll 1
        for (; c0 + 32 <= ncol; c0 += 32) {
          uint32_t r[32];
          tmem_ld32(taddr + c0, r);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const int slot = slot0 + c0 + e;
            const float val = __uint_as_float(r[e]) * __ldg(kinv + slot);
            if (val > best) { best = val; best_slot = slot; }
          }
        }
      }
#pragma unroll 1
      for (int c = c0; c < ncol; c += 16) {
        uint32_t r[16];
        tmem_ld16(taddr + c, r);
        tmem_wait_ld();
        if (a.smat) {
          // matrix mode: S[p][q] = <h_p, h_q> * (1/||h_p|| * 1/||h_q||) for this thread's kept row p
          if (v < a.keep_k) {
            float *srow = a.smat + ((size_t)b * a.keep_k + v) * a.keep_k + slot0 + c;
            if (c + 16 <= ncol && (reinterpret_cast<size_t>(srow) & 15) == 0) {
#pragma unroll
              for (int e = 0; e < 16; e += 4)         // 16-byte stores: a quarter of the store requests
                reinterpret_cast<float4 *>(srow)[e >> 2] =
                    make_float4(__uint_as_float(r[e]) * (inv_p * __ldg(kinv + slot0 + c + e)),
                                __uint_as_float(r[e + 1]) * (inv_p * __ldg(kinv + slot0 + c + e + 1)),
                                __uint_as_float(r[e + 2]) * (inv_p * __ldg(kinv + slot0 + c + e + 2)),
                                __uint_as_float(r[e + 3]) * (inv_p * __ldg(kinv + slot0 + c + e + 3)));
            } else {
#pragma unroll
              for (int e = 0; e < 16; ++e)
                if (c + e < ncol) srow[e] = __uint_as_float(r[e]) * (inv_p * __ldg(kinv + slot0 + c + e));
            }
          }
          continue;
        }
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const int slot = slot0 + c + e;
          if (c + e < ncol) {
            const float val = __uint_as_float(r[e]) * __ldg(kinv + slot);
            if (val > best) { best = val; best_slot = slot; }
          }
        }
      }
    }
    tc_fence_before();
    bool finalize = !a.smat;
    if (a.groups > 1 && !a.smat) {
      // per pair: [group][best of 256 rows | slot of 256 rows], then the 256 squared norms
      float *pp = a.part + ((size_t)b * a.max_mt + pr) * (size_t)(a.groups * 512 + 256);
      pp[gz * 512 + prow] = best;
      reinterpret_cast<int *>(pp)[gz * 512 + 256 + prow] = best_slot;
      if (gz == 0) pp[a.groups * 512 + prow] = ss;
      __threadfence();
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (warp == 2 && lane == 0) {
        unsigned int *cnt = a.tile_counters + (size_t)b * a.max_mt + pr;
        const unsigned int old = atomicAdd(cnt, 1u);
        bk->is_last = (old == (unsigned int)(a.groups - 1));
        if (bk->is_last) *cnt = 0u;
      }
      asm volatile("bar.sync 1, 256;" ::: "memory");
      finalize = bk->is_last != 0;
      if (finalize) {
        __threadfence();
        best = -INFINITY;
        best_slot = 0;
        for (int g2 = 0; g2 < a.groups; ++g2) {           // ascending slots: the first maximum stays
          const float val = __ldcg(pp + g2 * 512 + prow);
          const int slot = __ldcg(reinterpret_cast<const int *>(pp) + g2 * 512 + 256 + prow);
          if (val > best) { best = val; best_slot = slot; }
        }
        ss = __ldcg(pp + a.groups * 512 + prow);
      }
    }
    int dp = -1;
    if (finalize && v < n_rows) {
      const int role = a.role[(size_t)b * a.max_vis + v];
      dp = role < 0 ? -role - 1 : -1;
    }
    if (dp >= 0 && dp < nd && !bk->abort_flag) {
      const bool zero_row = !(ss >= 1e-24f);             // ||h|| < 1e-12: similarity 0 to every slot
      const float sim = zero_row ? 0.f : best * rsqrtf(ss);
      const int slot = zero_row ? 0 : best_slot;
      const size_t o = (size_t)b * (a.max_vis - a.keep_k) + dp;
      a.assign[o] = (sim > a.threshold) ? slot : -1;
      if (a.best_sim) a.best_sim[o] = sim;
    }
    if (warp == 2 && lane == 0) bk->is_last = finalize ? 1 : 0;
    __threadfence();
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, a.tmem_cols);
  }
  if (!bk->is_last) return;                              // a group that did not finalize its pair (or matrix mode)
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned int n_pr = (unsigned int)((n_rows + 255) / 256);
    const unsigned int old = atomicAdd(a.counters + b, 1u);
    bk->is_last = (old == n_pr - 1u);
    if (bk->is_last) a.counters[b] = 0u;
  }
  __syncthreads();
  if (!bk->is_last) return;
  __threadfence();
  csr_block(d, b, a.max_vis, a.keep_k, a.assign, a.seg, a.members, reinterpret_cast<int *>(base_ptr),
            bk->scan, a.drop_all, a.salience, a.member_meta);
}

}  // namespace asap
