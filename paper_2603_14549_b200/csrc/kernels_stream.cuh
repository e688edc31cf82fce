// The memory-bound and latency-bound kernels of the ASAP prune step:
//   prepare        device-side validation, per-sample descriptors, output row offsets
//   qsum           sum of the visual query rows                       (Eq. 1, summed over i first)
//   mass_salience  s_j, then s_hat_j and m_j                          (Eq. 1, Eq. 2, Eq. 3)
//   salience_from_heads  the same from per-head masses the score kernel produced
//   select         stable radix top-k of the ranking scores           (Fig. 3)
//   role_map       kept slot / dropped position of every visual token
//   kept_gather    kept rows gathered for the similarity GEMM, with their inverse norms (Sec. 4.2)
//   csr_block      dropped tokens grouped by destination slot (tail of the similarity kernel)
//   merge_compact  Eq. 5 and the hand-off of Fig. 3
//   gather_rows    KV-cache compaction with the row map of the hand-off
#pragma once

#include "common.cuh"

namespace asap {

// =======================================================================================
// prepare
// =======================================================================================
struct PrepareArgs {
  int32_t B, total_tokens, min_vis, max_vis, max_seq, max_rank, keep_k, out_capacity;
  int32_t write_desc;        // query-sum kernel only: its first block also runs prepare_block
  const int32_t *cu_seqlens, *vis_start, *vis_len, *text_start, *text_len, *rank_start, *rank_len;
  SampleDesc *desc;          // [B]
  int32_t *out_cu_seqlens;   // [B+1] or nullptr
  uint32_t *status;
};

// Descriptor of sequence b with its validity (out_row0 is filled in by prepare_block).
__device__ __forceinline__ SampleDesc make_desc(const PrepareArgs &a, int b) {
  const int lo = a.cu_seqlens[b], hi = a.cu_seqlens[b + 1];
  const int n = hi - lo;
  const int v0 = a.vis_start[b], nv = a.vis_len[b];
  const int t0 = a.text_start[b], tl = a.text_len[b];
  const int r0 = a.rank_start ? a.rank_start[b] : t0;
  const int nr = a.rank_len ? a.rank_len[b] : tl;
  bool ok = lo >= 0 && n > 0 && n <= a.max_seq && hi <= a.total_tokens;
  ok = ok && v0 >= 0 && nv >= a.min_vis && nv <= a.max_vis && v0 + nv <= n;
  ok = ok && tl >= 0 && t0 >= v0 + nv && t0 + tl <= n;
  ok = ok && r0 >= 0 && nr >= 1 && nr <= a.max_rank && r0 + nr <= n;
  ok = ok && a.keep_k <= nv;
  if (b == 0) ok = ok && lo == 0;
  if (b == a.B - 1) ok = ok && hi == a.total_tokens;
  SampleDesc d;
  d.row0 = lo; d.n = n; d.v0 = v0; d.nv = nv; d.r0 = r0; d.nr = nr; d.out_row0 = 0;
  d.valid = ok ? 1 : 0;
  return d;
}

// Run by one whole block: validates every sequence, writes the descriptors, the output row
// offsets and the status bits.
__device__ __forceinline__ void prepare_block(const PrepareArgs &a) {
  __shared__ int s_bad;
  if (threadIdx.x == 0) s_bad = 0;
  __syncthreads();
  for (int b = threadIdx.x; b < a.B; b += blockDim.x) {
    const SampleDesc d = make_desc(a, b);
    a.desc[b] = d;
    if (!d.valid) s_bad = 1;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int acc = 0;
    for (int b = 0; b < a.B; ++b) {
      a.desc[b].out_row0 = acc;
      if (a.out_cu_seqlens) a.out_cu_seqlens[b] = acc;
      if (a.desc[b].valid) acc += a.desc[b].n - a.desc[b].nv + a.keep_k;
    }
    if (a.out_cu_seqlens) a.out_cu_seqlens[a.B] = acc;
    uint32_t bits = 0;
    if (s_bad) bits |= STATUS_BAD_SAMPLE;
    if (acc > a.out_capacity) {
      bits |= STATUS_OUT_CAPACITY;
      for (int b = 0; b < a.B; ++b) a.desc[b].valid = 0;   // nothing may be written
    }
    if (bits) atomicOr(a.status, bits);
  }
  __syncthreads();
}

__global__ void prepare_kernel(PrepareArgs a) {
  pdl_enter();
  prepare_block(a);
}

// =======================================================================================
// qsum: qbar[b, c] = sum over visual rows i of q[i, c]   (fp32, fixed summation order)
// grid (chunks, column blocks, B); a block sums QSUM_ROWS rows of 2048 columns and the block
// that finishes last for (b, column block) adds the chunk partials in chunk order.
// =======================================================================================
constexpr int QSUM_ROWS = 32;
constexpr int QSUM_THREADS = 256;
constexpr int QSUM_COLS = QSUM_THREADS * 8;

__global__ void __launch_bounds__(QSUM_THREADS)
qsum_kernel(const __nv_bfloat16 *__restrict__ q, PrepareArgs pa, int D,
            int max_chunks, int rows_per_chunk /* a multiple of QSUM_ROWS */, float *__restrict__ partial /*[B, max_chunks, D]*/,
            float *__restrict__ qbar /*[B, D]*/, unsigned int *__restrict__ counters) {
  pdl_enter();
  const int b = blockIdx.z, cb = blockIdx.y, chunk = blockIdx.x;
  // When this is the first kernel of the step, block (0,0,0) also does the device-side validation
  // and writes the descriptors every later kernel reads; each block derives its own copy.
  if (pa.write_desc && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0) prepare_block(pa);
  const SampleDesc d = make_desc(pa, b);
  if (!d.valid) return;
  const int nchunks = (d.nv + rows_per_chunk - 1) / rows_per_chunk;
  if (chunk >= nchunks) return;
  const int col = cb * QSUM_COLS + threadIdx.x * 8;
  const bool active = col < D;
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  if (active) {
    const int r_lo = chunk * rows_per_chunk;
    const int r_hi = min(d.nv, r_lo + rows_per_chunk);
    const uint4 *base =
        reinterpret_cast<const uint4 *>(q + (size_t)(d.row0 + d.v0) * D + col);
    const size_t pitch = (size_t)D / 8;
    int r = r_lo;
    for (; r + 8 <= r_hi; r += 8) {       // eight independent 16-byte loads in flight per thread
      uint4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = __ldg(base + (size_t)(r + u) * pitch);
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        float f[8];
        unpack8(v[u], f);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] += f[e];
      }
    }
    for (; r < r_hi; ++r) {
      uint4 v = __ldg(base + (size_t)r * pitch);
      float f[8];
      unpack8(v, f);
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] += f[e];
    }
    float4 *dst = reinterpret_cast<float4 *>(partial + ((size_t)b * max_chunks + chunk) * D + col);
    dst[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
    dst[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
  }
  // last block for (b, cb) reduces the chunk partials
  __shared__ int s_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned int *c = counters + (size_t)b * gridDim.y + cb;
    unsigned int old = atomicAdd(c, 1u);
    s_last = (old == (unsigned int)(nchunks - 1));
    if (s_last) *c = 0u;   // ready for the next call
  }
  __syncthreads();
  if (!s_last || !active) return;
  __threadfence();
  float tot[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
  for (int c = 0; c < nchunks; ++c) {
    const float4 *src =
        reinterpret_cast<const float4 *>(partial + ((size_t)b * max_chunks + c) * D + col);
    float4 a0 = __ldcg(src), a1 = __ldcg(src + 1);
    tot[0] += a0.x; tot[1] += a0.y; tot[2] += a0.z; tot[3] += a0.w;
    tot[4] += a1.x; tot[5] += a1.y; tot[6] += a1.z; tot[7] += a1.w;
  }
  float4 *dst = reinterpret_cast<float4 *>(qbar + (size_t)b * D + col);
  dst[0] = make_float4(tot[0], tot[1], tot[2], tot[3]);
  dst[1] = make_float4(tot[4], tot[5], tot[6], tot[7]);
}

// =======================================================================================
// mass_salience: s_j = qbar . k_j / (H sqrt(d))  (Eq. 1 with the sum over queries taken first
// and the mean over heads folded in); the block that finishes last for a sample then does the
// min-max normalisation (Eq. 2) and the mask vector (Eq. 3).
// grid (row blocks, B); 8 warps x 4 rows each.
// =======================================================================================
constexpr int MASS_THREADS = 256;
constexpr int MASS_ROWS_PER_WARP = 4;
constexpr int MASS_ROWS = (MASS_THREADS / 32) * MASS_ROWS_PER_WARP;

__global__ void __launch_bounds__(MASS_THREADS)
mass_salience_kernel(const __nv_bfloat16 *__restrict__ k, const SampleDesc *__restrict__ desc,
                     int D, int max_vis, float scale, float lambda_max, float eps,
                     const float *__restrict__ qbar, float *__restrict__ mass,
                     float *__restrict__ salience, float *__restrict__ mask_log,
                     float *__restrict__ rank_score, unsigned int *__restrict__ counters) {
  pdl_enter();
  extern __shared__ float s_q[];   // [D]
  __shared__ float s_red[2 * (MASS_THREADS / 32)];
  __shared__ int s_last;
  const int b = blockIdx.y;
  const SampleDesc d = desc[b];
  float *mass_b = mass + (size_t)b * max_vis;
  if (!d.valid) {
    for (int j = blockIdx.x * MASS_THREADS + threadIdx.x; j < max_vis; j += gridDim.x * MASS_THREADS) {
      mass_b[j] = 0.f; salience[(size_t)b * max_vis + j] = 0.f; mask_log[(size_t)b * max_vis + j] = 0.f;
      rank_score[(size_t)b * max_vis + j] = 0.f;   // the score kernel skips the sample
    }
    return;
  }
  const int nblocks = (d.nv + MASS_ROWS - 1) / MASS_ROWS;
  if ((int)blockIdx.x >= nblocks) return;
  for (int c = threadIdx.x * 4; c < D; c += MASS_THREADS * 4)
    *reinterpret_cast<float4 *>(s_q + c) = __ldcg(reinterpret_cast<const float4 *>(qbar + (size_t)b * D + c));
  __syncthreads();

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int j0 = blockIdx.x * MASS_ROWS + warp * MASS_ROWS_PER_WARP;
  const int nvec = D / 8;
  float acc[MASS_ROWS_PER_WARP];
  const uint4 *rowp[MASS_ROWS_PER_WARP];
#pragma unroll
  for (int r = 0; r < MASS_ROWS_PER_WARP; ++r) {
    acc[r] = 0.f;
    const int j = min(j0 + r, d.nv - 1);   // clamp: duplicates are discarded below
    rowp[r] = reinterpret_cast<const uint4 *>(k + (size_t)(d.row0 + d.v0 + j) * D);
  }
  for (int v0 = lane; v0 < nvec; v0 += 64) {   // two vectors x four rows in flight per lane
    uint4 kv[2][MASS_ROWS_PER_WARP];
#pragma unroll
    for (int t = 0; t < 2; ++t)
#pragma unroll
      for (int r = 0; r < MASS_ROWS_PER_WARP; ++r)
        if (v0 + 32 * t < nvec) kv[t][r] = __ldg(rowp[r] + v0 + 32 * t);
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      const int v = v0 + 32 * t;
      if (v < nvec) {
        const float4 qa = *reinterpret_cast<const float4 *>(s_q + v * 8);
        const float4 qb = *reinterpret_cast<const float4 *>(s_q + v * 8 + 4);
#pragma unroll
        for (int r = 0; r < MASS_ROWS_PER_WARP; ++r) {
          float f[8];
          unpack8(kv[t][r], f);
          acc[r] += f[0] * qa.x + f[1] * qa.y + f[2] * qa.z + f[3] * qa.w + f[4] * qb.x + f[5] * qb.y +
                    f[6] * qb.z + f[7] * qb.w;
        }
      }
    }
  }
#pragma unroll
  for (int r = 0; r < MASS_ROWS_PER_WARP; ++r) {
    const float tot = warp_sum(acc[r]);
    if (lane == 0 && j0 + r < d.nv) mass_b[j0 + r] = tot * scale;
  }

  // ---- last block of the sample: Eq. 2 and Eq. 3 over the whole image span ----
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned int old = atomicAdd(counters + b, 1u);
    s_last = (old == (unsigned int)(nblocks - 1));
    if (s_last) counters[b] = 0u;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  float lo = INFINITY, hi = -INFINITY;
  for (int j = threadIdx.x; j < d.nv; j += MASS_THREADS) {
    const float s = __ldcg(mass_b + j);
    lo = fminf(lo, s); hi = fmaxf(hi, s);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
    hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
  }
  if (lane == 0) { s_red[warp] = lo; s_red[MASS_THREADS / 32 + warp] = hi; }
  __syncthreads();
  lo = s_red[0]; hi = s_red[MASS_THREADS / 32];
#pragma unroll
  for (int w = 1; w < MASS_THREADS / 32; ++w) {
    lo = fminf(lo, s_red[w]); hi = fmaxf(hi, s_red[MASS_THREADS / 32 + w]);
  }
  const float inv = 1.0f / ((hi - lo) + eps);
  float *sal_b = salience + (size_t)b * max_vis, *msk_b = mask_log + (size_t)b * max_vis;
  for (int j = threadIdx.x; j < max_vis; j += MASS_THREADS) {
    if (j < d.nv) {
      const float sh = (__ldcg(mass_b + j) - lo) * inv;
      sal_b[j] = sh;
      msk_b[j] = logf(fmaxf(lambda_max * sh, eps));
    } else {
      mass_b[j] = 0.f; sal_b[j] = 0.f; msk_b[j] = 0.f;
    }
  }
}

// =======================================================================================
// salience_from_heads: the tail of Eq. 1 and Eq. 2-3 when the per-head masses qbar^h . k_j^h were
// produced elsewhere (by the score kernel, from the key tiles it streams anyway).  One block per
// sample: s_j = scale * sum_h heads[b, h, j] (heads in order), then the min-max normalisation and
// the mask vector over the image span; padding past the span is zeroed as mass_salience does.
// =======================================================================================
constexpr int SAL_THREADS = 1024;

__global__ void __launch_bounds__(SAL_THREADS)
salience_from_heads_kernel(const SampleDesc *__restrict__ desc, int H, int max_vis, float scale, float lambda_max,
                           float eps, const float *__restrict__ heads /*[B, H, max_vis]*/, float *__restrict__ mass,
                           float *__restrict__ salience, float *__restrict__ mask_log, float *__restrict__ rank_score) {
  pdl_enter();
  __shared__ float s_red[2 * (SAL_THREADS / 32)];
  const int b = blockIdx.x;
  const SampleDesc d = desc[b];
  float *mass_b = mass + (size_t)b * max_vis, *sal_b = salience + (size_t)b * max_vis, *msk_b = mask_log + (size_t)b * max_vis;
  if (!d.valid) {
    for (int j = threadIdx.x; j < max_vis; j += SAL_THREADS) {
      mass_b[j] = 0.f; sal_b[j] = 0.f; msk_b[j] = 0.f;
      rank_score[(size_t)b * max_vis + j] = 0.f;       // the score and selection kernels skip the sample
    }
    return;
  }
  const float *hb = heads + (size_t)b * H * max_vis;
  float lo = INFINITY, hi = -INFINITY;
  for (int j = threadIdx.x; j < d.nv; j += SAL_THREADS) {
    float tot = 0.f;
    int hh = 0;
    for (; hh + 8 <= H; hh += 8) {            // eight loads in flight
      float v[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] = __ldcg(hb + (size_t)(hh + e) * max_vis + j);
#pragma unroll
      for (int e = 0; e < 8; ++e) tot += v[e];
    }
    for (; hh < H; ++hh) tot += __ldcg(hb + (size_t)hh * max_vis + j);
    tot *= scale;
    mass_b[j] = tot;
    lo = fminf(lo, tot); hi = fmaxf(hi, tot);
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
    hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
  }
  if (lane == 0) { s_red[warp] = lo; s_red[SAL_THREADS / 32 + warp] = hi; }
  __syncthreads();
  lo = s_red[0]; hi = s_red[SAL_THREADS / 32];
#pragma unroll
  for (int w = 1; w < SAL_THREADS / 32; ++w) {
    lo = fminf(lo, s_red[w]); hi = fmaxf(hi, s_red[SAL_THREADS / 32 + w]);
  }
  const float inv = 1.0f / ((hi - lo) + eps);
  for (int j = threadIdx.x; j < max_vis; j += SAL_THREADS) {
    if (j < d.nv) {
      const float sh = (mass_b[j] - lo) * inv;      // this thread's own store above
      sal_b[j] = sh;
      msk_b[j] = logf(fmaxf(lambda_max * sh, eps));
    } else {
      mass_b[j] = 0.f; sal_b[j] = 0.f; msk_b[j] = 0.f;
    }
  }
}

// =======================================================================================
// mass_heads: Eq. 1-3 kept per head (the variant with one salience and one mask per head).
//   s_j^h = qbar^h . k_j^h / sqrt(d): one warp per visual key row; a 16-byte vector of the row lies
//   inside one head (16 vectors per head), so the two halves of the warp reduce two heads per pass.
//   The block that finishes last for a sample then does, per head, the min-max normalisation (Eq. 2)
//   and the mask vector (Eq. 3), and per token the head means: mass = mean_h s^h (equal to the
//   default mass), salience = mean_h s_hat^h (the Eq. 5 weight), mask_log = Eq. 3 of that mean.
// grid (row blocks, B); 8 warps x 4 rows each.  s_heads: scratch [B, H, max_vis].
// Dynamic shared memory: D + 2 H floats.
// =======================================================================================
__global__ void __launch_bounds__(MASS_THREADS)
mass_heads_kernel(const __nv_bfloat16 *__restrict__ k, const SampleDesc *__restrict__ desc, int D, int H,
                  int max_vis, float scale, float lambda_max, float eps, const float *__restrict__ qbar,
                  float *__restrict__ s_heads, float *__restrict__ mass, float *__restrict__ salience,
                  float *__restrict__ mask_log, float *__restrict__ mask_log_heads,
                  float *__restrict__ rank_score, unsigned int *__restrict__ counters) {
  pdl_enter();
  extern __shared__ float s_q[];   // [D] then lo[H], inv[H]
  __shared__ int s_last;
  const int b = blockIdx.y;
  const SampleDesc d = desc[b];
  float *mass_b = mass + (size_t)b * max_vis;
  float *sal_b = salience + (size_t)b * max_vis, *msk_b = mask_log + (size_t)b * max_vis;
  float *mh_b = mask_log_heads + (size_t)b * H * max_vis;
  float *sh_b = s_heads + (size_t)b * H * max_vis;
  if (!d.valid) {
    for (int j = blockIdx.x * MASS_THREADS + threadIdx.x; j < max_vis; j += gridDim.x * MASS_THREADS) {
      mass_b[j] = 0.f; sal_b[j] = 0.f; msk_b[j] = 0.f;
      rank_score[(size_t)b * max_vis + j] = 0.f;   // the score kernel skips the sample
      for (int h = 0; h < H; ++h) mh_b[(size_t)h * max_vis + j] = 0.f;
    }
    return;
  }
  const int nblocks = (d.nv + MASS_ROWS - 1) / MASS_ROWS;
  if ((int)blockIdx.x >= nblocks) return;
  for (int c = threadIdx.x * 4; c < D; c += MASS_THREADS * 4)
    *reinterpret_cast<float4 *>(s_q + c) = __ldcg(reinterpret_cast<const float4 *>(qbar + (size_t)b * D + c));
  __syncthreads();

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int j0 = blockIdx.x * MASS_ROWS + warp * MASS_ROWS_PER_WARP;
  const int nvec = D / 8;
  const uint4 *rowp[MASS_ROWS_PER_WARP];
#pragma unroll
  for (int r = 0; r < MASS_ROWS_PER_WARP; ++r) {
    const int j = min(j0 + r, d.nv - 1);   // clamp: duplicates are discarded below
    rowp[r] = reinterpret_cast<const uint4 *>(k + (size_t)(d.row0 + d.v0 + j) * D);
  }
  for (int v0 = 0; v0 < nvec; v0 += 32) {      // one pass = 32 vectors = two heads
    const int v = v0 + lane;
    uint4 kv[MASS_ROWS_PER_WARP];
#pragma unroll
    for (int r = 0; r < MASS_ROWS_PER_WARP; ++r)
      if (v < nvec) kv[r] = __ldg(rowp[r] + v);
    float4 qa = make_float4(0.f, 0.f, 0.f, 0.f), qb = qa;
    if (v < nvec) {
      qa = *reinterpret_cast<const float4 *>(s_q + v * 8);
      qb = *reinterpret_cast<const float4 *>(s_q + v * 8 + 4);
    }
    const int h = (v0 >> 4) + (lane >> 4);      // head of this half of the warp
#pragma unroll
    for (int r = 0; r < MASS_ROWS_PER_WARP; ++r) {
      float part = 0.f;
      if (v < nvec) {
        float f[8];
        unpack8(kv[r], f);
        part = f[0] * qa.x + f[1] * qa.y + f[2] * qa.z + f[3] * qa.w + f[4] * qb.x + f[5] * qb.y + f[6] * qb.z +
               f[7] * qb.w;
      }
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);   // inside the 16 lanes
      if ((lane & 15) == 0 && h < H && j0 + r < d.nv) sh_b[(size_t)h * max_vis + j0 + r] = part * scale;
    }
  }

  // ---- last block of the sample ----
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned int old = atomicAdd(counters + b, 1u);
    s_last = (old == (unsigned int)(nblocks - 1));
    if (s_last) counters[b] = 0u;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  float *s_lo = s_q + D, *s_inv = s_lo + H;
  for (int h = warp; h < H; h += MASS_THREADS / 32) {           // Eq. 2's extremes, one warp per head
    float lo = INFINITY, hi = -INFINITY;
    for (int j = lane; j < d.nv; j += 32) {
      const float sv = __ldcg(sh_b + (size_t)h * max_vis + j);
      lo = fminf(lo, sv); hi = fmaxf(hi, sv);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
      hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    if (lane == 0) { s_lo[h] = lo; s_inv[h] = 1.0f / ((hi - lo) + eps); }
  }
  __syncthreads();
  const float inv_h = 1.0f / (float)H;
  for (int j = threadIdx.x; j < max_vis; j += MASS_THREADS) {
    if (j < d.nv) {
      float acc_s = 0.f, acc_sh = 0.f;
      for (int h = 0; h < H; ++h) {                               // heads in order
        const float sv = __ldcg(sh_b + (size_t)h * max_vis + j);
        const float sh = (sv - s_lo[h]) * s_inv[h];
        mh_b[(size_t)h * max_vis + j] = logf(fmaxf(lambda_max * sh, eps));
        acc_s += sv;
        acc_sh += sh;
      }
      const float sal = acc_sh * inv_h;
      mass_b[j] = acc_s * inv_h;
      sal_b[j] = sal;
      msk_b[j] = logf(fmaxf(lambda_max * sal, eps));
    } else {
      mass_b[j] = 0.f; sal_b[j] = 0.f; msk_b[j] = 0.f;
      for (int h = 0; h < H; ++h) mh_b[(size_t)h * max_vis + j] = 0.f;
    }
  }
}

// =======================================================================================
// select: exact top-k by radix select over order-preserving 32-bit keys, equal scores resolved
// toward the lower index, outputs in ascending index order.  One block per sample.
// =======================================================================================
constexpr int SELECT_THREADS = 1024;

__device__ __forceinline__ uint32_t score_key(float f) {
  if (f != f) return 0u;                       // NaN ranks below everything
  uint32_t u = __float_as_uint(f);
  if (f == 0.f) u = 0u;                        // -0.0 and +0.0 are one score: they tie, the lower index wins
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// exclusive prefix sum of one int per thread across the block; returns the block total in `total`
__device__ __forceinline__ int block_exclusive_scan(int v, int *s_warp /*[32]*/, int &total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();   // s_warp may still be read from a previous scan
  if (lane == 31) s_warp[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    int w = (lane < (int)(blockDim.x >> 5)) ? s_warp[lane] : 0;
    int winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int t = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += t;
    }
    s_warp[lane] = winc - w;             // exclusive warp offsets
    if (lane == 31) s_warp[32] = winc;   // block total
  }
  __syncthreads();
  total = s_warp[32];
  return s_warp[warp] + inc - v;
}

__global__ void __launch_bounds__(SELECT_THREADS)
select_kernel(const float *__restrict__ rank_score, const SampleDesc *__restrict__ desc,
              int max_vis, int keep_k, int32_t *__restrict__ keep_idx, int32_t *__restrict__ drop_idx,
              int32_t *__restrict__ role /*[B, max_vis]*/, int32_t *__restrict__ assign /*nullable*/,
              float *__restrict__ best_sim /*nullable*/, int sim_follows,
              const float *__restrict__ head_partial /*nullable: [B, H, max_vis]*/, int H,
              float *__restrict__ rank_out /*[B, max_vis], written when head_partial is given*/) {
  pdl_enter();
  extern __shared__ uint32_t s_key[];   // [max_vis]
  __shared__ int s_hist[256];
  __shared__ int s_scan[33];
  __shared__ uint32_t s_prefix;
  __shared__ int s_remaining;
  const int b = blockIdx.x;
  const SampleDesc d = desc[b];
  const int nd_max = max_vis - keep_k;
  int32_t *keep_b = keep_idx + (size_t)b * keep_k;
  int32_t *drop_b = drop_idx + (size_t)b * nd_max;
  int32_t *role_b = role + (size_t)b * max_vis;
  // assign / best_sim entries the similarity kernel will not write: the padding past the last
  // dropped token, and everything when no similarity kernel follows or the sample is skipped
  if (assign) {
    const int first = (d.valid && sim_follows) ? d.nv - keep_k : 0;
    for (int j = first + threadIdx.x; j < nd_max; j += blockDim.x) {
      assign[(size_t)b * nd_max + j] = -1;
      if (best_sim) best_sim[(size_t)b * nd_max + j] = 0.f;
    }
  }
  if (!d.valid) {
    for (int j = threadIdx.x; j < keep_k; j += blockDim.x) keep_b[j] = -1;
    for (int j = threadIdx.x; j < nd_max; j += blockDim.x) drop_b[j] = -1;
    for (int j = threadIdx.x; j < max_vis; j += blockDim.x) role_b[j] = 0;
    return;
  }
  const int nv = d.nv;
  if (head_partial) {
    // r_j = mean over heads and ranking rows of the Eq. 4 probabilities: the per-head sums
    // over ranking rows are added here in head order, and r is also written out
    const float inv = 1.0f / ((float)H * (float)d.nr);
    for (int j = threadIdx.x; j < max_vis; j += blockDim.x) {
      float tot = 0.f;
      if (j < nv) {
        const float *p = head_partial + (size_t)b * H * max_vis + j;
        int hh = 0;
        for (; hh + 32 <= H; hh += 32) {         // 32 loads in flight: one round trip for 32 heads
          float v[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = __ldcg(p + (size_t)(hh + e) * max_vis);
#pragma unroll
          for (int e = 0; e < 32; ++e) tot += v[e];
        }
        for (; hh + 8 <= H; hh += 8) {
          float v[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) v[e] = __ldcg(p + (size_t)(hh + e) * max_vis);
#pragma unroll
          for (int e = 0; e < 8; ++e) tot += v[e];
        }
        for (; hh < H; ++hh) tot += __ldcg(p + (size_t)hh * max_vis);
        tot *= inv;
        s_key[j] = score_key(tot);
      }
      rank_out[(size_t)b * max_vis + j] = tot;
    }
  } else {
    for (int j = threadIdx.x; j < nv; j += blockDim.x)
      s_key[j] = score_key(rank_score[(size_t)b * max_vis + j]);
  }
  if (threadIdx.x == 0) { s_prefix = 0u; s_remaining = keep_k; }
  __syncthreads();

  // four 8-bit digits, most significant first: find the key of the keep_k-th largest score
  uint32_t known = 0u;   // mask of the digits fixed so far
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = threadIdx.x; i < 256; i += blockDim.x) s_hist[i] = 0;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    for (int j = threadIdx.x; j < nv; j += blockDim.x) {
      const uint32_t key = s_key[j];
      if ((key & known) == prefix) atomicAdd(&s_hist[(key >> shift) & 255u], 1);
    }
    __syncthreads();
    if (threadIdx.x < 32) {
      const int lane = threadIdx.x;
      // lane L owns digits 255-8L .. 248-8L (descending); find where the running count reaches `remaining`
      int mine = 0;
#pragma unroll
      for (int e = 0; e < 8; ++e) mine += s_hist[255 - 8 * lane - e];
      int inc = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
      }
      const int remaining = s_remaining;
      __syncwarp();   // every lane has read s_remaining before one of them rewrites it
      const int before = inc - mine;
      if (before < remaining && remaining <= inc) {
        int run = before;
        for (int e = 0; e < 8; ++e) {
          const int digit = 255 - 8 * lane - e;
          const int c = s_hist[digit];
          if (run + c >= remaining) {
            s_prefix = prefix | ((uint32_t)digit << shift);
            s_remaining = remaining - run;
            break;
          }
          run += c;
        }
      }
    }
    known |= 255u << shift;
    __syncthreads();
  }
  const uint32_t kth = s_prefix;      // key of the keep_k-th largest score
  const int take_equal = s_remaining; // how many tokens with exactly that key are kept (lowest indices)

  // ordered emission: thread t owns the contiguous indices [t*per, (t+1)*per)
  const int per = (nv + blockDim.x - 1) / blockDim.x;
  const int lo = min(nv, (int)threadIdx.x * per), hi = min(nv, lo + per);
  int n_eq = 0;
  for (int j = lo; j < hi; ++j) n_eq += (s_key[j] == kth);
  int tot;
  int eq_before = block_exclusive_scan(n_eq, s_scan, tot);
  int n_keep = 0;
  {
    int e = eq_before;
    for (int j = lo; j < hi; ++j) {
      const uint32_t key = s_key[j];
      n_keep += (key > kth) || (key == kth && e < take_equal);
      e += (key == kth);
    }
  }
  int keep_before = block_exclusive_scan(n_keep, s_scan, tot);
  {
    int e = eq_before, kp = keep_before;
    for (int j = lo; j < hi; ++j) {
      const uint32_t key = s_key[j];
      const bool kept = (key > kth) || (key == kth && e < take_equal);
      e += (key == kth);
      if (kept) {
        keep_b[kp] = j; role_b[j] = kp; ++kp;
      } else {
        const int dp = j - kp;
        drop_b[dp] = j; role_b[j] = -(dp + 1);
      }
    }
  }
  for (int j = nv - keep_k + threadIdx.x; j < nd_max; j += blockDim.x) drop_b[j] = -1;
  for (int j = nv + threadIdx.x; j < max_vis; j += blockDim.x) role_b[j] = 0;
}

// role map from caller-provided keep / drop lists (entry point asap_merge)
__global__ void role_map_kernel(const SampleDesc *__restrict__ desc, int max_vis, int keep_k,
                                const int32_t *__restrict__ keep_idx,
                                const int32_t *__restrict__ drop_idx, int32_t *__restrict__ role,
                                int32_t *__restrict__ assign, float *__restrict__ best_sim,
                                int sim_follows) {
  pdl_enter();
  const int b = blockIdx.y;
  const SampleDesc d = desc[b];
  const int nd_max = max_vis - keep_k;
  {
    const int first = (d.valid && sim_follows) ? d.nv - keep_k : 0;
    for (int j = first + blockIdx.x * blockDim.x + threadIdx.x; j < nd_max; j += gridDim.x * blockDim.x) {
      assign[(size_t)b * nd_max + j] = -1;
      if (best_sim) best_sim[(size_t)b * nd_max + j] = 0.f;
    }
  }
  if (!d.valid) return;
  for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < d.nv; t += gridDim.x * blockDim.x) {
    if (t < keep_k) {
      const int j = keep_idx[(size_t)b * keep_k + t];
      if (j >= 0 && j < d.nv) role[(size_t)b * max_vis + j] = t;
    } else {
      const int dp = t - keep_k;
      const int j = drop_idx[(size_t)b * nd_max + dp];
      if (j >= 0 && j < d.nv) role[(size_t)b * max_vis + j] = -(dp + 1);
    }
  }
}

// =======================================================================================
// kept_gather: one warp per kept slot.  The kept row is copied to its slot of the dense
// [B*keep_k, D] operand of the similarity GEMM and its inverse norm 1/||h|| is stored (0 if
// ||h|| < 1e-12, which makes every similarity to that slot 0)   (Sec. 4.2).
// =======================================================================================
constexpr int GATHER_THREADS = 256;

__global__ void __launch_bounds__(GATHER_THREADS)
kept_gather_kernel(const __nv_bfloat16 *__restrict__ hidden, const SampleDesc *__restrict__ desc,
                   int D, int keep_k, const int32_t *__restrict__ keep_idx,
                   __nv_bfloat16 *__restrict__ kept_rows /*[B*keep_k, D]*/,
                   float *__restrict__ kept_inv /*[B*keep_k]*/) {
  pdl_enter();
  const int b = blockIdx.y;
  const SampleDesc d = desc[b];
  if (!d.valid) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int slot = blockIdx.x * (GATHER_THREADS / 32) + warp;
  if (slot >= keep_k) return;
  const int j = min(max(keep_idx[(size_t)b * keep_k + slot], 0), d.nv - 1);
  const uint4 *src = reinterpret_cast<const uint4 *>(hidden + (size_t)(d.row0 + d.v0 + j) * D);
  uint4 *dst = reinterpret_cast<uint4 *>(kept_rows + ((size_t)b * keep_k + slot) * D);
  const int nvec = D / 8;
  float ss = 0.f;
  for (int v = lane; v < nvec; v += 256) {
    uint4 x[8];
#pragma unroll
    for (int u = 0; u < 8; ++u)
      if (v + 32 * u < nvec) x[u] = __ldg(src + v + 32 * u);
#pragma unroll
    for (int u = 0; u < 8; ++u)
      if (v + 32 * u < nvec) {
        float f[8];
        unpack8(x[u], f);
#pragma unroll
        for (int e = 0; e < 8; ++e) ss += f[e] * f[e];
        dst[v + 32 * u] = x[u];
      }
  }
  ss = warp_sum(ss);
  if (lane == 0) {
    const float nrm = sqrtf(ss);
    kept_inv[(size_t)b * keep_k + slot] = nrm >= 1e-12f ? 1.0f / nrm : 0.f;
  }
}

// =======================================================================================
// csr_block: group the dropped tokens of one sample by destination slot (counting sort, stable
// in dropped order so the merge adds its members in a fixed order).  Run by one whole block of
// W <= 8 warps: warp w owns the w-th contiguous chunk of dropped positions, counts its chunk
// into its own histogram, and after a scan over (slot, warp) writes its chunk's positions behind
// those of the warps before it.  s_cnt needs (W + 1) * keep_k ints, s_scan 33 ints.
// seg [B, keep_k+1], members [B, max_vis-keep_k] (dropped POSITIONS, ascending inside a slot).
// With drop_idx, salience and member_meta given, member_meta [B, max_vis-keep_k] receives, beside every
// entry of `members`, the member's visual index and its merge weight (the salience, as bits): the
// merge kernel then reaches a member's row in two dependent loads instead of four.
// =======================================================================================
__device__ __forceinline__ void csr_block(const SampleDesc &d, int b, int max_vis, int keep_k,
                                          const int32_t *__restrict__ assign,
                                          int32_t *__restrict__ seg, int32_t *__restrict__ members,
                                          int *s_cnt, int *s_scan,
                                          const int32_t *__restrict__ drop_idx = nullptr,
                                          const float *__restrict__ salience = nullptr,
                                          int2 *__restrict__ member_meta = nullptr) {
  int32_t *seg_b = seg + (size_t)b * (keep_k + 1);
  const int nd_max = max_vis - keep_k, nd = d.nv - keep_k;
  const int32_t *as_b = assign + (size_t)b * nd_max;
  int32_t *mem_b = members + (size_t)b * nd_max;
  const int W = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunk = (((nd + W - 1) / W) + 31) & ~31;        // positions per warp, a multiple of 32
  int *hist = s_cnt;                                         // [W][keep_k]
  int *tot = s_cnt + W * keep_k;                             // [keep_k] members per slot
  for (int i = threadIdx.x; i < (W + 1) * keep_k; i += blockDim.x) s_cnt[i] = 0;
  __syncthreads();
  const int p_lo = min(nd, warp * chunk), p_hi = min(nd, p_lo + chunk);
  for (int p = p_lo + lane; p < p_hi; p += 32) {
    const int a = __ldcg(as_b + p);
    if (a >= 0 && a < keep_k) atomicAdd(&hist[warp * keep_k + a], 1);
  }
  __syncthreads();
  // per slot: turn the per-warp counts into per-warp offsets inside the slot, and total them
  for (int i = threadIdx.x; i < keep_k; i += blockDim.x) {
    int run = 0;
    for (int w = 0; w < W; ++w) {
      const int c = hist[w * keep_k + i];
      hist[w * keep_k + i] = run;
      run += c;
    }
    tot[i] = run;
  }
  __syncthreads();
  // exclusive scan over slots; thread t owns a contiguous range of slots
  const int per = (keep_k + blockDim.x - 1) / blockDim.x;
  const int lo = min(keep_k, (int)threadIdx.x * per), hi = min(keep_k, lo + per);
  int mine = 0;
  for (int i = lo; i < hi; ++i) mine += tot[i];
  int total;
  int run = block_exclusive_scan(mine, s_scan, total);
  for (int i = lo; i < hi; ++i) {
    const int c = tot[i];
    seg_b[i] = run;
    tot[i] = run;        // becomes the slot's base
    run += c;
  }
  if (threadIdx.x == 0) seg_b[keep_k] = total;
  __syncthreads();
  // stable fill: every warp walks its chunk 32 positions at a time in ascending order
  const bool meta = drop_idx && salience && member_meta;
  for (int base = p_lo; base < p_hi; base += 32) {
    const int p = base + lane;
    int a = (p < p_hi) ? __ldcg(as_b + p) : -1;
    if (a >= keep_k) a = -1;
    int2 mm = make_int2(0, 0);
    if (meta && a >= 0) {
      mm.x = min(max(__ldg(drop_idx + (size_t)b * nd_max + p), 0), d.nv - 1);
      mm.y = __float_as_int(__ldcg(salience + (size_t)b * max_vis + mm.x));
    }
    const unsigned peers = __match_any_sync(0xffffffffu, a);
    const int rank = __popc(peers & ((1u << lane) - 1u));
    int cur = 0;
    if (a >= 0) cur = hist[warp * keep_k + a];
    __syncwarp();
    if (a >= 0) {
      mem_b[tot[a] + cur + rank] = p;
      if (meta) member_meta[(size_t)b * nd_max + tot[a] + cur + rank] = mm;
      if (rank == 0) hist[warp * keep_k + a] = cur + __popc(peers);
    }
    __syncwarp();
  }
}

// =======================================================================================
// route: Sec. 4.2 inside the kept set, one block per sample.  Input: the keep_k x keep_k cosine
// matrix S of the kept rows, the salience, the attention mass, stage 1's kept / pruned lists.
//   A  visiting order of the kept slots: salience descending, sequence index ascending.
//   B  bit matrix  M[p] = { q : S[p][q] > t }.
//   C  one warp walks the slots in visiting order.  A slot whose bit is set in the running union
//      of the anchors' rows is absorbed (while the pruned pool can still refill a slot, i.e. at
//      most nv - keep_k times); any other slot becomes an anchor and adds its row to the union.
//      This is the greedy rule "join the most similar earlier anchor if that similarity exceeds t,
//      else become an anchor" with the question WHICH anchor left to step D.
//   D  every absorbed slot finds the most similar anchor that was visited before it (lowest slot
//      among equals).
//   E  the vacated slots are refilled with the pruned tokens of largest attention mass (radix
//      select, lower index first among equals).
//   F  anchors and refilled tokens, in sequence order, form the final kept list; the absorbed
//      tokens, ascending, form the source list with their anchor's FINAL slot; CSR of that list.
// Outputs use the layouts of the merge kernel: final_keep [B, keep_k], src_idx / src_assign /
// src_sim [B, max_vis - keep_k] (padding -1 / 0), seg [B, keep_k + 1], members [B, max_vis - keep_k].
// =======================================================================================
constexpr int ROUTE_THREADS = 1024;
constexpr int ROUTE_LANE_WORDS = 4;                     // keep_k <= 32 * 32 * 4

// The sequential part of the routing, run by one warp, 32 candidates of the visiting order at a
// time.  Lane l holds words l, l + 32, ... of the union of the anchors' rows (LW words per lane;
// LW = 1 covers keep_k <= 1024).  Per group of 32: (1) each lane looks up whether its candidate is
// already covered by an anchor of an earlier group; (2) each lane gathers its candidate's row
// restricted to the group (32 bits); (3) the group is resolved in order from those 32 x 32 bits, in
// registers, by every lane alike; (4) the group's anchors add their full rows to the union.  Only
// step (3) is a dependent chain, and it touches no memory.  Returns the number of absorbed slots.
template <int LW>
__device__ __forceinline__ int route_walk(const int *s_order, const uint32_t *mask, int *s_flag, int k, int kw,
                                          int nd, int lane) {
  const unsigned full = 0xffffffffu;
  uint32_t supp[LW];
#pragma unroll
  for (int i = 0; i < LW; ++i) supp[i] = 0u;
  int n_abs = 0;
  for (int r0 = 0; r0 < k; r0 += 32) {
    const bool valid = r0 + lane < k;
    const int p = valid ? s_order[r0 + lane] : 0;
    const int w = p >> 5;
    uint32_t word = 0u;
#pragma unroll
    for (int i = 0; i < LW; ++i) {
      const uint32_t got = __shfl_sync(full, supp[i], w & 31);
      if ((w >> 5) == i) word = got;
    }
    uint32_t blk = __ballot_sync(full, valid && ((word >> (p & 31)) & 1u));
    uint32_t intra = 0u;
#pragma unroll
    for (int u = 0; u < 32; ++u) {
      const int pu = __shfl_sync(full, p, u);
      const uint32_t bit = (mask[(size_t)p * kw + (pu >> 5)] >> (pu & 31)) & 1u;
      if (valid && r0 + u < k) intra |= bit << u;
    }
    uint32_t absorbed_bits = 0u;
#pragma unroll
    for (int t = 0; t < 32; ++t) {
      const uint32_t row_t = __shfl_sync(full, intra, t);
      const bool ab = ((blk >> t) & 1u) && n_abs < nd && r0 + t < k;
      if (ab) {
        ++n_abs;
        absorbed_bits |= 1u << t;
      } else {
        blk |= row_t & ~((2u << t) - 1u);          // an anchor covers later candidates only
      }
    }
#pragma unroll
    for (int t = 0; t < 32; ++t) {
      const int pt = __shfl_sync(full, p, t);
      if (r0 + t < k && !((absorbed_bits >> t) & 1u)) {
#pragma unroll
        for (int i = 0; i < LW; ++i) {
          const int ww = i * 32 + lane;
          if (ww < kw) supp[i] |= mask[(size_t)pt * kw + ww];
        }
      }
    }
    if (valid) s_flag[p] = ((absorbed_bits >> lane) & 1u) ? 0 : 1;
  }
  return n_abs;
}

struct RouteArgs {
  const SampleDesc *desc;
  int max_vis, keep_k, kw;        // kw = ceil(keep_k / 32)
  float threshold;
  const float *smat;              // [B, keep_k, keep_k]
  uint32_t *mask_g;               // [B, keep_k, kw] or nullptr: the bit matrix lives in shared memory
  const float *salience, *mass;   // [B, max_vis]
  const int32_t *keep_idx;        // [B, keep_k]            stage 1
  const int32_t *drop_idx;        // [B, max_vis - keep_k]  stage 1
  int32_t *final_keep, *src_idx, *src_assign, *seg, *members, *n_absorbed;
  float *src_sim;                 // nullable
};

__global__ void __launch_bounds__(ROUTE_THREADS)
route_kernel(RouteArgs a) {
  pdl_enter();
  extern __shared__ uint32_t r_smem[];
  __shared__ int s_hist[256];
  __shared__ int s_scan[33];
  __shared__ uint32_t s_prefix;
  __shared__ int s_remaining, s_nabs;
  const int b = blockIdx.x;
  const SampleDesc d = a.desc[b];
  const int k = a.keep_k, kw = a.kw, nd_max = a.max_vis - k;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, nthr = blockDim.x;
  int32_t *fk_b = a.final_keep + (size_t)b * k;
  int32_t *si_b = a.src_idx + (size_t)b * nd_max;
  int32_t *sa_b = a.src_assign + (size_t)b * nd_max;
  float *ss_b = a.src_sim ? a.src_sim + (size_t)b * nd_max : nullptr;
  int32_t *seg_b = a.seg + (size_t)b * (k + 1);
  int32_t *mem_b = a.members + (size_t)b * nd_max;
  if (!d.valid) {
    for (int j = tid; j < k; j += nthr) fk_b[j] = -1;
    for (int j = tid; j < nd_max; j += nthr) { si_b[j] = -1; sa_b[j] = -1; if (ss_b) ss_b[j] = 0.f; }
    for (int j = tid; j <= k; j += nthr) seg_b[j] = 0;
    if (tid == 0 && a.n_absorbed) a.n_absorbed[b] = 0;
    return;
  }
  const int nv = d.nv, nd = nv - k;
  // shared memory: [order k][rank k][flag k][dest k][tmp k] [union: bit matrix k*kw | key nd_max + pos max_vis]
  int *s_order = reinterpret_cast<int *>(r_smem);
  int *s_rank = s_order + k;
  int *s_flag = s_rank + k;
  int *s_dest = s_flag + k;
  uint32_t *s_tmp = r_smem + 4 * (size_t)k;
  uint32_t *s_union = s_tmp + k;
  uint32_t *mask = a.mask_g ? a.mask_g + (size_t)b * k * kw : s_union;
  const int32_t *keep_b = a.keep_idx + (size_t)b * k;
  const int32_t *drop_b = a.drop_idx + (size_t)b * nd_max;
  const float *sal_b = a.salience + (size_t)b * a.max_vis;
  const float *S = a.smat + (size_t)b * k * k;

  // ---- A: visiting order.  Keys are order-preserving integers, so NaN cannot break the permutation.
  for (int p = tid; p < k; p += nthr) {
    const int j = min(max(keep_b[p], 0), nv - 1);
    s_tmp[p] = score_key(sal_b[j]);
  }
  __syncthreads();
  for (int p = tid; p < k; p += nthr) {
    const uint32_t mine = s_tmp[p];
    int r = 0;
    for (int q = 0; q < k; ++q) {
      const uint32_t o = s_tmp[q];
      r += (o > mine) || (o == mine && q < p);       // the kept list is ascending: q < p is the lower index
    }
    s_rank[p] = r;
    s_order[r] = p;
  }
  // ---- B: bit matrix, one warp per row, coalesced
  for (int p = warp; p < k; p += (nthr >> 5)) {
    const float *row = S + (size_t)p * k;
    for (int w0 = 0; w0 < kw; w0 += 16) {             // sixteen loads in flight per lane
      float v[16];
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        const int q = (w0 + e) * 32 + lane;
        v[e] = q < k ? __ldcg(row + q) : -INFINITY;
      }
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        const int q = (w0 + e) * 32 + lane;
        const unsigned bits = __ballot_sync(0xffffffffu, q < k && q != p && v[e] > a.threshold);
        if (lane == 0 && w0 + e < kw) mask[(size_t)p * kw + w0 + e] = bits;
      }
    }
  }
  __syncthreads();
  // ---- C: greedy walk by one warp; the union lives in registers, word w in lane w % 32
  if (warp == 0) {
    const int n_abs_w = kw <= 32 ? route_walk<1>(s_order, mask, s_flag, k, kw, nd, lane)
                                 : route_walk<ROUTE_LANE_WORDS>(s_order, mask, s_flag, k, kw, nd, lane);
    if (lane == 0) s_nabs = n_abs_w;
  }
  __syncthreads();
  const int n_abs = s_nabs;
  // ---- D: destination of every absorbed slot
  for (int p = warp; p < k; p += (nthr >> 5)) {
    if (s_flag[p]) { if (lane == 0) s_dest[p] = -1; continue; }
    const float *row = S + (size_t)p * k;
    const int rp = s_rank[p];
    float best = -INFINITY;
    int best_q = 0x7fffffff;
    for (int q0 = lane; q0 < k; q0 += 32 * 8) {       // eight loads in flight per lane
      float v[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int q = q0 + 32 * e;
        v[e] = (q < k && s_flag[q] && s_rank[q] < rp) ? __ldcg(row + q) : -INFINITY;
      }
#pragma unroll
      for (int e = 0; e < 8; ++e)                     // ascending q: the first maximum stays
        if (v[e] > best) { best = v[e]; best_q = q0 + 32 * e; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int oq = __shfl_xor_sync(0xffffffffu, best_q, o);
      if (ob > best || (ob == best && oq < best_q)) { best = ob; best_q = oq; }
    }
    if (lane == 0) {
      s_dest[p] = best_q < k ? best_q : -1;
      s_tmp[p] = __float_as_uint(best);
    }
  }
  __syncthreads();      // the bit matrix is dead from here on: its space is reused
  uint32_t *s_key = s_union;                                  // [nd]
  int *s_pos = reinterpret_cast<int *>(s_union + nd_max);     // [nv] 1 + final slot, 0 = not in the final list
  // ---- E: the n_abs pruned tokens of largest attention mass
  const float *mass_b = a.mass + (size_t)b * a.max_vis;
  for (int v = tid; v < nv; v += nthr) s_pos[v] = 0;
  for (int i = tid; i < nd; i += nthr) {
    const int j = min(max(drop_b[i], 0), nv - 1);
    s_key[i] = score_key(mass_b[j]);
  }
  if (tid == 0) { s_prefix = 0u; s_remaining = n_abs; }
  __syncthreads();
  if (n_abs > 0) {
    uint32_t known = 0u;
    for (int shift = 24; shift >= 0; shift -= 8) {
      for (int i = tid; i < 256; i += nthr) s_hist[i] = 0;
      __syncthreads();
      const uint32_t prefix = s_prefix;
      for (int i = tid; i < nd; i += nthr) {
        const uint32_t key = s_key[i];
        if ((key & known) == prefix) atomicAdd(&s_hist[(key >> shift) & 255u], 1);
      }
      __syncthreads();
      if (tid < 32) {
        int mine = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) mine += s_hist[255 - 8 * lane - e];
        int inc = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          int t = __shfl_up_sync(0xffffffffu, inc, o);
          if (lane >= o) inc += t;
        }
        const int remaining = s_remaining;
        __syncwarp();
        const int before = inc - mine;
        if (before < remaining && remaining <= inc) {
          int run = before;
          for (int e = 0; e < 8; ++e) {
            const int digit = 255 - 8 * lane - e;
            const int c = s_hist[digit];
            if (run + c >= remaining) {
              s_prefix = prefix | ((uint32_t)digit << shift);
              s_remaining = remaining - run;
              break;
            }
            run += c;
          }
        }
      }
      known |= 255u << shift;
      __syncthreads();
    }
    const uint32_t kth = s_prefix;
    const int take_equal = s_remaining;
    const int per = (nd + nthr - 1) / nthr;
    const int lo = min(nd, tid * per), hi = min(nd, lo + per);
    int n_eq = 0;
    for (int i = lo; i < hi; ++i) n_eq += (s_key[i] == kth);
    int tot;
    int e = block_exclusive_scan(n_eq, s_scan, tot);
    for (int i = lo; i < hi; ++i) {
      const uint32_t key = s_key[i];
      if (key > kth || (key == kth && e < take_equal)) s_pos[min(max(drop_b[i], 0), nv - 1)] = 1;
      e += (key == kth);
    }
  }
  for (int p = tid; p < k; p += nthr)
    if (s_flag[p]) s_pos[min(max(keep_b[p], 0), nv - 1)] = 1;
  __syncthreads();
  // ---- F: final kept list in sequence order
  {
    const int per = (nv + nthr - 1) / nthr;
    const int lo = min(nv, tid * per), hi = min(nv, lo + per);
    int cnt = 0;
    for (int v = lo; v < hi; ++v) cnt += s_pos[v];
    int tot;
    int run = block_exclusive_scan(cnt, s_scan, tot);
    for (int v = lo; v < hi; ++v) {
      if (s_pos[v]) {
        if (run < k) fk_b[run] = v;
        s_pos[v] = ++run;
      }
    }
    // fewer than keep_k can only come from malformed input lists: pad
    for (int j = tot + tid; j < k; j += nthr) fk_b[j] = -1;
  }
  __syncthreads();
  // source list: absorbed slots in ascending order, with the final slot of their anchor
  {
    const int per = (k + nthr - 1) / nthr;
    const int lo = min(k, tid * per), hi = min(k, lo + per);
    int cnt = 0;
    for (int p = lo; p < hi; ++p) cnt += !s_flag[p];
    int tot;
    int run = block_exclusive_scan(cnt, s_scan, tot);
    for (int p = lo; p < hi; ++p) {
      if (!s_flag[p] && run < nd_max) {
        const int q = s_dest[p];
        const int slot = q >= 0 ? s_pos[min(max(keep_b[q], 0), nv - 1)] - 1 : -1;
        si_b[run] = keep_b[p];
        sa_b[run] = (slot >= 0 && slot < k) ? slot : -1;
        if (ss_b) ss_b[run] = __uint_as_float(s_tmp[p]);
        s_key[run] = (uint32_t)((slot >= 0 && slot < k) ? slot : -1);     // for the grouping below
        ++run;
      }
    }
    for (int j = n_abs + tid; j < nd_max; j += nthr) { si_b[j] = -1; sa_b[j] = -1; if (ss_b) ss_b[j] = 0.f; }
  }
  if (tid == 0 && a.n_absorbed) a.n_absorbed[b] = n_abs;
  __syncthreads();
  // grouping by destination (counting sort, stable in source order)
  {
    int *s_cnt = s_order;                     // reuse: the visiting order is no longer needed
    for (int sl = tid; sl < k; sl += nthr) s_cnt[sl] = 0;
    __syncthreads();
    for (int i = tid; i < n_abs; i += nthr) {
      const int sl = (int)s_key[i];
      if (sl >= 0 && sl < k) atomicAdd(&s_cnt[sl], 1);
    }
    __syncthreads();
    const int per = (k + nthr - 1) / nthr;
    const int lo = min(k, tid * per), hi = min(k, lo + per);
    int mine = 0;
    for (int sl = lo; sl < hi; ++sl) mine += s_cnt[sl];
    int tot;
    int run = block_exclusive_scan(mine, s_scan, tot);
    for (int sl = lo; sl < hi; ++sl) {
      const int c = s_cnt[sl];
      seg_b[sl] = run;
      s_cnt[sl] = run;
      run += c;
    }
    if (tid == 0) seg_b[k] = tot;
    __syncthreads();
    // one warp walks the sources 32 at a time in ascending order, so members stay ascending inside a slot
    if (warp == 0) {
      for (int base = 0; base < n_abs; base += 32) {
        const int i = base + lane;
        int sl = i < n_abs ? (int)s_key[i] : -1;
        if (sl >= k) sl = -1;
        const unsigned peers = __match_any_sync(0xffffffffu, sl);
        const int rank = __popc(peers & ((1u << lane) - 1u));
        int at = 0;
        if (sl >= 0) at = s_cnt[sl];
        __syncwarp();
        if (sl >= 0) {
          mem_b[at + rank] = i;
          if (rank == 0) s_cnt[sl] = at + __popc(peers);
        }
        __syncwarp();
      }
    }
  }
}

// =======================================================================================
// merge_compact: grid (keep_k + copy-row groups, B).
//   blockIdx.x <  keep_k : the block owns one kept visual row.  Its members (the dropped tokens
//                          assigned to that slot) are first listed in shared memory with their
//                          weights, then their rows are streamed four at a time and accumulated
//                          in fp32 in CSR order:  (s_hat_i h_i + sum_j s_hat_j h_j) / (s_hat_i +
//                          sum_j s_hat_j)   (Eq. 5), rounded to bf16 once.  No members, merging
//                          off, or total weight <= eps: the row is copied.
//   blockIdx.x >= keep_k : each warp copies one prefix / suffix row.
// Every output row also gets its gathered position id and its source row (hand-off of Fig. 3).
// =======================================================================================
constexpr int MERGE_THREADS = 256;
constexpr int MERGE_COPY_ROWS = MERGE_THREADS / 32;   // copy rows per block
constexpr int MERGE_LIST = 256;                        // members listed per pass
constexpr int MERGE_BATCH = 4;                         // member rows in flight per thread

struct MergeArgs {
  const __nv_bfloat16 *hidden;
  const int32_t *pos_ids;
  const SampleDesc *desc;
  int D, max_vis, keep_k, merge_enable;
  float eps;
  const float *salience;
  const int32_t *keep_idx, *drop_idx, *seg, *members;
  const int2 *member_meta;   // [B, max_vis-keep_k] (visual index, weight bits) beside `members`, or nullptr
  __nv_bfloat16 *out_hidden;
  int32_t *out_pos, *src_row;
};

// NV: 16-byte vectors per thread (D <= NV * 256 * 8); wide rows keep fewer member rows in flight per thread
// so that three or four blocks still fit the register file of an SM.
// LEAN (rows of at most 4096 elements, launches of many waves): two member rows in flight as well, 60 registers,
// four blocks per SM -- more blocks in their dependent look-ups at any time (c4 398 -> 369 us); on launches of a
// few waves the shorter batches cost more than the occupancy gives (c2 24.8 -> 26.6 us), so those keep four rows.
// Rows of 4097-6144 elements (NV = 3): one member row in flight, 64 registers, four blocks per SM as well
// (D = 5120, 1152 of 2304 kept: 280 -> 241 us; 576 of 1152: 151 -> 133 us; 288 of 576: 85 -> 75 us).
template <int NV, bool LEAN = false>
__global__ void __launch_bounds__(MERGE_THREADS, NV >= 4 ? 2 : ((LEAN || NV == 3) ? 4 : 3))
merge_compact_kernel(MergeArgs a) {
  constexpr int BATCH = NV == 3 ? 1 : ((NV >= 4 || LEAN) ? 2 : MERGE_BATCH);
  pdl_enter();
  __shared__ int s_j[MERGE_LIST];
  __shared__ float s_w[MERGE_LIST];
  const int b = blockIdx.y;
  const SampleDesc d = a.desc[b];
  if (!d.valid) return;
  const int nvec = a.D / 8;
  const int k = a.keep_k;
  if ((int)blockIdx.x >= k) {
    // ---------------------------------------------------------------- copy rows, one per warp
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int c = ((int)blockIdx.x - k) * MERGE_COPY_ROWS + warp;     // index among prefix + suffix rows
    if (c >= d.n - d.nv) return;
    const int srow = c < d.v0 ? c : c + d.nv;
    const int orow = d.out_row0 + (c < d.v0 ? c : c + k);
    const size_t grow = (size_t)(d.row0 + srow);
    if (lane == 0) {
      a.out_pos[orow] = a.pos_ids[grow];
      a.src_row[orow] = (int32_t)grow;
    }
    const uint4 *src = reinterpret_cast<const uint4 *>(a.hidden + grow * a.D);
    uint4 *dst = reinterpret_cast<uint4 *>(a.out_hidden + (size_t)orow * a.D);
    for (int v = lane; v < nvec; v += 32 * 8) {
      uint4 x[8];
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (v + 32 * u < nvec) x[u] = __ldg(src + v + 32 * u);
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (v + 32 * u < nvec) dst[v + 32 * u] = x[u];
    }
    return;
  }
  // ------------------------------------------------------------------ one kept row
  const int slot = blockIdx.x;
  const int vi = min(max(a.keep_idx[(size_t)b * k + slot], 0), d.nv - 1);   // visual index
  const size_t grow = (size_t)(d.row0 + d.v0 + vi);
  const int orow = d.out_row0 + d.v0 + slot;
  if (threadIdx.x == 0) {
    a.out_pos[orow] = a.pos_ids[grow];
    a.src_row[orow] = (int32_t)grow;
  }
  const uint4 *src = reinterpret_cast<const uint4 *>(a.hidden + grow * a.D);
  uint4 *dst = reinterpret_cast<uint4 *>(a.out_hidden + (size_t)orow * a.D);
  const int nd_max = a.max_vis - k;
  int m_lo = 0, m_hi = 0;
  if (a.merge_enable) {
    m_lo = min(max(a.seg[(size_t)b * (k + 1) + slot], 0), nd_max);
    m_hi = min(max(a.seg[(size_t)b * (k + 1) + slot + 1], m_lo), nd_max);
  }
  uint4 self[NV];
#pragma unroll
  for (int u = 0; u < NV; ++u) {
    const int v = threadIdx.x + u * MERGE_THREADS;
    if (v < nvec) self[u] = __ldg(src + v);
  }
  if (m_hi <= m_lo) {
#pragma unroll
    for (int u = 0; u < NV; ++u) {
      const int v = threadIdx.x + u * MERGE_THREADS;
      if (v < nvec) dst[v] = self[u];
    }
    return;
  }
  const float *sal_b = a.salience + (size_t)b * a.max_vis;
  const int32_t *mem_b = a.members + (size_t)b * nd_max;
  const int32_t *drop_b = a.drop_idx + (size_t)b * nd_max;
  const float w_self = sal_b[vi];
  float acc[NV][8];
#pragma unroll
  for (int u = 0; u < NV; ++u) {
    float f[8];
    unpack8(self[u], f);
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[u][e] = w_self * f[e];
  }
  float den = w_self;
  const __nv_bfloat16 *vis0 = a.hidden + (size_t)(d.row0 + d.v0) * a.D;
  for (int base = m_lo; base < m_hi; base += MERGE_LIST) {
    const int cnt = min(MERGE_LIST, m_hi - base);
    __syncthreads();                      // the previous list has been consumed
    if ((int)threadIdx.x < cnt) {
      if (a.member_meta) {
        const int2 mm = __ldg(a.member_meta + (size_t)b * nd_max + base + threadIdx.x);
        s_j[threadIdx.x] = min(max(mm.x, 0), d.nv - 1);
        s_w[threadIdx.x] = __int_as_float(mm.y);
      } else {
        const int j = min(max(drop_b[min(max(mem_b[base + threadIdx.x], 0), nd_max - 1)], 0), d.nv - 1);
        s_j[threadIdx.x] = j;
        s_w[threadIdx.x] = sal_b[j];
      }
    }
    __syncthreads();
    for (int m0 = 0; m0 < cnt; m0 += BATCH) {
      uint4 x[BATCH][NV];
#pragma unroll
      for (int t = 0; t < BATCH; ++t) {
        if (m0 + t < cnt) {
          const uint4 *msrc = reinterpret_cast<const uint4 *>(vis0 + (size_t)s_j[m0 + t] * a.D);
#pragma unroll
          for (int u = 0; u < NV; ++u) {
            const int v = threadIdx.x + u * MERGE_THREADS;
            if (v < nvec) x[t][u] = __ldg(msrc + v);
          }
        }
      }
#pragma unroll
      for (int t = 0; t < BATCH; ++t) {
        if (m0 + t < cnt) {
          const float w = s_w[m0 + t];
          den += w;
#pragma unroll
          for (int u = 0; u < NV; ++u) {
            float f[8];
            unpack8(x[t][u], f);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[u][e] += w * f[e];
          }
        }
      }
    }
  }
  if (den <= a.eps) {
#pragma unroll
    for (int u = 0; u < NV; ++u) {
      const int v = threadIdx.x + u * MERGE_THREADS;
      if (v < nvec) dst[v] = self[u];
    }
  } else {
    const float inv = 1.0f / den;
#pragma unroll
    for (int u = 0; u < NV; ++u) {
      const int v = threadIdx.x + u * MERGE_THREADS;
      if (v < nvec) {
        uint4 o;
        o.x = pack2_rn(acc[u][0] * inv, acc[u][1] * inv);
        o.y = pack2_rn(acc[u][2] * inv, acc[u][3] * inv);
        o.z = pack2_rn(acc[u][4] * inv, acc[u][5] * inv);
        o.w = pack2_rn(acc[u][6] * inv, acc[u][7] * inv);
        dst[v] = o;
      }
    }
  }
}

// =======================================================================================
// gather_rows: KV-cache compaction.  Output row r of every tensor is input row src_row[r] (the
// row map the prune step wrote); one warp per (row, tensor), 16-byte vectors, eight in flight.
// Rows at or past *n_rows (a device-side count, e.g. out_cu_seqlens[B]) are left untouched.
// =======================================================================================
constexpr int KV_MAX_TENSORS = 64;
constexpr int KV_THREADS = 256;

struct GatherArgs {
  const void *src[KV_MAX_TENSORS];
  void *dst[KV_MAX_TENSORS];
  const int32_t *src_row;
  const int32_t *n_rows;      // device scalar
  int32_t rows_capacity, src_rows, row_vecs;   // row_vecs = row bytes / 16
};

__global__ void __launch_bounds__(KV_THREADS)
gather_rows_kernel(GatherArgs a) {
  pdl_enter();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = blockIdx.x * (KV_THREADS / 32) + warp;
  if (r >= a.rows_capacity || r >= *a.n_rows) return;
  const int sr = a.src_row[r];
  if (sr < 0 || sr >= a.src_rows) return;                 // not a valid source row: leave the output row alone
  const uint4 *src = reinterpret_cast<const uint4 *>(a.src[blockIdx.y]) + (size_t)sr * a.row_vecs;
  uint4 *dst = reinterpret_cast<uint4 *>(a.dst[blockIdx.y]) + (size_t)r * a.row_vecs;
  for (int v = lane; v < a.row_vecs; v += 32 * 8) {
    uint4 x[8];
#pragma unroll
    for (int u = 0; u < 8; ++u)
      if (v + 32 * u < a.row_vecs) x[u] = __ldg(src + v + 32 * u);
#pragma unroll
    for (int u = 0; u < 8; ++u)
      if (v + 32 * u < a.row_vecs) dst[v + 32 * u] = x[u];
  }
}

}  // namespace asap
