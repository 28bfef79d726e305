// AttnGate (Sec. 3.1, Eq. 1) in two kernels:
//   pool_project_kernel : streams Q and K once (HBM-bound), average-pools each 64-token block per head and
//                         multiplies the pooled vectors by the head's gate matrix (fp32 on the CUDA cores) -> gq, gk
//   gate_scores_kernel  : logits = gq gk^T / sqrt(dg) over the causal blocks, row softmax -> scores
// The logits need fp32-grade products (plain bf16 or tf32 tensor-core inputs would not hold the 1e-3 relative bound on
// softmax outputs when logits reach tens), so gq and gk are stored as three bf16 planes each, x = hi + mid + lo with
// every part the bf16 rounding of what is left, and the product is taken on the tensor cores (mma.sync, fp32
// accumulation) as the six terms hi*hi + hi*mid + mid*hi + hi*lo + lo*hi + mid*mid: what is dropped is below 2^-24 of
// the product.
#include <cuda_bf16.h>
#include <math_constants.h>

#include <cstddef>
#include <mutex>

#include "seer_internal.cuh"

namespace seer {

// ----------------------------------------------------------------------------------------------- kernel 1
constexpr int kPoolThreads = 256;

// x = hi + mid + lo, each part the bf16 (round-to-nearest-even) of the remainder; the three planes of a tensor lie
// `plane` elements apart.
__device__ __forceinline__ void store_split3(uint16_t* __restrict__ dst, size_t plane, float x) {
  const __nv_bfloat16 hi = __float2bfloat16_rn(x);
  const float r1 = x - __bfloat162float(hi);
  const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
  const float r2 = r1 - __bfloat162float(mid);
  const __nv_bfloat16 lo = __float2bfloat16_rn(r2);
  dst[0] = __bfloat16_as_ushort(hi);
  dst[plane] = __bfloat16_as_ushort(mid);
  dst[2 * plane] = __bfloat16_as_ushort(lo);
}

__device__ __forceinline__ uint4 ld_stream_16(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
  return r;
}

__device__ __forceinline__ void acc_bf16x8(float (&a)[8], const uint4& u) {
  a[0] += __uint_as_float(u.x << 16); a[1] += __uint_as_float(u.x & 0xffff0000u);
  a[2] += __uint_as_float(u.y << 16); a[3] += __uint_as_float(u.y & 0xffff0000u);
  a[4] += __uint_as_float(u.z << 16); a[5] += __uint_as_float(u.z & 0xffff0000u);
  a[6] += __uint_as_float(u.w << 16); a[7] += __uint_as_float(u.w & 0xffff0000u);
}

// grid.x = total_chunks * (Hq + Hkv); the head varies fastest so that CTAs running together read
// neighbouring 256-byte segments of the same token rows.  A chunk is 16 consecutive blocks of the packed batch, whatever
// sequences they belong to (a chunk per sequence would leave most of a CTA idle on batches of short sequences).
__global__ void __launch_bounds__(kPoolThreads)
pool_project_kernel(SeqMeta m, const uint16_t* __restrict__ q, const uint16_t* __restrict__ k,
                    const float* __restrict__ Wq, const float* __restrict__ Wk, uint16_t* __restrict__ gq,
                    uint16_t* __restrict__ gk) {
  __shared__ __align__(16) float pooled[kPoolChunk][kHeadDim];

  const int heads_total = m.num_q_heads + m.num_kv_heads;
  const int chunk = blockIdx.x / heads_total;
  int hh = blockIdx.x - chunk * heads_total;
  const bool is_q = hh < m.num_q_heads;
  const int H = is_q ? m.num_q_heads : m.num_kv_heads;
  const int h = is_q ? hh : hh - m.num_q_heads;
  const uint16_t* __restrict__ x = is_q ? q : k;
  const float* __restrict__ W = (is_q ? Wq : Wk) + (size_t)h * kHeadDim * kGateDim;
  uint16_t* __restrict__ out = is_q ? gq : gk;
  const size_t plane = (size_t)H * m.total_blocks * kGateDim;   // elements between the hi / mid / lo planes

  const int g0 = chunk * kPoolChunk;                            // first block of the chunk, numbered over the batch
  const int nblk = min(kPoolChunk, m.total_blocks - g0);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int half = lane >> 4, cchunk = lane & 15;
  const size_t row_stride = (size_t)H * kHeadDim;  // elements between consecutive tokens
  bool any = false;

  for (int bi = warp; bi < nblk; bi += kPoolThreads / 32) {
    const int b = find_sequence(m.blk_off, m.batch, g0 + bi);
    const int i = g0 + bi - m.blk_off[b];
    const int s0 = m.cu_seqlens[b], s1 = m.cu_seqlens[b + 1];
    // chunked prefill: q holds the last positions only; query blocks before the chunk are skipped (projected as zeros)
    const int q_first = (m.chunked && is_q) ? m.qoff[b] : 0;
    const int q_shift = (m.chunked && is_q) ? m.qdelta[b] : 0;
    const int t0 = s0 + i * m.block;
    const int cnt = (i < q_first) ? 0 : min(m.block, s1 - t0);
    any |= cnt > 0;
    const uint16_t* base = x + ((ptrdiff_t)t0 + q_shift) * (ptrdiff_t)row_stride + (size_t)h * kHeadDim + cchunk * 8;
    float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
    for (int it = 0; it < m.block / 2; it += 8) {
      uint4 u[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int row = 2 * (it + j) + half;
        u[j] = row < cnt ? ld_stream_16(base + (size_t)row * row_stride) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) acc_bf16x8(a, u[j]);
    }
    const float inv = cnt > 0 ? 1.0f / (float)cnt : 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      a[j] += __shfl_xor_sync(0xffffffffu, a[j], 16);
      a[j] *= inv;
    }
    if (half == 0) {
      float4* dst = reinterpret_cast<float4*>(&pooled[bi][cchunk * 8]);
      dst[0] = make_float4(a[0], a[1], a[2], a[3]);
      dst[1] = make_float4(a[4], a[5], a[6], a[7]);
    }
  }
  if (!__syncthreads_or(any ? 1 : 0)) return;                   // every block of the chunk lies before its queries

  // projection: thread -> output column o, 8 of the 16 blocks
  const int o = threadIdx.x & (kGateDim - 1);
  const int grp = threadIdx.x >> 7;  // 0 or 1
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll 8
  for (int c = 0; c < kHeadDim; ++c) {
    const float w = __ldg(W + (size_t)c * kGateDim + o);
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = fmaf(pooled[grp * 8 + j][c], w, acc[j]);
  }
  const size_t obase = ((size_t)h * m.total_blocks + g0) * kGateDim;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int bi = grp * 8 + j;
    if (bi < nblk) store_split3(out + obase + (size_t)bi * kGateDim + o, plane, acc[j]);
  }
}


// ----------------------------------------------------------------------------------------------- kernel 1, variants
// Sec. 3.1, "Pooling Method Selection" and "Block-level RoPE in AttnGate": the same single pass over Q and K, but
//   * a tensor may be pooled by any subset of {average, max, min}; the pooled vectors are concatenated in that order
//     in the hidden dimension, so the head's gate matrix is [n * d, dg] (n = methods chosen for that tensor);
//   * with rope_theta > 0 the projected vector of block i is rotated as position i with base rope_theta / B
//     (pairs (c, c + dg/2), frequency base^(-2c/dg)); the angle and its sine / cosine are taken in double precision
//     (an fp32 angle near position 2000 would already cost more than the 1e-3 bound on large logits).
// max and min ride along the average's loads: the kernel stays one HBM pass.
__device__ __forceinline__ void max_bf16x8(float (&a)[8], const uint4& u) {
  a[0] = fmaxf(a[0], __uint_as_float(u.x << 16)); a[1] = fmaxf(a[1], __uint_as_float(u.x & 0xffff0000u));
  a[2] = fmaxf(a[2], __uint_as_float(u.y << 16)); a[3] = fmaxf(a[3], __uint_as_float(u.y & 0xffff0000u));
  a[4] = fmaxf(a[4], __uint_as_float(u.z << 16)); a[5] = fmaxf(a[5], __uint_as_float(u.z & 0xffff0000u));
  a[6] = fmaxf(a[6], __uint_as_float(u.w << 16)); a[7] = fmaxf(a[7], __uint_as_float(u.w & 0xffff0000u));
}
__device__ __forceinline__ void min_bf16x8(float (&a)[8], const uint4& u) {
  a[0] = fminf(a[0], __uint_as_float(u.x << 16)); a[1] = fminf(a[1], __uint_as_float(u.x & 0xffff0000u));
  a[2] = fminf(a[2], __uint_as_float(u.y << 16)); a[3] = fminf(a[3], __uint_as_float(u.y & 0xffff0000u));
  a[4] = fminf(a[4], __uint_as_float(u.z << 16)); a[5] = fminf(a[5], __uint_as_float(u.z & 0xffff0000u));
  a[6] = fminf(a[6], __uint_as_float(u.w << 16)); a[7] = fminf(a[7], __uint_as_float(u.w & 0xffff0000u));
}


__global__ void __launch_bounds__(kPoolThreads)
pool_project_ex_kernel(SeqMeta m, const uint16_t* __restrict__ q, const uint16_t* __restrict__ k,
                       const float* __restrict__ Wq, const float* __restrict__ Wk, uint16_t* __restrict__ gq,
                       uint16_t* __restrict__ gk, uint32_t pool_q, uint32_t pool_k, float rope_theta) {
  __shared__ __align__(16) float pooled[kPoolChunk][3 * kHeadDim];
  __shared__ int block_pos[kPoolChunk];                        // position of each block in its sequence (block RoPE)

  const int heads_total = m.num_q_heads + m.num_kv_heads;
  const int chunk = blockIdx.x / heads_total;
  int hh = blockIdx.x - chunk * heads_total;
  const bool is_q = hh < m.num_q_heads;
  const int H = is_q ? m.num_q_heads : m.num_kv_heads;
  const int h = is_q ? hh : hh - m.num_q_heads;
  const uint32_t methods = is_q ? pool_q : pool_k;
  const int nparts = __popc(methods);
  const int width = nparts * kHeadDim;                       // rows of the head's gate matrix
  const uint16_t* __restrict__ x = is_q ? q : k;
  const float* __restrict__ W = (is_q ? Wq : Wk) + (size_t)h * width * kGateDim;
  uint16_t* __restrict__ out = is_q ? gq : gk;
  const size_t plane = (size_t)H * m.total_blocks * kGateDim;   // elements between the hi / mid / lo planes
  // offsets of the parts inside the concatenated vector (order: average, max, min)
  const int off_avg = 0;
  const int off_max = (methods & SEER_POOL_AVG) ? kHeadDim : 0;
  const int off_min = off_max + ((methods & SEER_POOL_MAX) ? kHeadDim : 0);

  const int g0 = chunk * kPoolChunk;                            // first block of the chunk, numbered over the batch
  const int nblk = min(kPoolChunk, m.total_blocks - g0);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int half = lane >> 4, cchunk = lane & 15;
  const size_t row_stride = (size_t)H * kHeadDim;
  bool any = false;

  for (int bi = warp; bi < nblk; bi += kPoolThreads / 32) {
    const int b = find_sequence(m.blk_off, m.batch, g0 + bi);
    const int i = g0 + bi - m.blk_off[b];
    const int s0 = m.cu_seqlens[b], s1 = m.cu_seqlens[b + 1];
    // chunked prefill: q holds the last positions only; query blocks before the chunk are skipped (projected as zeros)
    const int q_first = (m.chunked && is_q) ? m.qoff[b] : 0;
    const int q_shift = (m.chunked && is_q) ? m.qdelta[b] : 0;
    const int t0 = s0 + i * m.block;
    const int cnt = (i < q_first) ? 0 : min(m.block, s1 - t0);
    any |= cnt > 0;
    if (lane == 0) block_pos[bi] = i;
    const uint16_t* base = x + ((ptrdiff_t)t0 + q_shift) * (ptrdiff_t)row_stride + (size_t)h * kHeadDim + cchunk * 8;
    float a[8], hi[8], lo[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) { a[j] = 0.f; hi[j] = -CUDART_INF_F; lo[j] = CUDART_INF_F; }
#pragma unroll 1
    for (int it = 0; it < m.block / 2; it += 8) {
      uint4 u[8];
      bool live[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int row = 2 * (it + j) + half;
        live[j] = row < cnt;
        u[j] = live[j] ? ld_stream_16(base + (size_t)row * row_stride) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        acc_bf16x8(a, u[j]);
        if (live[j]) { max_bf16x8(hi, u[j]); min_bf16x8(lo, u[j]); }   // rows past the end of the sequence take no part
      }
    }
    const float inv = cnt > 0 ? 1.0f / (float)cnt : 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      a[j] = (a[j] + __shfl_xor_sync(0xffffffffu, a[j], 16)) * inv;
      hi[j] = fmaxf(hi[j], __shfl_xor_sync(0xffffffffu, hi[j], 16));
      lo[j] = fminf(lo[j], __shfl_xor_sync(0xffffffffu, lo[j], 16));
      if (cnt == 0) { hi[j] = 0.f; lo[j] = 0.f; }      // a skipped block: zeros, not the identities of max and min
    }
    if (half == 0) {
      if (methods & SEER_POOL_AVG) {
        float4* dst = reinterpret_cast<float4*>(&pooled[bi][off_avg + cchunk * 8]);
        dst[0] = make_float4(a[0], a[1], a[2], a[3]); dst[1] = make_float4(a[4], a[5], a[6], a[7]);
      }
      if (methods & SEER_POOL_MAX) {
        float4* dst = reinterpret_cast<float4*>(&pooled[bi][off_max + cchunk * 8]);
        dst[0] = make_float4(hi[0], hi[1], hi[2], hi[3]); dst[1] = make_float4(hi[4], hi[5], hi[6], hi[7]);
      }
      if (methods & SEER_POOL_MIN) {
        float4* dst = reinterpret_cast<float4*>(&pooled[bi][off_min + cchunk * 8]);
        dst[0] = make_float4(lo[0], lo[1], lo[2], lo[3]); dst[1] = make_float4(lo[4], lo[5], lo[6], lo[7]);
      }
    }
  }
  if (!__syncthreads_or(any ? 1 : 0)) return;                   // every block of the chunk lies before its queries

  // projection: thread -> output column o, 8 of the 16 blocks
  const int o = threadIdx.x & (kGateDim - 1);
  const int grp = threadIdx.x >> 7;  // 0 or 1
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll 8
  for (int c = 0; c < width; ++c) {
    const float w = __ldg(W + (size_t)c * kGateDim + o);
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = fmaf(pooled[grp * 8 + j][c], w, acc[j]);
  }
  if (rope_theta > 0.f) {
    // rotate (o, o + dg/2) pairs: the partner's value goes through shared memory (the pooled vectors are no longer needed)
    __syncthreads();
#pragma unroll
    for (int j = 0; j < 8; ++j) pooled[grp * 8 + j][o] = acc[j];
    __syncthreads();
    const int f = o & (kGateDim / 2 - 1);
    const double freq = pow((double)rope_theta / (double)m.block, -2.0 * (double)f / (double)kGateDim);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int bi = grp * 8 + j;
      double sn, cs;
      sincos((double)(bi < nblk ? block_pos[bi] : 0) * freq, &sn, &cs);
      const float partner = pooled[bi][o ^ (kGateDim / 2)];
      // first half: x1 cos - x2 sin; second half: x2 cos + x1 sin
      acc[j] = (o < kGateDim / 2) ? (float)((double)acc[j] * cs - (double)partner * sn)
                                  : (float)((double)acc[j] * cs + (double)partner * sn);
    }
  }
  const size_t obase = ((size_t)h * m.total_blocks + g0) * kGateDim;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int bi = grp * 8 + j;
    if (bi < nblk) store_split3(out + obase + (size_t)bi * kGateDim + o, plane, acc[j]);
  }
}

// ----------------------------------------------------------------------------------------------- kernel 2
// 64 score rows of one head per CTA, walked over the causal columns 64 at a time (the next column tile is copied in
// while the current one is multiplied).  Eight warps; warp w owns rows 16 (w & 3) .. + 15 and the column half w >> 2
// (mma.sync m16n8k16, bf16 in, fp32 out): per 16-wide k step three A fragments (hi, mid, lo planes of gq) and, for each
// of its four 8-column groups, three B fragments of gk; six MMAs per group.  Tiles sit in shared memory as
// [plane][64 rows][128 k] bf16 with the 16-byte chunks of a row XOR-swizzled by the row (conflict-free ldmatrix).
constexpr int kScoreThreads = 256;
constexpr int kPlaneTile = kScoreTile * kGateDim * 2;                       // 16 KB: one plane of a 64 x 128 tile
constexpr int kScoreSmem = 9 * kPlaneTile + 6 * kScoreTile * (int)sizeof(float);   // A planes, two sets of B planes, row statistics

__device__ __forceinline__ uint32_t gs_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t gs_tile_off(int row, int chunk) { return (uint32_t)(row * 256 + ((chunk ^ (row & 7)) << 4)); }
__device__ __forceinline__ void gs_ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void gs_mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// Copies rows r0 .. r0+63 of the three planes of src ([rows][128] bf16 each, `plane` elements apart) into dst; rows at or
// beyond rows_valid are zero-filled.
__device__ __forceinline__ void gs_load_planes(uint32_t dst, const uint16_t* __restrict__ src, size_t plane, int r0,
                                               int rows_valid) {
  for (int idx = threadIdx.x; idx < 3 * kScoreTile * 16; idx += kScoreThreads) {
    const int pl = idx / (kScoreTile * 16), rem = idx - pl * (kScoreTile * 16);
    const int row = rem >> 4, chunk = rem & 15;
    const bool ok = row < rows_valid;
    const uint16_t* g = src + (size_t)pl * plane + (size_t)(r0 + (ok ? row : 0)) * kGateDim + chunk * 8;
    const int sz = ok ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst + (uint32_t)pl * kPlaneTile + gs_tile_off(row, chunk)),
                 "l"(g), "r"(sz) : "memory");
  }
}

// grid.x = tiles * band.heads (head fastest; tiles are visited from the last rows to the first).  A tile is 64
// consecutive block rows of the packed batch, counted from band.blk_lo, whatever sequences they belong to (a tile per
// sequence would leave most of a CTA idle on batches of short sequences): row r of the tile is query block i_r of
// sequence b_r, its causal columns are that sequence's blocks 0..i_r, i.e. the blocks seq_start_r .. r of the batch.  The
// CTA walks the column tiles from the sequence start of its first row to its last row; entries of other sequences are
// masked.  The whole problem is the band (0, total_blocks, 0, Hq, 0).  Scores are written at their offset in the full
// matrix minus band.score_base.
__global__ void __launch_bounds__(kScoreThreads)
gate_scores_kernel(SeqMeta m, ScoreBand band, const uint16_t* __restrict__ gq, const uint16_t* __restrict__ gk,
                   float* __restrict__ scores) {
  extern __shared__ __align__(128) unsigned char gs_smem[];
  const uint32_t sA = gs_smem_u32(gs_smem), sB0 = sA + 3 * kPlaneTile;
  float* row_m = reinterpret_cast<float*>(gs_smem + 9 * kPlaneTile);     // [64]
  float* row_l = row_m + kScoreTile;                                      // [64]
  float* part_m = row_l + kScoreTile;                                     // [2 column halves][64]
  float* part_l = part_m + 2 * kScoreTile;
  __shared__ int row_start[kScoreTile];        // first block of the row's sequence, numbered over the batch
  __shared__ int row_last[kScoreTile];         // the row's own block (its last causal column); -1: nothing to compute
  __shared__ long long row_off[kScoreTile];    // element offset of the row's scores (column 0) in the buffer

  const int tiles = (band.blk_hi - band.blk_lo + kScoreTile - 1) / kScoreTile;
  const int tile = tiles - 1 - (int)(blockIdx.x / band.heads);
  const int h = band.head_lo + (int)(blockIdx.x % band.heads);
  const int g = h / m.group;
  const int r0 = band.blk_lo + tile * kScoreTile;                          // first block row of the tile
  const int rows_valid = min(kScoreTile, band.blk_hi - r0);
  int live = 0;
  if (threadIdx.x < kScoreTile) {
    const int r = threadIdx.x;
    int start = 0, last = -1;
    long long off = 0;
    if (r < rows_valid) {
      const int gb = r0 + r;
      const int b = find_sequence(m.blk_off, m.batch, gb);
      const int nb = m.blk_off[b + 1] - m.blk_off[b];
      const int i = gb - m.blk_off[b];
      start = m.blk_off[b];
      off = m.score_off[b] + ((long long)h * nb + i) * nb - band.score_base;
      if (!(m.chunked && i < m.qoff[b])) last = gb;                       // chunked prefill: rows before the chunk are skipped
    }
    row_start[r] = start; row_last[r] = last; row_off[r] = off;
    live = last >= 0;
  }
  if (!__syncthreads_or(live)) return;                                     // a tile of query blocks before their chunks
  const size_t plane_q = (size_t)m.num_q_heads * m.total_blocks * kGateDim;
  const size_t plane_k = (size_t)m.num_kv_heads * m.total_blocks * kGateDim;
  const uint16_t* gq_h = gq + (size_t)h * m.total_blocks * kGateDim;
  const uint16_t* gk_g = gk + (size_t)g * m.total_blocks * kGateDim;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int wr = warp & 3, wc = warp >> 2;                               // row group, column half
  const int gid = lane >> 2, tig = lane & 3;
  const float scale = rsqrtf((float)kGateDim);

  const int first_col = row_start[0];                                     // rows ascend, so do their sequence starts
  const int last_col = r0 + rows_valid - 1;
  gs_load_planes(sA, gq_h, plane_q, r0, rows_valid);
  gs_load_planes(sB0, gk_g, plane_k, first_col, min(kScoreTile, last_col + 1 - first_col));
  asm volatile("cp.async.commit_group;" ::: "memory");

  // the two rows of this thread: r = wr * 16 + gid + 8 e
  int my_start[2], my_last[2];
  long long my_off[2];
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const int r = wr * 16 + gid + e * 8;
    my_start[e] = row_start[r]; my_last[e] = row_last[r]; my_off[e] = row_off[r];
  }
  float run_m[2] = {-CUDART_INF_F, -CUDART_INF_F}, run_l[2] = {0.f, 0.f};
  // the warp's A fragments (16 rows x 128 k, three planes) stay in registers for the whole row tile
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();
  uint32_t a[8][3][4];
#pragma unroll
  for (int ks = 0; ks < 8; ++ks)
#pragma unroll
    for (int pl = 0; pl < 3; ++pl) {
      const int row = wr * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
      gs_ldsm_x4(a[ks][pl], sA + (uint32_t)pl * kPlaneTile + gs_tile_off(row, ks * 2 + (lane >> 4)));
    }
  int buf = 0;
  for (int j0 = first_col; j0 <= last_col; j0 += kScoreTile, buf ^= 1) {
    const uint32_t sB = sB0 + (uint32_t)buf * 3 * kPlaneTile;
    __syncthreads();                                   // the other B buffer's fragments have been read
    if (j0 + kScoreTile <= last_col)
      gs_load_planes(sB0 + (uint32_t)(buf ^ 1) * 3 * kPlaneTile, gk_g, plane_k, j0 + kScoreTile,
                     min(kScoreTile, last_col + 1 - j0 - kScoreTile));
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 1;" ::: "memory");   // everything but the copy just started has landed
    __syncthreads();
    // two accumulators per 8-column group: the small terms and the large ones are independent MMA chains (the kernel is
    // bound by the latency of dependent MMAs, eight warps per SM), added once per column tile, small to large
    float acc[4][4], accs[4][4];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
      for (int c = 0; c < 4; ++c) { acc[nt][c] = 0.f; accs[nt][c] = 0.f; }
#pragma unroll
    for (int kk = 0; kk < 8; kk += 2) {                // two 16-wide k steps per pass (one B ldmatrix.x4 covers both)
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        uint32_t bf[3][4];                             // [plane]: b0, b1 of step kk, then of step kk + 1
#pragma unroll
        for (int pl = 0; pl < 3; ++pl)
          gs_ldsm_x4(bf[pl], sB + (uint32_t)pl * kPlaneTile + gs_tile_off((wc * 4 + nt) * 8 + (lane & 7), kk * 2 + (lane >> 3)));
#pragma unroll
        for (int s2 = 0; s2 < 2; ++s2) {
          // small chain: hi*lo, lo*hi, mid*mid; large chain: hi*mid, mid*hi, hi*hi
          gs_mma(accs[nt], a[kk + s2][0], bf[2][2 * s2], bf[2][2 * s2 + 1]);
          gs_mma(acc[nt], a[kk + s2][0], bf[1][2 * s2], bf[1][2 * s2 + 1]);
          gs_mma(accs[nt], a[kk + s2][2], bf[0][2 * s2], bf[0][2 * s2 + 1]);
          gs_mma(acc[nt], a[kk + s2][1], bf[0][2 * s2], bf[0][2 * s2 + 1]);
          gs_mma(accs[nt], a[kk + s2][1], bf[1][2 * s2], bf[1][2 * s2 + 1]);
          gs_mma(acc[nt], a[kk + s2][0], bf[0][2 * s2], bf[0][2 * s2 + 1]);
        }
      }
    }
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[nt][c] += accs[nt][c];
    // thread holds rows (gid, gid + 8) of the warp's 16 and columns (4 wc + nt) * 8 + 2 * tig + {0, 1} of the tile
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      if (my_last[e] < 0) continue;
      float x[4][2];
      float tmax = -CUDART_INF_F;
#pragma unroll
      for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          const int j = j0 + (wc * 4 + nt) * 8 + 2 * tig + c;              // block of the batch
          x[nt][c] = (j >= my_start[e] && j <= my_last[e]) ? acc[nt][2 * e + c] * scale : -CUDART_INF_F;
          tmax = fmaxf(tmax, x[nt][c]);
        }
      if (tmax == -CUDART_INF_F) continue;             // nothing causal for this thread in this tile
      const float nm = fmaxf(run_m[e], tmax);
      float sum = 0.f;
#pragma unroll
      for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int c = 0; c < 2; ++c) sum += x[nt][c] == -CUDART_INF_F ? 0.f : __expf(x[nt][c] - nm);
      run_l[e] = run_l[e] * __expf(run_m[e] - nm) + sum;  // exp(-inf) = 0 on the first contribution
      run_m[e] = nm;
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        const int j = j0 + (wc * 4 + nt) * 8 + 2 * tig;
        const long long at = my_off[e] + (j - my_start[e]);                // element offset of (row, j)
        float* dst = scores + at;
        const bool in0 = j >= my_start[e] && j <= my_last[e], in1 = j + 1 >= my_start[e] && j + 1 <= my_last[e];
        if (in0 && in1 && (at & 1) == 0) {
          *reinterpret_cast<float2*>(dst) = make_float2(x[nt][0], x[nt][1]);
        } else {
          if (in0) dst[0] = x[nt][0];
          if (in1) dst[1] = x[nt][1];
        }
      }
    }
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  // combine the partial (max, sum) pairs of each row: the four lanes of a quad, then the two column halves
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    float mm = run_m[e], ll = run_l[e];
#pragma unroll
    for (int off = 1; off < 4; off <<= 1) {
      const float om = __shfl_xor_sync(0xffffffffu, mm, off);
      const float ol = __shfl_xor_sync(0xffffffffu, ll, off);
      const float nm = fmaxf(mm, om);
      const float fa = (mm == -CUDART_INF_F) ? 0.f : __expf(mm - nm);
      const float fb = (om == -CUDART_INF_F) ? 0.f : __expf(om - nm);
      ll = ll * fa + ol * fb;
      mm = nm;
    }
    if (tig == 0) { part_m[wc * kScoreTile + wr * 16 + gid + e * 8] = mm; part_l[wc * kScoreTile + wr * 16 + gid + e * 8] = ll; }
  }
  __syncthreads();
  if (threadIdx.x < kScoreTile) {
    const float m0 = part_m[threadIdx.x], m1 = part_m[kScoreTile + threadIdx.x];
    const float nm = fmaxf(m0, m1);
    const float f0 = (m0 == -CUDART_INF_F) ? 0.f : __expf(m0 - nm), f1 = (m1 == -CUDART_INF_F) ? 0.f : __expf(m1 - nm);
    row_m[threadIdx.x] = nm;
    row_l[threadIdx.x] = part_l[threadIdx.x] * f0 + part_l[kScoreTile + threadIdx.x] * f1;
  }
  __syncthreads();
  // normalise in place: the logits this CTA just wrote are re-read (L2) and replaced by exp(x - m) / l; a warp per row,
  // four columns per lane and step, so that many independent loads are in flight
  for (int r = warp; r < rows_valid; r += kScoreThreads / 32) {
    if (row_last[r] < 0) continue;
    const int n = row_last[r] - row_start[r] + 1;      // causal columns of the row
    const float mm = row_m[r];
    const float inv = 1.0f / row_l[r];
    float* dst = scores + row_off[r];
    if ((row_off[r] & 3) == 0) {
      const int full = n & ~3;                         // columns 0 .. full-1 in whole float4s
      int j = lane * 4;
      for (; j + 384 < full; j += 512) {               // four loads in flight per lane (the loop is bound by their latency)
        float4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = *reinterpret_cast<float4*>(dst + j + u * 128);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          v[u].x = __expf(v[u].x - mm) * inv; v[u].y = __expf(v[u].y - mm) * inv;
          v[u].z = __expf(v[u].z - mm) * inv; v[u].w = __expf(v[u].w - mm) * inv;
          *reinterpret_cast<float4*>(dst + j + u * 128) = v[u];
        }
      }
      for (; j < full; j += 128) {
        float4 v = *reinterpret_cast<float4*>(dst + j);
        v.x = __expf(v.x - mm) * inv; v.y = __expf(v.y - mm) * inv; v.z = __expf(v.z - mm) * inv; v.w = __expf(v.w - mm) * inv;
        *reinterpret_cast<float4*>(dst + j) = v;
      }
      for (int j = full + lane; j < n; j += 32) dst[j] = __expf(dst[j] - mm) * inv;
    } else {
      for (int j = lane; j < n; j += 32) dst[j] = __expf(dst[j] - mm) * inv;
    }
  }
}

int launch_gate(seer_ctx* ctx, const SeqMeta& m, const void* q, const void* k, const float* Wq, const float* Wk,
                float* scores, void* ws, cudaStream_t stream) {
  (void)ctx;
  // three bf16 planes per tensor (hi, mid, lo of the fp32 value)
  size_t gq_bytes = ((size_t)m.num_q_heads * m.total_blocks * kGateDim * 6 + 255) / 256 * 256;
  uint16_t* gq = (uint16_t*)ws;
  uint16_t* gk = (uint16_t*)((char*)ws + gq_bytes);
  const unsigned grid1 = (unsigned)m.total_chunks * (unsigned)(m.num_q_heads + m.num_kv_heads);
  pool_project_kernel<<<grid1, kPoolThreads, 0, stream>>>(m, (const uint16_t*)q, (const uint16_t*)k, Wq, Wk, gq, gk);
  if (scores == nullptr) {                             // projection only: the scores follow band by band
    cudaError_t e0 = cudaGetLastError();
    return e0 == cudaSuccess ? 1 : -(int)e0;
  }
  const ScoreBand all = {0, m.total_blocks, 0, m.num_q_heads, 0};
  const unsigned grid2 = (unsigned)((m.total_blocks + kScoreTile - 1) / kScoreTile) * (unsigned)m.num_q_heads;
  gate_scores_kernel<<<grid2, kScoreThreads, kScoreSmem, stream>>>(m, all, gq, gk, scores);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 2 : -(int)e;
}

int launch_gate_ex(seer_ctx* ctx, const SeqMeta& m, const seer_gate_options& opt, const void* q, const void* k,
                   const float* Wq, const float* Wk, float* scores, void* ws, cudaStream_t stream) {
  (void)ctx;
  // three bf16 planes per tensor (hi, mid, lo of the fp32 value)
  size_t gq_bytes = ((size_t)m.num_q_heads * m.total_blocks * kGateDim * 6 + 255) / 256 * 256;
  uint16_t* gq = (uint16_t*)ws;
  uint16_t* gk = (uint16_t*)((char*)ws + gq_bytes);
  const unsigned grid1 = (unsigned)m.total_chunks * (unsigned)(m.num_q_heads + m.num_kv_heads);
  pool_project_ex_kernel<<<grid1, kPoolThreads, 0, stream>>>(m, (const uint16_t*)q, (const uint16_t*)k, Wq, Wk, gq, gk,
                                                              opt.pool_q, opt.pool_k, opt.rope_theta);
  if (scores == nullptr) {                             // projection only: the scores follow band by band
    cudaError_t e0 = cudaGetLastError();
    return e0 == cudaSuccess ? 1 : -(int)e0;
  }
  const ScoreBand all = {0, m.total_blocks, 0, m.num_q_heads, 0};
  const unsigned grid2 = (unsigned)((m.total_blocks + kScoreTile - 1) / kScoreTile) * (unsigned)m.num_q_heads;
  gate_scores_kernel<<<grid2, kScoreThreads, kScoreSmem, stream>>>(m, all, gq, gk, scores);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 2 : -(int)e;
}

// Scores of one band from the projected vectors launch_gate_ex(scores = nullptr) left in `ws`.
int launch_gate_scores_band(const SeqMeta& m, const ScoreBand& band, const void* ws, float* scores, cudaStream_t stream) {
  size_t gq_bytes = ((size_t)m.num_q_heads * m.total_blocks * kGateDim * 6 + 255) / 256 * 256;
  const uint16_t* gq = (const uint16_t*)ws;
  const uint16_t* gk = (const uint16_t*)((const char*)ws + gq_bytes);
  const unsigned grid = (unsigned)((band.blk_hi - band.blk_lo + kScoreTile - 1) / kScoreTile) * (unsigned)band.heads;
  if (grid == 0) return 0;
  gate_scores_kernel<<<grid, kScoreThreads, kScoreSmem, stream>>>(m, band, gq, gk, scores);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 1 : -(int)e;
}

// ----------------------------------------------------------------------------------------------- allocation-free variant
// Scratch for seer_gate_scores_static lives in the library image: every GPU that loads the library carries these
// bytes until the process exits.  Host code must never hand the symbol itself to a kernel; its device address is
// looked up once per device with cudaGetSymbolAddress.
constexpr int kStaticMaxBatch = SEER_STATIC_MAX_BATCH;
constexpr size_t kStaticMetaBytes = 16 * 1024;                              // cu_seqlens and the two offset arrays (block, score)
constexpr size_t kStaticScratchBytes = (size_t)SEER_STATIC_SCRATCH_BYTES;   // projected pooled Q and K, three bf16 planes each (768 B per (head, block))
static __device__ __align__(256) unsigned char g_static_scratch[kStaticMetaBytes + kStaticScratchBytes];

constexpr int kStaticMaxDevices = 64;
static std::mutex g_static_mutex;
static void* g_static_addr[kStaticMaxDevices];     // device address of g_static_scratch, per device ordinal
static bool g_static_ready[kStaticMaxDevices];

// Once per device, with that device current: resolve the array's device address and lift the score kernel's
// shared-memory limit.  Neither call allocates.
static seer_status static_setup(int dev, unsigned char** out) {
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_ready[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) return SEER_ERR_CUDA;
    if (cudaFuncSetAttribute(gate_scores_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kScoreSmem) != cudaSuccess)
      return SEER_ERR_CUDA;
    g_static_addr[dev] = ptr;
    g_static_ready[dev] = true;
  }
  *out = (unsigned char*)g_static_addr[dev];
  return SEER_OK;
}

seer_status gate_scores_static(const seer_shape* shape, const void* q, const void* k, const float* Wq, const float* Wk,
                               float* scores, cudaStream_t stream) {
  ShapeTotals t;
  seer_status st = shape_totals(shape, &t);
  if (st != SEER_OK) return st;
  if (shape->cu_seqlens_q_host) return SEER_ERR_UNSUPPORTED;   // no chunked prefill through the built-in scratch
  if (t.total_blocks == 0) return SEER_OK;
  if (!q || !k || !Wq || !Wk || !scores) return SEER_ERR_INVALID_ARG;
  // sizes beyond the built-in scratch are refused, never truncated
  if (shape->batch > kStaticMaxBatch || gate_workspace_bytes(t, shape) > kStaticScratchBytes) return SEER_ERR_WORKSPACE;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kStaticMaxDevices) return SEER_ERR_CUDA;
  unsigned char* base = nullptr;
  st = static_setup(dev, &base);
  if (st != SEER_OK) return st;

  // per-batch offsets, built in a host staging area that lives as long as the library (one per device, so that the
  // copy below never refers to a stack frame that has gone) and copied into the head of the array
  struct HostMeta {
    int32_t cu[kStaticMaxBatch + 4], blk[kStaticMaxBatch + 4];
    int64_t score[kStaticMaxBatch + 2];
  };
  static_assert(sizeof(HostMeta) <= kStaticMetaBytes, "metadata region too small");
  static HostMeta g_host_meta[kStaticMaxDevices];
  std::lock_guard<std::mutex> lock(g_static_mutex);   // (static_setup has released it)
  HostMeta& hm = g_host_meta[dev];
  hm.blk[0] = 0;
  hm.score[0] = 0;
  for (int b = 0; b < shape->batch; ++b) {
    hm.cu[b] = shape->cu_seqlens_host[b];
    const int32_t nb = (shape->cu_seqlens_host[b + 1] - shape->cu_seqlens_host[b] + shape->block - 1) / shape->block;
    hm.blk[b + 1] = hm.blk[b] + nb;
    hm.score[b + 1] = hm.score[b] + (int64_t)shape->num_q_heads * nb * nb;
  }
  hm.cu[shape->batch] = shape->cu_seqlens_host[shape->batch];
  // pageable source: the runtime stages the bytes before returning, so the next call may refill the staging area
  if (cudaMemcpyAsync(base, &hm, sizeof(HostMeta), cudaMemcpyHostToDevice, stream) != cudaSuccess) return SEER_ERR_CUDA;

  SeqMeta m;
  m.cu_seqlens = (const int32_t*)(base + offsetof(HostMeta, cu));
  m.blk_off = (const int32_t*)(base + offsetof(HostMeta, blk));
  m.score_off = (const int64_t*)(base + offsetof(HostMeta, score));
  m.batch = shape->batch;
  m.num_q_heads = shape->num_q_heads;
  m.num_kv_heads = shape->num_kv_heads;
  m.group = shape->num_q_heads / shape->num_kv_heads;
  m.total_tokens = (int32_t)t.total_tokens;
  m.total_blocks = (int32_t)t.total_blocks;
  m.total_chunks = (int32_t)t.total_chunks;
  m.max_nb = t.max_nb;
  m.rows = t.rows;
  m.score_elems = t.score_elems;
  m.softmax_scale = 0.f;   // unused by the gate
  m.block = shape->block;
  m.qoff = nullptr; m.qdelta = nullptr; m.chunked = 0;
  m.total_q_tokens = (int32_t)t.total_tokens;
  m.wait_limit_us = 0u; m.lose_v_copy = -1;   // unused by the gate
  // The two kernels below are the ones seer_gate_scores launches; only the scratch pointer differs.  Nothing in the
  // scratch has to start at zero: the first kernel writes every projected vector the second one reads.
  const int n = launch_gate(nullptr, m, q, k, Wq, Wk, scores, base + kStaticMetaBytes, stream);
  return n < 0 ? SEER_ERR_CUDA : SEER_OK;
}

seer_status init_gate(seer_ctx* ctx) {
  (void)ctx;
  cudaError_t e = cudaFuncSetAttribute(gate_scores_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kScoreSmem);
  return e == cudaSuccess ? SEER_OK : SEER_ERR_CUDA;
}

}  // namespace seer

extern "C" seer_status seer_gate_scores_static(const seer_shape* shape, const void* q, const void* k, const float* Wq,
                                               const float* Wk, float* scores, void* stream) {
  if (!shape) return SEER_ERR_INVALID_ARG;
  return seer::gate_scores_static(shape, q, k, Wq, Wk, scores, (cudaStream_t)stream);
}
