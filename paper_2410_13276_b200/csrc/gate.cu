// AttnGate (Sec. 3.1, Eq. 1) in two kernels:
//   pool_project_kernel : streams Q and K once (HBM-bound), average-pools each 64-token block per head and
//                         multiplies the pooled vectors by the head's gate matrix  -> gq, gk (fp32 workspace)
//   gate_scores_kernel  : logits = gq gk^T / sqrt(dg) over the causal blocks, row softmax -> scores
// All gate arithmetic is fp32 on the CUDA cores (tensor-core bf16/tf32 would not hold the 1e-3 relative bound
// on softmax outputs when logits reach tens).
#include <math_constants.h>

#include <cstddef>
#include <mutex>

#include "seer_internal.cuh"

namespace seer {

// ----------------------------------------------------------------------------------------------- kernel 1
constexpr int kPoolThreads = 256;

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
// neighbouring 256-byte segments of the same token rows.
__global__ void __launch_bounds__(kPoolThreads)
pool_project_kernel(SeqMeta m, const uint16_t* __restrict__ q, const uint16_t* __restrict__ k,
                    const float* __restrict__ Wq, const float* __restrict__ Wk, float* __restrict__ gq,
                    float* __restrict__ gk) {
  __shared__ __align__(16) float pooled[kPoolChunk][kHeadDim];

  const int heads_total = m.num_q_heads + m.num_kv_heads;
  const int chunk = blockIdx.x / heads_total;
  int hh = blockIdx.x - chunk * heads_total;
  const bool is_q = hh < m.num_q_heads;
  const int H = is_q ? m.num_q_heads : m.num_kv_heads;
  const int h = is_q ? hh : hh - m.num_q_heads;
  const uint16_t* __restrict__ x = is_q ? q : k;
  const float* __restrict__ W = (is_q ? Wq : Wk) + (size_t)h * kHeadDim * kGateDim;
  float* __restrict__ out = is_q ? gq : gk;

  const int b = find_sequence(m.chunk_off, m.batch, chunk);
  const int s0 = m.cu_seqlens[b], s1 = m.cu_seqlens[b + 1];
  const int nb = m.blk_off[b + 1] - m.blk_off[b];
  const int i0 = (chunk - m.chunk_off[b]) * kPoolChunk;
  const int nblk = min(kPoolChunk, nb - i0);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int half = lane >> 4, cchunk = lane & 15;
  const size_t row_stride = (size_t)H * kHeadDim;  // elements between consecutive tokens

  for (int bi = warp; bi < nblk; bi += kPoolThreads / 32) {
    const int t0 = s0 + (i0 + bi) * kBlock;
    const int cnt = min(kBlock, s1 - t0);
    const uint16_t* base = x + (size_t)t0 * row_stride + (size_t)h * kHeadDim + cchunk * 8;
    float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
    for (int it = 0; it < kBlock / 2; it += 8) {
      uint4 u[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int row = 2 * (it + j) + half;
        u[j] = row < cnt ? ld_stream_16(base + (size_t)row * row_stride) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) acc_bf16x8(a, u[j]);
    }
    const float inv = 1.0f / (float)cnt;
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
  __syncthreads();

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
  const size_t obase = ((size_t)h * m.total_blocks + m.blk_off[b] + i0) * kGateDim;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int bi = grp * 8 + j;
    if (bi < nblk) out[obase + (size_t)bi * kGateDim + o] = acc[j];
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

constexpr int kPoolExSmem = kPoolChunk * 3 * kHeadDim * (int)sizeof(float);   // 24 KB: [16 blocks][up to 3 parts][128]

__global__ void __launch_bounds__(kPoolThreads)
pool_project_ex_kernel(SeqMeta m, const uint16_t* __restrict__ q, const uint16_t* __restrict__ k,
                       const float* __restrict__ Wq, const float* __restrict__ Wk, float* __restrict__ gq,
                       float* __restrict__ gk, uint32_t pool_q, uint32_t pool_k, float rope_theta) {
  __shared__ __align__(16) float pooled[kPoolChunk][3 * kHeadDim];

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
  float* __restrict__ out = is_q ? gq : gk;
  // offsets of the parts inside the concatenated vector (order: average, max, min)
  const int off_avg = 0;
  const int off_max = (methods & SEER_POOL_AVG) ? kHeadDim : 0;
  const int off_min = off_max + ((methods & SEER_POOL_MAX) ? kHeadDim : 0);

  const int b = find_sequence(m.chunk_off, m.batch, chunk);
  const int s0 = m.cu_seqlens[b], s1 = m.cu_seqlens[b + 1];
  const int nb = m.blk_off[b + 1] - m.blk_off[b];
  const int i0 = (chunk - m.chunk_off[b]) * kPoolChunk;
  const int nblk = min(kPoolChunk, nb - i0);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int half = lane >> 4, cchunk = lane & 15;
  const size_t row_stride = (size_t)H * kHeadDim;

  for (int bi = warp; bi < nblk; bi += kPoolThreads / 32) {
    const int t0 = s0 + (i0 + bi) * kBlock;
    const int cnt = min(kBlock, s1 - t0);
    const uint16_t* base = x + (size_t)t0 * row_stride + (size_t)h * kHeadDim + cchunk * 8;
    float a[8], hi[8], lo[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) { a[j] = 0.f; hi[j] = -CUDART_INF_F; lo[j] = CUDART_INF_F; }
#pragma unroll 1
    for (int it = 0; it < kBlock / 2; it += 8) {
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
    const float inv = 1.0f / (float)cnt;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      a[j] = (a[j] + __shfl_xor_sync(0xffffffffu, a[j], 16)) * inv;
      hi[j] = fmaxf(hi[j], __shfl_xor_sync(0xffffffffu, hi[j], 16));
      lo[j] = fminf(lo[j], __shfl_xor_sync(0xffffffffu, lo[j], 16));
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
  __syncthreads();

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
    const double freq = pow((double)rope_theta / (double)kBlock, -2.0 * (double)f / (double)kGateDim);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int bi = grp * 8 + j;
      double sn, cs;
      sincos((double)(i0 + bi) * freq, &sn, &cs);
      const float partner = pooled[bi][o ^ (kGateDim / 2)];
      // first half: x1 cos - x2 sin; second half: x2 cos + x1 sin
      acc[j] = (o < kGateDim / 2) ? (float)((double)acc[j] * cs - (double)partner * sn)
                                  : (float)((double)acc[j] * cs + (double)partner * sn);
    }
  }
  const size_t obase = ((size_t)h * m.total_blocks + m.blk_off[b] + i0) * kGateDim;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int bi = grp * 8 + j;
    if (bi < nblk) out[obase + (size_t)bi * kGateDim + o] = acc[j];
  }
}

// ----------------------------------------------------------------------------------------------- kernel 2
constexpr int kScoreThreads = 256;
constexpr int kScoreSmem = 2 * kGateDim * kScoreTile * (int)sizeof(float) + 2 * kScoreTile * (int)sizeof(float);

// Loads a [64 rows x 128] fp32 tile (rows r0.. of src, row stride kGateDim) transposed into dst[k][row].
__device__ __forceinline__ void load_tile_transposed(float* dst, const float* __restrict__ src, int r0, int rows_valid) {
  for (int idx = threadIdx.x; idx < kScoreTile * (kGateDim / 4); idx += kScoreThreads) {
    const int row = idx & (kScoreTile - 1);
    const int k4 = idx / kScoreTile;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (row < rows_valid) v = __ldg(reinterpret_cast<const float4*>(src + (size_t)(r0 + row) * kGateDim) + k4);
    dst[(k4 * 4 + 0) * kScoreTile + row] = v.x;
    dst[(k4 * 4 + 1) * kScoreTile + row] = v.y;
    dst[(k4 * 4 + 2) * kScoreTile + row] = v.z;
    dst[(k4 * 4 + 3) * kScoreTile + row] = v.w;
  }
}

// grid.x = total_tiles * Hq (head fastest; tiles are visited from the last rows, the longest, to the first)
__global__ void __launch_bounds__(kScoreThreads)
gate_scores_kernel(SeqMeta m, const float* __restrict__ gq, const float* __restrict__ gk, float* __restrict__ scores) {
  extern __shared__ __align__(16) float smem[];
  float* As = smem;                              // [128][64]  gq tile, k-major
  float* Bs = smem + kGateDim * kScoreTile;      // [128][64]  gk tile, k-major
  float* row_m = Bs + kGateDim * kScoreTile;     // [64]
  float* row_l = row_m + kScoreTile;             // [64]

  const int tile_g = m.total_tiles - 1 - (int)(blockIdx.x / m.num_q_heads);
  const int h = blockIdx.x % m.num_q_heads;
  const int g = h / m.group;
  const int b = find_sequence(m.tile_off, m.batch, tile_g);
  const int nb = m.blk_off[b + 1] - m.blk_off[b];
  const int i0 = (tile_g - m.tile_off[b]) * kScoreTile;
  const int rows_valid = min(kScoreTile, nb - i0);
  const float* gq_h = gq + ((size_t)h * m.total_blocks + m.blk_off[b]) * kGateDim;
  const float* gk_g = gk + ((size_t)g * m.total_blocks + m.blk_off[b]) * kGateDim;
  float* sc = scores + m.score_off[b] + (size_t)h * nb * nb;

  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const float scale = rsqrtf((float)kGateDim);
  const bool vec_ok = (nb & 3) == 0 && (m.score_off[b] & 3) == 0;

  load_tile_transposed(As, gq_h, i0, rows_valid);

  float run_m[4], run_l[4];
#pragma unroll
  for (int r = 0; r < 4; ++r) { run_m[r] = -CUDART_INF_F; run_l[r] = 0.f; }

  const int last_col = i0 + rows_valid - 1;
  for (int j0 = 0; j0 <= last_col; j0 += kScoreTile) {
    __syncthreads();  // previous tile's Bs reads done (and As visible on the first pass)
    load_tile_transposed(Bs, gk_g, j0, min(kScoreTile, nb - j0));
    __syncthreads();
    float acc[4][4];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[r][c] = 0.f;
#pragma unroll 8
    for (int kk = 0; kk < kGateDim; ++kk) {
      const float4 a = *reinterpret_cast<const float4*>(As + kk * kScoreTile + ty * 4);
      const float4 bb = *reinterpret_cast<const float4*>(Bs + kk * kScoreTile + tx * 4);
      const float av[4] = {a.x, a.y, a.z, a.w};
      const float bv[4] = {bb.x, bb.y, bb.z, bb.w};
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(av[r], bv[c], acc[r][c]);
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int i = i0 + ty * 4 + r;
      if (i >= nb) continue;
      const int jb = j0 + tx * 4;
      float x[4];
      float tmax = -CUDART_INF_F;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        x[c] = (jb + c <= i) ? acc[r][c] * scale : -CUDART_INF_F;
        tmax = fmaxf(tmax, x[c]);
      }
      if (jb <= i) {
        const float nm = fmaxf(run_m[r], tmax);
        float s = 0.f;
#pragma unroll
        for (int c = 0; c < 4; ++c) s += (jb + c <= i) ? expf(x[c] - nm) : 0.f;
        run_l[r] = run_l[r] * expf(run_m[r] - nm) + s;   // exp(-inf) = 0 on the first contribution
        run_m[r] = nm;
        float* dst = sc + (size_t)i * nb + jb;
        if (vec_ok && jb + 3 <= i) {
          *reinterpret_cast<float4*>(dst) = make_float4(x[0], x[1], x[2], x[3]);
        } else {
#pragma unroll
          for (int c = 0; c < 4; ++c)
            if (jb + c <= i) dst[c] = x[c];
        }
      }
    }
  }
  // combine the 16 partial (max, sum) pairs of each row
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    float mm = run_m[r], ll = run_l[r];
#pragma unroll
    for (int off = 1; off < 16; off <<= 1) {
      const float om = __shfl_xor_sync(0xffffffffu, mm, off);
      const float ol = __shfl_xor_sync(0xffffffffu, ll, off);
      const float nm = fmaxf(mm, om);
      const float fa = (mm == -CUDART_INF_F) ? 0.f : expf(mm - nm);
      const float fb = (om == -CUDART_INF_F) ? 0.f : expf(om - nm);
      ll = ll * fa + ol * fb;
      mm = nm;
    }
    if (tx == 0) { row_m[ty * 4 + r] = mm; row_l[ty * 4 + r] = ll; }
  }
  __syncthreads();
  // normalise in place: the logits this CTA just wrote are re-read (L2) and replaced by exp(x - m) / l
  for (int r = 0; r < rows_valid; ++r) {
    const int i = i0 + r;
    const float mm = row_m[r];
    const float inv = 1.0f / row_l[r];
    float* dst = sc + (size_t)i * nb;
    for (int j = threadIdx.x; j <= i; j += kScoreThreads) dst[j] = expf(dst[j] - mm) * inv;
  }
}

int launch_gate(seer_ctx* ctx, const SeqMeta& m, const void* q, const void* k, const float* Wq, const float* Wk,
                float* scores, void* ws, cudaStream_t stream) {
  (void)ctx;
  size_t gq_bytes = ((size_t)m.num_q_heads * m.total_blocks * kGateDim * sizeof(float) + 255) / 256 * 256;
  float* gq = (float*)ws;
  float* gk = (float*)((char*)ws + gq_bytes);
  const unsigned grid1 = (unsigned)m.total_chunks * (unsigned)(m.num_q_heads + m.num_kv_heads);
  pool_project_kernel<<<grid1, kPoolThreads, 0, stream>>>(m, (const uint16_t*)q, (const uint16_t*)k, Wq, Wk, gq, gk);
  const unsigned grid2 = (unsigned)m.total_tiles * (unsigned)m.num_q_heads;
  gate_scores_kernel<<<grid2, kScoreThreads, kScoreSmem, stream>>>(m, gq, gk, scores);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 2 : -(int)e;
}

int launch_gate_ex(seer_ctx* ctx, const SeqMeta& m, const seer_gate_options& opt, const void* q, const void* k,
                   const float* Wq, const float* Wk, float* scores, void* ws, cudaStream_t stream) {
  (void)ctx;
  size_t gq_bytes = ((size_t)m.num_q_heads * m.total_blocks * kGateDim * sizeof(float) + 255) / 256 * 256;
  float* gq = (float*)ws;
  float* gk = (float*)((char*)ws + gq_bytes);
  const unsigned grid1 = (unsigned)m.total_chunks * (unsigned)(m.num_q_heads + m.num_kv_heads);
  pool_project_ex_kernel<<<grid1, kPoolThreads, 0, stream>>>(m, (const uint16_t*)q, (const uint16_t*)k, Wq, Wk, gq, gk,
                                                              opt.pool_q, opt.pool_k, opt.rope_theta);
  const unsigned grid2 = (unsigned)m.total_tiles * (unsigned)m.num_q_heads;
  gate_scores_kernel<<<grid2, kScoreThreads, kScoreSmem, stream>>>(m, gq, gk, scores);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 2 : -(int)e;
}

// ----------------------------------------------------------------------------------------------- allocation-free variant
// Scratch for seer_gate_scores_static lives in the library image: every GPU that loads the library carries these
// bytes until the process exits.  Host code must never hand the symbol itself to a kernel; its device address is
// looked up once per device with cudaGetSymbolAddress.
constexpr int kStaticMaxBatch = SEER_STATIC_MAX_BATCH;
constexpr size_t kStaticMetaBytes = 16 * 1024;                              // cu_seqlens + four offset arrays
constexpr size_t kStaticScratchBytes = (size_t)SEER_STATIC_SCRATCH_BYTES;   // projected pooled Q and K (fp32)
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
  if (t.total_blocks == 0) return SEER_OK;
  if (!q || !k || !Wq || !Wk || !scores) return SEER_ERR_INVALID_ARG;
  // sizes beyond the built-in scratch are refused, never truncated
  if (shape->batch > kStaticMaxBatch || gate_workspace_bytes(t, shape) > kStaticScratchBytes) return SEER_ERR_WORKSPACE;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kStaticMaxDevices) return SEER_ERR_CUDA;
  unsigned char* base = nullptr;
  st = static_setup(dev, &base);
  if (st != SEER_OK) return st;

  // per-batch offsets, built on the host stack and copied into the head of the array
  struct HostMeta {
    int32_t cu[kStaticMaxBatch + 4], blk[kStaticMaxBatch + 4], chunk[kStaticMaxBatch + 4], tile[kStaticMaxBatch + 4];
    int64_t score[kStaticMaxBatch + 2];
  } hm;
  static_assert(sizeof(HostMeta) <= kStaticMetaBytes, "metadata region too small");
  hm.blk[0] = hm.chunk[0] = hm.tile[0] = 0;
  hm.score[0] = 0;
  for (int b = 0; b < shape->batch; ++b) {
    hm.cu[b] = shape->cu_seqlens_host[b];
    const int32_t nb = (shape->cu_seqlens_host[b + 1] - shape->cu_seqlens_host[b] + kBlock - 1) / kBlock;
    hm.blk[b + 1] = hm.blk[b] + nb;
    hm.chunk[b + 1] = hm.chunk[b] + (nb + kPoolChunk - 1) / kPoolChunk;
    hm.tile[b + 1] = hm.tile[b] + (nb + kScoreTile - 1) / kScoreTile;
    hm.score[b + 1] = hm.score[b] + (int64_t)shape->num_q_heads * nb * nb;
  }
  hm.cu[shape->batch] = shape->cu_seqlens_host[shape->batch];
  // pageable source: the runtime stages the bytes before returning, so the stack buffer may go out of scope
  if (cudaMemcpyAsync(base, &hm, sizeof(HostMeta), cudaMemcpyHostToDevice, stream) != cudaSuccess) return SEER_ERR_CUDA;

  SeqMeta m;
  m.cu_seqlens = (const int32_t*)(base + offsetof(HostMeta, cu));
  m.blk_off = (const int32_t*)(base + offsetof(HostMeta, blk));
  m.chunk_off = (const int32_t*)(base + offsetof(HostMeta, chunk));
  m.tile_off = (const int32_t*)(base + offsetof(HostMeta, tile));
  m.score_off = (const int64_t*)(base + offsetof(HostMeta, score));
  m.batch = shape->batch;
  m.num_q_heads = shape->num_q_heads;
  m.num_kv_heads = shape->num_kv_heads;
  m.group = shape->num_q_heads / shape->num_kv_heads;
  m.total_tokens = (int32_t)t.total_tokens;
  m.total_blocks = (int32_t)t.total_blocks;
  m.total_chunks = (int32_t)t.total_chunks;
  m.total_tiles = (int32_t)t.total_tiles;
  m.max_nb = t.max_nb;
  m.rows = t.rows;
  m.score_elems = t.score_elems;
  m.softmax_scale = 0.f;   // unused by the gate
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
