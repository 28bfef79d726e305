// AttnGate (Sec. 3.1, Eq. 1) in two kernels:
//   pool_project_kernel : streams Q and K once (HBM-bound), average-pools each 64-token block per head and
//                         multiplies the pooled vectors by the head's gate matrix (fp32 on the CUDA cores) -> gq, gk
//   gate_scores_kernel  : logits = gq gk^T / sqrt(dg) over the causal blocks, row softmax -> scores (gate_scores.cu)
// The logits need fp32-grade products (plain bf16 or tf32 tensor-core inputs would not hold the 1e-3 relative bound on
// softmax outputs when logits reach tens), so gq and gk are stored as three bf16 planes each, x = hi + mid + lo with
// every part the bf16 rounding of what is left, and the second kernel takes the product on the tensor cores as six
// bf16 terms.
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
// gate_scores_kernel (tcgen05) lives in gate_scores.cu.
int launch_gate_scores(const SeqMeta& m, const ScoreBand& band, const uint16_t* gq, const uint16_t* gk, float* scores,
                       int* status, cudaStream_t stream);
bool init_gate_scores();

int launch_gate(seer_ctx* ctx, const SeqMeta& m, const void* q, const void* k, const float* Wq, const float* Wk,
                float* scores, void* ws, cudaStream_t stream) {
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
  const int n2 = launch_gate_scores(m, all, gq, gk, scores, ctx ? ctx->d_status : nullptr, stream);
  return n2 < 0 ? n2 : 1 + n2;
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
  const int n2 = launch_gate_scores(m, all, gq, gk, scores, ctx ? ctx->d_status : nullptr, stream);
  return n2 < 0 ? n2 : 1 + n2;
}

// Scores of one band from the projected vectors launch_gate_ex(scores = nullptr) left in `ws`.
int launch_gate_scores_band(const SeqMeta& m, const ScoreBand& band, const void* ws, float* scores, cudaStream_t stream) {
  size_t gq_bytes = ((size_t)m.num_q_heads * m.total_blocks * kGateDim * 6 + 255) / 256 * 256;
  const uint16_t* gq = (const uint16_t*)ws;
  const uint16_t* gk = (const uint16_t*)((const char*)ws + gq_bytes);
  return launch_gate_scores(m, band, gq, gk, scores, nullptr, stream);
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
    if (!init_gate_scores()) return SEER_ERR_CUDA;
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
  return init_gate_scores() ? SEER_OK : SEER_ERR_CUDA;
}

}  // namespace seer

extern "C" seer_status seer_gate_scores_static(const seer_shape* shape, const void* q, const void* k, const float* Wq,
                                               const float* Wk, float* scores, void* stream) {
  if (!shape) return SEER_ERR_INVALID_ARG;
  return seer::gate_scores_static(shape, q, k, Wq, Wk, scores, (cudaStream_t)stream);
}
