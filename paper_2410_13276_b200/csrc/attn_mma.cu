// Block-sparse causal GQA attention (Sec. 3.3) on the legacy warp-level tensor path (mma.sync m16n8k16, bf16).
// Kept as an on-device cross-check for the tcgen05 kernel and as the baseline it is measured against.
// One CTA (4 warps) per (sequence, head, query block); warp w owns query rows 16w..16w+15; K/V blocks of the
// row's list stream through a two-stage cp.async ring; online softmax in registers.
#include <math_constants.h>

#include "seer_internal.cuh"

namespace seer {

constexpr int kMmaThreads = 128;
constexpr int kTileBytes = kBlock * kHeadDim * 2;             // 16 KB
constexpr int kMmaSmem = kTileBytes * 5;                      // Q + 2 x (K, V)

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// byte offset of (row, 16-byte chunk) in a [64][128] bf16 tile with an XOR swizzle of the chunk index
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) { return (uint32_t)(row * 256 + ((chunk ^ (row & 7)) << 4)); }

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// Copies rows [row0, row0+64) x 128 of head `head` (of `heads`) into a swizzled tile; rows >= row_end are zero-filled.
__device__ __forceinline__ void load_tile_async(uint32_t dst, const uint16_t* __restrict__ x, int64_t tok0, int rows_valid,
                                                int heads, int head) {
  for (int idx = threadIdx.x; idx < kBlock * 16; idx += kMmaThreads) {
    const int row = idx >> 4, chunk = idx & 15;
    const bool ok = row < rows_valid;
    const uint16_t* src = x + ((tok0 + (ok ? row : 0)) * heads + head) * kHeadDim + chunk * 8;
    cp_async_16(dst + tile_off(row, chunk), src, ok);
  }
}

__global__ void __launch_bounds__(kMmaThreads)
attn_mma_kernel(SeqMeta m, const uint16_t* __restrict__ q, const uint16_t* __restrict__ k, const uint16_t* __restrict__ v,
                const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx, uint16_t* __restrict__ o,
                float* __restrict__ lse, int* __restrict__ status) {
  extern __shared__ __align__(128) unsigned char smem[];
  const uint32_t sQ = smem_u32(smem);
  const uint32_t sK0 = sQ + kTileBytes, sV0 = sK0 + kTileBytes, sK1 = sV0 + kTileBytes, sV1 = sK1 + kTileBytes;

  // work item: sequences in order, then KV head, then query blocks from the last (longest) to the first, then
  // the heads of the group -- neighbouring CTAs share one KV head's K/V in L2
  const int64_t w = blockIdx.x;
  const int b = find_sequence(m.blk_off, m.batch, (int)(w / m.num_q_heads));
  const int nb = m.blk_off[b + 1] - m.blk_off[b];
  const int local = (int)(w - (int64_t)m.num_q_heads * m.blk_off[b]);
  const int g = local / (nb * m.group);
  const int rem = local - g * nb * m.group;
  const int i = nb - 1 - rem / m.group;
  const int h = g * m.group + rem % m.group;
  const int64_t r = (int64_t)m.num_q_heads * m.blk_off[b] + (int64_t)h * nb + i;

  const int s0 = m.cu_seqlens[b];
  const int slen = m.cu_seqlens[b + 1] - s0;
  const int q_valid = min(kBlock, slen - i * kBlock);
  // chunked prefill: q / o / lse hold the last positions only (token index shifted by qdelta); blocks before the chunk do nothing
  if (m.chunked && i < m.qoff[b]) return;
  const int64_t tok0 = (int64_t)s0 + (int64_t)i * kBlock + (m.chunked ? m.qdelta[b] : 0);
  const int64_t lse_stride = m.chunked ? m.total_q_tokens : m.total_tokens;
  const int l0 = row_ptr[r], l1 = row_ptr[r + 1];
  const int nlist = l1 - l0;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gid = lane >> 2, tig = lane & 3;

  load_tile_async(sQ, q, tok0, q_valid, m.num_q_heads, h);
  cp_async_commit();

  auto fetch = [&](int it, uint32_t dK, uint32_t dV) -> int {
    int j = col_idx[l0 + it];
    if (j < 0 || j > i) {            // corrupt list entry: record it, never dereference it
      if (threadIdx.x == 0) atomicCAS(status, 0, (int)SEER_ERR_INVALID_INDEX);
      j = -1;
    } else {
      const int rows_valid = min(kBlock, slen - j * kBlock);
      load_tile_async(dK, k, (int64_t)s0 + (int64_t)j * kBlock, rows_valid, m.num_kv_heads, g);
      load_tile_async(dV, v, (int64_t)s0 + (int64_t)j * kBlock, rows_valid, m.num_kv_heads, g);
    }
    cp_async_commit();
    return j;
  };

  int j_cur = -1;
  if (nlist > 0) j_cur = fetch(0, sK0, sV0);

  float oacc[16][4];
#pragma unroll
  for (int n = 0; n < 16; ++n)
#pragma unroll
    for (int c = 0; c < 4; ++c) oacc[n][c] = 0.f;
  float row_m[2] = {-CUDART_INF_F, -CUDART_INF_F}, row_l[2] = {0.f, 0.f};
  const float sl2 = m.softmax_scale * 1.4426950408889634f;

  // Q fragments (registers for the whole item)
  uint32_t qf[8][4];
  if (nlist > 0) cp_async_wait<1>(); else cp_async_wait<0>();
  __syncthreads();
#pragma unroll
  for (int kk = 0; kk < 8; ++kk) {
    const int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
    ldsm_x4(qf[kk], sQ + tile_off(row, kk * 2 + (lane >> 4)));
  }

  for (int it = 0; it < nlist; ++it) {
    const uint32_t cK = (it & 1) ? sK1 : sK0, cV = (it & 1) ? sV1 : sV0;
    int j_next = -1;
    if (it + 1 < nlist) {
      j_next = fetch(it + 1, (it & 1) ? sK0 : sK1, (it & 1) ? sV0 : sV1);
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    if (j_cur >= 0) {
      float sacc[8][4];
#pragma unroll
      for (int n = 0; n < 8; ++n)
#pragma unroll
        for (int c = 0; c < 4; ++c) sacc[n][c] = 0.f;
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
        for (int kk = 0; kk < 8; kk += 2) {
          uint32_t bf[4];
          ldsm_x4(bf, cK + tile_off(nt * 8 + (lane & 7), kk * 2 + (lane >> 3)));
          mma_bf16(sacc[nt], qf[kk], bf[0], bf[1]);
          mma_bf16(sacc[nt], qf[kk + 1], bf[2], bf[3]);
        }
      }
      // scale, mask, online softmax.  Thread holds rows (gid, gid+8) x cols nt*8 + 2*tig + {0,1}
      const bool diag = j_cur == i;
      float tmax[2] = {-CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
      for (int nt = 0; nt < 8; ++nt)
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int rr = warp * 16 + gid + (c >> 1) * 8;
          const int cc = nt * 8 + 2 * tig + (c & 1);
          float x = sacc[nt][c] * sl2;
          if (diag && cc > rr) x = -CUDART_INF_F;
          sacc[nt][c] = x;
          tmax[c >> 1] = fmaxf(tmax[c >> 1], x);
        }
      float alpha[2], mref[2];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        tmax[e] = fmaxf(tmax[e], __shfl_xor_sync(0xffffffffu, tmax[e], 1));
        tmax[e] = fmaxf(tmax[e], __shfl_xor_sync(0xffffffffu, tmax[e], 2));
        const float nm = fmaxf(row_m[e], tmax[e]);
        mref[e] = nm == -CUDART_INF_F ? 0.f : nm;
        alpha[e] = exp2f(row_m[e] - mref[e]);
        row_m[e] = nm;
        row_l[e] *= alpha[e];
      }
      uint32_t pf[4][4];
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        const float p0 = exp2f(sacc[nt][0] - mref[0]), p1 = exp2f(sacc[nt][1] - mref[0]);
        const float p2 = exp2f(sacc[nt][2] - mref[1]), p3 = exp2f(sacc[nt][3] - mref[1]);
        const uint32_t lo = pack_bf16(p0, p1), hi = pack_bf16(p2, p3);
        // the denominator sums the bf16-rounded probabilities the P V product uses
        row_l[0] += __uint_as_float(lo << 16) + __uint_as_float(lo & 0xffff0000u);
        row_l[1] += __uint_as_float(hi << 16) + __uint_as_float(hi & 0xffff0000u);
        pf[nt >> 1][(nt & 1) * 2 + 0] = lo;
        pf[nt >> 1][(nt & 1) * 2 + 1] = hi;
      }
#pragma unroll
      for (int n = 0; n < 16; ++n) {
        oacc[n][0] *= alpha[0]; oacc[n][1] *= alpha[0];
        oacc[n][2] *= alpha[1]; oacc[n][3] *= alpha[1];
      }
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
        for (int nt = 0; nt < 16; nt += 2) {
          uint32_t bf[4];
          ldsm_x4_trans(bf, cV + tile_off(ks * 16 + ((lane >> 3) & 1) * 8 + (lane & 7), nt + (lane >> 4)));
          mma_bf16(oacc[nt], pf[ks], bf[0], bf[1]);
          mma_bf16(oacc[nt + 1], pf[ks], bf[2], bf[3]);
        }
      }
    }
    __syncthreads();   // everyone is done with this stage before the next prefetch overwrites it
    j_cur = j_next;
  }

  // epilogue: normalise, stage bf16 rows in the Q tile (each warp touches only its own 16 rows), coalesced stores
  float inv[2], lse_v[2];
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    float l = row_l[e];
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    inv[e] = l > 0.f ? 1.0f / l : 0.f;
    lse_v[e] = l > 0.f ? (row_m[e] + log2f(l)) * 0.6931471805599453f : -CUDART_INF_F;
  }
  __syncwarp();
#pragma unroll
  for (int n = 0; n < 16; ++n) {
    const int r0 = warp * 16 + gid;
    const uint32_t lo = pack_bf16(oacc[n][0] * inv[0], oacc[n][1] * inv[0]);
    const uint32_t hi = pack_bf16(oacc[n][2] * inv[1], oacc[n][3] * inv[1]);
    asm volatile("st.shared.b32 [%0], %1;" ::"r"(sQ + tile_off(r0, n) + tig * 4), "r"(lo) : "memory");
    asm volatile("st.shared.b32 [%0], %1;" ::"r"(sQ + tile_off(r0 + 8, n) + tig * 4), "r"(hi) : "memory");
  }
  __syncwarp();
#pragma unroll
  for (int rr = 0; rr < 16; rr += 2) {
    const int row = warp * 16 + rr + (lane >> 4);
    const int chunk = lane & 15;
    if (row < q_valid) {
      uint4 val;
      asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w)
                   : "r"(sQ + tile_off(row, chunk)));
      *reinterpret_cast<uint4*>(o + ((tok0 + row) * m.num_q_heads + h) * kHeadDim + chunk * 8) = val;
    }
  }
  if (lse != nullptr && tig == 0) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int row = warp * 16 + gid + e * 8;
      if (row < q_valid) lse[(int64_t)h * lse_stride + tok0 + row] = lse_v[e];
    }
  }
}


// ------------------------------------------------------------------------------------------------ max-pooled map
// Sec. 3.2, Eq. 2 (the distillation target of the gate; at inference a recall diagnostic): the 2D max-pool, window and
// stride B, of the attention map -- here the map the block lists define, a_ts = exp(r_ts - m_t) / l_t (appendix), given
// through the log-sum-exp the attention kernel wrote.  One value per list entry: the largest probability in that 64 x 64
// tile.  Same CTA layout as the kernel above, K tiles only; the tile maximum is reduced over the CTA through shared memory.
constexpr int kBmSmem = kTileBytes * 3 + 64;                   // Q + 2 x K + four per-warp maxima

__global__ void __launch_bounds__(kMmaThreads)
block_max_kernel(SeqMeta m, const uint16_t* __restrict__ q, const uint16_t* __restrict__ k,
                 const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx, const float* __restrict__ lse,
                 float* __restrict__ out, int* __restrict__ status) {
  extern __shared__ __align__(128) unsigned char smem[];
  const uint32_t sQ = smem_u32(smem);
  const uint32_t sK0 = sQ + kTileBytes, sK1 = sK0 + kTileBytes;
  float* wmax = reinterpret_cast<float*>(smem + 3 * kTileBytes);

  const int64_t w = blockIdx.x;
  const int b = find_sequence(m.blk_off, m.batch, (int)(w / m.num_q_heads));
  const int nb = m.blk_off[b + 1] - m.blk_off[b];
  const int local = (int)(w - (int64_t)m.num_q_heads * m.blk_off[b]);
  const int g = local / (nb * m.group);
  const int rem = local - g * nb * m.group;
  const int i = nb - 1 - rem / m.group;
  const int h = g * m.group + rem % m.group;
  const int64_t r = (int64_t)m.num_q_heads * m.blk_off[b] + (int64_t)h * nb + i;

  const int s0 = m.cu_seqlens[b];
  const int slen = m.cu_seqlens[b + 1] - s0;
  const int q_valid = min(kBlock, slen - i * kBlock);
  const int l0 = row_ptr[r], l1 = row_ptr[r + 1];
  const int nlist = l1 - l0;
  if (nlist <= 0) return;
  if (m.chunked && i < m.qoff[b]) return;                // chunked prefill: a block before the chunk

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gid = lane >> 2, tig = lane & 3;
  const int64_t tok0 = (int64_t)s0 + (int64_t)i * kBlock + (m.chunked ? m.qdelta[b] : 0);   // in q / lse
  const int64_t lse_stride = m.chunked ? m.total_q_tokens : m.total_tokens;

  load_tile_async(sQ, q, tok0, q_valid, m.num_q_heads, h);
  cp_async_commit();

  auto fetch = [&](int it, uint32_t dK) -> int {
    int j = col_idx[l0 + it];
    if (j < 0 || j > i) {            // corrupt list entry: record it, never dereference it
      if (threadIdx.x == 0) atomicCAS(status, 0, (int)SEER_ERR_INVALID_INDEX);
      j = -1;
    } else {
      load_tile_async(dK, k, (int64_t)s0 + (int64_t)j * kBlock, min(kBlock, slen - j * kBlock), m.num_kv_heads, g);
    }
    cp_async_commit();
    return j;
  };
  int j_cur = fetch(0, sK0);

  const float sl2 = m.softmax_scale * 1.4426950408889634f;
  // log2 of the softmax denominator of this thread's two query rows (gid, gid + 8 of the warp's 16)
  float lse2[2];
  bool row_ok[2];
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const int row = warp * 16 + gid + e * 8;
    row_ok[e] = row < q_valid;
    lse2[e] = row_ok[e] ? lse[(int64_t)h * lse_stride + tok0 + row] * 1.4426950408889634f : 0.f;
  }

  uint32_t qf[8][4];
  cp_async_wait<1>();
  __syncthreads();
#pragma unroll
  for (int kk = 0; kk < 8; ++kk) {
    const int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
    ldsm_x4(qf[kk], sQ + tile_off(row, kk * 2 + (lane >> 4)));
  }

  for (int it = 0; it < nlist; ++it) {
    const uint32_t cK = (it & 1) ? sK1 : sK0;
    int j_next = -1;
    if (it + 1 < nlist) {
      j_next = fetch(it + 1, (it & 1) ? sK0 : sK1);
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    float tmax = 0.f;                 // probabilities are positive; a tile with no causal pair gives 0
    if (j_cur >= 0) {
      float sacc[8][4];
#pragma unroll
      for (int n = 0; n < 8; ++n)
#pragma unroll
        for (int c = 0; c < 4; ++c) sacc[n][c] = 0.f;
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
        for (int kk = 0; kk < 8; kk += 2) {
          uint32_t bf[4];
          ldsm_x4(bf, cK + tile_off(nt * 8 + (lane & 7), kk * 2 + (lane >> 3)));
          mma_bf16(sacc[nt], qf[kk], bf[0], bf[1]);
          mma_bf16(sacc[nt], qf[kk + 1], bf[2], bf[3]);
        }
      }
      // the largest logit of each of the two rows, then one exponential per row (exp is monotone)
      const bool diag = j_cur == i;
      float xm[2] = {-CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
      for (int nt = 0; nt < 8; ++nt)
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int rr = warp * 16 + gid + (c >> 1) * 8;
          const int cc = nt * 8 + 2 * tig + (c & 1);
          if (!(diag && cc > rr)) xm[c >> 1] = fmaxf(xm[c >> 1], sacc[nt][c]);   // keys past the sequence end lie above the diagonal too
        }
#pragma unroll
      for (int e = 0; e < 2; ++e)
        if (row_ok[e] && xm[e] != -CUDART_INF_F) tmax = fmaxf(tmax, exp2f(xm[e] * sl2 - lse2[e]));
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, off));
    if (lane == 0) wmax[warp] = tmax;
    __syncthreads();   // also: everyone is done with this K stage before the next prefetch overwrites it
    if (threadIdx.x == 0) out[l0 + it] = fmaxf(fmaxf(wmax[0], wmax[1]), fmaxf(wmax[2], wmax[3]));
    __syncthreads();
    j_cur = j_next;
  }
}

seer_status init_attn_mma(seer_ctx* ctx) {
  (void)ctx;
  cudaError_t e = cudaFuncSetAttribute(attn_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMmaSmem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(block_max_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kBmSmem);
  return e == cudaSuccess ? SEER_OK : SEER_ERR_CUDA;
}

int launch_block_max(seer_ctx* ctx, const SeqMeta& m, const void* q, const void* k, const int32_t* row_ptr,
                     const int32_t* col_idx, const float* lse, float* out, cudaStream_t stream) {
  if (m.rows == 0) return 0;
  block_max_kernel<<<(unsigned)m.rows, kMmaThreads, kBmSmem, stream>>>(m, (const uint16_t*)q, (const uint16_t*)k, row_ptr,
                                                                       col_idx, lse, out, ctx->d_status);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 1 : -(int)e;
}

int launch_attn_mma(seer_ctx* ctx, const SeqMeta& m, const void* q, const void* k, const void* v,
                    const int32_t* row_ptr, const int32_t* col_idx, void* o, float* lse, cudaStream_t stream) {
  if (m.rows == 0) return 0;
  attn_mma_kernel<<<(unsigned)m.rows, kMmaThreads, kMmaSmem, stream>>>(
      m, (const uint16_t*)q, (const uint16_t*)k, (const uint16_t*)v, row_ptr, col_idx, (uint16_t*)o, lse, ctx->d_status);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 1 : -(int)e;
}

}  // namespace seer
