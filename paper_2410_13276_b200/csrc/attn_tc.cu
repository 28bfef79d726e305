// Block-sparse causal GQA attention (Sec. 3.3) on the Blackwell tensor path: tcgen05.mma with TMEM accumulators,
// TMA gathers of the listed K/V blocks, warp-specialised roles.
//
// Orientation.  A query block is 64 rows but the full-rate MMA shape is M = 128, and every (head, query block) has its
// own list, so rows of different work items cannot share an MMA.  The kernel therefore computes the transposed
// problem: two listed KV blocks (128 keys) form the M dimension and the 64 queries the N dimension,
//     S^T[128 keys x 64 q] = K_tile[128 x 128 d] * Q^T          (A, B K-major in shared memory)
//     O^T[128 d x 64 q]   += V_tile^T[128 d x 128 keys] * P^T    (A, B MN-major in shared memory)
// so every MMA row is useful for arbitrary lists (an odd list pads half a tile once).
//
// Softmax in this orientation: a thread owns one key row of S^T (64 query columns).  The per-query running reference
// m[c] lives in shared memory and is only a scaling reference, not the exact maximum: p = 2^(s - m[c]).  As long as no
// entry of a tile exceeds its reference by more than 2^8 the tile needs no cross-thread reduction at all; otherwise the
// work group computes exact column maxima, rebases m, rescales its partial sums and the O accumulator, and recomputes
// the tile.  Row sums are per-thread partials combined once per work item.
//
// Roles (192 threads): warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer, warps 2-5 = softmax / correction /
// epilogue.  One persistent CTA per SM walks the work items (longest rows first within each KV head).
// Every wait is bounded; a wait that runs out raises SEER_ERR_TIMEOUT and the CTA drains and exits.
#include <cuda.h>
#include <math_constants.h>

#include <map>

#include "seer_internal.cuh"

namespace seer {
namespace tc {

constexpr int kThreads = 192;
constexpr int kSoftmaxThreads = 128;
constexpr int kStages = 2;
constexpr uint32_t kHalfQ = 64 * 128;            // bytes of one d-half of a 64-row tile (8 KB)
constexpr uint32_t kHalfKV = 128 * 128;          // bytes of one d-half of a 128-row tile (16 KB)
constexpr uint32_t kQBytes = 2 * kHalfQ;         // 16 KB
constexpr uint32_t kKVBytes = 2 * kHalfKV;       // 32 KB (K or V of one stage)
constexpr uint32_t kPBytes = 128 * 128;          // 16 KB  P^T [128 keys][64 q] bf16
// shared memory map (offsets from a 1024-byte aligned base)
constexpr uint32_t kOffQ = 0;
constexpr uint32_t kOffK = kOffQ + kQBytes;                       // kStages x 32 KB
constexpr uint32_t kOffV = kOffK + kStages * kKVBytes;            // kStages x 32 KB
constexpr uint32_t kOffP = kOffV + kStages * kKVBytes;            // 16 KB (also epilogue staging)
constexpr uint32_t kOffRed = kOffP + kPBytes;                     // 128 x 65 floats for the row-sum reduction
constexpr uint32_t kRedBytes = 128 * 65 * 4;
constexpr uint32_t kOffMref = kOffRed + kRedBytes;                // 64 floats
constexpr uint32_t kOffAlpha = kOffMref + 256;                    // 64 floats
constexpr uint32_t kOffColmax = kOffAlpha + 256;                  // 64 ints
constexpr uint32_t kOffInvL = kOffColmax + 256;                   // 64 floats
constexpr uint32_t kOffBar = kOffInvL + 256;                      // mbarriers
constexpr uint32_t kNumBars = 16;
constexpr uint32_t kOffMisc = kOffBar + kNumBars * 8;             // tmem base, abort flag
constexpr uint32_t kSmemBytes = kOffMisc + 64 + 1024;             // + alignment slack

enum Bar { Q_FULL = 0, Q_EMPTY, KV_FULL0, KV_FULL1, KV_EMPTY0, KV_EMPTY1, S_FULL0, S_FULL1, S_EMPTY0, S_EMPTY1,
           P_FULL, PV_DONE };

constexpr uint32_t kTmemCols = 256;
constexpr uint32_t kColS0 = 0, kColS1 = 64, kColO = 128;

constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // a wait that lasts 2 s is declared lost

// ------------------------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}

struct Shared {
  uint32_t base;         // 1024-aligned shared address
  __device__ __forceinline__ uint32_t bar(int i) const { return base + kOffBar + 8u * (uint32_t)i; }
  __device__ __forceinline__ uint32_t abort_flag() const { return base + kOffMisc + 8; }
};

__device__ __forceinline__ uint32_t ld_shared_u32(uint32_t a) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
  return v;
}
__device__ __forceinline__ void st_shared_u32(uint32_t a, uint32_t v) {
  asm volatile("st.shared.u32 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}

__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait.  Returns false after the limit (or when another role has already given up); the caller drains.
__device__ __forceinline__ bool mbar_wait(const Shared& sh, int bar, uint32_t parity, int* status) {
  const uint32_t addr = sh.bar(bar);
  if (mbar_try(addr, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try(addr, parity)) return true;
    if ((it & 255u) == 0u) {
      if (ld_shared_u32(sh.abort_flag()) != 0u) return false;
      if (global_ns() - t0 > kWaitLimitNs) break;
    }
  }
  st_shared_u32(sh.abort_flag(), 1u);
  atomicCAS(status, 0, (int)SEER_ERR_TIMEOUT);
  return false;
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
               ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
               ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                 "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
               : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                 "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
// CTA-subset OR reduction of a predicate over `threads` threads on barrier `id`
__device__ __forceinline__ bool named_bar_or(int id, int threads, bool pred) {
  uint32_t r;
  asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 p, %3, 0;\n\tbar.red.or.pred q, %1, %2, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
               : "=r"(r) : "r"(id), "r"(threads), "r"((uint32_t)pred) : "memory");
  return r != 0;
}

// Shared-memory matrix descriptors (128-byte swizzle, descriptor version 1)
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((saddr & 0x3ffffu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// kind::f16 instruction descriptor: fp32 accumulate, bf16 x bf16, M = 128, N = 64
constexpr uint32_t make_idesc(bool a_mn_major, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
         ((64u >> 3) << 17) | ((128u >> 4) << 24);
}
constexpr uint32_t kIdescS = make_idesc(false, false);
constexpr uint32_t kIdescPV = make_idesc(true, true);

__device__ __forceinline__ int float_order_int(float x) {   // monotone float -> int map
  int i = __float_as_int(x);
  return i ^ ((i >> 31) & 0x7fffffff);
}
__device__ __forceinline__ float order_int_float(int i) { return __int_as_float(i ^ ((i >> 31) & 0x7fffffff)); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Wait used by the 128 softmax threads: all of them wait, then agree on the outcome, so that after a lost wait
// nobody is left behind at a named barrier.
__device__ __forceinline__ bool wg_wait(const Shared& sh, int bar, uint32_t parity, int* status) {
  const bool fail = !mbar_wait(sh, bar, parity, status);
  return !named_bar_or(3, kSoftmaxThreads, fail);
}

struct Item {
  int b, h, g, i, nb, s0, slen, l0, nlist, ntiles, q_valid;
  int64_t row;
};

__device__ __forceinline__ Item decode_item(const SeqMeta& m, const int32_t* __restrict__ row_ptr, int64_t w) {
  Item it;
  it.b = find_sequence(m.blk_off, m.batch, (int)(w / m.num_q_heads));
  it.nb = m.blk_off[it.b + 1] - m.blk_off[it.b];
  const int local = (int)(w - (int64_t)m.num_q_heads * m.blk_off[it.b]);
  it.g = local / (it.nb * m.group);
  const int rem = local - it.g * it.nb * m.group;
  it.i = it.nb - 1 - rem / m.group;
  it.h = it.g * m.group + rem % m.group;
  it.row = (int64_t)m.num_q_heads * m.blk_off[it.b] + (int64_t)it.h * it.nb + it.i;
  it.s0 = m.cu_seqlens[it.b];
  it.slen = m.cu_seqlens[it.b + 1] - it.s0;
  it.q_valid = min(kBlock, it.slen - it.i * kBlock);
  it.l0 = row_ptr[it.row];
  it.nlist = row_ptr[it.row + 1] - it.l0;
  it.ntiles = (it.nlist + 1) >> 1;
  return it;
}

// Block index of list position p of an item, or -1 when the position is past the list or the entry is out of range.
__device__ __forceinline__ int list_block(const Item& it, const int32_t* __restrict__ col_idx, int p) {
  if (p >= it.nlist) return -1;
  const int j = col_idx[it.l0 + p];
  return (j < 0 || j > it.i) ? -2 : j;
}

// ------------------------------------------------------------------------------------------------ kernel
__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v, SeqMeta m, const int32_t* __restrict__ row_ptr,
               const int32_t* __restrict__ col_idx, uint16_t* __restrict__ o, float* __restrict__ lse,
               int* __restrict__ status) {
  extern __shared__ unsigned char smem_raw[];
  Shared sh;
  sh.base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (sh.base - smem_u32(smem_raw));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + kOffMisc);

  if (threadIdx.x == 0) {
    mbar_init(sh.bar(Q_FULL), 1);
    mbar_init(sh.bar(Q_EMPTY), 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(sh.bar(KV_FULL0 + s), 1);
      mbar_init(sh.bar(KV_EMPTY0 + s), 1);
      mbar_init(sh.bar(S_FULL0 + s), 1);
      mbar_init(sh.bar(S_EMPTY0 + s), kSoftmaxThreads);
    }
    mbar_init(sh.bar(P_FULL), kSoftmaxThreads);
    mbar_init(sh.bar(PV_DONE), 1);
    st_shared_u32(sh.abort_flag(), 0u);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sh.base + kOffMisc), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  // ============================================================================================ producer
  if (warp == 0) {
    if (lane == 0) {
      uint32_t n_item = 0, n_tile = 0;
      for (int64_t w = blockIdx.x; w < m.rows; w += gridDim.x) {
        const Item it = decode_item(m, row_ptr, w);
        if (it.ntiles == 0) continue;   // empty list: nothing to load; only items with tiles advance n_item
        if (!mbar_wait(sh, Q_EMPTY, (n_item & 1u) ^ 1u, status)) break;
        ++n_item;
        mbar_expect_tx(sh.bar(Q_FULL), kQBytes);
        const int tq = it.s0 + it.i * kBlock;
        tma_load_3d(sh.base + kOffQ, &map_q, sh.bar(Q_FULL), 0, it.h, tq);
        tma_load_3d(sh.base + kOffQ + kHalfQ, &map_q, sh.bar(Q_FULL), 64, it.h, tq);
        bool ok = true;
        for (int t = 0; t < it.ntiles; ++t, ++n_tile) {
          const uint32_t st = n_tile & 1u;
          if (!mbar_wait(sh, KV_EMPTY0 + st, ((n_tile >> 1) & 1u) ^ 1u, status)) { ok = false; break; }
          int ja = list_block(it, col_idx, 2 * t), jb = list_block(it, col_idx, 2 * t + 1);
          if (ja == -2 || jb == -2) atomicCAS(status, 0, (int)SEER_ERR_INVALID_INDEX);
          const bool has_b = jb != -1;
          if (ja < 0) ja = 0;            // a rejected entry is replaced by block 0 and masked out in the softmax
          if (jb < 0) jb = 0;
          mbar_expect_tx(sh.bar(KV_FULL0 + st), has_b ? 2 * kKVBytes : kKVBytes);
          const uint32_t kdst = sh.base + kOffK + st * kKVBytes, vdst = sh.base + kOffV + st * kKVBytes;
          const uint32_t fb = sh.bar(KV_FULL0 + st);
          const int ta = it.s0 + ja * kBlock, tb = it.s0 + jb * kBlock;
          tma_load_3d(kdst, &map_k, fb, 0, it.g, ta);
          tma_load_3d(kdst + kHalfKV, &map_k, fb, 64, it.g, ta);
          if (has_b) {
            tma_load_3d(kdst + kHalfQ, &map_k, fb, 0, it.g, tb);
            tma_load_3d(kdst + kHalfKV + kHalfQ, &map_k, fb, 64, it.g, tb);
          }
          tma_load_3d(vdst, &map_v, fb, 0, it.g, ta);
          tma_load_3d(vdst + kHalfKV, &map_v, fb, 64, it.g, ta);
          if (has_b) {
            tma_load_3d(vdst + kHalfQ, &map_v, fb, 0, it.g, tb);
            tma_load_3d(vdst + kHalfKV + kHalfQ, &map_v, fb, 64, it.g, tb);
          }
        }
        if (!ok) break;
      }
    }
  }
  // ============================================================================================ MMA issuer
  else if (warp == 1) {
    if (lane == 0) {
      uint32_t n_item = 0, n_tile = 0;
      const uint32_t q_addr = sh.base + kOffQ;
      auto issue_s = [&](uint32_t n) -> bool {       // S^T(n) = K_tile * Q^T into S buffer n & 1
        const uint32_t st = n & 1u, use = n >> 1;
        if (!mbar_wait(sh, KV_FULL0 + st, use & 1u, status)) return false;
        if (!mbar_wait(sh, S_EMPTY0 + st, (use & 1u) ^ 1u, status)) return false;
        tc_fence_after();
        const uint32_t k_addr = sh.base + kOffK + st * kKVBytes;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint64_t a = make_desc(k_addr + (kk >> 2) * kHalfKV + (kk & 3) * 32, 16, 1024);
          const uint64_t b = make_desc(q_addr + (kk >> 2) * kHalfQ + (kk & 3) * 32, 16, 1024);
          tc_mma(tmem + (st ? kColS1 : kColS0), a, b, kIdescS, kk > 0);
        }
        tc_commit(sh.bar(S_FULL0 + st));
        return true;
      };
      bool ok = true;
      for (int64_t w = blockIdx.x; ok && w < m.rows; w += gridDim.x) {
        const Item it = decode_item(m, row_ptr, w);
        if (it.ntiles == 0) continue;
        if (!mbar_wait(sh, Q_FULL, n_item & 1u, status)) break;
        ++n_item;
        if (!issue_s(n_tile)) break;
        for (int t = 0; t < it.ntiles; ++t) {
          const uint32_t n = n_tile + t;
          if (t + 1 < it.ntiles) {
            if (!issue_s(n + 1)) { ok = false; break; }
          } else {
            tc_commit(sh.bar(Q_EMPTY));      // every S^T of this item has been issued: Q may be replaced once they finish
          }
          if (!mbar_wait(sh, P_FULL, n & 1u, status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t st = n & 1u;
          const uint32_t v_addr = sh.base + kOffV + st * kKVBytes, p_addr = sh.base + kOffP;
          const int nk = list_block(it, col_idx, 2 * t + 1) != -1 ? 8 : 4;   // 16-key groups to contract over
          for (int kk = 0; kk < nk; ++kk) {
            const uint64_t a = make_desc(v_addr + kk * 2048, kHalfKV, 1024);
            const uint64_t b = make_desc(p_addr + kk * 2048, kHalfKV, 1024);
            tc_mma(tmem + kColO, a, b, kIdescPV, (t > 0 || kk > 0) ? 1u : 0u);
          }
          tc_commit(sh.bar(KV_EMPTY0 + st));
          tc_commit(sh.bar(PV_DONE));
        }
        n_tile += it.ntiles;
      }
    }
  }
  // ============================================================================================ softmax work group
  else {
    const int wg_tid = threadIdx.x - 64;                 // 0..127
    const int quad = warp & 3;                           // TMEM lane quadrant this warp may access
    const int r = quad * 32 + lane;                      // key row of S^T / d row of O^T owned by this thread
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    float* mref = reinterpret_cast<float*>(smem + kOffMref);
    float* alpha = reinterpret_cast<float*>(smem + kOffAlpha);
    int* colmax = reinterpret_cast<int*>(smem + kOffColmax);
    float* inv_l = reinterpret_cast<float*>(smem + kOffInvL);
    float* red = reinterpret_cast<float*>(smem + kOffRed);
    const float sl2 = m.softmax_scale * 1.4426950408889634f;
    uint32_t n_tile = 0;
    bool ok = true;

    for (int64_t w = blockIdx.x; ok && w < m.rows; w += gridDim.x) {
      const Item it = decode_item(m, row_ptr, w);
      const int64_t tok0 = (int64_t)it.s0 + (int64_t)it.i * kBlock;
      float l_part[64];
#pragma unroll
      for (int c = 0; c < 64; ++c) l_part[c] = 0.f;
      if (wg_tid < 64) mref[wg_tid] = -CUDART_INF_F;
      named_bar_sync(1, kSoftmaxThreads);

      for (int t = 0; t < it.ntiles && ok; ++t, ++n_tile) {
        const uint32_t st = n_tile & 1u;
        const int ja = list_block(it, col_idx, 2 * t), jb = list_block(it, col_idx, 2 * t + 1);
        const int my_j = r < 64 ? ja : jb;
        const bool row_live = my_j >= 0;                 // absent / rejected blocks contribute nothing
        const bool diag = my_j == it.i;
        const int key_local = r & 63;
        if (!wg_wait(sh, S_FULL0 + st, (n_tile >> 1) & 1u, status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t s_addr = tmem + lane_addr + (st ? kColS1 : kColS0);

        uint32_t pk[32];
        for (int pass = 0; pass < 2; ++pass) {
          float xmax = -CUDART_INF_F;
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            uint32_t sv[16];
            tc_ld16(s_addr + ch * 16, sv);
            tc_wait_ld();
#pragma unroll
            for (int e = 0; e < 16; e += 2) {
              const int c = ch * 16 + e;
              const float2 mr = *reinterpret_cast<const float2*>(&mref[c]);
              float x0 = fmaf(__uint_as_float(sv[e]), sl2, -mr.x);
              float x1 = fmaf(__uint_as_float(sv[e + 1]), sl2, -mr.y);
              if (!row_live || (diag && key_local > c)) x0 = -CUDART_INF_F;
              if (!row_live || (diag && key_local > c + 1)) x1 = -CUDART_INF_F;
              xmax = fmaxf(xmax, fmaxf(x0, x1));
              pk[c >> 1] = pack_bf16(ex2f(fminf(x0, 64.f)), ex2f(fminf(x1, 64.f)));
            }
          }
          // does any entry of the tile exceed its reference by more than 2^8?
          const bool rebase = named_bar_or(2, kSoftmaxThreads, xmax > 8.f);
          if (!rebase) break;
          // ---- exact column maxima of this tile, then new references (pass 1 recomputes the tile with them)
          if (wg_tid < 64) colmax[wg_tid] = float_order_int(-CUDART_INF_F);
          named_bar_sync(1, kSoftmaxThreads);
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            uint32_t sv[16];
            tc_ld16(s_addr + ch * 16, sv);
            tc_wait_ld();
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              const int c = ch * 16 + e;
              float x = __uint_as_float(sv[e]) * sl2;
              if (!row_live || (diag && key_local > c)) x = -CUDART_INF_F;
              const int wm = __reduce_max_sync(0xffffffffu, float_order_int(x));
              if (lane == 0) atomicMax(&colmax[c], wm);
            }
          }
          named_bar_sync(1, kSoftmaxThreads);
          if (wg_tid < 64) {
            const float old = mref[wg_tid];
            float nm = fmaxf(old, order_int_float(colmax[wg_tid]));
            if (nm == -CUDART_INF_F) nm = 0.f;           // nothing visible in this column yet
            alpha[wg_tid] = old == -CUDART_INF_F ? 0.f : exp2f(old - nm);
            mref[wg_tid] = nm;
          }
          named_bar_sync(1, kSoftmaxThreads);
#pragma unroll
          for (int c = 0; c < 64; ++c) l_part[c] *= alpha[c];
          if (t > 0) {
            // O^T row r of this thread: scale column c by alpha[c].  The previous tile's P V must have finished.
            if (!wg_wait(sh, PV_DONE, (n_tile - 1) & 1u, status)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
              uint32_t ov[16];
              tc_ld16(tmem + lane_addr + kColO + ch * 16, ov);
              tc_wait_ld();
#pragma unroll
              for (int e = 0; e < 16; ++e) ov[e] = __float_as_uint(__uint_as_float(ov[e]) * alpha[ch * 16 + e]);
              tc_st16(tmem + lane_addr + kColO + ch * 16, ov);
            }
            tc_wait_st();
          }
        }
        if (!ok) break;
        // S^T buffer may be overwritten by the MMA of tile n + 2
        tc_fence_before();
        mbar_arrive(sh.bar(S_EMPTY0 + st));
        // row sums over the bf16-rounded probabilities the MMA will use
#pragma unroll
        for (int c2 = 0; c2 < 32; ++c2) {
          l_part[2 * c2] += __uint_as_float(pk[c2] << 16);
          l_part[2 * c2 + 1] += __uint_as_float(pk[c2] & 0xffff0000u);
        }
        // P^T row r -> shared memory (128-byte swizzle), after the previous P V has finished reading the buffer
        if (n_tile > 0 && !wg_wait(sh, PV_DONE, (n_tile - 1) & 1u, status)) { ok = false; break; }
        {
          const uint32_t prow = sh.base + kOffP + (uint32_t)r * 128u;
#pragma unroll
          for (int ck = 0; ck < 8; ++ck) {
            const uint32_t a = prow + (uint32_t)((ck ^ (r & 7)) << 4);
            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(pk[ck * 4]), "r"(pk[ck * 4 + 1]),
                         "r"(pk[ck * 4 + 2]), "r"(pk[ck * 4 + 3]) : "memory");
          }
          // ragged last block of a sequence: its V rows past the end belong to someone else -> zero them (0 * x must be 0)
          if (row_live && my_j * kBlock + key_local >= it.slen) {
            const uint32_t vrow = sh.base + kOffV + st * kKVBytes + (uint32_t)r * 128u;
#pragma unroll
            for (int ck = 0; ck < 8; ++ck) {
              asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(vrow + ck * 16), "r"(0u) : "memory");
              asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(vrow + kHalfKV + ck * 16), "r"(0u) : "memory");
            }
          }
        }
        fence_async_smem();
        tc_fence_before();
        mbar_arrive(sh.bar(P_FULL));
      }
      if (!ok) break;

      // ------------------------------------------------------------------------------------------ epilogue
      if (it.ntiles > 0) {
        if (!wg_wait(sh, PV_DONE, (n_tile - 1) & 1u, status)) { ok = false; break; }
        tc_fence_after();
      }
      // combine the 128 partial row sums of each query column
#pragma unroll
      for (int c = 0; c < 64; ++c) red[r * 65 + c] = l_part[c];
      named_bar_sync(1, kSoftmaxThreads);
      if (wg_tid < 64) {
        float l = 0.f;
        for (int rr = 0; rr < 128; ++rr) l += red[rr * 65 + wg_tid];
        inv_l[wg_tid] = l > 0.f ? 1.0f / l : 0.f;
        if (lse != nullptr && wg_tid < it.q_valid)
          lse[(int64_t)it.h * m.total_tokens + tok0 + wg_tid] =
              l > 0.f ? (mref[wg_tid] + log2f(l)) * 0.6931471805599453f : -CUDART_INF_F;
      }
      named_bar_sync(1, kSoftmaxThreads);
      // O^T row r (d = r) -> staging [q][d] bf16 in the P buffer
      {
        uint16_t* stage = reinterpret_cast<uint16_t*>(smem + kOffP);
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          uint32_t ov[16];
          if (it.ntiles > 0) {
            tc_ld16(tmem + lane_addr + kColO + ch * 16, ov);
            tc_wait_ld();
          } else {
#pragma unroll
            for (int e = 0; e < 16; ++e) ov[e] = 0u;
          }
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const int c = ch * 16 + e;
            const float val = it.ntiles > 0 ? __uint_as_float(ov[e]) * inv_l[c] : 0.f;
            stage[c * 128 + r] = (uint16_t)(pack_bf16(val, 0.f) & 0xffffu);
          }
        }
      }
      tc_fence_before();
      named_bar_sync(1, kSoftmaxThreads);
      {
        const uint4* stage4 = reinterpret_cast<const uint4*>(smem + kOffP);
        for (int idx = wg_tid; idx < 64 * 16; idx += kSoftmaxThreads) {
          const int qrow = idx >> 4, chunk = idx & 15;
          if (qrow < it.q_valid)
            *reinterpret_cast<uint4*>(o + ((tok0 + qrow) * m.num_q_heads + it.h) * kHeadDim + chunk * 8) = stage4[idx];
        }
      }
      named_bar_sync(1, kSoftmaxThreads);   // staging buffer is free again before the next item's P
    }
  }

  // ------------------------------------------------------------------------------------------------ teardown
  // After a lost wait give copies and MMAs still in flight time to land before shared memory and TMEM go away.
  if (ld_shared_u32(sh.abort_flag()) != 0u)
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

// ------------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// [T, H, 128] bf16 viewed as (d, head, token); box = 64 d x 1 head x 64 tokens, 128-byte swizzle, zero fill past T.
static bool make_map(seer_ctx* ctx, CUtensorMap* map, const void* base, int64_t tokens, int heads) {
  EncodeTiledFn fn = (EncodeTiledFn)ctx->tmap_encode;
  const cuuint64_t dims[3] = {(cuuint64_t)kHeadDim, (cuuint64_t)heads, (cuuint64_t)tokens};
  const cuuint64_t strides[2] = {(cuuint64_t)kHeadDim * 2, (cuuint64_t)heads * kHeadDim * 2};
  const cuuint32_t box[3] = {64, 1, 64};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tc

seer_status init_attn_tc(seer_ctx* ctx) {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess)
    return SEER_ERR_CUDA;
  ctx->tmap_encode = fn;
  cudaError_t e = cudaFuncSetAttribute(tc::attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::kSmemBytes);
  return e == cudaSuccess ? SEER_OK : SEER_ERR_CUDA;
}

int launch_attn_tc(seer_ctx* ctx, const SeqMeta& m, const void* q, const void* k, const void* v,
                   const int32_t* row_ptr, const int32_t* col_idx, void* o, float* lse, cudaStream_t stream) {
  if (m.rows == 0) return 0;
  // the input pointers must be 16-byte aligned for TMA
  if ((((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)o) & 15) != 0) return -(int)cudaErrorMisalignedAddress;
  CUtensorMap mq, mk, mv;
  if (!tc::make_map(ctx, &mq, q, m.total_tokens, m.num_q_heads) || !tc::make_map(ctx, &mk, k, m.total_tokens, m.num_kv_heads) ||
      !tc::make_map(ctx, &mv, v, m.total_tokens, m.num_kv_heads))
    return -(int)cudaErrorInvalidValue;
  const unsigned grid = (unsigned)min((int64_t)ctx->num_sms, m.rows);
  tc::attn_tc_kernel<<<grid, tc::kThreads, tc::kSmemBytes, stream>>>(mq, mk, mv, m, row_ptr, col_idx, (uint16_t*)o, lse,
                                                                    ctx->d_status);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 1 : -(int)e;
}

}  // namespace seer
