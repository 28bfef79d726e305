// Pieces shared by the tcgen05 attention kernels: PTX wrappers (mbarrier, TMA, tcgen05, named barriers), shared-memory
// matrix descriptors, the work-item decoder, warp-level column reductions and the optional cycle accounting.
#pragma once

#include <cuda.h>
#include <math_constants.h>

#include "seer_internal.cuh"

namespace seer {
namespace tcc {


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
  uint32_t bar0;         // shared address of mbarrier 0
  uint32_t abort_addr;   // shared address of the abort flag
  unsigned long long limit_ns;   // a wait that lasts this long is declared lost (2 s unless a test shortens it)
  __device__ __forceinline__ uint32_t bar(int i) const { return bar0 + 8u * (uint32_t)i; }
  __device__ __forceinline__ uint32_t abort_flag() const { return abort_addr; }
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
template <int kSleepNs = 0>
__device__ __forceinline__ bool mbar_wait(const Shared& sh, int bar, uint32_t parity, int* status) {
  const uint32_t addr = sh.bar(bar);
  {
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(addr), "r"(parity) : "memory");
    if (done) return true;
  }
  if (mbar_try(addr, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try(addr, parity)) return true;
    if (kSleepNs > 0) __nanosleep(kSleepNs);   // a waiting helper must not take issue slots from the softmax warps of its scheduler
    if ((it & 255u) == 0u) {
      if (ld_shared_u32(sh.abort_flag()) != 0u) return false;
      if (global_ns() - t0 > sh.limit_ns) break;
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
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                 "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                 "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                 "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
               : "r"(taddr) : "memory");
}
// Waits for the loads of this thread; the loaded registers are in/out operands so that no use of them moves above it.
__device__ __forceinline__ void tc_wait_ld32(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
                 "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
                 "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :: "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                 "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// Same wait, with the loaded registers as in/out operands so that no use of them can be scheduled above it.
__device__ __forceinline__ void tc_wait_ld(uint32_t (&r)[16]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
               :: "memory");
}
// No instruction: makes the registers of a load issued before the last wait depend on that wait.
__device__ __forceinline__ void tc_tie(uint32_t (&r)[16]) {
  asm volatile(""
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
               :: "memory");
}
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

struct Item {
  int b, h, g, i, nb, s0, slen, l0, nlist, ntiles, q_valid, dq;
  int64_t row;
};

// kChunk: chunked prefill.  q / o / lse hold the last positions of each sequence only: their token index is the k / v
// token index plus dq, and query blocks before the chunk have nothing to do whatever their lists say.
template <bool kChunk>
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
  it.dq = 0;
  if (kChunk) {
    it.dq = m.qdelta[it.b];
    if (it.i < m.qoff[it.b]) { it.nlist = 0; it.q_valid = 0; }   // no tiles, and no row of o / lse is written
  }
  it.ntiles = (it.nlist + 1) >> 1;
  return it;
}

// Block index of list position p of an item: -1 past the end of the list, -2 for an entry outside [0, i].
__device__ __forceinline__ int list_block(const Item& it, const int32_t* __restrict__ col_idx, int p) {
  if (p >= it.nlist) return -1;
  const int j = col_idx[it.l0 + p];
  return (j < 0 || j > it.i) ? -2 : j;
}

// The same in two steps, so that the load can be issued long before its result is looked at.
__device__ __forceinline__ int list_fetch(const Item& it, const int32_t* __restrict__ col_idx, int p) {
  return p < it.nlist ? __ldg(col_idx + it.l0 + p) : -1;
}
__device__ __forceinline__ int list_check(const Item& it, int p, int raw) {
  if (p >= it.nlist) return -1;
  return (raw < 0 || raw > it.i) ? -2 : raw;
}

// Maximum of each of 16 columns over the 32 lanes of a warp; lanes l and l ^ 1 end with column l >> 1.
__device__ __forceinline__ float warp_colmax16(const float (&x)[16], int lane) {
  float a[8], b[4], c[2];
  {
    const bool up = (lane & 16) != 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) a[i] = fmaxf(up ? x[i + 8] : x[i], __shfl_xor_sync(0xffffffffu, up ? x[i] : x[i + 8], 16));
  }
  {
    const bool up = (lane & 8) != 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) b[i] = fmaxf(up ? a[i + 4] : a[i], __shfl_xor_sync(0xffffffffu, up ? a[i] : a[i + 4], 8));
  }
  {
    const bool up = (lane & 4) != 0;
#pragma unroll
    for (int i = 0; i < 2; ++i) c[i] = fmaxf(up ? b[i + 2] : b[i], __shfl_xor_sync(0xffffffffu, up ? b[i] : b[i + 2], 4));
  }
  const bool up = (lane & 2) != 0;
  const float d = fmaxf(up ? c[1] : c[0], __shfl_xor_sync(0xffffffffu, up ? c[0] : c[1], 2));
  return fmaxf(d, __shfl_xor_sync(0xffffffffu, d, 1));
}

// Sums l[0..63] over the 32 lanes of a warp; lane ends with the totals of columns (2*bitrev-ish) base, base+1
// where base = 32*b4 + 16*b3 + 8*b2 + 4*b1 + 2*b0 (b_i = bit i of the lane id).
__device__ __forceinline__ void warp_colsum(float (&l)[64], int lane, float& out0, float& out1, int& base) {
  float a[32];
  {
    const bool up = (lane & 16) != 0;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      const float send = up ? l[i] : l[i + 32];
      const float recv = __shfl_xor_sync(0xffffffffu, send, 16);
      a[i] = (up ? l[i + 32] : l[i]) + recv;
    }
  }
  float b[16];
  {
    const bool up = (lane & 8) != 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const float send = up ? a[i] : a[i + 16];
      const float recv = __shfl_xor_sync(0xffffffffu, send, 8);
      b[i] = (up ? a[i + 16] : a[i]) + recv;
    }
  }
  float c[8];
  {
    const bool up = (lane & 4) != 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float send = up ? b[i] : b[i + 8];
      const float recv = __shfl_xor_sync(0xffffffffu, send, 4);
      c[i] = (up ? b[i + 8] : b[i]) + recv;
    }
  }
  float d[4];
  {
    const bool up = (lane & 2) != 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float send = up ? c[i] : c[i + 4];
      const float recv = __shfl_xor_sync(0xffffffffu, send, 2);
      d[i] = (up ? c[i + 4] : c[i]) + recv;
    }
  }
  {
    const bool up = (lane & 1) != 0;
    const float s0 = up ? d[0] : d[2], s1 = up ? d[1] : d[3];
    const float r0 = __shfl_xor_sync(0xffffffffu, s0, 1), r1 = __shfl_xor_sync(0xffffffffu, s1, 1);
    out0 = (up ? d[2] : d[0]) + r0;
    out1 = (up ? d[3] : d[1]) + r1;
  }
  base = ((lane >> 4) & 1) * 32 + ((lane >> 3) & 1) * 16 + ((lane >> 2) & 1) * 8 + ((lane >> 1) & 1) * 4 + (lane & 1) * 2;
}

// Optional cycle accounting of CTA 0 (diagnostics): every role attributes the clocks between two consecutive marks to the
// tag of the later mark, accumulates per tag in shared memory, and writes the sums and mark counts to
// trace[role * 8192 + tag * 2 ...] when it ends.
constexpr int kTraceTags = 48;
template <bool ON>
struct Tracer {
  unsigned long long* p;      // global destination (nullptr: off)
  unsigned long long* acc;    // shared accumulators of this role: [tag][sum, count]
  long long last;
  bool on;
  // Only every 8th tile is timed: the bookkeeping of a timed tile (~100 clocks per event) would otherwise slow the
  // traced CTA by a quarter and distort what it measures.
  __device__ __forceinline__ void sample(uint32_t ordinal) {
    const bool was = on;
    on = p != nullptr && (ordinal & 7u) == 0u;
    if (on && !was) last = clock64();
  }
  __device__ __forceinline__ void init(unsigned long long* base, int role, unsigned char* smem_trace) {
    p = (base != nullptr && blockIdx.x == 0) ? base + (size_t)role * 8192 : nullptr;
    acc = reinterpret_cast<unsigned long long*>(smem_trace) + role * kTraceTags * 2;
    if (p != nullptr) {
      for (int i = 0; i < kTraceTags * 2; ++i) acc[i] = 0;
      last = clock64();
    }
    on = false;
  }
  __device__ __forceinline__ void ev(uint32_t tag, uint32_t) {
    if (on) {
      const long long now = clock64();
      acc[2 * tag] += (unsigned long long)(now - last);
      acc[2 * tag + 1] += 1;
      last = clock64();
    }
  }
  __device__ __forceinline__ void flush() {
    if (p != nullptr)
      for (int i = 0; i < kTraceTags * 2; ++i) p[i] = acc[i];
  }
};
template <>
struct Tracer<false> {   // the production instantiation carries no state and no code
  __device__ __forceinline__ void sample(uint32_t) {}
  __device__ __forceinline__ void init(unsigned long long*, int, unsigned char*) {}
  __device__ __forceinline__ void ev(uint32_t, uint32_t) {}
  __device__ __forceinline__ void flush() {}
};

// kind::f16 instruction descriptor: fp32 accumulate, bf16 x bf16, M = 128, N = n
constexpr uint32_t make_idesc(bool a_mn_major, bool b_mn_major, uint32_t n = 64u) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
         ((n >> 3) << 17) | ((128u >> 4) << 24);
}


}  // namespace tcc
}  // namespace seer
