// Block-sparse causal GQA attention (Sec. 3.3) on the Blackwell tensor path, second arrangement of the softmax work
// (seer_set_attn_impl 3).  Same transposed formulation, roles, memory path and lazy-reference softmax as attn_tc.cu:
//     S^T[128 keys x 64 q] = K_tile[128 x 128 d] * Q^T,     O^T[128 d x 64 q] += V_tile^T[128 d x 128 keys] * P^T,
// but the two softmax groups do not alternate tiles: both work on every tile, group g on query columns 32 g .. 32 g + 31
// of S^T, of P^T, of the single O^T accumulator, of the references and of the row sums.  Consequences:
//   * nothing is merged at the end of a work item and the groups never meet at a barrier: a group finishes its own 32
//     query rows (row sums over its four warps, 1 / l, its columns of O^T, its rows of o and lse) and goes on;
//   * the first-tile rebase and every later one work on 32 columns;
//   * one ring of six S^T buffers and one ring of four P^T buffers, a tile per slot; a tile's P^T is complete, and its
//     S^T buffer free, when all eight softmax warps have arrived;
//   * TMEM: 6 x 64 columns of S^T, 64 of O^T, 64 of references (32 per group, replicated in every lane).
// Measured against attn_tc.cu: per work item it costs about half (prologue + epilogue 4 900 clocks against 9 900 per
// group), per tile slightly more (a tcgen05.ld round trip takes about 220 clocks when eight warps read at once, 110 with
// four), so it is faster where lists are short (65 536 tokens with a 92 % threshold mask: 7.2 against 8.9 ms) and 3 %
// slower on long lists (131 072 tokens, TopK 1/10: 23.0 against 22.3 ms).
#include <cuda.h>
#include <math_constants.h>

#include <map>

#include "seer_internal.cuh"

namespace seer {
namespace tc2 {

constexpr int kThreads = 512;               // warps 0-3: K(+Q) producer, S^T issuer, -, P V issuer; 4-7 / 8-11: softmax groups A / B; 12-15: V producers
constexpr int kVProducerWarps = 4;
constexpr float kRefShift = 7.f;   // softmax references are kept this far (log2) above the column maxima they were taken from
constexpr int kHelperRegs = 56, kSoftmaxRegs = 200;   // register split after the role dispatch: (2 * 56 + 2 * 200) * 128 = 65536
constexpr int kGroupThreads = 128;
constexpr uint32_t kHalfQ = 64 * 128;            // bytes of one d-half of a 64-row tile (8 KB)
constexpr uint32_t kHalfKV = 128 * 128;          // bytes of one d-half of a 128-row tile (16 KB)
constexpr uint32_t kQBytes = 2 * kHalfQ;         // 16 KB
constexpr uint32_t kKVBytes = 2 * kHalfKV;       // 32 KB (K or V tile of 128 keys)
constexpr uint32_t kPBytes = 128 * 128;          // 16 KB  P^T [128 keys][64 q] bf16
// shared memory map (offsets from a 1024-byte aligned base)
constexpr int kKSlots = 2, kVSlots = 2;
constexpr uint32_t kOffQ = 0;                                     // 16 KB
constexpr uint32_t kOffK = kOffQ + kQBytes;                       // kKSlots x 32 KB ring
constexpr uint32_t kOffV = kOffK + kKSlots * kKVBytes;            // kVSlots x 32 KB ring
constexpr uint32_t kOffP = kOffV + kVSlots * kKVBytes;            // 4 x 16 KB ring of P^T tiles (a group's half also serves as its epilogue staging)
constexpr uint32_t kOffGrp = kOffP + 4 * kPBytes;                 // per-group small arrays
constexpr uint32_t kGrpMref = 0, kGrpAlpha = 128, kGrpWinv = 256, kGrpLsum = 512;   // 32 floats each; lsum: 4 x 32 floats
constexpr uint32_t kGrpBytes = 1024;
constexpr uint32_t kOffBar = kOffGrp + 2 * kGrpBytes;             // mbarriers
constexpr uint32_t kNumBars = 32;
constexpr uint32_t kOffMisc = kOffBar + kNumBars * 8;             // tmem base, abort flag
constexpr uint32_t kOffTrace = kOffMisc + 64;                     // diagnostics: 6 roles x 48 tags x (sum, count)
constexpr uint32_t kSmemBytes = kOffTrace + 6 * 48 * 16 + 1024;   // + alignment slack
static_assert(kSmemBytes <= 232448, "shared memory budget of one CTA");

constexpr int kSSlots = 6;   // S^T buffers: one ring, a tile per slot; both softmax groups read every tile (32 query columns each)
enum Bar { Q_FULL = 0, Q_EMPTY = 1, K_FULL = 2 /* + slot */, K_EMPTY = 5, V_FULL = 8, V_EMPTY = 10,
           S_FULL = 12 /* + ring slot */, S_EMPTY = 18 /* + ring slot */, P_FULL = 24 /* + P^T buffer */, PV_DONE = 28 /* + P^T buffer */ };

// TMEM columns: S^T ring slot s at 64 s (0..383); the O^T accumulator at 384; the softmax references at 448 (replicated in
// every lane: a shared-memory read in the inner loop queues behind the operand traffic of the tensor pipe, a TMEM read
// does not).  Softmax group g owns query columns 32 g .. 32 g + 31 of all three.
constexpr uint32_t kTmemCols = 512;
__device__ __forceinline__ uint32_t col_s(uint32_t slot) { return slot * 64u; }
constexpr uint32_t kColO = 384u, kColM = 448u;

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
__device__ __forceinline__ void tc_ld8(uint32_t taddr, uint32_t (&r)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr) : "memory");
}
// Waits for the loads of this thread; the loaded registers are in/out operands so that no use of them moves above it.
__device__ __forceinline__ void tc_wait_ld8(uint32_t (&a)[8], uint32_t (&b)[8]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(a[0]), "+r"(a[1]), "+r"(a[2]), "+r"(a[3]), "+r"(a[4]), "+r"(a[5]), "+r"(a[6]), "+r"(a[7]),
                 "+r"(b[0]), "+r"(b[1]), "+r"(b[2]), "+r"(b[3]), "+r"(b[4]), "+r"(b[5]), "+r"(b[6]), "+r"(b[7])
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
// kind::f16 instruction descriptor: fp32 accumulate, bf16 x bf16, M = 128, N = 64
constexpr uint32_t make_idesc(bool a_mn_major, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
         ((64u >> 3) << 17) | ((128u >> 4) << 24);
}
constexpr uint32_t kIdescS = make_idesc(false, false);
constexpr uint32_t kIdescPV = make_idesc(true, true);


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

// One pass over this group's 32 query columns of a 128 x 64 S^T tile, for the key row of this thread:
// p = 2^(s * sl2 - mref[c]).  s_addr / m_addr point at the group's first column; c0 is that column's index in the tile.
//   SUBTRACT == false: adds p to l[c], packs p to bf16 pairs in pk, returns the OR of the packed words: bit 14 or 30
//                      set means some p >= 2 (the references sit kRefShift above the column maxima, so that is a score
//                      2^(kRefShift + 1) above its reference maximum, or an infinity / NaN).
//   SUBTRACT == true : removes p from l[c] again (used before a rebase; pk is not touched).
// MASKED applies the causal mask of a diagonal block / drops a dead row.
template <bool MASKED, bool SUBTRACT, class TR = Tracer<false>>
__device__ __forceinline__ uint32_t softmax_pass(uint32_t s_addr, uint32_t m_addr, float sl2, bool row_live,
                                              bool diag, int key_local, int c0, float (&l)[32], uint32_t (&pk)[16],
                                              TR* tr = nullptr) {
  uint32_t ored = 0u;
  uint32_t sv[2][8], mv[2][8];
  tc_ld8(s_addr, sv[0]);
  tc_ld8(m_addr, mv[0]);
#pragma unroll
  for (int ch = 0; ch < 4; ++ch) {
    tc_wait_ld8(sv[ch & 1], mv[ch & 1]);
    if (tr) tr->ev(40 + ch, 0);
    if (ch < 3) {
      tc_ld8(s_addr + (ch + 1) * 8, sv[(ch + 1) & 1]);
      tc_ld8(m_addr + (ch + 1) * 8, mv[(ch + 1) & 1]);
    }
#pragma unroll
    for (int e = 0; e < 8; e += 4) {
      const int c = ch * 8 + e;                        // column within the group
      float x0 = fmaf(__uint_as_float(sv[ch & 1][e]), sl2, -__uint_as_float(mv[ch & 1][e]));
      float x1 = fmaf(__uint_as_float(sv[ch & 1][e + 1]), sl2, -__uint_as_float(mv[ch & 1][e + 1]));
      float x2 = fmaf(__uint_as_float(sv[ch & 1][e + 2]), sl2, -__uint_as_float(mv[ch & 1][e + 2]));
      float x3 = fmaf(__uint_as_float(sv[ch & 1][e + 3]), sl2, -__uint_as_float(mv[ch & 1][e + 3]));
      if (MASKED) {
        if (!row_live || (diag && key_local > c0 + c)) x0 = -CUDART_INF_F;
        if (!row_live || (diag && key_local > c0 + c + 1)) x1 = -CUDART_INF_F;
        if (!row_live || (diag && key_local > c0 + c + 2)) x2 = -CUDART_INF_F;
        if (!row_live || (diag && key_local > c0 + c + 3)) x3 = -CUDART_INF_F;
      }
      const float p0 = ex2f(x0), p1 = ex2f(x1), p2 = ex2f(x2), p3 = ex2f(x3);
      if (SUBTRACT) {
        l[c] -= p0; l[c + 1] -= p1; l[c + 2] -= p2; l[c + 3] -= p3;
      } else {
        l[c] += p0; l[c + 1] += p1; l[c + 2] += p2; l[c + 3] += p3;
        pk[c >> 1] = pack_bf16(p0, p1);
        pk[(c >> 1) + 1] = pack_bf16(p2, p3);
        ored |= pk[c >> 1] | pk[(c >> 1) + 1];
      }
    }
  }
  return ored;
}

// Sums l[0..31] over the 32 lanes of a warp: lane n ends with the total of column n.
__device__ __forceinline__ float warp_colsum32(const float (&l)[32], int lane) {
  float a[16], b[8], c[4], d[2];
  {
    const bool up = (lane & 16) != 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) a[i] = (up ? l[i + 16] : l[i]) + __shfl_xor_sync(0xffffffffu, up ? l[i] : l[i + 16], 16);
  }
  {
    const bool up = (lane & 8) != 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) b[i] = (up ? a[i + 8] : a[i]) + __shfl_xor_sync(0xffffffffu, up ? a[i] : a[i + 8], 8);
  }
  {
    const bool up = (lane & 4) != 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) c[i] = (up ? b[i + 4] : b[i]) + __shfl_xor_sync(0xffffffffu, up ? b[i] : b[i + 4], 4);
  }
  {
    const bool up = (lane & 2) != 0;
#pragma unroll
    for (int i = 0; i < 2; ++i) d[i] = (up ? c[i + 2] : c[i]) + __shfl_xor_sync(0xffffffffu, up ? c[i] : c[i + 2], 2);
  }
  const bool up = (lane & 1) != 0;
  return (up ? d[1] : d[0]) + __shfl_xor_sync(0xffffffffu, up ? d[0] : d[1], 1);
}

// ------------------------------------------------------------------------------------------------ kernel
template <bool kTrace, bool kChunk>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc2_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v, SeqMeta m, const int32_t* __restrict__ row_ptr,
               const int32_t* __restrict__ col_idx, const void* __restrict__ k_ptr, const void* __restrict__ v_ptr,
               uint16_t* __restrict__ o,
               float* __restrict__ lse, int* __restrict__ status, unsigned long long* __restrict__ trace) {
  extern __shared__ unsigned char smem_raw[];
  Shared sh;
  sh.base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (sh.base - smem_u32(smem_raw));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + kOffMisc);

  if (threadIdx.x == 0) {
    mbar_init(sh.bar(Q_FULL), 1);
    mbar_init(sh.bar(Q_EMPTY), 1);
    for (int i = 0; i < kKSlots; ++i) {
      mbar_init(sh.bar(K_FULL + i), 1);
      mbar_init(sh.bar(K_EMPTY + i), 1);
    }
    for (int i = 0; i < kVSlots; ++i) {
      mbar_init(sh.bar(V_FULL + i), 32 * kVProducerWarps);   // one arrival per producer lane, when its copies have landed
      mbar_init(sh.bar(V_EMPTY + i), 1);
    }
    for (int i = 0; i < 4; ++i) {
      mbar_init(sh.bar(P_FULL + i), 2 * kGroupThreads / 32);   // one arrival per softmax warp, both groups
      mbar_init(sh.bar(PV_DONE + i), 1);
    }
    for (int i = 0; i < kSSlots; ++i) {
      mbar_init(sh.bar(S_FULL + i), 1);
      mbar_init(sh.bar(S_EMPTY + i), 1);                   // passed on by the P V issuer when it has seen P_FULL
    }
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
  const unsigned long long cta_t0 = kTrace ? global_ns() : 0ull;
  const long long cta_c0 = kTrace ? clock64() : 0ll;

  // Ordinals shared by all roles: k = non-empty items seen by this CTA, g = tiles seen, cnt_a / cnt_b = tiles handed to
  // softmax group A / B.  Every role walks the same items and tiles, so the counters agree without communication.

  // Register split: the two helper warpgroups (warps 0-3, 12-15) give registers up, the softmax warpgroups take them.
  if (warp < 4 || warp >= 12) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kHelperRegs));
  // ============================================================================================ K (+Q) producer (TMA)
  if (warp == 0) {
    if (lane == 0) {
      Tracer<kTrace> tr; tr.init(trace, 0, smem + kOffTrace);
      uint32_t k = 0, g = 0, slot = 0, use = 0;
      bool ok = true;
      for (int64_t w = blockIdx.x; ok && w < m.rows; w += gridDim.x) {
        const Item it = decode_item<kChunk>(m, row_ptr, w);
        if (it.ntiles == 0) continue;
        if (!mbar_wait(sh, Q_EMPTY, (k & 1u) ^ 1u, status)) break;
        mbar_expect_tx(sh.bar(Q_FULL), kQBytes);
        const int tq = it.s0 + it.i * kBlock + (kChunk ? it.dq : 0);
        tma_load_3d(sh.base + kOffQ, &map_q, sh.bar(Q_FULL), 0, it.h, tq);
        tma_load_3d(sh.base + kOffQ + kHalfQ, &map_q, sh.bar(Q_FULL), 64, it.h, tq);
        ++k;
        int ja = list_block(it, col_idx, 0), jb = list_block(it, col_idx, 1);
        for (int t = 0; t < it.ntiles; ++t, ++g) {
          const int na = list_block(it, col_idx, 2 * t + 2), nb2 = list_block(it, col_idx, 2 * t + 3);   // next pair
          if (ja == -2 || jb == -2) atomicCAS(status, 0, (int)SEER_ERR_INVALID_INDEX);
          tr.sample(g); tr.ev(1, g);
          if (!mbar_wait(sh, K_EMPTY + (int)slot, (use & 1u) ^ 1u, status)) { ok = false; break; }
          tr.ev(2, g);
          const bool has_b = jb != -1;
          const int xa = ja < 0 ? 0 : ja, xb = jb < 0 ? 0 : jb;   // a rejected entry: any valid block, masked out in the softmax
          const uint32_t fb = sh.bar(K_FULL + (int)slot), dst = sh.base + kOffK + slot * kKVBytes;
          mbar_expect_tx(fb, has_b ? kKVBytes : kKVBytes / 2);
          const int ta = it.s0 + xa * kBlock, tb = it.s0 + xb * kBlock;
          tma_load_3d(dst, &map_k, fb, 0, it.g, ta);
          tma_load_3d(dst + kHalfKV, &map_k, fb, 64, it.g, ta);
          if (has_b) {
            tma_load_3d(dst + kHalfQ, &map_k, fb, 0, it.g, tb);
            tma_load_3d(dst + kHalfKV + kHalfQ, &map_k, fb, 64, it.g, tb);
          }
          if (++slot == (uint32_t)kKSlots) { slot = 0; ++use; }
          ja = na; jb = nb2;
        }
      }
      tr.flush();
    }
  }
  // ============================================================================================ V producers (cp.async)
  // V tiles come through the LSU path (cp.async, 16 bytes per request).  Measured on this part: TMA box gathers of
  // 128-byte rows sustain ~41 B/clk per SM, cp.async ~80, both together ~85 (the SM's fill limit) and neither slows the
  // MMAs, so K goes by TMA and V by cp.async.  Producer warp pw copies rows 16 pw .. 16 pw + 15 of each block of the tile;
  // each lane writes the 128-byte-swizzled layout the MMA descriptor expects (rows past the end of the sequence are
  // zero-filled: 0 * x must be 0); completion is asynchronous: every lane's copies arrive on the slot's mbarrier when they
  // have landed.
  else if (warp >= 12) {
    const int pw = warp - 12;
    Tracer<kTrace> tr; tr.init(lane == 0 && pw == 0 ? trace : nullptr, 2, smem + kOffTrace);
    const unsigned char* __restrict__ xg = reinterpret_cast<const unsigned char*>(v_ptr);
    const size_t row_bytes = (size_t)m.num_kv_heads * kHeadDim * 2;      // bytes between consecutive tokens
    const int chunk = lane & 15, rsub = lane >> 4;
    const int row0 = pw * (kBlock / kVProducerWarps);                    // first row of this warp's share of a block
    constexpr int kIters = kBlock / kVProducerWarps / 2;                 // 2 rows per warp instruction
    // destination offset of (row0 + 2 * itc + rsub, this lane's chunk) inside a block half, for itc mod 4 = 0..3
    uint32_t doff[4];
#pragma unroll
    for (int q4 = 0; q4 < 4; ++q4) {
      const int row = 2 * q4 + rsub;
      doff[q4] = (uint32_t)(chunk >> 3) * kHalfKV + (uint32_t)(row0 + row) * 128u + (uint32_t)(((chunk & 7) ^ (row & 7)) << 4);
    }
    uint32_t g = 0;
    bool ok = true;
    for (int64_t w = blockIdx.x; ok && w < m.rows; w += gridDim.x) {
      const Item it = decode_item<kChunk>(m, row_ptr, w);
      if (it.ntiles == 0) continue;
      int ja = list_block(it, col_idx, 0), jb = list_block(it, col_idx, 1);
      const unsigned char* seq_base = xg + ((size_t)it.s0 * m.num_kv_heads + it.g) * (kHeadDim * 2) + (size_t)chunk * 16 +
                                      (size_t)(row0 + rsub) * row_bytes;
      for (int t = 0; t < it.ntiles; ++t, ++g) {
        const int na = list_block(it, col_idx, 2 * t + 2), nb2 = list_block(it, col_idx, 2 * t + 3);
        const uint32_t st = g & 1u;
        tr.sample(g); tr.ev(3, g);
        if (!mbar_wait(sh, V_EMPTY + (int)st, ((g >> 1) & 1u) ^ 1u, status)) { ok = false; break; }
        tr.ev(4, g);
        const uint32_t dst0 = sh.base + kOffV + st * kKVBytes;
#pragma unroll 1
        for (int half_tile = 0; half_tile < 2; ++half_tile) {
          int j = half_tile ? jb : ja;
          if (j == -1) continue;                       // odd list: no second block
          if (j < 0) j = 0;                            // rejected entry: any valid block, masked out in the softmax
          const int rows_valid = it.slen - j * kBlock - row0 - rsub;   // this lane's rows 2 * itc below this are real
          const unsigned char* src = seq_base + (size_t)j * kBlock * row_bytes;
          const uint32_t dst = dst0 + (uint32_t)half_tile * 8192u;
#pragma unroll
          for (int itc = 0; itc < kIters; ++itc) {
            const bool valid = 2 * itc < rows_valid;
            const int sz = valid ? 16 : 0;
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst + doff[itc & 3] + (uint32_t)(itc >> 2) * 1024u),
                         "l"(valid ? src + (size_t)(2 * itc) * row_bytes : seq_base), "r"(sz) : "memory");
          }
        }
        asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(sh.bar(V_FULL + (int)st)) : "memory");
        ja = na; jb = nb2;
      }
    }
    asm volatile("cp.async.wait_all;" ::: "memory");   // nothing of this warp is in flight when the CTA ends
    tr.flush();
  }
  // ============================================================================================ S^T issuer
  else if (warp == 1) {
    if (lane == 0) {
      Tracer<kTrace> tr; tr.init(trace, 1, smem + kOffTrace);
      uint32_t k = 0, g = 0, slot = 0, use = 0, ss = 0, sph = 0;   // ss / sph: S^T ring slot and its use parity
      // descriptor bases; per K-step the start address advances by 32 bytes inside a 64-element swizzle atom and by
      // one d-half (16 KB / 8 KB) between atoms
      const uint64_t kd0 = make_desc(sh.base + kOffK, 16, 1024);
      const uint64_t qd = make_desc(sh.base + kOffQ, 16, 1024);
      bool ok = true;
      for (int64_t w = blockIdx.x; ok && w < m.rows; w += gridDim.x) {
        const Item it = decode_item<kChunk>(m, row_ptr, w);
        if (it.ntiles == 0) continue;
        if (!mbar_wait(sh, Q_FULL, k & 1u, status)) break;
        for (int t = 0; t < it.ntiles; ++t, ++g) {
          tr.sample(g); tr.ev(10, g);
          if (!mbar_wait(sh, K_FULL + (int)slot, use & 1u, status)) { ok = false; break; }
          tr.ev(11, g);
          if (!mbar_wait(sh, S_EMPTY + (int)ss, sph ^ 1u, status)) { ok = false; break; }
          tr.ev(12, g);
          tc_fence_after();
          const uint64_t kd = kd0 + (uint64_t)(slot * (kKVBytes >> 4));
          const uint32_t d = tmem + col_s(ss);
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            tc_mma(d, kd + (uint64_t)((kk >> 2) * (kHalfKV >> 4) + (kk & 3) * 2),
                   qd + (uint64_t)((kk >> 2) * (kHalfQ >> 4) + (kk & 3) * 2), kIdescS, kk > 0);
          tc_commit(sh.bar(S_FULL + (int)ss));
          tc_commit(sh.bar(K_EMPTY + (int)slot));
          if (t == it.ntiles - 1) tc_commit(sh.bar(Q_EMPTY));   // last S^T of the item: Q may be replaced
          tr.ev(17, g);
          if (++ss == (uint32_t)kSSlots) { ss = 0; sph ^= 1u; }
          if (++slot == (uint32_t)kKSlots) { slot = 0; ++use; }
        }
        ++k;
      }
      tr.flush();
    }
  }
  // ============================================================================================ P V issuer
  else if (warp == 3) {
    if (lane == 0) {
      Tracer<kTrace> tr; tr.init(trace, 3, smem + kOffTrace);
      uint32_t g = 0, ss = 0;                              // ss: S^T ring slot of tile g
      const uint64_t vd0 = make_desc(sh.base + kOffV, kHalfKV, 1024), vd1 = make_desc(sh.base + kOffV + kKVBytes, kHalfKV, 1024);
      const uint64_t pd0 = make_desc(sh.base + kOffP, kHalfKV, 1024);   // P^T buffer b lies b buffers on
      bool ok = true;
      for (int64_t w = blockIdx.x; ok && w < m.rows; w += gridDim.x) {
        const Item it = decode_item<kChunk>(m, row_ptr, w);
        for (int t = 0; t < it.ntiles; ++t, ++g) {
          const uint32_t st = g & 1u, pb = g & 3u;
          tr.sample(g); tr.ev(13, g);
          if (!mbar_wait(sh, V_FULL + st, (g >> 1) & 1u, status)) { ok = false; break; }
          tr.ev(14, g);
          if (!mbar_wait(sh, P_FULL + (int)pb, (g >> 2) & 1u, status)) { ok = false; break; }
          // both softmax groups have finished with the tile's S^T buffer as well (they read it before they wrote P^T)
          mbar_arrive(sh.bar(S_EMPTY + (int)ss));
          if (++ss == (uint32_t)kSSlots) ss = 0;
          tr.ev(15, g);
          fence_async_smem();     // V was written through the generic proxy (cp.async); the MMA reads through the async proxy
          tc_fence_after();
          const uint64_t vd = st ? vd1 : vd0, pd = pd0 + (uint64_t)(pb * (kPBytes >> 4));
          const uint32_t d = tmem + kColO;
          const uint32_t acc0 = t >= 1 ? 1u : 0u;                  // the first tile of an item starts O^T afresh
          // 16 keys (2048 bytes of 128-byte rows) per step; an odd list leaves the second block of its last tile out
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) tc_mma(d, vd + (uint64_t)(kk * 128), pd + (uint64_t)(kk * 128), kIdescPV, kk > 0 ? 1u : acc0);
          if (2 * t + 1 < it.nlist) {
#pragma unroll
            for (int kk = 4; kk < 8; ++kk) tc_mma(d, vd + (uint64_t)(kk * 128), pd + (uint64_t)(kk * 128), kIdescPV, 1u);
          }
          tc_commit(sh.bar(V_EMPTY + st));
          tc_commit(sh.bar(PV_DONE + (int)pb));
          tr.ev(19, g);
        }
      }
      tr.flush();
    }
  }
  }   // helper warpgroups
  // ============================================================================================ softmax groups
  // Both groups work on every tile: group g owns query columns 32 g .. 32 g + 31 (of S^T, of P^T, of the accumulator, of
  // the references and of the row sums), so nothing is ever merged between them and they never wait for each other;
  // a tile's P^T is complete, and its S^T buffer free, when all eight warps have arrived.
  else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kSoftmaxRegs));
    const int grp = (warp - 4) >> 2;                     // 0: columns 0..31, 1: columns 32..63
    const int gt = threadIdx.x - 128 - grp * kGroupThreads;   // 0..127 within the group
    const int gw = (warp - 4) & 3;                       // warp within the group
    const int quad = warp & 3;                           // TMEM lane quadrant this warp may access
    const int r = quad * 32 + lane;                      // key row of S^T / d row of O^T owned by this thread
    const int c0 = grp * 32;                             // first query column of the group
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    unsigned char* gsm = smem + kOffGrp + grp * kGrpBytes;
    float* mref = reinterpret_cast<float*>(gsm + kGrpMref);    // [32]
    float* alpha = reinterpret_cast<float*>(gsm + kGrpAlpha);  // [32]
    float* winv = reinterpret_cast<float*>(gsm + kGrpWinv);    // [32]
    float* lsum = reinterpret_cast<float*>(gsm + kGrpLsum);    // [4 warps][32]
    const int bar_sync = 1 + grp, bar_vote = 3 + grp;
    const float sl2 = m.softmax_scale * 1.4426950408889634f;
    const int key_local = r & 63;
    const uint32_t m_addr = tmem + lane_addr + kColM + (uint32_t)c0;
    const uint32_t o_addr = tmem + lane_addr + kColO + (uint32_t)c0;
    Tracer<kTrace> tr; tr.init(gt == 0 ? trace : nullptr, 4 + grp, smem + kOffTrace);
    uint32_t cnt = 0;                                    // tiles of this CTA so far
    uint32_t ss = 0, sph = 0;                            // S^T ring slot of tile cnt and its use parity
    bool ok = true;

    for (int64_t w = blockIdx.x; w < m.rows; w += gridDim.x) {
      tr.sample(0);
      const Item it = decode_item<kChunk>(m, row_ptr, w);
      const int64_t tok0 = (int64_t)it.s0 + (int64_t)it.i * kBlock + (kChunk ? it.dq : 0);   // first row of the item in q / o / lse
      float l_part[32];
#pragma unroll
      for (int c = 0; c < 32; ++c) l_part[c] = 0.f;
      if (gt < 32) mref[gt] = -CUDART_INF_F;
      named_bar_sync(bar_sync, kGroupThreads);

      int nja = list_block(it, col_idx, 0), njb = list_block(it, col_idx, 1);
      tr.ev(29, 0);
      for (int t = 0; t < it.ntiles; ++t, ++cnt) {
        const uint32_t pbuf = cnt & 3u;                  // P^T buffer of the tile
        tr.sample(cnt); tr.ev(20, cnt);
        bool fail = !mbar_wait(sh, S_FULL + (int)ss, sph, status);
        tr.ev(21, cnt);
        tc_fence_after();
        const int ja = nja, jb = njb;
        // the next tile: the loads are issued here and looked at after the pass
        const int raw_a = list_fetch(it, col_idx, 2 * t + 2), raw_b = list_fetch(it, col_idx, 2 * t + 3);
        const int my_j = r < 64 ? ja : jb;
        const bool row_live = my_j >= 0;                 // absent / rejected blocks contribute nothing
        const bool diag = my_j == it.i;
        const bool masked = !row_live || diag;           // uniform per warp (a warp lies in one block half)
        const uint32_t s_addr = tmem + lane_addr + col_s(ss) + (uint32_t)c0;
        if (++ss == (uint32_t)kSSlots) { ss = 0; sph ^= 1u; }
        uint32_t pk[16];
        // the first tile of an item has no references yet: it goes straight to the rebase path
        uint32_t over = 0x40004000u;
        if (!fail && t >= 1) over = masked ? softmax_pass<true, false, Tracer<kTrace>>(s_addr, m_addr, sl2, row_live, diag, key_local, c0, l_part, pk, &tr)
                                 : softmax_pass<false, false, Tracer<kTrace>>(s_addr, m_addr, sl2, row_live, diag, key_local, c0, l_part, pk, &tr);
        nja = list_check(it, 2 * t + 2, raw_a); njb = list_check(it, 2 * t + 3, raw_b);
        tr.ev(23, cnt);
        // P^T goes to buffer cnt & 3; the P V that read that buffer four tiles ago has normally long finished
        if (!fail && cnt >= 4) fail = !mbar_wait(sh, PV_DONE + (int)pbuf, ((cnt >> 2) - 1) & 1u, status);
        tr.ev(22, cnt);
        // one vote per tile: does any entry reach 2^(kRefShift + 1) times its reference maximum (or has a wait been lost)?
        const bool slow = named_bar_or(bar_vote, kGroupThreads, fail || (over & 0x40004000u) != 0u);
        tr.ev(24, cnt);
        if (slow) {
          // the group's columns of O^T are rescaled below: the P V of the previous tile must have finished (the P V of this
          // tile cannot start before this group arrives)
          if (!fail && t >= 1) fail = !mbar_wait(sh, PV_DONE + (int)((cnt - 1) & 3u), ((cnt - 1) >> 2) & 1u, status);
          tc_fence_after();
          if (named_bar_or(bar_vote, kGroupThreads, fail)) { ok = false; break; }
          // ---- rebase: take this tile's contribution out of the row sums again, find the exact column maxima, move
          // the references, rescale the row sums and O^T, and recompute the tile
          if (t >= 1) {
            if (masked) softmax_pass<true, true>(s_addr, m_addr, sl2, row_live, diag, key_local, c0, l_part, pk);
            else softmax_pass<false, true>(s_addr, m_addr, sl2, row_live, diag, key_local, c0, l_part, pk);
          }
          // column maxima of the tile: over the lanes of each warp by shuffles (16 columns at a time: lane pair l, l ^ 1
          // ends with column l >> 1 of the chunk), over the four warps through shared memory
#pragma unroll
          for (int ch = 0; ch < 2; ++ch) {
            uint32_t sv[16];
            tc_ld16(s_addr + ch * 16, sv);
            tc_wait_ld(sv);
            float xv[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              const int c = c0 + ch * 16 + e;
              float x = __uint_as_float(sv[e]) * sl2;
              if (!row_live || (diag && key_local > c)) x = -CUDART_INF_F;
              xv[e] = x;
            }
            const float cm = warp_colmax16(xv, lane);
            if ((lane & 1) == 0) lsum[gw * 32 + ch * 16 + (lane >> 1)] = cm;
          }
          named_bar_sync(bar_sync, kGroupThreads);
          if (gt < 32) {
            const float old = mref[gt];
            const float cm = fmaxf(fmaxf(lsum[gt], lsum[32 + gt]), fmaxf(lsum[64 + gt], lsum[96 + gt]));
            float nm = fmaxf(old, cm + kRefShift);
            if (nm == -CUDART_INF_F) nm = 0.f;           // nothing visible in this column yet
            // a query column past the end of a ragged block holds whatever tokens follow in the packed tensor: an
            // unreachable reference makes its p = 0, so that it can never ask for a rebase (results must not depend on
            // the neighbours in the batch)
            if (c0 + gt >= it.q_valid) nm = 1.0e30f;
            alpha[gt] = old == -CUDART_INF_F ? 0.f : exp2f(old - nm);
            mref[gt] = nm;
          }
          named_bar_sync(bar_sync, kGroupThreads);
#pragma unroll
          for (int ch = 0; ch < 2; ++ch) {                // this lane's copy of the new references
            uint32_t mv[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) mv[e] = __float_as_uint(mref[ch * 16 + e]);
            tc_st16(m_addr + ch * 16, mv);
          }
          tc_wait_st();
          // a reference that moved by more than 2^30 makes everything accumulated so far negligible (and the value
          // taken out above may not have been finite): start the column afresh
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            const float a = alpha[c];
            l_part[c] = (t < 1 || a < 9.3e-10f) ? 0.f : l_part[c] * a;
          }
          if (t >= 1) {                                  // O^T already holds earlier tiles of the item
#pragma unroll 1
            for (int ch = 0; ch < 2; ++ch) {
              uint32_t ov[16];
              tc_ld16(o_addr + ch * 16, ov);
              tc_wait_ld(ov);
#pragma unroll
              for (int e = 0; e < 16; ++e) ov[e] = __float_as_uint(__uint_as_float(ov[e]) * alpha[ch * 16 + e]);
              tc_st16(o_addr + ch * 16, ov);
            }
            tc_wait_st();
          }
          if (masked) softmax_pass<true, false>(s_addr, m_addr, sl2, row_live, diag, key_local, c0, l_part, pk);
          else softmax_pass<false, false>(s_addr, m_addr, sl2, row_live, diag, key_local, c0, l_part, pk);
        }
        tr.ev(26, 0);
        // this group's 64 bytes of P^T row r -> buffer cnt & 3 (128-byte swizzle: 16-byte chunks 4 g .. 4 g + 3 of the row)
        {
          const uint32_t prow = sh.base + kOffP + pbuf * kPBytes + (uint32_t)r * 128u;
#pragma unroll
          for (int ck = 0; ck < 4; ++ck) {
            const uint32_t a = prow + (uint32_t)(((4 * grp + ck) ^ (r & 7)) << 4);
            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(pk[ck * 4]), "r"(pk[ck * 4 + 1]),
                         "r"(pk[ck * 4 + 2]), "r"(pk[ck * 4 + 3]) : "memory");
          }
        }
        tr.ev(27, 0);
        fence_async_smem();
        tr.ev(28, 0);
        // one arrival per warp (128 would serialise on the barrier word); it also hands the S^T buffer back
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(sh.bar(P_FULL + (int)pbuf));
        tr.ev(25, cnt);
      }

      // ------------------------------------------------------------------------------------------ epilogue
      // The group's 32 query columns are its own: row sums over its four warps, 1 / l, its columns of O^T, its 32 rows
      // of o and lse.  Nothing is shared with the other group.
      tr.sample(0); tr.ev(30, (uint32_t)(w / gridDim.x));
      bool efail = !ok;
      if (ok && it.ntiles > 0)                           // the last P V of the item (completion is in order)
        efail = !mbar_wait(sh, PV_DONE + (int)((cnt - 1) & 3u), ((cnt - 1) >> 2) & 1u, status);
      tc_fence_after();
      lsum[gw * 32 + lane] = warp_colsum32(l_part, lane);
      if (named_bar_or(bar_vote, kGroupThreads, efail)) { ok = false; break; }
      if (gt < 32) {
        const float l = (lsum[gt] + lsum[32 + gt]) + (lsum[64 + gt] + lsum[96 + gt]);
        const bool live = l > 0.f;
        winv[gt] = live ? 1.0f / l : 0.f;
        if (lse != nullptr && c0 + gt < it.q_valid)
          lse[(int64_t)it.h * (kChunk ? m.total_q_tokens : m.total_tokens) + tok0 + c0 + gt] =
              live ? (mref[gt] + log2f(l)) * 0.6931471805599453f : -CUDART_INF_F;
      }
      named_bar_sync(bar_sync, kGroupThreads);
      // staging [32 q][128 d] bf16 in the group's half of P^T buffer 0 (its 64 bytes of each 128-byte row): nobody else
      // writes there, and the P V of a later tile reads the buffer only after this group has arrived for that tile
      unsigned char* stage = smem + kOffP + grp * 64;
      auto stage_at = [&](int byte) -> unsigned char* { return stage + (byte >> 6) * 128 + (byte & 63); };
      {
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          uint32_t ov[16];
          if (it.ntiles > 0) { tc_ld16(o_addr + ch * 16, ov); tc_wait_ld(ov); }
#pragma unroll
          for (int e = 0; e < 16; e += 4) {
            const float4 wv = *reinterpret_cast<const float4*>(&winv[ch * 16 + e]);
            const float w4[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const float val = it.ntiles > 0 ? __uint_as_float(ov[e + u]) * w4[u] : 0.f;
              *reinterpret_cast<uint16_t*>(stage_at(((ch * 16 + e + u) * 128 + r) * 2)) = (uint16_t)(pack_bf16(val, 0.f) & 0xffffu);
            }
          }
        }
      }
      tc_fence_before();
      named_bar_sync(bar_sync, kGroupThreads);   // staging complete; every TMEM read of the item by this group is done
      for (int idx = gt; idx < 32 * 16; idx += kGroupThreads) {
        const int qrow = c0 + (idx >> 4), chunk = idx & 15;
        if (qrow < it.q_valid)
          *reinterpret_cast<uint4*>(o + ((tok0 + qrow) * m.num_q_heads + it.h) * kHeadDim + chunk * 8) =
              *reinterpret_cast<const uint4*>(stage_at(idx * 16));
      }
      named_bar_sync(bar_sync, kGroupThreads);   // staging is free again before this group's next P^T
      tr.ev(31, (uint32_t)(w / gridDim.x));
    }
    tr.flush();
  }

  // ------------------------------------------------------------------------------------------------ teardown
  // After a lost wait give copies and MMAs still in flight time to land before shared memory and TMEM go away.
  if (ld_shared_u32(sh.abort_flag()) != 0u)
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  tc_fence_before();
  __syncthreads();
  if (kTrace && trace != nullptr && threadIdx.x == 0) { trace[6 * 8192 + blockIdx.x] = global_ns() - cta_t0; trace[6 * 8192 + 256 + blockIdx.x] = (unsigned long long)(clock64() - cta_c0); }  // wall time of this CTA: ns, SM clocks
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

}  // namespace tc2

seer_status init_attn_tc2(seer_ctx* ctx) {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess)
    return SEER_ERR_CUDA;
  ctx->tmap_encode = fn;
  cudaError_t e = cudaFuncSetAttribute(tc2::attn_tc2_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc2::kSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(tc2::attn_tc2_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc2::kSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(tc2::attn_tc2_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc2::kSmemBytes);
  return e == cudaSuccess ? SEER_OK : SEER_ERR_CUDA;
}

int launch_attn_tc2(seer_ctx* ctx, const SeqMeta& m, const void* q, const void* k, const void* v,
                   const int32_t* row_ptr, const int32_t* col_idx, void* o, float* lse, cudaStream_t stream) {
  if (m.rows == 0) return 0;
  // the input pointers must be 16-byte aligned for TMA
  if ((((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)o) & 15) != 0) return -(int)cudaErrorMisalignedAddress;
  CUtensorMap mq, mk, mv;
  if (!tc2::make_map(ctx, &mq, q, m.total_q_tokens, m.num_q_heads) || !tc2::make_map(ctx, &mk, k, m.total_tokens, m.num_kv_heads) ||
      !tc2::make_map(ctx, &mv, v, m.total_tokens, m.num_kv_heads))
    return -(int)cudaErrorInvalidValue;
  const unsigned grid = (unsigned)min((int64_t)ctx->num_sms, m.rows);
  if (m.chunked)               // chunked prefill (never instrumented)
    tc2::attn_tc2_kernel<false, true><<<grid, tc2::kThreads, tc2::kSmemBytes, stream>>>(mq, mk, mv, m, row_ptr, col_idx, k, v, (uint16_t*)o, lse,
                                                                          ctx->d_status, (unsigned long long*)ctx->trace);
  else if (ctx->trace != nullptr)   // the instrumented instantiation
    tc2::attn_tc2_kernel<true, false><<<grid, tc2::kThreads, tc2::kSmemBytes, stream>>>(mq, mk, mv, m, row_ptr, col_idx, k, v, (uint16_t*)o, lse,
                                                                    ctx->d_status, (unsigned long long*)ctx->trace);
  else
    tc2::attn_tc2_kernel<false, false><<<grid, tc2::kThreads, tc2::kSmemBytes, stream>>>(mq, mk, mv, m, row_ptr, col_idx, k, v, (uint16_t*)o, lse,
                                                                    ctx->d_status, (unsigned long long*)ctx->trace);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 1 : -(int)e;
}

}  // namespace seer
