// Block-sparse causal GQA attention (Sec. 3.3) on the Blackwell tensor path, two work items in flight per CTA.
//
// Orientation (as in every tcgen05 kernel of this library): a query block is 64 rows but the full-rate MMA shape is
// M = 128, and every (head, query block) has its own list, so the kernel computes the transposed problem: two listed KV
// blocks (128 keys) form the M dimension and the 64 queries the N dimension,
//     S^T[128 keys x 64 q] = K_tile[128 x 128 d] * Q^T          (A, B K-major in shared memory)
//     O^T[128 d x 64 q]   += V_tile^T[128 d x 128 keys] * P^T    (A, B MN-major in shared memory)
//
// Softmax references ride in the MMA.  A thread owns a key row of S^T (64 query columns) and would need all 64
// per-query references in every pass.  Instead the reference of column c, R[c] (a bf16 number in units of raw scores),
// is subtracted by the tensor core: a ninth K-step multiplies a column of ones (A) by a row holding -R[c] (B, 2 KB,
// written by the softmax group), so the accumulator holds s - R[c] and a pass is p = 2^(scale * x) with no per-column
// operand: half the TMEM reads of a pass and no reference registers.  R[c] sits 2^7 above the largest score its column
// had when it was taken; a tile whose entries all stay below 2 (seen on the packed bf16 words) needs no cross-thread
// reduction.  Otherwise, and on the first tile of a work item, the group rebases: exact column maxima, new R, row sums
// and O^T rescaled, the -R row rewritten.  The (at most two) S^T tiles already computed with the old row are corrected in
// place by one more MMA each, issued by a thread of the group: ones x (R_old - R_new), the difference split into three
// bf16 terms so that it is exact.
//
// Arrangement.  A CTA runs two independent streams; a stream owns a whole work item (head, query block) from its first
// tile to its stores: Q tile, K tile, V tile, P^T buffer, two S^T accumulators and one O^T accumulator in TMEM, its own
// producer threads (K and Q; V), MMA-issuing thread and softmax warpgroup.  The streams never meet at a barrier: while
// one sits in the first-tile rebase or the epilogue of its item, the other keeps the tensor pipe busy.  The issuing
// thread of a stream starts S^T of tile t + 2 right after P V of tile t.  Roles (512 threads): warps 0 / 2 = TMA
// producer of Q and K for stream 0 / 1, warps 1 / 3 = MMA issuer of stream 0 / 1 (warp 1 owns TMEM), warps 4-7 / 8-11
// = softmax group of stream 0 / 1, warps 12 / 13 = TMA producer of V for stream 0 / 1.  K and V have producers of their
// own because a copy takes ~700 clocks to land and each buffer is refilled as soon as its product has been read: one
// producer thread per stream would hold the K copy back behind the wait for the V buffer.  Every wait is bounded; a
// wait that runs out raises SEER_ERR_TIMEOUT and the CTA drains and exits.
#include <cuda.h>
#include <math_constants.h>

#include "attn_tc_common.cuh"

namespace seer {
namespace tc {

using namespace tcc;

constexpr int kThreads = 512;
constexpr float kRefShift = 7.f;   // softmax references are kept this far (log2) above the column maxima they were taken from
constexpr float kFirstShift = 12.f; // ... and this far above the score of the single key an item's first references are taken from
constexpr float kNoRef = -32768.f; // reference of a column that has not seen a key yet: the first visible score overflows it
constexpr int kHelperRegs = 56, kSoftmaxRegs = 200;   // (2 * 56 + 2 * 200) * 128 = 65536
constexpr int kGroupThreads = 128;
// a helper thread that polls a barrier shares its scheduler with two softmax warps: it sleeps between polls
constexpr int kProducerSleepNs = 128, kIssuerSleepNs = 0;
// of every eight column pairs of a pass this many take their exponentials on the FMA pipe, the others on the
// special-function unit (the pass alone is fastest with 3; the kernel, where the pass shares its schedulers with the
// other stream's, with 2: 19.9 ms against 20.4 with 3, 20.3 with 0 and 21.5 with 4 on the 128k TopK 1/10 workload)
constexpr int kPolyPairsOf8 = 2;
constexpr uint32_t kHalfQ = 64 * 128;            // bytes of one d-half of a 64-row tile (8 KB)
constexpr uint32_t kHalfKV = 128 * 128;          // bytes of one d-half of a 128-row tile (16 KB)
constexpr uint32_t kQBytes = 2 * kHalfQ;         // 16 KB
constexpr uint32_t kKVBytes = 2 * kHalfKV;       // 32 KB (K or V tile of 128 keys)
constexpr uint32_t kPBytes = 128 * 128;          // 16 KB  P^T [128 keys][64 q] bf16 (also the epilogue's staging)
// shared memory map (offsets from a 1024-byte aligned base); the big buffers of a stream are contiguous
constexpr uint32_t kStQ = 0, kStK = kQBytes, kStV = kStK + kKVBytes, kStP = kStV + kKVBytes;
constexpr uint32_t kStreamBytes = kStP + kPBytes;                 // 96 KB
constexpr uint32_t kOffOnes = 2 * kStreamBytes;                   // [128 x 16] bf16, columns 0..2 = 1 (no swizzle): 4 KB
constexpr uint32_t kOffQext = kOffOnes + 4096;                    // per stream [64 x 16] bf16, column 0 = -R[c]: 2 KB
constexpr uint32_t kOffQfix = kOffQext + 2 * 2048;                // per stream [64 x 16] bf16, columns 0..2 = R_old - R_new in three terms
constexpr uint32_t kOffGrp = kOffQfix + 2 * 2048;                 // per-group small arrays
constexpr uint32_t kGrpRcur = 0, kGrpAlpha = 256, kGrpLsum = 1024;   // lsum: 4 x 64 floats
constexpr uint32_t kGrpBytes = 2048;
constexpr uint32_t kOffBar = kOffGrp + 2 * kGrpBytes;             // mbarriers
constexpr int kBarsPerStream = 20;
constexpr uint32_t kNumBars = 2 * kBarsPerStream;
constexpr uint32_t kOffMisc = kOffBar + kNumBars * 8;             // tmem base, abort flag, the two streams' rings of work items (at +16, +32)
constexpr uint32_t kOffTrace = kOffMisc + 64;                     // diagnostics: 6 roles x 48 tags x (sum, count)
constexpr uint32_t kSmemBytes = kOffTrace + 6 * 48 * 16 + 1024;   // + alignment slack
static_assert(kSmemBytes <= 232448, "shared memory budget of one CTA");

enum Bar { Q_FULL = 0, Q_EMPTY = 1, K_FULL = 2, K_EMPTY = 3, V_FULL = 4, V_EMPTY = 5, S_FULL = 6 /* + buf */, P_FULL = 8,
           PV_DONE = 9, FIXED = 10, ITEM_FULL = 12 /* + slot, 4 slots */, ITEM_EMPTY = 16 /* + slot */ };
constexpr int kItemRing = 4;

constexpr uint32_t kTmemCols = 512;
// TMEM columns of a stream: two S^T accumulators, O^T
__device__ __forceinline__ uint32_t col_s(int s, uint32_t buf) { return (uint32_t)s * 256u + buf * 64u; }
__device__ __forceinline__ uint32_t col_o(int s) { return (uint32_t)s * 256u + 128u; }

constexpr uint32_t kIdescS = make_idesc(false, false);
constexpr uint32_t kIdescPV = make_idesc(true, true);

// shared-memory matrix descriptor without swizzle (K-major: 8 x 16-byte core matrices; lbo = distance between the two
// 16-byte K chunks, sbo = distance between 8-row groups)
__device__ __forceinline__ uint64_t make_desc_ns(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((saddr & 0x3ffffu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) | (1ull << 46);
}

__device__ __forceinline__ bool mbar_test(uint32_t addr, uint32_t parity) {
  uint32_t done;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(done) : "r"(addr), "r"(parity) : "memory");
  return done != 0;
}

// The smallest bf16 number >= v (v finite), as a float.
__device__ __forceinline__ float bf16_ceil(float v) {
  uint32_t b = __float_as_uint(v);
  if ((b & 0xffffu) != 0u) b = v >= 0.f ? ((b + 0x10000u) & 0xffff0000u) : (b & 0xffff0000u);
  return __uint_as_float(b);
}

// 2^x for two values at once on the FMA pipe (the special-function unit does 16 exponentials per clock and SM, a
// quarter of what the pass would need): x = n + f with n = round(x), 2^f by a cubic (relative error 7.5e-5, far below
// the bf16 rounding of P), 2^n by adding n to the exponent field.  x is clamped to [-125, 128] so that the exponent
// field stays in 1..254: below gives ~2^-125, above ~2^128 (finite in fp32, an infinity as bf16, which the caller's
// overflow test sees).
__device__ __forceinline__ float2 exp2_poly2(float2 x) {
  x.x = fminf(fmaxf(x.x, -125.f), 128.f); x.y = fminf(fmaxf(x.y, -125.f), 128.f);
  const float2 magic = make_float2(12582912.f, 12582912.f);        // 1.5 * 2^23: the sum's low mantissa bits are round(x)
  const float2 t = __fadd2_rn(x, magic);
  const float2 n = __fadd2_rn(t, make_float2(-12582912.f, -12582912.f));
  const float2 f = __fadd2_rn(x, make_float2(-n.x, -n.y));         // in [-0.5, 0.5]
  float2 r = __ffma2_rn(make_float2(0.05517168343067169f, 0.05517168343067169f), f, make_float2(0.2426111251115799f, 0.2426111251115799f));
  r = __ffma2_rn(r, f, make_float2(0.6932609677314758f, 0.6932609677314758f));
  r = __ffma2_rn(r, f, make_float2(0.9999280571937561f, 0.9999280571937561f));
  r.x = __int_as_float(__float_as_int(r.x) + (__float_as_int(t.x) << 23));
  r.y = __int_as_float(__float_as_int(r.y) + (__float_as_int(t.y) << 23));
  return r;
}

// One pass over a 128 x 64 S^T tile for the key row of this thread: p = 2^(sl2 * x), x = s - R[c] as the MMA left it.
// kPolyPairsOf8 of every eight column pairs take their exponentials on the FMA pipe, the others on the special-function unit.
//   SUBTRACT == false: adds p to l[c], packs p to bf16 pairs in pk, returns the OR of the packed words: bit 14 or 30
//                      set means some p >= 2, i.e. a score 2^(kRefShift + 1) above the maximum its reference was taken
//                      from, or an infinity / NaN.
//   SUBTRACT == true : removes p from l[c] again (used before a rebase; pk is not touched).
// MASKED applies the causal mask of a diagonal block, drops a dead row and the query columns past a ragged block.
template <bool MASKED, bool SUBTRACT>
__device__ __forceinline__ uint32_t tile_pass(uint32_t s_addr, float sl2, bool row_live, bool diag,
                                              int key_local, int q_valid, float (&l)[64], uint32_t (&pk)[32], uint32_t early_bar = 0u,
                                              uint32_t early_parity = 0u, bool* early_done = nullptr) {
  uint32_t ored = 0u;
  const float2 sl22 = make_float2(sl2, sl2);
  // two TMEM round trips per pass: the second half is requested before the first is worked on
  uint32_t sv[2][32];
  tc_ld32(s_addr, sv[0]);
#pragma unroll
  for (int ch = 0; ch < 2; ++ch) {
    tc_wait_ld32(sv[ch]);
    if (ch == 0) tc_ld32(s_addr + 32, sv[1]);
    // a barrier the caller needs after the pass is looked at here, so that the answer has arrived by then
    if (ch == 1 && early_done != nullptr) *early_done = mbar_test(early_bar, early_parity);
    // stage by stage over the 32 columns, each stage a run of independent instructions, in place
    float2 v[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __fmul2_rn(make_float2(__uint_as_float(sv[ch][2 * i]), __uint_as_float(sv[ch][2 * i + 1])), sl22);
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      if ((i & 7) < kPolyPairsOf8) v[i] = exp2_poly2(v[i]);
      else v[i] = make_float2(ex2f(v[i].x), ex2f(v[i].y));
    }
    if (MASKED) {
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int c = ch * 32 + 2 * i;
        if (!row_live || (diag && key_local > c) || c >= q_valid) v[i].x = 0.f;
        if (!row_live || (diag && key_local > c + 1) || c + 1 >= q_valid) v[i].y = 0.f;
      }
    }
    if (!SUBTRACT) {
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        pk[ch * 16 + i] = pack_bf16(v[i].x, v[i].y);
        ored |= pk[ch * 16 + i];
      }
    } else {
#pragma unroll
      for (int i = 0; i < 16; ++i) { v[i].x = -v[i].x; v[i].y = -v[i].y; }
    }
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const int c = ch * 32 + 2 * i;
      const float2 la = __fadd2_rn(make_float2(l[c], l[c + 1]), v[i]);
      l[c] = la.x; l[c + 1] = la.y;
    }
  }
  return ored;
}

// ------------------------------------------------------------------------------------------------ kernel
// kBlockMax: the same pipeline without V: instead of softmax(S) V the kernel writes, for every list entry, the largest
// probability exp(scale * s - lse) of its 64 x 64 tile (Sec. 3.2, Eq. 2 on the listed blocks), `lse` being an input.
// The log-sum-exp of a query column is subtracted by the tensor core exactly like a softmax reference (as three bf16
// terms, so exactly to fp32), a thread takes the maximum of its key row, a block's maximum is one redux per warp.
template <bool kTrace, bool kChunk, bool kBlockMax = false>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, SeqMeta m,
                const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx,
                uint16_t* __restrict__ o, float* __restrict__ lse, int* __restrict__ status,
                unsigned long long* __restrict__ trace, float* __restrict__ block_max = nullptr,
                int* __restrict__ work_counter = nullptr) {
  extern __shared__ unsigned char smem_raw[];
  Shared sh;
  sh.base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  sh.bar0 = sh.base + kOffBar;
  sh.abort_addr = sh.base + kOffMisc + 8;
  sh.limit_ns = (unsigned long long)m.wait_limit_us * 1000ull;
  unsigned char* smem = smem_raw + (sh.base - smem_u32(smem_raw));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + kOffMisc);

  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; ++s) {
      const int b = s * kBarsPerStream;
      mbar_init(sh.bar(b + Q_FULL), 1);
      mbar_init(sh.bar(b + Q_EMPTY), 1);
      mbar_init(sh.bar(b + K_FULL), 1);
      mbar_init(sh.bar(b + K_EMPTY), 1);
      mbar_init(sh.bar(b + V_FULL), 1);
      mbar_init(sh.bar(b + V_EMPTY), 1);
      mbar_init(sh.bar(b + S_FULL), 1);
      mbar_init(sh.bar(b + S_FULL + 1), 1);
      mbar_init(sh.bar(b + P_FULL), 4);                       // one arrival per warp of the softmax group
      mbar_init(sh.bar(b + PV_DONE), 1);
      mbar_init(sh.bar(b + FIXED), 1);
      for (int i = 0; i < kItemRing; ++i) {
        mbar_init(sh.bar(b + ITEM_FULL + i), 1);
        mbar_init(sh.bar(b + ITEM_EMPTY + i), 3);             // the V producer, the issuer and the softmax group have read the slot
      }
    }
    st_shared_u32(sh.abort_flag(), 0u);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // the column of ones, the two -R rows (R = 0) and the per-group arrays that must start defined
  for (uint32_t i = threadIdx.x; i < (4096u + 4u * 2048u) / 4u; i += kThreads) {
    const uint32_t off = i * 4u;   // rows of the first K chunk are 16 bytes apart: elements 0, 1 | 2, 3 | ...
    reinterpret_cast<uint32_t*>(smem + kOffOnes)[i] = off >= 2048u ? 0u : (off & 15u) == 0u ? 0x3f803f80u : (off & 15u) == 4u ? 0x3f80u : 0u;
  }
  for (uint32_t i = threadIdx.x; i < 2u * kGrpBytes / 4u; i += kThreads) reinterpret_cast<uint32_t*>(smem + kOffGrp)[i] = 0u;
  fence_async_smem();
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

  // Every role of stream s walks the same items w = 2 * blockIdx.x + s, + 2 * gridDim.x, ... and the same tiles, so
  // their ordinals (items seen, tiles seen) agree without communication.
  const int64_t w_step = 2 * (int64_t)gridDim.x;
  // Work items.  Without a counter a stream takes the items 2 * CTA + stream, + 2 * grid, ... (static deal).  With one
  // (`work_counter`, zero at launch) the stream's Q / K producer draws the next item number from it when it starts an
  // item and passes it to the stream's other roles through a ring of four shared-memory words, each with a full and an
  // empty mbarrier: a slot is rewritten only when the V producer, the issuer and the softmax group have all read it
  // (items with empty lists cost their roles nothing, so without the empty barrier the producer could lap the ring).
  // A negative number ends the stream.  Results do not depend on which stream runs an item.
  const bool dyn = !kBlockMax && work_counter != nullptr;
  auto ring_addr = [&](int s, uint32_t n) -> uint32_t { return sh.base + kOffMisc + 16u + (uint32_t)s * 16u + (n & 3u) * 4u; };
  // consumer side: the n-th item of stream s (false: no more items, or a lost wait)
  auto next_item = [&](int s, uint32_t n, int64_t& w) -> bool {
    if (!dyn) { w = 2 * (int64_t)blockIdx.x + s + (int64_t)n * w_step; return w < m.rows; }
    if (!mbar_wait<kProducerSleepNs>(sh, s * kBarsPerStream + ITEM_FULL + (int)(n & 3u), (n >> 2) & 1u, status)) return false;
    w = (int64_t)(int32_t)ld_shared_u32(ring_addr(s, n));
    return w >= 0;
  };
  // a single-thread role has read slot n (the softmax group arrives once, after it has met)
  auto release_item = [&](int s, uint32_t n) {
    if (dyn) mbar_arrive(sh.bar(s * kBarsPerStream + ITEM_EMPTY + (int)(n & 3u)));
  };

  if (warp < 4 || warp >= 12) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kHelperRegs));
    // ========================================================================================== producers (TMA)
    // warps 0 / 2: Q and K of stream 0 / 1; warps 12 / 13: V of stream 0 / 1
    if (warp == 0 || warp == 2 || warp == 12 || warp == 13) {
      if (lane == 0 && !(kBlockMax && warp >= 12)) {       // (no V in the block-maximum pass)
        const bool is_v = warp >= 12;
        const int s = is_v ? warp - 12 : warp >> 1, bb = s * kBarsPerStream;
        const uint32_t sbase = sh.base + (uint32_t)s * kStreamBytes;
        Tracer<kTrace> tr; tr.init(s == 0 ? trace : nullptr, is_v ? 2 : 0, smem + kOffTrace);
        const CUtensorMap* map = is_v ? &map_v : &map_k;
        const int full = bb + (is_v ? V_FULL : K_FULL), empty = bb + (is_v ? V_EMPTY : K_EMPTY);
        const uint32_t dst = sbase + (is_v ? kStV : kStK);
        uint32_t nitem = 0, cnt = 0;
        bool ok = true;
        int drawn = (dyn && !is_v) ? atomicAdd(work_counter, 1) : 0;   // the Q / K producer draws the stream's items
        for (uint32_t n = 0; ok; ++n) {
          int64_t w;
          if (dyn && !is_v) {
            w = drawn;
            const bool more = w < m.rows;
            // the slot's previous content (item n - 4) has been read by everyone
            if (!mbar_wait<kProducerSleepNs>(sh, bb + ITEM_EMPTY + (int)(n & 3u), ((n >> 2) & 1u) ^ 1u, status)) break;
            st_shared_u32(ring_addr(s, n), more ? (uint32_t)drawn : 0xffffffffu);
            mbar_arrive(sh.bar(bb + ITEM_FULL + (int)(n & 3u)));
            if (!more) break;
            drawn = atomicAdd(work_counter, 1);                        // the next one is on its way while this one is copied
          } else {
            const bool more = next_item(s, n, w);
            release_item(s, n);
            if (!more) break;
          }
          const Item it = decode_item<kChunk>(m, row_ptr, w);
          if (it.ntiles == 0) continue;
          if (!is_v) {
            if (!mbar_wait<kProducerSleepNs>(sh, bb + Q_EMPTY, (nitem & 1u) ^ 1u, status)) break;
            mbar_expect_tx(sh.bar(bb + Q_FULL), kQBytes);
            const int tq = it.s0 + it.i * kBlock + (kChunk ? it.dq : 0);
            tma_load_3d(sbase + kStQ, &map_q, sh.bar(bb + Q_FULL), 0, it.h, tq);
            tma_load_3d(sbase + kStQ + kHalfQ, &map_q, sh.bar(bb + Q_FULL), 64, it.h, tq);
            ++nitem;
          }
          int ja = list_block(it, col_idx, 0), jb = list_block(it, col_idx, 1);
          for (int t = 0; t < it.ntiles; ++t, ++cnt) {
            const int na = list_block(it, col_idx, 2 * t + 2), nb2 = list_block(it, col_idx, 2 * t + 3);   // next pair
            if (!is_v && (ja == -2 || jb == -2)) atomicCAS(status, 0, (int)SEER_ERR_INVALID_INDEX);
            tr.sample(cnt); tr.ev(1, cnt);
            if (!mbar_wait<kProducerSleepNs>(sh, empty, (cnt & 1u) ^ 1u, status)) { ok = false; break; }
            tr.ev(2, cnt);
            const bool has_b = jb != -1;
            const int xa = ja < 0 ? 0 : ja, xb = jb < 0 ? 0 : jb;   // a rejected entry: any valid block, masked out in the softmax
            // test hook: one V copy that is never issued, so that the issuer's wait for it runs out
            if (is_v && s == 0 && blockIdx.x == 0 && m.lose_v_copy >= 0 && cnt == (uint32_t)m.lose_v_copy) { ja = na; jb = nb2; continue; }
            const uint32_t fb = sh.bar(full);
            mbar_expect_tx(fb, has_b ? kKVBytes : kKVBytes / 2);
            const int ta = it.s0 + xa * kBlock, tb = it.s0 + xb * kBlock;
            tma_load_3d(dst, map, fb, 0, it.g, ta);
            tma_load_3d(dst + kHalfKV, map, fb, 64, it.g, ta);
            if (has_b) {
              tma_load_3d(dst + kHalfQ, map, fb, 0, it.g, tb);
              tma_load_3d(dst + kHalfKV + kHalfQ, map, fb, 64, it.g, tb);
            }
            ja = na; jb = nb2;
          }
        }
        tr.flush();
      }
    }
    // ========================================================================================== MMA issuer of a stream
    else if (warp == 1 || warp == 3) {
      if (lane == 0) {
        const int s = warp >> 1, bb = s * kBarsPerStream;
        const uint32_t sbase = sh.base + (uint32_t)s * kStreamBytes;
        Tracer<kTrace> tr; tr.init(trace, s == 0 ? 1 : 3, smem + kOffTrace);
        // (the low word of a descriptor holds the start address and the leading-dimension offset, the high word is constant)
        const uint64_t desc_hi_k = make_desc(0, 16, 1024) & 0xffffffff00000000ull;
        const uint64_t desc_hi_v = make_desc(0, kHalfKV, 1024) & 0xffffffff00000000ull;
        const uint32_t kd_lo = (uint32_t)make_desc(sbase + kStK, 16, 1024), qd_lo = (uint32_t)make_desc(sbase + kStQ, 16, 1024);
        const uint32_t vd_lo = (uint32_t)make_desc(sbase + kStV, kHalfKV, 1024), pd_lo = (uint32_t)make_desc(sbase + kStP, kHalfKV, 1024);
        const uint64_t ones_d = make_desc_ns(sh.base + kOffOnes, 2048, 128);
        const uint64_t qext_d = make_desc_ns(sh.base + kOffQext + (uint32_t)s * 2048u, 1024, 128);
        const uint32_t d_o = tmem + col_o(s);
        uint32_t nitem = 0, cs = 0, cp = 0;   // items, S^T tiles issued, P V tiles issued (of this stream)
        bool ok = true;
        // S^T of the next tile of the stream (ordinal cs) into buffer cs & 1: eight K-steps over d, a ninth that
        // subtracts the softmax references
        auto issue_s = [&](bool last_of_item, bool with_refs) -> bool {
          tr.ev(10, cs);
          if (!mbar_wait(sh, bb + K_FULL, cs & 1u, status)) return false;
          tr.ev(11, cs);
          tc_fence_after();
          const uint32_t d = tmem + col_s(s, cs & 1u);
          uint32_t klo = kd_lo, qlo = qd_lo;
          asm volatile("" : "+r"(klo), "+r"(qlo));   // the descriptors are formed here, not kept in registers across the loop
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            tc_mma(d, desc_hi_k | (uint64_t)(klo + (uint32_t)((kk >> 2) * (kHalfKV >> 4) + (kk & 3) * 2)),
                   desc_hi_k | (uint64_t)(qlo + (uint32_t)((kk >> 2) * (kHalfQ >> 4) + (kk & 3) * 2)), kIdescS, kk > 0);
          if (with_refs) tc_mma(d, ones_d, qext_d, kIdescS, 1u);
          tc_commit(sh.bar(bb + S_FULL + (int)(cs & 1u)));
          tc_commit(sh.bar(bb + K_EMPTY));
          if (last_of_item) tc_commit(sh.bar(bb + Q_EMPTY));   // last S^T of the item: Q may be replaced
          tr.ev(12, cs);
          ++cs;
          return true;
        };
        for (uint32_t n = 0; ok; ++n) {
          int64_t w;
          const bool more = next_item(s, n, w);
          release_item(s, n);
          if (!more) break;
          const Item it = decode_item<kChunk>(m, row_ptr, w);
          if (it.ntiles == 0) continue;
          tr.sample(cs);
          if (!mbar_wait(sh, bb + Q_FULL, nitem & 1u, status)) break;
          ++nitem;
          // the first two tiles of an item are computed without references (the row still holds those of the previous
          // item, and a result must not depend on which item came before): the group subtracts its first references
          // from them in place
          if (!issue_s(it.ntiles == 1, false)) break;
          if (it.ntiles > 1 && !issue_s(it.ntiles == 2, false)) break;
          for (int t = 0; t < it.ntiles; ++t, ++cp) {
            tr.sample(cp); tr.ev(13, cp);
            if constexpr (kBlockMax) {
              // the group has taken the maxima of S^T buffer cp & 1: the buffer is free for the tile after next
              if (!mbar_wait<kIssuerSleepNs>(sh, bb + P_FULL, cp & 1u, status)) { ok = false; break; }
              if (t + 2 < it.ntiles && !issue_s(t + 3 == it.ntiles, true)) { ok = false; break; }
              continue;
            }
            if (!mbar_wait(sh, bb + V_FULL, cp & 1u, status)) { ok = false; break; }
            tr.ev(14, cp);
            // P^T of tile t is complete; the group has also finished with S^T buffer cp & 1 (and, at t = 0, with the
            // O^T accumulator of the previous item)
            if (!mbar_wait<kIssuerSleepNs>(sh, bb + P_FULL, cp & 1u, status)) { ok = false; break; }
            tr.ev(15, cp);
            tc_fence_after();
            // 16 keys (2048 bytes of 128-byte rows) per step; an odd list leaves the second block of its last tile out
            uint32_t vlo = vd_lo, plo = pd_lo;
            asm volatile("" : "+r"(vlo), "+r"(plo));
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              tc_mma(d_o, desc_hi_v | (uint64_t)(vlo + (uint32_t)(kk * 128)), desc_hi_v | (uint64_t)(plo + (uint32_t)(kk * 128)), kIdescPV, (kk > 0 || t > 0) ? 1u : 0u);
            if (2 * t + 1 < it.nlist) {
#pragma unroll
              for (int kk = 4; kk < 8; ++kk)
                tc_mma(d_o, desc_hi_v | (uint64_t)(vlo + (uint32_t)(kk * 128)), desc_hi_v | (uint64_t)(plo + (uint32_t)(kk * 128)), kIdescPV, 1u);
            }
            tc_commit(sh.bar(bb + V_EMPTY));
            tc_commit(sh.bar(bb + PV_DONE));
            tr.ev(16, cp);
            if (t + 2 < it.ntiles && !issue_s(t + 3 == it.ntiles, true)) { ok = false; break; }
          }
        }
        tr.flush();
      }
    }
  }   // helper warpgroups
  // ============================================================================================ softmax groups
  else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kSoftmaxRegs));
    const int s = (warp - 4) >> 2, bb = s * kBarsPerStream;
    const int gt = threadIdx.x - 128 - s * kGroupThreads;   // 0..127 within the group
    const int gw = (warp - 4) & 3;                          // warp within the group
    const int quad = warp & 3;                              // TMEM lane quadrant this warp may access
    const int r = quad * 32 + lane;                         // key row of S^T / d row of O^T owned by this thread
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    unsigned char* gsm = smem + kOffGrp + s * kGrpBytes;
    float* rcur = reinterpret_cast<float*>(gsm + kGrpRcur);   // R[c], in units of raw scores (always a bf16 number)
    float* alpha = reinterpret_cast<float*>(gsm + kGrpAlpha);
    float* lsum = reinterpret_cast<float*>(gsm + kGrpLsum);
    uint16_t* qext = reinterpret_cast<uint16_t*>(smem + kOffQext + s * 2048);
    uint16_t* qfix = reinterpret_cast<uint16_t*>(smem + kOffQfix + s * 2048);
    const uint64_t ones_d = make_desc_ns(sh.base + kOffOnes, 2048, 128);
    const uint64_t qfix_d = make_desc_ns(sh.base + kOffQfix + (uint32_t)s * 2048u, 1024, 128);
    uint32_t nfix = 0;                                      // rebases of this stream so far
    const int bar_sync = 1 + s, bar_vote = 3 + s;
    const float sl2 = m.softmax_scale * 1.4426950408889634f;
    const float shift_raw = kRefShift / sl2;
    const int key_local = r & 63;
    const uint32_t p_base = sh.base + (uint32_t)s * kStreamBytes + kStP;
    unsigned char* p_gen = smem + (size_t)s * kStreamBytes + kStP;
    const uint32_t o_addr = tmem + lane_addr + col_o(s);
    Tracer<kTrace> tr; tr.init(gt == 0 ? trace : nullptr, 4 + s, smem + kOffTrace);
    uint32_t cnt = 0;                                       // tiles this stream has processed
    bool ok = true;
    // diagnostics (traced build): clocks of every steady-state tile by segment, kept in registers
    long long seg[16] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0}, seg_last = 0;
    unsigned seg_n = 0, nreb = 0;
#define SEG(k) do { if constexpr (kTrace) { const long long now_ = clock64(); seg[k] += now_ - seg_last; seg_last = now_; } } while (0)

    if constexpr (kBlockMax) {
      int* wmax = reinterpret_cast<int*>(lsum);             // [2 tile parities][4 warps]: maxima as order-preserving integers
      bool sticky_fail = false;
      const float inv_scale = 1.0f / m.softmax_scale;
      for (int64_t w = 2 * (int64_t)blockIdx.x + s; ok && w < m.rows; w += w_step) {
        const Item it = decode_item<kChunk>(m, row_ptr, w);
        if (it.ntiles == 0) continue;
        const int64_t tok0 = (int64_t)it.s0 + (int64_t)it.i * kBlock + (kChunk ? it.dq : 0);
        // -R[c], R[c] = lse[c] / scale (the log-sum-exp in units of raw scores), as three truncated bf16 terms in
        // columns 0..2 of both reference rows (the first two tiles are corrected in place, the later ones get it from the
        // ninth K-step of their MMA)
        if (gt < 64) {
          float L = gt < it.q_valid ? lse[(int64_t)it.h * (kChunk ? m.total_q_tokens : m.total_tokens) + tok0 + gt] : 0.f;
          if (!(fabsf(L) < 3.0e38f)) L = 0.f;               // a query without a key has no probabilities to report
          const float d = -L * inv_scale;
          const uint32_t hi = __float_as_uint(d) & 0xffff0000u;
          const float r1 = d - __uint_as_float(hi);
          const uint32_t mid = __float_as_uint(r1) & 0xffff0000u;
          const uint32_t lo = __float_as_uint(r1 - __uint_as_float(mid)) & 0xffff0000u;
          *reinterpret_cast<uint2*>(qfix + gt * 8) = make_uint2((hi >> 16) | mid, lo >> 16);
          *reinterpret_cast<uint2*>(qext + gt * 8) = make_uint2((hi >> 16) | mid, lo >> 16);
          fence_async_smem();
        }
        int ja = list_block(it, col_idx, 0), jb = list_block(it, col_idx, 1);
        for (int t = 0; t < it.ntiles; ++t, ++cnt) {
          const uint32_t sbuf = cnt & 1u;
          // (a lost wait does not leave the loop here: the warps of a group meet only at an item's first tile, and all
          // of them have to get there; the failure is voted on at that point)
          bool fail = !mbar_wait(sh, bb + S_FULL + (int)sbuf, (cnt >> 1) & 1u, status);
          if (t == 0) {
            fail = fail || sticky_fail;
            if (!fail && it.ntiles > 1) fail = !mbar_wait(sh, bb + S_FULL + (int)(sbuf ^ 1u), ((cnt + 1) >> 1) & 1u, status);
            tc_fence_after();
            if (named_bar_or(bar_vote, kGroupThreads, fail)) { ok = false; break; }
            if (gt == 0) {
              tc_mma(tmem + col_s(s, sbuf), ones_d, qfix_d, kIdescS, 1u);
              if (it.ntiles > 1) tc_mma(tmem + col_s(s, sbuf ^ 1u), ones_d, qfix_d, kIdescS, 1u);
              tc_commit(sh.bar(bb + FIXED));
            }
            if (named_bar_or(bar_vote, kGroupThreads, !mbar_wait(sh, bb + FIXED, nfix & 1u, status))) { ok = false; break; }
            ++nfix;
          }
          tc_fence_after();
          const int na = list_block(it, col_idx, 2 * t + 2), nb2 = list_block(it, col_idx, 2 * t + 3);
          const int my_j = r < 64 ? ja : jb;
          const bool diag = my_j == it.i;
          const uint32_t s_addr = tmem + lane_addr + col_s(s, sbuf);
          float mx = -CUDART_INF_F;                         // largest s - R over the causal queries of this key row
#pragma unroll
          for (int ch = 0; ch < 2; ++ch) {
            uint32_t sv[32];
            tc_ld32(s_addr + ch * 32, sv);
            tc_wait_ld32(sv);
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              const int c = ch * 32 + e;
              if (c < it.q_valid && !(diag && key_local > c)) mx = fmaxf(mx, __uint_as_float(sv[e]));
            }
          }
          if (my_j < 0 || fail || !(mx == mx)) mx = -CUDART_INF_F;
          int key = __float_as_int(mx);
          key ^= (key >> 31) & 0x7fffffff;                  // order-preserving map float -> int
          key = __reduce_max_sync(0xffffffffu, key);
          if (lane == 0) wmax[sbuf * 4 + gw] = key;
          // this warp is done with the S^T buffer (four arrivals free it); the two warps of a key block meet to
          // combine their maxima, the group as a whole does not
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(sh.bar(bb + P_FULL));
          const int half = gw >> 1;
          named_bar_sync(5 + 2 * s + half, 64);
          if ((gw & 1) == 0 && lane == 0 && 2 * t + half < it.nlist) {
            int kx = max(wmax[sbuf * 4 + 2 * half], wmax[sbuf * 4 + 2 * half + 1]);
            kx ^= (kx >> 31) & 0x7fffffff;
            block_max[it.l0 + 2 * t + half] = exp2f(__int_as_float(kx) * sl2);   // 2^(-inf) = 0: no causal pair, or a rejected entry
          }
          sticky_fail |= fail;
          ja = na; jb = nb2;
        }
      }
    } else
    for (uint32_t n = 0;; ++n) {
      tr.sample(0);
      int64_t w;
      const bool more = next_item(s, n, w);
      // (with a counter the answer comes from a wait, which can be lost: the group leaves together or not at all)
      const bool stop = dyn ? named_bar_or(bar_vote, kGroupThreads, !more) : !more;
      if (gt == 0) release_item(s, n);                      // (every thread of the group has read the slot)
      if (stop) break;
      const Item it = decode_item<kChunk>(m, row_ptr, w);
      const int64_t tok0 = (int64_t)it.s0 + (int64_t)it.i * kBlock + (kChunk ? it.dq : 0);   // first row of the item in q / o / lse
      if (it.ntiles == 0) {                                 // no visible key: o = 0, lse = -inf
        for (int idx = gt; idx < 64 * 16; idx += kGroupThreads) {
          const int qrow = idx >> 4, chunk = idx & 15;
          if (qrow < it.q_valid)
            *reinterpret_cast<uint4*>(o + ((tok0 + qrow) * m.num_q_heads + it.h) * kHeadDim + chunk * 8) = make_uint4(0u, 0u, 0u, 0u);
        }
        if (lse != nullptr && gt < it.q_valid)
          lse[(int64_t)it.h * (kChunk ? m.total_q_tokens : m.total_tokens) + tok0 + gt] = -CUDART_INF_F;
        continue;
      }
      float l_part[64];
#pragma unroll
      for (int c = 0; c < 64; ++c) l_part[c] = 0.f;
      const bool ragged_q = it.q_valid < kBlock;

      int nja = list_block(it, col_idx, 0), njb = list_block(it, col_idx, 1);
      tr.ev(29, 0);
      bool s_seen = false;                                  // S_FULL of the coming tile was already seen complete
      for (int t = 0; t < it.ntiles; ++t, ++cnt) {
        const uint32_t sbuf = cnt & 1u;
        if constexpr (kTrace) { seg_last = clock64(); ++seg_n; }
        bool fail = false;
        if (!s_seen) fail = !mbar_wait(sh, bb + S_FULL + (int)sbuf, (cnt >> 1) & 1u, status);
        SEG(0);
        tc_fence_after();
        const int ja = nja, jb = njb;
        // the next tile's list entries: the loads are issued here and looked at after the pass
        const int raw_a = list_fetch(it, col_idx, 2 * t + 2), raw_b = list_fetch(it, col_idx, 2 * t + 3);
        const int my_j = r < 64 ? ja : jb;
        const bool row_live = my_j >= 0;                 // absent / rejected blocks contribute nothing
        const bool diag = my_j == it.i;
        const bool masked = !row_live || diag || ragged_q;   // uniform per warp (a warp lies in one block half)
        const uint32_t s_addr = tmem + lane_addr + col_s(s, sbuf);
        uint32_t pk[32];
        // First tile of an item: the references are still those of another item.  Column c takes the score of the
        // tile's first key (visible to every query of the block: it is the first key of a block not later than the
        // query block) plus kFirstShift as its reference: no reduction over the keys.  A reference taken from a key of
        // the column itself can never be too high (what it would flush to zero is negligible next to that key), and
        // if it is too low the pass below says so and the group rebases on exact maxima.
        bool have_ref = t >= 1;
        if (t == 0 && ja >= 0) {
          if (!fail && it.ntiles > 1) fail = !mbar_wait(sh, bb + S_FULL + (int)(sbuf ^ 1u), ((cnt + 1) >> 1) & 1u, status);
          tc_fence_after();
          if (!fail && gw == 0) {                         // (the TMEM load is a warp-wide instruction; lane 0 holds key row 0)
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
              uint32_t sv[16];
              tc_ld16(s_addr + ch * 16, sv);
              tc_wait_ld(sv);
              if (lane == 0) {
#pragma unroll
                for (int e = 0; e < 16; e += 4)
                  *reinterpret_cast<uint4*>(&lsum[ch * 16 + e]) = make_uint4(sv[e], sv[e + 1], sv[e + 2], sv[e + 3]);
              }
            }
          }
          tc_fence_before();
          if (named_bar_or(bar_vote, kGroupThreads, fail)) { ok = false; break; }
          if (gt < 64) {
            const float old = 0.f;                       // the first two S^T tiles of an item hold the raw scores
            float nr = bf16_ceil(lsum[gt] + kFirstShift / sl2);
            if (gt >= it.q_valid || !(fabsf(nr) < 3.0e38f)) nr = old;   // not a column of this block / not a finite score
            const float d = old - nr;
            rcur[gt] = nr;
            qext[gt * 8] = (uint16_t)((__float_as_uint(nr) >> 16) ^ 0x8000u);
            const uint32_t hi = __float_as_uint(d) & 0xffff0000u;
            const float r1 = d - __uint_as_float(hi);
            const uint32_t mid = __float_as_uint(r1) & 0xffff0000u;
            const uint32_t lo = __float_as_uint(r1 - __uint_as_float(mid)) & 0xffff0000u;
            *reinterpret_cast<uint2*>(qfix + gt * 8) = make_uint2((hi >> 16) | mid, lo >> 16);
            fence_async_smem();
          }
          named_bar_sync(bar_sync, kGroupThreads);
          if (gt == 0) {
            tc_fence_after();
            tc_mma(tmem + col_s(s, sbuf), ones_d, qfix_d, kIdescS, 1u);
            if (it.ntiles > 1) tc_mma(tmem + col_s(s, sbuf ^ 1u), ones_d, qfix_d, kIdescS, 1u);
            tc_commit(sh.bar(bb + FIXED));
          }
          if (named_bar_or(bar_vote, kGroupThreads, !mbar_wait(sh, bb + FIXED, nfix & 1u, status))) { ok = false; break; }
          ++nfix;
          tc_fence_after();
          have_ref = true;
        }
        // without references (the first key of the first tile is not a valid entry) the tile goes straight to the rebase
        uint32_t over = 0x40004000u;
        bool pv_seen = t == 0;                           // the P V of the previous tile has finished: the P^T buffer is free, O^T at rest
        if (!fail && have_ref)
          over = masked ? tile_pass<true, false>(s_addr, sl2, row_live, diag, key_local, it.q_valid, l_part, pk)
                        : tile_pass<false, false>(s_addr, sl2, row_live, diag, key_local, it.q_valid, l_part, pk,
                                                  sh.bar(bb + PV_DONE), (cnt - 1) & 1u, t >= 1 ? &pv_seen : nullptr);
        SEG(1);
        nja = list_check(it, 2 * t + 2, raw_a); njb = list_check(it, 2 * t + 3, raw_b);
        SEG(2);
        if (!fail && !pv_seen) fail = !mbar_wait(sh, bb + PV_DONE, (cnt - 1) & 1u, status);
        SEG(3);
        // P^T is stored at once; the vote on the tile (does any entry reach 2^(kRefShift + 1) times its reference
        // maximum, or has a wait been lost?) comes after the stores, where the group has to meet anyway, and the
        // issuer is told only after it
        auto store_p = [&]() {
          const uint32_t prow = p_base + (uint32_t)r * 128u;
#pragma unroll
          for (int ck = 0; ck < 8; ++ck) {
            const uint32_t a = prow + (uint32_t)((ck ^ (r & 7)) << 4);
            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(pk[ck * 4]), "r"(pk[ck * 4 + 1]),
                         "r"(pk[ck * 4 + 2]), "r"(pk[ck * 4 + 3]) : "memory");
          }
        };
        store_p();
        SEG(6);
        // the next tile's S^T: asked now, looked at when the next tile starts
        s_seen = t + 1 < it.ntiles && mbar_test(sh.bar(bb + S_FULL + (int)(sbuf ^ 1u)), ((cnt + 1) >> 1) & 1u);
        tc_fence_before();
        SEG(15);
        // the vote comes before the proxy fence: the stores drain (behind the MMAs' operand reads) while the group meets
        const bool slow = named_bar_or(bar_vote, kGroupThreads, fail || (over & 0x40004000u) != 0u);
        SEG(4);
        if (slow) {
          // the -R row may only change when the S^T of the next tile, issued with the old row, has been computed
          if (!fail && t + 1 < it.ntiles) fail = !mbar_wait(sh, bb + S_FULL + (int)(sbuf ^ 1u), ((cnt + 1) >> 1) & 1u, status);
          tc_fence_after();
          if (named_bar_or(bar_vote, kGroupThreads, fail)) { ok = false; break; }
          SEG(8);
          if constexpr (kTrace) ++nreb;
          // ---- rebase: take this tile's contribution out of the row sums again, find the exact column maxima, move
          // the references, rescale the row sums and O^T, and recompute the tile
          if (have_ref) {
            if (masked) tile_pass<true, true>(s_addr, sl2, row_live, diag, key_local, it.q_valid, l_part, pk);
            else tile_pass<false, true>(s_addr, sl2, row_live, diag, key_local, it.q_valid, l_part, pk);
          }
          // column maxima of the accumulator (s - R of the buffer): over the lanes of each warp by shuffles (16 columns
          // at a time: lane pair l, l ^ 1 ends with column l >> 1 of the chunk), over the four warps through shared memory
#pragma unroll 2
          for (int ch = 0; ch < 4; ++ch) {
            uint32_t sv[16];
            tc_ld16(s_addr + ch * 16, sv);
            tc_wait_ld(sv);
            SEG(9);
            float xv[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              const int c = ch * 16 + e;
              float x = __uint_as_float(sv[e]);
              if (!row_live || (diag && key_local > c)) x = -CUDART_INF_F;
              xv[e] = x;
            }
            const float cm = warp_colmax16(xv, lane);
            if ((lane & 1) == 0) lsum[gw * 64 + ch * 16 + (lane >> 1)] = cm;
            SEG(10);
          }
          tc_fence_before();                             // this thread's reads of the S^T buffer are done
          named_bar_sync(bar_sync, kGroupThreads);
          if (gt < 64) {
            const float old = have_ref ? rcur[gt] : 0.f;   // (an item's first tiles hold the raw scores)
            // largest raw score of the column in this tile
            const float cm = fmaxf(fmaxf(lsum[gt], lsum[64 + gt]), fmaxf(lsum[128 + gt], lsum[192 + gt])) + old;
            float nr;
            if (!have_ref) nr = cm == -CUDART_INF_F ? kNoRef : bf16_ceil(cm + shift_raw);
            else nr = cm == -CUDART_INF_F ? old : fmaxf(old, bf16_ceil(cm + shift_raw));
            // a query column past the end of a ragged block holds whatever tokens follow in the packed tensor; the
            // masked pass drops it, and it never moves a reference (results must not depend on the neighbours in the batch)
            if (gt >= it.q_valid) nr = old;
            const float d = old - nr;
            alpha[gt] = have_ref ? exp2f(d * sl2) : 0.f;
            rcur[gt] = nr;
            qext[gt * 8] = (uint16_t)((__float_as_uint(nr) >> 16) ^ 0x8000u);   // -R[c] as bf16, column 0 of row c
            // d = R_old - R_new in three bf16 terms (truncations, so every remainder is exact), columns 0..2 of row c
            const uint32_t hi = __float_as_uint(d) & 0xffff0000u;
            const float r1 = d - __uint_as_float(hi);
            const uint32_t mid = __float_as_uint(r1) & 0xffff0000u;
            const uint32_t lo = __float_as_uint(r1 - __uint_as_float(mid)) & 0xffff0000u;
            *reinterpret_cast<uint2*>(qfix + gt * 8) = make_uint2((hi >> 16) | mid, lo >> 16);
            fence_async_smem();
          }
          named_bar_sync(bar_sync, kGroupThreads);
          SEG(11);
          // the S^T tiles computed with the old row (this one and the next) get ones x (R_old - R_new) added in place
          if (gt == 0) {
            tc_fence_after();
            tc_mma(tmem + col_s(s, sbuf), ones_d, qfix_d, kIdescS, 1u);
            if (t + 1 < it.ntiles) tc_mma(tmem + col_s(s, sbuf ^ 1u), ones_d, qfix_d, kIdescS, 1u);
            tc_commit(sh.bar(bb + FIXED));
          }
          if (have_ref) {                                // row sums (and, after the first tile, O^T) accumulated so far
            // a reference that moved by more than 2^30 makes everything accumulated so far negligible (and the value
            // taken out above may not have been finite): start the column afresh
#pragma unroll
            for (int c = 0; c < 64; c += 4) {
              const float4 a = *reinterpret_cast<const float4*>(&alpha[c]);
              l_part[c] = a.x < 9.3e-10f ? 0.f : l_part[c] * a.x;
              l_part[c + 1] = a.y < 9.3e-10f ? 0.f : l_part[c + 1] * a.y;
              l_part[c + 2] = a.z < 9.3e-10f ? 0.f : l_part[c + 2] * a.z;
              l_part[c + 3] = a.w < 9.3e-10f ? 0.f : l_part[c + 3] * a.w;
            }
#pragma unroll 1
            for (int ch = 0; ch < (t >= 1 ? 4 : 0); ++ch) {
              uint32_t ov[16];
              tc_ld16(o_addr + ch * 16, ov);
              tc_wait_ld(ov);
#pragma unroll
              for (int e = 0; e < 16; e += 4) {
                const float4 a = *reinterpret_cast<const float4*>(&alpha[ch * 16 + e]);
                ov[e] = __float_as_uint(__uint_as_float(ov[e]) * a.x);
                ov[e + 1] = __float_as_uint(__uint_as_float(ov[e + 1]) * a.y);
                ov[e + 2] = __float_as_uint(__uint_as_float(ov[e + 2]) * a.z);
                ov[e + 3] = __float_as_uint(__uint_as_float(ov[e + 3]) * a.w);
              }
              tc_st16(o_addr + ch * 16, ov);
            }
            tc_wait_st();
          }
          SEG(12);
          if (named_bar_or(bar_vote, kGroupThreads, !mbar_wait(sh, bb + FIXED, nfix & 1u, status))) { ok = false; break; }
          SEG(13);
          ++nfix;
          tc_fence_after();
          if (masked) tile_pass<true, false>(s_addr, sl2, row_live, diag, key_local, it.q_valid, l_part, pk);
          else tile_pass<false, false>(s_addr, sl2, row_live, diag, key_local, it.q_valid, l_part, pk);
          store_p();
          fence_async_smem();
          tc_fence_before();
          named_bar_sync(bar_sync, kGroupThreads);
          s_seen = false;
          SEG(14);
        }
        SEG(5);
        // a warp whose stores are visible to the MMA arrives; four arrivals hand P^T over and the S^T buffer back
        if (!slow) fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(sh.bar(bb + P_FULL));
        SEG(7);
      }
      if (!ok) break;

      // ------------------------------------------------------------------------------------------ epilogue
      tr.sample(0); tr.ev(30, 0);
      const bool efail = !mbar_wait(sh, bb + PV_DONE, (cnt - 1) & 1u, status);   // the last P V of the item
      tc_fence_after();
      {
        float s0, s1; int base;
        warp_colsum(l_part, lane, s0, s1, base);
        lsum[gw * 64 + base] = s0;
        lsum[gw * 64 + base + 1] = s1;
      }
      if (named_bar_or(bar_vote, kGroupThreads, efail)) { ok = false; break; }
      if (gt < 64) {
        const float l = (lsum[gt] + lsum[64 + gt]) + (lsum[128 + gt] + lsum[192 + gt]);
        alpha[gt] = l > 0.f ? 1.f / l : 0.f;
        if (lse != nullptr && gt < it.q_valid)
          lse[(int64_t)it.h * (kChunk ? m.total_q_tokens : m.total_tokens) + tok0 + gt] =
              l > 0.f ? (rcur[gt] * sl2 + log2f(l)) * 0.6931471805599453f : -CUDART_INF_F;
      }
      named_bar_sync(bar_sync, kGroupThreads);
      // O^T row r (one d of all 64 queries) -> staging in the stream's P^T buffer as [32 query pairs][128 d] words, a
      // word holding the two queries of a pair for one d: every store is a full word per lane, a warp's stores one
      // 128-byte line (two-byte stores of single elements cost two wavefronts each and twice as many instructions)
      {
        uint32_t* stage = reinterpret_cast<uint32_t*>(p_gen);
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          uint32_t ov[16];
          tc_ld16(o_addr + ch * 16, ov);
          tc_wait_ld(ov);
#pragma unroll
          for (int e = 0; e < 16; e += 4) {
            const float4 f = *reinterpret_cast<const float4*>(&alpha[ch * 16 + e]);
            stage[((ch * 16 + e) >> 1) * 128 + r] = pack_bf16(__uint_as_float(ov[e]) * f.x, __uint_as_float(ov[e + 1]) * f.y);
            stage[((ch * 16 + e + 2) >> 1) * 128 + r] = pack_bf16(__uint_as_float(ov[e + 2]) * f.z, __uint_as_float(ov[e + 3]) * f.w);
          }
        }
      }
      tc_fence_before();
      named_bar_sync(bar_sync, kGroupThreads);   // O^T has been read (the next item's first P V waits for this group's P^T anyway)
      {
        // a thread takes eight d of a query pair: eight words in, the low halves are query 2p, the high halves query 2p + 1
        const uint4* stage4 = reinterpret_cast<const uint4*>(p_gen);
        for (int idx = gt; idx < 32 * 16; idx += kGroupThreads) {
          const int pair = idx >> 4, chunk = idx & 15;
          const uint4 w0 = stage4[pair * 32 + chunk * 2], w1 = stage4[pair * 32 + chunk * 2 + 1];
          const uint4 lo = make_uint4(__byte_perm(w0.x, w0.y, 0x5410), __byte_perm(w0.z, w0.w, 0x5410),
                                      __byte_perm(w1.x, w1.y, 0x5410), __byte_perm(w1.z, w1.w, 0x5410));
          const uint4 hi = make_uint4(__byte_perm(w0.x, w0.y, 0x7632), __byte_perm(w0.z, w0.w, 0x7632),
                                      __byte_perm(w1.x, w1.y, 0x7632), __byte_perm(w1.z, w1.w, 0x7632));
          uint16_t* dst = o + ((tok0 + 2 * pair) * m.num_q_heads + it.h) * kHeadDim + chunk * 8;
          if (2 * pair < it.q_valid) *reinterpret_cast<uint4*>(dst) = lo;
          if (2 * pair + 1 < it.q_valid) *reinterpret_cast<uint4*>(dst + (size_t)m.num_q_heads * kHeadDim) = hi;
        }
      }
      named_bar_sync(bar_sync, kGroupThreads);   // staging is free again before the next P^T
      tr.ev(31, 0);
    }
    if constexpr (kTrace) if (tr.p != nullptr)
      for (int k = 0; k < 16; ++k) { tr.acc[2 * (32 + k)] = (unsigned long long)seg[k]; tr.acc[2 * (32 + k) + 1] = (k >= 8 && k < 15) ? nreb : seg_n; }
    tr.flush();
#undef SEG
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

}  // namespace tc

seer_status init_attn_tc(seer_ctx* ctx) {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess)
    return SEER_ERR_CUDA;
  ctx->tmap_encode = fn;
  cudaError_t e = cudaFuncSetAttribute(tc::attn_tc_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::kSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(tc::attn_tc_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::kSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(tc::attn_tc_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::kSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(tc::attn_tc_kernel<false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::kSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(tc::attn_tc_kernel<false, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::kSmemBytes);
  return e == cudaSuccess ? SEER_OK : SEER_ERR_CUDA;
}

int launch_attn_tc(seer_ctx* ctx, const SeqMeta& m, const void* q, const void* k, const void* v,
                    const int32_t* row_ptr, const int32_t* col_idx, void* o, float* lse, int* work_counter,
                    cudaStream_t stream) {
  if (m.rows == 0) return 0;
  // the counter the streams draw their work items from (in the caller's workspace; without one the deal is static)
  if (work_counter != nullptr && cudaMemsetAsync(work_counter, 0, sizeof(int), stream) != cudaSuccess) return -(int)cudaErrorInvalidValue;
  // the input pointers must be 16-byte aligned for TMA
  if ((((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)o) & 15) != 0) return -(int)cudaErrorMisalignedAddress;
  CUtensorMap mq, mk, mv;
  if (!tc::make_map(ctx, &mq, q, m.total_q_tokens, m.num_q_heads) || !tc::make_map(ctx, &mk, k, m.total_tokens, m.num_kv_heads) ||
      !tc::make_map(ctx, &mv, v, m.total_tokens, m.num_kv_heads))
    return -(int)cudaErrorInvalidValue;
  const unsigned grid = (unsigned)min((int64_t)ctx->num_sms, (m.rows + 1) / 2);
  unsigned long long* tb = (unsigned long long*)ctx->trace;
  if (m.chunked)               // chunked prefill (never instrumented)
    tc::attn_tc_kernel<false, true><<<grid, tc::kThreads, tc::kSmemBytes, stream>>>(mq, mk, mv, m, row_ptr, col_idx, (uint16_t*)o, lse, ctx->d_status, tb, nullptr, work_counter);
  else if (tb != nullptr)      // the instrumented instantiation
    tc::attn_tc_kernel<true, false><<<grid, tc::kThreads, tc::kSmemBytes, stream>>>(mq, mk, mv, m, row_ptr, col_idx, (uint16_t*)o, lse, ctx->d_status, tb, nullptr, work_counter);
  else
    tc::attn_tc_kernel<false, false><<<grid, tc::kThreads, tc::kSmemBytes, stream>>>(mq, mk, mv, m, row_ptr, col_idx, (uint16_t*)o, lse, ctx->d_status, tb, nullptr, work_counter);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 1 : -(int)e;
}

// Max-pooled attention map on the listed blocks (Sec. 3.2, Eq. 2): the attention pipeline without V.
int launch_block_max_tc(seer_ctx* ctx, const SeqMeta& m, const void* q, const void* k, const int32_t* row_ptr,
                        const int32_t* col_idx, const float* lse, float* out, cudaStream_t stream) {
  if (m.rows == 0) return 0;
  if ((((uintptr_t)q | (uintptr_t)k) & 15) != 0) return -(int)cudaErrorMisalignedAddress;
  CUtensorMap mq, mk;
  if (!tc::make_map(ctx, &mq, q, m.total_q_tokens, m.num_q_heads) || !tc::make_map(ctx, &mk, k, m.total_tokens, m.num_kv_heads))
    return -(int)cudaErrorInvalidValue;
  const unsigned grid = (unsigned)min((int64_t)ctx->num_sms, (m.rows + 1) / 2);
  float* lse_in = const_cast<float*>(lse);   // read only in this mode
  if (m.chunked)
    tc::attn_tc_kernel<false, true, true><<<grid, tc::kThreads, tc::kSmemBytes, stream>>>(mq, mk, mk, m, row_ptr, col_idx, nullptr, lse_in, ctx->d_status, nullptr, out);
  else
    tc::attn_tc_kernel<false, false, true><<<grid, tc::kThreads, tc::kSmemBytes, stream>>>(mq, mk, mk, m, row_ptr, col_idx, nullptr, lse_in, ctx->d_status, nullptr, out);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 1 : -(int)e;
}

}  // namespace seer
