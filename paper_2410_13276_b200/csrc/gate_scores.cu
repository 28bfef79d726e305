// AttnGate, second kernel (Sec. 3.1, Eq. 1): logits = gq gk^T / sqrt(dg) over the causal blocks, row softmax -> scores.
//
// The logits need fp32-grade products (bf16 or tf32 inputs would not hold the 1e-3 relative bound on softmax outputs
// when logits reach tens), so gq and gk arrive as three bf16 planes each, x = hi + mid + lo, and the product is the six
// terms hi*lo + lo*hi + mid*mid (small) and hi*mid + mid*hi + hi*hi (large) (what is dropped is below 2^-24 of the
// product), accumulated in fp32 TMEM accumulators by tcgen05.mma: 6 x 8 K-steps of M = 128, N = 64, K = 16 per tile.
//
// One CTA = 128 consecutive block rows of one head (rows of the packed batch, whatever sequences they belong to), walked
// over the causal column tiles of 64 blocks twice: the first sweep keeps the running maximum and sum of every row (a
// thread owns a row: TMEM lane = row, so neither needs a shuffle), the second recomputes the logits and writes
// exp(x - m) / l: every score is written once and never read back.  The finished tile goes through shared memory so
// that a warp writes whole 256-byte row segments (a thread storing its own row scatters 16-byte pieces over 32 rows
// per instruction: measured three times slower).
//
// Roles (320 threads): warps 0-3 own the rows (epilogue), warps 6-9 copy the operand tiles (cp.async into the 128-byte
// swizzled K-major layout the MMA descriptors expect); one thread of warp 4 and one of warp 5 issue the MMAs, one the
// three small terms, the other the three large ones, each into its own accumulator (one thread starts an MMA about every 100 clocks, two
// keep the pipe at the 48 clocks an N = 64 instruction occupies it); the rows add the two.  Two accumulator pairs and
// two B buffers: the MMAs of tile n + 1 run while the rows work on tile n.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "attn_tc_common.cuh"
#include "seer_internal.cuh"

namespace seer {

using namespace tcc;

namespace gs {
constexpr int kRows = 128;                         // score rows per CTA
constexpr int kCols = kScoreTile;                  // columns per tile (64)
constexpr int kThreads = 320;
constexpr uint32_t kAPlane = kRows * kGateDim * 2;   // 32 KB: one plane of the 128 x 128 A tile, [2 k halves][128 rows][128 B]
constexpr uint32_t kBPlane = kCols * kGateDim * 2;   // 16 KB: one plane of a 64 x 128 B tile
constexpr uint32_t kOffA = 0;
constexpr uint32_t kOffB = 3 * kAPlane;              // two buffers of three planes
constexpr uint32_t kBBuf = 3 * kBPlane;
constexpr uint32_t kOffStage = kOffB + 2 * kBBuf;    // [128 rows][64 columns] fp32, 16-byte chunks XOR (row % 16): 32 KB
constexpr uint32_t kOffMeta = kOffStage + kRows * kCols * 4;   // per row: element offset of column 0 (int64), first and last causal block
constexpr uint32_t kOffBar = kOffMeta + kRows * 16;  // mbarriers: ACC_FULL[2], ACC_EMPTY[2], B_FULL[2]
constexpr uint32_t kOffMisc = kOffBar + 64;          // tmem base, abort flag
constexpr uint32_t kSmemBytes = kOffMisc + 64;
static_assert(kSmemBytes <= 232448, "shared memory budget of one CTA");
enum Bar { ACC_FULL = 0, ACC_EMPTY = 2, B_FULL = 4 };
constexpr int kLoaders = 128;                       // threads of the four copying warps
constexpr uint32_t kTmemCols = 256;                  // two buffers x (small terms, large terms) x 64 columns
constexpr uint32_t kIdesc = make_idesc(false, false, kCols);
constexpr uint32_t kWaitSpins = 1u << 24;          // a wait that lasts this many polls (seconds) is declared lost

// Bounded wait that never changes the control flow: after the limit the error is recorded and the wait counts as
// satisfied, so every role still reaches its barriers and the CTA ends normally (with a wrong result and a status).
__device__ __forceinline__ void wait_bar(uint32_t bar, uint32_t parity, uint32_t abort_addr, int* status) {
  for (uint32_t it = 0; it < kWaitSpins; ++it)
    if (mbar_try(bar, parity)) return;
  st_shared_u32(abort_addr, 1u);
  if (status != nullptr) atomicCAS(status, 0, (int)SEER_ERR_TIMEOUT);
}

// Rows r0 .. r0 + rows - 1 of the three planes of src ([blocks][128] bf16 each, `plane` elements apart) into the
// swizzled K-major tile layout: k half (64 elements = 128 bytes per row) -> 8-row group (1024 bytes) -> row -> 16-byte
// chunk XOR (row % 8).  Rows at or beyond rows_valid are zero-filled.
template <int ROWS>
__device__ __forceinline__ void load_planes(uint32_t dst, uint32_t plane_bytes, const uint16_t* __restrict__ src, size_t plane,
                                            int r0, int rows_valid, int tid, int nthreads) {
  for (int idx = tid; idx < 3 * ROWS * 16; idx += nthreads) {
    const int pl = idx / (ROWS * 16), rem = idx - pl * (ROWS * 16);
    const int row = rem >> 4, chunk = rem & 15;
    const bool ok = row < rows_valid;
    const uint16_t* g = src + (size_t)pl * plane + (size_t)(r0 + (ok ? row : 0)) * kGateDim + chunk * 8;
    const uint32_t at = dst + (uint32_t)pl * plane_bytes + (uint32_t)(chunk >> 3) * (ROWS * 128u) + (uint32_t)(row >> 3) * 1024u +
                        (uint32_t)(row & 7) * 128u + (uint32_t)(((chunk & 7) ^ (row & 7)) << 4);
    const int sz = ok ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(at), "l"(g), "r"(sz) : "memory");
  }
}
}  // namespace gs

// grid.x = row tiles * band.heads (head fastest; row tiles are visited from the last rows to the first).  Row r of a
// tile is query block i_r of sequence b_r; its causal columns are that sequence's blocks 0 .. i_r, i.e. the blocks
// seq_start_r .. r of the batch.  The CTA walks the column tiles from the sequence start of its first row to its last
// row; entries of other sequences are masked.  The whole problem is the band (0, total_blocks, 0, Hq, 0).  Scores are
// written at their offset in the full matrix minus band.score_base.
__global__ void __launch_bounds__(gs::kThreads, 1)
gate_scores_kernel(SeqMeta m, ScoreBand band, const uint16_t* __restrict__ gq, const uint16_t* __restrict__ gk,
                   float* __restrict__ scores, int* __restrict__ status) {
  using namespace gs;
  extern __shared__ __align__(1024) unsigned char gs_raw[];   // (the swizzled tiles need 1024-byte alignment; no slack is left to round up)
  const uint32_t base = (uint32_t)__cvta_generic_to_shared(gs_raw);
  unsigned char* smem = gs_raw;
  if ((base & 1023u) != 0u) {
    if (threadIdx.x == 0 && status != nullptr) atomicCAS(status, 0, (int)SEER_ERR_CUDA);
    return;
  }
  const uint32_t bar0 = base + kOffBar, abort_addr = base + kOffMisc + 4;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + kOffMisc);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const int row_tiles = (band.blk_hi - band.blk_lo + kRows - 1) / kRows;
  const int tile = row_tiles - 1 - (int)(blockIdx.x / band.heads);
  const int h = band.head_lo + (int)(blockIdx.x % band.heads);
  const int g = h / m.group;
  const int r0 = band.blk_lo + tile * kRows;                              // first block row of the tile
  const int rows_valid = min(kRows, band.blk_hi - r0);

  // this thread's row (threads 0..127); the helpers only need the tile's column range
  int my_start = 0, my_last = -1;
  long long my_off = 0;
  if (threadIdx.x < kRows && (int)threadIdx.x < rows_valid) {
    const int gb = r0 + (int)threadIdx.x;
    const int b = find_sequence(m.blk_off, m.batch, gb);
    const int nb = m.blk_off[b + 1] - m.blk_off[b];
    const int i = gb - m.blk_off[b];
    my_start = m.blk_off[b];
    my_off = m.score_off[b] + ((long long)h * nb + i) * nb - band.score_base;
    if (!(m.chunked && i < m.qoff[b])) my_last = gb;                      // chunked prefill: rows before the chunk are skipped
  }
  if (threadIdx.x < kRows) {
    *reinterpret_cast<long long*>(smem + kOffMeta + threadIdx.x * 16) = my_off - my_start;   // + j = element of column j
    *reinterpret_cast<int2*>(smem + kOffMeta + threadIdx.x * 16 + 8) = make_int2(my_start, my_last);
  }
  if (!__syncthreads_or(my_last >= 0 ? 1 : 0)) return;                    // a tile of query blocks before their chunks
  const int first_col = m.blk_off[find_sequence(m.blk_off, m.batch, r0)];  // rows ascend, so do their sequence starts
  const int last_col = r0 + rows_valid - 1;
  const int ntiles = (last_col - first_col) / kCols + 1;                  // column tiles of one sweep
  const int total = 2 * ntiles;                                           // both sweeps

  if (threadIdx.x == 0) {
    mbar_init(bar0 + 8 * (ACC_FULL + 0), 2); mbar_init(bar0 + 8 * (ACC_FULL + 1), 2);   // one commit per issuing thread
    mbar_init(bar0 + 8 * (ACC_EMPTY + 0), kRows); mbar_init(bar0 + 8 * (ACC_EMPTY + 1), kRows);
    mbar_init(bar0 + 8 * (B_FULL + 0), kLoaders); mbar_init(bar0 + 8 * (B_FULL + 1), kLoaders);
    st_shared_u32(abort_addr, 0u);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(base + kOffMisc), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  const size_t plane_q = (size_t)m.num_q_heads * m.total_blocks * kGateDim;
  const size_t plane_k = (size_t)m.num_kv_heads * m.total_blocks * kGateDim;
  const uint16_t* gq_h = gq + (size_t)h * m.total_blocks * kGateDim;
  const uint16_t* gk_g = gk + (size_t)g * m.total_blocks * kGateDim;

  if (warp >= 6) {
    // ------------------------------------------------------------------------------------------ copies
    const int tid = threadIdx.x - 192;                    // warps 6..9
    load_planes<kRows>(base + kOffA, kAPlane, gq_h, plane_q, r0, rows_valid, tid, kLoaders);
    for (int n = 0; n < total; ++n) {
      const int buf = n & 1;
      const int j0 = first_col + (n % ntiles) * kCols;
      // the MMAs of tile n - 2 read this B buffer: their completion is ACC_FULL of that tile
      if (n >= 2) wait_bar(bar0 + 8 * (ACC_FULL + buf), ((n - 2) >> 1) & 1u, abort_addr, status);
      load_planes<kCols>(base + kOffB + (uint32_t)buf * kBBuf, kBPlane, gk_g, plane_k, j0, min(kCols, last_col + 1 - j0), tid, kLoaders);
      asm volatile("cp.async.commit_group;" ::: "memory");
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      fence_async_smem();                                 // the copies (generic proxy) before the MMAs' reads (async proxy)
      mbar_arrive(bar0 + 8 * (B_FULL + buf));
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------------------------------ MMAs
    // (the issuing threads copy nothing: a thread that waits for its own copies between two batches of MMAs leaves
    // the pipe idle for the latency of a copy, which was 40 % of the kernel)
    if (lane == 0) {
      const int part = warp - 4;                          // 0: small terms, 1: large terms
      // (A plane, B plane): small = (hi, lo), (lo, hi), (mid, mid); large = (hi, mid), (mid, hi), (hi, hi)
      const int pa[3] = {0, part ? 1 : 2, part ? 0 : 1}, pb[3] = {part ? 1 : 2, 0, part ? 0 : 1};
      for (int n = 0; n < total; ++n) {
        const int buf = n & 1;
        wait_bar(bar0 + 8 * (B_FULL + buf), (n >> 1) & 1u, abort_addr, status);
        // the rows have taken tile n - 2 out of this accumulator pair
        if (n >= 2) wait_bar(bar0 + 8 * (ACC_EMPTY + buf), ((n - 2) >> 1) & 1u, abort_addr, status);
        tc_fence_after();
        const uint32_t d = tmem + (uint32_t)buf * 2u * kCols + (uint32_t)part * kCols;
        const uint32_t sa = base + kOffA, sb = base + kOffB + (uint32_t)buf * kBBuf;
#pragma unroll
        for (int t = 0; t < 3; ++t)
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint64_t ad = make_desc(sa + (uint32_t)pa[t] * kAPlane + (uint32_t)(kk >> 2) * (kRows * 128u) + (uint32_t)(kk & 3) * 32u, 16, 1024);
            const uint64_t bd = make_desc(sb + (uint32_t)pb[t] * kBPlane + (uint32_t)(kk >> 2) * (kCols * 128u) + (uint32_t)(kk & 3) * 32u, 16, 1024);
            tc_mma(d, ad, bd, kIdesc, (t | kk) != 0 ? 1u : 0u);
          }
        tc_commit(bar0 + 8 * (ACC_FULL + buf));
      }
    }
  } else {
    // ------------------------------------------------------------------------------------------ rows
    // everything in units of log2: x2 = logit * log2(e); m2 the running maximum of x2; p = 2^(x2 - m2) / l
    const float scale2 = rsqrtf((float)kGateDim) * 1.4426950408889634f;
    const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
    float run_m = -CUDART_INF_F, run_l = 0.f, inv_l = 0.f;
    for (int n = 0; n < total; ++n) {
      const int buf = n & 1;
      const int sweep = n / ntiles;
      const int j0 = first_col + (n - sweep * ntiles) * kCols;
      if (n == ntiles) inv_l = run_l > 0.f ? 1.0f / run_l : 0.f;
      wait_bar(bar0 + 8 * (ACC_FULL + buf), (n >> 1) & 1u, abort_addr, status);
      tc_fence_after();
      const uint32_t acc = tmem + lane_addr + (uint32_t)buf * 2u * kCols;
      // columns of this tile that are causal for this row: j in [my_start, my_last]
      const int lo = max(my_start - j0, 0), hi = min(my_last - j0, kCols - 1);   // hi < lo: nothing (also my_last = -1)
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        uint32_t vs[32], vl[32];
        tc_ld32(acc + half * 32, vs);
        tc_ld32(acc + kCols + half * 32, vl);
        tc_wait_ld32(vs);
        tc_wait_ld32(vl);
        const int c0 = half * 32;
        if (hi < c0 || lo > c0 + 31) continue;
        const bool whole = lo <= c0 && hi >= c0 + 31;     // no column of this half is masked
        float x[32];
#pragma unroll
        for (int c = 0; c < 32; ++c) x[c] = (__uint_as_float(vs[c]) + __uint_as_float(vl[c])) * scale2;
        if (sweep == 0) {
          if (!whole) {
#pragma unroll
            for (int c = 0; c < 32; ++c) if (c0 + c < lo || c0 + c > hi) x[c] = -CUDART_INF_F;
          }
          float tmax = x[0];
#pragma unroll
          for (int c = 1; c < 32; ++c) tmax = fmaxf(tmax, x[c]);
          const float nm = fmaxf(run_m, tmax);            // finite: the half holds a causal column
          float sum = 0.f;
#pragma unroll
          for (int c = 0; c < 32; ++c) sum += ex2f(x[c] - nm);   // 2^(-inf) = 0 for the masked columns
          run_l = run_l * ex2f(run_m - nm) + sum;         // 2^(-inf) = 0 on the first contribution
          run_m = nm;
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c) x[c] = ex2f(x[c] - run_m) * inv_l;
          float* srow = reinterpret_cast<float*>(smem + kOffStage) + threadIdx.x * kCols;
#pragma unroll
          for (int c = 0; c < 32; c += 4)
            *reinterpret_cast<float4*>(srow + ((((c0 + c) >> 2) ^ (threadIdx.x & 15)) << 2)) = make_float4(x[c], x[c + 1], x[c + 2], x[c + 3]);
        }
      }
      if (sweep == 1) {
        // the warp's 32 rows, two rows per step: a half-warp takes a row, a lane four consecutive columns of it
        __syncwarp();
#pragma unroll 4
        for (int rr = 0; rr < 32; rr += 2) {
          const int row = warp * 32 + rr + (lane >> 4);
          const long long off = *reinterpret_cast<const long long*>(smem + kOffMeta + row * 16);
          const int2 se = *reinterpret_cast<const int2*>(smem + kOffMeta + row * 16 + 8);
          const int c = 4 * (lane & 15), j = j0 + c;
          const float4 v = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(smem + kOffStage) + row * kCols +
                                                            (((c >> 2) ^ (row & 15)) << 2));
          float* dst = scores + (off + j);
          if (j >= se.x && j + 3 <= se.y && ((off + j) & 3) == 0) *reinterpret_cast<float4*>(dst) = v;
          else {
            if (j >= se.x && j <= se.y) dst[0] = v.x;
            if (j + 1 >= se.x && j + 1 <= se.y) dst[1] = v.y;
            if (j + 2 >= se.x && j + 2 <= se.y) dst[2] = v.z;
            if (j + 3 >= se.x && j + 3 <= se.y) dst[3] = v.w;
          }
        }
        __syncwarp();                                    // the staging rows are free again
      }
      tc_fence_before();
      mbar_arrive(bar0 + 8 * (ACC_EMPTY + buf));
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

int launch_gate_scores(const SeqMeta& m, const ScoreBand& band, const uint16_t* gq, const uint16_t* gk, float* scores,
                       int* status, cudaStream_t stream) {
  const unsigned grid = (unsigned)((band.blk_hi - band.blk_lo + gs::kRows - 1) / gs::kRows) * (unsigned)band.heads;
  if (grid == 0) return 0;
  gate_scores_kernel<<<grid, gs::kThreads, gs::kSmemBytes, stream>>>(m, band, gq, gk, scores, status);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 1 : -(int)e;
}

// Lifts the kernel's shared-memory limit on the current device (no allocation).
bool init_gate_scores() {
  return cudaFuncSetAttribute(gate_scores_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gs::kSmemBytes) == cudaSuccess;
}

}  // namespace seer
