// Binary block mask (Sec. 3.3, Eq. 3 TopK / Eq. 4 threshold) as CSR index lists.
//   count_kernel : one warp per (sequence, head, query-block) row -> number of kept blocks
//   scan_kernel  : exclusive prefix sum of the counts -> row_ptr, nnz, capacity check
//   fill_kernel  : one warp per row repeats the selection and writes the ascending list by ballot compaction
// Selection order in the TopK modes is (score descending, block index ascending): scores become order-preserving
// 32-bit keys, the key of the last kept candidate is found by a radix select over the row held in shared memory (at most
// four 8-bit passes with warp-private histograms; batches with rows too long to stage re-read the scores in every pass), and ties
// at that key are resolved by rank in index order.
#include "seer_internal.cuh"

namespace seer {

constexpr int kMaskWarps = 4;
// Rows are staged in shared memory when the longest row of the batch has at most this many blocks (16 bytes of shared
// memory per block and CTA).  Beyond that the staging buffer would cost more in occupancy than it saves in reads
// (measured: 4096 blocks 4.6 ms staged, 3.1 ms not; 10240 blocks 103 ms against 27 ms), and every pass re-reads the
// scores, which stay in L1 / L2 between the passes of a row.
constexpr int kMaskSmemRowMax = 2048;

struct RowInfo {
  const float* s;   // scores of this row
  int i;            // query block index (row has n = i + 1 causal blocks)
  bool valid;
  bool skip;        // chunked prefill: a query block before the chunk, its list is empty
  int nb;           // blocks of the row's sequence
};

// Rows [row_lo, row_hi) of the CSR structure whose scores sit at (offset in the full matrix - score_base) in `scores`.
struct RowBand {
  int64_t row_lo, row_hi, score_base;
};

__device__ __forceinline__ RowInfo decode_row(const SeqMeta& m, const RowBand& band, const float* __restrict__ scores, int64_t r) {
  RowInfo ri;
  ri.valid = r < band.row_hi;
  ri.skip = false;
  ri.nb = 0;
  if (!ri.valid) { ri.s = nullptr; ri.i = 0; return ri; }
  // (the host refuses shapes with 2^31 rows or more: 32-bit divisions)
  const int b = find_sequence(m.blk_off, m.batch, (int)((uint32_t)r / (uint32_t)m.num_q_heads));
  const int nb = m.blk_off[b + 1] - m.blk_off[b];
  const uint32_t local = (uint32_t)r - (uint32_t)m.num_q_heads * (uint32_t)m.blk_off[b];
  const int h = (int)(local / (uint32_t)nb);
  ri.i = (int)(local - (uint32_t)h * (uint32_t)nb);
  ri.s = scores + (m.score_off[b] + ((int64_t)h * nb + ri.i) * nb - band.score_base);
  ri.skip = m.chunked && ri.i < m.qoff[b];
  ri.nb = nb;
  return ri;
}

// Order-preserving map fp32 -> uint32 (larger score = larger key); -0 equals +0; NaN -> 0 (never a candidate).
__device__ __forceinline__ uint32_t score_key(float s) {
  uint32_t u = __float_as_uint(s);
  if ((u & 0x7fffffffu) > 0x7f800000u) return 0u;
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ bool is_forced(int j, int i, uint32_t flags) {
  return ((flags & SEER_FORCE_DIAG) && j == i) || ((flags & SEER_FORCE_SINK) && j == 0);
}

__device__ __forceinline__ int num_forced(int i, uint32_t flags) {
  int nf = (flags & SEER_FORCE_DIAG) ? 1 : 0;
  if ((flags & SEER_FORCE_SINK) && !((flags & SEER_FORCE_DIAG) && i == 0)) nf += 1;
  return nf;
}

__device__ __forceinline__ int keep_count(int n, const seer_mask_params& p) {
  if (p.mode == SEER_TOPK_RATIO) {
    long long k = ((long long)p.keep_num * n + p.keep_den - 1) / p.keep_den;
    if (k < 1) k = 1;
    if (k > n) k = n;
    return (int)k;
  }
  int k = p.k < 0 ? 0 : p.k;
  return k < n ? k : n;
}

__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__global__ void __launch_bounds__(kMaskWarps * 32)
count_kernel(SeqMeta m, RowBand band, const float* __restrict__ scores, seer_mask_params p, int32_t* __restrict__ row_ptr) {
  const int lane = threadIdx.x & 31;
  const int64_t r = band.row_lo + (int64_t)blockIdx.x * kMaskWarps + (threadIdx.x >> 5);
  const RowInfo ri = decode_row(m, band, scores, r);
  if (!ri.valid) return;
  const int n = ri.i + 1;
  int c = 0;
  if (ri.skip) {
    // nothing listed
  } else if (ri.i >= ri.nb - p.dense_tail_blocks) {
    c = n;                                             // a dense row at the end of the sequence
  } else if (p.mode == SEER_THRESHOLD) {
    int head = 0;
    if ((reinterpret_cast<uintptr_t>(ri.s) & 15) == 0) {       // four scores per lane and load where the row is aligned
      head = n & ~3;
      for (int j = lane * 4; j < head; j += 128) {
        const float4 v = *reinterpret_cast<const float4*>(ri.s + j);
        c += (is_forced(j, ri.i, p.flags) || v.x > p.threshold) ? 1 : 0;
        c += (is_forced(j + 1, ri.i, p.flags) || v.y > p.threshold) ? 1 : 0;
        c += (is_forced(j + 2, ri.i, p.flags) || v.z > p.threshold) ? 1 : 0;
        c += (is_forced(j + 3, ri.i, p.flags) || v.w > p.threshold) ? 1 : 0;
      }
    }
    for (int j = head + lane; j < n; j += 32) c += (is_forced(j, ri.i, p.flags) || ri.s[j] > p.threshold) ? 1 : 0;
    c = warp_sum(c);
  } else {
    int head = 0;
    if ((reinterpret_cast<uintptr_t>(ri.s) & 15) == 0) {
      head = n & ~3;
      for (int j = lane * 4; j < head; j += 128) {
        const float4 v = *reinterpret_cast<const float4*>(ri.s + j);
        c += (!is_forced(j, ri.i, p.flags) && score_key(v.x) != 0u) ? 1 : 0;
        c += (!is_forced(j + 1, ri.i, p.flags) && score_key(v.y) != 0u) ? 1 : 0;
        c += (!is_forced(j + 2, ri.i, p.flags) && score_key(v.z) != 0u) ? 1 : 0;
        c += (!is_forced(j + 3, ri.i, p.flags) && score_key(v.w) != 0u) ? 1 : 0;
      }
    }
    for (int j = head + lane; j < n; j += 32) c += (!is_forced(j, ri.i, p.flags) && score_key(ri.s[j]) != 0u) ? 1 : 0;
    const int ncand = warp_sum(c);
    const int nf = num_forced(ri.i, p.flags);
    const int take = max(keep_count(n, p) - nf, 0);
    c = nf + min(take, ncand);
  }
  if (lane == 0) row_ptr[r + 1] = c;
}

// Single CTA: in-place inclusive scan of row_ptr[1..rows].  `first`: row_ptr[0] = 0; otherwise the scan continues from
// row_ptr[0], the last entry of the rows scanned before.  Tiles of 4096 counts go through shared memory (coalesced loads
// and stores), four consecutive counts per thread, warp shuffles inside a warp, one carry per tile.
__global__ void __launch_bounds__(1024)
scan_kernel(int64_t rows, int32_t* __restrict__ row_ptr, int first, int64_t col_capacity, int64_t* __restrict__ nnz_out,
            int* __restrict__ status) {
  __shared__ int32_t tile[4096];
  __shared__ long long warp_tot[32];
  __shared__ long long carry_s;
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  long long carry = first ? 0 : row_ptr[0];
  for (int64_t base = 0; base < rows; base += 4096) {
    const int n = (int)min((int64_t)4096, rows - base);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int idx = t + k * 1024;
      tile[idx] = idx < n ? row_ptr[base + idx + 1] : 0;
    }
    __syncthreads();
    long long v[4];
    v[0] = tile[4 * t];
    v[1] = v[0] + tile[4 * t + 1];
    v[2] = v[1] + tile[4 * t + 2];
    v[3] = v[2] + tile[4 * t + 3];
    long long incl = v[3];
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const long long o = __shfl_up_sync(0xffffffffu, incl, off);
      if (lane >= off) incl += o;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      long long w = warp_tot[lane];
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const long long o = __shfl_up_sync(0xffffffffu, w, off);
        if (lane >= off) w += o;
      }
      warp_tot[lane] = w;                              // inclusive over warps
      if (lane == 31) carry_s = w;                     // total of the tile
    }
    __syncthreads();
    const long long before = carry + (warp > 0 ? warp_tot[warp - 1] : 0) + (incl - v[3]);
#pragma unroll
    for (int k = 0; k < 4; ++k) tile[4 * t + k] = (int32_t)(before + v[k]);
    carry += carry_s;
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int idx = t + k * 1024;
      if (idx < n) row_ptr[base + idx + 1] = tile[idx];
    }
    __syncthreads();
  }
  if (t == 0) {
    if (first) row_ptr[0] = 0;
    if (nnz_out) *nnz_out = carry;
    if (carry > col_capacity) atomicCAS(status, 0, (int)SEER_ERR_CAPACITY);
  }
}

__global__ void __launch_bounds__(kMaskWarps * 32)
fill_kernel(SeqMeta m, RowBand band, const float* __restrict__ scores, seer_mask_params p, const int32_t* __restrict__ row_ptr,
            int32_t* __restrict__ col_idx, int64_t col_capacity, int stage_cap) {
  extern __shared__ __align__(16) uint32_t key_smem[];
  uint32_t* hist_smem = key_smem + (size_t)kMaskWarps * stage_cap;   // 256 bins per warp
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t r = band.row_lo + (int64_t)blockIdx.x * kMaskWarps + warp;
  const RowInfo ri = decode_row(m, band, scores, r);
  if (!ri.valid || ri.skip) return;
  const int n = ri.i + 1;
  const int32_t out0 = row_ptr[r], out1 = row_ptr[r + 1];
  if ((int64_t)out1 > col_capacity) return;   // this row (and all later ones) do not fit; status already raised
  int32_t* __restrict__ out = col_idx + out0;
  const uint32_t lt_mask = (1u << lane) - 1u;

  if (ri.i >= ri.nb - p.dense_tail_blocks) {           // a dense row at the end of the sequence: every causal block
    for (int j = lane; j < n; j += 32) out[j] = j;
    return;
  }
  if (p.mode == SEER_THRESHOLD) {
    int written = 0;
    int head = 0;
    if ((reinterpret_cast<uintptr_t>(ri.s) & 15) == 0) {
      // four consecutive columns per lane: the lane's kept columns follow those of the lanes below it
      head = n & ~127;
      for (int base = 0; base < head; base += 128) {
        const int j = base + 4 * lane;
        const float4 v = *reinterpret_cast<const float4*>(ri.s + j);
        const bool k0 = is_forced(j, ri.i, p.flags) || v.x > p.threshold, k1 = is_forced(j + 1, ri.i, p.flags) || v.y > p.threshold;
        const bool k2 = is_forced(j + 2, ri.i, p.flags) || v.z > p.threshold, k3 = is_forced(j + 3, ri.i, p.flags) || v.w > p.threshold;
        const int mine = (int)k0 + (int)k1 + (int)k2 + (int)k3;
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int u = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += u;
        }
        int at = written + incl - mine;
        if (k0) out[at++] = j;
        if (k1) out[at++] = j + 1;
        if (k2) out[at++] = j + 2;
        if (k3) out[at++] = j + 3;
        written += __shfl_sync(0xffffffffu, incl, 31);
      }
    }
    for (int base = head; base < n; base += 32) {
      const int j = base + lane;
      const bool keep = j < n && (is_forced(j, ri.i, p.flags) || ri.s[j] > p.threshold);
      const uint32_t bal = __ballot_sync(0xffffffffu, keep);
      if (keep) out[written + __popc(bal & lt_mask)] = j;
      written += __popc(bal);
    }
    return;
  }

  // ---- TopK
  const int nf = num_forced(ri.i, p.flags);
  const int take = max(keep_count(n, p) - nf, 0);
  uint32_t* keys = key_smem + (size_t)warp * stage_cap;
  const bool staged = n <= stage_cap;
  int c = 0;
  uint32_t k_and = 0xffffffffu, k_or = 0u;     // over the candidates' keys: the bits all of them share are k_and | ~k_or
  // The same key as score_key in fewer instructions (this loop is bound by instruction issue); forced blocks are not
  // told apart here: they are taken out again below.  (Their keys stay in k_and / k_or: the bits a superset shares are
  // shared by the candidates too.)
  auto lean_key = [](float sc) -> uint32_t {
    const float z = sc + 0.0f;                                   // -0 -> +0
    const uint32_t u = __float_as_uint(z);
    const uint32_t kk = u ^ ((uint32_t)((int32_t)u >> 31) | 0x80000000u);
    return z != z ? 0u : kk;                                     // NaN: never a candidate
  };
  auto make_key = [&](int, float sc) -> uint32_t {
    const uint32_t kk = lean_key(sc);
    c += kk != 0u;
    k_or |= kk;
    k_and &= kk != 0u ? kk : 0xffffffffu;
    return kk;
  };
  // four scores per lane and load where the row is 16-byte aligned (the loop is bound by the latency of its loads);
  // the staged row is padded with zero keys (never candidates) to a multiple of 128
  const bool vec = (reinterpret_cast<uintptr_t>(ri.s) & 15) == 0;
  const int head = vec ? (n & ~3) : 0;
  // (four loads in flight per lane: one load per step left the loop waiting a memory latency per 128 columns, 45 % of
  // the kernel)
  for (int j0 = lane * 4; j0 < head; j0 += 512) {
    float4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u)
      v[u] = j0 + u * 128 < head ? *reinterpret_cast<const float4*>(ri.s + j0 + u * 128) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int j = j0 + u * 128;
      if (j < head) {
        const uint4 kq = make_uint4(make_key(j, v[u].x), make_key(j + 1, v[u].y), make_key(j + 2, v[u].z), make_key(j + 3, v[u].w));
        if (staged) *reinterpret_cast<uint4*>(keys + j) = kq;
      }
    }
  }
  for (int j = head + lane; j < n; j += 32) {
    const uint32_t kk = make_key(j, ri.s[j]);
    if (staged) keys[j] = kk;
  }
  const int n_pad = (n + 127) & ~127;
  if (staged) for (int j = n + lane; j < n_pad; j += 32) keys[j] = 0u;
  // forced blocks are not candidates: out of the count, and their staged keys blanked (a zero key is never kept by the
  // selection; the list writer below puts the forced blocks in their places: block 0 first, block i last)
  const bool sink_f = (p.flags & SEER_FORCE_SINK) != 0u;
  const bool diag_f = (p.flags & SEER_FORCE_DIAG) != 0u && !(sink_f && ri.i == 0);
  __syncwarp();
  if (lane == 0) {                                  // (the staged key where there is one: a global load here costs a memory latency per row)
    if (sink_f) { c -= (staged ? keys[0] : lean_key(ri.s[0])) != 0u; if (staged) keys[0] = 0u; }
    if (diag_f) { c -= (staged ? keys[ri.i] : lean_key(ri.s[ri.i])) != 0u; if (staged) keys[ri.i] = 0u; }
  }
  const int ncand = warp_sum(c);
  k_and = __reduce_and_sync(0xffffffffu, k_and);
  k_or = __reduce_or_sync(0xffffffffu, k_or);
  __syncwarp();
  auto key_at = [&](int j) -> uint32_t {
    return is_forced(j, ri.i, p.flags) ? 0u : score_key(ri.s[j]);
  };

  uint32_t T = 0u;      // key of the last kept candidate; kept: key > T, plus the first need_eq with key == T
  int need_eq = 0;
  if (take >= ncand) {
    T = 0u; need_eq = 0;            // every candidate is kept (key >= 1 > 0)
  } else if (take == 0) {
    T = 0xffffffffu; need_eq = 0;   // nothing beyond the forced blocks
  } else {
    // Radix select, up to 8 bits per pass from the top (rows too long to stage re-read their scores in every pass):
    // histogram the current digit of the keys that match the prefix found so far (warp-private shared-memory bins), walk
    // the bins from the largest digit down until `remaining` is covered.
    uint32_t* hist = hist_smem + warp * 256;
    // The scores of a row are close together (probabilities of one softmax): the leading bits all candidate keys share
    // need no pass, and the first digit starts at the highest bit in which two keys differ, so that it spreads the keys
    // over all 256 bins (a byte-aligned first digit put a whole row into two or three bins: 32 lanes adding to one
    // shared-memory word).
    const uint32_t differ = k_and ^ k_or;                                 // bit set: not all keys agree there
    int hi_bit = differ == 0u ? 0 : 31 - __clz(differ);                   // highest differing bit
    uint32_t prefix_mask = hi_bit >= 31 ? 0u : ~((2u << hi_bit) - 1u);    // the shared leading bits
    uint32_t prefix = k_or & prefix_mask;
    int remaining = take;           // rank (1-based, from the top) still to locate inside the current prefix class
    for (int top = hi_bit; top >= 0; top -= 8) {                          // this pass: bits top .. max(top - 7, 0)
      const int shift = max(top - 7, 0);
      const uint32_t dmask = (2u << (top - shift)) - 1u;
      for (int b = lane; b < 256; b += 32) hist[b] = 0u;
      __syncwarp();
      if (staged) {
        for (int j = lane * 4; j < n_pad; j += 128) {
          const uint4 kq = *reinterpret_cast<const uint4*>(keys + j);
          if (kq.x != 0u && (kq.x & prefix_mask) == prefix) atomicAdd(&hist[(kq.x >> shift) & dmask], 1u);
          if (kq.y != 0u && (kq.y & prefix_mask) == prefix) atomicAdd(&hist[(kq.y >> shift) & dmask], 1u);
          if (kq.z != 0u && (kq.z & prefix_mask) == prefix) atomicAdd(&hist[(kq.z >> shift) & dmask], 1u);
          if (kq.w != 0u && (kq.w & prefix_mask) == prefix) atomicAdd(&hist[(kq.w >> shift) & dmask], 1u);
        }
      } else {
        for (int j = lane; j < n; j += 32) {
          const uint32_t kk = key_at(j);
          if (kk != 0u && (kk & prefix_mask) == prefix) atomicAdd(&hist[(kk >> shift) & dmask], 1u);
        }
      }
      __syncwarp();
      // lane l owns digits 8l .. 8l+7; suffix sums over lanes give the number of keys with a larger digit
      uint32_t c[8], lane_total = 0u;
      {
        const uint4 h0 = *reinterpret_cast<const uint4*>(hist + lane * 8), h1 = *reinterpret_cast<const uint4*>(hist + lane * 8 + 4);
        c[0] = h0.x; c[1] = h0.y; c[2] = h0.z; c[3] = h0.w; c[4] = h1.x; c[5] = h1.y; c[6] = h1.z; c[7] = h1.w;
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) lane_total += c[e];
      uint32_t above = lane_total;                       // inclusive suffix sum over lanes >= this lane
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_down_sync(0xffffffffu, above, o);
        if (lane + o < 32) above += v;
      }
      above -= lane_total;                               // keys in lanes with larger digits
      // the digit holding rank `remaining` lies in the lane where above < remaining <= above + lane_total
      const bool mine = (int)above < remaining && remaining <= (int)(above + lane_total);
      uint32_t digit = 0u, sel_cnt = 0u; int new_remaining = 0;
      if (mine) {
        uint32_t acc = above;
#pragma unroll
        for (int e = 7; e >= 0; --e) {
          if ((int)acc < remaining && remaining <= (int)(acc + c[e])) { digit = (uint32_t)(lane * 8 + e); new_remaining = remaining - (int)acc; sel_cnt = c[e]; }
          acc += c[e];
        }
      }
      const uint32_t owner = __ballot_sync(0xffffffffu, mine);
      const int src = __ffs(owner) - 1;
      digit = __shfl_sync(0xffffffffu, digit, src);
      remaining = __shfl_sync(0xffffffffu, new_remaining, src);
      const uint32_t class_cnt = __shfl_sync(0xffffffffu, sel_cnt, src);   // keys that share the prefix found so far
      prefix |= digit << shift;
      prefix_mask |= dmask << shift;
      __syncwarp();
      // A class of at most 32 keys (the usual case after one pass: a row of <= 2048 keys over 256 bins) is finished in
      // registers: one sweep gathers its keys, every lane ranks one of them against the others.
      if (staged && shift > 0 && class_cnt <= 32u) {
        int found = 0;
        for (int j = lane * 4; j < n_pad; j += 128) {
          const uint4 kq = *reinterpret_cast<const uint4*>(keys + j);
          const uint32_t kk[4] = {kq.x, kq.y, kq.z, kq.w};
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const bool mt = kk[u] != 0u && (kk[u] & prefix_mask) == prefix;
            const uint32_t bal = __ballot_sync(0xffffffffu, mt);
            if (mt) hist[found + __popc(bal & lt_mask)] = kk[u];
            found += __popc(bal);
          }
        }
        __syncwarp();
        const uint32_t x = lane < (int)class_cnt ? hist[lane] : 0u;
        int G = 0, E = 0;                              // keys of the class larger than / equal to this lane's
#pragma unroll
        for (int l = 0; l < 32; ++l) {
          const uint32_t y = __shfl_sync(0xffffffffu, x, l);
          G += y > x; E += y == x;
        }
        const bool is_t = x != 0u && G < remaining && remaining <= G + E;
        const int ts = __ffs(__ballot_sync(0xffffffffu, is_t)) - 1;
        prefix = __shfl_sync(0xffffffffu, x, ts);
        remaining -= __shfl_sync(0xffffffffu, G, ts);
        __syncwarp();
        break;
      }
    }
    T = prefix;                      // the take-th largest key; `remaining` of the keys equal to it are kept
    need_eq = remaining;
  }
  int written = 0, eq_seen = 0;
  if (staged) {
    if (sink_f) { if (lane == 0) out[0] = 0; written = 1; }
    // 128 columns at a time, four consecutive ones per lane: a lane's kept columns follow those of the lanes below it
    for (int base = 0; base < n_pad; base += 128) {
      const int j = base + 4 * lane;
      const uint4 kq = *reinterpret_cast<const uint4*>(keys + j);
      const uint32_t kk[4] = {kq.x, kq.y, kq.z, kq.w};
      bool eq[4], keep[4];
      int my_eq = 0;
#pragma unroll
      for (int u = 0; u < 4; ++u) { eq[u] = kk[u] != 0u && kk[u] == T; my_eq += (int)eq[u]; }
      int eq_incl = my_eq;
      if (__any_sync(0xffffffffu, my_eq != 0)) {          // ties at the selection key are rare
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int u = __shfl_up_sync(0xffffffffu, eq_incl, o);
          if (lane >= o) eq_incl += u;
        }
      }
      int eq_rank = eq_seen + eq_incl - my_eq;            // ties before this lane's first column
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        keep[u] = (kk[u] != 0u && kk[u] > T) || (eq[u] && eq_rank < need_eq);
        eq_rank += (int)eq[u];
      }
      // kept columns of the lanes below this one: four independent ballots instead of a five-step scan
      const uint32_t b0 = __ballot_sync(0xffffffffu, keep[0]), b1 = __ballot_sync(0xffffffffu, keep[1]);
      const uint32_t b2 = __ballot_sync(0xffffffffu, keep[2]), b3 = __ballot_sync(0xffffffffu, keep[3]);
      int at = written + __popc(b0 & lt_mask) + __popc(b1 & lt_mask) + __popc(b2 & lt_mask) + __popc(b3 & lt_mask);
#pragma unroll
      for (int u = 0; u < 4; ++u) if (keep[u]) out[at++] = j + u;
      written += __popc(b0) + __popc(b1) + __popc(b2) + __popc(b3);
      eq_seen += __shfl_sync(0xffffffffu, eq_incl, 31);
    }
    if (diag_f && lane == 0) out[written] = ri.i;
    return;
  }
  for (int base = 0; base < n; base += 32) {
    const int j = base + lane;
    const uint32_t kk = j < n ? key_at(j) : 0u;
    const bool forced = j < n && is_forced(j, ri.i, p.flags);
    const bool eq = kk != 0u && kk == T;
    const uint32_t eq_bal = __ballot_sync(0xffffffffu, eq);
    const bool keep = forced || (kk != 0u && kk > T) || (eq && eq_seen + __popc(eq_bal & lt_mask) < need_eq);
    const uint32_t bal = __ballot_sync(0xffffffffu, keep);
    if (keep) out[written + __popc(bal & lt_mask)] = j;
    written += __popc(bal);
    eq_seen += __popc(eq_bal);
  }
}

int launch_mask_band(seer_ctx* ctx, const SeqMeta& m, const float* scores, int64_t score_base, int64_t row_lo,
                     int64_t row_hi, bool first, const seer_mask_params& p, int32_t* row_ptr, int32_t* col_idx,
                     int64_t col_capacity, int64_t* nnz_out, cudaStream_t stream) {
  if (row_hi <= row_lo) return 0;
  const RowBand band = {row_lo, row_hi, score_base};
  const unsigned grid = (unsigned)((row_hi - row_lo + kMaskWarps - 1) / kMaskWarps);
  count_kernel<<<grid, kMaskWarps * 32, 0, stream>>>(m, band, scores, p, row_ptr);
  scan_kernel<<<1, 1024, 0, stream>>>(row_hi - row_lo, row_ptr + row_lo, first ? 1 : 0, col_capacity, nnz_out, ctx->d_status);
  const int stage_cap = m.max_nb <= kMaskSmemRowMax ? (m.max_nb + 127) & ~127 : 0;   // long rows re-read their scores instead
  const size_t smem = (size_t)kMaskWarps * (stage_cap + 256) * sizeof(uint32_t);
  fill_kernel<<<grid, kMaskWarps * 32, smem, stream>>>(m, band, scores, p, row_ptr, col_idx, col_capacity, stage_cap);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 3 : -(int)e;
}

int launch_mask(seer_ctx* ctx, const SeqMeta& m, const float* scores, const seer_mask_params& p, int32_t* row_ptr,
                int32_t* col_idx, int64_t col_capacity, int64_t* nnz_out, cudaStream_t stream) {
  if (m.rows == 0) {
    cudaMemsetAsync(row_ptr, 0, sizeof(int32_t), stream);
    if (nnz_out) cudaMemsetAsync(nnz_out, 0, sizeof(int64_t), stream);
    return 0;
  }
  return launch_mask_band(ctx, m, scores, 0, 0, m.rows, true, p, row_ptr, col_idx, col_capacity, nnz_out, stream);
}

// ----------------------------------------------------------------------------------------------- 128-token lists -> 64-token lists
// A 128-token block j is the pair of 64-token blocks (2j, 2j + 1); the query rows of 128-token block i are the 64-token
// rows 2i and 2i + 1.  Causality inside the diagonal block: row 2i sees 2i only, row 2i + 1 sees 2i and 2i + 1.  Every
// other listed block j < i contributes both halves to both rows (they exist: only a sequence's last block can be
// shorter than 65 tokens).  An entry j > i is not causal; it is passed on as (2j, 2j + 1) and the attention call
// reports it.  One warp per 64-token row; `fill` = false counts, true writes.
template <bool kFill>
__global__ void __launch_bounds__(kMaskWarps * 32)
expand_kernel(SeqMeta m128, SeqMeta m64, const int32_t* __restrict__ row_ptr128, const int32_t* __restrict__ col_idx128,
              int32_t* __restrict__ row_ptr64, int32_t* __restrict__ col_idx64, int64_t col_capacity64) {
  const int lane = threadIdx.x & 31;
  const int64_t r = (int64_t)blockIdx.x * kMaskWarps + (threadIdx.x >> 5);
  if (r >= m64.rows) return;
  const int b = find_sequence(m64.blk_off, m64.batch, (int)(r / m64.num_q_heads));
  const int nb64 = m64.blk_off[b + 1] - m64.blk_off[b], nb128 = m128.blk_off[b + 1] - m128.blk_off[b];
  const int64_t local = r - (int64_t)m64.num_q_heads * m64.blk_off[b];
  const int h = (int)(local / nb64);
  const int i64 = (int)(local - (int64_t)h * nb64);
  const int i128 = i64 >> 1;
  const bool odd = (i64 & 1) != 0;
  const int64_t src = (int64_t)m128.num_q_heads * m128.blk_off[b] + (int64_t)h * nb128 + i128;
  const int32_t s0 = row_ptr128[src], s1 = row_ptr128[src + 1];
  int32_t out0 = 0;
  if (kFill) {
    out0 = row_ptr64[r];
    if ((int64_t)row_ptr64[r + 1] > col_capacity64) return;    // does not fit; status already raised by the scan
  }
  int written = 0;
  for (int base = s0; base < s1; base += 32) {
    const int e = base + lane;
    const int j = e < s1 ? col_idx128[e] : -1;
    const int c = e < s1 ? ((j == i128 && !odd) ? 1 : 2) : 0;
    int incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (kFill && c > 0) {
      int32_t* dst = col_idx64 + out0 + written + incl - c;
      dst[0] = 2 * j;
      if (c == 2) dst[1] = 2 * j + 1;
    }
    written += __shfl_sync(0xffffffffu, incl, 31);
  }
  if (!kFill && lane == 0) row_ptr64[r + 1] = written;
}

int launch_expand_lists(seer_ctx* ctx, const SeqMeta& m128, const SeqMeta& m64, const int32_t* row_ptr128,
                        const int32_t* col_idx128, int32_t* row_ptr64, int32_t* col_idx64, int64_t col_capacity64,
                        int64_t* nnz_out, cudaStream_t stream) {
  if (m64.rows == 0) {
    cudaMemsetAsync(row_ptr64, 0, sizeof(int32_t), stream);
    if (nnz_out) cudaMemsetAsync(nnz_out, 0, sizeof(int64_t), stream);
    return 0;
  }
  const unsigned grid = (unsigned)((m64.rows + kMaskWarps - 1) / kMaskWarps);
  expand_kernel<false><<<grid, kMaskWarps * 32, 0, stream>>>(m128, m64, row_ptr128, col_idx128, row_ptr64, col_idx64, col_capacity64);
  scan_kernel<<<1, 1024, 0, stream>>>(m64.rows, row_ptr64, 1, col_capacity64, nnz_out, ctx->d_status);
  expand_kernel<true><<<grid, kMaskWarps * 32, 0, stream>>>(m128, m64, row_ptr128, col_idx128, row_ptr64, col_idx64, col_capacity64);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 3 : -(int)e;
}

seer_status init_mask(seer_ctx* ctx) {
  (void)ctx;
  cudaError_t e = cudaFuncSetAttribute(fill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kMaskWarps * (kMaskSmemRowMax + 256) * (int)sizeof(uint32_t));
  return e == cudaSuccess ? SEER_OK : SEER_ERR_CUDA;
}

}  // namespace seer
