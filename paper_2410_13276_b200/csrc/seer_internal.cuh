// Internal declarations shared by the library's translation units (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "seer.h"

namespace seer {

constexpr int kBlock = 64;      // attention tile; the gate block is 64 or 128 tokens (SeqMeta::block)
constexpr int kHeadDim = 128;
constexpr int kGateDim = 128;
constexpr int kMaxBatch = 4096;
constexpr int kMetaSlots = 8;
constexpr int kPoolChunk = 16;  // blocks pooled and projected by one CTA of the gate's first kernel
constexpr int kScoreTile = 64;  // score rows (blocks of the packed batch) handled by one CTA of the gate's second kernel

// Per-batch metadata the kernels read from device memory.
struct SeqMeta {
  const int32_t* cu_seqlens;   // [batch+1] token offsets
  const int32_t* blk_off;      // [batch+1] cumulative number of blocks
  const int64_t* score_off;    // [batch+1] Hq * cumulative nb^2
  int32_t batch;
  int32_t num_q_heads;
  int32_t num_kv_heads;
  int32_t group;               // Hq / Hkv
  int32_t total_tokens;
  int32_t total_blocks;
  int32_t total_chunks;
  int32_t max_nb;
  int64_t rows;                // Hq * total_blocks
  int64_t score_elems;
  float softmax_scale;
  int32_t block;               // tokens per gate block: 64, or 128 (gate and mask only)
  // chunked prefill (all zero without a chunk): the queries of sequence b are its last positions
  const int32_t* qoff;         // [batch] block position of the chunk's first query block
  const int32_t* qdelta;       // [batch] token index in q / o / lse = token index in k / v + qdelta
  int32_t total_q_tokens;      // tokens in q / o / lse
  int32_t chunked;             // 1 if the shape carries cu_seqlens_q
  // bounded waits of the tcgen05 attention kernel, and the test hook that makes one of them run out
  uint32_t wait_limit_us;      // a barrier wait that lasts this long is declared lost
  int32_t lose_v_copy;         // >= 0: stream 0 of CTA 0 never issues the V copy of its tile with this ordinal
};

// A rectangle of (block row of the packed batch, query head) pairs whose scores are produced and consumed together.
// score_base is the offset, in the full score matrix, of the band's first element: the band's scores live at
// (full offset - score_base) in whatever buffer the kernels are given.
struct ScoreBand {
  int32_t blk_lo, blk_hi;      // block rows [blk_lo, blk_hi), numbered over the batch (blk_off)
  int32_t head_lo, heads;
  int64_t score_base;
};

struct MetaSlot {
  std::vector<int32_t> key;    // cu_seqlens + Hq: what the slot currently describes
  void* dev = nullptr;
  void* pinned = nullptr;
  cudaEvent_t ready = nullptr;     // upload finished
  cudaEvent_t last_use = nullptr;  // last library call that read the slot
  uint64_t stamp = 0;
};

}  // namespace seer

struct seer_ctx {
  int device = 0;
  int num_sms = 0;
  int* d_status = nullptr;
  int attn_impl = 0;
  int64_t launches = 0;
  uint64_t clock = 0;
  seer::MetaSlot slots[seer::kMetaSlots];
  void* tmap_encode = nullptr;   // cuTensorMapEncodeTiled, resolved at run time
  void* trace = nullptr;         // optional device buffer for the attention kernel's timeline (diagnostics)
  uint32_t wait_limit_us = 2000000u;   // seer_debug_lost_wait
  int32_t lose_v_copy = -1;
  // seer_prefill_host: copy streams and the events of its two-deep pipeline over KV-head slices
  cudaStream_t h2d_stream = nullptr, d2h_stream = nullptr;
  cudaEvent_t ev_start = nullptr, ev_h2d[2] = {nullptr, nullptr}, ev_comp[2] = {nullptr, nullptr},
              ev_d2h[2] = {nullptr, nullptr};
};

namespace seer {

// Validates the shape, makes its metadata resident on the device (ordered before later work on `stream`)
// and fills `m`.  `slot_out` identifies the slot to pass to finish_call.
seer_status prepare(seer_ctx* ctx, const seer_shape* shape, cudaStream_t stream, SeqMeta* m, int* slot_out);
void finish_call(seer_ctx* ctx, int slot, cudaStream_t stream);

// Host-only shape arithmetic (no CUDA calls): returns SEER_OK and fills totals.
struct ShapeTotals {
  int64_t total_tokens, total_q_tokens, total_blocks, total_chunks, rows, score_elems, causal_blocks;
  int32_t max_nb;
};
seer_status shape_totals(const seer_shape* shape, ShapeTotals* t);

size_t gate_workspace_bytes(const ShapeTotals& t, const seer_shape* shape);

// Kernel launchers (each returns the number of kernels it launched, or a negative cudaError).
int launch_gate(seer_ctx* ctx, const SeqMeta& m, const void* q, const void* k, const float* Wq, const float* Wk,
                float* scores, void* ws, cudaStream_t stream);
int launch_gate_ex(seer_ctx* ctx, const SeqMeta& m, const seer_gate_options& opt, const void* q, const void* k,
                   const float* Wq, const float* Wk, float* scores, void* ws, cudaStream_t stream);
int launch_gate_scores_band(const SeqMeta& m, const ScoreBand& band, const void* ws, float* scores, cudaStream_t stream);
// Mask rows [row_lo, row_hi) from a band of scores; `first` starts row_ptr at 0, later bands continue from the
// previous band's last entry.
int launch_mask_band(seer_ctx* ctx, const SeqMeta& m, const float* scores, int64_t score_base, int64_t row_lo,
                     int64_t row_hi, bool first, const seer_mask_params& p, int32_t* row_ptr, int32_t* col_idx,
                     int64_t col_capacity, int64_t* nnz_out, cudaStream_t stream);
// 128-token block lists -> the 64-token lists the attention kernels take (m128 and m64 describe the same batch).
int launch_expand_lists(seer_ctx* ctx, const SeqMeta& m128, const SeqMeta& m64, const int32_t* row_ptr128,
                        const int32_t* col_idx128, int32_t* row_ptr64, int32_t* col_idx64, int64_t col_capacity64,
                        int64_t* nnz_out, cudaStream_t stream);
int launch_mask(seer_ctx* ctx, const SeqMeta& m, const float* scores, const seer_mask_params& p, int32_t* row_ptr,
                int32_t* col_idx, int64_t col_capacity, int64_t* nnz_out, cudaStream_t stream);
int launch_attn_mma(seer_ctx* ctx, const SeqMeta& m, const void* q, const void* k, const void* v,
                    const int32_t* row_ptr, const int32_t* col_idx, void* o, float* lse, cudaStream_t stream);
int launch_block_max(seer_ctx* ctx, const SeqMeta& m, const void* q, const void* k, const int32_t* row_ptr,
                     const int32_t* col_idx, const float* lse, float* out, cudaStream_t stream);
int launch_block_max_tc(seer_ctx* ctx, const SeqMeta& m, const void* q, const void* k, const int32_t* row_ptr,
                        const int32_t* col_idx, const float* lse, float* out, cudaStream_t stream);
int launch_attn_tc(seer_ctx* ctx, const SeqMeta& m, const void* q, const void* k, const void* v,
                   const int32_t* row_ptr, const int32_t* col_idx, void* o, float* lse, int* work_counter,
                   cudaStream_t stream);
seer_status init_gate(seer_ctx* ctx);
seer_status init_mask(seer_ctx* ctx);
seer_status init_attn_mma(seer_ctx* ctx);
seer_status init_attn_tc(seer_ctx* ctx);


// Sequence that owns global block index gb: largest b with blk_off[b] <= gb (empty sequences are skipped).
__device__ __forceinline__ int find_sequence(const int32_t* __restrict__ off, int batch, int x) {
  int lo = 0, hi = batch;  // off[lo] <= x < off[hi]
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (off[mid] <= x) lo = mid; else hi = mid;
  }
  return lo;
}

}  // namespace seer
