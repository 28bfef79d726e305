// Context, shape validation, per-batch metadata upload and the three ABI entry points.
#include <cstring>

#include "seer_internal.cuh"

namespace seer {

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Byte offsets of the four arrays inside a metadata slot.
constexpr size_t kOffCu = 0;
constexpr size_t kOffBlk = kOffCu + sizeof(int32_t) * (kMaxBatch + 1 + 3);
constexpr size_t kOffScore = kOffBlk + sizeof(int32_t) * (kMaxBatch + 1 + 3);
constexpr size_t kOffQoff = kOffScore + sizeof(int64_t) * (kMaxBatch + 1);
constexpr size_t kOffQdelta = kOffQoff + sizeof(int32_t) * (kMaxBatch + 4);
constexpr size_t kSlotBytes = kOffQdelta + sizeof(int32_t) * (kMaxBatch + 4);

seer_status shape_totals(const seer_shape* s, ShapeTotals* t) {
  if (!s || !s->cu_seqlens_host || s->batch < 1) return SEER_ERR_INVALID_ARG;
  if (s->num_q_heads < 1 || s->num_kv_heads < 1) return SEER_ERR_INVALID_ARG;
  if (s->batch > kMaxBatch) return SEER_ERR_UNSUPPORTED;
  if (s->head_dim != kHeadDim || (s->block != kBlock && s->block != 2 * kBlock) || s->gate_dim != kGateDim)
    return SEER_ERR_UNSUPPORTED;
  if (s->num_q_heads % s->num_kv_heads != 0) return SEER_ERR_UNSUPPORTED;
  const int32_t* cu = s->cu_seqlens_host;
  if (cu[0] != 0) return SEER_ERR_INVALID_ARG;
  if (const int32_t* cq = s->cu_seqlens_q_host) {
    // the queries are the last positions of each sequence and start on a block boundary
    if (cq[0] != 0) return SEER_ERR_INVALID_ARG;
    for (int b = 0; b < s->batch; ++b) {
      if (cu[b + 1] < cu[b]) return SEER_ERR_INVALID_ARG;
      const int64_t sq = (int64_t)cq[b + 1] - cq[b], sk = (int64_t)cu[b + 1] - cu[b];
      if (sq < 0 || sq > sk) return SEER_ERR_INVALID_ARG;
      if (sq > 0 && (sk - sq) % s->block != 0) return SEER_ERR_UNSUPPORTED;
    }
  }
  int64_t blocks = 0, sq = 0, causal = 0;
  int32_t max_nb = 0;
  for (int b = 0; b < s->batch; ++b) {
    if (cu[b + 1] < cu[b]) return SEER_ERR_INVALID_ARG;
    int64_t nb = ((int64_t)cu[b + 1] - cu[b] + s->block - 1) / s->block;
    blocks += nb;
    sq += nb * nb;
    causal += nb * (nb + 1) / 2;
    if (nb > max_nb) max_nb = (int32_t)nb;
  }
  t->total_tokens = cu[s->batch];
  t->total_q_tokens = s->cu_seqlens_q_host ? s->cu_seqlens_q_host[s->batch] : cu[s->batch];
  t->total_blocks = blocks;
  t->total_chunks = (blocks + kPoolChunk - 1) / kPoolChunk;   // chunks of the gate's first kernel run over the whole batch
  t->rows = blocks * s->num_q_heads;
  t->score_elems = sq * s->num_q_heads;
  t->causal_blocks = causal * s->num_q_heads;
  t->max_nb = max_nb;
  // int32 row ids / CSR offsets and 32-bit grids
  if (t->rows >= (int64_t)1 << 31 || t->causal_blocks >= (int64_t)1 << 31) return SEER_ERR_UNSUPPORTED;
  if ((int64_t)t->total_tokens * s->num_q_heads * kHeadDim >= (int64_t)1 << 40) return SEER_ERR_UNSUPPORTED;
  return SEER_OK;
}

size_t gate_workspace_bytes(const ShapeTotals& t, const seer_shape* s) {
  // projected pooled Q [Hq, blocks, dg] and K [Hkv, blocks, dg], each as three bf16 planes (hi, mid, lo of the fp32 value)
  size_t gq = align_up((size_t)s->num_q_heads * t.total_blocks * kGateDim * 6, 256);
  size_t gk = align_up((size_t)s->num_kv_heads * t.total_blocks * kGateDim * 6, 256);
  return gq + gk;
}

seer_status prepare(seer_ctx* ctx, const seer_shape* shape, cudaStream_t stream, SeqMeta* m, int* slot_out) {
  if (!ctx) return SEER_ERR_INVALID_ARG;
  ShapeTotals t;
  seer_status st = shape_totals(shape, &t);
  if (st != SEER_OK) return st;
  if (cudaSetDevice(ctx->device) != cudaSuccess) return SEER_ERR_CUDA;

  const int n = shape->batch + 1;
  std::vector<int32_t> key(shape->cu_seqlens_host, shape->cu_seqlens_host + n);
  key.push_back(shape->num_q_heads);
  key.push_back(shape->block);
  if (shape->cu_seqlens_q_host) key.insert(key.end(), shape->cu_seqlens_q_host, shape->cu_seqlens_q_host + n);
  int slot = -1;
  for (int i = 0; i < kMetaSlots; ++i)
    if (ctx->slots[i].key == key) { slot = i; break; }
  if (slot < 0) {
    // the least recently used slot whose last reader and last upload have finished; only if every slot is still
    // in flight (more than kMetaSlots shapes cycling faster than the GPU works through them) does the call wait
    // for the oldest one
    slot = -1;
    int oldest = 0;
    for (int i = 0; i < kMetaSlots; ++i) {
      if (ctx->slots[i].stamp < ctx->slots[oldest].stamp) oldest = i;
      if (cudaEventQuery(ctx->slots[i].last_use) == cudaSuccess && cudaEventQuery(ctx->slots[i].ready) == cudaSuccess &&
          (slot < 0 || ctx->slots[i].stamp < ctx->slots[slot].stamp))
        slot = i;
    }
    (void)cudaGetLastError();                        // cudaErrorNotReady from the queries is not an error
    if (slot < 0) {
      slot = oldest;
      if (cudaEventSynchronize(ctx->slots[slot].last_use) != cudaSuccess) return SEER_ERR_CUDA;
      if (cudaEventSynchronize(ctx->slots[slot].ready) != cudaSuccess) return SEER_ERR_CUDA;
    }
    MetaSlot& s = ctx->slots[slot];
    char* h = (char*)s.pinned;
    int32_t* cu = (int32_t*)(h + kOffCu);
    int32_t* blk = (int32_t*)(h + kOffBlk);
    int64_t* sc = (int64_t*)(h + kOffScore);
    int32_t* qo = (int32_t*)(h + kOffQoff);
    int32_t* qd = (int32_t*)(h + kOffQdelta);
    blk[0] = 0; sc[0] = 0;
    for (int b = 0; b < shape->batch; ++b) {
      cu[b] = shape->cu_seqlens_host[b];
      int32_t nb = (shape->cu_seqlens_host[b + 1] - shape->cu_seqlens_host[b] + shape->block - 1) / shape->block;
      blk[b + 1] = blk[b] + nb;
      sc[b + 1] = sc[b] + (int64_t)shape->num_q_heads * nb * nb;
      qo[b] = 0; qd[b] = 0;
      if (const int32_t* cq = shape->cu_seqlens_q_host) {
        const int32_t sq = cq[b + 1] - cq[b], sk = shape->cu_seqlens_host[b + 1] - shape->cu_seqlens_host[b];
        qo[b] = sq > 0 ? (sk - sq) / shape->block : nb;          // no queries: past the last block
        qd[b] = cq[b] - (shape->cu_seqlens_host[b] + (sk - sq));  // first query token <-> key token cu[b] + sk - sq
      }
    }
    cu[shape->batch] = shape->cu_seqlens_host[shape->batch];
    if (cudaMemcpyAsync(s.dev, s.pinned, kSlotBytes, cudaMemcpyHostToDevice, stream) != cudaSuccess) return SEER_ERR_CUDA;
    if (cudaEventRecord(s.ready, stream) != cudaSuccess) return SEER_ERR_CUDA;
    s.key = key;
  } else {
    // another stream may have uploaded it
    if (cudaStreamWaitEvent(stream, ctx->slots[slot].ready, 0) != cudaSuccess) return SEER_ERR_CUDA;
  }
  MetaSlot& s = ctx->slots[slot];
  s.stamp = ++ctx->clock;
  const char* d = (const char*)s.dev;
  m->cu_seqlens = (const int32_t*)(d + kOffCu);
  m->blk_off = (const int32_t*)(d + kOffBlk);
  m->score_off = (const int64_t*)(d + kOffScore);
  m->batch = shape->batch;
  m->num_q_heads = shape->num_q_heads;
  m->num_kv_heads = shape->num_kv_heads;
  m->group = shape->num_q_heads / shape->num_kv_heads;
  m->total_tokens = (int32_t)t.total_tokens;
  m->total_blocks = (int32_t)t.total_blocks;
  m->total_chunks = (int32_t)t.total_chunks;
  m->max_nb = t.max_nb;
  m->rows = t.rows;
  m->score_elems = t.score_elems;
  m->softmax_scale = shape->softmax_scale > 0.f ? shape->softmax_scale : 0.08838834764831845f;  // 1/sqrt(128)
  m->block = shape->block;
  m->qoff = (const int32_t*)(d + kOffQoff);
  m->qdelta = (const int32_t*)(d + kOffQdelta);
  m->total_q_tokens = (int32_t)t.total_q_tokens;
  m->chunked = shape->cu_seqlens_q_host ? 1 : 0;
  m->wait_limit_us = ctx->wait_limit_us;
  m->lose_v_copy = ctx->lose_v_copy;
  *slot_out = slot;
  return SEER_OK;
}

void finish_call(seer_ctx* ctx, int slot, cudaStream_t stream) {
  cudaEventRecord(ctx->slots[slot].last_use, stream);
}

static bool ws_ok(const void* ws, size_t have, size_t need) {
  if (need == 0) return true;
  return ws && ((uintptr_t)ws & 255) == 0 && have >= need;
}

}  // namespace seer

using namespace seer;

extern "C" {

const char* seer_status_string(seer_status s) {
  switch (s) {
    case SEER_OK: return "ok";
    case SEER_ERR_INVALID_ARG: return "invalid argument";
    case SEER_ERR_UNSUPPORTED: return "unsupported shape";
    case SEER_ERR_WORKSPACE: return "workspace too small or misaligned";
    case SEER_ERR_CAPACITY: return "col_idx capacity exceeded";
    case SEER_ERR_INVALID_INDEX: return "block index out of range";
    case SEER_ERR_TIMEOUT: return "bounded device wait expired";
    case SEER_ERR_CUDA: return "CUDA call failed";
  }
  return "unknown status";
}

seer_status seer_create(seer_ctx** out, int device) {
  if (!out) return SEER_ERR_INVALID_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return SEER_ERR_CUDA;
  if (cudaSetDevice(device) != cudaSuccess) return SEER_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return SEER_ERR_CUDA;
  if (prop.major != 10) return SEER_ERR_CUDA;  // kernels are built for sm_100a only
  seer_ctx* ctx = new seer_ctx();
  ctx->device = device;
  ctx->num_sms = prop.multiProcessorCount;
  bool ok = cudaMalloc(&ctx->d_status, sizeof(int)) == cudaSuccess &&
            cudaMemset(ctx->d_status, 0, sizeof(int)) == cudaSuccess;
  for (int i = 0; ok && i < kMetaSlots; ++i) {
    MetaSlot& s = ctx->slots[i];
    ok = cudaMalloc(&s.dev, kSlotBytes) == cudaSuccess && cudaMallocHost(&s.pinned, kSlotBytes) == cudaSuccess &&
         cudaEventCreateWithFlags(&s.ready, cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&s.last_use, cudaEventDisableTiming) == cudaSuccess;
  }
  if (ok) ok = cudaStreamCreateWithFlags(&ctx->h2d_stream, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&ctx->d2h_stream, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&ctx->ev_start, cudaEventDisableTiming) == cudaSuccess;
  for (int i = 0; ok && i < 2; ++i)
    ok = cudaEventCreateWithFlags(&ctx->ev_h2d[i], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&ctx->ev_comp[i], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&ctx->ev_d2h[i], cudaEventDisableTiming) == cudaSuccess;
  if (ok) ok = init_gate(ctx) == SEER_OK && init_mask(ctx) == SEER_OK && init_attn_mma(ctx) == SEER_OK &&
              init_attn_tc(ctx) == SEER_OK;
  if (!ok) { seer_destroy(ctx); return SEER_ERR_CUDA; }
  *out = ctx;
  return SEER_OK;
}

void seer_destroy(seer_ctx* ctx) {
  if (!ctx) return;
  cudaSetDevice(ctx->device);
  cudaDeviceSynchronize();
  for (int i = 0; i < kMetaSlots; ++i) {
    MetaSlot& s = ctx->slots[i];
    if (s.dev) cudaFree(s.dev);
    if (s.pinned) cudaFreeHost(s.pinned);
    if (s.ready) cudaEventDestroy(s.ready);
    if (s.last_use) cudaEventDestroy(s.last_use);
  }
  if (ctx->d_status) cudaFree(ctx->d_status);
  if (ctx->h2d_stream) cudaStreamDestroy(ctx->h2d_stream);
  if (ctx->d2h_stream) cudaStreamDestroy(ctx->d2h_stream);
  if (ctx->ev_start) cudaEventDestroy(ctx->ev_start);
  for (int i = 0; i < 2; ++i) {
    if (ctx->ev_h2d[i]) cudaEventDestroy(ctx->ev_h2d[i]);
    if (ctx->ev_comp[i]) cudaEventDestroy(ctx->ev_comp[i]);
    if (ctx->ev_d2h[i]) cudaEventDestroy(ctx->ev_d2h[i]);
  }
  delete ctx;
}

size_t seer_workspace_bytes(const seer_shape* shape) {
  ShapeTotals t;
  if (shape_totals(shape, &t) != SEER_OK) return 0;
  return gate_workspace_bytes(t, shape);
}

size_t seer_scores_elems(const seer_shape* shape) {
  ShapeTotals t;
  if (shape_totals(shape, &t) != SEER_OK) return 0;
  return (size_t)t.score_elems;
}

int64_t seer_mask_rows(const seer_shape* shape) {
  ShapeTotals t;
  if (shape_totals(shape, &t) != SEER_OK) return -1;
  return t.rows;
}

int64_t seer_causal_blocks(const seer_shape* shape) {
  ShapeTotals t;
  if (shape_totals(shape, &t) != SEER_OK) return -1;
  return t.causal_blocks;
}

seer_status seer_gate_scores(seer_ctx* ctx, const seer_shape* shape, const void* q, const void* k, const float* Wq,
                             const float* Wk, float* scores, void* ws, size_t ws_bytes, void* stream_) {
  cudaStream_t stream = (cudaStream_t)stream_;
  if (!ctx || !shape) return SEER_ERR_INVALID_ARG;
  ShapeTotals t;
  seer_status st = shape_totals(shape, &t);
  if (st != SEER_OK) return st;
  if (t.total_blocks == 0 || t.total_q_tokens == 0) return SEER_OK;   // no score row to write
  if (!q || !k || !Wq || !Wk || !scores) return SEER_ERR_INVALID_ARG;
  if (!ws_ok(ws, ws_bytes, gate_workspace_bytes(t, shape))) return SEER_ERR_WORKSPACE;
  SeqMeta m; int slot;
  st = prepare(ctx, shape, stream, &m, &slot);
  if (st != SEER_OK) return st;
  int n = launch_gate(ctx, m, q, k, Wq, Wk, scores, ws, stream);
  finish_call(ctx, slot, stream);
  if (n < 0) return SEER_ERR_CUDA;
  ctx->launches += n;
  return SEER_OK;
}

seer_status seer_gate_project(seer_ctx* ctx, const seer_shape* shape, const void* q, const void* k, const float* Wq,
                              const float* Wk, void* ws, size_t ws_bytes, void* stream_) {
  cudaStream_t stream = (cudaStream_t)stream_;
  if (!ctx || !shape) return SEER_ERR_INVALID_ARG;
  ShapeTotals t;
  seer_status st = shape_totals(shape, &t);
  if (st != SEER_OK) return st;
  if (t.total_blocks == 0 || t.total_q_tokens == 0) return SEER_OK;
  if (!q || !k || !Wq || !Wk) return SEER_ERR_INVALID_ARG;
  if (!ws_ok(ws, ws_bytes, gate_workspace_bytes(t, shape))) return SEER_ERR_WORKSPACE;
  SeqMeta m; int slot;
  st = prepare(ctx, shape, stream, &m, &slot);
  if (st != SEER_OK) return st;
  int n = launch_gate(ctx, m, q, k, Wq, Wk, nullptr, ws, stream);   // no score buffer: pooling and projection only
  finish_call(ctx, slot, stream);
  if (n < 0) return SEER_ERR_CUDA;
  ctx->launches += n;
  return SEER_OK;
}

seer_status seer_gate_scores_ex(seer_ctx* ctx, const seer_shape* shape, const seer_gate_options* opt, const void* q,
                                const void* k, const float* Wq, const float* Wk, float* scores, void* ws, size_t ws_bytes,
                                void* stream_) {
  cudaStream_t stream = (cudaStream_t)stream_;
  if (!ctx || !shape || !opt) return SEER_ERR_INVALID_ARG;
  const uint32_t all = SEER_POOL_AVG | SEER_POOL_MAX | SEER_POOL_MIN;
  if (opt->pool_q == 0 || opt->pool_k == 0 || (opt->pool_q & ~all) || (opt->pool_k & ~all)) return SEER_ERR_INVALID_ARG;
  if (!(opt->rope_theta >= 0.f) || opt->rope_theta > 3.0e38f) return SEER_ERR_INVALID_ARG;   // also rejects NaN
  ShapeTotals t;
  seer_status st = shape_totals(shape, &t);
  if (st != SEER_OK) return st;
  if (t.total_blocks == 0 || t.total_q_tokens == 0) return SEER_OK;   // no score row to write
  if (!q || !k || !Wq || !Wk || !scores) return SEER_ERR_INVALID_ARG;
  if (!ws_ok(ws, ws_bytes, gate_workspace_bytes(t, shape))) return SEER_ERR_WORKSPACE;
  SeqMeta m; int slot;
  st = prepare(ctx, shape, stream, &m, &slot);
  if (st != SEER_OK) return st;
  int n = launch_gate_ex(ctx, m, *opt, q, k, Wq, Wk, scores, ws, stream);
  finish_call(ctx, slot, stream);
  if (n < 0) return SEER_ERR_CUDA;
  ctx->launches += n;
  return SEER_OK;
}

seer_status seer_block_mask(seer_ctx* ctx, const seer_shape* shape, const float* scores, const seer_mask_params* p,
                            int32_t* row_ptr, int32_t* col_idx, int64_t col_capacity, int64_t* nnz_out, void* ws,
                            size_t ws_bytes, void* stream_) {
  (void)ws; (void)ws_bytes;
  cudaStream_t stream = (cudaStream_t)stream_;
  if (!ctx || !shape || !p) return SEER_ERR_INVALID_ARG;
  ShapeTotals t;
  seer_status st = shape_totals(shape, &t);
  if (st != SEER_OK) return st;
  if (!row_ptr || col_capacity < 0 || (col_capacity > 0 && !col_idx)) return SEER_ERR_INVALID_ARG;
  if (p->mode != SEER_TOPK_RATIO && p->mode != SEER_TOPK_COUNT && p->mode != SEER_THRESHOLD) return SEER_ERR_INVALID_ARG;
  if (p->mode == SEER_TOPK_RATIO && (p->keep_num < 0 || p->keep_den < 1)) return SEER_ERR_INVALID_ARG;
  if (p->flags & ~(uint32_t)(SEER_FORCE_DIAG | SEER_FORCE_SINK)) return SEER_ERR_INVALID_ARG;
  if (p->dense_tail_blocks < 0) return SEER_ERR_INVALID_ARG;
  if (t.total_blocks > 0 && !scores) return SEER_ERR_INVALID_ARG;
  SeqMeta m; int slot;
  st = prepare(ctx, shape, stream, &m, &slot);
  if (st != SEER_OK) return st;
  int n = launch_mask(ctx, m, scores, *p, row_ptr, col_idx, col_capacity, nnz_out, stream);
  finish_call(ctx, slot, stream);
  if (n < 0) return SEER_ERR_CUDA;
  ctx->launches += n;
  return SEER_OK;
}

seer_status seer_sparse_attn(seer_ctx* ctx, const seer_shape* shape, const void* q, const void* k, const void* v,
                             const int32_t* row_ptr, const int32_t* col_idx, void* o, float* lse, void* ws,
                             size_t ws_bytes, void* stream_) {
  cudaStream_t stream = (cudaStream_t)stream_;
  if (!ctx || !shape) return SEER_ERR_INVALID_ARG;
  ShapeTotals t;
  seer_status st = shape_totals(shape, &t);
  if (st != SEER_OK) return st;
  if (shape->block != kBlock) return SEER_ERR_UNSUPPORTED;   // 128-token lists go through seer_expand_block_lists first
  // the first word of the workspace is the counter the tcgen05 kernel's streams draw their work items from; without
  // a workspace the items are dealt statically
  int* work_counter = ws_ok(ws, ws_bytes, 256) ? (int*)ws : nullptr;
  if (t.total_blocks == 0 || t.total_q_tokens == 0) return SEER_OK;   // no output row
  if (!q || !k || !v || !row_ptr || !col_idx || !o) return SEER_ERR_INVALID_ARG;
  SeqMeta m; int slot;
  st = prepare(ctx, shape, stream, &m, &slot);
  if (st != SEER_OK) return st;
  // impl 2: by shape.  The lists are at most the causal blocks; rows that short cost the persistent kernel more in
  // per-row hand-over than the legacy kernel needs for the whole row.
  const bool legacy = ctx->attn_impl == 1 || (ctx->attn_impl == 2 && t.causal_blocks <= 8 * t.rows);
  int n = legacy ? launch_attn_mma(ctx, m, q, k, v, row_ptr, col_idx, o, lse, stream)
                 : launch_attn_tc(ctx, m, q, k, v, row_ptr, col_idx, o, lse, work_counter, stream);
  finish_call(ctx, slot, stream);
  if (n < 0) return SEER_ERR_CUDA;
  ctx->launches += n;
  return SEER_OK;
}

seer_status seer_attn_block_max(seer_ctx* ctx, const seer_shape* shape, const void* q, const void* k,
                                const int32_t* row_ptr, const int32_t* col_idx, const float* lse, float* block_max,
                                void* stream_) {
  cudaStream_t stream = (cudaStream_t)stream_;
  if (!ctx || !shape) return SEER_ERR_INVALID_ARG;
  ShapeTotals t;
  seer_status st = shape_totals(shape, &t);
  if (st != SEER_OK) return st;
  if (shape->block != kBlock) return SEER_ERR_UNSUPPORTED;
  if (t.total_blocks == 0 || t.total_q_tokens == 0) return SEER_OK;
  if (!q || !k || !row_ptr || !col_idx || !lse || !block_max) return SEER_ERR_INVALID_ARG;
  SeqMeta m; int slot;
  st = prepare(ctx, shape, stream, &m, &slot);
  if (st != SEER_OK) return st;
  // the same choice of kernel as seer_sparse_attn: the tcgen05 pipeline without V, or the mma.sync kernel
  const bool legacy = ctx->attn_impl == 1 || (ctx->attn_impl == 2 && t.causal_blocks <= 8 * t.rows);
  int n = legacy ? launch_block_max(ctx, m, q, k, row_ptr, col_idx, lse, block_max, stream)
                 : launch_block_max_tc(ctx, m, q, k, row_ptr, col_idx, lse, block_max, stream);
  finish_call(ctx, slot, stream);
  if (n < 0) return SEER_ERR_CUDA;
  ctx->launches += n;
  return SEER_OK;
}

// ---- gate and mask in one call, the scores held one band at a time
namespace {
constexpr size_t kBandSlackElems = 4;   // the band's base is rounded down to a multiple of four elements

size_t min_band_bytes(const ShapeTotals& t) { return ((size_t)kScoreTile * (size_t)t.max_nb + kBandSlackElems) * sizeof(float); }
}  // namespace

size_t seer_gate_mask_workspace_bytes(const seer_shape* shape, size_t band_bytes) {
  ShapeTotals t;
  if (shape_totals(shape, &t) != SEER_OK) return 0;
  const size_t need = min_band_bytes(t);
  return gate_workspace_bytes(t, shape) + align_up(band_bytes > need ? band_bytes : need, 256);
}

seer_status seer_gate_block_mask(seer_ctx* ctx, const seer_shape* shape, const seer_gate_options* opt, const void* q,
                                 const void* k, const float* Wq, const float* Wk, const seer_mask_params* p,
                                 int32_t* row_ptr, int32_t* col_idx, int64_t col_capacity, int64_t* nnz_out, void* ws,
                                 size_t ws_bytes, void* stream_) {
  cudaStream_t stream = (cudaStream_t)stream_;
  if (!ctx || !shape || !p) return SEER_ERR_INVALID_ARG;
  if (opt) {
    const uint32_t all = SEER_POOL_AVG | SEER_POOL_MAX | SEER_POOL_MIN;
    if (opt->pool_q == 0 || opt->pool_k == 0 || (opt->pool_q & ~all) || (opt->pool_k & ~all)) return SEER_ERR_INVALID_ARG;
    if (!(opt->rope_theta >= 0.f) || opt->rope_theta > 3.0e38f) return SEER_ERR_INVALID_ARG;
  }
  ShapeTotals t;
  seer_status st = shape_totals(shape, &t);
  if (st != SEER_OK) return st;
  if (!row_ptr || col_capacity < 0 || (col_capacity > 0 && !col_idx)) return SEER_ERR_INVALID_ARG;
  if (p->mode != SEER_TOPK_RATIO && p->mode != SEER_TOPK_COUNT && p->mode != SEER_THRESHOLD) return SEER_ERR_INVALID_ARG;
  if (p->mode == SEER_TOPK_RATIO && (p->keep_num < 0 || p->keep_den < 1)) return SEER_ERR_INVALID_ARG;
  if (p->flags & ~(uint32_t)(SEER_FORCE_DIAG | SEER_FORCE_SINK)) return SEER_ERR_INVALID_ARG;
  if (p->dense_tail_blocks < 0) return SEER_ERR_INVALID_ARG;
  if (t.total_blocks > 0 && ((!q && t.total_q_tokens > 0) || !k || !Wq || !Wk)) return SEER_ERR_INVALID_ARG;
  const size_t gate_bytes = gate_workspace_bytes(t, shape);
  if (t.total_blocks > 0 && !ws_ok(ws, ws_bytes, gate_bytes + min_band_bytes(t))) return SEER_ERR_WORKSPACE;
  SeqMeta m; int slot;
  st = prepare(ctx, shape, stream, &m, &slot);
  if (st != SEER_OK) return st;
  if (t.total_blocks == 0) {
    int n0 = launch_mask(ctx, m, nullptr, *p, row_ptr, col_idx, col_capacity, nnz_out, stream);
    finish_call(ctx, slot, stream);
    return n0 < 0 ? SEER_ERR_CUDA : SEER_OK;
  }
  float* band_buf = (float*)((char*)ws + gate_bytes);
  const int64_t cap = (int64_t)((ws_bytes - gate_bytes) / sizeof(float)) - (int64_t)kBandSlackElems;   // elements per band
  int64_t launched = 0;
  bool bad = false, first = true;
  {
    int n = opt ? launch_gate_ex(ctx, m, *opt, q, k, Wq, Wk, nullptr, ws, stream)
                : launch_gate(ctx, m, q, k, Wq, Wk, nullptr, ws, stream);
    if (n < 0) bad = true; else launched += n;
  }
  // One band after the other, in CSR row order: scores of the band -> counts -> row_ptr (continued) -> lists.
  auto run_band = [&](int64_t blk_lo, int64_t blk_hi, int head_lo, int heads, int64_t base, int64_t row_lo, int64_t row_hi) {
    if (bad || row_hi <= row_lo) return;
    const ScoreBand band = {(int32_t)blk_lo, (int32_t)blk_hi, head_lo, heads, base & ~(int64_t)3};
    int n = launch_gate_scores_band(m, band, ws, band_buf, stream);
    if (n >= 0) {
      launched += n;
      n = launch_mask_band(ctx, m, band_buf, band.score_base, row_lo, row_hi, first, *p, row_ptr, col_idx, col_capacity,
                           nnz_out, stream);
    }
    if (n < 0) { bad = true; return; }
    launched += n;
    first = false;
  };
  const int32_t* cu = shape->cu_seqlens_host;
  const int Hq = shape->num_q_heads;
  auto blocks_of = [&](int b) { return ((int64_t)cu[b + 1] - cu[b] + shape->block - 1) / shape->block; };
  int64_t blk_off = 0, score_off = 0;                  // of sequence b
  for (int b = 0; b < shape->batch && !bad;) {
    const int64_t nb = blocks_of(b);
    if ((int64_t)Hq * nb * nb <= cap) {
      // whole sequences, as many as fit
      int b1 = b;
      int64_t blocks = 0, elems = 0;
      while (b1 < shape->batch) {
        const int64_t n1 = blocks_of(b1);
        if (elems + (int64_t)Hq * n1 * n1 > cap) break;
        elems += (int64_t)Hq * n1 * n1; blocks += n1;
        ++b1;
      }
      run_band(blk_off, blk_off + blocks, 0, Hq, score_off, Hq * blk_off, Hq * (blk_off + blocks));
      blk_off += blocks; score_off += elems;
      b = b1;
      continue;
    }
    const int64_t ntile = (nb + kScoreTile - 1) / kScoreTile;
    if (nb * nb <= cap) {
      // whole heads of this sequence
      const int hb = (int)(cap / (nb * nb));
      for (int h0 = 0; h0 < Hq; h0 += hb) {
        const int h1 = h0 + hb < Hq ? h0 + hb : Hq;
        run_band(blk_off, blk_off + nb, h0, h1 - h0, score_off + (int64_t)h0 * nb * nb, Hq * blk_off + (int64_t)h0 * nb,
                 Hq * blk_off + (int64_t)h1 * nb);
      }
    } else {
      // runs of 64-row tiles of one head
      const int64_t tb = cap / ((int64_t)kScoreTile * nb);   // >= 1: the workspace check above
      for (int h = 0; h < Hq; ++h)
        for (int64_t t0 = 0; t0 < ntile; t0 += tb) {
          const int64_t t1 = t0 + tb < ntile ? t0 + tb : ntile;
          const int64_t i0 = t0 * kScoreTile, i1 = t1 * kScoreTile < nb ? t1 * kScoreTile : nb;
          run_band(blk_off + i0, blk_off + i1, h, 1, score_off + ((int64_t)h * nb + i0) * nb,
                   Hq * blk_off + (int64_t)h * nb + i0, Hq * blk_off + (int64_t)h * nb + i1);
        }
    }
    blk_off += nb; score_off += (int64_t)Hq * nb * nb;
    ++b;
  }
  finish_call(ctx, slot, stream);
  if (bad) return SEER_ERR_CUDA;
  ctx->launches += launched;
  return SEER_OK;
}

seer_status seer_expand_block_lists(seer_ctx* ctx, const seer_shape* shape, const int32_t* row_ptr, const int32_t* col_idx,
                                    int32_t* row_ptr64, int32_t* col_idx64, int64_t col_capacity64, int64_t* nnz_out,
                                    void* stream_) {
  cudaStream_t stream = (cudaStream_t)stream_;
  if (!ctx || !shape) return SEER_ERR_INVALID_ARG;
  if (shape->block != 2 * kBlock) return SEER_ERR_UNSUPPORTED;
  seer_shape fine = *shape;
  fine.block = kBlock;
  ShapeTotals t128, t64;
  seer_status st = shape_totals(shape, &t128);
  if (st == SEER_OK) st = shape_totals(&fine, &t64);
  if (st != SEER_OK) return st;
  if (!row_ptr64 || col_capacity64 < 0 || (col_capacity64 > 0 && !col_idx64)) return SEER_ERR_INVALID_ARG;
  if (t128.total_blocks > 0 && !row_ptr) return SEER_ERR_INVALID_ARG;
  SeqMeta m128, m64; int slot128, slot64;
  st = prepare(ctx, shape, stream, &m128, &slot128);
  if (st != SEER_OK) return st;
  st = prepare(ctx, &fine, stream, &m64, &slot64);
  if (st != SEER_OK) { finish_call(ctx, slot128, stream); return st; }
  int n = launch_expand_lists(ctx, m128, m64, row_ptr, col_idx, row_ptr64, col_idx64, col_capacity64, nnz_out, stream);
  finish_call(ctx, slot128, stream);
  finish_call(ctx, slot64, stream);
  if (n < 0) return SEER_ERR_CUDA;
  ctx->launches += n;
  return SEER_OK;
}

seer_status seer_debug_lost_wait(seer_ctx* ctx, uint32_t wait_limit_us, int32_t lose_v_copy_of_tile) {
  if (!ctx || wait_limit_us == 0u) return SEER_ERR_INVALID_ARG;
  ctx->wait_limit_us = wait_limit_us;
  ctx->lose_v_copy = lose_v_copy_of_tile;
  return SEER_OK;
}

seer_status seer_set_attn_impl(seer_ctx* ctx, int impl) {
  if (!ctx || impl < 0 || impl > 2) return SEER_ERR_INVALID_ARG;
  ctx->attn_impl = impl;
  return SEER_OK;
}

seer_status seer_poll_device_status(seer_ctx* ctx, void* stream_) {
  if (!ctx) return SEER_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)stream_;
  if (cudaSetDevice(ctx->device) != cudaSuccess) return SEER_ERR_CUDA;
  int h = 0;
  if (cudaMemcpyAsync(&h, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, stream) != cudaSuccess) return SEER_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return SEER_ERR_CUDA;
  if (h != 0) {
    if (cudaMemsetAsync(ctx->d_status, 0, sizeof(int), stream) != cudaSuccess) return SEER_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return SEER_ERR_CUDA;
  }
  return (seer_status)h;
}

int64_t seer_launch_count(const seer_ctx* ctx) { return ctx ? ctx->launches : -1; }

seer_status seer_set_trace_buffer(seer_ctx* ctx, void* device_buffer) {
  if (!ctx) return SEER_ERR_INVALID_ARG;
  ctx->trace = device_buffer;
  return SEER_OK;
}

namespace {
// seer_prefill_host works on one KV head (and the query heads of its group) at a time: a slice is a problem of its own
// with num_q_heads = G, num_kv_heads = 1.  The arena holds two sets of slice inputs and outputs (copy of slice s + 1 and
// read-back of slice s - 1 overlap the kernels of slice s) and one set of intermediates.
struct ArenaLayout {
  size_t q[2], k[2], v[2], o[2], lse[2], wq[2], wk[2], scores, row_ptr, col_idx, nnz, ws, total;
};
ArenaLayout arena_layout(const seer_shape* slice, const ShapeTotals& t) {   // shape and totals of ONE slice
  ArenaLayout a;
  size_t p = 0;
  auto take = [&](size_t bytes) { size_t at = p; p = align_up(p + bytes, 256); return at; };
  const size_t T = (size_t)t.total_tokens;
  for (int b = 0; b < 2; ++b) {
    a.q[b] = take(T * slice->num_q_heads * kHeadDim * 2);
    a.k[b] = take(T * kHeadDim * 2);
    a.v[b] = take(T * kHeadDim * 2);
    a.o[b] = take(T * slice->num_q_heads * kHeadDim * 2);
    a.lse[b] = take(T * slice->num_q_heads * 4);
    a.wq[b] = take((size_t)slice->num_q_heads * kHeadDim * kGateDim * 4);
    a.wk[b] = take((size_t)kHeadDim * kGateDim * 4);
  }
  a.scores = take((size_t)t.score_elems * 4);
  a.row_ptr = take(((size_t)t.rows + 1) * 4);
  a.col_idx = take((size_t)t.causal_blocks * 4);
  a.nnz = take(8);
  a.ws = take(gate_workspace_bytes(t, slice));
  a.total = p;
  return a;
}
}  // namespace

static bool slice_of(const seer_shape* shape, seer_shape* slice, ShapeTotals* t) {
  *slice = *shape;
  if (shape->num_kv_heads <= 0 || shape->num_q_heads % shape->num_kv_heads != 0) return false;
  slice->num_q_heads = shape->num_q_heads / shape->num_kv_heads;
  slice->num_kv_heads = 1;
  return shape_totals(slice, t) == SEER_OK;
}

size_t seer_prefill_host_arena_bytes(const seer_shape* shape) {
  ShapeTotals full, t;
  seer_shape slice;
  if (!shape || shape_totals(shape, &full) != SEER_OK || !slice_of(shape, &slice, &t)) return 0;
  return arena_layout(&slice, t).total;
}

seer_status seer_prefill_host(seer_ctx* ctx, const seer_shape* shape, const void* q_host, const void* k_host,
                              const void* v_host, const float* Wq_host, const float* Wk_host,
                              const seer_mask_params* params, void* o_host, float* lse_host, void* arena,
                              size_t arena_bytes, void* stream_) {
  cudaStream_t stream = (cudaStream_t)stream_;
  if (!ctx || !shape || !params) return SEER_ERR_INVALID_ARG;
  ShapeTotals full, t;
  seer_status st = shape_totals(shape, &full);
  if (st != SEER_OK) return st;
  if (shape->block != kBlock || shape->cu_seqlens_q_host) return SEER_ERR_UNSUPPORTED;
  if (full.total_blocks == 0) return SEER_OK;
  if (!q_host || !k_host || !v_host || !Wq_host || !Wk_host || !o_host) return SEER_ERR_INVALID_ARG;
  seer_shape slice;
  if (!slice_of(shape, &slice, &t)) return SEER_ERR_INVALID_ARG;
  const ArenaLayout a = arena_layout(&slice, t);
  if (!ws_ok(arena, arena_bytes, a.total)) return SEER_ERR_WORKSPACE;
  if (cudaSetDevice(ctx->device) != cudaSuccess) return SEER_ERR_CUDA;
  char* d = (char*)arena;
  const size_t T = (size_t)t.total_tokens;
  const int Hq = shape->num_q_heads, Hkv = shape->num_kv_heads, G = slice.num_q_heads;
  const size_t head_bytes = (size_t)kHeadDim * 2;                       // one head of one token
  const size_t wq_bytes = (size_t)G * kHeadDim * kGateDim * 4, wk_bytes = (size_t)kHeadDim * kGateDim * 4;
  cudaStream_t h2d = ctx->h2d_stream, d2h = ctx->d2h_stream;
#define SEER_TRY(call) do { if ((call) != cudaSuccess) return SEER_ERR_CUDA; } while (0)
  // the copy streams start after whatever precedes this call on the caller's stream
  SEER_TRY(cudaEventRecord(ctx->ev_start, stream));
  SEER_TRY(cudaStreamWaitEvent(h2d, ctx->ev_start, 0));
  SEER_TRY(cudaStreamWaitEvent(d2h, ctx->ev_start, 0));
  for (int g = 0; g < Hkv; ++g) {
    const int b = g & 1;
    // ---- host -> device: the slice's heads are strided in the host tensors ([T, H, 128]) and packed on the device
    if (g >= 2) SEER_TRY(cudaStreamWaitEvent(h2d, ctx->ev_comp[b], 0));   // slice g - 2 has finished with these buffers
    SEER_TRY(cudaMemcpy2DAsync(d + a.q[b], (size_t)G * head_bytes, (const char*)q_host + (size_t)g * G * head_bytes,
                               (size_t)Hq * head_bytes, (size_t)G * head_bytes, T, cudaMemcpyHostToDevice, h2d));
    SEER_TRY(cudaMemcpy2DAsync(d + a.k[b], head_bytes, (const char*)k_host + (size_t)g * head_bytes, (size_t)Hkv * head_bytes,
                               head_bytes, T, cudaMemcpyHostToDevice, h2d));
    SEER_TRY(cudaMemcpy2DAsync(d + a.v[b], head_bytes, (const char*)v_host + (size_t)g * head_bytes, (size_t)Hkv * head_bytes,
                               head_bytes, T, cudaMemcpyHostToDevice, h2d));
    SEER_TRY(cudaMemcpyAsync(d + a.wq[b], (const char*)Wq_host + (size_t)g * wq_bytes, wq_bytes, cudaMemcpyHostToDevice, h2d));
    SEER_TRY(cudaMemcpyAsync(d + a.wk[b], (const char*)Wk_host + (size_t)g * wk_bytes, wk_bytes, cudaMemcpyHostToDevice, h2d));
    SEER_TRY(cudaEventRecord(ctx->ev_h2d[b], h2d));
    // ---- the three calls on the slice, on the caller's stream
    SEER_TRY(cudaStreamWaitEvent(stream, ctx->ev_h2d[b], 0));
    if (g >= 2) SEER_TRY(cudaStreamWaitEvent(stream, ctx->ev_d2h[b], 0));  // o / lse of slice g - 2 have been read back
    st = seer_gate_scores(ctx, &slice, d + a.q[b], d + a.k[b], (const float*)(d + a.wq[b]), (const float*)(d + a.wk[b]),
                          (float*)(d + a.scores), d + a.ws, a.total - a.ws, stream);
    if (st != SEER_OK) return st;
    st = seer_block_mask(ctx, &slice, (const float*)(d + a.scores), params, (int32_t*)(d + a.row_ptr),
                         (int32_t*)(d + a.col_idx), t.causal_blocks, (int64_t*)(d + a.nnz), nullptr, 0, stream);
    if (st != SEER_OK) return st;
    st = seer_sparse_attn(ctx, &slice, d + a.q[b], d + a.k[b], d + a.v[b], (const int32_t*)(d + a.row_ptr),
                          (const int32_t*)(d + a.col_idx), d + a.o[b], lse_host ? (float*)(d + a.lse[b]) : nullptr, d + a.ws,
                          a.total - a.ws, stream);   // (the gate's workspace is free again: the attention's work counter)
    if (st != SEER_OK) return st;
    SEER_TRY(cudaEventRecord(ctx->ev_comp[b], stream));
    // ---- device -> host
    SEER_TRY(cudaStreamWaitEvent(d2h, ctx->ev_comp[b], 0));
    SEER_TRY(cudaMemcpy2DAsync((char*)o_host + (size_t)g * G * head_bytes, (size_t)Hq * head_bytes, d + a.o[b],
                               (size_t)G * head_bytes, (size_t)G * head_bytes, T, cudaMemcpyDeviceToHost, d2h));
    if (lse_host)
      SEER_TRY(cudaMemcpyAsync(lse_host + (size_t)g * G * T, d + a.lse[b], (size_t)G * T * 4, cudaMemcpyDeviceToHost, d2h));
    SEER_TRY(cudaEventRecord(ctx->ev_d2h[b], d2h));
  }
  // the caller's stream is complete when the last read-backs are
  SEER_TRY(cudaStreamWaitEvent(stream, ctx->ev_d2h[(Hkv - 1) & 1], 0));
  if (Hkv >= 2) SEER_TRY(cudaStreamWaitEvent(stream, ctx->ev_d2h[Hkv & 1], 0));
#undef SEER_TRY
  return SEER_OK;
}

}  // extern "C"
