// Context, shape validation, per-batch metadata upload and the three ABI entry points.
#include <cstring>

#include "seer_internal.cuh"

namespace seer {

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Byte offsets of the four arrays inside a metadata slot.
constexpr size_t kOffCu = 0;
constexpr size_t kOffBlk = kOffCu + sizeof(int32_t) * (kMaxBatch + 1 + 3);
constexpr size_t kOffChunk = kOffBlk + sizeof(int32_t) * (kMaxBatch + 1 + 3);
constexpr size_t kOffTile = kOffChunk + sizeof(int32_t) * (kMaxBatch + 1 + 3);
constexpr size_t kOffScore = kOffTile + sizeof(int32_t) * (kMaxBatch + 1 + 3);
constexpr size_t kSlotBytes = kOffScore + sizeof(int64_t) * (kMaxBatch + 1);

seer_status shape_totals(const seer_shape* s, ShapeTotals* t) {
  if (!s || !s->cu_seqlens_host || s->batch < 1) return SEER_ERR_INVALID_ARG;
  if (s->num_q_heads < 1 || s->num_kv_heads < 1) return SEER_ERR_INVALID_ARG;
  if (s->batch > kMaxBatch) return SEER_ERR_UNSUPPORTED;
  if (s->head_dim != kHeadDim || s->block != kBlock || s->gate_dim != kGateDim) return SEER_ERR_UNSUPPORTED;
  if (s->num_q_heads % s->num_kv_heads != 0) return SEER_ERR_UNSUPPORTED;
  const int32_t* cu = s->cu_seqlens_host;
  if (cu[0] != 0) return SEER_ERR_INVALID_ARG;
  int64_t blocks = 0, chunks = 0, tiles = 0, sq = 0, causal = 0;
  int32_t max_nb = 0;
  for (int b = 0; b < s->batch; ++b) {
    if (cu[b + 1] < cu[b]) return SEER_ERR_INVALID_ARG;
    int64_t nb = ((int64_t)cu[b + 1] - cu[b] + kBlock - 1) / kBlock;
    blocks += nb;
    chunks += (nb + kPoolChunk - 1) / kPoolChunk;
    tiles += (nb + kScoreTile - 1) / kScoreTile;
    sq += nb * nb;
    causal += nb * (nb + 1) / 2;
    if (nb > max_nb) max_nb = (int32_t)nb;
  }
  t->total_tokens = cu[s->batch];
  t->total_blocks = blocks;
  t->total_chunks = chunks;
  t->total_tiles = tiles;
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
  // projected pooled Q [Hq, blocks, dg] and K [Hkv, blocks, dg], fp32
  size_t gq = align_up((size_t)s->num_q_heads * t.total_blocks * kGateDim * sizeof(float), 256);
  size_t gk = align_up((size_t)s->num_kv_heads * t.total_blocks * kGateDim * sizeof(float), 256);
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
  int slot = -1;
  for (int i = 0; i < kMetaSlots; ++i)
    if (ctx->slots[i].key == key) { slot = i; break; }
  if (slot < 0) {
    slot = 0;
    for (int i = 1; i < kMetaSlots; ++i)
      if (ctx->slots[i].stamp < ctx->slots[slot].stamp) slot = i;
    MetaSlot& s = ctx->slots[slot];
    // The slot may still be read by kernels of earlier calls, and its staging buffer by an earlier upload.
    if (cudaEventSynchronize(s.last_use) != cudaSuccess) return SEER_ERR_CUDA;
    if (cudaEventSynchronize(s.ready) != cudaSuccess) return SEER_ERR_CUDA;
    char* h = (char*)s.pinned;
    int32_t* cu = (int32_t*)(h + kOffCu);
    int32_t* blk = (int32_t*)(h + kOffBlk);
    int32_t* chk = (int32_t*)(h + kOffChunk);
    int32_t* til = (int32_t*)(h + kOffTile);
    int64_t* sc = (int64_t*)(h + kOffScore);
    blk[0] = 0; chk[0] = 0; til[0] = 0; sc[0] = 0;
    for (int b = 0; b < shape->batch; ++b) {
      cu[b] = shape->cu_seqlens_host[b];
      int32_t nb = (shape->cu_seqlens_host[b + 1] - shape->cu_seqlens_host[b] + kBlock - 1) / kBlock;
      blk[b + 1] = blk[b] + nb;
      chk[b + 1] = chk[b] + (nb + kPoolChunk - 1) / kPoolChunk;
      til[b + 1] = til[b] + (nb + kScoreTile - 1) / kScoreTile;
      sc[b + 1] = sc[b] + (int64_t)shape->num_q_heads * nb * nb;
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
  m->chunk_off = (const int32_t*)(d + kOffChunk);
  m->tile_off = (const int32_t*)(d + kOffTile);
  m->score_off = (const int64_t*)(d + kOffScore);
  m->batch = shape->batch;
  m->num_q_heads = shape->num_q_heads;
  m->num_kv_heads = shape->num_kv_heads;
  m->group = shape->num_q_heads / shape->num_kv_heads;
  m->total_tokens = (int32_t)t.total_tokens;
  m->total_blocks = (int32_t)t.total_blocks;
  m->total_chunks = (int32_t)t.total_chunks;
  m->total_tiles = (int32_t)t.total_tiles;
  m->max_nb = t.max_nb;
  m->rows = t.rows;
  m->score_elems = t.score_elems;
  m->softmax_scale = shape->softmax_scale > 0.f ? shape->softmax_scale : 0.08838834764831845f;  // 1/sqrt(128)
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
  if (t.total_blocks == 0) return SEER_OK;
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
  if (t.total_blocks == 0) return SEER_OK;
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
  (void)ws; (void)ws_bytes;
  cudaStream_t stream = (cudaStream_t)stream_;
  if (!ctx || !shape) return SEER_ERR_INVALID_ARG;
  ShapeTotals t;
  seer_status st = shape_totals(shape, &t);
  if (st != SEER_OK) return st;
  if (t.total_blocks == 0) return SEER_OK;
  if (!q || !k || !v || !row_ptr || !o) return SEER_ERR_INVALID_ARG;
  SeqMeta m; int slot;
  st = prepare(ctx, shape, stream, &m, &slot);
  if (st != SEER_OK) return st;
  int n = ctx->attn_impl == 1 ? launch_attn_mma(ctx, m, q, k, v, row_ptr, col_idx, o, lse, stream)
                              : launch_attn_tc(ctx, m, q, k, v, row_ptr, col_idx, o, lse, stream);
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
  if (t.total_blocks == 0) return SEER_OK;
  if (!q || !k || !row_ptr || !lse) return SEER_ERR_INVALID_ARG;
  SeqMeta m; int slot;
  st = prepare(ctx, shape, stream, &m, &slot);
  if (st != SEER_OK) return st;
  int n = launch_block_max(ctx, m, q, k, row_ptr, col_idx, lse, block_max, stream);
  finish_call(ctx, slot, stream);
  if (n < 0) return SEER_ERR_CUDA;
  ctx->launches += n;
  return SEER_OK;
}

seer_status seer_set_attn_impl(seer_ctx* ctx, int impl) {
  if (!ctx || (impl != 0 && impl != 1)) return SEER_ERR_INVALID_ARG;
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
struct ArenaLayout {
  size_t q, k, v, o, wq, wk, scores, row_ptr, col_idx, nnz, lse, ws, total;
};
ArenaLayout arena_layout(const seer_shape* s, const ShapeTotals& t) {
  ArenaLayout a;
  size_t p = 0;
  auto take = [&](size_t bytes) { size_t at = p; p = align_up(p + bytes, 256); return at; };
  const size_t T = (size_t)t.total_tokens;
  a.q = take(T * s->num_q_heads * kHeadDim * 2);
  a.k = take(T * s->num_kv_heads * kHeadDim * 2);
  a.v = take(T * s->num_kv_heads * kHeadDim * 2);
  a.o = take(T * s->num_q_heads * kHeadDim * 2);
  a.wq = take((size_t)s->num_q_heads * kHeadDim * kGateDim * 4);
  a.wk = take((size_t)s->num_kv_heads * kHeadDim * kGateDim * 4);
  a.scores = take((size_t)t.score_elems * 4);
  a.row_ptr = take(((size_t)t.rows + 1) * 4);
  a.col_idx = take((size_t)t.causal_blocks * 4);
  a.nnz = take(8);
  a.lse = take(T * s->num_q_heads * 4);
  a.ws = take(gate_workspace_bytes(t, s));
  a.total = p;
  return a;
}
}  // namespace

size_t seer_prefill_host_arena_bytes(const seer_shape* shape) {
  ShapeTotals t;
  if (shape_totals(shape, &t) != SEER_OK) return 0;
  return arena_layout(shape, t).total;
}

seer_status seer_prefill_host(seer_ctx* ctx, const seer_shape* shape, const void* q_host, const void* k_host,
                              const void* v_host, const float* Wq_host, const float* Wk_host,
                              const seer_mask_params* params, void* o_host, float* lse_host, void* arena,
                              size_t arena_bytes, void* stream_) {
  cudaStream_t stream = (cudaStream_t)stream_;
  if (!ctx || !shape || !params) return SEER_ERR_INVALID_ARG;
  ShapeTotals t;
  seer_status st = shape_totals(shape, &t);
  if (st != SEER_OK) return st;
  if (t.total_blocks == 0) return SEER_OK;
  if (!q_host || !k_host || !v_host || !Wq_host || !Wk_host || !o_host) return SEER_ERR_INVALID_ARG;
  const ArenaLayout a = arena_layout(shape, t);
  if (!ws_ok(arena, arena_bytes, a.total)) return SEER_ERR_WORKSPACE;
  if (cudaSetDevice(ctx->device) != cudaSuccess) return SEER_ERR_CUDA;
  char* d = (char*)arena;
  const size_t T = (size_t)t.total_tokens;
  const size_t qb = T * shape->num_q_heads * kHeadDim * 2, kb = T * shape->num_kv_heads * kHeadDim * 2;
  bool ok = cudaMemcpyAsync(d + a.q, q_host, qb, cudaMemcpyHostToDevice, stream) == cudaSuccess &&
            cudaMemcpyAsync(d + a.k, k_host, kb, cudaMemcpyHostToDevice, stream) == cudaSuccess &&
            cudaMemcpyAsync(d + a.v, v_host, kb, cudaMemcpyHostToDevice, stream) == cudaSuccess &&
            cudaMemcpyAsync(d + a.wq, Wq_host, (size_t)shape->num_q_heads * kHeadDim * kGateDim * 4,
                            cudaMemcpyHostToDevice, stream) == cudaSuccess &&
            cudaMemcpyAsync(d + a.wk, Wk_host, (size_t)shape->num_kv_heads * kHeadDim * kGateDim * 4,
                            cudaMemcpyHostToDevice, stream) == cudaSuccess;
  if (!ok) return SEER_ERR_CUDA;
  st = seer_gate_scores(ctx, shape, d + a.q, d + a.k, (const float*)(d + a.wq), (const float*)(d + a.wk),
                        (float*)(d + a.scores), d + a.ws, a.total - a.ws, stream);
  if (st != SEER_OK) return st;
  st = seer_block_mask(ctx, shape, (const float*)(d + a.scores), params, (int32_t*)(d + a.row_ptr),
                       (int32_t*)(d + a.col_idx), t.causal_blocks, (int64_t*)(d + a.nnz), nullptr, 0, stream);
  if (st != SEER_OK) return st;
  st = seer_sparse_attn(ctx, shape, d + a.q, d + a.k, d + a.v, (const int32_t*)(d + a.row_ptr),
                        (const int32_t*)(d + a.col_idx), d + a.o, lse_host ? (float*)(d + a.lse) : nullptr, nullptr, 0,
                        stream);
  if (st != SEER_OK) return st;
  if (cudaMemcpyAsync(o_host, d + a.o, qb, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return SEER_ERR_CUDA;
  if (lse_host &&
      cudaMemcpyAsync(lse_host, d + a.lse, T * shape->num_q_heads * 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
    return SEER_ERR_CUDA;
  return SEER_OK;
}

}  // extern "C"
