/*
 * seer.h -- C ABI of the B200 (sm_100a) SeerAttention prefill hot path.
 *
 *   seer_gate_scores : Q, K, Wq, Wk        -> block-level gating scores   (Sec. 3.1, Eq. 1)
 *   seer_block_mask  : scores, TopK | thr  -> per-row sorted KV-block index lists (Sec. 3.3, Eq. 3 / Eq. 4)
 *   seer_sparse_attn : Q, K, V, lists      -> O, visiting only listed blocks (Sec. 3.3, "Block Sparse Flash-Attn Kernel")
 *
 * General rules
 *  - Every tensor pointer is a DEVICE pointer owned by the caller and must stay valid until the work
 *    enqueued by the call has completed on `stream`.  `cu_seqlens_host` and the parameter structs are
 *    HOST memory and are consumed before the call returns.
 *  - Calls enqueue kernels on `stream` (a cudaStream_t passed as void*; NULL = default stream) and return
 *    without synchronising, with one exception: the context keeps the batch metadata (sequence offsets) of the
 *    8 most recent shapes on the device; a call with a ninth shape reuses the least recently used entry whose
 *    work has finished, and only if all 8 are still in flight does it wait on the host for the oldest one.
 *    The library allocates device memory only in seer_create; per-call scratch comes from the caller's
 *    workspace `ws` (>= seer_workspace_bytes(shape), 256-byte aligned).
 *  - The tcgen05 attention kernel takes all 512 tensor-memory columns and 219 KB of shared memory of an SM, the
 *    gate's score kernel 256 columns and 226 KB: one CTA of either is resident per SM (the two cannot share an SM
 *    either), so a tensor-memory allocation never waits on another CTA of this library.  A kernel of ANOTHER
 *    library that holds tensor memory on the same device at the same time (another stream or process) can make
 *    that allocation wait; it is the one wait in these kernels the library cannot bound.
 *  - Nothing throws across the ABI.  Host-detectable errors are returned at once and enqueue nothing.
 *    Errors only the device can see (list capacity exceeded, a list entry out of range, a bounded wait
 *    that ran out) are recorded in a status word owned by the context; the offending work is skipped and
 *    the kernel exits normally.  seer_poll_device_status reads that word.
 *  - bf16 tensors are passed as const void* / void*; element type is the 16-bit bfloat16 bit pattern.
 *
 * Shapes and layouts ("THD", packed variable-length batch)
 *    T            total tokens of all sequences = cu_seqlens[batch]
 *    q, o         [T, num_q_heads,  head_dim]   row-major bf16
 *    k, v         [T, num_kv_heads, head_dim]   row-major bf16
 *    Wq           [num_q_heads,  head_dim, gate_dim] fp32,  gate input x Wq[h] (row vector times matrix, no bias)
 *    Wk           [num_kv_heads, head_dim, gate_dim] fp32;  query head h pairs with KV head h / (Hq/Hkv)
 *    nb_b         ceil(len_b / block) blocks in sequence b
 *    scores       sequence after sequence, each [num_q_heads][nb_b][nb_b] fp32; entry (h,i,j) is defined for
 *                 j <= i only, the rest is never written nor read
 *    mask rows    row id of (b, h, i) = num_q_heads * (blocks of sequences before b) + h * nb_b + i
 *    row_ptr      int32 [rows + 1], col_idx int32 [nnz]: CSR lists of KV block indices, local to the sequence,
 *                 ascending, unique, 0 <= j <= i
 *
 * Supported: head_dim = 128, gate_dim = 128, block = 64 (every call) or 128 (gate and mask calls; the attention takes
 * their lists through seer_expand_block_lists), num_q_heads a multiple of num_kv_heads, batch <= 4096.
 * Anything else returns SEER_ERR_UNSUPPORTED.
 */
#ifndef SEER_H_
#define SEER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SEER_OK = 0,
  SEER_ERR_INVALID_ARG = 1,   /* null pointer, negative size, non-monotone cu_seqlens, bad mode */
  SEER_ERR_UNSUPPORTED = 2,   /* shape outside the supported set (see above), or more than 2^31-1 mask rows / score elements per sequence */
  SEER_ERR_WORKSPACE = 3,     /* ws too small or misaligned */
  SEER_ERR_CAPACITY = 4,      /* device: nnz exceeds col_capacity; row_ptr and nnz_out are still complete */
  SEER_ERR_INVALID_INDEX = 5, /* device: a list entry outside [0, i] */
  SEER_ERR_TIMEOUT = 6,       /* device: a bounded wait expired */
  SEER_ERR_CUDA = 7           /* a CUDA runtime / driver call failed (including: no device, no sm_100 device) */
} seer_status;

typedef struct seer_ctx seer_ctx;

/* Creates a context on CUDA device `device`: queries the SM count, raises the kernels' shared-memory limits,
 * allocates the device status word and a small metadata buffer.  Not thread-safe per context: use one
 * context per host thread or serialise calls. */
seer_status seer_create(seer_ctx** out, int device);
void seer_destroy(seer_ctx* ctx);
const char* seer_status_string(seer_status s);

typedef struct {
  int32_t batch;                  /* number of packed sequences, >= 1 */
  const int32_t* cu_seqlens_host; /* HOST [batch + 1], cu[0] = 0, non-decreasing; empty sequences are allowed */
  int32_t num_q_heads;
  int32_t num_kv_heads;
  int32_t head_dim;               /* 128 */
  int32_t block;                  /* 64: gate pooling window = attention tile (Sec. 4: B fixed at 64); or 128, see
                                     seer_expand_block_lists */
  int32_t gate_dim;               /* 128: output width of the gate's linear layers */
  float softmax_scale;            /* attention logit scale; <= 0 selects 1/sqrt(head_dim) (Sec. 2) */
  const int32_t* cu_seqlens_q_host; /* HOST [batch + 1] or NULL.  NULL: every sequence has as many queries as keys.
                                     Otherwise chunked prefill, see below */
} seer_shape;

/* Chunked prefill (the paper prefills whole prompts; a serving stack feeds them in pieces against a growing KV cache).
 *
 * With cu_seqlens_q_host set, sequence b has S_k = cu_seqlens[b+1] - cu_seqlens[b] keys and S_q = cu_q[b+1] - cu_q[b]
 * queries, which are the LAST S_q positions of the sequence; S_q <= S_k, and the chunk starts on a block boundary
 * ((S_k - S_q) a multiple of `block`) unless S_q = 0.  q, o are [cu_q[batch], num_q_heads, head_dim] and lse
 * [num_q_heads, cu_q[batch]]: they hold the chunk's tokens only; k, v hold all S_k tokens.
 * Everything indexed by blocks keeps the numbering of the whole sequence: nb_b = ceil(S_k / block), the score matrix is
 * [num_q_heads][nb_b][nb_b] per sequence, the CSR structure has num_q_heads * nb_b rows per sequence, and block-level
 * RoPE rotates a query block by its position in the sequence.  Only the rows of the chunk's query blocks are produced:
 * score rows before the chunk are not written, their CSR rows are empty, and lists given for them are ignored by the
 * attention.  The results are those of the whole problem restricted to the chunk (same kernels, same arithmetic).
 * A score buffer of full size is only needed by the separate gate and mask calls; seer_gate_block_mask needs none.
 * With no query at all (cu_q[batch] = 0) the gate and attention calls return SEER_OK without work (q, o, scores may be
 * NULL) and the mask calls write empty rows.
 * Not supported with a chunk (SEER_ERR_UNSUPPORTED): seer_prefill_host, seer_gate_scores_static. */

/* Sizing helpers (pure host arithmetic; return 0 / -1 on an invalid shape). */
size_t seer_workspace_bytes(const seer_shape* shape); /* enough for any of the three calls */
size_t seer_scores_elems(const seer_shape* shape);    /* num_q_heads * sum_b nb_b^2 */
int64_t seer_mask_rows(const seer_shape* shape);      /* num_q_heads * sum_b nb_b   */
int64_t seer_causal_blocks(const seer_shape* shape);  /* num_q_heads * sum_b nb_b (nb_b + 1) / 2: capacity that always suffices */

/* 1. AttnGate (Sec. 3.1, Eq. 1): score = softmax((Pq(Q) Wq)(Pk(K) Wk)^T / sqrt(gate_dim)).
 *    Pq, Pk: average pooling over non-overlapping blocks of `block` tokens (a ragged last block averages the
 *    tokens it has).  The softmax of row i runs over the causal blocks j <= i, so each row sums to 1.
 *    Pooling, projection and the softmax are fp32; the logits are fp32-grade products of the projected vectors
 *    (each split into three bf16 terms, six tensor-core products accumulated in fp32: what is dropped is below
 *    2^-24 of the product).  Writes `scores` (layout above). */
seer_status seer_gate_scores(seer_ctx* ctx, const seer_shape* shape, const void* q, const void* k,
                             const float* Wq, const float* Wk, float* scores, void* ws, size_t ws_bytes,
                             void* stream);

/* The first half of call 1 alone (Sec. 3.1, Eq. 1: the pooling P(.) and the linear layers W): pools Q and K per block
 * and projects the pooled vectors; the result stays in `ws` (>= seer_workspace_bytes) in the library's internal
 * layout.  The bandwidth-bound stage of the gate, exported so that it can be timed on its own. */
seer_status seer_gate_project(seer_ctx* ctx, const seer_shape* shape, const void* q, const void* k,
                              const float* Wq, const float* Wk, void* ws, size_t ws_bytes, void* stream);

enum { SEER_TOPK_RATIO = 0, SEER_TOPK_COUNT = 1, SEER_THRESHOLD = 2 };
enum { SEER_FORCE_DIAG = 1u, SEER_FORCE_SINK = 2u };

typedef struct {
  int32_t mode;      /* SEER_TOPK_RATIO: keep k_i = clamp(ceil(keep_num * (i+1) / keep_den), 1, i+1) blocks in row i;
                        SEER_TOPK_COUNT: keep min(k, i+1);  SEER_THRESHOLD: keep score > threshold (strict, fp32) */
  int32_t keep_num;  /* ratio numerator   (>= 0) */
  int32_t keep_den;  /* ratio denominator (>= 1) */
  int32_t k;
  float threshold;
  uint32_t flags;    /* SEER_FORCE_DIAG keeps block i, SEER_FORCE_SINK keeps block 0, in every row.  In the TopK modes
                        forced blocks count toward k_i; the other places go to the best remaining blocks ordered by
                        (score descending, block index ascending).  NaN scores are never selected. */
  int32_t dense_tail_blocks; /* >= 0: the last dense_tail_blocks query blocks of every sequence keep all their causal
                        blocks whatever their scores ("sparsity in the context, not in the question", Sec. 4) */
} seer_mask_params;

/* 2. Binary block mask (Sec. 3.3, Eq. 3 TopK / Eq. 4 threshold) as CSR index lists.
 *    row_ptr [rows+1] and nnz_out (device int64, may be NULL) are always written in full.  col_idx receives the lists
 *    of the rows that fit entirely below col_capacity; if nnz > col_capacity the device status becomes
 *    SEER_ERR_CAPACITY and the caller may re-allocate and call again. */
seer_status seer_block_mask(seer_ctx* ctx, const seer_shape* shape, const float* scores,
                            const seer_mask_params* params, int32_t* row_ptr, int32_t* col_idx,
                            int64_t col_capacity, int64_t* nnz_out, void* ws, size_t ws_bytes, void* stream);

/* 3. Causal GQA block-sparse attention (Sec. 3.3): for every query token, softmax(scale * q k^T) v over the keys of the
 *    blocks listed for its (sequence, head, query block) row that are not later than the query.  bf16 operands, fp32
 *    accumulation and softmax, probabilities rounded to bf16 before the P V product, o written as bf16.
 *    lse (optional, may be NULL): [num_q_heads, T] fp32, natural log of the softmax denominator of the scaled logits.
 *    A row with an empty list yields o = 0 and lse = -inf.
 *    ws (optional): with a workspace of at least 256 bytes (256-byte aligned, as for the other calls) the first word
 *    becomes the counter from which the tcgen05 kernel's persistent CTAs draw their (head, query block) work items,
 *    so that a CTA that finishes early takes more of them; without one (NULL) the items are dealt statically.  The
 *    results are identical bit for bit.  Calls that may run at the same time must not share the workspace. */
seer_status seer_sparse_attn(seer_ctx* ctx, const seer_shape* shape, const void* q, const void* k, const void* v,
                             const int32_t* row_ptr, const int32_t* col_idx, void* o, float* lse, void* ws,
                             size_t ws_bytes, void* stream);

/* Max-pooled attention map on the listed blocks (Sec. 3.2, Eq. 2: the 2D max-pooling, window and stride = block, of the
 * attention map, which the paper uses as the gate's distillation target; here also a diagnostic of what the gate kept).
 * For every entry p of col_idx, belonging to row (b, h, i) and naming key block j: block_max[p] = the largest softmax
 * probability exp(scale * q_t . k_s - lse[h, t]) over the causal (t, s) pairs of that 64 x 64 tile, lse being the
 * [num_q_heads, T] output of seer_sparse_attn for the same lists (so the probabilities are those of the block-sparse
 * softmax; with full causal lists, those of dense causal attention).  A tile with no causal pair gives 0.
 * q, k, row_ptr, col_idx as for seer_sparse_attn; lse and block_max (fp32, [nnz]) are device pointers owned by the
 * caller; no workspace.  Entries outside [0, i] raise SEER_ERR_INVALID_INDEX on the device status and give 0. */
seer_status seer_attn_block_max(seer_ctx* ctx, const seer_shape* shape, const void* q, const void* k,
                                const int32_t* row_ptr, const int32_t* col_idx, const float* lse, float* block_max,
                                void* stream);

/* Selects the attention kernel used by seer_sparse_attn (and, by the same rule, the kernel of seer_attn_block_max: the
 * tcgen05 pipeline without V, or the mma.sync kernel): 0 = tcgen05 / TMEM / TMA kernel (default),
 * 1 = mma.sync kernel (on-device cross-check; also the faster one for very short lists), 2 = chosen per call from
 * the shape: the persistent tcgen05 kernel pays a few microseconds per (head, query block) row whatever its list
 * length, so batches whose rows have at most 8 causal blocks on average (many short sequences) go to the mma.sync
 * kernel and everything else to the tcgen05 kernel.  Returns SEER_ERR_INVALID_ARG for other values. */
seer_status seer_set_attn_impl(seer_ctx* ctx, int impl);

/* Test hook for the bounded waits of the tcgen05 attention kernel (no counterpart in the paper).  Every barrier
 * wait in that kernel gives up after wait_limit_us microseconds (default 2 000 000): the thread raises
 * SEER_ERR_TIMEOUT on the device status, sets a flag that every other role of its CTA polls, the CTA lets the copies
 * and MMAs in flight land, frees its tensor memory and returns; rows it had not finished are not written.
 * lose_v_copy_of_tile >= 0 makes exactly one wait run out: the first stream of CTA 0 never issues the V copy of its
 * tile with that ordinal (counted over the CTA's work items from 0), so the MMA issuer's wait for it expires;
 * nothing faults and the context stays usable.  -1 switches the hook off.  wait_limit_us = 0 is rejected. */
seer_status seer_debug_lost_wait(seer_ctx* ctx, uint32_t wait_limit_us, int32_t lose_v_copy_of_tile);

/* Synchronises `stream`, returns the device status word (SEER_OK if nothing was raised) and clears it. */
seer_status seer_poll_device_status(seer_ctx* ctx, void* stream);

/* Whole path from HOST buffers (Sec. 3.3: "Inference with SeerAttention"): for one KV head at a time (with the query heads
 * of its group: the path is independent per KV head) it copies that slice of q, k, v, Wq, Wk to the device, runs
 * seer_gate_scores -> seer_block_mask -> seer_sparse_attn on it and copies the slice of o (and of lse if lse_host is not
 * NULL) back.  The copy of slice s + 1 and the read-back of slice s - 1 run on two copy streams of the context while the
 * kernels of slice s run on `stream`; everything is ordered after the work already on `stream`, and `stream` is complete
 * only when the last read-back is.  The result is bit for bit that of the three calls on device-resident tensors.
 * Host buffers should be page-locked for the copies to be asynchronous; they must stay valid, and o_host must not be read,
 * until `stream` has been synchronised.  `arena` is a caller-owned DEVICE buffer of at least
 * seer_prefill_host_arena_bytes(shape) bytes, 256-byte aligned, that holds two sets of slice inputs / outputs and one set of
 * slice intermediates; the call allocates nothing.  col_idx inside the arena is sized for the full causal mask of a slice,
 * so SEER_ERR_CAPACITY cannot occur.  One call at a time per context. */
size_t seer_prefill_host_arena_bytes(const seer_shape* shape);
seer_status seer_prefill_host(seer_ctx* ctx, const seer_shape* shape, const void* q_host, const void* k_host,
                              const void* v_host, const float* Wq_host, const float* Wk_host,
                              const seer_mask_params* params, void* o_host, float* lse_host, void* arena,
                              size_t arena_bytes, void* stream);

/* Gate scores without any allocation (the paper has no counterpart; this is a deployment variant of call 1).
 *
 * Who needs it: code that may not allocate device memory at the point where it runs the gate -- a serving process whose
 * memory pool has handed every byte to the KV cache, a plugin that runs inside another framework's allocator and must not
 * call cudaMalloc behind its back, a latency-critical loop where cudaMalloc's implicit device synchronisation is not
 * acceptable.  Such a caller cannot create a seer_ctx (seer_create allocates) nor provide a workspace.
 *
 * What it does: the same two kernels as seer_gate_scores, same arguments and results (q, k, Wq, Wk in, scores out, all
 * DEVICE pointers owned by the caller), on the CURRENT device, without a context and without a workspace.  The
 * intermediate projected vectors and the per-batch offsets live in a fixed array inside the library image: every GPU
 * that loads the library holds SEER_STATIC_SCRATCH_BYTES + 16 KiB for it until the process exits.
 *
 * Limits: shape->batch <= SEER_STATIC_MAX_BATCH and (num_q_heads + num_kv_heads) * total_blocks * 768 bytes (rounded up to
 * 256 per tensor) <= SEER_STATIC_SCRATCH_BYTES, i.e. 10922 (head, block) pairs: e.g. 40 heads x 17000 tokens.  Larger shapes
 * return SEER_ERR_WORKSPACE and enqueue nothing.
 *
 * First call on a device: looks up the array's device address and raises one kernel's shared-memory limit (no allocation).
 * Make that first call outside of any stream capture.  The call itself performs no cudaMalloc / cudaFree and uses no
 * allocating library routine; it copies about 5 KiB of offsets from the host stack with cudaMemcpyAsync and launches.
 *
 * Sharing: all calls on a device use the same array, which keeps whatever the last call left there.  Nothing in it needs to
 * start at zero (the first kernel rewrites all that the second reads).  Two calls that overlap on the GPU -- different
 * streams without an ordering between them, or different host threads -- race on it: keep the calls of one device on one
 * stream, or order them yourself. */
#define SEER_STATIC_SCRATCH_BYTES (8u << 20)
#define SEER_STATIC_MAX_BATCH 256
seer_status seer_gate_scores_static(const seer_shape* shape, const void* q, const void* k, const float* Wq,
                                    const float* Wk, float* scores, void* stream);

/* AttnGate with the two refinements of Sec. 3.1 beyond the simplest form of Eq. 1.
 *
 * "Pooling Method Selection": Q and K may each be pooled by any non-empty subset of {average, max, min} (kernel = stride
 * = block); the pooled tensors are concatenated in the hidden dimension, in the order average, max, min, before the
 * linear layer.  The paper's best configuration is pool_q = SEER_POOL_AVG, pool_k = SEER_POOL_AVG | SEER_POOL_MAX |
 * SEER_POOL_MIN.  Wq is then [num_q_heads, nq * head_dim, gate_dim] and Wk [num_kv_heads, nk * head_dim, gate_dim], fp32,
 * row-major, nq / nk the number of methods chosen.  A ragged last block pools the tokens it has.
 *
 * "Block-level RoPE in AttnGate": with rope_theta > 0 the projected vector of block i (i local to its sequence) is
 * rotated as position i with the reduced base rope_theta / block: pairs (c, c + gate_dim/2), frequency
 * (rope_theta / block)^(-2c / gate_dim).  The gate is then meant to be fed Q and K from before the model's own RoPE;
 * the library applies no RoPE to q and k themselves.  rope_theta = 0 switches it off.
 *
 * With pool_q = pool_k = SEER_POOL_AVG and rope_theta = 0 the result is that of seer_gate_scores.  All other
 * arguments, the workspace (seer_workspace_bytes), layouts, ownership and errors are those of seer_gate_scores;
 * SEER_ERR_INVALID_ARG for an empty or unknown pooling subset or a negative / non-finite rope_theta. */
#define SEER_POOL_AVG 1u
#define SEER_POOL_MAX 2u
#define SEER_POOL_MIN 4u
typedef struct {
  uint32_t pool_q;
  uint32_t pool_k;
  float rope_theta;
} seer_gate_options;
seer_status seer_gate_scores_ex(seer_ctx* ctx, const seer_shape* shape, const seer_gate_options* options, const void* q,
                                const void* k, const float* Wq, const float* Wk, float* scores, void* ws, size_t ws_bytes,
                                void* stream);

/* Gate and block mask in one call, without the quadratic score matrix (calls 1 and 2 fused at the level of the stream;
 * Sec. 3.1 and 3.3, Eq. 1, 3, 4).
 *
 * seer_gate_scores + seer_block_mask need scores[num_q_heads * sum nb^2] in device memory: 537 MB at 131072 tokens and
 * 32 heads, 34 GB at a million tokens.  This call projects the pooled Q and K once and then walks the rows of the CSR
 * structure in bands: the scores of a band (whole sequences, else whole heads of a sequence, else runs of 64-row tiles
 * of one head) are written to a scratch buffer, the band's rows are counted, row_ptr is continued from the previous
 * band, and the band's lists are written, before the next band overwrites the scratch.  A band of up to ~100 MB stays in
 * the L2 cache, so the scores never reach DRAM.
 *
 * Results (row_ptr, col_idx, *nnz_out) are identical, bit for bit, to seer_gate_scores (options == NULL) or
 * seer_gate_scores_ex (options != NULL) followed by seer_block_mask with the same params: the same kernels compute
 * the same scores in the same order.  Arguments, layouts, ownership and errors are those of these calls.
 *
 * Workspace: DEVICE memory, 256-byte aligned, seer_gate_mask_workspace_bytes(shape, band_bytes) bytes: the projected
 * vectors (seer_workspace_bytes) followed by the band scratch.  The call uses whatever follows the projected vectors
 * as scratch, so `band_bytes` is the caller's choice; at least 64 rows of the longest sequence (64 * max nb * 4 + 16
 * bytes) are needed and the size query never returns less.  SEER_ERR_WORKSPACE if ws is smaller than that. */
size_t seer_gate_mask_workspace_bytes(const seer_shape* shape, size_t band_bytes);
seer_status seer_gate_block_mask(seer_ctx* ctx, const seer_shape* shape, const seer_gate_options* options, const void* q,
                                 const void* k, const float* Wq, const float* Wk, const seer_mask_params* params,
                                 int32_t* row_ptr, int32_t* col_idx, int64_t col_capacity, int64_t* nnz_out, void* ws,
                                 size_t ws_bytes, void* stream);

/* 128-token gate blocks (Sec. 4 evaluates 64; the kernel section mentions 128-sized tiles).
 *
 * shape->block may be 64 or 128.  With 128, seer_gate_scores / _ex / _static, seer_block_mask and seer_gate_block_mask
 * work on 128-token blocks throughout: nb = ceil(S / 128) per sequence, scores [num_q_heads, nb, nb], CSR rows and block
 * indices in units of 128 tokens, block-level RoPE with base theta / 128.  The attention kernels tile by 64 tokens, so
 * seer_sparse_attn, seer_attn_block_max and seer_prefill_host return SEER_ERR_UNSUPPORTED for block = 128; instead
 * seer_expand_block_lists rewrites the 128-token lists as 64-token lists that select exactly the same (query, key)
 * pairs, and seer_sparse_attn runs on those with the same shape at block = 64:
 *   block j -> (2j, 2j + 1); query rows 2i and 2i + 1 inherit the list of row i; in the diagonal block, row 2i takes 2i
 *   only (2i + 1 lies in its future), row 2i + 1 takes both.
 * `shape` is the 128-token shape; row_ptr / col_idx the lists seer_block_mask produced for it (DEVICE, read only);
 * row_ptr64 [num_q_heads * sum ceil(S / 64) + 1] and col_idx64 [col_capacity64] are written (DEVICE, caller-owned;
 * four times the entries of col_idx always suffice); *nnz_out (DEVICE int64, may be NULL) receives the entry count.
 * SEER_ERR_CAPACITY through the device status if col_capacity64 is too small (row_ptr64 and *nnz_out are still
 * complete).  An entry j > i is passed on as (2j, 2j + 1) and reported by the attention call. */
seer_status seer_expand_block_lists(seer_ctx* ctx, const seer_shape* shape, const int32_t* row_ptr, const int32_t* col_idx,
                                    int32_t* row_ptr64, int32_t* col_idx64, int64_t col_capacity64, int64_t* nnz_out,
                                    void* stream);

/* Diagnostics (the paper has no counterpart): when `device_buffer` is not NULL, the tcgen05 attention kernel runs in an
 * instrumented instantiation.  CTA 0 adds up the SM clocks its pipeline roles spend between marked points, on every
 * 8th tile (role r at uint64 offset r * 8192: 48 tags x (clock sum, count)); every CTA writes its wall time in ns at
 * offset 6 * 8192 + blockIdx.x and in SM clocks at 6 * 8192 + 256 + blockIdx.x.  The buffer is device memory of at
 * least 7 * 8192 * 8 bytes, zero-initialised by the caller.  NULL switches it off (default). */
seer_status seer_set_trace_buffer(seer_ctx* ctx, void* device_buffer);

/* Number of kernels the library has launched through this context since creation (for launch accounting). */
int64_t seer_launch_count(const seer_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* SEER_H_ */
