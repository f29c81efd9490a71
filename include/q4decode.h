/*
 * q4decode — C ABI of the B200 decode-step library.
 *
 * One call, q4d_decode_step, is the body of the generation loop of the paper's
 * continuous-batching scheduler (Algorithm 1, generation loop): one new token
 * for every request of the active batch, from that request's own KV cache.
 * Membership of the batch changes only between steps (Algorithm 1, admission
 * and removal loops), which is what q4d_request_admit / q4d_request_release
 * express.  Models are 4-bit quantised
 * (Section 4, "Setup"); the forward pass is the pre-norm decoder of the model
 * families of Table 1.
 *
 * Conventions
 *  - Every function returns 0 (Q4D_OK) or a negative Q4D_ERR_* code.  A call
 *    that fails its host-side validation changes no state; a CUDA error in the
 *    middle of a step (Q4D_ERR_CUDA) leaves that step partially applied (K, V of
 *    the new token written for the layers that ran; request lengths not
 *    advanced).  q4d_last_error() gives the message of the calling thread's
 *    last failure.
 *  - "device" pointers are CUDA device memory owned by the caller and must
 *    outlive the object they are given to; "host" pointers are ordinary host
 *    memory read before the call returns.  The library allocates no device
 *    memory; q4d_model_create allocates pinned host staging and events.  It
 *    never frees memory it was given.
 *  - Work is enqueued on the given CUDA stream (a cudaStream_t passed as
 *    void*; NULL = the default stream) and is asynchronous unless stated.
 *  - bf16 values are passed as uint16_t bit patterns.
 *
 * 4-bit tensor format (a projection with K input and N output features):
 *    q      uint32 [N][K/8]   element k of a row sits in word k>>3, bits 4*(k&7)..+3
 *    scales bf16   [N][K/64]  one per group of 64 consecutive input features
 *    biases bf16   [N][K/64]
 *    w[j][k] = fl32(scales[j][k/64] * q[j][k] + biases[j][k/64])   (never rounded to bf16)
 *  K must be a multiple of 256.
 *
 * KV pool layout (bf16): [layer][0=K,1=V][block][kv_head][slot 0..15][128];
 * one block id names the same block in every layer.  Keys are stored after
 * the rotary embedding.
 */
#ifndef Q4DECODE_H
#define Q4DECODE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define Q4D_OK 0
#define Q4D_ERR_INVALID_ARG (-1)
#define Q4D_ERR_UNKNOWN_REQUEST (-2)
#define Q4D_ERR_DUPLICATE_REQUEST (-3)
#define Q4D_ERR_BATCH_TOO_LARGE (-4)
#define Q4D_ERR_BLOCK_TABLE_TOO_SHORT (-5)
#define Q4D_ERR_BLOCK_OUT_OF_RANGE (-6)
#define Q4D_ERR_POSITION_OVERFLOW (-7)
#define Q4D_ERR_WORKSPACE_TOO_SMALL (-8)
#define Q4D_ERR_CUDA (-9)
#define Q4D_ERR_TIMEOUT (-10)
#define Q4D_ERR_UNSUPPORTED (-11)

#define Q4D_MAX_BATCH 16
#define Q4D_BLOCK_SIZE 16
#define Q4D_HEAD_DIM 128

/* Shape of the model (plain data). */
typedef struct {
  int32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim; /* head_dim must be 128 */
  int32_t mlp_inter, vocab;
  int32_t group_size /* 64 */, bits /* 4 */;
  int32_t qk_norm /* 0|1: per-head RMSNorm of q and k before the rotary embedding */;
  int32_t tie_embeddings /* informational: embed and lm_head may alias */;
  float rms_eps;
  int32_t n_experts /* 0 = dense MLP */, top_k, expert_inter, norm_topk_prob;
  int32_t max_batch /* <= 16 */, max_positions /* rows of the rotary table */;
} q4d_shape;

/* One 4-bit tensor: three device pointers (format above). */
typedef struct {
  const uint32_t* q;
  const uint16_t* scales;
  const uint16_t* biases;
} q4d_qtensor;

/* Per-layer device pointers.  Norm weights are bf16 vectors. */
typedef struct {
  const uint16_t *attn_norm, *mlp_norm; /* [hidden] */
  const uint16_t *q_norm, *k_norm;      /* [128], NULL unless qk_norm */
  q4d_qtensor wqkv;      /* [(nq+2nkv)*128][hidden], rows: q heads, k heads, v heads */
  q4d_qtensor wo;        /* [hidden][nq*128] */
  q4d_qtensor w_gate_up; /* [2*mlp_inter][hidden], rows: gate then up (dense only) */
  q4d_qtensor w_down;    /* [hidden][mlp_inter] (dense only) */
  const uint16_t* router;      /* bf16 [n_experts][hidden] (MoE only) */
  q4d_qtensor experts_gate_up; /* [n_experts][2*expert_inter][hidden] stacked (MoE only) */
  q4d_qtensor experts_down;    /* [n_experts][hidden][expert_inter] stacked (MoE only) */
} q4d_layer_weights;

typedef struct {
  const q4d_layer_weights* layers; /* host array of n_layers entries (copied by model_create) */
  const uint16_t* final_norm;      /* bf16 [hidden] */
  q4d_qtensor embed;               /* [vocab][hidden] */
  q4d_qtensor lm_head;             /* [vocab][hidden] */
  const float* rope_cos_sin;       /* f32 [max_positions][64][2] = (cos, sin) of position * frequency_i */
} q4d_weights;

typedef struct q4d_model q4d_model;
typedef struct q4d_kv_pool q4d_kv_pool;

const char* q4d_last_error(void);

/* ---- model -------------------------------------------------------------- */

/* Bytes of device workspace q4d_model_create needs for this shape (activations,
 * split-K and split-KV partial sums, per-step metadata).  0 if the shape is
 * not supported. */
size_t q4d_model_workspace_bytes(const q4d_shape* shape);

/* Binds a shape to its weights ("model_create(shape config, device weight
 * pointers)").  `weights` is a host struct of device pointers; the per-layer
 * array is copied, the tensors are not.  `workspace` is device memory of at
 * least q4d_model_workspace_bytes(shape), 256-byte aligned, used exclusively by
 * this model until it is destroyed.  Errors: INVALID_ARG (NULL pointer,
 * missing tensor), UNSUPPORTED (head_dim != 128, group_size != 64, bits != 4,
 * widths not multiples of 256, more than 16 q heads per kv head, max_batch
 * > 16), WORKSPACE_TOO_SMALL, CUDA. */
int q4d_model_create(const q4d_shape* shape, const q4d_weights* weights, void* workspace,
                     size_t workspace_bytes, q4d_model** out);
int q4d_model_destroy(q4d_model* model);

/* ---- paged KV pool and batch membership ------------------------------- */

size_t q4d_kv_pool_bytes(const q4d_shape* shape, int32_t num_blocks, int32_t block_size);

/* Wraps caller-owned device memory (layout in the file header) as the block
 * pool of `model` ("kv_pool_create(blocks, block_size)").  block_size must be
 * 16.  The caller allocates blocks to requests and fills prefilled KV; the
 * library only reads the blocks named in block tables and appends one token
 * per step. */
int q4d_kv_pool_create(q4d_model* model, int32_t num_blocks, int32_t block_size, void* pool_mem,
                       size_t pool_bytes, q4d_kv_pool** out);
int q4d_kv_pool_destroy(q4d_kv_pool* pool);

/* A request joins the batch between steps (Algorithm 1, admission loop).  Its
 * first `prefilled_len` tokens already have K, V in the caller's blocks.
 * Errors: DUPLICATE_REQUEST, POSITION_OVERFLOW (prefilled_len < 0 or
 * >= max_positions). */
int q4d_request_admit(q4d_kv_pool* pool, int64_t request_id, int32_t prefilled_len);
/* A request leaves the batch between steps (Algorithm 1, removal loop). */
int q4d_request_release(q4d_kv_pool* pool, int64_t request_id);
/* Tokens cached so far for a request. */
int q4d_request_len(q4d_kv_pool* pool, int64_t request_id, int32_t* len_out);
/* Number of admitted requests. */
int q4d_request_count(q4d_kv_pool* pool, int32_t* count_out);

/* ---- the decode step ---------------------------------------------------- */

/* One token for each of the n listed requests (Algorithm 1, generation loop).
 *   request_ids   host  [n]   distinct, all admitted
 *   last_tokens   host  [n]   the token each request feeds in (0 <= t < vocab)
 *   block_tables  host  [n][max_blocks]  physical block of tokens 16*i..16*i+15;
 *                 row r must cover len_r + 1 tokens; the block receiving the
 *                 new token must not be shared with another request
 *   next_tokens   device [n]  greedy token (argmax of the logits, lowest index on ties)
 *   logits        device [n][vocab] f32, or NULL
 * Outputs are in the order of request_ids.  On success each listed request's
 * length grows by one; n = 0 is a no-op.  The call validates everything on
 * the host first (UNKNOWN_REQUEST, DUPLICATE_REQUEST, BATCH_TOO_LARGE,
 * BLOCK_TABLE_TOO_SHORT, BLOCK_OUT_OF_RANGE, POSITION_OVERFLOW, INVALID_ARG),
 * then enqueues the kernels and returns without synchronising. */
int q4d_decode_step(q4d_model* model, q4d_kv_pool* pool, int32_t n, const int64_t* request_ids,
                    const int32_t* last_tokens, const int32_t* block_tables, int32_t max_blocks,
                    int32_t* next_tokens, float* logits, void* cuda_stream);

/* Prompt processing for one request (Section 3.2, "Text Prefix Caching": the forward pass over the prompt, which a
 * cache hit skips for the cached tokens and resumes after them; Table 7 measures its latency as time to first
 * token).  Computes K, V of tokens[start_pos .. n_tokens) at their positions, writes them into the request's blocks,
 * and returns the greedy token that follows the prompt.  tokens and block_table are host arrays (block_table[i]
 * holds tokens 16 i .. 16 i + 15 and must cover n_tokens; the blocks of positions < start_pos already hold their
 * K, V, e.g. from q4d_prefix_lookup; a partly cached block that receives new tokens must be the request's own).
 * next_token (device, 1 value) and logits (device f32 [vocab]) may be NULL.  The result is, by definition, what
 * n_tokens - start_pos decode steps feeding the prompt's tokens one by one would leave behind; the library gets
 * there sixteen tokens at a time (one pass over the weights per sixteen tokens, each token attending to the cached
 * ones and to the earlier tokens of its chunk).  On success the request is admitted with n_tokens cached tokens.
 * Errors: DUPLICATE_REQUEST (already admitted), POSITION_OVERFLOW, BLOCK_TABLE_TOO_SHORT, BLOCK_OUT_OF_RANGE,
 * INVALID_ARG (start_pos outside [0, n_tokens): to reuse a fully cached prompt pass start_pos = n_tokens - 1). */
int q4d_prefill(q4d_model* model, q4d_kv_pool* pool, int64_t request_id, const int32_t* tokens, int32_t n_tokens,
                int32_t start_pos, const int32_t* block_table, int32_t max_blocks, int32_t* next_token, float* logits,
                void* cuda_stream);

/* Per-request sampling settings of one step (host arrays of n entries each, read before the call returns).  The
 * paper's scheduler only says that a token is generated per request (Algorithm 1, generation loop) and is silent on
 * how it is chosen; this is the usual temperature / top-k / top-p rule with the random draw supplied by the caller,
 * so that a run is reproducible from its seed:
 *   temperature <= 0 : the greedy token (largest logit, lowest index among equals); the other fields are ignored
 *   otherwise        : integer weights w_j = rint(2^40 exp((l_j - max l) / temperature));
 *                      top_k in 1..vocab-1 keeps the tokens whose logit is >= the k-th largest (ties at the cut
 *                      stay), any other value keeps all; top_p < 1 then keeps { l_j >= c } for the largest c whose
 *                      set holds at least ceil(top_p * kept weight); with W the weight kept and t = floor(u * W)
 *                      (u in [0, 1)), the tokens are walked by descending logit, ascending index among equal
 *                      logits, and the first whose running weight exceeds t is the result. */
typedef struct {
  const float* temperature;
  const int32_t* top_k;
  const float* top_p;
  const float* u;
} q4d_sampling;

/* q4d_decode_step whose next_tokens are drawn by the rule above from the step's logits instead of the argmax. */
int q4d_decode_step_sampled(q4d_model* model, q4d_kv_pool* pool, int32_t n, const int64_t* request_ids,
                            const int32_t* last_tokens, const int32_t* block_tables, int32_t max_blocks,
                            const q4d_sampling* sampling, int32_t* next_tokens, float* logits, void* cuda_stream);

/* Same step, but the fed-in tokens are read from device memory when the
 * kernels run (e.g. the next_tokens buffer of the previous step), so a loop
 * of steps needs no host round trip.  Token values are then not validated on
 * the host; out-of-range values are clamped into the vocabulary. */
int q4d_decode_step_chained(q4d_model* model, q4d_kv_pool* pool, int32_t n, const int64_t* request_ids,
                            const int32_t* last_tokens_device, const int32_t* block_tables,
                            int32_t max_blocks, int32_t* next_tokens, float* logits,
                            void* cuda_stream);

/* Same step with host outputs: next_tokens_host [n] and, if not NULL,
 * logits_host [n][vocab] are filled and the stream is synchronised before the
 * call returns. */
int q4d_decode_step_host(q4d_model* model, q4d_kv_pool* pool, int32_t n, const int64_t* request_ids,
                         const int32_t* last_tokens, const int32_t* block_tables, int32_t max_blocks,
                         int32_t* next_tokens_host, float* logits_host, void* cuda_stream);

/* ---- caches of the serving loop (host side) ------------------------------ */

/* SHA-256 (FIPS 180-4) of a byte string, the hash both caches key on (Algorithm 2, Algorithm 3). */
int q4d_sha256(const void* data, size_t bytes, uint8_t* out32);

/* Text prefix cache (Algorithm 2, "Text Prefix Cache Lookup"; Section 3.2 "Text Prefix Caching").  The KV state of
 * a prompt prefix is a list of 16-token blocks of the caller's pool; the cache stores one entry per block-aligned
 * prefix, keyed by SHA-256(key of the prefix one block shorter || the block's 16 int32 token ids), so a lookup costs
 * one hash per block and finds exactly the prefixes Algorithm 2 finds when it tries every prefix length from |P|
 * down to 1: the longest cached one.  Entries are evicted least-recently-used first within a byte budget (Section
 * 3.3, "Memory Management": 512 MB by default), never while a request reads them and never before the longer
 * prefixes that build on them.  The cache owns no device memory: it deals in block ids.
 *   capacity_bytes   0 = 512 MiB
 *   bytes_per_block  what one block costs in the pool (all layers, K and V): q4d_kv_pool_bytes(shape, 1, 16) */
typedef struct q4d_prefix_cache q4d_prefix_cache;
int q4d_prefix_cache_create(size_t capacity_bytes, size_t bytes_per_block, q4d_prefix_cache** out);
int q4d_prefix_cache_destroy(q4d_prefix_cache* cache);
/* Longest cached prefix of the prompt (host tokens): its blocks (blocks_out) and one handle per block (handles_out),
 * both [max_blocks]; *n_hit_blocks of them are filled, and generation resumes at position 16 * *n_hit_blocks
 * (Algorithm 2's "start position"; 0 = miss).  The returned blocks are read-only for the caller and stay pinned
 * until their handles are released. */
int q4d_prefix_lookup(q4d_prefix_cache* cache, const int32_t* tokens, int32_t n_tokens, int32_t max_blocks,
                      int32_t* blocks_out, int32_t* handles_out, int32_t* n_hit_blocks);
/* After the prompt's KV is in the pool: offers the first n_blocks full blocks of the request's block table.  For
 * block i, adopted_out[i] = 1 if the cache now (or already) holds exactly this block for this prefix (the caller
 * must not free it while it is cached), 0 if the prefix was cached before with another block (the caller's block
 * stays its own); handles_out[i] is a new pinned handle for blocks the call added, -1 otherwise. */
int q4d_prefix_insert(q4d_prefix_cache* cache, const int32_t* tokens, int32_t n_tokens, const int32_t* block_table,
                      int32_t n_blocks, int32_t* handles_out, int32_t* adopted_out);
/* A request stops reading: its handles (negative ones are skipped) are unpinned. */
int q4d_prefix_release(q4d_prefix_cache* cache, const int32_t* handles, int32_t n);
/* Evicts least-recently-used unpinned leaf entries until the cache is within its budget and at least bytes_to_free
 * bytes are gone (or nothing evictable is left, or max_out entries were evicted); the blocks given up are returned
 * for the caller's allocator. */
int q4d_prefix_evict(q4d_prefix_cache* cache, size_t bytes_to_free, int32_t max_out, int32_t* freed_blocks,
                     int32_t* n_freed);
int q4d_prefix_cache_stats(q4d_prefix_cache* cache, int64_t* entries, int64_t* bytes, int64_t* lookups,
                           int64_t* hit_blocks);

/* Content-hash store of the multimodal path (Algorithm 3, "Cache-Aware Multimodal Generation"; Section 3.3).  An
 * image is identified by the SHA-256 of its decoded pixel bytes, whatever form it arrived in; an entry keeps what
 * Algorithm 3 stores for reuse: the vision embeddings (a caller-owned device buffer) and the KV state (blocks of
 * the pool).  The vision encoder itself is outside this library.  LRU eviction within a byte budget (0 = 512 MiB),
 * never of an entry a request is using. */
typedef struct {
  uint8_t hash[32];   /* SHA-256 of the pixel bytes (filled by q4d_content_lookup) */
  void* embeddings;   /* device buffer with the vision embeddings, owned by the caller */
  int64_t bytes;      /* bytes the entry accounts for (embeddings + its KV blocks) */
  int32_t n_tokens;   /* tokens of KV state stored with it */
  int32_t n_blocks;   /* blocks of the pool holding that KV state */
} q4d_content_entry;
typedef struct q4d_content_cache q4d_content_cache;
int q4d_content_cache_create(size_t capacity_bytes, q4d_content_cache** out);
int q4d_content_cache_destroy(q4d_content_cache* cache);
/* Hashes the pixels and looks the hash up.  *hit = 1: entry_out and blocks_out[0..n_blocks) hold the stored
 * embeddings and KV state (skip the vision encoder and the prompt processing for this image) and the entry is
 * pinned until q4d_content_release; *hit = 0: only entry_out->hash is filled, to be completed and stored. */
int q4d_content_lookup(q4d_content_cache* cache, const void* pixels, size_t pixel_bytes, q4d_content_entry* entry_out,
                       int32_t max_blocks, int32_t* blocks_out, int32_t* hit);
/* Stores an entry after a miss (Algorithm 3, last step); it starts pinned by the storing request.
 * DUPLICATE_REQUEST if the hash is present. */
int q4d_content_store(q4d_content_cache* cache, const q4d_content_entry* entry, const int32_t* blocks);
int q4d_content_release(q4d_content_cache* cache, const uint8_t* hash32);
/* Evicts the least-recently-used unpinned entry if the store is over its budget or bytes_to_free > 0; *did_evict
 * says whether one went, and evicted_out / blocks_out name what the caller may now free.  Call until *did_evict = 0. */
int q4d_content_evict(q4d_content_cache* cache, size_t bytes_to_free, q4d_content_entry* evicted_out,
                      int32_t max_blocks, int32_t* blocks_out, int32_t* did_evict);
int q4d_content_cache_stats(q4d_content_cache* cache, int64_t* entries, int64_t* bytes);

/* ---- instrumentation ---------------------------------------------------- */

/* Kernel classes timed by the profile mode. */
enum {
  Q4D_K_EMBED = 0, Q4D_K_RMSNORM, Q4D_K_GEMM_QKV, Q4D_K_ROPE_APPEND, Q4D_K_ATTENTION,
  Q4D_K_ATTN_MERGE, Q4D_K_GEMM_O, Q4D_K_GEMM_GATE_UP, Q4D_K_GEMM_DOWN, Q4D_K_MOE_ROUTER,
  Q4D_K_MOE_GATE_UP, Q4D_K_MOE_DOWN, Q4D_K_LM_HEAD, Q4D_K_ARGMAX, Q4D_K_FUSED_STEP, Q4D_K_COUNT
};
/* With profiling on, every kernel launch of a step is bracketed by CUDA events
 * on the step's stream.  q4d_profile_read synchronises, adds up the elapsed
 * milliseconds and launches per class since the last read into ms[Q4D_K_COUNT]
 * and launches[Q4D_K_COUNT] (host arrays), and clears the record. */
int q4d_profile_enable(q4d_model* model, int32_t on);
int q4d_profile_read(q4d_model* model, float* ms, int32_t* launches);
/* Kernel launches enqueued by this model since creation. */
int64_t q4d_launch_count(q4d_model* model);
/* 1 if the model runs a step as one persistent kernel (every phase of the step in one cooperative launch,
 * class Q4D_K_FUSED_STEP in the profile), 0 if it launches one kernel per operation (the default).  The
 * persistent kernel is chosen by the environment variable Q4D_STEP_KERNEL=fused at model creation and is
 * available for dense models with at most 8 query heads per kv head and at most 96 layers. */
int q4d_step_is_fused(q4d_model* model);
/* Phase timeline of the persistent kernel.  While enabled, the kernel stamps the nanosecond clock after
 * every grid barrier.  q4d_timeline_read synchronises the device and adds up, for the most recent step,
 * the microseconds and the number of phases per class into us[Q4D_K_COUNT], phases[Q4D_K_COUNT] (host
 * arrays); a phase is filed under the class of the kernel it replaces (attention includes qk-norm, rotary
 * embedding, append and merge; projections include the RMSNorm they read through; the LM head includes the
 * argmax).  All zeros for a model that is not fused. */
int q4d_timeline_enable(q4d_model* model, int32_t on);
int q4d_timeline_read(q4d_model* model, float* us, int32_t* phases);
/* Bytes the most recent step copied host -> device (per-step metadata: tokens,
 * lengths, block tables, attention work list) and device -> host (only the
 * host-output variant copies anything back). */
int q4d_step_io_bytes(q4d_model* model, int64_t* h2d_bytes, int64_t* d2h_bytes);
/* Mixture-of-experts models: the number of (layer, expert) pairs the most recent step routed at least one request
 * to, i.e. the expert tensors it actually streamed (the grouped dequant-GEMM runs over the experts touched per
 * step).  Synchronises the device.  0 for dense models. */
int q4d_moe_touched_experts(q4d_model* model, int64_t* total);

/* ---- single operations (the kernels of the step, callable alone) -------- */
/* All pointers are device memory; n <= 16.  `scratch` is device memory of at
 * least q4d_op_scratch_bytes() bytes, zero-initialised once by the caller and
 * owned by one stream at a time. */
size_t q4d_op_scratch_bytes(void);

/* y[r][j] = sum_k w[j][k] x[r][k] with w dequantised on the fly.
 *   prologue 0: x is bf16 [n][K] (row stride x_stride elements)
 *   prologue 1: x is bf16 [n][2K] = gate | up; the operand is bf16(silu(gate) * up)
 *   epilogue 0: out bf16 [n][N] = bf16(y)
 *   epilogue 1: out bf16 [n][N] updated in place: out = bf16(out + bf16(y))   (residual)
 *   epilogue 2: out f32  [n][N] = y
 * out_stride is the element distance between requests in out. */
int q4d_q4_gemm(const q4d_qtensor* w, int32_t N, int32_t K, const uint16_t* x, int32_t x_stride,
                int32_t n, int32_t prologue, int32_t epilogue, void* out, int32_t out_stride,
                void* scratch, void* cuda_stream);

/* The same projection for callers that may not allocate device memory at all (the paper has no
 * counterpart; this is a deployment convenience).  Typical users: a plugin running inside a host
 * process that has given all device memory to its own arena, code called from an allocator or
 * memory-pool callback, or a serving loop where cudaMalloc is banned because it synchronises the
 * device.  Arguments and results are those of q4d_q4_gemm without `scratch`: the split-K scratch is
 * a fixed array inside the library (q4d_noalloc_max_scratch_bytes() = 8 MiB of partial sums, plus
 * 4096 row-tile counters and 0.6 MiB in which the activations are rearranged for the kernel) that
 * every GPU holds from the moment the library is loaded until the process exits.  The call allocates
 * and frees nothing.
 *  - Projections whose split-K partial sums exceed the array, or with K > 16384, are refused with
 *    WORKSPACE_TOO_SMALL (for example a 69632 x 8192 projection); use q4d_q4_gemm then.
 *  - The first call on each device looks up the array's device address; make that first call
 *    outside any stream capture, with the device current.  The kernels' shared-memory limits are set
 *    once per process, on the device that is current at the first projection call: use one device per
 *    process.
 *  - The call returns once the work is enqueued.  Should a bounded wait inside the kernel give up (a
 *    copy that never lands), the results are void and nothing reports it here; the step entry points,
 *    which own a status word, do report it.
 *  - Every call reuses the same array and finds in it what the previous call left; the counters are
 *    cleared on the stream before each launch.  Calls whose kernels can overlap on the GPU (different
 *    streams without an ordering between them) race on the array: keep them on one stream or order
 *    them with events. */
int q4d_q4_gemm_noalloc(const q4d_qtensor* w, int32_t N, int32_t K, const uint16_t* x, int32_t x_stride,
                        int32_t n, int32_t prologue, int32_t epilogue, void* out, int32_t out_stride,
                        void* cuda_stream);
size_t q4d_noalloc_max_scratch_bytes(void);

/* y = bf16(x * rsqrt(mean(x^2) + eps) * w), rows of length H. */
int q4d_rmsnorm(const uint16_t* x, const uint16_t* w, float eps, int32_t n, int32_t H, uint16_t* y,
                void* cuda_stream);

/* x[r] = bf16(dequantised row tokens[r] of the table). */
int q4d_embed(const q4d_qtensor* table, int32_t vocab, int32_t H, const int32_t* tokens, int32_t n,
              uint16_t* x, void* cuda_stream);

/* Per-head RMSNorm (if q_norm/k_norm given) and rotary embedding of q and k at
 * position lens[r]; q goes to q_out bf16 [n][nq][128]; k and v are appended to
 * the pool at token slot lens[r].  qkv is bf16 [n][(nq+2nkv)*128]. */
int q4d_rope_append(const uint16_t* qkv, const uint16_t* q_norm, const uint16_t* k_norm, float eps,
                    const float* rope_cos_sin, int32_t n, int32_t nq, int32_t nkv, const int32_t* lens,
                    const int32_t* block_tables, int32_t max_blocks, uint16_t* pool_layer_k,
                    uint16_t* pool_layer_v, uint16_t* q_out, void* cuda_stream);

/* Decode attention of q bf16 [n][nq][128] over tokens 0..lens[r] of each
 * request in one layer of the pool (split over the KV length, partial results
 * merged by log-sum-exp).  The lengths are given twice: the host copy plans
 * the split, the device copy is read by the kernels.  out bf16 [n][nq][128].
 * The call synchronises the stream before it returns. */
int q4d_paged_attention(const uint16_t* q, const uint16_t* pool_layer_k, const uint16_t* pool_layer_v,
                        int32_t n, int32_t nq, int32_t nkv, const int32_t* lens_host,
                        const int32_t* lens_device, const int32_t* block_tables_device,
                        int32_t max_blocks, int32_t chunk_tokens /* 0 = auto */, uint16_t* out,
                        void* scratch, void* cuda_stream);

/* next[r] drawn from logits f32 [n][vocab] (device) by the rule of q4d_sampling (host arrays). */
int q4d_sample(const float* logits, int32_t n, int32_t vocab, const q4d_sampling* sampling, int32_t* next,
               void* cuda_stream);

/* next[r] = argmax_j logits[r][j], lowest index on ties. */
int q4d_argmax(const float* logits, int32_t n, int32_t vocab, int32_t* next, void* cuda_stream);

/* ---- parity exports ----------------------------------------------------- */

/* Layers [layer_begin, layer_end) of the step, exactly as q4d_decode_step launches them (including the append of
 * K, V at each request's current length), starting from the hidden state x_in bf16 [n][hidden] (device) and
 * returning the hidden state after the last of them in x_out.  Request lengths do not change.  Used to compare
 * single layers of the production path with the oracle from identical inputs. */
int q4d_debug_run_layers(q4d_model* model, q4d_kv_pool* pool, int32_t n, const int64_t* request_ids,
                         const int32_t* block_tables, int32_t max_blocks, int32_t layer_begin, int32_t layer_end,
                         const uint16_t* x_in_device, uint16_t* x_out_device, void* cuda_stream);

/* Writes `value` into the device word in which the step's kernels report a bounded wait that gave up (a bulk copy
 * that never landed, a grid barrier that never completed).  The kernels only ever set it from inside such a wait;
 * this export lets a test exercise the host side of the report without making any wait on the GPU run out: after a
 * non-zero value the next step still runs and reads the word back, the step after it returns Q4D_ERR_TIMEOUT, and
 * so does every later step of this model (its results are void: destroy and re-create it). */
int q4d_debug_set_status(q4d_model* model, uint32_t value);

/* out f32 [N][K] = the dequantised weights (bit-exact definition above). */
int q4d_debug_dequant(const q4d_qtensor* w, int32_t N, int32_t K, float* out_device, void* cuda_stream);
/* Tokens 0..len-1 of one layer of the pool, gathered through a device block
 * table into k_out, v_out bf16 [len][n_kv_heads][128]. */
int q4d_debug_kv_gather(q4d_kv_pool* pool, int32_t layer, const int32_t* block_table_device,
                        int32_t len, uint16_t* k_out, uint16_t* v_out, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* Q4DECODE_H */
