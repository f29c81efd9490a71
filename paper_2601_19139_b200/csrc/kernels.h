// Host-side launch interface of the q4decode kernels (internal to the library).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace q4d {

constexpr int kMaxBatch = 16;
constexpr int kHeadDim = 128;
constexpr int kBlockSize = 16;

// ---- launch helper -----------------------------------------------------------------
// Launches with the programmatic-dependent-launch attribute when `pdl` is set: the kernel may start while its
// predecessor on the stream drains; every kernel of the library waits (griddepcontrol.wait) before it touches
// memory that another kernel writes.
void set_pdl_enabled(bool on);
bool pdl_enabled();

// ---- fragment-ordered GEMM operand ---------------------------------------------------
// xp bf16 [16][K] (chunks of 8 permuted), xs f32 [K/64][16] (group sums); see common.cuh.
// Three layouts of the bf16 elements exist: OPERAND_ROWS, [16][K] (the grouped projections of the MoE layers),
// OPERAND_BLOCKED, [K/8][16][8] (the tcgen05 kernel: a K-range of all requests is one contiguous block that the
// tensor core reads as 8-request x 16-byte core matrices), and OPERAND_SLICED, [K/ks][16][ks + 8] (the mma.sync
// kernels of the dense projections: a slice of ks features of all requests is one contiguous block, already padded
// like its shared-memory image).  All keep the order 0,4,1,5,2,6,3,7 inside a chunk of 8.
enum GemmPrologue { PRO_PLAIN = 0, PRO_SILU_MUL = 1 };
enum OperandLayout { OPERAND_ROWS = 0, OPERAND_BLOCKED = 1, OPERAND_SLICED = 2 };
__host__ __device__ __forceinline__ int operand_slice_features(int K) {
  const int quads = K >> 8;  // slices are the largest of 1024, 768, 512, 256 features that divides K
  for (int c = 4; c > 1; --c)
    if (quads % c == 0) return c << 8;
  return 256;
}
__host__ __device__ __forceinline__ size_t operand_elements(int layout, int K) {  // elements an operand buffer needs
  return layout == OPERAND_SLICED ? (size_t)(K / operand_slice_features(K)) * 16 * (operand_slice_features(K) + 8) : (size_t)16 * K;
}

cudaError_t launch_pack_operand(const uint16_t* x, int x_stride, int K, int n, int prologue, uint16_t* xp, float* xs,
                                int layout, cudaStream_t s);

// ---- 4-bit skinny GEMM ------------------------------------------------------------
// EPI_SILU_PACK: the tensor has 2*I rows (gate rows then up rows); the output is the operand of the next GEMM,
// h = bf16(silu(bf16(gate)) * bf16(up)), written in fragment order to out_xp [16][I] and out_xs [I/64][16].
enum GemmEpilogue { EPI_BF16 = 0, EPI_RESIDUAL = 1, EPI_F32 = 2, EPI_SILU_PACK = 3 };

struct GemmArgs {
  const uint32_t* qw;      // [N][K/8]
  const uint16_t* scales;  // [N][K/64]
  const uint16_t* biases;  // [N][K/64]
  int N, K;
  const uint16_t* xp;  // fragment-ordered operand
  const float* xs;
  int n;
  int epilogue;
  void* out;
  int out_stride;
  uint16_t* out_xp;  // EPI_SILU_PACK only
  float* out_xs;
  float2* argmax_partial;  // EPI_F32 only, optional: [row blocks][16] = (max, index as float bits) per request
  float* partial;          // split-K partial sums
  size_t partial_bytes;
  int* counters;  // zero between launches
  int counters_len;
  unsigned int* status = nullptr;  // device word set non-zero when a bounded wait inside the kernel gives up
  // grouped mode (MoE): one GEMM per slot of a device-side list of touched experts; the tensors hold
  // `N` rows per expert, stacked.  NULL expert_ids = a single GEMM.
  const int* expert_ids = nullptr;  // [max_slots]
  const int* n_touched = nullptr;   // number of valid slots
  int max_slots = 0;
  size_t xp_slot_stride = 0, xs_slot_stride = 0, out_slot_stride = 0, out_xs_slot_stride = 0;  // elements
};

// Bytes of split-K scratch a GEMM of this shape may use (upper bound over batch sizes).
size_t gemm_partial_bytes(int N, int K, int epilogue);
int gemm_counters_needed(int N);
int gemm_row_blocks(int N, int K, int n, int epilogue);  // grid.x of the launch (size of argmax_partial)
cudaError_t launch_q4_gemm(const GemmArgs& a, cudaStream_t s);
// The operand layout launch_q4_gemm expects for this call (grouped: the mixture-of-experts mode).
int gemm_operand_layout(bool grouped, int n);  // n: requests of the call

// tcgen05 kernel (q4_umma.cu): tiles of 128 rows, K in `parts` across CTAs, stages of 256 features.
struct UmmaPlan {
  int tiles, parts, ns;
  size_t partial_bytes;
};
UmmaPlan plan_umma(int N, int K, int epilogue, int sm_count);
bool umma_supported(int N, int K, int epilogue);
cudaError_t launch_q4_umma(const GemmArgs& a, int sm_count, cudaStream_t s);
cudaError_t gemm_init();  // sets the dynamic shared memory limits once per process/device
cudaError_t launch_argmax_finish(const float2* partial, int row_blocks, int n, int32_t* next, cudaStream_t s);

// ---- paged decode attention -------------------------------------------------------
struct AttnPlan {   // filled on the host from the request lengths
  int n_work;       // (request, chunk) items
  int n_slots;      // partial-result slots = n_work
  int chunk_tiles;  // tiles (16 tokens) per chunk
};
// work: int4 {request, first tile, end tile, slot}; slot_base/nchunks per request.
// wave_ctas: CTAs resident at once (attention_wave_ctas); the automatic chunk size fills one such wave.
AttnPlan plan_attention(const int32_t* lens, int n, int nkv, int chunk_tokens, int wave_ctas, int4* work,
                        int32_t* slot_base, int32_t* nchunks, int max_work);
int attention_wave_ctas(int nq, int nkv);
int attention_max_work(int max_batch, int max_positions);

struct AttnArgs {
  const uint16_t* q;  // [n][nq][128]
  const uint16_t* kpool;
  const uint16_t* vpool;  // this layer: [blocks][nkv][16][128]
  const int32_t* block_tables;
  const int32_t* lens;
  const int4* work;
  const int32_t* slot_base;
  const int32_t* nchunks;
  int n_work, n, nq, nkv, max_blocks;
  float* part_acc;  // [slots][nq][128]
  float* part_ml;   // [slots][nq][2]
  uint16_t* out;    // plain [n][nq][128], or NULL
  uint16_t* out_xp; // fragment-ordered operand [16][nq*128] of the O projection, or NULL
  float* out_xs;    // its group sums [nq*2][16]
  int out_layout = OPERAND_ROWS;  // layout of out_xp
  int* merge_counters = nullptr;  // [16][nkv], zero between launches: the attention kernel merges the chunks itself
  // The kernel requests its first K, V tiles before it waits for the preceding kernel (cached K, V do not depend on
  // it).  Set when they do (the preceding kernel appends tokens this launch reads): the launch then carries no
  // programmatic-dependent-launch attribute and starts only after the preceding kernel has completed.
  bool after_predecessor = false;
  // With qkv given (bf16 [n][(nq+2nkv)*128], the QKV projection's output) the kernel prepares q itself (qk-norm,
  // rotary embedding) and appends k, v of the new token to the pool; `q` is then unused.
  const uint16_t* qkv = nullptr;
  const uint16_t* q_norm = nullptr;  // bf16 [128] or NULL
  const uint16_t* k_norm = nullptr;
  float eps = 0.0f;
  const float* rope = nullptr;  // f32 [positions][64][2]
  uint16_t* kpool_w = nullptr;  // this layer of the pool, writable
  uint16_t* vpool_w = nullptr;
};
cudaError_t launch_paged_attention(const AttnArgs& a, cudaStream_t s);
cudaError_t launch_attention_merge(const AttnArgs& a, cudaStream_t s);
cudaError_t attention_init();

struct RopeArgs {
  const uint16_t* qkv;
  const uint16_t* q_norm;
  const uint16_t* k_norm;
  float eps;
  const float* rope;
  int n, nq, nkv;
  const int32_t* lens;
  const int32_t* block_tables;
  int max_blocks;
  uint16_t* kpool;
  uint16_t* vpool;
  uint16_t* q_out;
};
cudaError_t launch_rope_append(const RopeArgs& a, cudaStream_t s);

// ---- mixture of experts ------------------------------------------------------------
struct MoeRouteArgs {
  const uint16_t* y;       // plain normed hidden state bf16 [n][H]
  const uint16_t* router;  // bf16 [E][H]
  int H, E, top_k, norm;
  int32_t* idx;         // [16][top_k] selected experts, by decreasing logit
  float* wgt;           // [16][top_k] their weights
  int32_t* flags;       // [E], zero between launches
  int32_t* counter;     // zero between launches
  int32_t* expert_ids;  // [E] touched experts, ascending
  int32_t* slot_of;     // [E] position of an expert in expert_ids
  int32_t* n_touched;
  float* logits;           // [16][E] scratch
  int32_t* slice_counter;  // [16], zero between launches
  int32_t* touched_total = nullptr;  // optional: running sum of n_touched over the launches of a step
};
struct MoeCombineArgs {
  uint16_t* x;        // residual stream bf16 [n][H], updated in place
  const uint16_t* o;  // expert outputs bf16 [slot][16][H]
  const int32_t* idx;
  const float* wgt;
  const int32_t* slot_of;
  int H, top_k;
};
cudaError_t launch_moe_router(const MoeRouteArgs& a, int n, cudaStream_t s);
cudaError_t launch_moe_combine(const MoeCombineArgs& a, int n, cudaStream_t s);

// ---- sampling ------------------------------------------------------------------------
struct SampleArgs {  // passed to the kernel by value: the per-request settings travel with the launch
  const float* logits;  // f32 [n][vocab]
  int32_t* next;        // [n]
  int vocab;
  float temperature[kMaxBatch];  // <= 0: greedy
  int top_k[kMaxBatch];          // <= 0 or >= vocab: off
  float top_p[kMaxBatch];        // >= 1: off
  float u[kMaxBatch];            // the draw, in [0, 1)
};
cudaError_t launch_sample(const SampleArgs& a, int n, cudaStream_t s);

// ---- small kernels ----------------------------------------------------------------
cudaError_t launch_embed(const uint32_t* q, const uint16_t* scales, const uint16_t* biases, int vocab, int H,
                         const int32_t* tokens, int n, uint16_t* x, cudaStream_t s);
// y (plain, optional) and/or the fragment-ordered operand (yp, ys) of the next GEMM.
cudaError_t launch_rmsnorm(const uint16_t* x, const uint16_t* w, float eps, int n, int H, uint16_t* y,
                           uint16_t* yp, float* ys, int layout, cudaStream_t s);
cudaError_t launch_argmax(const float* logits, int n, int vocab, int32_t* next, cudaStream_t s);
cudaError_t launch_dequant(const uint32_t* q, const uint16_t* scales, const uint16_t* biases, int N, int K,
                           float* out, cudaStream_t s);
cudaError_t launch_kv_gather(const uint16_t* kpool, const uint16_t* vpool, int nkv, const int32_t* block_table,
                             int len, uint16_t* k_out, uint16_t* v_out, cudaStream_t s);

}  // namespace q4d
