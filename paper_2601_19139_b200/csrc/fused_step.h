// Host/device interface of the persistent whole-step kernel (internal to the library).
//
// One cooperative launch runs every phase of a decode step for a dense model: embedding, then per layer the QKV
// projection, attention (qk-norm, rotary embedding, KV append, split-KV attention and its merge), the O projection,
// the gate/up projection with SiLU gating and the down projection, then the LM head with the greedy argmax.  Phases
// are separated by grid-wide barriers; weights and cached KV of later phases are prefetched across them.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace q4d {

enum FusedPhaseType { PH_EMBED = 0, PH_GEMM = 1, PH_ATTN = 2, PH_NORM = 3 };
// Phases of a layer: norm, QKV, attention, O, norm, gate/up, down.
constexpr int kFusedPhasesPerLayer = 7;
constexpr int kFusedDimKinds = 10;  // embedding, the phases of a layer, final norm, LM head

// Dimensions of one kind of phase.  Every layer has the same seven kinds, so the kernel keeps ten of these in its
// parameters (embedding, the phases of a layer, final norm, LM head) and reads only pointers from the phase table.
struct FusedDims {
  int type;    // FusedPhaseType
  int epi;     // GemmEpilogue
  int N, K;
  int ntiles;  // 16-row tiles (SiLU epilogue: 8 gate rows + the 8 matching up rows)
  int S;       // K-slices of at most 1024 input features
  int norm;    // unused
  int pad;
};

// Device pointers of one layer, by projection: 0 QKV, 1 O, 2 gate/up, 3 down.
struct FusedLayerPtrs {
  const uint32_t* qw[4];
  const uint16_t* scales[4];
  const uint16_t* biases[4];
  const uint16_t* norm[2];  // attention norm, MLP norm
  const uint16_t* q_norm;   // bf16 [128] or NULL
  const uint16_t* k_norm;
};
constexpr int kFusedMaxLayers = 96;  // the pointers travel in the kernel parameters (constant bank: no loads on the way)

struct FusedStep {
  FusedLayerPtrs layer[kFusedMaxLayers];
  const uint32_t* lm_qw;
  const uint16_t* lm_scales;
  const uint16_t* lm_biases;
  const uint16_t* final_norm;
  FusedDims dims[kFusedDimKinds];  // by kind: 0 embedding, 1..7 the phases of a layer in order, 8 final norm, 9 LM head
  int n_phases;                    // phases of a whole step: 3 + 7 * layers
  int ph_begin, ph_end;
  int n;             // active requests
  int embed_from_x;  // first phase: take x as given (sums of squares only) instead of embedding tokens
  const int32_t* tokens;  // device [n]
  const int32_t* bt;      // device [n][max_blocks]
  int max_blocks;
  int32_t lens[16];
  // attention plan: request r has ceil(blocks_r / chunk_blocks) chunks; items are (request, chunk, kv head)
  int chunk_blocks, n_items;
  int32_t item_prefix[17];
  int32_t nch[16];  // chunks per (request, kv head)
  // shape
  int H, nq, nkv, V;
  float eps;
  const float* rope;
  const uint32_t* embed_q;
  const uint16_t* embed_s;
  const uint16_t* embed_b;
  // pool
  uint16_t* pool;
  size_t layer_elems;
  // workspace
  uint16_t* x;      // residual stream bf16 [16][H]
  uint16_t* y;      // normed hidden state, operand layout (K = H)
  uint16_t* h;      // gated MLP activations, operand layout (K = mlp_inter)
  uint16_t* qkv;    // bf16 [16][(nq+2nkv)*128]
  uint16_t* attn;   // attention output, operand layout (K = nq*128)
  float* ss;        // sums of squares of x: [H/16][16]
  float* pacc;      // split-KV partial accumulators [item][128][Gs], Gs = G rounded up to even
  float* pml;       // [item][Gs][2] = (max in log2 units, sum)
  int* attn_counters;  // [16][nkv], zero between phases
  float2* amax;     // [ctas][16] (best logit, index bits)
  int32_t* next;    // [n]
  float* logits;    // [n][V] or NULL
  unsigned int* control;  // [0] barrier arrivals, [1] status (0 = ok)
  unsigned long long* timeline;  // [phases + 1] nanosecond stamps, or NULL
};

constexpr int kFusedThreads = 512;
constexpr int kFusedSliceK = 1024;

size_t fused_smem_bytes();
// Largest cooperative grid of the kernel on the current device (0 if it cannot run).
cudaError_t fused_init(int* max_ctas);
cudaError_t launch_fused_step(const FusedStep& p, int ctas, cudaStream_t s);

}  // namespace q4d
