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

// One phase of the step.  The table is built once per model and lives in device memory.
struct alignas(128) FusedPhase {
  int type;    // FusedPhaseType
  int epi;     // PH_GEMM: GemmEpilogue
  int N, K;    // PH_GEMM: output and input features
  int ntiles;  // PH_GEMM: 16-row tiles (SiLU epilogue: 8 gate rows + the 8 matching up rows)
  int S;       // PH_GEMM: K-slices of at most 1024 input features (the activations are staged slice by slice)
  int norm;    // unused
  int layer;   // PH_ATTN: layer of the pool
  const uint32_t* qw;
  const uint16_t* scales;
  const uint16_t* biases;
  const uint16_t* in;      // PH_GEMM: operand bf16 [16][K], chunks of 8 in fragment order; PH_NORM: x, plain
  const uint16_t* norm_w;  // PH_NORM: bf16 [K]
  void* out;               // PH_GEMM: output (bf16 [16][out_stride]; ignored for the f32 epilogue); PH_NORM: operand
  const uint16_t* q_norm;  // PH_ATTN: bf16 [128] or NULL
  const uint16_t* k_norm;
  int out_stride;
  int cls;                 // timeline class (Q4D_K_* of the unfused kernel this phase replaces)
};

struct FusedStep {
  const FusedPhase* phases;
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
  uint16_t* qkv;    // bf16 [16][(nq+2nkv)*128]
  uint16_t* attn;   // attention output bf16 [16][nq*128], chunks of 8 in fragment order (operand of the O projection)
  float* ss;        // sums of squares of x: [H/16][16]
  float* pacc;      // split-KV partial accumulators [item][G][128]
  float* pml;       // [item][G][2] = (max in log2 units, sum)
  int* attn_counters;  // [16][nkv], zero between phases
  float2* amax;     // [ctas][16] (best logit, index bits)
  int32_t* next;    // [n]
  float* logits;    // [n][V] or NULL
  unsigned int* control;  // [0] barrier arrivals, [1] status (0 = ok)
  unsigned long long* timeline;  // [phases + 1] nanosecond stamps, or NULL
};

constexpr int kFusedThreads = 256;
constexpr int kFusedSliceK = 1024;

size_t fused_smem_bytes();
// Largest cooperative grid of the kernel on the current device (0 if it cannot run).
cudaError_t fused_init(int* max_ctas);
cudaError_t launch_fused_step(const FusedStep& p, int ctas, cudaStream_t s);

}  // namespace q4d
