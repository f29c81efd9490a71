// The persistent whole-step kernel: one cooperative launch per decode step.
//
// The grid has one CTA of eight warps per SM.  A step is a list of phases (embedding; per layer QKV projection,
// attention, O projection, gate/up projection, down projection; LM head) separated by grid-wide barriers.  Every
// warp owns a ring of shared-memory slots that it fills itself with cp.async and consumes in order; the stream of
// slots runs through the whole step, so while a warp finishes a phase and waits at the barrier, the packed weights
// (and the cached K, V blocks) of its first stages of the next phases are already on their way from HBM.  Nothing a
// warp prefetches is produced inside the step, except the pool slot of the token being appended, which the
// attention code overwrites in shared memory with the freshly computed k, v.
//
// Projections.  The 16-row tiles of the tensor are dealt to the CTAs in contiguous ranges.  A CTA works through its
// tiles in groups of up to eight; within a group every warp owns one tile (or a half or a quarter of the K range
// of one when the group has fewer tiles than the CTA has warps) and keeps its accumulators in registers while the
// CTA walks the K range slice by slice (1024 input features): the activations of the next slice are fetched into
// registers during the multiplication of the current one, normalised (RMSNorm), permuted into MMA fragment order
// and stored to the other of two shared-memory buffers with their group sums.  A warp's stage is 16 rows x 256
// input features of packed codes with their scales and biases; it multiplies with mma.sync on the exact integers
// 16 + q (see q4_gemm.cu for the arithmetic).  Warps that share a tile add their sums in shared memory in a fixed
// order.  No partial sum leaves the SM, so a projection costs no global synchronisation besides the phase barrier.
// The epilogues write plain bf16 activations (with the residual add and the per-tile sums of squares the next
// RMSNorm needs, or SiLU gating), or fp32 logits with a running argmax.
//
// Attention.  An item is (request, kv head, chunk of 16-token blocks); a warp prepares q for the G query heads of
// the kv head (qk-norm, rotary embedding), the warp with the request's last chunk also prepares and appends k, v,
// and each block streams through four ring slots (two 8-token halves of K, two of V).  The warp that finishes the
// last chunk of a (request, kv head) merges the chunks' partial results in chunk order.
//
// Every wait in the kernel is bounded: a barrier that does not complete within two seconds sets the status word
// and all CTAs leave.
#include <math.h>

#include "common.cuh"
#include "fused_step.h"
#include "kernels.h"

namespace q4d {

namespace {

constexpr int kWarps = kFusedThreads / 32;
constexpr int kDepth = 4;             // ring slots per warp (power of two)
constexpr int kSlot = 2304;           // 16 rows x 128 B of codes (16-byte chunks XOR-swizzled) + 16 x (4 scales + 4 biases)
constexpr int kSlotSb = 2048;         // offset of the scales/biases inside a slot
constexpr int kActRows = 16 * 2 * kFusedSliceK;     // bytes of a staged slice: 16 request rows, swizzled, no padding
constexpr int kActBytes = kActRows + (kFusedSliceK / 64) * 16 * 4;  // rows + group sums
constexpr int kRingBytes = kWarps * kDepth * kSlot;
constexpr int kPartFloats = (kWarps - 2) * 256;  // accumulators of the warps that share a tile with a lead warp
constexpr int kMiscFloats = 32 + 2 * kWarps * 16;  // reduction scratch, argmax values, argmax indices
constexpr size_t kSmemBytes = (size_t)kRingBytes + 2 * kActBytes + (kPartFloats + kMiscFloats) * 4;
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t v) {
  uint32_t r;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(r) : "r"(v));
  return r;
}

constexpr float kScaleLog2 = 0.08838834764831845f * 1.4426950408889634f;  // log2(e) / sqrt(128)
constexpr unsigned long long kBarrierTimeoutNs = 2000000000ull;

static_assert((kDepth & (kDepth - 1)) == 0, "ring depth must be a power of two");
static_assert(kDepth >= 4, "an attention block occupies four slots");
static_assert(kFusedThreads == kWarps * 32, "thread count");
static_assert(kSmemBytes <= 227 * 1024 - 256, "shared memory");

__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ unsigned int ld_relaxed_u32(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_add_u32(unsigned int* p, unsigned int v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ int atom_acq_rel_add_s32(int* p, int v) {
  int old;
  asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
  return old;
}

// ---- mbarrier + 1-D bulk copy (global -> shared), used to stage the activations
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_copy_g2s(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(smem_dst)),
               "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
// Waits for the phase with the given parity to complete; gives up (false) after a bounded number of tries.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  for (int tries = 0; tries < (1 << 17); ++tries) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    if (done) return true;
  }
  return false;
}

__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c) {  // (a & b) | c
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
// bf16x2 registers {16 + code j, 16 + code j + 4}, j = 0..3, of one packed word (exact in bf16).
__device__ __forceinline__ void unpack_word(uint32_t w, uint32_t (&p)[4]) {
  const uint32_t kMask = 0x00780078u, kSixteen = 0x41804180u;
  p[0] = and_or(w << 3, kMask, kSixteen);
  p[1] = and_or(w >> 1, kMask, kSixteen);
  p[2] = and_or(w >> 5, kMask, kSixteen);
  p[3] = and_or(w >> 9, kMask, kSixteen);
}
__device__ __forceinline__ float bf16_at(const uint2& v, int i) {
  const uint32_t w = (i >> 1) ? v.y : v.x;
  return (i & 1) ? bf16_hi(w) : bf16_lo(w);
}
__device__ __forceinline__ float bf16_round(float v) { return bf16_to_f32(f32_to_bf16(v)); }

// Row of the tensor behind local row i of a tile.  SiLU tiles pair 8 gate rows with the 8 up rows of the same
// columns of h; other tiles are 16 consecutive rows (clamped at the ragged end, masked when stored).
__device__ __forceinline__ int unit_row(int epi, int N, int tile, int i) {
  if (epi == EPI_SILU_PACK) return i < 8 ? tile * 8 + i : (N >> 1) + tile * 8 + (i - 8);
  const int r = tile * 16 + i;
  return r < N ? r : N - 1;
}

// Kind of a phase: 0 embedding, 1..7 the phases of a layer, 8 final norm, 9 LM head.
__device__ __forceinline__ int dims_index(const FusedStep& p, int ph) {
  return ph == 0 ? 0 : (ph >= p.n_phases - 2 ? 8 + (ph - (p.n_phases - 2)) : 1 + (ph - 1) % kFusedPhasesPerLayer);
}
__device__ __forceinline__ int phase_layer(int ph) { return (ph - 1) / kFusedPhasesPerLayer; }
// Tensors of a projection phase (kind 2 QKV, 4 O, 6 gate/up, 7 down, 9 LM head), from the kernel parameters.
struct GemmPtrs {
  const uint32_t* qw;
  const uint16_t* scales;
  const uint16_t* biases;
};
__device__ __forceinline__ GemmPtrs gemm_ptrs(const FusedStep& p, int ph, int kind) {
  GemmPtrs w;
  if (kind == 9) {
    w.qw = p.lm_qw, w.scales = p.lm_scales, w.biases = p.lm_biases;
  } else {
    const int j = kind == 2 ? 0 : (kind == 4 ? 1 : (kind == 6 ? 2 : 3));
    const FusedLayerPtrs& L = p.layer[phase_layer(ph)];
    w.qw = L.qw[j], w.scales = L.scales[j], w.biases = L.biases[j];
  }
  return w;
}
// Position of element e of a chunk of 8 in fragment order {0,4,1,5,2,6,3,7}.
__device__ __forceinline__ int frag_pos(int e) { return (e & 3) * 2 + (e >> 2); }

// A CTA's tiles are processed in groups.  A group of T tiles gives every tile 16 / ceilpow2(T) warps, which split
// the K range between them (ksh = log2 of the warps per tile; with 8 warps per tile a warp takes one quad of every
// other slice).  The table picks the first group for a number of remaining tiles so that the chain of stages a warp
// runs through is shortest, e.g. 11 tiles = 8 tiles x 2 warps, then 3 tiles x 4 warps.
static_assert(kWarps == 16, "the group table is written for 16 warps");
__device__ __forceinline__ void group_shape(int remaining, int& T_g, int& ksh) {
  if (remaining >= 16) {
    T_g = 16, ksh = 0;
  } else {
    // remaining:           1  2  3  4  5  6  7  8  9 10 11 12 13 14 15
    const unsigned long long tg = 0xF88888887444321ull, ks = 0x011111111222233ull;
    T_g = (int)((tg >> (4 * (remaining - 1))) & 0xF);
    ksh = (int)((ks >> (4 * (remaining - 1))) & 0xF);
  }
}
// The quads (256 input features) of slice s that belong to part pw of 1 << ksh: first quad and count.
__device__ __forceinline__ void my_quads(int K, int s, int ksh, int pw, int& first, int& count) {
  const int nqs = min(4, (K - s * kFusedSliceK) >> 8);
  if (ksh == 3) {  // eight warps per tile: quad pw & 3 of the slices of parity pw >> 2
    first = pw & 3;
    count = ((s & 1) == (pw >> 2) && first < nqs) ? 1 : 0;
    return;
  }
  const int qpp = 4 >> ksh;
  first = pw * qpp;
  const int c = nqs - first;
  count = c < 0 ? 0 : (c > qpp ? qpp : c);
}
// Where input feature k of request r sits in a projection's operand (K features), in elements.  The operand is
// stored slice by slice (1024 features; all requests of a slice are contiguous, so one bulk copy stages a slice),
// a request's slice as chunks of 8 features in MMA fragment order, and the 16-byte chunks of every 128 bytes
// XOR-swizzled with the request index so that the fragment loads from shared memory are free of bank conflicts.
__device__ __forceinline__ size_t operand_chunk(int K, int r, int k) {  // k a multiple of 8: offset of its chunk
  const int k0 = k & ~(kFusedSliceK - 1), kw = min(kFusedSliceK, K - k0), chunk = (k - k0) >> 3;
  return (size_t)16 * k0 + (size_t)r * kw + (size_t)((chunk ^ (r & 7)) << 3);
}

struct AttnItem {
  int r, kvh, chunk, nch, blk0, nblk, T;
};
__device__ __forceinline__ AttnItem decode_item(const FusedStep& p, int item) {
  AttnItem it;
  int r = 0;
  while (r + 1 < p.n && item >= p.item_prefix[r + 1]) ++r;
  const int rem = item - p.item_prefix[r];
  it.r = r;
  it.T = p.lens[r] + 1;
  const int nb = (it.T + 15) >> 4;
  it.nch = p.nch[r];
  it.kvh = rem / it.nch;  // the chunks of a (request, kv head) are consecutive items
  it.chunk = rem - it.kvh * it.nch;
  it.blk0 = it.chunk * p.chunk_blocks;
  it.nblk = min(p.chunk_blocks, nb - it.blk0);
  return it;
}

// Position of a warp's prefetch in its stream of ring stages (warp-uniform except the lane's source pointers).
// The integer fields mean different things in projection and attention phases (a warp is in one at a time).
struct IssueState {
  int ph, type;
  int u[10];
  const void* q[5];
};
// PH_GEMM: the walk over groups, slices and quads; q[0..3]: this lane's four 16-byte chunks of the tile's rows at
// input feature 0; q[4]: this lane's scale (lanes 0..15) or bias (16..31) row at group 0
enum { IG_TLO = 0, IG_TC, IG_DONE, IG_KSPLIT, IG_S, IG_K, IG_SLICE, IG_QI, IG_QFIRST, IG_QCOUNT };
// PH_ATTN: the item and the stage within it; q[0]: K of the layer
enum { IA_ITEM = 0, IA_ST, IA_NST, IA_R, IA_KVH, IA_BLK0, IA_NBLK };

__global__ void __launch_bounds__(kFusedThreads, 1) fused_step_kernel(const FusedStep p) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ int s_abort;
  __shared__ __align__(8) uint64_t s_mbar[2];  // one per activation buffer
  __shared__ int s_tlo[kFusedDimKinds], s_tc[kFusedDimKinds];  // this CTA's first tile and tile count by phase kind
  unsigned char* acts = smem + kRingBytes;
  float* s_part = reinterpret_cast<float*>(acts + 2 * kActBytes);  // [non-lead warp][8 values][32 lanes]
  float* s_red = s_part + kPartFloats;                             // [warps]
  float* s_bestv = s_red + 32;                                     // [warps][16]
  int* s_besti = reinterpret_cast<int*>(s_bestv + kWarps * 16);    // [warps][16]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int cta = blockIdx.x, ncta = gridDim.x;
  unsigned char* ring = smem + warp * (kDepth * kSlot);
  const int G = p.nq / p.nkv;
  const int nqkv = (p.nq + 2 * p.nkv) * kHeadDim;
  if (ld_acquire_u32(p.control + 1) != 0u) return;  // an earlier step timed out: the model must be re-created
  // The activation buffers start as zeros (rows of absent requests are never copied into); their mbarriers take
  // one arrival (the thread that issues the bulk copies) per use.
  for (int i = threadIdx.x; i < 2 * kActBytes / 16; i += kFusedThreads)
    reinterpret_cast<uint4*>(acts)[i] = make_uint4(0u, 0u, 0u, 0u);
  if (threadIdx.x < kFusedDimKinds) {
    const int nt = p.dims[threadIdx.x].type == PH_GEMM ? p.dims[threadIdx.x].ntiles : 0;
    s_tlo[threadIdx.x] = (int)((long long)cta * nt / ncta);
    s_tc[threadIdx.x] = (int)((long long)(cta + 1) * nt / ncta) - s_tlo[threadIdx.x];
  }
  if (threadIdx.x == 0) {
    s_abort = 0;
    mbar_init(&s_mbar[0], 1u);
    mbar_init(&s_mbar[1], 1u);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();
  int staged = 0;  // activation slices staged so far: slice number i uses buffer i & 1, mbarrier parity (i >> 1) & 1

  // ---------------------------------------------------------------- the issue side of the stage stream
  IssueState iss;
  iss.ph = p.ph_begin, iss.type = -1;
#pragma unroll
  for (int i = 0; i < 10; ++i) iss.u[i] = 0;
#pragma unroll
  for (int i = 0; i < 5; ++i) iss.q[i] = nullptr;
  int islot = 0;
  int win = 0, win_item = -1;  // window of block ids (blk0 + 32 * window + lane) of an attention item, and which item

  // PH_GEMM: moves to the next (group, slice) at or after the current one in which this warp has quads; `fresh`
  // says that the tile may have changed, so the lane's row pointers are loaded.
  auto iss_gemm_seek = [&](bool fresh) -> bool {
    for (;;) {
      if (iss.u[IG_DONE] >= iss.u[IG_TC]) return false;
      int T_g, ksh;
      group_shape(iss.u[IG_TC] - iss.u[IG_DONE], T_g, ksh);
      const int tw = warp >> ksh, pw = warp & ((1 << ksh) - 1);
      if (tw < T_g) {
        while (iss.u[IG_SLICE] < iss.u[IG_S]) {
          my_quads(iss.u[IG_K], iss.u[IG_SLICE], ksh, pw, iss.u[IG_QFIRST], iss.u[IG_QCOUNT]);
          if (iss.u[IG_QCOUNT] > 0) break;
          ++iss.u[IG_SLICE];
        }
        if (iss.u[IG_SLICE] < iss.u[IG_S]) {
          if (fresh) {
            const int kind = dims_index(p, iss.ph);
            const FusedDims& D = p.dims[kind];
            const GemmPtrs P = gemm_ptrs(p, iss.ph, kind);
            const int tile = iss.u[IG_TLO] + iss.u[IG_DONE] + tw, K = iss.u[IG_K];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int row = unit_row(D.epi, D.N, tile, i * 4 + (lane >> 3));
              iss.q[i] = P.qw + (size_t)row * (K >> 3) + (lane & 7) * 4;
            }
            const int row = unit_row(D.epi, D.N, tile, lane & 15);
            iss.q[4] = (lane < 16 ? P.scales : P.biases) + (size_t)row * (K >> 6);
          }
          return true;
        }
      }
      iss.u[IG_DONE] += T_g;
      iss.u[IG_SLICE] = 0;
      fresh = true;
    }
  };
  auto iss_attn_load = [&]() {
    const AttnItem it = decode_item(p, iss.u[IA_ITEM]);
    iss.u[IA_R] = it.r, iss.u[IA_KVH] = it.kvh, iss.u[IA_BLK0] = it.blk0, iss.u[IA_NBLK] = it.nblk;
    iss.u[IA_NST] = 4 * it.nblk, iss.u[IA_ST] = 0;
  };
  auto iss_load_phase = [&]() {  // moves to the first phase at or after iss.ph in which this warp has stages
    while (iss.ph < p.ph_end) {
      const int kind = dims_index(p, iss.ph);
      const FusedDims& D = p.dims[kind];
      iss.type = D.type;
      if (D.type == PH_GEMM) {
        iss.u[IG_TLO] = s_tlo[kind];
        iss.u[IG_TC] = s_tc[kind];
        iss.u[IG_DONE] = 0, iss.u[IG_SLICE] = 0, iss.u[IG_QI] = 0, iss.u[IG_S] = D.S, iss.u[IG_K] = D.K;
        if (iss.u[IG_TC] > 0 && iss_gemm_seek(true)) break;
      } else if (D.type == PH_ATTN) {
        iss.u[IA_ITEM] = cta * kWarps + warp;
        if (iss.u[IA_ITEM] < p.n_items) {
          iss.q[0] = p.pool + (size_t)(2 * phase_layer(iss.ph)) * p.layer_elems;
          iss_attn_load();
          break;
        }
      }
      ++iss.ph;
    }
  };
  // Issues the next stage of the stream (if any) into the next ring slot and closes a cp.async group either way.
  auto issue_next = [&]() {
    if (iss.ph < p.ph_end) {
      unsigned char* stg = ring + islot * kSlot;
      if (iss.type == PH_GEMM) {
        const int k = iss.u[IG_SLICE] * kFusedSliceK + (iss.u[IG_QFIRST] + iss.u[IG_QI]) * 256;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int r = i * 4 + (lane >> 3);
          cp_async16(stg + r * 128 + (((lane & 7) ^ (r & 7)) << 4), static_cast<const uint32_t*>(iss.q[i]) + (k >> 3));
        }
        cp_async8(stg + kSlotSb + (lane & 15) * 16 + (lane >> 4) * 8, static_cast<const uint16_t*>(iss.q[4]) + (k >> 6));
        if (++iss.u[IG_QI] == iss.u[IG_QCOUNT]) {
          iss.u[IG_QI] = 0;
          ++iss.u[IG_SLICE];
          if (!iss_gemm_seek(false)) {
            ++iss.ph;
            iss_load_phase();
          }
        }
      } else {
        const int b = iss.u[IA_ST] >> 2, part = iss.u[IA_ST] & 3;
        if (part == 0 && (b & 31) == 0 && (b != 0 || win_item != iss.u[IA_ITEM])) {
          // block ids do not depend on the layer: the first window of an item is kept from one layer to the next
          const int idx = b + lane;
          win = idx < iss.u[IA_NBLK] ? p.bt[(size_t)iss.u[IA_R] * p.max_blocks + iss.u[IA_BLK0] + idx] : 0;
          win_item = b == 0 ? iss.u[IA_ITEM] : -1;
        }
        const int blk = __shfl_sync(0xffffffffu, win, b & 31);
        const uint16_t* kbase = static_cast<const uint16_t*>(iss.q[0]);
        const uint16_t* base = (part < 2 ? kbase : kbase + p.layer_elems) +
                               ((size_t)(blk * p.nkv + iss.u[IA_KVH]) * 16 + (part & 1) * 8) * kHeadDim;
        const unsigned char* src = reinterpret_cast<const unsigned char*>(base);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int c = i * 32 + lane, tok = c >> 4, c16 = c & 15;
          cp_async16(stg + tok * 256 + ((c16 ^ tok) << 4), src + c * 16);
        }
        if (++iss.u[IA_ST] == iss.u[IA_NST]) {
          iss.u[IA_ITEM] += ncta * kWarps;
          if (iss.u[IA_ITEM] < p.n_items) {
            iss_attn_load();
          } else {
            ++iss.ph;
            iss_load_phase();
          }
        }
      }
    }
    cp_async_commit();
    islot = (islot + 1) & (kDepth - 1);
  };

  iss_load_phase();
#pragma unroll 1
  for (int i = 0; i < kDepth - 1; ++i) issue_next();
  int cslot = 0;

  // ---------------------------------------------------------------- grid barrier
  unsigned int bar_target = 0;
  auto grid_barrier = [&](int ph) -> bool {
    bar_target += ncta;
    __syncthreads();
    if (threadIdx.x == 0) {
      red_release_add_u32(p.control, 1u);
      const unsigned long long t0 = global_ns();
      unsigned int polls = 0;
      while (ld_relaxed_u32(p.control) < bar_target) {
        if ((++polls & 63u) == 0) {
          if (ld_acquire_u32(p.control + 1) != 0u) {
            s_abort = 1;
            break;
          }
          if (global_ns() - t0 > kBarrierTimeoutNs) {
            atomicExch(p.control + 1, 1u);
            s_abort = 1;
            break;
          }
        }
      }
      asm volatile("fence.acq_rel.gpu;" ::: "memory");
      if (p.timeline && cta == 0) p.timeline[ph - p.ph_begin + 1] = global_ns();
    }
    __syncthreads();
    return s_abort == 0;
  };
  if (p.timeline && cta == 0 && threadIdx.x == 0) p.timeline[0] = global_ns();

  // running argmax of the logits this thread finalises: requests nt * 8 + 2t + j
  float bestv[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
  int besti[4] = {0x7fffffff, 0x7fffffff, 0x7fffffff, 0x7fffffff};

#pragma unroll 1
  for (int ph = p.ph_begin; ph < p.ph_end; ++ph) {
    const FusedDims& D = p.dims[dims_index(p, ph)];

    if (D.type == PH_EMBED) {
      // ---------------------------------------------------------- embedding (or sums of squares of a given x)
      if (cta < p.n) {
        const int r = cta, H = p.H;
        int tok = 0;
        if (!p.embed_from_x) {
          tok = p.tokens[r];
          tok = tok < 0 ? 0 : (tok >= p.V ? p.V - 1 : tok);
        }
        for (int tile = threadIdx.x; tile < (H >> 4); tile += kFusedThreads) {
          uint32_t out[8];
          float ss = 0.0f;
          if (!p.embed_from_x) {
            const uint2 w = *reinterpret_cast<const uint2*>(p.embed_q + (size_t)tok * (H >> 3) + tile * 2);
            const float sc = bf16_to_f32(p.embed_s[(size_t)tok * (H >> 6) + (tile >> 2)]);
            const float bi = bf16_to_f32(p.embed_b[(size_t)tok * (H >> 6) + (tile >> 2)]);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const uint32_t word = i < 4 ? w.x : w.y;
              const float a = __fmaf_rn(sc, (float)((word >> (8 * (i & 3))) & 0xFu), bi);
              const float b = __fmaf_rn(sc, (float)((word >> (8 * (i & 3) + 4)) & 0xFu), bi);
              out[i] = pack_bf16x2(a, b);
            }
            uint4* dst = reinterpret_cast<uint4*>(p.x + (size_t)r * H + tile * 16);
            dst[0] = make_uint4(out[0], out[1], out[2], out[3]);
            dst[1] = make_uint4(out[4], out[5], out[6], out[7]);
          } else {
            const uint4* src = reinterpret_cast<const uint4*>(p.x + (size_t)r * H + tile * 16);
            const uint4 a = __ldcg(src), b = __ldcg(src + 1);
            out[0] = a.x, out[1] = a.y, out[2] = a.z, out[3] = a.w;
            out[4] = b.x, out[5] = b.y, out[6] = b.z, out[7] = b.w;
          }
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float a = bf16_lo(out[i]), b = bf16_hi(out[i]);
            ss = fmaf(a, a, ss);
            ss = fmaf(b, b, ss);
          }
          p.ss[(size_t)tile * 16 + r] = ss;
        }
      }
    } else if (D.type == PH_NORM) {
      // ---------------------------------------------------------- RMSNorm: y = bf16(x / rms(x) * w), written once
      // for all CTAs as the operand of the next projection (chunks of 8 in fragment order)
      const int nkind = dims_index(p, ph);
      const uint16_t* norm_w = nkind == 8 ? p.final_norm : p.layer[phase_layer(ph)].norm[nkind == 1 ? 0 : 1];
      const int H = D.K, cpr = H >> 3, total = p.n * cpr;
      const int lo = (int)((long long)cta * total / ncta), hi = (int)((long long)(cta + 1) * total / ncta);
      if (hi > lo) {
        uint16_t* out = p.y;
        for (int r = lo / cpr; r <= (hi - 1) / cpr; ++r) {
          float sq = 0.0f;
          for (int j = threadIdx.x; j < (H >> 4); j += kFusedThreads) sq += __ldcg(p.ss + (size_t)j * 16 + r);
          sq = warp_sum(sq);
          if (lane == 0) s_red[warp] = sq;
          __syncthreads();
          float tot = 0.0f;
#pragma unroll
          for (int w = 0; w < kWarps; ++w) tot += s_red[w];
          const float inv = 1.0f / sqrtf(tot / (float)H + p.eps);
          const int c_lo = max(lo, r * cpr), c_hi = min(hi, (r + 1) * cpr);
          for (int c = c_lo + threadIdx.x; c < c_hi; c += kFusedThreads) {
            const int kc = c - r * cpr;
            const uint4 v = __ldcg(reinterpret_cast<const uint4*>(p.x + (size_t)r * H + kc * 8));
            const uint4 wv = *reinterpret_cast<const uint4*>(norm_w + kc * 8);
            const uint32_t e[4] = {v.x, v.y, v.z, v.w}, ww[4] = {wv.x, wv.y, wv.z, wv.w};
            uint32_t o[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
              o[j] = pack_bf16x2(bf16_lo(e[j]) * inv * bf16_lo(ww[j]), bf16_hi(e[j]) * inv * bf16_hi(ww[j]));
            *reinterpret_cast<uint4*>(out + operand_chunk(H, r, kc * 8)) = permute_chunk(make_uint4(o[0], o[1], o[2], o[3]));
          }
          __syncthreads();
        }
      }
    } else if (D.type == PH_GEMM) {
      // ---------------------------------------------------------- projection
      const int t_lo = s_tlo[dims_index(p, ph)], T_c = s_tc[dims_index(p, ph)];
      if (T_c > 0) {
        // operand (as its producer wrote it) and output by kind: 2 QKV, 4 O, 6 gate/up, 7 down, 9 LM head
        const int kind = dims_index(p, ph);
        const uint16_t* in = kind == 4 ? p.attn : (kind == 7 ? p.h : p.y);
        uint16_t* outp = kind == 2 ? p.qkv : (kind == 6 ? p.h : p.x);
        const int out_stride = kind == 2 ? nqkv : p.H;
        const int K = D.K, S = D.S;

        // A slice of the operand goes to shared memory as one bulk copy per request row, tracked by the buffer's
        // mbarrier; the sums over every group of 64 input features come from the tensor cores (ones x operand).
        auto stage_issue = [&](int slice, int idx) {
          if (threadIdx.x == kFusedThreads - 32) {  // a lane of the last warp, which computes least often
            const int k0 = slice * kFusedSliceK;
            const uint32_t bytes = (uint32_t)(min(kFusedSliceK, K - k0) * 2 * p.n);  // rows 0..n-1 are contiguous
            mbar_expect_tx(&s_mbar[idx & 1], bytes);
            bulk_copy_g2s(acts + (idx & 1) * kActBytes, in + (size_t)16 * k0, bytes, &s_mbar[idx & 1]);
          }
          // the other lanes of the issuing warp go on to spin on the mbarrier: they must not starve the issuing lane
          __syncwarp();
        };
        auto stage_finish = [&](int slice, int idx) {
          if (!mbar_wait(&s_mbar[idx & 1], (uint32_t)((idx >> 1) & 1))) {
            if (lane == 0) atomicExch(p.control + 1, 2u);  // the copy never landed: report, results are void
          }
          const unsigned char* sB = acts + (idx & 1) * kActBytes;
          float* sX = reinterpret_cast<float*>(acts + (idx & 1) * kActBytes + kActRows);
          const int kw2 = min(kFusedSliceK, K - slice * kFusedSliceK) * 2, groups = kw2 >> 7;
          const uint32_t one2 = 0x3F803F80u;  // bf16 {1, 1}
          for (int gi = warp; gi < groups; gi += kWarps) {
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
              const unsigned char* row = sB + (nt * 8 + g) * kw2;
              const uint4 b0 = *reinterpret_cast<const uint4*>(row + (((gi * 8 + t * 2) ^ g) << 4));
              const uint4 b1 = *reinterpret_cast<const uint4*>(row + (((gi * 8 + t * 2 + 1) ^ g) << 4));
              float d[4];
              mma_bf16_first(d, one2, one2, one2, one2, b0.x, b0.y);
              mma_bf16(d, one2, one2, one2, one2, b0.z, b0.w);
              mma_bf16(d, one2, one2, one2, one2, b1.x, b1.y);
              mma_bf16(d, one2, one2, one2, one2, b1.z, b1.w);
              if (g == 0) *reinterpret_cast<float2*>(sX + gi * 16 + nt * 8 + 2 * t) = make_float2(d[0], d[1]);
            }
          }
        };

        // The CTA walks Q = groups x S slices; two of them are in flight at any time: slice q + 2 is requested as
        // soon as slice q's buffer is free.
        int n_groups = 0;
        for (int d2 = 0; d2 < T_c; ++n_groups) {
          int tg, kk;
          group_shape(T_c - d2, tg, kk);
          d2 += tg;
        }
        const int Q = n_groups * S, idx0 = staged;
        staged += Q;
        stage_issue(0, idx0);
        if (Q > 1) stage_issue(1 % S, idx0 + 1);
        stage_finish(0, idx0);
        __syncthreads();
        int q = 0;  // position in the walk: buffer (idx0 + q) & 1

        int done = 0;
#pragma unroll 1
        while (done < T_c) {
          int T_g, ksh;
          group_shape(T_c - done, T_g, ksh);
          const int ksplit = 1 << ksh, tw = warp >> ksh, pw = warp & (ksplit - 1);
          const bool mine = tw < T_g, lead = mine && pw == 0;
          const int tile = t_lo + done + tw;
          float acc[2][4];
#pragma unroll
          for (int nt = 0; nt < 2; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.0f;
          // the lead warp of a residual tile fetches the old values early
          uint16_t xold[8];
          if (lead && D.epi == EPI_RESIDUAL) {
            const uint16_t* out = outp;
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
              for (int c = 0; c < 4; ++c) {
                const int req = nt * 8 + 2 * t + (c & 1), row = tile * 16 + g + (c >> 1) * 8;
                xold[nt * 4 + c] = (req < p.n && row < D.N) ? __ldcg(out + (size_t)req * out_stride + row) : (uint16_t)0;
              }
          }

#pragma unroll 1
          for (int s = 0; s < S; ++s) {
            if (mine) {
              int q_first, q_count;
              my_quads(K, s, ksh, pw, q_first, q_count);
              const unsigned char* sB = acts + ((idx0 + q) & 1) * kActBytes;
              const float* sX = reinterpret_cast<const float*>(sB + kActRows);
              const int kw2 = min(kFusedSliceK, K - s * kFusedSliceK) * 2;  // bytes per request row of this slice
#pragma unroll 1
              for (int qi = 0; qi < q_count; ++qi) {
                const int qd = q_first + qi;
                issue_next();
                cp_async_wait<kDepth - 1>();
                __syncwarp();
                const unsigned char* stg = ring + cslot * kSlot;
                const uint4 sb_lo = *reinterpret_cast<const uint4*>(stg + kSlotSb + g * 16);
                const uint4 sb_hi = *reinterpret_cast<const uint4*>(stg + kSlotSb + (g + 8) * 16);
                const uint2 sc_lo = make_uint2(sb_lo.x, sb_lo.y), bi_lo = make_uint2(sb_lo.z, sb_lo.w);
                const uint2 sc_hi = make_uint2(sb_hi.x, sb_hi.y), bi_hi = make_uint2(sb_hi.z, sb_hi.w);
#pragma unroll
                for (int gi = 0; gi < 4; ++gi) {
                  const int gidx = qd * 4 + gi;
                  uint4 bf[2][2];
                  float2 xs[2];
#pragma unroll
                  for (int nt = 0; nt < 2; ++nt) {
                    const unsigned char* row = sB + (nt * 8 + g) * kw2;
                    bf[nt][0] = *reinterpret_cast<const uint4*>(row + (((gidx * 8 + t * 2) ^ g) << 4));
                    bf[nt][1] = *reinterpret_cast<const uint4*>(row + (((gidx * 8 + t * 2 + 1) ^ g) << 4));
                    xs[nt] = *reinterpret_cast<const float2*>(sX + gidx * 16 + nt * 8 + 2 * t);
                  }
                  const int off = (((gi * 2 + (t >> 1)) ^ g) << 4) + (t & 1) * 8;  // g: swizzle key of rows g, g + 8
                  const uint2 wl = *reinterpret_cast<const uint2*>(stg + g * 128 + off);
                  const uint2 wh = *reinterpret_cast<const uint2*>(stg + (g + 8) * 128 + off);
                  uint32_t l0[4], l1[4], h0[4], h1[4];
                  unpack_word(wl.x, l0);
                  unpack_word(wl.y, l1);
                  unpack_word(wh.x, h0);
                  unpack_word(wh.y, h1);
                  // sum (16 + q) x = 16 X + sum q x: the bias that multiplies X becomes b - 16 s
                  const float s_l = bf16_at(sc_lo, gi), s_h = bf16_at(sc_hi, gi);
                  const float b_l = fmaf(-16.0f, s_l, bf16_at(bi_lo, gi)), b_h = fmaf(-16.0f, s_h, bf16_at(bi_hi, gi));
#pragma unroll
                  for (int nt = 0; nt < 2; ++nt) {
                    float pc[4];
                    mma_bf16_first(pc, l0[0], h0[0], l0[1], h0[1], bf[nt][0].x, bf[nt][0].y);
                    mma_bf16(pc, l0[2], h0[2], l0[3], h0[3], bf[nt][0].z, bf[nt][0].w);
                    mma_bf16(pc, l1[0], h1[0], l1[1], h1[1], bf[nt][1].x, bf[nt][1].y);
                    mma_bf16(pc, l1[2], h1[2], l1[3], h1[3], bf[nt][1].z, bf[nt][1].w);
                    acc[nt][0] = fmaf(s_l, pc[0], fmaf(b_l, xs[nt].x, acc[nt][0]));
                    acc[nt][1] = fmaf(s_l, pc[1], fmaf(b_l, xs[nt].y, acc[nt][1]));
                    acc[nt][2] = fmaf(s_h, pc[2], fmaf(b_h, xs[nt].x, acc[nt][2]));
                    acc[nt][3] = fmaf(s_h, pc[3], fmaf(b_h, xs[nt].y, acc[nt][3]));
                  }
                }
                __syncwarp();
                cslot = (cslot + 1) & (kDepth - 1);
              }
            }
            if (q + 1 < Q) stage_finish((q + 1) % S, idx0 + q + 1);
            __syncthreads();
            if (q + 2 < Q) stage_issue((q + 2) % S, idx0 + q + 2);
            ++q;
          }

          // ---- warps that shared a tile: the lead warp adds the others' sums in warp order
          if (ksplit > 1) {
            if (mine && !lead) {
#pragma unroll
              for (int i = 0; i < 8; ++i) s_part[((warp - tw - 1) * 8 + i) * 32 + lane] = acc[i >> 2][i & 3];
            }
            __syncthreads();
            if (lead) {
              for (int o = 1; o < ksplit; ++o)
#pragma unroll
                for (int i = 0; i < 8; ++i) acc[i >> 2][i & 3] += s_part[((warp + o - tw - 1) * 8 + i) * 32 + lane];
            }
          }

          // ---- epilogue: acc[nt][c]: row g + 8 * (c >> 1) of the tile, request nt * 8 + 2t + (c & 1)
          if (lead) {
            if (D.epi == EPI_SILU_PACK) {
              uint16_t* out = outp;
              // the tile's 8 columns are one chunk of the down projection's operand (N / 2 input features)
#pragma unroll
              for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                  const int req = nt * 8 + 2 * t + j;
                  const float gt = bf16_round(acc[nt][j]), up = bf16_round(acc[nt][2 + j]);
                  if (req < p.n)
                    out[operand_chunk(D.N >> 1, req, tile * 8) + frag_pos(g)] = f32_to_bf16((gt / (1.0f + expf(-gt))) * up);
                }
            } else if (D.epi == EPI_F32) {
#pragma unroll
              for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                  const int req = nt * 8 + 2 * t + (c & 1), row = tile * 16 + g + (c >> 1) * 8;
                  if (req < p.n && row < D.N) {
                    const float v = acc[nt][c];
                    if (p.logits) p.logits[(size_t)req * D.N + row] = v;
                    const int bi = nt * 2 + (c & 1);
                    if (v > bestv[bi] || (v == bestv[bi] && row < besti[bi])) bestv[bi] = v, besti[bi] = row;
                  }
                }
            } else {
              uint16_t* out = outp;
              float sq[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
              for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                  const int req = nt * 8 + 2 * t + (c & 1), row = tile * 16 + g + (c >> 1) * 8;
                  if (req < p.n && row < D.N) {
                    uint16_t y = f32_to_bf16(acc[nt][c]);
                    if (D.epi == EPI_RESIDUAL) {
                      y = f32_to_bf16(bf16_to_f32(xold[nt * 4 + c]) + bf16_to_f32(y));
                      const float f = bf16_to_f32(y);
                      sq[nt * 2 + (c & 1)] = fmaf(f, f, sq[nt * 2 + (c & 1)]);
                    }
                    out[(size_t)req * out_stride + row] = y;
                  }
                }
              if (D.epi == EPI_RESIDUAL) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  sq[i] += __shfl_xor_sync(0xffffffffu, sq[i], 4);
                  sq[i] += __shfl_xor_sync(0xffffffffu, sq[i], 8);
                  sq[i] += __shfl_xor_sync(0xffffffffu, sq[i], 16);
                }
                if (g == 0) {
#pragma unroll
                  for (int i = 0; i < 4; ++i) p.ss[(size_t)tile * 16 + (i >> 1) * 8 + 2 * t + (i & 1)] = sq[i];
                }
              }
            }
          }
          done += T_g;
        }
      }

      if (D.epi == EPI_F32) {
        // the CTA's best logit per request, then (after the barrier) the best over all CTAs
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int o = 4; o <= 16; o <<= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bestv[i], o);
            const int oi = __shfl_xor_sync(0xffffffffu, besti[i], o);
            if (ov > bestv[i] || (ov == bestv[i] && oi < besti[i])) bestv[i] = ov, besti[i] = oi;
          }
        if (g == 0) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int req = (i >> 1) * 8 + 2 * t + (i & 1);
            s_bestv[warp * 16 + req] = bestv[i], s_besti[warp * 16 + req] = besti[i];
          }
        }
        __syncthreads();
        if (threadIdx.x < 16) {
          float bv = s_bestv[threadIdx.x];
          int bi = s_besti[threadIdx.x];
          for (int w = 1; w < kWarps; ++w) {
            const float ov = s_bestv[w * 16 + threadIdx.x];
            const int oi = s_besti[w * 16 + threadIdx.x];
            if (ov > bv || (ov == bv && oi < bi)) bv = ov, bi = oi;
          }
          p.amax[(size_t)cta * 16 + threadIdx.x] = make_float2(bv, __int_as_float(bi));
        }
      }
    } else {
      // ---------------------------------------------------------- attention
      // Per 16-token block: S^T[token][head] = K q^T (tokens are the MMA rows, the G <= 8 query heads of the kv head
      // the columns), online softmax down the columns, P^T transposed in registers (movmatrix) into the B operand of
      // O^T[d][head] += V^T P^T with P split into two bf16 terms.
      const int layer = phase_layer(ph);
      const FusedLayerPtrs& P = p.layer[layer];
      uint16_t* kpool_w = p.pool + (size_t)(2 * layer) * p.layer_elems;
      const int Gs = (G + 1) & ~1;  // heads stored per partial result
      // Items are dealt 16 consecutive ones to a CTA, one per warp, so the chunks of a (request, kv head) mostly meet
      // in one CTA and are merged in shared memory (the activation buffers are idle during attention).
      float* s_o = reinterpret_cast<float*>(acts);  // [warp][32 accumulator values][lane]
      float* s_ml = s_part;                         // [warp][heads 2t, 2t+1 of t = 0..3][m, l]
      const int per_round = ncta * kWarps;
#pragma unroll 1
      for (int base = cta * kWarps; base < p.n_items; base += per_round) {
        const int item = base + warp;
        const bool valid = item < p.n_items;
        AttnItem it = decode_item(p, valid ? item : base);
        const int r = it.r, h = it.kvh, pos = it.T - 1;
        if (!valid) it.nblk = 0;
        const uint16_t* qrow = p.qkv + (size_t)r * nqkv;
        const bool appends = valid && it.chunk == it.nch - 1;

        // loads first: q of head g, k and v of the new token, block id of the append
        uint32_t qb[8][2];  // head g: dims 16ks + 2t, +1 and 16ks + 2t + 8, +9
        uint32_t wa = 0u, wb = 0u, nv_a = 0u, nv_b = 0u;
        int append_blk = 0;
        {
          const uint16_t* q0 = qrow + (size_t)(h * G + g) * kHeadDim;
          const bool v0 = g < G;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            qb[ks][0] = v0 ? __ldcg(reinterpret_cast<const uint32_t*>(q0 + 16 * ks + 2 * t)) : 0u;
            qb[ks][1] = v0 ? __ldcg(reinterpret_cast<const uint32_t*>(q0 + 16 * ks + 2 * t + 8)) : 0u;
          }
          if (appends) {
            const uint16_t* ksrc = qrow + (size_t)(p.nq + h) * kHeadDim;
            const uint16_t* vsrc = qrow + (size_t)(p.nq + p.nkv + h) * kHeadDim;
            wa = __ldcg(reinterpret_cast<const uint32_t*>(ksrc + 2 * lane));
            wb = __ldcg(reinterpret_cast<const uint32_t*>(ksrc + 64 + 2 * lane));
            nv_a = __ldcg(reinterpret_cast<const uint32_t*>(vsrc + 2 * lane));
            nv_b = __ldcg(reinterpret_cast<const uint32_t*>(vsrc + 64 + 2 * lane));
            append_blk = p.bt[(size_t)r * p.max_blocks + (pos >> 4)];
          }
        }
        if (P.q_norm) {
          float ss = 0.0f;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            ss += bf16_lo(qb[ks][0]) * bf16_lo(qb[ks][0]) + bf16_hi(qb[ks][0]) * bf16_hi(qb[ks][0]) +
                  bf16_lo(qb[ks][1]) * bf16_lo(qb[ks][1]) + bf16_hi(qb[ks][1]) * bf16_hi(qb[ks][1]);
          ss += __shfl_xor_sync(0xffffffffu, ss, 1);
          ss += __shfl_xor_sync(0xffffffffu, ss, 2);
          const float inv = 1.0f / sqrtf(ss * (1.0f / kHeadDim) + p.eps);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
              const uint32_t nw = *reinterpret_cast<const uint32_t*>(P.q_norm + 16 * ks + 2 * t + hf * 8);
              qb[ks][hf] = pack_bf16x2(bf16_lo(qb[ks][hf]) * inv * bf16_lo(nw), bf16_hi(qb[ks][hf]) * inv * bf16_hi(nw));
            }
        }
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) {
            const int col = 16 * ks + 2 * t + hf * 8;  // even, < 64
            const float4 cs = *reinterpret_cast<const float4*>(p.rope + ((size_t)pos * 64 + col) * 2);  // c0 s0 c1 s1
            const float a0 = bf16_lo(qb[ks][hf]), a1 = bf16_hi(qb[ks][hf]);
            const float b0 = bf16_lo(qb[ks + 4][hf]), b1 = bf16_hi(qb[ks + 4][hf]);
            qb[ks][hf] = pack_bf16x2(a0 * cs.x - b0 * cs.y, a1 * cs.z - b1 * cs.w);
            qb[ks + 4][hf] = pack_bf16x2(b0 * cs.x + a0 * cs.y, b1 * cs.z + a1 * cs.w);
          }

        // The warp with the request's last chunk prepares k, v of the new token and appends them to the pool.
        uint32_t nk_a = 0u, nk_b = 0u;  // elements 2*lane, 2*lane+1 and 64+2*lane, 64+2*lane+1
        if (appends) {
          float a0 = bf16_lo(wa), a1 = bf16_hi(wa), b0 = bf16_lo(wb), b1 = bf16_hi(wb);
          if (P.k_norm) {
            const float ss = warp_sum(a0 * a0 + a1 * a1 + b0 * b0 + b1 * b1);
            const float inv = 1.0f / sqrtf(ss * (1.0f / kHeadDim) + p.eps);
            const uint32_t na = *reinterpret_cast<const uint32_t*>(P.k_norm + 2 * lane);
            const uint32_t nb = *reinterpret_cast<const uint32_t*>(P.k_norm + 64 + 2 * lane);
            a0 = bf16_round(a0 * inv * bf16_lo(na));
            a1 = bf16_round(a1 * inv * bf16_hi(na));
            b0 = bf16_round(b0 * inv * bf16_lo(nb));
            b1 = bf16_round(b1 * inv * bf16_hi(nb));
          }
          const float4 cs = *reinterpret_cast<const float4*>(p.rope + ((size_t)pos * 64 + 2 * lane) * 2);
          nk_a = pack_bf16x2(a0 * cs.x - b0 * cs.y, a1 * cs.z - b1 * cs.w);
          nk_b = pack_bf16x2(b0 * cs.x + a0 * cs.y, b1 * cs.z + a1 * cs.w);
          uint16_t* kd = kpool_w + ((size_t)(append_blk * p.nkv + h) * 16 + (pos & 15)) * kHeadDim;
          uint16_t* vd = kd + p.layer_elems;
          *reinterpret_cast<uint32_t*>(kd + 2 * lane) = nk_a;
          *reinterpret_cast<uint32_t*>(kd + 64 + 2 * lane) = nk_b;
          *reinterpret_cast<uint32_t*>(vd + 2 * lane) = nv_a;
          *reinterpret_cast<uint32_t*>(vd + 64 + 2 * lane) = nv_b;
        }

        // o[dt][c]: d = 16 dt + g + 8 (c >> 1), head 2t + (c & 1); m, l of heads 2t (index 0) and 2t + 1 (index 1)
        float o[8][4];
#pragma unroll
        for (int j = 0; j < 8; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.0f;
        float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.0f, l1 = 0.0f;

#pragma unroll 1
        for (int bi = 0; bi < it.nblk; ++bi) {
          const int tile = it.blk0 + bi;
          const bool patch = appends && tile == (pos >> 4);  // fetched before k, v of the new token existed
          const int tk = pos & 7;
          const int off_a = tk * 256 + (((lane >> 2) ^ tk) << 4) + (lane & 3) * 4;
          const int off_b = tk * 256 + (((8 + (lane >> 2)) ^ tk) << 4) + (lane & 3) * 4;
          unsigned char* sK0 = ring + cslot * kSlot;
          unsigned char* sK1 = ring + ((cslot + 1) & (kDepth - 1)) * kSlot;
          unsigned char* sV0 = ring + ((cslot + 2) & (kDepth - 1)) * kSlot;
          unsigned char* sV1 = ring + ((cslot + 3) & (kDepth - 1)) * kSlot;

          // K: kDepth stages are committed after this issue; the two K halves are the oldest two
          issue_next();
          cp_async_wait<kDepth - 2>();
          __syncwarp();
          if (patch) {
            unsigned char* kd = (pos & 8) ? sK1 : sK0;
            *reinterpret_cast<uint32_t*>(kd + off_a) = nk_a;
            *reinterpret_cast<uint32_t*>(kd + off_b) = nk_b;
            __syncwarp();
          }
          // scores: rows = tokens g, g + 8 of the block; columns = heads 2t, 2t + 1
          float s[4] = {0.0f, 0.0f, 0.0f, 0.0f};
          {
            const int mi = lane >> 3, tok = lane & 7;
            const unsigned char* kb = ((mi & 1) ? sK1 : sK0) + tok * 256;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              uint32_t ka[4];
              ldmatrix_x4(ka, kb + (((2 * ks + (mi >> 1)) ^ tok) << 4));
              mma_bf16(s, ka[0], ka[1], ka[2], ka[3], qb[ks][0], qb[ks][1]);
            }
          }
          __syncwarp();
          // the K slots are free: two more stages go out while V is awaited
          issue_next();
          issue_next();
          if (tile * 16 + 16 > it.T) {  // ragged last block: tokens at or beyond T do not exist
            if (tile * 16 + g >= it.T) s[0] = s[1] = -INFINITY;
            if (tile * 16 + g + 8 >= it.T) s[2] = s[3] = -INFINITY;
          }

          // online softmax down the columns; m is kept in log2 units
          float mx0 = fmaxf(s[0], s[2]), mx1 = fmaxf(s[1], s[3]);
#pragma unroll
          for (int sh = 4; sh <= 16; sh <<= 1) {
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, sh));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, sh));
          }
          const float mn0 = fmaxf(m0, mx0 * kScaleLog2), mn1 = fmaxf(m1, mx1 * kScaleLog2);
          const bool grow = (mn0 > m0) || (mn1 > m1);
          if (__any_sync(0xffffffffu, grow)) {
            const float c0 = exp2f(m0 - mn0), c1 = exp2f(m1 - mn1);
            l0 *= c0;
            l1 *= c1;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              o[j][0] *= c0, o[j][2] *= c0;
              o[j][1] *= c1, o[j][3] *= c1;
            }
            m0 = mn0, m1 = mn1;
          }
          uint32_t pH[2], pL[2];  // B fragments of P^T (head g; tokens 2t, 2t+1 and 2t+8, 2t+9): hi and lo bf16 terms
          {
            const float p0 = exp2f(fmaf(s[0], kScaleLog2, -m0)), p1 = exp2f(fmaf(s[1], kScaleLog2, -m1));
            const float p2 = exp2f(fmaf(s[2], kScaleLog2, -m0)), p3 = exp2f(fmaf(s[3], kScaleLog2, -m1));
            l0 += p0 + p2;
            l1 += p1 + p3;
            const uint32_t h01 = pack_bf16x2(p0, p1), h23 = pack_bf16x2(p2, p3);  // (token g | g + 8; heads 2t, 2t+1)
            const uint32_t e01 = pack_bf16x2(p0 - bf16_lo(h01), p1 - bf16_hi(h01));
            const uint32_t e23 = pack_bf16x2(p2 - bf16_lo(h23), p3 - bf16_hi(h23));
            pH[0] = movmatrix_trans(h01), pH[1] = movmatrix_trans(h23);
            pL[0] = movmatrix_trans(e01), pL[1] = movmatrix_trans(e23);
          }

          // V: kDepth + 2 stages are committed since the block began; the V halves are the third and fourth
          cp_async_wait<kDepth - 2>();
          __syncwarp();
          if (patch) {
            unsigned char* vd = (pos & 8) ? sV1 : sV0;
            *reinterpret_cast<uint32_t*>(vd + off_a) = nv_a;
            *reinterpret_cast<uint32_t*>(vd + off_b) = nv_b;
            __syncwarp();
          }
          // O^T[d][head] += V^T[d][token] P^T[token][head]
          {
            const int mi = lane >> 3, tok = lane & 7;
            const unsigned char* vbase = ((mi >> 1) ? sV1 : sV0) + tok * 256;
#pragma unroll
            for (int dt = 0; dt < 8; ++dt) {
              uint32_t va[4];
              ldmatrix_x4_trans(va, vbase + (((2 * dt + (mi & 1)) ^ tok) << 4));
              mma_bf16(o[dt], va[0], va[1], va[2], va[3], pH[0], pH[1]);
              mma_bf16(o[dt], va[0], va[1], va[2], va[3], pL[0], pL[1]);
            }
          }
          __syncwarp();
          cslot = (cslot + 4) & (kDepth - 1);
          issue_next();
        }

#pragma unroll
        for (int sh = 4; sh <= 16; sh <<= 1) {
          l0 += __shfl_xor_sync(0xffffffffu, l0, sh);
          l1 += __shfl_xor_sync(0xffffffffu, l1, sh);
        }

        // ---- merge inside the CTA: every warp leaves its state in shared memory, the first warp of each run of
        // chunks of one (request, kv head) adds the others' in chunk order
        if (valid) {
#pragma unroll
          for (int j = 0; j < 32; ++j) s_o[(warp * 32 + j) * 32 + lane] = o[j >> 2][j & 3];
          if (g == 0) *reinterpret_cast<float4*>(s_ml + warp * 16 + 4 * t) = make_float4(m0, l0, m1, l1);
        }
        __syncthreads();
        if (valid && (it.chunk == 0 || warp == 0)) {
          const int count = min(kWarps - warp, it.nch - it.chunk);
          float M0 = m0, M1 = m1;
          for (int w = 1; w < count; ++w) {
            const float4 ml = *reinterpret_cast<const float4*>(s_ml + (warp + w) * 16 + 4 * t);
            M0 = fmaxf(M0, ml.x), M1 = fmaxf(M1, ml.z);
          }
          {
            const float c0 = exp2f(m0 - M0), c1 = exp2f(m1 - M1);
            l0 *= c0, l1 *= c1;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              o[j][0] *= c0, o[j][2] *= c0;
              o[j][1] *= c1, o[j][3] *= c1;
            }
          }
          for (int w = 1; w < count; ++w) {
            const float4 ml = *reinterpret_cast<const float4*>(s_ml + (warp + w) * 16 + 4 * t);
            const float e0 = exp2f(ml.x - M0), e1 = exp2f(ml.z - M1);
            l0 = fmaf(e0, ml.y, l0), l1 = fmaf(e1, ml.w, l1);
            const float* so = s_o + (size_t)(warp + w) * 32 * 32 + lane;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              o[j][0] = fmaf(e0, so[(j * 4 + 0) * 32], o[j][0]);
              o[j][1] = fmaf(e1, so[(j * 4 + 1) * 32], o[j][1]);
              o[j][2] = fmaf(e0, so[(j * 4 + 2) * 32], o[j][2]);
              o[j][3] = fmaf(e1, so[(j * 4 + 3) * 32], o[j][3]);
            }
          }

          uint16_t* arow = p.attn;  // operand of the O projection: feature (h G + head) 128 + d of request r
          const int Kq = p.nq * kHeadDim, feat0 = h * G * kHeadDim;
          if (it.chunk == 0 && count == it.nch) {
            // the whole (request, kv head): d = 16 dt + g (+ 8) is element g of chunk 2 dt (+ 1) of the head
            const float i0 = 1.0f / l0, i1 = 1.0f / l1;
            const int fp = frag_pos(g);
#pragma unroll
            for (int dt = 0; dt < 8; ++dt) {
              if (2 * t < G) {
                const int f = feat0 + (2 * t) * kHeadDim + 16 * dt;
                arow[operand_chunk(Kq, r, f) + fp] = f32_to_bf16(o[dt][0] * i0);
                arow[operand_chunk(Kq, r, f + 8) + fp] = f32_to_bf16(o[dt][2] * i0);
              }
              if (2 * t + 1 < G) {
                const int f = feat0 + (2 * t + 1) * kHeadDim + 16 * dt;
                arow[operand_chunk(Kq, r, f) + fp] = f32_to_bf16(o[dt][1] * i1);
                arow[operand_chunk(Kq, r, f + 8) + fp] = f32_to_bf16(o[dt][3] * i1);
              }
            }
          } else {
            // the run is a part of the (request, kv head): publish it [d][Gs heads]; the last run to finish merges
            float* pa = p.pacc + (size_t)item * kHeadDim * Gs;
            float* pm = p.pml + (size_t)item * Gs * 2;
            if (2 * t < Gs) {
#pragma unroll
              for (int dt = 0; dt < 8; ++dt) {
                *reinterpret_cast<float2*>(pa + (size_t)(16 * dt + g) * Gs + 2 * t) = make_float2(o[dt][0], o[dt][1]);
                *reinterpret_cast<float2*>(pa + (size_t)(16 * dt + g + 8) * Gs + 2 * t) = make_float2(o[dt][2], o[dt][3]);
              }
              if (g == 0) *reinterpret_cast<float4*>(pm + 4 * t) = make_float4(M0, l0, M1, l1);
            }
            __syncwarp();
            const int i0 = item - it.chunk;  // first item of this (request, kv head)
            const int runs = ((i0 + it.nch - 1) / kWarps) - (i0 / kWarps) + 1;
            int last = 0;
            if (lane == 0) {
              __threadfence();  // the other lanes' stores, ordered before this by the warp barrier, become visible too
              last = atom_acq_rel_add_s32(p.attn_counters + r * p.nkv + h, 1) == runs - 1;
            }
            last = __shfl_sync(0xffffffffu, last, 0);
            if (last) {
              __threadfence();
              // lane: dims 4 lane .. 4 lane + 3, all heads; runs start at i0 and at every multiple of 16 after it
              float M[8], den[8], num[4][8];
#pragma unroll
              for (int a = 0; a < 8; ++a) {
                M[a] = -INFINITY, den[a] = 0.0f;
                num[0][a] = num[1][a] = num[2][a] = num[3][a] = 0.0f;
              }
              for (int c = 0; c < runs; ++c) {
                const int slot = c == 0 ? i0 : (i0 / kWarps + c) * kWarps;
                const float* pmc = p.pml + (size_t)slot * Gs * 2;
#pragma unroll
                for (int a = 0; a < 8; ++a)
                  if (a < Gs) M[a] = fmaxf(M[a], __ldcg(pmc + 2 * a));
              }
#pragma unroll 2
              for (int c = 0; c < runs; ++c) {
                const size_t slot = (size_t)(c == 0 ? i0 : (i0 / kWarps + c) * kWarps);
                const float* pmc = p.pml + slot * Gs * 2;
                const float* pac = p.pacc + slot * kHeadDim * Gs + (size_t)(4 * lane) * Gs;
                float e[8];
#pragma unroll
                for (int a = 0; a < 8; ++a) {
                  e[a] = 0.0f;
                  if (a < Gs) {
                    const float2 ml = __ldcg(reinterpret_cast<const float2*>(pmc + 2 * a));
                    e[a] = exp2f(ml.x - M[a]);
                    den[a] = fmaf(e[a], ml.y, den[a]);
                  }
                }
#pragma unroll
                for (int dd = 0; dd < 4; ++dd)
#pragma unroll
                  for (int a2 = 0; a2 < 4; ++a2)
                    if (2 * a2 < Gs) {
                      const float2 u = __ldcg(reinterpret_cast<const float2*>(pac + (size_t)dd * Gs + 2 * a2));
                      num[dd][2 * a2] = fmaf(e[2 * a2], u.x, num[dd][2 * a2]);
                      num[dd][2 * a2 + 1] = fmaf(e[2 * a2 + 1], u.y, num[dd][2 * a2 + 1]);
                    }
              }
              // dims 4 lane .. + 3: elements (lane & 1) * 4 .. + 3 of chunk lane >> 1 of the head
              const int e0 = (lane & 1) * 4;
#pragma unroll
              for (int a = 0; a < 8; ++a)
                if (a < G) {
                  uint16_t* d = arow + operand_chunk(Kq, r, feat0 + a * kHeadDim + (lane >> 1) * 8);
#pragma unroll
                  for (int dd = 0; dd < 4; ++dd) d[frag_pos(e0 + dd)] = f32_to_bf16(num[dd][a] / den[a]);
                }
              if (lane == 0) p.attn_counters[r * p.nkv + h] = 0;
            }
          }
        }
        __syncthreads();  // the next round reuses the shared-memory states
      }
      // the activation buffers were written with ordinary stores; bulk copies (async proxy) write them next
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }

    if (!grid_barrier(ph)) {
      cp_async_wait<0>();
      return;
    }
    if (D.type == PH_GEMM && D.epi == EPI_F32 && cta == 0 && threadIdx.x < p.n) {
      float bv = -INFINITY;
      int bi = 0x7fffffff;
      for (int c = 0; c < ncta; ++c) {
        const float2 v = __ldcg(p.amax + (size_t)c * 16 + threadIdx.x);
        const int oi = __float_as_int(v.y);
        if (v.x > bv || (v.x == bv && oi < bi)) bv = v.x, bi = oi;
      }
      p.next[threadIdx.x] = bi == 0x7fffffff ? 0 : bi;
    }
  }
  cp_async_wait<0>();
}

int g_fused_max_ctas = -1;

}  // namespace

size_t fused_smem_bytes() { return kSmemBytes; }

cudaError_t fused_init(int* max_ctas) {
  if (g_fused_max_ctas < 0) {
    int dev = 0, sms = 0, per_sm = 0, coop = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(fused_step_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e == cudaSuccess)
      e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fused_step_kernel, kFusedThreads, kSmemBytes);
    if (e != cudaSuccess) return e;
    g_fused_max_ctas = (coop && per_sm >= 1) ? sms : 0;
  }
  *max_ctas = g_fused_max_ctas;
  return cudaSuccess;
}

cudaError_t launch_fused_step(const FusedStep& p, int ctas, cudaStream_t s) {
  if (ctas < 1 || ctas > g_fused_max_ctas) return cudaErrorInvalidValue;
  void* args[] = {const_cast<FusedStep*>(&p)};
  return cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(fused_step_kernel), dim3(ctas), dim3(kFusedThreads),
                                     args, kSmemBytes, s);
}

}  // namespace q4d
