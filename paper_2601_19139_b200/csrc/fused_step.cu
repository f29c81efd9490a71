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

constexpr int kWarps = 8;
constexpr int kDepth = 8;             // ring slots per warp (power of two)
constexpr int kSlot = 2304;           // 16 rows x 128 B of codes (16-byte chunks XOR-swizzled) + 16 x (4 scales + 4 biases)
constexpr int kSlotSb = 2048;         // offset of the scales/biases inside a slot
constexpr int kActStride = 2 * kFusedSliceK + 16;  // bytes per request row of a staged slice (pad: no bank conflicts)
constexpr int kActBytes = 16 * kActStride + (kFusedSliceK / 64) * 16 * 4;  // rows + group sums
constexpr int kRingBytes = kWarps * kDepth * kSlot;
constexpr int kPartFloats = kWarps * 256;          // accumulators of the warps that share a tile
constexpr int kMiscFloats = 16 + 256 + 128 + 128;  // inv, reduction scratch, argmax values, argmax indices
constexpr size_t kSmemBytes = (size_t)kRingBytes + 2 * kActBytes + (kPartFloats + kMiscFloats) * 4;
constexpr float kScaleLog2 = 0.08838834764831845f * 1.4426950408889634f;  // log2(e) / sqrt(128)
constexpr unsigned long long kBarrierTimeoutNs = 2000000000ull;

static_assert((kDepth & (kDepth - 1)) == 0, "ring depth must be a power of two");
static_assert(kDepth == 8, "the attention wait pattern assumes eight slots");
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
__device__ __forceinline__ void red_release_add_u32(unsigned int* p, unsigned int v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ int atom_acq_rel_add_s32(int* p, int v) {
  int old;
  asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
  return old;
}
__device__ __forceinline__ void prefetch_l1(const void* p) { asm volatile("prefetch.global.L1 [%0];" ::"l"(p)); }

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
// Position of element e of a chunk of 8 in fragment order {0,4,1,5,2,6,3,7}.
__device__ __forceinline__ int frag_pos(int e) { return (e & 3) * 2 + (e >> 2); }

// A CTA's tiles are processed in groups: with five or more tiles left a warp owns a whole tile, with three or four
// two warps share a tile (half of every slice each), with one or two four warps do.
__device__ __forceinline__ void group_shape(int remaining, int& T_g, int& ksplit) {
  if (remaining >= 5) {
    T_g = remaining < 8 ? remaining : 8, ksplit = 1;
  } else if (remaining >= 3) {
    T_g = remaining, ksplit = 2;
  } else {
    T_g = remaining, ksplit = 4;
  }
}
// The quads (256 input features) of slice s that belong to part pw of ksplit: first quad and count.
__device__ __forceinline__ void my_quads(int K, int s, int ksplit, int pw, int& first, int& count) {
  const int nqs = min(4, (K - s * kFusedSliceK) >> 8), qpp = 4 / ksplit;
  first = pw * qpp;
  const int c = nqs - first;
  count = c < 0 ? 0 : (c > qpp ? qpp : c);
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
  it.chunk = rem / p.nkv;
  it.kvh = rem - it.chunk * p.nkv;
  it.T = p.lens[r] + 1;
  const int nb = (it.T + 15) >> 4;
  it.nch = (nb + p.chunk_blocks - 1) / p.chunk_blocks;
  it.blk0 = it.chunk * p.chunk_blocks;
  it.nblk = min(p.chunk_blocks, nb - it.blk0);
  return it;
}

// Position of a warp's prefetch in its stream of ring stages (warp-uniform except the lane's source pointers).
struct IssueState {
  int ph, type;
  // PH_GEMM: the walk over groups, slices and quads
  int t_lo, T_c, done, T_g, ksplit, S, K, s, qi, q_first, q_count, rows_done;
  const uint32_t* qw;
  const uint16_t* scales;
  const uint16_t* biases;
  const uint32_t* qrow[4];  // this lane's four 16-byte chunks of the tile's rows, input feature 0
  const uint16_t* sbrow;    // this lane's scale (lanes 0..15) or bias (16..31) row, group 0
  // PH_ATTN
  int item, st, nst, r, kvh, blk0, nblk, win;
  const uint16_t* kbase;
};

__global__ void __launch_bounds__(kFusedThreads, 1) fused_step_kernel(const FusedStep p) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ int s_abort;
  __shared__ __align__(8) uint64_t s_mbar[2];  // one per activation buffer
  unsigned char* acts = smem + kRingBytes;
  float* s_part = reinterpret_cast<float*>(acts + 2 * kActBytes);  // [8 values][8 warps][32 lanes]
  float* s_inv = s_part + kPartFloats;                             // [16]
  float* s_red = s_inv + 16;                                       // [16][16]
  float* s_bestv = s_red + 256;                                    // [8][16]
  int* s_besti = reinterpret_cast<int*>(s_bestv + 128);            // [8][16]

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
  iss.t_lo = iss.T_c = iss.done = iss.T_g = iss.ksplit = iss.S = iss.K = iss.s = iss.qi = 0;
  iss.q_first = iss.q_count = 0, iss.rows_done = -1;
  iss.qw = nullptr, iss.scales = nullptr, iss.biases = nullptr, iss.sbrow = nullptr;
  iss.qrow[0] = iss.qrow[1] = iss.qrow[2] = iss.qrow[3] = nullptr;
  iss.item = iss.st = iss.nst = iss.r = iss.kvh = iss.blk0 = iss.nblk = iss.win = 0;
  iss.kbase = nullptr;
  int islot = 0;

  // PH_GEMM: moves to the next (group, slice) at or after the current one in which this warp has quads.
  auto iss_gemm_seek = [&]() -> bool {
    for (;;) {
      if (iss.done >= iss.T_c) return false;
      group_shape(iss.T_c - iss.done, iss.T_g, iss.ksplit);
      const int tw = warp / iss.ksplit, pw = warp % iss.ksplit;
      if (tw < iss.T_g) {
        while (iss.s < iss.S) {
          my_quads(iss.K, iss.s, iss.ksplit, pw, iss.q_first, iss.q_count);
          if (iss.q_count > 0) break;
          ++iss.s;
        }
        if (iss.s < iss.S) {
          if (iss.rows_done != iss.done) {  // a new tile: this lane's row pointers
            const FusedDims& D = p.dims[dims_index(p, iss.ph)];
            const int tile = iss.t_lo + iss.done + tw;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int row = unit_row(D.epi, D.N, tile, i * 4 + (lane >> 3));
              iss.qrow[i] = iss.qw + (size_t)row * (iss.K >> 3) + (lane & 7) * 4;
            }
            const int row = unit_row(D.epi, D.N, tile, lane & 15);
            iss.sbrow = (lane < 16 ? iss.scales : iss.biases) + (size_t)row * (iss.K >> 6);
            iss.rows_done = iss.done;
          }
          return true;
        }
      }
      iss.done += iss.T_g;
      iss.s = 0;
    }
  };
  auto iss_attn_load = [&]() {
    const AttnItem it = decode_item(p, iss.item);
    iss.r = it.r, iss.kvh = it.kvh, iss.blk0 = it.blk0, iss.nblk = it.nblk;
    iss.nst = 4 * it.nblk, iss.st = 0;
  };
  auto iss_load_phase = [&]() {  // moves to the first phase at or after iss.ph in which this warp has stages
    while (iss.ph < p.ph_end) {
      const FusedDims& D = p.dims[dims_index(p, iss.ph)];
      iss.type = D.type;
      if (D.type == PH_GEMM) {
        iss.t_lo = (int)((long long)cta * D.ntiles / ncta);
        iss.T_c = (int)((long long)(cta + 1) * D.ntiles / ncta) - iss.t_lo;
        iss.done = 0, iss.s = 0, iss.qi = 0, iss.S = D.S, iss.K = D.K, iss.rows_done = -1;
        if (iss.T_c > 0) {
          const FusedPhase& P = p.phases[iss.ph];
          iss.qw = P.qw, iss.scales = P.scales, iss.biases = P.biases;
          if (iss_gemm_seek()) break;
        }
      } else if (D.type == PH_ATTN) {
        iss.item = cta + ncta * warp;
        if (iss.item < p.n_items) {
          iss.kbase = p.pool + (size_t)(2 * phase_layer(iss.ph)) * p.layer_elems;
          iss_attn_load();
          break;
        }
      }
      ++iss.ph;
    }
    if (iss.ph + 1 < p.ph_end) prefetch_l1(p.phases + iss.ph + 1);
  };
  // Issues the next stage of the stream (if any) into the next ring slot and closes a cp.async group either way.
  auto issue_next = [&]() {
    if (iss.ph < p.ph_end) {
      unsigned char* stg = ring + islot * kSlot;
      if (iss.type == PH_GEMM) {
        const int k = iss.s * kFusedSliceK + (iss.q_first + iss.qi) * 256;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int r = i * 4 + (lane >> 3);
          cp_async16(stg + r * 128 + (((lane & 7) ^ (r & 7)) << 4), iss.qrow[i] + (k >> 3));
        }
        cp_async8(stg + kSlotSb + (lane & 15) * 16 + (lane >> 4) * 8, iss.sbrow + (k >> 6));
        if (++iss.qi == iss.q_count) {
          iss.qi = 0;
          ++iss.s;
          if (!iss_gemm_seek()) {
            ++iss.ph;
            iss_load_phase();
          }
        }
      } else {
        const int b = iss.st >> 2, part = iss.st & 3;
        if (part == 0 && (b & 31) == 0) {
          const int idx = b + lane;
          iss.win = idx < iss.nblk ? p.bt[(size_t)iss.r * p.max_blocks + iss.blk0 + idx] : 0;
        }
        const int blk = __shfl_sync(0xffffffffu, iss.win, b & 31);
        const uint16_t* base = (part < 2 ? iss.kbase : iss.kbase + p.layer_elems) +
                               ((size_t)(blk * p.nkv + iss.kvh) * 16 + (part & 1) * 8) * kHeadDim;
        const unsigned char* src = reinterpret_cast<const unsigned char*>(base);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int c = i * 32 + lane, tok = c >> 4, c16 = c & 15;
          cp_async16(stg + tok * 256 + ((c16 ^ tok) << 4), src + c * 16);
        }
        if (++iss.st == iss.nst) {
          iss.item += ncta * kWarps;
          if (iss.item < p.n_items) {
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
      while (ld_acquire_u32(p.control) < bar_target) {
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
    if (ph + 1 < p.ph_end) prefetch_l1(p.phases + ph + 1);

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
      const FusedPhase& P = p.phases[ph];
      const int H = D.K, cpr = H >> 3, total = p.n * cpr;
      const int lo = (int)((long long)cta * total / ncta), hi = (int)((long long)(cta + 1) * total / ncta);
      if (hi > lo) {
        uint16_t* out = reinterpret_cast<uint16_t*>(P.out);
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
            const uint4 v = __ldcg(reinterpret_cast<const uint4*>(P.in + (size_t)r * H + kc * 8));
            const uint4 wv = *reinterpret_cast<const uint4*>(P.norm_w + kc * 8);
            const uint32_t e[4] = {v.x, v.y, v.z, v.w}, ww[4] = {wv.x, wv.y, wv.z, wv.w};
            uint32_t o[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
              o[j] = pack_bf16x2(bf16_lo(e[j]) * inv * bf16_lo(ww[j]), bf16_hi(e[j]) * inv * bf16_hi(ww[j]));
            *reinterpret_cast<uint4*>(out + (size_t)r * H + kc * 8) = permute_chunk(make_uint4(o[0], o[1], o[2], o[3]));
          }
          __syncthreads();
        }
      }
    } else if (D.type == PH_GEMM) {
      // ---------------------------------------------------------- projection
      const int t_lo = (int)((long long)cta * D.ntiles / ncta);
      const int T_c = (int)((long long)(cta + 1) * D.ntiles / ncta) - t_lo;
      if (T_c > 0) {
        const FusedPhase& P = p.phases[ph];
        const uint16_t* in = P.in;  // the operand as its producer wrote it: chunks of 8 in fragment order
        const int K = D.K, S = D.S;

        // A slice of the operand goes to shared memory as one bulk copy per request row, tracked by the buffer's
        // mbarrier; the sums over every group of 64 input features come from the tensor cores (ones x operand).
        auto stage_issue = [&](int slice, int idx) {
          if (threadIdx.x == 0) {
            const int k0 = slice * kFusedSliceK, bytes = min(kFusedSliceK, K - k0) * 2;
            unsigned char* dst = acts + (idx & 1) * kActBytes;
            mbar_expect_tx(&s_mbar[idx & 1], (uint32_t)(bytes * p.n));
            for (int r = 0; r < p.n; ++r)
              bulk_copy_g2s(dst + r * kActStride, in + (size_t)r * K + k0, (uint32_t)bytes, &s_mbar[idx & 1]);
          }
        };
        auto stage_finish = [&](int slice, int idx) {
          if (!mbar_wait(&s_mbar[idx & 1], (uint32_t)((idx >> 1) & 1))) {
            if (lane == 0) atomicExch(p.control + 1, 2u);  // the copy never landed: report, results are void
          }
          const unsigned char* sB = acts + (idx & 1) * kActBytes;
          float* sX = reinterpret_cast<float*>(acts + (idx & 1) * kActBytes + 16 * kActStride);
          const int groups = min(kFusedSliceK, K - slice * kFusedSliceK) >> 6;
          const uint32_t one2 = 0x3F803F80u;  // bf16 {1, 1}
          for (int gi = warp; gi < groups; gi += kWarps) {
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
              const unsigned char* bp = sB + (nt * 8 + g) * kActStride + gi * 128 + t * 32;
              const uint4 b0 = *reinterpret_cast<const uint4*>(bp), b1 = *reinterpret_cast<const uint4*>(bp + 16);
              float d[4];
              mma_bf16_first(d, one2, one2, one2, one2, b0.x, b0.y);
              mma_bf16(d, one2, one2, one2, one2, b0.z, b0.w);
              mma_bf16(d, one2, one2, one2, one2, b1.x, b1.y);
              mma_bf16(d, one2, one2, one2, one2, b1.z, b1.w);
              if (g == 0) *reinterpret_cast<float2*>(sX + gi * 16 + nt * 8 + 2 * t) = make_float2(d[0], d[1]);
            }
          }
        };

        // prologue: the first slice
        stage_issue(0, staged);
        stage_finish(0, staged);
        __syncthreads();
        int flat = staged++;  // index of the current slice's staging: buffer flat & 1

        int done = 0;
#pragma unroll 1
        while (done < T_c) {
          int T_g, ksplit;
          group_shape(T_c - done, T_g, ksplit);
          const int tw = warp / ksplit, pw = warp % ksplit;
          const bool mine = tw < T_g, lead = mine && pw == 0;
          const int tile = t_lo + done + tw;
          const bool more_groups = done + T_g < T_c;
          float acc[2][4];
#pragma unroll
          for (int nt = 0; nt < 2; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.0f;
          // the lead warp of a residual tile fetches the old values early
          uint16_t xold[8];
          if (lead && D.epi == EPI_RESIDUAL) {
            const uint16_t* out = reinterpret_cast<const uint16_t*>(P.out);
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
              for (int c = 0; c < 4; ++c) {
                const int req = nt * 8 + 2 * t + (c & 1), row = tile * 16 + g + (c >> 1) * 8;
                xold[nt * 4 + c] = (req < p.n && row < D.N) ? __ldcg(out + (size_t)req * P.out_stride + row) : (uint16_t)0;
              }
          }

#pragma unroll 1
          for (int s = 0; s < S; ++s) {
            const bool has_next = (s + 1 < S) || more_groups;
            const int next_slice = (s + 1 < S) ? s + 1 : 0;
            const int next_idx = staged;
            if (has_next) stage_issue(next_slice, next_idx);
            if (mine) {
              int q_first, q_count;
              my_quads(K, s, ksplit, pw, q_first, q_count);
              const unsigned char* sB = acts + (flat & 1) * kActBytes;
              const float* sX = reinterpret_cast<const float*>(sB + 16 * kActStride);
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
                    const unsigned char* bp = sB + (nt * 8 + g) * kActStride + gidx * 128 + t * 32;
                    bf[nt][0] = *reinterpret_cast<const uint4*>(bp);
                    bf[nt][1] = *reinterpret_cast<const uint4*>(bp + 16);
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
            if (has_next) {
              stage_finish(next_slice, next_idx);
              ++staged;
            }
            __syncthreads();
            flat = next_idx;
          }

          // ---- warps that shared a tile: the lead warp adds the others' sums in warp order
          if (ksplit > 1) {
            if (mine && !lead) {
#pragma unroll
              for (int i = 0; i < 8; ++i) s_part[(i * kWarps + warp) * 32 + lane] = acc[i >> 2][i & 3];
            }
            __syncthreads();
            if (lead) {
              for (int o = 1; o < ksplit; ++o)
#pragma unroll
                for (int i = 0; i < 8; ++i) acc[i >> 2][i & 3] += s_part[(i * kWarps + warp + o) * 32 + lane];
            }
          }

          // ---- epilogue: acc[nt][c]: row g + 8 * (c >> 1) of the tile, request nt * 8 + 2t + (c & 1)
          if (lead) {
            if (D.epi == EPI_SILU_PACK) {
              uint16_t* out = reinterpret_cast<uint16_t*>(P.out);
              const int col = tile * 8 + frag_pos(g);  // the tile's 8 columns are one chunk of the down projection's operand
#pragma unroll
              for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                  const int req = nt * 8 + 2 * t + j;
                  const float gt = bf16_round(acc[nt][j]), up = bf16_round(acc[nt][2 + j]);
                  if (req < p.n) out[(size_t)req * P.out_stride + col] = f32_to_bf16((gt / (1.0f + expf(-gt))) * up);
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
              uint16_t* out = reinterpret_cast<uint16_t*>(P.out);
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
                    out[(size_t)req * P.out_stride + row] = y;
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
      const FusedPhase& P = p.phases[ph];
      const int layer = phase_layer(ph);
      uint16_t* kpool_w = p.pool + (size_t)(2 * layer) * p.layer_elems;
#pragma unroll 1
      for (int item = cta + ncta * warp; item < p.n_items; item += ncta * kWarps) {
        const AttnItem it = decode_item(p, item);
        const int r = it.r, h = it.kvh, pos = it.T - 1;
        const uint16_t* qrow = p.qkv + (size_t)r * nqkv;
        const bool appends = it.chunk == it.nch - 1;

        // loads first: q of the G query heads, k and v of the new token, rotary table, block id of the append
        uint32_t qa[8][4];
        uint32_t wa = 0u, wb = 0u, nv_a = 0u, nv_b = 0u;
        int append_blk = 0;
        {
          const uint16_t* q0 = qrow + (size_t)(h * G + g) * kHeadDim;
          const uint16_t* q1 = q0 + 8 * kHeadDim;
          const bool v0 = g < G, v1 = g + 8 < G;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            qa[ks][0] = v0 ? __ldcg(reinterpret_cast<const uint32_t*>(q0 + 16 * ks + 2 * t)) : 0u;
            qa[ks][1] = v1 ? __ldcg(reinterpret_cast<const uint32_t*>(q1 + 16 * ks + 2 * t)) : 0u;
            qa[ks][2] = v0 ? __ldcg(reinterpret_cast<const uint32_t*>(q0 + 16 * ks + 2 * t + 8)) : 0u;
            qa[ks][3] = v1 ? __ldcg(reinterpret_cast<const uint32_t*>(q1 + 16 * ks + 2 * t + 8)) : 0u;
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
        {
          if (P.q_norm) {
            float ss0 = 0.0f, ss1 = 0.0f;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              ss0 += bf16_lo(qa[ks][0]) * bf16_lo(qa[ks][0]) + bf16_hi(qa[ks][0]) * bf16_hi(qa[ks][0]) +
                     bf16_lo(qa[ks][2]) * bf16_lo(qa[ks][2]) + bf16_hi(qa[ks][2]) * bf16_hi(qa[ks][2]);
              ss1 += bf16_lo(qa[ks][1]) * bf16_lo(qa[ks][1]) + bf16_hi(qa[ks][1]) * bf16_hi(qa[ks][1]) +
                     bf16_lo(qa[ks][3]) * bf16_lo(qa[ks][3]) + bf16_hi(qa[ks][3]) * bf16_hi(qa[ks][3]);
            }
            ss0 += __shfl_xor_sync(0xffffffffu, ss0, 1);
            ss0 += __shfl_xor_sync(0xffffffffu, ss0, 2);
            ss1 += __shfl_xor_sync(0xffffffffu, ss1, 1);
            ss1 += __shfl_xor_sync(0xffffffffu, ss1, 2);
            const float inv0 = 1.0f / sqrtf(ss0 * (1.0f / kHeadDim) + p.eps);
            const float inv1 = 1.0f / sqrtf(ss1 * (1.0f / kHeadDim) + p.eps);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
#pragma unroll
              for (int rr = 0; rr < 4; ++rr) {
                const int col = 16 * ks + 2 * t + (rr >> 1) * 8;
                const uint32_t nw = *reinterpret_cast<const uint32_t*>(P.q_norm + col);
                const float inv = (rr & 1) ? inv1 : inv0;
                qa[ks][rr] = pack_bf16x2(bf16_lo(qa[ks][rr]) * inv * bf16_lo(nw), bf16_hi(qa[ks][rr]) * inv * bf16_hi(nw));
              }
          }
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
              const int col = 16 * ks + 2 * t + hf * 8;  // even, < 64
              const float4 cs = *reinterpret_cast<const float4*>(p.rope + ((size_t)pos * 64 + col) * 2);  // c0 s0 c1 s1
#pragma unroll
              for (int rw = 0; rw < 2; ++rw) {
                const int rr = hf * 2 + rw;
                const float a0 = bf16_lo(qa[ks][rr]), a1 = bf16_hi(qa[ks][rr]);
                const float b0 = bf16_lo(qa[ks + 4][rr]), b1 = bf16_hi(qa[ks + 4][rr]);
                qa[ks][rr] = pack_bf16x2(a0 * cs.x - b0 * cs.y, a1 * cs.z - b1 * cs.w);
                qa[ks + 4][rr] = pack_bf16x2(b0 * cs.x + a0 * cs.y, b1 * cs.z + a1 * cs.w);
              }
            }
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

        float o[16][4];
#pragma unroll
        for (int j = 0; j < 16; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.0f;
        float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.0f, l_hi = 0.0f;

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

          // K: eight stages are committed after this issue; the two K halves are the oldest two
          issue_next();
          cp_async_wait<kDepth - 2>();
          __syncwarp();
          if (patch) {
            unsigned char* kd = (pos & 8) ? sK1 : sK0;
            *reinterpret_cast<uint32_t*>(kd + off_a) = nk_a;
            *reinterpret_cast<uint32_t*>(kd + off_b) = nk_b;
            __syncwarp();
          }
          // scores S[head][token] for the 16 tokens of the block
          float s[2][4];
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const unsigned char* sK = j ? sK1 : sK0;
            s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.0f;
#pragma unroll
            for (int kp = 0; kp < 4; ++kp) {
              uint32_t kb[4];
              const int tok = lane & 7, chunk = 4 * kp + (lane >> 3);
              ldmatrix_x4(kb, sK + tok * 256 + ((chunk ^ tok) << 4));
              mma_bf16(s[j], qa[2 * kp][0], qa[2 * kp][1], qa[2 * kp][2], qa[2 * kp][3], kb[0], kb[1]);
              mma_bf16(s[j], qa[2 * kp + 1][0], qa[2 * kp + 1][1], qa[2 * kp + 1][2], qa[2 * kp + 1][3], kb[2], kb[3]);
            }
          }
          __syncwarp();
          // the K slots are free: two more stages go out while V is awaited
          issue_next();
          issue_next();
          if (tile * 16 + 16 > it.T) {  // ragged last block: tokens at or beyond T do not exist
#pragma unroll
            for (int j = 0; j < 2; ++j)
#pragma unroll
              for (int c = 0; c < 4; ++c)
                if (tile * 16 + 8 * j + 2 * t + (c & 1) >= it.T) s[j][c] = -INFINITY;
          }

          // online softmax, rows g (lo) and g + 8 (hi); m is kept in log2 units
          float mx_lo = fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1]));
          float mx_hi = fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3]));
          mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
          mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
          mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
          mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
          const float mn_lo = fmaxf(m_lo, mx_lo * kScaleLog2), mn_hi = fmaxf(m_hi, mx_hi * kScaleLog2);
          const bool grow = (mn_lo > m_lo) || (mn_hi > m_hi);
          if (__any_sync(0xffffffffu, grow)) {
            const float c_lo = exp2f(m_lo - mn_lo), c_hi = exp2f(m_hi - mn_hi);
            l_lo *= c_lo;
            l_hi *= c_hi;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              o[j][0] *= c_lo, o[j][1] *= c_lo;
              o[j][2] *= c_hi, o[j][3] *= c_hi;
            }
            m_lo = mn_lo, m_hi = mn_hi;
          }
          uint32_t pH[4], pL[4];  // A fragments of P: hi and lo bf16 terms
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const float p0 = exp2f(fmaf(s[j][0], kScaleLog2, -m_lo)), p1 = exp2f(fmaf(s[j][1], kScaleLog2, -m_lo));
            const float p2 = exp2f(fmaf(s[j][2], kScaleLog2, -m_hi)), p3 = exp2f(fmaf(s[j][3], kScaleLog2, -m_hi));
            l_lo += p0 + p1;
            l_hi += p2 + p3;
            const uint32_t h01 = pack_bf16x2(p0, p1), h23 = pack_bf16x2(p2, p3);
            pH[2 * j] = h01, pH[2 * j + 1] = h23;
            pL[2 * j] = pack_bf16x2(p0 - bf16_lo(h01), p1 - bf16_hi(h01));
            pL[2 * j + 1] = pack_bf16x2(p2 - bf16_lo(h23), p3 - bf16_hi(h23));
          }

          // V: ten stages are committed since the block began; the V halves are the third and fourth
          cp_async_wait<kDepth - 2>();
          __syncwarp();
          if (patch) {
            unsigned char* vd = (pos & 8) ? sV1 : sV0;
            *reinterpret_cast<uint32_t*>(vd + off_a) = nv_a;
            *reinterpret_cast<uint32_t*>(vd + off_b) = nv_b;
            __syncwarp();
          }
          // O[head][d] += P[head][token] V[token][d]
#pragma unroll
          for (int jp = 0; jp < 8; ++jp) {
            uint32_t vb[4];
            const int i = lane >> 3, tok = lane & 7, chunk = 2 * jp + (i >> 1);
            ldmatrix_x4_trans(vb, ((i & 1) ? sV1 : sV0) + tok * 256 + ((chunk ^ tok) << 4));
            mma_bf16(o[2 * jp], pH[0], pH[1], pH[2], pH[3], vb[0], vb[1]);
            mma_bf16(o[2 * jp], pL[0], pL[1], pL[2], pL[3], vb[0], vb[1]);
            mma_bf16(o[2 * jp + 1], pH[0], pH[1], pH[2], pH[3], vb[2], vb[3]);
            mma_bf16(o[2 * jp + 1], pL[0], pL[1], pL[2], pL[3], vb[2], vb[3]);
          }
          __syncwarp();
          cslot = (cslot + 4) & (kDepth - 1);
          issue_next();
        }

        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);

        uint16_t* arow = p.attn + (size_t)r * p.nq * kHeadDim + (size_t)h * G * kHeadDim;
        if (it.nch == 1) {
          const float i_lo = 1.0f / l_lo, i_hi = 1.0f / l_hi;
          const int p0 = frag_pos(2 * t), p1 = frag_pos(2 * t + 1);  // chunk j of the head, elements 2t and 2t + 1
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            if (g < G) {
              uint16_t* d = arow + (size_t)g * kHeadDim + 8 * j;
              d[p0] = f32_to_bf16(o[j][0] * i_lo), d[p1] = f32_to_bf16(o[j][1] * i_lo);
            }
            if (g + 8 < G) {
              uint16_t* d = arow + (size_t)(g + 8) * kHeadDim + 8 * j;
              d[p0] = f32_to_bf16(o[j][2] * i_hi), d[p1] = f32_to_bf16(o[j][3] * i_hi);
            }
          }
          continue;
        }

        // publish the chunk's partial result; the last chunk to finish merges all of them in chunk order
        {
          float* pa = p.pacc + (size_t)item * G * kHeadDim;
          float* pm = p.pml + (size_t)item * G * 2;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            if (g < G) *reinterpret_cast<float2*>(pa + (size_t)g * kHeadDim + 8 * j + 2 * t) = make_float2(o[j][0], o[j][1]);
            if (g + 8 < G)
              *reinterpret_cast<float2*>(pa + (size_t)(g + 8) * kHeadDim + 8 * j + 2 * t) = make_float2(o[j][2], o[j][3]);
          }
          if (t == 0) {
            if (g < G) *reinterpret_cast<float2*>(pm + g * 2) = make_float2(m_lo, l_lo);
            if (g + 8 < G) *reinterpret_cast<float2*>(pm + (g + 8) * 2) = make_float2(m_hi, l_hi);
          }
          __syncwarp();
          int last = 0;
          if (lane == 0) {
            __threadfence();  // the other lanes' stores, ordered before this by the warp barrier, become visible too
            last = atom_acq_rel_add_s32(p.attn_counters + r * p.nkv + h, 1) == it.nch - 1;
          }
          last = __shfl_sync(0xffffffffu, last, 0);
          if (!last) continue;
          __threadfence();
          const int item0 = p.item_prefix[r] + h;  // chunk c of this (request, kv head) is item0 + c * nkv
          for (int a = 0; a < G; ++a) {
            float M = -INFINITY;
            for (int c = lane; c < it.nch; c += 32)
              M = fmaxf(M, __ldcg(p.pml + ((size_t)(item0 + c * p.nkv) * G + a) * 2));
#pragma unroll
            for (int sh = 16; sh > 0; sh >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, sh));
            float4 num = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            float den = 0.0f;
#pragma unroll 4
            for (int c = 0; c < it.nch; ++c) {
              const size_t row = (size_t)(item0 + c * p.nkv) * G + a;
              const float2 ml = __ldcg(reinterpret_cast<const float2*>(p.pml + row * 2));
              const float4 u = __ldcg(reinterpret_cast<const float4*>(p.pacc + row * kHeadDim + lane * 4));
              const float e = exp2f(ml.x - M);
              num.x = fmaf(e, u.x, num.x), num.y = fmaf(e, u.y, num.y);
              num.z = fmaf(e, u.z, num.z), num.w = fmaf(e, u.w, num.w);
              den = fmaf(e, ml.y, den);
            }
            // dims 4 * lane .. + 3: elements (lane & 1) * 4 .. + 3 of chunk lane >> 1
            uint16_t* d = arow + (size_t)a * kHeadDim + (lane >> 1) * 8;
            const int e0 = (lane & 1) * 4;
            d[frag_pos(e0)] = f32_to_bf16(num.x / den), d[frag_pos(e0 + 1)] = f32_to_bf16(num.y / den);
            d[frag_pos(e0 + 2)] = f32_to_bf16(num.z / den), d[frag_pos(e0 + 3)] = f32_to_bf16(num.w / den);
          }
          if (lane == 0) p.attn_counters[r * p.nkv + h] = 0;
        }
      }
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
