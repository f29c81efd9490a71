// Fused dequantise-and-multiply of 4-bit affine group-64 weights on the fifth-generation tensor cores
// (tcgen05.mma with the weight operand in tensor memory).
//
//   y[r][j] = sum_g scale[j][g] * (sum_{k in g} q[j][k] x[r][k]) + bias[j][g] * (sum_{k in g} x[r][k])
//
// A CTA owns one tile of 128 weight rows and one part of K.  Row i of the tile is lane i of tensor memory: the thread
// that owns the lane unpacks the row's 4-bit codes into exact bf16 integers 16 + q (one shift and one logic operation
// per pair of codes) and stores them with tcgen05.st as the A operand of a 128 x 16 x 64 product; the activations of
// the 16 requests are the B operand, read from shared memory in the layout the tensor core wants (the producing
// kernels write it that way, so a stage is one bulk copy).  Every group of 64 input features gets its own 16-column
// fp32 accumulator, which is read back (tcgen05.ld) and folded into registers with the group's scale and bias:
// products are exact, accumulation is fp32, and no dequantised weight is ever rounded to bf16.  The offset 16 leaves
// through the bias term (bias - 16 scale multiplies the group's sum of x).
//
// Roles (warp-specialised, 13 warps):
//   warps 0..3  unpack: wait for a stage of packed codes (128 rows x 256 features, brought by TMA with the 128-byte
//               swizzle, so that a lane reads its row's 16-byte chunks without bank conflicts), unpack, store A.
//   warps 4..7  scale/bias: wait for a group's MMAs, read its accumulator, acc += scale * D + (bias - 16 scale) * X
//               with packed fp32 FMAs; their registers hold the tile's running sums.  Scales and biases of the
//               thread's row arrive through a private cp.async ring, six stages ahead.
//   warp 8      producer (one thread): tensor-map loads of the codes (started before the preceding kernel is
//               awaited: weights do not depend on it) and bulk copies of the operand and its group sums.
//   warps 9..12 MMA issue, one thread each, warp 9 + g for the groups that pass through A slot g (a single thread
//               issues a group's four MMAs and its commit in about a thousand cycles: too slow for all groups);
//               warp 9 owns the tensor-memory allocation.
// Four A slots and eight accumulator slots of tensor memory keep the three stages of the pipeline apart.
//
// K is cut into parts across CTAs where the tiles alone would not fill the machine; the parts of a tile meet in
// global scratch and the last CTA to arrive adds them in part order (deterministic) and applies the epilogue.
#include <cuda.h>

#include <mutex>
#include <unordered_map>

#include "common.cuh"
#include "kernels.h"
#include "launch.h"

namespace q4d {

namespace {

constexpr int kUmThreads = 32 * 13;
constexpr int kUmWStages = 4;                      // stages of codes in flight
constexpr int kUmWStage = 128 * 128;               // 128 rows x 256 codes
constexpr int kUmBStage = 32 * 256 + 4 * 16 * 4;   // 256 features x 16 requests bf16 (8 KB) + the 4 groups' sums
constexpr int kUmBStages = 4;
constexpr int kUmTmemCols = 256;                   // A: 4 slots x 32 columns at 0; D: 8 slots x 16 columns at 128
constexpr uint32_t kUmDCol0 = 128;
constexpr int kUmSbStages = 6;                     // stages of scales and biases in flight (one 16-byte entry per row)
constexpr int kUmSbStage = 128 * 16;
constexpr int kUmSmem = kUmWStages * kUmWStage + kUmBStages * kUmBStage + kUmSbStages * kUmSbStage + 1024;  // + room to align to 1024

struct UmmaParams {
  const uint16_t* scales;
  const uint16_t* biases;
  const uint16_t* xb;  // operand [K/8][16][8] (chunks of 8 features in the order 0,4,1,5,2,6,3,7)
  const float* xs;     // group sums [K/64][16]
  void* out;
  uint16_t* out_xb;    // EPI_SILU_PACK: the next projection's operand [N/2/8][16][8]
  float* out_xs;       //                and its group sums [N/2/64][16]
  float2* argmax_partial;  // [tiles * 4][16]
  unsigned int* status;
  float* partial;      // [parts][tiles][128][16]
  int* counters;       // [tiles], zero between launches
  int N, K, n, out_stride, epilogue;
  int tiles, parts, ns;  // ns: stages of 256 features in K
};

__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c) {  // (a & b) | c
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

__device__ __forceinline__ void um_mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void um_mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void um_mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void um_bulk_g2s(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(smem_dst)),
               "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
// A box of the tensor map at element (x, row y) into shared memory (this GPU's memory only, no multicast).
__device__ __forceinline__ void um_tma_2d(void* smem_dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
                   smem_u32(smem_dst)),
               "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
               : "memory");
}
// Waits for the phase of the given parity.  Each try suspends the thread in hardware until the phase completes or the
// hint (in nanoseconds) runs out, so that waiting warps do not occupy issue slots and the shared-memory pipeline;
// gives up (false) after a bounded number of tries (about two seconds).
__device__ __forceinline__ bool um_mbar_wait(uint64_t* bar, uint32_t parity) {
  for (int tries = 0; tries < 20000; ++tries) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_u32(bar)), "r"(parity), "r"(100000u)
        : "memory");
    if (done) return true;
  }
  return false;
}
// The same for a whole warp: every lane polls, the verdict is the warp's (uniform control flow for the callers).
__device__ __forceinline__ bool um_mbar_wait_warp(uint64_t* bar, uint32_t parity) {
  for (int tries = 0; tries < 20000; ++tries) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_u32(bar)), "r"(parity), "r"(100000u)
        : "memory");
    if (__all_sync(0xffffffffu, done != 0u)) return true;
  }
  return false;
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D(128 x 16, f32, tensor memory) (+)= A(128 x 16 bf16, tensor memory) * B(16 x 16 bf16, shared memory, K-major)
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,"
      "%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
      "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]),
      "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]),
      "r"(r[31])
      : "memory");
}
// 16 accumulator columns of this lane as 8 pairs
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, unsigned long long (&v)[8]) {
  uint32_t u[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]), "=r"(u[8]), "=r"(u[9]),
        "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 8; ++i) asm("mov.b64 %0, {%1, %2};" : "=l"(v[i]) : "r"(u[2 * i]), "r"(u[2 * i + 1]));
}
// two fp32 FMAs in one instruction: c = a * b + c on both halves
__device__ __forceinline__ void ffma2(unsigned long long& c, unsigned long long a, unsigned long long b) {
  asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(c) : "l"(a), "l"(b));
}
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ float2 unpack2(unsigned long long v) {
  float2 r;
  asm("mov.b64 {%0, %1}, %2;" : "=f"(r.x), "=f"(r.y) : "l"(v));
  return r;
}

__device__ __forceinline__ void um_bar_sync_epilogue() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

__global__ void __launch_bounds__(kUmThreads, 2)
q4_umma_kernel(const UmmaParams p, const __grid_constant__ CUtensorMap map_codes) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t w_full[kUmWStages], w_empty[kUmWStages];
  __shared__ __align__(8) uint64_t b_full[kUmBStages], b_empty[kUmBStages];
  __shared__ __align__(8) uint64_t a_full[4];   // A slot g written by all unpack threads
  __shared__ __align__(8) uint64_t done[8];     // the MMAs of (stage & 1, g) have completed
  __shared__ __align__(8) uint64_t d_empty[8];  // accumulator slot read back by all scale/bias threads
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_is_last;

  grid_launch_dependents();

  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* sW = smem;                                 // code stages, 1024-byte aligned (swizzle atoms)
  unsigned char* sB = smem + kUmWStages * kUmWStage;
  unsigned char* sSb = sB + kUmBStages * kUmBStage;         // [stage][row]{4 scales, 4 biases}

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool silu = p.epilogue == EPI_SILU_PACK;
  const int half_n = p.N >> 1;
  const int tile = blockIdx.x / p.parts, part = blockIdx.x - tile * p.parts;
  const int j0 = (int)((long long)part * p.ns / p.parts), j1 = (int)((long long)(part + 1) * p.ns / p.parts);
  const int ns = j1 - j0;  // stages of this CTA
  // the tile's rows: two runs of 64 consecutive rows of the tensor (gate rows and the matching up rows for the SiLU tile)
  const int run0 = silu ? tile * 64 : tile * 128, run1 = silu ? half_n + tile * 64 : tile * 128 + 64;

  if (threadIdx.x == 0) {
    // one arrival per warp (its lane 0, after the warp has synchronised): arrivals on one barrier are serialised
    // shared-memory atomics, and 128 of them per group from every role occupied that unit for most of the time
    for (int s = 0; s < kUmWStages; ++s) um_mbar_init(&w_full[s], 1), um_mbar_init(&w_empty[s], 4);
    for (int s = 0; s < kUmBStages; ++s) um_mbar_init(&b_full[s], 1), um_mbar_init(&b_empty[s], 4);
    for (int g = 0; g < 4; ++g) um_mbar_init(&a_full[g], 4);
    for (int d = 0; d < 8; ++d) um_mbar_init(&done[d], 1), um_mbar_init(&d_empty[d], 4);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  auto load_codes = [&](int i) {  // stage i of this CTA into slot i % kUmWStages: two boxes of 64 rows x 128 bytes
    const int slot = i % kUmWStages;
    um_mbar_expect_tx(&w_full[slot], (uint32_t)kUmWStage);
    um_tma_2d(sW + slot * kUmWStage, &map_codes, (j0 + i) * 128, run0, &w_full[slot]);
    um_tma_2d(sW + slot * kUmWStage + 64 * 128, &map_codes, (j0 + i) * 128, run1, &w_full[slot]);
  };
  if (warp == 8 && lane == 0) {
    // Weights do not depend on the preceding kernel: fill the ring before anything else (tensor memory may still be
    // held by the preceding kernel's CTAs on this SM; the allocation below waits for it).
    for (int i = 0; i < kUmWStages && i < ns; ++i) load_codes(i);
  }
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)), "n"(kUmTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tbase = s_tmem_base;

  bool ok = true;
  unsigned long long acc[8];  // scale/bias warps: the row's 16 running sums as pairs
#pragma unroll
  for (int r = 0; r < 8; ++r) acc[r] = 0ull;

  if (warp == 8) {
    // ---- producer (one thread) ----
    if (lane == 0) {
      grid_dependency_wait();
      for (int i = 0; i < ns && ok; ++i) {
        const int bslot = i % kUmBStages;
        if (i >= kUmBStages && !um_mbar_wait(&b_empty[bslot], (uint32_t)((i / kUmBStages - 1) & 1))) ok = false;
        if (ok) {
          unsigned char* dst = sB + bslot * kUmBStage;
          um_mbar_expect_tx(&b_full[bslot], (uint32_t)kUmBStage);
          um_bulk_g2s(dst, p.xb + (size_t)(j0 + i) * 32 * 128, 32 * 256, &b_full[bslot]);
          um_bulk_g2s(dst + 32 * 256, p.xs + (size_t)(j0 + i) * 4 * 16, 4 * 16 * 4, &b_full[bslot]);
        }
        const int i2 = i + kUmWStages;  // refill the slot of stage i once the unpack warps have left it
        if (ok && i2 < ns) {
          if (!um_mbar_wait(&w_empty[i % kUmWStages], (uint32_t)((i / kUmWStages) & 1))) ok = false;
          if (ok) load_codes(i2);
        }
      }
      if (!ok && p.status) atomicExch(p.status, 3u);
    }
    __syncwarp();
  } else if (warp >= 9) {
    // ---- MMA issue: warp 9 + g serves A slot g (one thread each; a single thread cannot issue fast enough) ----
    if (lane == 0) {
      const int g = warp - 9;
      // D f32, A and B bf16, both K-major, N = 16, M = 128
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((16u >> 3) << 17) | ((128u >> 4) << 24);
      for (int i = 0; i < ns && ok; ++i) {
        const uint32_t sb_addr = smem_u32(sB + (i % kUmBStages) * kUmBStage);
        // shared-memory descriptor, no swizzle: 8-request core matrices 128 B apart, chunks of 8 features 256 B apart
        const uint64_t desc0 = (uint64_t)((sb_addr & 0x3FFFFu) >> 4) | ((uint64_t)(256u >> 4) << 16) | ((uint64_t)(128u >> 4) << 32) |
                               (1ull << 46);
        const int d = (i & 1) * 4 + g;
        if (!um_mbar_wait(&b_full[i % kUmBStages], (uint32_t)((i / kUmBStages) & 1))) ok = false;
        // A slot g holds the group, and (the unpack threads have checked) accumulator slot d has been read back
        if (ok && !um_mbar_wait(&a_full[g], (uint32_t)(i & 1))) ok = false;
        if (!ok) break;
        tc_fence_after();
        const uint32_t dcol = tbase + kUmDCol0 + (uint32_t)(d * 16);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
          umma_bf16(dcol, tbase + (uint32_t)(g * 32 + ks * 8), desc0 + (uint64_t)(((g * 4 + ks) * 512) >> 4), idesc, ks != 0);
        umma_commit(&done[d]);
      }
      if (!ok && p.status) atomicExch(p.status, 3u);
    }
    __syncwarp();
  } else if (warp < 4) {
    // ---- unpack warps ----
    const uint32_t lane_addr = tbase + ((uint32_t)(warp * 32) << 16);
    const int row = warp * 32 + lane;  // row of the tile = lane of tensor memory
    for (int i = 0; i < ns && ok; ++i) {
      const unsigned char* stg = sW + (i % kUmWStages) * kUmWStage + row * 128;
      if (!um_mbar_wait_warp(&w_full[i % kUmWStages], (uint32_t)((i / kUmWStages) & 1))) ok = false;
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        if (!ok) break;
        // codes of group g of this row: logical 16-byte chunks 2g, 2g + 1, stored at chunk ^ (row & 7)
        const uint4 w0 = *reinterpret_cast<const uint4*>(stg + (((2 * g) ^ (lane & 7)) << 4));
        const uint4 w1 = *reinterpret_cast<const uint4*>(stg + (((2 * g + 1) ^ (lane & 7)) << 4));
        const uint32_t w[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
        uint32_t a[32];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          // {16 + code j, 16 + code j + 4}: the code sits in mantissa bits 3..6 of bf16 16.0, where 16 + code is exact
          // (the smallest offset this placement allows: the fp32 rounding of the group sums grows with it)
          a[4 * j + 0] = and_or(w[j] << 3, 0x00780078u, 0x41804180u);
          a[4 * j + 1] = and_or(w[j] >> 1, 0x00780078u, 0x41804180u);
          a[4 * j + 2] = and_or(w[j] >> 5, 0x00780078u, 0x41804180u);
          a[4 * j + 3] = and_or(w[j] >> 9, 0x00780078u, 0x41804180u);
        }
        // the MMAs that read A slot g for the previous stage must have completed, and the accumulator slot this
        // group's MMAs will write (last used two stages ago) must have been read back
        if (i >= 1 && !um_mbar_wait_warp(&done[((i - 1) & 1) * 4 + g], (uint32_t)(((i - 1) >> 1) & 1))) ok = false;
        if (ok && i >= 2 && !um_mbar_wait_warp(&d_empty[(i & 1) * 4 + g], (uint32_t)(((i >> 1) - 1) & 1))) ok = false;
        if (!ok) break;
        tc_fence_after();
        tmem_st32(lane_addr + (uint32_t)(g * 32), a);
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        tc_fence_before();
        __syncwarp();
        if (lane == 0) um_mbar_arrive(&a_full[g]);
      }
      __syncwarp();
      if (ok && lane == 0) um_mbar_arrive(&w_empty[i % kUmWStages]);  // this warp has read its rows of the stage
    }
    if (!ok && lane == 0 && p.status) atomicExch(p.status, 3u);
  } else {
    // ---- scale/bias warps ----
    const int q = warp - 4;  // lane quarter of tensor memory
    const uint32_t lane_addr = tbase + ((uint32_t)(q * 32) << 16);
    const int local = q * 32 + lane;
    // this thread's row of the tensor (clamped: rows beyond the tensor are computed and dropped)
    const int grow = local < 64 ? min(run0 + local, (silu ? half_n : p.N) - 1) : min(run1 + local - 64, p.N - 1);
    // Scales and biases of this thread's row reach it through a private ring of asynchronous copies, six stages
    // ahead: a load from DRAM takes longer than a stage under load, and nothing else in this warp can hide it.
    const uint16_t* srow = p.scales + (size_t)grow * (p.K >> 6) + (size_t)j0 * 4;  // 4 scales per stage
    const uint16_t* brow = p.biases + (size_t)grow * (p.K >> 6) + (size_t)j0 * 4;
    unsigned char* my_sb = sSb + local * 16;
    auto issue_sb = [&](int i) {
      unsigned char* dst = my_sb + (i % kUmSbStages) * kUmSbStage;
      cp_async8(dst, srow + (size_t)i * 4);
      cp_async8(dst + 8, brow + (size_t)i * 4);
    };
#pragma unroll
    for (int i = 0; i < kUmSbStages; ++i) {
      if (i < ns) issue_sb(i);
      cp_async_commit();
    }
    for (int i = 0; i < ns && ok; ++i) {
      cp_async_wait<kUmSbStages - 1>();
      const uint4 sbv = *reinterpret_cast<const uint4*>(my_sb + (i % kUmSbStages) * kUmSbStage);
      const uint2 scw = make_uint2(sbv.x, sbv.y), biw = make_uint2(sbv.z, sbv.w);
      if (i + kUmSbStages < ns) issue_sb(i + kUmSbStages);  // the slot just read (by this thread alone)
      cp_async_commit();
      const int bslot = i % kUmBStages;
      if (!um_mbar_wait_warp(&b_full[bslot], (uint32_t)((i / kUmBStages) & 1))) ok = false;  // the group sums came with the operand
      const float* sX = reinterpret_cast<const float*>(sB + bslot * kUmBStage + 32 * 256);
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        if (!ok) break;
        const int d = (i & 1) * 4 + g;
        const uint32_t sw = g < 2 ? scw.x : scw.y, bw = g < 2 ? biw.x : biw.y;
        const float sc = (g & 1) ? bf16_hi(sw) : bf16_lo(sw);
        const float bi = fmaf(-16.0f, sc, (g & 1) ? bf16_hi(bw) : bf16_lo(bw));
        const unsigned long long sc2 = pack2(sc, sc), bi2 = pack2(bi, bi);
        unsigned long long xv[8];
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          const ulonglong2 t = *reinterpret_cast<const ulonglong2*>(sX + g * 16 + q4 * 4);
          xv[2 * q4] = t.x, xv[2 * q4 + 1] = t.y;
        }
        if (!um_mbar_wait_warp(&done[d], (uint32_t)((i >> 1) & 1))) ok = false;
        if (!ok) break;
        tc_fence_after();
        unsigned long long dv[8];
        tmem_ld16(lane_addr + kUmDCol0 + (uint32_t)(d * 16), dv);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) um_mbar_arrive(&d_empty[d]);
#pragma unroll
        for (int r = 0; r < 8; ++r) {
          ffma2(acc[r], bi2, xv[r]);
          ffma2(acc[r], sc2, dv[r]);
        }
      }
      __syncwarp();
      if (ok && lane == 0) um_mbar_arrive(&b_empty[bslot]);
    }
    cp_async_wait<0>();
    if (!ok && lane == 0 && p.status) atomicExch(p.status, 3u);

    // ---- parts of K meet; epilogue ----
    grid_dependency_wait();  // the residual stream and the scratch below belong to the preceding kernel until it ends
    float accf[16];
#pragma unroll
    for (int r = 0; r < 8; ++r) {
      const float2 t = unpack2(acc[r]);
      accf[2 * r] = t.x, accf[2 * r + 1] = t.y;
    }
    bool finish = true;
    if (p.parts > 1) {
      float4* dst = reinterpret_cast<float4*>(p.partial + (((size_t)part * p.tiles + tile) * 128 + local) * 16);
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) dst[q4] = make_float4(accf[q4 * 4], accf[q4 * 4 + 1], accf[q4 * 4 + 2], accf[q4 * 4 + 3]);
      __threadfence();
      um_bar_sync_epilogue();
      if (local == 0) {
        const int prev = atomicAdd(p.counters + tile, 1);
        s_is_last = prev == p.parts - 1;
        if (s_is_last) p.counters[tile] = 0;
      }
      um_bar_sync_epilogue();
      finish = s_is_last != 0;
      if (finish) {
        __threadfence();
#pragma unroll
        for (int r = 0; r < 16; ++r) accf[r] = 0.0f;
        for (int y0 = 0; y0 < p.parts; y0 += 2) {  // two parts at a time: their loads go out together
          float4 v[2][4];
#pragma unroll
          for (int y = 0; y < 2; ++y)
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4)
              v[y][q4] = y0 + y < p.parts
                             ? __ldcg(reinterpret_cast<const float4*>(p.partial + (((size_t)(y0 + y) * p.tiles + tile) * 128 + local) * 16) + q4)
                             : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
#pragma unroll
          for (int y = 0; y < 2; ++y)
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
              accf[q4 * 4 + 0] += v[y][q4].x, accf[q4 * 4 + 1] += v[y][q4].y;
              accf[q4 * 4 + 2] += v[y][q4].z, accf[q4 * 4 + 3] += v[y][q4].w;
            }
        }
      }
    }
    if (finish) {
      if (silu) {
        // rows 0..63 of the tile are gate rows j, rows 64..127 the matching up rows: h = bf16(silu(bf16(g)) * bf16(u))
        // meets in shared memory (every MMA has completed, so the code stages are idle) and leaves as 16-byte chunks
        // of the next operand.
        um_bar_sync_epilogue();
        uint16_t* sU = reinterpret_cast<uint16_t*>(sW);         // [16][64]
        uint16_t* sH = reinterpret_cast<uint16_t*>(sW) + 1024;  // [16][66]
        if (local >= 64) {
#pragma unroll
          for (int r = 0; r < 16; ++r) sU[r * 64 + (local - 64)] = f32_to_bf16(accf[r]);
        }
        um_bar_sync_epilogue();
        if (local < 64) {
#pragma unroll
          for (int r = 0; r < 16; ++r) {
            const float gt = bf16_to_f32(f32_to_bf16(accf[r])), up = bf16_to_f32(sU[r * 64 + local]);
            sH[r * 66 + local] = f32_to_bf16((gt / (1.0f + expf(-gt))) * up);
          }
        }
        um_bar_sync_epilogue();
        const int c = local >> 4, r = local & 15;  // chunk of 8 columns, request
        if (r < p.n) {
          const uint16_t* h = sH + r * 66 + c * 8;
          uint4 v;
          v.x = (uint32_t)h[0] | ((uint32_t)h[4] << 16);
          v.y = (uint32_t)h[1] | ((uint32_t)h[5] << 16);
          v.z = (uint32_t)h[2] | ((uint32_t)h[6] << 16);
          v.w = (uint32_t)h[3] | ((uint32_t)h[7] << 16);
          *reinterpret_cast<uint4*>(p.out_xb + ((size_t)(tile * 8 + c) * 16 + r) * 8) = v;
          if (c == 0 && p.out_xs) {  // the tile's 64 columns are one group of the next projection
            const uint32_t* hw = reinterpret_cast<const uint32_t*>(sH + r * 66);
            float s8[8];
#pragma unroll
            for (int ch = 0; ch < 8; ++ch)
              s8[ch] = ((bf16_lo(hw[ch * 4]) + bf16_hi(hw[ch * 4])) + (bf16_lo(hw[ch * 4 + 1]) + bf16_hi(hw[ch * 4 + 1]))) +
                       ((bf16_lo(hw[ch * 4 + 2]) + bf16_hi(hw[ch * 4 + 2])) + (bf16_lo(hw[ch * 4 + 3]) + bf16_hi(hw[ch * 4 + 3])));
            p.out_xs[(size_t)tile * 16 + r] = ((s8[0] + s8[1]) + (s8[2] + s8[3])) + ((s8[4] + s8[5]) + (s8[6] + s8[7]));
          }
        }
      } else {
        const int row = tile * 128 + local;
        const bool row_ok = row < p.N;
        if (p.epilogue == EPI_F32) {
          float* o = reinterpret_cast<float*>(p.out) + row;
#pragma unroll
          for (int r = 0; r < 16; ++r)
            if (row_ok && r < p.n) o[(size_t)r * p.out_stride] = accf[r];
          if (p.argmax_partial) {
#pragma unroll
            for (int r = 0; r < 16; ++r) {
              float best = row_ok ? accf[r] : -INFINITY;
              int bidx = row_ok ? row : 0x7fffffff;
#pragma unroll
              for (int o2 = 16; o2 > 0; o2 >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, best, o2);
                const int oi = __shfl_xor_sync(0xffffffffu, bidx, o2);
                if (ov > best || (ov == best && oi < bidx)) best = ov, bidx = oi;
              }
              if (lane == 0 && r < p.n) p.argmax_partial[((size_t)tile * 4 + q) * 16 + r] = make_float2(best, __int_as_float(bidx));
            }
          }
        } else {
          uint16_t* o = reinterpret_cast<uint16_t*>(p.out) + row;
          const bool res = p.epilogue == EPI_RESIDUAL;
#pragma unroll
          for (int r = 0; r < 16; ++r)
            if (row_ok && r < p.n) {
              uint16_t y = f32_to_bf16(accf[r]);
              if (res) y = f32_to_bf16(bf16_to_f32(o[(size_t)r * p.out_stride]) + bf16_to_f32(y));
              o[(size_t)r * p.out_stride] = y;
            }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 9) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "n"(kUmTmemCols) : "memory");
}

// ---- tensor maps of the packed codes, one per tensor, made on first use ----
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct MapKey {
  const void* ptr;
  long long rows, row_bytes;
  bool operator==(const MapKey& o) const { return ptr == o.ptr && rows == o.rows && row_bytes == o.row_bytes; }
};
struct MapKeyHash {
  size_t operator()(const MapKey& k) const {
    return std::hash<const void*>()(k.ptr) ^ (std::hash<long long>()(k.rows) * 1000003u) ^ (std::hash<long long>()(k.row_bytes) * 7919u);
  }
};

std::mutex g_map_mutex;
std::unordered_map<MapKey, CUtensorMap, MapKeyHash> g_maps;
EncodeTiledFn g_encode = nullptr;
bool g_umma_init = false;

// The packed codes as a 2-D byte tensor [rows][K/2]; a box is 64 rows x 128 bytes (256 codes), 128-byte swizzle.
// The map depends only on the address and the extents, so an entry stays valid for as long as those describe a tensor.
cudaError_t codes_map(const uint32_t* qw, long long rows, int K, CUtensorMap* out) {
  const MapKey key{qw, rows, (long long)K / 2};
  std::lock_guard<std::mutex> lock(g_map_mutex);
  auto it = g_maps.find(key);
  if (it != g_maps.end()) {
    *out = it->second;
    return cudaSuccess;
  }
  if (!g_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return e;
    if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  }
  if (reinterpret_cast<uintptr_t>(qw) % 16 || (K / 2) % 16) return cudaErrorInvalidValue;
  const cuuint64_t dims[2] = {(cuuint64_t)(K / 2), (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)(K / 2)};
  const cuuint32_t box[2] = {128u, 64u}, elem[2] = {1u, 1u};
  CUtensorMap m;
  const CUresult r = g_encode(&m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint32_t*>(qw), dims, strides, box, elem,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
  if (g_maps.size() > 65536) g_maps.clear();
  g_maps.emplace(key, m);
  *out = m;
  return cudaSuccess;
}

cudaError_t umma_init() {
  cudaError_t e = cudaFuncSetAttribute(q4_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kUmSmem);
  if (e == cudaSuccess) g_umma_init = true;
  return e;
}

}  // namespace

UmmaPlan plan_umma(int N, int K, int epilogue, int sm_count) {
  UmmaPlan t;
  t.tiles = epilogue == EPI_SILU_PACK ? (N / 2) / 64 : (N + 127) / 128;
  t.ns = K / 256;
  // Parts of K: the count that minimises waves x (stages per part + the fixed cost of a CTA and of the hand-over),
  // with two CTAs resident per SM.
  const int slots = 2 * (sm_count > 0 ? sm_count : 148);
  int best = 1;
  double best_t = 1e30;
  for (int parts = 1; parts <= t.ns && parts <= 16; ++parts) {
    const long long units = (long long)t.tiles * parts;
    const double waves = (double)((units + slots - 1) / slots);
    const double per = (double)((t.ns + parts - 1) / parts) + (parts > 1 ? 2.0 : 1.0);
    const double tt = waves * per;
    if (tt < best_t - 1e-9) best_t = tt, best = parts;
  }
  t.parts = best;
  t.partial_bytes = t.parts > 1 ? (size_t)t.parts * t.tiles * 128 * 16 * sizeof(float) : 0;
  return t;
}

bool umma_supported(int N, int K, int epilogue) {
  if (N <= 0 || K <= 0 || (K % 256)) return false;
  if (epilogue == EPI_SILU_PACK && (N % 128)) return false;
  return true;
}

cudaError_t launch_q4_umma(const GemmArgs& a, int sm_count, cudaStream_t s) {
  if (!g_umma_init) {
    cudaError_t e = umma_init();
    if (e != cudaSuccess) return e;
  }
  const UmmaPlan t = plan_umma(a.N, a.K, a.epilogue, sm_count);
  UmmaParams p;
  p.scales = a.scales, p.biases = a.biases, p.xb = a.xp, p.xs = a.xs, p.out = a.out;
  p.out_xb = a.out_xp, p.out_xs = a.out_xs, p.argmax_partial = a.argmax_partial, p.status = a.status;
  p.partial = a.partial, p.counters = a.counters;
  p.N = a.N, p.K = a.K, p.n = a.n, p.out_stride = a.out_stride, p.epilogue = a.epilogue;
  p.tiles = t.tiles, p.parts = t.parts, p.ns = t.ns;
  if (!a.xs) return cudaErrorInvalidValue;
  if (t.parts > 1 && (!a.partial || !a.counters || t.partial_bytes > a.partial_bytes || t.tiles > a.counters_len))
    return cudaErrorInvalidValue;
  CUtensorMap map;
  cudaError_t e = codes_map(a.qw, a.N, a.K, &map);
  if (e != cudaSuccess) return e;
  return launch_kernel(q4_umma_kernel, dim3(t.tiles * t.parts), dim3(kUmThreads), kUmSmem, s, p, map);
}

}  // namespace q4d
