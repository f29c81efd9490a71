// Fused dequantise-and-multiply of 4-bit affine group-64 weights on the fifth-generation tensor cores
// (tcgen05.mma with the weight operand in tensor memory).
//
//   y[r][j] = sum_g scale[j][g] * (sum_{k in g} q[j][k] x[r][k]) + bias[j][g] * (sum_{k in g} x[r][k])
//
// A CTA owns one tile of 128 weight rows and one part of K.  Row i of the tile is lane i of tensor memory: the thread
// that owns the lane unpacks the row's 4-bit codes into exact bf16 integers 16 + q (one shift and one logic operation per
// pair of codes) and stores them with tcgen05.st as the A operand of a 128 x 16 x 64 product; the
// activations of the 16 requests are the B operand, read from shared memory in the layout the tensor core wants (the
// producing kernels write it that way, so a stage is one bulk copy).  Every group of 64 input features gets its own
// 16-column fp32 accumulator, which the lane's thread reads back (tcgen05.ld) and folds into registers with the
// group's scale and bias: products are exact, accumulation is fp32, and no dequantised weight is ever rounded to
// bf16.  The offset 16 leaves through the bias term (bias - 16 scale multiplies the group's sum of x).
//
// Roles: warps 0..3 stream the packed rows of their 32 lanes through private cp.async rings (started before the
// preceding kernel is awaited: weights do not depend on it), unpack, store A, and run the scale/bias epilogue of the
// group issued four groups earlier; one thread of warp 4 stages the operand with bulk copies and issues the MMAs.
// Four A slots and eight accumulator slots of tensor memory keep four groups in flight between the two.
//
// K is cut into parts across CTAs where the tiles alone would not fill the machine; the parts of a tile meet in
// global scratch and the last CTA to arrive adds them in part order (deterministic) and applies the epilogue.
#include "common.cuh"
#include "kernels.h"
#include "launch.h"

namespace q4d {

namespace {

constexpr int kUmWarps = 4;                        // unpack warps = the four lane quarters of tensor memory
constexpr int kUmThreads = 32 * (kUmWarps + 1);    // + the control warp
constexpr int kUmWStage = 32 * 128 + 32 * 16;      // a warp's stage: 32 rows x 256 codes (128 B) + 4 scales, 4 biases each
constexpr int kUmBStage = 32 * 256 + 4 * 16 * 4;   // 256 features x 16 requests bf16 (8 KB) + the 4 groups' sums
constexpr int kUmBStages = 4;
constexpr int kUmTmemCols = 256;                   // A: 4 slots x 32 columns at 0; D: 8 slots x 16 columns at 128
constexpr uint32_t kUmDCol0 = 128;

struct UmmaParams {
  const uint32_t* qw;
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
// Waits for the phase of the given parity; gives up (false) after a bounded number of tries.
__device__ __forceinline__ bool um_mbar_wait(uint64_t* bar, uint32_t parity) {
  for (int tries = 0; tries < (1 << 18); ++tries) {
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
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t u[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]), "=r"(u[8]), "=r"(u[9]),
        "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(u[i]);
}

__device__ __forceinline__ void um_bar_sync_unpackers() { asm volatile("bar.sync 1, %0;" ::"n"(32 * kUmWarps) : "memory"); }

template <int WST>
__global__ void __launch_bounds__(kUmThreads, 2) q4_umma_kernel(const UmmaParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) uint64_t bar_full[4];  // A slot g written by all unpack threads (stage parity)
  __shared__ __align__(8) uint64_t bar_done[8];  // the MMAs of (stage & 1, g) have completed
  __shared__ __align__(8) uint64_t bar_b[kUmBStages];
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_is_last;

  grid_launch_dependents();

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool silu = p.epilogue == EPI_SILU_PACK;
  const int half_n = p.N >> 1;
  const int tile = blockIdx.x / p.parts, part = blockIdx.x - tile * p.parts;
  const int j0 = (int)((long long)part * p.ns / p.parts), j1 = (int)((long long)(part + 1) * p.ns / p.parts);
  const int ns = j1 - j0;  // stages of this CTA

  unsigned char* sB = smem + kUmWarps * WST * kUmWStage;

  // rows of this warp (warps 0..3): 32 consecutive rows of the tensor
  const int local0 = warp * 32;
  int warp_row0, row_limit;
  if (!silu) {
    warp_row0 = tile * 128 + local0, row_limit = p.N;
  } else if (local0 < 64) {
    warp_row0 = tile * 64 + local0, row_limit = half_n;  // gate rows
  } else {
    warp_row0 = half_n + tile * 64 + (local0 - 64), row_limit = p.N;  // the matching up rows
  }
  unsigned char* ring = smem + warp * (WST * kUmWStage);

  auto issue_stage = [&](int slot, int j) {  // stage j of the tensor's K
    unsigned char* stg = ring + slot * kUmWStage;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int r = i * 4 + (lane >> 3), c = lane & 7;
      const int grow = min(warp_row0 + r, row_limit - 1);
      const unsigned char* src = reinterpret_cast<const unsigned char*>(p.qw + (size_t)grow * (p.K >> 3) + (size_t)j * 32) + c * 16;
      cp_async16(stg + r * 128 + ((c ^ (r & 7)) << 4), src);
    }
    const int grow = min(warp_row0 + lane, row_limit - 1);
    const size_t off = (size_t)grow * (p.K >> 6) + (size_t)j * 4;
    cp_async8(stg + 32 * 128 + lane * 16, p.scales + off);
    cp_async8(stg + 32 * 128 + lane * 16 + 8, p.biases + off);
  };

  if (warp < kUmWarps) {
    // Weights do not depend on the preceding kernel: fill the ring before waiting for it.
#pragma unroll
    for (int s = 0; s < WST; ++s) {
      if (s < ns) issue_stage(s, j0 + s);
      cp_async_commit();
    }
  } else {
    if (lane == 0) {
      for (int g = 0; g < 4; ++g) um_mbar_init(&bar_full[g], 32 * kUmWarps);
      for (int d = 0; d < 8; ++d) um_mbar_init(&bar_done[d], 1);
      for (int b = 0; b < kUmBStages; ++b) um_mbar_init(&bar_b[b], 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)), "n"(kUmTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tbase = s_tmem_base;

  grid_dependency_wait();

  bool ok = true;
  float acc[16];
#pragma unroll
  for (int r = 0; r < 16; ++r) acc[r] = 0.0f;

  if (warp == kUmWarps) {
    // ---- control: operand staging and MMA issue (one thread) ----
    if (lane == 0) {
      auto stage_b = [&](int i) {  // stage i of this CTA into slot i % kUmBStages
        unsigned char* dst = sB + (i % kUmBStages) * kUmBStage;
        uint64_t* bar = &bar_b[i % kUmBStages];
        um_mbar_expect_tx(bar, (uint32_t)kUmBStage);
        um_bulk_g2s(dst, p.xb + (size_t)(j0 + i) * 32 * 128, 32 * 256, bar);
        um_bulk_g2s(dst + 32 * 256, p.xs + (size_t)(j0 + i) * 4 * 16, 4 * 16 * 4, bar);
      };
      for (int i = 0; i < kUmBStages && i < ns; ++i) stage_b(i);
      // D f32, A and B bf16, both K-major, N = 16, M = 128
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((16u >> 3) << 17) | ((128u >> 4) << 24);
      for (int i = 0; i < ns && ok; ++i) {
        const uint32_t sb_addr = smem_u32(sB + (i % kUmBStages) * kUmBStage);
        // shared-memory descriptor, no swizzle: 8-request core matrices 128 B apart, chunks of 8 features 256 B apart
        const uint64_t desc0 = (uint64_t)((sb_addr & 0x3FFFFu) >> 4) | ((uint64_t)(256u >> 4) << 16) | ((uint64_t)(128u >> 4) << 32) |
                               (1ull << 46);
        if (!um_mbar_wait(&bar_b[i % kUmBStages], (uint32_t)((i / kUmBStages) & 1))) ok = false;
        for (int g = 0; g < 4 && ok; ++g) {
          if (!um_mbar_wait(&bar_full[g], (uint32_t)(i & 1))) {
            ok = false;
            break;
          }
          tc_fence_after();
          if (g == 0 && i >= 2 && i + 2 < ns) stage_b(i + 2);  // its slot held stage i - 2, which every thread has left
          const uint32_t d = tbase + kUmDCol0 + (uint32_t)(((i & 1) * 4 + g) * 16);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            umma_bf16(d, tbase + (uint32_t)(g * 32 + ks * 8), desc0 + (uint64_t)(((g * 4 + ks) * 512) >> 4), idesc, ks != 0);
          umma_commit(&bar_done[(i & 1) * 4 + g]);
        }
      }
      if (!ok && p.status) atomicExch(p.status, 3u);
    }
    __syncwarp();
  } else {
    // ---- unpack warps ----
    const uint32_t lane_addr = tbase + ((uint32_t)(warp * 32) << 16);
    uint4 sb_prev = make_uint4(0u, 0u, 0u, 0u);
    for (int i = 0; i <= ns && ok; ++i) {
      const unsigned char* stg = ring + (i % WST) * kUmWStage;
      uint4 sb = make_uint4(0u, 0u, 0u, 0u);
      if (i < ns) {
        cp_async_wait<WST - 1>();
        __syncwarp();
        sb = *reinterpret_cast<const uint4*>(stg + 32 * 128 + lane * 16);
      }
      const float* sX = reinterpret_cast<const float*>(sB + ((i + kUmBStages - 1) % kUmBStages) * kUmBStage + 32 * 256);
      if (i >= 1 && !um_mbar_wait(&bar_b[(i - 1) % kUmBStages], (uint32_t)(((i - 1) / kUmBStages) & 1))) ok = false;
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        if (i >= 1 && ok) {
          // scale/bias epilogue of group g of stage i - 1
          if (!um_mbar_wait(&bar_done[((i - 1) & 1) * 4 + g], (uint32_t)(((i - 1) >> 1) & 1))) ok = false;
          if (ok) {
            tc_fence_after();
            float d[16];
            tmem_ld16(lane_addr + kUmDCol0 + (uint32_t)((((i - 1) & 1) * 4 + g) * 16), d);
            const uint32_t sw = g < 2 ? sb_prev.x : sb_prev.y, bw = g < 2 ? sb_prev.z : sb_prev.w;
            const float sc = (g & 1) ? bf16_hi(sw) : bf16_lo(sw);
            const float bi = fmaf(-16.0f, sc, (g & 1) ? bf16_hi(bw) : bf16_lo(bw));
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
              const float4 xv = *reinterpret_cast<const float4*>(sX + g * 16 + q4 * 4);
              acc[q4 * 4 + 0] = fmaf(sc, d[q4 * 4 + 0], fmaf(bi, xv.x, acc[q4 * 4 + 0]));
              acc[q4 * 4 + 1] = fmaf(sc, d[q4 * 4 + 1], fmaf(bi, xv.y, acc[q4 * 4 + 1]));
              acc[q4 * 4 + 2] = fmaf(sc, d[q4 * 4 + 2], fmaf(bi, xv.z, acc[q4 * 4 + 2]));
              acc[q4 * 4 + 3] = fmaf(sc, d[q4 * 4 + 3], fmaf(bi, xv.w, acc[q4 * 4 + 3]));
            }
          }
        }
        if (i < ns && ok) {
          // codes of group g of this lane's row: logical 16-byte chunks 2g, 2g + 1, stored at chunk ^ (row & 7)
          const uint4 w0 = *reinterpret_cast<const uint4*>(stg + lane * 128 + (((2 * g) ^ (lane & 7)) << 4));
          const uint4 w1 = *reinterpret_cast<const uint4*>(stg + lane * 128 + (((2 * g + 1) ^ (lane & 7)) << 4));
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
          tmem_st32(lane_addr + (uint32_t)(g * 32), a);
          asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
          tc_fence_before();
          um_mbar_arrive(&bar_full[g]);
        }
      }
      if (i < ns) {
        sb_prev = sb;
        __syncwarp();  // every lane has read the stage: refill its slot
        if (i + WST < ns) issue_stage(i % WST, j0 + i + WST);
        cp_async_commit();
      }
    }
    cp_async_wait<0>();
    if (!ok && lane == 0 && p.status) atomicExch(p.status, 3u);
  }

  // ---- parts of K meet; epilogue (unpack warps only) ----
  if (warp < kUmWarps) {
    const int local = warp * 32 + lane;
    bool finish = true;
    if (p.parts > 1) {
      float4* dst = reinterpret_cast<float4*>(p.partial + (((size_t)part * p.tiles + tile) * 128 + local) * 16);
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) dst[q4] = make_float4(acc[q4 * 4], acc[q4 * 4 + 1], acc[q4 * 4 + 2], acc[q4 * 4 + 3]);
      __threadfence();
      um_bar_sync_unpackers();
      if (threadIdx.x == 0) {
        const int prev = atomicAdd(p.counters + tile, 1);
        s_is_last = prev == p.parts - 1;
        if (s_is_last) p.counters[tile] = 0;
      }
      um_bar_sync_unpackers();
      finish = s_is_last != 0;
      if (finish) {
        __threadfence();
#pragma unroll
        for (int r = 0; r < 16; ++r) acc[r] = 0.0f;
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
              acc[q4 * 4 + 0] += v[y][q4].x, acc[q4 * 4 + 1] += v[y][q4].y;
              acc[q4 * 4 + 2] += v[y][q4].z, acc[q4 * 4 + 3] += v[y][q4].w;
            }
        }
      }
    }
    if (finish) {
      if (silu) {
        // rows of warps 0, 1 are gate rows j, rows of warps 2, 3 the matching up rows: h = bf16(silu(bf16(g)) * bf16(u))
        // meets in shared memory (the rings are idle now) and leaves as 16-byte chunks of the next operand.
        um_bar_sync_unpackers();  // every warp has left its ring
        uint16_t* sU = reinterpret_cast<uint16_t*>(smem);         // [16][64]
        uint16_t* sH = reinterpret_cast<uint16_t*>(smem) + 1024;  // [16][66]
        if (local >= 64) {
#pragma unroll
          for (int r = 0; r < 16; ++r) sU[r * 64 + (local - 64)] = f32_to_bf16(acc[r]);
        }
        um_bar_sync_unpackers();
        if (local < 64) {
#pragma unroll
          for (int r = 0; r < 16; ++r) {
            const float gt = bf16_to_f32(f32_to_bf16(acc[r])), up = bf16_to_f32(sU[r * 64 + local]);
            sH[r * 66 + local] = f32_to_bf16((gt / (1.0f + expf(-gt))) * up);
          }
        }
        um_bar_sync_unpackers();
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
            if (row_ok && r < p.n) o[(size_t)r * p.out_stride] = acc[r];
          if (p.argmax_partial) {
#pragma unroll
            for (int r = 0; r < 16; ++r) {
              float best = row_ok ? acc[r] : -INFINITY;
              int bidx = row_ok ? row : 0x7fffffff;
#pragma unroll
              for (int o2 = 16; o2 > 0; o2 >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, best, o2);
                const int oi = __shfl_xor_sync(0xffffffffu, bidx, o2);
                if (ov > best || (ov == best && oi < bidx)) best = ov, bidx = oi;
              }
              if (lane == 0 && r < p.n) p.argmax_partial[((size_t)tile * 4 + warp) * 16 + r] = make_float2(best, __int_as_float(bidx));
            }
          }
        } else {
          uint16_t* o = reinterpret_cast<uint16_t*>(p.out) + row;
          const bool res = p.epilogue == EPI_RESIDUAL;
#pragma unroll
          for (int r = 0; r < 16; ++r)
            if (row_ok && r < p.n) {
              uint16_t y = f32_to_bf16(acc[r]);
              if (res) y = f32_to_bf16(bf16_to_f32(o[(size_t)r * p.out_stride]) + bf16_to_f32(y));
              o[(size_t)r * p.out_stride] = y;
            }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == kUmWarps)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "n"(kUmTmemCols) : "memory");
}

constexpr int kUmWStagesDefault = 3;

size_t umma_smem_bytes(int wst) { return (size_t)kUmWarps * wst * kUmWStage + (size_t)kUmBStages * kUmBStage; }

bool g_umma_init = false;

cudaError_t umma_init() {
  cudaError_t e = cudaFuncSetAttribute(q4_umma_kernel<kUmWStagesDefault>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)umma_smem_bytes(kUmWStagesDefault));
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
  p.qw = a.qw, p.scales = a.scales, p.biases = a.biases, p.xb = a.xp, p.xs = a.xs, p.out = a.out;
  p.out_xb = a.out_xp, p.out_xs = a.out_xs, p.argmax_partial = a.argmax_partial, p.status = a.status;
  p.partial = a.partial, p.counters = a.counters;
  p.N = a.N, p.K = a.K, p.n = a.n, p.out_stride = a.out_stride, p.epilogue = a.epilogue;
  p.tiles = t.tiles, p.parts = t.parts, p.ns = t.ns;
  if (!a.xs) return cudaErrorInvalidValue;
  if (t.parts > 1 && (!a.partial || !a.counters || t.partial_bytes > a.partial_bytes || t.tiles > a.counters_len))
    return cudaErrorInvalidValue;
  return launch_kernel(q4_umma_kernel<kUmWStagesDefault>, dim3(t.tiles * t.parts), dim3(kUmThreads),
                       umma_smem_bytes(kUmWStagesDefault), s, p);
}

}  // namespace q4d
