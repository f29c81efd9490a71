// Fused dequantise-and-multiply of 4-bit affine group-64 weights against bf16
// activations for 1..16 requests (the QKV, O, gate/up, down and LM-head
// projections of the decode step).
//
// y[r][j] = sum_k (scale[j][k/64] * q[j][k] + bias[j][k/64]) * x[r][k]
//         = sum_g scale[j][g] * (sum_{k in g} q[j][k] x[r][k]) + bias[j][g] * (sum_{k in g} x[r][k])
//
// The inner sums run on the tensor cores with the 4-bit codes converted to
// exact bf16 integers 16 + q (products are exact, accumulation is fp32), so
// no dequantised weight is ever rounded to bf16; scale and bias (less 16 * scale,
// which removes the offset again) are applied to the fp32 group sums.
//
// Layout of the work.  One CTA of 12 warps per SM owns a contiguous range of 16-row tiles (and, for K > 4096, one
// part of K).  q4_span_kernel serves CTAs with at most 12 tiles (the projections of a layer): every slice of the
// operand is resident, each warp streams an equal contiguous span of the CTA's stages, partial tiles meet in shared
// memory.  q4_round_kernel serves longer tile ranges (the LM head): rounds of 12 tiles, the operand slices double
// buffered with a CTA barrier per slice.  In both the weight stream does not depend on the preceding kernel, so it
// is started before the grid dependency is awaited.  q4_gemm_kernel is the older CTA-granular form (a CTA owns 128
// rows and one K-slice, split-K through global scratch); the grouped mode of the mixture-of-experts layers still
// runs on it.
#include <stdlib.h>
#include <string.h>

#include "common.cuh"
#include "kernels.h"
#include "launch.h"

namespace q4d {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = 8;
constexpr int kRowStride = 160;  // bytes per row per stage in smem: 128 data + 32 pad (conflict-free 8-byte reads)
constexpr int kSbBytes = 16;     // per row per stage: 4 scales + 4 biases (bf16)
constexpr int kMaxQuadsPerSlice = 4;  // K-slice <= 1024

struct GemmParams {
  const uint32_t* qw;
  const uint16_t* scales;
  const uint16_t* biases;
  const uint16_t* xp;
  const float* xs;
  void* out;
  uint16_t* out_xp;
  float* out_xs;
  float2* argmax_partial;
  float* partial;
  int* counters;
  int N, K, n, out_stride;
  int ks;      // nominal K-slice (multiple of 256)
  int splits;  // gridDim.y
  int epilogue;
  int out_ks, out_row_stride, out_slice_stride;  // out_xp: features per slice, elements between rows and between slices
  // grouped mode (MoE experts): blockIdx.z is a slot of the touched-expert list; the tensors of expert
  // expert_ids[slot] start expert_rows rows further per expert; operand and output move by their slot strides.
  const int* expert_ids;
  const int* n_touched;
  int expert_rows;
  size_t xp_slot_stride, xs_slot_stride, out_slot_stride, out_xs_slot_stride;  // elements
};

// Four bf16x2 registers {16 + code j, 16 + code j+4}, j = 0..3, from one packed word: the code is placed in
// mantissa bits 3..6 of bf16 16.0 (0x4180), where 16 + code is exact.  One shift and one logic op per register;
// the constant 16 is taken out again through the group sums (16 * sum x is subtracted via the bias term).
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c) {  // (a & b) | c in one LOP3
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
__device__ __forceinline__ void unpack_word(uint32_t w, uint32_t (&p)[4]) {
  const uint32_t kMask = 0x00780078u, kSixteen = 0x41804180u;
  p[0] = and_or(w << 3, kMask, kSixteen);
  p[1] = and_or(w >> 1, kMask, kSixteen);
  p[2] = and_or(w >> 5, kMask, kSixteen);
  p[3] = and_or(w >> 9, kMask, kSixteen);
}

// two fp32 FMAs in one instruction: c = a * b + c on both halves, each rounded like a scalar FMA
__device__ __forceinline__ void fma_f32x2(unsigned long long& c, unsigned long long a, unsigned long long b) {
  asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(c) : "l"(a), "l"(b));
}
__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack_f32x2(unsigned long long v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}

// acc += s * pc + b * xs for the 2 x 2 block of an MMA fragment (rows g, g + 8; requests 2t, 2t + 1): s and b per row,
// xs per request; two requests per packed instruction, each half rounded like the scalar fmaf(s, pc, fmaf(b, xs, acc)).
__device__ __forceinline__ void scale_bias_fma(float (&acc)[4], const float (&pc)[4], float s_lo, float s_hi, float b_lo,
                                               float b_hi, float2 xs) {
  const unsigned long long x2 = pack_f32x2(xs.x, xs.y);
  unsigned long long a01 = pack_f32x2(acc[0], acc[1]), a23 = pack_f32x2(acc[2], acc[3]);
  fma_f32x2(a01, pack_f32x2(b_lo, b_lo), x2);
  fma_f32x2(a23, pack_f32x2(b_hi, b_hi), x2);
  fma_f32x2(a01, pack_f32x2(s_lo, s_lo), pack_f32x2(pc[0], pc[1]));
  fma_f32x2(a23, pack_f32x2(s_hi, s_hi), pack_f32x2(pc[2], pc[3]));
  unpack_f32x2(a01, acc[0], acc[1]);
  unpack_f32x2(a23, acc[2], acc[3]);
}

__device__ __forceinline__ float bf16_at(const uint2& v, int i) {
  uint32_t w = (i >> 1) ? v.y : v.x;
  return (i & 1) ? bf16_hi(w) : bf16_lo(w);
}

__device__ __forceinline__ void store_out(const GemmParams& p, int row, int req, float v) {
  if (p.epilogue == EPI_F32) {
    reinterpret_cast<float*>(p.out)[(size_t)req * p.out_stride + row] = v;
  } else {
    uint16_t* o = reinterpret_cast<uint16_t*>(p.out) + (size_t)req * p.out_stride + row;
    uint16_t y = f32_to_bf16(v);
    if (p.epilogue == EPI_RESIDUAL) y = f32_to_bf16(bf16_to_f32(*o) + bf16_to_f32(y));
    *o = y;
  }
}

template <int MT, int NT, int STAGES>
__global__ void __launch_bounds__(kThreads, (MT == 1) ? 2 : 1) q4_gemm_kernel(const GemmParams pin) {
  constexpr int R = 16 * MT;        // rows per warp
  constexpr int NP = 8 * NT;        // padded request count
  constexpr int kRows = kWarps * R; // rows per CTA
  constexpr int kStage = R * (kRowStride + kSbBytes);
  constexpr int kTs = NP + 1;       // row stride of the final tile (floats)
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ int s_is_last;

  grid_launch_dependents();

  GemmParams p = pin;
  if (pin.expert_ids) {
    // the expert list is written by the preceding kernel: wait for it before anything else
    grid_dependency_wait();
    const int slot = blockIdx.z;
    if (slot >= *pin.n_touched) return;
    const size_t e = (size_t)pin.expert_ids[slot];
    p.qw += e * pin.expert_rows * (size_t)(pin.K >> 3);
    p.scales += e * pin.expert_rows * (size_t)(pin.K >> 6);
    p.biases += e * pin.expert_rows * (size_t)(pin.K >> 6);
    p.xp += (size_t)slot * pin.xp_slot_stride;
    p.xs += (size_t)slot * pin.xs_slot_stride;
    if (p.out_xs) p.out_xs += (size_t)slot * pin.out_xs_slot_stride;
    if (p.out_xp) p.out_xp += (size_t)slot * pin.out_slot_stride;
    if (p.out) p.out = reinterpret_cast<uint16_t*>(p.out) + (size_t)slot * pin.out_slot_stride;
  }

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const bool silu = p.epilogue == EPI_SILU_PACK;
  const int half_n = p.N >> 1;  // silu: rows [0, half_n) are gate rows, [half_n, N) up rows
  // local row of the CTA -> row of the tensor.  With the SiLU epilogue the first half of the CTA's rows are
  // gate rows and the second half the matching up rows, so that one CTA ends up with both.
  auto global_row = [&](int lrow) -> int {
    if (!silu) return blockIdx.x * kRows + lrow;
    return lrow < kRows / 2 ? blockIdx.x * (kRows / 2) + lrow : half_n + blockIdx.x * (kRows / 2) + (lrow - kRows / 2);
  };
  const int row_limit_first = silu ? half_n : p.N;  // rows of the first half must stay below this
  const int warp_row0 = global_row(warp * R);
  const int warp_limit = (silu && warp * R >= kRows / 2) ? p.N : row_limit_first;
  const int k0 = blockIdx.y * p.ks;
  const int kend = min(p.K, k0 + p.ks);
  const int kslice = kend - k0;
  const int nquads = kslice >> 8;
  const int b_stride = p.ks * 2 + 16;  // bytes per request row of the staged activations

  unsigned char* ring = smem + warp * (STAGES * kStage);
  unsigned char* sB = smem + kWarps * STAGES * kStage;
  float* sX = reinterpret_cast<float*>(sB + NP * b_stride);  // [group][NP]

  auto issue_stage = [&](int qd) {
    unsigned char* stg = ring + (qd % STAGES) * kStage;
    const int kq = k0 + qd * 256;
#pragma unroll
    for (int i = 0; i < R / 4; ++i) {
      const int r = i * 4 + (lane >> 3);
      const int grow = min(warp_row0 + r, warp_limit - 1);
      const unsigned char* src =
          reinterpret_cast<const unsigned char*>(p.qw + (size_t)grow * (p.K >> 3) + (kq >> 3)) + (lane & 7) * 16;
      cp_async16(stg + r * kRowStride + (lane & 7) * 16, src);
    }
    for (int r = lane; r < R; r += 32) {
      const int grow = min(warp_row0 + r, warp_limit - 1);
      const size_t off = (size_t)grow * (p.K >> 6) + (kq >> 6);
      cp_async8(stg + R * kRowStride + r * kSbBytes, p.scales + off);
      cp_async8(stg + R * kRowStride + r * kSbBytes + 8, p.biases + off);
    }
  };

  // Weights do not depend on the preceding kernel: start streaming them before waiting for it.
#pragma unroll
  for (int s = 0; s < STAGES - 1; ++s) {
    if (s < nquads) issue_stage(s);
    cp_async_commit();
  }

  grid_dependency_wait();

  // Activations (already in fragment order) and their group sums: straight copies.
  {
    const int cpr = kslice >> 3;  // 16-byte chunks per request row
    for (int c = threadIdx.x; c < NP * cpr; c += kThreads) {
      const int r = c / cpr, kc = c - r * cpr;
      cp_async16(sB + r * b_stride + kc * 16, p.xp + (size_t)r * p.K + k0 + kc * 8);
    }
    const int groups = kslice >> 6;
    for (int c = threadIdx.x; c < groups * (NP / 4); c += kThreads) {
      const int gq = c / (NP / 4), q4 = c - gq * (NP / 4);
      cp_async16(sX + gq * NP + q4 * 4, p.xs + (size_t)((k0 >> 6) + gq) * 16 + q4 * 4);
    }
    cp_async_commit();
    cp_async_wait<0>();
  }
  __syncthreads();

  float acc[MT][NT][4];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[mt][nt][c] = 0.0f;

  for (int qd = 0; qd < nquads; ++qd) {
    if (qd + STAGES - 1 < nquads) issue_stage(qd + STAGES - 1);
    cp_async_commit();
    cp_async_wait<STAGES - 1>();
    __syncwarp();
    const unsigned char* stg = ring + (qd % STAGES) * kStage;

    uint2 sc[MT][2], bi[MT][2];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const uint4 v = *reinterpret_cast<const uint4*>(stg + R * kRowStride + (mt * 16 + g + 8 * h) * kSbBytes);
        sc[mt][h] = make_uint2(v.x, v.y);
        bi[mt][h] = make_uint2(v.z, v.w);
      }

#pragma unroll
    for (int gi = 0; gi < 4; ++gi) {
      const int gidx = qd * 4 + gi;
      uint4 bf[NT][2];
      float2 xs[NT];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const unsigned char* bp = sB + (nt * 8 + g) * b_stride + gidx * 128 + t * 32;
        bf[nt][0] = *reinterpret_cast<const uint4*>(bp);
        bf[nt][1] = *reinterpret_cast<const uint4*>(bp + 16);
        xs[nt] = *reinterpret_cast<const float2*>(sX + gidx * NP + nt * 8 + 2 * t);
      }
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        const uint2 wl = *reinterpret_cast<const uint2*>(stg + (mt * 16 + g) * kRowStride + gi * 32 + t * 8);
        const uint2 wh = *reinterpret_cast<const uint2*>(stg + (mt * 16 + g + 8) * kRowStride + gi * 32 + t * 8);
        uint32_t l0[4], l1[4], h0[4], h1[4];
        unpack_word(wl.x, l0);
        unpack_word(wl.y, l1);
        unpack_word(wh.x, h0);
        unpack_word(wh.y, h1);
        // sum (16 + q) x = 16 X + sum q x, so the bias that multiplies X becomes b - 16 s
        const float s_lo = bf16_at(sc[mt][0], gi), s_hi = bf16_at(sc[mt][1], gi);
        const float b_lo = fmaf(-16.0f, s_lo, bf16_at(bi[mt][0], gi)), b_hi = fmaf(-16.0f, s_hi, bf16_at(bi[mt][1], gi));
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          float pc[4];
          mma_bf16_first(pc, l0[0], h0[0], l0[1], h0[1], bf[nt][0].x, bf[nt][0].y);
          mma_bf16(pc, l0[2], h0[2], l0[3], h0[3], bf[nt][0].z, bf[nt][0].w);
          mma_bf16(pc, l1[0], h1[0], l1[1], h1[1], bf[nt][1].x, bf[nt][1].y);
          mma_bf16(pc, l1[2], h1[2], l1[3], h1[3], bf[nt][1].z, bf[nt][1].w);
          scale_bias_fma(acc[mt][nt], pc, s_lo, s_hi, b_lo, b_hi, xs[nt]);
        }
      }
    }
    __syncwarp();
  }
  cp_async_wait<0>();
  __syncthreads();  // every warp is done with its ring: the final tile may overlay them

  float* sT = reinterpret_cast<float*>(smem);  // [kRows][kTs]
  if (p.splits == 1) {
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int c = 0; c < 4; ++c)
          sT[(warp * R + mt * 16 + g + (c >> 1) * 8) * kTs + nt * 8 + 2 * t + (c & 1)] = acc[mt][nt][c];
  } else {
    // Split-K: publish this CTA's partial sums, then the last CTA of the row block reduces them.
    const size_t tile = (size_t)kRows * NP;
    float* part = p.partial + ((size_t)blockIdx.y * gridDim.x + blockIdx.x) * tile;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int h = 0; h < 2; ++h)
          *reinterpret_cast<float2*>(part + (size_t)(warp * R + mt * 16 + g + h * 8) * NP + nt * 8 + 2 * t) =
              make_float2(acc[mt][nt][2 * h], acc[mt][nt][2 * h + 1]);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
      const int prev = atomicAdd(p.counters + blockIdx.x, 1);
      s_is_last = (prev == p.splits - 1);
    }
    __syncthreads();
    if (!s_is_last) return;
    __threadfence();
    for (int idx = threadIdx.x; idx < kRows * NP / 4; idx += kThreads) {
      const int lrow = idx / (NP / 4), q4 = idx - lrow * (NP / 4);
      float4 v = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
      for (int s = 0; s < p.splits; ++s) {
        const float4 a = __ldcg(reinterpret_cast<const float4*>(p.partial + ((size_t)s * gridDim.x + blockIdx.x) * tile +
                                                               (size_t)lrow * NP + q4 * 4));
        v.x += a.x, v.y += a.y, v.z += a.z, v.w += a.w;
      }
      float* d = sT + lrow * kTs + q4 * 4;
      d[0] = v.x, d[1] = v.y, d[2] = v.z, d[3] = v.w;
    }
    if (threadIdx.x == 0) p.counters[blockIdx.x] = 0;
  }
  __syncthreads();

  if (silu) {
    // h = bf16(silu(bf16(gate)) * bf16(up)) for the CTA's kRows/2 columns, as the next GEMM's operand.
    constexpr int kCh = kRows / 16;  // chunks of 8 columns
    const int idx = threadIdx.x;
    if (idx < kCh * NP) {
      const int c = idx % kCh, req = idx / kCh;
      uint32_t hw[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float hv[2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int col = c * 8 + 2 * i + j;
          const float gt = bf16_to_f32(f32_to_bf16(sT[col * kTs + req]));
          const float up = bf16_to_f32(f32_to_bf16(sT[(kRows / 2 + col) * kTs + req]));
          hv[j] = (gt / (1.0f + expf(-gt))) * up;
        }
        hw[i] = pack_bf16x2(hv[0], hv[1]);
      }
      const uint4 v = make_uint4(hw[0], hw[1], hw[2], hw[3]);
      const float gsum = group_sum_8lanes(chunk_sum(v));
      const int col0 = blockIdx.x * (kRows / 2) + c * 8;
      if (col0 < half_n && req < p.n) {
        *reinterpret_cast<uint4*>(p.out_xp + (size_t)req * half_n + col0) = permute_chunk(v);
        if ((c & 7) == 0 && p.out_xs) p.out_xs[(size_t)(col0 >> 6) * 16 + req] = gsum;
      }
    }
    return;
  }

  for (int idx = threadIdx.x; idx < kRows * NP; idx += kThreads) {
    const int req = idx / kRows, lrow = idx - req * kRows;
    const int row = blockIdx.x * kRows + lrow;
    if (row < p.N && req < p.n) store_out(p, row, req, sT[lrow * kTs + req]);
  }
  if (p.epilogue == EPI_F32 && p.argmax_partial) {
    // Per request: the largest value of this row block and its row (lowest row among equals).
    for (int req = warp; req < NP; req += kWarps) {
      float best = -INFINITY;
      int bidx = 0x7fffffff;
      for (int lrow = lane; lrow < kRows; lrow += 32) {
        const int row = blockIdx.x * kRows + lrow;
        const float v = sT[lrow * kTs + req];
        if (row < p.N && (v > best || (v == best && row < bidx))) best = v, bidx = row;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bidx, o);
        if (ov > best || (ov == best && oi < bidx)) best = ov, bidx = oi;
      }
      if (lane == 0 && req < p.n) p.argmax_partial[(size_t)blockIdx.x * 16 + req] = make_float2(best, __int_as_float(bidx));
    }
  }
}

// ---- epilogue of a row tile ------------------------------------------------------------------------------------
// Epilogue of one finished row tile from the accumulators in MMA fragment layout (lane holds rows g, g + 8 and
// requests 2t, 2t + 1 of each block of 8 requests).  sE is 16 * (8 NT + 1) floats of the warp's own.
template <int NT, class Params>
__device__ __forceinline__ void tile_epilogue(const Params& p, const float (&acc)[NT][4], int tile, float* sE,
                                              int lane, float& best, int& bidx) {
  constexpr int NP = 8 * NT, kEs = NP + 1;
  const int g = lane >> 2, t = lane & 3;
  if (p.epilogue == EPI_SILU_PACK) {
    // rows g are gate rows, rows g + 8 the matching up rows: h = bf16(silu(bf16(gate)) * bf16(up)) is lane-local
    const int half_n = p.N >> 1;
    uint16_t* sH = reinterpret_cast<uint16_t*>(sE);  // [NP][8]
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const float gt = bf16_to_f32(f32_to_bf16(acc[nt][j]));
        const float up = bf16_to_f32(f32_to_bf16(acc[nt][2 + j]));
        sH[(nt * 8 + 2 * t + j) * 8 + g] = f32_to_bf16((gt / (1.0f + expf(-gt))) * up);
      }
    __syncwarp();
    const int col0 = tile * 8;
    if (lane < NP && lane < p.n && col0 < half_n) {
      const uint4 v = *reinterpret_cast<const uint4*>(sH + lane * 8);
      // element (lane, col0) of the consumer's operand: slices of out_ks features, strides set by the host
      const int sl = col0 / p.out_ks;
      *reinterpret_cast<uint4*>(p.out_xp + (size_t)sl * p.out_slice_stride + (size_t)lane * p.out_row_stride +
                                (col0 - sl * p.out_ks)) = permute_chunk(v);
    }
    __syncwarp();
    return;
  }
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
#pragma unroll
    for (int c = 0; c < 4; ++c) sE[(g + (c >> 1) * 8) * kEs + nt * 8 + 2 * t + (c & 1)] = acc[nt][c];
  __syncwarp();
  const int req = lane >> 1, half = lane & 1;
  const int row0 = tile * 16 + half * 8;
  float tb = -INFINITY;
  int ti = 0x7fffffff;
  if (req < NP && req < p.n && row0 < p.N) {
    float v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = sE[(half * 8 + i) * kEs + req];
    const bool full = row0 + 8 <= p.N && p.vec_ok;
    if (p.epilogue == EPI_F32) {
      float* o = reinterpret_cast<float*>(p.out) + (size_t)req * p.out_stride + row0;
      if (full) {
        *reinterpret_cast<float4*>(o) = make_float4(v[0], v[1], v[2], v[3]);
        *reinterpret_cast<float4*>(o + 4) = make_float4(v[4], v[5], v[6], v[7]);
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (row0 + i < p.N) o[i] = v[i];
      }
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (row0 + i < p.N && v[i] > tb) tb = v[i], ti = row0 + i;  // ascending rows: the lowest row among equals
    } else {
      uint16_t* o = reinterpret_cast<uint16_t*>(p.out) + (size_t)req * p.out_stride + row0;
      const bool res = p.epilogue == EPI_RESIDUAL;
      if (full) {
        uint4 old = make_uint4(0, 0, 0, 0);
        if (res) old = *reinterpret_cast<const uint4*>(o);
        const uint32_t ow[4] = {old.x, old.y, old.z, old.w};
        uint32_t nw[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          float a = bf16_to_f32(f32_to_bf16(v[2 * i])), b = bf16_to_f32(f32_to_bf16(v[2 * i + 1]));
          if (res) a += bf16_lo(ow[i]), b += bf16_hi(ow[i]);
          nw[i] = pack_bf16x2(a, b);
        }
        *reinterpret_cast<uint4*>(o) = make_uint4(nw[0], nw[1], nw[2], nw[3]);
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (row0 + i < p.N) {
            uint16_t y = f32_to_bf16(v[i]);
            if (res) y = f32_to_bf16(bf16_to_f32(o[i]) + bf16_to_f32(y));
            o[i] = y;
          }
      }
    }
  }
  if (p.epilogue == EPI_F32 && p.argmax_partial) {
    // the two lanes of a request cover rows 0..7 and 8..15 of the tile; both keep the request's running best
    const float ov = __shfl_xor_sync(0xffffffffu, tb, 1);
    const int oi = __shfl_xor_sync(0xffffffffu, ti, 1);
    if (ov > tb || (ov == tb && oi < ti)) tb = ov, ti = oi;
    if (tb > best || (tb == best && ti < bidx)) best = tb, bidx = ti;
  }
  __syncwarp();
}

// ---- round kernel ------------------------------------------------------------------------------------------------
// One CTA of kRoundWarps warps per SM owns a contiguous range of row tiles (of 16 rows) and one part of K (at most
// four slices of 1024 input features; most projections have a single part).  It walks its tiles in rounds of at
// most kRoundWarps / kw tiles; kw warps share a tile
// (stage j of the tile's stages goes to warp j mod kw of the tile) and add their accumulators through shared
// memory at the end of the round.  The CTA moves through the slices together: the activations of the
// next slice arrive by bulk copy in the other of two buffers while the warps multiply the current one, with one CTA
// barrier per slice.  The weight rings (XOR-swizzled, no padding) run ahead across slices, tiles and rounds.  With
// several parts of K the first warp of a tile hands its sums over through global scratch at the end of the round,
// and the last part to arrive adds them in part order and applies the epilogue.
struct RoundParams {
  const uint32_t* qw;
  const uint16_t* scales;
  const uint16_t* biases;
  const uint16_t* xp;
  const float* xs;  // group sums of the operand, or NULL: the CTA adds them up itself
  void* out;
  uint16_t* out_xp;
  float2* argmax_partial;  // [warps of the grid][16]
  unsigned int* status;    // set to 3 when a wait gives up (may be NULL)
  float* partial;          // [parts][T][MT * 16 * 8 NT] sums of a tile over one part of K (parts > 1 only)
  int* counters;           // [T], zero between launches (parts > 1 only)
  int N, K, n, out_stride, epilogue;
  int out_ks, out_row_stride, out_slice_stride;  // out_xp: features per slice, elements between rows and between slices
  int xp_layout;   // layout of xp: OPERAND_SLICED (one copy per slice) or OPERAND_ROWS (one copy per row and slice)
  int T;   // row tiles of MT sub-tiles
  int Tsub;  // sub-tiles of 16 rows (SiLU epilogue: 8 gate rows and the 8 matching up rows)
  int Q;   // stages per K-slice
  int S;   // K-slices per part; gridDim.y parts
  int kw;  // warps per tile
  int vec_ok;
};

constexpr int kRoundMT = 1;  // sub-tiles of 16 rows per warp tile (2, with 8 warps of 198 registers, measured no faster)
// 12 warps of up to 170 registers: with 16 the 128-register cap cost more in instruction scheduling than the four
// extra warps gave (LM head 175 -> 138 us, the batch-1 step of the 8B shape 3.00 -> 2.70 ms)
constexpr int kRoundWarps = 12, kRoundThreads = 32 * kRoundWarps;
// a stage: 16 MT rows of 128 B of codes, 16-byte chunks swizzled by row, then the rows' scales and biases
constexpr int kRoundRows = 16 * kRoundMT, kRoundStage = kRoundRows * (128 + kSbBytes);

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

template <int NT, int STAGES, bool SLICED>  // SLICED: the operand's layout (one copy per slice) or plain rows
__global__ void __launch_bounds__(kRoundThreads, 1) q4_round_kernel(const RoundParams p) {
  constexpr int NP = 8 * NT, MT = kRoundMT, RW = kRoundRows;
  constexpr int kEs = NP + 1;
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) uint64_t s_mbar[2];

  grid_launch_dependents();

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const bool silu = p.epilogue == EPI_SILU_PACK;
  const int half_n = p.N >> 1;
  const int Q = p.Q, S = p.S, SQ = S * Q, kw = p.kw;
  const int parts = gridDim.y, part_j0 = blockIdx.y * SQ;  // this CTA's part of K starts at stage part_j0
  const int ks = Q * 256;
  const int b_stride = ks * 2 + 16;        // bytes per request row of a staged slice
  const int act_bytes = NP * b_stride;     // one activation buffer
  const int sum_bytes = Q * 4 * 16 * 4;    // group sums of a slice: [group][16]

  unsigned char* ring = smem + warp * (STAGES * kRoundStage);
  unsigned char* sAct = smem + kRoundWarps * STAGES * kRoundStage;  // two buffers
  float* sSum = reinterpret_cast<float*>(sAct + 2 * act_bytes);     // two buffers
  (void)kEs;

  // the CTA's tiles and rounds
  const int t0 = (int)((long long)blockIdx.x * p.T / gridDim.x), t1 = (int)((long long)(blockIdx.x + 1) * p.T / gridDim.x);
  const int Tc = t1 - t0, tpr = kRoundWarps / kw;
  const int R = (Tc + tpr - 1) / tpr;
  const int base = R ? Tc / R : 0, rem = R ? Tc - base * R : 0;  // rounds [0, rem) hold base + 1 tiles
  const int ts = warp / kw, kp = warp - ts * kw;
  const int my_rounds = ts < base ? R : (ts == base ? rem : 0);  // the warp has a tile in rounds [0, my_rounds)
  auto tile_of = [&](int r) -> int { return t0 + r * base + min(r, rem) + ts; };

  // row r of a tile belongs to sub-tile tile * MT + r / 16
  auto row_of = [&](int tile, int r) -> int {
    const int sub = tile * MT + (r >> 4), rr = r & 15;
    if (!silu) return min(sub * 16 + rr, p.N - 1);
    return rr < 8 ? min(sub * 8 + rr, half_n - 1) : min(half_n + sub * 8 + (rr - 8), p.N - 1);
  };
  auto issue_stage = [&](int slot, int tile, int j) {
    unsigned char* stg = ring + slot * kRoundStage;
    const int kq = (part_j0 + j) * 256;
#pragma unroll
    for (int i = 0; i < RW / 4; ++i) {
      const int r = i * 4 + (lane >> 3);
      const int grow = row_of(tile, r);
      const unsigned char* src =
          reinterpret_cast<const unsigned char*>(p.qw + (size_t)grow * (p.K >> 3) + (kq >> 3)) + (lane & 7) * 16;
      cp_async16(stg + r * 128 + (((lane & 7) ^ (r & 7)) << 4), src);
    }
    if (lane < RW) {
      const int grow = row_of(tile, lane);
      const size_t off = (size_t)grow * (p.K >> 6) + (kq >> 6);
      cp_async8(stg + RW * 128 + lane * kSbBytes, p.scales + off);
      cp_async8(stg + RW * 128 + lane * kSbBytes + 8, p.biases + off);
    }
  };

  // cursors over the warp's stages: (round, stage of the tile), stage = kp, kp + kw, ...
  int ir = 0, ij = kp;  // next stage to request
  int cr = 0, cj = kp;  // next stage to multiply
  int islot = 0, cslot = 0;
  const bool any = my_rounds > 0 && kp < SQ;
  // Weights do not depend on the preceding kernel: start streaming them before waiting for it.
#pragma unroll
  for (int s = 0; s < STAGES - 1; ++s) {
    if (any && ir < my_rounds) {
      issue_stage(islot, tile_of(ir), ij);
      ij += kw;
      if (ij >= SQ) ij = kp, ++ir;
      if (++islot == STAGES) islot = 0;
    }
    cp_async_commit();
  }

  if (threadIdx.x == 0) {
    mbar_init(&s_mbar[0], 1u);
    mbar_init(&s_mbar[1], 1u);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  grid_dependency_wait();

  // A slice arrives as one bulk copy of all its rows (sliced layout) or one per request row (plain rows), plus one
  // for its group sums, tracked by the buffer's mbarrier.
  // Only the rows of requests that exist are fetched; the other columns of the MMAs multiply whatever the buffer
  // holds and their results are never stored.
  const int rows_used = p.n < NP ? p.n : NP;
  constexpr bool sliced = SLICED;  // a sliced row comes with its padding
  const uint32_t slice_bytes = (uint32_t)(rows_used * (sliced ? b_stride : ks * 2) + (p.xs ? sum_bytes : 0));
  auto stage_acts = [&](int gstep) {  // the lanes of warp 0 issue the copies side by side
    if (warp == 0) {
      const int buf = gstep & 1, slice = blockIdx.y * S + gstep % S;
      if (lane == 0) mbar_expect_tx(&s_mbar[buf], slice_bytes);
      if (sliced && lane == 0)  // the slice's rows are one contiguous block, padded like their image here
        bulk_copy_g2s(sAct + buf * act_bytes, p.xp + (size_t)slice * 16 * (ks + 8), (uint32_t)(rows_used * b_stride),
                      &s_mbar[buf]);
      else if (!sliced && lane < rows_used)
        bulk_copy_g2s(sAct + buf * act_bytes + lane * b_stride, p.xp + (size_t)lane * p.K + (size_t)slice * ks,
                      (uint32_t)(ks * 2), &s_mbar[buf]);
      else if (lane == NP && p.xs)
        bulk_copy_g2s(sSum + buf * (sum_bytes / 4), p.xs + (size_t)slice * Q * 4 * 16, (uint32_t)sum_bytes, &s_mbar[buf]);
    }
    __syncwarp();  // lanes that have nothing to issue go on to poll the mbarrier: they must not starve the others
  };
  const int steps = R * S;
  if (steps > 0) stage_acts(0);

  float acc[MT][NT][4];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[mt][nt][c] = 0.0f;
  float best = -INFINITY;
  int bidx = 0x7fffffff;

  int gstep = 0;
  for (int r = 0; r < R; ++r) {
    for (int s = 0; s < S; ++s, ++gstep) {
      // the other buffer was last read in step gstep - 1, which every warp has left (barrier below)
      if (gstep + 1 < steps) stage_acts(gstep + 1);
      const int b = gstep & 1;
      if (!mbar_wait(&s_mbar[b], (uint32_t)((gstep >> 1) & 1))) {
        if (lane == 0 && p.status) atomicExch(p.status, 3u);  // the copy never landed: report, results are void
      }
      const unsigned char* sB = sAct + b * act_bytes;
      float* sX = sSum + b * (sum_bytes / 4);
      if (!p.xs) {
        // the producer left no group sums: add up the 64 staged elements of every (group, request) of the slice
        for (int c = threadIdx.x; c < Q * 4 * NP; c += kRoundThreads) {
          const int gq = c / NP, rq = c - gq * NP;
          const uint4* src = reinterpret_cast<const uint4*>(sB + rq * b_stride + gq * 128);
          float sum = 0.0f;
#pragma unroll
          for (int i = 0; i < 8; ++i) sum += chunk_sum(src[i]);
          sX[gq * 16 + rq] = sum;
        }
        __syncthreads();
      }

      while (any && cr == r && cr < my_rounds && cj < (s + 1) * Q) {
        if (ir < my_rounds) {
          issue_stage(islot, tile_of(ir), ij);
          ij += kw;
          if (ij >= SQ) ij = kp, ++ir;
          if (++islot == STAGES) islot = 0;
        }
        cp_async_commit();
        cp_async_wait<STAGES - 1>();
        __syncwarp();
        const unsigned char* stg = ring + cslot * kRoundStage;
        if (++cslot == STAGES) cslot = 0;
        const int cq = cj - s * Q;

        uint2 sc[MT][2], bi[MT][2];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const uint4 v = *reinterpret_cast<const uint4*>(stg + RW * 128 + (mt * 16 + g + 8 * h) * kSbBytes);
            sc[mt][h] = make_uint2(v.x, v.y);
            bi[mt][h] = make_uint2(v.z, v.w);
          }
#pragma unroll
        for (int gi = 0; gi < 4; ++gi) {
          const int gidx = cq * 4 + gi;
          uint4 bf[NT][2];
          float2 xs[NT];
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            const unsigned char* bp = sB + (nt * 8 + g) * b_stride + gidx * 128 + t * 32;
            bf[nt][0] = *reinterpret_cast<const uint4*>(bp);
            bf[nt][1] = *reinterpret_cast<const uint4*>(bp + 16);
            xs[nt] = *reinterpret_cast<const float2*>(sX + gidx * 16 + nt * 8 + 2 * t);
          }
          // 16-byte chunk c of row r sits at chunk c ^ (r & 7); rows g, g + 8, g + 16, ... share the swizzle
          const int woff = g * 128 + (((gi * 2 + (t >> 1)) ^ g) << 4) + (t & 1) * 8;
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
            const uint2 wl = *reinterpret_cast<const uint2*>(stg + mt * 16 * 128 + woff);
            const uint2 wh = *reinterpret_cast<const uint2*>(stg + mt * 16 * 128 + woff + 8 * 128);
            uint32_t l0[4], l1[4], h0[4], h1[4];
            unpack_word(wl.x, l0);
            unpack_word(wl.y, l1);
            unpack_word(wh.x, h0);
            unpack_word(wh.y, h1);
            // sum (16 + q) x = 16 X + sum q x, so the bias that multiplies X becomes b - 16 s
            const float s_lo = bf16_at(sc[mt][0], gi), s_hi = bf16_at(sc[mt][1], gi);
            const float b_lo = fmaf(-16.0f, s_lo, bf16_at(bi[mt][0], gi)), b_hi = fmaf(-16.0f, s_hi, bf16_at(bi[mt][1], gi));
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              float pc[4];
              mma_bf16_first(pc, l0[0], h0[0], l0[1], h0[1], bf[nt][0].x, bf[nt][0].y);
              mma_bf16(pc, l0[2], h0[2], l0[3], h0[3], bf[nt][0].z, bf[nt][0].w);
              mma_bf16(pc, l1[0], h1[0], l1[1], h1[1], bf[nt][1].x, bf[nt][1].y);
              mma_bf16(pc, l1[2], h1[2], l1[3], h1[3], bf[nt][1].z, bf[nt][1].w);
              scale_bias_fma(acc[mt][nt], pc, s_lo, s_hi, b_lo, b_hi, xs[nt]);
            }
          }
        }
        __syncwarp();
        cj += kw;
        if (cj >= SQ) cj = kp, ++cr;
      }

      if (s == S - 1 && kw > 1 && kp != 0 && r < my_rounds) {
        // hand the accumulators to the tile's first warp through the ring slot this warp has just multiplied: it
        // is free until the warp requests its next stage (lane-major: conflict-free both ways)
        float4* dst = reinterpret_cast<float4*>(ring + (cslot == 0 ? STAGES - 1 : cslot - 1) * kRoundStage);
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int nt = 0; nt < NT; ++nt)
            dst[(mt * NT + nt) * 32 + lane] = make_float4(acc[mt][nt][0], acc[mt][nt][1], acc[mt][nt][2], acc[mt][nt][3]);
      }
      __syncthreads();
    }
    // round end: the first warp of every tile adds its partners in warp order and applies the epilogue
    if (r < my_rounds && kp == 0) {
      for (int k = 1; k < kw; ++k) {
        // partner k has multiplied (r + 1) * ceil((SQ - k) / kw) stages so far: its last slot follows from that
        const int pslot = ((r + 1) * ((SQ - k + kw - 1) / kw) - 1) % STAGES;
        const float4* src = reinterpret_cast<const float4*>(smem + (warp + k) * (STAGES * kRoundStage) + pslot * kRoundStage);
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            const float4 a = src[(mt * NT + nt) * 32 + lane];
            acc[mt][nt][0] += a.x, acc[mt][nt][1] += a.y, acc[mt][nt][2] += a.z, acc[mt][nt][3] += a.w;
          }
      }
      const int tile = tile_of(r);
      bool finish = true;
      if (parts > 1) {
        // several CTAs hold parts of this tile's sums: publish, and the last to arrive adds them in part order
        constexpr int kF4 = 32 * MT * NT;  // float4 per tile and part
        float4* part = reinterpret_cast<float4*>(p.partial) + ((size_t)blockIdx.y * p.T + tile) * kF4;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int nt = 0; nt < NT; ++nt)
            part[(mt * NT + nt) * 32 + lane] = make_float4(acc[mt][nt][0], acc[mt][nt][1], acc[mt][nt][2], acc[mt][nt][3]);
        __threadfence();
        __syncwarp();
        int prev = 0;
        if (lane == 0) prev = atomicAdd(p.counters + tile, 1);
        prev = __shfl_sync(0xffffffffu, prev, 0);
        finish = prev == parts - 1;
        if (finish) {
          __threadfence();
          if (lane == 0) p.counters[tile] = 0;
#pragma unroll
          for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
              for (int c = 0; c < 4; ++c) acc[mt][nt][c] = 0.0f;
          for (int y0 = 0; y0 < parts; y0 += 2) {  // two parts at a time: their loads go out together
            float4 v[2][MT * NT];
#pragma unroll
            for (int y = 0; y < 2; ++y)
#pragma unroll
              for (int i = 0; i < MT * NT; ++i)
                v[y][i] = y0 + y < parts
                              ? __ldcg(reinterpret_cast<const float4*>(p.partial) + ((size_t)(y0 + y) * p.T + tile) * kF4 + i * 32 + lane)
                              : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
#pragma unroll
            for (int y = 0; y < 2; ++y)
#pragma unroll
              for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                  const float4 a = v[y][mt * NT + nt];
                  acc[mt][nt][0] += a.x, acc[mt][nt][1] += a.y, acc[mt][nt][2] += a.z, acc[mt][nt][3] += a.w;
                }
          }
        }
      }
      // the epilogue transposes through the ring slot the warp has just multiplied, one sub-tile at a time
      if (finish) {
        float* sE = reinterpret_cast<float*>(ring + (cslot == 0 ? STAGES - 1 : cslot - 1) * kRoundStage);
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
          if (tile * MT + mt < p.Tsub) tile_epilogue<NT>(p, acc[mt], tile * MT + mt, sE, lane, best, bidx);
      }
    }
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[mt][nt][c] = 0.0f;
    if (kw > 1) __syncthreads();  // the partners' slots are read before anyone requests a stage into them
  }
  cp_async_wait<0>();

  if (p.epilogue == EPI_F32 && p.argmax_partial && (lane & 1) == 0) {
    const int req = lane >> 1;
    if (req < NP && req < p.n)
      p.argmax_partial[((size_t)(blockIdx.y * gridDim.x + blockIdx.x) * kRoundWarps + warp) * 16 + req] =
          make_float2(best, __int_as_float(bidx));
  }
}

// ---- span kernel: projections whose CTAs hold at most kRoundWarps row tiles ---------------------------------------
// All K-slices of the CTA's part of K (at most four) are resident in shared memory, so nothing ties the warps to one
// another while they multiply.  The CTA's stages, row tile major, are cut into equal contiguous spans, one per
// warp: every warp streams the same number of stages (to within one) whatever the number of tiles, a span covers the
// tail of one tile and the head of the next at most, and each warp refills the ring slot it has just multiplied.
// At the end the warps leave their (one or two) partial sums in shared memory, and the warp that holds a tile's first
// stage adds the tile's partial sums in warp order and applies the epilogue.
// acc += the stage's 16 rows x 256 input features against the staged operand (sB: the slice, sX: its group sums,
// cq: the stage's place in the slice).
template <int NT>
__device__ __forceinline__ void span_multiply_stage(const unsigned char* stg, const unsigned char* sB, const float* sX,
                                                    int b_stride, int cq, int g, int t, float (&acc)[NT][4]) {
  uint2 sc[2], bi[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const uint4 v = *reinterpret_cast<const uint4*>(stg + 16 * 128 + (g + 8 * h) * kSbBytes);
    sc[h] = make_uint2(v.x, v.y);
    bi[h] = make_uint2(v.z, v.w);
  }
#pragma unroll
  for (int gi = 0; gi < 4; ++gi) {
    const int gidx = cq * 4 + gi;
    uint4 bf[NT][2];
    float2 xs[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const unsigned char* bp = sB + (nt * 8 + g) * b_stride + gidx * 128 + t * 32;
      bf[nt][0] = *reinterpret_cast<const uint4*>(bp);
      bf[nt][1] = *reinterpret_cast<const uint4*>(bp + 16);
      xs[nt] = *reinterpret_cast<const float2*>(sX + gidx * 16 + nt * 8 + 2 * t);
    }
    // 16-byte chunk c of row r sits at chunk c ^ (r & 7); rows g and g + 8 share the swizzle
    const int woff = g * 128 + (((gi * 2 + (t >> 1)) ^ g) << 4) + (t & 1) * 8;
    const uint2 wl = *reinterpret_cast<const uint2*>(stg + woff);
    const uint2 wh = *reinterpret_cast<const uint2*>(stg + woff + 8 * 128);
    uint32_t l0[4], l1[4], h0[4], h1[4];
    unpack_word(wl.x, l0);
    unpack_word(wl.y, l1);
    unpack_word(wh.x, h0);
    unpack_word(wh.y, h1);
    // sum (16 + q) x = 16 X + sum q x, so the bias that multiplies X becomes b - 16 s
    const float s_lo = bf16_at(sc[0], gi), s_hi = bf16_at(sc[1], gi);
    const float b_lo = fmaf(-16.0f, s_lo, bf16_at(bi[0], gi)), b_hi = fmaf(-16.0f, s_hi, bf16_at(bi[1], gi));
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      float pc[4];
      mma_bf16_first(pc, l0[0], h0[0], l0[1], h0[1], bf[nt][0].x, bf[nt][0].y);
      mma_bf16(pc, l0[2], h0[2], l0[3], h0[3], bf[nt][0].z, bf[nt][0].w);
      mma_bf16(pc, l1[0], h1[0], l1[1], h1[1], bf[nt][1].x, bf[nt][1].y);
      mma_bf16(pc, l1[2], h1[2], l1[3], h1[3], bf[nt][1].z, bf[nt][1].w);
      scale_bias_fma(acc[nt], pc, s_lo, s_hi, b_lo, b_hi, xs[nt]);
    }
  }
}

template <int NT, int STAGES, bool SLICED>  // SLICED: the operand's layout (one copy per slice) or plain rows
__global__ void __launch_bounds__(kRoundThreads, 1) q4_span_kernel(const RoundParams p) {
  static_assert(kRoundMT == 1, "the span kernel works on 16-row tiles");
  constexpr int NP = 8 * NT, W = kRoundWarps;
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) uint64_t s_mbar;

  grid_launch_dependents();

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const bool silu = p.epilogue == EPI_SILU_PACK;
  const int half_n = p.N >> 1;
  const int Q = p.Q, S = p.S, SQ = S * Q;
  const int parts = gridDim.y, part_j0 = blockIdx.y * SQ;
  const int ks = Q * 256;
  const int b_stride = ks * 2 + 16;
  const int act_bytes = NP * b_stride;
  const int sum_bytes = Q * 4 * 16 * 4;

  unsigned char* ring = smem + warp * (STAGES * kRoundStage);
  unsigned char* sAct = smem + W * STAGES * kRoundStage;             // S buffers; the partial sums at the end
  float* sSum = reinterpret_cast<float*>(sAct + S * act_bytes);     // S buffers

  // the CTA's tiles, and this warp's span of their stages
  const int t0 = (int)((long long)blockIdx.x * p.T / gridDim.x), t1 = (int)((long long)(blockIdx.x + 1) * p.T / gridDim.x);
  const int Tc = t1 - t0, Lc = Tc * SQ;
  // Span (w % 4) * (W / 4) + w / 4 belongs to warp w: when only every second or fourth span holds a stage (few stages per
  // CTA) the busy warps still spread over the four schedulers of the SM.
  const int span = (warp & 3) * (W / 4) + (warp >> 2);
  auto span_begin = [&](int i) -> int { return i * Lc / W; };
  const int a = span_begin(span), cnt = span_begin(span + 1) - a;
  const int tlA = a / SQ, jA0 = a - tlA * SQ;
  const int lenA = min(cnt, SQ - jA0);  // stages in the first tile; the rest belong to tile tlA + 1, from its stage 0
  auto stage_of = [&](int i, int& tl, int& j) {
    if (i < lenA) tl = tlA, j = jA0 + i;
    else tl = tlA + 1, j = i - lenA;
  };

  const int q_recip = (65536 + Q - 1) / Q;  // j / Q == (j * q_recip) >> 16 for j < 4096 and Q <= 4
  // The addresses of a tile's rows are worked out once per tile (a span touches two tiles at most), not per stage:
  // a stage then costs five additions instead of five 64-bit multiplications with their row clamps.
  const unsigned char* row_src[4];  // rows 4i + lane / 8 of the tile, at this lane's 16 bytes of feature 0
  size_t sb_off = 0;                // row `lane` of the tile in the scale / bias tensors (lanes < 16)
  int rows_tl = -1;
  auto issue_stage = [&](unsigned char* stg, int tl, int j) {
    if (tl != rows_tl) {
      rows_tl = tl;
      const int sub = t0 + tl;
      auto row_of = [&](int r) -> int {
        if (!silu) return min(sub * 16 + r, p.N - 1);
        return r < 8 ? min(sub * 8 + r, half_n - 1) : min(half_n + sub * 8 + (r - 8), p.N - 1);
      };
#pragma unroll
      for (int i = 0; i < 4; ++i)
        row_src[i] = reinterpret_cast<const unsigned char*>(p.qw + (size_t)row_of(i * 4 + (lane >> 3)) * (p.K >> 3)) +
                     (lane & 7) * 16;
      sb_off = (size_t)row_of(lane & 15) * (p.K >> 6);
    }
    const int kq = (part_j0 + j) * 256;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int r = i * 4 + (lane >> 3);
      cp_async16(stg + r * 128 + (((lane & 7) ^ (r & 7)) << 4), row_src[i] + (kq >> 1));
    }
    if (lane < 16) {
      cp_async8(stg + 16 * 128 + lane * kSbBytes, p.scales + sb_off + (kq >> 6));
      cp_async8(stg + 16 * 128 + lane * kSbBytes + 8, p.biases + sb_off + (kq >> 6));
    }
  };

  // Weights do not depend on the preceding kernel: fill the ring before waiting for it.
#pragma unroll
  for (int i = 0; i < STAGES; ++i) {
    if (i < cnt) {
      int tl, j;
      stage_of(i, tl, j);
      issue_stage(ring + i * kRoundStage, tl, j);
    }
    cp_async_commit();
  }

  if (threadIdx.x == 0) {
    mbar_init(&s_mbar, 1u);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  grid_dependency_wait();

  // every slice of the operand (and its group sums) on one mbarrier: one bulk copy per slice in the sliced layout,
  // one per request row and slice with plain rows, issued by the lanes of warp 0 side by side
  if (warp == 0) {
    // only the rows of requests that exist are fetched: the other columns of the MMAs multiply whatever the buffer
    // holds and their results are never stored
    const int rows_used = p.n < NP ? p.n : NP;
    const int row_bytes = SLICED ? b_stride : ks * 2;  // a sliced row comes with its padding
    if (lane == 0) mbar_expect_tx(&s_mbar, (uint32_t)(rows_used * row_bytes + (p.xs ? sum_bytes : 0)) * (uint32_t)S);
    // a slice of the operand is one contiguous block in global memory, padded like its image here: one copy each
    // for the rows and for the sums (the copy engine's time goes with the number of copies, not with their bytes)
    const int per = NP + 1;  // copies per slice at most: the rows, then the sums
    for (int i = lane; i < S * per; i += 32) {
      const int sl = i / per, r = i - sl * per, slice = blockIdx.y * S + sl;
      if (r == NP) {
        if (p.xs) bulk_copy_g2s(sSum + sl * (sum_bytes / 4), p.xs + (size_t)slice * Q * 4 * 16, (uint32_t)sum_bytes, &s_mbar);
      } else if (SLICED) {
        if (r == 0)
          bulk_copy_g2s(sAct + sl * act_bytes, p.xp + (size_t)slice * 16 * (ks + 8), (uint32_t)(rows_used * b_stride), &s_mbar);
      } else if (r < rows_used) {
        bulk_copy_g2s(sAct + sl * act_bytes + r * b_stride, p.xp + (size_t)r * p.K + (size_t)slice * ks, (uint32_t)(ks * 2),
                      &s_mbar);
      }
    }
  }
  __syncwarp();  // lanes that have nothing to issue go on to poll the mbarrier: they must not starve the others
  if (!mbar_wait(&s_mbar, 0u)) {
    if (lane == 0 && p.status) atomicExch(p.status, 3u);  // the copies never landed: report, results are void
  }
  if (!p.xs) {
    // the producer left no group sums: add up the 64 staged elements of every (slice, group, request)
    const int per = Q * 4 * NP;
    for (int c = threadIdx.x; c < S * per; c += kRoundThreads) {
      const int sl = c / per, cc = c - sl * per;
      const int gq = cc / NP, rq = cc - gq * NP;
      const uint4* src = reinterpret_cast<const uint4*>(sAct + sl * act_bytes + rq * b_stride + gq * 128);
      float sum = 0.0f;
#pragma unroll
      for (int i = 0; i < 8; ++i) sum += chunk_sum(src[i]);
      sSum[sl * (sum_bytes / 4) + gq * 16 + rq] = sum;
    }
    __syncthreads();
  }

  float acc[NT][4], first[NT][4];  // the tile being multiplied; the finished part of the span's first tile
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
#pragma unroll
    for (int c = 0; c < 4; ++c) acc[nt][c] = 0.0f, first[nt][c] = 0.0f;

  int slot = 0;
  for (int i = 0; i < cnt; ++i) {
    cp_async_wait<STAGES - 1>();
    __syncwarp();
    int tl, j;
    stage_of(i, tl, j);
    if (i == lenA) {  // the span moves on to its second tile
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int c = 0; c < 4; ++c) first[nt][c] = acc[nt][c], acc[nt][c] = 0.0f;
    }
    const int sl = (j * q_recip) >> 16, cq = j - sl * Q;  // j / Q for the few stages of a tile
    span_multiply_stage<NT>(ring + slot * kRoundStage, sAct + sl * act_bytes, sSum + sl * (sum_bytes / 4), b_stride, cq, g, t,
                            acc);
    __syncwarp();
    if (i + STAGES < cnt) {  // refill the slot just multiplied
      int tl2, j2;
      stage_of(i + STAGES, tl2, j2);
      issue_stage(ring + slot * kRoundStage, tl2, j2);
    }
    cp_async_commit();
    if (++slot == STAGES) slot = 0;
  }
  cp_async_wait<0>();
  const bool two = cnt > lenA;  // the span reached a second tile: `first` holds tile tlA, acc tile tlA + 1
  __syncthreads();              // nobody reads the operand any more: its buffers take the partial sums

  // partial sums, lane-major: [span][first or second tile of the span][NT][32 lanes] float4
  float4* sP = reinterpret_cast<float4*>(sAct);
  if (cnt > 0) {
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const float (&fa)[4] = two ? first[nt] : acc[nt];
      sP[((span * 2 + 0) * NT + nt) * 32 + lane] = make_float4(fa[0], fa[1], fa[2], fa[3]);
      if (two) sP[((span * 2 + 1) * NT + nt) * 32 + lane] = make_float4(acc[nt][0], acc[nt][1], acc[nt][2], acc[nt][3]);
    }
  }
  __syncthreads();

  float best = -INFINITY;
  int bidx = 0x7fffffff;
  // The warp whose span holds a tile's first stage finishes the tile (it adds the spans' partial sums in span order): its own first tile if the span starts at the
  // tile's stage 0, and its second tile always.
  for (int which = 0; which < 2; ++which) {
    const bool own = which == 0 ? (cnt > 0 && jA0 == 0) : two;
    if (!own) continue;
    const int tl = tlA + which;
    const int last = ((tl * SQ + SQ) * W - 1) / Lc;  // the span that holds the tile's last stage
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[nt][c] = 0.0f;
    const int tile_first = tl * SQ;  // the tile's first stage
#pragma unroll 4
    for (int w2 = span; w2 <= last; ++w2) {
      const int b0 = span_begin(w2);
      if (span_begin(w2 + 1) == b0) continue;  // an empty span (fewer stages than warps)
      const int sel = b0 < tile_first ? 1 : 0;  // the tile is that span's first tile, or its second
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const float4 v = sP[((w2 * 2 + sel) * NT + nt) * 32 + lane];
        acc[nt][0] += v.x, acc[nt][1] += v.y, acc[nt][2] += v.z, acc[nt][3] += v.w;
      }
    }
    const int tile = t0 + tl;
    bool finish = true;
    if (parts > 1) {
      // several CTAs hold parts of this tile's sums: publish, and the last to arrive adds them in part order
      float4* part = reinterpret_cast<float4*>(p.partial) + ((size_t)blockIdx.y * p.T + tile) * (32 * NT);
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) part[nt * 32 + lane] = make_float4(acc[nt][0], acc[nt][1], acc[nt][2], acc[nt][3]);
      __threadfence();
      __syncwarp();
      int prev = 0;
      if (lane == 0) prev = atomicAdd(p.counters + tile, 1);
      prev = __shfl_sync(0xffffffffu, prev, 0);
      finish = prev == parts - 1;
      if (finish) {
        __threadfence();
        if (lane == 0) p.counters[tile] = 0;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int c = 0; c < 4; ++c) acc[nt][c] = 0.0f;
        for (int y0 = 0; y0 < parts; y0 += 4) {  // four parts at a time: their loads go out together
          float4 v[4][NT];
#pragma unroll
          for (int y = 0; y < 4; ++y)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
              v[y][nt] = y0 + y < parts ? __ldcg(reinterpret_cast<const float4*>(p.partial) +
                                                 ((size_t)(y0 + y) * p.T + tile) * (32 * NT) + nt * 32 + lane)
                                        : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
#pragma unroll
          for (int y = 0; y < 4; ++y)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
              acc[nt][0] += v[y][nt].x, acc[nt][1] += v[y][nt].y, acc[nt][2] += v[y][nt].z, acc[nt][3] += v[y][nt].w;
        }
      }
    }
    // the epilogue transposes through the warp's ring, which is idle now
    if (finish && tile < p.Tsub) tile_epilogue<NT>(p, acc, tile, reinterpret_cast<float*>(ring), lane, best, bidx);
  }

  if (p.epilogue == EPI_F32 && p.argmax_partial && (lane & 1) == 0) {
    const int req = lane >> 1;
    if (req < NP && req < p.n)
      p.argmax_partial[((size_t)(blockIdx.y * gridDim.x + blockIdx.x) * W + warp) * 16 + req] =
          make_float2(best, __int_as_float(bidx));
  }
}

constexpr int g_part_slices = 4;  // K-slices per part of K

struct RoundPlan {
  int nt, stages, Q, S, parts, T, Tsub, ctas, kw;
  bool span;  // at most 16 tiles per CTA: the span kernel
  int span_stages;
  size_t span_smem;
  size_t smem, partial_bytes;
};

RoundPlan plan_rounds(int N, int K, int n, int epilogue, int sm_count) {
  RoundPlan t;
  t.nt = n <= 8 ? 1 : 2;
  t.stages = t.nt == 1 ? 3 : 2;  // ring slots per warp; deeper rings measured slower (LM head: 4 -> 142 us, 5 -> 171 us, 2 -> 137 us)
  const int quads = K / 256;
  static_assert(kMaxQuadsPerSlice == 4, "operand_slice_features cuts K into slices of at most 4 x 256 features");
  t.Q = operand_slice_features(K) / 256;  // the producers lay the operand out in these slices
  const int slices = quads / t.Q;
  // A CTA re-reads the activations of its part of K for every round, so K is cut into parts of at most four
  // slices: beyond that the activations would outweigh the CTA's weights.
  t.parts = 1;
  while (slices % t.parts || slices / t.parts > g_part_slices) ++t.parts;
  t.S = slices / t.parts;
  t.Tsub = epilogue == EPI_SILU_PACK ? (N / 2 + 7) / 8 : (N + 15) / 16;
  t.T = (t.Tsub + kRoundMT - 1) / kRoundMT;
  int ctas = sm_count / t.parts;
  if (ctas < 1) ctas = 1;
  t.ctas = t.T < ctas ? t.T : ctas;
  const int per_cta = (t.T + t.ctas - 1) / t.ctas;
  int kw = 1;
  while (kw * 2 <= kRoundWarps / per_cta && kw * 2 <= t.S * t.Q) kw *= 2;  // fill the CTA's warps, a stage each at least
  t.kw = kw;
  const int np = 8 * t.nt;
  t.smem = (size_t)kRoundWarps * t.stages * kRoundStage + 2 * ((size_t)np * (t.Q * 512 + 16) + (size_t)t.Q * 4 * 16 * 4);
  t.partial_bytes = t.parts > 1 ? (size_t)t.parts * t.T * kRoundRows * np * sizeof(float) : 0;
  t.span = per_cta <= kRoundWarps && kRoundMT == 1;
  // Two ring slots per warp, each refilled as soon as it is multiplied.  Measured: deeper rings are slower (8B shape,
  // batch 16, three slots instead of two: gate/up 29 -> 37 us, down 23 -> 27 us) — more requests in flight than the
  // memory system serves well, and a larger footprint keeps the next projection's CTAs off the SM for longer.
  t.span_stages = 2;
  const size_t operand = t.S * ((size_t)np * (t.Q * 512 + 16) + (size_t)t.Q * 4 * 16 * 4);
  const size_t handover = (size_t)kRoundWarps * 2 * 16 * np * sizeof(float);  // two partial tiles per warp, in the operand's place
  t.span_smem = (size_t)kRoundWarps * t.span_stages * kRoundStage + (operand > handover ? operand : handover);
  return t;
}

template <int MT, int NT, int STAGES>
size_t smem_bytes(int ks) {
  return (size_t)kWarps * STAGES * (16 * MT) * (kRowStride + kSbBytes) + (size_t)(8 * NT) * (ks * 2 + 16) +
         (size_t)(ks / 64) * (8 * NT) * sizeof(float);
}

struct Tiling {
  int cfg;  // 0: <1,1,4>  1: <2,2,4>  2: <1,2,3>
  int nt, rows_cta, rowblocks, qps, splits;
};

int g_sm_count = 0;

Tiling choose_tiling(int N, int K, int n, int epilogue, int sm_count, bool grouped = false) {
  Tiling t;
  const int rows_logical = epilogue == EPI_SILU_PACK ? N / 2 : N;  // rows that index row blocks
  const int quads = K / 256;
  if (n <= 8) {
    t.cfg = 0, t.nt = 1, t.rows_cta = 128;
  } else {
    t.cfg = 2;  // two 128-row CTAs per SM hide more latency than one 256-row CTA (measured)
    t.nt = 2, t.rows_cta = 128;
  }
  const int rows_per_block = epilogue == EPI_SILU_PACK ? t.rows_cta / 2 : t.rows_cta;
  t.rowblocks = (rows_logical + rows_per_block - 1) / rows_per_block;
  const int wave = sm_count * (t.cfg == 1 ? 1 : 2);
  int qps = 1;
  for (int c = (quads < kMaxQuadsPerSlice ? quads : kMaxQuadsPerSlice); c >= 1; --c) {
    if (quads % c) continue;
    if ((long long)t.rowblocks * (quads / c) >= wave || c == 1) {
      qps = c;
      break;
    }
  }
  if (grouped) qps = quads;  // experts: many small GEMMs fill the machine without split-K (K <= 2048)
  t.qps = qps;
  t.splits = quads / qps;
  return t;
}

size_t tiling_partial_bytes(const Tiling& t) {
  return t.splits > 1 ? (size_t)t.splits * t.rowblocks * t.rows_cta * (8 * t.nt) * sizeof(float) : 0;
}

int sm_count_or_default() {
  if (g_sm_count == 0) {
    if (gemm_init() != cudaSuccess) {
      (void)cudaGetLastError();
      return 148;  // sizing only: no device in this process
    }
  }
  return g_sm_count;
}

// next[r] = the best of the row-block partial results, lowest index among equals.
__global__ void __launch_bounds__(256) argmax_finish_kernel(const float2* partial, int row_blocks, int32_t* next) {
  __shared__ float sv[8];
  __shared__ int si[8];
  grid_launch_dependents();
  grid_dependency_wait();
  const int req = blockIdx.x;
  float best = -INFINITY;
  int bidx = 0x7fffffff;
  for (int b = threadIdx.x; b < row_blocks; b += blockDim.x) {
    const float2 v = partial[(size_t)b * 16 + req];
    const int i = __float_as_int(v.y);
    if (v.x > best || (v.x == best && i < bidx)) best = v.x, bidx = i;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, best, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bidx, o);
    if (ov > best || (ov == best && oi < bidx)) best = ov, bidx = oi;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) sv[warp] = best, si[warp] = bidx;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w)
      if (sv[w] > best || (sv[w] == best && si[w] < bidx)) best = sv[w], bidx = si[w];
    next[req] = bidx == 0x7fffffff ? 0 : bidx;
  }
}

}  // namespace

// Dense projections run on the span/round kernels; Q4D_GEMM_KERNEL=tcgen05 (read once per process) selects the
// tcgen05 kernel of q4_umma.cu instead, which is correct on every shape but, as measured, not yet faster.
static bool g_legacy = true;
static bool use_umma(int N, int K, int epilogue) { return !g_legacy && umma_supported(N, K, epilogue); }

size_t gemm_partial_bytes(int N, int K, int epilogue) {
  const int sms = sm_count_or_default();
  if (use_umma(N, K, epilogue)) return plan_umma(N, K, epilogue, sms).partial_bytes;
  const size_t a = plan_rounds(N, K, 8, epilogue, sms).partial_bytes, b = plan_rounds(N, K, 16, epilogue, sms).partial_bytes;
  return a > b ? a : b;
}

int gemm_counters_needed(int N) { return (N + 15) / 16 + 1; }

int gemm_row_blocks(int N, int K, int n, int epilogue) {
  if (use_umma(N, K, epilogue)) return plan_umma(N, K, epilogue, sm_count_or_default()).tiles * 4;  // one per warp of a tile
  const RoundPlan t = plan_rounds(N, K, n, epilogue, sm_count_or_default());
  return t.ctas * t.parts * kRoundWarps;  // one argmax partial per warp of the grid
}

int gemm_operand_layout(bool grouped, int n) {
  (void)sm_count_or_default();
  if (grouped) return OPERAND_ROWS;
  if (!g_legacy) return OPERAND_BLOCKED;
  // One or two requests: a slice is one or two row copies either way, and plain rows measured faster there
  // (8B-shaped batch 1: 2.76 against 2.84 ms per step); from three requests on one copy per slice wins.
  return n <= 2 ? OPERAND_ROWS : OPERAND_SLICED;
}

cudaError_t gemm_init() {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  int sms = 0;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  // 227 KB is the per-CTA limit for static + dynamic shared memory; leave room for the static part.
  const int big = 227 * 1024 - 1024;
  e = cudaFuncSetAttribute(q4_gemm_kernel<1, 1, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(q4_gemm_kernel<2, 2, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(q4_gemm_kernel<1, 2, 3>, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
  auto big_smem = [&](auto kernel) {
    if (e == cudaSuccess) e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
  };
  big_smem(q4_round_kernel<1, 3, true>), big_smem(q4_round_kernel<1, 3, false>), big_smem(q4_round_kernel<2, 2, true>);
  big_smem(q4_span_kernel<1, 2, true>), big_smem(q4_span_kernel<1, 2, false>), big_smem(q4_span_kernel<2, 2, true>);
  if (e != cudaSuccess) return e;
  if (const char* f = getenv("Q4D_GEMM_KERNEL")) g_legacy = strcmp(f, "tcgen05") != 0;
  g_sm_count = sms;
  return cudaSuccess;
}

cudaError_t launch_q4_gemm(const GemmArgs& a, cudaStream_t s) {
  if (g_sm_count == 0) {
    cudaError_t e = gemm_init();
    if (e != cudaSuccess) return e;
  }
  if (a.n <= 0) return cudaSuccess;
  if (a.N <= 0 || a.K <= 0 || (a.K % 256) || a.n > kMaxBatch) return cudaErrorInvalidValue;
  const bool grouped = a.expert_ids != nullptr;
  if (a.epilogue == EPI_SILU_PACK && ((a.N % 16) || !a.out_xp || (grouped && !a.out_xs))) return cudaErrorInvalidValue;
  if (grouped && (a.K > 2048 || !a.n_touched || a.max_slots < 1)) return cudaErrorInvalidValue;
  if (!grouped && use_umma(a.N, a.K, a.epilogue)) return launch_q4_umma(a, g_sm_count, s);
  if (!grouped) {
    const RoundPlan t = plan_rounds(a.N, a.K, a.n, a.epilogue, g_sm_count);
    RoundParams p;
    p.qw = a.qw, p.scales = a.scales, p.biases = a.biases, p.xp = a.xp, p.xs = a.xs, p.out = a.out;
    p.out_xp = a.out_xp, p.argmax_partial = a.argmax_partial, p.status = a.status;
    p.N = a.N, p.K = a.K, p.n = a.n, p.out_stride = a.out_stride, p.epilogue = a.epilogue;
    p.xp_layout = gemm_operand_layout(false, a.n);
    {  // the SiLU epilogue feeds a dense projection of N / 2 input features in the same layout
      const int k2 = a.N / 2, ks2 = p.xp_layout == OPERAND_SLICED && k2 % 256 == 0 ? operand_slice_features(k2) : k2;
      const bool sl2 = p.xp_layout == OPERAND_SLICED && k2 % 256 == 0;
      p.out_ks = ks2, p.out_row_stride = sl2 ? ks2 + 8 : k2, p.out_slice_stride = sl2 ? 16 * (ks2 + 8) : 0;
    }
    p.T = t.T, p.Tsub = t.Tsub, p.Q = t.Q, p.S = t.S, p.kw = t.kw;
    p.partial = a.partial, p.counters = a.counters;
    if (t.parts > 1 && (!a.partial || !a.counters || t.partial_bytes > a.partial_bytes || t.T > a.counters_len))
      return cudaErrorInvalidValue;
    const int elem = a.epilogue == EPI_F32 ? 4 : 2;
    p.vec_ok = a.out && (reinterpret_cast<uintptr_t>(a.out) % 16 == 0) && ((size_t)a.out_stride * elem % 16 == 0);
    const dim3 grid(t.ctas, t.parts), block(kRoundThreads);
    const bool sliced = p.xp_layout == OPERAND_SLICED;
    if (t.nt == 2 && !sliced) return cudaErrorInvalidValue;  // more than eight requests always come sliced
    if (t.span) {
      if (t.nt == 2) return launch_kernel(q4_span_kernel<2, 2, true>, grid, block, t.span_smem, s, p);
      if (sliced) return launch_kernel(q4_span_kernel<1, 2, true>, grid, block, t.span_smem, s, p);
      return launch_kernel(q4_span_kernel<1, 2, false>, grid, block, t.span_smem, s, p);
    }
    if (t.nt == 2) return launch_kernel(q4_round_kernel<2, 2, true>, grid, block, t.smem, s, p);
    if (sliced) return launch_kernel(q4_round_kernel<1, 3, true>, grid, block, t.smem, s, p);
    return launch_kernel(q4_round_kernel<1, 3, false>, grid, block, t.smem, s, p);
  }
  const Tiling t = choose_tiling(a.N, a.K, a.n, a.epilogue, g_sm_count, grouped);
  GemmParams p;
  p.expert_ids = a.expert_ids, p.n_touched = a.n_touched, p.expert_rows = a.N;
  p.xp_slot_stride = a.xp_slot_stride, p.xs_slot_stride = a.xs_slot_stride;
  p.out_slot_stride = a.out_slot_stride, p.out_xs_slot_stride = a.out_xs_slot_stride;
  p.qw = a.qw, p.scales = a.scales, p.biases = a.biases, p.xp = a.xp, p.xs = a.xs, p.out = a.out;
  p.out_xp = a.out_xp, p.out_xs = a.out_xs, p.argmax_partial = a.argmax_partial;
  p.partial = a.partial, p.counters = a.counters;
  p.N = a.N, p.K = a.K, p.n = a.n, p.out_stride = a.out_stride;
  p.ks = t.qps * 256, p.splits = t.splits, p.epilogue = a.epilogue;
  p.out_ks = a.N / 2 > 0 ? a.N / 2 : 1, p.out_row_stride = a.N / 2, p.out_slice_stride = 0;  // plain rows
  if (t.splits > 1) {
    if (!a.partial || !a.counters || tiling_partial_bytes(t) > a.partial_bytes || t.rowblocks > a.counters_len)
      return cudaErrorInvalidValue;
  }
  const dim3 grid(t.rowblocks, t.splits, grouped ? a.max_slots : 1), block(kThreads);
  switch (t.cfg) {
    case 0:
      return launch_kernel(q4_gemm_kernel<1, 1, 4>, grid, block, smem_bytes<1, 1, 4>(p.ks), s, p);
    case 1:
      return launch_kernel(q4_gemm_kernel<2, 2, 4>, grid, block, smem_bytes<2, 2, 4>(p.ks), s, p);
    default:
      return launch_kernel(q4_gemm_kernel<1, 2, 3>, grid, block, smem_bytes<1, 2, 3>(p.ks), s, p);
  }
}

cudaError_t launch_argmax_finish(const float2* partial, int row_blocks, int n, int32_t* next, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  return launch_kernel(argmax_finish_kernel, dim3(n), dim3(256), 0, s, partial, row_blocks, next);
}

}  // namespace q4d
