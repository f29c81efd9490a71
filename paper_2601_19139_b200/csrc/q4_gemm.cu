// Fused dequantise-and-multiply of 4-bit affine group-64 weights against bf16
// activations for 1..16 requests (the QKV, O, gate/up, down and LM-head
// projections of the decode step).
//
// y[r][j] = sum_k (scale[j][k/64] * q[j][k] + bias[j][k/64]) * x[r][k]
//         = sum_g scale[j][g] * (sum_{k in g} q[j][k] x[r][k]) + bias[j][g] * (sum_{k in g} x[r][k])
//
// The inner sums run on the tensor cores with the 4-bit codes converted to
// exact bf16 integers (products code * x are exact, accumulation is fp32), so
// no dequantised weight is ever rounded to bf16; scale and bias are applied to
// the fp32 group sums.
//
// Layout of the work.  A CTA of 8 warps owns 8*16*MT consecutive output rows
// and one K-slice; each warp owns 16*MT rows and streams their packed codes,
// scales and biases through a private cp.async ring in shared memory, 256 input
// features (one "quad" of four groups, 128 B per row) per stage.  The
// activation slice is staged once per CTA in shared memory in the element
// order the MMA fragments need.  Split-K partial sums go to a scratch buffer;
// the last CTA to arrive for a row block adds them in split order (so the
// result does not depend on arrival order) and applies the epilogue.
#include "common.cuh"
#include "kernels.h"

namespace q4d {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = 8;
constexpr int kRowStride = 160;  // bytes per row per stage in smem: 128 data + 32 pad (conflict-free 8-byte reads)
constexpr int kSbBytes = 16;     // per row per stage: 4 scales + 4 biases (bf16)
constexpr int kStages = 3;
constexpr int kMaxQuadsPerSlice = 8;  // K-slice <= 2048

struct GemmParams {
  const uint32_t* qw;
  const uint16_t* scales;
  const uint16_t* biases;
  const uint16_t* x;
  void* out;
  float* partial;
  int* counters;
  int N, K, n, x_stride, out_stride;
  int ks;      // nominal K-slice (multiple of 256)
  int splits;  // gridDim.y
  int prologue, epilogue;
};

// Four bf16x2 registers {code j, code j+4}, j = 0..3, as exact integers, from one packed word.
__device__ __forceinline__ void unpack_word(uint32_t w, uint32_t (&p)[4]) {
  constexpr uint32_t kMask = 0x000F000Fu, kMagic = 0x43004300u;  // bf16 128.0 in both halves
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    uint32_t v = ((w >> (4 * j)) & kMask) | kMagic;  // 128 + code, exact
    asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(p[j]) : "r"(v), "r"(kMagic));
  }
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

template <int MT, int NT>
__global__ void __launch_bounds__(kThreads, (MT == 1 && NT == 1) ? 2 : 1) q4_gemm_kernel(const GemmParams p) {
  constexpr int R = 16 * MT;  // rows per warp
  constexpr int NP = 8 * NT;  // padded request count
  constexpr int kStage = R * (kRowStride + kSbBytes);
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ int s_is_last;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int row_block = blockIdx.x * (kWarps * R);
  const int warp_row0 = row_block + warp * R;
  const int k0 = blockIdx.y * p.ks;
  const int kend = min(p.K, k0 + p.ks);
  const int kslice = kend - k0;
  const int nquads = kslice >> 8;
  const int b_stride = p.ks * 2 + 16;  // bytes per request row of the staged activations

  unsigned char* ring = smem + warp * (kStages * kStage);
  unsigned char* sB = smem + kWarps * kStages * kStage;
  float* sX = reinterpret_cast<float*>(sB + NP * b_stride);  // [group][NP]

  auto issue_stage = [&](int qd) {
    unsigned char* stg = ring + (qd % kStages) * kStage;
    const int kq = k0 + qd * 256;
#pragma unroll
    for (int i = 0; i < R / 4; ++i) {
      const int r = i * 4 + (lane >> 3);
      const int grow = min(warp_row0 + r, p.N - 1);
      const unsigned char* src =
          reinterpret_cast<const unsigned char*>(p.qw + (size_t)grow * (p.K >> 3) + (kq >> 3)) + (lane & 7) * 16;
      cp_async16(stg + r * kRowStride + (lane & 7) * 16, src);
    }
    for (int r = lane; r < R; r += 32) {
      const int grow = min(warp_row0 + r, p.N - 1);
      const size_t off = (size_t)grow * (p.K >> 6) + (kq >> 6);
      cp_async8(stg + R * kRowStride + r * kSbBytes, p.scales + off);
      cp_async8(stg + R * kRowStride + r * kSbBytes + 8, p.biases + off);
    }
  };

  // Weights do not depend on the preceding kernel: start streaming them before waiting for it.
#pragma unroll
  for (int s = 0; s < kStages - 1; ++s) {
    if (s < nquads) issue_stage(s);
    cp_async_commit();
  }

  grid_dependency_wait();

  // Stage the activation slice: permute each 8-element chunk to {0,4,1,5,2,6,3,7} so that a lane's
  // 16 elements of a group are its B fragments of the four k-steps, and form the fp32 group sums.
  {
    const int cpr = kslice >> 3;  // 16-byte chunks per request row
    const int total = NP * cpr;   // multiple of 256
    for (int c = threadIdx.x; c < total; c += kThreads) {
      const int r = c / cpr, kc = c - r * cpr;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (r < p.n) {
        const uint16_t* src = p.x + (size_t)r * p.x_stride + k0 + kc * 8;
        v = *reinterpret_cast<const uint4*>(src);
        if (p.prologue == PRO_SILU_MUL) {
          const uint4 u = *reinterpret_cast<const uint4*>(src + p.K);
          uint32_t gw[4] = {v.x, v.y, v.z, v.w}, uw[4] = {u.x, u.y, u.z, u.w}, hw[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float g0 = bf16_lo(gw[i]), g1 = bf16_hi(gw[i]);
            const float h0 = (g0 / (1.0f + expf(-g0))) * bf16_lo(uw[i]);
            const float h1 = (g1 / (1.0f + expf(-g1))) * bf16_hi(uw[i]);
            hw[i] = pack_bf16x2(h0, h1);
          }
          v = make_uint4(hw[0], hw[1], hw[2], hw[3]);
        }
      }
      float sum = ((bf16_lo(v.x) + bf16_hi(v.x)) + (bf16_lo(v.y) + bf16_hi(v.y))) +
                  ((bf16_lo(v.z) + bf16_hi(v.z)) + (bf16_lo(v.w) + bf16_hi(v.w)));
      sum += __shfl_xor_sync(0xffffffffu, sum, 1);
      sum += __shfl_xor_sync(0xffffffffu, sum, 2);
      sum += __shfl_xor_sync(0xffffffffu, sum, 4);
      uint4 o;
      o.x = __byte_perm(v.x, v.z, 0x5410);
      o.y = __byte_perm(v.x, v.z, 0x7632);
      o.z = __byte_perm(v.y, v.w, 0x5410);
      o.w = __byte_perm(v.y, v.w, 0x7632);
      *reinterpret_cast<uint4*>(sB + r * b_stride + kc * 16) = o;
      if ((kc & 7) == 0) sX[(kc >> 3) * NP + r] = sum;
    }
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
    if (qd + kStages - 1 < nquads) issue_stage(qd + kStages - 1);
    cp_async_commit();
    cp_async_wait<kStages - 1>();
    __syncwarp();
    const unsigned char* stg = ring + (qd % kStages) * kStage;

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
        const float s_lo = bf16_at(sc[mt][0], gi), s_hi = bf16_at(sc[mt][1], gi);
        const float b_lo = bf16_at(bi[mt][0], gi), b_hi = bf16_at(bi[mt][1], gi);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          float pc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
          mma_bf16(pc, l0[0], h0[0], l0[1], h0[1], bf[nt][0].x, bf[nt][0].y);
          mma_bf16(pc, l0[2], h0[2], l0[3], h0[3], bf[nt][0].z, bf[nt][0].w);
          mma_bf16(pc, l1[0], h1[0], l1[1], h1[1], bf[nt][1].x, bf[nt][1].y);
          mma_bf16(pc, l1[2], h1[2], l1[3], h1[3], bf[nt][1].z, bf[nt][1].w);
          acc[mt][nt][0] = fmaf(s_lo, pc[0], fmaf(b_lo, xs[nt].x, acc[mt][nt][0]));
          acc[mt][nt][1] = fmaf(s_lo, pc[1], fmaf(b_lo, xs[nt].y, acc[mt][nt][1]));
          acc[mt][nt][2] = fmaf(s_hi, pc[2], fmaf(b_hi, xs[nt].x, acc[mt][nt][2]));
          acc[mt][nt][3] = fmaf(s_hi, pc[3], fmaf(b_hi, xs[nt].y, acc[mt][nt][3]));
        }
      }
    }
    __syncwarp();
  }
  cp_async_wait<0>();

  if (p.splits == 1) {
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int row = warp_row0 + mt * 16 + g + (c >> 1) * 8;
          const int req = nt * 8 + 2 * t + (c & 1);
          if (row < p.N && req < p.n) store_out(p, row, req, acc[mt][nt][c]);
        }
    return;
  }

  // Split-K: publish this CTA's partial sums, then the last CTA of the row block reduces them.
  const int n_pad = gridDim.x * (kWarps * R);
  {
    float* part = p.partial + (size_t)blockIdx.y * n_pad * NP;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int row = warp_row0 + mt * 16 + g + h * 8;
          *reinterpret_cast<float2*>(part + (size_t)row * NP + nt * 8 + 2 * t) =
              make_float2(acc[mt][nt][2 * h], acc[mt][nt][2 * h + 1]);
        }
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const int prev = atomicAdd(p.counters + blockIdx.x, 1);
    s_is_last = (prev == p.splits - 1);
  }
  __syncthreads();
  if (!s_is_last) return;
  __threadfence();
  constexpr int kRows = kWarps * R;
  for (int idx = threadIdx.x; idx < kRows * NP; idx += kThreads) {
    const int req = idx / kRows, row = row_block + (idx - req * kRows);
    if (row >= p.N || req >= p.n) continue;
    float v = 0.0f;
    for (int s = 0; s < p.splits; ++s) v += __ldcg(p.partial + ((size_t)s * n_pad + row) * NP + req);
    store_out(p, row, req, v);
  }
  if (threadIdx.x == 0) p.counters[blockIdx.x] = 0;
}

template <int MT, int NT>
size_t smem_bytes(int ks) {
  return (size_t)kWarps * kStages * (16 * MT) * (kRowStride + kSbBytes) + (size_t)(8 * NT) * (ks * 2 + 16) +
         (size_t)(ks / 64) * (8 * NT) * sizeof(float);
}

struct Tiling {
  int mt, nt, rows_cta, rowblocks, qps, splits;
};

Tiling choose_tiling(int N, int K, int n, int sm_count) {
  Tiling t;
  t.nt = n > 8 ? 2 : 1;
  t.mt = t.nt == 2 ? 2 : 1;
  t.rows_cta = kWarps * 16 * t.mt;
  t.rowblocks = (N + t.rows_cta - 1) / t.rows_cta;
  const int quads = K / 256;
  const int wave = sm_count * ((t.mt == 1 && t.nt == 1) ? 2 : 1);
  int qps = 1;
  for (int c = (quads < kMaxQuadsPerSlice ? quads : kMaxQuadsPerSlice); c >= 1; --c) {
    if (quads % c) continue;
    if ((long long)t.rowblocks * (quads / c) >= wave || c == 1) {
      qps = c;
      break;
    }
  }
  t.qps = qps;
  t.splits = quads / qps;
  return t;
}

int g_sm_count = 0;

}  // namespace

size_t gemm_partial_bytes(int N, int K) {
  int sms = g_sm_count;
  if (sms == 0) {
    if (gemm_init() == cudaSuccess) {
      sms = g_sm_count;
    } else {
      (void)cudaGetLastError();
      sms = 148;  // sizing only: no device in this process
    }
  }
  size_t need = 0;
  for (int n = 8; n <= 16; n += 8) {  // the two tilings: up to 8 requests, 9..16 requests
    const Tiling t = choose_tiling(N, K, n, sms);
    const size_t b = t.splits > 1 ? (size_t)t.splits * t.rowblocks * t.rows_cta * (8 * t.nt) * sizeof(float) : 0;
    if (b > need) need = b;
  }
  return need;
}

int gemm_counters_needed(int N) { return (N + 127) / 128 + 1; }

cudaError_t gemm_init() {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  int sms = 0;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  // 227 KB is the per-CTA limit for static + dynamic shared memory; leave room for the static part.
  const int big = 227 * 1024 - 1024;
  e = cudaFuncSetAttribute(q4_gemm_kernel<1, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, big / 2 - 1024);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(q4_gemm_kernel<2, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
  if (e != cudaSuccess) return e;
  g_sm_count = sms;
  return cudaSuccess;
}

cudaError_t launch_q4_gemm(const GemmArgs& a, cudaStream_t s) {
  if (g_sm_count == 0) {
    cudaError_t e = gemm_init();
    if (e != cudaSuccess) return e;
  }
  if (a.n <= 0) return cudaSuccess;
  if (a.N <= 0 || a.K <= 0 || (a.K % 256) || a.n > kMaxBatch || (a.x_stride % 8)) return cudaErrorInvalidValue;
  const Tiling t = choose_tiling(a.N, a.K, a.n, g_sm_count);
  GemmParams p;
  p.qw = a.qw, p.scales = a.scales, p.biases = a.biases, p.x = a.x, p.out = a.out;
  p.partial = a.partial, p.counters = a.counters;
  p.N = a.N, p.K = a.K, p.n = a.n, p.x_stride = a.x_stride, p.out_stride = a.out_stride;
  p.ks = t.qps * 256, p.splits = t.splits, p.prologue = a.prologue, p.epilogue = a.epilogue;
  if (t.splits > 1) {
    const size_t need = (size_t)t.splits * t.rowblocks * t.rows_cta * (8 * t.nt) * sizeof(float);
    if (!a.partial || !a.counters || need > a.partial_bytes || t.rowblocks > a.counters_len)
      return cudaErrorInvalidValue;
  }
  const dim3 grid(t.rowblocks, t.splits), block(kThreads);
  if (t.mt == 1 && t.nt == 1)
    q4_gemm_kernel<1, 1><<<grid, block, smem_bytes<1, 1>(p.ks), s>>>(p);
  else
    q4_gemm_kernel<2, 2><<<grid, block, smem_bytes<2, 2>(p.ks), s>>>(p);
  return cudaGetLastError();
}

}  // namespace q4d
