// Small kernels of the decode step: embedding lookup, RMSNorm, greedy argmax,
// and the two parity exports (dequantised weights, gathered KV).
#include <math.h>

#include "common.cuh"
#include "kernels.h"
#include "launch.h"

namespace q4d {

namespace {

__device__ __forceinline__ float dequant(const uint32_t* qrow, const uint16_t* srow, const uint16_t* brow, int k) {
  const uint32_t code = (qrow[k >> 3] >> (4 * (k & 7))) & 0xFu;
  return __fmaf_rn(bf16_to_f32(srow[k >> 6]), (float)code, bf16_to_f32(brow[k >> 6]));
}

// x[r][k] = bf16(w[tok_r][k]); token ids outside the vocabulary are clamped.
__global__ void embed_kernel(const uint32_t* q, const uint16_t* scales, const uint16_t* biases, int vocab, int H,
                             const int32_t* tokens, uint16_t* x) {
  grid_launch_dependents();
  grid_dependency_wait();
  const int r = blockIdx.x;
  int tok = tokens[r];
  tok = tok < 0 ? 0 : (tok >= vocab ? vocab - 1 : tok);
  const uint32_t* qrow = q + (size_t)tok * (H >> 3);
  const uint16_t* srow = scales + (size_t)tok * (H >> 6);
  const uint16_t* brow = biases + (size_t)tok * (H >> 6);
  // one packed word (8 elements) per thread and pass: its three loads go out together, one 16-byte store
  for (int w8 = threadIdx.x; w8 < (H >> 3); w8 += blockDim.x) {
    const uint32_t word = qrow[w8];
    const float sc = bf16_to_f32(srow[w8 >> 3]), bi = bf16_to_f32(brow[w8 >> 3]);
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j)
      o[j] = pack_bf16x2(__fmaf_rn(sc, (float)((word >> (8 * j)) & 0xFu), bi), __fmaf_rn(sc, (float)((word >> (8 * j + 4)) & 0xFu), bi));
    *reinterpret_cast<uint4*>(x + (size_t)r * H + w8 * 8) = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

__device__ __forceinline__ float block_sum(float v, float* red) {
  v = warp_sum(v);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float tot = 0.0f;
  for (int i = 0; i < nw; ++i) tot += red[i];  // same order in every thread
  __syncthreads();
  return tot;
}

// y = bf16(x / sqrt(mean(x^2) + eps) * w); one CTA per request row.  The row is held in registers (up to 8 chunks
// of 8 elements per thread: H <= 16384).  Writes y in plain layout and/or as the next GEMM's operand.
__global__ void __launch_bounds__(256) rmsnorm_kernel(const uint16_t* x, const uint16_t* w, float eps, int H,
                                                       uint16_t* y, uint16_t* yp, float* ys, int layout) {
  __shared__ float red[8];
  grid_launch_dependents();
  const int r = blockIdx.x, nch = H >> 3;
  uint4 wv[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {  // norm weights do not depend on the preceding kernel
    const int c = threadIdx.x + i * 256;
    wv[i] = c < nch ? *reinterpret_cast<const uint4*>(w + c * 8) : make_uint4(0u, 0u, 0u, 0u);
  }
  grid_dependency_wait();
  uint4 xv[8];
  float ss = 0.0f;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int c = threadIdx.x + i * 256;
    xv[i] = c < nch ? *reinterpret_cast<const uint4*>(x + (size_t)r * H + c * 8) : make_uint4(0u, 0u, 0u, 0u);
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const uint32_t e[4] = {xv[i].x, xv[i].y, xv[i].z, xv[i].w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float a = bf16_lo(e[j]), b = bf16_hi(e[j]);
      ss = fmaf(a, a, ss);
      ss = fmaf(b, b, ss);
    }
  }
  ss = block_sum(ss, red);
  const float inv = 1.0f / sqrtf(ss / (float)H + eps);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int c = threadIdx.x + i * 256;
    if (i * 256 >= nch) break;  // uniform across the CTA
    const uint32_t e[4] = {xv[i].x, xv[i].y, xv[i].z, xv[i].w}, ww[4] = {wv[i].x, wv[i].y, wv[i].z, wv[i].w};
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j)
      o[j] = pack_bf16x2(bf16_lo(e[j]) * inv * bf16_lo(ww[j]), bf16_hi(e[j]) * inv * bf16_hi(ww[j]));
    const uint4 v = make_uint4(o[0], o[1], o[2], o[3]);
    const float gsum = group_sum_8lanes(chunk_sum(v));  // lanes of an aligned group of 8 hold one 64-element group
    if (c < nch) {
      if (y) *reinterpret_cast<uint4*>(y + (size_t)r * H + c * 8) = v;
      if (yp) {
        *reinterpret_cast<uint4*>(yp + operand_chunk_offset(layout, H, r, c)) = permute_chunk(v);
        if ((c & 7) == 0) ys[(size_t)(c >> 3) * 16 + r] = gsum;
      }
    }
  }
}

// Plain activations -> the GEMM's fragment-ordered operand (optionally h = bf16(silu(gate) * up) first).
// One thread per chunk of 8 elements; x is [n][x_stride] (with the SiLU prologue: gate at [0, K), up at [K, 2K)).
__global__ void __launch_bounds__(256) pack_operand_kernel(const uint16_t* x, int x_stride, int K, int n, int prologue,
                                                            uint16_t* xp, float* xs, int layout) {
  grid_launch_dependents();
  grid_dependency_wait();
  const int cpr = K >> 3;
  const int c = blockIdx.x * blockDim.x + threadIdx.x;  // cpr is a multiple of 32: warps never straddle rows
  const int r = c / cpr, kc = c - r * cpr;
  uint4 v = make_uint4(0u, 0u, 0u, 0u);
  if (r < n) {
    const uint16_t* src = x + (size_t)r * x_stride + kc * 8;
    v = *reinterpret_cast<const uint4*>(src);
    if (prologue == PRO_SILU_MUL) {
      const uint4 u = *reinterpret_cast<const uint4*>(src + K);
      const uint32_t gw[4] = {v.x, v.y, v.z, v.w}, uw[4] = {u.x, u.y, u.z, u.w};
      uint32_t hw[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float g0 = bf16_lo(gw[i]), g1 = bf16_hi(gw[i]);
        hw[i] = pack_bf16x2((g0 / (1.0f + expf(-g0))) * bf16_lo(uw[i]), (g1 / (1.0f + expf(-g1))) * bf16_hi(uw[i]));
      }
      v = make_uint4(hw[0], hw[1], hw[2], hw[3]);
    }
  }
  const float gsum = group_sum_8lanes(chunk_sum(v));
  if (r < n) {
    *reinterpret_cast<uint4*>(xp + operand_chunk_offset(layout, K, r, kc)) = permute_chunk(v);
    if ((kc & 7) == 0) xs[(size_t)(kc >> 3) * 16 + r] = gsum;
  }
}

// next[r] = index of the largest logit, the lowest index among equals.
__global__ void __launch_bounds__(1024) argmax_kernel(const float* logits, int vocab, int32_t* next) {
  __shared__ float sv[32];
  __shared__ int si[32];
  grid_launch_dependents();
  grid_dependency_wait();
  const float* row = logits + (size_t)blockIdx.x * vocab;
  float best = -INFINITY;
  int idx = 0x7fffffff;
  for (int j = threadIdx.x; j < vocab; j += blockDim.x) {
    const float v = row[j];
    if (v > best || (v == best && j < idx)) best = v, idx = j;
  }
  auto better = [](float v, int i, float bv, int bi) { return v > bv || (v == bv && i < bi); };
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, best, o);
    const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
    if (better(ov, oi, best, idx)) best = ov, idx = oi;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) sv[warp] = best, si[warp] = idx;
  __syncthreads();
  if (warp == 0) {
    const int nw = blockDim.x >> 5;
    best = lane < nw ? sv[lane] : -INFINITY;
    idx = lane < nw ? si[lane] : 0x7fffffff;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, best, o);
      const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
      if (better(ov, oi, best, idx)) best = ov, idx = oi;
    }
    if (lane == 0) next[blockIdx.x] = idx == 0x7fffffff ? 0 : idx;
  }
}

__global__ void dequant_kernel(const uint32_t* q, const uint16_t* scales, const uint16_t* biases, int N, int K,
                               float* out) {
  const size_t total = (size_t)N * K;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const size_t j = i / K;
    const int k = (int)(i - j * K);
    out[i] = dequant(q + j * (K >> 3), scales + j * (K >> 6), biases + j * (K >> 6), k);
  }
}

// k_out, v_out [len][nkv][128] from one layer of the pool through a block table.
__global__ void kv_gather_kernel(const uint16_t* kpool, const uint16_t* vpool, int nkv, const int32_t* block_table,
                                 int len, uint16_t* k_out, uint16_t* v_out) {
  const int tok = blockIdx.x, h = blockIdx.y, d = threadIdx.x;
  if (tok >= len) return;
  const int blk = block_table[tok / kBlockSize], slot = tok % kBlockSize;
  const size_t src = (((size_t)blk * nkv + h) * kBlockSize + slot) * kHeadDim + d;
  const size_t dst = ((size_t)tok * nkv + h) * kHeadDim + d;
  k_out[dst] = kpool[src];
  v_out[dst] = vpool[src];
}

}  // namespace

cudaError_t launch_embed(const uint32_t* q, const uint16_t* scales, const uint16_t* biases, int vocab, int H,
                         const int32_t* tokens, int n, uint16_t* x, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  return launch_kernel(embed_kernel, dim3(n), dim3(256), 0, s, q, scales, biases, vocab, H, tokens, x);
}

cudaError_t launch_rmsnorm(const uint16_t* x, const uint16_t* w, float eps, int n, int H, uint16_t* y,
                           uint16_t* yp, float* ys, int layout, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  if (H % 64 || H > 16384 || (yp && !ys)) return cudaErrorInvalidValue;
  return launch_kernel(rmsnorm_kernel, dim3(n), dim3(256), 0, s, x, w, eps, H, y, yp, ys, layout);
}

cudaError_t launch_pack_operand(const uint16_t* x, int x_stride, int K, int n, int prologue, uint16_t* xp, float* xs,
                                int layout, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  if (K % 256 || x_stride % 8) return cudaErrorInvalidValue;
  const int chunks = n * (K >> 3);
  return launch_kernel(pack_operand_kernel, dim3((chunks + 255) / 256), dim3(256), 0, s, x, x_stride, K, n, prologue,
                       xp, xs, layout);
}

cudaError_t launch_argmax(const float* logits, int n, int vocab, int32_t* next, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  return launch_kernel(argmax_kernel, dim3(n), dim3(1024), 0, s, logits, vocab, next);
}

cudaError_t launch_dequant(const uint32_t* q, const uint16_t* scales, const uint16_t* biases, int N, int K,
                           float* out, cudaStream_t s) {
  if (N <= 0 || K <= 0) return cudaSuccess;
  const size_t total = (size_t)N * K;
  const int blocks = (int)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
  dequant_kernel<<<blocks, 256, 0, s>>>(q, scales, biases, N, K, out);
  return cudaGetLastError();
}

cudaError_t launch_kv_gather(const uint16_t* kpool, const uint16_t* vpool, int nkv, const int32_t* block_table,
                             int len, uint16_t* k_out, uint16_t* v_out, cudaStream_t s) {
  if (len <= 0) return cudaSuccess;
  kv_gather_kernel<<<dim3(len, nkv), kHeadDim, 0, s>>>(kpool, vpool, nkv, block_table, len, k_out, v_out);
  return cudaGetLastError();
}

}  // namespace q4d
