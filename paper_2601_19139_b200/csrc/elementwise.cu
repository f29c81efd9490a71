// Small kernels of the decode step: embedding lookup, RMSNorm, greedy argmax,
// and the two parity exports (dequantised weights, gathered KV).
#include <math.h>

#include "common.cuh"
#include "kernels.h"

namespace q4d {

namespace {

__device__ __forceinline__ float dequant(const uint32_t* qrow, const uint16_t* srow, const uint16_t* brow, int k) {
  const uint32_t code = (qrow[k >> 3] >> (4 * (k & 7))) & 0xFu;
  return __fmaf_rn(bf16_to_f32(srow[k >> 6]), (float)code, bf16_to_f32(brow[k >> 6]));
}

// x[r][k] = bf16(w[tok_r][k]); token ids outside the vocabulary are clamped.
__global__ void embed_kernel(const uint32_t* q, const uint16_t* scales, const uint16_t* biases, int vocab, int H,
                             const int32_t* tokens, uint16_t* x) {
  grid_dependency_wait();
  const int r = blockIdx.x;
  int tok = tokens[r];
  tok = tok < 0 ? 0 : (tok >= vocab ? vocab - 1 : tok);
  const uint32_t* qrow = q + (size_t)tok * (H >> 3);
  const uint16_t* srow = scales + (size_t)tok * (H >> 6);
  const uint16_t* brow = biases + (size_t)tok * (H >> 6);
  for (int k = threadIdx.x; k < H; k += blockDim.x) x[(size_t)r * H + k] = f32_to_bf16(dequant(qrow, srow, brow, k));
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

// y = bf16(x / sqrt(mean(x^2) + eps) * w); one CTA per request row.
__global__ void __launch_bounds__(256) rmsnorm_kernel(const uint16_t* x, const uint16_t* w, float eps, int H,
                                                       uint16_t* y) {
  __shared__ float red[8];
  grid_dependency_wait();
  const uint16_t* xr = x + (size_t)blockIdx.x * H;
  uint16_t* yr = y + (size_t)blockIdx.x * H;
  float ss = 0.0f;
  for (int i = threadIdx.x * 2; i < H; i += blockDim.x * 2) {
    const uint32_t v = *reinterpret_cast<const uint32_t*>(xr + i);
    const float a = bf16_lo(v), b = bf16_hi(v);
    ss = fmaf(a, a, ss);
    ss = fmaf(b, b, ss);
  }
  ss = block_sum(ss, red);
  const float inv = 1.0f / sqrtf(ss / (float)H + eps);
  for (int i = threadIdx.x * 2; i < H; i += blockDim.x * 2) {
    const uint32_t v = *reinterpret_cast<const uint32_t*>(xr + i);
    const uint32_t ww = *reinterpret_cast<const uint32_t*>(w + i);
    *reinterpret_cast<uint32_t*>(yr + i) = pack_bf16x2(bf16_lo(v) * inv * bf16_lo(ww), bf16_hi(v) * inv * bf16_hi(ww));
  }
}

// next[r] = index of the largest logit, the lowest index among equals.
__global__ void __launch_bounds__(1024) argmax_kernel(const float* logits, int vocab, int32_t* next) {
  __shared__ float sv[32];
  __shared__ int si[32];
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
  embed_kernel<<<n, 256, 0, s>>>(q, scales, biases, vocab, H, tokens, x);
  return cudaGetLastError();
}

cudaError_t launch_rmsnorm(const uint16_t* x, const uint16_t* w, float eps, int n, int H, uint16_t* y,
                           cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  if (H % 2) return cudaErrorInvalidValue;
  rmsnorm_kernel<<<n, 256, 0, s>>>(x, w, eps, H, y);
  return cudaGetLastError();
}

cudaError_t launch_argmax(const float* logits, int n, int vocab, int32_t* next, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  argmax_kernel<<<n, 1024, 0, s>>>(logits, vocab, next);
  return cudaGetLastError();
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
