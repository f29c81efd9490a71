// Mixture-of-experts routing for the decode step: router logits, softmax, top-k, the list of experts
// touched by the batch, and the weighted combination of the expert outputs into the residual stream.
//
//   z = Wr y (bf16 dense router, fp32 accumulation);  pi = softmax(z) over all experts;
//   the top_k experts by z (lower index wins a tie), weights pi_k, renormalised to sum 1 if asked;
//   x = bf16(x + bf16(sum_k pi_k * bf16(expert_k output)))
//
// The expert projections themselves run as grouped 4-bit GEMMs over the touched-expert list
// (q4_gemm.cu); every touched expert is evaluated for all requests of the batch and the routing
// weights select what is used, so the packed weights of an expert are streamed once per step.
#include <math.h>

#include "common.cuh"
#include "kernels.h"
#include "launch.h"

namespace q4d {

namespace {

constexpr int kMaxExperts = 256;

constexpr int kRouterThreads = 256;
constexpr int kRouterWarps = kRouterThreads / 32;

// CTA (slice, request): the request's row is staged in shared memory and each warp computes the logits of one or
// more experts of the slice, keeping eight 16-byte loads of a router row in flight per lane (the router matrix is
// small, 512 KB for 128 experts of width 2048, so it is spread over many SMs and the loads overlap).  A lane adds
// its chunks lane, lane + 32, ... in ascending order.  The logits go to global memory; the CTA that finishes a
// request's last slice selects its experts, and the CTA that finishes the last request compacts the touched-expert
// flags into a list.
__global__ void __launch_bounds__(kRouterThreads) moe_router_kernel(const MoeRouteArgs p) {
  extern __shared__ __align__(16) unsigned char router_smem[];
  uint4* sy = reinterpret_cast<uint4*>(router_smem);  // the row: H / 8 chunks of 8 bf16
  __shared__ float sz[kMaxExperts];
  __shared__ int s_last;
  __shared__ int s_warp_base[kRouterWarps];
  grid_launch_dependents();
  const int r = blockIdx.y, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunks = p.H >> 3;
  const int per_slice = (p.E + (int)gridDim.x - 1) / (int)gridDim.x;
  const int e_begin = blockIdx.x * per_slice, e_end = min(p.E, e_begin + per_slice);
  grid_dependency_wait();
  {
    const uint4* y = reinterpret_cast<const uint4*>(p.y + (size_t)r * p.H);
    for (int c = threadIdx.x; c < chunks; c += kRouterThreads) sy[c] = y[c];
  }
  __syncthreads();
  for (int e = e_begin + warp; e < e_end; e += kRouterWarps) {
    const uint4* wr = reinterpret_cast<const uint4*>(p.router + (size_t)e * p.H);
    float acc = 0.0f;
    for (int c0 = lane; c0 < chunks; c0 += 32 * 8) {
      uint4 a[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int c = c0 + 32 * i;
        a[i] = c < chunks ? __ldg(wr + c) : make_uint4(0u, 0u, 0u, 0u);
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int c = c0 + 32 * i;
        if (c < chunks) {
          const uint4 b = sy[c];
          const uint32_t aw[4] = {a[i].x, a[i].y, a[i].z, a[i].w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            acc = fmaf(bf16_lo(aw[j]), bf16_lo(bw[j]), acc);
            acc = fmaf(bf16_hi(aw[j]), bf16_hi(bw[j]), acc);
          }
        }
      }
    }
    acc = warp_sum(acc);
    if (lane == 0) p.logits[(size_t)r * p.E + e] = acc;
  }
  // ---- the CTA with the request's last slice selects the experts ----
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    s_last = (atomicAdd(p.slice_counter + r, 1) == (int)gridDim.x - 1);
    if (s_last) p.slice_counter[r] = 0;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  for (int e = threadIdx.x; e < p.E; e += kRouterThreads) sz[e] = __ldcg(p.logits + (size_t)r * p.E + e);
  __syncthreads();
  if (warp == 0) {
    // each lane owns experts lane, lane + 32, ...
    float v[kMaxExperts / 32];
    float m = -INFINITY;
#pragma unroll
    for (int i = 0; i < kMaxExperts / 32; ++i) {
      const int e = lane + 32 * i;
      v[i] = e < p.E ? sz[e] : -INFINITY;
      m = fmaxf(m, v[i]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float Z = 0.0f;
#pragma unroll
    for (int i = 0; i < kMaxExperts / 32; ++i)
      if (lane + 32 * i < p.E) Z += expf(v[i] - m);
    Z = warp_sum(Z);
    float sel_sum = 0.0f, my_w = 0.0f;
    int my_e = 0;
    for (int k = 0; k < p.top_k; ++k) {
      float best = -INFINITY;
      int bidx = 0x7fffffff;
#pragma unroll
      for (int i = 0; i < kMaxExperts / 32; ++i) {
        const int e = lane + 32 * i;
        if (v[i] > best || (v[i] == best && v[i] != -INFINITY && e < bidx)) best = v[i], bidx = e;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bidx, o);
        if (ov > best || (ov == best && oi < bidx)) best = ov, bidx = oi;
      }
      const float wk = expf(best - m) / Z;
      sel_sum += wk;
      if (lane == k) my_e = bidx, my_w = wk;
      if ((bidx & 31) == lane) {  // remove the winner from its owner's candidates
#pragma unroll
        for (int i = 0; i < kMaxExperts / 32; ++i)
          if (i == (bidx >> 5)) v[i] = -INFINITY;
      }
    }
    if (lane < p.top_k) {
      p.idx[r * p.top_k + lane] = my_e;
      p.wgt[r * p.top_k + lane] = p.norm ? my_w / sel_sum : my_w;
      p.flags[my_e] = 1;
    }
  }
  // ---- the last CTA builds the list of touched experts, in ascending expert order ----
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = (atomicAdd(p.counter, 1) == (int)gridDim.y - 1);
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const int e = threadIdx.x;
  const int f = (e < p.E) ? __ldcg(p.flags + e) : 0;
  const unsigned ball = __ballot_sync(0xffffffffu, f != 0);
  if (lane == 0) s_warp_base[warp] = __popc(ball);
  __syncthreads();
  int base = 0;
  for (int w = 0; w < warp; ++w) base += s_warp_base[w];
  if (f) {
    const int pos = base + __popc(ball & ((1u << lane) - 1u));
    p.expert_ids[pos] = e;
    p.slot_of[e] = pos;
  }
  if (e < p.E) p.flags[e] = 0;
  if (threadIdx.x == 0) {
    int tot = 0;
    for (int w = 0; w < kMaxExperts / 32; ++w) tot += s_warp_base[w];
    *p.n_touched = tot;
    *p.counter = 0;
    if (p.touched_total) *p.touched_total += tot;  // one CTA per launch, launches of a step are stream-ordered
  }
}

// x[r] = bf16(x[r] + bf16(sum_k wgt[r][k] * o[slot_of[idx[r][k]]][r])); a thread takes 8 consecutive elements.
__global__ void __launch_bounds__(256) moe_combine_kernel(const MoeCombineArgs p) {
  grid_launch_dependents();
  grid_dependency_wait();
  const int r = blockIdx.y;
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= (p.H >> 3)) return;
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  for (int k = 0; k < p.top_k; ++k) {
    const int slot = p.slot_of[p.idx[r * p.top_k + k]];
    const float w = p.wgt[r * p.top_k + k];
    const uint4 v = *reinterpret_cast<const uint4*>(p.o + ((size_t)slot * 16 + r) * p.H + c * 8);
    const uint32_t vw[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      acc[2 * i] = fmaf(w, bf16_lo(vw[i]), acc[2 * i]);
      acc[2 * i + 1] = fmaf(w, bf16_hi(vw[i]), acc[2 * i + 1]);
    }
  }
  uint16_t* xr = p.x + (size_t)r * p.H + c * 8;
  const uint4 xv = *reinterpret_cast<const uint4*>(xr);
  const uint32_t xw[4] = {xv.x, xv.y, xv.z, xv.w};
  uint32_t ow[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float d0 = bf16_to_f32(f32_to_bf16(acc[2 * i])), d1 = bf16_to_f32(f32_to_bf16(acc[2 * i + 1]));
    ow[i] = pack_bf16x2(bf16_lo(xw[i]) + d0, bf16_hi(xw[i]) + d1);
  }
  *reinterpret_cast<uint4*>(xr) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
}

}  // namespace

cudaError_t launch_moe_router(const MoeRouteArgs& a, int n, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  if (a.E < 1 || a.E > kMaxExperts || a.top_k < 1 || a.top_k > 32 || a.top_k > a.E || a.H % 8) return cudaErrorInvalidValue;
  if ((size_t)a.H * 2 > 48 * 1024 || !a.logits || !a.slice_counter) return cudaErrorInvalidValue;
  const int slices = (a.E + kRouterWarps - 1) / kRouterWarps;  // one expert per warp while that gives at most 32 slices
  return launch_kernel(moe_router_kernel, dim3(slices < 32 ? slices : 32, n), dim3(kRouterThreads), (size_t)a.H * 2, s, a);
}

cudaError_t launch_moe_combine(const MoeCombineArgs& a, int n, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  const int chunks = a.H >> 3;
  return launch_kernel(moe_combine_kernel, dim3((chunks + 255) / 256, n), dim3(256), 0, s, a);
}

}  // namespace q4d
