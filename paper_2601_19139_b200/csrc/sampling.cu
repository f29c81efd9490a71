// Seeded temperature / top-k / top-p sampling of the next token from fp32 logits (GenerateToken beyond greedy).
//
// Definition (per request; l = logits, T = temperature > 0, V = vocabulary):
//   w_j    = rint(2^40 * exp((l_j - max l) / T))                     integer weights: sums are exact in any order
//   top-k  : keep { j : l_j >= the k-th largest logit }              (k <= 0 or k >= V: keep all; ties at the cut stay)
//   top-p  : with W_k the kept weight, keep { j : l_j >= c } for the largest value c whose set weighs >= top_p * W_k
//   draw   : W = weight of the kept set, t = floor(u * W) for the given u in [0, 1); walk the kept tokens by
//            descending logit, ascending index among equal logits, and take the first whose running weight exceeds t.
// T <= 0 selects the greedy token (largest logit, lowest index among equals).
//
// One CTA per request.  Nothing is sorted: the k-th largest logit, the top-p cut and the drawn token are each found
// by a radix descent over the order-preserving 32-bit image of the logits (four passes of 256-bin histograms of
// counts and weights, private to each warp, lanes that meet in a bin added up before the bin is touched), and the
// position among equal logits by one pass over contiguous index ranges.  Once a cut leaves at most 4096 tokens they
// are gathered into shared memory and the remaining steps run on that list instead of the vocabulary.
#include <math.h>

#include "common.cuh"
#include "kernels.h"
#include "launch.h"

namespace q4d {

namespace {

constexpr int kSampleThreads = 1024;
constexpr int kSampleList = 4096;  // candidates kept in shared memory once the cut leaves no more than this many

// larger float <=> larger key
__device__ __forceinline__ uint32_t order_key(float l) {
  const uint32_t u = __float_as_uint(l);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct Descent {
  uint32_t key;               // the value at which the running total first reaches the target
  unsigned long long w_gt;    // weight of the elements with larger keys (within the restriction)
  unsigned long long w_eq;    // weight of the elements with this key
  uint32_t c_gt, c_eq;        // the same as counts
};

__global__ void __launch_bounds__(kSampleThreads) sample_kernel(const SampleArgs a) {
  extern __shared__ __align__(16) unsigned char dyn_smem[];  // per-warp histograms: counts then weights
  __shared__ unsigned long long s_mass[256];
  __shared__ uint32_t s_cnt[256];
  __shared__ float s_redf[32];
  __shared__ int s_redi[32];
  __shared__ Descent s_d;
  __shared__ uint32_t s_scan[kSampleThreads / 32];
  __shared__ int s_pick, s_count;

  grid_launch_dependents();
  grid_dependency_wait();

  const int r = blockIdx.x, V = a.vocab, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* row = a.logits + (size_t)r * V;
  const float T = a.temperature[r];

  // ---- largest logit and its first index ----
  float best = -INFINITY;
  int bidx = 0x7fffffff;
  for (int j = tid; j < V; j += kSampleThreads) {
    const float v = row[j];
    if (v > best || (v == best && j < bidx)) best = v, bidx = j;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, best, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bidx, o);
    if (ov > best || (ov == best && oi < bidx)) best = ov, bidx = oi;
  }
  if (lane == 0) s_redf[warp] = best, s_redi[warp] = bidx;
  __syncthreads();
  best = s_redf[0], bidx = s_redi[0];
  for (int w = 1; w < kSampleThreads / 32; ++w)
    if (s_redf[w] > best || (s_redf[w] == best && s_redi[w] < bidx)) best = s_redf[w], bidx = s_redi[w];
  __syncthreads();
  if (!(T > 0.0f)) {
    if (tid == 0) a.next[r] = bidx == 0x7fffffff ? 0 : bidx;
    return;
  }
  const float m = best, inv_t = 1.0f / T;
  auto weight = [&](float l) -> unsigned long long {
    return (unsigned long long)__float2ull_rn(expf((l - m) * inv_t) * 1099511627776.0f);  // 2^40
  };

  // Radix descent: among the elements with key >= floor_key, in descending key order, the key at which the running
  // total (of counts if by_count, else of weights) first reaches target (target >= 1, and at most the total).
  // Histograms are private to a warp (no contention between warps: the leading digits of the keys are shared by most
  // of the vocabulary) and the lanes of a warp that hit the same bin are added up first, so a bin sees one update
  // per warp and step.
  uint32_t* w_cnt = reinterpret_cast<uint32_t*>(dyn_smem) + warp * 256;                               // [32 warps][256]
  unsigned long long* w_mass = reinterpret_cast<unsigned long long*>(dyn_smem + 32 * 256 * 4) + warp * 256;
  // candidate list (shared memory): the tokens with key >= the current cut, once there are few enough of them
  int* c_idx = reinterpret_cast<int*>(dyn_smem + 32 * 256 * 12);
  float* c_l = reinterpret_cast<float*>(dyn_smem + 32 * 256 * 12 + kSampleList * 4);
  bool use_list = false;
  int M = 0;
  auto descend = [&](bool by_count, unsigned long long target, uint32_t floor_key) {
    const int count = use_list ? M : V;
    const float* src = use_list ? c_l : row;
    uint32_t prefix = 0;
    unsigned long long w_gt = 0;
    uint32_t c_gt = 0;
    for (int shift = 24; shift >= 0; shift -= 8) {
      for (int b = lane; b < 256; b += 32) w_cnt[b] = 0u, w_mass[b] = 0ull;
      __syncwarp();
      const uint32_t hi_mask = shift == 24 ? 0u : (0xffffffffu << (shift + 8));
      constexpr int kBatch = 16;  // loads in flight per thread: the logits come from L2, one load at a time is all latency
      for (int j0 = 0; j0 < count; j0 += kBatch * kSampleThreads) {
        float lv[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
          const int j = j0 + u * kSampleThreads + tid;
          lv[u] = j < count ? src[j] : 0.0f;
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
          const int j = j0 + u * kSampleThreads + tid;
          const float l = lv[u];
          const uint32_t k = order_key(l);
          const bool in = j < count && k >= floor_key && (k & hi_mask) == prefix;
          const uint32_t active = __ballot_sync(0xffffffffu, in);
          if (active == 0u) continue;
          if (in && by_count) {
            atomicAdd(&w_cnt[(k >> shift) & 255u], 1u);  // counts only: the hardware merges a warp's hits on one bin
          } else if (in) {
            const uint32_t b = (k >> shift) & 255u;
            const uint32_t peers = __match_any_sync(active, b);
            const unsigned long long w = weight(l);
            // the peers' weights (below 2^41 each) in two halves that 32 lanes cannot overflow
            const uint32_t lo = __reduce_add_sync(peers, (uint32_t)(w & 0xfffffu));
            const uint32_t hi = __reduce_add_sync(peers, (uint32_t)(w >> 20));
            if ((int)(__ffs(peers) - 1) == lane) {
              atomicAdd(&w_cnt[b], (uint32_t)__popc(peers));
              atomicAdd(&w_mass[b], ((unsigned long long)hi << 20) + lo);
            }
          }
        }
      }
      __syncthreads();
      if (tid < 256) {  // add the warps' histograms up
        uint32_t c = 0;
        unsigned long long mm = 0;
        const uint32_t* ac = reinterpret_cast<const uint32_t*>(dyn_smem) + tid;
        const unsigned long long* am = reinterpret_cast<const unsigned long long*>(dyn_smem + 32 * 256 * 4) + tid;
        for (int w2 = 0; w2 < kSampleThreads / 32; ++w2) c += ac[w2 * 256], mm += am[w2 * 256];
        s_cnt[tid] = c, s_mass[tid] = mm;
      }
      __syncthreads();
      if (tid == 0) {
        int b = 255;
        for (; b > 0; --b) {
          const unsigned long long have = by_count ? (unsigned long long)(c_gt + s_cnt[b]) : w_gt + s_mass[b];
          if (have >= target) break;
          w_gt += s_mass[b], c_gt += s_cnt[b];
        }
        s_d.key = prefix | ((uint32_t)b << shift);
        s_d.w_gt = w_gt, s_d.c_gt = c_gt, s_d.w_eq = s_mass[b], s_d.c_eq = s_cnt[b];
      }
      __syncthreads();
      prefix = s_d.key, w_gt = s_d.w_gt, c_gt = s_d.c_gt;
      __syncthreads();
    }
  };
  // weight of the elements with key >= floor_key (every thread returns the block's total)
  auto weight_at_least = [&](uint32_t floor_key) -> unsigned long long {
    unsigned long long part = 0;
    const int count = use_list ? M : V;
    const float* src = use_list ? c_l : row;
    for (int j = tid; j < count; j += kSampleThreads) {
      const float l = src[j];
      if (order_key(l) >= floor_key) part += weight(l);
    }
    if (tid == 0) s_mass[0] = 0ull;
    __syncthreads();
    const uint32_t lo = __reduce_add_sync(0xffffffffu, (uint32_t)(part & 0xfffffu));
    const unsigned long long hi = part >> 20;  // up to 2^29 per thread: add the halves as 64-bit values across the warp
    unsigned long long hs = hi;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) hs += __shfl_xor_sync(0xffffffffu, hs, o);
    if (lane == 0) atomicAdd(&s_mass[0], (hs << 20) + lo);
    __syncthreads();
    const unsigned long long tot = s_mass[0];
    __syncthreads();
    return tot;
  };

  // Gathers the tokens with key >= floor_key (at most kSampleList of them: the caller has counted) into the list;
  // everything after works on the list.
  auto gather = [&](uint32_t floor_key) {
    if (tid == 0) s_count = 0;
    __syncthreads();
    for (int j = tid; j < V; j += kSampleThreads) {
      const float l = row[j];
      if (order_key(l) >= floor_key) {
        const int pos = atomicAdd(&s_count, 1);
        if (pos < kSampleList) c_idx[pos] = j, c_l[pos] = l;
      }
    }
    __syncthreads();
    M = min(s_count, kSampleList);
    use_list = true;
    __syncthreads();
  };

  // ---- top-k cut and the weight it keeps ----
  uint32_t floor_key = 0u;
  unsigned long long W = 0;
  const int k = a.top_k[r];
  if (k > 0 && k < V) {
    descend(true, (unsigned long long)k, 0u);  // by counts alone: no exponentials in these passes
    floor_key = s_d.key;
    if (s_d.c_gt + s_d.c_eq <= (uint32_t)kSampleList) gather(floor_key);
  }
  W = weight_at_least(floor_key);
  // ---- top-p cut ----
  const float p = a.top_p[r];
  if (p < 1.0f) {
    unsigned long long target = (unsigned long long)ceil((double)p * (double)W);
    if (target < 1ull) target = 1ull;
    if (target > W) target = W;
    descend(false, target, floor_key);
    floor_key = s_d.key;
    W = s_d.w_gt + s_d.w_eq;
    if (!use_list && s_d.c_gt + s_d.c_eq <= (uint32_t)kSampleList) gather(floor_key);
  }
  // ---- the draw ----
  unsigned long long t = (unsigned long long)((double)a.u[r] * (double)W);
  if (t >= W) t = W - 1ull;
  descend(false, t + 1ull, floor_key);
  const Descent d = s_d;
  // position among the tokens of this logit, in index order (they weigh the same)
  const unsigned long long each = d.c_eq ? d.w_eq / d.c_eq : 1ull;
  unsigned long long rho = t + 1ull - d.w_gt;  // 1 .. w_eq
  uint32_t want = each ? (uint32_t)((rho + each - 1ull) / each) : 1u;
  if (want < 1u) want = 1u;
  if (want > d.c_eq) want = d.c_eq;
  if (tid == 0) s_pick = bidx;  // never left unset
  __syncthreads();
  if (use_list) {
    // the list is in no particular order: an entry of this logit is the wanted one when want - 1 others precede it
    for (int i = tid; i < M; i += kSampleThreads) {
      if (order_key(c_l[i]) != d.key) continue;
      uint32_t before = 0;
      for (int o = 0; o < M; ++o) before += order_key(c_l[o]) == d.key && c_idx[o] < c_idx[i];
      if (before == want - 1u) s_pick = c_idx[i];
    }
  } else {
    // contiguous index ranges: thread tid owns [tid * L, (tid + 1) * L)
    const int L = (V + kSampleThreads - 1) / kSampleThreads;
    const int j0 = tid * L, j1 = min(V, j0 + L);
    uint32_t mine = 0;
    for (int j = j0; j < j1; ++j) mine += order_key(row[j]) == d.key;
    // exclusive prefix over the threads
    uint32_t incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) s_scan[warp] = incl;
    __syncthreads();
    uint32_t base = 0;
    for (int w = 0; w < warp; ++w) base += s_scan[w];
    const uint32_t before = base + incl - mine;
    if (mine && before < want && want <= before + mine) {
      uint32_t seen = before;
      for (int j = j0; j < j1; ++j)
        if (order_key(row[j]) == d.key && ++seen == want) s_pick = j;
    }
  }
  __syncthreads();
  if (tid == 0) a.next[r] = s_pick;
}

}  // namespace

cudaError_t launch_sample(const SampleArgs& a, int n, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  if (n > kMaxBatch || a.vocab < 1 || !a.logits || !a.next) return cudaErrorInvalidValue;
  static bool attr_set = false;
  constexpr int kDyn = 32 * 256 * (4 + 8) + kSampleList * 8;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(sample_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDyn);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  return launch_kernel(sample_kernel, dim3(n), dim3(kSampleThreads), kDyn, s, a);
}

}  // namespace q4d
