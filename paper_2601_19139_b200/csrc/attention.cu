// GQA decode attention over a paged KV pool, split over the KV length with a
// log-sum-exp merge, plus the kernel that prepares q and appends k, v.
//
// For request r, q head a (kv head h = a / G) and cached tokens t = 0..len_r:
//   s_t = q_a . k_t / sqrt(128),  P = softmax(s),  out_a = bf16(sum_t P_t v_t)
//
// Work item = (request, kv head, chunk of consecutive 16-token blocks).  A CTA
// of four warps takes one item; each warp walks its share of the chunk's
// blocks through a private cp.async ring (one stage = the 4 KB K block and the
// 4 KB V block of that kv head), computes scores for the G query heads of the
// kv head with m16n8k16 MMAs (rows = query heads, padded to 16), keeps a
// running (max, sum, accumulator) per head, and multiplies P into V with P
// split into two bf16 terms so the product keeps ~16 bits of P.  The warps'
// states are merged in shared memory and written as one partial result per
// item; a second kernel merges the partial results of a request.
#include <math.h>

#include "common.cuh"
#include "kernels.h"
#include "launch.h"

namespace q4d {

namespace {

constexpr int kAttnThreads = 128;
constexpr int kAttnWarps = 4;
constexpr int kAttnStages = 3;
constexpr int kTileBytes = 16 * 128 * 2;    // one block of one kv head: 16 tokens x 128 x bf16
constexpr int kAttnStage = 2 * kTileBytes;  // K then V
constexpr float kScaleLog2 = 0.08838834764831845f * 1.4426950408889634f;  // log2(e) / sqrt(128)

// out[r][a] = bf16(sum_c 2^(m_c - M) acc_c / sum_c 2^(m_c - M) l_c) over the request's chunks, in chunk order.
// One call handles 8 consecutive elements (index ch of 16) of head a; the 8 lanes of an aligned lane group must hold
// the 8 chunks of one 64-element group and all call together (group sums).  Writes the plain layout and/or the
// fragment-ordered operand of the O projection (K = nq * 128) with its group sums.
__device__ __forceinline__ void merge_head_chunk(const AttnArgs& p, int r, int a, int ch, bool valid) {
  const int s0 = p.slot_base[r], nc = p.nchunks[r];
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  float den = 0.0f;
  if (valid) {
    float M = -INFINITY;
    // the merge runs in the last CTA of a request, after everything else: its loads go out in batches (16 maxima,
    // then 8 chunks' partial results at a time) so that a request of a dozen chunks costs two round trips, not four
#pragma unroll 16
    for (int c = 0; c < nc; ++c) M = fmaxf(M, __ldcg(p.part_ml + ((size_t)(s0 + c) * p.nq + a) * 2));
#pragma unroll 8
    for (int c = 0; c < nc; ++c) {
      const size_t qh = (size_t)(s0 + c) * p.nq + a;
      const float2 ml = __ldcg(reinterpret_cast<const float2*>(p.part_ml + qh * 2));
      const float4 u = __ldcg(reinterpret_cast<const float4*>(p.part_acc + qh * kHeadDim + ch * 8));
      const float4 v = __ldcg(reinterpret_cast<const float4*>(p.part_acc + qh * kHeadDim + ch * 8 + 4));
      const float e = exp2f(ml.x - M);
      acc[0] = fmaf(e, u.x, acc[0]), acc[1] = fmaf(e, u.y, acc[1]), acc[2] = fmaf(e, u.z, acc[2]);
      acc[3] = fmaf(e, u.w, acc[3]), acc[4] = fmaf(e, v.x, acc[4]), acc[5] = fmaf(e, v.y, acc[5]);
      acc[6] = fmaf(e, v.z, acc[6]), acc[7] = fmaf(e, v.w, acc[7]);
      den = fmaf(e, ml.y, den);
    }
  } else {
    den = 1.0f;
  }
  uint4 o;
  o.x = pack_bf16x2(acc[0] / den, acc[1] / den);
  o.y = pack_bf16x2(acc[2] / den, acc[3] / den);
  o.z = pack_bf16x2(acc[4] / den, acc[5] / den);
  o.w = pack_bf16x2(acc[6] / den, acc[7] / den);
  const float gsum = group_sum_8lanes(chunk_sum(o));  // 8 lanes = 64 elements = one group of the O projection's K
  if (!valid) return;
  const size_t col = (size_t)a * kHeadDim + ch * 8;
  const size_t K = (size_t)p.nq * kHeadDim;
  if (p.out) *reinterpret_cast<uint4*>(p.out + (size_t)r * K + col) = o;
  if (p.out_xp) {
    *reinterpret_cast<uint4*>(p.out_xp + operand_chunk_offset(p.out_layout, (int)K, r, (int)(col >> 3))) = permute_chunk(o);
    if ((ch & 7) == 0) p.out_xs[(col >> 6) * 16 + r] = gsum;
  }
}

__global__ void __launch_bounds__(kAttnThreads) paged_attention_kernel(const AttnArgs p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int G = p.nq / p.nkv;
  const int h = blockIdx.y;

  grid_launch_dependents();
  // The cached K, V, the lengths, the block tables and the work list are not written by the preceding kernel, so
  // the first tiles are requested before it is awaited; q (and k, v of the new token) are read after the wait.
  bool waited = false;

  for (int item = blockIdx.x; item < p.n_work; item += gridDim.x) {
    const int4 w = p.work[item];
    const int r = w.x, tile_begin = w.y, tile_end = w.z, slot = w.w;
    const int T = p.lens[r] + 1, pos = T - 1;
    const int32_t* bt = p.block_tables + (size_t)r * p.max_blocks;
    unsigned char* ring = smem + warp * (kAttnStages * kAttnStage);

    auto issue_tile = [&](int tile, int stage) {
      const int blk = bt[tile];
      const size_t base = ((size_t)blk * p.nkv + h) * (16 * kHeadDim);
      const unsigned char* ksrc = reinterpret_cast<const unsigned char*>(p.kpool + base);
      const unsigned char* vsrc = reinterpret_cast<const unsigned char*>(p.vpool + base);
      unsigned char* dst = ring + stage * kAttnStage;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int c = i * 32 + lane;  // 16-byte chunk of the 4 KB block
        const int tok = c >> 4, c16 = c & 15;
        const int off = tok * 256 + ((c16 ^ (tok & 7)) << 4);
        cp_async16(dst + off, ksrc + c * 16);
        cp_async16(dst + kTileBytes + off, vsrc + c * 16);
      }
    };

    float o[16][4];
#pragma unroll
    for (int j = 0; j < 16; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.0f;
    float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.0f, l_hi = 0.0f;

    const int first = tile_begin + warp;
    const int my_tiles = (first < tile_end) ? (tile_end - first + kAttnWarps - 1) / kAttnWarps : 0;
#pragma unroll
    for (int s = 0; s < kAttnStages - 1; ++s) {
      if (s < my_tiles) issue_tile(first + s * kAttnWarps, s);
      cp_async_commit();
    }

    if (!waited) {
      grid_dependency_wait();
      waited = true;
    }

    // Q fragments: rows = query heads of this kv head (zero beyond G), k = head dimension.  With `qkv` given the
    // kernel prepares q itself (per-head RMSNorm, rotary embedding at the request's position) and the CTA that holds
    // the request's last tile also prepares k, v of the new token and appends them to the pool.
    uint32_t qa[8][4];
    const bool prep = p.qkv != nullptr;
    {
      const int heads = p.nq + 2 * p.nkv;
      const uint16_t* qbase = prep ? p.qkv + (size_t)r * heads * kHeadDim : p.q + (size_t)r * p.nq * kHeadDim;
      const uint16_t* q0 = qbase + (size_t)(h * G + g) * kHeadDim;
      const uint16_t* q1 = q0 + 8 * kHeadDim;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        qa[ks][0] = (g < G) ? *reinterpret_cast<const uint32_t*>(q0 + 16 * ks + 2 * t) : 0u;
        qa[ks][1] = (g + 8 < G) ? *reinterpret_cast<const uint32_t*>(q1 + 16 * ks + 2 * t) : 0u;
        qa[ks][2] = (g < G) ? *reinterpret_cast<const uint32_t*>(q0 + 16 * ks + 2 * t + 8) : 0u;
        qa[ks][3] = (g + 8 < G) ? *reinterpret_cast<const uint32_t*>(q1 + 16 * ks + 2 * t + 8) : 0u;
      }
    }
    if (prep) {
      if (p.q_norm) {
        float ss0 = 0.0f, ss1 = 0.0f;  // rows g and g + 8
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
            const uint32_t nw = *reinterpret_cast<const uint32_t*>(p.q_norm + 16 * ks + 2 * t + (rr >> 1) * 8);
            const float inv = (rr & 1) ? inv1 : inv0;
            qa[ks][rr] = pack_bf16x2(bf16_lo(qa[ks][rr]) * inv * bf16_lo(nw), bf16_hi(qa[ks][rr]) * inv * bf16_hi(nw));
          }
      }
#pragma unroll
      for (int ks = 0; ks < 4; ++ks)
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          const int col = 16 * ks + 2 * t + hf * 8;  // even, < 64; its partner is col + 64 (k-step ks + 4)
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
    // k, v of the new token: the warp that walks the request's last tile prepares them, appends them to the pool and
    // later puts them into its staged copy of that tile (which was fetched before they existed)
    const int last_tile = pos >> 4;
    const bool appends = prep && last_tile >= first && last_tile < tile_end && ((last_tile - first) % kAttnWarps) == 0;
    uint32_t nk_a = 0u, nk_b = 0u, nv_a = 0u, nv_b = 0u;  // elements 2*lane, 2*lane+1 and 64+2*lane, 64+2*lane+1
    if (appends) {
      const int heads = p.nq + 2 * p.nkv;
      const uint16_t* ksrc = p.qkv + ((size_t)r * heads + p.nq + h) * kHeadDim;
      const uint16_t* vsrc = ksrc + (size_t)p.nkv * kHeadDim;
      const uint32_t wa = *reinterpret_cast<const uint32_t*>(ksrc + 2 * lane);
      const uint32_t wb = *reinterpret_cast<const uint32_t*>(ksrc + 64 + 2 * lane);
      nv_a = *reinterpret_cast<const uint32_t*>(vsrc + 2 * lane);
      nv_b = *reinterpret_cast<const uint32_t*>(vsrc + 64 + 2 * lane);
      float a0 = bf16_lo(wa), a1 = bf16_hi(wa), b0 = bf16_lo(wb), b1 = bf16_hi(wb);
      if (p.k_norm) {
        const float ss = warp_sum(a0 * a0 + a1 * a1 + b0 * b0 + b1 * b1);
        const float inv = 1.0f / sqrtf(ss * (1.0f / kHeadDim) + p.eps);
        const uint32_t na = *reinterpret_cast<const uint32_t*>(p.k_norm + 2 * lane);
        const uint32_t nb = *reinterpret_cast<const uint32_t*>(p.k_norm + 64 + 2 * lane);
        a0 = bf16_to_f32(f32_to_bf16(a0 * inv * bf16_lo(na)));
        a1 = bf16_to_f32(f32_to_bf16(a1 * inv * bf16_hi(na)));
        b0 = bf16_to_f32(f32_to_bf16(b0 * inv * bf16_lo(nb)));
        b1 = bf16_to_f32(f32_to_bf16(b1 * inv * bf16_hi(nb)));
      }
      const float4 cs = *reinterpret_cast<const float4*>(p.rope + ((size_t)pos * 64 + 2 * lane) * 2);
      nk_a = pack_bf16x2(a0 * cs.x - b0 * cs.y, a1 * cs.z - b1 * cs.w);
      nk_b = pack_bf16x2(b0 * cs.x + a0 * cs.y, b1 * cs.z + a1 * cs.w);
      const size_t dst = (((size_t)bt[last_tile] * p.nkv + h) * kBlockSize + (pos & 15)) * kHeadDim;
      *reinterpret_cast<uint32_t*>(p.kpool_w + dst + 2 * lane) = nk_a;
      *reinterpret_cast<uint32_t*>(p.kpool_w + dst + 64 + 2 * lane) = nk_b;
      *reinterpret_cast<uint32_t*>(p.vpool_w + dst + 2 * lane) = nv_a;
      *reinterpret_cast<uint32_t*>(p.vpool_w + dst + 64 + 2 * lane) = nv_b;
    }

    for (int it = 0; it < my_tiles; ++it) {
      const int tile = first + it * kAttnWarps;
      if (it + kAttnStages - 1 < my_tiles)
        issue_tile(first + (it + kAttnStages - 1) * kAttnWarps, (it + kAttnStages - 1) % kAttnStages);
      cp_async_commit();
      cp_async_wait<kAttnStages - 1>();
      __syncwarp();
      unsigned char* sK = ring + (it % kAttnStages) * kAttnStage;
      unsigned char* sV = sK + kTileBytes;
      if (appends && tile == last_tile) {
        const int tk = pos & 15;
        const int off_a = tk * 256 + (((lane >> 2) ^ (tk & 7)) << 4) + (lane & 3) * 4;
        const int off_b = tk * 256 + (((8 + (lane >> 2)) ^ (tk & 7)) << 4) + (lane & 3) * 4;
        *reinterpret_cast<uint32_t*>(sK + off_a) = nk_a;
        *reinterpret_cast<uint32_t*>(sK + off_b) = nk_b;
        *reinterpret_cast<uint32_t*>(sV + off_a) = nv_a;
        *reinterpret_cast<uint32_t*>(sV + off_b) = nv_b;
        __syncwarp();
      }

      // scores S[head][token] for the 16 tokens of the block
      float s[2][4];
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.0f;
#pragma unroll
        for (int kp = 0; kp < 4; ++kp) {
          uint32_t kb[4];
          const int tok = 8 * j + (lane & 7), chunk = 4 * kp + (lane >> 3);
          ldmatrix_x4(kb, sK + tok * 256 + ((chunk ^ (tok & 7)) << 4));
          mma_bf16(s[j], qa[2 * kp][0], qa[2 * kp][1], qa[2 * kp][2], qa[2 * kp][3], kb[0], kb[1]);
          mma_bf16(s[j], qa[2 * kp + 1][0], qa[2 * kp + 1][1], qa[2 * kp + 1][2], qa[2 * kp + 1][3], kb[2], kb[3]);
        }
      }
      if (tile * 16 + 16 > T) {  // ragged last block: tokens at or beyond T do not exist
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
          for (int c = 0; c < 4; ++c)
            if (tile * 16 + 8 * j + 2 * t + (c & 1) >= T) s[j][c] = -INFINITY;
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
      uint32_t ph[4], pl[4];  // A fragments of P: hi and lo bf16 terms
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const float p0 = exp2f(fmaf(s[j][0], kScaleLog2, -m_lo)), p1 = exp2f(fmaf(s[j][1], kScaleLog2, -m_lo));
        const float p2 = exp2f(fmaf(s[j][2], kScaleLog2, -m_hi)), p3 = exp2f(fmaf(s[j][3], kScaleLog2, -m_hi));
        l_lo += p0 + p1;
        l_hi += p2 + p3;
        const uint32_t h01 = pack_bf16x2(p0, p1), h23 = pack_bf16x2(p2, p3);
        ph[2 * j] = h01, ph[2 * j + 1] = h23;
        pl[2 * j] = pack_bf16x2(p0 - bf16_lo(h01), p1 - bf16_hi(h01));
        pl[2 * j + 1] = pack_bf16x2(p2 - bf16_lo(h23), p3 - bf16_hi(h23));
      }

      // O[head][d] += P[head][token] V[token][d]
#pragma unroll
      for (int jp = 0; jp < 8; ++jp) {
        uint32_t vb[4];
        const int i = lane >> 3;
        const int tok = (i & 1) * 8 + (lane & 7), chunk = 2 * jp + (i >> 1);
        ldmatrix_x4_trans(vb, sV + tok * 256 + ((chunk ^ (tok & 7)) << 4));
        mma_bf16(o[2 * jp], ph[0], ph[1], ph[2], ph[3], vb[0], vb[1]);
        mma_bf16(o[2 * jp], pl[0], pl[1], pl[2], pl[3], vb[0], vb[1]);
        mma_bf16(o[2 * jp + 1], ph[0], ph[1], ph[2], ph[3], vb[2], vb[3]);
        mma_bf16(o[2 * jp + 1], pl[0], pl[1], pl[2], pl[3], vb[2], vb[3]);
      }
      __syncwarp();
    }
    cp_async_wait<0>();

    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);

    // merge the four warps through shared memory (overlays the rings)
    __syncthreads();
    float* sO = reinterpret_cast<float*>(smem);   // [warp][16][128]
    float* sM = sO + kAttnWarps * 16 * kHeadDim;  // [warp][16]
    float* sL = sM + kAttnWarps * 16;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      float* row_lo = sO + ((warp * 16 + g) * kHeadDim) + 8 * j + 2 * t;
      *reinterpret_cast<float2*>(row_lo) = make_float2(o[j][0], o[j][1]);
      *reinterpret_cast<float2*>(row_lo + 8 * kHeadDim) = make_float2(o[j][2], o[j][3]);
    }
    if (t == 0) {
      sM[warp * 16 + g] = m_lo, sM[warp * 16 + g + 8] = m_hi;
      sL[warp * 16 + g] = l_lo, sL[warp * 16 + g + 8] = l_hi;
    }
    __syncthreads();
    {
      const int d = threadIdx.x;
      for (int a = 0; a < G; ++a) {
        float M = sM[a];
#pragma unroll
        for (int ww = 1; ww < kAttnWarps; ++ww) M = fmaxf(M, sM[ww * 16 + a]);
        float num = 0.0f, den = 0.0f;
#pragma unroll
        for (int ww = 0; ww < kAttnWarps; ++ww) {
          const float e = exp2f(sM[ww * 16 + a] - M);
          num = fmaf(e, sO[(ww * 16 + a) * kHeadDim + d], num);
          den = fmaf(e, sL[ww * 16 + a], den);
        }
        const size_t qh = (size_t)slot * p.nq + (size_t)h * G + a;
        p.part_acc[qh * kHeadDim + d] = num;
        if (d == 0) {
          p.part_ml[qh * 2] = M;
          p.part_ml[qh * 2 + 1] = den;
        }
      }
    }
    if (p.merge_counters) {
      // the CTA that finishes the last chunk of this (request, kv head) merges all of them in chunk order
      __shared__ int s_last;
      __threadfence();
      __syncthreads();
      if (threadIdx.x == 0) {
        const int prev = atomicAdd(p.merge_counters + r * p.nkv + h, 1);
        s_last = prev == p.nchunks[r] - 1;
        if (s_last) p.merge_counters[r * p.nkv + h] = 0;
      }
      __syncthreads();
      if (s_last) {
        __threadfence();
        for (int a0 = 0; a0 < G; a0 += 8) {  // 16 threads per head, 8 heads per pass
          const int a = a0 + (threadIdx.x >> 4);
          merge_head_chunk(p, r, h * G + a, threadIdx.x & 15, a < G);
        }
      }
    }
    __syncthreads();
  }
}

// ---- the same work with the 16 tokens of a block as the MMA rows (kv groups of at most 8 query heads) ----
//
// S^T[token][head] = K q^T: A = the K block (rows = tokens), B = q of the G <= 8 heads (columns), 8 MMAs per block
// instead of 16; online softmax down the columns; P^T is moved from accumulator layout into B-fragment layout with
// movmatrix; O^T[d][head] += V^T[d][token] P^T[token][head] with P in two bf16 terms: 16 MMAs instead of 32 and 32
// accumulator registers instead of 64, so three CTAs fit on an SM with two-stage rings.
constexpr int kAttnTStages = 2;
constexpr int kAttnTPad = 132;  // floats per head row of the cross-warp merge buffer: conflict-free for the fragment layout

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t v) {
  uint32_t r;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(r) : "r"(v));
  return r;
}

__global__ void __launch_bounds__(kAttnThreads) paged_attention_t_kernel(const AttnArgs p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int G = p.nq / p.nkv;
  const int h = blockIdx.y;

  grid_launch_dependents();
  bool waited = false;  // as in the kernel above: cached K, V are requested before the preceding kernel is awaited

  for (int item = blockIdx.x; item < p.n_work; item += gridDim.x) {
    const int4 w = p.work[item];
    const int r = w.x, tile_begin = w.y, tile_end = w.z, slot = w.w;
    const int T = p.lens[r] + 1, pos = T - 1;
    const int32_t* bt = p.block_tables + (size_t)r * p.max_blocks;
    unsigned char* ring = smem + warp * (kAttnTStages * kAttnStage);

    auto issue_tile = [&](int tile, int stage) {
      const int blk = bt[tile];
      const size_t base = ((size_t)blk * p.nkv + h) * (16 * kHeadDim);
      const unsigned char* ksrc = reinterpret_cast<const unsigned char*>(p.kpool + base);
      const unsigned char* vsrc = reinterpret_cast<const unsigned char*>(p.vpool + base);
      unsigned char* dst = ring + stage * kAttnStage;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int c = i * 32 + lane;  // 16-byte chunk of the 4 KB block
        const int tok = c >> 4, c16 = c & 15;
        const int off = tok * 256 + ((c16 ^ (tok & 7)) << 4);
        cp_async16(dst + off, ksrc + c * 16);
        cp_async16(dst + kTileBytes + off, vsrc + c * 16);
      }
    };

    const int first = tile_begin + warp;
    const int my_tiles = (first < tile_end) ? (tile_end - first + kAttnWarps - 1) / kAttnWarps : 0;
#pragma unroll
    for (int s = 0; s < kAttnTStages - 1; ++s) {
      if (s < my_tiles) issue_tile(first + s * kAttnWarps, s);
      cp_async_commit();
    }

    // the rotary table and the norm weights do not depend on the preceding kernel either
    const bool prep = p.qkv != nullptr;
    float4 rope_cs[4][2];   // c0 s0 c1 s1 of columns 16ks + 2t + 8hf, +1 (their partners are 64 further)
    uint32_t qn_w[8][2];
    if (prep) {
#pragma unroll
      for (int ks = 0; ks < 4; ++ks)
#pragma unroll
        for (int hf = 0; hf < 2; ++hf)
          rope_cs[ks][hf] = __ldg(reinterpret_cast<const float4*>(p.rope + ((size_t)pos * 64 + 16 * ks + 2 * t + hf * 8) * 2));
      if (p.q_norm) {
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
#pragma unroll
          for (int hf = 0; hf < 2; ++hf)
            qn_w[ks][hf] = __ldg(reinterpret_cast<const uint32_t*>(p.q_norm + 16 * ks + 2 * t + hf * 8));
      }
    }

    if (!waited) {
      grid_dependency_wait();
      waited = true;
    }

    // q of head g of this kv head (zero beyond G): dims 16ks + 2t, +1 and 16ks + 2t + 8, +9 -- the B fragments
    uint32_t qb[8][2];
    {
      const int heads = p.nq + 2 * p.nkv;
      const uint16_t* qbase = prep ? p.qkv + (size_t)r * heads * kHeadDim : p.q + (size_t)r * p.nq * kHeadDim;
      const uint16_t* q0 = qbase + (size_t)(h * G + g) * kHeadDim;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        qb[ks][0] = (g < G) ? *reinterpret_cast<const uint32_t*>(q0 + 16 * ks + 2 * t) : 0u;
        qb[ks][1] = (g < G) ? *reinterpret_cast<const uint32_t*>(q0 + 16 * ks + 2 * t + 8) : 0u;
      }
    }
    if (prep) {
      if (p.q_norm) {
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
            const uint32_t nw = qn_w[ks][hf];
            qb[ks][hf] = pack_bf16x2(bf16_lo(qb[ks][hf]) * inv * bf16_lo(nw), bf16_hi(qb[ks][hf]) * inv * bf16_hi(nw));
          }
      }
#pragma unroll
      for (int ks = 0; ks < 4; ++ks)
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          const float4 cs = rope_cs[ks][hf];  // column 16ks + 2t + 8hf (even, < 64); its partner is k-step ks + 4
          const float a0 = bf16_lo(qb[ks][hf]), a1 = bf16_hi(qb[ks][hf]);
          const float b0 = bf16_lo(qb[ks + 4][hf]), b1 = bf16_hi(qb[ks + 4][hf]);
          qb[ks][hf] = pack_bf16x2(a0 * cs.x - b0 * cs.y, a1 * cs.z - b1 * cs.w);
          qb[ks + 4][hf] = pack_bf16x2(b0 * cs.x + a0 * cs.y, b1 * cs.z + a1 * cs.w);
        }
    }
    // k, v of the new token: prepared and appended by the warp that walks the request's last tile, which later puts
    // them into its staged copy of that tile (fetched before they existed)
    const int last_tile = pos >> 4;
    const bool appends = prep && last_tile >= first && last_tile < tile_end && ((last_tile - first) % kAttnWarps) == 0;
    uint32_t nk_a = 0u, nk_b = 0u, nv_a = 0u, nv_b = 0u;  // elements 2*lane, 2*lane+1 and 64+2*lane, 64+2*lane+1
    if (appends) {
      const int heads = p.nq + 2 * p.nkv;
      const uint16_t* ksrc = p.qkv + ((size_t)r * heads + p.nq + h) * kHeadDim;
      const uint16_t* vsrc = ksrc + (size_t)p.nkv * kHeadDim;
      const uint32_t wa = *reinterpret_cast<const uint32_t*>(ksrc + 2 * lane);
      const uint32_t wb = *reinterpret_cast<const uint32_t*>(ksrc + 64 + 2 * lane);
      nv_a = *reinterpret_cast<const uint32_t*>(vsrc + 2 * lane);
      nv_b = *reinterpret_cast<const uint32_t*>(vsrc + 64 + 2 * lane);
      float a0 = bf16_lo(wa), a1 = bf16_hi(wa), b0 = bf16_lo(wb), b1 = bf16_hi(wb);
      if (p.k_norm) {
        const float ss = warp_sum(a0 * a0 + a1 * a1 + b0 * b0 + b1 * b1);
        const float inv = 1.0f / sqrtf(ss * (1.0f / kHeadDim) + p.eps);
        const uint32_t na = *reinterpret_cast<const uint32_t*>(p.k_norm + 2 * lane);
        const uint32_t nb = *reinterpret_cast<const uint32_t*>(p.k_norm + 64 + 2 * lane);
        a0 = bf16_to_f32(f32_to_bf16(a0 * inv * bf16_lo(na)));
        a1 = bf16_to_f32(f32_to_bf16(a1 * inv * bf16_hi(na)));
        b0 = bf16_to_f32(f32_to_bf16(b0 * inv * bf16_lo(nb)));
        b1 = bf16_to_f32(f32_to_bf16(b1 * inv * bf16_hi(nb)));
      }
      const float4 cs = *reinterpret_cast<const float4*>(p.rope + ((size_t)pos * 64 + 2 * lane) * 2);
      nk_a = pack_bf16x2(a0 * cs.x - b0 * cs.y, a1 * cs.z - b1 * cs.w);
      nk_b = pack_bf16x2(b0 * cs.x + a0 * cs.y, b1 * cs.z + a1 * cs.w);
      const size_t dst = (((size_t)bt[last_tile] * p.nkv + h) * kBlockSize + (pos & 15)) * kHeadDim;
      *reinterpret_cast<uint32_t*>(p.kpool_w + dst + 2 * lane) = nk_a;
      *reinterpret_cast<uint32_t*>(p.kpool_w + dst + 64 + 2 * lane) = nk_b;
      *reinterpret_cast<uint32_t*>(p.vpool_w + dst + 2 * lane) = nv_a;
      *reinterpret_cast<uint32_t*>(p.vpool_w + dst + 64 + 2 * lane) = nv_b;
    }

    // o[dt][c]: d = 16 dt + g + 8 (c >> 1), head 2t + (c & 1); m, l of heads 2t (index 0) and 2t + 1 (index 1)
    float o[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.0f;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.0f, l1 = 0.0f;

    for (int it = 0; it < my_tiles; ++it) {
      const int tile = first + it * kAttnWarps;
      if (it + kAttnTStages - 1 < my_tiles)
        issue_tile(first + (it + kAttnTStages - 1) * kAttnWarps, (it + kAttnTStages - 1) % kAttnTStages);
      cp_async_commit();
      cp_async_wait<kAttnTStages - 1>();
      __syncwarp();
      unsigned char* sK = ring + (it % kAttnTStages) * kAttnStage;
      unsigned char* sV = sK + kTileBytes;
      if (appends && tile == last_tile) {
        const int tk = pos & 15;
        const int off_a = tk * 256 + (((lane >> 2) ^ (tk & 7)) << 4) + (lane & 3) * 4;
        const int off_b = tk * 256 + (((8 + (lane >> 2)) ^ (tk & 7)) << 4) + (lane & 3) * 4;
        *reinterpret_cast<uint32_t*>(sK + off_a) = nk_a;
        *reinterpret_cast<uint32_t*>(sK + off_b) = nk_b;
        *reinterpret_cast<uint32_t*>(sV + off_a) = nv_a;
        *reinterpret_cast<uint32_t*>(sV + off_b) = nv_b;
        __syncwarp();
      }

      // scores: rows = tokens g, g + 8 of the block; columns = heads 2t, 2t + 1.  Two accumulators halve the
      // chain of dependent MMAs.
      float s[4] = {0.0f, 0.0f, 0.0f, 0.0f}, s2[4] = {0.0f, 0.0f, 0.0f, 0.0f};
      {
        const int mi = lane >> 3, tok = (mi & 1) * 8 + (lane & 7);
        const unsigned char* kb = sK + tok * 256;
#pragma unroll
        for (int ks = 0; ks < 8; ks += 2) {
          uint32_t ka[4], kc[4];
          ldmatrix_x4(ka, kb + (((2 * ks + (mi >> 1)) ^ (tok & 7)) << 4));
          ldmatrix_x4(kc, kb + (((2 * ks + 2 + (mi >> 1)) ^ (tok & 7)) << 4));
          mma_bf16(s, ka[0], ka[1], ka[2], ka[3], qb[ks][0], qb[ks][1]);
          mma_bf16(s2, kc[0], kc[1], kc[2], kc[3], qb[ks + 1][0], qb[ks + 1][1]);
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) s[c] += s2[c];
      }
      if (tile * 16 + 16 > T) {  // ragged last block: tokens at or beyond T do not exist
        if (tile * 16 + g >= T) s[0] = s[1] = -INFINITY;
        if (tile * 16 + g + 8 >= T) s[2] = s[3] = -INFINITY;
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
        const uint32_t h01 = pack_bf16x2(p0, p1), h23 = pack_bf16x2(p2, p3);  // token g | g + 8; heads 2t, 2t + 1
        const uint32_t e01 = pack_bf16x2(p0 - bf16_lo(h01), p1 - bf16_hi(h01));
        const uint32_t e23 = pack_bf16x2(p2 - bf16_lo(h23), p3 - bf16_hi(h23));
        pH[0] = movmatrix_trans(h01), pH[1] = movmatrix_trans(h23);
        pL[0] = movmatrix_trans(e01), pL[1] = movmatrix_trans(e23);
      }

      // O^T[d][head] += V^T[d][token] P^T[token][head]
      {
        const int mi = lane >> 3, tok = (mi >> 1) * 8 + (lane & 7);
        const unsigned char* vb = sV + tok * 256;
#pragma unroll
        for (int dt = 0; dt < 8; ++dt) {
          uint32_t va[4];
          ldmatrix_x4_trans(va, vb + (((2 * dt + (mi & 1)) ^ (tok & 7)) << 4));
          mma_bf16(o[dt], va[0], va[1], va[2], va[3], pH[0], pH[1]);
          mma_bf16(o[dt], va[0], va[1], va[2], va[3], pL[0], pL[1]);
        }
      }
      __syncwarp();
    }
    cp_async_wait<0>();

#pragma unroll
    for (int sh = 4; sh <= 16; sh <<= 1) {
      l0 += __shfl_xor_sync(0xffffffffu, l0, sh);
      l1 += __shfl_xor_sync(0xffffffffu, l1, sh);
    }

    // merge the four warps through shared memory (overlays the rings)
    __syncthreads();
    float* sO = reinterpret_cast<float*>(smem);    // [warp][8 heads][kAttnTPad]
    float* sM = sO + kAttnWarps * 8 * kAttnTPad;   // [warp][8]
    float* sL = sM + kAttnWarps * 8;
#pragma unroll
    for (int dt = 0; dt < 8; ++dt)
#pragma unroll
      for (int c = 0; c < 4; ++c)
        sO[(warp * 8 + 2 * t + (c & 1)) * kAttnTPad + 16 * dt + g + 8 * (c >> 1)] = o[dt][c];
    if (g == 0) {
      sM[warp * 8 + 2 * t] = m0, sM[warp * 8 + 2 * t + 1] = m1;
      sL[warp * 8 + 2 * t] = l0, sL[warp * 8 + 2 * t + 1] = l1;
    }
    __syncthreads();
    {
      const int d = threadIdx.x;
      for (int a = 0; a < G; ++a) {
        float M = sM[a];
#pragma unroll
        for (int ww = 1; ww < kAttnWarps; ++ww) M = fmaxf(M, sM[ww * 8 + a]);
        float num = 0.0f, den = 0.0f;
#pragma unroll
        for (int ww = 0; ww < kAttnWarps; ++ww) {
          const float e = exp2f(sM[ww * 8 + a] - M);
          num = fmaf(e, sO[(ww * 8 + a) * kAttnTPad + d], num);
          den = fmaf(e, sL[ww * 8 + a], den);
        }
        const size_t qh = (size_t)slot * p.nq + (size_t)h * G + a;
        p.part_acc[qh * kHeadDim + d] = num;
        if (d == 0) {
          p.part_ml[qh * 2] = M;
          p.part_ml[qh * 2 + 1] = den;
        }
      }
    }
    if (p.merge_counters) {
      // the CTA that finishes the last chunk of this (request, kv head) merges all of them in chunk order
      __shared__ int s_last;
      __threadfence();
      __syncthreads();
      if (threadIdx.x == 0) {
        const int prev = atomicAdd(p.merge_counters + r * p.nkv + h, 1);
        s_last = prev == p.nchunks[r] - 1;
        if (s_last) p.merge_counters[r * p.nkv + h] = 0;
      }
      __syncthreads();
      if (s_last) {
        __threadfence();
        merge_head_chunk(p, r, h * G + (threadIdx.x >> 4), threadIdx.x & 15, (threadIdx.x >> 4) < G);  // 16 threads per head
      }
    }
    __syncthreads();
  }
}

// The merge as a kernel of its own: 16 threads per head; a CTA of 128 threads takes 8 heads.
__global__ void __launch_bounds__(128) attention_merge_kernel(const AttnArgs p) {
  grid_launch_dependents();
  grid_dependency_wait();
  const int r = blockIdx.x, a = blockIdx.y * 8 + (threadIdx.x >> 4), ch = threadIdx.x & 15;
  merge_head_chunk(p, r, a, ch, a < p.nq);
}

// One warp per (request, head of qkv): optional RMSNorm over the head, rotary embedding at the
// request's position, then q -> q_out, k and v -> the pool slot of the new token.
__global__ void __launch_bounds__(128) rope_append_kernel(const RopeArgs p) {
  grid_launch_dependents();
  grid_dependency_wait();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int heads = p.nq + 2 * p.nkv;
  const int hd = blockIdx.x * 4 + warp, r = blockIdx.y;
  if (hd >= heads) return;
  const uint16_t* src = p.qkv + ((size_t)r * heads + hd) * kHeadDim;
  const int pos = p.lens[r];
  // lane holds elements 2*lane, 2*lane+1 and their rotary partners 64 + 2*lane, 64 + 2*lane + 1
  const uint32_t wa = *reinterpret_cast<const uint32_t*>(src + 2 * lane);
  const uint32_t wb = *reinterpret_cast<const uint32_t*>(src + 64 + 2 * lane);
  uint32_t oa = wa, ob = wb;
  if (hd < p.nq + p.nkv) {
    float a0 = bf16_lo(wa), a1 = bf16_hi(wa), b0 = bf16_lo(wb), b1 = bf16_hi(wb);
    const uint16_t* nw = (hd < p.nq) ? p.q_norm : p.k_norm;
    if (nw) {
      const float ss = warp_sum(a0 * a0 + a1 * a1 + b0 * b0 + b1 * b1);
      const float inv = 1.0f / sqrtf(ss * (1.0f / kHeadDim) + p.eps);
      const uint32_t na = *reinterpret_cast<const uint32_t*>(nw + 2 * lane);
      const uint32_t nb = *reinterpret_cast<const uint32_t*>(nw + 64 + 2 * lane);
      a0 = bf16_to_f32(f32_to_bf16(a0 * inv * bf16_lo(na)));
      a1 = bf16_to_f32(f32_to_bf16(a1 * inv * bf16_hi(na)));
      b0 = bf16_to_f32(f32_to_bf16(b0 * inv * bf16_lo(nb)));
      b1 = bf16_to_f32(f32_to_bf16(b1 * inv * bf16_hi(nb)));
    }
    const float4 cs = *reinterpret_cast<const float4*>(p.rope + ((size_t)pos * 64 + 2 * lane) * 2);  // c0 s0 c1 s1
    oa = pack_bf16x2(a0 * cs.x - b0 * cs.y, a1 * cs.z - b1 * cs.w);
    ob = pack_bf16x2(b0 * cs.x + a0 * cs.y, b1 * cs.z + a1 * cs.w);
  }
  uint16_t* dst;
  if (hd < p.nq) {
    dst = p.q_out + ((size_t)r * p.nq + hd) * kHeadDim;
  } else {
    const int kvh = (hd - p.nq) % p.nkv;
    const bool is_v = hd >= p.nq + p.nkv;
    const int blk = p.block_tables[(size_t)r * p.max_blocks + pos / kBlockSize], slot = pos % kBlockSize;
    dst = (is_v ? p.vpool : p.kpool) + (((size_t)blk * p.nkv + kvh) * kBlockSize + slot) * kHeadDim;
  }
  *reinterpret_cast<uint32_t*>(dst + 2 * lane) = oa;
  *reinterpret_cast<uint32_t*>(dst + 64 + 2 * lane) = ob;
}

int g_attn_sm_count = 0;
int g_attn_ctas_per_sm[2] = {0, 0};  // resident CTAs per SM: [0] heads as MMA rows, [1] tokens as MMA rows

constexpr int kAttnSmem = kAttnWarps * kAttnStages * kAttnStage;
constexpr int kAttnTSmem = kAttnWarps * kAttnTStages * kAttnStage;

}  // namespace

cudaError_t attention_init() {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  int sms = 0;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(paged_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmem);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(paged_attention_t_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnTSmem);
  if (e != cudaSuccess) return e;
  // the neighbouring projection kernels run with the largest shared-memory carve-out; asking for the same one here
  // keeps the SMs from being reconfigured (and drained) between the kernels of a layer
  e = cudaFuncSetAttribute(paged_attention_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(paged_attention_t_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  if (e != cudaSuccess) return e;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&g_attn_ctas_per_sm[0], paged_attention_kernel, kAttnThreads, kAttnSmem);
  if (e != cudaSuccess) return e;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&g_attn_ctas_per_sm[1], paged_attention_t_kernel, kAttnThreads, kAttnTSmem);
  if (e != cudaSuccess) return e;
  if (g_attn_ctas_per_sm[0] < 1 || g_attn_ctas_per_sm[1] < 1) return cudaErrorInvalidConfiguration;
  g_attn_sm_count = sms;
  return cudaSuccess;
}

// CTAs of the attention kernel that are resident at once for this head grouping (one wave of the grid).
int attention_wave_ctas(int nq, int nkv) {
  if (g_attn_sm_count == 0 && attention_init() != cudaSuccess) return 0;
  return g_attn_sm_count * g_attn_ctas_per_sm[nq / nkv <= 8 ? 1 : 0];
}

int attention_max_work(int max_batch, int max_positions) {
  // smallest automatic chunk is 4 tiles (64 tokens)
  return max_batch * ((max_positions + 63) / 64 + 1);
}

AttnPlan plan_attention(const int32_t* lens, int n, int nkv, int chunk_tokens, int wave_ctas, int4* work,
                        int32_t* slot_base, int32_t* nchunks, int max_work) {
  AttnPlan plan;
  long long total_tiles = 0;
  for (int r = 0; r < n; ++r) total_tiles += (lens[r] + 1 + 15) / 16;
  int chunk_tiles;
  if (chunk_tokens > 0) {
    chunk_tiles = (chunk_tokens + 15) / 16;
  } else {
    // One wave: aim at as many (item, kv head) CTAs as are resident at once, of equal size (a multiple of 4 tiles so
    // that the four warps of a CTA get equal shares), at least 4 tiles and at most 512: a second, partly filled
    // wave of shorter items costs more than one wave of longer ones.
    const long long slots = wave_ctas > 0 ? wave_ctas : 1;
    long long ct = (total_tiles * nkv + slots - 1) / slots;
    ct = (ct + 3) / 4 * 4;
    chunk_tiles = (int)(ct < 4 ? 4 : (ct > 512 ? 512 : ct));
    // requests add a ragged last chunk each: grow the chunk until the items fit the wave
    for (;;) {
      long long items = 0;
      for (int r = 0; r < n; ++r) items += ((lens[r] + 1 + 15) / 16 + chunk_tiles - 1) / chunk_tiles;
      if (items * nkv <= slots || chunk_tiles >= 512) break;
      chunk_tiles += 4;
    }
  }
  if (chunk_tiles < 1) chunk_tiles = 1;
  int w = 0;
  for (int r = 0; r < n; ++r) {
    const int tiles = (lens[r] + 1 + 15) / 16;
    slot_base[r] = w;
    int c = 0;
    for (int t0 = 0; t0 < tiles && w < max_work; t0 += chunk_tiles, ++c, ++w)
      work[w] = make_int4(r, t0, t0 + chunk_tiles < tiles ? t0 + chunk_tiles : tiles, w);
    nchunks[r] = c;
  }
  plan.n_work = w;
  plan.n_slots = w;
  plan.chunk_tiles = chunk_tiles;
  return plan;
}

cudaError_t launch_paged_attention(const AttnArgs& a, cudaStream_t s) {
  if (g_attn_sm_count == 0) {
    cudaError_t e = attention_init();
    if (e != cudaSuccess) return e;
  }
  if (a.n_work <= 0) return cudaSuccess;
  const int G = a.nq / a.nkv;
  if (G < 1 || G > 16 || a.nq % a.nkv) return cudaErrorInvalidValue;
  const dim3 grid(a.n_work, a.nkv), block(kAttnThreads);
  if (G <= 8) return launch_kernel_pdl(!a.after_predecessor, paged_attention_t_kernel, grid, block, kAttnTSmem, s, a);
  return launch_kernel_pdl(!a.after_predecessor, paged_attention_kernel, grid, block, kAttnSmem, s, a);
}

cudaError_t launch_attention_merge(const AttnArgs& a, cudaStream_t s) {
  if (a.n <= 0) return cudaSuccess;
  return launch_kernel(attention_merge_kernel, dim3(a.n, (a.nq + 7) / 8), dim3(128), 0, s, a);
}

cudaError_t launch_rope_append(const RopeArgs& a, cudaStream_t s) {
  if (a.n <= 0) return cudaSuccess;
  const int heads = a.nq + 2 * a.nkv;
  return launch_kernel(rope_append_kernel, dim3((heads + 3) / 4, a.n), dim3(128), 0, s, a);
}

}  // namespace q4d
