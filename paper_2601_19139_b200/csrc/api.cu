// C ABI of the q4decode library: objects, host-side validation, and the
// stream-ordered launch sequence of one decode step.
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <new>
#include <string>
#include <unordered_map>
#include <unordered_set>
#include <vector>

#include "../../include/q4decode.h"
#include "fused_step.h"
#include "kernels.h"

using namespace q4d;

namespace {

thread_local std::string g_last_error;

int fail(int code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  g_last_error = buf;
  return code;
}

int fail_cuda(cudaError_t e, const char* what) {
  return fail(Q4D_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

bool g_pdl = true;

constexpr size_t kAlign = 256;
size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

// Per-step metadata, one contiguous block: header, attention work list, block tables.
struct MetaLayout {
  int max_blocks_cap, max_work;
  size_t off_tokens, off_lens, off_slot_base, off_nchunks, off_bt, off_work, bytes;
  void init(int max_positions) {
    max_blocks_cap = (max_positions + kBlockSize - 1) / kBlockSize;
    max_work = attention_max_work(kMaxBatch, max_positions);
    size_t o = 0;
    off_tokens = o, o += kMaxBatch * 4;
    off_lens = o, o += kMaxBatch * 4;
    off_slot_base = o, o += kMaxBatch * 4;
    off_nchunks = o, o += kMaxBatch * 4;
    off_work = o, o += (size_t)max_work * sizeof(int4);
    off_bt = o, o += (size_t)kMaxBatch * max_blocks_cap * 4;
    bytes = align_up(o);
  }
};

struct Workspace {
  // x: residual stream (plain).  yp/ys, ap/as, hp/hs: GEMM operands in fragment order with their group sums
  // (normed hidden state, attention output, silu(gate)*up).
  size_t x, yp, ys, qkv, qbuf, ap, as, hp, hs, logits, next, amax, gemm_partial, gemm_partial_bytes, counters,
      part_acc, part_ml, attn_merge_counters, meta, bytes;
  // MoE: plain normed state, routing results, touched-expert list, per-slot expert activations and outputs
  size_t yplain, m_idx, m_wgt, m_ints, m_hp, m_hs, m_o;
  int counters_len, amax_blocks;
  // persistent whole-step kernel (dense models): plain attention output and gated MLP activations, sums of squares
  // of the residual stream, split-KV scratch, argmax partials, barrier/status words, phase table
  size_t f_attn, f_h, f_ss, f_pacc, f_pml, f_attn_counters, f_amax, f_control, f_timeline, chain_status;
  int f_max_items, f_max_ctas, f_n_phases;
};

// The CTA count the whole-step kernel is sized for: one per SM of the current device (148 when there is none).
int fused_cta_bound() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    (void)cudaGetLastError();
    return 148;
  }
  return sms > 0 ? sms : 148;
}

struct FusedGemmDims {
  int N, K, ntiles, S;
};
FusedGemmDims fused_dims(int N, int K, int epi) {
  FusedGemmDims d;
  d.N = N, d.K = K;
  d.ntiles = epi == EPI_SILU_PACK ? N / 16 : (N + 15) / 16;  // SiLU tiles: 8 gate rows + 8 up rows of N/2 columns
  d.S = (K + kFusedSliceK - 1) / kFusedSliceK;
  return d;
}

bool shape_supported(const q4d_shape& s, std::string* why) {
  auto bad = [&](const char* m) {
    if (why) *why = m;
    return false;
  };
  if (s.n_layers < 1 || s.hidden < 256 || s.n_q_heads < 1 || s.n_kv_heads < 1 || s.vocab < 1)
    return bad("non-positive dimension");
  if (s.head_dim != kHeadDim) return bad("head_dim must be 128");
  if (s.group_size != 64 || s.bits != 4) return bad("only 4-bit group-64 weights are supported");
  if (s.n_q_heads % s.n_kv_heads || s.n_q_heads / s.n_kv_heads > 16) return bad("q heads per kv head must be 1..16");
  if (s.hidden % 256 || (s.n_q_heads * s.head_dim) % 256) return bad("hidden and nq*128 must be multiples of 256");
  if (s.hidden > 16384) return bad("hidden must be at most 16384 (the RMSNorm kernel holds a row in registers)");
  if (s.max_batch < 1 || s.max_batch > kMaxBatch) return bad("max_batch must be 1..16");
  if (s.max_positions < 1) return bad("max_positions must be positive");
  if (s.n_experts == 0) {
    if (s.mlp_inter < 256 || s.mlp_inter % 256) return bad("mlp_inter must be a positive multiple of 256");
  } else {
    if (s.n_experts > 256 || s.top_k < 1 || s.top_k > 32 || s.top_k > s.n_experts) return bad("need 1 <= top_k <= min(32, n_experts), n_experts <= 256");
    if (s.expert_inter < 256 || s.expert_inter % 256 || s.expert_inter > 2048) return bad("expert_inter must be a multiple of 256, at most 2048");
    if (s.hidden > 2048) return bad("MoE layers need hidden <= 2048");
  }
  return true;
}

Workspace carve(const q4d_shape& s, const MetaLayout& ml) {
  Workspace w;
  size_t o = 0;
  auto take = [&](size_t bytes) {
    size_t at = o;
    o += align_up(bytes);
    return at;
  };
  const size_t B = kMaxBatch;
  const int nqkv = (s.n_q_heads + 2 * s.n_kv_heads) * kHeadDim;
  const size_t qdim = (size_t)s.n_q_heads * kHeadDim;
  w.x = take(B * s.hidden * 2);
  w.yp = take(operand_elements(OPERAND_SLICED, s.hidden) * 2);  // the largest of the layouts
  w.ys = take((size_t)(s.hidden / 64) * 16 * 4);
  w.qkv = take(B * nqkv * 2);
  w.qbuf = take(B * qdim * 2);
  w.ap = take(operand_elements(OPERAND_SLICED, qdim) * 2);
  w.as = take((qdim / 64) * 16 * 4);
  w.hp = take(operand_elements(OPERAND_SLICED, s.mlp_inter) * 2 + 256);
  w.hs = take((size_t)(s.mlp_inter / 64) * 16 * 4 + 256);
  w.yplain = w.m_idx = w.m_wgt = w.m_ints = w.m_hp = w.m_hs = w.m_o = 0;
  if (s.n_experts) {
    const size_t E = s.n_experts;
    w.yplain = take(B * s.hidden * 2);
    w.m_idx = take(B * s.top_k * 4);
    w.m_wgt = take(B * s.top_k * 4);
    // flags[E], expert_ids[E], slot_of[E], counter, n_touched, touched_total, slice_counter[16], then logits[16][E]
    w.m_ints = take((3 * E + 3 + kMaxBatch) * 4 + B * E * 4);
    w.m_hp = take(E * B * s.expert_inter * 2);
    w.m_hs = take(E * (size_t)(s.expert_inter / 64) * 16 * 4);
    w.m_o = take(E * B * s.hidden * 2);
  }
  w.logits = take(B * (size_t)s.vocab * 4);
  w.next = take(B * 4);
  w.amax_blocks = std::max(gemm_row_blocks(s.vocab, s.hidden, 8, EPI_F32), gemm_row_blocks(s.vocab, s.hidden, 16, EPI_F32));
  w.amax = take((size_t)w.amax_blocks * 16 * sizeof(float2));
  size_t pb = 0;
  int cl = 0;
  auto gemm = [&](int N, int K, int epi) {
    pb = std::max(pb, gemm_partial_bytes(N, K, epi));
    cl = std::max(cl, gemm_counters_needed(N));
  };
  gemm(nqkv, s.hidden, EPI_BF16);
  gemm(s.hidden, s.n_q_heads * kHeadDim, EPI_RESIDUAL);
  if (!s.n_experts) {
    gemm(2 * s.mlp_inter, s.hidden, EPI_SILU_PACK);
    gemm(s.hidden, s.mlp_inter, EPI_RESIDUAL);
  }
  gemm(s.vocab, s.hidden, EPI_F32);
  w.gemm_partial_bytes = pb;
  w.gemm_partial = take(pb);
  w.counters_len = cl;
  w.counters = take((size_t)cl * 4);
  w.part_acc = take((size_t)ml.max_work * s.n_q_heads * kHeadDim * 4);
  w.part_ml = take((size_t)ml.max_work * s.n_q_heads * 2 * 4);
  w.attn_merge_counters = take((size_t)16 * s.n_kv_heads * 4);
  w.meta = take(ml.bytes);
  w.f_attn = w.f_h = w.f_ss = w.f_pacc = w.f_pml = w.f_attn_counters = w.f_amax = 0;
  w.f_control = w.f_timeline = 0;
  w.chain_status = take(256);  // status word of the chain's kernels (a bounded wait that gave up)
  w.f_max_items = w.f_max_ctas = w.f_n_phases = 0;
  if (!s.n_experts) {
    const int G = s.n_q_heads / s.n_kv_heads;
    w.f_max_ctas = fused_cta_bound();
    w.f_max_items = std::max(w.f_max_ctas * (kFusedThreads / 32), 16 * s.n_kv_heads);
    w.f_n_phases = 3 + kFusedPhasesPerLayer * s.n_layers;
    w.f_attn = take(B * qdim * 2);
    w.f_h = take(B * (size_t)s.mlp_inter * 2);
    w.f_ss = take((size_t)(s.hidden / 16) * 16 * 4);
    const int Gs = (G + 1) & ~1;  // heads per split-KV partial result
    w.f_pacc = take((size_t)w.f_max_items * Gs * kHeadDim * 4);
    w.f_pml = take((size_t)w.f_max_items * Gs * 2 * 4);
    w.f_attn_counters = take((size_t)16 * s.n_kv_heads * 4);
    w.f_amax = take((size_t)w.f_max_ctas * 16 * sizeof(float2));
    w.f_control = take(256);
    w.f_timeline = take((size_t)(w.f_n_phases + 1) * 8);
  }
  w.bytes = o;
  return w;
}

constexpr int kStagingSlots = 8;

struct ProfileRec {
  cudaEvent_t a, b;
  int cls;
};

}  // namespace

struct q4d_model {
  q4d_shape sh;
  std::vector<q4d_layer_weights> layers;
  q4d_weights w;
  unsigned char* ws;
  Workspace lay;
  MetaLayout ml;
  int sm_count;
  // pinned staging ring for the per-step metadata
  unsigned char* staging[kStagingSlots];
  cudaEvent_t staging_done[kStagingSlots];
  bool staging_used[kStagingSlots];
  int staging_next;
  // instrumentation
  bool profile;
  std::vector<ProfileRec> prof_recs;
  std::vector<cudaEvent_t> prof_free;
  int64_t launches;
  int64_t last_h2d, last_d2h;
  int32_t* host_next;  // pinned, for the host-output variant
  // persistent whole-step kernel
  bool fused;
  int fused_ctas;
  FusedStep* fused_params;  // host template of the kernel parameters
  bool timeline;
  uint32_t* host_status;  // pinned copy of the kernel's status word, read back after every step
  cudaEvent_t status_done;
  bool status_pending;
  bool timed_out;  // a kernel of an earlier step reported a wait that gave up: every later step is refused
};

struct q4d_kv_pool {
  q4d_model* model;
  int32_t num_blocks;
  uint16_t* mem;
  std::unordered_map<int64_t, int32_t> lens;
};

namespace {

template <typename T>
T* at(q4d_model* m, size_t off) {
  return reinterpret_cast<T*>(m->ws + off);
}

// Runs one launch, bracketed by events in profile mode.
template <typename F>
cudaError_t timed(q4d_model* m, int cls, cudaStream_t s, F&& f) {
  ProfileRec rec{nullptr, nullptr, cls};
  if (m->profile) {
    for (cudaEvent_t* ev : {&rec.a, &rec.b}) {
      if (!m->prof_free.empty()) {
        *ev = m->prof_free.back();
        m->prof_free.pop_back();
      } else {
        cudaError_t e = cudaEventCreate(ev);
        if (e != cudaSuccess) return e;
      }
    }
    cudaEventRecord(rec.a, s);
  }
  cudaError_t e = f();
  m->launches++;
  if (m->profile) {
    cudaEventRecord(rec.b, s);
    m->prof_recs.push_back(rec);
  }
  return e;
}

GemmArgs gemm_args(q4d_model* m, const q4d_qtensor& t, int N, int K, const uint16_t* xp, const float* xs, int n,
                   int epi, void* out, int out_stride) {
  GemmArgs a;
  a.qw = t.q, a.scales = t.scales, a.biases = t.biases;
  a.N = N, a.K = K, a.xp = xp, a.xs = xs, a.n = n, a.epilogue = epi;
  a.out = out, a.out_stride = out_stride;
  a.out_xp = nullptr, a.out_xs = nullptr, a.argmax_partial = nullptr;
  a.partial = at<float>(m, m->lay.gemm_partial), a.partial_bytes = m->lay.gemm_partial_bytes;
  a.counters = at<int>(m, m->lay.counters), a.counters_len = m->lay.counters_len;
  a.status = at<unsigned int>(m, m->lay.chain_status);
  return a;
}

bool qt_ok(const q4d_qtensor& t) { return t.q && t.scales && t.biases; }

// ---- persistent whole-step kernel: phase table and per-step launch ----

// Phase kinds of the whole-step kernel (index into FusedStep::dims) and the timeline class each is filed under.
const int kFusedKindClass[kFusedDimKinds] = {Q4D_K_EMBED,  Q4D_K_RMSNORM,      Q4D_K_GEMM_QKV,  Q4D_K_ATTENTION, Q4D_K_GEMM_O,
                                             Q4D_K_RMSNORM, Q4D_K_GEMM_GATE_UP, Q4D_K_GEMM_DOWN, Q4D_K_RMSNORM,   Q4D_K_LM_HEAD};
int fused_kind(int ph, int n_phases) {
  return ph == 0 ? 0 : (ph >= n_phases - 2 ? 8 + (ph - (n_phases - 2)) : 1 + (ph - 1) % kFusedPhasesPerLayer);
}

// Everything of the kernel's parameters that does not change from step to step.
void build_fused_params(const q4d_model* m, FusedStep* fp) {
  const q4d_shape& sh = m->sh;
  const Workspace& lay = m->lay;
  const int H = sh.hidden, nq = sh.n_q_heads, nkv = sh.n_kv_heads, I = sh.mlp_inter, V = sh.vocab;
  const int nqkv = (nq + 2 * nkv) * kHeadDim, qdim = nq * kHeadDim;
  memset(fp, 0, sizeof *fp);
  for (int l = 0; l < sh.n_layers; ++l) {
    const q4d_layer_weights& lw = m->layers[l];
    FusedLayerPtrs& L = fp->layer[l];
    const q4d_qtensor* t[4] = {&lw.wqkv, &lw.wo, &lw.w_gate_up, &lw.w_down};
    for (int j = 0; j < 4; ++j) L.qw[j] = t[j]->q, L.scales[j] = t[j]->scales, L.biases[j] = t[j]->biases;
    L.norm[0] = lw.attn_norm, L.norm[1] = lw.mlp_norm;
    L.q_norm = sh.qk_norm ? lw.q_norm : nullptr, L.k_norm = sh.qk_norm ? lw.k_norm : nullptr;
  }
  fp->lm_qw = m->w.lm_head.q, fp->lm_scales = m->w.lm_head.scales, fp->lm_biases = m->w.lm_head.biases;
  fp->final_norm = m->w.final_norm;
  auto dims = [&](int kind, int type, int N, int K, int epi) {
    FusedDims& D = fp->dims[kind];
    D.type = type, D.epi = epi, D.N = N, D.K = K, D.norm = 0, D.pad = 0, D.ntiles = 0, D.S = 0;
    if (type == PH_GEMM) {
      const FusedGemmDims d = fused_dims(N, K, epi);
      D.ntiles = d.ntiles, D.S = d.S;
    }
  };
  dims(0, PH_EMBED, 0, H, 0);
  dims(1, PH_NORM, 0, H, 0);
  dims(2, PH_GEMM, nqkv, H, EPI_BF16);
  dims(3, PH_ATTN, 0, 0, 0);
  dims(4, PH_GEMM, H, qdim, EPI_RESIDUAL);
  dims(5, PH_NORM, 0, H, 0);
  dims(6, PH_GEMM, 2 * I, H, EPI_SILU_PACK);
  dims(7, PH_GEMM, H, I, EPI_RESIDUAL);
  dims(8, PH_NORM, 0, H, 0);
  dims(9, PH_GEMM, V, H, EPI_F32);
  fp->n_phases = lay.f_n_phases;
  fp->H = H, fp->nq = nq, fp->nkv = nkv, fp->V = V, fp->eps = sh.rms_eps;
  fp->rope = m->w.rope_cos_sin;
  fp->embed_q = m->w.embed.q, fp->embed_s = m->w.embed.scales, fp->embed_b = m->w.embed.biases;
  fp->x = reinterpret_cast<uint16_t*>(m->ws + lay.x), fp->y = reinterpret_cast<uint16_t*>(m->ws + lay.yp);
  fp->h = reinterpret_cast<uint16_t*>(m->ws + lay.f_h), fp->qkv = reinterpret_cast<uint16_t*>(m->ws + lay.qkv);
  fp->attn = reinterpret_cast<uint16_t*>(m->ws + lay.f_attn);
  fp->ss = reinterpret_cast<float*>(m->ws + lay.f_ss);
  fp->pacc = reinterpret_cast<float*>(m->ws + lay.f_pacc), fp->pml = reinterpret_cast<float*>(m->ws + lay.f_pml);
  fp->attn_counters = reinterpret_cast<int*>(m->ws + lay.f_attn_counters);
  fp->amax = reinterpret_cast<float2*>(m->ws + lay.f_amax);
  fp->control = reinterpret_cast<unsigned int*>(m->ws + lay.f_control);
}

// Reports a wait that gave up inside a kernel of an earlier step (a grid barrier of the persistent kernel, a bulk
// copy of the projection kernel) once the step's status word has come back.
int fused_check_status(q4d_model* m, bool wait) {
  if (m->timed_out)
    return fail(Q4D_ERR_TIMEOUT, "decode_step: a bounded wait inside a kernel of an earlier step gave up; destroy and re-create the model");
  if (!m->status_pending) return Q4D_OK;
  cudaError_t e = wait ? cudaEventSynchronize(m->status_done) : cudaEventQuery(m->status_done);
  if (e == cudaErrorNotReady) return Q4D_OK;
  if (e != cudaSuccess) return fail_cuda(e, "status read-back");
  m->status_pending = false;
  if (*m->host_status != 0u) m->timed_out = true;
  if (m->timed_out)
    return fail(Q4D_ERR_TIMEOUT, "decode_step: a bounded wait inside a kernel of an earlier step gave up; destroy and re-create the model");
  return Q4D_OK;
}

int run_fused(q4d_model* m, q4d_kv_pool* pool, int n, const int32_t* lens, const int32_t* d_tokens, const int32_t* d_bt,
              int32_t* next_dev, float* logits_dev, cudaStream_t s, int layer_begin, int layer_end, const uint16_t* x_in,
              uint16_t* x_out, bool ranged) {
  const q4d_shape& sh = m->sh;
  const Workspace& lay = m->lay;
  FusedStep& fp = *m->fused_params;  // the model's template; the per-step fields are filled in below
  fp.n = n, fp.tokens = d_tokens, fp.bt = d_bt, fp.max_blocks = m->ml.max_blocks_cap;
  // attention plan: equal chunks of whole blocks, at most one (request, chunk, kv head) item per warp of the grid
  const int W = m->fused_ctas * (kFusedThreads / 32), nkv = sh.n_kv_heads;
  long long total = 0;
  int nb[kMaxBatch], maxnb = 1;
  for (int r = 0; r < n; ++r) {
    fp.lens[r] = lens[r];
    nb[r] = (lens[r] + 1 + kBlockSize - 1) / kBlockSize;
    total += nb[r];
    maxnb = std::max(maxnb, nb[r]);
  }
  int C = (int)std::max<long long>(1, (total * nkv + W - 1) / W);
  for (;; ++C) {
    long long items = 0;
    for (int r = 0; r < n; ++r) items += (long long)((nb[r] + C - 1) / C) * nkv;
    if (items <= W || C >= maxnb) break;
  }
  fp.chunk_blocks = C;
  fp.item_prefix[0] = 0;
  for (int r = 0; r < n; ++r) {
    fp.nch[r] = (nb[r] + C - 1) / C;
    fp.item_prefix[r + 1] = fp.item_prefix[r] + fp.nch[r] * nkv;
  }
  for (int r = n; r < kMaxBatch; ++r) fp.item_prefix[r + 1] = fp.item_prefix[n];
  fp.n_items = fp.item_prefix[n];
  if (fp.n_items > lay.f_max_items) return fail(Q4D_ERR_WORKSPACE_TOO_SMALL, "decode_step: split-KV scratch too small");
  fp.pool = pool->mem;
  fp.layer_elems = (size_t)pool->num_blocks * nkv * kBlockSize * kHeadDim;
  fp.next = next_dev, fp.logits = logits_dev;
  fp.timeline = m->timeline ? at<unsigned long long>(m, lay.f_timeline) : nullptr;

  auto launch = [&](int ph_begin, int ph_end, int from_x) -> int {
    fp.ph_begin = ph_begin, fp.ph_end = ph_end, fp.embed_from_x = from_x;
    cudaError_t e = cudaMemsetAsync(fp.control, 0, sizeof(unsigned int), s);  // barrier arrivals; the status word stays
    if (e != cudaSuccess) return fail_cuda(e, "barrier reset");
    e = timed(m, Q4D_K_FUSED_STEP, s, [&]() -> cudaError_t { return launch_fused_step(fp, m->fused_ctas, s); });
    return e == cudaSuccess ? Q4D_OK : fail_cuda(e, "fused step launch");
  };
  int rc = Q4D_OK;
  if (!ranged) {
    rc = launch(0, lay.f_n_phases, 0);
  } else {
    cudaError_t ce = cudaMemcpyAsync(fp.x, x_in, (size_t)n * sh.hidden * 2, cudaMemcpyDeviceToDevice, s);
    if (ce != cudaSuccess) return fail_cuda(ce, "hidden state copy");
    rc = launch(0, 1, 1);  // sums of squares of the given hidden state
    if (rc == Q4D_OK && layer_end > layer_begin) rc = launch(1 + kFusedPhasesPerLayer * layer_begin, 1 + kFusedPhasesPerLayer * layer_end, 0);
    if (rc != Q4D_OK) return rc;
    ce = cudaMemcpyAsync(x_out, fp.x, (size_t)n * sh.hidden * 2, cudaMemcpyDeviceToDevice, s);
    if (ce != cudaSuccess) return fail_cuda(ce, "hidden state copy");
  }
  if (rc != Q4D_OK) return rc;
  if (!m->status_pending) {
    cudaError_t e = cudaMemcpyAsync(m->host_status, fp.control + 1, sizeof(uint32_t), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaEventRecord(m->status_done, s);
    if (e != cudaSuccess) return fail_cuda(e, "status read-back");
    m->status_pending = true;
  }
  return Q4D_OK;
}

// The launch sequence of a step.  A whole step embeds the tokens, runs every layer and the head, and advances the
// requests.  The parity export runs only layers [layer_begin, layer_end) from a given hidden state (x_in) and
// returns the hidden state (x_out) without advancing anything.
struct LayerRange {
  int begin, end;
  const uint16_t* x_in;
  uint16_t* x_out;
};

// Prompt processing: the n rows of the launch sequence are n consecutive tokens of ONE request, row r at position
// start + r, all reading the same block table.  K, V of the rows are appended by a kernel of their own before the
// attention kernel runs (a row attends to the rows before it), and only the last chunk of a prompt needs the head.
struct PrefillRows {
  int start;
  bool want_head;
};

int step_impl(q4d_model* m, q4d_kv_pool* pool, int32_t n, const int64_t* ids, const int32_t* tokens_host,
              const int32_t* tokens_dev, const int32_t* bt, int32_t max_blocks, int32_t* next_dev, float* logits_dev,
              cudaStream_t s, const LayerRange* range = nullptr, const PrefillRows* pf = nullptr) {
  if (!m || !pool || pool->model != m) return fail(Q4D_ERR_INVALID_ARG, "decode_step: model/pool mismatch or NULL");
  if (n < 0) return fail(Q4D_ERR_INVALID_ARG, "decode_step: n < 0");
  if (n == 0) return Q4D_OK;
  if (n > m->sh.max_batch)
    return fail(Q4D_ERR_BATCH_TOO_LARGE, "decode_step: n = %d exceeds max_batch %d", n, m->sh.max_batch);
  if ((!ids && !pf) || !bt || max_blocks < 1 || (!range && ((!tokens_host && !tokens_dev) || !next_dev)))
    return fail(Q4D_ERR_INVALID_ARG, "decode_step: NULL argument");
  const q4d_shape& sh = m->sh;
  {
    const int rc = fused_check_status(m, false);
    if (rc != Q4D_OK) return rc;
  }

  // ---- validate on the host; nothing is changed before this block passes ----
  int32_t lens[kMaxBatch];
  if (pf) {  // validated by the caller (q4d_prefill): one request, consecutive positions
    for (int r = 0; r < n; ++r) lens[r] = pf->start + r;
  } else {
    std::unordered_set<int64_t> seen;
    for (int r = 0; r < n; ++r) {
      const long long id = (long long)ids[r];
      if (!seen.insert(ids[r]).second)
        return fail(Q4D_ERR_DUPLICATE_REQUEST, "decode_step: request %lld listed twice", id);
      auto it = pool->lens.find(ids[r]);
      if (it == pool->lens.end())
        return fail(Q4D_ERR_UNKNOWN_REQUEST, "decode_step: request %lld was not admitted", id);
      lens[r] = it->second;
      if (lens[r] + 1 > sh.max_positions)
        return fail(Q4D_ERR_POSITION_OVERFLOW, "decode_step: request %lld is at max_positions", id);
      const int need = (lens[r] + 1 + kBlockSize - 1) / kBlockSize;
      if (need > max_blocks)
        return fail(Q4D_ERR_BLOCK_TABLE_TOO_SHORT, "decode_step: request %lld needs %d blocks, table has %d", id, need,
                    max_blocks);
      for (int i = 0; i < need; ++i) {
        const int b = bt[(size_t)r * max_blocks + i];
        if (b < 0 || b >= pool->num_blocks)
          return fail(Q4D_ERR_BLOCK_OUT_OF_RANGE, "decode_step: request %lld block %d = %d outside the pool", id, i, b);
      }
      if (tokens_host && (tokens_host[r] < 0 || tokens_host[r] >= sh.vocab))
        return fail(Q4D_ERR_INVALID_ARG, "decode_step: token %d outside the vocabulary", tokens_host[r]);
    }
  }

  // ---- per-step metadata: stage in pinned memory, copy to the device ----
  const MetaLayout& ml = m->ml;
  const int slot = m->staging_next;
  m->staging_next = (slot + 1) % kStagingSlots;
  if (m->staging_used[slot]) {
    cudaError_t e = cudaEventSynchronize(m->staging_done[slot]);
    if (e != cudaSuccess) return fail_cuda(e, "staging wait");
  }
  unsigned char* st = m->staging[slot];
  int32_t* h_tokens = reinterpret_cast<int32_t*>(st + ml.off_tokens);
  int32_t* h_lens = reinterpret_cast<int32_t*>(st + ml.off_lens);
  int32_t* h_slot = reinterpret_cast<int32_t*>(st + ml.off_slot_base);
  int32_t* h_nch = reinterpret_cast<int32_t*>(st + ml.off_nchunks);
  int4* h_work = reinterpret_cast<int4*>(st + ml.off_work);
  int32_t* h_bt = reinterpret_cast<int32_t*>(st + ml.off_bt);
  for (int r = 0; r < n; ++r) {
    h_tokens[r] = tokens_host ? tokens_host[r] : 0;
    h_lens[r] = lens[r];
    const int need = (lens[r] + 1 + kBlockSize - 1) / kBlockSize;  // <= max_blocks_cap since len < max_positions
    const int32_t* bt_row = bt + (pf ? 0 : (size_t)r * max_blocks);
    for (int i = 0; i < ml.max_blocks_cap; ++i) h_bt[(size_t)r * ml.max_blocks_cap + i] = i < need ? bt_row[i] : 0;
  }
  AttnPlan plan = {0, 0, 0};  // the whole-step kernel plans its attention items from the lengths alone
  if (!m->fused || pf) plan = plan_attention(lens, n, sh.n_kv_heads, 0, attention_wave_ctas(sh.n_q_heads, sh.n_kv_heads), h_work, h_slot, h_nch, ml.max_work);
  unsigned char* dmeta = m->ws + m->lay.meta;
  const size_t head_bytes = ml.off_work + (size_t)plan.n_work * sizeof(int4);
  const size_t bt_bytes = (size_t)n * ml.max_blocks_cap * 4;
  cudaError_t e = cudaMemcpyAsync(dmeta, st, head_bytes, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(dmeta + ml.off_bt, st + ml.off_bt, bt_bytes, cudaMemcpyHostToDevice, s);
  if (e != cudaSuccess) return fail_cuda(e, "metadata copy");
  cudaEventRecord(m->staging_done[slot], s);
  m->staging_used[slot] = true;
  m->last_h2d = (int64_t)(head_bytes + bt_bytes);
  m->last_d2h = 0;

  const int32_t* d_tokens = tokens_dev ? tokens_dev : reinterpret_cast<const int32_t*>(dmeta + ml.off_tokens);
  const int32_t* d_lens = reinterpret_cast<const int32_t*>(dmeta + ml.off_lens);
  const int32_t* d_bt = reinterpret_cast<const int32_t*>(dmeta + ml.off_bt);

  if (m->fused && !pf) {
    const int rc = run_fused(m, pool, n, lens, d_tokens, d_bt, next_dev, logits_dev, s, range ? range->begin : 0,
                             range ? range->end : 0, range ? range->x_in : nullptr, range ? range->x_out : nullptr,
                             range != nullptr);
    if (rc != Q4D_OK || range) return rc;
    for (int r = 0; r < n; ++r) pool->lens[ids[r]] = lens[r] + 1;
    return Q4D_OK;
  }

  // ---- the launch sequence ----
  const int H = sh.hidden, nq = sh.n_q_heads, nkv = sh.n_kv_heads, I = sh.mlp_inter, V = sh.vocab;
  const int nqkv = (nq + 2 * nkv) * kHeadDim;
  uint16_t* x = at<uint16_t>(m, m->lay.x);
  uint16_t* yp = at<uint16_t>(m, m->lay.yp);
  float* ys = at<float>(m, m->lay.ys);
  uint16_t* qkv = at<uint16_t>(m, m->lay.qkv);
  uint16_t* qbuf = at<uint16_t>(m, m->lay.qbuf);
  uint16_t* ap = at<uint16_t>(m, m->lay.ap);
  float* as = at<float>(m, m->lay.as);
  uint16_t* hp = at<uint16_t>(m, m->lay.hp);
  float* hs = at<float>(m, m->lay.hs);
  float2* amax = at<float2>(m, m->lay.amax);
  float* logits = logits_dev ? logits_dev : at<float>(m, m->lay.logits);
  const size_t layer_elems = (size_t)pool->num_blocks * nkv * kBlockSize * kHeadDim;
  const int qdim = nq * kHeadDim;
  const int dense_layout = gemm_operand_layout(false, n);  // of the operands of the dense projections

#define Q4D_LAUNCH(cls, expr)                                                 \
  do {                                                                        \
    cudaError_t le = timed(m, cls, s, [&]() -> cudaError_t { return expr; }); \
    if (le != cudaSuccess) return fail_cuda(le, #cls);                        \
  } while (0)

  if (sh.n_experts) {  // the step's count of routed experts starts at zero
    cudaError_t ce = cudaMemsetAsync(at<int32_t>(m, m->lay.m_ints) + 3 * sh.n_experts + 2, 0, 4, s);
    if (ce != cudaSuccess) return fail_cuda(ce, "routed-expert counter reset");
  }
  if (range) {
    cudaError_t ce = cudaMemcpyAsync(x, range->x_in, (size_t)n * H * 2, cudaMemcpyDeviceToDevice, s);
    if (ce != cudaSuccess) return fail_cuda(ce, "hidden state copy");
  } else {
    Q4D_LAUNCH(Q4D_K_EMBED, launch_embed(m->w.embed.q, m->w.embed.scales, m->w.embed.biases, V, H, d_tokens, n, x, s));
  }
  for (int l = range ? range->begin : 0; l < (range ? range->end : sh.n_layers); ++l) {
    const q4d_layer_weights& lw = m->layers[l];
    uint16_t* kpool = pool->mem + (size_t)(2 * l) * layer_elems;
    uint16_t* vpool = kpool + layer_elems;
    Q4D_LAUNCH(Q4D_K_RMSNORM, launch_rmsnorm(x, lw.attn_norm, sh.rms_eps, n, H, nullptr, yp, ys, dense_layout, s));
    Q4D_LAUNCH(Q4D_K_GEMM_QKV, launch_q4_gemm(gemm_args(m, lw.wqkv, nqkv, H, yp, ys, n, EPI_BF16, qkv, nqkv), s));
    AttnArgs aa;
    aa.q = qbuf, aa.kpool = kpool, aa.vpool = vpool, aa.block_tables = d_bt, aa.lens = d_lens;
    aa.work = reinterpret_cast<const int4*>(dmeta + ml.off_work);
    aa.slot_base = reinterpret_cast<const int32_t*>(dmeta + ml.off_slot_base);
    aa.nchunks = reinterpret_cast<const int32_t*>(dmeta + ml.off_nchunks);
    aa.n_work = plan.n_work, aa.n = n, aa.nq = nq, aa.nkv = nkv, aa.max_blocks = ml.max_blocks_cap;
    aa.part_acc = at<float>(m, m->lay.part_acc), aa.part_ml = at<float>(m, m->lay.part_ml);
    aa.out = nullptr, aa.out_xp = ap, aa.out_xs = as, aa.out_layout = dense_layout;
    aa.merge_counters = at<int>(m, m->lay.attn_merge_counters);  // the last CTA of a (request, kv head) merges its chunks
    // q preparation (qk-norm, rotary embedding) and the append of k, v happen inside the attention kernel
    aa.qkv = qkv, aa.q_norm = sh.qk_norm ? lw.q_norm : nullptr, aa.k_norm = sh.qk_norm ? lw.k_norm : nullptr;
    aa.eps = sh.rms_eps, aa.rope = m->w.rope_cos_sin, aa.kpool_w = kpool, aa.vpool_w = vpool;
    if (pf) {
      // prompt rows: append k, v of all rows first; the attention kernel then starts after that kernel has ended
      RopeArgs ra;
      ra.qkv = qkv, ra.q_norm = aa.q_norm, ra.k_norm = aa.k_norm, ra.eps = sh.rms_eps, ra.rope = m->w.rope_cos_sin;
      ra.n = n, ra.nq = nq, ra.nkv = nkv, ra.lens = d_lens, ra.block_tables = d_bt, ra.max_blocks = ml.max_blocks_cap;
      ra.kpool = kpool, ra.vpool = vpool, ra.q_out = qbuf;
      Q4D_LAUNCH(Q4D_K_ROPE_APPEND, launch_rope_append(ra, s));
      aa.qkv = nullptr, aa.after_predecessor = true;
    }
    Q4D_LAUNCH(Q4D_K_ATTENTION, launch_paged_attention(aa, s));
    Q4D_LAUNCH(Q4D_K_GEMM_O, launch_q4_gemm(gemm_args(m, lw.wo, H, qdim, ap, as, n, EPI_RESIDUAL, x, H), s));
    if (sh.n_experts == 0) {
      Q4D_LAUNCH(Q4D_K_RMSNORM, launch_rmsnorm(x, lw.mlp_norm, sh.rms_eps, n, H, nullptr, yp, ys, dense_layout, s));
      GemmArgs gu = gemm_args(m, lw.w_gate_up, 2 * I, H, yp, ys, n, EPI_SILU_PACK, nullptr, 0);
      gu.out_xp = hp, gu.out_xs = hs;
      Q4D_LAUNCH(Q4D_K_GEMM_GATE_UP, launch_q4_gemm(gu, s));
      Q4D_LAUNCH(Q4D_K_GEMM_DOWN, launch_q4_gemm(gemm_args(m, lw.w_down, H, I, hp, dense_layout == OPERAND_BLOCKED ? hs : nullptr, n, EPI_RESIDUAL, x, H), s));
    } else {
      const int E = sh.n_experts, Ie = sh.expert_inter;
      uint16_t* yplain = at<uint16_t>(m, m->lay.yplain);
      int32_t* ints = at<int32_t>(m, m->lay.m_ints);
      MoeRouteArgs mr;
      mr.y = yplain, mr.router = lw.router, mr.H = H, mr.E = E, mr.top_k = sh.top_k, mr.norm = sh.norm_topk_prob;
      mr.idx = at<int32_t>(m, m->lay.m_idx), mr.wgt = at<float>(m, m->lay.m_wgt);
      mr.flags = ints, mr.expert_ids = ints + E, mr.slot_of = ints + 2 * E, mr.counter = ints + 3 * E;
      mr.n_touched = ints + 3 * E + 1;
      mr.touched_total = ints + 3 * E + 2;
      mr.slice_counter = ints + 3 * E + 3;
      mr.logits = reinterpret_cast<float*>(ints + 3 * E + 3 + kMaxBatch);
      uint16_t* ehp = at<uint16_t>(m, m->lay.m_hp);
      float* ehs = at<float>(m, m->lay.m_hs);
      uint16_t* eo = at<uint16_t>(m, m->lay.m_o);
      Q4D_LAUNCH(Q4D_K_RMSNORM, launch_rmsnorm(x, lw.mlp_norm, sh.rms_eps, n, H, yplain, yp, ys, gemm_operand_layout(true, n), s));
      Q4D_LAUNCH(Q4D_K_MOE_ROUTER, launch_moe_router(mr, n, s));
      GemmArgs gu = gemm_args(m, lw.experts_gate_up, 2 * Ie, H, yp, ys, n, EPI_SILU_PACK, nullptr, 0);
      gu.out_xp = ehp, gu.out_xs = ehs;
      gu.expert_ids = mr.expert_ids, gu.n_touched = mr.n_touched, gu.max_slots = E;
      gu.out_slot_stride = (size_t)16 * Ie, gu.out_xs_slot_stride = (size_t)(Ie / 64) * 16;
      Q4D_LAUNCH(Q4D_K_MOE_GATE_UP, launch_q4_gemm(gu, s));
      GemmArgs dn = gemm_args(m, lw.experts_down, H, Ie, ehp, ehs, n, EPI_BF16, eo, H);
      dn.expert_ids = mr.expert_ids, dn.n_touched = mr.n_touched, dn.max_slots = E;
      dn.xp_slot_stride = (size_t)16 * Ie, dn.xs_slot_stride = (size_t)(Ie / 64) * 16;
      dn.out_slot_stride = (size_t)16 * H;
      Q4D_LAUNCH(Q4D_K_MOE_DOWN, launch_q4_gemm(dn, s));
      MoeCombineArgs mc;
      mc.x = x, mc.o = eo, mc.idx = mr.idx, mc.wgt = mr.wgt, mc.slot_of = mr.slot_of, mc.H = H, mc.top_k = sh.top_k;
      Q4D_LAUNCH(Q4D_K_MOE_DOWN, launch_moe_combine(mc, n, s));
    }
  }
  if (range) {
    cudaError_t ce = cudaMemcpyAsync(range->x_out, x, (size_t)n * H * 2, cudaMemcpyDeviceToDevice, s);
    return ce == cudaSuccess ? Q4D_OK : fail_cuda(ce, "hidden state copy");
  }
  if (pf && !pf->want_head) return Q4D_OK;  // an inner chunk of a prompt: its K, V are in the pool, nothing else is needed
  Q4D_LAUNCH(Q4D_K_RMSNORM, launch_rmsnorm(x, m->w.final_norm, sh.rms_eps, n, H, nullptr, yp, ys, dense_layout, s));
  GemmArgs lm = gemm_args(m, m->w.lm_head, V, H, yp, ys, n, EPI_F32, logits, V);
  lm.argmax_partial = amax;
  const int lm_blocks = gemm_row_blocks(V, H, n, EPI_F32);
  if (lm_blocks > m->lay.amax_blocks) return fail(Q4D_ERR_WORKSPACE_TOO_SMALL, "decode_step: argmax scratch too small");
  Q4D_LAUNCH(Q4D_K_LM_HEAD, launch_q4_gemm(lm, s));
  Q4D_LAUNCH(Q4D_K_ARGMAX, launch_argmax_finish(amax, lm_blocks, n, next_dev, s));
#undef Q4D_LAUNCH
  if (!m->status_pending) {
    cudaError_t se = cudaMemcpyAsync(m->host_status, m->ws + m->lay.chain_status, sizeof(uint32_t), cudaMemcpyDeviceToHost, s);
    if (se == cudaSuccess) se = cudaEventRecord(m->status_done, s);
    if (se != cudaSuccess) return fail_cuda(se, "status read-back");
    m->status_pending = true;
  }

  if (!pf)
    for (int r = 0; r < n; ++r) pool->lens[ids[r]] = lens[r] + 1;
  return Q4D_OK;
}

}  // namespace

namespace q4d {
void set_pdl_enabled(bool on) { g_pdl = on; }
bool pdl_enabled() { return g_pdl; }
}  // namespace q4d

extern "C" {

const char* q4d_last_error(void) { return g_last_error.c_str(); }

// Lets the other translation units of the library record an error message.
int q4d_internal_fail(int code, const char* msg) { return fail(code, "%s", msg); }

size_t q4d_model_workspace_bytes(const q4d_shape* shape) {
  std::string why;
  if (!shape || !shape_supported(*shape, &why)) {
    fail(Q4D_ERR_UNSUPPORTED, "workspace_bytes: %s", shape ? why.c_str() : "NULL shape");
    return 0;
  }
  MetaLayout ml;
  ml.init(shape->max_positions);
  return carve(*shape, ml).bytes;
}

int q4d_model_create(const q4d_shape* shape, const q4d_weights* weights, void* workspace, size_t workspace_bytes,
                     q4d_model** out) {
  if (!shape || !weights || !workspace || !out) return fail(Q4D_ERR_INVALID_ARG, "model_create: NULL argument");
  std::string why;
  if (!shape_supported(*shape, &why)) return fail(Q4D_ERR_UNSUPPORTED, "model_create: %s", why.c_str());
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign)
    return fail(Q4D_ERR_INVALID_ARG, "model_create: workspace must be 256-byte aligned");
  if (!weights->layers || !weights->final_norm || !weights->rope_cos_sin || !qt_ok(weights->embed) ||
      !qt_ok(weights->lm_head))
    return fail(Q4D_ERR_INVALID_ARG, "model_create: missing tensor");
  for (int l = 0; l < shape->n_layers; ++l) {
    const q4d_layer_weights& lw = weights->layers[l];
    const bool mlp_ok = shape->n_experts ? (lw.router && qt_ok(lw.experts_gate_up) && qt_ok(lw.experts_down))
                                         : (qt_ok(lw.w_gate_up) && qt_ok(lw.w_down));
    if (!lw.attn_norm || !lw.mlp_norm || !qt_ok(lw.wqkv) || !qt_ok(lw.wo) || !mlp_ok ||
        (shape->qk_norm && (!lw.q_norm || !lw.k_norm)))
      return fail(Q4D_ERR_INVALID_ARG, "model_create: layer %d has a missing tensor", l);
  }
  MetaLayout ml;
  ml.init(shape->max_positions);
  if (const char* v = getenv("Q4D_NO_PDL")) set_pdl_enabled(v[0] == '0');
  cudaError_t e = gemm_init();
  if (e == cudaSuccess) e = attention_init();
  if (e != cudaSuccess) return fail_cuda(e, "kernel init");
  const Workspace lay = carve(*shape, ml);
  if (workspace_bytes < lay.bytes)
    return fail(Q4D_ERR_WORKSPACE_TOO_SMALL, "model_create: workspace %zu < %zu", workspace_bytes, lay.bytes);
  q4d_model* m = new (std::nothrow) q4d_model();
  if (!m) return fail(Q4D_ERR_INVALID_ARG, "model_create: out of host memory");
  m->sh = *shape;
  m->layers.assign(weights->layers, weights->layers + shape->n_layers);
  m->w = *weights;
  m->w.layers = m->layers.data();
  m->ws = static_cast<unsigned char*>(workspace);
  m->lay = lay;
  m->ml = ml;
  m->profile = false;
  m->launches = 0;
  m->last_h2d = m->last_d2h = 0;
  m->staging_next = 0;
  m->host_next = nullptr;
  m->fused = false, m->fused_ctas = 0, m->timeline = false, m->fused_params = nullptr;
  m->host_status = nullptr, m->status_done = nullptr, m->status_pending = false, m->timed_out = false;
  int dev = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&m->sm_count, cudaDevAttrMultiProcessorCount, dev);
  for (int i = 0; i < kStagingSlots; ++i)
    m->staging[i] = nullptr, m->staging_done[i] = nullptr, m->staging_used[i] = false;
  for (int i = 0; i < kStagingSlots && e == cudaSuccess; ++i) {
    e = cudaMallocHost(reinterpret_cast<void**>(&m->staging[i]), ml.bytes);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&m->staging_done[i], cudaEventDisableTiming);
  }
  if (e == cudaSuccess) e = cudaMallocHost(reinterpret_cast<void**>(&m->host_next), kMaxBatch * sizeof(int32_t));
  if (e == cudaSuccess) e = cudaMemset(m->ws + lay.counters, 0, (size_t)lay.counters_len * 4);
  if (e == cudaSuccess) e = cudaMemset(m->ws + lay.attn_merge_counters, 0, (size_t)16 * shape->n_kv_heads * 4);
  if (e == cudaSuccess && shape->n_experts)
    e = cudaMemset(m->ws + lay.m_ints, 0, (3 * (size_t)shape->n_experts + 3 + kMaxBatch) * 4);
  if (e == cudaSuccess) e = cudaMemset(m->ws + lay.chain_status, 0, 256);
  if (e == cudaSuccess) e = cudaMallocHost(reinterpret_cast<void**>(&m->host_status), sizeof(uint32_t));
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&m->status_done, cudaEventDisableTiming);
  if (e == cudaSuccess) *m->host_status = 0u;
  // The step runs as a chain of kernels (one per operation, programmatic dependent launches).  Dense models with at
  // most 8 query heads per kv head can instead run the whole step as one persistent kernel: Q4D_STEP_KERNEL=fused at
  // model creation.  On B200 the chain is the faster of the two, so it is the default.
  const char* step_kernel = getenv("Q4D_STEP_KERNEL");
  const bool want_fused = step_kernel && strcmp(step_kernel, "fused") == 0;
  const bool narrow_gqa = shape->n_q_heads / shape->n_kv_heads <= 8;
  if (e == cudaSuccess && want_fused && !shape->n_experts && narrow_gqa) {
    int max_ctas = 0;
    e = fused_init(&max_ctas);
    if (e == cudaSuccess && max_ctas > 0 && max_ctas <= lay.f_max_ctas && shape->n_layers <= kFusedMaxLayers) {
      m->fused = true;
      m->fused_ctas = max_ctas;
      m->fused_params = new (std::nothrow) FusedStep;
      if (!m->fused_params) {
        q4d_model_destroy(m);
        return fail(Q4D_ERR_INVALID_ARG, "model_create: out of host memory");
      }
      build_fused_params(m, m->fused_params);
      if (e == cudaSuccess) e = cudaMemset(m->ws + lay.f_attn_counters, 0, (size_t)16 * shape->n_kv_heads * 4);
      if (e == cudaSuccess) e = cudaMemset(m->ws + lay.f_control, 0, 256);
    }
  }
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) {
    q4d_model_destroy(m);
    return fail_cuda(e, "model_create");
  }
  *out = m;
  return Q4D_OK;
}

int q4d_model_destroy(q4d_model* m) {
  if (!m) return Q4D_OK;
  for (int i = 0; i < kStagingSlots; ++i) {
    if (m->staging[i]) cudaFreeHost(m->staging[i]);
    if (m->staging_done[i]) cudaEventDestroy(m->staging_done[i]);
  }
  if (m->host_next) cudaFreeHost(m->host_next);
  delete m->fused_params;
  if (m->host_status) cudaFreeHost(m->host_status);
  if (m->status_done) cudaEventDestroy(m->status_done);
  for (auto& r : m->prof_recs) cudaEventDestroy(r.a), cudaEventDestroy(r.b);
  for (auto ev : m->prof_free) cudaEventDestroy(ev);
  delete m;
  return Q4D_OK;
}

size_t q4d_kv_pool_bytes(const q4d_shape* shape, int32_t num_blocks, int32_t block_size) {
  if (!shape || num_blocks < 1 || block_size != kBlockSize) return 0;
  return (size_t)shape->n_layers * 2 * num_blocks * shape->n_kv_heads * block_size * shape->head_dim * 2;
}

int q4d_kv_pool_create(q4d_model* model, int32_t num_blocks, int32_t block_size, void* pool_mem, size_t pool_bytes,
                       q4d_kv_pool** out) {
  if (!model || !pool_mem || !out) return fail(Q4D_ERR_INVALID_ARG, "kv_pool_create: NULL argument");
  if (block_size != kBlockSize) return fail(Q4D_ERR_UNSUPPORTED, "kv_pool_create: block_size must be 16");
  if (num_blocks < 1) return fail(Q4D_ERR_INVALID_ARG, "kv_pool_create: num_blocks < 1");
  if (reinterpret_cast<uintptr_t>(pool_mem) % 16)
    return fail(Q4D_ERR_INVALID_ARG, "kv_pool_create: pool must be 16-byte aligned");
  const size_t need = q4d_kv_pool_bytes(&model->sh, num_blocks, block_size);
  if (pool_bytes < need) return fail(Q4D_ERR_INVALID_ARG, "kv_pool_create: pool %zu < %zu bytes", pool_bytes, need);
  q4d_kv_pool* p = new (std::nothrow) q4d_kv_pool();
  if (!p) return fail(Q4D_ERR_INVALID_ARG, "kv_pool_create: out of host memory");
  p->model = model, p->num_blocks = num_blocks, p->mem = static_cast<uint16_t*>(pool_mem);
  *out = p;
  return Q4D_OK;
}

int q4d_kv_pool_destroy(q4d_kv_pool* p) {
  delete p;
  return Q4D_OK;
}

int q4d_request_admit(q4d_kv_pool* p, int64_t id, int32_t prefilled_len) {
  if (!p) return fail(Q4D_ERR_INVALID_ARG, "request_admit: NULL pool");
  if (prefilled_len < 0 || prefilled_len >= p->model->sh.max_positions)
    return fail(Q4D_ERR_POSITION_OVERFLOW, "request_admit: prefilled_len %d outside [0, %d)", prefilled_len,
                p->model->sh.max_positions);
  if (p->lens.count(id))
    return fail(Q4D_ERR_DUPLICATE_REQUEST, "request_admit: request %lld already admitted", (long long)id);
  p->lens[id] = prefilled_len;
  return Q4D_OK;
}

int q4d_request_release(q4d_kv_pool* p, int64_t id) {
  if (!p) return fail(Q4D_ERR_INVALID_ARG, "request_release: NULL pool");
  if (!p->lens.erase(id))
    return fail(Q4D_ERR_UNKNOWN_REQUEST, "request_release: request %lld was not admitted", (long long)id);
  return Q4D_OK;
}

int q4d_request_len(q4d_kv_pool* p, int64_t id, int32_t* len_out) {
  if (!p || !len_out) return fail(Q4D_ERR_INVALID_ARG, "request_len: NULL argument");
  auto it = p->lens.find(id);
  if (it == p->lens.end())
    return fail(Q4D_ERR_UNKNOWN_REQUEST, "request_len: request %lld was not admitted", (long long)id);
  *len_out = it->second;
  return Q4D_OK;
}

int q4d_request_count(q4d_kv_pool* p, int32_t* count_out) {
  if (!p || !count_out) return fail(Q4D_ERR_INVALID_ARG, "request_count: NULL argument");
  *count_out = (int32_t)p->lens.size();
  return Q4D_OK;
}

int q4d_decode_step(q4d_model* m, q4d_kv_pool* pool, int32_t n, const int64_t* ids, const int32_t* last_tokens,
                    const int32_t* bt, int32_t max_blocks, int32_t* next_tokens, float* logits, void* stream) {
  if (n > 0 && !last_tokens) return fail(Q4D_ERR_INVALID_ARG, "decode_step: NULL last_tokens");
  return step_impl(m, pool, n, ids, last_tokens, nullptr, bt, max_blocks, next_tokens, logits,
                   static_cast<cudaStream_t>(stream));
}

namespace {
int fill_sample_args(const q4d_sampling* sp, int n, int vocab, SampleArgs* a) {
  if (!sp || !sp->temperature || !sp->top_k || !sp->top_p || !sp->u) return fail(Q4D_ERR_INVALID_ARG, "sampling: NULL argument");
  for (int r = 0; r < n; ++r) {
    if (!(sp->u[r] >= 0.0f && sp->u[r] < 1.0f)) return fail(Q4D_ERR_INVALID_ARG, "sampling: u[%d] outside [0, 1)", r);
    if (sp->temperature[r] > 0.0f && !(sp->top_p[r] > 0.0f)) return fail(Q4D_ERR_INVALID_ARG, "sampling: top_p[%d] must be positive", r);
    a->temperature[r] = sp->temperature[r], a->top_k[r] = sp->top_k[r], a->top_p[r] = sp->top_p[r], a->u[r] = sp->u[r];
  }
  for (int r = n; r < kMaxBatch; ++r) a->temperature[r] = 0.0f, a->top_k[r] = 0, a->top_p[r] = 1.0f, a->u[r] = 0.0f;
  a->vocab = vocab;
  return Q4D_OK;
}
}  // namespace

int q4d_decode_step_sampled(q4d_model* m, q4d_kv_pool* pool, int32_t n, const int64_t* ids, const int32_t* last_tokens,
                            const int32_t* bt, int32_t max_blocks, const q4d_sampling* sampling, int32_t* next_tokens,
                            float* logits, void* stream) {
  if (!m) return fail(Q4D_ERR_INVALID_ARG, "decode_step_sampled: NULL model");
  if (n > 0 && !last_tokens) return fail(Q4D_ERR_INVALID_ARG, "decode_step_sampled: NULL last_tokens");
  if (n < 0 || n > kMaxBatch) return fail(Q4D_ERR_BATCH_TOO_LARGE, "decode_step_sampled: n outside 0..16");
  SampleArgs sa;
  int rc = fill_sample_args(sampling, n, m->sh.vocab, &sa);
  if (rc != Q4D_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  float* lg = logits ? logits : at<float>(m, m->lay.logits);  // the draw reads the logits: they are always produced
  rc = step_impl(m, pool, n, ids, last_tokens, nullptr, bt, max_blocks, next_tokens, lg, s);
  if (rc != Q4D_OK || n == 0) return rc;
  sa.logits = lg, sa.next = next_tokens;
  cudaError_t e = launch_sample(sa, n, s);
  m->launches++;
  return e == cudaSuccess ? Q4D_OK : fail_cuda(e, "sample");
}

int q4d_sample(const float* logits, int32_t n, int32_t vocab, const q4d_sampling* sampling, int32_t* next, void* stream) {
  if (!logits || !next || n < 0 || n > kMaxBatch || vocab < 1) return fail(Q4D_ERR_INVALID_ARG, "sample: bad argument");
  SampleArgs sa;
  const int rc = fill_sample_args(sampling, n, vocab, &sa);
  if (rc != Q4D_OK) return rc;
  sa.logits = logits, sa.next = next;
  cudaError_t e = launch_sample(sa, n, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? Q4D_OK : fail_cuda(e, "sample");
}

int q4d_prefill(q4d_model* m, q4d_kv_pool* pool, int64_t request_id, const int32_t* tokens, int32_t n_tokens,
                int32_t start_pos, const int32_t* block_table, int32_t max_blocks, int32_t* next_token, float* logits,
                void* stream) {
  if (!m || !pool || pool->model != m) return fail(Q4D_ERR_INVALID_ARG, "prefill: model/pool mismatch or NULL");
  if (!tokens || !block_table || n_tokens < 1 || start_pos < 0 || start_pos >= n_tokens || max_blocks < 1)
    return fail(Q4D_ERR_INVALID_ARG, "prefill: need 0 <= start_pos < n_tokens and a block table");
  const q4d_shape& sh = m->sh;
  if (n_tokens >= sh.max_positions)
    return fail(Q4D_ERR_POSITION_OVERFLOW, "prefill: %d tokens do not leave a position to generate at (max_positions %d)",
                n_tokens, sh.max_positions);
  if (pool->lens.count(request_id))
    return fail(Q4D_ERR_DUPLICATE_REQUEST, "prefill: request %lld already admitted", (long long)request_id);
  const int need = (n_tokens + kBlockSize - 1) / kBlockSize;
  if (need > max_blocks)
    return fail(Q4D_ERR_BLOCK_TABLE_TOO_SHORT, "prefill: %d tokens need %d blocks, table has %d", n_tokens, need, max_blocks);
  for (int i = 0; i < need; ++i)
    if (block_table[i] < 0 || block_table[i] >= pool->num_blocks)
      return fail(Q4D_ERR_BLOCK_OUT_OF_RANGE, "prefill: block %d = %d outside the pool", i, block_table[i]);
  for (int t = start_pos; t < n_tokens; ++t)
    if (tokens[t] < 0 || tokens[t] >= sh.vocab) return fail(Q4D_ERR_INVALID_ARG, "prefill: token %d outside the vocabulary", tokens[t]);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int32_t* ws_next = at<int32_t>(m, m->lay.next);
  float* ws_logits = at<float>(m, m->lay.logits);
  int last_rows = 0;
  for (int c = start_pos; c < n_tokens; c += kMaxBatch) {
    const int n = std::min(kMaxBatch, n_tokens - c);
    const PrefillRows pf{c, c + n == n_tokens};
    const int rc = step_impl(m, pool, n, nullptr, tokens + c, nullptr, block_table, max_blocks, ws_next,
                             pf.want_head ? ws_logits : nullptr, s, nullptr, &pf);
    if (rc != Q4D_OK) return rc;
    last_rows = n;
  }
  cudaError_t e = cudaSuccess;
  if (next_token) e = cudaMemcpyAsync(next_token, ws_next + (last_rows - 1), sizeof(int32_t), cudaMemcpyDeviceToDevice, s);
  if (e == cudaSuccess && logits)
    e = cudaMemcpyAsync(logits, ws_logits + (size_t)(last_rows - 1) * sh.vocab, (size_t)sh.vocab * sizeof(float),
                        cudaMemcpyDeviceToDevice, s);
  if (e != cudaSuccess) return fail_cuda(e, "prefill outputs");
  pool->lens[request_id] = n_tokens;
  return Q4D_OK;
}

int q4d_decode_step_chained(q4d_model* m, q4d_kv_pool* pool, int32_t n, const int64_t* ids,
                            const int32_t* last_tokens_device, const int32_t* bt, int32_t max_blocks,
                            int32_t* next_tokens, float* logits, void* stream) {
  if (n > 0 && !last_tokens_device) return fail(Q4D_ERR_INVALID_ARG, "decode_step_chained: NULL last_tokens_device");
  return step_impl(m, pool, n, ids, nullptr, last_tokens_device, bt, max_blocks, next_tokens, logits,
                   static_cast<cudaStream_t>(stream));
}

int q4d_decode_step_host(q4d_model* m, q4d_kv_pool* pool, int32_t n, const int64_t* ids, const int32_t* last_tokens,
                         const int32_t* bt, int32_t max_blocks, int32_t* next_tokens_host, float* logits_host,
                         void* stream) {
  if (!m) return fail(Q4D_ERR_INVALID_ARG, "decode_step_host: NULL model");
  if (n > 0 && (!last_tokens || !next_tokens_host))
    return fail(Q4D_ERR_INVALID_ARG, "decode_step_host: NULL argument");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int32_t* d_next = at<int32_t>(m, m->lay.next);
  float* d_logits = (logits_host || !m->fused) ? at<float>(m, m->lay.logits) : nullptr;
  const int rc = step_impl(m, pool, n, ids, last_tokens, nullptr, bt, max_blocks, d_next, d_logits, s);
  if (rc != Q4D_OK || n == 0) return rc;
  cudaError_t e = cudaMemcpyAsync(m->host_next, d_next, (size_t)n * 4, cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess && logits_host)
    e = cudaMemcpyAsync(logits_host, d_logits, (size_t)n * m->sh.vocab * 4, cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return fail_cuda(e, "decode_step_host");
  {
    const int st = fused_check_status(m, true);
    if (st != Q4D_OK) return st;
  }
  memcpy(next_tokens_host, m->host_next, (size_t)n * 4);
  m->last_d2h = (int64_t)n * 4 + (logits_host ? (int64_t)n * m->sh.vocab * 4 : 0);
  return Q4D_OK;
}

int q4d_profile_enable(q4d_model* m, int32_t on) {
  if (!m) return fail(Q4D_ERR_INVALID_ARG, "profile_enable: NULL model");
  m->profile = on != 0;
  return Q4D_OK;
}

int q4d_profile_read(q4d_model* m, float* ms, int32_t* launches) {
  if (!m || !ms || !launches) return fail(Q4D_ERR_INVALID_ARG, "profile_read: NULL argument");
  for (int i = 0; i < Q4D_K_COUNT; ++i) ms[i] = 0.0f, launches[i] = 0;
  for (auto& r : m->prof_recs) {
    cudaError_t e = cudaEventSynchronize(r.b);
    float t = 0.0f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&t, r.a, r.b);
    if (e != cudaSuccess) return fail_cuda(e, "profile_read");
    ms[r.cls] += t;
    launches[r.cls] += 1;
    m->prof_free.push_back(r.a);
    m->prof_free.push_back(r.b);
  }
  m->prof_recs.clear();
  return Q4D_OK;
}

int64_t q4d_launch_count(q4d_model* m) { return m ? m->launches : 0; }

int q4d_step_is_fused(q4d_model* m) { return m && m->fused ? 1 : 0; }

int q4d_timeline_enable(q4d_model* m, int32_t on) {
  if (!m) return fail(Q4D_ERR_INVALID_ARG, "timeline_enable: NULL model");
  m->timeline = on != 0 && m->fused;
  return Q4D_OK;
}

int q4d_timeline_read(q4d_model* m, float* us, int32_t* phases) {
  if (!m || !us || !phases) return fail(Q4D_ERR_INVALID_ARG, "timeline_read: NULL argument");
  for (int i = 0; i < Q4D_K_COUNT; ++i) us[i] = 0.0f, phases[i] = 0;
  if (!m->fused) return Q4D_OK;
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return fail_cuda(e, "timeline_read");
  const int np = m->lay.f_n_phases;
  std::vector<unsigned long long> stamps(np + 1);
  e = cudaMemcpy(stamps.data(), m->ws + m->lay.f_timeline, stamps.size() * 8, cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return fail_cuda(e, "timeline_read");
  for (int i = 0; i < np; ++i) {
    const int c = kFusedKindClass[fused_kind(i, np)];
    if (stamps[i + 1] < stamps[i]) continue;
    us[c] += (float)((double)(stamps[i + 1] - stamps[i]) * 1e-3);
    phases[c] += 1;
  }
  return Q4D_OK;
}

int q4d_moe_touched_experts(q4d_model* m, int64_t* total) {
  if (!m || !total) return fail(Q4D_ERR_INVALID_ARG, "moe_touched_experts: NULL argument");
  *total = 0;
  if (!m->sh.n_experts) return Q4D_OK;
  int32_t v = 0;
  cudaError_t e = cudaDeviceSynchronize();
  if (e == cudaSuccess)
    e = cudaMemcpy(&v, at<int32_t>(m, m->lay.m_ints) + 3 * m->sh.n_experts + 2, 4, cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return fail_cuda(e, "moe_touched_experts");
  *total = v;
  return Q4D_OK;
}

int q4d_step_io_bytes(q4d_model* m, int64_t* h2d, int64_t* d2h) {
  if (!m || !h2d || !d2h) return fail(Q4D_ERR_INVALID_ARG, "step_io_bytes: NULL argument");
  *h2d = m->last_h2d, *d2h = m->last_d2h;
  return Q4D_OK;
}

// ---- single operations ------------------------------------------------------------

namespace {
constexpr size_t kOpCounters = 64 * 1024;  // bytes
constexpr size_t kOpGemmPartial = 48ull << 20;
constexpr size_t kOpAttnMeta = 1ull << 20;
constexpr size_t kOpPartAcc = 64ull << 20;
constexpr size_t kOpPartMl = 1ull << 20;
constexpr int kOpMaxK = 32768;                         // widest operand the pack buffers hold
constexpr size_t kOpPackXp = (size_t)16 * kOpMaxK * 2 + kOpMaxK;  // fragment-ordered operand, with the sliced layout's padding
constexpr size_t kOpPackXs = (size_t)(kOpMaxK / 64) * 16 * 4;
constexpr size_t kOpPackOff = kOpCounters + kOpGemmPartial + kOpAttnMeta + kOpPartAcc + kOpPartMl;
}  // namespace

size_t q4d_op_scratch_bytes(void) { return kOpPackOff + kOpPackXp + kOpPackXs; }

int q4d_q4_gemm(const q4d_qtensor* w, int32_t N, int32_t K, const uint16_t* x, int32_t x_stride, int32_t n,
                int32_t prologue, int32_t epilogue, void* out, int32_t out_stride, void* scratch, void* stream) {
  if (!w || !qt_ok(*w) || !x || !out || !scratch) return fail(Q4D_ERR_INVALID_ARG, "q4_gemm: NULL argument");
  if (n < 0 || n > kMaxBatch || N < 1 || K < 256 || K % 256 || x_stride % 8 || prologue < 0 || prologue > 1 ||
      epilogue < 0 || epilogue > 2)
    return fail(Q4D_ERR_INVALID_ARG, "q4_gemm: bad shape (K must be a multiple of 256, n <= 16)");
  if (x_stride < K * (1 + prologue)) return fail(Q4D_ERR_INVALID_ARG, "q4_gemm: x_stride is smaller than a row of the operand");
  if (K > kOpMaxK || gemm_partial_bytes(N, K, epilogue) > kOpGemmPartial ||
      (size_t)gemm_counters_needed(N) * 4 > kOpCounters)
    return fail(Q4D_ERR_WORKSPACE_TOO_SMALL, "q4_gemm: shape needs more scratch than q4d_op_scratch_bytes provides");
  unsigned char* sc = static_cast<unsigned char*>(scratch);
  uint16_t* xp = reinterpret_cast<uint16_t*>(sc + kOpPackOff);
  float* xs = reinterpret_cast<float*>(sc + kOpPackOff + kOpPackXp);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = launch_pack_operand(x, x_stride, K, n, prologue, xp, xs, gemm_operand_layout(false, n), st);
  if (e != cudaSuccess) return fail_cuda(e, "q4_gemm (operand)");
  GemmArgs a;
  a.qw = w->q, a.scales = w->scales, a.biases = w->biases, a.N = N, a.K = K, a.xp = xp, a.xs = xs, a.n = n;
  a.epilogue = epilogue, a.out = out, a.out_stride = out_stride;
  a.out_xp = nullptr, a.out_xs = nullptr, a.argmax_partial = nullptr;
  a.counters = reinterpret_cast<int*>(sc), a.counters_len = (int)(kOpCounters / 4);
  a.partial = reinterpret_cast<float*>(sc + kOpCounters), a.partial_bytes = kOpGemmPartial;
  e = launch_q4_gemm(a, st);
  return e == cudaSuccess ? Q4D_OK : fail_cuda(e, "q4_gemm");
}

int q4d_rmsnorm(const uint16_t* x, const uint16_t* w, float eps, int32_t n, int32_t H, uint16_t* y, void* stream) {
  if (!x || !w || !y || n < 0 || H < 64 || H % 64 || H > 16384)
    return fail(Q4D_ERR_INVALID_ARG, "rmsnorm: bad argument (H must be a multiple of 64, at most 16384)");
  cudaError_t e = launch_rmsnorm(x, w, eps, n, H, y, nullptr, nullptr, OPERAND_ROWS, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? Q4D_OK : fail_cuda(e, "rmsnorm");
}

int q4d_embed(const q4d_qtensor* t, int32_t vocab, int32_t H, const int32_t* tokens, int32_t n, uint16_t* x,
              void* stream) {
  if (!t || !qt_ok(*t) || !tokens || !x || n < 0 || H % 64) return fail(Q4D_ERR_INVALID_ARG, "embed: bad argument");
  cudaError_t e = launch_embed(t->q, t->scales, t->biases, vocab, H, tokens, n, x, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? Q4D_OK : fail_cuda(e, "embed");
}

int q4d_rope_append(const uint16_t* qkv, const uint16_t* q_norm, const uint16_t* k_norm, float eps, const float* rope,
                    int32_t n, int32_t nq, int32_t nkv, const int32_t* lens, const int32_t* bt, int32_t max_blocks,
                    uint16_t* kpool, uint16_t* vpool, uint16_t* q_out, void* stream) {
  if (!qkv || !rope || !lens || !bt || !kpool || !vpool || !q_out || n < 0 || nq < 1 || nkv < 1)
    return fail(Q4D_ERR_INVALID_ARG, "rope_append: bad argument");
  RopeArgs a;
  a.qkv = qkv, a.q_norm = q_norm, a.k_norm = k_norm, a.eps = eps, a.rope = rope, a.n = n, a.nq = nq, a.nkv = nkv;
  a.lens = lens, a.block_tables = bt, a.max_blocks = max_blocks, a.kpool = kpool, a.vpool = vpool, a.q_out = q_out;
  cudaError_t e = launch_rope_append(a, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? Q4D_OK : fail_cuda(e, "rope_append");
}

int q4d_paged_attention(const uint16_t* q, const uint16_t* kpool, const uint16_t* vpool, int32_t n, int32_t nq,
                        int32_t nkv, const int32_t* lens_host, const int32_t* lens_device, const int32_t* bt_device,
                        int32_t max_blocks, int32_t chunk_tokens, uint16_t* out, void* scratch, void* stream) {
  if (!q || !kpool || !vpool || !lens_host || !lens_device || !bt_device || !out || !scratch)
    return fail(Q4D_ERR_INVALID_ARG, "paged_attention: NULL argument");
  if (n < 0 || n > kMaxBatch || nq < 1 || nkv < 1 || nq % nkv || nq / nkv > 16)
    return fail(Q4D_ERR_INVALID_ARG, "paged_attention: bad head counts or batch");
  if (n == 0) return Q4D_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t by_meta = (kOpAttnMeta - 1024) / sizeof(int4);
  const size_t by_acc = kOpPartAcc / ((size_t)nq * kHeadDim * 4), by_ml = kOpPartMl / ((size_t)nq * 8);
  const int max_work = (int)std::min(by_meta, std::min(by_acc, by_ml));
  std::vector<int4> work(max_work);
  int32_t head[2 * kMaxBatch];
  const AttnPlan plan =
      plan_attention(lens_host, n, nkv, chunk_tokens, attention_wave_ctas(nq, nkv), work.data(), head, head + kMaxBatch, max_work);
  long long want = 0;
  for (int r = 0; r < n; ++r) want += ((lens_host[r] + 1 + 15) / 16 + plan.chunk_tiles - 1) / plan.chunk_tiles;
  if (want != plan.n_work)
    return fail(Q4D_ERR_WORKSPACE_TOO_SMALL, "paged_attention: too many chunks for the op scratch");
  unsigned char* sc = static_cast<unsigned char*>(scratch) + kOpCounters + kOpGemmPartial;
  cudaError_t e = cudaMemcpyAsync(sc, head, sizeof head, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(sc + 1024, work.data(), (size_t)plan.n_work * sizeof(int4), cudaMemcpyHostToDevice, s);
  if (e != cudaSuccess) return fail_cuda(e, "paged_attention metadata");
  AttnArgs a;
  a.q = q, a.kpool = kpool, a.vpool = vpool, a.block_tables = bt_device, a.lens = lens_device;
  a.work = reinterpret_cast<const int4*>(sc + 1024);
  a.slot_base = reinterpret_cast<const int32_t*>(sc), a.nchunks = reinterpret_cast<const int32_t*>(sc) + kMaxBatch;
  a.n_work = plan.n_work, a.n = n, a.nq = nq, a.nkv = nkv, a.max_blocks = max_blocks;
  a.part_acc = reinterpret_cast<float*>(sc + kOpAttnMeta);
  a.part_ml = reinterpret_cast<float*>(sc + kOpAttnMeta + kOpPartAcc);
  a.out = out, a.out_xp = nullptr, a.out_xs = nullptr;
  e = launch_paged_attention(a, s);
  if (e == cudaSuccess) e = launch_attention_merge(a, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);  // the host work list must outlive the copy
  return e == cudaSuccess ? Q4D_OK : fail_cuda(e, "paged_attention");
}

int q4d_argmax(const float* logits, int32_t n, int32_t vocab, int32_t* next, void* stream) {
  if (!logits || !next || n < 0 || vocab < 1) return fail(Q4D_ERR_INVALID_ARG, "argmax: bad argument");
  cudaError_t e = launch_argmax(logits, n, vocab, next, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? Q4D_OK : fail_cuda(e, "argmax");
}

int q4d_debug_run_layers(q4d_model* m, q4d_kv_pool* pool, int32_t n, const int64_t* ids, const int32_t* bt,
                         int32_t max_blocks, int32_t layer_begin, int32_t layer_end, const uint16_t* x_in,
                         uint16_t* x_out, void* stream) {
  if (!m || !x_in || !x_out || layer_begin < 0 || layer_end > m->sh.n_layers || layer_begin > layer_end)
    return fail(Q4D_ERR_INVALID_ARG, "debug_run_layers: bad argument");
  const LayerRange range{layer_begin, layer_end, x_in, x_out};
  return step_impl(m, pool, n, ids, nullptr, nullptr, bt, max_blocks, nullptr, nullptr,
                   static_cast<cudaStream_t>(stream), &range);
}

int q4d_debug_set_status(q4d_model* m, uint32_t value) {
  if (!m) return fail(Q4D_ERR_INVALID_ARG, "debug_set_status: NULL model");
  cudaError_t e = cudaDeviceSynchronize();
  if (e == cudaSuccess)
    e = cudaMemcpy(m->fused ? reinterpret_cast<unsigned char*>(m->fused_params->control + 1) : m->ws + m->lay.chain_status,
                   &value, sizeof value, cudaMemcpyHostToDevice);
  return e == cudaSuccess ? Q4D_OK : fail_cuda(e, "debug_set_status");
}

int q4d_debug_dequant(const q4d_qtensor* w, int32_t N, int32_t K, float* out, void* stream) {
  if (!w || !qt_ok(*w) || !out || N < 1 || K < 64 || K % 64)
    return fail(Q4D_ERR_INVALID_ARG, "debug_dequant: bad argument");
  cudaError_t e = launch_dequant(w->q, w->scales, w->biases, N, K, out, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? Q4D_OK : fail_cuda(e, "debug_dequant");
}

int q4d_debug_kv_gather(q4d_kv_pool* p, int32_t layer, const int32_t* bt_device, int32_t len, uint16_t* k_out,
                        uint16_t* v_out, void* stream) {
  if (!p || !bt_device || !k_out || !v_out || len < 0 || layer < 0 || layer >= p->model->sh.n_layers)
    return fail(Q4D_ERR_INVALID_ARG, "debug_kv_gather: bad argument");
  const size_t layer_elems = (size_t)p->num_blocks * p->model->sh.n_kv_heads * kBlockSize * kHeadDim;
  const uint16_t* kpool = p->mem + (size_t)(2 * layer) * layer_elems;
  cudaError_t e = launch_kv_gather(kpool, kpool + layer_elems, p->model->sh.n_kv_heads, bt_device, len, k_out, v_out,
                                   static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? Q4D_OK : fail_cuda(e, "debug_kv_gather");
}

}  // extern "C"
