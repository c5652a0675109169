// C ABI of the ltri library: host-side stream state, arena layout and the launch sequences of a prefill call
// and a decode step.  Everything that computes runs in the kernels; this file only orders them.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <deque>
#include <new>
#include <vector>

#include "../../include/ltri.h"
#include "common.cuh"

using namespace ltri;

namespace {

struct Region {
  int start, end, slot;
};

struct LayerState {
  long long t = 0;  // tokens appended
  int E = 0;        // end of the indexed prefix
  bool decoding = false;
  std::deque<Region> pending;
  long long span_ub = 0;  // upper bound of the device-side span count
  int last_m = 0;
  long long base = 0;  // sliding slabs: first token the window region of this layer's slabs holds
  int slides = 0;      // times the live rows were moved to the start of the window region
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Carver {
  char* base;
  size_t off = 0;
  template <typename T>
  T* take(size_t count) {
    off = align_up(off, 256);
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += count * sizeof(T);
    return p;
  }
};

bool validate(const ltri_params* p) {
  if (!p) return false;
  if (p->n_layers < 1 || p->n_q_heads < 1 || p->n_kv_heads < 1 || p->head_dim != kD) return false;
  if (p->n_q_heads % p->n_kv_heads) return false;
  const int G = p->n_q_heads / p->n_kv_heads;
  if (!(G == 1 || G == 2 || G == 4 || G == 8)) return false;
  if (p->max_seqs < 1 || p->max_tokens < 1 || p->max_tokens > (1ll << 30)) return false;
  if (p->chunk < 16 || p->chunk > 1024 || p->chunk % 16) return false;
  if (p->window < 1 || p->n_sink < 1 || p->n_sink > p->chunk) return false;
  if (p->top_k < 1 || p->top_k > kMaxTopK) return false;
  if (p->reps_per_span < 0 || p->reps_per_span > kMaxReps) return false;
  if (p->max_spans_per_region < 0 || p->max_spans_per_region > kMaxTopK) return false;
  if (p->theta_mode != 0 && p->theta_mode != 1) return false;
  if (!(p->theta >= 0.f) || (p->theta_mode == 1 && p->theta > 1.f)) return false;
  if (!(p->softmax_scale >= 0.f)) return false;
  if (p->flags & ~(uint32_t)(LTRI_FLAG_PERSIST_DECODE | LTRI_FLAG_HOST_STAGING | LTRI_FLAG_COLLAB_VOTE |
                              LTRI_FLAG_SEGMENT_PER_UNIT | LTRI_FLAG_HOST_KV))
    return false;
  if ((p->flags & LTRI_FLAG_COLLAB_VOTE) && (p->unit_tokens == 0 || !p->retrieval_head)) return false;
  if (p->flags & LTRI_FLAG_HOST_KV) {
    if (p->unit_tokens == 0) return false;
    const int need = p->top_k * ((p->flags & LTRI_FLAG_PERSIST_DECODE) ? 2 : 1);
    if (p->cache_units < need || p->cache_units > 128) return false;
    if (!(p->score_decay >= 0.f && p->score_decay <= 1.f)) return false;
  }
  if (p->flags & LTRI_FLAG_SEGMENT_PER_UNIT) {
    // a call of up to `chunk` tokens touches at most this many units; their kept spans share the segmenter's arrays
    if (p->unit_tokens == 0) return false;
    const int nun = (p->chunk + p->unit_tokens - 2) / p->unit_tokens + 1;
    const int cu = p->max_spans_per_region > 0 ? p->max_spans_per_region : std::max(1, p->unit_tokens / 32);
    if (cu * nun > kMaxTopK) return false;
  }
  if (p->retrieval_head)
    for (int l = 0; l < p->n_layers; ++l) {
      if (p->retrieval_head[l] < -1 || p->retrieval_head[l] >= p->n_q_heads) return false;
      if (p->retrieval_head_score && !(p->retrieval_head_score[l] >= 0.f && p->retrieval_head_score[l] < 1e30f))
        return false;
    }
  if (p->nms_iou_milli < 0 || p->nms_iou_milli > 999) return false;
  if (p->unit_tokens != 0) {
    if (p->unit_tokens < 8 || p->unit_tokens > p->chunk || p->unit_tokens % 8) return false;
    if (p->max_tokens / p->unit_tokens + 2 > 12288) return false;  // unit keys of the top-k kernel: 48 KB of shared memory
  }
  for (int l = 0; l < p->n_layers; ++l) {
    if (p->layer_theta && (!(p->layer_theta[l] >= 0.f) || (p->theta_mode == 1 && p->layer_theta[l] > 1.f))) return false;
    if (p->layer_nms_iou_milli && (p->layer_nms_iou_milli[l] < 0 || p->layer_nms_iou_milli[l] > 999)) return false;
    if (p->layer_rep_lambda && !(p->layer_rep_lambda[l] >= 0.f)) return false;
  }
  if (p->rep_mode != 0 && p->rep_mode != 1) return false;
  if (p->rep_mode == 1) {
    if (p->ratio_kind < 0 || p->ratio_kind > 2) return false;
    if (p->min_reps < 1 || p->max_reps < p->min_reps || p->max_reps > kMaxReps) return false;
    if (!(p->rep_lambda >= 0.f)) return false;
  }
  return true;
}

// bytes of one staging set of the host-buffer entry: q, k, v and out of a full call
size_t stage_set_bytes(const ltri_params& p) {
  const size_t rows = (size_t)p.n_layers * p.chunk;
  return align_up(rows * p.n_q_heads * kD * 2, 256) * 2 + align_up(rows * p.n_kv_heads * kD * 2, 256) * 2;
}

// rows of the window region of a sliding slab (see layout): 2 x (window + 2 chunks) + tile slack
long long window_rows(const ltri_params& p) { return 2ll * ((long long)p.window + 2ll * p.chunk) + 2 * kTokPad; }

// fills every pointer of `d` relative to `base` (nullptr: sizing only) and returns the bytes used
size_t layout(const ltri_params& p, DevCtx& d, char* base, char** stage_out = nullptr) {
  d.NL = p.n_layers;
  d.Hq = p.n_q_heads;
  d.Hkv = p.n_kv_heads;
  d.G = d.Hq / d.Hkv;
  d.NS = p.max_seqs;
  d.Tmax = p.max_tokens;
  d.Tpad = (long long)align_up((size_t)p.max_tokens, 128) + kTokPad;
  d.chunk = p.chunk;
  d.W = p.window;
  d.Ls = p.n_sink;
  d.topk = p.top_k;
  d.rcap = 2 * p.top_k + 2;
  d.persist = (p.flags & LTRI_FLAG_PERSIST_DECODE) ? 1 : 0;
  d.vote = (p.flags & LTRI_FLAG_COLLAB_VOTE) ? 1 : 0;
  d.reps = p.reps_per_span > 0 ? p.reps_per_span : 1;
  d.seg_unit = (p.flags & LTRI_FLAG_SEGMENT_PER_UNIT) ? p.unit_tokens : 0;
  d.C = p.max_spans_per_region > 0 ? p.max_spans_per_region
                                   : std::max(1, (d.seg_unit > 0 ? p.unit_tokens : p.chunk) / 32);
  d.Jmax = 2 * d.C + 1;
  if (d.seg_unit > 0) d.Jmax *= (p.chunk + p.unit_tokens - 2) / p.unit_tokens + 1;  // every unit a call can touch
  d.slots = (p.window + p.chunk - 1) / p.chunk + 8;
  d.cap = (int)std::min<long long>((long long)1 << 30, ((p.max_tokens + p.chunk - 1) / p.chunk + 8) * d.Jmax);
  d.theta_mode = p.theta_mode;
  d.theta = p.theta;
  d.unit = p.unit_tokens;
  d.phi_milli = p.nms_iou_milli;
  d.rep_mode = p.rep_mode;
  d.ratio_kind = p.ratio_kind;
  d.min_reps = p.min_reps;
  d.max_reps = p.max_reps;
  d.rep_lambda = p.rep_lambda;
  d.scale = p.softmax_scale > 0.f ? p.softmax_scale : 1.0f / std::sqrt((float)kD);
  const size_t units = (size_t)d.NS * d.NL;
  Carver cv{base};
  d.host_kv = (p.flags & LTRI_FLAG_HOST_KV) ? 1 : 0;
  d.cache_units = d.host_kv ? p.cache_units : 0;
  d.score_decay = p.score_decay;
  const size_t cache_rows = d.host_kv ? units * d.Hkv * (size_t)d.cache_units * p.unit_tokens : 0;
  // K/V slabs.  Resident: a row per token.  Paged: the sink, then a window region that holds twice what a call can
  // touch (tokens since the last eviction before the call + the call + tile slack), so that when it runs full the
  // live rows can be moved to its start without overlapping themselves.
  d.paged = d.host_kv;
  d.Lsp = d.paged ? (int)align_up((size_t)p.n_sink + 8, 8) : 0;
  d.SR = d.paged ? d.Lsp + window_rows(p) + kTokPad : d.Tpad;
  d.Kc = cv.take<__nv_bfloat16>(units * d.Hkv * d.SR * kD);
  d.Vc = cv.take<__nv_bfloat16>(units * d.Hkv * d.SR * kD);
  d.Kcache = cv.take<__nv_bfloat16>(cache_rows * kD);
  d.Vcache = cv.take<__nv_bfloat16>(cache_rows * kD);
  d.ctag = cv.take<int>(d.host_kv ? units * d.Hkv * d.cache_units : 0);
  d.cscore = cv.take<float>(d.host_kv ? units * d.Hkv * d.cache_units : 0);
  d.cstat = cv.take<unsigned long long>(d.host_kv ? units * 2 : 0);
  d.rng_koff = cv.take<int>(d.host_kv ? units * d.Hkv * d.rcap : 0);
  d.pl_id = cv.take<int>(d.host_kv ? units * d.Hkv * 2 * kMaxTopK : 0);
  d.pl_src = cv.take<int>(d.host_kv ? units * d.Hkv * 2 * kMaxTopK : 0);
  d.pl_start = cv.take<int>(d.host_kv ? units * d.Hkv * 2 * kMaxTopK : 0);
  d.pl_len = cv.take<int>(d.host_kv ? units * d.Hkv * 2 * kMaxTopK : 0);
  d.pl_cnt = cv.take<int>(d.host_kv ? units * d.Hkv : 0);
  d.votes = cv.take<long long>(units * d.Tpad);
  d.span_start = cv.take<int>(units * d.cap);
  d.span_len = cv.take<int>(units * d.cap);
  d.n_spans = cv.take<int>(units);
  d.KR = cv.take<__nv_bfloat16>(units * d.Hkv * d.cap * kD);
  d.pend_start = cv.take<int>(units * (d.slots + 1) * d.Jmax);
  d.pend_len = cv.take<int>(units * (d.slots + 1) * d.Jmax);
  d.pend_cnt = cv.take<int>(units * (d.slots + 1));
  d.pend_nrep = cv.take<int>(units * (d.slots + 1) * d.Jmax);
  d.sel = cv.take<int>(units * d.Hkv * d.topk);
  d.persist_sel = cv.take<int>(units * d.Hkv * d.topk);
  d.sel_tokens = cv.take<long long>(units * d.Hkv);
  {
    // (carved whether or not a layer has a retrieval head, so that the arena size does not depend on host arrays)
    int* rh = cv.take<int>(d.NL);
    float* hw = cv.take<float>(d.NL);
    d.ret_head = p.retrieval_head ? rh : nullptr;
    d.head_w = p.retrieval_head ? hw : nullptr;
    d.ballot = cv.take<int>(units * d.topk);
    float* th = cv.take<float>(d.NL);
    int* ph = cv.take<int>(d.NL);
    float* la = cv.take<float>(d.NL);
    d.theta_l = p.layer_theta ? th : nullptr;
    d.phi_l = p.layer_nms_iou_milli ? ph : nullptr;
    d.lambda_l = p.layer_rep_lambda ? la : nullptr;
  }
  d.Mq = cv.take<int>((size_t)d.NL * d.chunk * d.chunk);
  d.Rsuf = cv.take<long long>((size_t)d.NL * d.chunk * d.chunk);
  d.best = cv.take<long long>((size_t)d.NL * 2 * d.chunk);
  d.thetaq = cv.take<long long>(d.NL);
  d.rowstat = cv.take<float2>((size_t)d.NL * d.chunk * d.Hq);
  d.rowq = cv.take<float>((size_t)d.NL * d.chunk * d.Hq);
  // rows padded to whole 256-row work items of the tensor-core attention kernel
  d.Oacc = cv.take<float>((size_t)d.NL * align_up((size_t)d.chunk * d.G, 256) * d.Hkv * kD);
  d.u = cv.take<float>((size_t)d.NL * d.Hkv * d.Jmax * kD);
  d.Jcnt = cv.take<int>(d.NL);
  d.nrep_last = cv.take<int>((size_t)d.NL * d.Jmax);
  d.Rcap = (long long)align_up((size_t)d.topk * d.chunk, 128) + kTokPad;
  d.Kg = cv.take<__nv_bfloat16>((size_t)d.NL * d.Hkv * d.Rcap * kD);
  d.Vg = cv.take<__nv_bfloat16>((size_t)d.NL * d.Hkv * d.Rcap * kD);
  d.gcnt = cv.take<int>((size_t)d.NL * d.Hkv);
  d.scores = cv.take<float>(units * d.Hkv * d.cap);
  d.rng_start = cv.take<int>(units * d.Hkv * d.rcap);
  d.rng_len = cv.take<int>(units * d.Hkv * d.rcap);
  d.rng_cnt = cv.take<int>(units * d.Hkv);
  d.dec_part = cv.take<float>(units * d.Hq * kMaxDecSplit * (kD + 2));
  d.status = cv.take<int>(4);
  d.tc_redo = cv.take<int>(kTcMaxCtas);
  d.wait_limit = kDefaultWaitLimit;
  d.slots += 1;  // the extra slot is scratch for ltri_debug_segment_map
  if (p.flags & LTRI_FLAG_HOST_STAGING) {
    const size_t set_bytes = stage_set_bytes(p);
    for (int s = 0; s < 2; ++s) {
      char* ptr = cv.take<char>(set_bytes);
      if (stage_out) stage_out[s] = ptr;
    }
  }
  return align_up(cv.off, 256);
}

}  // namespace

struct ltri_ctx {
  ltri_params p;
  DevCtx d;
  std::vector<LayerState> st;  // [max_seqs][n_layers]
  std::vector<int> ret_head;   // [n_layers] copy of the caller's retrieval heads (empty: none)
  std::vector<float> head_w;
  int last_cuda = 0;
  int sm_count = 148;
  bool use_tc = false;     // tcgen05/TMEM/TMA attention kernels (default when available)
  int dec_fused = -1;      // decode retrieval in one launch: -1 auto, 0 never, 1 whenever the index fits, 2 cluster kernel
  // host-buffer entry (LTRI_FLAG_HOST_STAGING): two staging sets in the arena, a copy-up and a copy-down stream, and
  // events that order every reuse of a set's layer-group slices
  static constexpr int kHostGroups = 4;
  char* stage[2] = {nullptr, nullptr};   // per set: q | k | v | out of one call, [NL][chunk][H][128] bf16 each
  cudaStream_t s_up = nullptr, s_down = nullptr;
  // host-memory pager: evicted rows are mirrored to the host on their own stream
  cudaStream_t s_spill = nullptr;
  cudaEvent_t ev_pre = nullptr, ev_spill = nullptr;
  // pulls of a prefill call run per layer group on their own stream (see ltri_prefill_chunk)
  static constexpr int kMaxGroups = 4;
  cudaStream_t s_pull = nullptr;
  cudaEvent_t ev_sel[kMaxGroups] = {}, ev_pull[kMaxGroups] = {};
  int pager_groups = kMaxGroups;  // layer groups of a paged prefill call (testing aid: LTRI_PAGER_GROUPS)
  char* host_kv = nullptr;   // the caller's mirror (host address)
  bool spilled = false;      // ev_spill has been recorded at least once
  cudaEvent_t ev_up[2][kHostGroups] = {}, ev_run[2][kHostGroups] = {}, ev_down[2][kHostGroups] = {};
  int ret_phase = 2;       // retrieved attention: 2 merges with the stored local state, 1 continues from it (testing aid)
  bool grp_used[2][kHostGroups] = {};  // the events of (set, group) have been recorded at least once
  long long host_calls = 0;
  alignas(64) unsigned char kv_maps[kTcMapBytes];  // TMA descriptors of the K/V cache
  long long launches = 0;  // kernels launched since creation
  // optional per-kernel-class timing with CUDA events on the launching stream
  bool profiling = false;
  struct Timed {
    cudaEvent_t a, b;
    int cls;
  };
  std::vector<Timed> timed;      // recorded since the last read
  std::vector<Timed> free_pool;  // reusable event pairs
  long long cls_launches[LTRI_K_COUNT] = {0};
  LayerState& at(int seq, int layer) { return st[(size_t)seq * d.NL + layer]; }
};

namespace {

int cuda_fail(ltri_ctx* ctx, cudaError_t e) {
  if (e == cudaSuccess) return LTRI_OK;
  ctx->last_cuda = (int)e;
  return LTRI_ECUDA;
}
#define LTRI_CUDA(ctx, expr)                                                         \
  do {                                                                               \
    cudaError_t e__ = (expr);                                                        \
    if (e__ != cudaSuccess) {                                                        \
      if (std::getenv("LTRI_DEBUG"))                                                 \
        fprintf(stderr, "ltri: %s failed at line %d: %s\n", #expr, __LINE__, cudaGetErrorString(e__)); \
      return cuda_fail(ctx, e__);                                                    \
    }                                                                                \
  } while (0)

bool aligned16(const void* p) { return p && (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// Brackets one kernel group with events when profiling is on, and counts its kernels.
struct Scope {
  ltri_ctx* ctx;
  cudaStream_t st;
  ltri_ctx::Timed t;
  bool on;
  Scope(ltri_ctx* c, cudaStream_t s, int cls, int kernels) : ctx(c), st(s), on(false) {
    ctx->launches += kernels;
    ctx->cls_launches[cls] += kernels;
    if (!ctx->profiling) return;
    if (!ctx->free_pool.empty()) {
      t = ctx->free_pool.back();
      ctx->free_pool.pop_back();
    } else if (cudaEventCreate(&t.a) != cudaSuccess || cudaEventCreate(&t.b) != cudaSuccess) {
      return;
    }
    t.cls = cls;
    on = cudaEventRecord(t.a, st) == cudaSuccess;
  }
  ~Scope() {
    if (!on) return;
    cudaEventRecord(t.b, st);
    ctx->timed.push_back(t);
  }
};

}  // namespace

extern "C" {

size_t ltri_host_kv_bytes(const ltri_params* p) {
  if (!validate(p) || !(p->flags & LTRI_FLAG_HOST_KV)) return 0;
  DevCtx d;
  layout(*p, d, nullptr);
  return (size_t)d.NS * d.NL * d.Hkv * (size_t)d.Tpad * kD * sizeof(__nv_bfloat16) * 2;
}

size_t ltri_arena_bytes(const ltri_params* p) {
  if (!validate(p)) return 0;
  DevCtx d;
  return layout(*p, d, nullptr);
}

int ltri_create(const ltri_params* p, void* cuda_stream, ltri_ctx** out) {
  if (!out) return LTRI_EINVAL;
  *out = nullptr;
  if (!validate(p)) return LTRI_EINVAL;
  if (!p->arena || (reinterpret_cast<uintptr_t>(p->arena) & 255)) return LTRI_EINVAL;
  DevCtx d;
  const size_t need = layout(*p, d, nullptr);
  if (p->arena_bytes < need) return LTRI_ECAPACITY;
  const __nv_bfloat16* host_dev = nullptr;
  if (p->flags & LTRI_FLAG_HOST_KV) {
    // the mirror must be page-locked host memory that kernels can read; checked here, on the host, so that a wrong
    // pointer is an error code and never a device fault
    if (!p->host_kv || (reinterpret_cast<uintptr_t>(p->host_kv) & 255)) return LTRI_EINVAL;
    if (p->host_kv_bytes < ltri_host_kv_bytes(p)) return LTRI_ECAPACITY;
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, p->host_kv) != cudaSuccess || attr.type != cudaMemoryTypeHost) {
      cudaGetLastError();
      return LTRI_EINVAL;
    }
    void* dp = nullptr;
    if (cudaHostGetDevicePointer(&dp, p->host_kv, 0) != cudaSuccess || !dp) {
      cudaGetLastError();
      return LTRI_EINVAL;
    }
    host_dev = static_cast<const __nv_bfloat16*>(dp);
  }
  ltri_ctx* ctx = new (std::nothrow) ltri_ctx();
  if (!ctx) return LTRI_ECAPACITY;
  ctx->p = *p;
  layout(*p, ctx->d, static_cast<char*>(p->arena), ctx->stage);
  if (host_dev) {
    const size_t half = (size_t)ctx->d.NS * ctx->d.NL * ctx->d.Hkv * (size_t)ctx->d.Tpad * kD;
    ctx->d.hostK = host_dev;
    ctx->d.hostV = host_dev + half;
    ctx->host_kv = static_cast<char*>(p->host_kv);
    bool ok = cudaStreamCreateWithFlags(&ctx->s_spill, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&ctx->s_pull, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&ctx->ev_pre, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&ctx->ev_spill, cudaEventDisableTiming) == cudaSuccess;
    for (int g = 0; g < ltri_ctx::kMaxGroups && ok; ++g)
      ok = cudaEventCreateWithFlags(&ctx->ev_sel[g], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&ctx->ev_pull[g], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
      ltri_destroy(ctx);
      return LTRI_ECUDA;
    }
    if (const char* f = std::getenv("LTRI_PAGER_GROUPS"))  // testing aid
      ctx->pager_groups = std::max(1, std::min((int)ltri_ctx::kMaxGroups, std::atoi(f)));
  }
  if (p->retrieval_head) {  // the caller's arrays are read now and not kept
    ctx->ret_head.assign(p->retrieval_head, p->retrieval_head + p->n_layers);
    ctx->head_w.assign((size_t)p->n_layers, 1.0f);
    if (p->retrieval_head_score) ctx->head_w.assign(p->retrieval_head_score, p->retrieval_head_score + p->n_layers);
  }
  ctx->p.retrieval_head = nullptr;
  ctx->p.retrieval_head_score = nullptr;
  ctx->p.layer_theta = nullptr;
  ctx->p.layer_nms_iou_milli = nullptr;
  ctx->p.layer_rep_lambda = nullptr;
  if (p->flags & LTRI_FLAG_HOST_STAGING) {
    bool ok = cudaStreamCreateWithFlags(&ctx->s_up, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&ctx->s_down, cudaStreamNonBlocking) == cudaSuccess;
    for (int s = 0; s < 2 && ok; ++s)
      for (int g = 0; g < ltri_ctx::kHostGroups && ok; ++g)
        ok = cudaEventCreateWithFlags(&ctx->ev_up[s][g], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&ctx->ev_run[s][g], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&ctx->ev_down[s][g], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
      ltri_destroy(ctx);
      return LTRI_ECUDA;
    }
  }
  if (const char* f = std::getenv("LTRI_ATTN_CONT"))  // testing aid
    if (std::atoi(f) != 0) ctx->ret_phase = 1;
  ctx->st.resize((size_t)p->max_seqs * p->n_layers);
  for (auto& s : ctx->st) s.E = p->n_sink;
  int dev = 0;
  if (cudaGetDevice(&dev) == cudaSuccess) {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0) ctx->sm_count = sms;
  }
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  // testing aid: 0 two launches, 1 one launch, 2 one launch with the cluster kernel whatever the index size
  if (const char* f = std::getenv("LTRI_DEC_FUSED")) ctx->dec_fused = std::max(0, std::min(2, std::atoi(f)));
  const char* impl = std::getenv("LTRI_ATTN_IMPL");  // "mma" selects the warp-MMA kernels (debugging aid)
  ctx->use_tc = tc_attention_supported(ctx->d) && !(impl && std::strcmp(impl, "mma") == 0) &&
                tc_encode_kv_maps(ctx->d, ctx->kv_maps);
  // unfilled tile slots and over-fetched rows must hold finite values: start from an all-zero cache
  const size_t kv_bytes = (size_t)p->max_seqs * p->n_layers * ctx->d.Hkv * (size_t)ctx->d.SR * kD * 2 * sizeof(__nv_bfloat16);
  // (paged decode numbers K rows from the start of the K slabs through the unit caches in 31 bits)
  const bool rows_fit = !ctx->d.paged ||
                        (size_t)(ctx->d.Kcache - ctx->d.Kc) / kD + (size_t)(ctx->d.Vcache - ctx->d.Kcache) / kD < (1ull << 31);
  if (((!ctx->ret_head.empty() || ctx->d.paged) && !ctx->use_tc) || !rows_fit) {
    // retrieval heads are built into the tensor-core map pass only, sliding slabs into the tensor-core kernels only
    ltri_destroy(ctx);
    return LTRI_EINVAL;
  }
  cudaError_t e = cudaMemsetAsync(ctx->d.Kc, 0, kv_bytes, s);
  if (e == cudaSuccess && ctx->d.host_kv)  // (the two unit caches are adjacent)
    e = cudaMemsetAsync(ctx->d.Kcache, 0,
                        (size_t)ctx->d.NS * ctx->d.NL * ctx->d.Hkv * ctx->d.cache_units * (size_t)ctx->d.unit * kD * 2 *
                            sizeof(__nv_bfloat16),
                        s);
  if (e == cudaSuccess && !ctx->ret_head.empty()) {
    e = cudaMemcpyAsync(const_cast<int*>(ctx->d.ret_head), ctx->ret_head.data(), ctx->ret_head.size() * sizeof(int),
                        cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess)
      e = cudaMemcpyAsync(const_cast<float*>(ctx->d.head_w), ctx->head_w.data(), ctx->head_w.size() * sizeof(float),
                          cudaMemcpyHostToDevice, s);
  }
  // per-layer tables: copied from the caller's arrays (the stream is synchronised below, before this call returns)
  auto up = [&](const void* dst, const void* src, size_t bytes) {
    if (e == cudaSuccess && dst && src) e = cudaMemcpyAsync(const_cast<void*>(dst), src, bytes, cudaMemcpyHostToDevice, s);
  };
  up(ctx->d.theta_l, p->layer_theta, (size_t)p->n_layers * sizeof(float));
  up(ctx->d.phi_l, p->layer_nms_iou_milli, (size_t)p->n_layers * sizeof(int));
  up(ctx->d.lambda_l, p->layer_rep_lambda, (size_t)p->n_layers * sizeof(float));
  if (e == cudaSuccess) e = launch_init(ctx->d, -1, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) {
    delete ctx;
    return LTRI_ECUDA;
  }
  *out = ctx;
  return LTRI_OK;
}

int ltri_destroy(ltri_ctx* ctx) {
  if (!ctx) return LTRI_EINVAL;
  if (ctx->s_up) {  // copies of the host-buffer entry may still be in flight
    cudaStreamSynchronize(ctx->s_up);
    cudaStreamDestroy(ctx->s_up);
  }
  if (ctx->s_down) {
    cudaStreamSynchronize(ctx->s_down);
    cudaStreamDestroy(ctx->s_down);
  }
  if (ctx->s_spill) {  // copies into the caller's host mirror may still be in flight
    cudaStreamSynchronize(ctx->s_spill);
    cudaStreamDestroy(ctx->s_spill);
  }
  if (ctx->s_pull) {
    cudaStreamSynchronize(ctx->s_pull);
    cudaStreamDestroy(ctx->s_pull);
  }
  for (int g = 0; g < ltri_ctx::kMaxGroups; ++g) {
    if (ctx->ev_sel[g]) cudaEventDestroy(ctx->ev_sel[g]);
    if (ctx->ev_pull[g]) cudaEventDestroy(ctx->ev_pull[g]);
  }
  if (ctx->ev_pre) cudaEventDestroy(ctx->ev_pre);
  if (ctx->ev_spill) cudaEventDestroy(ctx->ev_spill);
  for (int s = 0; s < 2; ++s)
    for (int g = 0; g < ltri_ctx::kHostGroups; ++g) {
      if (ctx->ev_up[s][g]) cudaEventDestroy(ctx->ev_up[s][g]);
      if (ctx->ev_run[s][g]) cudaEventDestroy(ctx->ev_run[s][g]);
      if (ctx->ev_down[s][g]) cudaEventDestroy(ctx->ev_down[s][g]);
    }
  for (auto* pool : {&ctx->timed, &ctx->free_pool})
    for (auto& t : *pool) {
      cudaEventDestroy(t.a);
      cudaEventDestroy(t.b);
    }
  delete ctx;
  return LTRI_OK;
}

int ltri_reset_sequence(ltri_ctx* ctx, int seq, void* cuda_stream) {
  if (!ctx || seq < 0 || seq >= ctx->d.NS) return LTRI_EINVAL;
  for (int l = 0; l < ctx->d.NL; ++l) {
    LayerState fresh;
    fresh.E = ctx->d.Ls;
    ctx->at(seq, l) = fresh;
  }
  LTRI_CUDA(ctx, launch_init(ctx->d, seq, static_cast<cudaStream_t>(cuda_stream)));
  return LTRI_OK;
}

// Sliding slabs: can tokens up to `t_end` (exclusive) be given rows in the window region of this layer's slabs?
// Returns 0 when they already fit, 1 when the live rows have to be moved to the start of the region first, and
// LTRI_ECAPACITY when even that would not make room (decode ran past what a sliding slab can hold).  No side effects.
static int slide_check(const ltri_ctx* ctx, const LayerState& s0, long long t_end) {
  const DevCtx& d = ctx->d;
  const long long cap = d.SR - d.Lsp - kTokPad;  // rows of the window region that may hold tokens
  if (t_end - s0.base <= cap) return 0;
  const long long nb = s0.E, live = s0.t - nb, dist = nb - s0.base;
  if (t_end - nb > cap || dist < live) return LTRI_ECAPACITY;
  return 1;
}

// Sliding slabs: make room for tokens up to `t_end` (exclusive) in the window region of the slabs of the given layers.
// When the region is full, the live rows -- everything since the last eviction, [E, t) -- are moved to its start with
// one strided device copy for K and one for V; the region is sized so that source and destination cannot overlap.
// Rows that leave the slab this way were mirrored to the host when their region was evicted: the copy waits for that.
static int slide_window(ltri_ctx* ctx, int seq, int layer_begin, int layer_count, long long t_end, cudaStream_t st) {
  const DevCtx& d = ctx->d;
  LayerState& s0 = ctx->at(seq, layer_begin);
  const int need = slide_check(ctx, s0, t_end);
  if (need <= 0) return need;
  const long long nb = s0.E, live = s0.t - nb, dist = nb - s0.base;
  if (ctx->spilled) LTRI_CUDA(ctx, cudaStreamWaitEvent(st, ctx->ev_spill, 0));
  if (live > 0) {
    const size_t row_bytes = kD * sizeof(__nv_bfloat16), pitch = (size_t)d.SR * row_bytes;
    const size_t slab0 = unit_of(d, seq, layer_begin) * d.Hkv;
    const size_t to = (slab0 * (size_t)d.SR + d.Lsp) * row_bytes, from = to + (size_t)dist * row_bytes;
    for (__nv_bfloat16* base : {d.Kc, d.Vc})
      LTRI_CUDA(ctx, cudaMemcpy2DAsync(reinterpret_cast<char*>(base) + to, pitch, reinterpret_cast<const char*>(base) + from,
                                       pitch, (size_t)live * row_bytes, (size_t)layer_count * d.Hkv,
                                       cudaMemcpyDeviceToDevice, st));
  }
  for (int l = 0; l < layer_count; ++l) {
    ctx->at(seq, layer_begin + l).base = nb;
    ctx->at(seq, layer_begin + l).slides += 1;
  }
  return LTRI_OK;
}

// Everything a prefill call decides on the host before it enqueues work: which regions leave the window, where the
// indexed prefix ends afterwards, the call's own region and the pending slot it gets.
struct PrefillPlan {
  std::vector<Region> ev;
  int E = 0, t0 = 0, reg_start = 0, m = 0, slot = -1;
  long long ub = 0;
};

// All host-side checks of a prefill call over layers [layer_begin, layer_begin + layer_count); fills `plan`.
// Changes nothing: a call that fails here leaves the context as it was.
static int plan_prefill(ltri_ctx* ctx, int seq, int layer_begin, int layer_count, int n_tokens, PrefillPlan& plan) {
  const DevCtx& d = ctx->d;
  if (seq < 0 || seq >= d.NS || layer_begin < 0 || layer_count < 1 || layer_begin + layer_count > d.NL)
    return LTRI_EINVAL;
  if (n_tokens < 1 || n_tokens > d.chunk) return LTRI_EINVAL;
  const LayerState& s0 = ctx->at(seq, layer_begin);
  for (int l = 0; l < layer_count; ++l) {
    const LayerState& s = ctx->at(seq, layer_begin + l);
    if (s.decoding) return LTRI_ESTATE;
    if (s.t != s0.t || s.E != s0.E || s.pending.size() != s0.pending.size() || s.base != s0.base) return LTRI_ESTATE;
  }
  if (s0.t + n_tokens > d.Tmax) return LTRI_ECAPACITY;
  const int t0 = (int)s0.t;
  // the evictions (the host knows the region boundaries; the span counts live on the device)
  plan.ev.clear();
  int E = s0.E;
  long long ub = s0.span_ub;
  for (const Region& r : s0.pending) {
    if (r.end <= t0 - d.W) {
      plan.ev.push_back(r);
      E = r.end;
      ub += std::min(d.Jmax, r.end - r.start);
    } else
      break;
  }
  if (ub > d.cap) return LTRI_ECAPACITY;
  const int reg_start = std::max(d.Ls, t0);
  const int m = std::max(0, t0 + n_tokens - reg_start);
  const int user_slots = d.slots - 1;
  if (m > 0 && (int)(s0.pending.size() - plan.ev.size()) + 1 > user_slots) return LTRI_ECAPACITY;
  int slot = -1;
  if (m > 0) {
    // first slot not used by a region that stays pending
    std::vector<char> used(user_slots, 0);
    for (size_t i = plan.ev.size(); i < s0.pending.size(); ++i) used[s0.pending[i].slot] = 1;
    for (int i = 0; i < user_slots; ++i)
      if (!used[i]) {
        slot = i;
        break;
      }
  }
  if (d.paged && slide_check(ctx, s0, (long long)t0 + n_tokens) < 0) return LTRI_ECAPACITY;
  plan.E = E;
  plan.ub = ub;
  plan.t0 = t0;
  plan.reg_start = reg_start;
  plan.m = m;
  plan.slot = slot;
  return LTRI_OK;
}

int ltri_prefill_chunk(ltri_ctx* ctx, int seq, int layer_begin, int layer_count, int n_tokens, const void* q,
                       const void* k, const void* v, void* out, void* cuda_stream) {
  if (!ctx) return LTRI_EINVAL;
  const DevCtx& d = ctx->d;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return LTRI_EINVAL;
  PrefillPlan plan;
  {
    const int rc = plan_prefill(ctx, seq, layer_begin, layer_count, n_tokens, plan);
    if (rc != LTRI_OK) return rc;
  }
  LayerState& s0 = ctx->at(seq, layer_begin);
  const std::vector<Region>& ev = plan.ev;
  const int t0 = plan.t0, E = plan.E, reg_start = plan.reg_start, m = plan.m, slot = plan.slot;
  const long long ub = plan.ub;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  PrefillArgs a;
  a.seq = seq;
  a.layer_begin = layer_begin;
  a.layer_count = layer_count;
  a.n = n_tokens;
  a.t0 = t0;
  a.sink_end = std::min(d.Ls, t0);
  a.loc_begin = std::min(E, t0);
  a.reg_start = reg_start;
  a.m = m;
  a.slot = slot;
  a.q = static_cast<const __nv_bfloat16*>(q);
  a.k = static_cast<const __nv_bfloat16*>(k);
  a.v = static_cast<const __nv_bfloat16*>(v);
  a.out = static_cast<__nv_bfloat16*>(out);

  // every host-side check has passed: from here on work is enqueued
  if (d.paged) {
    const int rc = slide_window(ctx, seq, layer_begin, layer_count, t0 + n_tokens, st);
    if (rc != LTRI_OK) return rc;
  }
  const long long shift = d.paged ? s0.base - d.Lsp : 0;
  a.shift = shift;
  // The eviction kernel (one CTA per layer) goes first and releases the append kernel behind it at once: the two
  // touch different data and run side by side; the append kernel waits for the eviction kernel at its end.  They are
  // timed together (class LTRI_K_EVICT); a call that evicts nothing times its append kernel alone (LTRI_K_APPEND).
  {
    const int n_ev = (int)((ev.size() + 7) / 8);
    Scope sc(ctx, st, n_ev > 0 ? LTRI_K_EVICT : LTRI_K_APPEND, n_ev + 1);
    for (size_t i = 0; i < ev.size(); i += 8) {
      EvictArgs ea;
      ea.seq = seq;
      ea.shift = shift;
      ea.layer_begin = layer_begin;
      ea.nslots = (int)std::min<size_t>(8, ev.size() - i);
      ea.release = i + 8 >= ev.size() ? 1 : 0;
      for (int j = 0; j < ea.nslots; ++j) ea.slot[j] = ev[i + j].slot;
      LTRI_CUDA(ctx, launch_evict_index(d, ea, layer_count, st));
    }
    LTRI_CUDA(ctx, launch_append_prefill(d, a, /*clear_maps=*/ctx->use_tc, /*late_wait=*/n_ev > 0, st));
  }
  if (d.host_kv && !ev.empty()) {
    // mirror the rows that just left the window to the host: one strided copy for K and one for V per region (the
    // slabs of consecutive (layer, KV head) pairs are Tpad rows apart on both sides), on the spill stream, behind
    // everything submitted before this call (the rows were appended by earlier calls); the top-k kernel, which may
    // pull them back, waits for the copies
    LTRI_CUDA(ctx, cudaEventRecord(ctx->ev_pre, st));
    LTRI_CUDA(ctx, cudaStreamWaitEvent(ctx->s_spill, ctx->ev_pre, 0));
    const size_t row_bytes = kD * sizeof(__nv_bfloat16);
    const size_t half = (size_t)d.NS * d.NL * d.Hkv * (size_t)d.Tpad * row_bytes;
    const size_t hpitch = (size_t)d.Tpad * row_bytes, dpitch = (size_t)d.SR * row_bytes;
    const size_t slab0 = unit_of(d, seq, layer_begin) * d.Hkv;  // first slab of the call's layers
    for (const Region& r : ev) {
      const size_t hoff = (slab0 * (size_t)d.Tpad + r.start) * row_bytes;  // mirror: a row per token
      const size_t doff = (slab0 * (size_t)d.SR + (size_t)slab_row(d, r.start, shift)) * row_bytes;
      const size_t width = (size_t)(r.end - r.start) * row_bytes;
      LTRI_CUDA(ctx, cudaMemcpy2DAsync(ctx->host_kv + hoff, hpitch, reinterpret_cast<const char*>(d.Kc) + doff, dpitch,
                                       width, (size_t)layer_count * d.Hkv, cudaMemcpyDeviceToHost, ctx->s_spill));
      LTRI_CUDA(ctx, cudaMemcpy2DAsync(ctx->host_kv + half + hoff, hpitch, reinterpret_cast<const char*>(d.Vc) + doff,
                                       dpitch, width, (size_t)layer_count * d.Hkv, cudaMemcpyDeviceToHost, ctx->s_spill));
    }
    LTRI_CUDA(ctx, cudaEventRecord(ctx->ev_spill, ctx->s_spill));
    ctx->spilled = true;
  }
  const bool has_index = ub > 0;
  // Layer groups.  Resident contexts run every kernel once over all layers of the call.  Under the host-memory pager
  // the call is issued in up to four groups of layers: a group's top-k only decides what has to come over the bus;
  // the transfer and the gather (k_pull_pack) follow on the pager's own stream while the next groups compute, and
  // the retrieved attention of each group is issued at the end, once its rows are in place.
  const int NG = (d.host_kv && has_index) ? std::min(ctx->pager_groups, layer_count) : 1;
  long long thq_abs = 0;
  if (d.theta_mode == 0) thq_abs = (long long)std::nearbyint((double)d.theta * (double)d.Hq * (double)kQScale);
  PrefillArgs grp[ltri_ctx::kMaxGroups];
  for (int g = 0; g < NG; ++g) {
    const int lo = layer_count * g / NG, hi = layer_count * (g + 1) / NG;  // call-relative layers of the group
    PrefillArgs& ag = grp[g];
    ag = a;
    ag.layer_begin = layer_begin + lo;
    ag.layer_count = hi - lo;
    ag.q = a.q + (size_t)lo * n_tokens * d.Hq * kD;
    ag.k = a.k + (size_t)lo * n_tokens * d.Hkv * kD;
    ag.v = a.v + (size_t)lo * n_tokens * d.Hkv * kD;
    ag.out = a.out + (size_t)lo * n_tokens * d.Hq * kD;
    {
      Scope sc(ctx, st, LTRI_K_ATTN_LOCAL, ctx->use_tc ? 2 : 1);
      LTRI_CUDA(ctx, ctx->use_tc ? launch_attn_prefill_tc(d, ag, 0, !has_index, ctx->kv_maps, st)
                                 : launch_attn_prefill(d, ag, 0, !has_index, st));
    }
    {
      // (the tensor-core pass is one kernel; the warp-MMA fallback has one for the local keys and one for the call's own)
      Scope sc(ctx, st, LTRI_K_MAP, ctx->use_tc ? 1 : ((a.t0 - a.loc_begin > 0 && a.loc_begin >= d.Ls) ? 2 : 1));
      LTRI_CUDA(ctx, ctx->use_tc ? launch_map_pass_tc(d, ag, ctx->kv_maps, st) : launch_map_pass(d, ag, st));
    }
    if (m > 0) {
      Scope sc(ctx, st, LTRI_K_SEGMENT, 4);
      LTRI_CUDA(ctx, launch_segment(d, seq, ag.layer_begin, ag.layer_count, m, reg_start, slot, d.theta_mode, d.theta,
                                    thq_abs, d.C, n_tokens, t0, ag.q, st, /*tables=*/true, d.seg_unit));
    }
    if (!has_index) continue;
    {
      Scope sc(ctx, st, LTRI_K_SCORE_TOPK, d.vote ? 3 : 2);
      if (ctx->use_tc && score_tc_supported(d))
        LTRI_CUDA(ctx, launch_score_prefill_tc(d, ag, (int)ub, ctx->kv_maps, st));
      else if (ctx->use_tc)
        LTRI_CUDA(ctx, launch_score_prefill_mma(d, ag, (int)ub, st));
      else
        LTRI_CUDA(ctx, launch_score_prefill(d, ag, (int)ub, st));
      LTRI_CUDA(ctx, launch_topk_prefill(d, ag, st));
    }
    if (d.host_kv) {
      // the group's selection is known: its units travel on the pager's stream (behind this call's spill copies, whose
      // rows a pull may want back) while the caller's stream goes on with the next group
      cudaStream_t sp = ctx->s_pull;
      LTRI_CUDA(ctx, cudaEventRecord(ctx->ev_sel[g], st));
      LTRI_CUDA(ctx, cudaStreamWaitEvent(sp, ctx->ev_sel[g], 0));
      if (!ev.empty()) LTRI_CUDA(ctx, cudaStreamWaitEvent(sp, ctx->ev_spill, 0));
      {
        Scope sc(ctx, sp, LTRI_K_PAGER_PULL, 1);
        LTRI_CUDA(ctx, launch_pull_pack(d, ag, sp));
      }
      LTRI_CUDA(ctx, cudaEventRecord(ctx->ev_pull[g], sp));
    }
  }
  if (has_index)
    for (int g = 0; g < NG; ++g) {
      if (d.host_kv) LTRI_CUDA(ctx, cudaStreamWaitEvent(st, ctx->ev_pull[g], 0));
      Scope sc(ctx, st, LTRI_K_ATTN_RET, ctx->use_tc ? 2 : 1);
      LTRI_CUDA(ctx, ctx->use_tc ? launch_attn_prefill_tc(d, grp[g], ctx->ret_phase, true, ctx->kv_maps, st)
                                 : launch_attn_prefill(d, grp[g], 1, true, st));
    }
  // commit the host state
  for (int l = 0; l < layer_count; ++l) {
    LayerState& s = ctx->at(seq, layer_begin + l);
    for (size_t i = 0; i < ev.size(); ++i) s.pending.pop_front();
    s.E = E;
    s.span_ub = ub;
    s.t += n_tokens;
    s.last_m = m;
    if (m > 0) s.pending.push_back(Region{reg_start, t0 + n_tokens, slot});
  }
  return LTRI_OK;
}

int ltri_prefill_chunk_host(ltri_ctx* ctx, int seq, int layer_begin, int layer_count, int n_tokens, const void* q_host,
                            const void* k_host, const void* v_host, void* out_host, void* cuda_stream) {
  if (!ctx) return LTRI_EINVAL;
  if (!ctx->stage[0]) return LTRI_ESTATE;  // created without LTRI_FLAG_HOST_STAGING
  const DevCtx& d = ctx->d;
  if (!q_host || !k_host || !v_host || !out_host) return LTRI_EINVAL;
  {
    // every host-side check of the whole call first: the layers of a call are in the same state, so what holds for
    // the full range holds for each layer group, and an error return leaves the sequence untouched
    PrefillPlan plan;
    const int rc = plan_prefill(ctx, seq, layer_begin, layer_count, n_tokens, plan);
    if (rc != LTRI_OK) return rc;
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int set = (int)(ctx->host_calls & 1);
  const size_t rows = (size_t)d.NL * d.chunk;
  const size_t qb = align_up(rows * d.Hq * kD * 2, 256), kb = align_up(rows * d.Hkv * kD * 2, 256);
  char* sq = ctx->stage[set];
  char* sk = sq + qb;
  char* sv = sk + kb;
  char* so = sv + kb;
  // The layer groups are those of the CONTEXT (layers [NL g / G, NL (g + 1) / G) for group g), whatever range the call
  // covers, and a layer's staging bytes start at layer * chunk rows: a group always owns the same bytes of a staging
  // set, so the events of (set, group) order every reuse of them, also between calls of different sizes.  Inside a
  // group's slice the call's layers are dense (n_tokens rows apart), as the device entry wants them.
  const int G = std::min((int)ltri_ctx::kHostGroups, d.NL);
  const size_t qrow = (size_t)n_tokens * d.Hq * kD * 2, krow = (size_t)n_tokens * d.Hkv * kD * 2;  // bytes per layer
  const size_t qlay = (size_t)d.chunk * d.Hq * kD * 2, klay = (size_t)d.chunk * d.Hkv * kD * 2;     // staging stride
  for (int g = 0; g < G; ++g) {
    const int lo = std::max(layer_begin, d.NL * g / G), hi = std::min(layer_begin + layer_count, d.NL * (g + 1) / G);
    if (lo >= hi) continue;
    const size_t qs = lo * qlay, ks = lo * klay;                                  // staging offsets of the slice
    const size_t qh = (lo - layer_begin) * qrow, kh = (lo - layer_begin) * krow;  // offsets in the caller's tensors
    const size_t qn = (hi - lo) * qrow, kn = (hi - lo) * krow;
    // up: the kernels that read this group's slice of the set (two calls ago) are done
    if (ctx->grp_used[set][g]) LTRI_CUDA(ctx, cudaStreamWaitEvent(ctx->s_up, ctx->ev_run[set][g], 0));
    LTRI_CUDA(ctx, cudaMemcpyAsync(sq + qs, static_cast<const char*>(q_host) + qh, qn, cudaMemcpyHostToDevice, ctx->s_up));
    LTRI_CUDA(ctx, cudaMemcpyAsync(sk + ks, static_cast<const char*>(k_host) + kh, kn, cudaMemcpyHostToDevice, ctx->s_up));
    LTRI_CUDA(ctx, cudaMemcpyAsync(sv + ks, static_cast<const char*>(v_host) + kh, kn, cudaMemcpyHostToDevice, ctx->s_up));
    LTRI_CUDA(ctx, cudaEventRecord(ctx->ev_up[set][g], ctx->s_up));
    // run: inputs are up, and the output slice written two calls ago has gone down
    LTRI_CUDA(ctx, cudaStreamWaitEvent(st, ctx->ev_up[set][g], 0));
    if (ctx->grp_used[set][g]) LTRI_CUDA(ctx, cudaStreamWaitEvent(st, ctx->ev_down[set][g], 0));
    // (after the checks above this can only fail in the CUDA runtime)
    const int rc = ltri_prefill_chunk(ctx, seq, lo, hi - lo, n_tokens, sq + qs, sk + ks, sv + ks, so + qs, st);
    if (rc != LTRI_OK) return rc;
    LTRI_CUDA(ctx, cudaEventRecord(ctx->ev_run[set][g], st));
    // down
    LTRI_CUDA(ctx, cudaStreamWaitEvent(ctx->s_down, ctx->ev_run[set][g], 0));
    LTRI_CUDA(ctx, cudaMemcpyAsync(static_cast<char*>(out_host) + qh, so + qs, qn, cudaMemcpyDeviceToHost, ctx->s_down));
    LTRI_CUDA(ctx, cudaEventRecord(ctx->ev_down[set][g], ctx->s_down));
    ctx->grp_used[set][g] = true;
  }
  ctx->host_calls += 1;
  return LTRI_OK;
}

int ltri_host_outputs_ready(ltri_ctx* ctx, void* cuda_stream) {
  if (!ctx) return LTRI_EINVAL;
  if (!ctx->stage[0]) return LTRI_ESTATE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  for (int s = 0; s < 2; ++s)
    for (int g = 0; g < ltri_ctx::kHostGroups; ++g)
      if (ctx->grp_used[s][g]) LTRI_CUDA(ctx, cudaStreamWaitEvent(st, ctx->ev_down[s][g], 0));
  return LTRI_OK;
}

int ltri_decode_step(ltri_ctx* ctx, const int32_t* seq_ids, int n_seqs, int layer_begin, int layer_count,
                     const void* q, const void* k, const void* v, void* out, void* cuda_stream) {
  if (!ctx || !seq_ids) return LTRI_EINVAL;
  const DevCtx& d = ctx->d;
  if (n_seqs < 1 || n_seqs > d.NS || layer_begin < 0 || layer_count < 1 || layer_begin + layer_count > d.NL)
    return LTRI_EINVAL;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return LTRI_EINVAL;
  std::vector<char> seen(d.NS, 0);
  long long ub = 0;
  for (int i = 0; i < n_seqs; ++i) {
    const int sq = seq_ids[i];
    if (sq < 0 || sq >= d.NS || seen[sq]) return LTRI_EINVAL;
    seen[sq] = 1;
    const LayerState& s0 = ctx->at(sq, layer_begin);
    if (s0.t < 1) return LTRI_ESTATE;
    if (s0.t + 1 > d.Tmax) return LTRI_ECAPACITY;
    if (d.paged && slide_check(ctx, s0, s0.t + 1) < 0) return LTRI_ECAPACITY;  // (before anything is enqueued)
    for (int l = 0; l < layer_count; ++l) {
      const LayerState& s = ctx->at(sq, layer_begin + l);
      if (s.t != s0.t || s.E != s0.E || s.base != s0.base) return LTRI_ESTATE;
    }
    ub = std::max(ub, s0.span_ub);
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (d.paged)
    for (int i = 0; i < n_seqs; ++i) {
      const int rc = slide_window(ctx, seq_ids[i], layer_begin, layer_count, ctx->at(seq_ids[i], layer_begin).t + 1, st);
      if (rc != LTRI_OK) return rc;
    }
  const __nv_bfloat16* qb = static_cast<const __nv_bfloat16*>(q);
  const __nv_bfloat16* kb = static_cast<const __nv_bfloat16*>(k);
  const __nv_bfloat16* vb = static_cast<const __nv_bfloat16*>(v);
  __nv_bfloat16* ob = static_cast<__nv_bfloat16*>(out);
  // persistent mechanism: before a sequence's first decode step overwrites the selection of its last prefill call,
  // that selection is set aside; every decode step then attends over it as well
  if (d.persist) {
    for (int i = 0; i < n_seqs; ++i) {
      const int sq = seq_ids[i];
      for (int l = 0; l < layer_count; ++l) {
        if (ctx->at(sq, layer_begin + l).decoding) continue;
        const size_t off = unit_of(d, sq, layer_begin + l) * d.Hkv * (size_t)d.topk;
        LTRI_CUDA(ctx, cudaMemcpyAsync(d.persist_sel + off, d.sel + off, (size_t)d.Hkv * d.topk * sizeof(int),
                                       cudaMemcpyDeviceToDevice, st));
      }
    }
  }
  for (int i0 = 0; i0 < n_seqs; i0 += kDecBatch) {
    DecBatch b;
    b.n = std::min(kDecBatch, n_seqs - i0);
    for (int i = 0; i < b.n; ++i) {
      const LayerState& s = ctx->at(seq_ids[i0 + i], layer_begin);
      b.seq[i] = seq_ids[i0 + i];
      b.pos[i] = (int)s.t;
      b.loc_begin[i] = s.E;
      b.src[i] = i0 + i;
      b.shift[i] = d.paged ? s.base - d.Lsp : 0;
    }
    const int units = b.n * layer_count * d.Hkv;
    // split count of the decode attention: three CTAs fit an SM, so the grid runs in waves of 3 x SMs CTAs.  Among
    // the split counts that leave a CTA at least ~512 tokens (of the tokens known on the host: sink + everything
    // since the last eviction) take the one whose last wave is fullest; ties go to fewer, longer slices.
    int nsplit = 1;
    {
      const LayerState& s0 = ctx->at(seq_ids[i0], layer_begin);
      const long long known = d.Ls + (s0.t + 1 - s0.E);
      const int wave = 3 * ctx->sm_count;
      const int max_split = (int)std::max<long long>(1, std::min<long long>(kMaxDecSplit, known / 512));
      double best = -1.0;
      for (int ns = 1; ns <= max_split; ++ns) {
        const long long ctas = (long long)units * ns;
        const long long waves = (ctas + wave - 1) / wave;
        const double eff = (double)ctas / (double)(waves * wave);
        if (eff > best + 1e-9) {
          best = eff;
          nsplit = ns;
        }
      }
    }
    // retrieval in one launch with the scores in shared memory: one CTA per (sequence, layer, KV head) when there are
    // enough heads to fill the GPU and the index fits one CTA (12K spans), a cluster of eight CTAs per head for a larger
    // index (up to 98K spans); otherwise the scores go through global memory in two launches
    const bool one_cta = ub <= 12288;
    // (unit-granular retrieval ranks units, which only the two-launch path does)
    const bool fused = d.unit == 0 && ub <= dec_retrieve_fused_max_spans() &&
                       (ctx->dec_fused >= 1 || (ctx->dec_fused < 0 && (!one_cta || units >= ctx->sm_count)));
    if (!fused) {
      Scope sc(ctx, st, LTRI_K_APPEND, 1);
      LTRI_CUDA(ctx, launch_append_decode(d, b, layer_begin, layer_count, n_seqs, kb, vb, st));
    }
    if (fused) {
      // (the one-launch kernels also store the step's K/V rows: no append launch)
      Scope sc(ctx, st, LTRI_K_DEC_RETRIEVE, 1);
      // CTA size of the one-CTA kernel: 1024 threads fit once per SM, 512 twice; with more CTAs than SMs the smaller
      // size keeps all of them resident instead of running a second, partly empty wave
      const int ret_threads = units > ctx->sm_count ? 512 : 1024;
      LTRI_CUDA(ctx, launch_dec_retrieve_fused(d, b, layer_begin, layer_count, qb, kb, vb, (int)ub, ctx->dec_fused == 2,
                                               ret_threads, st));
    } else {
      Scope sc(ctx, st, LTRI_K_DEC_RETRIEVE, d.vote ? 3 : 2);
      LTRI_CUDA(ctx, launch_score_decode(d, b, layer_begin, layer_count, n_seqs, qb, (int)ub, st));
      LTRI_CUDA(ctx, launch_topk_decode(d, b, layer_begin, layer_count, st));
    }
    Scope sc(ctx, st, LTRI_K_DEC_ATTN, 2);
    LTRI_CUDA(ctx, launch_decode_attn(d, b, layer_begin, layer_count, n_seqs, qb, ob, nsplit, st));
  }
  for (int i = 0; i < n_seqs; ++i)
    for (int l = 0; l < layer_count; ++l) {
      LayerState& s = ctx->at(seq_ids[i], layer_begin + l);
      s.t += 1;
      s.decoding = true;
    }
  return LTRI_OK;
}

// ---- introspection ---------------------------------------------------------------------------
static int copy_back(ltri_ctx* ctx, void* dst, const void* src, size_t bytes, cudaStream_t st) {
  if (bytes == 0) return LTRI_OK;
  LTRI_CUDA(ctx, cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, st));
  LTRI_CUDA(ctx, cudaStreamSynchronize(st));
  return LTRI_OK;
}

int ltri_get_spans(ltri_ctx* ctx, int seq, int layer, int32_t* pairs, int cap, int* n_out, void* cuda_stream) {
  if (!ctx || !n_out || seq < 0 || seq >= ctx->d.NS || layer < 0 || layer >= ctx->d.NL || cap < 0) return LTRI_EINVAL;
  const DevCtx& d = ctx->d;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t unit = unit_of(d, seq, layer);
  int n = 0;
  int rc = copy_back(ctx, &n, d.n_spans + unit, sizeof(int), st);
  if (rc) return rc;
  *n_out = n;
  const int take = std::min(n, cap);
  if (take > 0 && pairs) {
    std::vector<int> a(take), b(take);
    rc = copy_back(ctx, a.data(), d.span_start + unit * d.cap, take * sizeof(int), st);
    if (rc) return rc;
    rc = copy_back(ctx, b.data(), d.span_len + unit * d.cap, take * sizeof(int), st);
    if (rc) return rc;
    for (int i = 0; i < take; ++i) {
      pairs[2 * i] = a[i];
      pairs[2 * i + 1] = b[i];
    }
  }
  return LTRI_OK;
}

int ltri_get_pending_spans(ltri_ctx* ctx, int seq, int layer, int32_t* pairs, int cap, int* n_out, void* cuda_stream) {
  if (!ctx || !n_out || seq < 0 || seq >= ctx->d.NS || layer < 0 || layer >= ctx->d.NL || cap < 0) return LTRI_EINVAL;
  const DevCtx& d = ctx->d;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t unit = unit_of(d, seq, layer);
  int total = 0;
  for (const Region& r : ctx->at(seq, layer).pending) {
    int cnt = 0;
    int rc = copy_back(ctx, &cnt, d.pend_cnt + unit * d.slots + r.slot, sizeof(int), st);
    if (rc) return rc;
    cnt = std::max(0, std::min(cnt, d.Jmax));
    std::vector<int> a(cnt), b(cnt);
    rc = copy_back(ctx, a.data(), d.pend_start + (unit * d.slots + r.slot) * d.Jmax, cnt * sizeof(int), st);
    if (rc) return rc;
    rc = copy_back(ctx, b.data(), d.pend_len + (unit * d.slots + r.slot) * d.Jmax, cnt * sizeof(int), st);
    if (rc) return rc;
    for (int i = 0; i < cnt; ++i, ++total)
      if (total < cap && pairs) {
        pairs[2 * total] = a[i];
        pairs[2 * total + 1] = b[i];
      }
  }
  *n_out = total;
  return LTRI_OK;
}

int ltri_get_selected(ltri_ctx* ctx, int seq, int layer, int32_t* ids, void* cuda_stream) {
  if (!ctx || !ids || seq < 0 || seq >= ctx->d.NS || layer < 0 || layer >= ctx->d.NL) return LTRI_EINVAL;
  const DevCtx& d = ctx->d;
  return copy_back(ctx, ids, d.sel + unit_of(d, seq, layer) * d.Hkv * d.topk, (size_t)d.Hkv * d.topk * sizeof(int),
                   static_cast<cudaStream_t>(cuda_stream));
}

int ltri_get_stats(ltri_ctx* ctx, int seq, int layer, ltri_stats* out, void* cuda_stream) {
  if (!ctx || !out || seq < 0 || seq >= ctx->d.NS || layer < 0 || layer >= ctx->d.NL) return LTRI_EINVAL;
  const DevCtx& d = ctx->d;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t unit = unit_of(d, seq, layer);
  const LayerState& s = ctx->at(seq, layer);
  std::memset(out, 0, sizeof(*out));
  int n = 0;
  long long rt = 0;
  int rc = copy_back(ctx, &n, d.n_spans + unit, sizeof(int), st);
  if (rc) return rc;
  {
    std::vector<long long> per_head(d.Hkv, 0);
    rc = copy_back(ctx, per_head.data(), d.sel_tokens + unit * d.Hkv, (size_t)d.Hkv * sizeof(long long), st);
    for (long long v : per_head) rt += v;
  }
  if (rc) return rc;
  out->tokens = s.t;
  out->evicted_end = s.E;
  out->n_spans = n;
  out->n_pending_regions = (int)s.pending.size();
  out->index_bytes = (int64_t)n * d.Hkv * kD * 2;
  out->retrieved_tokens = rt;
  out->slab_slides = s.slides;
  if (!s.pending.empty() && !s.decoding) {
    int cnt = 0;
    rc = copy_back(ctx, &cnt, d.pend_cnt + unit * d.slots + s.pending.back().slot, sizeof(int), st);
    if (rc) return rc;
    out->last_call_spans = cnt;
  }
  return LTRI_OK;
}

int ltri_sync_status(ltri_ctx* ctx, void* cuda_stream) {
  if (!ctx) return LTRI_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int w[4] = {0, 0, 0, 0};
  int rc = copy_back(ctx, w, ctx->d.status, sizeof(w), st);
  if (rc) return rc;
  if (w[0] != 0) {
    LTRI_CUDA(ctx, cudaMemsetAsync(ctx->d.status, 0, sizeof(w), st));
    LTRI_CUDA(ctx, cudaStreamSynchronize(st));
    return (w[0] <= LTRI_EINVAL && w[0] >= LTRI_ETIMEOUT) ? w[0] : LTRI_EDEVICE;
  }
  return LTRI_OK;
}

int ltri_last_cuda_error(const ltri_ctx* ctx) { return ctx ? ctx->last_cuda : 0; }

int64_t ltri_launch_count(const ltri_ctx* ctx) { return ctx ? ctx->launches : 0; }

int ltri_profile_enable(ltri_ctx* ctx, int on) {
  if (!ctx) return LTRI_EINVAL;
  ctx->profiling = on != 0;
  return LTRI_OK;
}

int ltri_profile_read(ltri_ctx* ctx, float* ms, int64_t* launches, void* cuda_stream) {
  if (!ctx || !ms || !launches) return LTRI_EINVAL;
  LTRI_CUDA(ctx, cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)));
  for (int i = 0; i < LTRI_K_COUNT; ++i) {
    ms[i] = 0.f;
    launches[i] = ctx->cls_launches[i];
    ctx->cls_launches[i] = 0;
  }
  for (auto& t : ctx->timed) {
    float e = 0.f;
    if (cudaEventElapsedTime(&e, t.a, t.b) == cudaSuccess) ms[t.cls] += e;
    ctx->free_pool.push_back(t);
  }
  ctx->timed.clear();
  return LTRI_OK;
}

const char* ltri_strerror(int code) {
  switch (code) {
    case LTRI_OK: return "ok";
    case LTRI_EINVAL: return "invalid argument";
    case LTRI_ECAPACITY: return "capacity exceeded";
    case LTRI_ESTATE: return "call order violated";
    case LTRI_ECUDA: return "CUDA runtime error";
    case LTRI_EDEVICE: return "device-side check failed";
    case LTRI_ETIMEOUT: return "device-side wait expired";
  }
  return "unknown error";
}

int ltri_span_capacity(const ltri_ctx* ctx) { return ctx ? ctx->d.cap : LTRI_EINVAL; }

int ltri_debug_read(ltri_ctx* ctx, int what, int seq, int layer, void* dst, size_t cap_bytes, size_t* bytes_out,
                    void* cuda_stream) {
  if (!ctx || seq < 0 || seq >= ctx->d.NS || layer < 0 || layer >= ctx->d.NL) return LTRI_EINVAL;
  const DevCtx& d = ctx->d;
  const size_t unit = unit_of(d, seq, layer);
  const void* src = nullptr;
  size_t bytes = 0;
  switch (what) {
    case LTRI_BUF_MAP:
      src = d.Mq + (size_t)layer * d.chunk * d.chunk;
      bytes = (size_t)d.chunk * d.chunk * sizeof(int);
      break;
    case LTRI_BUF_VOTES:
      src = d.votes + unit * d.Tpad;
      bytes = (size_t)d.Tmax * sizeof(long long);
      break;
    case LTRI_BUF_INDEX:
      src = d.KR + unit * d.Hkv * (size_t)d.cap * kD;
      bytes = (size_t)d.Hkv * d.cap * kD * 2;
      break;
    case LTRI_BUF_THETA:
      src = d.thetaq + layer;
      bytes = sizeof(long long);
      break;
    case LTRI_BUF_SCORES:
      src = d.scores + unit * d.Hkv * (size_t)d.cap;
      bytes = (size_t)d.Hkv * d.cap * sizeof(float);
      break;
    case LTRI_BUF_QREPS:
      src = d.u + (size_t)layer * d.Hkv * d.Jmax * kD;
      bytes = (size_t)d.Hkv * d.Jmax * kD * sizeof(float);
      break;
    case LTRI_BUF_NREPS:
      src = d.nrep_last + (size_t)layer * d.Jmax;
      bytes = (size_t)d.Jmax * sizeof(int);
      break;
    case LTRI_BUF_CACHE_TAGS:
      if (!d.host_kv) return LTRI_ESTATE;
      src = d.ctag + unit_of(d, seq, layer) * d.Hkv * d.cache_units;
      bytes = (size_t)d.Hkv * d.cache_units * sizeof(int);
      break;
    case LTRI_BUF_CACHE_SCORES:
      if (!d.host_kv) return LTRI_ESTATE;
      src = d.cscore + unit_of(d, seq, layer) * d.Hkv * d.cache_units;
      bytes = (size_t)d.Hkv * d.cache_units * sizeof(float);
      break;
    case LTRI_BUF_CACHE_STATS:
      if (!d.host_kv) return LTRI_ESTATE;
      src = d.cstat + unit_of(d, seq, layer) * 2;
      bytes = 2 * sizeof(unsigned long long);
      break;
    case LTRI_BUF_BALLOT:
      src = d.ballot + unit_of(d, seq, layer) * d.topk;
      bytes = (size_t)d.topk * sizeof(int);
      break;
    case LTRI_BUF_ROWSTAT:
      src = d.rowstat + (size_t)layer * d.chunk * d.Hq;
      bytes = (size_t)d.chunk * d.Hq * sizeof(float2);
      break;
    default: return LTRI_EINVAL;
  }
  if (bytes_out) *bytes_out = bytes;
  if (!dst) return LTRI_OK;
  return copy_back(ctx, dst, src, std::min(bytes, cap_bytes), static_cast<cudaStream_t>(cuda_stream));
}

int ltri_debug_segment_map(ltri_ctx* ctx, const int32_t* Mq, int m, int theta_mode, float theta, int64_t theta_q,
                           int max_spans, int32_t* pairs, int cap, int* n_out, void* cuda_stream) {
  if (!ctx || !Mq || !n_out || !pairs) return LTRI_EINVAL;
  const DevCtx& d = ctx->d;
  if (m < 1 || m > d.chunk || theta_mode < 0 || theta_mode > 2 || max_spans < 1 || max_spans > d.C) return LTRI_EINVAL;
  if (theta_mode == 1 && !(theta >= 0.f && theta <= 1.f)) return LTRI_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  LTRI_CUDA(ctx, cudaMemcpy2DAsync(d.Mq, (size_t)d.chunk * sizeof(int), Mq, (size_t)m * sizeof(int),
                                   (size_t)m * sizeof(int), m, cudaMemcpyHostToDevice, st));
  long long thq = theta_q;
  if (theta_mode == 0) thq = (long long)std::nearbyint((double)theta * (double)d.Hq * (double)kQScale);
  const int slot = d.slots - 1;
  LTRI_CUDA(ctx, launch_segment(d, 0, 0, 1, m, 0, slot, theta_mode == 1 ? 1 : 0, theta, thq, max_spans, 0, 0, nullptr,
                                st));
  int cnt = 0;
  int rc = copy_back(ctx, &cnt, d.pend_cnt + slot, sizeof(int), st);
  if (rc) return rc;
  *n_out = cnt;
  cnt = std::max(0, std::min(std::min(cnt, cap), d.Jmax));
  std::vector<int> a(cnt), b(cnt);
  rc = copy_back(ctx, a.data(), d.pend_start + (size_t)slot * d.Jmax, cnt * sizeof(int), st);
  if (rc) return rc;
  rc = copy_back(ctx, b.data(), d.pend_len + (size_t)slot * d.Jmax, cnt * sizeof(int), st);
  if (rc) return rc;
  for (int i = 0; i < cnt; ++i) {
    pairs[2 * i] = a[i];
    pairs[2 * i + 1] = b[i];
  }
  return LTRI_OK;
}

int ltri_debug_load_index(ltri_ctx* ctx, int seq, int layer, int64_t evicted_end, const int32_t* pairs, int n_spans,
                          const void* index_bf16, void* cuda_stream) {
  if (!ctx || seq < 0 || seq >= ctx->d.NS || layer < 0 || layer >= ctx->d.NL || n_spans < 0) return LTRI_EINVAL;
  const DevCtx& d = ctx->d;
  LayerState& s = ctx->at(seq, layer);
  if (n_spans > 0 && (!pairs || !index_bf16)) return LTRI_EINVAL;
  if (evicted_end != s.E) return LTRI_ESTATE;  // the cache, the votes and the pending regions stay as they are
  if (n_spans > d.cap) return LTRI_ECAPACITY;
  // the spans must cover [n_sink, E) in token order (they may overlap, as the spans of an NMS with phi > 0 do)
  long long reach = d.Ls;
  std::vector<int> st_(n_spans), ln_(n_spans);
  for (int i = 0; i < n_spans; ++i) {
    const long long a = pairs[2 * i], len = pairs[2 * i + 1];
    if (len < 1 || a < d.Ls || a > reach || a + len > s.E || (i > 0 && a < pairs[2 * i - 2])) return LTRI_EINVAL;
    reach = std::max(reach, a + len);
    st_[i] = (int)a;
    ln_[i] = (int)len;
  }
  if (reach != s.E) return LTRI_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t unit = unit_of(d, seq, layer);
  if (n_spans > 0) {
    LTRI_CUDA(ctx, cudaMemcpyAsync(d.span_start + unit * d.cap, st_.data(), n_spans * sizeof(int), cudaMemcpyHostToDevice, st));
    LTRI_CUDA(ctx, cudaMemcpyAsync(d.span_len + unit * d.cap, ln_.data(), n_spans * sizeof(int), cudaMemcpyHostToDevice, st));
    for (int g = 0; g < d.Hkv; ++g)
      LTRI_CUDA(ctx, cudaMemcpyAsync(d.KR + (unit * d.Hkv + g) * (size_t)d.cap * kD,
                                     static_cast<const __nv_bfloat16*>(index_bf16) + (size_t)g * n_spans * kD,
                                     (size_t)n_spans * kD * sizeof(__nv_bfloat16), cudaMemcpyHostToDevice, st));
  }
  LTRI_CUDA(ctx, cudaMemcpyAsync(d.n_spans + unit, &n_spans, sizeof(int), cudaMemcpyHostToDevice, st));
  LTRI_CUDA(ctx, cudaStreamSynchronize(st));  // the host buffers (and the locals above) may go away on return
  s.span_ub = n_spans;
  return LTRI_OK;
}

int ltri_debug_wait_timeout(ltri_ctx* ctx, int64_t limit_cycles, int64_t* waited_cycles, void* cuda_stream) {
  if (!ctx || !waited_cycles || limit_cycles < 1 || limit_cycles > 100000000ll) return LTRI_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  ctx->launches += 1;
  LTRI_CUDA(ctx, launch_wait_probe(ctx->d, (long long)limit_cycles, st));
  int w[4] = {0, 0, 0, 0};
  const int rc = copy_back(ctx, w, ctx->d.status, sizeof(w), st);
  if (rc) return rc;
  waited_cycles[0] = w[2];
  waited_cycles[1] = w[3];
  return LTRI_OK;
}

}  // extern "C"
