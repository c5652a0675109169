// Shared declarations of the ltri CUDA library (sm_100a): the device-side view of a
// context and the host launch wrappers of every kernel file.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ltri {

constexpr int kD = 128;               // head_dim (fixed)
constexpr int kQBits = 20;            // fixed-point fraction bits of the local attention map
constexpr float kQScale = 1048576.0f;
constexpr int kMaxReps = 8;
constexpr int kMaxTopK = 64;
constexpr int kMaxDecSplit = 32;
constexpr int kMaxRanges = 2 * kMaxTopK + 2;  // sink + local + the spans of this step's and of the persistent selection
constexpr float kMapMargin = 0.0078125f;          // safety margin (in log2 units) of the map pass's skip test
constexpr float kMapScale = 0.4972997117f;         // 2^-(1 + kMapMargin)
constexpr int kTokPad = 128;          // rows of slack after every K/V slab so tile over-reads stay inside it
constexpr int kTcMaxCtas = 1024;      // most persistent CTAs the tensor-core attention kernel is launched with
constexpr long long kDefaultWaitLimit = 2000000000ll;  // device-side waits give up after about a second

// Device-side view of one context.  Passed to kernels by value.
struct DevCtx {
  int NL, Hq, Hkv, G, NS;
  long long Tpad;        // token capacity of a (seq, layer): max_tokens + slack (votes, host mirror of the pager)
  long long SR;          // rows of a per-(seq, layer, KV head) K/V slab.  Resident context: Tpad, row = token.
                         // Paged context (sliding slab): rows [0, Ls) hold the sink for good; behind them, from row
                         // Lsp on, sits the window: the row of token tok is tok - shift, where shift = (first token
                         // the window region holds) - Lsp moves up whenever the host compacts the slab
  int paged;             // 1: sliding slabs (host-memory pager)
  int Lsp;               // first row of the window region of a sliding slab
  long long Tmax;
  int chunk, W, Ls, topk, reps, C, Jmax, cap, slots;
  int rcap;              // token ranges kept per (seq, layer, KV head): 2 * top_k + 2
  int phi_milli;         // NMS IoU threshold in thousandths (0: spans never overlap)
  int unit;              // retrieval granularity: 0 = span, U > 0 = units of U tokens (Eq. 8 as printed)
  int seg_unit;          // > 0: every unit of this many tokens is segmented on its own (C spans kept per unit)
  int persist;           // decode keeps the spans selected by the last prefill call (Sec. 3.5, persistent mechanism)
  int theta_mode;
  float theta, scale;
  int rep_mode, ratio_kind, min_reps, max_reps;  // dynamic span index vectors (Sec. 3.3.2); rep_mode 0: static count
  float rep_lambda;
  // persistent state
  __nv_bfloat16* Kc;     // [NS][NL][Hkv][SR][128]
  __nv_bfloat16* Vc;
  long long* votes;      // [NS][NL][Tpad]
  int* span_start;       // [NS][NL][cap]
  int* span_len;
  int* n_spans;          // [NS][NL]
  __nv_bfloat16* KR;     // [NS][NL][Hkv][cap][128]
  int* pend_start;       // [NS][NL][slots][Jmax]
  int* pend_len;
  int* pend_cnt;         // [NS][NL][slots]
  int* pend_nrep;        // [NS][NL][slots][Jmax]  representative count of every pending span
  int* sel;              // [NS][NL][Hkv][topk]  ascending ids, -1 padded
  int* persist_sel;      // [NS][NL][Hkv][topk]  selection of the last prefill call, kept through decode
  // retrieval heads and collaborative voting (Sec. 3.5)
  int vote;              // rank units by the tally of the layers' ballots before their own scores
  const int* ret_head;   // [NL]  retrieval head of the layer, -1 none; nullptr: no layer has one
  const float* head_w;   // [NL]  its score = the weight of the layer's ballot
  int* ballot;           // [NS][NL][topk]  own top-k units of a layer with a retrieval head (ascending, -1 padded)
  // host-memory pager (Sec. 3.4): evicted rows mirrored in mapped host memory, unit cache in device memory
  int host_kv;                  // 1: retrieved units of prefill calls come from the unit cache / the host mirror
  int cache_units;              // slots per (seq, layer, KV head)
  float score_decay;
  const __nv_bfloat16* hostK;   // [NS][NL][Hkv][Tpad][128] in mapped host memory (device-visible address)
  const __nv_bfloat16* hostV;
  __nv_bfloat16* Kcache;        // [NS][NL][Hkv][cache_units][unit][128]
  __nv_bfloat16* Vcache;
  int* ctag;                    // [NS][NL][Hkv][cache_units]  unit held by the slot, -1 empty
  float* cscore;                // [NS][NL][Hkv][cache_units]  usage score
  unsigned long long* cstat;    // [NS][NL][2]  hits, misses
  // what a prefill call's top-k kernel asks k_pull_pack to move, per (seq, layer, KV head): the units named (ascending),
  // each with the cache slot that holds it (-1: read from the mirror; bit 16: the slot has to be filled first) and
  // its valid token range
  int* pl_id;                   // [NS*NL][Hkv][2 * kMaxTopK]
  int* pl_src;
  int* pl_start;
  int* pl_len;
  int* pl_cnt;                  // [NS*NL][Hkv]
  int* rng_koff;                // [NS*NL][Hkv][rcap]  decode: K row of a range's first token, counted from Kc (a slab
                                //                     row or a unit-cache row; the V row follows from it)
  // per-layer tables of the paper's configuration appendix (nullptr: the scalar holds for every layer)
  const float* theta_l;  // [NL]  theta
  const int* phi_l;      // [NL]  NMS IoU threshold in thousandths
  const float* lambda_l; // [NL]  lambda of Eq. r_v
  long long* sel_tokens; // [NS][NL][Hkv]  retrieved tokens of the last call
  // per-layer scratch of the prefill call in flight
  int* Mq;               // [NL][chunk][chunk]
  long long* Rsuf;       // [NL][chunk][chunk]
  long long* best;       // [NL][2*chunk]
  long long* thetaq;     // [NL]
  float2* rowstat;       // [NL][chunk][Hq]   (reference maximum m in scaled log2 units, row sum l)
  float* rowq;           // [NL][chunk][Hq]   -m - log2(l) + 21 + kMapMargin: offset that turns a scaled logit into
                         //                   log2 of its Q20 probability (see kernels_map_tc.cu)
  float* Oacc;           // [NL][chunk][Hq][128]  unnormalised accumulator of the local part
  float* u;              // [NL][Hkv][Jmax][128]  summed query representatives
  __nv_bfloat16* Kg;     // [NL][Hkv][Rcap][128]  keys of the spans selected for the call in flight, packed
  __nv_bfloat16* Vg;     //                       (directly behind Kg) their values
  int* gcnt;             // [NL][Hkv]             packed rows (retrieved tokens) per KV head
  long long Rcap;        // row capacity of a packed slab: top_k spans of at most `chunk` tokens, rounded up
  int* Jcnt;             // [NL]
  int* nrep_last;        // [NL][Jmax]  representative counts of the spans of the call in flight
  // per-(seq,layer) scratch
  float* scores;         // [NS*NL][Hkv][cap]
  int* rng_start;        // [NS*NL][Hkv][rcap]
  int* rng_len;
  int* rng_cnt;          // [NS*NL][Hkv]
  float* dec_part;       // [NS*NL][Hq][kMaxDecSplit][128+2]
  int* status;           // [4]: first error code, detail...
  int* tc_redo;          // [kTcMaxCtas]  per CTA of the tensor-core attention kernel: its work has to be redone
  long long wait_limit;  // upper bound of any single device-side wait, in SM clock cycles
};

__host__ __device__ inline size_t unit_of(const DevCtx& c, int seq, int layer) { return (size_t)seq * c.NL + layer; }

// Row of token `tok` inside its K/V slab (see DevCtx::SR).  Sink tokens are also written to their window row while
// they are inside the window, so a range that starts in the window may be read with window rows throughout.
__host__ __device__ inline long long slab_row(const DevCtx& c, long long tok, long long shift) {
  return (c.paged && tok >= c.Ls) ? tok - shift : tok;
}

#ifdef __CUDACC__
// Retrieval head of a layer (Sec. 3.5): -1 when the layer locates evidence with all its heads.
__device__ __forceinline__ int ret_head_of(const DevCtx& c, int layer) { return c.ret_head ? c.ret_head[layer] : -1; }
#endif

// Decode batch descriptor (passed by value; at most 64 sequences per launch).
constexpr int kDecBatch = 64;
struct DecBatch {
  int n;
  int seq[kDecBatch];
  int pos[kDecBatch];        // position of the new token
  int loc_begin[kDecBatch];  // E' of the sequence/layer
  int src[kDecBatch];        // index into the caller's [n_seqs] arrays
  long long shift[kDecBatch];  // sliding slabs: token - shift = row of the sequence's window tokens
};

struct EvictArgs {
  int seq, layer_begin;
  int nslots;
  int slot[8];
  long long shift;  // sliding slabs: token - shift = row
  int release;      // let the kernel launched behind this one (the call's append kernel) start at once
};

struct PrefillArgs {
  int seq, layer_begin, layer_count;
  int n, t0;
  int sink_end, loc_begin;  // sink = [0,sink_end), local = [loc_begin,t0)
  int reg_start, m;         // region [reg_start, t0+n), m tokens
  int slot;                 // pending slot of this region (-1 if the region is empty)
  long long shift;          // sliding slabs: token - shift = row of the window tokens (0 in a resident context)
  const __nv_bfloat16* q;   // [layer_count][n][Hq][128]
  const __nv_bfloat16* k;
  const __nv_bfloat16* v;
  __nv_bfloat16* out;
};

// ---- launch wrappers (each returns the cudaError_t of the launch) -------------------
cudaError_t launch_init(const DevCtx& c, int seq /* -1: all */, cudaStream_t s);
cudaError_t launch_append_prefill(const DevCtx& c, const PrefillArgs& a, bool clear_maps, bool late_wait, cudaStream_t s);
cudaError_t launch_append_decode(const DevCtx& c, const DecBatch& b, int layer_begin, int layer_count, int n_seqs_total,
                                 const __nv_bfloat16* k, const __nv_bfloat16* v, cudaStream_t s);
cudaError_t launch_evict_index(const DevCtx& c, const EvictArgs& a, int layer_count, cudaStream_t s);
// segmenter on Mq of the given layers; writes spans (absolute tokens = reg_start + x) into pending slot `slot`
// and, when q != nullptr, the summed query representatives of every span.  theta_mode 0/2: theta_q_abs is used.
cudaError_t launch_segment(const DevCtx& c, int seq, int layer_begin, int layer_count, int m, int reg_start, int slot,
                           int theta_mode, float theta, long long theta_q_abs, int max_spans, int n, int t0,
                           const __nv_bfloat16* q, cudaStream_t s, bool tables = false, int seg_unit = 0);
cudaError_t launch_score_prefill(const DevCtx& c, const PrefillArgs& a, int span_bound, cudaStream_t s);
// tensor-core version of launch_score_prefill (split-bf16 representatives)
cudaError_t launch_score_prefill_mma(const DevCtx& c, const PrefillArgs& a, int span_bound, cudaStream_t s);
cudaError_t launch_topk_prefill(const DevCtx& c, const PrefillArgs& a, cudaStream_t s);
// host-memory pager: pulls of the missing units + gather of the selected units' rows (after launch_topk_prefill)
cudaError_t launch_pull_pack(const DevCtx& c, const PrefillArgs& a, cudaStream_t s);
cudaError_t launch_score_decode(const DevCtx& c, const DecBatch& b, int layer_begin, int layer_count, int n_seqs_total,
                                const __nv_bfloat16* q, int span_bound, cudaStream_t s);
// decode scores + top-k + range list in one launch (span_bound <= dec_retrieve_fused_max_spans())
cudaError_t launch_dec_retrieve_fused(const DevCtx& c, const DecBatch& b, int layer_begin, int layer_count,
                                      const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v, int span_bound, bool force_cluster, int threads,
                                      cudaStream_t s);
int dec_retrieve_fused_max_spans();
cudaError_t launch_topk_decode(const DevCtx& c, const DecBatch& b, int layer_begin, int layer_count, cudaStream_t s);

// prefill attention.  phase 0: local part over sink|local|cur, stores state (+ final output if `final`);
// phase 1: continues from the stored state over the selected spans and writes the output; phase 2 (tensor-core
// kernel only): the same result, with the selected spans accumulated from scratch and merged with the stored state.
// The tensor-core version is two launches: the second redoes, with exact per-tile maxima, the work of CTAs that met
// logits too far above their running reference (it returns at once otherwise).
cudaError_t launch_attn_prefill(const DevCtx& c, const PrefillArgs& a, int phase, bool final, cudaStream_t s);
// tcgen05/TMEM/TMA version of launch_attn_prefill (same contract) and its availability check
// host storage for a context's tensor maps: five box heights of the K/V cache, the index, five of the packed slabs
constexpr int kTcMapBytes = 11 * 128;
cudaError_t launch_attn_prefill_tc(const DevCtx& c, const PrefillArgs& a, int phase, bool final, const void* kv_maps,
                                   cudaStream_t s);
bool tc_attention_supported(const DevCtx& c);
bool tc_encode_kv_maps(const DevCtx& c, void* out_bytes);
cudaError_t launch_map_pass_tc(const DevCtx& c, const PrefillArgs& a, const void* kv_maps, cudaStream_t s);
// tcgen05 version of the prefill scores; returns cudaErrorNotSupported when the query-span count does not fit
cudaError_t launch_score_prefill_tc(const DevCtx& c, const PrefillArgs& a, int span_bound, const void* kv_maps,
                                    cudaStream_t s);
bool score_tc_supported(const DevCtx& c);
cudaError_t launch_map_pass(const DevCtx& c, const PrefillArgs& a, cudaStream_t s);

cudaError_t launch_decode_attn(const DevCtx& c, const DecBatch& b, int layer_begin, int layer_count, int n_seqs_total,
                               const __nv_bfloat16* q, __nv_bfloat16* out, int nsplit, cudaStream_t s);

// test kernel for the bounded waits: one wait with `short_limit` cycles on a barrier nothing completes (kernels_probe.cu)
cudaError_t launch_wait_probe(const DevCtx& c, long long short_limit, cudaStream_t s);

// ---- programmatic dependent launch -------------------------------------------------------
// The kernels of a prefill call and of a decode step form a chain on one stream.  Launched through launch_chained,
// a kernel's launch is prepared while its predecessor is still running and its CTAs start as soon as the predecessor
// grid has finished; it touches global memory only after chain_wait(), which returns once that grid's writes are
// visible.  No kernel releases its successor early: with one large CTA per SM (or a tuned number of them) the
// successor's CTAs would only take resources away from the kernel that is still working (measured: decode 0.250
// instead of 0.225 ms per step).  Launched the ordinary way, chain_wait() does nothing.
#ifdef __CUDACC__
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the kernel launched behind this one start now instead of when this grid has finished.  Used in one place only:
// the eviction kernel (a few CTAs) releases the call's append kernel, which does not depend on it and whose threads
// wait for the eviction kernel at their end instead of their beginning, so that the two run side by side and
// everything behind the append kernel still follows both.
__device__ __forceinline__ void chain_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                  Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// ---- small device helpers --------------------------------------------------------------
__device__ __forceinline__ void set_status(const DevCtx& c, int code, int detail) {
  if (atomicCAS(&c.status[0], 0, code) == 0) c.status[1] = detail;
}

__device__ __forceinline__ long long shfl_xor_ll(long long v, int m) {
  int lo = __shfl_xor_sync(0xffffffffu, (int)(v & 0xffffffffll), m);
  int hi = __shfl_xor_sync(0xffffffffu, (int)(v >> 32), m);
  return ((long long)hi << 32) | (unsigned int)lo;
}
__device__ __forceinline__ long long shfl_up_ll(long long v, int d) {
  int lo = __shfl_up_sync(0xffffffffu, (int)(v & 0xffffffffll), d);
  int hi = __shfl_up_sync(0xffffffffu, (int)(v >> 32), d);
  return ((long long)hi << 32) | (unsigned int)lo;
}
__device__ __forceinline__ long long shfl_ll(long long v, int src) {
  int lo = __shfl_sync(0xffffffffu, (int)(v & 0xffffffffll), src);
  int hi = __shfl_sync(0xffffffffu, (int)(v >> 32), src);
  return ((long long)hi << 32) | (unsigned int)lo;
}

// Warp-cooperative choice of the min(reps,len) tokens of [start,start+len) with the largest votes
// (ties -> lower token index), returned ascending in toks[] (Eq. 6 / Sec. 3.3.1).  All lanes get the result.
__device__ inline int select_reps(const long long* __restrict__ votes, int start, int len, int reps, int* toks) {
  const int lane = threadIdx.x & 31;
  int cnt = reps < len ? reps : len;
  for (int r = 0; r < cnt; ++r) {
    long long bv = (long long)0x8000000000000000ull;
    int bi = 0x7fffffff;
    for (int i = lane; i < len; i += 32) {
      int tok = start + i;
      bool used = false;
      for (int q = 0; q < r; ++q) used |= (toks[q] == tok);
      if (used) continue;
      long long v = votes[tok];
      if (v > bv || (v == bv && tok < bi)) {
        bv = v;
        bi = tok;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      long long ov = shfl_xor_ll(bv, o);
      int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ov > bv || (ov == bv && oi < bi)) {
        bv = ov;
        bi = oi;
      }
    }
    toks[r] = bi;
  }
  for (int a = 1; a < cnt; ++a) {  // insertion sort, ascending token
    int x = toks[a], b = a - 1;
    while (b >= 0 && toks[b] > x) {
      toks[b + 1] = toks[b];
      --b;
    }
    toks[b + 1] = x;
  }
  return cnt;
}

}  // namespace ltri
