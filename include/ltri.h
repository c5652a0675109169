/* ltri.h -- C ABI of the B200 (sm_100a) streaming span-retrieval attention library.
 *
 * The library implements, per streamed chunk or decode step, the hot path of Ltri-LLM
 * (arXiv 2412.04757): segment the KV stream into semantic spans from the triangular
 * pattern of the local attention map (Sec. 3.2, Eq. 1-5, App. "NMS Input Filtration"),
 * keep one representative key (or a small key set) per span in a device-resident index
 * (Sec. 3.3.1, Eq. 6), score the queries against the index and take the top-k spans
 * (Sec. 3.4 step 2, Eq. 7-8), gather those spans' K/V and run exact softmax attention
 * over [sink | retrieved spans | local window | current tokens] (Sec. 3.4 step 3).
 *
 * Conventions
 *  - All tensor arguments are DEVICE pointers to bf16 unless stated otherwise, 16-byte
 *    aligned, dense row-major in the layout written beside the argument.
 *  - The caller owns every buffer, including the arena all library state lives in; the
 *    library never allocates or frees device memory.  The handle owns host metadata only.
 *  - Calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*) and return
 *    without synchronising unless stated.  All calls on one context must use one stream
 *    (or be ordered by the caller).
 *  - Return value: 0 (LTRI_OK) or a negative LTRI_E* code.  Parameter, state and capacity
 *    errors are detected on the host before anything is launched and leave the context
 *    unchanged (ltri_prefill_chunk_host included: it checks the whole call before its first
 *    layer group starts).  LTRI_ECUDA means the CUDA runtime refused a launch or a copy part
 *    of the way through a call; the sequence is then in an undefined state: reset it.
 *    Device-side checks record a code in a status word read by ltri_sync_status; nothing
 *    traps or spins without bound.
 *  - Numeric range.  Inputs are finite bf16 values of any magnitude for which the scaled
 *    logits q.k * softmax_scale stay below about 2000 in absolute value (the local-map
 *    pass carries the row offsets -max - log2(sum) through an fp32 accumulator clamped at
 *    that size); inside that range every softmax is exact however far a later key tile
 *    exceeds the running maximum: the prefill attention kernel notices when a tile's
 *    maximum outruns its late-moving reference maximum by more than 2^90 and flags its
 *    CTA; a second launch of the same kernel (it returns at once for CTAs without a flag)
 *    then recomputes those CTAs' work with the true maximum exchanged on every tile.
 */
#ifndef LTRI_H_
#define LTRI_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  LTRI_OK = 0,
  LTRI_EINVAL = -1,    /* bad geometry / parameter / null or misaligned pointer */
  LTRI_ECAPACITY = -2, /* tokens, sequences, spans or arena size exceeded */
  LTRI_ESTATE = -3,    /* call order violated (e.g. prefill after decode, layers out of step) */
  LTRI_ECUDA = -4,     /* a CUDA runtime call failed; see ltri_last_cuda_error */
  LTRI_EDEVICE = -5,   /* a device-side bounds or numeric-range check failed */
  LTRI_ETIMEOUT = -6   /* a bounded device-side wait expired */
};

typedef struct ltri_ctx ltri_ctx; /* opaque host-side handle */

typedef struct {
  int32_t n_layers, n_q_heads, n_kv_heads, head_dim; /* head_dim must be 128; n_q_heads % n_kv_heads == 0,
                                                        group size n_q_heads/n_kv_heads in {1,2,4,8} */
  int32_t max_seqs;                                  /* independent sequences held at once */
  int64_t max_tokens;                                /* per-sequence capacity, prefill + decode */
  int32_t chunk;                                     /* max tokens per prefill call, 16..1024, multiple of 16 */
  int32_t window;                                    /* local window L_win >= 1 (Sec. 3.4) */
  int32_t n_sink;                                    /* initial tokens L_init, 1..chunk */
  int32_t top_k;                                     /* spans retrieved per (layer, KV head), 1..64 (Eq. 8) */
  int32_t reps_per_span;                             /* index vectors per span, 1..8; 0 -> 1 (Sec. 3.3.1) */
  int32_t max_spans_per_region;                      /* NMS keeps at most this many per call; 0 -> chunk/32 */
  int32_t theta_mode;                                /* 0: theta is an absolute head-mean probability,
                                                        1: theta is a quantile level of the region map (Eq. 5) */
  float theta;                                       /* mode 1 default 0.90 */
  float softmax_scale;                               /* 0 -> 1/sqrt(head_dim) */
  uint32_t flags;                                    /* LTRI_FLAG_* */
  /* Dynamic span index vectors (Sec. 3.3.2, Eq. r_v).  rep_mode 0: every span keeps reps_per_span representatives.
   * rep_mode 1: a span of L tokens keeps round(L * exp(-rep_lambda * (1 - r_a))) of them, clamped to
   * [min_reps, max_reps] and to L, where r_a = T / (T + neighbours) on the call's head-summed Q20 region map: T is
   * the mass of the span's own triangle; the neighbours are the mass its rows give to earlier tokens of the region
   * (ratio_kind 0, "row"), the mass later rows of the region give to its columns (1, "column"), or both (2).  The
   * same count is used for the query side while the region is current and for the key side when it is indexed. */
  int32_t rep_mode;                                  /* 0 static, 1 dynamic */
  int32_t ratio_kind;                                /* 0 row, 1 column, 2 both */
  int32_t min_reps, max_reps;                        /* 1 <= min_reps <= max_reps <= 8 (rep_mode 1 only) */
  float rep_lambda;                                  /* >= 0 (rep_mode 1 only) */
  int32_t unit_tokens;                               /* retrieval granularity.  0: the k best spans are fetched.
                                                        U (multiple of 8, 8..chunk): Eq. 8 as printed -- the tokens are
                                                        cut into fixed units of U on the absolute token grid, a unit's
                                                        score is the maximum over the spans it meets, the k best units
                                                        are fetched whole (clipped to the indexed range) and
                                                        ltri_get_selected reports unit numbers (token / U) */
  int32_t nms_iou_milli;                             /* NMS IoU threshold phi in thousandths, 0..999 (App. "NMS Input
                                                        Filtration", boxes = squares on the diagonal).  0: kept spans
                                                        never overlap and the spans partition the region; > 0: kept
                                                        spans may overlap, the gaps are the runs none of them covers */
  /* Retrieval heads (Sec. 3.5).  HOST arrays of n_layers entries, read at ltri_create and not kept; NULL: no layer
   * has one.  retrieval_head[l] = -1: layer l locates evidence with all its heads (the default path).
   * retrieval_head[l] = h in [0, n_q_heads): layer l uses head h alone -- the local map of Eq. 1-4, the threshold
   * (mode 0: theta in that head's probability units), the votes of Eq. 6, the query representatives and the scores
   * of Eq. 7 (against the index of h's KV head) come from h, and the one selection serves every KV head of the layer.
   * retrieval_head_score[l] >= 0 is the head's score, its weight under LTRI_FLAG_COLLAB_VOTE (ignored where
   * retrieval_head[l] < 0; NULL: every weight 1).  Which heads these are is a property of the model; the caller
   * supplies them. */
  const int32_t* retrieval_head;
  const float* retrieval_head_score;
  /* Per-layer tables (App. "Experimental Details": theta and phi are searched per layer, lambda is larger for the
   * first layers).  HOST arrays of n_layers entries, read at ltri_create and not kept; NULL: the scalar above holds
   * for every layer.  Same meaning and range as theta, nms_iou_milli and rep_lambda. */
  const float* layer_theta;
  const int32_t* layer_nms_iou_milli;
  const float* layer_rep_lambda;
  /* Context memory on the host (Sec. 3.4: evicted tokens live in CPU memory behind a cache of memory units on the
   * GPU; used with LTRI_FLAG_HOST_KV, which needs unit_tokens > 0).
   * host_kv: caller-owned HOST memory, page-locked and mapped for the device (cudaHostAlloc / cudaHostRegister /
   * a pinned torch tensor), 256-byte aligned, ltri_host_kv_bytes(params) bytes: the K rows of every (sequence, layer,
   * KV head) slab, then the V rows.  cache_units: memory units of unit_tokens tokens kept in device memory per
   * (sequence, layer, KV head), top_k..128 (2 * top_k with LTRI_FLAG_PERSIST_DECODE); score_decay in [0, 1]: at every
   * retrieval the usage score of a cached unit becomes score_decay * score (+ 1 if the retrieval names it), and a
   * unit that has to make room is the one with the lowest score (lowest slot among equals). */
  void* host_kv;
  size_t host_kv_bytes;
  int32_t cache_units;
  float score_decay;
  void* arena;                                       /* caller-owned device memory, 256-byte aligned */
  size_t arena_bytes;                                /* >= ltri_arena_bytes(params) */
} ltri_params;

enum {
  LTRI_FLAG_NONE = 0,
  /* Persistent mechanism (Sec. 3.5): the spans selected by the last prefill call of a sequence stay in the attention
   * of every decode step, next to the spans the step retrieves itself. */
  LTRI_FLAG_PERSIST_DECODE = 1,
  /* Reserve two staging sets in the arena (q, k, v and out of one full call each) for ltri_prefill_chunk_host. */
  LTRI_FLAG_HOST_STAGING = 2,
  /* Collaborative voting (Sec. 3.5); needs unit_tokens > 0 (unit numbers mean the same tokens in every layer) and
   * retrieval_head.  Every layer with a retrieval head casts a ballot: its k best units by its own scores, weighted
   * by retrieval_head_score.  Layer K ranks its units by tally -- the summed weights of the ballots of layers 0..K
   * (fp32, ascending layer order) that name the unit -- then by its own score, then by lower unit number, and fetches
   * the first k.  The layers of a chunk (or decode step) must be submitted in ascending order, each layer of a
   * sequence exactly once, so that the ballots a layer reads are those of the same chunk. */
  LTRI_FLAG_COLLAB_VOTE = 4,
  /* Segmentation per memory unit (Sec. 3.3: every block is divided into spans); needs unit_tokens > 0.  The part of a
   * call's region inside each unit of unit_tokens tokens (absolute grid) is segmented on its own: only intervals
   * inside one unit are candidates, NMS keeps max_spans_per_region spans PER UNIT (0 -> unit_tokens/32), uncovered
   * runs are cut at the unit boundaries; theta is still that of the whole region.  Spans never cross a unit boundary.
   * max_spans_per_region * (units a call can touch = (chunk + unit_tokens - 2) / unit_tokens + 1) must be <= 64. */
  LTRI_FLAG_SEGMENT_PER_UNIT = 8,
  /* Host-memory pager for retrieved tokens (Sec. 3.4, "Implementation Details": GPU cache size, score decay).  When a
   * region leaves the window its K/V rows are also copied to host_kv (on an internal stream, overlapping the call's
   * attention).  Retrieved units are then no longer read from the device-resident K/V slabs: a unit found in the
   * (sequence, layer, KV head)'s unit cache is read from there; a missing one is pulled from host_kv over the bus by
   * the top-k kernel itself, into the slot of the unit with the lowest usage score.  Prefill calls pack the units'
   * rows from the cache slots (the unit the indexed range ends in, while still growing, straight from the mirror);
   * decode steps attend over the cache slots in place.  Results are bit-identical to the default path.
   * The device then keeps, per (sequence, layer, KV head), only the sink and a sliding window of
   * 2 * (window + 2 * chunk) + 256 rows instead of max_tokens rows: when the window region is full the rows since the
   * last eviction are moved to its start (ltri_stats.slab_slides counts these moves).  Decode never evicts, so a
   * sequence can take about window + 2 * chunk decode steps beyond that before ltri_decode_step returns
   * LTRI_ECAPACITY.  Needs the tensor-core kernels. */
  LTRI_FLAG_HOST_KV = 16
};

typedef struct {
  int64_t tokens;          /* tokens appended so far (prefill + decode) */
  int64_t evicted_end;     /* E: tokens [n_sink, E) are covered by indexed spans */
  int32_t n_spans;         /* indexed spans N_s */
  int32_t n_pending_regions;
  int64_t index_bytes;     /* N_s * n_kv_heads * head_dim * 2 */
  int64_t retrieved_tokens; /* sum of the lengths of the spans selected by the last call, over KV heads */
  int32_t last_call_spans; /* spans the last prefill call cut its region into */
  int32_t slab_slides;     /* LTRI_FLAG_HOST_KV: times the live rows of this layer's sliding K/V slabs were moved to the
                              start of their window region (0 in a resident context) */
} ltri_stats;

/* Bytes of device memory the arena must provide for these parameters (host only; the
 * `arena` and `arena_bytes` fields are ignored).  Returns 0 if the parameters are invalid. */
size_t ltri_arena_bytes(const ltri_params* p);

/* Bytes of host memory that host_kv must provide under LTRI_FLAG_HOST_KV (0 if the parameters are invalid). */
size_t ltri_host_kv_bytes(const ltri_params* p);

/* Create a context over the caller's arena and initialise its device state on
 * `cuda_stream` (synchronises that stream once).  Streaming attention with parameters
 * init / window / chunk / top-K as in Sec. "Implementation Details". */
int ltri_create(const ltri_params* p, void* cuda_stream, ltri_ctx** out);

/* Free the host handle.  Device memory stays with the caller. */
int ltri_destroy(ltri_ctx* ctx);

/* Forget all tokens of one sequence so that its slot can stream a new context. */
int ltri_reset_sequence(ltri_ctx* ctx, int seq, void* cuda_stream);

/* One streamed prefill call (Sec. 3.4, steps 1-3) for `n_tokens` (1..chunk) new tokens of
 * sequence `seq`, for layers [layer_begin, layer_begin+layer_count).  Every call is a region
 * of its own (it is segmented once, while current) and stays pending until it has left the
 * window; a context has room for window/chunk (rounded up) + 8 pending regions, so a caller
 * that streams calls much shorter than `chunk` gets LTRI_ECAPACITY once more calls than that
 * fit into the window (e.g. window 4096, chunk 512: the 17th 64-token call in a row).
 *   q   [layer_count][n_tokens][n_q_heads ][head_dim]
 *   k,v [layer_count][n_tokens][n_kv_heads][head_dim]   (copied into the library's cache)
 *   out [layer_count][n_tokens][n_q_heads ][head_dim]   (fully overwritten)
 * Per layer: regions that left the window are indexed (Eq. 6); the local map over
 * [sink | local | current] is computed and the call's own region is segmented (Eq. 1-5);
 * query representatives are scored against the index and the top-k spans selected
 * (Eq. 7-8); attention runs over [sink | selected spans | local | current (causal)].
 * Each (sequence, layer) is its own stream: its tokens must arrive in order, and a layer
 * that already decoded cannot prefill again (LTRI_ESTATE).  The layers of one call must
 * all be at the same position. */
int ltri_prefill_chunk(ltri_ctx* ctx, int seq, int layer_begin, int layer_count, int n_tokens, const void* q,
                       const void* k, const void* v, void* out, void* cuda_stream);

/* ltri_prefill_chunk for a caller whose tensors live in HOST memory (pinned memory for the copies to overlap): same
 * shapes and meaning, but q_host, k_host, v_host and out_host are host pointers.  The context must have been created
 * with LTRI_FLAG_HOST_STAGING.  The layers of a call are independent, so the call is carried out in up to four layer
 * groups: a group's inputs go up on an internal copy stream while the previous group computes on `cuda_stream` and the
 * group before that sends its output down on a second internal stream; two staging sets alternate between calls, so
 * the copies of one call also overlap the kernels of its neighbours.  The host inputs must stay valid, and out_host
 * must not be read, until the work is done: make a stream wait for it with ltri_host_outputs_ready (or synchronise
 * the device).  All parameter, state and capacity checks of the whole call are made before the first group is
 * enqueued, so those errors leave the sequence unchanged; only LTRI_ECUDA can leave some layers advanced (reset the
 * sequence then).  The groups are fixed layer ranges of the context (a quarter of its layers each), so calls of any
 * size and layer range may follow each other.
 * The streamed-context setting of Sec. 3.4 with the context memory on the host side. */
int ltri_prefill_chunk_host(ltri_ctx* ctx, int seq, int layer_begin, int layer_count, int n_tokens, const void* q_host,
                            const void* k_host, const void* v_host, void* out_host, void* cuda_stream);

/* Make `cuda_stream` wait until every output of earlier ltri_prefill_chunk_host calls has reached host memory. */
int ltri_host_outputs_ready(ltri_ctx* ctx, void* cuda_stream);

/* One decode step (Sec. 3.5: during decoding the current block is one token) for `n_seqs` sequences.
 *   seq_ids  HOST array [n_seqs] of distinct sequence slots
 *   q   [n_seqs][layer_count][n_q_heads ][head_dim]
 *   k,v [n_seqs][layer_count][n_kv_heads][head_dim]
 *   out [n_seqs][layer_count][n_q_heads ][head_dim]
 * Appends the token, scores the summed query of each KV-head group against the index,
 * selects top-k spans and attends over [sink | selected spans | every token since the
 * last eviction].  Decode never evicts, votes or segments. */
int ltri_decode_step(ltri_ctx* ctx, const int32_t* seq_ids, int n_seqs, int layer_begin, int layer_count,
                     const void* q, const void* k, const void* v, void* out, void* cuda_stream);

/* ---- introspection (synchronise `cuda_stream`; HOST output buffers) ---- */

/* Indexed spans of (seq, layer) as {start,len} pairs in token order; *n_out = N_s (even if > cap). */
int ltri_get_spans(ltri_ctx* ctx, int seq, int layer, int32_t* start_len_pairs, int cap, int* n_out, void* cuda_stream);
/* Spans of the regions still inside the window, oldest first, as {start,len} pairs. */
int ltri_get_pending_spans(ltri_ctx* ctx, int seq, int layer, int32_t* start_len_pairs, int cap, int* n_out,
                           void* cuda_stream);
/* Span ids chosen by the last call, ascending, -1 padded: ids[n_kv_heads][top_k]. */
int ltri_get_selected(ltri_ctx* ctx, int seq, int layer, int32_t* ids, void* cuda_stream);
int ltri_get_stats(ltri_ctx* ctx, int seq, int layer, ltri_stats* out, void* cuda_stream);
/* First device-side error recorded since the last call of this function (then cleared). */
int ltri_sync_status(ltri_ctx* ctx, void* cuda_stream);
/* cudaError_t of the last failed runtime call (0 if none). */
int ltri_last_cuda_error(const ltri_ctx* ctx);
const char* ltri_strerror(int code);

/* ---- measurement hooks ---- */

/* Kernel classes reported by ltri_profile_read. */
enum {
  LTRI_K_APPEND = 0,   /* K/V cache append of a call that evicts nothing (and of the two-launch decode path) */
  LTRI_K_EVICT,        /* eviction + span index build (Eq. 6), together with the call's K/V cache append, which runs
                          beside it */
  LTRI_K_ATTN_LOCAL,   /* prefill attention over sink | local | current */
  LTRI_K_MAP,          /* local-map pass: votes + region map (Eq. 4, Eq. 6) */
  LTRI_K_SEGMENT,      /* theta, cumulative sums, anti-diagonal filter, NMS, query representatives */
  LTRI_K_SCORE_TOPK,   /* prefill similarity scores + top-k (Eq. 7-8) */
  LTRI_K_ATTN_RET,     /* prefill attention over the retrieved spans + merge */
  LTRI_K_DEC_RETRIEVE, /* decode scores + top-k */
  LTRI_K_DEC_ATTN,     /* decode split-KV attention + merge */
  LTRI_K_PAGER_PULL,   /* host-memory pager: pulls of missing units + gather (on the pager's own stream: overlaps
                          the other classes) */
  LTRI_K_COUNT
};
/* Kernels launched by this context since it was created (host counter). */
int64_t ltri_launch_count(const ltri_ctx* ctx);
/* While enabled, every kernel class of a call is bracketed by CUDA events on the call's stream. */
int ltri_profile_enable(ltri_ctx* ctx, int on);
/* Synchronises the stream; writes, per class, the summed event time in ms (0 if profiling was off) and the
 * kernels launched since the previous read: ms[LTRI_K_COUNT], launches[LTRI_K_COUNT] (HOST). */
int ltri_profile_read(ltri_ctx* ctx, float* ms, int64_t* launches, void* cuda_stream);

/* ---- debug / test entry points ---- */

enum {
  LTRI_BUF_MAP = 1,      /* int32 [chunk][chunk]: the last prefill call's head-summed Q20 region map (row-major,
                            leading dimension chunk; entries above the diagonal are unspecified) */
  LTRI_BUF_VOTES = 2,    /* int64 [max_tokens]: accumulated votes v_x in Q20 units (Eq. 6) */
  LTRI_BUF_INDEX = 3,    /* bf16  [n_kv_heads][span_capacity][head_dim]: the span index K^R */
  LTRI_BUF_THETA = 4,    /* int64 [1]: theta of the last prefill call in Q20 head-sum units */
  LTRI_BUF_SCORES = 5,   /* float [n_kv_heads][span_capacity]: similarity scores of the last call (Eq. 7) */
  LTRI_BUF_QREPS = 6,    /* float [n_kv_heads][J][head_dim]: summed query representatives; J = 2*max_spans_per_region+1
                            (times the units a call can touch under LTRI_FLAG_SEGMENT_PER_UNIT) */
  LTRI_BUF_NREPS = 8,    /* int32 [2*max_spans_per_region+1]: representative counts of the spans of the last prefill
                            call's region (Sec. 3.3.2) */
  LTRI_BUF_CACHE_TAGS = 10,   /* int32 [n_kv_heads][cache_units]: unit held by every slot of the unit cache, -1 empty */
  LTRI_BUF_CACHE_SCORES = 11, /* float [n_kv_heads][cache_units]: usage scores of the slots */
  LTRI_BUF_CACHE_STATS = 12,  /* int64 [2]: units found in the cache / pulled from the host so far (all KV heads) */
  LTRI_BUF_BALLOT = 9,   /* int32 [top_k]: the layer's own ballot under LTRI_FLAG_COLLAB_VOTE (ascending unit numbers,
                            -1 padded; all -1 for a layer without a retrieval head) */
  LTRI_BUF_ROWSTAT = 7   /* float [chunk][n_q_heads][2]: reference maximum m (logits * scale * log2(e); may lag the true
                            row maximum by up to 8) and the matching row sum of exp2(logit - m) of the local softmax
                            of the last prefill call */
};
/* Copy an internal buffer of (seq, layer) to HOST memory `dst`; *bytes_out = full size.  Synchronises. */
int ltri_debug_read(ltri_ctx* ctx, int what, int seq, int layer, void* dst, size_t cap_bytes, size_t* bytes_out,
                    void* cuda_stream);
/* Span capacity per (seq, layer) (leading dimension of LTRI_BUF_INDEX / LTRI_BUF_SCORES). */
int ltri_span_capacity(const ltri_ctx* ctx);

/* Run the segmenter (Eq. 4-5 cumulative sums, anti-diagonal filter, greedy NMS with IoU threshold 0, gap
 * fill) on a caller-supplied HOST map Mq [m][m] int32 row-major (lower triangle used, 1 <= m <= chunk).
 * theta_mode/theta as in ltri_params, except mode 2: `theta_q` is given directly in map units.
 * Writes {start,len} pairs (HOST) partitioning [0,m); uses layer 0's scratch of the context.  Synchronises. */
int ltri_debug_segment_map(ltri_ctx* ctx, const int32_t* Mq, int m, int theta_mode, float theta, int64_t theta_q,
                           int max_spans, int32_t* start_len_pairs, int cap, int* n_out, void* cuda_stream);

/* Bring-up hook: replace the span table and the span index K^R of (seq, layer) -- what Sec. 3.3 builds from the
 * evicted tokens and Sec. 3.4 step 2 (Eq. 7-8) scores against -- with a state computed elsewhere, so that retrieval
 * and attention can be driven from spans and index vectors the library did not produce itself.
 *   evicted_end   must equal the layer's current E (ltri_stats.evicted_end): the K/V cache, the votes and the
 *                 pending regions are left as they are (LTRI_ESTATE otherwise)
 *   start_len_pairs HOST int32 [n_spans][2], in token order, covering [n_sink, E) without a gap (spans may overlap,
 *                 as those of an NMS with phi > 0 do); n_spans = 0 only if E = n_sink
 *   index_bf16    HOST bf16 [n_kv_heads][n_spans][head_dim]
 * n_spans beyond ltri_span_capacity is LTRI_ECAPACITY.  Synchronises `cuda_stream`; the host buffers are not kept. */
int ltri_debug_load_index(ltri_ctx* ctx, int seq, int layer, int64_t evicted_end, const int32_t* start_len_pairs,
                          int n_spans, const void* index_bf16, void* cuda_stream);

/* Test hook for the bounded device-side waits (no counterpart in the paper; failure detection).  Runs a one-CTA
 * kernel in which one thread waits, for at most `limit_cycles` SM clock cycles (1..10^8), on a barrier that nothing
 * ever completes, while a second thread waits on it with the context's normal limit.  The first wait expires and
 * raises the CTA's abort flag, which releases the second; the kernel then records LTRI_ETIMEOUT in the status word
 * the way the tensor-core kernels do, so the next ltri_sync_status returns it (and clears it).  Nothing faults or
 * hangs, and the context stays usable.  waited_cycles HOST int64 [2]: cycles each of the two waits lasted (-1: the
 * wait reported success).  Synchronises `cuda_stream`. */
int ltri_debug_wait_timeout(ltri_ctx* ctx, int64_t limit_cycles, int64_t* waited_cycles, void* cuda_stream);

/* ---- allocation-free entry point ---- */

/* The paper has no counterpart for this call; it exists for callers that cannot allocate device memory at the
 * point of use (code inside a fully committed memory pool, plugins of a host that forbids cudaMalloc after
 * start-up, service threads that must stay off the allocator).  It runs the same segmenter as
 * ltri_debug_segment_map, but needs no context and no arena: its scratch is a fixed array inside the library
 * image (about 0.5 MiB, held by every GPU that loads the library until the process exits).
 *   Mq     DEVICE int32 [m][m] dense row-major map (lower triangle used), 1 <= m <= LTRI_STATIC_SEGMENT_MAX_M,
 *          in the memory of the CURRENT device (the scratch that is used is the current device's; a pointer that
 *          the runtime attributes to another device is LTRI_EINVAL)
 *   theta_q threshold in map units (Eq. 5), max_spans 1..64 (NMS cap)
 *   pairs  DEVICE int32 [cap_pairs][2]: {start,len} spans partitioning [0,m); n_out DEVICE int32[1]: span count.
 *          At most cap_pairs pairs are written; *n_out is the full count even when it exceeds cap_pairs (the
 *          segmenter yields at most 2 * max_spans + 1 spans).  If a device-side check of the segmenter fails,
 *          *n_out is the negative LTRI_E* code instead and no pair is valid.
 * Larger m or max_spans return LTRI_ECAPACITY and launch nothing.  The call allocates nothing and returns
 * without synchronising.  The first call on each device also looks up the scratch array's device address; make
 * that first call outside any stream capture.  All calls share the one scratch array, which keeps the previous
 * call's contents (the call clears what has to start at zero), so two calls that overlap on the GPU race: keep
 * them on one stream or order them yourself. */
#define LTRI_STATIC_SEGMENT_MAX_M 256
int ltri_segment_map_static(const int32_t* Mq, int m, int64_t theta_q, int max_spans, int32_t* pairs, int cap_pairs,
                            int32_t* n_out, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* LTRI_H_ */
