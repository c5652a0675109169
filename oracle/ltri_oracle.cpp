// Ltri-LLM streaming attention -- CPU ORACLE (test infrastructure, not product code).
//
// A plain, slow, fp32 restatement of the method's hot path, one thread per query
// head, written from the paper's equations.  It shares no code with the CUDA path
// and must never be imported, linked or executed by it.  Only the tests, the smoke
// check and the benchmark's CPU-baseline leg call into this file.
//
// One `Stream` object is one (sequence, layer): the method treats layers and
// sequences independently.
//
// Steps (paper passage each follows):
//   O1  append K/V of the call                               Sec. 3.4 "Overall Framework"
//   O2  evict regions that left the window; pick the most     Sec. 3.4 step 1; Eq. 6 (votes v_x),
//       voted token(s) of each span as its index vector       Sec. 3.3.1 (static index vectors)
//   O3  local attention rows: softmax over sink+local+cur     Eq. 1-3 restricted to the local map
//   O4  Q20 fixed-point map, head sum, votes                  Eq. 4 (sum over heads), Eq. 6
//   O5  threshold theta                                       Eq. 5, App. "Configuration" (quantile)
//   O6  triangle scores, anti-diagonal filter, greedy NMS     Eq. 4-5, App. "NMS Input Filtration"
//   O7  query representatives of the call's spans             Sec. 3.4 step 2
//   O8  similarity of query reps vs span index                Eq. 7
//   O9  top-k spans                                           Eq. 8 (unit = span)
//   O10 softmax attention over sink+retrieved+local+cur       Sec. 3.4 step 3
//   O11 decode step (one query, no eviction, no votes)        Sec. 3.5 "Persistent Mechanism" (while
//                                                             decoding, the current block is one token)
//   O12 full causal attention (reference for the pin
//       "top-k covers every span => method == full attention")
// Optional modes (off by default):
//   O7'  dynamic number of representatives per span            Sec. 3.3.2, Eq. r_v
//   O6'  NMS with an IoU threshold above zero                  App. "NMS Input Filtration"
//   O9'  retrieval in fixed token units, unit score = max      Eq. 8 as printed
//        over the unit's spans
//   O11' decode keeps the last prefill call's selection        Sec. 3.5 "Persistent Mechanism"
//   O3'  a layer locates evidence with its retrieval head      Sec. 3.5 "Retrieval Heads"
//        alone (map, theta, votes, representatives, scores)
//   O9'' units ranked by the weighted ballots of the layers    Sec. 3.5 "Collaborative Voting"
//        up to this one, then by the layer's own scores
//   O6'' every memory unit of the region segmented on its own  Sec. 3.3 (blocks divided into spans)
// (The policy of the device-side cache of memory units, Sec. 3.4, changes no result of attention; its model,
//  UnitCachePolicy, lives in the Python wrapper beside this file.)
//
// Parity status: O3/O10/O12 are pinned by softmax invariants and by the full-attention
// equivalence; O6 is pinned by brute force, by hand-built block maps and by a library
// NMS; O8/O9 by brute force.  "parity unpinned" (defined only by this build's readings
// of passages the paper leaves open, checked by brute force and hand-built cases but by
// nothing the paper prints): the quantile convention of theta, the Q20 rounding of the
// map, gap filling, the vote-based choice of representative tokens and its tie rule,
// the max over query spans of summed representatives, the decode rules, and (optional
// modes) the definition of the area ratio r_a behind Eq. r_v, which the paper gives only
// as a figure.  Pinned among the optional modes: the shape of Eq. r_v and its clamps, the
// IoU NMS against a library NMS, the unit scores and the tokens a unit-granular step
// attends over, the union semantics of the persistent mechanism, the retrieval-head layer
// against the one-head model of that head, the vote ranking against a restated sort.
// "parity unpinned" there too: what a ballot is and how tallies and own scores combine,
// which the paper describes in one sentence.
//
// Build: g++ -O2 -std=c++17 -shared -fPIC -pthread ltri_oracle.cpp -o libltri_oracle.so

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <deque>
#include <functional>
#include <thread>
#include <vector>

namespace {

constexpr int kQ = 20;  // fixed-point fraction bits of the attention map
constexpr float kQScale = 1048576.0f;

inline float bf16_to_f32(uint16_t b) {
  uint32_t u = (uint32_t)b << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return f;
}

inline uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  std::memcpy(&u, &f, 4);
  if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x40);  // NaN
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  return (uint16_t)(u >> 16);
}

struct Span {
  int start, len;
  int nrep = 0;  // number of representative tokens (0: not decided yet -> static count)
};

struct Region {
  int start, end;
  std::vector<Span> spans;
};

struct Params {
  int32_t n_q_heads, n_kv_heads, head_dim;
  int32_t chunk, window, n_sink, top_k;
  int32_t reps_per_span, max_spans_per_region;
  int32_t theta_mode;
  float theta;
  float softmax_scale;
  int64_t max_tokens;
  // dynamic span index vectors (Sec. 3.3.2): rep_mode 0 = static count reps_per_span, 1 = count from the area ratio
  int32_t rep_mode, ratio_kind;  // ratio_kind 0: row neighbours, 1: column neighbours, 2: both
  int32_t min_reps, max_reps;
  float rep_lambda;
  // persistent mechanism (Sec. 3.5): decode keeps the spans selected by the last prefill call
  int32_t persist_decode;
  // retrieval granularity (Eq. 8 as printed): 0 = the span; U > 0 = fixed units of U tokens on the absolute token
  // grid, scored by the maximum over the spans they meet and fetched whole (clipped to the indexed range)
  int32_t unit_tokens;
  // NMS IoU threshold phi in thousandths (0: spans never overlap)
  int32_t nms_iou_milli;
  // 1: every unit of unit_tokens tokens is segmented on its own, max_spans_per_region spans kept per unit
  int32_t segment_per_unit;
  // retrieval head of this layer (Sec. 3.5): -1 = none, the layer locates evidence with all its heads; h >= 0 = the
  // local map, the votes, the query representatives and the scores come from head h alone, and its one selection
  // serves every KV head of the layer.  head_weight is that head's score, its voting weight.
  int32_t ret_head;
  float head_weight;
  // collaborative voting (Sec. 3.5): rank the units by the summed weights of the ballots (own top-k of this and of the
  // preceding layers that have a retrieval head) before their own scores; needs unit_tokens > 0
  int32_t collab_vote;
};

// ---------------------------------------------------------------------------
// O5: threshold in Q20 units of the head-summed map.
// mode 0: absolute head-mean probability -> theta * Hq * 2^20, rounded to nearest even.
// mode 1: lower nearest-rank quantile of the causal entries of the region map.
int64_t theta_q(const int32_t* Mq, int m, int ld, int mode, float theta, int Hq) {
  if (m <= 0) return 0;
  if (mode == 0) return (int64_t)std::nearbyint((double)theta * (double)Hq * (double)kQScale);
  int64_t N = (int64_t)m * (m + 1) / 2;
  std::vector<int32_t> vals;
  vals.reserve((size_t)N);
  for (int i = 0; i < m; ++i)
    for (int j = 0; j <= i; ++j) vals.push_back(Mq[(size_t)i * ld + j]);
  int64_t rank = (int64_t)std::floor((double)theta * (double)(N - 1));
  if (rank < 0) rank = 0;
  if (rank > N - 1) rank = N - 1;
  std::nth_element(vals.begin(), vals.begin() + rank, vals.end());
  return vals[(size_t)rank];
}

// Sec. 3.3.2 (dynamic span index vectors), written out from its definition on the raw region map:
// T = mass of the span's own triangle, R = mass its rows give to earlier tokens of the region ("row neighbours"),
// C = mass later rows of the region give to its columns ("column neighbours").  r_a = T / (T + neighbours) for the
// chosen kind (1 when there is no mass at all), r_v = 1 / e^(lambda (1 - r_a)) (Eq. r_v), and the span keeps
// round(len * r_v) representatives, clamped to [min_reps, max_reps] and to the span length.  All sums are integers;
// the ratio, the exponential and the rounding (to nearest even) are taken in double precision.
int dynamic_rep_count(const int32_t* Mq, int m, int ld, int x, int y, int kind, double lambda, int min_reps,
                      int max_reps) {
  int64_t T = 0, R = 0, Cn = 0;
  for (int i = x; i <= y; ++i) {
    for (int j = 0; j < x; ++j) R += Mq[(size_t)i * ld + j];
    for (int j = x; j <= i; ++j) T += Mq[(size_t)i * ld + j];
  }
  for (int i = y + 1; i < m; ++i)
    for (int j = x; j <= y; ++j) Cn += Mq[(size_t)i * ld + j];
  const int64_t nb = kind == 0 ? R : kind == 1 ? Cn : R + Cn;
  const double ra = (T + nb) > 0 ? (double)T / (double)(T + nb) : 1.0;
  const double rv = 1.0 / std::exp(lambda * (1.0 - ra));
  const int len = y - x + 1;
  int cnt = (int)std::nearbyint((double)len * rv);
  cnt = std::max(cnt, min_reps);
  cnt = std::min(cnt, max_reps);
  cnt = std::min(cnt, len);
  return std::max(cnt, 1);
}

// Eq. 4-5 by the two cumulative sums of Fig. 2: S(x,y) = sum_{x<=j<=i<=y} (Mq[i][j]-theta).
// Rsuf[i][x] = sum_{j=x..i} D[i][j]  (suffix sum along the row, "sum the right elements"),
// S(x,y)     = sum_{i=x..y} Rsuf[i][x] (prefix sum down the column, "sum the upper elements").
// Output S is m x m, entry [x*m+y] defined for x<=y.
void ta_scores(const int32_t* Mq, int m, int ld, int64_t thq, std::vector<int64_t>& S) {
  std::vector<int64_t> R((size_t)m * m, 0);
  for (int i = 0; i < m; ++i) {
    int64_t acc = 0;
    for (int x = i; x >= 0; --x) {
      acc += (int64_t)Mq[(size_t)i * ld + x] - thq;
      R[(size_t)i * m + x] = acc;
    }
  }
  S.assign((size_t)m * m, 0);
  for (int x = 0; x < m; ++x) {
    int64_t acc = 0;
    for (int y = x; y < m; ++y) {
      acc += R[(size_t)y * m + x];
      S[(size_t)x * m + y] = acc;
    }
  }
}

struct Cand {
  int64_t S;
  int x, y;
};

inline double rel_gap(int64_t a, int64_t b) {
  double da = (double)a, db = (double)b;
  double den = std::max(std::fabs(da), std::fabs(db));
  if (den == 0.0) return 0.0;
  return std::fabs(da - db) / den;
}

// O6: anti-diagonal filter, sort, greedy NMS, gap fill.  A candidate is suppressed when its IoU with a kept one
// exceeds phi = phi_milli / 1000, the boxes being the squares (x, x, y+1, y+1) on the diagonal: two spans that share
// `inter` tokens have IoU = inter^2 / (L1^2 + L2^2 - inter^2).  phi = 0: any overlap suppresses and the spans
// partition the region; phi > 0: kept spans may overlap, and the gaps are the runs no kept span covers.
// `min_gap` (optional) receives the smallest relative gap between two quantities whose
// comparison decided something: best vs runner-up on an anti-diagonal that produced a
// candidate; the best point's triangle mass vs its theta*area (the sign test S>0) on every
// anti-diagonal; and neighbours in the sorted candidate list up to the last one the
// greedy pass looked at.
void segment_map(const int32_t* Mq, int m, int ld, int64_t thq, int C, int phi_milli, std::vector<Span>& out,
                 double* min_gap) {
  out.clear();
  double gap = 1.0;
  if (m <= 0) {
    if (min_gap) *min_gap = gap;
    return;
  }
  std::vector<int64_t> S;
  ta_scores(Mq, m, ld, thq, S);
  std::vector<Cand> cands;
  for (int c = 0; c <= 2 * m - 2; ++c) {
    bool have = false;
    Cand best{0, 0, 0};
    int64_t second = 0;
    bool have2 = false;
    // walk from the shortest interval outwards so that ties keep the shorter span
    int y0 = (c + 1) / 2;
    for (int y = y0; y < m && c - y >= 0; ++y) {
      int x = c - y;
      int64_t s = S[(size_t)x * m + y];
      if (!have || s > best.S) {
        if (have) {
          second = have2 ? std::max(second, best.S) : best.S;
          have2 = true;
        }
        best = Cand{s, x, y};
        have = true;
      } else {
        second = have2 ? std::max(second, s) : s;
        have2 = true;
      }
    }
    if (have) {
      int64_t len = best.y - best.x + 1;
      int64_t tarea = thq * (len * (len + 1) / 2);
      gap = std::min(gap, rel_gap(best.S + tarea, tarea));
    }
    if (have && best.S > 0) {
      cands.push_back(best);
      if (have2) gap = std::min(gap, rel_gap(best.S, second));
    }
  }
  std::sort(cands.begin(), cands.end(), [](const Cand& a, const Cand& b) {
    if (a.S != b.S) return a.S > b.S;
    int la = a.y - a.x, lb = b.y - b.x;
    if (la != lb) return la < lb;
    return a.x < b.x;
  });
  std::vector<Cand> kept;
  size_t examined = 0;
  for (size_t ci = 0; ci < cands.size() && (int)kept.size() < C; ++ci) {
    examined = ci + 1;
    const Cand& c = cands[ci];
    bool ok = true;
    for (const Cand& k : kept) {
      const int64_t inter = std::min(c.y, k.y) - std::max(c.x, k.x) + 1;
      if (inter <= 0) continue;
      const int64_t l1 = c.y - c.x + 1, l2 = k.y - k.x + 1, i2 = inter * inter;
      if (i2 * 1000 > (int64_t)phi_milli * (l1 * l1 + l2 * l2 - i2)) {
        ok = false;
        break;
      }
    }
    if (ok) kept.push_back(c);
  }
  for (size_t ci = 0; ci + 1 < cands.size() && ci < examined; ++ci)
    gap = std::min(gap, rel_gap(cands[ci].S, cands[ci + 1].S));
  std::sort(kept.begin(), kept.end(), [](const Cand& a, const Cand& b) { return a.x != b.x ? a.x < b.x : a.y < b.y; });
  int pos = 0;  // first token no span emitted so far covers
  for (const Cand& k : kept) {
    if (k.x > pos) out.push_back(Span{pos, k.x - pos});
    out.push_back(Span{k.x, k.y - k.x + 1});
    pos = std::max(pos, k.y + 1);
  }
  if (pos < m) out.push_back(Span{pos, m - pos});
  if (min_gap) *min_gap = gap;
}

// O6 per memory unit (Sec. 3.3 "each block ... divided into spans"): the region starts at absolute token `origin`;
// the tokens are cut into units of `unit` tokens on the absolute grid and every unit's part of the region is segmented
// on its own -- its own triangle of the map, its own candidates, NMS and cap C, its own gap fill -- with the region's
// one threshold.  unit <= 0: the region is one piece.
void segment_region(const int32_t* Mq, int m, int ld, int64_t thq, int C, int phi_milli, int unit, int origin,
                    std::vector<Span>& out, double* min_gap) {
  if (unit <= 0) {
    segment_map(Mq, m, ld, thq, C, phi_milli, out, min_gap);
    return;
  }
  out.clear();
  double gap = 1.0;
  for (int a = 0; a < m;) {
    const int b = std::min(m, ((origin + a) / unit + 1) * unit - origin);  // end of the unit that holds token a
    std::vector<Span> part;
    double g = 1.0;
    segment_map(Mq + (size_t)a * ld + a, b - a, ld, thq, C, phi_milli, part, &g);
    for (const Span& sp : part) out.push_back(Span{sp.start + a, sp.len});
    gap = std::min(gap, g);
    a = b;
  }
  if (min_gap) *min_gap = gap;
}

// O9: the min(k,n) largest scores, ties -> lower id.  ids in rank order, -1 padded.
void top_k(const float* score, int n, int k, int* ids, double* cut_gap) {
  std::vector<int> order(n);
  for (int i = 0; i < n; ++i) order[i] = i;
  std::stable_sort(order.begin(), order.end(),
                   [&](int a, int b) { return score[a] > score[b]; });
  int kk = std::min(k, n);
  for (int i = 0; i < k; ++i) ids[i] = i < kk ? order[i] : -1;
  if (cut_gap) {
    *cut_gap = 1.0;
    if (kk < n && kk > 0) {
      double a = score[order[kk - 1]], b = score[order[kk]];
      double den = std::max(std::fabs(a), std::fabs(b));
      *cut_gap = den == 0.0 ? 0.0 : std::fabs(a - b) / den;
    }
  }
}

void run_heads(int H, const std::function<void(int)>& fn) {
  std::vector<std::thread> th;
  th.reserve(H);
  for (int h = 0; h < H; ++h) th.emplace_back(fn, h);
  for (auto& t : th) t.join();
}

struct Stream {
  Params p;
  int Hq, Hkv, G, d;
  float scale;
  int t = 0;  // tokens appended so far
  int E;      // end of the evicted (indexed) prefix
  bool decoding = false;
  std::vector<float> K, V;  // [Hkv][max_tokens][d]
  std::vector<int64_t> votes;
  std::deque<Region> pending;
  std::vector<Span> spans;    // indexed spans, tile [Ls,E)
  std::vector<uint16_t> KR;   // [span][Hkv][d] bf16 bits
  // state of the current call
  int t0 = 0, n = 0;
  std::vector<float> Q;  // [n][Hq][d]
  int reg_start = 0, m = 0;
  std::vector<int32_t> Mq;  // [m][m]
  int64_t thq = 0;
  double seg_gap = 1.0;
  std::vector<float> u;  // [Hkv][J][d]
  int J = 0;
  std::vector<float> score;  // [Hkv][Ns]
  std::vector<float> unit_score;  // [Hkv][units] (unit mode)
  std::vector<int> sel;      // [Hkv][top_k]
  std::vector<int> persist;  // [Hkv][top_k] selection of the last prefill call, kept through decode (Sec. 3.5)
  // collaborative voting: ballots of the preceding layers for the current call (set by the caller in layer order),
  // this layer's own ballot (its top-k by its own scores, absolute unit ids, -1 padded) and the tallies of the units
  struct Ballot {
    float w;
    std::vector<int> ids;
  };
  std::vector<Ballot> ballots;
  std::vector<int> own_ballot;
  std::vector<float> tally;  // [units]
  std::vector<double> cut_gap;  // [Hkv]
  std::vector<int> qrep_tok;    // [J][reps] absolute tokens, -1 padded

  explicit Stream(const Params& pp) : p(pp) {
    Hq = p.n_q_heads;
    Hkv = p.n_kv_heads;
    G = Hq / Hkv;
    d = p.head_dim;
    scale = p.softmax_scale > 0 ? p.softmax_scale : 1.0f / std::sqrt((float)d);
    E = p.n_sink;
    K.assign((size_t)Hkv * p.max_tokens * d, 0.f);
    V.assign((size_t)Hkv * p.max_tokens * d, 0.f);
    votes.assign((size_t)p.max_tokens, 0);
    sel.assign((size_t)Hkv * p.top_k, -1);
    cut_gap.assign(Hkv, 1.0);
  }

  const float* krow(int g, int tok) const { return &K[((size_t)g * p.max_tokens + tok) * d]; }
  const float* vrow(int g, int tok) const { return &V[((size_t)g * p.max_tokens + tok) * d]; }

  // O1
  void append(int cnt, const uint16_t* kb, const uint16_t* vb) {
    for (int r = 0; r < cnt; ++r)
      for (int g = 0; g < Hkv; ++g)
        for (int e = 0; e < d; ++e) {
          size_t src = ((size_t)r * Hkv + g) * d + e;
          size_t dst = ((size_t)g * p.max_tokens + (t + r)) * d + e;
          K[dst] = bf16_to_f32(kb[src]);
          V[dst] = bf16_to_f32(vb[src]);
        }
    t += cnt;
  }

  // units (of unit_tokens tokens on the absolute grid) that meet the indexed range [n_sink, E)
  int unit_count() const {
    if (p.unit_tokens <= 0 || E <= p.n_sink) return 0;
    return (E + p.unit_tokens - 1) / p.unit_tokens - p.n_sink / p.unit_tokens;
  }
  int rep_stride() const { return p.rep_mode == 1 ? std::max(p.max_reps, 1) : p.reps_per_span; }
  // representative counts of the spans of the newest region (the region map of the current call is still there)
  void decide_rep_counts(Region& reg) const {
    for (Span& s : reg.spans) {
      if (p.rep_mode == 1)
        s.nrep = dynamic_rep_count(Mq.data(), m, m, s.start - reg_start, s.start - reg_start + s.len - 1, p.ratio_kind,
                                   (double)p.rep_lambda, p.min_reps, p.max_reps);
      else
        s.nrep = std::min(p.reps_per_span, s.len);
    }
  }

  // tokens of [lo,hi) with the largest votes, ties -> lower index; returned ascending.
  std::vector<int> rep_tokens(int lo, int len, int nrep) const {
    int cnt = std::min(nrep > 0 ? nrep : p.reps_per_span, len);
    std::vector<int> idx(len);
    for (int i = 0; i < len; ++i) idx[i] = lo + i;
    std::stable_sort(idx.begin(), idx.end(), [&](int a, int b) { return votes[a] > votes[b]; });
    idx.resize(cnt);
    std::sort(idx.begin(), idx.end());
    return idx;
  }

  // ---- test hooks (no arithmetic of the method): let a test continue the stream from a given state --------------
  // append tokens without any processing (O1 only)
  int append_only(int cnt, const uint16_t* kb, const uint16_t* vb) {
    if (cnt < 0 || (int64_t)t + cnt > p.max_tokens) return -2;
    append(cnt, kb, vb);
    return 0;
  }
  // replace the indexed prefix: evicted end, span table and (optionally) index vectors; pending regions are dropped
  int load_state(int evicted_end, int nspans, const int* start_len, const uint16_t* kr) {
    if (evicted_end < p.n_sink || evicted_end > t) return -1;
    spans.clear();
    int pos = p.n_sink;
    for (int i = 0; i < nspans; ++i) {
      if (start_len[2 * i] != pos || start_len[2 * i + 1] < 1) return -1;
      spans.push_back(Span{start_len[2 * i], start_len[2 * i + 1]});
      pos += start_len[2 * i + 1];
    }
    if (pos != evicted_end) return -1;
    KR.assign((size_t)nspans * Hkv * d, 0);
    if (kr) std::memcpy(KR.data(), kr, KR.size() * sizeof(uint16_t));
    E = evicted_end;
    pending.clear();
    return 0;
  }
  // test hook: replace the span table and the index vectors of the indexed prefix [n_sink, E) and leave everything
  // else (E, the pending regions, the votes) as it is; no arithmetic of the method
  int replace_index(int nspans, const int* start_len, const uint16_t* kr) {
    std::vector<Span> fresh;
    int pos = p.n_sink;
    for (int i = 0; i < nspans; ++i) {
      if (start_len[2 * i] != pos || start_len[2 * i + 1] < 1) return -1;
      fresh.push_back(Span{start_len[2 * i], start_len[2 * i + 1]});
      pos += start_len[2 * i + 1];
    }
    if (pos != E || !kr) return -1;
    spans.swap(fresh);
    KR.assign((size_t)nspans * Hkv * d, 0);
    std::memcpy(KR.data(), kr, KR.size() * sizeof(uint16_t));
    return 0;
  }
  // append a region that is still inside the window, with its spans (its votes start from zero)
  int add_pending(int start, int end, int nspans, const int* start_len) {
    if (start < E || end <= start || end > t) return -1;
    if (!pending.empty() && pending.back().end != start) return -1;
    if (pending.empty() && start != E) return -1;
    Region r;
    r.start = start;
    r.end = end;
    int pos = start;
    for (int i = 0; i < nspans; ++i) {
      if (start_len[2 * i] != pos || start_len[2 * i + 1] < 1) return -1;
      r.spans.push_back(Span{start_len[2 * i], start_len[2 * i + 1]});
      pos += start_len[2 * i + 1];
    }
    if (pos != end) return -1;
    pending.push_back(r);
    return 0;
  }
  // make the last `cnt` appended tokens the current call (sets t0, n, Q) without running the local pass
  int begin_call(int cnt, const uint16_t* qb) {
    if (cnt < 1 || cnt > t) return -1;
    t0 = t - cnt;
    n = cnt;
    m = 0;
    Q.resize((size_t)n * Hq * d);
    for (size_t i = 0; i < Q.size(); ++i) Q[i] = bf16_to_f32(qb[i]);
    return 0;
  }

  // O2
  void evict(int t0_) {
    while (!pending.empty() && pending.front().end <= t0_ - p.window) {
      Region& r = pending.front();
      for (const Span& s : r.spans) {
        std::vector<int> reps = rep_tokens(s.start, s.len, s.nrep);
        size_t base = KR.size();
        KR.resize(base + (size_t)Hkv * d);
        for (int g = 0; g < Hkv; ++g)
          for (int e = 0; e < d; ++e) {
            float acc = 0.f;
            for (int tok : reps) acc += krow(g, tok)[e];
            KR[base + (size_t)g * d + e] = f32_to_bf16_rne(acc);
          }
        spans.push_back(s);
      }
      E = r.end;
      pending.pop_front();
    }
  }

  struct KeySet {
    // half-open token ranges in the order sink, retrieved..., local, cur
    std::vector<std::pair<int, int>> ranges;
  };

  // softmax statistics + probabilities of one (head,row) over a key list; fp32 throughout.
  void softmax_row(const float* qv, int g, const std::vector<std::pair<int, int>>& ranges,
                   std::vector<float>& pbuf, float& l_out) const {
    pbuf.clear();
    float mx = -INFINITY;
    for (auto& rg : ranges)
      for (int j = rg.first; j < rg.second; ++j) {
        const float* kr = krow(g, j);
        float acc = 0.f;
        for (int e = 0; e < d; ++e) acc += qv[e] * kr[e];
        float s = acc * scale;
        pbuf.push_back(s);
        mx = std::max(mx, s);
      }
    float l = 0.f;
    for (float& s : pbuf) {
      s = std::exp(s - mx);
      l += s;
    }
    l_out = l;
  }

  // O1-O6
  int prefill_local(int cnt, const uint16_t* qb, const uint16_t* kb, const uint16_t* vb) {
    if (decoding) return -3;
    if (cnt < 1 || cnt > p.chunk || (int64_t)t + cnt > p.max_tokens) return -2;
    t0 = t;
    n = cnt;
    append(cnt, kb, vb);
    evict(t0);
    Q.resize((size_t)n * Hq * d);
    for (size_t i = 0; i < Q.size(); ++i) Q[i] = bf16_to_f32(qb[i]);
    reg_start = std::max(p.n_sink, t0);
    m = std::max(0, t0 + n - reg_start);
    const int sink_end = std::min(p.n_sink, t0);
    const int loc_begin = std::min(E, t0);
    std::vector<std::vector<int32_t>> Mh(Hq);
    std::vector<std::vector<int64_t>> vh(Hq);
    const int vbase = loc_begin;  // votes touched lie in [loc_begin, t0+n)
    run_heads(Hq, [&](int h) {
      int g = h / G;
      Mh[h].assign((size_t)m * m, 0);
      vh[h].assign((size_t)(t0 + n - vbase), 0);
      if (p.ret_head >= 0 && h != p.ret_head) return;  // the layer's retrieval head alone draws the map and votes
      std::vector<float> pbuf;
      std::vector<std::pair<int, int>> ranges(3);
      for (int r = 0; r < n; ++r) {
        int i = t0 + r;
        ranges[0] = {0, sink_end};
        ranges[1] = {loc_begin, t0};
        ranges[2] = {t0, i + 1};
        float l;
        softmax_row(&Q[((size_t)r * Hq + h) * d], g, ranges, pbuf, l);
        size_t pi = 0;
        for (auto& rg : ranges)
          for (int j = rg.first; j < rg.second; ++j, ++pi) {
            float a = pbuf[pi] / l;
            int32_t aq = (int32_t)std::nearbyintf(a * kQScale);
            if (j >= loc_begin && j >= p.n_sink) vh[h][j - vbase] += aq;  // O4 votes (Eq. 6)
            if (j >= reg_start && i >= reg_start)
              Mh[h][(size_t)(i - reg_start) * m + (j - reg_start)] += aq;  // O4 map
          }
      }
    });
    Mq.assign((size_t)m * m, 0);
    for (int h = 0; h < Hq; ++h) {
      for (size_t i = 0; i < Mq.size(); ++i) Mq[i] += Mh[h][i];
      for (size_t i = 0; i < vh[h].size(); ++i) votes[vbase + i] += vh[h][i];
    }
    Region reg;
    reg.start = reg_start;
    reg.end = t0 + n;
    if (m > 0) {
      thq = theta_q(Mq.data(), m, m, p.theta_mode, p.theta, p.ret_head >= 0 ? 1 : Hq);
      std::vector<Span> sp;
      segment_region(Mq.data(), m, m, thq, p.max_spans_per_region, p.nms_iou_milli,
                     p.segment_per_unit ? p.unit_tokens : 0, reg_start, sp, &seg_gap);
      for (Span& s : sp) s.start += reg_start;
      reg.spans = sp;
      decide_rep_counts(reg);
      pending.push_back(reg);
    } else {
      thq = 0;
      seg_gap = 1.0;
    }
    return 0;
  }

  // O7-O9 for the current prefill call (uses the spans stored for the newest region).
  void prefill_retrieve() {
    J = 0;
    u.clear();
    qrep_tok.clear();
    if (m > 0) {
      const Region& reg = pending.back();
      J = (int)reg.spans.size();
      u.assign((size_t)Hkv * J * d, 0.f);
      qrep_tok.assign((size_t)J * rep_stride(), -1);
      for (int j = 0; j < J; ++j) {
        std::vector<int> reps = rep_tokens(reg.spans[j].start, reg.spans[j].len, reg.spans[j].nrep);
        for (size_t r = 0; r < reps.size(); ++r) qrep_tok[(size_t)j * rep_stride() + r] = reps[r];
        for (int g = 0; g < Hkv; ++g)
          for (int e = 0; e < d; ++e) {
            // the heads whose queries locate the evidence for KV head g: its own group, or the layer's retrieval head
            const int h_lo = p.ret_head >= 0 ? p.ret_head : g * G, h_hi = p.ret_head >= 0 ? p.ret_head + 1 : (g + 1) * G;
            float ug = 0.f;
            for (int h = h_lo; h < h_hi; ++h) {
              float qr = 0.f;
              for (int tok : reps) qr += Q[((size_t)(tok - t0) * Hq + h) * d + e];
              ug += qr;
            }
            u[((size_t)g * J + j) * d + e] = ug;
          }
      }
    }
    score_and_select();
  }

  // O8 + O9 with the representatives in `u` ([Hkv][J][d]).  A layer with a retrieval head scores against the index
  // of that head's KV head, so every row of its scores and of its selection is the same.
  void score_and_select() {
    int Ns = (int)spans.size();
    score.assign((size_t)Hkv * Ns, -INFINITY);
    if (p.unit_tokens > 0) unit_score.assign((size_t)Hkv * unit_count(), -INFINITY);
    own_ballot.assign(p.top_k, -1);
    tally.clear();
    for (int g = 0; g < Hkv; ++g) {
      const int gk = p.ret_head >= 0 ? p.ret_head / G : g;  // KV head whose index vectors are scored
      for (int s = 0; s < Ns; ++s) {
        float best = -INFINITY;
        for (int j = 0; j < J; ++j) {
          const float* uj = &u[((size_t)g * J + j) * d];
          const uint16_t* kr = &KR[((size_t)s * Hkv + gk) * d];
          float acc = 0.f;
          for (int e = 0; e < d; ++e) acc += uj[e] * bf16_to_f32(kr[e]);
          best = std::max(best, acc);
        }
        score[(size_t)g * Ns + s] = best;
      }
      if (J > 0 && p.unit_tokens > 0) {
        // Eq. 8: the score of a unit is the maximum over its spans; the top-k units are fetched
        const int U = p.unit_tokens, u0 = p.n_sink / U, nu = unit_count();
        float* us = &unit_score[(size_t)g * nu];
        for (int u = 0; u < nu; ++u) us[u] = -INFINITY;
        for (int s = 0; s < Ns; ++s)
          for (int u = spans[s].start / U; u <= (spans[s].start + spans[s].len - 1) / U; ++u)
            us[u - u0] = std::max(us[u - u0], score[(size_t)g * Ns + s]);
        int* sg = &sel[(size_t)g * p.top_k];
        top_k(us, nu, p.top_k, sg, &cut_gap[g]);
        for (int i = 0; i < p.top_k; ++i)
          if (sg[i] >= 0) sg[i] += u0;  // absolute unit ids
      } else if (J > 0)
        top_k(&score[(size_t)g * Ns], Ns, p.top_k, &sel[(size_t)g * p.top_k], &cut_gap[g]);
      else {
        for (int i = 0; i < p.top_k; ++i) sel[(size_t)g * p.top_k + i] = -1;
        cut_gap[g] = 1.0;
      }
    }
    if (p.collab_vote && J > 0 && p.unit_tokens > 0) {
      // the layer's ballot: its top-k by its own scores (every row is the same under a retrieval head); layers
      // without a retrieval head cast none
      if (p.ret_head >= 0) own_ballot.assign(sel.begin(), sel.begin() + p.top_k);
      vote_select();
    }
  }

  // Sec. 3.5, collaborative voting.  A ballot counts with its layer's retrieval-head score.  Tally of a unit = sum of
  // the weights of the ballots that name it, preceding layers first (ascending), then this layer's own.  The units
  // are ranked by tally, then own score, then lower id, and the first top_k are fetched.
  void vote_select() {
    const int U = p.unit_tokens, u0 = p.n_sink / U, nu = unit_count();
    tally.assign(nu, 0.f);
    for (const Ballot& b : ballots)
      for (int id : b.ids)
        if (id >= u0 && id - u0 < nu) tally[id - u0] += b.w;
    if (p.ret_head >= 0)
      for (int id : own_ballot)
        if (id >= u0 && id - u0 < nu) tally[id - u0] += p.head_weight;
    for (int g = 0; g < Hkv; ++g) {
      const float* us = &unit_score[(size_t)g * nu];
      int* sg = &sel[(size_t)g * p.top_k];
      std::vector<int> order(nu);
      for (int i = 0; i < nu; ++i) order[i] = i;
      std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
        if (tally[a] != tally[b]) return tally[a] > tally[b];
        return us[a] > us[b];
      });
      const int kk = std::min(p.top_k, nu);
      for (int i = 0; i < p.top_k; ++i) sg[i] = i < kk ? order[i] + u0 : -1;
      cut_gap[g] = 1.0;
      if (kk < nu && kk > 0 && tally[order[kk - 1]] == tally[order[kk]]) {
        double a = us[order[kk - 1]], b = us[order[kk]];
        double den = std::max(std::fabs(a), std::fabs(b));
        cut_gap[g] = den == 0.0 ? 0.0 : std::fabs(a - b) / den;
      }
    }
  }

  std::vector<std::pair<int, int>> key_ranges(int g, int sink_end, int loc_begin, int loc_end) const {
    std::vector<std::pair<int, int>> ranges;
    ranges.push_back({0, sink_end});
    // the spans selected now (rank order) and, in a decode step under the persistent mechanism, those the last
    // prefill call selected that are not among them; every span once
    std::vector<int> ids;
    for (int i = 0; i < p.top_k; ++i) {
      int s = sel[(size_t)g * p.top_k + i];
      if (s >= 0) ids.push_back(s);
    }
    if (decoding && p.persist_decode && !persist.empty())
      for (int i = 0; i < p.top_k; ++i) {
        int s = persist[(size_t)g * p.top_k + i];
        if (s >= 0 && std::find(ids.begin(), ids.end(), s) == ids.end()) ids.push_back(s);
      }
    if (p.nms_iou_milli > 0 && p.unit_tokens == 0) {
      // selected spans may overlap: every token once (ranges in position order, overlaps merged)
      std::sort(ids.begin(), ids.end());
      for (int s : ids) {
        const int a = spans[s].start, b = spans[s].start + spans[s].len;
        if (ranges.size() > 1 && a <= ranges.back().second)
          ranges.back().second = std::max(ranges.back().second, b);
        else
          ranges.push_back({a, b});
      }
      ranges.push_back({loc_begin, loc_end});
      return ranges;
    }
    for (int s : ids) {
      if (p.unit_tokens > 0)  // the unit's tokens inside the indexed range [n_sink, E)
        ranges.push_back({std::max(s * p.unit_tokens, p.n_sink), std::min((s + 1) * p.unit_tokens, E)});
      else
        ranges.push_back({spans[s].start, spans[s].start + spans[s].len});
    }
    ranges.push_back({loc_begin, loc_end});
    return ranges;
  }

  void attend_row(const float* qv, int g, std::vector<std::pair<int, int>>& ranges, float* out) const {
    std::vector<float> pbuf;
    float l;
    softmax_row(qv, g, ranges, pbuf, l);
    std::vector<float> acc(d, 0.f);
    size_t pi = 0;
    for (auto& rg : ranges)
      for (int j = rg.first; j < rg.second; ++j, ++pi) {
        const float* vr = vrow(g, j);
        float pj = pbuf[pi];
        for (int e = 0; e < d; ++e) acc[e] += pj * vr[e];
      }
    for (int e = 0; e < d; ++e) out[e] = acc[e] / l;
  }

  // O10 for rows [r0,r1) of the current call; out is [r1-r0][Hq][d] fp32.
  void prefill_attend(int r0, int r1, float* out) const {
    const int sink_end = std::min(p.n_sink, t0);
    const int loc_begin = std::min(E, t0);
    run_heads(Hq, [&](int h) {
      int g = h / G;
      for (int r = r0; r < r1; ++r) {
        auto ranges = key_ranges(g, sink_end, loc_begin, t0);
        ranges.push_back({t0, t0 + r + 1});
        attend_row(&Q[((size_t)r * Hq + h) * d], g, ranges, &out[((size_t)(r - r0) * Hq + h) * d]);
      }
    });
  }

  // O11: retrieval part of a decode step.
  int decode_retrieve(const uint16_t* qb, const uint16_t* kb, const uint16_t* vb) {
    if ((int64_t)t + 1 > p.max_tokens) return -2;
    if (!decoding && p.persist_decode) persist = sel;  // what the last prefill call retrieved (may be empty)
    decoding = true;
    t0 = t;
    n = 1;
    m = 0;
    append(1, kb, vb);
    Q.resize((size_t)Hq * d);
    for (size_t i = 0; i < Q.size(); ++i) Q[i] = bf16_to_f32(qb[i]);
    J = 1;
    u.assign((size_t)Hkv * d, 0.f);
    for (int g = 0; g < Hkv; ++g)
      for (int e = 0; e < d; ++e) {
        const int h_lo = p.ret_head >= 0 ? p.ret_head : g * G, h_hi = p.ret_head >= 0 ? p.ret_head + 1 : (g + 1) * G;
        float ug = 0.f;
        for (int h = h_lo; h < h_hi; ++h) ug += Q[(size_t)h * d + e];
        u[(size_t)g * d + e] = ug;
      }
    score_and_select();
    return 0;
  }

  // O11: attention part of a decode step; out is [Hq][d] fp32.
  void decode_attend(float* out) const {
    const int pos = t0;  // the decode token's own position
    const int sink_end = std::min(p.n_sink, pos + 1);
    const int loc_begin = std::min(E, pos + 1);
    run_heads(Hq, [&](int h) {
      int g = h / G;
      auto ranges = key_ranges(g, sink_end, loc_begin, pos + 1);
      attend_row(&Q[(size_t)h * d], g, ranges, &out[(size_t)h * d]);
    });
  }

  // O12: causal attention over every cached token <= position, for given query rows.
  void full_attention(int cnt, const int* positions, const uint16_t* qb, float* out) const {
    std::vector<float> Qf((size_t)cnt * Hq * d);
    for (size_t i = 0; i < Qf.size(); ++i) Qf[i] = bf16_to_f32(qb[i]);
    run_heads(Hq, [&](int h) {
      int g = h / G;
      for (int r = 0; r < cnt; ++r) {
        std::vector<std::pair<int, int>> ranges{{0, positions[r] + 1}};
        attend_row(&Qf[((size_t)r * Hq + h) * d], g, ranges, &out[((size_t)r * Hq + h) * d]);
      }
    });
  }
};

}  // namespace

// ---------------------------------------------------------------------------
// C interface for the ctypes wrapper
extern "C" {

void* orc_create(const Params* p) {
  if (!p || p->n_q_heads < 1 || p->n_kv_heads < 1 || p->n_q_heads % p->n_kv_heads) return nullptr;
  if (p->head_dim < 1 || p->chunk < 1 || p->window < 1 || p->n_sink < 1 || p->top_k < 1) return nullptr;
  if (p->reps_per_span < 1 || p->max_spans_per_region < 1 || p->max_tokens < 1) return nullptr;
  if (p->unit_tokens < 0 || p->nms_iou_milli < 0 || p->nms_iou_milli >= 1000) return nullptr;
  if (p->ret_head < -1 || p->ret_head >= p->n_q_heads || !(p->head_weight >= 0.f)) return nullptr;
  if (p->collab_vote && p->unit_tokens <= 0) return nullptr;
  if (p->segment_per_unit && p->unit_tokens <= 0) return nullptr;
  if (p->rep_mode != 0 && p->rep_mode != 1) return nullptr;
  if (p->rep_mode == 1 && (p->ratio_kind < 0 || p->ratio_kind > 2 || p->min_reps < 1 || p->max_reps < p->min_reps ||
                           !(p->rep_lambda >= 0.f)))
    return nullptr;
  return new Stream(*p);
}
void orc_destroy(void* h) { delete (Stream*)h; }

int orc_prefill_local(void* h, int n, const uint16_t* q, const uint16_t* k, const uint16_t* v) {
  return ((Stream*)h)->prefill_local(n, q, k, v);
}
void orc_prefill_retrieve(void* h) { ((Stream*)h)->prefill_retrieve(); }
void orc_prefill_attend(void* h, int r0, int r1, float* out) { ((Stream*)h)->prefill_attend(r0, r1, out); }
int orc_decode_retrieve(void* h, const uint16_t* q, const uint16_t* k, const uint16_t* v) {
  return ((Stream*)h)->decode_retrieve(q, k, v);
}
void orc_decode_attend(void* h, float* out) { ((Stream*)h)->decode_attend(out); }
void orc_full_attention(void* h, int cnt, const int* pos, const uint16_t* q, float* out) {
  ((Stream*)h)->full_attention(cnt, pos, q, out);
}

// --- test hooks ---------------------------------------------------------------
int orc_append_only(void* h, int n, const uint16_t* k, const uint16_t* v) { return ((Stream*)h)->append_only(n, k, v); }
int orc_load_state(void* h, int evicted_end, int nspans, const int* start_len, const uint16_t* kr) {
  return ((Stream*)h)->load_state(evicted_end, nspans, start_len, kr);
}
int orc_replace_index(void* h, int nspans, const int* start_len, const uint16_t* kr) {
  return ((Stream*)h)->replace_index(nspans, start_len, kr);
}
int orc_begin_call(void* h, int n, const uint16_t* q) { return ((Stream*)h)->begin_call(n, q); }
int orc_add_pending(void* h, int start, int end, int nspans, const int* start_len) {
  return ((Stream*)h)->add_pending(start, end, nspans, start_len);
}

// --- state access -----------------------------------------------------------
int orc_tokens(void* h) { return ((Stream*)h)->t; }
int orc_evicted_end(void* h) { return ((Stream*)h)->E; }
int orc_num_spans(void* h) { return (int)((Stream*)h)->spans.size(); }
void orc_get_spans(void* h, int* start_len) {
  Stream* s = (Stream*)h;
  for (size_t i = 0; i < s->spans.size(); ++i) {
    start_len[2 * i] = s->spans[i].start;
    start_len[2 * i + 1] = s->spans[i].len;
  }
}
void orc_get_index(void* h, uint16_t* kr) {  // [span][Hkv][d] bf16 bits
  Stream* s = (Stream*)h;
  std::memcpy(kr, s->KR.data(), s->KR.size() * sizeof(uint16_t));
}
int orc_num_pending_regions(void* h) { return (int)((Stream*)h)->pending.size(); }
// region r of the pending queue (0 = oldest): returns span count, writes {start,end} and spans
int orc_get_pending(void* h, int r, int* start_end, int* start_len, int cap) {
  Stream* s = (Stream*)h;
  if (r < 0 || r >= (int)s->pending.size()) return -1;
  const Region& reg = s->pending[r];
  start_end[0] = reg.start;
  start_end[1] = reg.end;
  int c = (int)reg.spans.size();
  for (int i = 0; i < c && i < cap; ++i) {
    start_len[2 * i] = reg.spans[i].start;
    start_len[2 * i + 1] = reg.spans[i].len;
  }
  return c;
}
// replace the spans of the newest pending region (re-synchronisation after a tolerated near-tie)
int orc_set_newest_spans(void* h, const int* start_len, int cnt) {
  Stream* s = (Stream*)h;
  if (s->pending.empty()) return -1;
  Region& reg = s->pending.back();
  int pos = reg.start;  // first token not covered yet: the spans come sorted by start and leave no hole
  for (int i = 0; i < cnt; ++i) {
    const int st = start_len[2 * i], ln = start_len[2 * i + 1];
    if (ln < 1 || st > pos || st < reg.start || (s->p.nms_iou_milli == 0 && st != pos)) return -1;
    if (i > 0 && st < start_len[2 * i - 2]) return -1;
    pos = std::max(pos, st + ln);
  }
  if (pos != reg.end) return -1;
  reg.spans.clear();
  for (int i = 0; i < cnt; ++i) reg.spans.push_back(Span{start_len[2 * i], start_len[2 * i + 1]});
  if (s->m > 0 && reg.start == s->reg_start) s->decide_rep_counts(reg);
  return 0;
}
// representative counts of the newest pending region's spans
int orc_get_newest_rep_counts(void* h, int* out, int cap) {
  Stream* s = (Stream*)h;
  if (s->pending.empty()) return 0;
  const Region& reg = s->pending.back();
  int c = (int)reg.spans.size();
  for (int i = 0; i < c && i < cap; ++i) out[i] = reg.spans[i].nrep > 0 ? reg.spans[i].nrep : std::min(s->p.reps_per_span, reg.spans[i].len);
  return c;
}
// overwrite the representative counts of the newest region's spans (re-synchronisation after a tolerated rounding flip)
int orc_set_newest_rep_counts(void* h, const int* counts, int cnt) {
  Stream* s = (Stream*)h;
  if (s->pending.empty() || (int)s->pending.back().spans.size() != cnt) return -1;
  for (int i = 0; i < cnt; ++i) {
    if (counts[i] < 1 || counts[i] > s->pending.back().spans[i].len) return -1;
    s->pending.back().spans[i].nrep = counts[i];
  }
  return 0;
}
int orc_num_units(void* h) { return ((Stream*)h)->unit_count(); }
// collaborative voting: the ballots of the preceding layers for the next retrieval (ascending layer order);
// ids [n][top_k] absolute unit ids, -1 padded
void orc_set_ballots(void* h, int n, const float* w, const int* ids) {
  Stream* s = (Stream*)h;
  s->ballots.clear();
  for (int i = 0; i < n; ++i) {
    Stream::Ballot b;
    b.w = w[i];
    for (int j = 0; j < s->p.top_k; ++j)
      if (ids[(size_t)i * s->p.top_k + j] >= 0) b.ids.push_back(ids[(size_t)i * s->p.top_k + j]);
    s->ballots.push_back(b);
  }
}
// this layer's own ballot of the last retrieval ([top_k], -1 padded; all -1 for a layer without a retrieval head)
void orc_get_ballot(void* h, int* ids) {
  Stream* s = (Stream*)h;
  for (int i = 0; i < s->p.top_k; ++i) ids[i] = i < (int)s->own_ballot.size() ? s->own_ballot[i] : -1;
}
void orc_set_ballot(void* h, const int* ids) {  // test hook: adopt a tolerated pick and count the votes again
  Stream* s = (Stream*)h;
  s->own_ballot.assign(ids, ids + s->p.top_k);
  if (s->p.collab_vote && s->J > 0 && s->p.unit_tokens > 0 && s->unit_count() > 0) s->vote_select();
}
void orc_get_tally(void* h, float* out) {  // [units]
  Stream* s = (Stream*)h;
  std::memcpy(out, s->tally.data(), s->tally.size() * sizeof(float));
}
void orc_get_unit_scores(void* h, float* out) {  // [Hkv][units]
  Stream* s = (Stream*)h;
  std::memcpy(out, s->unit_score.data(), s->unit_score.size() * sizeof(float));
}
int orc_rep_stride(void* h) { return ((Stream*)h)->rep_stride(); }
int orc_dynamic_rep_count(const int32_t* Mq, int m, int x, int y, int kind, double lambda, int min_reps, int max_reps) {
  return dynamic_rep_count(Mq, m, m, x, y, kind, lambda, min_reps, max_reps);
}
void orc_get_votes(void* h, int lo, int hi, int64_t* out) {
  Stream* s = (Stream*)h;
  for (int i = lo; i < hi; ++i) out[i - lo] = s->votes[i];
}
// current call
int orc_region_len(void* h) { return ((Stream*)h)->m; }
int orc_region_start(void* h) { return ((Stream*)h)->reg_start; }
void orc_get_map(void* h, int32_t* Mq) {
  Stream* s = (Stream*)h;
  std::memcpy(Mq, s->Mq.data(), s->Mq.size() * sizeof(int32_t));
}
int64_t orc_get_theta_q(void* h) { return ((Stream*)h)->thq; }
double orc_get_seg_gap(void* h) { return ((Stream*)h)->seg_gap; }
int orc_num_query_reps(void* h) { return ((Stream*)h)->J; }
void orc_get_query_reps(void* h, float* u) {  // [Hkv][J][d]
  Stream* s = (Stream*)h;
  std::memcpy(u, s->u.data(), s->u.size() * sizeof(float));
}
void orc_get_query_rep_tokens(void* h, int* tok) {  // [J][reps]
  Stream* s = (Stream*)h;
  std::memcpy(tok, s->qrep_tok.data(), s->qrep_tok.size() * sizeof(int));
}
void orc_get_scores(void* h, float* sc) {  // [Hkv][Ns]
  Stream* s = (Stream*)h;
  std::memcpy(sc, s->score.data(), s->score.size() * sizeof(float));
}
void orc_get_selected(void* h, int* ids, double* gaps) {  // [Hkv][top_k], [Hkv]
  Stream* s = (Stream*)h;
  std::memcpy(ids, s->sel.data(), s->sel.size() * sizeof(int));
  if (gaps) std::memcpy(gaps, s->cut_gap.data(), s->cut_gap.size() * sizeof(double));
}
// [Hkv][top_k] span ids kept through decode by the persistent mechanism (-1 padded; all -1 before the first decode step)
void orc_get_persistent(void* h, int* ids) {
  Stream* s = (Stream*)h;
  for (size_t i = 0; i < s->sel.size(); ++i) ids[i] = i < s->persist.size() ? s->persist[i] : -1;
}
void orc_set_selected(void* h, const int* ids) {
  Stream* s = (Stream*)h;
  std::memcpy(s->sel.data(), ids, s->sel.size() * sizeof(int));
}

// --- stateless pieces, exposed so that each can be pinned on its own ---------
int64_t orc_theta_q(const int32_t* Mq, int m, int mode, float theta, int Hq) {
  return theta_q(Mq, m, m, mode, theta, Hq);
}
void orc_ta_scores(const int32_t* Mq, int m, int64_t thq, int64_t* S) {  // S[x*m+y], x<=y
  std::vector<int64_t> s;
  ta_scores(Mq, m, m, thq, s);
  std::memcpy(S, s.data(), s.size() * sizeof(int64_t));
}
int orc_segment_map(const int32_t* Mq, int m, int64_t thq, int C, int phi_milli, int unit, int origin, int* start_len,
                    int cap, double* gap) {
  std::vector<Span> sp;
  segment_region(Mq, m, m, thq, C, phi_milli, unit, origin, sp, gap);
  for (size_t i = 0; i < sp.size() && (int)i < cap; ++i) {
    start_len[2 * i] = sp[i].start;
    start_len[2 * i + 1] = sp[i].len;
  }
  return (int)sp.size();
}
void orc_top_k(const float* score, int n, int k, int* ids, double* gap) { top_k(score, n, k, ids, gap); }
uint16_t orc_f32_to_bf16(float f) { return f32_to_bf16_rne(f); }

}  // extern "C"
