// State kernels: cache append, eviction + span index build (Sec. 3.3.1, Eq. 6), span segmenter
// (Eq. 4-5, App. "NMS Input Filtration"), query representatives, similarity scores (Eq. 7) and
// top-k selection (Eq. 8).  All segmentation arithmetic is integer and order-independent.
#include <cooperative_groups.h>

#include "common.cuh"

namespace ltri {

// ------------------------------------------------------------------------------------------
__global__ void k_init(DevCtx c, int seq) {
  const int s0 = seq < 0 ? 0 : seq, s1 = seq < 0 ? c.NS : seq + 1;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  for (int s = s0; s < s1; ++s) {
    const size_t u0 = (size_t)s * c.NL;
    for (size_t i = tid; i < (size_t)c.NL; i += stride) {
      c.n_spans[u0 + i] = 0;
    }
    for (size_t i = tid; i < (size_t)c.NL * c.Hkv; i += stride) c.sel_tokens[u0 * c.Hkv + i] = 0;
    for (size_t i = tid; i < (size_t)c.NL * c.slots; i += stride) c.pend_cnt[u0 * c.slots + i] = 0;
    for (size_t i = tid; i < (size_t)c.NL * c.Hkv * c.topk; i += stride) {
      c.sel[u0 * c.Hkv * c.topk + i] = -1;
      c.persist_sel[u0 * c.Hkv * c.topk + i] = -1;
    }
    for (size_t i = tid; i < (size_t)c.NL * c.Hkv; i += stride) c.rng_cnt[u0 * c.Hkv + i] = 0;
    for (size_t i = tid; i < (size_t)c.NL * c.topk; i += stride) c.ballot[u0 * c.topk + i] = -1;
    if (c.host_kv) {  // empty unit caches
      const size_t nslot = (size_t)c.NL * c.Hkv * c.cache_units;
      for (size_t i = tid; i < nslot; i += stride) {
        c.ctag[u0 * c.Hkv * c.cache_units + i] = -1;
        c.cscore[u0 * c.Hkv * c.cache_units + i] = 0.f;
      }
      for (size_t i = tid; i < (size_t)c.NL * 2; i += stride) c.cstat[u0 * 2 + i] = 0ull;
    }
  }
  if (seq < 0 && tid < 4) c.status[tid] = 0;
  if (seq < 0)
    for (size_t i = tid; i < (size_t)kTcMaxCtas; i += stride) c.tc_redo[i] = 0;
  if (seq < 0)
    for (size_t i = tid; i < (size_t)c.NL; i += stride) c.Jcnt[i] = 0;
}

cudaError_t launch_init(const DevCtx& c, int seq, cudaStream_t s) {
  k_init<<<64, 256, 0, s>>>(c, seq);
  return cudaGetLastError();
}


// ------------------------------------------------------------------------------------------
// a0: copy the call's K/V rows into the cache slabs; 16 threads move one 256-byte row.  The threads behind the copy
// (zero_vec of them, 16 bytes each) clear the region maps of the call's layers, which the tensor-core map pass
// accumulates into with integer reductions: nothing reads a layer's map between the segmenter of the layer's previous
// call and that pass, so clearing it here, in the first kernel of the call, keeps a memset out of the kernel chain.
__global__ void k_append_prefill(DevCtx c, PrefillArgs a, unsigned long long zero_vec, int late_wait) {
  // late_wait: the kernel in front of this one is the call's eviction kernel, which has released this one (see
  // chain_release): everything older is complete and visible, the two kernels touch different data, and this one
  // waits for the eviction kernel at its end (in its last CTA), so that whatever follows it follows both.
  if (!late_wait) chain_wait();
  const size_t gid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int c16 = gid & 15;
  size_t row = gid >> 4;  // over [layer_count][n][Hkv]
  const size_t nrows = (size_t)a.layer_count * a.n * c.Hkv;
  if (row >= nrows) {
    const size_t zi = gid - nrows * 16;
    if (zi < zero_vec)
      reinterpret_cast<uint4*>(c.Mq + (size_t)a.layer_begin * c.chunk * c.chunk)[zi] = make_uint4(0u, 0u, 0u, 0u);
  } else {
    const int g = row % c.Hkv;
    const int r = (row / c.Hkv) % a.n;
    const int l = row / ((size_t)c.Hkv * a.n);
    const size_t unit = unit_of(c, a.seq, a.layer_begin + l);
    const long long tok = a.t0 + r;
    const long long wrow = c.paged ? tok - a.shift : tok;  // window row (a sink token has one too while it is current)
    if (wrow < 0 || wrow >= c.SR) {                         // cannot happen: the host keeps the window inside the slab
      set_status(c, -2, (int)tok);
    } else {
      const size_t dst = ((unit * c.Hkv + g) * c.SR + wrow) * kD + c16 * 8;
      const size_t src = row * kD + c16 * 8;
      const uint4 kv = *reinterpret_cast<const uint4*>(a.k + src), vv = *reinterpret_cast<const uint4*>(a.v + src);
      *reinterpret_cast<uint4*>(c.Kc + dst) = kv;
      *reinterpret_cast<uint4*>(c.Vc + dst) = vv;
      if (c.paged && tok < c.Ls) {  // the sink's permanent rows
        const size_t sd = ((unit * c.Hkv + g) * c.SR + tok) * kD + c16 * 8;
        *reinterpret_cast<uint4*>(c.Kc + sd) = kv;
        *reinterpret_cast<uint4*>(c.Vc + sd) = vv;
      }
      if (g == 0 && c16 == 0) c.votes[unit * c.Tpad + a.t0 + r] = 0;
    }
  }
  // (only the last CTA waits: the grid is not complete before it is, and CTAs that sat waiting in every slot of an SM
  // would keep the rest of the grid from starting)
  if (late_wait && blockIdx.x == gridDim.x - 1) chain_wait();
}

cudaError_t launch_append_prefill(const DevCtx& c, const PrefillArgs& a, bool clear_maps, bool late_wait,
                                  cudaStream_t s) {
  const unsigned long long zero_vec = clear_maps ? (unsigned long long)a.layer_count * c.chunk * c.chunk / 4 : 0ull;
  const size_t threads = (size_t)a.layer_count * a.n * c.Hkv * 16 + zero_vec;
  return launch_chained(k_append_prefill, dim3((unsigned)((threads + 255) / 256)), dim3(256), 0, s, c, a, zero_vec,
                        late_wait ? 1 : 0);
}

__global__ void k_append_decode(DevCtx c, DecBatch b, int layer_begin, int layer_count,
                                const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v) {
  chain_wait();
  const size_t gid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int c16 = gid & 15;
  size_t row = gid >> 4;  // over [b.n][layer_count][Hkv]
  if (row >= (size_t)b.n * layer_count * c.Hkv) return;
  const int g = row % c.Hkv;
  const int l = (row / c.Hkv) % layer_count;
  const int bi = row / ((size_t)c.Hkv * layer_count);
  const size_t unit = unit_of(c, b.seq[bi], layer_begin + l);
  const long long tok = b.pos[bi];
  const long long wrow = c.paged ? tok - b.shift[bi] : tok;
  if (wrow < 0 || wrow >= c.SR) {  // cannot happen: the host keeps the window inside the slab
    set_status(c, -2, (int)tok);
    return;
  }
  const size_t dst = ((unit * c.Hkv + g) * c.SR + wrow) * kD + c16 * 8;
  const size_t src = (((size_t)b.src[bi] * layer_count + l) * c.Hkv + g) * kD + c16 * 8;
  const uint4 kv = *reinterpret_cast<const uint4*>(k + src), vv = *reinterpret_cast<const uint4*>(v + src);
  *reinterpret_cast<uint4*>(c.Kc + dst) = kv;
  *reinterpret_cast<uint4*>(c.Vc + dst) = vv;
  if (c.paged && tok < c.Ls) {  // the sink's permanent rows
    const size_t sd = ((unit * c.Hkv + g) * c.SR + tok) * kD + c16 * 8;
    *reinterpret_cast<uint4*>(c.Kc + sd) = kv;
    *reinterpret_cast<uint4*>(c.Vc + sd) = vv;
  }
  if (g == 0 && c16 == 0) {
    c.votes[unit * c.Tpad + b.pos[bi]] = 0;
  }
}

cudaError_t launch_append_decode(const DevCtx& c, const DecBatch& b, int layer_begin, int layer_count, int,
                                 const __nv_bfloat16* k, const __nv_bfloat16* v, cudaStream_t s) {
  const size_t threads = (size_t)b.n * layer_count * c.Hkv * 16;
  return launch_chained(k_append_decode, dim3((unsigned)((threads + 255) / 256)), dim3(256), 0, s, c, b, layer_begin,
                        layer_count, k, v);
}

// ------------------------------------------------------------------------------------------
// a1: regions that left the window: every span gets its index vector, the bf16 sum of the keys of
// its most voted token(s), and is appended to the span table.  One CTA per layer, one warp per span (32 warps).
__global__ void __launch_bounds__(1024) k_evict_index(DevCtx c, EvictArgs a) {
  chain_wait();
  if (a.release) chain_release();
  const int layer = a.layer_begin + blockIdx.x;
  const size_t unit = unit_of(c, a.seq, layer);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  const int base = c.n_spans[unit];
  const long long* votes = c.votes + unit * c.Tpad;
  int off = 0;
  for (int si = 0; si < a.nslots; ++si) {
    const size_t ps = (unit * c.slots + a.slot[si]) * c.Jmax;
    const int cnt = c.pend_cnt[unit * c.slots + a.slot[si]];
    for (int i = warp; i < cnt; i += nwarps) {
      const int start = c.pend_start[ps + i], len = c.pend_len[ps + i];
      const int dst = base + off + i;
      if (dst >= c.cap) {
        if (lane == 0) set_status(c, -2, dst);
        continue;
      }
      if (lane == 0) {
        c.span_start[unit * c.cap + dst] = start;
        c.span_len[unit * c.cap + dst] = len;
      }
      int toks[kMaxReps];
      const int nrep = select_reps(votes, start, len, c.rep_mode == 1 ? c.pend_nrep[ps + i] : c.reps, toks);
      for (int g = 0; g < c.Hkv; ++g) {
        const __nv_bfloat16* kslab = c.Kc + ((unit * c.Hkv + g) * c.SR) * kD;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int r = 0; r < nrep; ++r) {
          const uint2 raw =
              *reinterpret_cast<const uint2*>(kslab + (size_t)slab_row(c, toks[r], a.shift) * kD + lane * 4);
          const __nv_bfloat162 p0 = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
          const __nv_bfloat162 p1 = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
          acc[0] += __bfloat162float(p0.x);
          acc[1] += __bfloat162float(p0.y);
          acc[2] += __bfloat162float(p1.x);
          acc[3] += __bfloat162float(p1.y);
        }
        __nv_bfloat162 o0 = __floats2bfloat162_rn(acc[0], acc[1]);
        __nv_bfloat162 o1 = __floats2bfloat162_rn(acc[2], acc[3]);
        uint2 w;
        w.x = *reinterpret_cast<uint32_t*>(&o0);
        w.y = *reinterpret_cast<uint32_t*>(&o1);
        *reinterpret_cast<uint2*>(c.KR + ((unit * c.Hkv + g) * c.cap + dst) * kD + lane * 4) = w;
      }
    }
    off += cnt;
  }
  __syncthreads();
  if (threadIdx.x == 0) c.n_spans[unit] = min(base + off, c.cap);
}

cudaError_t launch_evict_index(const DevCtx& c, const EvictArgs& a, int layer_count, cudaStream_t s) {
  // a warp per span: one round for a region of up to 32 spans
  return launch_chained(k_evict_index, dim3(layer_count), dim3(1024), 0, s, c, a);
}

// ------------------------------------------------------------------------------------------
// Warp-parallel walks over a shared-memory histogram (all 32 lanes of one warp call them).
// pick_from_top: the largest bin b with  sum(hist[b+1..nb-1]) < need <= sum(hist[b..nb-1]);  `need` becomes the rank
// inside that bin.  pick_from_bottom: the smallest bin b with  rank < sum(hist[0..b]);  `rank` becomes the rank inside
// the bin.  Both clamp to the last bin they look at when the counts do not reach the target.  nb is a multiple of 32.
__device__ __forceinline__ int pick_from_top(const unsigned* hist, int nb, unsigned& need) {
  const int lane = threadIdx.x & 31, per = nb >> 5;
  const int b1 = nb - lane * per;  // lane 0 owns the top `per` bins
  unsigned mine = 0;
  for (int i = 1; i <= per; ++i) mine += hist[b1 - i];
  unsigned incl = mine;  // counts of this lane's bins and of all higher ones
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  const unsigned hit = __ballot_sync(0xffffffffu, incl >= need);
  const int src = hit ? __ffs(hit) - 1 : 31;
  int bin = 0;
  unsigned left = 0;
  if (lane == src) {
    left = need - (incl - mine);
    bin = b1 - 1;
    for (; bin > b1 - per; --bin) {
      if (left <= hist[bin]) break;
      left -= hist[bin];
    }
    if (!hit && left > hist[bin]) left = hist[bin];
  }
  need = __shfl_sync(0xffffffffu, left, src);
  return __shfl_sync(0xffffffffu, bin, src);
}

__device__ __forceinline__ unsigned pick_from_bottom(const unsigned* hist, int nb, long long& rank) {
  const int lane = threadIdx.x & 31, per = nb >> 5;
  const int b0 = lane * per;
  long long mine = 0;
  for (int i = 0; i < per; ++i) mine += hist[b0 + i];
  long long incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const long long t = shfl_up_ll(incl, o);
    if (lane >= o) incl += t;
  }
  const unsigned hit = __ballot_sync(0xffffffffu, rank < incl);
  const int src = hit ? __ffs(hit) - 1 : 31;
  unsigned bin = 0;
  long long left = 0;
  if (lane == src) {
    left = rank - (incl - mine);
    bin = (unsigned)b0;
    for (; bin < (unsigned)(b0 + per - 1); ++bin) {
      if (left < (long long)hist[bin]) break;
      left -= hist[bin];
    }
  }
  rank = shfl_ll(left, src);
  return __shfl_sync(0xffffffffu, bin, src);
}

// Counting one radix digit of many keys with few shared-memory atomics.  Scores of one head share their leading bits,
// so in the first passes nearly every key falls into the same bin and one atomic per key would serialise on it.  A
// thread adds up runs of equal digits among its own keys; when all lanes of a warp end on the same digit, the warp
// adds their last runs with one atomic.  flush() is called by all 32 lanes of a warp, converged.
struct DigitRuns {
  int cur = -1;
  unsigned run = 0;
  __device__ __forceinline__ void add(unsigned* hist, int d) {
    if (d == cur) {
      ++run;
    } else {
      if (run) atomicAdd(&hist[cur], run);
      cur = d;
      run = 1;
    }
  }
  __device__ __forceinline__ void flush(unsigned* hist) {
    const int top = __reduce_max_sync(0xffffffffu, cur);  // (-1: a lane without a matching key)
    if (__all_sync(0xffffffffu, cur == top || cur < 0)) {
      const unsigned sum = __reduce_add_sync(0xffffffffu, run);
      if ((threadIdx.x & 31) == 0 && sum) atomicAdd(&hist[top], sum);
    } else if (run) {
      atomicAdd(&hist[cur], run);
    }
    cur = -1;
    run = 0;
  }
};

// Exclusive scan of the nt (a multiple of 32, at most 1024) counts in s_scan by the first warp of the CTA; returns the
// total to every thread of that warp.  The caller brackets it with __syncthreads().
__device__ __forceinline__ int warp0_exclusive_scan(int* s_scan, int nt) {
  const int lane = threadIdx.x & 31;
  int run = 0;
  for (int blk = 0; blk < nt; blk += 32) {
    const int v = s_scan[blk + lane];
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += t;
    }
    s_scan[blk + lane] = run + inc - v;
    run += __shfl_sync(0xffffffffu, inc, 31);
  }
  return run;
}

// ------------------------------------------------------------------------------------------
// a3 segmenter, step 1: exact rank selection of theta (quantile mode) over the causal entries of Mq.
// Pass 1 counts negatives (only hand-built maps have any) and zeros (a sparse map is mostly zeros) and builds a
// log-scale histogram of the positive entries: bin = (position of the leading one, next four bits), which is monotone
// in the value and spreads a heavy-tailed map over many bins.  If the rank falls among the positives, the remaining
// low bits of the selected bin are resolved by MSB radix passes of 9 bits.  One private histogram per warp, four loads
// in flight per lane; a thread-block cluster of eight CTAs shares a layer: each counts its share of the rows, then
// every CTA adds up the eight histograms through distributed shared memory and takes the same decision.
constexpr int kThetaBits = 9;
constexpr int kThetaBins = 1 << kThetaBits;

// visits the causal entries of the m x m map: f(value) for every (i, j <= i).  The rows are dealt to the warps of the
// `nparts` CTAs that share a map in pairs (i, m-1-i), so every warp sees about the same number of entries.
template <typename F>
__device__ __forceinline__ void for_each_causal(const int* __restrict__ Mq, int ld, int m, int part, int nparts, F&& f) {
  const int lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  const int gw = part * nwarps + (threadIdx.x >> 5), step = nparts * nwarps;
  for (int idx = gw; 2 * idx < m; idx += step) {
#pragma unroll 1
    for (int side = 0; side < 2; ++side) {
      const int i = side == 0 ? idx : m - 1 - idx;
      if (side == 1 && i == idx) break;
      const int* row = Mq + (size_t)i * ld;
      for (int j0 = 0; j0 <= i; j0 += 128) {
        int v[4];
        bool ok[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int j = j0 + u * 32 + lane;
          ok[u] = j <= i;
          v[u] = ok[u] ? row[j] : 0;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (ok[u]) f(v[u]);
      }
    }
  }
}

// monotone log-scale bin of a positive value: 16 bins per power of two
__device__ __forceinline__ unsigned log_bin(unsigned v) {
  const int e = 31 - __clz(v);
  const unsigned frac = e >= 4 ? (v >> (e - 4)) & 15u : (v << (4 - e)) & 15u;
  return ((unsigned)e << 4) | frac;
}

constexpr int kThetaCluster = 8;   // CTAs (one thread-block cluster) per layer
constexpr int kThetaThreads = 512;

__global__ void __cluster_dims__(kThetaCluster, 1, 1) __launch_bounds__(kThetaThreads)
    k_theta_select(DevCtx c, int layer_begin, int m, long long rank, int tables) {
  chain_wait();
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  extern __shared__ unsigned hist[];  // [warps][kThetaBins]
  constexpr int NW = kThetaThreads / 32;
  const int layer = layer_begin + blockIdx.x / kThetaCluster;
  const int part = (int)cluster.block_rank();
  if (tables && c.theta_l) {  // the layer's own quantile level: the same double arithmetic as on the host
    const long long N = (long long)m * (m + 1) / 2;
    rank = (long long)floor((double)c.theta_l[layer] * (double)(N - 1));
    rank = rank < 0 ? 0 : (rank > N - 1 ? N - 1 : rank);
  }
  const int* Mq = c.Mq + (size_t)layer * c.chunk * c.chunk;
  __shared__ unsigned loc[kThetaBins + 2];  // this CTA's histogram, then its counts of negatives and zeros
  __shared__ unsigned tot[kThetaBins];      // the cluster's histogram (every CTA builds its own copy)
  __shared__ unsigned s_red[NW][2];
  __shared__ unsigned s_prefix, s_lo_bits;
  __shared__ long long s_rank, s_cn, s_cz;
  __shared__ int s_cls;  // 0: answer found, 1: among positives (bin chosen), -1: among negatives
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  unsigned* myhist = hist + warp * kThetaBins;
  // sums the per-warp histograms into loc, then the cluster's loc arrays into tot.  The second cluster barrier keeps
  // every CTA's loc intact until all have read it (and keeps a CTA from exiting while it can still be read).
  auto combine = [&](bool with_counts) {
    __syncthreads();
    if (threadIdx.x < kThetaBins) {
      unsigned sum = 0;
      for (int w = 0; w < NW; ++w) sum += hist[w * kThetaBins + threadIdx.x];
      loc[threadIdx.x] = sum;
    }
    if (with_counts && threadIdx.x == 0) {
      unsigned cn = 0, cz = 0;
      for (int w = 0; w < NW; ++w) {
        cn += s_red[w][0];
        cz += s_red[w][1];
      }
      loc[kThetaBins] = cn;
      loc[kThetaBins + 1] = cz;
    }
    cluster.sync();
    if (threadIdx.x < kThetaBins) {
      unsigned sum = 0;
      for (int r = 0; r < kThetaCluster; ++r) sum += cluster.map_shared_rank(loc, r)[threadIdx.x];
      tot[threadIdx.x] = sum;
    }
    if (with_counts && threadIdx.x == 0) {
      long long cn = 0, cz = 0;
      for (int r = 0; r < kThetaCluster; ++r) {
        const unsigned* rl = cluster.map_shared_rank(loc, r);
        cn += rl[kThetaBins];
        cz += rl[kThetaBins + 1];
      }
      s_cn = cn;
      s_cz = cz;
    }
    cluster.sync();
  };
  for (int t = threadIdx.x; t < NW * kThetaBins; t += blockDim.x) hist[t] = 0;
  __syncthreads();
  unsigned nneg = 0, nzero = 0;
  for_each_causal(Mq, c.chunk, m, part, kThetaCluster, [&](int v) {
    if (v > 0)
      atomicAdd(&myhist[log_bin((unsigned)v)], 1u);
    else if (v == 0)
      ++nzero;
    else
      ++nneg;
  });
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    nneg += __shfl_xor_sync(0xffffffffu, nneg, o);
    nzero += __shfl_xor_sync(0xffffffffu, nzero, o);
  }
  if (lane == 0) {
    s_red[warp][0] = nneg;
    s_red[warp][1] = nzero;
  }
  combine(true);
  if (threadIdx.x < 32) {
    const long long cn = s_cn, cz = s_cz;
    if (rank < cn) {
      if (lane == 0) {
        s_cls = -1;
        s_rank = rank;
      }
    } else if (rank < cn + cz) {
      if (lane == 0) {
        s_cls = 0;
        if (part == 0) c.thetaq[layer] = 0;
      }
    } else {
      long long r = rank - cn - cz;
      const unsigned b = pick_from_bottom(tot, kThetaBins, r);
      const int e = (int)(b >> 4);
      const unsigned frac = b & 15u;
      if (lane == 0) {
        s_rank = r;
        if (e <= 4) {  // the bin holds a single value
          s_cls = 0;
          if (part == 0) c.thetaq[layer] = (long long)((1u << e) | (frac >> (4 - e)));
        } else {
          s_cls = 1;
          s_prefix = (1u << e) | (frac << (e - 4));  // leading one and the next four bits
          s_lo_bits = (unsigned)(e - 4);             // bits still unknown
        }
      }
    }
  }
  __syncthreads();
  const int cls = s_cls;
  if (cls == 0) return;  // the same decision in every CTA of the cluster
  // remaining bits: [0, hi).  Negatives: plain MSB radix over the sign-flipped key.
  int hi = cls > 0 ? (int)s_lo_bits : 31;
  if (cls < 0 && threadIdx.x == 0) s_prefix = 0;
  __syncthreads();
  while (hi > 0) {
    const int lo = max(0, hi - kThetaBits);
    const unsigned dmask = (1u << (hi - lo)) - 1u;
    for (int t = threadIdx.x; t < NW * kThetaBins; t += blockDim.x) hist[t] = 0;
    __syncthreads();
    const unsigned prefix = s_prefix;
    for_each_causal(Mq, c.chunk, m, part, kThetaCluster, [&](int v) {
      const bool in_cls = cls > 0 ? v > 0 : v < 0;
      const unsigned key = cls > 0 ? (unsigned)v : ((unsigned)v ^ 0x80000000u);
      if (in_cls && (key >> hi) == (prefix >> hi)) atomicAdd(&myhist[(key >> lo) & dmask], 1u);
    });
    combine(false);
    if (threadIdx.x < 32) {
      long long r = s_rank;
      unsigned b = pick_from_bottom(tot, kThetaBins, r);  // bins above dmask are empty
      if (b > dmask) b = dmask;
      if (threadIdx.x == 0) {
        s_rank = r;
        s_prefix = prefix | (b << lo);
      }
    }
    __syncthreads();
    hi = lo;
  }
  if (threadIdx.x == 0 && part == 0)
    c.thetaq[layer] = cls > 0 ? (long long)s_prefix : (long long)(int)(s_prefix ^ 0x80000000u);
}

// absolute threshold: thq in units of the map summed over all heads, thq1 in units of a single (retrieval) head's map;
// with per-layer tables the layer's own theta, scaled here
__global__ void k_theta_set(DevCtx c, int layer_begin, long long thq, long long thq1, int tables) {
  chain_wait();
  const int layer = layer_begin + blockIdx.x;
  const bool one = ret_head_of(c, layer) >= 0;
  long long t = one ? thq1 : thq;
  if (tables && c.theta_l) t = (long long)rint((double)c.theta_l[layer] * (one ? 1.0 : (double)c.Hq) * (double)kQScale);
  c.thetaq[layer] = t;
}

// step 2: suffix sums along each row of D = Mq - theta ("sum the right elements", Fig. 2):
// Rsuf[i][x] = sum_{j=x..i} D[i][j].  One warp per row, 32-wide shuffle scans from the diagonal leftwards.
__global__ void __launch_bounds__(256) k_seg_rowscan(DevCtx c, int layer_begin, int m) {
  chain_wait();
  const int layer = layer_begin + blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int i = blockIdx.x * 8 + warp;
  if (blockIdx.x == 0)
    for (int t = threadIdx.x; t < 2 * c.chunk; t += blockDim.x) c.best[(size_t)layer * 2 * c.chunk + t] = 0;
  if (i >= m) return;
  const long long thq = c.thetaq[layer];
  const int* row = c.Mq + ((size_t)layer * c.chunk + i) * c.chunk;
  long long* out = c.Rsuf + ((size_t)layer * c.chunk + i) * c.chunk;
  long long carry = 0;
  for (int hi = i; hi >= 0; hi -= 32) {
    const int x = hi - lane;  // lane 0 is the rightmost element of this group
    long long v = x >= 0 ? (long long)row[x] - thq : 0;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const long long t = shfl_up_ll(v, o);
      if (lane >= o) v += t;
    }
    v += carry;
    if (x >= 0) out[x] = v;
    carry = shfl_ll(v, 31);
  }
}

// step 3: prefix sums down each column ("sum the upper elements"): S(x,y) = sum_{i=x..y} Rsuf[i][x], and the
// best point of every anti-diagonal x+y=c (max S, ties -> shorter span), kept only when S > 0.
// A CTA owns 32 columns; thread (cx, ry) scans rows [ry*R, ry*R+R) of its column, a shared-memory scan over ry
// supplies the offsets, and a second pass emits S.  key = (S << 10) | (1023 - (y-x)).
// seg_unit > 0 (segmentation per memory unit): only intervals inside one unit of seg_unit tokens on the absolute grid
// are candidates; `origin` is the absolute position of the region's first token.
// HOLD: a thread keeps its (at most 16) entries of the column in registers between the two passes (m <= 512).
template <bool HOLD>
__global__ void __launch_bounds__(1024) k_seg_colscan(DevCtx c, int layer_begin, int m, int seg_unit, int origin) {
  chain_wait();
  extern __shared__ long long sm[];
  long long* part = sm;             // [32 ry][32 cx]
  long long* sbest = sm + 32 * 32;  // [m + 32]
  const int layer = layer_begin + blockIdx.y;
  const int cx = threadIdx.x & 31, ry = threadIdx.x >> 5;
  const int x0 = blockIdx.x * 32, x = x0 + cx;
  const int R = (m + 31) / 32;
  const long long* Rs = c.Rsuf + (size_t)layer * c.chunk * c.chunk;
  for (int t = threadIdx.x; t < m + 32; t += blockDim.x) sbest[t] = 0;
  const int ylo = ry * R, yhi = min(m, ylo + R);
  long long acc = 0;
  long long cv[HOLD ? 16 : 1];
  if (HOLD) {
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      const int y = ylo + k;
      cv[k] = (x < m && y >= x && y < yhi) ? Rs[(size_t)y * c.chunk + x] : 0;
    }
#pragma unroll
    for (int k = 0; k < 16; ++k) acc += cv[k];
  } else if (x < m) {
    for (int y = max(ylo, x); y < yhi; ++y) acc += Rs[(size_t)y * c.chunk + x];
  }
  part[ry * 32 + cx] = acc;
  __syncthreads();
  if (ry == 0) {  // exclusive scan over ry for column cx
    long long run = 0;
    for (int r = 0; r < 32; ++r) {
      const long long t = part[r * 32 + cx];
      part[r * 32 + cx] = run;
      run += t;
    }
  }
  __syncthreads();
  if (x < m) {
    long long S = part[ry * 32 + cx];
    // last token of the unit that holds x (region-relative)
    const int ymax = seg_unit > 0 ? ((origin + x) / seg_unit + 1) * seg_unit - origin - 1 : m;
    if (HOLD) {
#pragma unroll
      for (int k = 0; k < 16; ++k) {
        const int y = ylo + k;
        if (y < x || y >= yhi) continue;
        S += cv[k];
        if (S > 0 && y <= ymax) {
          const long long key = (S << 10) | (long long)(1023 - (y - x));
          atomicMax(&sbest[x + y - 2 * x0], key);
        }
      }
    } else {
      for (int y = max(ylo, x); y < yhi; ++y) {
        S += Rs[(size_t)y * c.chunk + x];
        if (S > 0 && y <= ymax) {
          const long long key = (S << 10) | (long long)(1023 - (y - x));
          atomicMax(&sbest[x + y - 2 * x0], key);
        }
      }
    }
  }
  __syncthreads();
  long long* gbest = c.best + (size_t)layer * 2 * c.chunk;
  for (int t = threadIdx.x; t < m + 32; t += blockDim.x) {
    const long long key = sbest[t];
    const int cd = 2 * x0 + t;
    if (key > 0 && cd <= 2 * m - 2) atomicMax(&gbest[cd], key);
  }
}

// step 4: the <= 2m-1 candidates in the order (S desc, length asc, start asc), greedy non-maximum suppression with
// IoU threshold 0 until max_spans are kept, gap fill, store the region's spans in its pending slot; then the
// query representatives of every span (Sec. 3.4 step 2): u[g][j] = sum_{h in g} sum_{rep tokens} q_h[tok].
// NMS on the squares (x, x, y+1, y+1): a candidate is suppressed by a kept span when their IoU exceeds phi_milli/1000;
// two spans that share `inter` tokens have IoU = inter^2 / (L1^2 + L2^2 - inter^2).  Integer arithmetic; phi = 0
// means any overlap suppresses.
__device__ __forceinline__ bool nms_suppressed(int x, int y, int kx, int ky, int phi_milli) {
  const long long inter = (long long)min(y, ky) - max(x, kx) + 1;
  if (inter <= 0) return false;
  const long long l1 = y - x + 1, l2 = ky - kx + 1, i2 = inter * inter;
  return i2 * 1000 > (long long)phi_milli * (l1 * l1 + l2 * l2 - i2);
}

struct NmsArgs {
  int seq, layer_begin, m, reg_start, slot, max_spans;
  int n, t0;                 // query tensor geometry (q == nullptr: skip the representatives)
  const __nv_bfloat16* q;
  int tables;                // use the context's per-layer phi and lambda tables where it has them
  int seg_unit;              // > 0: every unit of this many tokens (absolute grid) keeps max_spans spans of its own
};

__global__ void __launch_bounds__(1024) k_seg_nms(DevCtx c, NmsArgs a) {
  chain_wait();
  __shared__ long long skey[768];  // scratch of the query representatives: token lists and counts per span
  __shared__ int kx[kMaxTopK], ky[kMaxTopK];
  __shared__ int out_start[2 * kMaxTopK + 1], out_len[2 * kMaxTopK + 1];
  __shared__ int s_nout;
  __shared__ int s_ucnt[kMaxTopK + 2];  // segmentation per unit: spans kept in every unit the region touches
  const int layer = a.layer_begin + blockIdx.x;
  const size_t unit = unit_of(c, a.seq, layer);
  const int m = a.m;
  const int SU = a.seg_unit;
  auto unit_idx = [&](int x) { return (a.reg_start + x) / SU - a.reg_start / SU; };
  const int cap_total = SU > 0 ? kMaxTopK : a.max_spans;
  const int phi_milli = a.tables && c.phi_l ? c.phi_l[layer] : c.phi_milli;
  const float rep_lambda = a.tables && c.lambda_l ? c.lambda_l[layer] : c.rep_lambda;
  const int ncand = 2 * m - 1;
  const long long* gbest = c.best + (size_t)layer * 2 * c.chunk;
  // Greedy NMS without a sort: the candidate the sorted sweep would reach next is the best one that is still alive
  // (key larger, or equal key and smaller anti-diagonal), so every round takes the block-wide maximum over the alive
  // candidates, keeps it, and lets every thread strike out its own candidates that the new span suppresses (or whose
  // unit is full).  At most max_spans rounds of two barriers each instead of sorting up to 2047 keys.
  // Candidate of anti-diagonal cd: key = (S << 10) | (1023 - len) > 0; x = (cd - len) / 2, y = x + len.
  __shared__ long long s_wkey[32];
  __shared__ int s_wcd[32];
  const int tid = threadIdx.x, wlane = tid & 31, wid = tid >> 5;
  long long ckey[2];
  int cx[2], cy[2];
  bool alive[2];
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    const int cd = tid + u * 1024;
    ckey[u] = cd < ncand ? gbest[cd] : 0;
    const int len = 1023 - (int)(ckey[u] & 1023);
    cx[u] = (cd - len) >> 1;
    cy[u] = cx[u] + len;
    alive[u] = ckey[u] > 0;
  }
  for (int t = tid; t < kMaxTopK + 2; t += blockDim.x) s_ucnt[t] = 0;
  int kept = 0;
  auto better = [](long long ka, int ca, long long kb, int cb) { return ka > kb || (ka == kb && ca < cb); };
  while (kept < cap_total) {
    long long bk = 0;
    int bc = 0x7fffffff;
#pragma unroll
    for (int u = 0; u < 2; ++u)
      if (alive[u] && better(ckey[u], tid + u * 1024, bk, bc)) {
        bk = ckey[u];
        bc = tid + u * 1024;
      }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const long long ok = shfl_xor_ll(bk, o);
      const int oc = __shfl_xor_sync(0xffffffffu, bc, o);
      if (better(ok, oc, bk, bc)) {
        bk = ok;
        bc = oc;
      }
    }
    if (wlane == 0) {
      s_wkey[wid] = bk;
      s_wcd[wid] = bc;
    }
    __syncthreads();
    bk = s_wkey[wlane];  // every warp reduces the 32 partial results itself: all threads learn the winner
    bc = s_wcd[wlane];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const long long ok = shfl_xor_ll(bk, o);
      const int oc = __shfl_xor_sync(0xffffffffu, bc, o);
      if (better(ok, oc, bk, bc)) {
        bk = ok;
        bc = oc;
      }
    }
    if (bk <= 0) break;  // nothing alive is left (the same decision in every thread)
    const int wl = 1023 - (int)(bk & 1023);
    const int wx = (bc - wl) >> 1, wy = wx + wl;
    if (tid == 0) {
      kx[kept] = wx;
      ky[kept] = wy;
      if (SU > 0) ++s_ucnt[unit_idx(wx)];
    }
    ++kept;
    __syncthreads();  // the unit counts are up to date; s_wkey may be overwritten
#pragma unroll
    for (int u = 0; u < 2; ++u)
      alive[u] = alive[u] && tid + u * 1024 != bc && !nms_suppressed(cx[u], cy[u], wx, wy, phi_milli) &&
                 (SU == 0 || s_ucnt[unit_idx(cx[u])] < a.max_spans);
  }
  __syncthreads();
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    // order the kept spans by start (rank sort), then gap fill
    int rank0 = 0, rank1 = 0;
    const int x0 = lane < kept ? kx[lane] : 0x7fffffff;
    const int x1 = lane + 32 < kept ? kx[lane + 32] : 0x7fffffff;
    const int y0 = lane < kept ? ky[lane] : 0, y1 = lane + 32 < kept ? ky[lane + 32] : 0;
    for (int q = 0; q < kept; ++q) {  // with phi > 0 two kept spans may share their start: then the shorter first
      rank0 += kx[q] < x0 || (kx[q] == x0 && ky[q] < y0);
      rank1 += kx[q] < x1 || (kx[q] == x1 && ky[q] < y1);
    }
    __syncwarp();
    if (lane < kept) kx[rank0] = x0;
    if (lane + 32 < kept) kx[rank1] = x1;
    __syncwarp();
    if (lane < kept) ky[rank0] = y0;
    if (lane + 32 < kept) ky[rank1] = y1;
    __syncwarp();
    if (lane == 0) {
      int pos = 0, no = 0;
      // an uncovered run [g0, g1) becomes a span; under segmentation per unit it is cut at the unit boundaries
      auto emit_gap = [&](int g0, int g1) {
        while (g0 < g1 && no < 2 * kMaxTopK + 1) {
          const int e = SU > 0 ? min(g1, ((a.reg_start + g0) / SU + 1) * SU - a.reg_start) : g1;
          out_start[no] = g0;
          out_len[no++] = e - g0;
          g0 = e;
        }
      };
      for (int q = 0; q < kept; ++q) {
        if (kx[q] > pos) emit_gap(pos, kx[q]);
        if (no < 2 * kMaxTopK + 1) {
          out_start[no] = kx[q];
          out_len[no++] = ky[q] - kx[q] + 1;
        }
        pos = max(pos, ky[q] + 1);  // kept spans may overlap when phi > 0
      }
      if (pos < m) emit_gap(pos, m);
      s_nout = no;
    }
  }
  __syncthreads();
  const int nout = s_nout;
  const size_t ps = (unit * c.slots + a.slot) * c.Jmax;
  if (nout > c.Jmax) {
    if (threadIdx.x == 0) set_status(c, -5, nout);
    return;
  }
  for (int t = threadIdx.x; t < nout; t += blockDim.x) {
    c.pend_start[ps + t] = a.reg_start + out_start[t];
    c.pend_len[ps + t] = out_len[t];
  }
  if (threadIdx.x == 0) {
    c.pend_cnt[unit * c.slots + a.slot] = nout;
    c.Jcnt[layer] = a.q ? nout : 0;
  }
  // query representatives.  First one warp per span picks the representative tokens, then one warp per
  // (span, KV head) sums their query rows with all loads of the head group in flight at once.
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  const long long* votes = c.votes + unit * c.Tpad;
  const __nv_bfloat16* q = a.q + (size_t)blockIdx.x * a.n * c.Hq * kD;
  int* rep_tok = reinterpret_cast<int*>(skey);          // [Jmax][kMaxReps]
  int* rep_cnt = rep_tok + (2 * kMaxTopK + 1) * kMaxReps;
  __syncthreads();
  // representative count of every span: static, or from the area ratio of Sec. 3.3.2 on the raw region map.  The
  // row-suffix table holds sums of (Mq - theta), so a raw sum over w entries is the table value + theta * w.
  int* nrep_of = rep_cnt + (2 * kMaxTopK + 1);
  for (int j = warp; j < nout; j += nwarps) {
    int cnt = min(c.reps, out_len[j]);
    if (c.rep_mode == 1) {
      const long long* Rs = c.Rsuf + (size_t)layer * c.chunk * c.chunk;
      const long long th = c.thetaq[layer];
      const int x = out_start[j], y = x + out_len[j] - 1;
      long long T = 0, TR = 0, Cn = 0;
      for (int i = x + lane; i <= y; i += 32) {
        T += Rs[(size_t)i * c.chunk + x] + th * (i - x + 1);
        TR += Rs[(size_t)i * c.chunk] + th * (i + 1);
      }
      for (int i = y + 1 + lane; i < m; i += 32)
        Cn += Rs[(size_t)i * c.chunk + x] - Rs[(size_t)i * c.chunk + y + 1] + th * (y - x + 1);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        T += shfl_xor_ll(T, o);
        TR += shfl_xor_ll(TR, o);
        Cn += shfl_xor_ll(Cn, o);
      }
      const long long R = TR - T;
      const long long nb = c.ratio_kind == 0 ? R : c.ratio_kind == 1 ? Cn : R + Cn;
      const double ra = (T + nb) > 0 ? (double)T / (double)(T + nb) : 1.0;
      const double rv = 1.0 / exp((double)rep_lambda * (1.0 - ra));
      cnt = (int)rint((double)out_len[j] * rv);  // to nearest even
      cnt = max(cnt, c.min_reps);
      cnt = min(cnt, c.max_reps);
      cnt = min(cnt, out_len[j]);
      cnt = max(cnt, 1);
    }
    if (lane == 0) {
      nrep_of[j] = cnt;
      if (c.pend_nrep) c.pend_nrep[ps + j] = cnt;  // (absent in the scratch-only context of the static entry)
      if (c.nrep_last) c.nrep_last[(size_t)layer * c.Jmax + j] = cnt;
    }
  }
  __syncthreads();
  if (!a.q) return;
  for (int j = warp; j < nout; j += nwarps) {
    int toks[kMaxReps];
    const int nrep = select_reps(votes, a.reg_start + out_start[j], out_len[j], nrep_of[j], toks);
    if (lane == 0) {
      rep_cnt[j] = nrep;
      for (int r = 0; r < nrep; ++r) rep_tok[j * kMaxReps + r] = toks[r];
    }
  }
  __syncthreads();
  // a half-warp per (span, KV head): sixteen lanes x eight dimensions; the rows of the heads of the group are all in
  // flight before they are added up, per head over the representative tokens (ascending) and then over the heads in
  // ascending order
  const int hw = lane >> 4, hl = lane & 15;
  const int rh = ret_head_of(c, layer);
  for (int task = 2 * warp + hw; task < nout * c.Hkv; task += 2 * nwarps) {
    const int j = task / c.Hkv, g = task % c.Hkv;
    const int nrep = rep_cnt[j];
    const __nv_bfloat16* qg = q + (size_t)g * c.G * kD + hl * 8;
    // a layer with a retrieval head (Sec. 3.5) has one representative per span, that head's: the other heads add zero
    auto counts = [&](int hh) { return hh < c.G && (rh < 0 || g * c.G + hh == rh); };
    auto add8 = [](float (&acc)[8], const uint4& w) {
      const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&w);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = __bfloat1622float2(p2[i]);
        acc[2 * i] += f.x;
        acc[2 * i + 1] += f.y;
      }
    };
    float ug[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) ug[e] = 0.f;
    if (nrep == 1) {
      const __nv_bfloat16* row = qg + (size_t)(rep_tok[j * kMaxReps] - a.t0) * c.Hq * kD;
      for (int h0 = 0; h0 < c.G; h0 += 8) {
        uint4 raw[8];
#pragma unroll
        for (int hh = 0; hh < 8; ++hh)
          raw[hh] = counts(h0 + hh) ? *reinterpret_cast<const uint4*>(row + (size_t)(h0 + hh) * kD) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int hh = 0; hh < 8; ++hh) {
          float one[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) one[e] = 0.f;
          add8(one, raw[hh]);  // (0 + x first, as the general path does)
#pragma unroll
          for (int e = 0; e < 8; ++e) ug[e] += one[e];
        }
      }
    } else {
      for (int hh = 0; hh < c.G; ++hh) {
        if (!counts(hh)) continue;
        uint4 raw[kMaxReps];
#pragma unroll
        for (int r = 0; r < kMaxReps; ++r)
          raw[r] = r < nrep ? *reinterpret_cast<const uint4*>(qg + ((size_t)(rep_tok[j * kMaxReps + r] - a.t0) * c.Hq + hh) * kD)
                            : make_uint4(0u, 0u, 0u, 0u);
        float one[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) one[e] = 0.f;
#pragma unroll
        for (int r = 0; r < kMaxReps; ++r)
          if (r < nrep) add8(one, raw[r]);
#pragma unroll
        for (int e = 0; e < 8; ++e) ug[e] += one[e];
      }
    }
    float* up = c.u + (((size_t)layer * c.Hkv + g) * c.Jmax + j) * kD + hl * 8;
    *reinterpret_cast<float4*>(up) = make_float4(ug[0], ug[1], ug[2], ug[3]);
    *reinterpret_cast<float4*>(up + 4) = make_float4(ug[4], ug[5], ug[6], ug[7]);
  }
}

cudaError_t launch_segment(const DevCtx& c, int seq, int layer_begin, int layer_count, int m, int reg_start,
                             int slot, int theta_mode, float theta, long long theta_q_abs, int max_spans, int n,
                             int t0, const __nv_bfloat16* q, cudaStream_t s, bool tables, int seg_unit) {
  if (theta_mode == 1) {
    const long long N = (long long)m * (m + 1) / 2;
    long long rank = (long long)floor((double)theta * (double)(N - 1));
    if (rank < 0) rank = 0;
    if (rank > N - 1) rank = N - 1;
    const int hsmem = (kThetaThreads / 32) * kThetaBins * (int)sizeof(unsigned);
    launch_chained(k_theta_select, dim3(layer_count * kThetaCluster), dim3(kThetaThreads), hsmem, s, c, layer_begin, m,
                   rank, tables ? 1 : 0);
  } else {
    launch_chained(k_theta_set, dim3(layer_count), dim3(1), 0, s, c, layer_begin, theta_q_abs,
                   (long long)nearbyint((double)theta * (double)kQScale), tables ? 1 : 0);
  }
  launch_chained(k_seg_rowscan, dim3((m + 7) / 8, layer_count), dim3(256), 0, s, c, layer_begin, m);
  const size_t smem = (size_t)(32 * 32 + m + 32) * sizeof(long long);
  if (m <= 512)
    launch_chained(k_seg_colscan<true>, dim3((m + 31) / 32, layer_count), dim3(1024), smem, s, c, layer_begin, m, seg_unit,
                   reg_start);
  else
    launch_chained(k_seg_colscan<false>, dim3((m + 31) / 32, layer_count), dim3(1024), smem, s, c, layer_begin, m,
                   seg_unit, reg_start);
  NmsArgs a{seq, layer_begin, m, reg_start, slot, max_spans, n, t0, q, tables ? 1 : 0, seg_unit};
  launch_chained(k_seg_nms, dim3(layer_count), dim3(1024), 0, s, c, a);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// a4 scores (Eq. 7 with summed representatives, max over the call's query spans):
// score[g][s] = max_j u[g][j] . K^R[g][s].  One warp per span, 4 dims per lane.
template <bool DECODE>
__global__ void __launch_bounds__(256) k_score(DevCtx c, int seq, int layer_begin, DecBatch b, int layer_count,
                                               const __nv_bfloat16* __restrict__ q) {
  extern __shared__ float su[];  // [J][128]
  int layer, sq, J;
  const int g = blockIdx.y;
  if (DECODE) {
    const int bi = blockIdx.z / layer_count;
    layer = layer_begin + blockIdx.z % layer_count;
    sq = b.seq[bi];
    J = 1;
    if (threadIdx.x < kD) {
      const __nv_bfloat16* qp =
          q + (((size_t)b.src[bi] * layer_count + (layer - layer_begin)) * c.Hq + g * c.G) * kD + threadIdx.x;
      float acc = 0.f;
      for (int hh = 0; hh < c.G; ++hh) acc += __bfloat162float(qp[(size_t)hh * kD]);
      su[threadIdx.x] = acc;
    }
  } else {
    layer = layer_begin + blockIdx.z;
    sq = seq;
    J = c.Jcnt[layer];
    const float* up = c.u + ((size_t)layer * c.Hkv + g) * c.Jmax * kD;
    for (int t = threadIdx.x; t < J * kD; t += blockDim.x) su[t] = up[t];
  }
  const size_t unit = unit_of(c, sq, layer);
  __syncthreads();
  const int N = c.n_spans[unit];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int s0 = blockIdx.x * 64;
  const __nv_bfloat16* KR = c.KR + (unit * c.Hkv + g) * (size_t)c.cap * kD;
  float* sc = c.scores + (unit * c.Hkv + g) * (size_t)c.cap;
  for (int s = s0 + warp; s < min(s0 + 64, N); s += 8) {
    const uint2 raw = *reinterpret_cast<const uint2*>(KR + (size_t)s * kD + lane * 4);
    const __nv_bfloat162 p0 = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
    const __nv_bfloat162 p1 = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
    const float k0 = __bfloat162float(p0.x), k1 = __bfloat162float(p0.y), k2 = __bfloat162float(p1.x),
                k3 = __bfloat162float(p1.y);
    float best = -INFINITY;
    for (int j = 0; j < J; ++j) {
      const float4 uv = *reinterpret_cast<const float4*>(su + j * kD + lane * 4);
      float d = uv.x * k0;
      d = fmaf(uv.y, k1, d);
      d = fmaf(uv.z, k2, d);
      d = fmaf(uv.w, k3, d);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
      best = fmaxf(best, d);
    }
    if (lane == 0) sc[s] = best;
  }
}

cudaError_t launch_score_prefill(const DevCtx& c, const PrefillArgs& a, int span_bound, cudaStream_t s) {
  DecBatch dummy;
  dummy.n = 0;
  const size_t smem = (size_t)c.Jmax * kD * sizeof(float);
  if (smem > 48 * 1024) cudaFuncSetAttribute(k_score<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  k_score<false><<<dim3((span_bound + 63) / 64, c.Hkv, a.layer_count), 256, smem, s>>>(c, a.seq, a.layer_begin, dummy,
                                                                                       a.layer_count, nullptr);
  return cudaGetLastError();
}

// decode scores, memory-bound index scan: one query representative per KV head (the summed query of the group).
// Half-warp per 256-byte index row, 16 bytes per lane, four rows in flight; grid (span tiles of 256, Hkv, units).
__global__ void __launch_bounds__(256) k_score_dec(DevCtx c, int layer_begin, DecBatch b, int layer_count,
                                                   const __nv_bfloat16* __restrict__ q) {
  chain_wait();
  __shared__ float su[kD];
  const int g = blockIdx.y;
  const int bi = blockIdx.z / layer_count, l = blockIdx.z % layer_count, layer = layer_begin + l;
  const size_t unit = unit_of(c, b.seq[bi], layer);
  const int tid = threadIdx.x;
  const int N = c.n_spans[unit];
  // a layer with a retrieval head (Sec. 3.5) scores that head's query against the index of its KV head, for every g
  const int rh = ret_head_of(c, layer), gk = rh >= 0 ? rh / c.G : g;
  const int s0 = blockIdx.x * 256;
  if (s0 >= N) return;
  if (tid < kD) {
    const __nv_bfloat16* qp = q + (((size_t)b.src[bi] * layer_count + l) * c.Hq + gk * c.G) * kD + tid;
    float acc = 0.f;
    for (int hh = 0; hh < c.G; ++hh)
      if (rh < 0 || gk * c.G + hh == rh) acc += __bfloat162float(qp[(size_t)hh * kD]);
    su[tid] = acc;
  }
  __syncthreads();
  const int hw = tid >> 4, hl = tid & 15;  // 16 half-warps
  float uf[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) uf[e] = su[hl * 8 + e];
  const __nv_bfloat16* KR = c.KR + (unit * c.Hkv + gk) * (size_t)c.cap * kD + hl * 8;
  float* sc = c.scores + (unit * c.Hkv + g) * (size_t)c.cap;
#pragma unroll
  for (int rep = 0; rep < 4; ++rep) {
    uint4 raw[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const int s = s0 + rep * 64 + t * 16 + hw;
      raw[t] = s < N ? __ldg(reinterpret_cast<const uint4*>(KR + (size_t)s * kD)) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&raw[t]);
      float d = 0.f;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = __bfloat1622float2(p2[i]);
        d = fmaf(uf[2 * i], f.x, d);
        d = fmaf(uf[2 * i + 1], f.y, d);
      }
      d += __shfl_xor_sync(0xffffffffu, d, 1);
      d += __shfl_xor_sync(0xffffffffu, d, 2);
      d += __shfl_xor_sync(0xffffffffu, d, 4);
      d += __shfl_xor_sync(0xffffffffu, d, 8);
      const int s = s0 + rep * 64 + t * 16 + hw;
      if (hl == 0 && s < N) sc[s] = d;
    }
  }
}

cudaError_t launch_score_decode(const DevCtx& c, const DecBatch& b, int layer_begin, int layer_count, int,
                                const __nv_bfloat16* q, int span_bound, cudaStream_t s) {
  if (span_bound <= 0) span_bound = 1;
  return launch_chained(k_score_dec, dim3((span_bound + 255) / 256, c.Hkv, b.n * layer_count), dim3(256), 0, s, c,
                        layer_begin, b, layer_count, q);
}

// ------------------------------------------------------------------------------------------
// a4 top-k (Eq. 8 with unit = span): the min(k, N_s) largest scores, ties -> lower span id.  4-pass radix select on
// order-preserving keys, then an id-ordered pick of the threshold ties.  Writes the ascending id list and the token
// ranges the attention kernels walk (adjacent spans merged).  One CTA per (unit, KV head).
// Union of this step's selection (s_ids[0..cnt), ascending) with the selection the last prefill call left in
// persist_sel (ascending, -1 padded): the persistent mechanism of Sec. 3.5.  Writes the ascending, duplicate-free id
// list to s_all and returns its length.  Called by every thread of the CTA; s_tmp has room for kMaxTopK ints.
__device__ __forceinline__ int union_with_persistent(const DevCtx& c, size_t unit, int g, const int* s_ids, int cnt,
                                                     int* s_tmp, int* s_all, int* s_nall) {
  const int tid = threadIdx.x;
  if (tid < c.topk) s_tmp[tid] = c.persist ? c.persist_sel[(unit * c.Hkv + g) * (size_t)c.topk + tid] : -1;
  __syncthreads();
  if (tid == 0) {
    int a = 0, b = 0, n = 0;
    while (b < c.topk && s_tmp[b] < 0) ++b;  // (-1 padding sits at the end, but tolerate it anywhere)
    while (a < cnt || b < c.topk) {
      const int va = a < cnt ? s_ids[a] : 0x7fffffff;
      const int vb = b < c.topk && s_tmp[b] >= 0 ? s_tmp[b] : 0x7fffffff;
      if (va == 0x7fffffff && vb == 0x7fffffff) break;
      const int v = va < vb ? va : vb;
      s_all[n++] = v;
      if (va == v) ++a;
      if (vb == v) {
        ++b;
        while (b < c.topk && s_tmp[b] < 0) ++b;
      }
    }
    *s_nall = n;
  }
  __syncthreads();
  return *s_nall;
}

__device__ __forceinline__ unsigned order_key(float f) {
  const unsigned u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Radix select of the K largest keys among KEY(0..N) (ties: lower index first), one 8-bit digit per pass from the top.
// Writes the chosen indices, unordered, to s_ids and their number to *s_cnt (which the caller has zeroed).  Called by
// every thread of the CTA; K < N.  R > 0 (keys that are expensive to read, 32-bit): up to R keys per thread are read
// once and kept in registers (thread t holds keys t, t + nt, ...); with more keys than that, or R = 0, every pass
// reads them through KEY.
constexpr int kSelCand = 256;  // keys the short cut of radix_select_top ranks against each other

template <typename KT, int R, typename KeyF>
__device__ __forceinline__ void radix_select_top(KeyF&& KEY, int N, int K, unsigned* hist, KT* s_prefix,
                                                 unsigned* s_need, int* s_scan, int* s_cnt, int* s_ids,
                                                 unsigned* s_ckey = nullptr) {
  static_assert(R == 0 || sizeof(KT) == 4, "register copies are kept of 32-bit keys only");
  const int tid = threadIdx.x, nt = blockDim.x;
  constexpr int kPasses = (int)sizeof(KT);
  const bool inreg = R > 0 && N <= R * nt;
  unsigned kr[R > 0 ? R : 1];
  if (inreg) {
#pragma unroll
    for (int i = 0; i < R; ++i) {
      const int s = tid + i * nt;
      kr[i] = s < N ? (unsigned)KEY(s) : 0u;
    }
  }
  // f(index, key) for every key of this thread
  auto for_each_key = [&](auto&& f) {
    if (inreg) {
#pragma unroll
      for (int i = 0; i < R; ++i) {
        const int s = tid + i * nt;
        if (s < N) f(s, (KT)kr[i]);
      }
    } else {
      // eight keys in flight per thread (KEY may be a load from global memory)
      for (int base = tid; base < N; base += 8 * nt) {
        KT k8[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int s = base + u * nt;
          k8[u] = s < N ? (KT)KEY(s) : (KT)0;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int s = base + u * nt;
          if (s < N) f(s, k8[u]);
        }
      }
    }
  };
  if (sizeof(KT) == 4 && s_ckey != nullptr && nt >= 64 + kSelCand) {
    // Short cut for 32-bit keys (K is small against N): with the block's largest key M known, one histogram
    // of how far a key's upper 16 bits lie below M's (256 bins; further away: the last bin) gives the smallest
    // distance b within which at least K keys lie; those keys -- usually a few more than K -- are listed in shared
    // memory and ranked against each other (key, then lower index).  Four barriers instead of twelve and about a
    // third of the instructions of the four radix passes.  The radix passes below remain for the cases this does not
    // cover: the K-th key more than 255 bins below M, or more than kSelCand keys within b (many equal keys).
    int* s_cid = s_scan + 64;  // (s_scan[32..34]: scratch words)
    const int lane = tid & 31, wid = tid >> 5, nw = nt >> 5;
    unsigned m = 0;
    for_each_key([&](int, KT key) { m = max(m, (unsigned)key); });
    m = __reduce_max_sync(0xffffffffu, m);
    if (lane == 0) s_scan[wid] = (int)m;
    if (tid < 256) hist[tid] = 0;
    if (tid == 0) s_scan[34] = 0;
    __syncthreads();
    m = __reduce_max_sync(0xffffffffu, (unsigned)s_scan[lane < nw ? lane : 0]);
    const unsigned M16 = m >> 16;
    DigitRuns dr;
    for_each_key([&](int, KT key) { dr.add(hist, (int)min(M16 - ((unsigned)key >> 16), 255u)); });
    dr.flush(hist);
    __syncthreads();
    if (tid < 32) {
      long long rank = K - 1;  // (0-based from the top = from bin 0)
      const unsigned b = pick_from_bottom(hist, 256, rank);
      if (tid == 0) s_scan[33] = (int)b;
    }
    __syncthreads();
    const unsigned bcut = (unsigned)s_scan[33];
    if (bcut < 255u) {
      for_each_key([&](int s, KT key) {
        if (M16 - ((unsigned)key >> 16) <= bcut) {
          const int j = atomicAdd(&s_scan[34], 1);
          if (j < kSelCand) {
            s_ckey[j] = (unsigned)key;
            s_cid[j] = s;
          }
        }
      });
      __syncthreads();
      const int nc = s_scan[34];
      if (nc <= kSelCand) {
        for (int j = tid; j < nc; j += nt) {
          const unsigned key = s_ckey[j];
          const int id = s_cid[j];
          int rank = 0;
          for (int i = 0; i < nc; ++i) rank += (s_ckey[i] > key) || (s_ckey[i] == key && s_cid[i] < id);
          if (rank < K) {
            const int slot = atomicAdd(s_cnt, 1);
            if (slot < kMaxTopK) s_ids[slot] = id;
          }
        }
        return;
      }
    }
    __syncthreads();  // (the scratch words are free again)
  }
  if (tid == 0) {
    *s_prefix = 0;
    *s_need = K;  // rank from the top, 1-based: find key T with #(key > T) < K <= #(key >= T)
  }
  for (int pass = 0; pass < kPasses; ++pass) {
    const int shift = 8 * (kPasses - 1 - pass);
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    const KT prefix = *s_prefix;
    const KT himask = pass == 0 ? (KT)0 : (KT)(~(KT)0 << (shift + 8));
    DigitRuns dr;
    for_each_key([&](int, KT key) {
      if ((key & himask) == prefix) dr.add(hist, (int)((unsigned)(key >> shift) & 255u));
    });
    dr.flush(hist);
    __syncthreads();
    if (tid < 32) {
      unsigned need = *s_need;
      const int bin = pick_from_top(hist, 256, need);
      if (tid == 0) {
        *s_need = need;
        *s_prefix = prefix | ((KT)bin << shift);
      }
    }
    __syncthreads();
  }
  const KT T = *s_prefix;
  const unsigned need_eq = *s_need;  // how many of the == T elements are taken (lowest ids first)
  // the last pass counted the keys equal to T in the bin of T's low digit (the histogram is still there)
  if (hist[(unsigned)T & 255u] == need_eq) {
    // every key equal to the threshold is taken: no order among them is needed
    for_each_key([&](int s, KT key) {
      if (key >= T) {
        const int slot = atomicAdd(s_cnt, 1);
        if (slot < kMaxTopK) s_ids[slot] = s;
      }
    });
    return;
  }
  // ties at the cut: contiguous id partition so that they are picked in id order
  const int per = (N + nt - 1) / nt;
  const int lo = min(N, tid * per), hi = min(N, lo + per);
  int eq = 0;
  for (int s = lo; s < hi; ++s) eq += KEY(s) == T;
  s_scan[tid] = eq;
  __syncthreads();
  if (tid < 32) warp0_exclusive_scan(s_scan, nt);
  __syncthreads();
  int eqrank = s_scan[tid];
  for (int s = lo; s < hi; ++s) {
    const KT key = KEY(s);
    bool take = key > T;
    if (key == T) {
      take = (unsigned)eqrank < need_eq;
      ++eqrank;
    }
    if (take) {
      const int slot = atomicAdd(s_cnt, 1);
      if (slot < kMaxTopK) s_ids[slot] = s;
    }
  }
}

// What a launch of k_topk does.  kTopkSelect: the selection, the token ranges and (prefill) the gather.  The other
// two are the collaborative voting of Sec. 3.5: kTopkBallot only records the own top-k units of every layer that has a
// retrieval head; kTopkVote then ranks a layer's units by the tally of the ballots of the layers up to it before
// their own scores and goes on like kTopkSelect.
enum { kTopkSelect = 0, kTopkBallot = 1, kTopkVote = 2 };
constexpr int kTopkSelRegs = 24;  // scores of up to 12K spans (512 threads) are read from global memory once

template <bool DECODE>
__global__ void __launch_bounds__(512) k_topk(DevCtx c, int seq, int layer_begin, DecBatch b, int layer_count,
                                              int evicted_end, int mode) {
  chain_wait();
  __shared__ unsigned hist[256];
  __shared__ unsigned s_prefix, s_need;
  __shared__ unsigned long long s_prefix64;
  __shared__ int s_ids[kMaxTopK];
  __shared__ int s_cnt;
  __shared__ int s_scan[512];
  __shared__ unsigned s_ckey[kSelCand];
  __shared__ int s_rs[kMaxRanges], s_rl[kMaxRanges], s_pre[kMaxRanges + 1], s_nr;  // merged ranges, packed-row prefix
  __shared__ int s_sst[2 * kMaxTopK], s_sln[2 * kMaxTopK];  // extents of the selected spans
  __shared__ int s_all[2 * kMaxTopK], s_nall;            // decode: this step's selection united with the persistent one
  __shared__ int s_ko[kMaxRanges];  // pager, decode: first K row of every range, counted from the start of the K slabs
  const int g = blockIdx.x;
  int layer, sq, pos = 0, loc_begin = 0;
  if (DECODE) {
    const int bi = blockIdx.y / layer_count;
    layer = layer_begin + blockIdx.y % layer_count;
    sq = b.seq[bi];
    pos = b.pos[bi];
    loc_begin = b.loc_begin[bi];
  } else {
    layer = layer_begin + blockIdx.y;
    sq = seq;
  }
  // a layer with a retrieval head (Sec. 3.5) has one selection, made from the scores of that head's KV head
  const int rh = ret_head_of(c, layer);
  if (mode == kTopkBallot && (rh < 0 || g != 0)) return;
  const size_t unit = unit_of(c, sq, layer);
  const int nspans = c.n_spans[unit];
  const float* sc = c.scores + (unit * c.Hkv + (rh >= 0 ? rh / c.G : g)) * (size_t)c.cap;
  const int tid = threadIdx.x, nt = blockDim.x;
  // What is ranked: the spans themselves, or (Eq. 8 as printed) fixed units of c.unit tokens on the absolute token
  // grid, each scored by the maximum over the spans it meets.  N = number of candidates, KEY(i) = order key of
  // candidate i.
  extern __shared__ unsigned ukey[];  // unit mode: order key of every unit that meets the indexed range [Ls, E)
  const int U = c.unit;
  int N = nspans, u0 = 0, Eend = 0;
  if (U > 0) {
    Eend = nspans > 0 ? (DECODE ? loc_begin : evicted_end) : c.Ls;  // end of the indexed range
    u0 = c.Ls / U;
    N = Eend > c.Ls ? (Eend + U - 1) / U - u0 : 0;
    for (int i = tid; i < N; i += nt) ukey[i] = 0u;  // below the key of every real score
    __syncthreads();
    for (int s = tid; s < nspans; s += nt) {
      const int st = c.span_start[unit * c.cap + s], ln = c.span_len[unit * c.cap + s];
      const unsigned key = order_key(sc[s]);
      for (int u = st / U; u <= (st + ln - 1) / U; ++u) atomicMax(&ukey[u - u0], key);
    }
    __syncthreads();
  }
  // voting: tally of every unit = summed weights of the ballots that name it, layers in ascending order (fp32)
  float* utally = reinterpret_cast<float*>(ukey + ((N + 3) & ~3));
  if (mode == kTopkVote) {
    for (int i = tid; i < N; i += nt) utally[i] = 0.f;
    __syncthreads();
    for (int l = 0; l <= layer; ++l) {
      if (ret_head_of(c, l) < 0) continue;
      const float w = c.head_w[l];
      if (tid < c.topk) {
        const int id = c.ballot[unit_of(c, sq, l) * c.topk + tid];  // distinct within a ballot
        if (id >= u0 && id - u0 < N) utally[id - u0] += w;
      }
      __syncthreads();
    }
  }
  auto KEY = [&](int i) -> unsigned { return U > 0 ? ukey[i] : order_key(sc[i]); };
  auto KEY64 = [&](int i) -> unsigned long long {
    return ((unsigned long long)order_key(utally[i]) << 32) | ukey[i];
  };
  const int K = min(c.topk, N);
  if (tid == 0) s_cnt = 0;
  __syncthreads();
  if (K == N) {
    for (int t = tid; t < K; t += nt) s_ids[t] = t;
    if (tid == 0) s_cnt = K;
  } else if (mode == kTopkVote) {
    radix_select_top<unsigned long long, 0>(KEY64, N, K, hist, &s_prefix64, &s_need, s_scan, &s_cnt, s_ids);
  } else {
    radix_select_top<unsigned, kTopkSelRegs>(KEY, N, K, hist, &s_prefix, &s_need, s_scan, &s_cnt, s_ids, s_ckey);
  }
  __syncthreads();
  const int cnt = min(s_cnt, K);
  // rank sort ascending
  int myid = -1, rank = 0;
  if (tid < cnt) {
    myid = s_ids[tid];
    for (int t = 0; t < cnt; ++t) rank += s_ids[t] < myid;
  }
  __syncthreads();
  if (tid < cnt) s_ids[rank] = myid;
  __syncthreads();
  if (U > 0 && tid < cnt) s_ids[tid] += u0;  // absolute unit ids
  __syncthreads();
  if (mode == kTopkBallot) {
    for (int t = tid; t < c.topk; t += nt) c.ballot[unit * c.topk + t] = t < cnt ? s_ids[t] : -1;
    return;
  }
  int* sel = c.sel + (unit * c.Hkv + g) * (size_t)c.topk;
  for (int t = tid; t < c.topk; t += nt) sel[t] = t < cnt ? s_ids[t] : -1;
  // token ranges of the attention kernels: the spans' extents are fetched in parallel, merged (adjacent spans become
  // one range) by one thread in shared memory and written out in parallel
  const int* ids_all = s_ids;
  int nall = cnt;
  if (DECODE && c.persist) {
    nall = union_with_persistent(c, unit, g, s_ids, cnt, s_scan, s_all, &s_nall);
    ids_all = s_all;
  }
  if (tid < nall) {
    if (U > 0) {  // the unit's tokens inside the indexed range
      const int st = max(ids_all[tid] * U, c.Ls);
      s_sst[tid] = st;
      s_sln[tid] = min((ids_all[tid] + 1) * U, Eend) - st;
    } else {
      s_sst[tid] = c.span_start[unit * c.cap + ids_all[tid]];
      s_sln[tid] = c.span_len[unit * c.cap + ids_all[tid]];
    }
  }
  __syncthreads();
  // Host-memory pager (Sec. 3.4).  The units named by this retrieval are looked up in this (sequence, layer, KV
  // head)'s unit cache; every slot's usage score decays, a unit named now gains 1; a missing unit takes the slot with
  // the lowest score among the slots not named now (lowest slot among equals) and its rows are pulled from the host
  // mirror.  A prefill call caches only whole units: the unit the indexed range ends in, while it is still growing,
  // is read from the mirror every time.  (During decode the indexed range no longer grows, so that unit is cached
  // like the others.)  s_src[t]: slot of named unit t, -1 = straight from the host.
  __shared__ int s_tag[128], s_src[2 * kMaxTopK], s_fill[2 * kMaxTopK];
  __shared__ float s_sco[128];
  __shared__ unsigned char s_named[128];
  if (c.host_kv) {
    const int CU = c.cache_units;
    const size_t cb = (unit * c.Hkv + g) * (size_t)CU;
    if (tid < CU) {
      s_tag[tid] = c.ctag[cb + tid];
      s_sco[tid] = __fmul_rn(c.cscore[cb + tid], c.score_decay);
      s_named[tid] = 0;
    }
    __syncthreads();
    if (tid == 0) {
      unsigned long long hits = 0, misses = 0;
      auto growing = [&](int id) { return !DECODE && (id + 1) * U > Eend; };
      for (int t = 0; t < nall; ++t) {  // first the units that are there, so that none of them is pushed out
        const int id = ids_all[t];
        s_src[t] = -1;
        s_fill[t] = 0;
        if (growing(id)) continue;
        for (int sl = 0; sl < CU; ++sl)
          if (s_tag[sl] == id) {
            s_src[t] = sl;
            s_named[sl] = 1;
            s_sco[sl] = __fadd_rn(s_sco[sl], 1.f);
            ++hits;
            break;
          }
      }
      for (int t = 0; t < nall; ++t) {
        const int id = ids_all[t];
        if (growing(id) || s_src[t] >= 0) continue;
        int victim = -1;
        for (int sl = 0; sl < CU; ++sl)
          if (!s_named[sl] && (victim < 0 || s_sco[sl] < s_sco[victim])) victim = sl;
        if (victim < 0) continue;  // (cannot happen: cache_units >= the units one retrieval names)
        s_tag[victim] = id;
        s_sco[victim] = 1.f;
        s_named[victim] = 1;
        s_src[t] = victim;
        s_fill[t] = 1;
        ++misses;
      }
      atomicAdd(&c.cstat[unit * 2], hits);
      atomicAdd(&c.cstat[unit * 2 + 1], misses);
    }
    __syncthreads();
    if (tid < CU) {
      c.ctag[cb + tid] = s_tag[tid];
      c.cscore[cb + tid] = s_sco[tid];
    }
    if (!DECODE) {
      // A prefill call leaves the data movement to k_pull_pack, which runs on a stream of its own while the kernels
      // of the call's other layers compute: this kernel only records what has to be brought in and from where.
      const size_t pb = (unit * c.Hkv + g) * (size_t)(2 * kMaxTopK);
      if (tid < nall) {
        c.pl_id[pb + tid] = ids_all[tid];
        c.pl_src[pb + tid] = s_src[tid] < 0 ? -1 : (s_src[tid] | (s_fill[tid] ? 0x10000 : 0));
        c.pl_start[pb + tid] = s_sst[tid];
        c.pl_len[pb + tid] = s_sln[tid];
      }
      if (tid == 0) c.pl_cnt[unit * c.Hkv + g] = nall;
    }
    if (DECODE) {
      // a decode step pulls its missing units here: the unit's valid rows [s_sst, s_sst + s_sln) go to the same row
      // offsets of its slot (the attention kernel, launched next, reads the slots in place)
      const size_t hslab = (unit * c.Hkv + g) * (size_t)c.Tpad;
      for (int t = 0; t < nall; ++t) {
        if (!s_fill[t]) continue;
        const int st = s_sst[t], ln = s_sln[t];
        const size_t drow = (cb + s_src[t]) * (size_t)U + (st - ids_all[t] * U);
        const uint4* hk = reinterpret_cast<const uint4*>(c.hostK + (hslab + st) * kD);
        const uint4* hv = reinterpret_cast<const uint4*>(c.hostV + (hslab + st) * kD);
        uint4* dk = reinterpret_cast<uint4*>(c.Kcache + drow * kD);
        uint4* dv = reinterpret_cast<uint4*>(c.Vcache + drow * kD);
        for (int i = tid; i < ln * 16; i += nt) {
          dk[i] = hk[i];
          dv[i] = hv[i];
        }
      }
    }
  }
  if (!(DECODE && c.host_kv)) {
    // (ranges in place, adjacent spans merged: one warp)
    if (tid < 32) {
      const int first = DECODE ? 1 : 0;  // decode: the sink in front of the spans, the recent tokens behind them
      const int rbeg = DECODE ? min(loc_begin, pos + 1) : 0;
      const int nr = merge_ranges_warp(
          nall + 2 * first,
          [&](int i, int& st, int& ln) {
            if (i < first) {
              st = 0;
              ln = min(c.Ls, pos + 1);
            } else if (i - first < nall) {
              st = s_sst[i - first];
              ln = s_sln[i - first];
            } else {
              st = rbeg;
              ln = pos + 1 - rbeg;
            }
          },
          s_rs, s_rl);
      long long tokens = 0;
      for (int t = tid; t < nall; t += 32) tokens += s_sln[t];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) tokens += shfl_xor_ll(tokens, o);
      // packed-row prefix of the ranges
      int run = 0;
      for (int base = 0; base < nr; base += 32) {
        const int i = base + tid;
        const int v = i < nr ? s_rl[i] : 0;
        int inc = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int t = __shfl_up_sync(0xffffffffu, inc, o);
          if (tid >= o) inc += t;
        }
        if (i < nr) s_pre[i] = run + inc - v;
        run += __shfl_sync(0xffffffffu, inc, 31);
      }
      if (tid == 0) {
        s_pre[nr] = run;
        s_nr = nr;
        c.rng_cnt[unit * c.Hkv + g] = nr;
        c.sel_tokens[unit * c.Hkv + g] = tokens;  // (summed over the KV heads by ltri_get_stats)
        if (!DECODE) c.gcnt[(size_t)layer * c.Hkv + g] = run;
      }
    }
  } else
  if (tid == 0) {
    int nr = 0;
    long long tokens = 0;
    // under the pager a decode step reads every named unit from its cache slot, so the units stay ranges of their own
    // and every range carries the K row it starts at, counted from the start of the K slabs (the V row follows from it)
    const bool paged = DECODE && c.host_kv;
    const long long slab0 = (long long)((unit * c.Hkv + g) * (size_t)c.SR);
    auto push = [&](int st, int ln, int slot) {
      if (ln <= 0) return;
      if (!paged && nr > 0 && s_rs[nr - 1] + s_rl[nr - 1] >= st)  // adjacent, or (NMS with phi > 0) overlapping
        s_rl[nr - 1] = max(s_rl[nr - 1], st + ln - s_rs[nr - 1]);
      else {
        s_rs[nr] = st;
        s_rl[nr] = ln;
        if (paged) {
          if (slot >= 0) {
            const long long crow =
                (long long)(((unit * c.Hkv + g) * (size_t)c.cache_units + slot) * (size_t)U) + (st - (st / U) * U);
            s_ko[nr] = (int)((long long)((c.Kcache - c.Kc) / kD) + crow);
          } else {
            s_ko[nr] = (int)(slab0 + slab_row(c, st, DECODE ? b.shift[blockIdx.y / layer_count] : 0));
          }
        }
        ++nr;
      }
    };
    if (DECODE) push(0, min(c.Ls, pos + 1), -1);
    for (int t = 0; t < nall; ++t) {
      tokens += s_sln[t];
      push(s_sst[t], s_sln[t], paged ? s_src[t] : -1);
    }
    if (DECODE) push(min(loc_begin, pos + 1), pos + 1 - min(loc_begin, pos + 1), -1);
    int run = 0;
    for (int i = 0; i < nr; ++i) {
      s_pre[i] = run;
      run += s_rl[i];
    }
    s_pre[nr] = run;
    s_nr = nr;
    c.rng_cnt[unit * c.Hkv + g] = nr;
    c.sel_tokens[unit * c.Hkv + g] = tokens;  // (summed over the KV heads by ltri_get_stats)
    if (!DECODE) c.gcnt[(size_t)layer * c.Hkv + g] = run;
  }
  __syncthreads();
  {
    const size_t rb = (unit * c.Hkv + g) * (size_t)c.rcap;
    for (int t = tid; t < s_nr; t += nt) {
      c.rng_start[rb + t] = s_rs[t];
      c.rng_len[rb + t] = s_rl[t];
      if (DECODE && c.host_kv) c.rng_koff[rb + t] = s_ko[t];
    }
  }
  if (!DECODE && c.host_kv) {
    // (a5 gather from the unit cache / the host mirror: k_pull_pack)
  } else if (!DECODE) {
    // a5 gather: pack the K and V rows of the selected spans into one contiguous slab per (layer, KV head), so the
    // attention kernel that continues over them reads whole 128-row tiles.  16 threads per 256-byte row, four rows
    // of K and of V in flight per thread; the rows up to the next multiple of 8 are zero-filled.
    const int nr = s_nr, R = s_pre[nr], Rz = (R + 7) & ~7;
    const size_t slab = (unit * c.Hkv + g) * (size_t)c.SR;  // (resident contexts only: row = token)
    const uint4* Ksrc = reinterpret_cast<const uint4*>(c.Kc + slab * kD);
    const uint4* Vsrc = reinterpret_cast<const uint4*>(c.Vc + slab * kD);
    const size_t gslab = ((size_t)layer * c.Hkv + g) * (size_t)c.Rcap;
    uint4* Kdst = reinterpret_cast<uint4*>(c.Kg + gslab * kD);
    uint4* Vdst = reinterpret_cast<uint4*>(c.Vg + gslab * kD);
    const int ch = tid & 15, rpp = nt >> 4;  // 16-byte chunk of the row, rows per pass
    for (int r0 = tid >> 4; r0 < Rz; r0 += 4 * rpp) {
      uint4 kv[4], vv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int r = r0 + i * rpp;
        kv[i] = vv[i] = make_uint4(0u, 0u, 0u, 0u);
        if (r < R) {
          int lo = 0, hi = nr - 1;  // last range whose first packed row is <= r
          while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (s_pre[mid] <= r) lo = mid; else hi = mid - 1;
          }
          const size_t tok = (size_t)(s_rs[lo] + (r - s_pre[lo]));
          kv[i] = __ldg(Ksrc + tok * 16 + ch);
          vv[i] = __ldg(Vsrc + tok * 16 + ch);
        }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int r = r0 + i * rpp;
        if (r < Rz) {
          Kdst[(size_t)r * 16 + ch] = kv[i];
          Vdst[(size_t)r * 16 + ch] = vv[i];
        }
      }
    }
  }
}

// Host-memory pager (Sec. 3.4), data movement of a prefill call.  A task = one (named unit, KV head, layer): bring
// the unit's rows to the slab the retrieved attention reads (a5 gather) -- from its cache slot, or over the bus from
// the host mirror, in which case the rows also go into the slot the top-k kernel chose for the unit (unless the unit
// is the one the indexed range ends in and still grows: that one is never cached).  A few small persistent CTAs
// (128 threads, few registers, no dynamic shared memory) walk the tasks: small and few on purpose, so that each fits
// onto an SM beside the one large CTA of the attention and map kernels and the bus transfer really runs under the
// computation of the call's other layers instead of taking SMs away from it.  Eight 16-byte loads per thread are in
// flight on the bus at a time, which keeps the bus busy with far fewer threads than the GPU has.
constexpr int kPullThreads = 128;
constexpr int kPullCtas = 32;

__global__ void __launch_bounds__(kPullThreads) k_pull_pack(DevCtx c, int seq, int layer_begin, int layer_count, int max_units) {
  __shared__ int s_off;
  const int tid = threadIdx.x;
  const int ntasks = max_units * c.Hkv * layer_count;
  for (int task = blockIdx.x; task < ntasks; task += gridDim.x) {
  const int t = task % max_units, g = (task / max_units) % c.Hkv, layer = layer_begin + task / (max_units * c.Hkv);
  const size_t unit = unit_of(c, seq, layer);
  const int nall = min(c.pl_cnt[unit * c.Hkv + g], 2 * kMaxTopK);
  if (t >= nall) continue;
  __syncthreads();  // (s_off of the previous task has been read by everyone)
  const size_t pb = (unit * c.Hkv + g) * (size_t)(2 * kMaxTopK);
  // first packed row of this unit: the units are packed in ascending order, every token once
  if (tid < 32) {
    int part = 0;
    for (int i = tid; i < t; i += 32) part += c.pl_len[pb + i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    if (tid == 0) s_off = part;
  }
  __syncthreads();
  const int U = c.unit;
  const int id = c.pl_id[pb + t], src = c.pl_src[pb + t], st = c.pl_start[pb + t], ln = c.pl_len[pb + t];
  const size_t gslab = ((size_t)layer * c.Hkv + g) * (size_t)c.Rcap + s_off;
  uint4* Kdst = reinterpret_cast<uint4*>(c.Kg + gslab * kD);
  uint4* Vdst = reinterpret_cast<uint4*>(c.Vg + gslab * kD);
  const uint4 *Ksrc, *Vsrc;
  uint4 *Kslot = nullptr, *Vslot = nullptr;
  const size_t hslab = (unit * c.Hkv + g) * (size_t)c.Tpad;
  if (src >= 0) {
    const size_t row = ((unit * c.Hkv + g) * (size_t)c.cache_units + (src & 0xffff)) * (size_t)U + (st - id * U);
    Ksrc = reinterpret_cast<const uint4*>(c.Kcache + row * kD);
    Vsrc = reinterpret_cast<const uint4*>(c.Vcache + row * kD);
    if (src & 0x10000) {  // not there yet: over the bus, and into the slot as well
      Kslot = reinterpret_cast<uint4*>(c.Kcache + row * kD);
      Vslot = reinterpret_cast<uint4*>(c.Vcache + row * kD);
      Ksrc = reinterpret_cast<const uint4*>(c.hostK + (hslab + st) * kD);
      Vsrc = reinterpret_cast<const uint4*>(c.hostV + (hslab + st) * kD);
    }
  } else {
    Ksrc = reinterpret_cast<const uint4*>(c.hostK + (hslab + st) * kD);
    Vsrc = reinterpret_cast<const uint4*>(c.hostV + (hslab + st) * kD);
  }
  const int n16 = ln * 16;
  for (int i0 = tid; i0 < n16; i0 += 4 * kPullThreads) {
    uint4 kv[4], vv[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = i0 + u * kPullThreads;
      if (i < n16) {
        kv[u] = Ksrc[i];
        vv[u] = Vsrc[i];
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = i0 + u * kPullThreads;
      if (i < n16) {
        Kdst[i] = kv[u];
        Vdst[i] = vv[u];
        if (Kslot) {
          Kslot[i] = kv[u];
          Vslot[i] = vv[u];
        }
      }
    }
  }
  if (t == nall - 1) {
    // the packed rows up to the next multiple of eight are zero (tile pieces are eight rows high)
    const int R = s_off + ln, pad = ((R + 7) & ~7) - R;
    for (int i = tid; i < pad * 16; i += kPullThreads) {
      Kdst[n16 + i] = make_uint4(0u, 0u, 0u, 0u);
      Vdst[n16 + i] = make_uint4(0u, 0u, 0u, 0u);
    }
  }
  }  // task
}

cudaError_t launch_pull_pack(const DevCtx& c, const PrefillArgs& a, cudaStream_t s) {
  k_pull_pack<<<kPullCtas, kPullThreads, 0, s>>>(c, a.seq, a.layer_begin, a.layer_count, c.topk);
  return cudaGetLastError();
}

// Decode retrieval in one launch: a CTA owns one (sequence, layer, KV head), streams that head's index once
// (half-warp per 256-byte row, 16 bytes per lane, four rows in flight), keeps the scores in shared memory, selects the
// top-k there (same radix select as k_topk) and writes the selection and the token ranges of the attention kernel.
// Token ranges of the attention kernels from M items (start, length) in ascending order of start: items of length
// zero are dropped, an item that starts at or before the end of what came before it (adjacent spans, or overlapping
// ones under NMS with phi > 0) extends the current range.  One warp, 32 items per round: an item opens a range iff it
// starts beyond the largest end seen so far (a prefix maximum), its range number is the count of such items up to
// it, and a range's end is the prefix maximum in front of the next opener.  Returns the number of ranges; s_rs / s_rl
// receive their starts and lengths.  Called by all 32 lanes of one warp.
template <typename ItemF>
__device__ __forceinline__ int merge_ranges_warp(int M, ItemF&& item, int* s_rs, int* s_rl) {
  const int lane = threadIdx.x & 31;
  constexpr int kNone = -0x7fffffff;
  int far = kNone, nr = 0;  // largest end so far, ranges so far
  for (int base = 0; base < M; base += 32) {
    const int i = base + lane;
    int st = 0, ln = 0;
    if (i < M) item(i, st, ln);
    const bool valid = i < M && ln > 0;
    const int en = valid ? st + ln : kNone;
    int inc = en;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc = max(inc, t);
    }
    int before = __shfl_up_sync(0xffffffffu, inc, 1);
    if (lane == 0) before = kNone;
    before = max(before, far);
    const bool opens = valid && st > before;
    const unsigned ob = __ballot_sync(0xffffffffu, opens);
    if (opens) {
      const int idx = nr + __popc(ob & ((2u << lane) - 1u)) - 1;
      s_rs[idx] = st;
      if (idx > 0) s_rl[idx - 1] = before;  // (the end of the range before it; turned into a length below)
    }
    far = max(far, __shfl_sync(0xffffffffu, inc, 31));
    nr += __popc(ob);
  }
  if (lane == 0 && nr > 0) s_rl[nr - 1] = far;
  __syncwarp();
  for (int r = lane; r < nr; r += 32) s_rl[r] -= s_rs[r];
  __syncwarp();
  return nr;
}

constexpr int kFusedMaxSpans = 12288;  // scores kept in shared memory (48 KB)
constexpr int kDecSelRegs = 16;        // keys per thread the select holds in registers (8K spans at 512 threads)

// a0 inside the one-launch decode retrieval: the CTA of (sequence, layer, KV head) also stores that head's new K and V
// row (threads 0-31: sixteen 16-byte pieces each), so a decode step needs no separate append launch.  The attention
// kernel, launched next, is the first reader of the row.  (Resident contexts only: the one-launch path is never paged.)
__device__ __forceinline__ void append_decode_row(const DevCtx& c, const DecBatch& b, int bi, int l, int layer_count,
                                                  size_t unit, int g, const __nv_bfloat16* __restrict__ k,
                                                  const __nv_bfloat16* __restrict__ v) {
  const int tid = threadIdx.x;
  if (tid < 32) {
    const int c16 = tid & 15;
    const __nv_bfloat16* src = (tid < 16 ? k : v) + (((size_t)b.src[bi] * layer_count + l) * c.Hkv + g) * kD + c16 * 8;
    __nv_bfloat16* dst = (tid < 16 ? c.Kc : c.Vc) + ((unit * c.Hkv + g) * (size_t)c.SR + b.pos[bi]) * kD + c16 * 8;
    *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
    if (g == 0 && tid == 0) c.votes[unit * c.Tpad + b.pos[bi]] = 0;
  }
}

__global__ void __launch_bounds__(1024) k_dec_retrieve(DevCtx c, int layer_begin, DecBatch b, int layer_count,
                                                       const __nv_bfloat16* __restrict__ q,
                                                       const __nv_bfloat16* __restrict__ knew,
                                                       const __nv_bfloat16* __restrict__ vnew) {
  chain_wait();
  extern __shared__ unsigned sck[];  // [N] order-preserving keys of the scores
  __shared__ float su[kD];
  __shared__ unsigned hist[256];
  __shared__ unsigned s_prefix, s_need;
  __shared__ int s_ids[kMaxTopK];
  __shared__ int s_cnt;
  __shared__ int s_scan[1024];
  __shared__ unsigned s_ckey[kSelCand];
  __shared__ int s_rs[kMaxRanges], s_rl[kMaxRanges], s_nr, s_sst[2 * kMaxTopK], s_sln[2 * kMaxTopK];
  __shared__ int s_all[2 * kMaxTopK], s_nall;
  const int g = blockIdx.x;
  const int bi = blockIdx.y / layer_count, l = blockIdx.y % layer_count, layer = layer_begin + l;
  const int sq = b.seq[bi], pos = b.pos[bi], loc_begin = b.loc_begin[bi];
  const size_t unit = unit_of(c, sq, layer);
  const int tid = threadIdx.x, nt = blockDim.x;
  const int N = min(c.n_spans[unit], kFusedMaxSpans);
  const int rh = ret_head_of(c, layer), gk = rh >= 0 ? rh / c.G : g;  // retrieval head of the layer (Sec. 3.5)
  append_decode_row(c, b, bi, l, layer_count, unit, g, knew, vnew);
  // ---- scores.  The first four index rows of every half-warp are requested before the query sum below is formed,
  // so that their latency and that of the query loads pass together.
  const int hw = tid >> 4, hl = tid & 15, nhw = nt >> 4;  // half-warps of the CTA (the launch picks its size)
  const __nv_bfloat16* KR = c.KR + (unit * c.Hkv + gk) * (size_t)c.cap * kD + hl * 8;
  // software pipeline: the next four rows are in flight while the current four are reduced
  auto fetch = [&](int base, uint4 (&raw)[4]) {
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const int s = base + t * nhw + hw;
      raw[t] = s < N ? __ldg(reinterpret_cast<const uint4*>(KR + (size_t)s * kD)) : make_uint4(0, 0, 0, 0);
    }
  };
  uint4 cur[4], nxt[4];
  fetch(0, cur);
  if (tid < kD) {
    const __nv_bfloat16* qp = q + (((size_t)b.src[bi] * layer_count + l) * c.Hq + gk * c.G) * kD + tid;
    float acc = 0.f;
    for (int hh = 0; hh < c.G; ++hh)
      if (rh < 0 || gk * c.G + hh == rh) acc += __bfloat162float(qp[(size_t)hh * kD]);
    su[tid] = acc;
  }
  if (tid == 0) s_cnt = 0;
  __syncthreads();
  {
    float uf[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) uf[e] = su[hl * 8 + e];
    for (int base = 0; base < N; base += nhw * 4) {  // uniform trip count (shuffles inside)
      fetch(base + nhw * 4, nxt);                    // past the end: zeros, no loads
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&cur[t]);
        float d = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 f = __bfloat1622float2(p2[i]);
          d = fmaf(uf[2 * i], f.x, d);
          d = fmaf(uf[2 * i + 1], f.y, d);
        }
        d += __shfl_xor_sync(0xffffffffu, d, 1);
        d += __shfl_xor_sync(0xffffffffu, d, 2);
        d += __shfl_xor_sync(0xffffffffu, d, 4);
        d += __shfl_xor_sync(0xffffffffu, d, 8);
        const int s = base + t * nhw + hw;
        if (hl == 0 && s < N) sck[s] = order_key(d);
      }
#pragma unroll
      for (int t = 0; t < 4; ++t) cur[t] = nxt[t];
    }
  }
  __syncthreads();
  // ---- top-k over the shared-memory scores
  const int K = min(c.topk, N);
  if (K == N) {
    for (int t = tid; t < K; t += nt) s_ids[t] = t;
    if (tid == 0) s_cnt = K;
  } else {
    radix_select_top<unsigned, kDecSelRegs>([&](int i) { return sck[i]; }, N, K, hist, &s_prefix, &s_need, s_scan,
                                            &s_cnt, s_ids, s_ckey);
  }
  __syncthreads();
  const int cnt = min(s_cnt, K);
  int myid = -1, rank = 0;
  if (tid < cnt) {
    myid = s_ids[tid];
    for (int t = 0; t < cnt; ++t) rank += s_ids[t] < myid;
  }
  __syncthreads();
  if (tid < cnt) s_ids[rank] = myid;
  __syncthreads();
  int* sel = c.sel + (unit * c.Hkv + g) * (size_t)c.topk;
  for (int t = tid; t < c.topk; t += nt) sel[t] = t < cnt ? s_ids[t] : -1;
  const int* ids_all = s_ids;
  int nall = cnt;
  if (c.persist) {
    nall = union_with_persistent(c, unit, g, s_ids, cnt, s_scan, s_all, &s_nall);
    ids_all = s_all;
  }
  if (tid < nall) {
    s_sst[tid] = c.span_start[unit * c.cap + ids_all[tid]];
    s_sln[tid] = c.span_len[unit * c.cap + ids_all[tid]];
  }
  __syncthreads();
  if (tid < 32) {
    // items: the sink, the selected spans, the recent tokens
    const int rb = min(loc_begin, pos + 1);
    const int nr = merge_ranges_warp(
        nall + 2,
        [&](int i, int& st, int& ln) {
          if (i == 0) {
            st = 0;
            ln = min(c.Ls, pos + 1);
          } else if (i <= nall) {
            st = s_sst[i - 1];
            ln = s_sln[i - 1];
          } else {
            st = rb;
            ln = pos + 1 - rb;
          }
        },
        s_rs, s_rl);
    long long tokens = 0;
    for (int t = tid; t < nall; t += 32) tokens += s_sln[t];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) tokens += shfl_xor_ll(tokens, o);
    if (tid == 0) {
      s_nr = nr;
      c.rng_cnt[unit * c.Hkv + g] = nr;
      c.sel_tokens[unit * c.Hkv + g] = tokens;  // (summed over the KV heads by ltri_get_stats)
    }
  }
  __syncthreads();
  const size_t rbb = (unit * c.Hkv + g) * (size_t)c.rcap;
  for (int t = tid; t < s_nr; t += nt) {
    c.rng_start[rbb + t] = s_rs[t];
    c.rng_len[rbb + t] = s_rl[t];
  }
}

// Decode retrieval in one launch for an index too large for one CTA's shared memory (up to 98K spans, the 1M-token
// workload): a thread-block cluster of eight CTAs owns one (sequence, layer, KV head).  Each
// CTA streams its eighth of that head's index once (half-warp per 256-byte row, 16 bytes per lane, four rows in
// flight, the next four prefetched) and keeps its scores in shared memory; the cluster then selects the top-k with
// the radix select of k_topk, every CTA counting its own scores and all of them adding the eight histograms up
// through distributed shared memory; the selected ids meet in the first CTA, which writes the selection and the
// token ranges of the attention kernel.
constexpr int kRetCluster = 8;
constexpr int kRetThreads = 512;
constexpr int kRetSliceMax = 12288;  // scores a CTA keeps in shared memory (48 KB)

__global__ void __cluster_dims__(kRetCluster, 1, 1) __launch_bounds__(kRetThreads)
    k_dec_retrieve_cl(DevCtx c, int layer_begin, DecBatch b, int layer_count, const __nv_bfloat16* __restrict__ q,
                      const __nv_bfloat16* __restrict__ knew, const __nv_bfloat16* __restrict__ vnew) {
  chain_wait();
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  extern __shared__ float ssc[];  // this CTA's slice of the scores
  __shared__ float su[kD];
  __shared__ unsigned hist[256];  // this CTA's histogram (read by the whole cluster)
  __shared__ unsigned tot[256];   // the cluster's histogram (every CTA builds its own copy)
  __shared__ unsigned s_prefix, s_need;
  __shared__ int s_eq, s_take;    // this CTA's count of scores equal to the threshold / of selected scores
  __shared__ int s_ids[kMaxTopK]; // first CTA: all selected ids, ascending
  __shared__ int s_loc[kMaxTopK]; // this CTA's selected ids
  __shared__ int s_scan[kRetThreads];
  __shared__ int s_rs[kMaxRanges], s_rl[kMaxRanges], s_nr, s_sst[2 * kMaxTopK], s_sln[2 * kMaxTopK];
  __shared__ int s_all[2 * kMaxTopK], s_nall;
  const int rank = (int)cluster.block_rank();
  const int g = blockIdx.x / kRetCluster;
  const int bi = blockIdx.y / layer_count, l = blockIdx.y % layer_count, layer = layer_begin + l;
  const int sq = b.seq[bi], pos = b.pos[bi], loc_begin = b.loc_begin[bi];
  const size_t unit = unit_of(c, sq, layer);
  const int tid = threadIdx.x, nt = blockDim.x;
  const int N = min(c.n_spans[unit], kRetCluster * kRetSliceMax);
  const int per = (N + kRetCluster - 1) / kRetCluster;
  const int lo = min(N, rank * per), hi = min(N, lo + per), nloc = hi - lo;  // this CTA's spans [lo, hi)
  const int rh = ret_head_of(c, layer), gk = rh >= 0 ? rh / c.G : g;  // retrieval head of the layer (Sec. 3.5)
  if (rank == 0) append_decode_row(c, b, bi, l, layer_count, unit, g, knew, vnew);
  if (tid < kD) {
    const __nv_bfloat16* qp = q + (((size_t)b.src[bi] * layer_count + l) * c.Hq + gk * c.G) * kD + tid;
    float acc = 0.f;
    for (int hh = 0; hh < c.G; ++hh)
      if (rh < 0 || gk * c.G + hh == rh) acc += __bfloat162float(qp[(size_t)hh * kD]);
    su[tid] = acc;
  }
  __syncthreads();
  // ---- scores of the slice
  {
    constexpr int HW = kRetThreads / 16;  // half-warps
    const int hw = tid >> 4, hl = tid & 15;
    float uf[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) uf[e] = su[hl * 8 + e];
    const __nv_bfloat16* KR = c.KR + ((unit * c.Hkv + gk) * (size_t)c.cap + lo) * kD + hl * 8;
    auto fetch = [&](int base, uint4 (&raw)[4]) {
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const int s = base + t * HW + hw;
        raw[t] = s < nloc ? __ldg(reinterpret_cast<const uint4*>(KR + (size_t)s * kD)) : make_uint4(0, 0, 0, 0);
      }
    };
    uint4 cur[4], nxt[4];
    fetch(0, cur);
    for (int base = 0; base < nloc; base += HW * 4) {  // uniform trip count (shuffles inside)
      fetch(base + HW * 4, nxt);                       // past the end: zeros, no loads
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&cur[t]);
        float d = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 f = __bfloat1622float2(p2[i]);
          d = fmaf(uf[2 * i], f.x, d);
          d = fmaf(uf[2 * i + 1], f.y, d);
        }
        d += __shfl_xor_sync(0xffffffffu, d, 1);
        d += __shfl_xor_sync(0xffffffffu, d, 2);
        d += __shfl_xor_sync(0xffffffffu, d, 4);
        d += __shfl_xor_sync(0xffffffffu, d, 8);
        const int s = base + t * HW + hw;
        if (hl == 0 && s < nloc) ssc[s] = d;
      }
#pragma unroll
      for (int t = 0; t < 4; ++t) cur[t] = nxt[t];
    }
  }
  __syncthreads();
  // ---- top-k over the cluster's scores
  const int K = min(c.topk, N);
  if (tid == 0) s_take = 0;
  __syncthreads();
  if (K == N) {
    for (int t = tid; t < nloc; t += nt) s_loc[t] = lo + t;  // (N <= top_k <= 64)
    if (tid == 0) s_take = nloc;
  } else {
    if (tid == 0) {
      s_prefix = 0;
      s_need = K;  // rank from the top, 1-based: find key T with #(key > T) < K <= #(key >= T)
    }
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      if (tid < 256) hist[tid] = 0;
      __syncthreads();
      const unsigned prefix = s_prefix;
      const unsigned himask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
      DigitRuns dr;
      for (int s = tid; s < nloc; s += nt) {
        const unsigned key = order_key(ssc[s]);
        if ((key & himask) == prefix) dr.add(hist, (int)((key >> shift) & 255u));
      }
      dr.flush(hist);
      cluster.sync();
      if (tid < 256) {
        unsigned sum = 0;
        for (int r = 0; r < kRetCluster; ++r) sum += cluster.map_shared_rank(hist, r)[tid];
        tot[tid] = sum;
      }
      cluster.sync();  // every CTA has read every histogram: they may be reset
      if (tid < 32) {
        unsigned need = s_need;
        const int bin = pick_from_top(tot, 256, need);
        if (tid == 0) {
          s_need = need;
          s_prefix = prefix | ((unsigned)bin << shift);
        }
      }
      __syncthreads();
    }
    const unsigned T = s_prefix;
    const unsigned need_eq = s_need;  // how many of the == T elements are taken (lowest ids first, cluster-wide)
    if (tot[T & 255u] == need_eq) {
      // (the last pass counted the cluster's keys equal to T; every CTA holds the same tot) every key at the
      // threshold is taken: no order among them is needed, and no exchange of counts
      for (int s = tid; s < nloc; s += nt)
        if (order_key(ssc[s]) >= T) {
          const int slot = atomicAdd(&s_take, 1);
          if (slot < kMaxTopK) s_loc[slot] = lo + s;
        }
    } else {
    // contiguous id partition so that ties are picked in id order: inside the CTA by thread, across CTAs by rank
    const int pt = (nloc + nt - 1) / nt;
    const int tlo = min(nloc, tid * pt), thi = min(nloc, tlo + pt);
    int eq = 0;
    for (int s = tlo; s < thi; ++s) eq += order_key(ssc[s]) == T;
    s_scan[tid] = eq;
    __syncthreads();
    if (tid < 32) {
      const int run = warp0_exclusive_scan(s_scan, nt);
      if (tid == 0) s_eq = run;
    }
    cluster.sync();
    int eqrank = s_scan[tid];
    for (int r = 0; r < rank; ++r) eqrank += *cluster.map_shared_rank(&s_eq, r);
    for (int s = tlo; s < thi; ++s) {
      const unsigned key = order_key(ssc[s]);
      bool take = key > T;
      if (key == T) {
        take = (unsigned)eqrank < need_eq;
        ++eqrank;
      }
      if (take) {
        const int slot = atomicAdd(&s_take, 1);
        if (slot < kMaxTopK) s_loc[slot] = lo + s;
      }
    }
    }
  }
  __syncthreads();
  // this CTA's ids in ascending order (rank sort), then into the first CTA's list behind those of the lower ranks
  const int ntake = min(s_take, kMaxTopK);
  int myid = -1, myrank = 0;
  if (tid < ntake) {
    myid = s_loc[tid];
    for (int t = 0; t < ntake; ++t) myrank += s_loc[t] < myid;
  }
  cluster.sync();  // every CTA's s_take is final
  int offset = 0, total = 0;
  for (int r = 0; r < kRetCluster; ++r) {
    const int v = min(*cluster.map_shared_rank(&s_take, r), kMaxTopK);
    if (r < rank) offset += v;
    total += v;
  }
  if (tid < ntake && offset + myrank < kMaxTopK) cluster.map_shared_rank(s_ids, 0)[offset + myrank] = myid;
  cluster.sync();  // the list is complete; the other CTAs' shared memory is not read after this point
  if (rank != 0) return;
  const int cnt = min(total, K);
  int* sel = c.sel + (unit * c.Hkv + g) * (size_t)c.topk;
  for (int t = tid; t < c.topk; t += nt) sel[t] = t < cnt ? s_ids[t] : -1;
  const int* ids_all = s_ids;
  int nall = cnt;
  if (c.persist) {
    nall = union_with_persistent(c, unit, g, s_ids, cnt, s_scan, s_all, &s_nall);
    ids_all = s_all;
  }
  if (tid < nall) {
    s_sst[tid] = c.span_start[unit * c.cap + ids_all[tid]];
    s_sln[tid] = c.span_len[unit * c.cap + ids_all[tid]];
  }
  __syncthreads();
  if (tid < 32) {
    // items: the sink, the selected spans, the recent tokens
    const int rbeg = min(loc_begin, pos + 1);
    const int nr = merge_ranges_warp(
        nall + 2,
        [&](int i, int& st, int& ln) {
          if (i == 0) {
            st = 0;
            ln = min(c.Ls, pos + 1);
          } else if (i <= nall) {
            st = s_sst[i - 1];
            ln = s_sln[i - 1];
          } else {
            st = rbeg;
            ln = pos + 1 - rbeg;
          }
        },
        s_rs, s_rl);
    long long tokens = 0;
    for (int t = tid; t < nall; t += 32) tokens += s_sln[t];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) tokens += shfl_xor_ll(tokens, o);
    if (tid == 0) {
      s_nr = nr;
      c.rng_cnt[unit * c.Hkv + g] = nr;
      c.sel_tokens[unit * c.Hkv + g] = tokens;  // (summed over the KV heads by ltri_get_stats)
    }
  }
  __syncthreads();
  const size_t rbb = (unit * c.Hkv + g) * (size_t)c.rcap;
  for (int t = tid; t < s_nr; t += nt) {
    c.rng_start[rbb + t] = s_rs[t];
    c.rng_len[rbb + t] = s_rl[t];
  }
}

cudaError_t launch_dec_retrieve_fused(const DevCtx& c, const DecBatch& b, int layer_begin, int layer_count,
                                      const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                                      int span_bound, bool force_cluster, int threads, cudaStream_t s) {
  span_bound = max(span_bound, 1);
  if (span_bound <= kFusedMaxSpans && !force_cluster) {  // one CTA per head: no cluster barriers
    return launch_chained(k_dec_retrieve, dim3(c.Hkv, b.n * layer_count), dim3(threads), sizeof(float) * span_bound, s,
                          c, layer_begin, b, layer_count, q, k, v);
  }
  const int per = (span_bound + kRetCluster - 1) / kRetCluster;
  if (per > kRetSliceMax) return cudaErrorInvalidValue;
  return launch_chained(k_dec_retrieve_cl, dim3(c.Hkv * kRetCluster, b.n * layer_count), dim3(kRetThreads),
                        sizeof(float) * per, s, c, layer_begin, b, layer_count, q, k, v);
}
int dec_retrieve_fused_max_spans() { return kRetCluster * kRetSliceMax; }

// dynamic shared memory of k_topk: one order key per unit in unit mode (at most 12K units: 48 KB), nothing otherwise;
// under collaborative voting a tally per unit behind the keys
static int topk_unit_smem(const DevCtx& c) {
  if (c.unit <= 0) return 0;
  const int n = (int)(c.Tmax / c.unit + 2);
  return (int)sizeof(unsigned) * (c.vote ? 2 * n + 4 : n);
}

// Top-k of the call.  Under collaborative voting (Sec. 3.5) two launches: the ballots of the layers with a retrieval
// head, then the vote (a layer reads the ballots of the layers up to its own, also those of earlier calls for the same
// chunk or step).
template <bool DECODE>
static cudaError_t launch_topk(const DevCtx& c, int seq, int layer_begin, const DecBatch& b, int layer_count, int gy,
                               int evicted_end, cudaStream_t s) {
  const int smem = topk_unit_smem(c);
  if (smem > 32 * 1024) {  // (static shared memory comes on top: ask for the larger limit in good time)
    cudaError_t e = cudaFuncSetAttribute(k_topk<DECODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
  }
  if (c.vote)
    launch_chained(k_topk<DECODE>, dim3(c.Hkv, gy), dim3(512), smem, s, c, seq, layer_begin, b, layer_count, evicted_end,
                   (int)kTopkBallot);
  launch_chained(k_topk<DECODE>, dim3(c.Hkv, gy), dim3(512), smem, s, c, seq, layer_begin, b, layer_count, evicted_end,
                 (int)(c.vote ? kTopkVote : kTopkSelect));
  return cudaGetLastError();
}

cudaError_t launch_topk_prefill(const DevCtx& c, const PrefillArgs& a, cudaStream_t s) {
  DecBatch dummy;
  dummy.n = 0;
  return launch_topk<false>(c, a.seq, a.layer_begin, dummy, a.layer_count, a.layer_count, a.loc_begin, s);
}

cudaError_t launch_topk_decode(const DevCtx& c, const DecBatch& b, int layer_begin, int layer_count, cudaStream_t s) {
  return launch_topk<true>(c, 0, layer_begin, b, layer_count, b.n * layer_count, 0, s);
}

}  // namespace ltri
