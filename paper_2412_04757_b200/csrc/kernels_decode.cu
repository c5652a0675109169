// Decode attention (Sec. 3.5: the block becomes a single token): memory-bound split-KV flash-decoding over the
// token ranges [sink | selected spans | tokens since the last eviction].  Every K/V row is read once with 16-byte
// loads and shared by the G query heads of its KV group; softmax reductions use warp shuffles.
#include "common.cuh"

namespace ltri {

constexpr float kLog2eD = 1.4426950408889634f;
constexpr int kDecThreads = 128;  // 4 warps = 8 half-warps, each half-warp owns one token at a time

__device__ __forceinline__ void unpack8(const uint4& raw, float (&f)[8]) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 t = __bfloat1622float2(p[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}

// grid (nsplit, Hkv, b.n*layer_count).  Partial results (m, l, O[128]) per (unit, head, split) go to dec_part.
template <int G>
__global__ void __launch_bounds__(kDecThreads) k_decode_attn(DevCtx c, DecBatch b, int layer_begin, int layer_count,
                                                             const __nv_bfloat16* __restrict__ q, int nsplit) {
  __shared__ int rs[kMaxTopK + 2], rl[kMaxTopK + 2], rp[kMaxTopK + 3];
  __shared__ float sm_m[8][G], sm_l[8][G];
  __shared__ float sm_o[8][G][kD];
  const int tid = threadIdx.x;
  const int hw = tid >> 4, hl = tid & 15;  // half-warp id (0..7), lane in half-warp
  const int split = blockIdx.x, g = blockIdx.y;
  const int bi = blockIdx.z / layer_count, l = blockIdx.z % layer_count, layer = layer_begin + l;
  const size_t unit = unit_of(c, b.seq[bi], layer);
  const size_t rb = (unit * c.Hkv + g) * (size_t)(c.topk + 2);
  const int nr = min(c.rng_cnt[unit * c.Hkv + g], c.topk + 2);
  if (tid == 0) {
    int run = 0;
    for (int i = 0; i < nr; ++i) {
      rs[i] = c.rng_start[rb + i];
      rl[i] = c.rng_len[rb + i];
      rp[i] = run;
      run += rl[i];
    }
    rp[nr] = run;
  }
  __syncthreads();
  const int total = rp[nr];
  const int per = (total + nsplit - 1) / nsplit;
  const int v0 = split * per, v1 = min(total, v0 + per);

  // this lane's 8 dims of the G query heads, pre-scaled
  float qf[G][8];
  const float c2 = c.scale * kLog2eD;
  const __nv_bfloat16* qp = q + (((size_t)b.src[bi] * layer_count + l) * c.Hq + (size_t)g * G) * kD + hl * 8;
#pragma unroll
  for (int hh = 0; hh < G; ++hh) {
    const uint4 raw = *reinterpret_cast<const uint4*>(qp + (size_t)hh * kD);
    unpack8(raw, qf[hh]);
#pragma unroll
    for (int e = 0; e < 8; ++e) qf[hh][e] *= c2;
  }
  const __nv_bfloat16* Kslab = c.Kc + (unit * c.Hkv + g) * (size_t)c.Tpad * kD + hl * 8;
  const __nv_bfloat16* Vslab = c.Vc + (unit * c.Hkv + g) * (size_t)c.Tpad * kD + hl * 8;

  float m[G], lsum[G], O[G][8];
#pragma unroll
  for (int hh = 0; hh < G; ++hh) {
    m[hh] = -INFINITY;
    lsum[hh] = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) O[hh][e] = 0.f;
  }
  // range cursor of this half-warp
  int ri = 0;
  constexpr int U = 4;  // tokens in flight per half-warp
  for (int base = v0; base < v1; base += 8 * U) {  // trip count is uniform over the CTA (shuffles inside)
    const int vb = base + hw * U;
    uint4 kraw[U], vraw[U];
    bool ok[U];
#pragma unroll
    for (int t = 0; t < U; ++t) {
      const int v = vb + t;
      ok[t] = v < v1;
      int tok = 0;
      if (ok[t]) {
        while (v >= rp[ri + 1]) ++ri;
        tok = rs[ri] + (v - rp[ri]);
      }
      kraw[t] = ok[t] ? __ldg(reinterpret_cast<const uint4*>(Kslab + (size_t)tok * kD)) : make_uint4(0, 0, 0, 0);
      vraw[t] = ok[t] ? __ldg(reinterpret_cast<const uint4*>(Vslab + (size_t)tok * kD)) : make_uint4(0, 0, 0, 0);
    }
    float s[U][G];
#pragma unroll
    for (int t = 0; t < U; ++t) {
      float kf[8];
      unpack8(kraw[t], kf);
#pragma unroll
      for (int hh = 0; hh < G; ++hh) {
        float d = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) d = fmaf(qf[hh][e], kf[e], d);
        s[t][hh] = d;
      }
    }
#pragma unroll
    for (int t = 0; t < U; ++t)
#pragma unroll
      for (int hh = 0; hh < G; ++hh) {
        float d = s[t][hh];
        d += __shfl_xor_sync(0xffffffffu, d, 1);
        d += __shfl_xor_sync(0xffffffffu, d, 2);
        d += __shfl_xor_sync(0xffffffffu, d, 4);
        d += __shfl_xor_sync(0xffffffffu, d, 8);
        s[t][hh] = ok[t] ? d : -INFINITY;
      }
#pragma unroll
    for (int hh = 0; hh < G; ++hh) {
      float mx = m[hh];
#pragma unroll
      for (int t = 0; t < U; ++t) mx = fmaxf(mx, s[t][hh]);
      const float mu = mx == -INFINITY ? 0.f : mx;  // a half-warp may have seen no token yet
      const float alpha = exp2f(m[hh] - mu);
      m[hh] = mx;
      lsum[hh] *= alpha;
#pragma unroll
      for (int e = 0; e < 8; ++e) O[hh][e] *= alpha;
#pragma unroll
      for (int t = 0; t < U; ++t) s[t][hh] = exp2f(s[t][hh] - mu);
    }
#pragma unroll
    for (int t = 0; t < U; ++t) {
      float vf[8];
      unpack8(vraw[t], vf);
#pragma unroll
      for (int hh = 0; hh < G; ++hh) {
        const float p = s[t][hh];
        lsum[hh] += p;
#pragma unroll
        for (int e = 0; e < 8; ++e) O[hh][e] = fmaf(p, vf[e], O[hh][e]);
      }
    }
  }
  // merge the 8 half-warps through shared memory
#pragma unroll
  for (int hh = 0; hh < G; ++hh) {
    if (hl == 0) {
      sm_m[hw][hh] = m[hh];
      sm_l[hw][hh] = lsum[hh];
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) sm_o[hw][hh][hl * 8 + e] = O[hh][e];
  }
  __syncthreads();
  for (int idx = tid; idx < G * kD; idx += kDecThreads) {
    const int hh = idx / kD, e = idx % kD;
    float mx = -INFINITY;
#pragma unroll
    for (int w = 0; w < 8; ++w) mx = fmaxf(mx, sm_m[w][hh]);
    float lt = 0.f, ot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) {
      const float sc = sm_m[w][hh] == -INFINITY ? 0.f : exp2f(sm_m[w][hh] - mx);
      lt += sm_l[w][hh] * sc;
      ot += sm_o[w][hh][e] * sc;
    }
    float* part = c.dec_part + ((unit * c.Hq + g * G + hh) * (size_t)kMaxDecSplit + split) * (kD + 2);
    part[e] = ot;
    if (e == 0) {
      part[kD] = mx;
      part[kD + 1] = lt;
    }
  }
}

// merge of the split partials: grid (Hq, b.n*layer_count), 128 threads (one per output dim).
__global__ void __launch_bounds__(kD) k_decode_merge(DevCtx c, DecBatch b, int layer_begin, int layer_count,
                                                     __nv_bfloat16* __restrict__ out, int nsplit) {
  const int h = blockIdx.x, e = threadIdx.x;
  const int bi = blockIdx.y / layer_count, l = blockIdx.y % layer_count;
  const size_t unit = unit_of(c, b.seq[bi], layer_begin + l);
  const float* part = c.dec_part + (unit * c.Hq + h) * (size_t)kMaxDecSplit * (kD + 2);
  float mx = -INFINITY;
  for (int s = 0; s < nsplit; ++s) mx = fmaxf(mx, part[(size_t)s * (kD + 2) + kD]);
  float lt = 0.f, ot = 0.f;
  for (int s = 0; s < nsplit; ++s) {
    const float ms = part[(size_t)s * (kD + 2) + kD];
    const float sc = ms == -INFINITY ? 0.f : exp2f(ms - mx);
    lt += part[(size_t)s * (kD + 2) + kD + 1] * sc;
    ot += part[(size_t)s * (kD + 2) + e] * sc;
  }
  out[(((size_t)b.src[bi] * layer_count + l) * c.Hq + h) * kD + e] = __float2bfloat16(ot / lt);
}

template <int G>
static cudaError_t launch_dec_g(const DevCtx& c, const DecBatch& b, int layer_begin, int layer_count,
                                const __nv_bfloat16* q, __nv_bfloat16* out, int nsplit, cudaStream_t s) {
  k_decode_attn<G><<<dim3(nsplit, c.Hkv, b.n * layer_count), kDecThreads, 0, s>>>(c, b, layer_begin, layer_count, q,
                                                                                 nsplit);
  k_decode_merge<<<dim3(c.Hq, b.n * layer_count), kD, 0, s>>>(c, b, layer_begin, layer_count, out, nsplit);
  return cudaGetLastError();
}

cudaError_t launch_decode_attn(const DevCtx& c, const DecBatch& b, int layer_begin, int layer_count, int,
                               const __nv_bfloat16* q, __nv_bfloat16* out, int nsplit, cudaStream_t s) {
  switch (c.G) {
    case 1: return launch_dec_g<1>(c, b, layer_begin, layer_count, q, out, nsplit, s);
    case 2: return launch_dec_g<2>(c, b, layer_begin, layer_count, q, out, nsplit, s);
    case 4: return launch_dec_g<4>(c, b, layer_begin, layer_count, q, out, nsplit, s);
    case 8: return launch_dec_g<8>(c, b, layer_begin, layer_count, q, out, nsplit, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace ltri
