// Decode attention (Sec. 3.5: while decoding, the current block is one token): memory-bound split-KV flash-decoding over the
// token ranges [sink | selected spans | tokens since the last eviction].  Every K/V row is read once with 16-byte
// loads and shared by the G query heads of its KV group; softmax reductions use warp shuffles.
#include "common.cuh"
#include "mma_util.cuh"

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

// grid (nsplit, Hkv, b.n*layer_count), 4 warps.  Each warp walks 16-token tiles of the CTA's slice of the virtual
// token list (sink | selected spans | recent tokens): the tile's K and V rows (two contiguous 256-byte rows per
// cp.async instruction, 16 bytes per lane) land in a warp-private, XOR-swizzled 2-stage ring; QK^T and PV run as
// m16n8k16 tensor-core MMAs with the G query heads of the group in the first rows of the 16-row operand, so the
// per-token ALU cost is a handful of instructions and the kernel stays bound by the K/V stream.
// Partial results (m, l, O[128]) per (unit, head, split) go to dec_part.
constexpr int kDTile = 16;
constexpr int kDStages = 2;     // two stages of 8 KB per warp: three CTAs (12 warps) fit an SM, which hides more latency
constexpr int kDecCtasPerSm = 3;  // than a deeper ring at two CTAs per SM
constexpr int kDWarpBytes = kDStages * 2 * kDTile * 256;  // K and V rows of every stage

template <int G>
__global__ void __launch_bounds__(kDecThreads, kDecCtasPerSm) k_decode_attn(DevCtx c, DecBatch b, int layer_begin, int layer_count,
                                                                const __nv_bfloat16* __restrict__ q, int nsplit) {
  chain_wait();
  extern __shared__ __align__(1024) unsigned char dsm[];
  // rs: first token of every range -- in a paged context (host-memory pager) its first K row, counted from the start
  // of the K slabs, instead: there a range lives in a sliding slab or in a slot of the unit cache
  __shared__ int rs[kMaxRanges], rp[kMaxRanges + 1];
  __shared__ float sm_m[4][G], sm_l[4][G];
  __shared__ float sm_o[4][G][kD];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int split = blockIdx.x, g = blockIdx.y;
  const int bi = blockIdx.z / layer_count, l = blockIdx.z % layer_count, layer = layer_begin + l;
  const size_t unit = unit_of(c, b.seq[bi], layer);
  const size_t rb = (unit * c.Hkv + g) * (size_t)c.rcap;
  const int nr = min(c.rng_cnt[unit * c.Hkv + g], c.rcap);
  if (tid == 0) {
    int run = 0;
    for (int i = 0; i < nr; ++i) {
      rs[i] = c.host_kv ? (int)c.rng_koff[rb + i] : c.rng_start[rb + i];
      rp[i] = run;
      run += c.rng_len[rb + i];
    }
    rp[nr] = run;
  }
  __syncthreads();
  const int total = rp[nr];
  const int per = (total + nsplit - 1) / nsplit;
  const int v0 = split * per, v1 = min(total, v0 + per);
  const int ntiles = v1 > v0 ? (v1 - v0 + kDTile - 1) / kDTile : 0;

  // query fragments: rows 0..G-1 of the 16-row A operand are the heads of the group, the rest are zero
  const int r = lane >> 2, qd = lane & 3;
  uint32_t qa[8][2];
  {
    const __nv_bfloat16* qp = q + (((size_t)b.src[bi] * layer_count + l) * c.Hq + (size_t)g * G + (r < G ? r : 0)) * kD;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      qa[ks][0] = r < G ? *reinterpret_cast<const uint32_t*>(qp + ks * 16 + 2 * qd) : 0u;
      qa[ks][1] = r < G ? *reinterpret_cast<const uint32_t*>(qp + ks * 16 + 8 + 2 * qd) : 0u;
    }
  }
  // (resident contexts: row = token; paged contexts address every range through rko / rvo below)
  const __nv_bfloat16* Kslab = c.Kc + (unit * c.Hkv + g) * (size_t)c.SR * kD;
  const __nv_bfloat16* Vslab = c.Vc + (unit * c.Hkv + g) * (size_t)c.SR * kD;
  const size_t cache_k0 = c.host_kv ? (size_t)((c.Kcache - c.Kc) / kD) : 0;
  const size_t cache_dv = c.host_kv ? (size_t)((c.Vcache - c.Vc) / kD) - cache_k0 : 0;
  const uint32_t wbase = smem_u32(dsm) + warp * kDWarpBytes;
  const float c2 = c.scale * kLog2eD;

  // this lane copies rows (lane>>4) + 2i of every tile, 16 bytes at chunk (lane&15)
  int ri = 0;
  const int ch = lane & 15;
  auto issue = [&](int t, int stage) {
    const uint32_t sk = wbase + stage * (2 * kDTile * 256), sv = sk + kDTile * 256;
    const int vb = v0 + t * kDTile;
#pragma unroll
    for (int i = 0; i < kDTile / 2; ++i) {
      const int row = 2 * i + (lane >> 4);
      const int v = vb + row;
      const bool okr = v < v1;
      size_t tok = 0;
      if (okr) {
        while (v >= rp[ri + 1]) ++ri;
        tok = (size_t)(rs[ri] + (v - rp[ri]));
      }
      const __nv_bfloat16* kp = Kslab + tok * kD;
      const __nv_bfloat16* vp = Vslab + tok * kD;
      if (c.host_kv) {
        // tok is a K row counted from c.Kc; its V row has the same number counted from c.Vc inside the slabs and is
        // cache_dv rows further inside the unit caches
        kp = c.Kc + tok * kD;
        vp = c.Vc + (tok >= cache_k0 ? tok + cache_dv : tok) * kD;
      }
      cp_async16(sk + tile_off(row, ch), kp + ch * 8, okr ? 16 : 0);
      cp_async16(sv + tile_off(row, ch), vp + ch * 8, okr ? 16 : 0);
    }
  };

  float O[16][4];
#pragma unroll
  for (int i = 0; i < 16; ++i) O[i][0] = O[i][1] = O[i][2] = O[i][3] = 0.f;
  float m = -INFINITY, lsum = 0.f;

  // tiles of this warp: warp, warp + 4, ...
  const int my_tiles = ntiles > warp ? (ntiles - warp + 3) / 4 : 0;
#pragma unroll
  for (int s = 0; s < kDStages - 1; ++s) {
    if (s < my_tiles) issue(warp + 4 * s, s);
    cp_async_commit();
  }
  for (int it = 0; it < my_tiles; ++it) {
    const int stage = it % kDStages;
    if (it + kDStages - 1 < my_tiles) issue(warp + 4 * (it + kDStages - 1), (it + kDStages - 1) % kDStages);
    cp_async_commit();
    cp_async_wait<kDStages - 1>();
    __syncwarp();
    const uint32_t sk = wbase + stage * (2 * kDTile * 256), sv = sk + kDTile * 256;
    const int vb = v0 + (warp + 4 * it) * kDTile;
    float S[2][4];
#pragma unroll
    for (int i = 0; i < 2; ++i) S[i][0] = S[i][1] = S[i][2] = S[i][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      uint32_t bf[4];
      ldsm_x4(bf, sk + tile_off((lane & 7) + ((lane >> 4) << 3), ks * 2 + ((lane >> 3) & 1)));
      const uint32_t a[4] = {qa[ks][0], 0u, qa[ks][1], 0u};
      mma_bf16(S[0], a, bf[0], bf[1]);
      mma_bf16(S[1], a, bf[2], bf[3]);
    }
    // row r of this lane: tokens nt*8 + 2*qd + e
    float tmax = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        if (vb + nt * 8 + 2 * qd + e >= v1) S[nt][e] = -INFINITY;
        tmax = fmaxf(tmax, S[nt][e]);
      }
    tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
    tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
    const float mnew = fmaxf(m, tmax * c2);
    const float mu = mnew == -INFINITY ? 0.f : mnew;
    const float alpha = exp2f(m - mu);
    m = mnew;
    float p[2][2];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
      for (int e = 0; e < 2; ++e) p[nt][e] = exp2f(fmaf(S[nt][e], c2, -mu));
    lsum = lsum * alpha + (p[0][0] + p[0][1] + p[1][0] + p[1][1]);
#pragma unroll
    for (int nt = 0; nt < 16; ++nt) {
      O[nt][0] *= alpha;
      O[nt][1] *= alpha;
    }
    const uint32_t pa[4] = {pack_bf16(p[0][0], p[0][1]), 0u, pack_bf16(p[1][0], p[1][1]), 0u};
#pragma unroll
    for (int dp = 0; dp < 8; ++dp) {
      uint32_t bf[4];
      ldsm_x4_t(bf, sv + tile_off((lane & 7) + (((lane >> 3) & 1) << 3), dp * 2 + (lane >> 4)));
      mma_bf16(O[2 * dp], pa, bf[0], bf[1]);
      mma_bf16(O[2 * dp + 1], pa, bf[2], bf[3]);
    }
    __syncwarp();
  }
  cp_async_wait<0>();
  lsum += __shfl_xor_sync(0xffffffffu, lsum, 1);
  lsum += __shfl_xor_sync(0xffffffffu, lsum, 2);
  if (r < G) {
    if (qd == 0) {
      sm_m[warp][r] = m;
      sm_l[warp][r] = lsum;
    }
#pragma unroll
    for (int nt = 0; nt < 16; ++nt) {
      sm_o[warp][r][nt * 8 + 2 * qd] = O[nt][0];
      sm_o[warp][r][nt * 8 + 2 * qd + 1] = O[nt][1];
    }
  }
  __syncthreads();
  for (int idx = tid; idx < G * kD; idx += kDecThreads) {
    const int hh = idx / kD, e = idx % kD;
    float mx = -INFINITY;
#pragma unroll
    for (int w = 0; w < 4; ++w) mx = fmaxf(mx, sm_m[w][hh]);
    float lt = 0.f, ot = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
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
  chain_wait();
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
  const int smem = 4 * kDWarpBytes;
  cudaFuncSetAttribute(k_decode_attn<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  launch_chained(k_decode_attn<G>, dim3(nsplit, c.Hkv, b.n * layer_count), dim3(kDecThreads), smem, s, c, b, layer_begin,
                 layer_count, q, nsplit);
  return launch_chained(k_decode_merge, dim3(c.Hq, b.n * layer_count), dim3(kD), 0, s, c, b, layer_begin, layer_count, out,
                        nsplit);
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
