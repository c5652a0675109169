// Prefill attention and local-map kernels, warp-MMA version (ldmatrix + mma.sync bf16, fp32 accumulate).
//   k_attn_prefill : exact softmax attention of the call's queries over a list of key ranges (Sec. 3.4 step 3).
//                    phase 0 walks sink | local | current (causal) and stores the softmax state; phase 1 resumes
//                    from that state over the retrieved spans and writes the output.
//   k_map_local / k_map_cur : second pass over local | current that turns the now-known row statistics into the
//                    Q20 fixed-point local attention map: votes (Eq. 6) and the region's head-summed map (Eq. 4).
#include "common.cuh"
#include "mma_util.cuh"

namespace ltri {

constexpr float kLog2e = 1.4426950408889634f;

struct Ranges {
  int n;
  int start[kMaxTopK + 2];
  int len[kMaxTopK + 2];
};

// ------------------------------------------------------------------------------------------
// grid (M tiles, Hkv, layers), 256 threads.  M tile = 128 rows = (128/G tokens) x (G heads of one KV group).
template <int G>
__global__ void __launch_bounds__(256, 1) k_attn_prefill(DevCtx c, PrefillArgs a, int phase, int final_out) {
  extern __shared__ __align__(1024) unsigned char smem[];
  __shared__ Ranges rg;
  constexpr int TOK = 128 / G;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = blockIdx.y, l = blockIdx.z, layer = a.layer_begin + l;
  const size_t unit = unit_of(c, a.seq, layer);
  const int tok0 = blockIdx.x * TOK;  // first token (call-relative) of this tile
  const uint32_t sQ = smem_u32(smem), sK = sQ + 32768, sV = sK + 32768;  // K,V: 2 stages x 16 KB

  const int last_tok = min(a.n, tok0 + TOK) - 1;  // call-relative, last valid token of the tile
  if (tid == 0) {
    if (phase == 0) {
      rg.n = 3;
      rg.start[0] = 0;
      rg.len[0] = a.sink_end;
      rg.start[1] = a.loc_begin;
      rg.len[1] = a.t0 - a.loc_begin;
      rg.start[2] = a.t0;
      rg.len[2] = last_tok + 1;  // causal range: keys up to the tile's last token
    } else {
      const size_t rb = (unit * c.Hkv + g) * (size_t)c.rcap;
      const int nr = min(c.rng_cnt[unit * c.Hkv + g], kMaxTopK + 2);
      rg.n = nr;
      for (int i = 0; i < nr; ++i) {
        rg.start[i] = c.rng_start[rb + i];
        rg.len[i] = c.rng_len[rb + i];
      }
    }
  }
  // Q tile
  {
    const __nv_bfloat16* qbase = a.q + (((size_t)l * a.n + tok0) * c.Hq + (size_t)g * G) * kD;
    for (int i = tid; i < 128 * 16; i += 256) {
      const int r = i >> 4, ch = i & 15;
      const int tk = r / G, hh = r % G;
      const bool ok = tok0 + tk < a.n;
      const __nv_bfloat16* src = qbase + (ok ? ((size_t)tk * c.Hq + hh) * kD : 0) + ch * 8;
      cp_async16(sQ + tile_off(r, ch), src, ok ? 16 : 0);
    }
  }
  __syncthreads();

  const __nv_bfloat16* Kslab = c.Kc + (unit * c.Hkv + g) * (size_t)c.SR * kD;
  const __nv_bfloat16* Vslab = c.Vc + (unit * c.Hkv + g) * (size_t)c.SR * kD;
  const float c2 = c.scale * kLog2e;

  // rows of this thread
  const int r0 = warp * 16 + (lane >> 2), r1 = r0 + 8;
  const int tk0 = tok0 + r0 / G, tk1 = tok0 + r1 / G;  // call-relative tokens
  const int h0 = g * G + r0 % G, h1 = g * G + r1 % G;

  float O[16][4];
  float mraw[2], lsum[2];
#pragma unroll
  for (int i = 0; i < 16; ++i) O[i][0] = O[i][1] = O[i][2] = O[i][3] = 0.f;
  mraw[0] = mraw[1] = -INFINITY;
  lsum[0] = lsum[1] = 0.f;
  if (phase == 1) {
    if (tk0 < a.n) {
      const float2 st = c.rowstat[((size_t)layer * c.chunk + tk0) * c.Hq + h0];
      mraw[0] = st.x / c2;
      lsum[0] = (lane & 3) == 0 ? st.y : 0.f;
      const float* op = c.Oacc + (((size_t)layer * c.chunk + tk0) * c.Hq + h0) * kD + 2 * (lane & 3);
#pragma unroll
      for (int nt = 0; nt < 16; ++nt) {
        const float2 v = *reinterpret_cast<const float2*>(op + nt * 8);
        O[nt][0] = v.x;
        O[nt][1] = v.y;
      }
    }
    if (tk1 < a.n) {
      const float2 st = c.rowstat[((size_t)layer * c.chunk + tk1) * c.Hq + h1];
      mraw[1] = st.x / c2;
      lsum[1] = (lane & 3) == 0 ? st.y : 0.f;
      const float* op = c.Oacc + (((size_t)layer * c.chunk + tk1) * c.Hq + h1) * kD + 2 * (lane & 3);
#pragma unroll
      for (int nt = 0; nt < 16; ++nt) {
        const float2 v = *reinterpret_cast<const float2*>(op + nt * 8);
        O[nt][2] = v.x;
        O[nt][3] = v.y;
      }
    }
  }

  // tile iterator over the ranges
  int ri = 0, off = 0;
  auto skip_empty = [&]() {
    while (ri < rg.n && off >= rg.len[ri]) {
      ++ri;
      off = 0;
    }
  };
  auto issue = [&](int stage, int rix, int offx) {
    const int kt = rg.start[rix] + offx;
    const int nvalid = min(64, rg.len[rix] - offx);
    load_tile_async(sK + stage * 16384, Kslab + (size_t)kt * kD, kD, 64, nvalid, tid, 256);
    load_tile_async(sV + stage * 16384, Vslab + (size_t)kt * kD, kD, 64, nvalid, tid, 256);
  };
  skip_empty();
  int stage = 0;
  if (ri < rg.n) issue(0, ri, off);
  cp_async_commit();

  while (ri < rg.n) {
    const int cri = ri, coff = off;
    off += 64;
    skip_empty();
    const bool more = ri < rg.n;
    if (more) issue(stage ^ 1, ri, off);
    cp_async_commit();
    if (more)
      cp_async_wait<1>();
    else
      cp_async_wait<0>();
    __syncthreads();

    const int kt = rg.start[cri] + coff;
    const int nvalid = min(64, rg.len[cri] - coff);
    const bool causal = phase == 0 && cri == 2;
    float S[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) S[i][0] = S[i][1] = S[i][2] = S[i][3] = 0.f;
    warp_qk_16x64(S, sQ, warp * 16, sK + stage * 16384, lane);
    // mask + row max
    float tmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int nt = 0; nt < 8; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int col = nt * 8 + 2 * (lane & 3) + (e & 1);
        const int rowtok = (e < 2) ? tk0 : tk1;
        bool ok = col < nvalid;
        if (causal) ok = ok && (kt + col <= a.t0 + rowtok);
        if (!ok) S[nt][e] = -INFINITY;
        tmax[e >> 1] = fmaxf(tmax[e >> 1], S[nt][e]);
      }
    float alpha[2], mc[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      tmax[r] = fmaxf(tmax[r], __shfl_xor_sync(0xffffffffu, tmax[r], 1));
      tmax[r] = fmaxf(tmax[r], __shfl_xor_sync(0xffffffffu, tmax[r], 2));
      const float mnew = fmaxf(mraw[r], tmax[r]);
      mc[r] = mnew == -INFINITY ? 0.f : mnew * c2;
      alpha[r] = exp2f(mraw[r] * c2 - mc[r]);  // mraw = -inf -> 0
      mraw[r] = mnew;
      lsum[r] *= alpha[r];
    }
    uint32_t P[4][4];
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const float p0 = exp2f(S[nt][0] * c2 - mc[0]);
      const float p1 = exp2f(S[nt][1] * c2 - mc[0]);
      const float p2 = exp2f(S[nt][2] * c2 - mc[1]);
      const float p3 = exp2f(S[nt][3] * c2 - mc[1]);
      lsum[0] += p0 + p1;
      lsum[1] += p2 + p3;
      P[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p0, p1);
      P[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2, p3);
    }
#pragma unroll
    for (int nt = 0; nt < 16; ++nt) {
      O[nt][0] *= alpha[0];
      O[nt][1] *= alpha[0];
      O[nt][2] *= alpha[1];
      O[nt][3] *= alpha[1];
    }
    const uint32_t vt = sV + stage * 16384;
#pragma unroll
    for (int kb = 0; kb < 4; ++kb) {
#pragma unroll
      for (int dp = 0; dp < 8; ++dp) {
        uint32_t b[4];
        ldsm_x4_t(b, vt + tile_off(kb * 16 + (lane & 7) + (((lane >> 3) & 1) << 3), dp * 2 + (lane >> 4)));
        mma_bf16(O[2 * dp], P[kb], b[0], b[1]);
        mma_bf16(O[2 * dp + 1], P[kb], b[2], b[3]);
      }
    }
    __syncthreads();
    stage ^= 1;
  }
  cp_async_wait<0>();

  // epilogue
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    lsum[r] += __shfl_xor_sync(0xffffffffu, lsum[r], 1);
    lsum[r] += __shfl_xor_sync(0xffffffffu, lsum[r], 2);
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int tk = r == 0 ? tk0 : tk1, h = r == 0 ? h0 : h1;
    if (tk >= a.n) continue;
    if (phase == 0) {
      if ((lane & 3) == 0) c.rowstat[((size_t)layer * c.chunk + tk) * c.Hq + h] = make_float2(mraw[r] * c2, lsum[r]);
      if (!final_out) {
        float* op = c.Oacc + (((size_t)layer * c.chunk + tk) * c.Hq + h) * kD + 2 * (lane & 3);
#pragma unroll
        for (int nt = 0; nt < 16; ++nt)
          *reinterpret_cast<float2*>(op + nt * 8) = make_float2(O[nt][2 * r], O[nt][2 * r + 1]);
      }
    }
    if (final_out) {
      const float inv = 1.f / lsum[r];
      __nv_bfloat16* op = a.out + (((size_t)l * a.n + tk) * c.Hq + h) * kD + 2 * (lane & 3);
#pragma unroll
      for (int nt = 0; nt < 16; ++nt)
        *reinterpret_cast<uint32_t*>(op + nt * 8) = pack_bf16(O[nt][2 * r] * inv, O[nt][2 * r + 1] * inv);
    }
  }
}

template <int G>
static cudaError_t launch_attn_g(const DevCtx& c, const PrefillArgs& a, int phase, bool final_out, cudaStream_t s) {
  constexpr int TOK = 128 / G;
  const int smem = 32768 * 3;
  cudaFuncSetAttribute(k_attn_prefill<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  k_attn_prefill<G><<<dim3((a.n + TOK - 1) / TOK, c.Hkv, a.layer_count), 256, smem, s>>>(c, a, phase, final_out ? 1 : 0);
  return cudaGetLastError();
}

cudaError_t launch_attn_prefill(const DevCtx& c, const PrefillArgs& a, int phase, bool final_out, cudaStream_t s) {
  switch (c.G) {
    case 1: return launch_attn_g<1>(c, a, phase, final_out, s);
    case 2: return launch_attn_g<2>(c, a, phase, final_out, s);
    case 4: return launch_attn_g<4>(c, a, phase, final_out, s);
    case 8: return launch_attn_g<8>(c, a, phase, final_out, s);
  }
  return cudaErrorInvalidValue;
}

// ------------------------------------------------------------------------------------------
// Quantised probability of one logit given its row statistics (reading of Eq. 1-3 in Q20 fixed point):
// Aq = rint(2^20 * exp2(s*scale*log2e - m) / sum), (m, sum) being the row statistics the attention kernel stored.
__device__ __forceinline__ int quant_prob(float s, float m_scaled, float inv_l_q, float c2) {
  return __float2int_rn(exp2f(fmaf(s, c2, -m_scaled)) * inv_l_q);
}

// reduce the per-thread column sums of a 16x64 warp tile over the 8 row groups and add them to sh_cols[64]
__device__ __forceinline__ void reduce_cols(int (&cs)[8][2], unsigned long long* sh_cols, int lane) {
#pragma unroll
  for (int nt = 0; nt < 8; ++nt)
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      int v = cs[nt][e];
      v += __shfl_xor_sync(0xffffffffu, v, 4);
      v += __shfl_xor_sync(0xffffffffu, v, 8);
      v += __shfl_xor_sync(0xffffffffu, v, 16);
      if (lane < 4 && v != 0) atomicAdd(&sh_cols[nt * 8 + 2 * lane + e], (unsigned long long)v);
    }
}

// votes of the local keys: grid (64-key tiles of [loc_begin,t0), Hkv, layers), 128 threads.  The key tile stays in
// shared memory while all n*G query rows stream through in 64-row tiles.
template <int G>
__global__ void __launch_bounds__(128) k_map_local(DevCtx c, PrefillArgs a) {
  extern __shared__ __align__(1024) unsigned char smem[];
  __shared__ unsigned long long sh_cols[64];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = blockIdx.y, l = blockIdx.z, layer = a.layer_begin + l;
  const size_t unit = unit_of(c, a.seq, layer);
  const int kt = a.loc_begin + blockIdx.x * 64;
  const int nvalid = min(64, a.t0 - kt);
  const uint32_t sK = smem_u32(smem), sQ = sK + 16384;  // Q: 2 stages x 16 KB
  constexpr int TOK = 64 / G;
  const int ntiles = (a.n + TOK - 1) / TOK;
  if (tid < 64) sh_cols[tid] = 0;
  const __nv_bfloat16* Kslab = c.Kc + (unit * c.Hkv + g) * (size_t)c.SR * kD;
  load_tile_async(sK, Kslab + (size_t)kt * kD, kD, 64, nvalid, tid, 128);
  auto issue_q = [&](int stage, int t) {
    const int tok0 = t * TOK;
    const __nv_bfloat16* qbase = a.q + (((size_t)l * a.n + tok0) * c.Hq + (size_t)g * G) * kD;
    for (int i = tid; i < 64 * 16; i += 128) {
      const int r = i >> 4, ch = i & 15;
      const int tk = r / G, hh = r % G;
      const bool ok = tok0 + tk < a.n;
      cp_async16(sQ + stage * 16384 + tile_off(r, ch), qbase + (ok ? ((size_t)tk * c.Hq + hh) * kD : 0) + ch * 8,
                 ok ? 16 : 0);
    }
  };
  issue_q(0, 0);
  cp_async_commit();
  const float c2 = c.scale * kLog2e;
  int cs[8][2];
#pragma unroll
  for (int i = 0; i < 8; ++i) cs[i][0] = cs[i][1] = 0;
  for (int t = 0; t < ntiles; ++t) {
    const int stage = t & 1;
    if (t + 1 < ntiles) issue_q(stage ^ 1, t + 1);
    cp_async_commit();
    if (t + 1 < ntiles)
      cp_async_wait<1>();
    else
      cp_async_wait<0>();
    __syncthreads();
    float S[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) S[i][0] = S[i][1] = S[i][2] = S[i][3] = 0.f;
    warp_qk_16x64(S, sQ + stage * 16384, warp * 16, sK, lane);
    const int r0 = warp * 16 + (lane >> 2), r1 = r0 + 8;
    const int tk0 = t * TOK + r0 / G, tk1 = t * TOK + r1 / G;
    float m0 = 0.f, m1 = 0.f, il0 = 0.f, il1 = 0.f;
    if (tk0 < a.n) {
      const float2 st = c.rowstat[((size_t)layer * c.chunk + tk0) * c.Hq + g * G + r0 % G];
      m0 = st.x;
      il0 = kQScale / st.y;
    }
    if (tk1 < a.n) {
      const float2 st = c.rowstat[((size_t)layer * c.chunk + tk1) * c.Hq + g * G + r1 % G];
      m1 = st.x;
      il1 = kQScale / st.y;
    }
#pragma unroll
    for (int nt = 0; nt < 8; ++nt)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int col = nt * 8 + 2 * (lane & 3) + e;
        if (col < nvalid) {
          if (tk0 < a.n) cs[nt][e] += quant_prob(S[nt][e], m0, il0, c2);
          if (tk1 < a.n) cs[nt][e] += quant_prob(S[nt][2 + e], m1, il1, c2);
        }
      }
    __syncthreads();
  }
  reduce_cols(cs, sh_cols, lane);
  __syncthreads();
  if (tid < nvalid && sh_cols[tid] != 0 && kt + tid >= c.Ls)
    atomicAdd((unsigned long long*)&c.votes[unit * c.Tpad + kt + tid], sh_cols[tid]);
}

// current-chunk block of the map: grid (tile pairs (it >= jt) of 64x64 token tiles, layers), 128 threads.
// Loops over all query heads so that the head sum of Eq. 4 needs no atomics; writes the region map tile and adds
// the tile's column sums to the votes.
template <int G>
__global__ void __launch_bounds__(128) k_map_cur(DevCtx c, PrefillArgs a) {
  extern __shared__ __align__(1024) unsigned char smem[];
  __shared__ unsigned long long sh_cols[64];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int l = blockIdx.y, layer = a.layer_begin + l;
  const size_t unit = unit_of(c, a.seq, layer);
  int it = 0, rem = blockIdx.x;
  while (rem > it) {
    rem -= it + 1;
    ++it;
  }
  const int jt = rem;
  const uint32_t sK = smem_u32(smem), sQ = sK + 2 * 16384;  // K: 2 stages, Q: 2 stages
  if (tid < 64) sh_cols[tid] = 0;
  const int i0 = it * 64, j0 = jt * 64;  // call-relative
  const int qvalid = min(64, a.n - i0), kvalid = min(64, a.n - j0);
  auto issue = [&](int h) {
    const int st = h & 1;
    load_tile_async(sQ + st * 16384, a.q + (((size_t)l * a.n + i0) * c.Hq + h) * kD, (size_t)c.Hq * kD, 64, qvalid, tid,
                    128);
    if (h % G == 0) {
      const int g = h / G;
      const __nv_bfloat16* Kslab = c.Kc + (unit * c.Hkv + g) * (size_t)c.SR * kD;
      load_tile_async(sK + (g & 1) * 16384, Kslab + (size_t)(a.t0 + j0) * kD, kD, 64, kvalid, tid, 128);
    }
  };
  issue(0);
  cp_async_commit();
  const float c2 = c.scale * kLog2e;
  int acc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0;
  const int r0 = warp * 16 + (lane >> 2), r1 = r0 + 8;
  const int ti0 = i0 + r0, ti1 = i0 + r1;  // call-relative query tokens
  for (int h = 0; h < c.Hq; ++h) {
    if (h + 1 < c.Hq) issue(h + 1);
    cp_async_commit();
    if (h + 1 < c.Hq)
      cp_async_wait<1>();
    else
      cp_async_wait<0>();
    __syncthreads();
    float S[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) S[i][0] = S[i][1] = S[i][2] = S[i][3] = 0.f;
    warp_qk_16x64(S, sQ + (h & 1) * 16384, warp * 16, sK + ((h / G) & 1) * 16384, lane);
    float m0 = 0.f, m1 = 0.f, il0 = 0.f, il1 = 0.f;
    if (ti0 < a.n) {
      const float2 st = c.rowstat[((size_t)layer * c.chunk + ti0) * c.Hq + h];
      m0 = st.x;
      il0 = kQScale / st.y;
    }
    if (ti1 < a.n) {
      const float2 st = c.rowstat[((size_t)layer * c.chunk + ti1) * c.Hq + h];
      m1 = st.x;
      il1 = kQScale / st.y;
    }
#pragma unroll
    for (int nt = 0; nt < 8; ++nt)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int tj = j0 + nt * 8 + 2 * (lane & 3) + e;  // call-relative key token
        if (tj < a.n && a.t0 + tj >= c.Ls) {
          if (ti0 < a.n && tj <= ti0) acc[nt][e] += quant_prob(S[nt][e], m0, il0, c2);
          if (ti1 < a.n && tj <= ti1) acc[nt][2 + e] += quant_prob(S[nt][2 + e], m1, il1, c2);
        }
      }
    __syncthreads();
  }
  // region map tile
  int* Mq = c.Mq + (size_t)layer * c.chunk * c.chunk;
  const int roff = a.t0 - a.reg_start;  // <= 0: region row = call-relative token + roff
  int cs[8][2];
#pragma unroll
  for (int nt = 0; nt < 8; ++nt)
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int tj = j0 + nt * 8 + 2 * (lane & 3) + e;
      cs[nt][e] = acc[nt][e] + acc[nt][2 + e];
      const int cj = tj + roff;
      if (tj < a.n && cj >= 0) {
        const int ri0 = ti0 + roff, ri1 = ti1 + roff;
        if (ti0 < a.n && ri0 >= 0 && tj <= ti0) Mq[(size_t)ri0 * c.chunk + cj] = acc[nt][e];
        if (ti1 < a.n && ri1 >= 0 && tj <= ti1) Mq[(size_t)ri1 * c.chunk + cj] = acc[nt][2 + e];
      }
    }
  reduce_cols(cs, sh_cols, lane);
  __syncthreads();
  if (tid < kvalid && sh_cols[tid] != 0)
    atomicAdd((unsigned long long*)&c.votes[unit * c.Tpad + a.t0 + j0 + tid], sh_cols[tid]);
}

template <int G>
static cudaError_t launch_map_g(const DevCtx& c, const PrefillArgs& a, cudaStream_t s) {
  const int nloc = a.t0 - a.loc_begin;
  if (nloc > 0 && a.loc_begin >= c.Ls) {
    cudaFuncSetAttribute(k_map_local<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, 3 * 16384);
    k_map_local<G><<<dim3((nloc + 63) / 64, c.Hkv, a.layer_count), 128, 3 * 16384, s>>>(c, a);
  }
  const int nt = (a.n + 63) / 64;
  cudaFuncSetAttribute(k_map_cur<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, 4 * 16384);
  k_map_cur<G><<<dim3(nt * (nt + 1) / 2, a.layer_count), 128, 4 * 16384, s>>>(c, a);
  return cudaGetLastError();
}

cudaError_t launch_map_pass(const DevCtx& c, const PrefillArgs& a, cudaStream_t s) {
  switch (c.G) {
    case 1: return launch_map_g<1>(c, a, s);
    case 2: return launch_map_g<2>(c, a, s);
    case 4: return launch_map_g<4>(c, a, s);
    case 8: return launch_map_g<8>(c, a, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace ltri
