// Prefill similarity scores (Eq. 7 with summed representatives, max over the call's query spans) on tensor cores:
// score[g][s] = max_j u[g][j] . K^R[g][s].  The fp32 query representatives are split into three bf16 terms
// (u = u1 + u2 + u3 to 2^-24), so three bf16 MMAs with fp32 accumulation reproduce the fp32 dot product to rounding
// order; the index vectors are bf16 already.  A CTA keeps the split representatives in shared memory and streams
// 64-span tiles of the index through them.
#include "common.cuh"
#include "mma_util.cuh"

namespace ltri {

constexpr int kScoreStages = 4;

// grid (tile groups, Hkv, layers), 128 threads (4 warps x 16 spans)
__global__ void __launch_bounds__(128) k_score_mma(DevCtx c, int seq, int layer_begin) {
  extern __shared__ __align__(1024) unsigned char smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = blockIdx.y, layer = layer_begin + blockIdx.z;
  const size_t unit = unit_of(c, seq, layer);
  const int N = c.n_spans[unit];
  const int J = c.Jcnt[layer];
  const int ntiles = (N + 63) / 64;
  if ((int)blockIdx.x >= ntiles) return;
  const int njb = (J + 63) / 64;                      // blocks of 64 query spans
  const uint32_t sU = smem_u32(smem);                 // [njb][3 terms][64 rows][128] bf16 = njb * 48 KB
  const uint32_t sA = sU + njb * 3 * 16384;           // kScoreStages x 16 KB of index rows
  // split the representatives
  const float* up = c.u + ((size_t)layer * c.Hkv + g) * c.Jmax * kD;
  for (int i = tid; i < njb * 64 * 16; i += 128) {
    const int j = i >> 4, ch = i & 15;
    float f[8];
    if (j < J) {
      const float4 a = *reinterpret_cast<const float4*>(up + (size_t)j * kD + ch * 8);
      const float4 b = *reinterpret_cast<const float4*>(up + (size_t)j * kD + ch * 8 + 4);
      f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) f[e] = 0.f;
    }
    const int jb = j >> 6, jr = j & 63;
#pragma unroll
    for (int t = 0; t < 3; ++t) {
      uint32_t w[4];
#pragma unroll
      for (int e = 0; e < 8; e += 2) {
        const __nv_bfloat16 h0 = __float2bfloat16_rn(f[e]), h1 = __float2bfloat16_rn(f[e + 1]);
        f[e] -= __bfloat162float(h0);
        f[e + 1] -= __bfloat162float(h1);
        __nv_bfloat162 pr;
        pr.x = h0;
        pr.y = h1;
        w[e >> 1] = *reinterpret_cast<uint32_t*>(&pr);
      }
      asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(sU + (jb * 3 + t) * 16384 + tile_off(jr, ch)), "r"(w[0]),
                   "r"(w[1]), "r"(w[2]), "r"(w[3])
                   : "memory");
    }
  }
  const __nv_bfloat16* KR = c.KR + (unit * c.Hkv + g) * (size_t)c.cap * kD;
  float* sc = c.scores + (unit * c.Hkv + g) * (size_t)c.cap;
  auto issue = [&](int stage, int tile) {
    load_tile_async(sA + stage * 16384, KR + (size_t)tile * 64 * kD, kD, 64, min(64, N - tile * 64), tid, 128);
  };
  // kScoreStages-deep cp.async ring over this CTA's tiles blockIdx.x, blockIdx.x + gridDim.x, ...
  const int my_tiles = (ntiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
#pragma unroll
  for (int s = 0; s < kScoreStages - 1; ++s) {
    if (s < my_tiles) issue(s, blockIdx.x + s * gridDim.x);
    cp_async_commit();
  }
  for (int it = 0; it < my_tiles; ++it) {
    const int stage = it % kScoreStages;
    const int tile = blockIdx.x + it * gridDim.x;
    if (it + kScoreStages - 1 < my_tiles)
      issue((it + kScoreStages - 1) % kScoreStages, blockIdx.x + (it + kScoreStages - 1) * gridDim.x);
    cp_async_commit();
    cp_async_wait<kScoreStages - 1>();
    __syncthreads();
    float best0 = -INFINITY, best1 = -INFINITY;
    for (int jb = 0; jb < njb; ++jb) {
      float S[8][4];
#pragma unroll
      for (int i = 0; i < 8; ++i) S[i][0] = S[i][1] = S[i][2] = S[i][3] = 0.f;
      const int npairs = min(4, (J - jb * 64 + 15) >> 4);  // only the column tiles that hold query spans
#pragma unroll 1
      for (int t = 2; t >= 0; --t)  // smallest term first
        warp_qk_16xN(S, sA + stage * 16384, warp * 16, sU + (jb * 3 + t) * 16384, lane, npairs);
#pragma unroll
      for (int nt = 0; nt < 8; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int j = jb * 64 + nt * 8 + 2 * (lane & 3) + e;
          if (j < J) {
            best0 = fmaxf(best0, S[nt][e]);
            best1 = fmaxf(best1, S[nt][2 + e]);
          }
        }
    }
    best0 = fmaxf(best0, __shfl_xor_sync(0xffffffffu, best0, 1));
    best0 = fmaxf(best0, __shfl_xor_sync(0xffffffffu, best0, 2));
    best1 = fmaxf(best1, __shfl_xor_sync(0xffffffffu, best1, 1));
    best1 = fmaxf(best1, __shfl_xor_sync(0xffffffffu, best1, 2));
    if ((lane & 3) == 0) {
      const int s0 = tile * 64 + warp * 16 + (lane >> 2), s1 = s0 + 8;
      if (s0 < N) sc[s0] = best0;
      if (s1 < N) sc[s1] = best1;
    }
    __syncthreads();
  }
}

cudaError_t launch_score_prefill_mma(const DevCtx& c, const PrefillArgs& a, int span_bound, cudaStream_t s) {
  const int njb_max = (c.Jmax + 63) / 64;
  const int smem = njb_max * 3 * 16384 + kScoreStages * 16384;
  cudaFuncSetAttribute(k_score_mma, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  const int tiles = (span_bound + 63) / 64;
  // enough tiles per CTA to amortise the split of the representatives, enough CTAs to fill the GPU
  const int per_cta = tiles >= 512 ? 32 : 16;
  const int gx = max(1, (tiles + per_cta - 1) / per_cta);
  k_score_mma<<<dim3(gx, c.Hkv, a.layer_count), 128, smem, s>>>(c, a.seq, a.layer_begin);
  return cudaGetLastError();
}

}  // namespace ltri
