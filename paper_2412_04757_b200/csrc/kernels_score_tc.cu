// Prefill similarity scores (Eq. 7 with summed representatives, max over the call's query spans) on tcgen05:
// score[g][s] = max_j u[g][j] . K^R[g][s].  The fp32 representatives are split into three bf16 terms
// (u = u1 + u2 + u3 to 2^-24) and written to shared memory in the 128-byte-swizzled K-major layout the tensor core
// reads; index rows arrive by TMA in 128-span tiles; 3 x 8 MMAs (M = 128 spans, N = padded span count, K = 16)
// accumulate one fp32 tile in TMEM, and each epilogue thread takes the maximum over its span's row.
// Roles: warps 0-3 epilogue (thread = span), warp 4 TMA producer, warp 5 MMA issuer.
#include <cuda.h>

#include <cstring>

#include "common.cuh"
#include "tc_util.cuh"

namespace ltri {

using namespace tc;

constexpr int kScThreads = 192;
// index-tile stages: two when the representatives are small enough for two CTAs to share an SM (one CTA's prologue
// -- splitting the representatives -- then overlaps the other's stream), three when only one CTA fits
constexpr int kScMaxN = 96;  // padded query-span count the kernel supports

template <int kScStages>
__global__ void __launch_bounds__(kScThreads, kScStages == 2 ? 2 : 1)
    k_score_tc(DevCtx c, int seq, int layer_begin, int tiles_per_cta, int npad_lay,
               const __grid_constant__ CUtensorMap kr_map) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long bars[2 * kScStages + 4];  // AFULL[3] AEMPTY[3] SFULL[2] SEMPTY[2]
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;
  chain_wait();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = blockIdx.y, layer = layer_begin + blockIdx.z;
  const size_t unit = unit_of(c, seq, layer);
  const int N = c.n_spans[unit];
  const int J = c.Jcnt[layer];
  const int ntiles = (N + 127) / 128;
  const int tile0 = blockIdx.x * tiles_per_cta;
  if (tile0 >= ntiles) return;
  const int my_tiles = min(tiles_per_cta, ntiles - tile0);
  const int Npad = max(16, (J + 15) & ~15);
  const uint32_t sbase = (smem_addr(smem_raw) + 1023u) & ~1023u;
  const uint32_t sA = sbase;                          // kScStages x 32 KB: [half d][128 spans][64]
  const uint32_t sU = sbase + kScStages * 32768;      // 3 terms x [half d][npad_lay rows][64]
  const uint32_t kHalfBytes = (uint32_t)npad_lay * 128;  // npad_lay: the context's largest padded query-span count
  const uint32_t kTermBytes = 2 * kHalfBytes;
  enum { B_AFULL = 0, B_AEMPTY = kScStages, B_SFULL = 2 * kScStages, B_SEMPTY = 2 * kScStages + 2 };
  auto bar = [&](int i) { return smem_addr(&bars[i]); };
  volatile int* abortp = &s_abort;
  if (tid == 0) {
    s_abort = 0;
    for (int s = 0; s < kScStages; ++s) {
      mbar_init(bar(B_AFULL + s), 1);
      mbar_init(bar(B_AEMPTY + s), 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(bar(B_SFULL + s), 1);
      mbar_init(bar(B_SEMPTY + s), 4);
    }
    fence_mbar_init();
  }
  // split the representatives into three bf16 terms, K-major rows of 64 elements, 16-byte chunks XOR-swizzled by row
  {
    const float* up = c.u + ((size_t)layer * c.Hkv + g) * c.Jmax * kD;
    for (int i = tid; i < Npad * 16; i += kScThreads) {
      const int j = i >> 4, ch = i & 15;  // chunk of 8 elements: half = ch >> 3, chunk in half = ch & 7
      float f[8];
      if (j < J) {
        const float4 a = *reinterpret_cast<const float4*>(up + (size_t)j * kD + ch * 8);
        const float4 b = *reinterpret_cast<const float4*>(up + (size_t)j * kD + ch * 8 + 4);
        f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) f[e] = 0.f;
      }
      const uint32_t off = (uint32_t)(ch >> 3) * kHalfBytes + (uint32_t)j * 128 + (uint32_t)(((ch & 7) ^ (j & 7)) << 4);
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
        asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(sU + t * kTermBytes + off), "r"(w[0]), "r"(w[1]),
                     "r"(w[2]), "r"(w[3])
                     : "memory");
      }
    }
  }
  fence_async_smem();  // the tensor core reads these tiles through the async proxy
  if (warp == 4) tmem_alloc(smem_addr(&s_tmem_base), 256);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem = s_tmem_base;
  const long long row0 = (long long)(unit * c.Hkv + g) * c.cap;

  if (warp == 4) {
    if (lane == 0) {
      bool ok = true;
      for (int it = 0; ok && it < my_tiles; ++it) {
        const int st = it % kScStages;
        if (it >= kScStages) ok = mbar_wait(bar(B_AEMPTY + st), ((it / kScStages) - 1) & 1, abortp, c.wait_limit);
        if (!ok) break;
        const long long row = row0 + (long long)(tile0 + it) * 128;
        mbar_expect_tx(bar(B_AFULL + st), 32768);
        tma_load_2d(sA + st * 32768, &kr_map, 0, (int)row, bar(B_AFULL + st));
        tma_load_2d(sA + st * 32768 + 16384, &kr_map, 64, (int)row, bar(B_AFULL + st));
      }
      for (int back = 1; back <= kScStages && back <= my_tiles; ++back) {  // no copy in flight at exit
        const int ii = my_tiles - back;
        if (!mbar_wait(bar(B_AEMPTY + (ii % kScStages)), (ii / kScStages) & 1, abortp, c.wait_limit)) break;
      }
    }
  } else if (warp == 5) {
    if (lane == 0) {
      const uint32_t idesc = make_idesc(128, Npad, false);
      const uint64_t dA = make_desc(sA, 16, 1024), dU = make_desc(sU, 16, 1024);
      bool ok = true;
      for (int it = 0; ok && it < my_tiles; ++it) {
        const int st = it % kScStages, buf = it & 1;
        ok = mbar_wait(bar(B_AFULL + st), (it / kScStages) & 1, abortp, c.wait_limit);
        if (!ok) break;
        if (it >= 2) ok = mbar_wait(bar(B_SEMPTY + buf), ((it >> 1) - 1) & 1, abortp, c.wait_limit);
        if (!ok) break;
        fence_after_sync();
        const uint64_t da = dA + (uint64_t)((st * 32768) >> 4);
#pragma unroll
        for (int t = 2; t >= 0; --t) {  // smallest term first
          const uint64_t db = dU + (uint64_t)((t * kTermBytes) >> 4);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const uint32_t kin = (ks & 3) * 32;
            mma_ss(tmem + buf * 128, da + (((ks >> 2) * 16384 + kin) >> 4), db + (((ks >> 2) * kHalfBytes + kin) >> 4),
                   idesc, !(t == 2 && ks == 0));
          }
        }
        mma_commit(bar(B_SFULL + buf));
        mma_commit(bar(B_AEMPTY + st));
      }
    }
  } else {
    // epilogue: thread = span row of the tile
    const int r = warp * 32 + lane;
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    float* sc = c.scores + (unit * c.Hkv + g) * (size_t)c.cap;
    bool ok = true;
    for (int it = 0; it < my_tiles; ++it) {
      const int buf = it & 1;
      ok = ok && mbar_wait(bar(B_SFULL + buf), (it >> 1) & 1, abortp, c.wait_limit);
      if (!ok) break;
      fence_after_sync();
      float best = -INFINITY;
      for (int c0 = 0; c0 < Npad; c0 += 16) {
        uint32_t v[16];
        tmem_ld16(tmem + lane_base + buf * 128 + c0, v);
        tmem_ld_wait();
#pragma unroll
        for (int e = 0; e < 16; ++e)
          if (c0 + e < J) best = fmaxf(best, __uint_as_float(v[e]));
      }
      fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_SEMPTY + buf));
      const int s = (tile0 + it) * 128 + r;
      if (s < N) sc[s] = best;
    }
  }
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  if (warp == 4) tmem_dealloc(tmem, 256);
  if (tid == 0 && s_abort) set_status(c, -6, 7000 + (int)blockIdx.x);
}

bool score_tc_supported(const DevCtx& c) { return ((c.Jmax + 15) & ~15) <= kScMaxN; }

cudaError_t launch_score_prefill_tc(const DevCtx& c, const PrefillArgs& a, int span_bound, const void* kv_maps,
                                    cudaStream_t s) {
  if (!score_tc_supported(c) || !kv_maps) return cudaErrorNotSupported;
  CUtensorMap kr;
  memcpy(&kr, static_cast<const CUtensorMap*>(kv_maps) + 5, sizeof(kr));
  const int npad_lay = max(16, (c.Jmax + 15) & ~15);
  const int rep_bytes = 3 * 2 * npad_lay * 128 + 1024;
  const bool two = 2 * (2 * 32768 + rep_bytes + 1024) <= 227 * 1024;  // two CTAs (with their reserved KB) per SM
  const int smem = (two ? 2 : 3) * 32768 + rep_bytes;
  const int tiles = (span_bound + 127) / 128;
  const int per_cta = tiles >= 256 ? 32 : (tiles >= 48 ? 16 : 8);  // amortise the split of the representatives
  const int gx = (tiles + per_cta - 1) / per_cta;
  const dim3 grid(gx > 0 ? gx : 1, c.Hkv, a.layer_count);
  if (two) {
    cudaFuncSetAttribute(k_score_tc<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    return launch_chained(k_score_tc<2>, grid, dim3(kScThreads), smem, s, c, a.seq, a.layer_begin, per_cta, npad_lay, kr);
  } else {
    cudaFuncSetAttribute(k_score_tc<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    return launch_chained(k_score_tc<3>, grid, dim3(kScThreads), smem, s, c, a.seq, a.layer_begin, per_cta, npad_lay, kr);
  }
  return cudaGetLastError();
}

}  // namespace ltri
