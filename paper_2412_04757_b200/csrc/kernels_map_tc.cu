// Local-map pass on tcgen05 tensor cores: with the row statistics of the local softmax known, recompute the logits of
// local | current keys and turn them into Q20 fixed-point probabilities (reading of Eq. 1-3), accumulating the votes of
// Eq. 6 (column sums over all rows and heads) and the head-summed region map of Eq. 4.
//
// The product is computed transposed, S^T = K Q^T: a CTA keeps up to four 128-key tiles in shared memory and streams
// all query rows of its KV group through them in 128-row blocks (row = (token, head)).  With keys on the TMEM lanes
// every epilogue thread owns one key, so a column sum of the map is a thread-local sum and needs no shuffles; the G
// heads of a token are adjacent columns, so their sum (Eq. 4) is thread-local too and goes to the region map with one
// integer reduction per (token, key, KV head).  Roles: warps 0-15 epilogue (four warps per lane quarter, 32 columns
// each), warp 16 TMA producer, warp 17 MMA issuer; four TMEM accumulators and two Q stages overlap the MMAs with the
// exp/round epilogue, which is bound by the special-function unit (one ex2 per map entry).  The rows' softmax
// offsets ride along in the contraction (a ninth K step against a tile of ones), so the epilogue is one multiply,
// one ex2, one fused scale-and-round and one integer add per entry, with no per-column operand to fetch.
#include <cuda.h>

#include <cstring>

#include "common.cuh"
#include "tc_util.cuh"

namespace ltri {

using namespace tc;

constexpr float kLog2eM = 1.4426950408889634f;
constexpr int kMapThreads = 576;  // 16 epilogue warps + TMA producer + MMA issuer
// The attention kernel stores per row off = -m - log2(l) + 21 + kMapMargin, so that x = logit*scale*log2e + off is
// log2(p * 2^20) + 1 + margin and the Q20 value is rint(2^x * kMapScale); x < 0 means the value is below
// 2^-(1+margin) < 0.5 and rounds to zero.

struct MapMaps {
  CUtensorMap q;    // [tokens][Hq][128] bf16, box {64, G, 128/G}
  CUtensorMap k128; // K slabs, box {64, 128}
};

__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float ex2m(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// grid (key-tile groups, Hkv, layers).  A CTA keeps up to kMapKT 128-key tiles of one KV head in shared memory (all
// from [loc_begin, t0) or all from the call's own tokens [t0, t0+n)) and streams the query blocks through them once,
// so the query tensor is re-read kMapKT times less often than with one key tile per CTA.
constexpr int kMapKT = 4;

template <int G>
__global__ void __launch_bounds__(kMapThreads, 1)
    k_map_tc(DevCtx c, PrefillArgs a, int n_local_groups, int n_local_tiles, int n_cur_tiles,
             const __grid_constant__ MapMaps maps) {
  extern __shared__ unsigned char smem_raw[];
  // KFULL[4] | QFULL[2] QEMPTY[2] | SFULL[4] SEMPTY[4]
  __shared__ __align__(8) unsigned long long bars[4 + 4 + 8];
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;
  constexpr int TPB = 128 / G;  // tokens per query block
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = blockIdx.y, l = blockIdx.z, layer = a.layer_begin + l;
  const size_t unit = unit_of(c, a.seq, layer);
  // a layer with a retrieval head (Sec. 3.5) draws its map and votes from that head alone: the other KV heads have
  // nothing to add, and in the head's own group the other heads' columns are switched off through their offsets
  int rh = -1;
  if (c.ret_head) {  // (a table in global memory, written once at ltri_create: older than any predecessor in the chain)
    rh = c.ret_head[layer];
    if (rh >= 0 && g != rh / G) return;
  }
  const bool is_cur = (int)blockIdx.x >= n_local_groups;
  const int tile0 = (is_cur ? (int)blockIdx.x - n_local_groups : (int)blockIdx.x) * kMapKT;
  const int ntile = min(kMapKT, (is_cur ? n_cur_tiles : n_local_tiles) - tile0);
  // first key (absolute) of key tile kt, the end of the range, and the first query block that sees the tile
  const int kbase = is_cur ? a.t0 : a.loc_begin;
  const int key_end = is_cur ? a.t0 + a.n : a.t0;
  auto key0_of = [&](int kt) { return kbase + (tile0 + kt) * 128; };
  auto blk0_of = [&](int kt) { return is_cur ? ((tile0 + kt) * 128) / TPB : 0; };
  const int nblocks = (a.n + TPB - 1) / TPB;
  const int bmin = blk0_of(0);

  const uint32_t sbase = (smem_addr(smem_raw) + 1023u) & ~1023u;
  const uint32_t sK = sbase;                      // kMapKT x 32 KB: [tile][half d][128 keys][64]
  const uint32_t sQ = sbase + kMapKT * 32768;     // 2 stages x 32 KB: [half d][128 rows][64]
  // One more step of the contraction carries the rows' offsets (see kMapMargin): the key side is a constant tile of
  // ones, the query side holds off / c2 of the block's 128 rows split into four bf16 terms, so the accumulator comes
  // out as logit + off / c2 and the epilogue needs no per-column offsets.  Both are 128 x 16 K-major tiles without
  // swizzle: 8-row x 16-byte core matrices, the two core matrices of a row group 128 bytes apart, row groups 256.
  const uint32_t sXa = sQ + 65536;                // 4 KB
  const uint32_t sXb = sXa + 4096;                // 2 stages x 4 KB
  auto xoff = [](int r, int kc) -> uint32_t { return (uint32_t)((r >> 3) * 256 + kc * 128 + (r & 7) * 16); };
  enum { B_KFULL = 0, B_QFULL = 4, B_QEMPTY = 6, B_SFULL = 8, B_SEMPTY = 12 };
  auto bar = [&](int i) { return smem_addr(&bars[i]); };
  volatile int* abortp = &s_abort;
  if (tid == 0) {
    s_abort = 0;
    for (int s = 0; s < 2; ++s) {
      mbar_init(bar(B_QFULL + s), 2);  // the copies of a block's queries (with their byte count), then its offsets
      mbar_init(bar(B_QEMPTY + s), 1);
    }
    for (int s = 0; s < 4; ++s) {
      mbar_init(bar(B_KFULL + s), 1);
      mbar_init(bar(B_SFULL + s), 1);
      mbar_init(bar(B_SEMPTY + s), 16);
    }
    fence_mbar_init();
  }
  if (tid < 256) {  // ones in the first four K slots of every key row, zeros behind them; the query side's second
    const int r = tid >> 1, kc = tid & 1;  // core matrix (K slots 8..15) stays zero for good
    const uint32_t one2 = kc == 0 ? 0x3F803F80u : 0u;
    asm volatile("st.shared.v4.b32 [%0], {%1,%1,%2,%2};" ::"r"(sXa + xoff(r, kc)), "r"(one2), "r"(0u) : "memory");
    if (kc == 1) {
      asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(sXb + xoff(r, 1)), "r"(0u) : "memory");
      asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(sXb + 4096 + xoff(r, 1)), "r"(0u) : "memory");
    }
  }
  fence_async_smem();
  if (warp == 16) tmem_alloc(smem_addr(&s_tmem_base), 512);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem = s_tmem_base;
  chain_wait();  // everything above set up shared memory, barriers and TMEM only

  if (warp == 16) {
    // Every key tile has its own barrier, and the first one is asked for before anything else, the others behind the
    // first query block: the first product starts as soon as one tile and one block have landed.
    auto load_keys = [&](int kt) {
      // (local and current keys: window rows of the slab)
      const long long krow = (long long)(unit * c.Hkv + g) * c.SR + key0_of(kt) - (c.paged ? a.shift : 0);
      mbar_expect_tx(bar(B_KFULL + kt), 32768u);
      tma_load_2d(sK + kt * 32768, &maps.k128, 0, (int)krow, bar(B_KFULL + kt));
      tma_load_2d(sK + kt * 32768 + 16384, &maps.k128, 64, (int)krow, bar(B_KFULL + kt));
    };
    if (lane == 0) load_keys(0);
    // lane 0 starts the copies of a block's queries (and, behind the first block's, of the other key tiles); then
    // every lane writes the offsets of four of the block's 128 rows (row = (token, head)) and lane 0 publishes them
    // with the second arrival on the block's barrier
    const float* rq = c.rowq + (size_t)layer * c.chunk * c.Hq + g * G;
    const float inv_c2 = 1.0f / (c.scale * kLog2eM);
    int ok = 1;
    int it = 0;
    for (int blk = bmin; ok && blk < nblocks; ++blk, ++it) {
      const int st = it & 1;
      if (lane == 0 && it >= 2) ok = mbar_wait(bar(B_QEMPTY + st), ((it >> 1) - 1) & 1, abortp, c.wait_limit) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      if (lane == 0) {
        mbar_expect_tx(bar(B_QFULL + st), 32768);
        tma_load_3d(sQ + st * 32768, &maps.q, 0, g * G, l * a.n + blk * TPB, bar(B_QFULL + st));
        tma_load_3d(sQ + st * 32768 + 16384, &maps.q, 64, g * G, l * a.n + blk * TPB, bar(B_QFULL + st));
        if (it == 0)
          for (int kt = 1; kt < ntile; ++kt) load_keys(kt);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int row = lane + 32 * i;
        const int tk = blk * TPB + row / G;
        // rows past the call's end, and (under a retrieval head) the other heads' rows, get an offset that sends
        // every entry to zero
        float v = -30000.f;
        if (tk < a.n && (rh < 0 || g * G + row % G == rh)) v = fmaxf(__ldg(rq + (size_t)tk * c.Hq + row % G) * inv_c2, -30000.f);
        uint32_t w[2];
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          const __nv_bfloat16 h0 = __float2bfloat16_rn(v);
          v -= __bfloat162float(h0);
          const __nv_bfloat16 h1 = __float2bfloat16_rn(v);
          v -= __bfloat162float(h1);
          __nv_bfloat162 pr;
          pr.x = h0;
          pr.y = h1;
          w[t] = *reinterpret_cast<uint32_t*>(&pr);
        }
        asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%3};" ::"r"(sXb + st * 4096 + xoff(row, 0)), "r"(w[0]), "r"(w[1]),
                     "r"(0u)
                     : "memory");
      }
      fence_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_QFULL + st));
    }
    if (lane == 0)
      for (int back = 1; back <= 2 && back <= it; ++back) {  // no copy may be in flight at exit
        const int ii = it - back;
        if (!mbar_wait(bar(B_QEMPTY + (ii & 1)), (ii >> 1) & 1, abortp, c.wait_limit)) break;
      }
  } else if (warp == 17) {
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(128, 128, false);
      const uint64_t dK = make_desc(sK, 16, 1024), dQ = make_desc(sQ, 16, 1024);
      const uint64_t dXa = make_desc_noswizzle(sXa, 128, 256), dXb = make_desc_noswizzle(sXb, 128, 256);
      bool ok = true;
      int it = 0, seq = 0;
      for (int blk = bmin; ok && blk < nblocks; ++blk, ++it) {
        const int st = it & 1;
        ok = mbar_wait(bar(B_QFULL + st), (it >> 1) & 1, abortp, c.wait_limit);
        if (!ok) break;
        const uint64_t db = dQ + (uint64_t)((st * 32768) >> 4);
        for (int kt = 0; ok && kt < ntile; ++kt) {
          if (blk < blk0_of(kt)) continue;
          // the first product on a tile waits for the tile
          if (blk == max(bmin, blk0_of(kt))) ok = mbar_wait(bar(B_KFULL + kt), 0, abortp, c.wait_limit);
          if (!ok) break;
          const int buf = seq & 3;
          if (seq >= 4) ok = mbar_wait(bar(B_SEMPTY + buf), ((seq >> 2) - 1) & 1, abortp, c.wait_limit);
          if (!ok) break;
          fence_after_sync();
          const uint64_t da = dK + (uint64_t)((kt * 32768) >> 4);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const uint32_t off = ((ks >> 2) * 16384 + (ks & 3) * 32) >> 4;
            mma_ss(tmem + buf * 128, da + off, db + off, idesc, ks > 0);
          }
          mma_ss(tmem + buf * 128, dXa, dXb + (uint64_t)((st * 4096) >> 4), idesc, true);  // + off / c2 per column
          mma_commit(bar(B_SFULL + buf));
          ++seq;
        }
        if (!ok) break;
        mma_commit(bar(B_QEMPTY + st));
      }
    }
  } else {
    // epilogue: thread = key (TMEM lane), columns [32*cq, +32) of every block
    const int cq = warp >> 2;
    const int krel = (warp & 3) * 32 + lane;  // key inside its tile
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const float c2 = c.scale * kLog2eM;
    int* Mq = c.Mq + (size_t)layer * c.chunk * c.chunk;
    const int roff = a.t0 - a.reg_start;      // region index = call-relative token + roff
    long long total[kMapKT];
#pragma unroll
    for (int kt = 0; kt < kMapKT; ++kt) total[kt] = 0;
    bool ok = true;
    int it = 0, seq = 0;
    const float2 c2v = make_float2(c2, c2);
    const float2 sc = make_float2(kMapScale, kMapScale), mg = make_float2(12582912.f, 12582912.f);
    for (int blk = bmin; ok && blk < nblocks; ++blk, ++it) {
      const int tokb = blk * TPB;  // first token of the block (call-relative)
#pragma unroll
      for (int kt = 0; kt < kMapKT; ++kt) {
        if (kt >= ntile || blk < blk0_of(kt)) continue;
        const int buf = seq & 3;
        ok = ok && mbar_wait(bar(B_SFULL + buf), (seq >> 2) & 1, abortp, c.wait_limit);
        ++seq;
        if (!ok) break;
        fence_after_sync();
        uint32_t v[32];
        tmem_ld32(tmem + lane_base + buf * 128 + cq * 32, v);
        tmem_ld_wait();
        // the accumulator is in registers: hand the TMEM buffer back
        fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(B_SEMPTY + buf));
        // x = log2 of (probability * 2^20) + 1 + margin; the Q20 value is rint(2^x * kMapScale), rounded to nearest
        // even by adding 1.5 * 2^23: the integer sits in the mantissa.
        if (!is_cur) {
          // keys before the call: every row sees them, only the column sum (votes) is wanted.  The mantissa
          // integers are summed as raw bit patterns (modulo 2^32) and the bias is taken off once per group.
          // (No test for all-zero groups here: with thousands of visible keys a whole 8 x 32 group of entries
          // below half a Q20 unit is rare, and the test costs more than the exponentials it saves.)
          uint32_t bsum = 0;
#pragma unroll
          for (int e8 = 0; e8 < 32; e8 += 8) {
            float2 x[4];  // (the accumulator already holds logit + off / c2)
            x[0] = __fmul2_rn(make_float2(__uint_as_float(v[e8]), __uint_as_float(v[e8 + 1])), c2v);
            x[1] = __fmul2_rn(make_float2(__uint_as_float(v[e8 + 2]), __uint_as_float(v[e8 + 3])), c2v);
            x[2] = __fmul2_rn(make_float2(__uint_as_float(v[e8 + 4]), __uint_as_float(v[e8 + 5])), c2v);
            x[3] = __fmul2_rn(make_float2(__uint_as_float(v[e8 + 6]), __uint_as_float(v[e8 + 7])), c2v);
            {
              uint32_t part = 0u - 8u * 0x4B400000u;
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float2 y = __ffma2_rn(make_float2(ex2m(x[e].x), ex2m(x[e].y)), sc, mg);
                part += __float_as_uint(y.x) + __float_as_uint(y.y);
              }
              bsum += part;
            }
          }
          total[kt] += (long long)bsum;
          continue;
        }
        const int key0 = key0_of(kt);
        const int key = key0 + krel;
        const bool key_ok = key < key_end && key >= c.Ls;
        const int jrel = key - a.t0;  // call-relative
        const bool diag = tokb < (key0 - a.t0) + 128;  // some token of the block precedes some key
        int bsum = 0;
        int aq[32];
#pragma unroll
        for (int e8 = 0; e8 < 32; e8 += 8) {
          float2 x[4];
          x[0] = __fmul2_rn(make_float2(__uint_as_float(v[e8]), __uint_as_float(v[e8 + 1])), c2v);
          x[1] = __fmul2_rn(make_float2(__uint_as_float(v[e8 + 2]), __uint_as_float(v[e8 + 3])), c2v);
          x[2] = __fmul2_rn(make_float2(__uint_as_float(v[e8 + 4]), __uint_as_float(v[e8 + 5])), c2v);
          x[3] = __fmul2_rn(make_float2(__uint_as_float(v[e8 + 6]), __uint_as_float(v[e8 + 7])), c2v);
          // an entry with x < 0 rounds to zero: a group of eight columns whose x is negative on every lane of the
          // warp (common under the causal diagonal) needs no exponentials at all
          const float xm = fmaxf(fmaxf(fmax3(x[0].x, x[0].y, x[1].x), fmax3(x[1].y, x[2].x, x[2].y)),
                                 fmaxf(x[3].x, x[3].y));
          if (__any_sync(0xffffffffu, xm >= 0.f)) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float2 y = __ffma2_rn(make_float2(ex2m(x[e].x), ex2m(x[e].y)), sc, mg);
              aq[e8 + 2 * e] = __float_as_int(y.x) - 0x4B400000;
              aq[e8 + 2 * e + 1] = __float_as_int(y.y) - 0x4B400000;
            }
          } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) aq[e8 + e] = 0;
          }
        }
        if (diag) {
#pragma unroll
          for (int e = 0; e < 32; ++e)
            if (tokb + (cq * 32 + e) / G < jrel) aq[e] = 0;
        }
        // head sum per token (Eq. 4) -> region map; causality already zeroed the invalid entries
#pragma unroll
        for (int t = 0; t < 32 / G; ++t) {
          int sv = 0;
#pragma unroll
          for (int hh = 0; hh < G; ++hh) sv += aq[t * G + hh];
          bsum += sv;
          const int tk = tokb + (cq * 32) / G + t;
          if (key_ok && sv != 0 && tk < a.n) atomicAdd(&Mq[(size_t)(tk + roff) * c.chunk + (jrel + roff)], sv);
        }
        total[kt] += bsum;
      }
    }
    if (ok) {
#pragma unroll
      for (int kt = 0; kt < kMapKT; ++kt) {
        const int key = key0_of(kt) + krel;
        if (kt < ntile && key < key_end && key >= c.Ls && total[kt] != 0)
          atomicAdd((unsigned long long*)&c.votes[unit * c.Tpad + key], (unsigned long long)total[kt]);
      }
    }
  }
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  if (warp == 16) tmem_dealloc(tmem, 512);
  if (tid == 0 && s_abort) set_status(c, -6, 5000 + (int)blockIdx.x);
}

typedef CUresult (*EncodeFnM)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

template <int G>
static cudaError_t launch_map_tc_g(const DevCtx& c, const PrefillArgs& a, const void* kv_maps, cudaStream_t s) {
  static EncodeFnM enc = nullptr;
  if (!enc) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return cudaErrorNotSupported;
    enc = reinterpret_cast<EncodeFnM>(p);
  }
  MapMaps maps;
  memcpy(&maps.k128, static_cast<const CUtensorMap*>(kv_maps) + 4, sizeof(CUtensorMap));  // the 128-row box
  cuuint64_t dims[3] = {128, (cuuint64_t)c.Hq, (cuuint64_t)a.layer_count * a.n};
  cuuint64_t strides[2] = {256, (cuuint64_t)c.Hq * 256};
  cuuint32_t box[3] = {64, (cuuint32_t)G, (cuuint32_t)(128 / G)};
  cuuint32_t es[3] = {1, 1, 1};
  if (enc(&maps.q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<__nv_bfloat16*>(a.q), dims, strides, box, es,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  // (the region maps, which the kernel accumulates into with integer reductions, were cleared by the call's append
  // kernel)
  const int nloc = (a.loc_begin >= c.Ls) ? (a.t0 - a.loc_begin + 127) / 128 : 0;
  const int ncur = (a.n + 127) / 128;
  const int gloc = (nloc + kMapKT - 1) / kMapKT, gcur = (ncur + kMapKT - 1) / kMapKT;
  const int smem = kMapKT * 32768 + 65536 + 3 * 4096 + 1024;  // key tiles, two query stages, the offset tiles
  cudaFuncSetAttribute(k_map_tc<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  return launch_chained(k_map_tc<G>, dim3(gloc + gcur, c.Hkv, a.layer_count), dim3(kMapThreads), smem, s, c, a, gloc, nloc,
                        ncur, maps);
}

cudaError_t launch_map_pass_tc(const DevCtx& c, const PrefillArgs& a, const void* kv_maps, cudaStream_t s) {
  switch (c.G) {
    case 1: return launch_map_tc_g<1>(c, a, kv_maps, s);
    case 2: return launch_map_tc_g<2>(c, a, kv_maps, s);
    case 4: return launch_map_tc_g<4>(c, a, kv_maps, s);
    case 8: return launch_map_tc_g<8>(c, a, kv_maps, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace ltri
