// Prefill attention on the 5th-generation tensor cores (tcgen05.mma, TMEM accumulators, TMA-fed shared memory).
//
// One CTA owns 256 query rows of one (layer, KV head): two 128-row tiles Q0/Q1, each row = (token, head of the
// group), so one K/V tile serves the whole GQA group.  Keys arrive in 128-slot tiles assembled by TMA from pieces of
// 8..128 rows, which lets a tile be packed from several short spans ("span-indirect" tiles): every range is padded
// to a multiple of 8 rows only.  Roles (18 warps):
//   warps 0-7 / 8-15 : softmax of S0 / S1, two threads per row (64 columns each), P written back to TMEM as bf16
//   warp 16          : TMA producer (Q once, K/V pieces through a 2-stage ring)
//   warp 17          : MMA issuer: S = Q K^T (both operands in shared memory), O += P V (P from TMEM, V MN-major)
// TMEM columns: S0 [0,128) S1 [128,256) O0 [256,384) O1 [384,512); P (bf16) aliases columns [0,32) and [64,96) of
// its S: every softmax thread overwrites only logit columns it has already read.
// The issue order QK0, QK1, {PV0_j, QK0_j+1, PV1_j, QK1_j+1} keeps the tensor pipe busy with one tile's MMAs while
// the other tile's softmax runs.  The running max is updated lazily (only when it grows by more than 2^8), in which
// case the softmax thread rescales its O row in TMEM; the in-order tensor pipe guarantees the row is quiescent then.
// Every wait is bounded; on expiry the CTA sets LTRI_ETIMEOUT in the status word, drains and frees its TMEM.
#include <cuda.h>

#include <cstdlib>
#include <cstring>

#include "common.cuh"
#include "tc_util.cuh"

namespace ltri {

using namespace tc;

constexpr float kLog2eT = 1.4426950408889634f;
constexpr int kTcThreads = 576;  // 16 softmax warps + TMA producer + MMA issuer
constexpr int kNumBoxes = 5;  // box heights 8,16,32,64,128
constexpr float kRescaleThreshold = 24.0f;
// Largest exponent (log2 units) a probability may carry above the softmax reference in the regular launch: 2^90 times
// the 2^7 keys of a tile, the 2^13 tiles of the longest item and values of up to 2^10 still fits fp32 (and the bf16
// P operand).
constexpr float kLazyRange = 90.0f;

struct TcMaps {
  CUtensorMap q;             // [tokens][Hq][128] bf16, box {64, G, 256/G}
  CUtensorMap kv[kNumBoxes]; // K slabs followed by V slabs: [rows][128] bf16, box {64, 8<<i}
};
static_assert(sizeof(CUtensorMap) * (2 * kNumBoxes + 1) <= kTcMapBytes, "kTcMapBytes too small");

struct RangeList {
  int n;
  int start[kMaxTopK + 2];
  int len[kMaxTopK + 2];
};

// What the softmax threads need to know about a tile: which of its 128 key slots hold keys, and for the causal
// (current-chunk) tile the absolute token of slot 0 (-1 otherwise).
struct __align__(16) TileDesc {
  unsigned m0, m1, m2, m3;
  int causal_tok0;
  int full;  // all 128 slots valid and no causal masking
  int pad0, pad1;
};

// Deterministic tile builder: every role walks the same range list and derives the same tiles.  All state lives in
// registers (no dynamically indexed arrays); only the producer asks for the piece list.
struct TileIter {
  const RangeList* rg;
  int ri = 0, off = 0;
  int causal_ri;  // index of the causal (current-chunk) range, -1 if none
  // description of the current tile
  unsigned m0, m1, m2, m3;  // valid-slot mask
  int causal_tok0;          // absolute token of slot 0 when the tile is causal, else -1
  bool full;                // all 128 slots valid and no causal masking
  __device__ __forceinline__ void set_bits(int lo, int cnt) {
    const int hi = lo + cnt;
    auto word = [&](int w) -> unsigned {
      const int a = max(lo, 32 * w), b = min(hi, 32 * w + 32);
      if (b <= a) return 0u;
      const int n = b - a;
      return (n == 32 ? 0xffffffffu : ((1u << n) - 1u)) << (a - 32 * w);
    };
    m0 |= word(0);
    m1 |= word(1);
    m2 |= word(2);
    m3 |= word(3);
  }
  // Advances to the next tile.  f(slot, token, box_index) is called for every piece when PIECES is set.
  template <bool PIECES, typename F>
  __device__ __forceinline__ bool next(F&& f) {
    m0 = m1 = m2 = m3 = 0u;
    causal_tok0 = -1;
    int slot = 0;
    while (slot < 128 && ri < rg->n) {
      const int rem = rg->len[ri] - off;
      if (rem <= 0) {
        ++ri;
        off = 0;
        continue;
      }
      const bool causal = ri == causal_ri;
      if (causal && slot != 0 && causal_tok0 < 0) break;  // the causal range starts a fresh tile
      const int need = (rem + 7) & ~7;
      const int room = 128 - slot;
      const int lim = need < room ? need : room;
      int bi = 4;
      while ((8 << bi) > lim) --bi;
      const int h = 8 << bi;
      const int nvalid = h < rem ? h : rem;
      const int tok = rg->start[ri] + off;
      if (causal && slot == 0) causal_tok0 = tok;
      if (PIECES) f(slot, tok, bi);
      set_bits(slot, nvalid);
      off += nvalid;
      slot += h;
    }
    full = causal_tok0 < 0 && (m0 & m1 & m2 & m3) == 0xffffffffu;
    return slot > 0;
  }
  __device__ __forceinline__ bool next() {
    return next<false>([](int, int, int) {});
  }
  __device__ __forceinline__ unsigned mask(int w) const { return w == 0 ? m0 : w == 1 ? m1 : w == 2 ? m2 : m3; }
};

// Number of tiles the iterator yields for a range list: every range is padded to 8 rows and the causal range starts
// a fresh tile.
__device__ __forceinline__ int count_tiles(const RangeList* rg, int causal_ri) {
  int slots = 0;
  for (int i = 0; i < rg->n; ++i) {
    const int len = rg->len[i];
    if (len <= 0) continue;
    if (i == causal_ri) slots = (slots + 127) & ~127;
    slots += (len + 7) & ~7;
  }
  return (slots + 127) >> 7;
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// MERGE: the launch may be asked for phase 2 (kept out of the instantiation that runs phases 0 and 1, whose inner
// loop is sensitive to every register).
template <int G, bool EXCH, bool MERGE>
__global__ void __launch_bounds__(kTcThreads, 1)
    k_attn_tc(DevCtx c, PrefillArgs a, int phase, int final_out, int* __restrict__ redo,
              const __grid_constant__ TcMaps maps, long long v_row_offset) {
  constexpr int exch = EXCH ? 1 : 0;
  // exch = 0: the regular launch.  Its softmax reference moves one tile late (see the softmax role); a CTA in which
  // some tile outran that reference by more than the exponent range allows leaves redo[blockIdx.x] = 1.
  // exch = 1: the launch that follows it with the same grid.  A CTA whose flag is clear returns at once; one whose
  // flag is set walks its work items again with the true maximum exchanged on every tile and overwrites what the
  // first launch stored, so inputs of any magnitude get the exact softmax.
  if (exch) {
    chain_wait();
    if (redo[blockIdx.x] == 0) return;
  }
  const CUtensorMap* kvmaps = maps.kv;
  extern __shared__ unsigned char smem_raw[];
  // QFULL QFREE ODONE[0] | KFULL[2] VFULL[2] KEMPTY[2] VEMPTY[2] | SREADY[2] PREADY[2][2] OFREE[2] | ODONE[1]
  __shared__ __align__(8) unsigned long long bars[3 + 8 + 8 + 1];
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;
  __shared__ RangeList rg;            // key ranges of the work item the producer is walking
  __shared__ int s_item_tiles[3];     // tile count of the work items in flight (roles may be up to two items apart)
  __shared__ TileDesc s_td[8];        // per-tile masks, written by the producer, read by the softmax threads
  __shared__ int s_quit[2];
  __shared__ int s_redo;              // some tile of this CTA outran the late softmax reference
  __shared__ int s_items_ready;       // number of work items whose key ranges the producer has published
  __shared__ float s_max[2][2][2][128];  // per tile parity, Q tile, column half, row: partial maxima
  __shared__ float s_sum[2][2][128];     // per Q tile, column half, row: partial row sums (end of an item)
  constexpr int TOKB = 256 / G;  // tokens per work item
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // persistent CTA: work items (token block, KV head, layer) are dealt round-robin
  const int MB = (a.n + TOKB - 1) / TOKB;
  const int nitems = MB * c.Hkv * a.layer_count;
  const uint32_t sbase = (smem_addr(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = sbase;                 // 64 KB: [half d][256 rows][64]
  const uint32_t sKV = sbase + 65536;        // 2 stages x (K 32 KB | V 32 KB), each [half d][128 slots][64]
  enum {
    B_QFULL = 0, B_QFREE = 1, B_ODONE = 2, B_KFULL = 3, B_VFULL = 5, B_KEMPTY = 7, B_VEMPTY = 9, B_SREADY = 11,
    B_PREADY = 13,  // + 2 * part + q: the two 32-column chunks of a thread's probabilities are handed over separately
    B_OFREE = 17, B_ODONE1 = 19
  };
  auto bar = [&](int i) { return smem_addr(&bars[i]); };
  volatile int* abortp = &s_abort;

  if (tid == 0) {
    s_abort = 0;
    s_quit[0] = s_quit[1] = 0;
    s_redo = 0;
    s_items_ready = 0;
    rg.n = 0;
    mbar_init(bar(B_QFULL), 1);
    mbar_init(bar(B_QFREE), 1);
    mbar_init(bar(B_ODONE), 1);
    mbar_init(bar(B_ODONE1), 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(bar(B_KFULL + s), 1);
      mbar_init(bar(B_VFULL + s), 1);
      mbar_init(bar(B_KEMPTY + s), 1);
      mbar_init(bar(B_VEMPTY + s), 1);
      mbar_init(bar(B_SREADY + s), 1);
      mbar_init(bar(B_PREADY + s), 8);
      mbar_init(bar(B_PREADY + 2 + s), 8);
      mbar_init(bar(B_OFREE + s), 8);
    }
    fence_mbar_init();
  }
  // stale shared memory must never hold non-finite bit patterns: unfilled key slots are multiplied by P = 0
  for (uint32_t i = tid; i < 131072 / 16; i += kTcThreads)
    asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(sKV + i * 16), "r"(0) : "memory");
  fence_async_smem();
  if (warp == 16) tmem_alloc(smem_addr(&s_tmem_base), 512);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem = s_tmem_base;
  if (!exch) chain_wait();  // everything above set up shared memory, barriers and TMEM only
  const int causal_ri = phase == 0 ? 2 : -1;

  // decode a work item
  struct Item {
    int mb, g, l, layer, tok0;
    size_t unit, slab_row0;
  };
  auto decode = [&](int item) {
    Item w;
    w.mb = item % MB;
    w.g = (item / MB) % c.Hkv;
    w.l = item / (MB * c.Hkv);
    w.layer = a.layer_begin + w.l;
    w.tok0 = w.mb * TOKB;
    w.unit = unit_of(c, a.seq, w.layer);
    // phase 0 reads the K/V cache of the (sequence, layer, KV head); phase 1 the packed slab of the selected spans
    w.slab_row0 = phase == 0 ? (w.unit * c.Hkv + w.g) * (size_t)c.SR
                             : ((size_t)w.layer * c.Hkv + w.g) * (size_t)c.Rcap;
    return w;
  };

  // unnormalised O state between the two phases: one 128 x 128 fp32 block per (layer, item, Q tile)
  auto oacc_base = [&](const Item& w, int q) -> size_t {
    return ((((size_t)w.layer * MB + w.mb) * c.Hkv + w.g) * 2 + q) * (size_t)(128 * kD);
  };

  if (warp == 16) {
    // ------------------------------------------------------------------ TMA producer
    // Every lane walks the tile list; lane 0 owns the barrier bookkeeping and lanes 0-3 issue the copies of
    // (K low half, K high half, V low half, V high half) so that many small pieces do not serialise on one thread.
    int jt = 0, ok = 1;
    if (lane == 0) prefetch_tmap(&maps.q);
    for (int item = blockIdx.x, wi = 0; ok && item < nitems; item += gridDim.x, ++wi) {
      const Item w = decode(item);
      if (lane == 0) {
        // the Q buffer is free once every QK^T product of the previous item has completed
        if (wi > 0) ok = mbar_wait(bar(B_QFREE), (wi - 1) & 1, abortp, c.wait_limit) ? 1 : 0;
        // the key ranges of this item (the other roles read them after they have seen its Q tile arrive)
        const int last_tok = min(a.n, w.tok0 + TOKB) - 1;
        if (phase == 0) {
          rg.n = 3;
          rg.start[0] = 0;
          rg.len[0] = a.sink_end;
          rg.start[1] = a.loc_begin;
          rg.len[1] = a.t0 - a.loc_begin;
          rg.start[2] = a.t0;
          rg.len[2] = last_tok + 1;
        } else {
          rg.n = 1;
          rg.start[0] = 0;
          rg.len[0] = c.gcnt[(size_t)w.layer * c.Hkv + w.g];
        }
        // publish the item's tile count with a monotonic counter: a softmax thread may look for item wi only after
        // the Q tile of item wi+1 has arrived, so a parity barrier could not tell the two apart
        s_item_tiles[wi % 3] = count_tiles(&rg, causal_ri);
        __threadfence_block();
        *reinterpret_cast<volatile int*>(&s_items_ready) = wi + 1;
        if (ok) {
          mbar_expect_tx(bar(B_QFULL), 65536);
          tma_load_3d(sQ, &maps.q, 0, w.g * G, w.l * a.n + w.tok0, bar(B_QFULL));
          tma_load_3d(sQ + 32768, &maps.q, 64, w.g * G, w.l * a.n + w.tok0, bar(B_QFULL));
        }
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      __syncwarp();
      TileIter it;
      it.rg = &rg;
      it.causal_ri = causal_ri;
      int pslot[16], ptok[16], pbox[16];
      while (true) {
        int np = 0;
        // (pieces are addressed by slab row: in a sliding slab the ranges behind the sink sit at token - shift)
        if (!it.next<true>([&](int slot, int tok, int bi) {
              pslot[np] = slot;
              ptok[np] = (phase == 0 && c.paged && it.ri > 0) ? (int)(tok - a.shift) : tok;
              pbox[np] = bi;
              ++np;
            }))
          break;
        const int st = jt & 1;
        const uint32_t par = ((jt >> 1) - 1) & 1;
        uint32_t bytes = 0;
        for (int p = 0; p < np; ++p) bytes += (uint32_t)(8 << pbox[p]) * 256u;
        if (lane == 0) {
          if (jt >= 2) ok = mbar_wait(bar(B_KEMPTY + st), par, abortp, c.wait_limit) ? 1 : 0;
          if (ok) {
            // the tile's masks travel to the softmax threads through the barrier chain KFULL -> SREADY; slot jt & 7
            // was last read for tile jt - 8, whose softmax ended before K stage jt - 2 was released
            TileDesc& td = s_td[jt & 7];
            td.m0 = it.m0;
            td.m1 = it.m1;
            td.m2 = it.m2;
            td.m3 = it.m3;
            // a tile of the current chunk that ends at or before the item's first token is visible to every row
            const bool all_slots = (it.m0 & it.m1 & it.m2 & it.m3) == 0xffffffffu;
            const bool below = it.causal_tok0 >= 0 && all_slots && it.causal_tok0 + 127 <= a.t0 + w.tok0;
            td.causal_tok0 = below ? -1 : it.causal_tok0;
            td.full = (it.full || below) ? 1 : 0;
            mbar_expect_tx(bar(B_KFULL + st), bytes);
          }
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        const uint32_t sK = sKV + st * 65536, sV = sK + 32768;
        if (lane < 2)
          for (int p = 0; p < np; ++p)
            tma_load_2d(sK + lane * 16384 + (uint32_t)pslot[p] * 128u, &kvmaps[pbox[p]], lane * 64,
                        (int)((long long)w.slab_row0 + ptok[p]), bar(B_KFULL + st));
        if (lane == 0) {
          if (jt >= 2) ok = mbar_wait(bar(B_VEMPTY + st), par, abortp, c.wait_limit) ? 1 : 0;
          if (ok) mbar_expect_tx(bar(B_VFULL + st), bytes);
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        if (lane == 2 || lane == 3)
          for (int p = 0; p < np; ++p)
            tma_load_2d(sV + (lane - 2) * 16384 + (uint32_t)pslot[p] * 128u, &kvmaps[pbox[p]], (lane - 2) * 64,
                        (int)((long long)w.slab_row0 + ptok[p] + v_row_offset), bar(B_VFULL + st));
        ++jt;
      }
    }
    // drain: wait until the MMA warp has released the last stages so that no copy is in flight at exit
    if (lane == 0)
      for (int back = 1; back <= 2 && back <= jt; ++back) {
        const int jj = jt - back;
        if (!mbar_wait(bar(B_VEMPTY + (jj & 1)), (jj >> 1) & 1, abortp, c.wait_limit)) break;
      }
    __syncwarp();
  } else if (warp == 17) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = make_idesc(128, 128, false);
      constexpr uint32_t idesc_pv = make_idesc(128, 128, true);
      // descriptors differ only in their start-address field: build one per operand, then add constants
      // (the address field holds bytes/16 and cannot carry out for any shared-memory offset)
      const uint64_t dQ = make_desc(sQ, 16, 1024);
      const uint64_t dK = make_desc(sKV, 16, 1024);
      const uint64_t dV = make_desc(sKV + 32768, 16384, 1024);
      auto issue_qk = [&](int q, int st) {
        const uint64_t da = dQ + (uint64_t)((q * 16384) >> 4);
        const uint64_t db = dK + (uint64_t)((st * 65536) >> 4);
        const uint32_t d = tmem + q * 128;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint32_t half = ks >> 2, kin = (ks & 3) * 32;
          mma_ss(d, da + ((half * 32768 + kin) >> 4), db + ((half * 16384 + kin) >> 4), idesc_qk, ks > 0);
        }
        mma_commit(bar(B_SREADY + q));
      };
      auto issue_pv = [&](int q, int st, bool acc, int part) {
        // 16 keys per step: 2 KB down the V tile; N = 128 spans both 64-wide halves (LBO = 16 KB).  Part 0 takes the
        // key steps whose probabilities the softmax threads write first (keys [0,32) and [64,96)), part 1 the rest.
        const uint64_t db = dV + (uint64_t)((st * 65536) >> 4);
        const uint32_t d = tmem + 256 + q * 128, pa = tmem + q * 128;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int ks = (i & 1) + 2 * part + 4 * (i >> 1);
          // P of keys [64h, 64h+64) sits in the first 32 columns of column half h of the S buffer
          mma_ts(d, pa + ks * 8 + (ks >> 2) * 32, db + ((ks * 2048) >> 4), idesc_pv, acc || part > 0 || i > 0);
        }
      };
      int jt = 0;
      bool ok = true;
      // Across work items the two Q tiles stay half a tile apart: when the last P.V product of Q tile 0 has been
      // issued, the first QK^T product of the NEXT item's Q tile 0 follows at once if that item's queries and first
      // key tile have landed (pre = true), so Q tile 0's logits are ready when its softmax threads come back from
      // their epilogue, and the tensor pipe has work while Q tile 1 finishes the current item.  Each Q tile has its
      // own "accumulator complete" barrier for the same reason.
      bool pre = false;
      int T_pre = 0;
      for (int item = blockIdx.x, wi = 0; ok && item < nitems; item += gridDim.x, ++wi) {
        int T = T_pre;
        if (!pre) {
          ok = mbar_wait(bar(B_QFULL), wi & 1, abortp, c.wait_limit);
          if (!ok) break;
          T = *reinterpret_cast<volatile int*>(&s_item_tiles[wi % 3]);
        }
        if (T > 0) {
          if (!pre) {
            ok = mbar_wait(bar(B_KFULL + (jt & 1)), (jt >> 1) & 1, abortp, c.wait_limit);
            if (!ok) break;
            fence_after_sync();
            issue_qk(0, jt & 1);
          }
          issue_qk(1, jt & 1);
          mma_commit(bar(B_KEMPTY + (jt & 1)));
          if (T == 1) mma_commit(bar(B_QFREE));
        } else {
          mma_commit(bar(B_QFREE));
        }
        pre = false;
        const bool has_next = item + (int)gridDim.x < nitems;
        for (int j = 0; ok && j < T; ++j, ++jt) {
          const int st = jt & 1, nst = st ^ 1;
          const bool acc = (j > 0) || (phase == 1);
          ok = mbar_wait(bar(B_VFULL + st), (jt >> 1) & 1, abortp, c.wait_limit);
          if (!ok) break;
          ok = mbar_wait(bar(B_PREADY + 0), jt & 1, abortp, c.wait_limit);
          if (!ok) break;
          // the first P.V product of an item overwrites O: the previous item's epilogue must have read it
          if (j == 0 && wi > 0) {
            ok = mbar_wait(bar(B_OFREE + 0), (wi - 1) & 1, abortp, c.wait_limit);
            if (!ok) break;
          }
          fence_after_sync();
          issue_pv(0, st, acc, 0);
          ok = mbar_wait(bar(B_PREADY + 2), jt & 1, abortp, c.wait_limit);
          if (!ok) break;
          fence_after_sync();
          issue_pv(0, st, acc, 1);
          if (j + 1 < T) {
            ok = mbar_wait(bar(B_KFULL + nst), ((jt + 1) >> 1) & 1, abortp, c.wait_limit);
            if (!ok) break;
            fence_after_sync();
            issue_qk(0, nst);
          } else {
            mma_commit(bar(B_ODONE));
            if (has_next && mbar_try(bar(B_QFULL), (wi + 1) & 1)) {
              const int Tn = *reinterpret_cast<volatile int*>(&s_item_tiles[(wi + 1) % 3]);
              if (Tn > 0 && mbar_try(bar(B_KFULL + nst), ((jt + 1) >> 1) & 1)) {
                fence_after_sync();
                issue_qk(0, nst);
                pre = true;
                T_pre = Tn;
              }
            }
          }
          ok = mbar_wait(bar(B_PREADY + 1), jt & 1, abortp, c.wait_limit);
          if (!ok) break;
          if (j == 0 && wi > 0) {
            ok = mbar_wait(bar(B_OFREE + 1), (wi - 1) & 1, abortp, c.wait_limit);
            if (!ok) break;
          }
          fence_after_sync();
          issue_pv(1, st, acc, 0);
          ok = mbar_wait(bar(B_PREADY + 3), jt & 1, abortp, c.wait_limit);
          if (!ok) break;
          fence_after_sync();
          issue_pv(1, st, acc, 1);
          mma_commit(bar(B_VEMPTY + st));
          if (j + 1 < T) {
            issue_qk(1, nst);
            mma_commit(bar(B_KEMPTY + nst));
            if (j + 2 == T) mma_commit(bar(B_QFREE));  // the last QK^T products of the item are in flight
          }
        }
        if (!ok) break;
        if (T == 0) mma_commit(bar(B_ODONE));
        mma_commit(bar(B_ODONE1));
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue
    // Two threads per row: warps 0-7 serve Q tile 0, warps 8-15 Q tile 1; inside a tile warps 0-3 take the columns
    // [0,64) of S and O, warps 4-7 the columns [64,128).  A thread writes its probabilities over its own logit
    // columns only, so the halves need no ordering between the loads of one and the stores of the other.
    const int q = warp >> 3;
    const int half = (warp >> 2) & 1;
    const int r = (warp & 3) * 32 + lane;        // row inside the 128-row tile = TMEM lane
    const int rr = q * 128 + r;                  // row inside the work item
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + lane_base + q * 128 + half * 64;   // this thread's 64 logits
    const uint32_t tP = tS;  // its 64 probabilities (bf16 pairs) overwrite the first 32 of its own logit columns
    const uint32_t tO = tmem + lane_base + 256 + q * 128 + half * 64;
    const float c2 = c.scale * kLog2eT;
    int jt = 0;
    bool ok = true;
    for (int item = blockIdx.x, wi = 0; item < nitems; item += gridDim.x, ++wi) {
      const Item w = decode(item);
      const int tk = w.tok0 + rr / G;              // call-relative token
      const int h = w.g * G + rr % G;
      const bool row_ok = tk < a.n;
      const int layer = w.layer;
      if (ok) {
        // wait (bounded) until the producer has published this item's key ranges
        const long long t0c = clock64();
        while (*reinterpret_cast<volatile int*>(&s_items_ready) <= wi) {
          if (*abortp) {
            ok = false;
            break;
          }
          if (clock64() - t0c > c.wait_limit) {
            *abortp = 1;
            ok = false;
            break;
          }
        }
        __threadfence_block();
      }
      // collective decision per Q tile: either all 256 threads walk the item's tiles or all leave here, so the named
      // barriers below always see every thread
      if (!ok) s_quit[q] = 1;
      asm volatile("bar.sync %0, 256;" ::"r"(1 + q) : "memory");
      if (s_quit[q]) break;
      const int T = *reinterpret_cast<volatile int*>(&s_item_tiles[wi % 3]);
      float m_used = -INFINITY, lsum = 0.f;
      float2 stat0 = make_float2(0.f, 1.f);  // phase 2: reference maximum and row sum of the local part
      if (MERGE && phase == 2 && row_ok) {
        // the state this item is merged with at its end: fetch the statistics now (used after the tile loop) and pull
        // the accumulator rows into L2 (one request per 128-byte line: eight rows of a column group)
        stat0 = c.rowstat[((size_t)layer * c.chunk + tk) * c.Hq + h];
        if ((r & 7) == 0) {
          const float* op = c.Oacc + oacc_base(w, q) + (size_t)(half * 16) * 512 + r * 4;
#pragma unroll
          for (int i = 0; i < 16; ++i) asm volatile("prefetch.global.L2 [%0];" ::"l"(op + (size_t)i * 512));
        }
      }
      if (ok && phase == 1) {
        // continue from the state the local pass stored: running max, row sum and the unnormalised O row
        const float* op = c.Oacc + oacc_base(w, q) + (size_t)(half * 16) * 512 + r * 4;
        if (row_ok) {
          const float2 stt = c.rowstat[((size_t)layer * c.chunk + tk) * c.Hq + h];
          m_used = stt.x;
          lsum = half == 0 ? stt.y : 0.f;
        }
        // all sixteen 16-byte loads of the row half in flight at once, then two TMEM stores
        uint32_t v[2][32];
#pragma unroll
        for (int ch = 0; ch < 2; ++ch)
#pragma unroll
          for (int e = 0; e < 32; e += 4) {
            const float4 f = row_ok ? *reinterpret_cast<const float4*>(op + (size_t)(ch * 8 + (e >> 2)) * 512)
                                    : make_float4(0, 0, 0, 0);
            v[ch][e] = __float_as_uint(f.x);
            v[ch][e + 1] = __float_as_uint(f.y);
            v[ch][e + 2] = __float_as_uint(f.z);
            v[ch][e + 3] = __float_as_uint(f.w);
          }
        tmem_st32(tO, v[0]);
        tmem_st32(tO + 32, v[1]);
        tmem_st_wait();
      }
      int j = 0;
      const int row_abs = a.t0 + tk;
      bool need_ref = true;   // no reference maximum yet: the first tile exchanges the halves' maxima
      float mprev = -INFINITY;
      while (j < T) {
        // after an expired wait every thread keeps walking the item's tiles (without computing) so that the named
        // barrier is still reached by all 256 threads of the tile
        ok = ok && mbar_wait(bar(B_SREADY + q), jt & 1, abortp, c.wait_limit);
        if (!ok) {
          if (need_ref) asm volatile("bar.sync %0, 256;" ::"r"(1 + q) : "memory");
          need_ref = EXCH;
          ++j;
          ++jt;
          continue;
        }
        fence_after_sync();
        uint32_t v[2][32];
        tmem_ld32(tS, v[0]);
        tmem_ld32(tS + 32, v[1]);
        tmem_ld_wait();
        const TileDesc& td = s_td[jt & 7];
        if (!td.full) {
          // valid-slot bits, and for the causal tile the last visible column of this row (keys are consecutive
          // tokens from slot 0): column c is visible iff c <= lim
          const int ctok = td.causal_tok0;
          const int lim = ctok >= 0 ? row_abs - ctok - half * 64 : 127;
          const uint2 mks = *reinterpret_cast<const uint2*>(&td.m0 + half * 2);
          if (MERGE) {
            // (the form that measured faster in this instantiation; the other one in the other)
            // one bit per column: the slot holds a key and the key is visible to this row
            const unsigned vis0 = lim >= 31 ? 0xffffffffu : (lim < 0 ? 0u : (2u << lim) - 1u);
            const unsigned vis1 = lim >= 63 ? 0xffffffffu : (lim < 32 ? 0u : (2u << (lim - 32)) - 1u);
#pragma unroll
            for (int ch = 0; ch < 2; ++ch) {
              const unsigned mk = ch == 0 ? (mks.x & vis0) : (mks.y & vis1);
#pragma unroll
              for (int e = 0; e < 32; ++e)
                if (!((mk >> e) & 1u)) v[ch][e] = 0xff800000u;  // -inf
            }
          } else {
#pragma unroll
            for (int ch = 0; ch < 2; ++ch) {
              const unsigned mk = ch == 0 ? mks.x : mks.y;
#pragma unroll
              for (int e = 0; e < 32; ++e)
                if (!((mk >> e) & 1u) || ch * 32 + e > lim) v[ch][e] = 0xff800000u;  // -inf
            }
          }
        }
        // maximum of this thread's 64 logits (four independent chains)
        float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int ch = 0; ch < 2; ++ch)
#pragma unroll
          for (int e = 0; e < 32; e += 8) {
#pragma unroll
            for (int u = 0; u < 4; ++u)
              mx[u] = max3(mx[u], __uint_as_float(v[ch][e + 2 * u]), __uint_as_float(v[ch][e + 2 * u + 1]));
          }
        const float mloc = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
        // The two threads of a row must scale by the same reference.  On an item's first tile (no reference yet)
        // they exchange their maxima through shared memory and a named barrier.  On later tiles the reference moves
        // one tile late: it is the maximum over the previous tiles, whose partner half is already visible (the
        // partner stored it before its PREADY arrival of the previous tile, which precedes this tile's SREADY), so
        // no barrier sits between the logits and the exponentials.  A tile that exceeds the late reference only
        // makes the exponent positive; if it does so by more than kLazyRange the probabilities may overflow, so the
        // thread flags the CTA for the second launch, in which every tile exchanges its maxima like the first one
        // and the exponent never exceeds the lazy threshold.
        s_max[jt & 1][q][half][r] = mloc;
        float mt;
        if (need_ref) {
          asm volatile("bar.sync %0, 256;" ::"r"(1 + q) : "memory");
          mt = fmaxf(mloc, s_max[jt & 1][q][half ^ 1][r]) * c2;
        } else {
          mt = fmaxf(mprev, s_max[(jt & 1) ^ 1][q][half ^ 1][r]) * c2;
          if (mloc > -INFINITY && !(mloc * c2 - m_used <= kLazyRange)) *reinterpret_cast<volatile int*>(&s_redo) = 1;
        }
        need_ref = EXCH;
        mprev = mloc;
        // lazy running maximum: move it only when it grows by more than the threshold (or on first use)
        float alpha = 1.f;
        const bool grow = mt > m_used + kRescaleThreshold || (m_used == -INFINITY && mt > -INFINITY);
        if (grow) {
          alpha = ex2(m_used - mt);  // 0 when m_used = -inf
          m_used = mt;
          lsum *= alpha;
        }
        const bool have_o = (j > 0) || (phase == 1);
        if (have_o && __any_sync(0xffffffffu, grow)) {
#pragma unroll 1
          for (int ch = 0; ch < 4; ++ch) {
            uint32_t wv[16];
            tmem_ld16(tO + ch * 16, wv);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 16; ++e) wv[e] = __float_as_uint(__uint_as_float(wv[e]) * alpha);
            tmem_st16(tO + ch * 16, wv);
          }
          tmem_st_wait();
        }
        // probabilities, row sum, P (bf16).  Masked entries are -inf -> exp2 gives 0.
        const float mneg = m_used == -INFINITY ? 0.f : -m_used;
        const float2 c2v = make_float2(c2, c2), mnv = make_float2(mneg, mneg);
        float2 ls = make_float2(0.f, 0.f);
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          uint32_t pk[16];
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            // packed fp32x2 arithmetic: one FFMA2 and one FADD2 per pair of logits
            const float2 x =
                __ffma2_rn(make_float2(__uint_as_float(v[ch][e]), __uint_as_float(v[ch][e + 1])), c2v, mnv);
            const float2 pp = make_float2(ex2(x.x), ex2(x.y));
            ls = __fadd2_rn(ls, pp);
            pk[e >> 1] = pack2(pp.x, pp.y);
          }
          tmem_st16(tP + ch * 16, pk);
          // hand this chunk over: the P.V product starts on it while the other chunk's exponentials run
          tmem_st_wait();
          fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(B_PREADY + 2 * ch + q));
        }
        lsum += ls.x + ls.y;
        ++j;
        ++jt;
      }
      // epilogue: the two halves of a row exchange their partial sums, then each writes its 64 output columns
      s_sum[q][half][r] = lsum;
      asm volatile("bar.sync %0, 256;" ::"r"(1 + q) : "memory");
      lsum += s_sum[q][half ^ 1][r];
      if (ok) ok = mbar_wait(bar(q ? B_ODONE1 : B_ODONE), wi & 1, abortp, c.wait_limit);
      if (!ok) s_quit[q] = 1;
      asm volatile("bar.sync %0, 256;" ::"r"(1 + q) : "memory");  // also: s_sum is reused by the next item
      if (s_quit[q]) break;  // collective decision: all 256 threads of the tile leave after the same item
      fence_after_sync();
      if (phase == 0 && row_ok && half == 0) {
        c.rowstat[((size_t)layer * c.chunk + tk) * c.Hq + h] = make_float2(m_used, lsum);
        c.rowq[((size_t)layer * c.chunk + tk) * c.Hq + h] = -m_used - __log2f(lsum) + (21.0f + kMapMargin);
      }
      const bool have_o = (j > 0) || (phase == 1);
      if (MERGE && phase == 2) {
        // merge of two partial softmaxes: the local part (reference m0, row sum l0, accumulator O0 in global memory)
        // and the retrieved part just computed (m_used, lsum, accumulator in TMEM)
        const float M = fmaxf(stat0.x, m_used);
        const float a0 = ex2(stat0.x - M), a1 = m_used == -INFINITY ? 0.f : ex2(m_used - M);
        const float inv = 1.f / fmaf(stat0.y, a0, lsum * a1);
        const float w0 = a0 * inv, w1 = a1 * inv;
        const float* op0 = c.Oacc + oacc_base(w, q) + (size_t)(half * 16) * 512 + r * 4;
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          float4 o0[8];
#pragma unroll
          for (int i = 0; i < 8; ++i)
            o0[i] = row_ok ? *reinterpret_cast<const float4*>(op0 + (size_t)(ch * 8 + i) * 512) : make_float4(0, 0, 0, 0);
          uint32_t ov[32];
          if (have_o) {
            tmem_ld32(tO + ch * 32, ov);
            tmem_ld_wait();
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) ov[e] = 0u;
          }
          if (ch == 1) {  // O is in registers: the next item's first P.V product may overwrite the accumulator
            fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(B_OFREE + q));
          }
          if (row_ok) {
            __nv_bfloat16* op = a.out + (((size_t)w.l * a.n + tk) * c.Hq + h) * kD + half * 64 + ch * 32;
#pragma unroll
            for (int e = 0; e < 32; e += 8) {
              const float4 x0 = o0[e >> 2], x1 = o0[(e >> 2) + 1];
              uint4 wv;
              wv.x = pack2(fmaf(x0.x, w0, __uint_as_float(ov[e]) * w1), fmaf(x0.y, w0, __uint_as_float(ov[e + 1]) * w1));
              wv.y = pack2(fmaf(x0.z, w0, __uint_as_float(ov[e + 2]) * w1), fmaf(x0.w, w0, __uint_as_float(ov[e + 3]) * w1));
              wv.z = pack2(fmaf(x1.x, w0, __uint_as_float(ov[e + 4]) * w1), fmaf(x1.y, w0, __uint_as_float(ov[e + 5]) * w1));
              wv.w = pack2(fmaf(x1.z, w0, __uint_as_float(ov[e + 6]) * w1), fmaf(x1.w, w0, __uint_as_float(ov[e + 7]) * w1));
              *reinterpret_cast<uint4*>(op + e) = wv;
            }
          }
        }
        continue;
      }
      const float inv = 1.f / lsum;
      uint32_t ov[2][32];
      if (have_o) {
        tmem_ld32(tO, ov[0]);
        tmem_ld32(tO + 32, ov[1]);
        tmem_ld_wait();
      } else {
#pragma unroll
        for (int e = 0; e < 32; ++e) ov[0][e] = ov[1][e] = 0u;
      }
      // O is in registers: the next item's first P.V product may overwrite the accumulator
      fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_OFREE + q));
      if (row_ok) {
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          if (phase == 0 && !final_out) {
            // scratch layout [4-float column group][row][4]: the 32 rows of a warp write 512 contiguous bytes
            float* op = c.Oacc + oacc_base(w, q) + (size_t)(half * 16 + ch * 8) * 512 + r * 4;
#pragma unroll
            for (int e = 0; e < 32; e += 4)
              *reinterpret_cast<uint4*>(op + (size_t)(e >> 2) * 512) =
                  make_uint4(ov[ch][e], ov[ch][e + 1], ov[ch][e + 2], ov[ch][e + 3]);
          }
          if (final_out) {
            __nv_bfloat16* op = a.out + (((size_t)w.l * a.n + tk) * c.Hq + h) * kD + half * 64 + ch * 32;
#pragma unroll
            for (int e = 0; e < 32; e += 8) {
              uint4 wv;
              wv.x = pack2(__uint_as_float(ov[ch][e]) * inv, __uint_as_float(ov[ch][e + 1]) * inv);
              wv.y = pack2(__uint_as_float(ov[ch][e + 2]) * inv, __uint_as_float(ov[ch][e + 3]) * inv);
              wv.z = pack2(__uint_as_float(ov[ch][e + 4]) * inv, __uint_as_float(ov[ch][e + 5]) * inv);
              wv.w = pack2(__uint_as_float(ov[ch][e + 6]) * inv, __uint_as_float(ov[ch][e + 7]) * inv);
              *reinterpret_cast<uint4*>(op + e) = wv;
            }
          }
        }
      }
    }
  }
  // ------------------------------------------------------------------ teardown
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  if (warp == 16) tmem_dealloc(tmem, 512);
  if (tid == 0 && s_abort) set_status(c, -6, (int)blockIdx.x);
  if (tid == 0) redo[blockIdx.x] = exch ? 0 : s_redo;  // (the second launch leaves the flags clear for the next call)
}

// ---------------------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeFn get_encode() {
  static EncodeFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeFn>(p);
  }
  return fn;
}

// K/V tensor maps of a context (box heights 8..128); `out` receives kNumBoxes CUtensorMap objects (host memory).
bool tc_encode_kv_maps(const DevCtx& c, void* out_bytes) {
  EncodeFn enc = get_encode();
  if (!enc) return false;
  CUtensorMap* out = static_cast<CUtensorMap*>(out_bytes);
  const cuuint64_t rows = (cuuint64_t)c.NS * c.NL * c.Hkv * (cuuint64_t)c.SR * 2;  // K slabs then V slabs
  for (int i = 0; i < kNumBoxes; ++i) {
    cuuint64_t dims[2] = {128, rows};
    cuuint64_t strides[1] = {256};
    cuuint32_t box[2] = {64, (cuuint32_t)(8 << i)};
    cuuint32_t es[2] = {1, 1};
    if (enc(&out[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, c.Kc, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  }
  // maps 6..10: the packed slabs of the selected spans (K slabs then V slabs), same box heights
  for (int i = 0; i < kNumBoxes; ++i) {
    cuuint64_t dims[2] = {128, (cuuint64_t)c.NL * c.Hkv * (cuuint64_t)c.Rcap * 2};
    cuuint64_t strides[1] = {256};
    cuuint32_t box[2] = {64, (cuuint32_t)(8 << i)};
    cuuint32_t es[2] = {1, 1};
    if (enc(&out[kNumBoxes + 1 + i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, c.Kg, dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  }
  // sixth map: the span index K^R, [rows][128] bf16 in 128-row boxes
  {
    cuuint64_t dims[2] = {128, (cuuint64_t)c.NS * c.NL * c.Hkv * (cuuint64_t)c.cap};
    cuuint64_t strides[1] = {256};
    cuuint32_t box[2] = {64, 128};
    cuuint32_t es[2] = {1, 1};
    if (enc(&out[kNumBoxes], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, c.KR, dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  }
  return true;
}

bool tc_attention_supported(const DevCtx& c) {
  // the V slabs must follow the K slabs directly (one tensor map covers both) and row indices must fit 31 bits
  const size_t rows = (size_t)c.NS * c.NL * c.Hkv * (size_t)c.SR;
  if (c.Vc != c.Kc + rows * kD) return false;
  if (rows * 2 >= (1ull << 31)) return false;
  const size_t grows = (size_t)c.NL * c.Hkv * (size_t)c.Rcap;
  if (c.Vg != c.Kg + grows * kD || grows * 2 >= (1ull << 31)) return false;
  return get_encode() != nullptr;
}

template <int G, bool MERGE>
static cudaError_t launch_tc_g(const DevCtx& c, const PrefillArgs& a, int phase, bool final_out, const void* kv_maps,
                               cudaStream_t s) {
  TcMaps maps;
  EncodeFn enc = get_encode();
  if (!enc || !kv_maps) return cudaErrorNotSupported;
  memcpy(maps.kv, static_cast<const CUtensorMap*>(kv_maps) + (phase == 0 ? 0 : kNumBoxes + 1), sizeof(maps.kv));
  {
    cuuint64_t dims[3] = {128, (cuuint64_t)c.Hq, (cuuint64_t)a.layer_count * a.n};
    cuuint64_t strides[2] = {256, (cuuint64_t)c.Hq * 256};
    cuuint32_t box[3] = {64, (cuuint32_t)G, (cuuint32_t)(256 / G)};
    cuuint32_t es[3] = {1, 1, 1};
    if (enc(&maps.q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<__nv_bfloat16*>(a.q), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
  }
  constexpr int TOKB = 256 / G;
  const int smem = 65536 + 131072 + 1024;
  cudaFuncSetAttribute(k_attn_tc<G, false, MERGE>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  cudaFuncSetAttribute(k_attn_tc<G, true, MERGE>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  const long long v_off = phase == 0 ? (long long)c.NS * c.NL * c.Hkv * c.SR : (long long)c.NL * c.Hkv * c.Rcap;
  static int sms = 0;
  if (sms == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
  }
  int ctas = sms;
  // testing aid: fewer CTAs make every CTA walk several work items even on small problems
  if (const char* cap = getenv("LTRI_TC_MAX_CTAS")) ctas = max(1, min(sms, atoi(cap)));
  // persistent CTAs: one per SM (the kernel needs the whole TMEM and most of the shared memory of an SM)
  const int nitems = ((a.n + TOKB - 1) / TOKB) * c.Hkv * a.layer_count;
  // the regular launch, then the one that redoes the work of the CTAs that asked for it (they return at once otherwise)
  const int grid = min(nitems, ctas);
  if (grid > kTcMaxCtas) return cudaErrorInvalidValue;
  launch_chained(k_attn_tc<G, false, MERGE>, dim3(grid), dim3(kTcThreads), smem, s, c, a, phase, final_out ? 1 : 0,
                 c.tc_redo, maps, v_off);
  return launch_chained(k_attn_tc<G, true, MERGE>, dim3(grid), dim3(kTcThreads), smem, s, c, a, phase, final_out ? 1 : 0,
                        c.tc_redo, maps, v_off);
}

cudaError_t launch_attn_prefill_tc(const DevCtx& c, const PrefillArgs& a, int phase, bool final_out,
                                   const void* kv_maps, cudaStream_t s) {
  switch (c.G) {
    case 1: return phase == 2 ? launch_tc_g<1, true>(c, a, phase, final_out, kv_maps, s) : launch_tc_g<1, false>(c, a, phase, final_out, kv_maps, s);
    case 2: return phase == 2 ? launch_tc_g<2, true>(c, a, phase, final_out, kv_maps, s) : launch_tc_g<2, false>(c, a, phase, final_out, kv_maps, s);
    case 4: return phase == 2 ? launch_tc_g<4, true>(c, a, phase, final_out, kv_maps, s) : launch_tc_g<4, false>(c, a, phase, final_out, kv_maps, s);
    case 8: return phase == 2 ? launch_tc_g<8, true>(c, a, phase, final_out, kv_maps, s) : launch_tc_g<8, false>(c, a, phase, final_out, kv_maps, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace ltri
