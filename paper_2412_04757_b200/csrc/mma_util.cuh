// Warp-level tensor-core building blocks (ldmatrix + mma.sync m16n8k16 bf16) and cp.async staging with the
// 16-byte-chunk XOR swizzle used by every shared-memory tile of 128-element (256-byte) rows.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace ltri {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// byte offset of 16-byte chunk `chunk` (0..15) of row `row` inside a tile of 256-byte rows
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) { return row * 256 + ((chunk ^ (row & 7)) << 4); }

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// 16-byte async copy; src_bytes = 0 zero-fills the destination
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Load `rows` rows of 128 bf16 from global (row r at base + r*row_stride elements) into a swizzled tile;
// rows >= valid_rows are zero-filled.  All `nthreads` threads of the CTA take part.
__device__ __forceinline__ void load_tile_async(uint32_t tile_smem, const __nv_bfloat16* base, size_t row_stride,
                                                int rows, int valid_rows, int tid, int nthreads) {
  for (int i = tid; i < rows * 16; i += nthreads) {
    const int r = i >> 4, ch = i & 15;
    const bool ok = r < valid_rows;
    const __nv_bfloat16* src = base + (ok ? (size_t)r * row_stride : 0) + ch * 8;
    cp_async16(tile_smem + tile_off(r, ch), src, ok ? 16 : 0);
  }
}

// S[16 x 64] += A[16 x 128] * B[64 x 128]^T for one warp: A rows a_row0.. of the A tile, all 64 rows of the B tile.
__device__ __forceinline__ void warp_qk_16x64(float (&S)[8][4], uint32_t a_tile, int a_row0, uint32_t b_tile, int lane) {
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    uint32_t a[4];
    ldsm_x4(a, a_tile + tile_off(a_row0 + (lane & 15), ks * 2 + (lane >> 4)));
#pragma unroll
    for (int np = 0; np < 4; ++np) {
      uint32_t b[4];
      ldsm_x4(b, b_tile + tile_off(np * 16 + (lane & 7) + ((lane >> 4) << 3), ks * 2 + ((lane >> 3) & 1)));
      mma_bf16(S[2 * np], a, b[0], b[1]);
      mma_bf16(S[2 * np + 1], a, b[2], b[3]);
    }
  }
}

// Same as warp_qk_16x64 but only the first `npairs` pairs of 8-column tiles (16 columns each) are computed.
__device__ __forceinline__ void warp_qk_16xN(float (&S)[8][4], uint32_t a_tile, int a_row0, uint32_t b_tile, int lane,
                                             int npairs) {
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    uint32_t a[4];
    ldsm_x4(a, a_tile + tile_off(a_row0 + (lane & 15), ks * 2 + (lane >> 4)));
#pragma unroll
    for (int np = 0; np < 4; ++np) {
      if (np < npairs) {
        uint32_t b[4];
        ldsm_x4(b, b_tile + tile_off(np * 16 + (lane & 7) + ((lane >> 4) << 3), ks * 2 + ((lane >> 3) & 1)));
        mma_bf16(S[2 * np], a, b[0], b[1]);
        mma_bf16(S[2 * np + 1], a, b[2], b[3]);
      }
    }
  }
}

}  // namespace ltri
