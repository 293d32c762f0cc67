// Warp-level pieces shared by the strided-attention kernels that run on mma.sync (Sec. 3.3): tile geometry,
// asynchronous tile loads, ldmatrix operand fetches and the m16n8k16 product with its published fragment layouts.
#pragma once
#include <cuda_bf16.h>

#include <cstdint>

namespace mst_attn {

constexpr int D = 64;        // head dimension
constexpr int TS = 64;       // tile side (queries and keys)
constexpr int BW_THREADS = 128;
constexpr int LDB = 72;      // row pitch of the bf16 tiles in shared memory (64 + 8: rows 144 bytes apart, no bank aliasing)
constexpr int LDF = 68;      // row pitch of the fp32 tiles
constexpr float SCALE = 0.125f;   // 1 / sqrt(64)

// One tile copy with the thread's share of the address arithmetic done by the caller: `dst_thread` = shared
// address of piece (threadIdx.x / 8, threadIdx.x % 8) of the tile, `src_thread` = that piece of the tile's first rows
// in global memory; thread t of THREADS copies the pieces THREADS / 8 rows apart
template <int THREADS>
__device__ __forceinline__ void copy_tile_async(uint32_t dst_thread, const __nv_bfloat16* src_thread, int64_t ld) {
#pragma unroll
  for (int k = 0; k < TS * 8 / THREADS; ++k)
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_thread + (uint32_t)(k * (THREADS / 8) * LDB * 2)),
                 "l"(src_thread + k * (THREADS / 8) * ld)
                 : "memory");
}
// rows [r0, r0 + 64) of one head's 64 columns -> dst[64][LDB] (row-major, bf16), issued asynchronously by the BW_THREADS
// threads of a block (cp.async, 16 bytes per request); complete after async_wait_all + a barrier
__device__ __forceinline__ void load_tile_async(__nv_bfloat16* dst, const __nv_bfloat16* src, int64_t ld, int64_t r0) {
  const int r = threadIdx.x >> 3, c = (threadIdx.x & 7) * 8;
  copy_tile_async<BW_THREADS>((uint32_t)__cvta_generic_to_shared(dst + r * LDB + c), src + (r0 + r) * ld + c, ld);
}
__device__ __forceinline__ void load_floats_async(float* dst, const float* src, int n) {
  for (int e = threadIdx.x; e < n; e += BW_THREADS) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst + e);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(d), "l"(src + e) : "memory");
  }
}
__device__ __forceinline__ void async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

// Warp-level tensor-core pieces (mma.sync m16n8k16, bf16 in, fp32 accumulate) with the published fragment layouts:
// with g = lane / 4 and t = lane % 4, an accumulator tile (16 x 8) holds rows g, g + 8 and columns 2t, 2t + 1 in its
// four registers, and an A operand (16 x 16, row-major) holds the same rows and columns 2t, 2t + 1, 2t + 8, 2t + 9 —
// so two neighbouring accumulator tiles, rounded to bf16, ARE the A operand of the next product and the scores never
// leave the registers.
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const __nv_bfloat16* p) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], const __nv_bfloat16* p) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
constexpr float SCALE_LOG2E = SCALE * 1.4426950408889634f;   // exp(s / sqrt(d) - lse) = 2^(s * SCALE_LOG2E - lse * log2(e))
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}
// A operand: rows r0 .. r0 + 16, columns 16 kb .. 16 kb + 16 of a bf16 tile with row pitch LDB
__device__ __forceinline__ void load_a(uint32_t (&a)[4], const __nv_bfloat16* tile, int r0, int kb, int lane) {
  ldsm_x4(a, tile + (r0 + (lane & 7) + ((lane >> 3) & 1) * 8) * LDB + kb * 16 + (lane >> 4) * 8);
}
// c[nb][16 x 8] += A strip (four k-steps over the 64 head dimensions, in registers) * rows n0 + 8 nb .. + 8 of `tile`,
// transposed, for NB neighbouring blocks of eight rows at once, k-step by k-step, so that consecutive products go to
// different accumulators and none waits for the one issued just before it
template <int NB>
__device__ __forceinline__ void mma_rows_wide(float (&c)[NB][4], const uint32_t (&a)[4][4], const __nv_bfloat16* tile, int n0, int lane) {
#pragma unroll
  for (int k2 = 0; k2 < 2; ++k2) {
    uint32_t b[NB][4];
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) ldsm_x4(b[nb], tile + (n0 + nb * 8 + (lane & 7)) * LDB + k2 * 32 + (lane >> 3) * 8);
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) mma_bf16(c[nb], a[2 * k2], b[nb][0], b[nb][1]);
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) mma_bf16(c[nb], a[2 * k2 + 1], b[nb][2], b[nb][3]);
  }
}
// acc[16 x 64] += A (16 x 16, in registers) * rows k0 .. k0 + 16 of `tile` (64 columns)
__device__ __forceinline__ void mma_cols(float (&acc)[8][4], const uint32_t (&a)[4], const __nv_bfloat16* tile, int k0, int lane) {
#pragma unroll
  for (int n2 = 0; n2 < 4; ++n2) {
    uint32_t b[4];
    ldsm_x4_t(b, tile + (k0 + (lane & 7) + ((lane >> 3) & 1) * 8) * LDB + n2 * 16 + (lane >> 4) * 8);
    mma_bf16(acc[2 * n2], a, b[0], b[1]);
    mma_bf16(acc[2 * n2 + 1], a, b[2], b[3]);
  }
}
// accumulators (16 x 64) -> fp32 tile in shared memory, rows r0 .. r0 + 16
__device__ __forceinline__ void store_acc(float* out, const float (&acc)[8][4], int r0, int lane) {
  const int g = lane >> 2, t = lane & 3;
#pragma unroll
  for (int nb = 0; nb < 8; ++nb) {
    *reinterpret_cast<float2*>(out + (r0 + g) * LDF + nb * 8 + 2 * t) = make_float2(acc[nb][0], acc[nb][1]);
    *reinterpret_cast<float2*>(out + (r0 + g + 8) * LDF + nb * 8 + 2 * t) = make_float2(acc[nb][2], acc[nb][3]);
  }
}

}  // namespace mst_attn
