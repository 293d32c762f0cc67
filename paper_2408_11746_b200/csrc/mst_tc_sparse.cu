// Forward and input gradient on the structured-sparse tensor-core instruction (tcgen05.mma.sp, 2:4 along K).
//
//   out[t, r] = sum_k in[t, k] * S[r, k]        S = W.M (forward: r = output feature, k = input feature)
//                                               S = (W.M)^T (input gradient: r = input feature, k = output feature)
//
// An unstructured mask of density d <= 0.1 has at most two entries in all but a few of its groups of four
// consecutive k: (1 - d)^4 + 4 d (1 - d)^3 + 6 d^2 (1 - d)^2 of the groups conform (99.6 % at d = 0.1).  S is split
// into a 2:4-conforming part (the first two entries of every group) and a spill list (third and fourth entries).
// The conforming part runs at the sparse rate of the tensor cores: it is the A operand, stored compressed
// ([rows x K/2] bf16, K-major) with its 2-bit position metadata in tensor memory; the activations are the B operand,
// read as stored.  The accumulator therefore holds the TRANSPOSE of the output tile (lanes = rows of S = output
// features, columns = tokens); the epilogue adds the spill entries of its row from a feature-major copy of the
// activation columns they touch, and writes 64-byte runs of the token-major output rows (32 consecutive features of
// one token per store instruction).  Every product is an exact bf16 x bf16 product accumulated in fp32, as on the
// dense path.
//
// Kernel: clusters of two blocks (an SM pair) share a 256 (rows of S) x 240 (tokens) tile with
// tcgen05.mma.sp.cta_group::2.  Per 128-deep K block a block loads its 128 compressed rows (16 KB), its 120 tokens of
// activations (two 64-wide swizzled boxes), and the 2 KB of metadata of its rows, which the MMA-issuing thread copies
// into tensor memory (tcgen05.cp) right before the four K = 32 instructions that use it.  Two 240-column
// accumulators (tile i's epilogue overlaps tile i+1's main loop) and two 4-column metadata slots fill 488 of the 512
// tensor-memory columns, which is why the token tile is 240 and not 256.  Roles, barriers and bounded waits are those
// of the dense contraction kernel (mst_tc_gemm.cu).
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstdlib>

#include "mst_internal.cuh"
#include "mst_tc_gemm.cuh"
#include "mst_tc_ptx.cuh"

namespace {

using namespace mst_ptx;

constexpr int SM_ROWS = 128;           // rows of S per block (256 per pair)
constexpr int SN = 240;                // tokens per tile; each block of the pair loads SN / 2
constexpr int SKB = 128;               // logical K per stage (64 compressed elements = one 128-byte swizzled row)
constexpr int S_STAGES = 4;
constexpr int SA_BYTES = SM_ROWS * (SKB / 2) * 2;       // 16 KiB
constexpr int SB_BOX_BYTES = (SN / 2) * 64 * 2;         // 15 KiB: 120 tokens x 64 k
constexpr int SB_BOX_STRIDE = SB_BOX_BYTES;             // 15 KiB: still a multiple of 1024 bytes (swizzle atoms)
constexpr int SE_BYTES = 128 * 16;                      // metadata of 128 rows x 128 k
constexpr int S_STAGE_BYTES = SA_BYTES + 2 * SB_BOX_STRIDE + SE_BYTES;   // 48 KiB
constexpr int S_TX_BYTES = SA_BYTES + 2 * SB_BOX_BYTES + SE_BYTES;
constexpr int S_EPI_WARPS = 8;
constexpr int S_THREADS = 64 + 32 * S_EPI_WARPS;
constexpr int S_CHUNK = 16;                             // tokens per epilogue step
constexpr int S_FAST_SPILLS = 4;                        // spills per row whose activations are fetched one step ahead
constexpr int S_TMEM_COLS = 512;
constexpr int S_META_COL = 2 * SN;                      // metadata slots behind the two accumulators
constexpr size_t S_SMEM_BYTES = (size_t)S_STAGES * S_STAGE_BYTES + 1024 + 256;
constexpr int XR_TOK = 64;                              // token tile of the feature-major column copy

__device__ int g_sp_error = 0;  // sticky: 1 = a bounded wait expired

// Cycle accounting of the roles (compiled in with -DMST_SP_PROFILE, off by default; no effect on results): per block
//   [0] producer waiting for a free stage   [1] MMA thread waiting for a full stage   [2] MMA thread waiting for a free
//   accumulator   [3] epilogue warp 2 waiting for a complete accumulator   [4] epilogue warp 2 working
//   [5] whole kernel
#ifdef MST_SP_PROFILE
__device__ long long g_sp_prof[160][8];
#define SP_PROF_DECL long long prof_t0 = 0, prof_acc0 = 0, prof_acc1 = 0, prof_t1 = 0, prof_acc2 = 0, prof_acc3 = 0
#define SP_PROF_BEGIN1() prof_t1 = clock64()
#define SP_PROF_END1(acc) acc += clock64() - prof_t1
#define SP_PROF_BEGIN() prof_t0 = clock64()
#define SP_PROF_END(acc) acc += clock64() - prof_t0
#define SP_PROF_STORE(slot, acc) g_sp_prof[blockIdx.x][slot] = acc
#else
#define SP_PROF_DECL
#define SP_PROF_BEGIN1()
#define SP_PROF_END1(acc)
#define SP_PROF_BEGIN()
#define SP_PROF_END(acc)
#define SP_PROF_STORE(slot, acc)
#endif

struct SpParams {
  int64_t R, T;           // rows of S (output features of the product), tokens
  uint16_t* out;          // [T x ldout] bf16
  int64_t ldout;
  int kblocks;            // kd_pad / 128
  int m_tiles, n_tiles;   // 256-row tiles of S, 240-token tiles
  int chunks;             // 16-k chunks per row of S
  const int32_t* scan;    // spills of row r: [scan[r * chunks], scan[(r + 1) * chunks])
  const uint32_t* spill;  // (row of xr << 16) | bf16 value
  const uint16_t* xr;     // [columns with spills x ldxr] bf16, feature-major copy of those activation columns
  int64_t ldxr;
};

__device__ __forceinline__ bool sp_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  return mst_ptx::mbar_wait(bar, parity, abort_flag, &g_sp_error);
}
__device__ __forceinline__ uint32_t sp_in_even_block(uint32_t local_addr) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(0u));
  return r;
}
__device__ __forceinline__ uint32_t sp_cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void sp_cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void sp_tma_load_2d_pair(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(tm), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
// K-major descriptor without swizzle: 8-row x 16-byte core matrices, `sbo` bytes between consecutive 8-row groups
__device__ __forceinline__ uint64_t sp_desc_plain(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;
  return d;
}
// sixteen columns of this thread's tensor-memory lane, issued without waiting: the registers are valid after sp_tmem_wait on them
__device__ __forceinline__ void sp_tmem_ld16_issue(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
// wait for the outstanding tensor-memory loads; the registers are operands so that no use of them moves above the wait
__device__ __forceinline__ void sp_tmem_wait(uint32_t (&r)[16]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
                 "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
               :
               : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(S_THREADS, 1)
tc_sp24_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ CUtensorMap tmE, const SpParams P) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles_base = (raw + 1023u) & ~1023u;
  const uint32_t bar_base = tiles_base + S_STAGES * S_STAGE_BYTES;
  const uint32_t full0 = bar_base, empty0 = bar_base + 8 * S_STAGES, tfull0 = bar_base + 16 * S_STAGES, tempty0 = tfull0 + 16;
  __shared__ uint32_t tmem_base_holder;
  __shared__ int abort_sh;
  volatile int* abort_flag = &abort_sh;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = sp_cluster_ctarank();  // 0 = even block (issues the MMAs), 1 = its peer
  if (threadIdx.x == 0) {
    abort_sh = 0;
    for (int s = 0; s < S_STAGES; ++s) {
      mbar_init(full0 + 8 * s, 2);
      mbar_init(empty0 + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull0 + 8 * a, 1);
      mbar_init(tempty0 + 8 * a, 2 * S_EPI_WARPS);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_holder)),
                 "r"(S_TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  sp_cluster_sync();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_holder;
  mst_grid_launch_dependents();
  mst_grid_dependency_wait();
#ifdef MST_SP_PROFILE
  const long long prof_kernel_t0 = clock64();
#endif

  // work item w: token tile w / m_tiles, row tile w % m_tiles.  Pairs that run at the same time share their token
  // tile (the activations stream through L2 once) and sweep the compressed operand, which stays L2-resident.
  const int64_t works = (int64_t)P.m_tiles * P.n_tiles;
  const int64_t pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer (both blocks)
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      SP_PROF_DECL;
      for (int64_t w = pair; w < works && !*abort_flag; w += npairs) {
        const int mt = (int)(w % P.m_tiles), nt = (int)(w / P.m_tiles);
        const int row0 = mt * (2 * SM_ROWS) + (int)rank * SM_ROWS;      // this block's rows of S
        const int tok0 = nt * SN + (int)rank * (SN / 2);                // this block's half of the tokens
        const int mt128 = mt * 2 + (int)rank;                           // 128-row tile index for the metadata
        for (int kb = 0; kb < P.kblocks; ++kb) {
          SP_PROF_BEGIN();
          if (!sp_wait(empty0 + 8 * s, ph ^ 1u, abort_flag)) break;
          SP_PROF_END(prof_acc0);
          const uint32_t fb = sp_in_even_block(full0 + 8 * s);
          const uint32_t sa = tiles_base + s * S_STAGE_BYTES, sb = sa + SA_BYTES, se = sb + 2 * SB_BOX_STRIDE;
          asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(fb), "r"(S_TX_BYTES) : "memory");
          sp_tma_load_2d_pair(sa, &tmA, kb * (SKB / 2), row0, fb);
          sp_tma_load_2d_pair(sb, &tmB, kb * SKB, tok0, fb);
          sp_tma_load_2d_pair(sb + SB_BOX_STRIDE, &tmB, kb * SKB + 64, tok0, fb);
          sp_tma_load_2d_pair(se, &tmE, 0, (mt128 * P.kblocks + kb) * 2, fb);   // two 1 KiB rows = the block's 2 KiB
          if (++s == S_STAGES) { s = 0; ph ^= 1u; }
        }
      }
      SP_PROF_STORE(0, prof_acc0);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (even block only)
    if (lane == 0 && rank == 0) {
      // sparse, fp32 accumulate, bf16 x bf16, both operands K-major, N = 240, M = 256
      const uint32_t idesc0 = (1u << 2) | (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(SN >> 3) << 17) |
                              ((uint32_t)((2 * SM_ROWS) >> 4) << 24);
      const uint64_t adesc0 = smem_desc(tiles_base, 16, 1024);
      const uint64_t bdesc0 = smem_desc(tiles_base + SA_BYTES, 16, 1024);
      const uint64_t edesc0 = sp_desc_plain(tiles_base + SA_BYTES + 2 * SB_BOX_STRIDE, 128, 128);
      int s = 0, acc = 0, eslot = 0;
      uint32_t ph = 0, acc_ph = 0;
      SP_PROF_DECL;
      for (int64_t w = pair; w < works && !*abort_flag; w += npairs) {
        SP_PROF_BEGIN();
        if (!sp_wait(tempty0 + 8 * acc, acc_ph ^ 1u, abort_flag)) break;
        SP_PROF_END(prof_acc1);
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * SN);
        bool ok = true;
        for (int kb = 0; kb < P.kblocks; ++kb) {
          SP_PROF_BEGIN();
          if (!sp_wait(full0 + 8 * s, ph, abort_flag)) { ok = false; break; }
          SP_PROF_END(prof_acc0);
          tc_fence_after();
          const uint64_t soff = (uint64_t)(uint32_t)(s * (S_STAGE_BYTES >> 4));
          const uint32_t e_tmem = tmem_base + (uint32_t)(S_META_COL + 4 * eslot);
          asm volatile("tcgen05.cp.cta_group::2.128x128b [%0], %1;" ::"r"(e_tmem), "l"(edesc0 + soff) : "memory");
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            // compressed A: 16 elements (32 bytes) per instruction; B: 32 elements (64 bytes), second box after two
            const uint64_t ad = adesc0 + soff + (uint64_t)(j * 2);
            const uint64_t bd = bdesc0 + soff + (uint64_t)((j >> 1) * (SB_BOX_STRIDE >> 4) + (j & 1) * 4);
            const uint32_t idesc = idesc0 | (uint32_t)(j & 1);           // metadata column inside its aligned pair
            const uint32_t e_addr = e_tmem + (uint32_t)(j & 2);
            const uint32_t accum = (kb > 0 || j > 0) ? 1u : 0u;
            asm volatile(
                "{\n\t.reg .pred p;\n\t"
                "setp.ne.b32 p, %5, 0;\n\t"
                "tcgen05.mma.sp.cta_group::2.kind::f16 [%0], %1, %2, [%3], %4, p;\n\t}" ::"r"(d_tmem),
                "l"(ad), "l"(bd), "r"(e_addr), "r"(idesc), "r"(accum)
                : "memory");
          }
          asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
                           empty0 + 8 * s),
                       "h"((uint16_t)3)
                       : "memory");
          eslot ^= 1;
          if (++s == S_STAGES) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
                         tfull0 + 8 * acc),
                     "h"((uint16_t)3)
                     : "memory");
        if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
      }
      SP_PROF_STORE(1, prof_acc0);
      SP_PROF_STORE(2, prof_acc1);
    }
  } else {
    // ------------------------------------------------------------------ epilogue (both blocks, own 128 rows of S)
    // A thread owns one output feature (tensor-memory lane) and reads 16 tokens of it at a time.  For a fixed token the
    // 32 lanes of a warp hold 32 consecutive features, so each store instruction writes one 64-byte run of an output
    // row.  (Staging the chunk in shared memory for a bulk tensor store was measured slower: 94 K against 87 K cycles
    // for the forward product of a 5120 x 1280 layer over 8192 tokens.)  The activations of the row's first spills are
    // fetched one step ahead (they come from L2: the latency would otherwise be paid once per step).
    const int q = warp & 3;                 // tensor-memory lane quarter
    const int c0 = (warp - 2) >> 2;         // the two warps of a quarter take alternate 16-token chunks
    int acc = 0;
    uint32_t acc_ph = 0;
    SP_PROF_DECL;
    for (int64_t w = pair; w < works; w += npairs) {
      const int mt = (int)(w % P.m_tiles), nt = (int)(w / P.m_tiles);
      const int64_t row0 = (int64_t)mt * (2 * SM_ROWS) + (int)rank * SM_ROWS + q * 32;
      const int64_t r = row0 + lane;        // this thread's row of S = output feature
      const int64_t tok0 = (int64_t)nt * SN;
      // third and fourth entries of this row's groups (rows beyond R have none: their counts are zero)
      SP_PROF_BEGIN1();
      const int32_t sp0 = P.scan[r * P.chunks], sp1 = P.scan[(r + 1) * P.chunks];
      const int n_fast = min(sp1 - sp0, S_FAST_SPILLS);
      const int n_fast_warp = __reduce_max_sync(0xffffffffu, n_fast);
      float wv[S_FAST_SPILLS];
      const uint16_t* xrow[S_FAST_SPILLS];
#pragma unroll
      for (int j = 0; j < S_FAST_SPILLS; ++j) {
        const uint32_t ent = j < n_fast ? __ldg(P.spill + sp0 + j) : 0u;
        wv[j] = __uint_as_float(ent << 16);
        xrow[j] = P.xr + (int64_t)(ent >> 16) * P.ldxr;
      }
      uint4 xn[S_FAST_SPILLS][2];           // activations of the fast spills for the next chunk
      auto fetch = [&](int c) {
        const int64_t t0 = tok0 + c * S_CHUNK;
#pragma unroll
        for (int j = 0; j < S_FAST_SPILLS; ++j) {
          xn[j][0] = xn[j][1] = make_uint4(0, 0, 0, 0);
          if (j < n_fast && c < SN / S_CHUNK && t0 < P.T) {
            const uint4* src = reinterpret_cast<const uint4*>(xrow[j] + t0);
            xn[j][0] = __ldg(src);
            xn[j][1] = __ldg(src + 1);
          }
        }
      };
      if (n_fast_warp > 0) fetch(c0);
      SP_PROF_END1(prof_acc3);
      SP_PROF_BEGIN();
      if (!sp_wait(tfull0 + 8 * acc, acc_ph, abort_flag)) break;
      SP_PROF_END(prof_acc0);
      tc_fence_after();
      SP_PROF_BEGIN();
      // one 16-token chunk: spills added, rounded, written.  The tensor-memory load of the warp's next chunk is issued
      // before the chunk in hand is processed, so its latency hides behind the stores.
      auto chunk = [&](int c, uint32_t (&v)[16]) {
        const int64_t t0 = tok0 + c * S_CHUNK;
        if (n_fast_warp > 0) {   // uniform over the warp: some row of this warp has spills in this tile
          uint4 xc[S_FAST_SPILLS][2];
#pragma unroll
          for (int j = 0; j < S_FAST_SPILLS; ++j) { xc[j][0] = xn[j][0]; xc[j][1] = xn[j][1]; }
          fetch(c + 2);
          auto add_spill = [&](float wj, const uint4& x0, const uint4& x1) {
            const uint32_t xw[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              v[2 * i] = __float_as_uint(fmaf(wj, __uint_as_float(xw[i] << 16), __uint_as_float(v[2 * i])));
              v[2 * i + 1] = __float_as_uint(fmaf(wj, __uint_as_float(xw[i] & 0xFFFF0000u), __uint_as_float(v[2 * i + 1])));
            }
          };
#pragma unroll
          for (int j = 0; j < S_FAST_SPILLS; ++j)
            if (j < n_fast) add_spill(wv[j], xc[j][0], xc[j][1]);
          // rows with more spills than the prefetch holds: one at a time
          for (int32_t e = sp0 + S_FAST_SPILLS; e < sp1; ++e) {
            const uint32_t ent = __ldg(P.spill + e);
            const uint4* src = reinterpret_cast<const uint4*>(P.xr + (int64_t)(ent >> 16) * P.ldxr + t0);
            add_spill(__uint_as_float(ent << 16), __ldg(src), __ldg(src + 1));
          }
        }
        if (r < P.R) {
          uint16_t* dst = P.out + t0 * P.ldout + r;
          if (t0 + S_CHUNK <= P.T) {   // uniform: the whole chunk lies inside
#pragma unroll
            for (int j = 0; j < 16; j += 2) {
              const uint32_t pk = pack_bf16(__uint_as_float(v[j]), __uint_as_float(v[j + 1]));
              dst[(int64_t)j * P.ldout] = (uint16_t)(pk & 0xFFFFu);
              dst[(int64_t)(j + 1) * P.ldout] = (uint16_t)(pk >> 16);
            }
          } else {
#pragma unroll
            for (int j = 0; j < 16; j += 2) {
              const uint32_t pk = pack_bf16(__uint_as_float(v[j]), __uint_as_float(v[j + 1]));
              if (t0 + j < P.T) dst[(int64_t)j * P.ldout] = (uint16_t)(pk & 0xFFFFu);
              if (t0 + j + 1 < P.T) dst[(int64_t)(j + 1) * P.ldout] = (uint16_t)(pk >> 16);
            }
          }
        }
      };
      const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * SN);
      auto chunk_valid = [&](int c) { return c < SN / S_CHUNK && tok0 + (int64_t)c * S_CHUNK < P.T; };   // uniform
      uint32_t va[16], vb[16];
      if (chunk_valid(c0)) sp_tmem_ld16_issue(tacc + (uint32_t)(c0 * S_CHUNK), va);
#pragma unroll 1
      for (int c = c0; chunk_valid(c); c += 4) {
        SP_PROF_BEGIN1();
        sp_tmem_wait(va);
        SP_PROF_END1(prof_acc2);
        if (chunk_valid(c + 2)) sp_tmem_ld16_issue(tacc + (uint32_t)((c + 2) * S_CHUNK), vb);
        chunk(c, va);
        if (!chunk_valid(c + 2)) break;
        SP_PROF_BEGIN1();
        sp_tmem_wait(vb);
        SP_PROF_END1(prof_acc2);
        if (chunk_valid(c + 4)) sp_tmem_ld16_issue(tacc + (uint32_t)((c + 4) * S_CHUNK), va);
        chunk(c + 2, vb);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(sp_in_even_block(tempty0 + 8 * acc)) : "memory");
      SP_PROF_END(prof_acc1);
      if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
    }
    if (warp == 2 && lane == 0) {
      SP_PROF_STORE(3, prof_acc0);
      SP_PROF_STORE(4, prof_acc1);
      SP_PROF_STORE(6, prof_acc2);
      SP_PROF_STORE(7, prof_acc3);
    }
  }

  // ------------------------------------------------------------------ teardown
  if (*abort_flag) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
#ifdef MST_SP_PROFILE
  if (threadIdx.x == 0) g_sp_prof[blockIdx.x][5] = clock64() - prof_kernel_t0;
#endif
  sp_cluster_sync();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(S_TMEM_COLS) : "memory");
  }
}

// ------------------------------------------------------------------------------------------- compression
// Metadata of one group of four: positions p0 < p1 of the two kept elements, p0 | p1 << 2.  A group with fewer than
// two entries keeps explicit zeros at free positions.
struct Group {
  uint32_t nib;      // metadata nibble
  int take0, take1;  // which of the group's entries (0 = first set bit, ...) fill slot 0 / slot 1; -1 = zero
};
__device__ __forceinline__ Group group_of(uint32_t bits4) {
  Group g;
  const int cnt = __popc(bits4);
  if (cnt == 0) {
    g.nib = 0u | (1u << 2);
    g.take0 = g.take1 = -1;
  } else if (cnt == 1) {
    const int p = __ffs(bits4) - 1;
    if (p < 3) { g.nib = (uint32_t)p | (3u << 2); g.take0 = 0; g.take1 = -1; }
    else { g.nib = 0u | (3u << 2); g.take0 = -1; g.take1 = 0; }
  } else {
    const int p0 = __ffs(bits4) - 1;
    const int p1 = __ffs(bits4 & ~(1u << p0)) - 1;
    g.nib = (uint32_t)p0 | ((uint32_t)p1 << 2);
    g.take0 = 0;
    g.take1 = 1;
  }
  return g;
}

// where the 16-bit metadata of (row r, logical k in [k0, k0 + 16)) lives: 128-row tile, 128-deep K block, tensor-memory
// lane (r % 8) + 8 * ((k0 / 16) % 2) + 16 * ((r % 128) / 16), 32-bit word (k0 % 128) / 32, upper half for rows 8..15 of
// each 16
__device__ __forceinline__ int64_t meta_half_index(int64_t r, int k0, int kblocks) {
  const int64_t mt = r >> 7;
  const int m = (int)(r & 127), m0 = m & 7, m1 = (m >> 3) & 1, m2 = m >> 4;
  const int kb = k0 >> 7, j = (k0 & 127) >> 5, k1 = (k0 >> 4) & 1;
  const int ln = m0 + 8 * k1 + 16 * m2;
  return ((((mt * kblocks + kb) * 128 + ln) * 4 + j) << 1) + m1;
}

// One thread per (row of S, 16 consecutive k).  DIR 0: S = W.M, consecutive threads walk along a row.  DIR 1:
// S = (W.M)^T, row = input feature i, k = output feature o; consecutive threads take consecutive i, so the 16 mask
// words a warp needs are the same for all its lanes.  Every element of the compressed rows and of the metadata
// (padding included) is written, so nothing has to be cleared beforehand.
//   mode 0 (the mask changed): also counts the chunk's spills and flags the activation columns they multiply
//   mode 1: also writes the chunk's spills (position from the scan of the counts, row of the column copy from the
//           scan of the flags)
template <int DIR>
__global__ void sp24_compress_kernel(const uint32_t* __restrict__ bits, const int32_t* __restrict__ wscan,
                                     const uint16_t* __restrict__ vals, int O, int I, int wpr, int64_t r_pad, int kd_pad,
                                     int kblocks, int chunks, uint16_t* __restrict__ ac, uint16_t* __restrict__ meta16,
                                     int32_t* __restrict__ cnt, const int32_t* __restrict__ scan,
                                     int32_t* __restrict__ col_flag, const int32_t* __restrict__ col_slot,
                                     uint32_t* __restrict__ spill, int64_t spill_cap, int32_t* __restrict__ place,
                                     int mode) {
  mst_grid_launch_dependents();
  mst_grid_dependency_wait();
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= r_pad * chunks) return;
  int64_t r;
  int chunk;
  if (DIR == 0) {
    r = idx / chunks;
    chunk = (int)(idx - r * chunks);
  } else {
    chunk = (int)(idx / r_pad);
    r = idx - (int64_t)chunk * r_pad;
  }
  const int k0 = chunk << 4;
  const int R = DIR == 0 ? O : I, Kd = DIR == 0 ? I : O;
  uint32_t half = 0;
  int32_t pos[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) pos[j] = 0;
  if (r < R && k0 < Kd) {
    if (DIR == 0) {
      const int64_t wi = r * wpr + (k0 >> 5);
      const uint32_t word = bits[wi];
      const int sh = k0 & 31;
      half = (word >> sh) & 0xFFFFu;
      const int32_t base = wscan[wi] + __popc(word & ((1u << sh) - 1u));
#pragma unroll
      for (int j = 0; j < 16; ++j) pos[j] = base + __popc(half & ((1u << j) - 1u));
    } else {
      const int sh = (int)(r & 31);
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const int o = k0 + j;
        if (o < O) {
          const int64_t wi = (int64_t)o * wpr + (r >> 5);
          const uint32_t word = bits[wi];
          if ((word >> sh) & 1u) {
            half |= 1u << j;
            pos[j] = wscan[wi] + __popc(word & ((1u << sh) - 1u));
          }
        }
      }
    }
  }
  uint32_t m16 = 0;
  uint32_t outw[4];
  int extra = 0;
  int32_t e_at = 0;
  if (mode == 1) e_at = scan[r * chunks + chunk];
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    const uint32_t b4 = (half >> (4 * g)) & 0xFu;
    const Group G = group_of(b4);
    // CSR positions of the group's entries in ascending k
    int32_t ent[4];
    int n = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      ent[j] = 0;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if ((b4 >> j) & 1u) {
        // n is at most j, so a small select chain places the entry without dynamic indexing
        if (n == 0) ent[0] = pos[4 * g + j];
        else if (n == 1) ent[1] = pos[4 * g + j];
        else if (n == 2) ent[2] = pos[4 * g + j];
        else ent[3] = pos[4 * g + j];
        ++n;
      }
    }
    const int s0 = G.take0 == 0 ? ent[0] : -1;
    const int s1 = G.take1 == 0 ? ent[0] : (G.take1 == 1 ? ent[1] : -1);
    const uint32_t lo = s0 >= 0 ? (uint32_t)vals[s0] : 0u;
    const uint32_t hi = s1 >= 0 ? (uint32_t)vals[s1] : 0u;
    outw[g] = lo | (hi << 16);
    if (place && mode == 1) {
      const int32_t at = (int32_t)(r * (kd_pad >> 1) + (k0 >> 1) + 2 * g);
      if (s0 >= 0) place[s0] = at;
      if (s1 >= 0) place[s1] = at + 1;
    }
    m16 |= G.nib << (4 * g);
    if (n > 2) {
      extra += n - 2;
      // the third and fourth set bits of the group
      int seen = 0;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if ((b4 >> j) & 1u) {
          if (seen >= 2) {
            const int k = k0 + 4 * g + j;
            if (mode == 0) {
              col_flag[k] = 1;
            } else if (e_at < spill_cap) {
              spill[e_at] = ((uint32_t)col_slot[k] << 16) | (uint32_t)vals[seen == 2 ? ent[2] : ent[3]];
              if (place) place[seen == 2 ? ent[2] : ent[3]] = -(e_at + 1);
              ++e_at;
            }
          }
          ++seen;
        }
      }
    }
  }
  *reinterpret_cast<uint4*>(ac + r * (kd_pad >> 1) + (k0 >> 1)) = make_uint4(outw[0], outw[1], outw[2], outw[3]);
  meta16[meta_half_index(r, k0, kblocks)] = (uint16_t)m16;
  if (mode == 0) cnt[r * chunks + chunk] = extra;
}

// The values of the stored entries have changed, the mask has not: every value goes to the place the last compression
// gave its entry (an element of the compressed operand, or the low half of a spill word).
__global__ void sp24_scatter_values_kernel(const uint16_t* __restrict__ vals, const int32_t* __restrict__ place, int64_t nnz,
                                           uint16_t* __restrict__ ac, uint32_t* __restrict__ spill) {
  mst_grid_launch_dependents();
  mst_grid_dependency_wait();
  const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= nnz) return;
  const int32_t at = place[e];
  const uint16_t v = vals[e];
  if (at >= 0) ac[at] = v;
  else reinterpret_cast<uint16_t*>(spill)[2 * (int64_t)(-(at + 1))] = v;   // little-endian: the value is the low half
}

__global__ void sp24_slot_cols_kernel(const int32_t* __restrict__ col_flag, const int32_t* __restrict__ col_slot, int kd_pad,
                                      int32_t* __restrict__ slot_col) {
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k < kd_pad && col_flag[k]) slot_col[col_slot[k]] = k;
}

// Feature-major copy of the activation columns that spills multiply: xr[slot][t] = in[t][slot_col[slot]], zero for
// t >= T.  A block moves 32 columns x 64 tokens through shared memory: reads walk along the token rows (consecutive
// slots are ascending, mostly adjacent columns), writes are 128-byte rows.  Blocks beyond the number of such columns
// do nothing.
__global__ void __launch_bounds__(256) sp24_gather_cols_kernel(const uint16_t* __restrict__ in, int64_t ldin, int64_t T,
                                                              const int32_t* __restrict__ slot_col,
                                                              const int32_t* __restrict__ n_cols_ptr,
                                                              uint16_t* __restrict__ xr, int64_t ldxr) {
  mst_grid_launch_dependents();
  mst_grid_dependency_wait();
  __shared__ uint16_t tile[32][XR_TOK + 2];
  const int n_cols = *n_cols_ptr;
  const int64_t tok_tiles = ldxr / XR_TOK;
  const int64_t items = (int64_t)((n_cols + 31) / 32) * tok_tiles;   // the grid is sized for the layer, not for n_cols
  const int x = threadIdx.x & 31, y = threadIdx.x >> 5;
  for (int64_t it = blockIdx.x; it < items; it += gridDim.x) {
    const int slot0 = (int)(it / tok_tiles) * 32;
    const int64_t t0 = (it % tok_tiles) * XR_TOK;
    const int slot = slot0 + x;
    const int k = slot < n_cols ? slot_col[slot] : -1;
#pragma unroll
    for (int j = 0; j < XR_TOK / 8; ++j) {
      const int tl = y * (XR_TOK / 8) + j;
      const int64_t t = t0 + tl;
      tile[x][tl] = (k >= 0 && t < T) ? in[t * ldin + k] : (uint16_t)0;
    }
    __syncthreads();
    // warp y writes slots 4y .. 4y+3; eight lanes per slot, eight tokens (16 bytes) per lane
    const int sl = y * 4 + (x >> 3), piece = x & 7;
    if (slot0 + sl < n_cols) {
      uint32_t w[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) w[j] = (uint32_t)tile[sl][piece * 8 + 2 * j] | ((uint32_t)tile[sl][piece * 8 + 2 * j + 1] << 16);
      *reinterpret_cast<uint4*>(xr + (int64_t)(slot0 + sl) * ldxr + t0 + piece * 8) = make_uint4(w[0], w[1], w[2], w[3]);
    }
    __syncthreads();
  }
}

// ------------------------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn sp_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}
bool sp_map_2d(CUtensorMap* tm, CUtensorMapDataType dt, int esize, const void* base, int64_t rows, int64_t cols, int64_t ld,
               int box_cols, int box_rows, CUtensorMapSwizzle sw) {
  EncodeTiledFn fn = sp_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * esize};
  cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1u, 1u};
  return fn(tm, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int sp_sm_count() {
  int dev = 0, n = 0;
  cudaGetDevice(&dev);
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
  return n;
}

struct Carve {
  size_t off = 0;
  size_t take(size_t bytes) {
    const size_t at = off;
    off += (bytes + 255) & ~(size_t)255;
    return at;
  }
};

mst_status_t sp24_ensure(mst_layer* L, int dir) {
  mst_sp24& S = L->sp[dir];
  if (S.base) return MST_OK;
  const int R = dir == 0 ? L->O : L->I, Kd = dir == 0 ? L->I : L->O;
  S.R = R;
  S.Kd = Kd;
  S.r_pad = ((int64_t)R + 255) / 256 * 256;
  S.kd_pad = (Kd + 127) / 128 * 128;
  S.kblocks = S.kd_pad / 128;
  S.chunks = S.kd_pad / 16;
  S.spill_cap = L->N / 8 + 16;
  const int64_t n_cnt = S.r_pad * S.chunks;
  Carve cv;
  const size_t o_ac = cv.take((size_t)S.r_pad * (S.kd_pad / 2) * 2);
  const size_t o_meta = cv.take((size_t)(S.r_pad / 128) * S.kblocks * 2048);
  const size_t o_cnt = cv.take(4 * (size_t)(n_cnt + 1));
  const size_t o_scan = cv.take(4 * (size_t)(n_cnt + 1));
  const size_t o_spill = cv.take(4 * (size_t)S.spill_cap);
  const size_t o_flag = cv.take(4 * (size_t)(S.kd_pad + 1));
  const size_t o_slot = cv.take(4 * (size_t)(S.kd_pad + 1));
  const size_t o_scol = cv.take(4 * (size_t)S.kd_pad);
  const size_t o_bsum = cv.take(4 * (size_t)(mst_scan_block_sums_len(n_cnt) + 1024));
  // places of the stored entries, when an element index of the compressed operand fits 32 bits
  const bool keep_place = S.r_pad * (S.kd_pad / 2) < 0x7FFFFFFFLL;
  const size_t o_place = keep_place ? cv.take(4 * (size_t)(L->cap > 0 ? L->cap : 1)) : 0;
  MST_CUDA_TRY(cudaMalloc((void**)&S.base, cv.off));
  S.ac = (uint16_t*)(S.base + o_ac);
  S.meta = (uint32_t*)(S.base + o_meta);
  S.cnt = (int32_t*)(S.base + o_cnt);
  S.scan = (int32_t*)(S.base + o_scan);
  S.spill = (uint32_t*)(S.base + o_spill);
  S.col_flag = (int32_t*)(S.base + o_flag);
  S.col_slot = (int32_t*)(S.base + o_slot);
  S.slot_col = (int32_t*)(S.base + o_scol);
  S.bsums = (int32_t*)(S.base + o_bsum);
  S.place = keep_place ? (int32_t*)(S.base + o_place) : nullptr;
  S.place_version = -1;
  S.struct_version = -1;
  return MST_OK;
}

template <int DIR>
mst_status_t sp24_launch_compress(mst_layer* L, int mode, cudaStream_t s) {
  mst_sp24& S = L->sp[DIR];
  const int c = L->cur;
  const int64_t threads = S.r_pad * S.chunks;
  const unsigned blocks = (unsigned)((threads + 255) / 256);
  MST_CUDA_TRY(mst_launch_overlapped(sp24_compress_kernel<DIR>, dim3(blocks), dim3(256), 0, s, (const uint32_t*)L->bits[c],
                                     (const int32_t*)L->wscan[c], (const uint16_t*)L->vals[c], L->O, L->I, L->wpr, S.r_pad,
                                     S.kd_pad, S.kblocks, S.chunks, S.ac, (uint16_t*)S.meta, S.cnt, (const int32_t*)S.scan,
                                     S.col_flag, (const int32_t*)S.col_slot, S.spill, S.spill_cap, S.place, mode));
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}

// Compressed operand, metadata and spill list of the live structure and the current values.  The positions depend on
// the mask only and are rebuilt when it has changed; the values may have been changed in place since the last call,
// so they are written again every time (a scatter over the stored entries to the places the compression recorded).
mst_status_t sp24_refresh(mst_layer* L, int dir, cudaStream_t s) {
  MST_TRY(sp24_ensure(L, dir));
  mst_sp24& S = L->sp[dir];
  if (S.struct_version != L->version) {
    MST_CUDA_TRY(cudaMemsetAsync(S.col_flag, 0, 4 * (size_t)(S.kd_pad + 1), s));
    MST_TRY(dir == 0 ? sp24_launch_compress<0>(L, 0, s) : sp24_launch_compress<1>(L, 0, s));
    MST_TRY(mst_scan_i32(S.cnt, S.scan, S.r_pad * S.chunks, S.bsums, s));
    MST_TRY(mst_scan_i32(S.col_flag, S.col_slot, S.kd_pad, S.bsums, s));
    sp24_slot_cols_kernel<<<(unsigned)((S.kd_pad + 255) / 256), 256, 0, s>>>(S.col_flag, S.col_slot, S.kd_pad, S.slot_col); MST_COUNT_LAUNCH();
    MST_CUDA_TRY(cudaGetLastError());
    S.struct_version = L->version;
    S.values_epoch = -1;
  }
  // with value tracking the compressed operand is reused until the values change
  if (L->track_values && S.values_epoch == L->values_epoch) return MST_OK;
  S.values_epoch = L->values_epoch;
  if (S.place && S.place_version == L->version) {
    if (L->nnz == 0) return MST_OK;
    MST_CUDA_TRY(mst_launch_overlapped(sp24_scatter_values_kernel, dim3((unsigned)((L->nnz + 255) / 256)), dim3(256), 0, s,
                                       (const uint16_t*)L->vals[L->cur], (const int32_t*)S.place, (int64_t)L->nnz, S.ac, S.spill));
    MST_CUDA_TRY(cudaGetLastError());
    return MST_OK;
  }
  MST_TRY(dir == 0 ? sp24_launch_compress<0>(L, 1, s) : sp24_launch_compress<1>(L, 1, s));
  S.place_version = L->version;
  return MST_OK;
}

}  // namespace

bool mst_sp24_usable(const mst_layer* L, int dir, const void* in, int64_t ldin, const void* out, int64_t ldout) {
  (void)dir;
  // at most half of the entries can be third or fourth in their group
  return L->dtype == MST_BF16 && L->nnz >= 0 && L->nnz / 2 <= L->N / 8 && (ldin % 8 == 0) && (ldout % 8 == 0) &&
         ((reinterpret_cast<uintptr_t>(in) & 15u) == 0) && ((reinterpret_cast<uintptr_t>(out) & 15u) == 0) &&
         sp_encode_fn() != nullptr;
}

void mst_sp24_free(mst_layer* L) {
  for (int d = 0; d < 2; ++d) {
    if (L->sp[d].base) cudaFree(L->sp[d].base);
    L->sp[d] = mst_sp24();
  }
}

mst_status_t mst_sp24_product(mst_layer* L, int dir, const void* in, int64_t ldin, int64_t T, void* out, int64_t ldout,
                              cudaStream_t s) {
  if (T <= 0) return MST_OK;
  MST_TRY(sp24_refresh(L, dir, s));
  const mst_sp24& S = L->sp[dir];
  // feature-major copy of the activation columns the spills multiply (all of them in the worst case)
  const int64_t ldxr = (T + XR_TOK - 1) / XR_TOK * XR_TOK;
  void* xr = nullptr;
  MST_TRY(mst_workspace_kind(MST_WS_COLUMNS, (size_t)S.kd_pad * ldxr * 2, &xr));
  const int64_t gather_items = (int64_t)(S.kd_pad / 32) * (ldxr / XR_TOK);
  const int64_t gather_grid = gather_items < (int64_t)sp_sm_count() * 8 ? gather_items : (int64_t)sp_sm_count() * 8;
  MST_CUDA_TRY(mst_launch_overlapped(sp24_gather_cols_kernel, dim3((unsigned)gather_grid), dim3(256), 0, s, (const uint16_t*)in, ldin, T, (const int32_t*)S.slot_col,
                                     (const int32_t*)(S.col_slot + S.kd_pad), (uint16_t*)xr, ldxr));
  MST_CUDA_TRY(cudaGetLastError());

  CUtensorMap tmA, tmB, tmE;
  const bool ok = sp_map_2d(&tmA, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, S.ac, S.r_pad, S.kd_pad / 2, S.kd_pad / 2, 64, SM_ROWS,
                            CU_TENSOR_MAP_SWIZZLE_128B) &&
                  sp_map_2d(&tmB, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, in, T, S.Kd, ldin, 64, SN / 2, CU_TENSOR_MAP_SWIZZLE_128B) &&
                  // metadata blocks are contiguous 2 KiB pieces: described as rows of 256 words so that a block is
                  // fetched as sixteen full lines (a box of 128 rows x 16 bytes would be 128 separate requests)
                  sp_map_2d(&tmE, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, S.meta, (int64_t)(S.r_pad / 128) * S.kblocks * 2, 256, 256, 256,
                            2, CU_TENSOR_MAP_SWIZZLE_NONE);
  if (!ok) return MST_ERR_SHAPE;
  SpParams P = {};
  P.R = S.R;
  P.T = T;
  P.out = (uint16_t*)out;
  P.ldout = ldout;
  P.kblocks = S.kblocks;
  P.m_tiles = (int)(S.r_pad / (2 * SM_ROWS));
  P.n_tiles = (int)((T + SN - 1) / SN);
  P.chunks = S.chunks;
  P.scan = S.scan;
  P.spill = S.spill;
  P.xr = (const uint16_t*)xr;
  P.ldxr = ldxr;
  MST_CUDA_TRY(cudaFuncSetAttribute(tc_sp24_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)S_SMEM_BYTES));
  const int64_t works = (int64_t)P.m_tiles * P.n_tiles;
  const int64_t max_pairs = sp_sm_count() / 2;
  const int grid = 2 * (int)(works < max_pairs ? works : max_pairs);
  MST_CUDA_TRY(mst_launch_overlapped(tc_sp24_pair_kernel, dim3(grid), dim3(S_THREADS), S_SMEM_BYTES, s, tmA, tmB, tmE, P));
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}

#ifdef MST_SP_PROFILE
// cycle counters of the last launch: out[block][8], `blocks` rows (profiling builds only)
extern "C" mst_status_t mst_sp24_profile(long long* out, int blocks) {
  if (!out || blocks < 0 || blocks > 160) return MST_ERR_INVALID_ARG;
  MST_CUDA_TRY(cudaDeviceSynchronize());
  MST_CUDA_TRY(cudaMemcpyFromSymbol(out, g_sp_prof, sizeof(long long) * 8 * (size_t)blocks));
  return MST_OK;
}
#endif

mst_status_t mst_sp24_error_flags(int32_t* flags) {
  int v = 0;
  MST_CUDA_TRY(cudaMemcpyFromSymbol(&v, g_sp_error, sizeof(int)));
  *flags = v;
  return MST_OK;
}
