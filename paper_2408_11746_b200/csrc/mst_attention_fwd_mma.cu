// Strided sparse self-attention, forward (Sec. 3.3), on warp-level tensor-core products:
//   Out[i] = sum_{j in S_i} P_ij v_j,   P = softmax over S_i of q_i . k_j / sqrt(d),
//   S_i = { j <= i : i - j < l  or  (i - j) mod l == 0 }.
// A block owns 64 queries of one (sequence, head) and each of its four warps a 16-row strip of them (the kernel is
// also built for 128-query blocks and for two strips per warp, which share every key / value fragment between two
// products; measured within 2 % of each other or slower, see MST_ATTN_FWD_SHAPE below).  The block walks 64-key tiles
// of the window (keys q0 - l .. q0 + 63; the tile that starts l positions back also holds the first strided key of
// every query); riding along with window tile `it` comes the tile of the strided position i - (it + 2) l, of which only
// the diagonal is attended: a warp forms the two 16 x 8 score tiles in line with its rows and one 16-key step of the
// second product.  Window tiles are scored 32 keys at a time, and a warp skips the keys none of its rows can see.
// The softmax is the running one in base 2 with the scale folded into one multiply-add; its reference follows the
// running maximum lazily (see softmax_step), so the output rows are rescaled rarely.  Scores never leave the
// registers: two neighbouring accumulator tiles, rounded to bf16, are the A operand of P V.  K / V tiles are
// double-buffered with cp.async, every thread copying the same piece of every tile (addresses formed once); the
// query tile passes through the second buffer once.  No atomics; the order of every sum is fixed.
// The kernel is bound by instruction issue, not by a pipe: per score it spends about 16 thread instructions of which
// the two products are one (executed-opcode counts in the profile summary).
#include <cuda_bf16.h>

#include <cstdlib>

#include "mst_attention_mma.cuh"
#include "mst_internal.cuh"

namespace {
using namespace mst_attn;


struct FwdParams {
  const __nv_bfloat16 *Q, *K, *V;
  int64_t ld;
  __nv_bfloat16* Out;
  int64_t ldo;
  float* lse;   // [batch, heads, seq] or null
  int batch, seq, heads, stride;
};

// One strip's share of the running softmax over the keys just scored.  x[nb][e]: raw dot products of rows g (e < 2)
// and g + 8 (e >= 2) with `NB` blocks of eight keys, -inf where the pair is not attended.  m is the REFERENCE the
// exponents are taken against (base 2, scale folded in): it follows the running maximum only when that has moved up
// by more than 8, so weights stay below 2^8 (no overflow in fp32 sums or bf16 operands, same relative rounding) and
// the output rows are rescaled rarely; the final division by the sum cancels the reference exactly.  On return x
// holds the weights 2^(x SCALE_LOG2E - m).
template <int NB>
__device__ __forceinline__ void softmax_step(float (&x)[NB][4], float (&acc)[8][4], float (&m)[2], float (&sum)[2]) {
  float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) {
    mx0 = fmaxf(mx0, fmaxf(x[nb][0], x[nb][1]));
    mx1 = fmaxf(mx1, fmaxf(x[nb][2], x[nb][3]));
  }
  mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
  mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
  mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
  mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
  const float n0 = mx0 * SCALE_LOG2E, n1 = mx1 * SCALE_LOG2E;
  const bool up0 = n0 > m[0] + 8.f, up1 = n1 > m[1] + 8.f;   // a first key (m = -inf) always moves the reference
  if (__any_sync(0xffffffffu, up0 || up1)) {
    const float c0 = up0 ? ex2_approx(m[0] - n0) : 1.f, c1 = up1 ? ex2_approx(m[1] - n1) : 1.f;
    if (up0) m[0] = n0;
    if (up1) m[1] = n1;
    sum[0] *= c0;
    sum[1] *= c1;
#pragma unroll
    for (int nb = 0; nb < 8; ++nb) {
      acc[nb][0] *= c0;
      acc[nb][1] *= c0;
      acc[nb][2] *= c1;
      acc[nb][3] *= c1;
    }
  }
  // a row that has seen no key yet keeps reference -inf; its exponents are taken against 0 and come out as 0
  const float u0 = m[0] == -INFINITY ? 0.f : m[0], u1 = m[1] == -INFINITY ? 0.f : m[1];
  float s0 = 0.f, s1 = 0.f;
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) {
    x[nb][0] = ex2_approx(fmaf(x[nb][0], SCALE_LOG2E, -u0));
    x[nb][1] = ex2_approx(fmaf(x[nb][1], SCALE_LOG2E, -u0));
    x[nb][2] = ex2_approx(fmaf(x[nb][2], SCALE_LOG2E, -u1));
    x[nb][3] = ex2_approx(fmaf(x[nb][3], SCALE_LOG2E, -u1));
    s0 += x[nb][0] + x[nb][1];
    s1 += x[nb][2] + x[nb][3];
  }
  sum[0] += s0;   // this lane's columns only: the four lanes of a row add up at the end
  sum[1] += s1;
}

// NS = 16-row strips per warp, HALVES = 64-query halves per block: a block's 64 HALVES queries are shared by
// 4 HALVES / NS warps
template <int NS, int HALVES>
__global__ void __launch_bounds__(128 * HALVES / NS, HALVES == 1 ? 3 : 2) attn_fwd_mma_kernel(FwdParams P) {
  constexpr int WR = 16 * NS;        // rows per warp
  constexpr int HW = 4 / NS;         // warps per 64-query half
  constexpr int FQ = 64 * HALVES;    // queries per block
  extern __shared__ __align__(128) unsigned char smem[];
  __nv_bfloat16* KV = reinterpret_cast<__nv_bfloat16*>(smem);   // 4 + 4 HALVES tiles of [64][LDB], see `slot`

  const int qt = (int)gridDim.x - 1 - (int)blockIdx.x;   // the blocks with the most tiles start first
  const int h = blockIdx.y, b = blockIdx.z;
  const int q0 = qt * FQ, l = P.stride;
  const int64_t row0 = (int64_t)b * P.seq;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int a_row = q0 + warp * WR;   // this warp's first query

  // Trip `it` of the block's loop brings window tile `it` (keys k_first + 64 it ...) and, riding along, the strided
  // position m = it + 2 of both 64-query halves (keys q0 + 64 half - m l ...), as long as each exists
  const int k_first = q0 - l > 0 ? q0 - l : 0;
  const int n_near = (q0 + (HALVES - 1) * TS - k_first) / TS + 1;
  const int far0 = q0 / l > 1 ? q0 / l - 1 : 0;
  const int far1 = HALVES == 2 && (q0 + TS) / l > 1 ? (q0 + TS) / l - 1 : 0;   // two halves: far0 <= far1
  const int far_max = far0 > far1 ? far0 : far1;
  const int n_trips = n_near > far_max ? n_near : far_max;
  auto slot = [&](int i) { return KV + i * TS * LDB; };   // 0..3: window K, V of buffers 0 and 1; from 4: far K, V per buffer and half
  // this thread's piece of every tile copy: row threadIdx.x / 8 (+ multiples of THREADS / 8), 16-byte column threadIdx.x % 8
  constexpr int THREADS = 128 * HALVES / NS;
  const uint32_t s_thr = (uint32_t)__cvta_generic_to_shared(KV + (threadIdx.x >> 3) * LDB + (threadIdx.x & 7) * 8);
  const int64_t g_thr = (row0 + (threadIdx.x >> 3)) * P.ld + h * D + (threadIdx.x & 7) * 8;
  const __nv_bfloat16 *Kt = P.K + g_thr, *Vt = P.V + g_thr;
  auto copy = [&](int sl, const __nv_bfloat16* src_thread, int first_row) {
    copy_tile_async<THREADS>(s_thr + (uint32_t)(sl * TS * LDB * 2), src_thread + (int64_t)first_row * P.ld, P.ld);
  };
  auto fetch = [&](int it, int bf) {
    if (it < n_near) {
      copy(2 * bf, Kt, k_first + it * TS);
      copy(2 * bf + 1, Vt, k_first + it * TS);
    }
    if (it < far0) {
      copy(4 + 2 * HALVES * bf, Kt, q0 - (it + 2) * l);
      copy(5 + 2 * HALVES * bf, Vt, q0 - (it + 2) * l);
    }
    if (HALVES == 2 && it < far1) {
      copy(6 + 4 * bf, Kt, q0 + TS - (it + 2) * l);
      copy(7 + 4 * bf, Vt, q0 + TS - (it + 2) * l);
    }
    async_commit();
  };
  copy(2, P.Q + g_thr, q0);             // queries through the second window buffer
  if (HALVES == 2) copy(3, P.Q + g_thr, q0 + TS);
  fetch(0, 0);
  async_wait_all();
  __syncthreads();
  uint32_t qa[NS][4][4];
  {
    const __nv_bfloat16* Qs = slot(2 + warp / HW);
#pragma unroll
    for (int s = 0; s < NS; ++s)
#pragma unroll
      for (int kb = 0; kb < 4; ++kb) load_a(qa[s][kb], Qs, (warp % HW) * WR + s * 16, kb, lane);
  }
  float acc[NS][8][4], m[NS][2], sum[NS][2];
#pragma unroll
  for (int s = 0; s < NS; ++s) {
    m[s][0] = m[s][1] = -INFINITY;
    sum[s][0] = sum[s][1] = 0.f;
#pragma unroll
    for (int nb = 0; nb < 8; ++nb) acc[s][nb][0] = acc[s][nb][1] = acc[s][nb][2] = acc[s][nb][3] = 0.f;
  }

  int buf = 0;
  for (int it = 0; it < n_trips; ++it, buf ^= 1) {
    async_wait_all();
    __syncthreads();   // this trip's tiles have landed for everyone; the other buffers (first: the queries) have been consumed
    if (it + 1 < n_trips) fetch(it + 1, buf ^ 1);
    if (it < (warp / HW ? far1 : far0)) {
      // the strided position: query r of this half sees key r of the half's tile only
      const __nv_bfloat16* Ks = slot(4 + 2 * HALVES * buf + 2 * (warp / HW));
      const __nv_bfloat16* Vs = Ks + TS * LDB;
      const int c0 = (warp % HW) * WR;   // strip s: the 16 keys c0 + 16 s ... in line with its rows
      float sc[NS][2][4];
#pragma unroll
      for (int s = 0; s < NS; ++s)
#pragma unroll
        for (int nb = 0; nb < 2; ++nb) sc[s][nb][0] = sc[s][nb][1] = sc[s][nb][2] = sc[s][nb][3] = 0.f;
#pragma unroll
      for (int k2 = 0; k2 < 2; ++k2) {
        uint32_t kf[NS][2][4];
#pragma unroll
        for (int s = 0; s < NS; ++s)
#pragma unroll
          for (int nb = 0; nb < 2; ++nb) ldsm_x4(kf[s][nb], Ks + (c0 + s * 16 + nb * 8 + (lane & 7)) * LDB + k2 * 32 + (lane >> 3) * 8);
#pragma unroll
        for (int kk = 0; kk < 2; ++kk)
#pragma unroll
          for (int s = 0; s < NS; ++s)
#pragma unroll
            for (int nb = 0; nb < 2; ++nb) mma_bf16(sc[s][nb], qa[s][2 * k2 + kk], kf[s][nb][2 * kk], kf[s][nb][2 * kk + 1]);
      }
#pragma unroll
      for (int s = 0; s < NS; ++s) {
#pragma unroll
        for (int nb = 0; nb < 2; ++nb)
#pragma unroll
          for (int e = 0; e < 4; ++e)   // row g + 8 (e >> 1) against key 8 nb + 2 t + (e & 1)
            if (g + (e >> 1) * 8 != nb * 8 + 2 * t + (e & 1)) sc[s][nb][e] = -INFINITY;
        softmax_step<2>(sc[s], acc[s], m[s], sum[s]);
        uint32_t pa[4];
        pa[0] = pack_bf16(sc[s][0][0], sc[s][0][1]);
        pa[1] = pack_bf16(sc[s][0][2], sc[s][0][3]);
        pa[2] = pack_bf16(sc[s][1][0], sc[s][1][1]);
        pa[3] = pack_bf16(sc[s][1][2], sc[s][1][3]);
        mma_cols(acc[s], pa, Vs, c0 + s * 16, lane);
      }
    }
    if (it >= n_near) continue;
    const int k0 = k_first + it * TS;
    const __nv_bfloat16* Ks = slot(2 * buf);
    const __nv_bfloat16* Vs = slot(2 * buf + 1);
    // window tile, 32 keys at a time: a pair is attended iff 0 <= i - j <= l (the window and the first strided position)
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const int kh = k0 + half * 32;
      if (a_row + WR - 1 - kh < 0 || a_row - (kh + 31) > l) continue;   // none of this warp's rows sees these keys
      float sc[NS][4][4];
#pragma unroll
      for (int s = 0; s < NS; ++s)
#pragma unroll
        for (int nb = 0; nb < 4; ++nb) sc[s][nb][0] = sc[s][nb][1] = sc[s][nb][2] = sc[s][nb][3] = 0.f;
#pragma unroll
      for (int k2 = 0; k2 < 2; ++k2) {   // k-step outermost: consecutive products go to different accumulators
        uint32_t kf[4][4];
#pragma unroll
        for (int nb = 0; nb < 4; ++nb) ldsm_x4(kf[nb], Ks + (half * 32 + nb * 8 + (lane & 7)) * LDB + k2 * 32 + (lane >> 3) * 8);
#pragma unroll
        for (int kk = 0; kk < 2; ++kk)
#pragma unroll
          for (int nb = 0; nb < 4; ++nb)
#pragma unroll
            for (int s = 0; s < NS; ++s) mma_bf16(sc[s][nb], qa[s][2 * k2 + kk], kf[nb][2 * kk], kf[nb][2 * kk + 1]);
      }
      uint32_t pa[NS][2][4];
#pragma unroll
      for (int s = 0; s < NS; ++s) {
        const int a_s = a_row + s * 16;
        const bool full = a_s - (kh + 31) >= 0 && a_s + 15 - kh <= l;   // uniform over the warp
        if (!full) {
          const int back0 = a_s + g - kh - 2 * t;   // i - j of this lane's first element of key block 0
#pragma unroll
          for (int nb = 0; nb < 4; ++nb) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int back = back0 + (e >> 1) * 8 - nb * 8 - (e & 1);
              if ((unsigned)back > (unsigned)l) sc[s][nb][e] = -INFINITY;   // back < 0 or back > l
            }
          }
        }
        softmax_step<4>(sc[s], acc[s], m[s], sum[s]);
#pragma unroll
        for (int j = 0; j < 2; ++j) {   // 16 keys per step of the second product
          pa[s][j][0] = pack_bf16(sc[s][2 * j][0], sc[s][2 * j][1]);
          pa[s][j][1] = pack_bf16(sc[s][2 * j][2], sc[s][2 * j][3]);
          pa[s][j][2] = pack_bf16(sc[s][2 * j + 1][0], sc[s][2 * j + 1][1]);
          pa[s][j][3] = pack_bf16(sc[s][2 * j + 1][2], sc[s][2 * j + 1][3]);
        }
      }
#pragma unroll
      for (int j = 0; j < 2; ++j) {
#pragma unroll
        for (int n2 = 0; n2 < 4; ++n2) {
          uint32_t vf[4];
          ldsm_x4_t(vf, Vs + (half * 32 + j * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * LDB + n2 * 16 + (lane >> 4) * 8);
#pragma unroll
          for (int s = 0; s < NS; ++s) {
            mma_bf16(acc[s][2 * n2], pa[s][j], vf[0], vf[1]);
            mma_bf16(acc[s][2 * n2 + 1], pa[s][j], vf[2], vf[3]);
          }
        }
      }
    }
  }
  __syncthreads();   // every warp is done with the tiles: their storage stages the output rows
  __nv_bfloat16* Ob = slot(0) + warp * WR * LDB;
  const int64_t stat0 = ((int64_t)b * P.heads + h) * P.seq;
#pragma unroll
  for (int s = 0; s < NS; ++s) {
    float s0 = sum[s][0], s1 = sum[s][1];
    s0 += __shfl_xor_sync(0xffffffffu, s0, 1);
    s1 += __shfl_xor_sync(0xffffffffu, s1, 1);
    s0 += __shfl_xor_sync(0xffffffffu, s0, 2);
    s1 += __shfl_xor_sync(0xffffffffu, s1, 2);
    const float i0 = 1.f / s0, i1 = 1.f / s1;   // every row attends at least itself
#pragma unroll
    for (int nb = 0; nb < 8; ++nb) {
      *reinterpret_cast<__nv_bfloat162*>(Ob + (s * 16 + g) * LDB + nb * 8 + 2 * t) = __floats2bfloat162_rn(acc[s][nb][0] * i0, acc[s][nb][1] * i0);
      *reinterpret_cast<__nv_bfloat162*>(Ob + (s * 16 + g + 8) * LDB + nb * 8 + 2 * t) = __floats2bfloat162_rn(acc[s][nb][2] * i1, acc[s][nb][3] * i1);
    }
    if (P.lse && t == 0) {
      P.lse[stat0 + a_row + s * 16 + g] = (m[s][0] + log2f(s0)) * 0.6931471805599453f;
      P.lse[stat0 + a_row + s * 16 + g + 8] = (m[s][1] + log2f(s1)) * 0.6931471805599453f;
    }
  }
  __syncwarp();
#pragma unroll
  for (int it = 0; it < 4 * NS; ++it) {   // eight lanes write one row of 128 bytes
    const int r = it * 4 + (lane >> 3), piece = lane & 7;
    const uint4 v = *reinterpret_cast<const uint4*>(Ob + r * LDB + piece * 8);
    *reinterpret_cast<uint4*>(P.Out + (row0 + a_row + r) * P.ldo + h * D + piece * 8) = v;
  }
}

}  // namespace

// Launch for the shapes the public entry point has checked: head dimension 64, seq_len a multiple of 128, stride a
// positive multiple of 64, 16-byte aligned pointers, leading dimensions multiples of 8.
mst_status_t mst_attention_fwd_mma(const void* Q, const void* K, const void* V, int64_t ld, int32_t batch, int32_t seq_len,
                                   int32_t heads, int32_t stride, void* Out, int64_t ldo, float* lse, cudaStream_t s) {
  if (seq_len % 128 != 0 || stride <= 0 || stride % TS != 0 || heads > 65535 || batch > 65535) return MST_ERR_SHAPE;
  FwdParams P;
  P.Q = (const __nv_bfloat16*)Q; P.K = (const __nv_bfloat16*)K; P.V = (const __nv_bfloat16*)V;
  P.ld = ld;
  P.Out = (__nv_bfloat16*)Out;
  P.ldo = ldo;
  P.lse = lse;
  P.batch = batch; P.seq = seq_len; P.heads = heads; P.stride = stride;
  int halves = 1, strips = 1;   // 64 queries per block, 16 rows per warp: four warps
  if (const char* e = getenv("MST_ATTN_FWD_SHAPE")) {   // measurement override: "<halves><strips>", e.g. 21
    halves = e[0] == '2' ? 2 : 1;
    strips = e[0] && e[1] == '2' ? 2 : 1;
  }
  const size_t smem = (size_t)((4 + 4 * halves) * TS * LDB) * 2;
  dim3 grid((unsigned)(seq_len / (64 * halves)), (unsigned)heads, (unsigned)batch);
#define MST_ATTN_LAUNCH(NS_, H_)                                                                                              \
  do {                                                                                                                        \
    MST_CUDA_TRY(cudaFuncSetAttribute(attn_fwd_mma_kernel<NS_, H_>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));  \
    attn_fwd_mma_kernel<NS_, H_><<<grid, 128 * H_ / NS_, smem, s>>>(P); MST_COUNT_LAUNCH();                                    \
  } while (0)
  if (halves == 2 && strips == 2) MST_ATTN_LAUNCH(2, 2);
  else if (halves == 2) MST_ATTN_LAUNCH(1, 2);
  else if (strips == 2) MST_ATTN_LAUNCH(2, 1);
  else MST_ATTN_LAUNCH(1, 1);
#undef MST_ATTN_LAUNCH
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}
