// Interface of the structured-sparse tensor-core path (tcgen05.mma.sp, 2:4 along the contraction dimension) for the
// forward product and the input gradient of bf16 layers.  Internal to libmst.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "mst.h"

struct mst_layer;

// One direction of the split of S = W.M (dir 0: forward, rows = output features, k = input features) or
// S = (W.M)^T (dir 1: input gradient, rows = input features, k = output features) into
//   - a 2:4-conforming part: the first two entries of every group of four consecutive k, stored compressed
//     ([r_pad x kd_pad/2] bf16) with 4 bits of position metadata per group, laid out as the tensor core reads it;
//   - a spill list: the third and fourth entries of the few groups that hold more than two, as a CSR-like list per
//     row whose entries name a row of a feature-major copy of the activation columns they multiply.
struct mst_sp24 {
  unsigned char* base = nullptr;  // one allocation
  uint16_t* ac = nullptr;         // compressed values
  uint32_t* meta = nullptr;       // metadata, one 2 KiB block per (128 rows, 128 k)
  int32_t* cnt = nullptr;         // [r_pad * chunks + 1] spills per (row, 16-k chunk)
  int32_t* scan = nullptr;        // [r_pad * chunks + 1] exclusive scan of cnt: row r's spills are [scan[r*chunks], scan[(r+1)*chunks])
  uint32_t* spill = nullptr;      // [spill_cap]  (slot << 16) | bf16 value
  int32_t* col_flag = nullptr;    // [kd_pad + 1] 1 = some spill multiplies activation column k
  int32_t* col_slot = nullptr;    // [kd_pad + 1] exclusive scan of col_flag; col_slot[kd_pad] = number of such columns
  int32_t* slot_col = nullptr;    // [kd_pad]     inverse map
  int32_t* bsums = nullptr;       // scan partials
  int32_t* place = nullptr;       // [cap] where stored entry e went: >= 0 element of ac, < 0 spill -(index + 1); nullptr: not kept
  int R = 0, Kd = 0;
  int64_t r_pad = 0;
  int kd_pad = 0, kblocks = 0, chunks = 0;
  int64_t spill_cap = 0;
  int64_t struct_version = -1;    // layer structure version the spill positions belong to
  int64_t values_epoch = -1;      // values epoch the compressed operand was built from (value tracking only)
  int64_t place_version = -1;     // layer structure version `place` belongs to
};

// true when the operands can be described to the TMA unit and the layer's nnz fits the spill capacity
bool mst_sp24_usable(const mst_layer* L, int dir, const void* in, int64_t ldin, const void* out, int64_t ldout);
// out[t, r] = sum_k in[t, k] * S[r, k]   (dir 0: forward, dir 1: input gradient); bf16 in and out, fp32 accumulation
mst_status_t mst_sp24_product(mst_layer* L, int dir, const void* in, int64_t ldin, int64_t T, void* out, int64_t ldout,
                              cudaStream_t s);
void mst_sp24_free(mst_layer* L);
mst_status_t mst_sp24_error_flags(int32_t* flags);
