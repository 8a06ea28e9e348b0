// Parameter block of the contraction families (GEMM / 1x1 convolution anchors).
#pragma once
#include <cuda.h>

#include "microop.h"

namespace dnnf {

// One GEMM operand as a strided 2-D matrix with up to two batch dims.
// A is [M x K] (row = m, col = k); B is [K x N] (row = k, col = n).
struct GemmOperand {
  void* ptr;
  int64_t base;            // elements
  int64_t stride_row, stride_col;
  int64_t batch_stride[2];
  int32_t dtype;
  int32_t pad;
};

struct GemmParams {
  int32_t M, N, K;
  int32_t batch_ext[2];    // batch_ext[0] is the inner batch dim; total batches = product
  GemmOperand A, B;
  // Epilogue iteration space, innermost first: n digits, then m digits, then batch digits.
  IterSpace it;
  int32_t n_nd, m_nd, b_nd;
  int32_t n_in, n_out;
  TensorArg in[kMaxIn];
  TensorArg out[kMaxOut];
  Program prog;
  int32_t vec_ok;          // every epilogue access along n is unit-stride and 4-element aligned
  int32_t tiles_m, tiles_n;
  int32_t* status;         // device status words (bounded-wait failures)
  int32_t block_index;
  uint32_t static_mask;     // bit 0: B, bit 1+i: epilogue input i is an external input of the graph (never written by a kernel)
};

// Tensor-core path extras (kept apart so the common block stays small).
struct GemmTcParams {
  CUtensorMap tmA, tmB;
  int32_t a_kmajor, b_kmajor;     // operand major-ness in shared memory
  int32_t k_tiles;
  int32_t bn;                      // N tile
  int32_t persistent_tiles;        // total output tiles
  int32_t debug;                   // ablation switches (development only)
  FastDiv fd_tiles_mn, fd_tiles_n, fd_batch0;   // tile index -> (batch, tile row, tile column), batch -> (b0, b1)
};

}  // namespace dnnf
