// Row family: a chain around a reduction over the last axis (Softmax, LayerNorm,
// ReduceSum/Mean/Max/Prod).  The whole row lives in registers from the first load
// to the last store: a warp (rows up to 1024 elements) or a CTA (up to 8192) owns
// a row, reductions are warp shuffles (plus one shared-memory exchange for
// CTA-wide rows), and the pre- and post-chains run on the register-resident row.
#include "chain.cuh"
#include "ir.h"

namespace dnnf {

__device__ __forceinline__ uint32_t fdiv_row(const IterSpace& it, int d, uint32_t n) {
  return it.extent[d] == 1 ? n : (__umulhi(n, it.div_m[d]) >> it.div_s[d]);
}

// NV vectors of V elements per thread; WPR warps cooperate on one row.
template <int V, int NV, int WPR>
struct RowIO {
  const RowParams& p;
  uint32_t outer[kMaxDims];
  int lane_in_row;                 // 0 .. 32*WPR-1
  float* xchg;                     // shared memory, WPR floats per row slot (WPR > 1)
  __device__ __forceinline__ int col(int j) const { return (j * 32 * WPR + lane_in_row) * V; }
  __device__ __forceinline__ int64_t row_offset(const TensorArg& a) const {
    int64_t off = a.base;
#pragma unroll
    for (int d = 0; d < kMaxDims - 1; ++d)
      if (d < p.it.ndim - 1) off += (int64_t)outer[d] * a.stride[d];
    return off;
  }
  __device__ __forceinline__ void load(int idx, float (&dst)[V * NV]) const {
    const TensorArg& a = p.in[idx];
    const int64_t si = a.stride[p.it.ndim - 1];
    const int64_t ro = row_offset(a);
    if (si == 0) {
      float x = load_scalar(a, ro);
#pragma unroll
      for (int v = 0; v < V * NV; ++v) dst[v] = x;
      return;
    }
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      int c = col(j);
      if (c < p.L) {
        if (V == 4) load_vec4(a, ro + c, &dst[j * V]);
        else dst[j] = load_scalar(a, ro + c);
      } else {
#pragma unroll
        for (int v = 0; v < V; ++v) dst[j * V + v] = 0.0f;
      }
    }
  }
  __device__ __forceinline__ void anchor(float (&dst)[V * NV]) const {
#pragma unroll
    for (int v = 0; v < V * NV; ++v) dst[v] = 0.0f;
  }
  __device__ __forceinline__ void store(int idx, const float (&val)[V * NV]) const {
    const TensorArg& a = p.out[idx];
    const int64_t si = a.stride[p.it.ndim - 1];
    const int64_t ro = row_offset(a);
    if (si == 0) {                                   // a per-row scalar (reduced output)
      if (lane_in_row == 0) store_scalar(a, ro, val[0], false);
      return;
    }
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      int c = col(j);
      if (c < p.L) {
        if (V == 4) store_vec4(a, ro + c, &val[j * V], false);
        else store_scalar(a, ro + c, val[j], false);
      }
    }
  }
  __device__ __forceinline__ void row_reduce(int op, float (&acc)[V * NV]) const {
    float r;
    if (op == M_ROWMAX) r = -CUDART_INF_F; else if (op == M_ROWPROD) r = 1.0f; else r = 0.0f;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      if (col(j) < p.L) {
#pragma unroll
        for (int v = 0; v < V; ++v) {
          float x = acc[j * V + v];
          if (op == M_ROWMAX) r = fmaxf(r, x); else if (op == M_ROWPROD) r *= x; else r += x;
        }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      float y = __shfl_xor_sync(0xffffffffu, r, o);
      if (op == M_ROWMAX) r = fmaxf(r, y); else if (op == M_ROWPROD) r *= y; else r += y;
    }
    if (WPR > 1) {
      __syncthreads();                               // previous exchange fully consumed
      if ((threadIdx.x & 31) == 0) xchg[threadIdx.x >> 5] = r;
      __syncthreads();
      float t = xchg[0];
#pragma unroll
      for (int w = 1; w < WPR; ++w) {
        float y = xchg[w];
        if (op == M_ROWMAX) t = fmaxf(t, y); else if (op == M_ROWPROD) t *= y; else t += y;
      }
      r = t;
    }
    if (op == M_ROWMEAN) r = r / (float)p.L;
#pragma unroll
    for (int v = 0; v < V * NV; ++v) acc[v] = r;
  }
};

constexpr int kRowWarpsPerCta = 4;

template <int V, int NV, int WPR>
__global__ void __launch_bounds__(WPR > 1 ? 32 * WPR : 32 * kRowWarpsPerCta)
row_kernel(const __grid_constant__ RowParams p) {
  __shared__ float xchg[WPR > 1 ? WPR : 1];
  RowIO<V, NV, WPR> io{p};
  io.xchg = xchg;
  uint32_t row;
  if (WPR > 1) { row = blockIdx.x; io.lane_in_row = threadIdx.x; }
  else { row = blockIdx.x * kRowWarpsPerCta + (threadIdx.x >> 5); io.lane_in_row = threadIdx.x & 31; }
  if (row >= (uint32_t)p.rows) return;               // whole warps (WPR == 1) or never (WPR > 1)
  uint32_t lin = row;
#pragma unroll
  for (int d = kMaxDims - 2; d >= 0; --d) {
    if (d < p.it.ndim - 1) {
      uint32_t q = fdiv_row(p.it, d, lin);
      io.outer[d] = lin - q * p.it.extent[d];
      lin = q;
    }
  }
  run_program<V * NV, 2>(p.prog, io);
}

template <int V, int NV, int WPR>
static void launch_one(const RowParams& p, int grid, cudaStream_t st) {
  row_kernel<V, NV, WPR><<<grid, WPR > 1 ? 32 * WPR : 32 * kRowWarpsPerCta, 0, st>>>(p);
}

// variant encoding: V * 10000 + NV * 100 + WPR
int launch_row(const Launch& L, cudaStream_t st) {
  const RowParams& p = L.row;
  switch (L.variant) {
    case 40101: launch_one<4, 1, 1>(p, L.grid, st); break;
    case 40201: launch_one<4, 2, 1>(p, L.grid, st); break;
    case 40401: launch_one<4, 4, 1>(p, L.grid, st); break;
    case 40601: launch_one<4, 6, 1>(p, L.grid, st); break;
    case 40801: launch_one<4, 8, 1>(p, L.grid, st); break;
    case 40208: launch_one<4, 2, 8>(p, L.grid, st); break;
    case 40408: launch_one<4, 4, 8>(p, L.grid, st); break;
    case 40808: launch_one<4, 8, 8>(p, L.grid, st); break;
    case 10101: launch_one<1, 1, 1>(p, L.grid, st); break;
    case 10401: launch_one<1, 4, 1>(p, L.grid, st); break;
    case 11601: launch_one<1, 16, 1>(p, L.grid, st); break;
    case 10808: launch_one<1, 8, 8>(p, L.grid, st); break;
    case 13208: launch_one<1, 32, 8>(p, L.grid, st); break;
    default: return 2;
  }
  return cudaGetLastError() == cudaSuccess ? 0 : 1;
}

bool finalize_row(Launch& L) {
  RowParams& p = L.row;
  int V = p.vec, Lr = p.L;
  int nv = 0, wpr = 0;
  if (V == 4) {
    int need = (Lr + 127) / 128;                   // vectors per lane with one warp per row
    if (need <= 8) { wpr = 1; nv = need <= 1 ? 1 : need <= 2 ? 2 : need <= 4 ? 4 : need <= 6 ? 6 : 8; }
    else { wpr = 8; int n8 = (Lr + 1023) / 1024; nv = n8 <= 2 ? 2 : n8 <= 4 ? 4 : 8; if (n8 > 8) return false; }
  } else {
    int need = (Lr + 31) / 32;
    if (need <= 16) { wpr = 1; nv = need <= 1 ? 1 : need <= 4 ? 4 : 16; }
    else { wpr = 8; int n8 = (Lr + 255) / 256; nv = n8 <= 8 ? 8 : 32; if (n8 > 32) return false; }
  }
  L.variant = V * 10000 + nv * 100 + wpr;
  L.grid = wpr > 1 ? (int)p.rows : (int)((p.rows + kRowWarpsPerCta - 1) / kRowWarpsPerCta);
  L.threads = wpr > 1 ? 32 * wpr : 32 * kRowWarpsPerCta;
  set_fastdiv(p.it);
  return true;
}

}  // namespace dnnf
