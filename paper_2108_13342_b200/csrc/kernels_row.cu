// Row family: a chain around a reduction over the last axis (Softmax, LayerNorm,
// ReduceSum/Mean/Max/Prod).  The whole row lives in registers from the first load
// to the last store: a warp (rows up to 1024 elements) or a CTA (up to 8192) owns
// a row -- short rows are processed RPW at a time per warp so that enough loads
// are in flight -- reductions are warp shuffles (plus one shared-memory exchange
// for CTA-wide rows), and the pre- and post-chains run on the register-resident row.
#include "chain.cuh"
#include "ir.h"

namespace dnnf {

__device__ __forceinline__ uint32_t fdiv_row(const IterSpace& it, int d, uint32_t n) {
  return it.extent[d] == 1 ? n : (__umulhi(n, it.div_m[d]) >> it.div_s[d]);
}

// Device dim 0 is the row (length L); dims 1.. are the outer dims, innermost first.
// NV vectors of V elements per thread and row; RPW rows per warp; WPR warps per row.
template <int V, int NV, int WPR, int RPW>
struct RowIO {
  static constexpr int VV = V * NV * RPW;
  const RowParams& p;
  uint32_t outer[RPW][kMaxDims];
  bool row_ok[RPW];
  int lane_in_row;                 // 0 .. 32*WPR-1
  float* xchg;                     // shared memory, WPR floats (WPR > 1)
  __device__ __forceinline__ int col(int j) const { return (j * 32 * WPR + lane_in_row) * V; }
  __device__ __forceinline__ int64_t row_offset(const TensorArg& a, int r) const {
    int64_t off = a.base;
#pragma unroll
    for (int d = 1; d < kMaxDims; ++d)
      if (d < p.it.ndim) off += (int64_t)outer[r][d] * a.stride[d];
    return off;
  }
  __device__ __forceinline__ void load(int idx, float (&dst)[VV]) const {
    const TensorArg& a = p.in[idx];
    const int64_t si = a.stride[0];
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
      const int64_t ro = row_offset(a, r);
      if (si == 0) {
        float x = row_ok[r] ? load_scalar(a, ro) : 0.0f;
#pragma unroll
        for (int e = 0; e < V * NV; ++e) dst[r * V * NV + e] = x;
        continue;
      }
#pragma unroll
      for (int j = 0; j < NV; ++j) {
        int c = col(j);
        float* d = &dst[(r * NV + j) * V];
        if (row_ok[r] && c < p.L) {
          if (V == 4) load_vec4(a, ro + c, d);
          else d[0] = load_scalar(a, ro + c);
        } else {
#pragma unroll
          for (int v = 0; v < V; ++v) d[v] = 0.0f;
        }
      }
    }
  }
  __device__ __forceinline__ void anchor(float (&dst)[VV]) const {
#pragma unroll
    for (int v = 0; v < VV; ++v) dst[v] = 0.0f;
  }
  __device__ __forceinline__ void store(int idx, const float (&val)[VV]) const {
    const TensorArg& a = p.out[idx];
    const int64_t si = a.stride[0];
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
      if (!row_ok[r]) continue;
      const int64_t ro = row_offset(a, r);
      if (si == 0) {                                 // a per-row scalar (reduced output)
        if (lane_in_row == 0) store_scalar(a, ro, val[r * V * NV], false);
        continue;
      }
#pragma unroll
      for (int j = 0; j < NV; ++j) {
        int c = col(j);
        if (c < p.L) {
          if (V == 4) store_vec4(a, ro + c, &val[(r * NV + j) * V], false);
          else store_scalar(a, ro + c, val[(r * NV + j) * V], false);
        }
      }
    }
  }
  __device__ __forceinline__ void row_reduce(int op, float (&acc)[VV]) const {
    float red[RPW];
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
      float x0 = op == M_ROWMAX ? -CUDART_INF_F : (op == M_ROWPROD ? 1.0f : 0.0f);
      float rr = x0;
#pragma unroll
      for (int j = 0; j < NV; ++j) {
        if (col(j) < p.L) {
#pragma unroll
          for (int v = 0; v < V; ++v) {
            float x = acc[(r * NV + j) * V + v];
            if (op == M_ROWMAX) rr = fmaxf(rr, x); else if (op == M_ROWPROD) rr *= x; else rr += x;
          }
        }
      }
      red[r] = rr;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
      for (int r = 0; r < RPW; ++r) {
        float y = __shfl_xor_sync(0xffffffffu, red[r], o);
        if (op == M_ROWMAX) red[r] = fmaxf(red[r], y); else if (op == M_ROWPROD) red[r] *= y; else red[r] += y;
      }
    }
    if (WPR > 1) {                                   // RPW == 1 here
      __syncthreads();                               // previous exchange fully consumed
      if ((threadIdx.x & 31) == 0) xchg[threadIdx.x >> 5] = red[0];
      __syncthreads();
      float t = xchg[0];
#pragma unroll
      for (int w = 1; w < WPR; ++w) {
        float y = xchg[w];
        if (op == M_ROWMAX) t = fmaxf(t, y); else if (op == M_ROWPROD) t *= y; else t += y;
      }
      red[0] = t;
    }
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
      float x = op == M_ROWMEAN ? red[r] / (float)p.L : red[r];
#pragma unroll
      for (int e = 0; e < V * NV; ++e) acc[r * V * NV + e] = x;
    }
  }
};

constexpr int kRowWarpsPerCta = 4;

template <int V, int NV, int WPR, int RPW, class SP>
__global__ void __launch_bounds__(WPR > 1 ? 32 * WPR : 32 * kRowWarpsPerCta)
row_kernel(const __grid_constant__ RowParams p) {
  __shared__ float xchg[WPR > 1 ? WPR : 1];
  RowIO<V, NV, WPR, RPW> io{p};
  io.xchg = xchg;
  uint32_t row0;
  if (WPR > 1) { row0 = blockIdx.x; io.lane_in_row = threadIdx.x; }
  else { row0 = (blockIdx.x * kRowWarpsPerCta + (threadIdx.x >> 5)) * RPW; io.lane_in_row = threadIdx.x & 31; }
  if (row0 >= (uint32_t)p.rows) return;              // whole warps (WPR == 1) or never (WPR > 1)
#pragma unroll
  for (int r = 0; r < RPW; ++r) {
    uint32_t row = row0 + r;
    io.row_ok[r] = row < (uint32_t)p.rows;
    uint32_t lin = io.row_ok[r] ? row : row0;
#pragma unroll
    for (int d = 1; d < kMaxDims; ++d) {
      io.outer[r][d] = 0;
      if (d < p.it.ndim) {
        uint32_t q = fdiv_row(p.it, d, lin);
        io.outer[r][d] = lin - q * p.it.extent[d];
        lin = q;
      }
    }
  }
  run_program<V * NV * RPW, SP>(p.prog, io);
}

template <int V, int NV, int WPR, int RPW>
struct RowLauncher {
  const Launch& L; cudaStream_t st;
  template <class SP> void run() {
    row_kernel<V, NV, WPR, RPW, SP><<<L.grid, L.threads, 0, st>>>(L.row);
  }
};

template <int V, int NV, int WPR, int RPW, bool kStatic>
static void launch_one(const Launch& L, cudaStream_t st) {
  RowLauncher<V, NV, WPR, RPW> F{L, st};
  if (kStatic && L.static_id > 0 && StaticSet<RowStatic>::dispatch(L.static_id, F)) return;
  F.template run<DynProg>();
}

// variant encoding: V * 100000 + NV * 1000 + WPR * 10 + RPW
int launch_row(const Launch& L, cudaStream_t st) {
  switch (L.variant) {
    case 401014: launch_one<4, 1, 1, 4, true>(L, st); break;
    case 402012: launch_one<4, 2, 1, 2, true>(L, st); break;
    case 404011: launch_one<4, 4, 1, 1, true>(L, st); break;
    case 406011: launch_one<4, 6, 1, 1, true>(L, st); break;
    case 408011: launch_one<4, 8, 1, 1, true>(L, st); break;
    case 402081: launch_one<4, 2, 8, 1, false>(L, st); break;
    case 404081: launch_one<4, 4, 8, 1, false>(L, st); break;
    case 408081: launch_one<4, 8, 8, 1, false>(L, st); break;
    case 101014: launch_one<1, 1, 1, 4, false>(L, st); break;
    case 104011: launch_one<1, 4, 1, 1, false>(L, st); break;
    case 116011: launch_one<1, 16, 1, 1, false>(L, st); break;
    case 108081: launch_one<1, 8, 8, 1, false>(L, st); break;
    case 132081: launch_one<1, 32, 8, 1, false>(L, st); break;
    default: return 2;
  }
  return cudaGetLastError() == cudaSuccess ? 0 : 1;
}

bool finalize_row(Launch& L) {
  RowParams& p = L.row;
  int nd = p.it.ndim;
  auto rev = [&](auto* arr) { for (int a = 0, b = nd - 1; a < b; ++a, --b) { auto t = arr[a]; arr[a] = arr[b]; arr[b] = t; } };
  rev(p.it.extent);
  for (int i = 0; i < p.n_in; ++i) rev(p.in[i].stride);
  for (int i = 0; i < p.n_out; ++i) rev(p.out[i].stride);
  int V = p.vec, Lr = p.L;
  int nv = 0, wpr = 1, rpw = 1;
  if (V == 4) {
    int need = (Lr + 127) / 128;                   // vectors per lane with one warp per row
    if (need <= 1) { nv = 1; rpw = 4; }
    else if (need <= 2) { nv = 2; rpw = 2; }
    else if (need <= 8) nv = need <= 4 ? 4 : need <= 6 ? 6 : 8;
    else { wpr = 8; int n8 = (Lr + 1023) / 1024; nv = n8 <= 2 ? 2 : n8 <= 4 ? 4 : 8; if (n8 > 8) return false; }
  } else {
    int need = (Lr + 31) / 32;
    if (need <= 1) { nv = 1; rpw = 4; }
    else if (need <= 16) nv = need <= 4 ? 4 : 16;
    else { wpr = 8; int n8 = (Lr + 255) / 256; nv = n8 <= 8 ? 8 : 32; if (n8 > 32) return false; }
  }
  L.variant = V * 100000 + nv * 1000 + wpr * 10 + rpw;
  int64_t warps = (p.rows + rpw - 1) / rpw;
  L.grid = wpr > 1 ? (int)p.rows : (int)((warps + kRowWarpsPerCta - 1) / kRowWarpsPerCta);
  L.threads = wpr > 1 ? 32 * wpr : 32 * kRowWarpsPerCta;
  L.static_id = (V == 4 && wpr == 1) ? StaticSet<RowStatic>::find(p.prog) : 0;
  set_fastdiv(p.it);
  return true;
}

}  // namespace dnnf
