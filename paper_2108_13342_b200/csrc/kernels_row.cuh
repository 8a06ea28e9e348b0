// Row family: a chain around a reduction over the last axis (Softmax, LayerNorm,
// ReduceSum/Mean/Max/Prod).  The whole row lives in registers from the first load
// to the last store: a warp (rows up to 1024 elements) or a CTA (up to 8192) owns
// a row -- short rows are processed RPW at a time per warp so that enough loads
// are in flight -- reductions are warp shuffles (plus one shared-memory exchange
// for CTA-wide rows), and the pre- and post-chains run on the register-resident row.
#pragma once
#include "chain.cuh"
#include "ir.h"

namespace dnnf {

__device__ __forceinline__ uint32_t fdiv_row(const IterSpace& it, int d, uint32_t n) {
  return it.extent[d] == 1 ? n : (__umulhi(n, it.div_m[d]) >> it.div_s[d]);
}

// Device dim 0 is the row (length L); dims 1.. are the outer dims, innermost first.
// NV vectors of V elements per thread and row; RPW rows per warp; WPR warps per row.
template <int V, int NV, int WPR, int RPW, bool F32>
struct RowIO {
  static constexpr int VV = V * NV * RPW;
  const RowParams& p;
  uint32_t outer[kMaxDims];        // coordinates of the warp's first row; its other rows follow along dim 1
  bool row_ok[RPW];
  int lane_in_row;                 // 0 .. 32*WPR-1
  float* xchg;                     // shared memory, 2 x WPR floats (WPR > 1)
  mutable int xslot = 0;
  __device__ __forceinline__ int col(int j) const { return (j * 32 * WPR + lane_in_row) * V; }
  __device__ __forceinline__ uint32_t row_offset(const TensorArg& a, int r) const {
    uint32_t off = (uint32_t)a.base + (uint32_t)r * (uint32_t)a.stride[1];
#pragma unroll
    for (int d = 1; d < kMaxDims; ++d) off += outer[d] * (uint32_t)a.stride[d];      // unused dims: coord 0
    return off;
  }
  __device__ __forceinline__ void load(int idx, float (&dst)[VV]) const {
    const TensorArg& a = p.in[idx];
    const int si = a.stride[0];
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
      const uint32_t ro = row_offset(a, r);
      if (si == 0) {
        float x = row_ok[r] ? load_scalar<F32>(a, ro) : 0.0f;
#pragma unroll
        for (int e = 0; e < V * NV; ++e) dst[r * V * NV + e] = x;
        continue;
      }
#pragma unroll
      for (int j = 0; j < NV; ++j) {
        int c = col(j);
        float* d = &dst[(r * NV + j) * V];
        if (row_ok[r] && c < p.L) {
          if (V == 4) load_vec4<F32>(a, ro + c, d);
          else d[0] = load_scalar<F32>(a, ro + c);
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
    const int si = a.stride[0];
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
      if (!row_ok[r]) continue;
      const uint32_t ro = row_offset(a, r);
      if (si == 0) {                                 // a per-row scalar (reduced output)
        if (lane_in_row == 0) store_scalar<F32>(a, ro, val[r * V * NV], false);
        continue;
      }
#pragma unroll
      for (int j = 0; j < NV; ++j) {
        int c = col(j);
        if (c < p.L) {
          if (V == 4) store_vec4<F32>(a, ro + c, &val[(r * NV + j) * V], false);
          else store_scalar<F32>(a, ro + c, val[(r * NV + j) * V], false);
        }
      }
    }
  }
  // Running sum along the row (CumSum).  The row's elements sit in scan order first inside a thread's vector, then
  // across the lanes (and warps) of one chunk of 32 * WPR vectors, then across the NV chunks: a serial scan of the
  // vector, a shuffle scan of the vector totals, one shared-memory exchange of the warp totals, and a carry from
  // chunk to chunk.  Exclusive: each element gets the sum of those before it; reverse: scan order runs from the far end.
  __device__ __forceinline__ void row_scan(int op, float (&acc)[VV]) const {
    const bool excl = op == M_ROWSCAN_X || op == M_ROWSCAN_RX, rev = op == M_ROWSCAN_R || op == M_ROWSCAN_RX;
    const int lane = threadIdx.x & 31;
    pdl_launch_dependents();
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
      float carry = 0.0f;
#pragma unroll
      for (int jj = 0; jj < NV; ++jj) {
        const int j = rev ? NV - 1 - jj : jj;
        float* a = &acc[(r * NV + j) * V];
        const bool inside = col(j) < p.L;
        float run = 0.0f;
#pragma unroll
        for (int vv = 0; vv < V; ++vv) {
          const int v = rev ? V - 1 - vv : vv;
          const float x = inside ? a[v] : 0.0f;
          a[v] = excl ? run : run + x;
          run += x;
        }
        float incl = run;                              // inclusive scan of the vector totals over the warp's lanes
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const float y = rev ? __shfl_down_sync(0xffffffffu, incl, o) : __shfl_up_sync(0xffffffffu, incl, o);
          if (rev ? lane + o < 32 : lane >= o) incl += y;
        }
        float before = rev ? __shfl_down_sync(0xffffffffu, incl, 1) : __shfl_up_sync(0xffffffffu, incl, 1);
        if (lane == (rev ? 31 : 0)) before = 0.0f;
        float chunk_total = __shfl_sync(0xffffffffu, incl, rev ? 0 : 31);
        if (WPR > 1) {
          float* x = xchg + xslot * WPR;
          xslot ^= 1;
          const int warp = threadIdx.x >> 5;
          if (lane == 0) x[warp] = chunk_total;
          __syncthreads();
          float wb = 0.0f, tot = 0.0f;
#pragma unroll
          for (int w = 0; w < WPR; ++w) {
            const float y = x[w];
            tot += y;
            if (rev ? w > warp : w < warp) wb += y;
          }
          before += wb;
          chunk_total = tot;
        }
#pragma unroll
        for (int v = 0; v < V; ++v) a[v] += before + carry;
        carry += chunk_total;
      }
    }
  }
  __device__ __forceinline__ void row_reduce(int op, float (&acc)[VV]) const {
    if (op >= M_ROWSCAN) { row_scan(op, acc); return; }
    // The row's loads have been issued by now: let the next kernel's CTAs start arriving.  (Triggering at
    // kernel entry parks them on the SMs for this kernel's whole load latency, where they take the
    // slots of independent kernels that could run.)  Only the first trigger of a CTA counts.
    pdl_launch_dependents();
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
      // two exchange areas used in turn: the barrier of this exchange also tells that everybody has
      // finished reading the one before, so one barrier per reduction is enough
      float* x = xchg + xslot * WPR;
      xslot ^= 1;
      if ((threadIdx.x & 31) == 0) x[threadIdx.x >> 5] = red[0];
      __syncthreads();
      float t = x[0];
#pragma unroll
      for (int w = 1; w < WPR; ++w) {
        float y = x[w];
        if (op == M_ROWMAX) t = fmaxf(t, y); else if (op == M_ROWPROD) t *= y; else t += y;
      }
      red[0] = t;
    }
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
      float x = op == M_ROWMEAN ? red[r] * p.inv_L : red[r];
#pragma unroll
      for (int e = 0; e < V * NV; ++e) acc[r * V * NV + e] = x;
    }
  }
};

constexpr int kRowWarpsPerCta = 4;

template <int V, int NV, int WPR, int RPW, class SP, bool F32>
__global__ void __launch_bounds__(WPR > 1 ? 32 * WPR : 32 * kRowWarpsPerCta)
row_kernel(const __grid_constant__ RowParams p) {
  __shared__ float xchg[WPR > 1 ? 2 * WPR : 1];
  RowIO<V, NV, WPR, RPW, F32> io{p};
  io.xchg = xchg;
  uint32_t row0;
  if (WPR > 1) { row0 = blockIdx.x; io.lane_in_row = threadIdx.x; }
  else { row0 = (blockIdx.x * kRowWarpsPerCta + (threadIdx.x >> 5)) * RPW; io.lane_in_row = threadIdx.x & 31; }
  if (row0 >= (uint32_t)p.rows) return;              // whole warps (WPR == 1) or never (WPR > 1)
#pragma unroll
  for (int r = 0; r < RPW; ++r) io.row_ok[r] = row0 + r < (uint32_t)p.rows;
  {
    uint32_t lin = row0;
#pragma unroll
    for (int d = 1; d < kMaxDims; ++d) {
      io.outer[d] = 0;
      if (d < p.it.ndim) {
        uint32_t q = fdiv_row(p.it, d, lin);
        io.outer[d] = lin - q * p.it.extent[d];
        lin = q;
      }
    }
  }
  pdl_wait();
  run_program<V * NV * RPW, SP>(p.prog, io);
}

template <int V, int NV, int WPR, int RPW, bool F32>
struct RowLauncher {
  const Launch& L; cudaStream_t st;
  template <class SP> void run() {
    launch_pdl(row_kernel<V, NV, WPR, RPW, SP, F32>, L.grid, L.threads, 0, st, L.row);
  }
};

static inline bool all_f32(const RowParams& p) {
  for (int i = 0; i < p.n_in; ++i) if (p.in[i].dtype != 0) return false;
  for (int i = 0; i < p.n_out; ++i) if (p.out[i].dtype != 0) return false;
  return true;
}

template <int V, int NV, int WPR, int RPW, bool kStatic>
static void launch_one(const Launch& L, cudaStream_t st) {
  if (kStatic && all_f32(L.row)) {
    RowLauncher<V, NV, WPR, RPW, true> F{L, st};
    if (L.static_id > 0 && StaticSet<RowStatic>::dispatch(L.static_id, F)) return;
    F.template run<DynProg>();
  } else {
    RowLauncher<V, NV, WPR, RPW, false> F{L, st};
    if (kStatic && L.static_id > 0 && StaticSet<RowStatic>::dispatch(L.static_id, F)) return;
    F.template run<DynProg>();
  }
}

}  // namespace dnnf
