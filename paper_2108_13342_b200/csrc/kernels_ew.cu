// Element-wise families: contiguous chains (one pass, 128-bit accesses) and chains
// with a Shuffle staged through shared memory so that both the load side and the
// store side stay coalesced.
#include "chain.cuh"
#include "ir.h"

namespace dnnf {

__device__ __forceinline__ uint32_t fdiv(const IterSpace& it, int d, uint32_t n) {
  return it.extent[d] == 1 ? n : (__umulhi(n, it.div_m[d]) >> it.div_s[d]);
}

// ---------------------------------------------------------------------------
// Contiguous chain.  Each thread owns U vectors of V elements, U*256*V elements
// per CTA, consecutive lanes on consecutive vectors.
// ---------------------------------------------------------------------------
template <int V, int U>
struct EwIO {
  const EwParams& p;
  uint32_t coord[U][kMaxDims];
  bool valid[U];
  __device__ __forceinline__ int64_t offset(const TensorArg& a, int u) const {
    int64_t off = a.base;
#pragma unroll
    for (int d = 0; d < kMaxDims; ++d)
      if (d < p.it.ndim) off += (int64_t)coord[u][d] * a.stride[d];
    return off;
  }
  __device__ __forceinline__ void load(int idx, float (&dst)[V * U]) const {
    const TensorArg& a = p.in[idx];
    const int inner = p.it.ndim - 1;
    const int64_t si = a.stride[inner];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      if (!valid[u]) {
#pragma unroll
        for (int v = 0; v < V; ++v) dst[u * V + v] = 0.0f;
        continue;
      }
      int64_t off = offset(a, u);
      if (V == 4 && si == 1 && a.mode == 0) {
        load_vec4(a, off, &dst[u * V]);
      } else if (si == 0) {
        float x = load_scalar(a, off);
#pragma unroll
        for (int v = 0; v < V; ++v) dst[u * V + v] = x;
      } else {
#pragma unroll
        for (int v = 0; v < V; ++v) dst[u * V + v] = load_scalar(a, off + v * si);
      }
    }
  }
  __device__ __forceinline__ void anchor(float (&dst)[V * U]) const {
#pragma unroll
    for (int v = 0; v < V * U; ++v) dst[v] = 0.0f;
  }
  __device__ __forceinline__ void store(int idx, const float (&val)[V * U]) const {
    const TensorArg& a = p.out[idx];
    const int inner = p.it.ndim - 1;
    const int64_t si = a.stride[inner];
    const bool exact = p.prog.flags & kProgPureMove;
#pragma unroll
    for (int u = 0; u < U; ++u) {
      if (!valid[u]) continue;
      int64_t off = offset(a, u);
      if (V == 4 && si == 1 && a.mode == 0) store_vec4(a, off, &val[u * V], exact);
      else {
#pragma unroll
        for (int v = 0; v < V; ++v) store_scalar(a, off + v * si, val[u * V + v], exact);
      }
    }
  }
  __device__ __forceinline__ void row_reduce(int, float (&)[V * U]) const {}
};

template <int V, int U>
__global__ void __launch_bounds__(256) ew_kernel(const __grid_constant__ EwParams p) {
  EwIO<V, U> io{p};
  const uint32_t nvec = (uint32_t)(p.total / V);
  const int nd = p.it.ndim;
#pragma unroll
  for (int u = 0; u < U; ++u) {
    uint32_t vi = blockIdx.x * (256u * U) + u * 256u + threadIdx.x;
    io.valid[u] = vi < nvec;
    uint32_t lin = vi;
    // innermost dim counts vectors
    {
      uint32_t e = p.inner_vecs;
      uint32_t q = e == 1 ? lin : (__umulhi(lin, p.inner_m) >> p.inner_s);
      io.coord[u][nd - 1] = (lin - q * e) * V;
      lin = q;
    }
#pragma unroll
    for (int d = kMaxDims - 2; d >= 0; --d) {
      if (d < nd - 1) {
        uint32_t q = fdiv(p.it, d, lin);
        io.coord[u][d] = lin - q * p.it.extent[d];
        lin = q;
      }
    }
  }
  run_program<V * U, kMaxTmp>(p.prog, io);
}

// ---------------------------------------------------------------------------
// Chain with a staged Shuffle.  Iteration dims are ordered so that dim nd-1 is the
// output-contiguous dim (i) and dim nd-2 is the dim along which the staged inputs
// are contiguous (t).  A CTA owns a TT x TI tile: staged inputs are read with
// lanes along t and written to padded shared memory, then every thread evaluates
// the chain on vectors along i, reading staged operands from shared memory and
// all others straight from global memory.
// ---------------------------------------------------------------------------
constexpr int TT = 64, TI = 64, TPITCH = TI + 1;

template <int V>
struct TrIO {
  const EwParams& p;
  const float* smem;       // [n_staged][TT][TPITCH]
  uint32_t outer[kMaxDims];
  uint32_t t0, i0;         // tile origin
  uint32_t tt, ti;         // this thread's element within the tile
  bool valid;
  __device__ __forceinline__ int64_t offset(const TensorArg& a) const {
    const int nd = p.it.ndim;
    int64_t off = a.base + (int64_t)(t0 + tt) * a.stride[nd - 2] + (int64_t)(i0 + ti) * a.stride[nd - 1];
#pragma unroll
    for (int d = 0; d < kMaxDims - 2; ++d)
      if (d < nd - 2) off += (int64_t)outer[d] * a.stride[d];
    return off;
  }
  __device__ __forceinline__ void load(int idx, float (&dst)[V]) const {
    const TensorArg& a = p.in[idx];
    if (!valid) {
#pragma unroll
      for (int v = 0; v < V; ++v) dst[v] = 0.0f;
      return;
    }
    if (a.mode & 1) {
      const float* s = smem + ((a.mode >> 1) * TT + tt) * TPITCH + ti;
#pragma unroll
      for (int v = 0; v < V; ++v) dst[v] = s[v];
      return;
    }
    const int64_t si = a.stride[p.it.ndim - 1];
    int64_t off = offset(a);
    if (V == 4 && si == 1 && a.mode == 0) load_vec4(a, off, dst);
    else if (si == 0) {
      float x = load_scalar(a, off);
#pragma unroll
      for (int v = 0; v < V; ++v) dst[v] = x;
    } else {
#pragma unroll
      for (int v = 0; v < V; ++v) dst[v] = load_scalar(a, off + v * si);
    }
  }
  __device__ __forceinline__ void anchor(float (&dst)[V]) const {
#pragma unroll
    for (int v = 0; v < V; ++v) dst[v] = 0.0f;
  }
  __device__ __forceinline__ void store(int idx, const float (&val)[V]) const {
    if (!valid) return;
    const TensorArg& a = p.out[idx];
    const int64_t si = a.stride[p.it.ndim - 1];
    const bool exact = p.prog.flags & kProgPureMove;
    int64_t off = offset(a);
    if (V == 4 && si == 1 && a.mode == 0) store_vec4(a, off, val, exact);
    else {
#pragma unroll
      for (int v = 0; v < V; ++v) store_scalar(a, off + v * si, val[v], exact);
    }
  }
  __device__ __forceinline__ void row_reduce(int, float (&)[V]) const {}
};

template <int V>
__global__ void __launch_bounds__(256) tr_kernel(const __grid_constant__ EwParams p) {
  extern __shared__ float smem[];
  const int nd = p.it.ndim;
  TrIO<V> io{p, smem};
  uint32_t b = blockIdx.x;
  uint32_t tile_i = b % (uint32_t)p.tiles_i; b /= (uint32_t)p.tiles_i;
  uint32_t tile_t = b % (uint32_t)p.tiles_t; b /= (uint32_t)p.tiles_t;
#pragma unroll
  for (int d = kMaxDims - 3; d >= 0; --d) {
    if (d < nd - 2) {
      uint32_t q = fdiv(p.it, d, b);
      io.outer[d] = b - q * p.it.extent[d];
      b = q;
    }
  }
  io.t0 = tile_t * TT; io.i0 = tile_i * TI;
  const uint32_t ext_t = p.it.extent[nd - 2], ext_i = p.it.extent[nd - 1];

  // Phase 1: staged inputs, lanes along t (their contiguous dim).
  for (int k = 0; k < p.n_in; ++k) {
    const TensorArg& a = p.in[k];
    if (!(a.mode & 1)) continue;
    float* s = smem + (a.mode >> 1) * TT * TPITCH;
    int64_t base = a.base + (int64_t)io.t0 * a.stride[nd - 2] + (int64_t)io.i0 * a.stride[nd - 1];
    for (int d = 0; d < nd - 2; ++d) base += (int64_t)io.outer[d] * a.stride[d];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int ti = warp; ti < TI; ti += 8) {
      bool iok = io.i0 + ti < ext_i;
#pragma unroll
      for (int h = 0; h < TT / 32; ++h) {
        int tt = lane + 32 * h;
        float x = 0.0f;
        if (iok && io.t0 + tt < ext_t) x = load_scalar(a, base + (int64_t)tt * a.stride[nd - 2] + (int64_t)ti * a.stride[nd - 1]);
        s[tt * TPITCH + ti] = x;
      }
    }
  }
  __syncthreads();

  // Phase 2: the chain, vectors along i.
  constexpr int VPR = TI / V;                    // vectors per tile row
  for (int v = threadIdx.x; v < TT * VPR; v += 256) {
    io.tt = v / VPR;
    io.ti = (v % VPR) * V;
    io.valid = (io.t0 + io.tt < ext_t) && (io.i0 + io.ti < ext_i);
    run_program<V, kMaxTmp>(p.prog, io);
  }
}

// ---------------------------------------------------------------------------
int launch_ew(const Launch& L, cudaStream_t st) {
  const EwParams& p = L.ew;
  if (L.family == DNNF_FAMILY_ELEMENTWISE) {
    if (p.vec == 4) ew_kernel<4, 2><<<L.grid, 256, 0, st>>>(p);
    else ew_kernel<1, 4><<<L.grid, 256, 0, st>>>(p);
  } else {
    if (p.vec == 4) tr_kernel<4><<<L.grid, 256, L.smem, st>>>(p);
    else tr_kernel<1><<<L.grid, 256, L.smem, st>>>(p);
  }
  return cudaGetLastError() == cudaSuccess ? 0 : 1;
}

// Host-side launch geometry for the element-wise families (called at plan time).
void finalize_ew(Launch& L) {
  EwParams& p = L.ew;
  int nd = p.it.ndim;
  if (L.family == DNNF_FAMILY_TRANSPOSE) {
    // move tdim to position nd-2
    int td = p.tdim;
    if (td != nd - 2) {
      auto rot = [&](auto* arr) { auto v = arr[td]; for (int d = td; d < nd - 2; ++d) arr[d] = arr[d + 1]; arr[nd - 2] = v; };
      rot(p.it.extent);
      for (int i = 0; i < p.n_in; ++i) rot(p.in[i].stride);
      for (int i = 0; i < p.n_out; ++i) rot(p.out[i].stride);
      p.tdim = nd - 2;
    }
    p.tiles_t = (p.it.extent[nd - 2] + TT - 1) / TT;
    p.tiles_i = (p.it.extent[nd - 1] + TI - 1) / TI;
    int64_t grid = (int64_t)p.tiles_t * p.tiles_i;
    for (int d = 0; d < nd - 2; ++d) grid *= p.it.extent[d];
    int staged = 0;
    for (int i = 0; i < p.n_in; ++i) if (p.in[i].mode == 1) { p.in[i].mode = 1 + 2 * staged; staged++; }
    L.smem = (size_t)staged * TT * TPITCH * sizeof(float);
    L.grid = (int)grid; L.threads = 256;
    L.variant = p.vec;
  } else {
    int U = p.vec == 4 ? 2 : 4;
    int64_t nvec = p.total / p.vec;
    L.grid = (int)((nvec + 256 * U - 1) / (256 * U));
    L.threads = 256;
    L.variant = p.vec;
    p.inner_vecs = p.it.extent[nd - 1] / p.vec;
    fastdiv_for(p.inner_vecs, p.inner_m, p.inner_s);
  }
  set_fastdiv(p.it);
}

}  // namespace dnnf
