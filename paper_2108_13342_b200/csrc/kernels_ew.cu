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
template <int V, int U, bool F32>
struct EwIO {
  const EwParams& p;
  uint32_t coord[U][kMaxDims];
  bool valid[U];
  __device__ __forceinline__ uint32_t offset(const TensorArg& a, int u) const {
    uint32_t off = (uint32_t)a.base;
#pragma unroll
    for (int d = 0; d < kMaxDims; ++d) off += coord[u][d] * (uint32_t)a.stride[d];   // unused dims: coord 0
    return off;
  }
  __device__ __forceinline__ void load(int idx, float (&dst)[V * U]) const {
    const TensorArg& a = p.in[idx];
    const int si = a.stride[0];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      if (!valid[u]) {
#pragma unroll
        for (int v = 0; v < V; ++v) dst[u * V + v] = 0.0f;
        continue;
      }
      uint32_t off = offset(a, u);
      if (V == 4 && si == 1 && a.mode == 0) {
        load_vec4<F32>(a, off, &dst[u * V]);
      } else if (si == 0) {
        float x = load_scalar<F32>(a, off);
#pragma unroll
        for (int v = 0; v < V; ++v) dst[u * V + v] = x;
      } else {
#pragma unroll
        for (int v = 0; v < V; ++v) dst[u * V + v] = load_scalar<F32>(a, off + v * si);
      }
    }
  }
  __device__ __forceinline__ void anchor(float (&dst)[V * U]) const {
#pragma unroll
    for (int v = 0; v < V * U; ++v) dst[v] = 0.0f;
  }
  __device__ __forceinline__ void store(int idx, const float (&val)[V * U]) const {
    pdl_launch_dependents();       // loads are done: the next kernel's CTAs may start arriving (first trigger counts)
    const TensorArg& a = p.out[idx];
    const int si = a.stride[0];
    const bool exact = p.prog.flags & kProgPureMove;
#pragma unroll
    for (int u = 0; u < U; ++u) {
      if (!valid[u]) continue;
      uint32_t off = offset(a, u);
      if (V == 4 && si == 1 && a.mode == 0) store_vec4<F32>(a, off, &val[u * V], exact);
      else {
#pragma unroll
        for (int v = 0; v < V; ++v) store_scalar<F32>(a, off + v * si, val[u * V + v], exact);
      }
    }
  }
  __device__ __forceinline__ void row_reduce(int, float (&)[V * U]) const {}
};

// NOTE: on the device the iteration dims are stored INNERMOST FIRST (dim 0 is the
// contiguous one), so that every index below is a compile-time constant.
template <int V, int U, class SP, bool F32>
__global__ void __launch_bounds__(256) ew_kernel(const __grid_constant__ EwParams p) {
  EwIO<V, U, F32> io{p};
  const uint32_t nvec = (uint32_t)(p.total / V);
#pragma unroll
  for (int u = 0; u < U; ++u) {
    uint32_t vi = blockIdx.x * (256u * U) + u * 256u + threadIdx.x;
    io.valid[u] = vi < nvec;
    uint32_t lin = vi;
    {
      uint32_t e = p.inner_vecs;
      uint32_t q = e == 1 ? lin : (__umulhi(lin, p.inner_m) >> p.inner_s);
      io.coord[u][0] = (lin - q * e) * V;
      lin = q;
    }
#pragma unroll
    for (int d = 1; d < kMaxDims; ++d) {
      io.coord[u][d] = 0;
      if (d < p.it.ndim) {
        uint32_t q = fdiv(p.it, d, lin);
        io.coord[u][d] = lin - q * p.it.extent[d];
        lin = q;
      }
    }
  }
  pdl_wait();
  run_program<V * U, SP>(p.prog, io);
}

// ---------------------------------------------------------------------------
// Chain with a staged Shuffle.  Device dim 0 is the output-contiguous dim (i) and
// dim 1 the dim along which the staged inputs are contiguous (t).  A CTA owns a
// TT x TI tile: staged inputs are read with lanes along t and written to padded
// shared memory, then every thread evaluates the chain on vectors along i,
// reading staged operands from shared memory and all others from global memory.
// ---------------------------------------------------------------------------
constexpr int TT = 64, TI = 64, TPITCH = TI + 1;

template <int V, int K, bool F32>      // K vectors per thread
struct TrIO {
  const EwParams& p;
  const float* smem;       // [n_staged][TT][TPITCH]
  uint32_t outer[kMaxDims];
  uint32_t t0, i0;         // tile origin
  uint32_t tt[K], ti;      // this thread's elements within the tile
  bool valid[K];
  __device__ __forceinline__ uint32_t offset(const TensorArg& a, int k) const {
    uint32_t off = (uint32_t)a.base + (t0 + tt[k]) * (uint32_t)a.stride[1] + (i0 + ti) * (uint32_t)a.stride[0];
#pragma unroll
    for (int d = 2; d < kMaxDims; ++d) off += outer[d] * (uint32_t)a.stride[d];
    return off;
  }
  __device__ __forceinline__ void load(int idx, float (&dst)[V * K]) const {
    const TensorArg& a = p.in[idx];
    const int si = a.stride[0];
#pragma unroll
    for (int k = 0; k < K; ++k) {
      if (!valid[k]) {
#pragma unroll
        for (int v = 0; v < V; ++v) dst[k * V + v] = 0.0f;
        continue;
      }
      if (a.mode & 1) {
        const float* s = smem + (((a.mode >> 1) & 1) * TT + tt[k]) * TPITCH + ti;
#pragma unroll
        for (int v = 0; v < V; ++v) dst[k * V + v] = s[v];
        continue;
      }
      uint32_t off = offset(a, k);
      if (V == 4 && si == 1 && a.mode == 0) load_vec4<F32>(a, off, &dst[k * V]);
      else if (si == 0) {
        float x = load_scalar<F32>(a, off);
#pragma unroll
        for (int v = 0; v < V; ++v) dst[k * V + v] = x;
      } else {
#pragma unroll
        for (int v = 0; v < V; ++v) dst[k * V + v] = load_scalar<F32>(a, off + v * si);
      }
    }
  }
  __device__ __forceinline__ void anchor(float (&dst)[V * K]) const {
#pragma unroll
    for (int v = 0; v < V * K; ++v) dst[v] = 0.0f;
  }
  __device__ __forceinline__ void store(int idx, const float (&val)[V * K]) const {
    const TensorArg& a = p.out[idx];
    const int si = a.stride[0];
    const bool exact = p.prog.flags & kProgPureMove;
#pragma unroll
    for (int k = 0; k < K; ++k) {
      if (!valid[k]) continue;
      uint32_t off = offset(a, k);
      if (V == 4 && si == 1 && a.mode == 0) store_vec4<F32>(a, off, &val[k * V], exact);
      else {
#pragma unroll
        for (int v = 0; v < V; ++v) store_scalar<F32>(a, off + v * si, val[k * V + v], exact);
      }
    }
  }
  __device__ __forceinline__ void row_reduce(int, float (&)[V * K]) const {}
};

template <int V, class SP, bool F32>
__global__ void __launch_bounds__(256) tr_kernel(const __grid_constant__ EwParams p) {
  extern __shared__ float smem[];
  pdl_launch_dependents();
  constexpr int K = 4;
  TrIO<V, K, F32> io{p, smem};
  uint32_t b = blockIdx.x;
  uint32_t u = fd_div(b, p.fd_tiles_i);
  const uint32_t tile_i = b - u * (uint32_t)p.tiles_i; b = u;
  u = fd_div(b, p.fd_tiles_t);
  const uint32_t tile_t = b - u * (uint32_t)p.tiles_t; b = u;
#pragma unroll
  for (int d = 2; d < kMaxDims; ++d) {
    io.outer[d] = 0;
    if (d < p.it.ndim) {
      uint32_t q = fdiv(p.it, d, b);
      io.outer[d] = b - q * p.it.extent[d];
      b = q;
    }
  }
  io.t0 = tile_t * TT; io.i0 = tile_i * TI;
  const uint32_t ext_t = p.it.extent[1], ext_i = p.it.extent[0];

  pdl_wait();
  // Phase 1: staged inputs, lanes along t (their contiguous dim).
  for (int k = 0; k < p.n_in; ++k) {
    const TensorArg& a = p.in[k];
    if (!(a.mode & 1)) continue;
    float* s = smem + ((a.mode >> 1) & 1) * TT * TPITCH;
    uint32_t base = (uint32_t)a.base + io.t0 * (uint32_t)a.stride[1] + io.i0 * (uint32_t)a.stride[0];
#pragma unroll
    for (int d = 2; d < kMaxDims; ++d) base += io.outer[d] * (uint32_t)a.stride[d];
    const bool full = io.t0 + TT <= ext_t && io.i0 + TI <= ext_i;
    if (V == 4 && a.mode >= 5 && full) {          // 128-bit loads along t (host verified alignment)
#pragma unroll
      for (int r = 0; r < (TT / 4) * TI / 256; ++r) {
        int idx = threadIdx.x + 256 * r;
        int t4 = (idx % (TT / 4)) * 4, ti = idx / (TT / 4);
        float x[4];
        load_vec4<F32>(a, base + t4 + ti * (uint32_t)a.stride[0], x);
#pragma unroll
        for (int j = 0; j < 4; ++j) s[(t4 + j) * TPITCH + ti] = x[j];
      }
    } else {
      const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
      for (int ti = warp; ti < TI; ti += 8) {
        bool iok = io.i0 + ti < ext_i;
#pragma unroll
        for (int h = 0; h < TT / 32; ++h) {
          int tt = lane + 32 * h;
          float x = 0.0f;
          if (iok && io.t0 + tt < ext_t) x = load_scalar<F32>(a, base + tt * (uint32_t)a.stride[1] + ti * (uint32_t)a.stride[0]);
          s[tt * TPITCH + ti] = x;
        }
      }
    }
  }
  __syncthreads();

  // Phase 2: the chain, vectors along i.
  if (V == 4) {
    io.ti = (threadIdx.x % (TI / 4)) * 4;
#pragma unroll
    for (int k = 0; k < K; ++k) {
      io.tt[k] = threadIdx.x / (TI / 4) + (256 / (TI / 4)) * k;
      io.valid[k] = (io.t0 + io.tt[k] < ext_t) && (io.i0 + io.ti < ext_i);
    }
    run_program<V * K, SP>(p.prog, io);
  } else {
    for (int r = 0; r < TT * TI / (256 * K); ++r) {
      io.ti = threadIdx.x % TI;
#pragma unroll
      for (int k = 0; k < K; ++k) {
        io.tt[k] = threadIdx.x / TI + (256 / TI) * (r * K + k);
        io.valid[k] = (io.t0 + io.tt[k] < ext_t) && (io.i0 + io.ti < ext_i);
      }
      run_program<V * K, SP>(p.prog, io);
    }
  }
}

// ---------------------------------------------------------------------------
// Vectors per thread for interpreted programs.
constexpr int kDynU = 2;     // (4 was measured: occupancy halves and it gets slower)

template <bool F32>
struct EwLauncher {
  const Launch& L; cudaStream_t st;
  template <class SP> void run() {
    if (SP::n == 0) launch_pdl(ew_kernel<4, kDynU, SP, F32>, L.grid, 256, 0, st, L.ew);
    else launch_pdl(ew_kernel<4, 2, SP, F32>, L.grid, 256, 0, st, L.ew);
  }
};
template <bool F32>
struct TrLauncher {
  const Launch& L; cudaStream_t st;
  template <class SP> void run() { launch_pdl(tr_kernel<4, SP, F32>, L.grid, 256, L.smem, st, L.ew); }
};

static bool all_f32(const EwParams& p) {
  for (int i = 0; i < p.n_in; ++i) if (p.in[i].dtype != 0) return false;
  for (int i = 0; i < p.n_out; ++i) if (p.out[i].dtype != 0) return false;
  return true;
}

int launch_ew(const Launch& L, cudaStream_t st) {
  const EwParams& p = L.ew;
  if (p.vec == 4 && L.family == DNNF_FAMILY_TRANSPOSE) {
    if (all_f32(p)) {
      TrLauncher<true> F{L, st};
      if (!(L.static_id > 0 && StaticSet<TrStatic>::dispatch(L.static_id, F))) F.run<DynProg>();
    } else {
      TrLauncher<false> F{L, st};
      if (!(L.static_id > 0 && StaticSet<TrStatic>::dispatch(L.static_id, F))) F.run<DynProg>();
    }
  } else if (p.vec == 4) {
    if (all_f32(p)) {
      EwLauncher<true> F{L, st};
      if (!(L.static_id > 0 && StaticSet<EwStatic>::dispatch(L.static_id, F))) F.run<DynProg>();
    } else {
      EwLauncher<false> F{L, st};
      if (!(L.static_id > 0 && StaticSet<EwStatic>::dispatch(L.static_id, F))) F.run<DynProg>();
    }
  } else {
    if (L.family == DNNF_FAMILY_ELEMENTWISE) launch_pdl(ew_kernel<1, 4, DynProg, false>, L.grid, 256, 0, st, p);
    else launch_pdl(tr_kernel<1, DynProg, false>, L.grid, 256, L.smem, st, p);
  }
  return cudaGetLastError() == cudaSuccess ? 0 : 1;
}

// Host-side launch geometry for the element-wise families (called at plan time).
// Reverses the dim order for the device (innermost first).
void finalize_ew(Launch& L) {
  EwParams& p = L.ew;
  int nd = p.it.ndim;
  if (L.family == DNNF_FAMILY_TRANSPOSE) {
    int td = p.tdim;                         // move tdim next to the innermost dim
    if (td != nd - 2) {
      auto rot = [&](auto* arr) { auto v = arr[td]; for (int d = td; d < nd - 2; ++d) arr[d] = arr[d + 1]; arr[nd - 2] = v; };
      rot(p.it.extent);
      for (int i = 0; i < p.n_in; ++i) rot(p.in[i].stride);
      for (int i = 0; i < p.n_out; ++i) rot(p.out[i].stride);
      p.tdim = nd - 2;
    }
  }
  auto rev = [&](auto* arr) { for (int a = 0, b = nd - 1; a < b; ++a, --b) { auto t = arr[a]; arr[a] = arr[b]; arr[b] = t; } };
  rev(p.it.extent);
  for (int i = 0; i < p.n_in; ++i) rev(p.in[i].stride);
  for (int i = 0; i < p.n_out; ++i) rev(p.out[i].stride);
  if (L.family == DNNF_FAMILY_TRANSPOSE) {
    p.tiles_t = (p.it.extent[1] + TT - 1) / TT;
    p.tiles_i = (p.it.extent[0] + TI - 1) / TI;
    p.fd_tiles_t = make_fastdiv((uint32_t)p.tiles_t); p.fd_tiles_i = make_fastdiv((uint32_t)p.tiles_i);
    int64_t grid = (int64_t)p.tiles_t * p.tiles_i;
    for (int d = 2; d < nd; ++d) grid *= p.it.extent[d];
    int staged = 0;
    for (int i = 0; i < p.n_in; ++i) if (p.in[i].mode == 1) {
      TensorArg& a = p.in[i];
      bool v4 = p.vec == 4 && a.base % 4 == 0 && a.stride[1] == 1 && p.it.extent[1] % 4 == 0;
      for (int d = 0; d < nd; ++d) if (d != 1 && a.stride[d] % 4) v4 = false;
      a.mode = 1 + 2 * staged + (v4 ? 4 : 0);          // bit0 staged, bit1 slot, bit2 vector loads
      staged++;
    }
    L.smem = (size_t)staged * TT * TPITCH * sizeof(float);
    L.grid = (int)grid; L.threads = 256;
  }
  L.static_id = p.vec != 4 ? 0 : (L.family == DNNF_FAMILY_TRANSPOSE ? StaticSet<TrStatic>::find(p.prog) : StaticSet<EwStatic>::find(p.prog));
  if (L.family != DNNF_FAMILY_TRANSPOSE) {
    int U = p.vec == 4 ? (L.static_id > 0 ? 2 : kDynU) : 4;
    int64_t nvec = p.total / p.vec;
    L.grid = (int)((nvec + 256 * U - 1) / (256 * U));
    L.threads = 256;
    p.inner_vecs = p.it.extent[0] / p.vec;
    fastdiv_for(p.inner_vecs, p.inner_m, p.inner_s);
  }
  L.variant = p.vec * 100 + L.static_id;
  set_fastdiv(p.it);
}

}  // namespace dnnf
