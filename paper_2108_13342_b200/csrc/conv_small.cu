// fp32 pointwise-convolution / matrix-product blocks with FEW rows (one image of 14 x 14 or 28 x 28 pixels): the
// shapes where the tall-and-skinny tensor-core kernel has no tiles to spread over the GPU and the register-tiled FMA
// kernel runs on a handful of CTAs that each fetch all of W first.
//
// The work is cut as finely as the instruction allows: a CTA owns ONE 16-row x 32-column tile of the result (16 columns where that leaves SMs idle), its eight
// warps split K between them and add their partial sums through shared memory in a fixed order.  No weights are staged:
// a lane reads the eight weight values of its B fragments straight from global memory (L2 serves the re-reads of the
// other row tiles), splits them on the fly, and reads its rows of A with 128-bit loads.  Split TF32 on mma.sync m16n8k8,
// three products per step (lo*hi + hi*lo + hi*hi, fp32 accumulate), the same k order inside an instruction as in the
// single-kernel inverted-residual block.  The block's chain runs on the summed fragments in warp 0.
#include <cuda_runtime.h>

#include <algorithm>

#include "chain.cuh"
#include "conv_params.h"
#include "gemm_params.h"
#include "launch_util.h"
#include "lower.h"

namespace dnnf {

namespace pws {

constexpr int WARPS = 8, THREADS = 32 * WARPS;               // the warps of a CTA split K; NT n-tiles of 8 columns per CTA (2 or 4)

__device__ __forceinline__ void mma_tf32(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void split(float x, uint32_t& hi, uint32_t& lo) {          // activations: cut
  hi = __float_as_uint(x) & 0xffffe000u;
  lo = __float_as_uint(x - __uint_as_float(hi));
}
__device__ __forceinline__ void split_rn(float x, uint32_t& hi, uint32_t& lo) {       // weights: rounded
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(hi) : "f"(x));
  lo = __float_as_uint(x - __uint_as_float(hi));
}

// rows pix0 and pix1 = pix0 + 8 of the result, columns col and col + 1
struct SmallIO {
  static constexpr int VV = 4;
  const GemmParams& p;
  float accv[4];
  uint32_t pix0, pix1, col;
  bool ok0, ok1, okc;
  __device__ __forceinline__ uint32_t off(const TensorArg& a, uint32_t pix) const {
    return (uint32_t)a.base + pix * (uint32_t)a.stride[1] + col * (uint32_t)a.stride[0];
  }
  __device__ __forceinline__ void load(int idx, float (&dst)[4]) const {
    const TensorArg& a = p.in[idx];
    const float* base = reinterpret_cast<const float*>(a.ptr);
    if (a.stride[0] == 0) {
      const float x = ok0 ? __ldg(base + off(a, pix0)) : 0.0f;
      const float y = ok1 ? __ldg(base + off(a, pix1)) : 0.0f;
      dst[0] = dst[1] = x; dst[2] = dst[3] = y;
      return;
    }
    const float2 z = make_float2(0.0f, 0.0f);
    const float2 u = ok0 && okc ? __ldg(reinterpret_cast<const float2*>(base + off(a, pix0))) : z;
    const float2 w = a.stride[1] == 0 ? u : (ok1 && okc ? __ldg(reinterpret_cast<const float2*>(base + off(a, pix1))) : z);
    dst[0] = u.x; dst[1] = u.y; dst[2] = w.x; dst[3] = w.y;
  }
  __device__ __forceinline__ void anchor(float (&dst)[4]) const {
#pragma unroll
    for (int v = 0; v < 4; ++v) dst[v] = accv[v];
  }
  __device__ __forceinline__ void store(int idx, const float (&val)[4]) const {
    const TensorArg& a = p.out[idx];
    float* base = reinterpret_cast<float*>(a.ptr);
    if (ok0 && okc) *reinterpret_cast<float2*>(base + off(a, pix0)) = make_float2(val[0], val[1]);
    if (ok1 && okc) *reinterpret_cast<float2*>(base + off(a, pix1)) = make_float2(val[2], val[3]);
  }
  __device__ __forceinline__ void row_reduce(int, float (&)[4]) const {}
};

__device__ __noinline__ void run_interpreted(const Program& prog, SmallIO& io) { run_program<4, DynProg>(prog, io); }

// K is a multiple of 8; N is even (the last column group of a row tile may hold fewer than 4 n-tiles, the last n-tile
// fewer than 8 columns).
template <int NT, class SP>
__global__ void __launch_bounds__(THREADS) conv_small_kernel(const __grid_constant__ GemmParams p) {
  __shared__ float part[WARPS - 1][NT * 4][32];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int n_groups = (p.N + 8 * NT - 1) / (8 * NT);
  const int mt = blockIdx.x / n_groups, ng = blockIdx.x - mt * n_groups;
  const int r0 = mt * 16 + g, r1 = r0 + 8;
  const bool ok0 = r0 < p.M, ok1 = r1 < p.M;
  const int n0 = ng * 8 * NT;
  const int nt_here = min(NT, (p.N - n0 + 7) >> 3);              // the last n-tile of a row may be narrower than 8 columns
  pdl_launch_dependents();
  pdl_wait();
  const float* X = reinterpret_cast<const float*>(p.A.ptr) + p.A.base;
  const float* W = reinterpret_cast<const float*>(p.B.ptr) + p.B.base;
  const float* x0 = X + (int64_t)(ok0 ? r0 : 0) * p.A.stride_row;
  const float* x1 = X + (int64_t)(ok1 ? r1 : 0) * p.A.stride_row;
  // this warp's share of the 16-wide k blocks
  const int blocks = p.K >> 4, per = (blocks + WARPS - 1) / WARPS;
  const int b_begin = warp * per, b_end = min(blocks, b_begin + per);
  float acc[NT][4];
#pragma unroll
  for (int j = 0; j < NT; ++j) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.0f;
  const float4 z4 = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
  // the loads of block b + 1 are issued before the instructions of block b (the loop is a chain of global-memory
  // latencies otherwise)
  float4 u = z4, w = z4, un = z4, wn = z4;
  float wv[NT][4], wvn[NT][4];
  auto fetch = [&](int b, float4& fu, float4& fw, float (&fv)[NT][4]) {
    const int kb = 16 * b + 4 * t;                                // this lane's four consecutive k
    fu = ok0 ? __ldg(reinterpret_cast<const float4*>(x0 + kb)) : z4;
    fw = ok1 ? __ldg(reinterpret_cast<const float4*>(x1 + kb)) : z4;
    // weights W[kb + {0, 1, 2, 3}][n0 + 8 j + g]: the B fragments of two steps
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      const bool in = j < nt_here && n0 + 8 * j + g < p.N;
      const float* wp = W + (size_t)kb * p.N + n0 + 8 * j + g;
#pragma unroll
      for (int e = 0; e < 4; ++e) fv[j][e] = in ? __ldg(wp + (size_t)e * p.N) : 0.0f;
    }
  };
  if (b_begin < b_end) fetch(b_begin, u, w, wv);
  for (int b = b_begin; b < b_end; ++b) {
    if (b + 1 < b_end) fetch(b + 1, un, wn, wvn);
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      uint32_t h0, h1, h2, h3, l0, l1, l2, l3;
      split(half ? u.z : u.x, h0, l0); split(half ? w.z : w.x, h1, l1);
      split(half ? u.w : u.y, h2, l2); split(half ? w.w : w.y, h3, l3);
      uint32_t bh0[NT], bl0[NT], bh1[NT], bl1[NT];
#pragma unroll
      for (int j = 0; j < NT; ++j) { split_rn(wv[j][2 * half], bh0[j], bl0[j]); split_rn(wv[j][2 * half + 1], bh1[j], bl1[j]); }
      // product by product over the accumulators: consecutive instructions do not depend on each other
#pragma unroll
      for (int j = 0; j < NT; ++j) mma_tf32(acc[j], l0, l1, l2, l3, bh0[j], bh1[j]);
#pragma unroll
      for (int j = 0; j < NT; ++j) mma_tf32(acc[j], h0, h1, h2, h3, bl0[j], bl1[j]);
#pragma unroll
      for (int j = 0; j < NT; ++j) mma_tf32(acc[j], h0, h1, h2, h3, bh0[j], bh1[j]);
    }
    u = un; w = wn;
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) wv[j][e] = wvn[j][e];
  }
  if ((p.K & 8) && warp == WARPS - 1) {                           // a K that is 8 mod 16 ends with one step on k = 16 blocks + 2 t + {0, 1}
    const int kb = 16 * blocks + 2 * t;
    const float2 u = ok0 ? __ldg(reinterpret_cast<const float2*>(x0 + kb)) : make_float2(0.0f, 0.0f);
    const float2 w = ok1 ? __ldg(reinterpret_cast<const float2*>(x1 + kb)) : make_float2(0.0f, 0.0f);
    uint32_t h0, h1, h2, h3, l0, l1, l2, l3;
    split(u.x, h0, l0); split(w.x, h1, l1); split(u.y, h2, l2); split(w.y, h3, l3);
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      const bool in = j < nt_here && n0 + 8 * j + g < p.N;
      const float* wp = W + (size_t)kb * p.N + n0 + 8 * j + g;
      const float w0 = in ? __ldg(wp) : 0.0f, w1 = in ? __ldg(wp + p.N) : 0.0f;
      uint32_t bh0, bl0, bh1, bl1;
      split_rn(w0, bh0, bl0); split_rn(w1, bh1, bl1);
      mma_tf32(acc[j], l0, l1, l2, l3, bh0, bh1);
      mma_tf32(acc[j], h0, h1, h2, h3, bl0, bl1);
      mma_tf32(acc[j], h0, h1, h2, h3, bh0, bh1);
    }
  }
  if (warp > 0) {
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
      for (int v = 0; v < 4; ++v) part[warp - 1][j * 4 + v][lane] = acc[j][v];
  }
  __syncthreads();
  if (warp != 0) return;
  SmallIO io{p};
  io.pix0 = (uint32_t)(ok0 ? r0 : 0); io.pix1 = (uint32_t)(ok1 ? r1 : 0);
  io.ok0 = ok0; io.ok1 = ok1;
#pragma unroll
  for (int j = 0; j < NT; ++j) {
    io.okc = j < nt_here && n0 + 8 * j + 2 * t < p.N;           // N is even: a pair of columns is inside or outside together
    io.col = (uint32_t)(io.okc ? n0 + 8 * j + 2 * t : 0);
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      float sum = acc[j][v];
#pragma unroll
      for (int r = 0; r < WARPS - 1; ++r) sum += part[r][j * 4 + v][lane];
      io.accv[v] = sum;
    }
    if (j >= nt_here) continue;
    if constexpr (SP::n == 0) run_interpreted(p.prog, io);
    else run_program<4, SP>(p.prog, io);
  }
}

}  // namespace pws

static const GemmParams& gp_of(const Launch& L) { return *reinterpret_cast<const GemmParams*>(L.blob.data()); }

// The part of the eligibility test that depends on the problem's shape alone (the planner's cost model for splitting a
// contraction asks it: this kernel, not the FMA kernels, is what an unsplit fp32 contraction of such a shape runs on).
bool conv_small_shape_fits(int64_t M, int64_t N, int64_t K) {
  if (plan_flag(DNNF_PLAN_NO_SMALL_CONV)) return false;
  // (beyond 1024 rows only where the tall-and-skinny tensor-core kernel does not apply, i.e. K x N too large for its
  // resident weights: the 576 -> 160 and 384 -> 64 projections on 6272 pixels ran at 99 and 86 us on the FMA kernels)
  { const char* e = dev_env("DNNF_SMALL_M_MAX"); if (M > (e ? atoi(e) : 65536)) return false; }
  return N % 2 == 0 && K % 8 == 0 && K >= 8;
}

// Taken where the tall-and-skinny kernels have too few rows to fill the GPU.
bool conv_small_eligible(const GemmParams& gp) {
  if (!conv_small_shape_fits(gp.M, gp.N, gp.K)) return false;
  if (gp.A.dtype != 0 || gp.B.dtype != 0) return false;
  if (gp.batch_ext[0] * gp.batch_ext[1] != 1) return false;
  if (gp.A.stride_col != 1 || gp.A.stride_row % 4 || gp.A.base % 4) return false;
  if (gp.B.stride_col != 1 || gp.B.stride_row != gp.N) return false;
  if (gp.n_nd != 1 || gp.m_nd != 1 || gp.b_nd != 1) return false;
  // the chain reads and writes pairs of neighbouring columns: 8-byte aligned wherever it walks along n
  auto pair_ok = [](const TensorArg& a) { return a.dtype == 0 && (a.stride[0] == 0 || (a.stride[0] == 1 && a.base % 2 == 0 && a.stride[1] % 2 == 0)); };
  for (int i = 0; i < gp.n_in; ++i) if (!pair_ok(gp.in[i]) || gp.in[i].mode == 2) return false;
  for (int i = 0; i < gp.n_out; ++i) if (!pair_ok(gp.out[i]) || gp.out[i].stride[0] != 1) return false;
  return true;
}

void conv_small_plan(Launch& L) {
  GemmParams& gp = *reinterpret_cast<GemmParams*>(L.blob.data());
  L.variant = 7;
  L.threads = pws::THREADS;
  L.smem = 0;
  // 16 x 32 tiles; 16 x 16 where those would leave SMs without a CTA
  const int64_t m_tiles = (gp.M + 15) / 16;
  int nt = 4;
  if (m_tiles * ((gp.N + 31) / 32) < sm_count() && gp.N > 16) nt = 2;
  gp.tiles_n = nt;
  L.grid = (int)(m_tiles * ((gp.N + 8 * nt - 1) / (8 * nt)));
  L.static_id = StaticSet<ConvStatic>::find(gp.prog);
}

namespace {
struct SmallLauncher {
  const Launch& L; cudaStream_t st; cudaError_t rc = cudaSuccess;
  template <class SP> void run() {
    if (gp_of(L).tiles_n == 2) rc = launch_pdl(pws::conv_small_kernel<2, SP>, L.grid, pws::THREADS, 0, st, gp_of(L));
    else rc = launch_pdl(pws::conv_small_kernel<4, SP>, L.grid, pws::THREADS, 0, st, gp_of(L));
  }
};
}  // namespace

int conv_small_launch(const Launch& L, cudaStream_t st) {
  SmallLauncher F{L, st};
  if (!(L.static_id > 0 && StaticSet<ConvStatic>::dispatch(L.static_id, F))) F.run<DynProg>();
  return F.rc == cudaSuccess ? 0 : 1;
}

}  // namespace dnnf
