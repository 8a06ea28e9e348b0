// A whole inverted-residual block as ONE kernel (an extension beyond Table 3, which keeps two Many-to-Many
// operators apart): pointwise expansion + chain -> depthwise 3x3 + chain -> pointwise projection + chain, fp32 NHWC.
// Under the paper's rules the block is three kernels and the expanded tensor travels through HBM twice; here it
// lives only in shared memory: a CTA owns an 8 x 16 tile of output pixels, computes the expansion on the tile plus
// its one-pixel halo (the halo is recomputed by the neighbouring tiles), applies the depthwise filter out of shared
// memory and feeds the result straight into the projection.
//
// Both pointwise convolutions run on warp-level tensor-core instructions (mma.sync m16n8k8, TF32 inputs, fp32
// accumulate) with every operand split in two, x = hi + lo, and the three products lo*hi + hi*lo + hi*hi summed:
// the error per product is below 2^-20 relative, within the 1e-5 parity bar of fp32 blocks.  A is split with a mask
// on the fly, the weights once per CTA into fragment order.  The depthwise stage computes each lane's results
// directly in the A-fragment layout of the projection (lane (g, t) owns pixels g and g + 8 of a 16-pixel tile and
// four consecutive channels), so its output never goes back to shared memory.  Every stage hands over through
// __syncthreads; there is no mbarrier, bulk copy or tensor memory in this kernel.
//
// Stage programs: the chains behind the three anchors are the blocks' own micro-op programs.  Operands of the first
// two must not depend on the pixel (batch-norm scale and shift); the last one takes any operand of a pointwise
// convolution block (the residual).
#include <cuda_runtime.h>

#include <algorithm>
#include <set>

#include "chain.cuh"
#include "conv_params.h"
#include "gemm_params.h"
#include "launch_util.h"
#include "lower.h"

namespace dnnf {

int lower_contraction(const Graph& g, const std::vector<int>& ops, uint32_t flags, int anchor, Block& out, std::string& why);

namespace mb {

constexpr int THREADS = 512, WARPS = 16;
constexpr int TH = 8, TW = 16, HH = TH + 2, HW = TW + 2, HALO = HH * HW, M1 = (HALO + 15) / 16;   // 180 halo pixels, 12 row tiles
constexpr int kSmemMax = 227 * 1024;

struct Params {
  int32_t N, H, W, Cin, Ce, Cout;
  int32_t tiles_w, tiles_h, total_tiles;
  const float *x, *w1, *kd, *w3;
  Program prog1, prog2, prog3;
  int32_t n_in1, n_in2, n_in3, n_out3;
  TensorArg in1[kMaxIn], in2[kMaxIn];        // per-channel operands: element c at base + c * stride[0]
  TensorArg in3[kMaxIn], out3[kMaxOut];      // stride[0]: channel, stride[1]: pixel (n, h, w flattened)
  uint32_t static_mask;                      // bit 0: all weights and per-channel operands are external inputs of the graph
};

__device__ __forceinline__ void mma_tf32(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float tf32_round(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return __uint_as_float(r);
}
// Order of k inside an instruction is free as long as A and B agree: lane (g, t) supplies k = 16 b + 4 t + {0, 1} to
// step 2 b and k = 16 b + 4 t + {2, 3} to step 2 b + 1, i.e. one 128-bit piece of a row feeds two steps; a K that is
// 8 mod 16 ends with one step on k = 16 b + 2 t + {0, 1}.
__device__ __forceinline__ int lane_k0(int s, int t, int K) {
  const int b = s >> 1;
  if (16 * b + 16 <= K) return 16 * b + 4 * t + 2 * (s & 1);
  return 16 * b + 2 * t;
}
// 16-byte asynchronous copy global -> shared; src_bytes = 0 writes zeros
__device__ __forceinline__ void cp_async_16(float* dst, const float* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void split(float x, uint32_t& hi, uint32_t& lo) {
  hi = __float_as_uint(x) & 0xffffe000u;
  lo = __float_as_uint(x - __uint_as_float(hi));
}

// weights [K x N] row-major -> fragment order [K / 8][N / 8][32 lanes] {hi(k0), hi(k0 + 1), lo(k0), lo(k0 + 1)}
__device__ __forceinline__ void make_fragments(float4* dst, const float* W, int K, int N) {
  const int S = K >> 3, NT = N >> 3;
  for (int i = threadIdx.x; i < S * NT * 32; i += THREADS) {
    const int l = i & 31, j = (i >> 5) % NT, s = (i >> 5) / NT;
    const int k0 = lane_k0(s, l & 3, K), n = 8 * j + (l >> 2);
    const float w0 = __ldg(W + (size_t)k0 * N + n), w1 = __ldg(W + (size_t)(k0 + 1) * N + n);
    const float h0 = tf32_round(w0), h1 = tf32_round(w1);
    dst[i] = make_float4(h0, h1, tf32_round(w0 - h0), tf32_round(w1 - h1));
  }
}

// ---- stage 1: expansion result (rows r0 and r0 + 8 of the halo tile, columns col and col + 1) -> expanded tile ----
struct ExpandIO {
  static constexpr int VV = 4;
  const float* vecs; int vec_pitch;        // staged per-channel operands
  float* es; int ep;                       // expanded tile, pitch in floats
  float accv[4];
  int r0, col;
  bool keep0, keep1, in0, in1;             // row exists in the halo tile / pixel lies inside the image
  __device__ __forceinline__ void load(int idx, float (&dst)[4]) const {
    const float2 u = *reinterpret_cast<const float2*>(vecs + idx * vec_pitch + col);
    dst[0] = u.x; dst[1] = u.y; dst[2] = u.x; dst[3] = u.y;
  }
  __device__ __forceinline__ void anchor(float (&dst)[4]) const {
#pragma unroll
    for (int v = 0; v < 4; ++v) dst[v] = accv[v];
  }
  // the depthwise filter pads the EXPANDED tensor with zeros: positions outside the image hold 0, not chain(0)
  __device__ __forceinline__ void store(int, const float (&val)[4]) const {
    if (keep0) *reinterpret_cast<float2*>(es + r0 * ep + col) = in0 ? make_float2(val[0], val[1]) : make_float2(0.0f, 0.0f);
    if (keep1) *reinterpret_cast<float2*>(es + (r0 + 8) * ep + col) = in1 ? make_float2(val[2], val[3]) : make_float2(0.0f, 0.0f);
  }
  __device__ __forceinline__ void row_reduce(int, float (&)[4]) const {}
};

// ---- stage 2: depthwise result of one pixel, four consecutive channels ch .. ch + 3 -> registers ----
struct DwIO2 {
  static constexpr int VV = 4;
  const float* vecs; int vec_pitch;
  float accv[4];
  float res[4];
  int ch;
  __device__ __forceinline__ void load(int idx, float (&dst)[4]) const {
    const float4 u = *reinterpret_cast<const float4*>(vecs + idx * vec_pitch + ch);
    dst[0] = u.x; dst[1] = u.y; dst[2] = u.z; dst[3] = u.w;
  }
  __device__ __forceinline__ void anchor(float (&dst)[4]) const {
#pragma unroll
    for (int v = 0; v < 4; ++v) dst[v] = accv[v];
  }
  __device__ __forceinline__ void store(int, const float (&val)[4]) {
#pragma unroll
    for (int v = 0; v < 4; ++v) res[v] = val[v];
  }
  __device__ __forceinline__ void row_reduce(int, float (&)[4]) const {}
};

// ---- stage 3: projection result (pixels pix0, pix1; columns col, col + 1) -> the block's outputs ----
struct ProjectIO {
  static constexpr int VV = 4;
  const Params& p;
  const float* vecs; int vec_pitch; uint32_t vec_mask;
  float accv[4];
  uint32_t pix0, pix1, col;
  bool ok0, ok1;
  __device__ __forceinline__ uint32_t off(const TensorArg& a, uint32_t pix) const {
    return (uint32_t)a.base + pix * (uint32_t)a.stride[1] + col * (uint32_t)a.stride[0];
  }
  __device__ __forceinline__ void load(int idx, float (&dst)[4]) const {
    if ((vec_mask >> idx) & 1u) {
      const float2 u = *reinterpret_cast<const float2*>(vecs + idx * vec_pitch + col);
      dst[0] = u.x; dst[1] = u.y; dst[2] = u.x; dst[3] = u.y;
      return;
    }
    const TensorArg& a = p.in3[idx];
    const float* base = reinterpret_cast<const float*>(a.ptr);
    if (a.stride[0] == 0) {
      const float x = ok0 ? __ldg(base + off(a, pix0)) : 0.0f;
      const float y = ok1 ? __ldg(base + off(a, pix1)) : 0.0f;
      dst[0] = dst[1] = x; dst[2] = dst[3] = y;
      return;
    }
    const float2 z = make_float2(0.0f, 0.0f);
    const float2 u = ok0 ? __ldg(reinterpret_cast<const float2*>(base + off(a, pix0))) : z;
    const float2 w = ok1 ? __ldg(reinterpret_cast<const float2*>(base + off(a, pix1))) : z;
    dst[0] = u.x; dst[1] = u.y; dst[2] = w.x; dst[3] = w.y;
  }
  __device__ __forceinline__ void anchor(float (&dst)[4]) const {
#pragma unroll
    for (int v = 0; v < 4; ++v) dst[v] = accv[v];
  }
  __device__ __forceinline__ void store(int idx, const float (&val)[4]) const {
    const TensorArg& a = p.out3[idx];
    float* base = reinterpret_cast<float*>(a.ptr);
    if (ok0) *reinterpret_cast<float2*>(base + off(a, pix0)) = make_float2(val[0], val[1]);
    if (ok1) *reinterpret_cast<float2*>(base + off(a, pix1)) = make_float2(val[2], val[3]);
  }
  __device__ __forceinline__ void row_reduce(int, float (&)[4]) const {}
};

__device__ __noinline__ void interp1(const Program& prog, ExpandIO& io) { run_program<4, DynProg>(prog, io); }
__device__ __noinline__ void interp2(const Program& prog, DwIO2& io) { run_program<4, DynProg>(prog, io); }
__device__ __noinline__ void interp3(const Program& prog, ProjectIO& io) { run_program<4, DynProg>(prog, io); }

// Shared-memory layout (bytes, all 16-byte aligned), computed the same way on the host.
struct Layout {
  int w1f, w3f, kd, vec1, vec2, vec3, xs, es, total;
  int xp, ep;     // pitches in floats
};
__host__ __device__ inline Layout layout_of(int Cin, int Ce, int Cout) {
  Layout L{};
  int o = 0;
  L.w1f = o; o += Cin * Ce * 8;
  L.w3f = o; o += Ce * Cout * 8;
  L.kd = o; o += 9 * Ce * 4;
  L.vec1 = o; o += kMaxIn * Ce * 4;
  L.vec2 = o; o += kMaxIn * Ce * 4;
  L.vec3 = o; o += kMaxIn * Cout * 4;
  L.xp = Cin + 4; L.ep = Ce + 4;
  L.xs = o; o += M1 * 16 * L.xp * 4;                   // the halo tile of X
  // the expanded tile; after stage 2 its place takes the partial sums of the projection: 4 pixel groups x 4 channel
  // quarters x (2 NT3 x 4 <= 32) values x 32 lanes of fp32, which a narrow expansion alone would not hold
  L.es = o; o += HALO * L.ep * 4 > 16 * 32 * 32 * 4 ? HALO * L.ep * 4 : 16 * 32 * 32 * 4;
  L.total = o;
  return L;
}

// NT3 = Cout / 8.  SP1 / SP2 / SP3: compile-time tables of the three chains, or DynProg (interpreted).
template <int NT3, class SP1, class SP2, class SP3>
__global__ void __launch_bounds__(THREADS, 1) mbconv_kernel(const __grid_constant__ Params p) {
  extern __shared__ __align__(16) uint8_t smem[];
  const int Cin = p.Cin, Ce = p.Ce, Cout = p.Cout;
  const Layout L = layout_of(Cin, Ce, Cout);
  float4* w1f = reinterpret_cast<float4*>(smem + L.w1f);
  float4* w3f = reinterpret_cast<float4*>(smem + L.w3f);
  float* kds = reinterpret_cast<float*>(smem + L.kd);
  float* vec1 = reinterpret_cast<float*>(smem + L.vec1);
  float* vec2 = reinterpret_cast<float*>(smem + L.vec2);
  float* vec3 = reinterpret_cast<float*>(smem + L.vec3);
  float* xs = reinterpret_cast<float*>(smem + L.xs);
  float* es = reinterpret_cast<float*>(smem + L.es);
  const int XP = L.xp, EP = L.ep;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int NT1 = Ce >> 3, S1 = Cin >> 3, NB = Ce >> 4;

  pdl_launch_dependents();
  if (!(p.static_mask & 1u)) pdl_wait();
  // ---- once per CTA: weights into fragment order, filter taps and per-channel operands into shared memory ----
  make_fragments(w1f, p.w1, Cin, Ce);
  make_fragments(w3f, p.w3, Ce, Cout);
  for (int i = threadIdx.x; i < 9 * Ce; i += THREADS) kds[i] = __ldg(p.kd + i);
  for (int i = 0; i < p.n_in1; ++i) {
    const float* src = reinterpret_cast<const float*>(p.in1[i].ptr) + p.in1[i].base;
    for (int c = threadIdx.x; c < Ce; c += THREADS) vec1[i * Ce + c] = __ldg(src + c * p.in1[i].stride[0]);
  }
  for (int i = 0; i < p.n_in2; ++i) {
    const float* src = reinterpret_cast<const float*>(p.in2[i].ptr) + p.in2[i].base;
    for (int c = threadIdx.x; c < Ce; c += THREADS) vec2[i * Ce + c] = __ldg(src + c * p.in2[i].stride[0]);
  }
  uint32_t vec3_mask = 0;
  for (int i = 0; i < p.n_in3; ++i) {
    const TensorArg& a = p.in3[i];
    if (a.stride[0] != 1 || a.stride[1] != 0) continue;
    vec3_mask |= 1u << i;
    const float* src = reinterpret_cast<const float*>(a.ptr) + a.base;
    for (int c = threadIdx.x; c < Cout; c += THREADS) vec3[i * Cout + c] = __ldg(src + c);
  }
  for (int i = threadIdx.x; i < (M1 * 16 - HALO) * XP; i += THREADS) xs[HALO * XP + i] = 0.0f;    // rows past the halo tile
  if (p.static_mask & 1u) pdl_wait();
  __syncthreads();

  ExpandIO io1{vec1, Ce, es, EP};
  DwIO2 io2{vec2, Ce};
  ProjectIO io3{p, vec3, Cout, vec3_mask};
  const int tiles_per_image = p.tiles_w * p.tiles_h;

  // the halo tile of X (zeros outside the image), copied asynchronously into shared memory
  auto load_x = [&](int tile_) {
    const int n_ = tile_ / tiles_per_image, tr_ = tile_ - n_ * tiles_per_image;
    const int hh = (tr_ / p.tiles_w) * TH, ww = (tr_ % p.tiles_w) * TW;
    const int q4 = Cin >> 2;
    for (int i = threadIdx.x; i < HALO * q4; i += THREADS) {
      const int px = i / q4, q = i - px * q4;
      const int gh = hh - 1 + px / HW, gw = ww - 1 + px % HW;
      const bool inside = gh >= 0 && gh < p.H && gw >= 0 && gw < p.W;
      const float* src = inside ? p.x + ((size_t)(n_ * p.H + gh) * p.W + gw) * Cin + 4 * q : p.x;
      cp_async_16(xs + px * XP + 4 * q, src, inside ? 16 : 0);
    }
  };
  if ((int)blockIdx.x < p.total_tiles) load_x(blockIdx.x);
  cp_async_commit();
  cp_async_wait_all();
  __syncthreads();

  for (int tile = blockIdx.x; tile < p.total_tiles; tile += gridDim.x) {
    const int n = tile / tiles_per_image, tr = tile - n * tiles_per_image;
    const int h0 = (tr / p.tiles_w) * TH, w0 = (tr % p.tiles_w) * TW;

    // ---- stage 1: expansion of the halo tile; a unit is 16 halo pixels x 24 channels ----
    for (int unit = warp; unit < M1 * (NT1 / 3); unit += WARPS) {
      const int m = unit % M1, jg = unit / M1;
      const int r0 = 16 * m + g, r1 = r0 + 8;
      float acc[3][4];
#pragma unroll
      for (int j = 0; j < 3; ++j) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.0f;
      const float* x0 = xs + r0 * XP;
      const float* x1 = xs + r1 * XP;
      for (int b = 0; 16 * b < Cin; ++b) {
        float4 u, w;
        const bool full = 16 * b + 16 <= Cin;
        if (full) {
          u = *reinterpret_cast<const float4*>(x0 + 16 * b + 4 * t);
          w = *reinterpret_cast<const float4*>(x1 + 16 * b + 4 * t);
        } else {
          const float2 a = *reinterpret_cast<const float2*>(x0 + 16 * b + 2 * t), c = *reinterpret_cast<const float2*>(x1 + 16 * b + 2 * t);
          u = make_float4(a.x, a.y, 0.0f, 0.0f); w = make_float4(c.x, c.y, 0.0f, 0.0f);
        }
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          if (half == 1 && !full) break;
          const int s = 2 * b + half;
          uint32_t h0_, h1_, h2_, h3_, l0_, l1_, l2_, l3_;
          split(half ? u.z : u.x, h0_, l0_); split(half ? w.z : w.x, h1_, l1_);
          split(half ? u.w : u.y, h2_, l2_); split(half ? w.w : w.y, h3_, l3_);
          const float4* bs = w1f + ((size_t)s * NT1 + 3 * jg) * 32 + lane;
          float4 bq[3];
#pragma unroll
          for (int j = 0; j < 3; ++j) bq[j] = bs[j * 32];
#pragma unroll
          for (int j = 0; j < 3; ++j) mma_tf32(acc[j], l0_, l1_, l2_, l3_, __float_as_uint(bq[j].x), __float_as_uint(bq[j].y));
#pragma unroll
          for (int j = 0; j < 3; ++j) mma_tf32(acc[j], h0_, h1_, h2_, h3_, __float_as_uint(bq[j].z), __float_as_uint(bq[j].w));
#pragma unroll
          for (int j = 0; j < 3; ++j) mma_tf32(acc[j], h0_, h1_, h2_, h3_, __float_as_uint(bq[j].x), __float_as_uint(bq[j].y));
        }
      }
      const int gh0 = h0 - 1 + r0 / HW, gw0 = w0 - 1 + r0 % HW, gh1 = h0 - 1 + r1 / HW, gw1 = w0 - 1 + r1 % HW;
      io1.r0 = r0;
      io1.keep0 = r0 < HALO; io1.keep1 = r1 < HALO;
      io1.in0 = gh0 >= 0 && gh0 < p.H && gw0 >= 0 && gw0 < p.W;
      io1.in1 = gh1 >= 0 && gh1 < p.H && gw1 >= 0 && gw1 < p.W;
#pragma unroll
      for (int j = 0; j < 3; ++j) {
        io1.col = 8 * (3 * jg + j) + 2 * t;
#pragma unroll
        for (int v = 0; v < 4; ++v) io1.accv[v] = acc[j][v];
        if constexpr (SP1::n == 0) interp1(p.prog1, io1);
        else run_program<4, SP1>(p.prog1, io1);
      }
    }
    __syncthreads();
    // The halo tile of X is consumed: the next tile's copy starts now and lands while stages 2 and 3 run.
    if (tile + (int)gridDim.x < p.total_tiles) load_x(tile + gridDim.x);
    cp_async_commit();

    // ---- stages 2 and 3: warp = (pixel group, channel quarter).  A pixel group is 4 rows x 8 columns of the tile: lane
    // (g, t) owns the four pixels of column 8 c + g in rows 4 rg .. 4 rg + 3 and four consecutive channels of every
    // 16-channel group of its quarter.  The two upper pixels are fragment rows g and g + 8 of one 16-pixel tile of the
    // projection, the two lower ones of a second tile.  Six rows of the expanded tile feed four results per column,
    // and a filter tap is read once for all four ----
    float acc3[2][NT3][4];
    const int grp = warp >> 2, quarter = warp & 3, rg = grp >> 1, c = grp & 1;
    {
#pragma unroll
      for (int u = 0; u < 2; ++u)
#pragma unroll
        for (int j = 0; j < NT3; ++j) acc3[u][j][0] = acc3[u][j][1] = acc3[u][j][2] = acc3[u][j][3] = 0.0f;
      const int b_begin = (NB * quarter + 3) >> 2, b_end = (NB * (quarter + 1) + 3) >> 2;
      const float* e_base = es + ((4 * rg) * HW + 8 * c + g) * EP;          // halo row 4 rg is the row above pixel row 4 rg
      for (int b = b_begin; b < b_end; ++b) {
        const int ch = 16 * b + 4 * t;
        float o[4][4];
#pragma unroll
        for (int rr = 0; rr < 4; ++rr) o[rr][0] = o[rr][1] = o[rr][2] = o[rr][3] = 0.0f;
        const float* e0 = e_base + ch;
#pragma unroll
        for (int dx = 0; dx < 3; ++dx) {
          float4 k[3];
#pragma unroll
          for (int dy = 0; dy < 3; ++dy) k[dy] = *reinterpret_cast<const float4*>(kds + (dy * 3 + dx) * Ce + ch);
#pragma unroll
          for (int er = 0; er < 6; ++er) {
            const float4 e = *reinterpret_cast<const float4*>(e0 + (er * HW + dx) * EP);
#pragma unroll
            for (int rr = 0; rr < 4; ++rr) {
              const int dy = er - rr;
              if (dy < 0 || dy > 2) continue;
              o[rr][0] = fmaf(e.x, k[dy].x, o[rr][0]); o[rr][1] = fmaf(e.y, k[dy].y, o[rr][1]);
              o[rr][2] = fmaf(e.z, k[dy].z, o[rr][2]); o[rr][3] = fmaf(e.w, k[dy].w, o[rr][3]);
            }
          }
        }
        io2.ch = ch;
#pragma unroll
        for (int rr = 0; rr < 4; ++rr) {
#pragma unroll
          for (int v = 0; v < 4; ++v) io2.accv[v] = o[rr][v];
          if constexpr (SP2::n == 0) interp2(p.prog2, io2);
          else run_program<4, SP2>(p.prog2, io2);
#pragma unroll
          for (int v = 0; v < 4; ++v) o[rr][v] = io2.res[v];
        }
        // two k-steps of the projection: channels ch, ch + 1 and ch + 2, ch + 3
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const int s = 2 * b + half;
          const float4* bs = w3f + (size_t)s * NT3 * 32 + lane;
          float4 bq[NT3];
#pragma unroll
          for (int j = 0; j < NT3; ++j) bq[j] = bs[j * 32];
          uint32_t hi[2][4], lo[2][4];
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            split(o[2 * u][2 * half], hi[u][0], lo[u][0]); split(o[2 * u + 1][2 * half], hi[u][1], lo[u][1]);
            split(o[2 * u][2 * half + 1], hi[u][2], lo[u][2]); split(o[2 * u + 1][2 * half + 1], hi[u][3], lo[u][3]);
          }
          // product by product over all accumulators: consecutive instructions do not depend on each other
#pragma unroll
          for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int j = 0; j < NT3; ++j) mma_tf32(acc3[u][j], lo[u][0], lo[u][1], lo[u][2], lo[u][3], __float_as_uint(bq[j].x), __float_as_uint(bq[j].y));
#pragma unroll
          for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int j = 0; j < NT3; ++j) mma_tf32(acc3[u][j], hi[u][0], hi[u][1], hi[u][2], hi[u][3], __float_as_uint(bq[j].z), __float_as_uint(bq[j].w));
#pragma unroll
          for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int j = 0; j < NT3; ++j) mma_tf32(acc3[u][j], hi[u][0], hi[u][1], hi[u][2], hi[u][3], __float_as_uint(bq[j].x), __float_as_uint(bq[j].y));
        }
      }
    }
    // dense operands of the last chain (the residual): ask for this warp's pieces now, they arrive during the exchange
    for (int i = 0; i < p.n_in3; ++i) {
      const TensorArg& a = p.in3[i];
      if ((vec3_mask >> i) & 1u) continue;
      const int gw = w0 + 8 * c + g;
      for (int f = quarter; f < 2 * NT3; f += 4) {
        const int u = f / NT3, j = f - u * NT3;
#pragma unroll
        for (int rr = 0; rr < 2; ++rr) {
          const int gh = h0 + 4 * rg + 2 * u + rr;
          if (gh < p.H && gw < p.W) {
            const float* q = reinterpret_cast<const float*>(a.ptr) + (uint32_t)a.base + (uint32_t)((n * p.H + gh) * p.W + gw) * (uint32_t)a.stride[1] + (uint32_t)(8 * j + 2 * t) * (uint32_t)a.stride[0];
            asm volatile("prefetch.global.L1 [%0];" ::"l"(q));
          }
        }
      }
    }
    __syncthreads();                       // every warp is done with the expanded tile: its place takes the partial sums
    float* part = es;                      // [pixel group][quarter][2 NT3 x 4 values][32 lanes]
    constexpr int kVals = 2 * NT3 * 4, kFrags = 2 * NT3;
    {
      float* r = part + ((size_t)(grp * 4 + quarter) * kVals) * 32 + lane;
#pragma unroll
      for (int u = 0; u < 2; ++u)
#pragma unroll
        for (int j = 0; j < NT3; ++j)
#pragma unroll
          for (int v = 0; v < 4; ++v) r[((u * NT3 + j) * 4 + v) * 32] = acc3[u][j][v];
    }
    __syncthreads();
    {
      // the group's fragments are shared out over its four warps: each adds the four partial sums of its fragments
      // (always in the same order) and runs the last chain on them
      const float* r = part + ((size_t)(grp * 4) * kVals) * 32 + lane;
      const int gw = w0 + 8 * c + g;
      for (int f = quarter; f < kFrags; f += 4) {
        const int u = f / NT3, j = f - u * NT3;
        const int gh = h0 + 4 * rg + 2 * u;
        io3.ok0 = gh < p.H && gw < p.W; io3.ok1 = gh + 1 < p.H && gw < p.W;
        io3.pix0 = io3.ok0 ? (uint32_t)((n * p.H + gh) * p.W + gw) : 0u;
        io3.pix1 = io3.ok1 ? (uint32_t)((n * p.H + gh + 1) * p.W + gw) : 0u;
        io3.col = (uint32_t)(8 * j + 2 * t);
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          const int slot = (f * 4 + v) * 32;
          io3.accv[v] = ((r[slot] + r[kVals * 32 + slot]) + r[2 * kVals * 32 + slot]) + r[3 * kVals * 32 + slot];
        }
        if constexpr (SP3::n == 0) interp3(p.prog3, io3);
        else run_program<4, SP3>(p.prog3, io3);
      }
    }
    cp_async_wait_all();
    __syncthreads();                       // the partial sums are read, the next halo tile of X has landed
  }
}

#define MO(o, s, i) MicroOp{o, s, i, 0}
DNNF_SP_BEGIN(MP_ScaleShift, 4)
  MO(M_MOV, S_ANCHOR, 0), MO(M_MUL, S_IN, 0), MO(M_ADD, S_IN, 1), MO(M_STORE, S_NONE, 0) DNNF_SP_END
#undef MO

struct Blob {
  Params q;
};

}  // namespace mb

static mb::Blob& mb_of(Launch& L) { return *reinterpret_cast<mb::Blob*>(L.blob.data()); }
static const mb::Blob& mb_of(const Launch& L) { return *reinterpret_cast<const mb::Blob*>(L.blob.data()); }
static const GemmParams& gemm_params(const Launch& L) { return *reinterpret_cast<const GemmParams*>(L.blob.data()); }
static const DwParams& dw_params(const Launch& L) { return *reinterpret_cast<const DwParams*>(L.blob.data()); }

// Conv1x1 + chain -> DwConv3x3 + chain -> Conv1x1 + chain.  `ops` is the union of the three blocks of the normal plan,
// in topological order.
int lower_mbconv(const Graph& g, const std::vector<int>& ops, uint32_t flags, Block& out, std::string& why) {
  auto refuse = [&](const char* m) { why = m; return DNNF_ERR_UNSUPPORTED_OP; };
  std::vector<int> anchors;
  for (int o : ops) { const int k = g.ops[o].kind; if (is_row_anchor(k) || is_contraction(k)) anchors.push_back(o); }
  if (anchors.size() != 3 || g.ops[anchors[0]].kind != DNNF_OP_CONV1X1 || g.ops[anchors[1]].kind != DNNF_OP_DWCONV3X3 ||
      g.ops[anchors[2]].kind != DNNF_OP_CONV1X1) return refuse("not a Conv1x1 - DwConv3x3 - Conv1x1 block");
  const Op& C1 = g.ops[anchors[0]];
  const Op& DW = g.ops[anchors[1]];
  const Op& C3 = g.ops[anchors[2]];
  const int t_e = DW.in[0], t_d = C3.in[0];
  for (int t : {t_e, t_d})
    if (g.tensors[t].is_output || g.tensors[t].consumers.size() != 1) return refuse("an intermediate of the block is needed elsewhere");
  // the three groups: operators up to the tensor the depthwise filter reads, up to the one the projection reads, the rest
  std::vector<int> g1, g2, g3;
  {
    int stage = 1;
    for (int o : ops) {
      if (o == anchors[1]) stage = 2;
      if (o == anchors[2]) stage = 3;
      (stage == 1 ? g1 : stage == 2 ? g2 : g3).push_back(o);
    }
  }
  Block bA, bB, bC;
  const uint32_t sub_flags = flags & ~DNNF_PLAN_BEYOND_TABLE3;
  int rc = lower_contraction(g, g1, sub_flags, anchors[0], bA, why);
  if (rc != DNNF_OK) return rc;
  rc = lower_contraction(g, g2, sub_flags, anchors[1], bB, why);
  if (rc != DNNF_OK) return rc;
  rc = lower_contraction(g, g3, sub_flags, anchors[2], bC, why);
  if (rc != DNNF_OK) return rc;
  if (bA.launch.family != DNNF_FAMILY_CONV1X1 || bB.launch.family != DNNF_FAMILY_DWCONV || bC.launch.family != DNNF_FAMILY_CONV1X1)
    return refuse("the three stages did not lower to convolution blocks");
  const GemmParams& ga = gemm_params(bA.launch);
  const DwParams& db = dw_params(bB.launch);
  const GemmParams& gc = gemm_params(bC.launch);
  const Tensor& X = g.tensors[C1.in[0]];
  if (X.dims.size() != 4) return refuse("input is not NHWC");
  const int N = (int)X.dims[0], H = (int)X.dims[1], W = (int)X.dims[2], Cin = (int)X.dims[3], Ce = ga.N, Cout = gc.N;
  if (bA.launch.out_tensors.size() != 1 || bA.launch.out_tensors[0] != t_e) return refuse("the expansion block stores something else than the depthwise input");
  if (bB.launch.out_tensors.size() != 1 || bB.launch.out_tensors[0] != t_d) return refuse("the depthwise block stores something else than the projection input");
  if (db.C != Ce || gc.K != Ce || db.H != H || db.W != W || db.N != N) return refuse("shapes of the stages do not chain");
  if ((int64_t)N * H * W >= (1ll << 31) / std::max(Ce, 1)) return refuse("tensor too large");
  auto dense_rows = [](const GemmOperand& a, int k) { return a.dtype == 0 && a.stride_col == 1 && a.stride_row == k && a.base == 0; };
  if (!dense_rows(ga.A, Cin) || !dense_rows(gc.A, Ce)) return refuse("a pointwise input is not a dense NHWC tensor");
  if (ga.B.dtype != 0 || ga.B.stride_col != 1 || ga.B.stride_row != Ce || gc.B.dtype != 0 || gc.B.stride_col != 1 || gc.B.stride_row != Cout)
    return refuse("weights are not dense row-major fp32");
  if (ga.batch_ext[0] * ga.batch_ext[1] != 1 || gc.batch_ext[0] * gc.batch_ext[1] != 1) return refuse("batched pointwise convolution");
  if (Cin % 8 || Ce % 48 || Cout % 8 || (Cout != 24 && Cout != 32)) return refuse("channel counts outside the single-kernel form");
  if (ga.n_nd != 1 || ga.m_nd != 1 || gc.n_nd != 1 || gc.m_nd != 1 || !gc.vec_ok) return refuse("index maps outside the single-kernel form");
  // chains 1 and 2: per-channel operands only, one result
  for (int i = 0; i < ga.n_in; ++i) {
    const TensorArg& a = ga.in[i];
    if (a.dtype != 0 || a.stride[0] != 1) return refuse("an operand behind the expansion depends on the pixel");
    for (int d = 1; d < kMaxDims; ++d) if (a.stride[d] != 0) return refuse("an operand behind the expansion depends on the pixel");
  }
  for (int i = 0; i < db.n_in; ++i) {
    const TensorArg& a = db.in[i];
    if (a.dtype != 0 || a.stride[0] != 1) return refuse("an operand behind the depthwise filter depends on the pixel");
    for (int d = 1; d < kMaxDims; ++d) if (a.stride[d] != 0) return refuse("an operand behind the depthwise filter depends on the pixel");
  }
  auto one_store = [](const Program& pr) { int n = 0; for (int i = 0; i < pr.n; ++i) if (pr.ops[i].op == M_STORE) ++n; return n == 1; };
  if (ga.n_out != 1 || db.n_out != 1 || !one_store(ga.prog) || !one_store(db.prog)) return refuse("a middle stage has more than one result");
  for (int i = 0; i < gc.n_in; ++i) if (gc.in[i].dtype != 0 || gc.in[i].mode == 2) return refuse("projection operand type");
  for (int i = 0; i < gc.n_out; ++i) if (gc.out[i].dtype != 0 || gc.out[i].stride[0] != 1) return refuse("projection output type");
  const mb::Layout lay = mb::layout_of(Cin, Ce, Cout);
  if (lay.total > mb::kSmemMax) return refuse("block does not fit shared memory");

  Launch& L = out.launch;
  L = Launch{};
  L.blob.assign(sizeof(mb::Blob), 0);
  mb::Params& q = mb_of(L).q;
  q.N = N; q.H = H; q.W = W; q.Cin = Cin; q.Ce = Ce; q.Cout = Cout;
  q.tiles_w = (W + mb::TW - 1) / mb::TW; q.tiles_h = (H + mb::TH - 1) / mb::TH;
  const int64_t total = (int64_t)N * q.tiles_w * q.tiles_h;
  if (total >= (1ll << 31)) return refuse("too many tiles");
  q.total_tiles = (int)total;
  // Measured (B200, CUDA-graph replays of the 24 -> 144 -> 24 block): one kernel against three is 15.1 against 21.7 us
  // on one 56 x 56 image (28 tiles; 17.3 against 20.4 us once the small-M pointwise kernel existed), but 30.1 against 26.8 us on 8 images
  // and 94.9 against 63.0 us on 32: once the tiles exceed one wave the kernel is bound by instruction issue and
  // shared-memory bandwidth (split-TF32 on warp-level instructions, the depthwise taps), the three kernels by HBM.
  if (total > sm_count() && !plan_flag(DNNF_PLAN_MBCONV_ALWAYS)) return refuse("more than one wave of tiles: the three kernels are faster");
  // ... and below 16 tiles its set-up (both weight matrices into fragment order, once per CTA) is not paid back: one
  // 14 x 14 image is 17.2 us against 11.5 us for the three kernels since the small-M pointwise kernel exists.
  { const char* e = dev_env("DNNF_MB_MIN_TILES"); const int min_tiles = e ? atoi(e) : 16;
    if (total < min_tiles && !plan_flag(DNNF_PLAN_MBCONV_ALWAYS)) return refuse("too few tiles to pay for the set-up: the three kernels are faster"); }
  q.prog1 = ga.prog; q.prog2 = db.prog; q.prog3 = gc.prog;
  q.n_in1 = ga.n_in; q.n_in2 = db.n_in; q.n_in3 = gc.n_in; q.n_out3 = gc.n_out;
  for (int i = 0; i < ga.n_in; ++i) q.in1[i] = ga.in[i];
  for (int i = 0; i < db.n_in; ++i) q.in2[i] = db.in[i];
  for (int i = 0; i < gc.n_in; ++i) q.in3[i] = gc.in[i];
  for (int i = 0; i < gc.n_out; ++i) q.out3[i] = gc.out[i];
  // tensors: X, W1, chain-1 operands, Kd, chain-2 operands, W3, chain-3 operands; the projection block's outputs
  L.in_tensors = {bA.launch.in_tensors[0], bA.launch.in_tensors[1]};
  for (size_t i = 2; i < bA.launch.in_tensors.size(); ++i) L.in_tensors.push_back(bA.launch.in_tensors[i]);
  L.in_tensors.push_back(bB.launch.in_tensors[1]);
  for (size_t i = 2; i < bB.launch.in_tensors.size(); ++i) L.in_tensors.push_back(bB.launch.in_tensors[i]);
  L.in_tensors.push_back(bC.launch.in_tensors[1]);
  for (size_t i = 2; i < bC.launch.in_tensors.size(); ++i) L.in_tensors.push_back(bC.launch.in_tensors[i]);
  L.out_tensors = bC.launch.out_tensors;
  bool all_static = true;
  for (size_t i = 1; i < L.in_tensors.size(); ++i) {
    const Tensor& T = g.tensors[L.in_tensors[i]];
    const bool is_static = T.external && T.producer < 0 && !T.is_output;
    // the dense operands of the last chain (the residual) are read after the wait in any case
    bool late = false;
    const size_t first3 = 2 + ga.n_in + 1 + db.n_in + 1;
    if (i >= first3) { const TensorArg& a = gc.in[i - first3]; late = !(a.stride[0] == 1 && a.stride[1] == 0); }
    if (!is_static && !late) all_static = false;
  }
  q.static_mask = all_static ? 1u : 0u;
  L.smem = (size_t)lay.total;
  L.threads = mb::THREADS;
  L.grid = (int)std::min<int64_t>(total, sm_count());
  L.family = DNNF_FAMILY_MBCONV;
  L.variant = 0;
  L.flops = bA.launch.flops + bB.launch.flops + bC.launch.flops;
  L.ew.prog = gc.prog;                 // introspection (dnnf_block_program): the chain behind the projection
  const bool s12 = program_matches<CP_ScaleShiftClip>(q.prog1) && program_matches<CP_ScaleShiftClip>(q.prog2);
  L.static_id = !s12 ? 0 : program_matches<CP_ScaleShiftResidual>(q.prog3) ? 1 : program_matches<mb::MP_ScaleShift>(q.prog3) ? 2 : 0;
  out.inputs.clear();
  for (int t : L.in_tensors) if (std::find(out.inputs.begin(), out.inputs.end(), t) == out.inputs.end()) out.inputs.push_back(t);
  out.outputs = L.out_tensors;
  out.lowered = true;
  return DNNF_OK;
}

void mbconv_patch(Launch& L, const std::vector<void*>& ip, const std::vector<void*>& op) {
  mb::Params& q = mb_of(L).q;
  size_t k = 0;
  q.x = reinterpret_cast<const float*>(ip[k++]);
  q.w1 = reinterpret_cast<const float*>(ip[k++]);
  for (int i = 0; i < q.n_in1; ++i) q.in1[i].ptr = ip[k++];
  q.kd = reinterpret_cast<const float*>(ip[k++]);
  for (int i = 0; i < q.n_in2; ++i) q.in2[i].ptr = ip[k++];
  q.w3 = reinterpret_cast<const float*>(ip[k++]);
  for (int i = 0; i < q.n_in3; ++i) q.in3[i].ptr = ip[k++];
  for (int i = 0; i < q.n_out3; ++i) q.out3[i].ptr = op[i];
}

namespace {
template <int NT3, class SP1, class SP2, class SP3>
int mb_launch_one(const Launch& L, cudaStream_t st) {
  static PerDeviceOnce once;
  if (once.first_use()) cudaFuncSetAttribute(mb::mbconv_kernel<NT3, SP1, SP2, SP3>, cudaFuncAttributeMaxDynamicSharedMemorySize, mb::kSmemMax);
  return launch_pdl(mb::mbconv_kernel<NT3, SP1, SP2, SP3>, L.grid, mb::THREADS, L.smem, st, mb_of(L).q) == cudaSuccess ? 0 : 1;
}
template <int NT3>
int mb_launch_nt(const Launch& L, cudaStream_t st) {
  if (L.static_id == 1) return mb_launch_one<NT3, CP_ScaleShiftClip, CP_ScaleShiftClip, CP_ScaleShiftResidual>(L, st);
  if (L.static_id == 2) return mb_launch_one<NT3, CP_ScaleShiftClip, CP_ScaleShiftClip, mb::MP_ScaleShift>(L, st);
  return mb_launch_one<NT3, DynProg, DynProg, DynProg>(L, st);
}
}  // namespace

int mbconv_launch(const Launch& L, cudaStream_t st) {
  const int nt3 = mb_of(L).q.Cout / 8;
  if (nt3 == 3) return mb_launch_nt<3>(L, st);
  if (nt3 == 4) return mb_launch_nt<4>(L, st);
  return 1;
}

}  // namespace dnnf
