// fp32 NHWC convolution anchors on CUDA cores, each with the block's epilogue program:
//  * pointwise (1x1) convolution as a register-tiled FMA GEMM for tall-skinny shapes: weights
//    resident in shared memory, pixel tile streamed through shared memory, 8 pixels x TN
//    channels per thread;
//  * depthwise 3x3, stride 1, zero padding 1: a thread owns one (image, column, 4-channel
//    group) and walks down the rows with a rolling 3x3 window, so every input value is
//    loaded three times from L1/L2 instead of nine.
// Both are bound by HBM traffic at the shapes of a MobileNet block (K = 24 / 144).
#include <cuda_runtime.h>

#include <algorithm>

#include "chain.cuh"
#include "conv_params.h"
#include "gemm_params.h"
#include "lower.h"

namespace dnnf {

// ---------------------------------------------------------------------------
// Pointwise convolution: [P x K] * [K x N], fp32, rows contiguous.
// Register-tiled FMA kernel for tall-skinny problems (K, N small): a CTA owns BM = PG*8
// pixels and all N channels; the [K x N] weights sit in shared memory for the CTA's
// lifetime, the pixel tile streams through shared memory 8 input channels at a time
// (transposed, so a thread reads its 8 pixels as two 128-bit words); a thread accumulates
// 8 pixels x TN channels.  Thread `chg` owns the float4 channel groups chg + CG*j, so the
// lanes of a warp write neighbouring 16-byte pieces of a pixel's row.
// ---------------------------------------------------------------------------
constexpr int PW_TM = 8, PW_KC = 8;

template <int TN>
struct PwIO {
  static constexpr int VV = TN;
  const GemmParams& p;
  float accv[TN];
  uint32_t pix;            // pixel index (row of the [P x N] result)
  int chg, cg;
  bool ok;
  __device__ __forceinline__ uint32_t off(const TensorArg& a, int j) const {
    return (uint32_t)a.base + pix * (uint32_t)a.stride[1] + (uint32_t)(4 * (chg + cg * j)) * (uint32_t)a.stride[0];
  }
  __device__ __forceinline__ void load(int idx, float (&dst)[VV]) const {
    const TensorArg& a = p.in[idx];
#pragma unroll
    for (int j = 0; j < TN / 4; ++j) {
      float* d = &dst[4 * j];
      if (!ok) { d[0] = d[1] = d[2] = d[3] = 0.0f; continue; }
      if (a.stride[0] == 0) { float x = load_scalar<true>(a, off(a, j)); d[0] = d[1] = d[2] = d[3] = x; }
      else load_vec4<true>(a, off(a, j), d);
    }
  }
  __device__ __forceinline__ void anchor(float (&dst)[VV]) const {
#pragma unroll
    for (int v = 0; v < VV; ++v) dst[v] = accv[v];
  }
  __device__ __forceinline__ void store(int idx, const float (&val)[VV]) const {
    if (!ok) return;
    const TensorArg& a = p.out[idx];
#pragma unroll
    for (int j = 0; j < TN / 4; ++j) store_vec4<true>(a, off(a, j), &val[4 * j], false);
  }
  __device__ __forceinline__ void row_reduce(int, float (&)[VV]) const {}
};

// THREADS = CG * PG; BM = PG * 8 pixels per CTA
template <int TN, int CG, int PG, class SP>
__global__ void __launch_bounds__(CG * PG) conv1x1_kernel(const __grid_constant__ GemmParams p) {
  constexpr int THREADS = CG * PG, BM = PG * PW_TM, APITCH = BM + 16;
  extern __shared__ float wsm[];                 // [K][N] weights, then [2][KC][APITCH] pixel chunks
  pdl_launch_dependents();
  pdl_wait();
  const int K = p.K, N = p.N;
  float* as = wsm + K * N;
  const float* W = reinterpret_cast<const float*>(p.B.ptr) + p.B.base;
  for (int i = threadIdx.x * 4; i < K * N; i += THREADS * 4)
    *reinterpret_cast<float4*>(&wsm[i]) = __ldg(reinterpret_cast<const float4*>(W + i));
  const float* X = reinterpret_cast<const float*>(p.A.ptr) + p.A.base;
  const int chg = threadIdx.x % CG, pxg = threadIdx.x / CG;
  const int64_t m0 = (int64_t)blockIdx.x * BM;
  // chunk loader: BM pixels x 8 input channels = 2*BM float4; thread t takes float4 (pixel t/2 + i*THREADS/2, half t%2)
  constexpr int LD = (2 * BM + THREADS - 1) / THREADS;
  float4 pre[LD];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int i = 0; i < LD; ++i) {
      int idx = threadIdx.x + i * THREADS;
      int px = idx >> 1, half = idx & 1;
      bool ok = idx < 2 * BM && m0 + px < p.M && k0 + half * 4 < K;
      pre[i] = ok ? __ldg(reinterpret_cast<const float4*>(X + (m0 + px) * p.A.stride_row + k0 + half * 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
  auto stash = [&](int buf) {
    float* dst = as + buf * (PW_KC * APITCH);
#pragma unroll
    for (int i = 0; i < LD; ++i) {
      int idx = threadIdx.x + i * THREADS;
      if (idx < 2 * BM) {
        int px = idx >> 1, half = idx & 1;
        dst[(half * 4 + 0) * APITCH + px] = pre[i].x; dst[(half * 4 + 1) * APITCH + px] = pre[i].y;
        dst[(half * 4 + 2) * APITCH + px] = pre[i].z; dst[(half * 4 + 3) * APITCH + px] = pre[i].w;
      }
    }
  };
  float acc[PW_TM][TN];
#pragma unroll
  for (int i = 0; i < PW_TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0.0f;
  fetch(0);
  stash(0);
  __syncthreads();
  const int nchunks = (K + PW_KC - 1) / PW_KC;
  for (int c = 0; c < nchunks; ++c) {
    if (c + 1 < nchunks) fetch((c + 1) * PW_KC);          // next chunk's global loads overlap this chunk's FMAs
    const float* a_s = as + (c & 1) * (PW_KC * APITCH) + pxg * PW_TM;
#pragma unroll
    for (int kk = 0; kk < PW_KC; ++kk) {
      const int k = c * PW_KC + kk;
      if (k < K) {
        float4 a0 = *reinterpret_cast<const float4*>(a_s + kk * APITCH), a1 = *reinterpret_cast<const float4*>(a_s + kk * APITCH + 4);
        const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
        float b[TN];
#pragma unroll
        for (int j = 0; j < TN / 4; ++j) {
          float4 w = *reinterpret_cast<const float4*>(wsm + k * N + 4 * (chg + CG * j));
          b[4 * j] = w.x; b[4 * j + 1] = w.y; b[4 * j + 2] = w.z; b[4 * j + 3] = w.w;
        }
#pragma unroll
        for (int i = 0; i < PW_TM; ++i)
#pragma unroll
          for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
      }
    }
    if (c + 1 < nchunks) stash((c + 1) & 1);
    __syncthreads();
  }
  PwIO<TN> io{p};
  io.chg = chg; io.cg = CG;
#pragma unroll
  for (int i = 0; i < PW_TM; ++i) {
    const int64_t pix = m0 + pxg * PW_TM + i;
    io.ok = pix < p.M;
    io.pix = (uint32_t)(io.ok ? pix : 0);
#pragma unroll
    for (int j = 0; j < TN; ++j) io.accv[j] = acc[i][j];
    run_program<TN, SP>(p.prog, io);
  }
}

static const GemmParams& gp_of(const Launch& L) { return *reinterpret_cast<const GemmParams*>(L.blob.data()); }

// Instantiated (TN, CG, PG) shapes; the host picks one with TN*CG == N.
struct PwShape { int tn, cg, pg; };
static bool pw_shape(int n, PwShape& s) {
  static const PwShape table[] = {{12, 12, 16}, {4, 6, 32}, {8, 8, 24}, {8, 16, 16}, {4, 4, 32}, {4, 8, 32}, {8, 4, 32}, {4, 2, 64}, {4, 1, 64}, {12, 4, 32}};
  for (auto& t : table) if (t.tn * t.cg == n) { s = t; return true; }
  return false;
}

bool conv1x1_direct_eligible(const GemmParams& gp) {
  if (gp.A.dtype != 0 || gp.B.dtype != 0) return false;
  if (gp.batch_ext[0] * gp.batch_ext[1] != 1) return false;
  if (gp.M < 128) return false;      // a handful of rows: one CTA would fetch all of B alone; the tiled kernel spreads N over CTAs
  if (gp.A.stride_col != 1 || gp.A.stride_row % 4 || gp.A.base % 4) return false;
  if (gp.B.stride_col != 1 || gp.B.stride_row != gp.N || gp.B.base % 4) return false;
  if (gp.N % 4 || gp.K % 4 || (int64_t)gp.K * gp.N * 4 > 96 * 1024) return false;
  if (gp.n_nd != 1 || gp.m_nd != 1 || gp.b_nd != 1 || !gp.vec_ok) return false;
  for (int i = 0; i < gp.n_in; ++i) if (gp.in[i].dtype != 0) return false;
  for (int i = 0; i < gp.n_out; ++i) if (gp.out[i].dtype != 0) return false;
  PwShape s;
  return pw_shape(gp.N, s);
}

void conv1x1_direct_plan(Launch& L) {
  GemmParams& gp = *reinterpret_cast<GemmParams*>(L.blob.data());
  PwShape s;
  pw_shape(gp.N, s);
  L.variant = 2;
  L.threads = s.cg * s.pg;
  const int bm = s.pg * PW_TM;
  L.smem = (size_t)gp.K * gp.N * 4 + 2 * PW_KC * (bm + 16) * 4;
  L.grid = (int)((gp.M + bm - 1) / bm);
  L.static_id = StaticSet<ConvStatic>::find(gp.prog);
}

template <int TN, int CG, int PG>
struct PwLauncher {
  const Launch& L; cudaStream_t st;
  template <class SP> void run() {
    static PerDeviceOnce once;       // per instantiation
    if (once.first_use()) cudaFuncSetAttribute(conv1x1_kernel<TN, CG, PG, SP>, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * 1024);
    launch_pdl(conv1x1_kernel<TN, CG, PG, SP>, L.grid, CG * PG, L.smem, st, gp_of(L));
  }
};
template <int TN, int CG, int PG, bool kStatic>
static void pw_launch(const Launch& L, cudaStream_t st) {
  PwLauncher<TN, CG, PG> F{L, st};
  if (kStatic && L.static_id > 0 && StaticSet<ConvStatic>::dispatch(L.static_id, F)) return;
  F.template run<DynProg>();
}

int conv1x1_direct_launch(const Launch& L, cudaStream_t st) {
  const GemmParams& gp = gp_of(L);
  PwShape s{0, 0, 0};
  pw_shape(gp.N, s);
  switch (s.tn * 10000 + s.cg * 100 + s.pg) {
    case 121216: pw_launch<12, 12, 16, true>(L, st); break;
    case 40632: pw_launch<4, 6, 32, true>(L, st); break;
    case 80824: pw_launch<8, 8, 24, false>(L, st); break;
    case 81616: pw_launch<8, 16, 16, false>(L, st); break;
    case 40432: pw_launch<4, 4, 32, false>(L, st); break;
    case 40832: pw_launch<4, 8, 32, false>(L, st); break;
    case 80432: pw_launch<8, 4, 32, false>(L, st); break;
    case 40264: pw_launch<4, 2, 64, false>(L, st); break;
    case 40164: pw_launch<4, 1, 64, false>(L, st); break;
    case 120432: pw_launch<12, 4, 32, false>(L, st); break;
    default: return 2;
  }
  return cudaGetLastError() == cudaSuccess ? 0 : 1;
}

// ---------------------------------------------------------------------------
// Depthwise 3x3
// ---------------------------------------------------------------------------
__device__ __forceinline__ float4 ld4_or_zero(const float* p, bool ok) {
  return ok ? __ldg(reinterpret_cast<const float4*>(p)) : make_float4(0.f, 0.f, 0.f, 0.f);
}
__device__ __forceinline__ void fma4(float (&acc)[4], const float4& x, const float4& k) {
  acc[0] = fmaf(x.x, k.x, acc[0]); acc[1] = fmaf(x.y, k.y, acc[1]); acc[2] = fmaf(x.z, k.z, acc[2]); acc[3] = fmaf(x.w, k.w, acc[3]);
}

// HS rows per thread: the grid covers (n, h-strip, w, c4).  The 3x3 weights sit in shared memory
// (a thread re-reads its nine 128-bit words per output row: conflict-free, neighbouring lanes hold
// neighbouring channels), which keeps the thread at 64 registers so that four CTAs fit an SM and
// enough loads are in flight to cover the memory latency.
template <class SP>
__global__ void __launch_bounds__(256, 4) dwconv_kernel(const __grid_constant__ DwParams p, int HS) {
  extern __shared__ float4 kws[];                // [9][C/4]
  pdl_launch_dependents();
  pdl_wait();
  const int C4 = p.C / 4;
  for (int i = threadIdx.x; i < 9 * C4; i += 256) kws[i] = __ldg(reinterpret_cast<const float4*>(p.k) + i);
  __syncthreads();
  const int strips = (p.H + HS - 1) / HS;
  int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x;
  const int64_t total = (int64_t)p.N * strips * p.W * C4;
  if (t >= total) return;
  const int c4 = (int)(t % C4); t /= C4;
  const int w = (int)(t % p.W); t /= p.W;
  const int s = (int)(t % strips); const int n = (int)(t / strips);
  const int h0 = s * HS, h1 = min(p.H, h0 + HS);
  const float4* kw = kws + c4;
  const float* xb = p.x + ((int64_t)n * p.H * p.W) * p.C + c4 * 4;
  const bool wl = w > 0, wr = w + 1 < p.W;
  auto row = [&](int h, float4 (&r)[3]) {
    const bool ok = h >= 0 && h < p.H;
    const float* q = xb + ((int64_t)h * p.W + w) * p.C;
    r[0] = ld4_or_zero(q - p.C, ok && wl); r[1] = ld4_or_zero(q, ok); r[2] = ld4_or_zero(q + p.C, ok && wr);
  };
  float4 r0[3], r1[3], r2[3], r3[3];
  row(h0 - 1, r0); row(h0, r1); row(h0 + 1, r2);
  DwIO io{p};
  io.n = n; io.w = w; io.c = c4 * 4;
  for (int h = h0; h < h1; ++h) {
    row(h + 2, r3);                              // the row needed by the NEXT output: in flight during this one
    io.accv[0] = io.accv[1] = io.accv[2] = io.accv[3] = 0.0f;
#pragma unroll
    for (int j = 0; j < 3; ++j) { fma4(io.accv, r0[j], kw[j * C4]); fma4(io.accv, r1[j], kw[(3 + j) * C4]); fma4(io.accv, r2[j], kw[(6 + j) * C4]); }
    io.h = h;
    run_program<4, SP>(p.prog, io);
#pragma unroll
    for (int j = 0; j < 3; ++j) { r0[j] = r1[j]; r1[j] = r2[j]; r2[j] = r3[j]; }
  }
}

size_t dwconv_tma_blob_bytes();
bool dwconv_tma_plan(Launch& L);
bool dwconv_tma_prepare(Launch& L, std::string& err);
int dwconv_tma_launch(const Launch& L, int32_t* status, int block_index, cudaStream_t st);

static const DwParams& dw_of(const Launch& L) { return *reinterpret_cast<const DwParams*>(L.blob.data()); }

struct DwLauncher {
  const Launch& L; cudaStream_t st; int hs;
  template <class SP> void run() { launch_pdl(dwconv_kernel<SP>, L.grid, 256, (size_t)9 * dw_of(L).C * 4, st, dw_of(L), hs); }
};

int dwconv_launch(const Launch& L, void* status_words, int block_index, cudaStream_t st) {
  if (L.variant < 0 && !L.tc_ready) return 1;        // never launch with a tensor map that was not encoded
  if (L.variant < 0) return dwconv_tma_launch(L, reinterpret_cast<int32_t*>(status_words), block_index, st);
  DwLauncher F{L, st, L.variant};
  if (!(L.static_id > 0 && StaticSet<ConvStatic>::dispatch(L.static_id, F))) F.run<DynProg>();
  return cudaGetLastError() == cudaSuccess ? 0 : 1;
}

void dwconv_patch(Launch& L, const std::vector<void*>& ip, const std::vector<void*>& op, std::string& err) {
  DwParams& dp = *reinterpret_cast<DwParams*>(L.blob.data());
  if (L.variant < 0 && (dp.x != ip[0] || !L.tc_ready)) {
    dp.x = reinterpret_cast<const float*>(ip[0]);
    L.tc_ready = dwconv_tma_prepare(L, err);
    if (!L.tc_ready && err.empty()) err = "cannot encode the tensor map of a depthwise convolution block";
  }
  dp.x = reinterpret_cast<const float*>(ip[0]);
  dp.k = reinterpret_cast<const float*>(ip[1]);
  for (int i = 0; i < dp.n_in; ++i) dp.in[i].ptr = ip[2 + i];
  for (int i = 0; i < dp.n_out; ++i) dp.out[i].ptr = op[i];
}

int lower_dwconv(const Graph& g, const std::vector<int>& ops, int anchor, Block& out, std::string& why) {
  const Op& A = g.ops[anchor];
  const Tensor& X = g.tensors[A.in[0]];
  const Tensor& Kt = g.tensors[A.in[1]];
  const Tensor& Y = g.tensors[A.out[0]];
  std::set<int> in_block(ops.begin(), ops.end());
  if (X.dtype != DNNF_F32 || Kt.dtype != DNNF_F32) { why = "depthwise convolution is fp32 only"; return DNNF_ERR_UNSUPPORTED_OP; }
  if (X.dims[3] % 4) { why = "depthwise convolution needs a channel count that is a multiple of 4"; return DNNF_ERR_UNSUPPORTED_OP; }
  if (X.dims[3] > 1280) { why = "depthwise convolution: more than 1280 channels"; return DNNF_ERR_UNSUPPORTED_OP; }   // weights in 48 KB of shared memory
  if (in_block.count(X.producer) || in_block.count(Kt.producer)) { why = "operators in front of a convolution anchor (no prologue fusion)"; return DNNF_ERR_UNSUPPORTED_OP; }
  if (X.numel() >= (1ll << 31)) { why = "tensor too large"; return DNNF_ERR_UNSUPPORTED_OP; }
  LowerCtx cx(g);
  cx.ops = ops; cx.in_block = in_block;
  cx.ext = Y.dims;
  if (!derive_views(cx, A.out[0], {anchor})) { why = cx.why; return DNNF_ERR_UNSUPPORTED_OP; }
  if (cx.ext != Y.dims) { why = "epilogue reshapes a depthwise convolution's result"; return DNNF_ERR_UNSUPPORTED_OP; }
  if (!emit_program(cx, A.out[0], 2)) { why = cx.why; return DNNF_ERR_UNSUPPORTED_OP; }
  Launch& L = out.launch;
  L = Launch{};
  L.blob.assign(sizeof(DwParams) + dwconv_tma_blob_bytes(), 0);
  DwParams& dp = *reinterpret_cast<DwParams*>(L.blob.data());
  dp.N = (int)Y.dims[0]; dp.H = (int)Y.dims[1]; dp.W = (int)Y.dims[2]; dp.C = (int)Y.dims[3];
  dp.n_in = (int)cx.ins.size(); dp.n_out = (int)cx.outs.size();
  auto fill = [&](TensorArg& a, const ExtArg& e, bool is_out) {
    a.ptr = nullptr; a.base = (int32_t)e.view.c0; a.dtype = g.tensors[e.tensor].dtype; a.mode = 0;
    for (int d = 0; d < kMaxDims; ++d) a.stride[d] = d < 4 ? (int32_t)e.view.coef[3 - d] : 0;
    if (a.dtype != DNNF_F32) return false;
    if (a.stride[0] == 1) { if (a.base % 4) return false; for (int d = 1; d < 4; ++d) if (a.stride[d] % 4) return false; }
    else if (!(a.stride[0] == 0 && !is_out)) return false;
    return true;
  };
  for (size_t i = 0; i < cx.ins.size(); ++i) if (!fill(dp.in[i], cx.ins[i], false)) { why = "depthwise epilogue operand is not fp32 / channel-contiguous"; return DNNF_ERR_UNSUPPORTED_OP; }
  for (size_t i = 0; i < cx.outs.size(); ++i) if (!fill(dp.out[i], cx.outs[i], true)) { why = "depthwise epilogue output is not fp32 / channel-contiguous"; return DNNF_ERR_UNSUPPORTED_OP; }
  dp.prog = cx.prog;
  L.ew.prog = cx.prog;
  L.in_tensors = {A.in[0], A.in[1]};
  out.inputs = {A.in[0], A.in[1]};
  out.outputs.clear();
  for (auto& a : cx.ins) { L.in_tensors.push_back(a.tensor); if (std::find(out.inputs.begin(), out.inputs.end(), a.tensor) == out.inputs.end()) out.inputs.push_back(a.tensor); }
  for (auto& a : cx.outs) { L.out_tensors.push_back(a.tensor); out.outputs.push_back(a.tensor); }
  L.family = DNNF_FAMILY_DWCONV;
  L.flops = 2ll * 9 * Y.numel();
  if (dwconv_tma_plan(L)) { out.lowered = true; return DNNF_OK; }
  // rows per thread: enough threads to fill the machine, long enough strips to reuse the window
  int hs = dp.H;
  int64_t threads_full = (int64_t)dp.N * dp.W * (dp.C / 4);
  while (hs > 7 && threads_full * ((dp.H + hs - 1) / hs) < 148 * 1024 * 4) hs = (hs + 1) / 2;
  // a problem with fewer threads than one CTA per SM is a chain of dependent row loads per thread: shorter strips, at
  // the price of reading the strips' halo rows again
  while (hs > 2 && threads_full * ((dp.H + hs - 1) / hs) < (int64_t)sm_count() * 256) hs = (hs + 1) / 2;
  L.variant = hs;
  int64_t total = threads_full * ((dp.H + hs - 1) / hs);
  L.grid = (int)((total + 255) / 256);
  L.threads = 256;
  L.flops = 2ll * 9 * Y.numel();
  L.static_id = StaticSet<ConvStatic>::find(dp.prog);
  out.lowered = true;
  return DNNF_OK;
}

}  // namespace dnnf
