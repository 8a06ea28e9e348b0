// MaxPool / AveragePool over an NHWC fp32 tensor with a fused epilogue chain.
//
// Table 2 lists both under Many-to-Many; like the other Many-to-Many anchors they take One-to-One successors as
// an epilogue (Table 3, Many-to-Many followed by One-to-One) and nothing in front.
//
// One thread owns four neighbouring channels of one output pixel and walks its window with 128-bit loads;
// neighbouring lanes hold neighbouring channels, so every load of a warp is one run of bytes.  The window's rows
// overlap between neighbouring outputs (stride < kernel) and are served by L1/L2; the kernel's HBM traffic is the
// input once plus the output once.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdlib>
#include <set>

#include "conv_params.h"
#include "launch_util.h"
#include "lower.h"

namespace dnnf {

struct PoolParams {
  DwParams d;              // N, H, W, C: the RESULT's dims; x: the pooled tensor; k unused; epilogue operands
  int32_t Hi, Wi;          // pooled tensor's height and width
  int32_t kernel, stride, pad;
  int32_t is_max;
  int32_t col2im;          // the tensor holds k x k patches per pixel ([N,Hi,Wi,k*k*C]); an output element adds the values that land on it
  int32_t Ci;              // channels per pixel of the tensor that is read (C, or k*k*C for col2im)
  FastDiv fd_c4, fd_w, fd_h, fd_s;   // fd_s: by the stride (col2im)
  // wide windows (a global pool): CTAs per (pixel, 128-channel group) and how the window is sliced over them
  int32_t groups, slices, per_slice;
  float* scratch;          // [unit][slice][128] partial results of a sliced window
  int32_t* counters;       // [unit] arrivals, zero between runs
};

template <class SP>
__global__ void __launch_bounds__(256) pool_kernel(const __grid_constant__ PoolParams p) {
  pdl_launch_dependents();
  pdl_wait();
  const uint32_t C4 = (uint32_t)p.d.C / 4;
  const uint32_t t = blockIdx.x * 256u + threadIdx.x;
  const uint32_t total = (uint32_t)p.d.N * p.d.H * p.d.W * C4;
  if (t >= total) return;
  const uint32_t q0 = fd_div(t, p.fd_c4), c4 = t - q0 * C4;
  const uint32_t q1 = fd_div(q0, p.fd_w), wo = q0 - q1 * (uint32_t)p.d.W;
  const uint32_t n = fd_div(q1, p.fd_h), ho = q1 - n * (uint32_t)p.d.H;
  const int h0 = (int)ho * p.stride - p.pad, w0 = (int)wo * p.stride - p.pad;
  const int ha = max(h0, 0), hb = min(h0 + p.kernel, p.Hi);
  const int wa = max(w0, 0), wb = min(w0 + p.kernel, p.Wi);
  const float* xb = p.d.x + ((size_t)n * p.Hi * p.Wi) * p.Ci + c4 * 4;
  DwIO io{p.d};
  const float init = p.is_max ? -INFINITY : 0.0f;
  io.accv[0] = io.accv[1] = io.accv[2] = io.accv[3] = init;
  if (p.col2im) {
    // transposed convolution, gather form: output row ho receives tap i of input row h where ho + pad = h * stride + i,
    // likewise for columns; at most ceil(k / s)^2 terms, added in a fixed order
    const int s = p.stride, k = p.kernel;
    const int hp = (int)ho + p.pad, wp = (int)wo + p.pad;
    if (k <= 2 * s) {
      // at most 2 x 2 terms (the usual k = 2s): their loads are issued together, then added in the same fixed order
      const int hq = (int)fd_div((uint32_t)hp, p.fd_s), wq = (int)fd_div((uint32_t)wp, p.fd_s);
      const int i0 = hp - hq * s, j0 = wp - wq * s;
      float4 v[4];
#pragma unroll
      for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int b = 0; b < 2; ++b) {
          const int i = i0 + a * s, j = j0 + b * s, h = hq - a, w = wq - b;
          const bool ok = i < k && j < k && h >= 0 && h < p.Hi && w >= 0 && w < p.Wi;
          v[a * 2 + b] = ok ? __ldg(reinterpret_cast<const float4*>(xb + ((size_t)h * p.Wi + w) * p.Ci + (size_t)(i * k + j) * p.d.C))
                            : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
      for (int e = 0; e < 4; ++e) { io.accv[0] += v[e].x; io.accv[1] += v[e].y; io.accv[2] += v[e].z; io.accv[3] += v[e].w; }
    } else
    for (int i = hp % s; i < k; i += s) {
      const int h = (hp - i) / s;
      if (hp - i < 0 || h >= p.Hi) continue;
      for (int j = wp % s; j < k; j += s) {
        const int w = (wp - j) / s;
        if (wp - j < 0 || w >= p.Wi) continue;
        const float4 v = __ldg(reinterpret_cast<const float4*>(xb + ((size_t)h * p.Wi + w) * p.Ci + (size_t)(i * k + j) * p.d.C));
        io.accv[0] += v.x; io.accv[1] += v.y; io.accv[2] += v.z; io.accv[3] += v.w;
      }
    }
    io.n = n; io.h = ho; io.w = wo; io.c = c4 * 4;
    run_program<4, SP>(p.d.prog, io);
    return;
  }
  if (p.kernel <= 3) {
    // up to nine loads, all issued before the first use (the window loop below would wait for each in turn)
    float4 v[9];
#pragma unroll
    for (int dh = 0; dh < 3; ++dh)
#pragma unroll
      for (int dw = 0; dw < 3; ++dw) {
        const int h = h0 + dh, w = w0 + dw;
        const bool ok = dh < p.kernel && dw < p.kernel && h >= 0 && h < p.Hi && w >= 0 && w < p.Wi;
        v[dh * 3 + dw] = ok ? __ldg(reinterpret_cast<const float4*>(xb + ((size_t)h * p.Wi + w) * p.d.C)) : make_float4(init, init, init, init);
      }
#pragma unroll
    for (int e = 0; e < 9; ++e) {
      if (p.is_max) { io.accv[0] = fmaxf(io.accv[0], v[e].x); io.accv[1] = fmaxf(io.accv[1], v[e].y); io.accv[2] = fmaxf(io.accv[2], v[e].z); io.accv[3] = fmaxf(io.accv[3], v[e].w); }
      else { io.accv[0] += v[e].x; io.accv[1] += v[e].y; io.accv[2] += v[e].z; io.accv[3] += v[e].w; }
    }
  } else {
    for (int h = ha; h < hb; ++h) {
      const float* row = xb + ((size_t)h * p.Wi) * p.d.C;
      for (int w = wa; w < wb; ++w) {
        const float4 v = __ldg(reinterpret_cast<const float4*>(row + (size_t)w * p.d.C));
        if (p.is_max) { io.accv[0] = fmaxf(io.accv[0], v.x); io.accv[1] = fmaxf(io.accv[1], v.y); io.accv[2] = fmaxf(io.accv[2], v.z); io.accv[3] = fmaxf(io.accv[3], v.w); }
        else { io.accv[0] += v.x; io.accv[1] += v.y; io.accv[2] += v.z; io.accv[3] += v.w; }
      }
    }
  }
  if (!p.is_max) {                                  // mean over the elements inside the image (padding is not counted)
    const float inv = 1.0f / (float)((hb - ha) * (wb - wa));
#pragma unroll
    for (int v = 0; v < 4; ++v) io.accv[v] *= inv;
  }
  io.n = n; io.h = ho; io.w = wo; io.c = c4 * 4;
  run_program<4, SP>(p.d.prog, io);
}

// Wide windows.  A CTA reduces one slice of one output pixel's window for 128 neighbouring channels: its eight
// warps stride over the slice's elements (a warp reads 512 contiguous bytes per element), then combine through
// shared memory.  With one slice the CTA finishes the pixel itself; otherwise the partial goes to scratch, an
// arrival counter per (pixel, channel group) finds the last CTA, and that CTA combines the slices in slice order
// (the result does not depend on which CTA came last) and runs the epilogue.
template <class SP>
__global__ void __launch_bounds__(256) pool_wide_kernel(const __grid_constant__ PoolParams p) {
  __shared__ float4 part[8][32];
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t slice = blockIdx.x % (uint32_t)p.slices;
  const uint32_t unit = blockIdx.x / (uint32_t)p.slices;
  const uint32_t grp = unit % (uint32_t)p.groups, pix = unit / (uint32_t)p.groups;
  const uint32_t q1 = fd_div(pix, p.fd_w), wo = pix - q1 * (uint32_t)p.d.W;
  const uint32_t n = fd_div(q1, p.fd_h), ho = q1 - n * (uint32_t)p.d.H;
  const int h0 = (int)ho * p.stride - p.pad, w0 = (int)wo * p.stride - p.pad;
  const int ha = max(h0, 0), hb = min(h0 + p.kernel, p.Hi);
  const int wa = max(w0, 0), wb = min(w0 + p.kernel, p.Wi);
  const int ww = wb - wa, count = (hb - ha) * ww;
  const int c = (int)grp * 128 + lane * 4;
  const bool live = c < p.d.C;
  const float init = p.is_max ? -INFINITY : 0.0f;
  float4 acc = make_float4(init, init, init, init);
  const float* xb = p.d.x + ((size_t)n * p.Hi * p.Wi) * p.d.C + c;
  const int e0 = (int)slice * p.per_slice, e1 = min(count, e0 + p.per_slice);
  if (live) {
    for (int eb = e0 + warp; eb < e1; eb += 32) {
      float4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {            // four independent loads in flight per warp
        const int e = eb + 8 * u;
        v[u] = make_float4(init, init, init, init);
        if (e < e1) {
          const int dh = e / ww, dw = e - dh * ww;
          v[u] = __ldg(reinterpret_cast<const float4*>(xb + ((size_t)(ha + dh) * p.Wi + (wa + dw)) * p.d.C));
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (p.is_max) { acc.x = fmaxf(acc.x, v[u].x); acc.y = fmaxf(acc.y, v[u].y); acc.z = fmaxf(acc.z, v[u].z); acc.w = fmaxf(acc.w, v[u].w); }
        else { acc.x += v[u].x; acc.y += v[u].y; acc.z += v[u].z; acc.w += v[u].w; }
      }
    }
  }
  part[warp][lane] = acc;
  __syncthreads();
  if (warp != 0) return;
  auto combine = [&](float4& a, const float4& b) {
    if (p.is_max) { a.x = fmaxf(a.x, b.x); a.y = fmaxf(a.y, b.y); a.z = fmaxf(a.z, b.z); a.w = fmaxf(a.w, b.w); }
    else { a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w; }
  };
  acc = part[0][lane];
#pragma unroll
  for (int w = 1; w < 8; ++w) combine(acc, part[w][lane]);
  if (p.slices > 1) {
    float4* mine = reinterpret_cast<float4*>(p.scratch) + ((size_t)unit * p.slices + slice) * 32;
    mine[lane] = acc;
    __threadfence();                         // the partial is visible before the counter moves
    __syncwarp();
    int old = 0;
    if (lane == 0) old = atomicAdd(&p.counters[unit], 1);
    old = __shfl_sync(0xffffffffu, old, 0);
    if (old != p.slices - 1) return;         // another CTA finishes this pixel
    if (lane == 0) p.counters[unit] = 0;     // ready for the next run
    __threadfence();
    const float4* all = reinterpret_cast<const float4*>(p.scratch) + (size_t)unit * p.slices * 32;
    acc = __ldcg(all + lane);
    for (int s = 1; s < p.slices; ++s) combine(acc, __ldcg(all + (size_t)s * 32 + lane));
  }
  if (!live) return;
  DwIO io{p.d};
  const float inv = p.is_max ? 1.0f : 1.0f / (float)count;
  io.accv[0] = acc.x * inv; io.accv[1] = acc.y * inv; io.accv[2] = acc.z * inv; io.accv[3] = acc.w * inv;
  io.n = n; io.h = ho; io.w = wo; io.c = (uint32_t)c;
  run_program<4, SP>(p.d.prog, io);
}

static const PoolParams& pool_of(const Launch& L) { return *reinterpret_cast<const PoolParams*>(L.blob.data()); }

struct PoolLauncher {
  const Launch& L; cudaStream_t st;
  template <class SP> void run() {
    if (pool_of(L).slices > 0) launch_pdl(pool_wide_kernel<SP>, L.grid, 256, 0, st, pool_of(L));
    else launch_pdl(pool_kernel<SP>, L.grid, 256, 0, st, pool_of(L));
  }
};

int pool_launch(const Launch& L, void* ws_base, cudaStream_t st) {
  {
    PoolParams& pp = *reinterpret_cast<PoolParams*>(const_cast<Launch&>(L).blob.data());
    pp.scratch = L.scratch_off >= 0 ? reinterpret_cast<float*>(reinterpret_cast<char*>(ws_base) + L.scratch_off) : nullptr;
    pp.counters = L.counter_off >= 0 ? reinterpret_cast<int32_t*>(reinterpret_cast<char*>(ws_base) + L.counter_off) : nullptr;
    if (pp.slices > 1 && (!pp.scratch || !pp.counters)) return 1;
  }
  PoolLauncher F{L, st};
  if (!(L.static_id > 0 && StaticSet<ConvStatic>::dispatch(L.static_id, F))) F.run<DynProg>();
  return cudaGetLastError() == cudaSuccess ? 0 : 1;
}

void pool_patch(Launch& L, const std::vector<void*>& ip, const std::vector<void*>& op) {
  PoolParams& pp = *reinterpret_cast<PoolParams*>(L.blob.data());
  pp.d.x = reinterpret_cast<const float*>(ip[0]);
  for (int i = 0; i < pp.d.n_in; ++i) pp.d.in[i].ptr = ip[1 + i];
  for (int i = 0; i < pp.d.n_out; ++i) pp.d.out[i].ptr = op[i];
}

int lower_pool(const Graph& g, const std::vector<int>& ops, int anchor, Block& out, std::string& why) {
  const Op& A = g.ops[anchor];
  const Tensor& X = g.tensors[A.in[0]];
  const Tensor& Y = g.tensors[A.out[0]];
  std::set<int> in_block(ops.begin(), ops.end());
  if (X.dtype != DNNF_F32) { why = "pooling is fp32 only"; return DNNF_ERR_UNSUPPORTED_OP; }
  if (Y.dims[3] % 4) { why = "pooling / col2im needs a channel count that is a multiple of 4"; return DNNF_ERR_UNSUPPORTED_OP; }
  if (in_block.count(X.producer)) { why = "operators in front of a pooling anchor (no prologue fusion)"; return DNNF_ERR_UNSUPPORTED_OP; }
  if (X.numel() >= (1ll << 31) || Y.numel() >= (1ll << 31)) { why = "tensor too large"; return DNNF_ERR_UNSUPPORTED_OP; }
  LowerCtx cx(g);
  cx.ops = ops; cx.in_block = in_block;
  cx.ext = Y.dims;
  if (!derive_views(cx, A.out[0], {anchor})) { why = cx.why; return DNNF_ERR_UNSUPPORTED_OP; }
  if (cx.ext != Y.dims) { why = "epilogue reshapes a pooling result"; return DNNF_ERR_UNSUPPORTED_OP; }
  if (!emit_program(cx, A.out[0], 2)) { why = cx.why; return DNNF_ERR_UNSUPPORTED_OP; }
  Launch& L = out.launch;
  L = Launch{};
  L.blob.assign(sizeof(PoolParams), 0);
  PoolParams& pp = *reinterpret_cast<PoolParams*>(L.blob.data());
  DwParams& dp = pp.d;
  dp.N = (int)Y.dims[0]; dp.H = (int)Y.dims[1]; dp.W = (int)Y.dims[2]; dp.C = (int)Y.dims[3];
  pp.Hi = (int)X.dims[1]; pp.Wi = (int)X.dims[2];
  pp.kernel = (int)A.at.kernel; pp.stride = (int)A.at.stride; pp.pad = (int)A.at.pad;
  pp.is_max = A.kind == DNNF_OP_MAXPOOL;
  pp.col2im = A.kind == DNNF_OP_COL2IM;
  pp.Ci = (int)X.dims[3];
  pp.fd_c4 = make_fastdiv((uint32_t)dp.C / 4); pp.fd_w = make_fastdiv((uint32_t)dp.W); pp.fd_h = make_fastdiv((uint32_t)dp.H);
  pp.fd_s = make_fastdiv((uint32_t)std::max(pp.stride, 1));
  dp.n_in = (int)cx.ins.size(); dp.n_out = (int)cx.outs.size();
  auto fill = [&](TensorArg& a, const ExtArg& e, bool is_out) {
    a.ptr = nullptr; a.base = (int32_t)e.view.c0; a.dtype = g.tensors[e.tensor].dtype; a.mode = 0;
    for (int d = 0; d < kMaxDims; ++d) a.stride[d] = d < 4 ? (int32_t)e.view.coef[3 - d] : 0;
    if (a.dtype != DNNF_F32) return false;
    if (a.stride[0] == 1) { if (a.base % 4) return false; for (int d = 1; d < 4; ++d) if (a.stride[d] % 4) return false; }
    else if (!(a.stride[0] == 0 && !is_out)) return false;
    return true;
  };
  for (size_t i = 0; i < cx.ins.size(); ++i) if (!fill(dp.in[i], cx.ins[i], false)) { why = "pooling epilogue operand is not fp32 / channel-contiguous"; return DNNF_ERR_UNSUPPORTED_OP; }
  for (size_t i = 0; i < cx.outs.size(); ++i) if (!fill(dp.out[i], cx.outs[i], true)) { why = "pooling epilogue output is not fp32 / channel-contiguous"; return DNNF_ERR_UNSUPPORTED_OP; }
  dp.prog = cx.prog;
  L.ew.prog = cx.prog;
  L.in_tensors = {A.in[0]};
  out.inputs = {A.in[0]};
  out.outputs.clear();
  for (auto& a : cx.ins) { L.in_tensors.push_back(a.tensor); if (std::find(out.inputs.begin(), out.inputs.end(), a.tensor) == out.inputs.end()) out.inputs.push_back(a.tensor); }
  for (auto& a : cx.outs) { L.out_tensors.push_back(a.tensor); out.outputs.push_back(a.tensor); }
  L.family = DNNF_FAMILY_POOL;
  L.flops = (int64_t)Y.numel() * pp.kernel * pp.kernel;
  const int64_t total = Y.numel() / 4;
  L.grid = (int)((total + 255) / 256);
  L.threads = 256;
  pp.slices = 0;
  if (!pp.col2im && pp.kernel * pp.kernel >= 64 && !dev_env("DNNF_NO_WIDE_POOL")) {
    // one thread per output would walk the window alone: give the window to whole CTAs instead
    pp.groups = (dp.C + 127) / 128;
    const int64_t units = (int64_t)dp.N * dp.H * dp.W * pp.groups;
    const int window = pp.kernel * pp.kernel;
    int slices = (int)std::min<int64_t>(std::max<int64_t>(1, (2 * 148 + units - 1) / units), std::max(1, window / 32));
    pp.per_slice = (window + slices - 1) / slices;
    pp.slices = (window + pp.per_slice - 1) / pp.per_slice;
    if (units * pp.slices < (1ll << 31)) {
      L.grid = (int)(units * pp.slices);
      if (pp.slices > 1) { L.counter_bytes = units * 4; L.scratch_bytes = units * pp.slices * 128 * 4; }
    } else {
      pp.slices = 0;
    }
  }
  L.variant = pp.is_max;
  L.static_id = StaticSet<ConvStatic>::find(dp.prog);
  out.lowered = true;
  return DNNF_OK;
}

}  // namespace dnnf
