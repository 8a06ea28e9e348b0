// InstanceNormalization over an NHWC fp32 tensor with a fused epilogue chain.
//
// Table 2 lists the operator under Many-to-Many: every result depends on all H x W positions of its own (image,
// channel) plane.  Like the other Many-to-Many anchors it takes One-to-One successors as an epilogue and nothing in
// front.  A CTA owns one image and a group of 4, 8, 16 or 32 neighbouring channels (one to eight 128-bit lanes; the host
// picks the widest group that still gives two CTAs per SM; where images and channels are few it also splits the plane over
// a cluster of 2, 4 or 8 CTAs whose partial sums meet through distributed shared memory and the cluster's hardware
// barrier) and walks its part of the plane three times: sum -> mean, sum of squared
// deviations -> variance (two passes, as the definition reads; no E[x^2] - mean^2 cancellation), then normalise, scale,
// shift, run the chain and store.  The second and third walk find the slab in L1 / L2 (H x W x 16..128 bytes), so the
// kernel's HBM traffic is the input once plus the output once.  Reductions: shuffles among the lanes of a warp that hold
// the same channels, then one shared-memory exchange between the warps, always in the same order.
#include <cooperative_groups.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <set>

#include "conv_params.h"
#include "launch_util.h"
#include "lower.h"

namespace dnnf {

struct InstNormParams {
  DwParams d;              // N, H, W, C; x: the normalised tensor; k unused; epilogue operands
  const float* scale;
  const float* shift;
  float eps;
  int32_t lanes;           // 128-bit lanes per pixel a CTA works on: 1, 2, 4 or 8 (4 channels each)
  int32_t groups;          // channel groups per image: ceil(C / (4 * lanes))
  int32_t split;           // CTAs (one cluster) that share a plane: 1, 2, 4 or 8
};

namespace {
constexpr int kThreads = 256;

// sum over all threads that hold the same channels (threads with equal threadIdx.x % lanes); every thread gets the result
__device__ __forceinline__ float4 plane_sum(float4 v, int lanes, float4 (*xchg)[8]) {
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) {
    if (o < lanes) break;
    v.x += __shfl_xor_sync(0xffffffffu, v.x, o); v.y += __shfl_xor_sync(0xffffffffu, v.y, o);
    v.z += __shfl_xor_sync(0xffffffffu, v.z, o); v.w += __shfl_xor_sync(0xffffffffu, v.w, o);
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __syncthreads();                                   // the exchange area is free again
  if (lane < lanes) xchg[warp][lane] = v;
  __syncthreads();
  float4 s = xchg[0][lane % lanes];
#pragma unroll
  for (int w = 1; w < kThreads / 32; ++w) {
    const float4 t = xchg[w][lane % lanes];
    s.x += t.x; s.y += t.y; s.z += t.z; s.w += t.w;
  }
  return s;
}

// sum of the CTAs' results over the cluster, in rank order; `mine` is this CTA's slot in its own shared memory
template <bool kCluster>
__device__ __forceinline__ float4 cluster_sum(float4 v, float4* mine, int lanes, int split) {
  if (!kCluster) return v;
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  if ((int)threadIdx.x < lanes) mine[threadIdx.x] = v;
  cluster.sync();
  float4 s = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
  for (int r = 0; r < split; ++r) {
    const float4 t = *cluster.map_shared_rank(mine + threadIdx.x % lanes, r);
    s.x += t.x; s.y += t.y; s.z += t.z; s.w += t.w;
  }
  return s;
}

template <class SP, bool kCluster>
__global__ void __launch_bounds__(kThreads) instnorm_kernel(const __grid_constant__ InstNormParams p) {
  __shared__ float4 xchg[kThreads / 32][8];
  __shared__ float4 cpart[2][8];                     // this CTA's sums for the cluster: one slot per pass
  pdl_launch_dependents();
  pdl_wait();
  const int lanes = p.lanes;
  const int split = kCluster ? p.split : 1;
  const int plane = blockIdx.x / split, rank = blockIdx.x - plane * split;     // a cluster is `split` consecutive CTAs
  const int n = plane / p.groups, grp = plane - n * p.groups;
  const int cl = threadIdx.x % lanes, pr = threadIdx.x / lanes, prs = kThreads / lanes;
  const int c = (grp * lanes + cl) * 4;
  const bool live = c < p.d.C;                       // the last group of an image may be narrower
  const int HW = p.d.H * p.d.W;
  const int per = (HW + split - 1) / split;
  const int q_begin = rank * per, q_end = min(HW, q_begin + per);
  const float* xb = p.d.x + (size_t)n * HW * p.d.C + (live ? c : 0);
  const float inv = 1.0f / (float)HW;

  float4 s = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
  const float4 zero4 = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
  if (live)
    for (int q = q_begin + pr; q < q_end; q += 4 * prs) {          // four loads in flight per thread
      float4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) v[u] = q + u * prs < q_end ? __ldg(reinterpret_cast<const float4*>(xb + (size_t)(q + u * prs) * p.d.C)) : zero4;
#pragma unroll
      for (int u = 0; u < 4; ++u) { s.x += v[u].x; s.y += v[u].y; s.z += v[u].z; s.w += v[u].w; }
    }
  s = cluster_sum<kCluster>(plane_sum(s, lanes, xchg), cpart[0], lanes, split);
  const float4 mean = make_float4(s.x * inv, s.y * inv, s.z * inv, s.w * inv);

  float4 m2 = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
  if (live)
    for (int q = q_begin + pr; q < q_end; q += 4 * prs) {
      float4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) v[u] = q + u * prs < q_end ? __ldg(reinterpret_cast<const float4*>(xb + (size_t)(q + u * prs) * p.d.C)) : mean;
#pragma unroll
      for (int u = 0; u < 4; ++u) {                                 // (a pixel past the end was given the mean: deviation 0)
        const float a = v[u].x - mean.x, b = v[u].y - mean.y, e = v[u].z - mean.z, f = v[u].w - mean.w;
        m2.x = fmaf(a, a, m2.x); m2.y = fmaf(b, b, m2.y); m2.z = fmaf(e, e, m2.z); m2.w = fmaf(f, f, m2.w);
      }
    }
  m2 = cluster_sum<kCluster>(plane_sum(m2, lanes, xchg), cpart[1], lanes, split);
  if (live) {
  const float4 sc = __ldg(reinterpret_cast<const float4*>(p.scale + c)), sh = __ldg(reinterpret_cast<const float4*>(p.shift + c));
  // y = (x - mean) / sqrt(var + eps) * scale + shift
  const float4 g = make_float4(sc.x / sqrtf(m2.x * inv + p.eps), sc.y / sqrtf(m2.y * inv + p.eps), sc.z / sqrtf(m2.z * inv + p.eps),
                               sc.w / sqrtf(m2.w * inv + p.eps));
  // four pixels per pass of the chain
  BatchIO<DwIO, 4> b{{DwIO{p.d}, DwIO{p.d}, DwIO{p.d}, DwIO{p.d}}, {false, false, false, false}};
  for (int q = q_begin + pr; q < q_end; q += 4 * prs) {
    float4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int qq = q + u * prs;
      b.on[u] = qq < q_end;
      v[u] = b.on[u] ? __ldg(reinterpret_cast<const float4*>(xb + (size_t)qq * p.d.C)) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int qq = q + u * prs;
      DwIO& io = b.io[u];
      io.accv[0] = fmaf(v[u].x - mean.x, g.x, sh.x); io.accv[1] = fmaf(v[u].y - mean.y, g.y, sh.y);
      io.accv[2] = fmaf(v[u].z - mean.z, g.z, sh.z); io.accv[3] = fmaf(v[u].w - mean.w, g.w, sh.w);
      io.n = n; io.c = c; io.h = qq / p.d.W; io.w = qq - io.h * p.d.W;
    }
    run_program<16, SP>(p.d.prog, b);
  }
  }
  if (kCluster) cooperative_groups::this_cluster().sync();      // nobody leaves while its sums may still be read
}

struct InLauncher {
  const Launch& L; cudaStream_t st; cudaError_t rc = cudaSuccess;
  template <class SP> void run() {
    const InstNormParams& q = *reinterpret_cast<const InstNormParams*>(L.blob.data());
    if (q.split == 1) { rc = launch_pdl(instnorm_kernel<SP, false>, L.grid, kThreads, 0, st, q); return; }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(L.grid); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = 0; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)q.split; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 2;
    rc = cudaLaunchKernelEx(&cfg, instnorm_kernel<SP, true>, q);
  }
};
}  // namespace

int instnorm_launch(const Launch& L, cudaStream_t st) {
  InLauncher F{L, st};
  if (!(L.static_id > 0 && StaticSet<ConvStatic>::dispatch(L.static_id, F))) F.run<DynProg>();
  return F.rc == cudaSuccess ? 0 : 1;
}

void instnorm_patch(Launch& L, const std::vector<void*>& ip, const std::vector<void*>& op) {
  InstNormParams& q = *reinterpret_cast<InstNormParams*>(L.blob.data());
  q.d.x = reinterpret_cast<const float*>(ip[0]);
  q.scale = reinterpret_cast<const float*>(ip[1]);
  q.shift = reinterpret_cast<const float*>(ip[2]);
  for (int i = 0; i < q.d.n_in; ++i) q.d.in[i].ptr = ip[3 + i];
  for (int i = 0; i < q.d.n_out; ++i) q.d.out[i].ptr = op[i];
}

int lower_instnorm(const Graph& g, const std::vector<int>& ops, int anchor, Block& out, std::string& why) {
  const Op& A = g.ops[anchor];
  const Tensor& X = g.tensors[A.in[0]];
  const Tensor& Y = g.tensors[A.out[0]];
  std::set<int> in_block(ops.begin(), ops.end());
  auto refuse = [&](const char* m) { why = m; return DNNF_ERR_UNSUPPORTED_OP; };
  if (X.dtype != DNNF_F32 || g.tensors[A.in[1]].dtype != DNNF_F32 || g.tensors[A.in[2]].dtype != DNNF_F32) return refuse("instance normalisation is fp32 only");
  if (X.dims[3] % 4) return refuse("instance normalisation needs a channel count that is a multiple of 4");
  for (int s = 0; s < 3; ++s) if (in_block.count(g.tensors[A.in[s]].producer)) return refuse("operators in front of an instance normalisation (no prologue fusion)");
  if (X.numel() >= (1ll << 31)) return refuse("tensor too large");
  LowerCtx cx(g);
  cx.ops = ops; cx.in_block = in_block;
  cx.ext = Y.dims;
  if (!derive_views(cx, A.out[0], {anchor})) { why = cx.why; return DNNF_ERR_UNSUPPORTED_OP; }
  if (cx.ext != Y.dims) return refuse("epilogue reshapes an instance normalisation's result");
  if (!emit_program(cx, A.out[0], 2)) { why = cx.why; return DNNF_ERR_UNSUPPORTED_OP; }
  Launch& L = out.launch;
  L = Launch{};
  L.blob.assign(sizeof(InstNormParams), 0);
  InstNormParams& q = *reinterpret_cast<InstNormParams*>(L.blob.data());
  DwParams& dp = q.d;
  dp.N = (int)Y.dims[0]; dp.H = (int)Y.dims[1]; dp.W = (int)Y.dims[2]; dp.C = (int)Y.dims[3];
  q.eps = (float)A.at.eps;
  dp.n_in = (int)cx.ins.size(); dp.n_out = (int)cx.outs.size();
  auto fill = [&](TensorArg& a, const ExtArg& e, bool is_out) {
    a.ptr = nullptr; a.base = (int32_t)e.view.c0; a.dtype = g.tensors[e.tensor].dtype; a.mode = 0;
    for (int d = 0; d < kMaxDims; ++d) a.stride[d] = d < 4 ? (int32_t)e.view.coef[3 - d] : 0;
    if (a.dtype != DNNF_F32) return false;
    if (a.stride[0] == 1) { if (a.base % 4) return false; for (int d = 1; d < 4; ++d) if (a.stride[d] % 4) return false; }
    else if (!(a.stride[0] == 0 && !is_out)) return false;
    return true;
  };
  for (size_t i = 0; i < cx.ins.size(); ++i) if (!fill(dp.in[i], cx.ins[i], false)) return refuse("instance normalisation epilogue operand is not fp32 / channel-contiguous");
  for (size_t i = 0; i < cx.outs.size(); ++i) if (!fill(dp.out[i], cx.outs[i], true)) return refuse("instance normalisation epilogue output is not fp32 / channel-contiguous");
  dp.prog = cx.prog;
  L.ew.prog = cx.prog;
  L.in_tensors = {A.in[0], A.in[1], A.in[2]};
  out.inputs = {A.in[0], A.in[1], A.in[2]};
  out.outputs.clear();
  for (auto& a : cx.ins) { L.in_tensors.push_back(a.tensor); if (std::find(out.inputs.begin(), out.inputs.end(), a.tensor) == out.inputs.end()) out.inputs.push_back(a.tensor); }
  for (auto& a : cx.outs) { L.out_tensors.push_back(a.tensor); out.outputs.push_back(a.tensor); }
  // Two CTAs per SM are wanted.  The widest channel group reads whole 128-byte lines per pixel; where images x groups are
  // too few, first the plane is split over a cluster (as long as every CTA keeps 512 pixels), then the group narrows.
  int lanes = 8, split = 1;
  while (lanes > 1 && lanes > dp.C / 4) lanes >>= 1;
  const int64_t hw = (int64_t)dp.H * dp.W, want = 2ll * sm_count();
  auto ctas = [&]() { return (int64_t)dp.N * ((dp.C / 4 + lanes - 1) / lanes) * split; };
  while (ctas() < want && split < 8 && hw / (2 * split) >= 512) split *= 2;
  while (ctas() < want && lanes > 1) lanes >>= 1;
  q.lanes = lanes; q.split = split;
  q.groups = (dp.C / 4 + lanes - 1) / lanes;
  const int64_t grid = ctas();
  if (grid >= (1ll << 31)) return refuse("too many planes");
  L.grid = (int)grid;
  L.threads = kThreads;
  L.family = DNNF_FAMILY_INSTNORM;
  L.variant = lanes * 10 + split;
  L.flops = 8 * Y.numel();
  L.static_id = StaticSet<ConvStatic>::find(dp.prog);
  out.lowered = true;
  return DNNF_OK;
}

}  // namespace dnnf
