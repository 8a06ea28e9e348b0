// Depthwise 3x3 convolution (stride 1, zero padding 1, fp32 NHWC) with the block's epilogue
// program, tiled through shared memory by TMA (sm_100a).
//
// A CTA owns a sequence of output tiles of HT rows x WT columns x CB channels.  One 4-D TMA
// box load brings the (HT+2) x (WT+2) x CB input patch of a tile into shared memory; the
// halo that falls outside the image is zero-filled by the TMA unit, which IS the
// convolution's padding.  Two patch buffers alternate: the load of tile i+1 is in flight
// while tile i is computed.  A thread owns one (column, 4-channel group) of the tile and
// walks down its rows with a rolling 3x3 register window: three 128-bit shared-memory reads
// and one 128-bit global store per output, every input element fetched from L2/HBM once per
// tile (plus halo) and never through the L1 load path.  Per-channel epilogue operands
// (scale, shift) are read once per thread, not once per output.
//
// Every TMA load in this file is a plain per-CTA load; no clusters are used.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdlib>
#include <mutex>
#include <string>

#include "conv_params.h"
#include "tma_host.h"

namespace dnnf {

namespace dwt {

constexpr int HT = 8, THREADS = 256;
constexpr unsigned long long kWaitLimitNs = 1000000000ull;   // 1 s

struct Params {
  CUtensorMap tmX;           // dims (C, W, H, N), box (cb, wt + 2, HT + 2, 1), no swizzle
  int32_t cb, wt;            // channels and columns per tile
  int32_t tiles_c, tiles_w, tiles_h, total_tiles;
  FastDiv fd_c, fd_w, fd_h, fd_c4; // tile index -> (channel block, column block, row block, image); item -> (column, channel group)
  int32_t invariant[kMaxIn]; // epilogue input i depends on the channel only
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long wall_ns() { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
// Bounded wait: false when the bound ran out (the caller records the failure and leaves).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  if (mbar_try(bar, parity)) return true;
  const unsigned long long t0 = wall_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i) if (mbar_try(bar, parity)) return true;
    if (wall_ns() - t0 > kWaitLimitNs) return false;
  }
}
__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* tm, uint64_t* bar, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
               ::"r"(smem_u32(dst)), "l"(tm), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

// Epilogue IO of one output position (n, h, w, 4 channels); channel-only operands come from registers.
struct TileIO {
  const DwParams& p;
  const Params& q;
  float accv[4];
  float4 inv[3];             // cached channel-only operands (inputs 0..2)
  uint32_t n, h, w, c;
  __device__ __forceinline__ uint32_t off(const TensorArg& a) const {
    return (uint32_t)a.base + c * (uint32_t)a.stride[0] + w * (uint32_t)a.stride[1] + h * (uint32_t)a.stride[2] + n * (uint32_t)a.stride[3];
  }
  __device__ __forceinline__ void fetch(int idx, float (&dst)[4]) const {
    const TensorArg& a = p.in[idx];
    if (a.stride[0] == 0) { float x = load_scalar<true>(a, off(a)); dst[0] = dst[1] = dst[2] = dst[3] = x; }
    else load_vec4<true>(a, off(a), dst);
  }
  __device__ __forceinline__ void load(int idx, float (&dst)[4]) const {
    if (idx < 3 && q.invariant[idx]) { dst[0] = inv[idx].x; dst[1] = inv[idx].y; dst[2] = inv[idx].z; dst[3] = inv[idx].w; return; }
    fetch(idx, dst);
  }
  __device__ __forceinline__ void anchor(float (&dst)[4]) const {
#pragma unroll
    for (int v = 0; v < 4; ++v) dst[v] = accv[v];
  }
  __device__ __forceinline__ void store(int idx, const float (&val)[4]) const { store_vec4<true>(p.out[idx], off(p.out[idx]), val, false); }
  __device__ __forceinline__ void row_reduce(int, float (&)[4]) const {}
};

__device__ __forceinline__ void fma4(float (&acc)[4], const float4& x, const float4& k) {
  acc[0] = fmaf(x.x, k.x, acc[0]); acc[1] = fmaf(x.y, k.y, acc[1]); acc[2] = fmaf(x.z, k.z, acc[2]); acc[3] = fmaf(x.w, k.w, acc[3]);
}

template <class SP>
__global__ void __launch_bounds__(THREADS, 2) dwconv_tma_kernel(const __grid_constant__ DwParams p, const __grid_constant__ Params q, int32_t* status,
                                                                  int block_index) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  const int cb = q.cb, wt = q.wt, c4n = cb / 4;
  const int patch_w = wt + 2;
  const uint32_t patch_bytes = (uint32_t)(HT + 2) * patch_w * cb * 4;
  const uint32_t patch_stride = (patch_bytes + 127u) & ~127u;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + 2 * (size_t)patch_stride);
  __shared__ int failed;

  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    mbar_init(&full_bar[0], 1); mbar_init(&full_bar[1], 1);
    failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  pdl_wait();

  auto issue = [&](int tile, int buf) {
    uint32_t t = (uint32_t)tile, u;
    u = fd_div(t, q.fd_c); const int tc = (int)(t - u * q.tiles_c); t = u;
    u = fd_div(t, q.fd_w); const int tw = (int)(t - u * q.tiles_w); t = u;
    u = fd_div(t, q.fd_h); const int th = (int)(t - u * q.tiles_h); const int n = (int)u;
    mbar_expect_tx(&full_bar[buf], patch_bytes);
    // the halo may start at -1: rows and columns outside the image arrive as zeros (the convolution's padding)
    tma_load_4d(smem + (size_t)buf * patch_stride, &q.tmX, &full_bar[buf], tc * cb, tw * wt - 1, th * HT - 1, n);
  };

  if (threadIdx.x == 0 && (int)blockIdx.x < q.total_tiles) issue(blockIdx.x, 0);
  const int items = c4n * wt;                       // (column, channel group) pairs of a tile
  // weights and channel-only epilogue operands of this thread's channel group: the same for every tile
  // when one channel block covers C and a thread owns one item
  const bool hoist = q.tiles_c == 1 && items <= THREADS;
  float4 kw[9];
  TileIO io{p, q};
  io.n = io.h = io.w = 0;
  auto load_consts = [&](int c) {
#pragma unroll
    for (int i = 0; i < 9; ++i) kw[i] = __ldg(reinterpret_cast<const float4*>(p.k + i * p.C + c));
    io.c = c;
#pragma unroll
    for (int i = 0; i < 3; ++i)
      if (i < p.n_in && q.invariant[i]) { float v[4]; io.fetch(i, v); io.inv[i] = make_float4(v[0], v[1], v[2], v[3]); }
  };
  if (hoist && (int)threadIdx.x < items) load_consts(((int)threadIdx.x - (int)fd_div(threadIdx.x, q.fd_c4) * c4n) * 4);
  uint32_t k = 0;
  for (int tile = blockIdx.x; tile < q.total_tiles; tile += gridDim.x, ++k) {
    const int buf = k & 1;
    const int next = tile + gridDim.x;
    // buffer buf^1 was read during iteration k-1, which ended with a barrier
    if (threadIdx.x == 0 && next < q.total_tiles) issue(next, buf ^ 1);
    if (!mbar_wait(&full_bar[buf], (k >> 1) & 1)) failed = 1;
    __syncthreads();
    if (failed) break;
    uint32_t t = (uint32_t)tile, u;
    u = fd_div(t, q.fd_c); const int tc = (int)(t - u * q.tiles_c); t = u;
    u = fd_div(t, q.fd_w); const int tw = (int)(t - u * q.tiles_w); t = u;
    u = fd_div(t, q.fd_h); const int th = (int)(t - u * q.tiles_h); const int n = (int)u;
    const float4* patch = reinterpret_cast<const float4*>(smem + (size_t)buf * patch_stride);
    for (int item = threadIdx.x; item < items; item += THREADS) {
      const int wl = (int)fd_div((uint32_t)item, q.fd_c4), c4 = item - wl * c4n;
      const int w = tw * wt + wl, c = tc * cb + c4 * 4;
      if (w >= p.W || c >= p.C) continue;
      if (!hoist) load_consts(c);
      io.n = n; io.w = w; io.c = c;
      // patch element (row r, column wl + dx, channel group c4)
      const float4* col = patch + wl * c4n + c4;
      const int row_stride = patch_w * c4n;
      float4 r[3][3];
#pragma unroll
      for (int dx = 0; dx < 3; ++dx) { r[0][dx] = col[dx * c4n]; r[1][dx] = col[row_stride + dx * c4n]; }
#pragma unroll
      for (int hl = 0; hl < HT; ++hl) {
        const float4* src = col + (hl + 2) * row_stride;
#pragma unroll
        for (int dx = 0; dx < 3; ++dx) r[(hl + 2) % 3][dx] = src[dx * c4n];
        io.accv[0] = io.accv[1] = io.accv[2] = io.accv[3] = 0.0f;
#pragma unroll
        for (int dy = 0; dy < 3; ++dy)
#pragma unroll
          for (int dx = 0; dx < 3; ++dx) fma4(io.accv, r[(hl + dy) % 3][dx], kw[dy * 3 + dx]);
        const int h = th * HT + hl;
        if (h < p.H) { io.h = h; run_program<4, SP>(p.prog, io); }
      }
    }
    __syncthreads();                                 // everyone is done with this buffer
  }
  if (failed && threadIdx.x == 0 && status) {
    atomicExch(&status[0], DNNF_ERR_TIMEOUT); atomicExch(&status[1], block_index);
    long long t0 = clock64(); while (clock64() - t0 < 2000000) {}      // let a copy that is still in flight land
  }
  __syncthreads();
}

}  // namespace dwt

// ---- host side ------------------------------------------------------------------------------------
static DwParams& dw_of(Launch& L) { return *reinterpret_cast<DwParams*>(L.blob.data()); }
static const DwParams& dw_of(const Launch& L) { return *reinterpret_cast<const DwParams*>(L.blob.data()); }
static dwt::Params& tq_of(Launch& L) { return *reinterpret_cast<dwt::Params*>(L.blob.data() + sizeof(DwParams)); }
static const dwt::Params& tq_of(const Launch& L) { return *reinterpret_cast<const dwt::Params*>(L.blob.data() + sizeof(DwParams)); }

size_t dwconv_tma_blob_bytes() { return sizeof(dwt::Params); }

// Picks the tile; false when the shape does not suit this kernel.
bool dwconv_tma_plan(Launch& L) {
  if (plan_flag(DNNF_PLAN_NO_TMA_DWCONV)) return false;
  const DwParams& dp = dw_of(L);
  dwt::Params& q = tq_of(L);
  if (dp.C % 4 || dp.H < 4 || dp.W < 4) return false;
  // channel block: the whole channel dim when a box can hold it, else the largest divisor-free split <= 256
  int cb = dp.C;
  if (cb > 256) cb = 256;
  // columns per tile: about 256 threads' worth of (column, channel group) pairs, both patch buffers within 106 KB (two CTAs per SM)
  int wt = std::max(1, std::min(dp.W, (dwt::THREADS * 4) / cb));
  while (wt > 1 && 2ll * (dwt::HT + 2) * (wt + 2) * cb * 4 > 106 * 1024) --wt;
  if (2ll * (dwt::HT + 2) * (wt + 2) * cb * 4 > 106 * 1024) return false;
  if (wt + 2 > 256) return false;
  q.cb = cb; q.wt = wt;
  q.tiles_c = (dp.C + cb - 1) / cb;
  q.tiles_w = (dp.W + wt - 1) / wt;
  q.tiles_h = (dp.H + dwt::HT - 1) / dwt::HT;
  q.fd_c = make_fastdiv((uint32_t)q.tiles_c); q.fd_w = make_fastdiv((uint32_t)q.tiles_w); q.fd_h = make_fastdiv((uint32_t)q.tiles_h);
  q.fd_c4 = make_fastdiv((uint32_t)(cb / 4));
  const int64_t total = (int64_t)q.tiles_c * q.tiles_w * q.tiles_h * dp.N;
  if (total >= (1ll << 31) || total < 148) return false;        // too small to fill the machine: the direct kernel is better
  q.total_tiles = (int)total;
  for (int i = 0; i < kMaxIn; ++i) {
    const TensorArg& a = dp.in[i];
    q.invariant[i] = i < dp.n_in && a.stride[1] == 0 && a.stride[2] == 0 && a.stride[3] == 0;
  }
  const size_t patch = ((size_t)(dwt::HT + 2) * (wt + 2) * cb * 4 + 127) & ~size_t(127);
  L.smem = 2 * patch + 128 + 64;
  L.threads = dwt::THREADS;
  L.grid = (int)std::min<int64_t>(total, 2 * 148);
  L.variant = -1;                                               // marks the TMA kernel (the direct kernel keeps its strip height here)
  L.static_id = StaticSet<ConvStatic>::find(dp.prog);
  return true;
}

bool dwconv_tma_prepare(Launch& L, std::string& err) {
  const DwParams& dp = dw_of(L);
  dwt::Params& q = tq_of(L);
  cuuint64_t dims[4] = {(cuuint64_t)dp.C, (cuuint64_t)dp.W, (cuuint64_t)dp.H, (cuuint64_t)dp.N};
  cuuint64_t strides[3] = {(cuuint64_t)dp.C * 4, (cuuint64_t)dp.W * dp.C * 4, (cuuint64_t)dp.H * dp.W * dp.C * 4};
  cuuint32_t box[4] = {(cuuint32_t)q.cb, (cuuint32_t)(q.wt + 2), (cuuint32_t)(dwt::HT + 2), 1};
  if (!tma_encode(&q.tmX, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float*>(dp.x), dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE, err)) return false;
  return true;
}

struct DwTmaLauncher {
  const Launch& L; cudaStream_t st; int32_t* status; int block_index;
  template <class SP> void run() {
    static PerDeviceOnce once;       // per instantiation
    if (once.first_use()) cudaFuncSetAttribute(dwt::dwconv_tma_kernel<SP>, cudaFuncAttributeMaxDynamicSharedMemorySize, 112 * 1024);
    launch_pdl(dwt::dwconv_tma_kernel<SP>, L.grid, dwt::THREADS, L.smem, st, dw_of(L), tq_of(L), status, block_index);
  }
};

int dwconv_tma_launch(const Launch& L, int32_t* status, int block_index, cudaStream_t st) {
  DwTmaLauncher F{L, st, status, block_index};
  if (!(L.static_id > 0 && StaticSet<ConvStatic>::dispatch(L.static_id, F))) F.run<DynProg>();
  return cudaGetLastError() == cudaSuccess ? 0 : 1;
}

}  // namespace dnnf
