// fp32 GEMM- and pointwise-convolution-anchored blocks on the tensor cores (sm_100a), for
// tall-and-skinny problems: M (pixels / rows) large, the whole [K x N] operand B small enough
// to live in shared memory.  On the FMA pipes such a block is bound by arithmetic; on the
// tensor cores it becomes bound by HBM, which is where a fused block belongs.
//
// fp32 accuracy comes from splitting every operand into two TF32 numbers, x = hi + lo, and accumulating the three
// products lo*hi + hi*lo + hi*hi in fp32 (tensor memory).  B is split once per CTA with rounding (hi = tf32(x),
// lo = tf32(x - hi)); A, which is split on the fly for every tile, with a mask (hi = x cut to 11 significant bits,
// lo = x - hi, cut once more by the tensor core): the dropped lo*lo term and the cut of lo are below 2^-20 relative
// per product, against a parity bar of 1e-5.
//
// One persistent CTA per SM, 448 threads, warp-specialised:
//   warp 0        TMA producer: raw fp32 row blocks of A (whole rows: one contiguous piece of memory
//                 per block when A is dense) into a shared-memory ring; it starts before B is ready
//   warp 1        TMEM allocation, then MMA issue (one elected lane); the A operand of every MMA
//                 comes from tensor memory, only B is read from shared memory
//   warps 2..9    epilogue.  Fast form (dense fp32 output, row-invariant or dense operands): a lane
//                 keeps 32 columns of its own row, row-invariant operands (scale, shift, bias) come
//                 from vectors staged once per CTA in shared memory, the result goes through a
//                 swizzled 32 x 32 chunk buffer to a TMA store.  General form: 32 x 32 transpose
//                 through shared memory, then loads and stores through the block's index maps.
//   warps 10..13  converters: a lane reads its row of a landed raw tile, splits it and writes hi and
//                 lo into a ring of A stages in tensor memory (tcgen05.st).  A small-N MMA is bound
//                 by the shared-memory reads of its operands; with A in tensor memory only the few
//                 rows of B are left.
// B is split once per CTA by all threads into K-major, 128-byte-swizzled hi and lo images (rows
// [0, NP) and [NP, 2NP) of each 32-wide K atom).  When 2*NP <= 256 one MMA multiplies A_hi with
// both images at once (N = 2*NP, two accumulator column ranges that the epilogue adds), so a
// k-step costs two MMAs and two passes over A instead of three.
// Two accumulator stages in TMEM overlap the epilogue of tile i with the main loop of tile i+1.
// Every wait is bounded: on expiry the CTA records DNNF_ERR_TIMEOUT, stops and frees TMEM.
//
// Every TMA load in this file is a plain per-CTA load; no clusters are used.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdlib>
#include <mutex>

#include "ir.h"
#include "tc_common.cuh"
#include "fp32_epilogues.h"
#include "tma_host.h"

namespace dnnf {

namespace tf32 {

#ifdef DNNF_TRACE_LITE
#define FACC3(slot, v) do {} while (0)
#else
#define FACC3(slot, v) FACC(slot, v)
#endif
#ifdef DNNF_TRACE
#define FACC(slot, v) do { if (blockIdx.x == 0 && p.status) atomicAdd(reinterpret_cast<unsigned long long*>(p.status) + 4 + (slot), (unsigned long long)(v)); } while (0)
#else
#define FACC(slot, v) do {} while (0)
#endif

constexpr int BM = 128, BK = 32, EPI_WARPS = 8, CONV_WARPS = 4, THREADS = 64 + 32 * (EPI_WARPS + CONV_WARPS);
constexpr int kSmemMax = 227 * 1024;
constexpr int kMaxStages = 8;                               // raw row blocks in the ring
constexpr int kAStageCols = 2 * BK;                         // TMEM columns of one A stage: hi, then lo
constexpr int kChunkBytes = 32 * 128;                       // 32 rows x 32 fp32, swizzled
constexpr int kMaxVec = 4, kVecFloats = 256 + 32;           // staged row-invariant operands
constexpr int kMinEpiBytes = EPI_WARPS * 2 * kChunkBytes;   // >= EPI_WARPS * kStageWords * 4 (the general form's staging)
constexpr int kFixedNoEpi = 1024 + 512 + kMaxVec * kVecFloats * 4;          // alignment slack, barriers, staged vectors
// chunk buffers of the fast epilogue: one per 32-column chunk a warp handles in a tile, so that a tile's stores are
// issued together and the wait for the buffers falls a whole tile later
inline int epi_bytes_for(int N, int K, bool fast) {
  const int n_epi = N <= 32 ? 4 : 8;
  const int chunks = (N + 31) / 32, per_warp = n_epi == 4 ? chunks : (chunks + 1) / 2;
  int b = n_epi * per_warp * kChunkBytes;
  if (!fast && b < kMinEpiBytes) b = kMinEpiBytes;                // the general form's transpose staging
  const int raw_b = ((K * N * 4 + 1023) / 1024) * 1024;          // a dense B block lands here before it is split
  return b < raw_b && raw_b <= 96 * 1024 ? raw_b : b;
}

constexpr int kMaxBBytes = 88 * 1024;                       // hi + lo images of B

struct Params {
  CUtensorMap tmA, tmD;
  int32_t k_chunks;          // ceil(K / 32)
  int32_t npad;              // N rounded up to 16
  int32_t total_tiles;
  int32_t stages;            // raw row blocks in the shared-memory ring
  int32_t epi_warps;         // 8 epilogue + 4 converter warps, or 4 + 8 when the tile is one 32-column chunk wide
  int32_t rb;                // rows per raw block: 128, 64 or 32
  int32_t pitch;             // floats per shared-memory row of a raw block (the TMA box width; >= K, zero beyond K)
  int32_t unit_stride;       // bytes between ring stages
  int32_t a_stages;          // A stages in tensor memory
  int32_t dual;              // A_hi x [B_hi | B_lo] in one MMA (two accumulator ranges)
  int32_t b_dense;           // B is a dense row-major [K x N] block: fetched with one bulk copy
  int32_t fast_epi;          // the fast epilogue form applies
  int32_t debug;             // ablation switches (development only)
  int32_t epi_bytes;         // chunk buffers / transpose staging / raw B
  int32_t chunks_per_warp;   // fast epilogue: chunk buffers of one warp
  FastDiv fd_n, fd_npad, fd_kpad;   // element index of B -> (k, n)
  int32_t b_static;          // B is an external input: it may be read before the previous kernel ends
  int8_t slot[kMaxIn];       // fast form: staged-vector slot of epilogue input i, or -1 for a dense operand
};

#ifdef DNNF_TF32_POLL
// non-suspending poll
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n.reg .pred p;\nmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_poll(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_test(bar, parity)) return true;
  const unsigned long long t0 = wall_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i) if (mbar_test(bar, parity)) return true;
    if (*abort_flag) return false;
    if (wall_ns() - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
  }
}
#define mbar_wait mbar_wait_poll
#endif
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* tm, uint64_t* bar, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(smem_u32(dst)), "l"(tm), "r"(smem_u32(bar)), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void mma_tf32(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n}"
               ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_tf32_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n}"
               ::"r"(tmem_d), "r"(tmem_a), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
                 "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]),
                 "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]),
                 "r"(r[30]), "r"(r[31]) : "memory");
}
__device__ __forceinline__ void tc_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float to_tf32(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return __uint_as_float(r);
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tm, const void* src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(tm), "r"(smem_u32(src)), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// Fast epilogue IO: a lane owns 32 consecutive columns [c, c+32) of its own row.
struct RowEpiIO {
  static constexpr int VV = 32;
  const GemmParams& p;
  const Params& q;
  float accv[32];
  uint8_t* chunk;            // this warp's current chunk buffer: 32 rows x 128 B, 128-byte swizzle
  const float* vec_s;        // staged row-invariant operands: [kMaxVec][kVecFloats]
  uint32_t row;              // global row of this lane
  bool row_ok;
  int lane, c;
  __device__ __forceinline__ void load(int idx, float (&dst)[VV]) const {
    const int slot = q.slot[idx];
    if (slot >= 0) {           // every lane reads the same words: broadcast
      const float* s = vec_s + slot * kVecFloats + c;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float4 w = *reinterpret_cast<const float4*>(s + 4 * j);
        dst[4 * j] = w.x; dst[4 * j + 1] = w.y; dst[4 * j + 2] = w.z; dst[4 * j + 3] = w.w;
      }
      return;
    }
    const TensorArg& a = p.in[idx];
    const float* src = reinterpret_cast<const float*>(a.ptr) + a.base + (int64_t)row * a.stride[1] + c;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      float4 w = make_float4(0.f, 0.f, 0.f, 0.f);
      if (row_ok && c + 4 * j < p.N) w = __ldg(reinterpret_cast<const float4*>(src + 4 * j));
      dst[4 * j] = w.x; dst[4 * j + 1] = w.y; dst[4 * j + 2] = w.z; dst[4 * j + 3] = w.w;
    }
  }
  __device__ __forceinline__ void anchor(float (&dst)[VV]) const {
#pragma unroll
    for (int v = 0; v < VV; ++v) dst[v] = accv[v];
  }
  __device__ __forceinline__ void store(int, const float (&val)[VV]) const {
#pragma unroll
    for (int j = 0; j < 8; ++j)
      *reinterpret_cast<float4*>(chunk + lane * 128 + ((j ^ (lane & 7)) << 4)) = make_float4(val[4 * j], val[4 * j + 1], val[4 * j + 2], val[4 * j + 3]);
  }
  __device__ __forceinline__ void row_reduce(int, float (&)[VV]) const {}
};

// The same for a result of at most 8 columns (a convolution onto a few channels): the chain runs on 8 values per row
// instead of 32, of which 24 would be padding.
struct RowEpiIO8 {
  static constexpr int VV = 8;
  const GemmParams& p;
  const Params& q;
  float accv[8];
  uint8_t* chunk;
  const float* vec_s;
  uint32_t row;
  bool row_ok;
  int lane;
  __device__ __forceinline__ void load(int idx, float (&dst)[VV]) const {
    const int slot = q.slot[idx];
    if (slot >= 0) {
      const float* s = vec_s + slot * kVecFloats;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        float4 w = *reinterpret_cast<const float4*>(s + 4 * j);
        dst[4 * j] = w.x; dst[4 * j + 1] = w.y; dst[4 * j + 2] = w.z; dst[4 * j + 3] = w.w;
      }
      return;
    }
    const TensorArg& a = p.in[idx];
    const float* src = reinterpret_cast<const float*>(a.ptr) + a.base + (int64_t)row * a.stride[1];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      float4 w = make_float4(0.f, 0.f, 0.f, 0.f);
      if (row_ok && 4 * j < p.N) w = __ldg(reinterpret_cast<const float4*>(src + 4 * j));
      dst[4 * j] = w.x; dst[4 * j + 1] = w.y; dst[4 * j + 2] = w.z; dst[4 * j + 3] = w.w;
    }
  }
  __device__ __forceinline__ void anchor(float (&dst)[VV]) const {
#pragma unroll
    for (int v = 0; v < VV; ++v) dst[v] = accv[v];
  }
  __device__ __forceinline__ void store(int, const float (&val)[VV]) const {
#pragma unroll
    for (int j = 0; j < 2; ++j)
      *reinterpret_cast<float4*>(chunk + lane * 128 + ((j ^ (lane & 7)) << 4)) = make_float4(val[4 * j], val[4 * j + 1], val[4 * j + 2], val[4 * j + 3]);
  }
  __device__ __forceinline__ void row_reduce(int, float (&)[VV]) const {}
};

// byte offset of element (row, k) inside a K-major, 128-byte-swizzled image whose 32-wide K atoms
// are `atom_bytes` apart
__device__ __forceinline__ uint32_t sw128_offset(uint32_t row, uint32_t k, uint32_t atom_bytes) {
  const uint32_t kk = k & 31u;
  return (k >> 5) * atom_bytes + row * 128u + (((kk >> 2) ^ (row & 7u)) << 4) + ((kk & 3u) << 2);
}

template <class SP, bool kFast>
__global__ void __launch_bounds__(THREADS, 1)
gemm_tf32_kernel(const __grid_constant__ GemmParams p, const __grid_constant__ Params q) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int stages = q.stages, NP = q.npad, k_chunks = q.k_chunks;
  const uint32_t atom_bytes = 2u * (uint32_t)NP * 128u;            // one 32-wide K atom of B: hi rows, then lo rows
  const uint32_t lo_off = (uint32_t)NP * 128u;
  const int nranges = q.dual ? 2 : 1;                              // NP-wide column ranges the epilogue adds up
  const int acc_cols = nranges * NP;                               // accumulator stage width in TMEM columns
  const int a_stages = q.a_stages;
  const uint32_t a_cols0 = 2u * (uint32_t)acc_cols;                // A stages follow the two accumulator stages
  uint8_t* ring = smem + (size_t)atom_bytes * k_chunks;            // raw row blocks of A
  uint8_t* epi = ring + (size_t)stages * q.unit_stride;            // chunk buffers (1024-aligned) / transpose staging / raw B
  float* vec_s = reinterpret_cast<float*>(epi + q.epi_bytes);
  uint64_t* raw_bar = reinterpret_cast<uint64_t*>(vec_s + kMaxVec * kVecFloats);
  uint64_t* empty_bar = raw_bar + kMaxStages;    // [stages]   raw block consumed by the converters
  uint64_t* conv_bar = empty_bar + kMaxStages;   // [a_stages] A stage written
  uint64_t* afree_bar = conv_bar + 8;            // [a_stages] A stage consumed by the MMAs
  uint64_t* tfull_bar = afree_bar + 8;           // [2]
  uint64_t* tempty_bar = tfull_bar + 2;          // [2]
  uint64_t* b_bar = tempty_bar + 2;              // raw B landed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(b_bar + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  uint32_t* stage_area = reinterpret_cast<uint32_t*>(epi);       // general form: EPI_WARPS x kStageWords

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_epi = q.epi_warps, conv_sets = (EPI_WARPS + CONV_WARPS - n_epi) / 4;   // converter sets take chunks in turn
  const int rb = q.rb, units = BM / rb;                            // a raw block holds rb rows; `units` blocks per tile
  pdl_launch_dependents();
  const long long t_begin = clock64();
  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { mbar_init(&raw_bar[s], 1); mbar_init(&empty_bar[s], (uint32_t)(rb / 32 * conv_sets)); }
    for (int s = 0; s < a_stages; ++s) { mbar_init(&conv_bar[s], 4); mbar_init(&afree_bar[s], 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(&tfull_bar[s], 1); mbar_init(&tempty_bar[s], (uint32_t)n_epi); }
    mbar_init(b_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int total_tiles = q.total_tiles;

  if (warp == 0) {
    // ---------------- TMA producer: starts at once, while the other warps still prepare B ----------------
    if (lane == 0) {
      pdl_wait();
      // (ring positions and phases advance by increments everywhere: a division by a run-time stage count
      // costs a lone thread some 200 cycles of dependent instructions)
      int s = 0; uint32_t ph = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        for (int u = 0; u < units; ++u) {
          { long long t0 = clock64(); if (!mbar_wait(&empty_bar[s], ph ^ 1, abort_flag)) { ok = false; break; } FACC(1, clock64() - t0); }
          mbar_expect_tx(&raw_bar[s], (uint32_t)(rb * q.pitch * 4));
          tma_load_2d(ring + (size_t)s * q.unit_stride, &q.tmA, &raw_bar[s], 0, tile * BM + u * rb);
          if (++s == stages) { s = 0; ph ^= 1; }
        }
      }
    }
  } else {
    // ---- B: split into hi / lo images, K-major, swizzled; rows >= N and k >= K are zero ----
    const int tid = threadIdx.x - 32, nthr = THREADS - 32;
    const float* W = reinterpret_cast<const float*>(p.B.ptr) + p.B.base;
    const int kpad = k_chunks * BK;
    auto put_b = [&](int k, int n, float x) {
      const float hi = to_tf32(x), lo = to_tf32(x - hi);
      const uint32_t off = sw128_offset((uint32_t)n, (uint32_t)k, atom_bytes);
      *reinterpret_cast<float*>(smem + off) = hi;
      *reinterpret_cast<float*>(smem + lo_off + off) = lo;
    };
    auto fetch_b = [&]() {        // dense B: one bulk copy into the (still unused) epilogue buffers
      if (tid == 0) {
        const uint32_t bytes = (uint32_t)(p.K * p.N * 4);
        mbar_expect_tx(b_bar, bytes);
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_u32(epi)), "l"(W), "r"(bytes), "r"(smem_u32(b_bar)) : "memory");
      }
    };
    auto split_b_strided = [&]() {
      const int total = kpad * NP;
      const bool n_fast = p.B.stride_col == 1;       // walk the contiguous direction of B in global memory
      for (int i0 = tid; i0 < total; i0 += 4 * nthr) {
        float x[4]; int kk[4], nn[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int i = i0 + u * nthr;
          int k, n;
          if (n_fast) { k = (int)fd_div((uint32_t)i, q.fd_npad); n = i - k * NP; } else { n = (int)fd_div((uint32_t)i, q.fd_kpad); k = i - n * kpad; }
          kk[u] = k; nn[u] = n;
          x[u] = (i < total && k < p.K && n < p.N) ? __ldg(W + (int64_t)k * p.B.stride_row + (int64_t)n * p.B.stride_col) : 0.0f;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) if (i0 + u * nthr < total) put_b(kk[u], nn[u], x[u]);
      }
    };
    auto stage_vectors = [&](bool want_static) {
      // row-invariant epilogue operands, once per CTA; zero beyond N
      for (int idx = 0; idx < p.n_in; ++idx) {
        const int slot = q.slot[idx];
        if (slot < 0 || (((p.static_mask >> (1 + idx)) & 1u) != 0) != want_static) continue;
        const TensorArg& a = p.in[idx];
        for (int n = tid; n < kVecFloats; n += nthr)
          vec_s[slot * kVecFloats + n] = n < p.N ? load_scalar<false>(a, (uint32_t)a.base + (uint32_t)n * (uint32_t)a.stride[0]) : 0.0f;
      }
    };
    // An external input is written by no kernel of the graph: reading it may overlap the previous kernel's tail.
    if (q.b_static) { if (q.b_dense) fetch_b(); else split_b_strided(); }
    if (kFast) stage_vectors(true);
    if (q.b_dense && (NP != p.N || kpad != p.K)) {           // zero the padding of the images
      float4* img = reinterpret_cast<float4*>(smem);
      for (int i = tid; i < (int)(atom_bytes / 16) * k_chunks; i += nthr) img[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    // nothing below may touch other global memory before the previous kernel has finished
    pdl_wait();
    if (!q.b_static) { if (q.b_dense) fetch_b(); else split_b_strided(); }
    if (kFast) stage_vectors(false);
    if (q.b_dense) {
      asm volatile("bar.sync 1, %0;" ::"r"(nthr) : "memory");   // zero fill done before values go in
      if (mbar_wait(b_bar, 0, abort_flag)) {
        const float* raw = reinterpret_cast<const float*>(epi);
        const int total = p.K * p.N;
        for (int i = tid; i < total; i += nthr) { const int k = (int)fd_div((uint32_t)i, q.fd_n); put_b(k, i - k * p.N, raw[i]); }
      }
    }
    fence_async_smem();
    asm volatile("bar.sync 1, %0;" ::"r"(nthr) : "memory");
    if (tid == 0) FACC(0, clock64() - t_begin);
  }

  if (warp == 1) {
    if (lane == 0) {
      // ---------------- MMA issuer ----------------
      // instruction descriptors: D fp32, A/B tf32, both K-major, M = 128, N = NP or 2*NP
      const uint32_t idesc0 = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(BM >> 4) << 24);
      const uint32_t idesc = idesc0 | ((uint32_t)(NP >> 3) << 17), idesc2 = idesc0 | ((uint32_t)(NP >> 2) << 17);
      const uint32_t b_base = smem_u32(smem);
      const bool dual = q.dual != 0;
      uint32_t tcount = 0;
      int s = 0; uint32_t ph = 0;
      bool ok = true;
      const uint64_t db0 = make_desc(b_base, 16, 1024);          // B_hi of K atom 0; + atom_bytes / 16 per atom, + lo_off / 16 for B_lo
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++tcount) {
        const int acc = tcount & 1;
        const uint32_t aph = (tcount >> 1) & 1;
        { long long t0 = clock64(); if (!mbar_wait(&tempty_bar[acc], aph ^ 1, abort_flag)) { ok = false; break; } FACC(2, clock64() - t0); }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * acc_cols);
        const long long t_tile = clock64();
        uint64_t dbh = db0;
        int k_left = p.K;
        for (int kc = 0; kc < k_chunks; ++kc, k_left -= BK, dbh += atom_bytes >> 4) {
          { long long t0 = clock64(); if (!mbar_wait(&conv_bar[s], ph, abort_flag)) { ok = false; break; } FACC3(3, clock64() - t0); }
          tc_fence_after();
          const long long t_issue = clock64();
          const int ksteps = min(BK, k_left + 7) >> 3;                   // 8 tf32 per MMA
          const uint32_t a_hi = tmem_base + a_cols0 + (uint32_t)(s * kAStageCols), a_lo = a_hi + BK;
          // B descriptors advance by 32 bytes (2 units of 16) per k-step inside the swizzled atom
          const uint64_t dbl = dbh + (lo_off >> 4);
          if (q.debug & 2) {
          } else if (dual) {
#pragma unroll
            for (int kk = 0; kk < BK / 8; ++kk) {
              if (kk < ksteps) {
                mma_tf32_ts(d_tmem, a_hi + 8 * kk, dbh + 2 * kk, idesc2, (kc | kk) ? 1u : 0u);   // [A_hi B_hi | A_hi B_lo]
                mma_tf32_ts(d_tmem, a_lo + 8 * kk, dbh + 2 * kk, idesc, 1u);                    // + A_lo B_hi on the first range
              }
            }
          } else {
#pragma unroll
            for (int kk = 0; kk < BK / 8; ++kk) {
              if (kk < ksteps) {
                mma_tf32_ts(d_tmem, a_lo + 8 * kk, dbh + 2 * kk, idesc, (kc | kk) ? 1u : 0u);   // small terms first
                mma_tf32_ts(d_tmem, a_hi + 8 * kk, dbl + 2 * kk, idesc, 1u);
                mma_tf32_ts(d_tmem, a_hi + 8 * kk, dbh + 2 * kk, idesc, 1u);
              }
            }
          }
          tc_commit(&afree_bar[s]);          // frees the A stage once these MMAs have read it
          if (++s == a_stages) { s = 0; ph ^= 1; }
          FACC3(4, clock64() - t_issue);
        }
        FACC(10, clock64() - t_tile);
        if (ok) tc_commit(&tfull_bar[acc]);  // accumulator complete
      }
      FACC(11, clock64() - t_begin);
    }
  } else if (warp >= 2 && warp < 2 + n_epi) {
    // ---------------- epilogue warps ----------------
    const int sub = warp & 3;                 // TMEM sub-partition this warp may read
    const int cgroup = (warp - 2) >> 2;       // with 8 warps: takes every second 32-column chunk
    const int cstep = 8 * n_epi;              // 64 or 32 columns
    uint32_t tcount = 0, nstore = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++tcount) {
      const int acc = tcount & 1;
      const uint32_t aph = (tcount >> 1) & 1;
      { long long t0 = clock64(); if (!mbar_wait(&tfull_bar[acc], aph, abort_flag)) { ok = false; break; } if (warp == 2 && lane == 0) FACC(5, clock64() - t0); }
      const long long t_epi = clock64();
      tc_fence_after();
      if (q.debug & 4) { __syncwarp(); if (lane == 0) mbar_arrive(&tempty_bar[acc]); continue; }
      const uint32_t t_row = tmem_base + ((uint32_t)(sub * 32) << 16) + (uint32_t)(acc * acc_cols);
      bool released = false;
      if (kFast) {
        RowEpiIO io{p, q};
        io.lane = lane;
        io.vec_s = vec_s;
        const int m = tile * BM + sub * 32 + lane;
        io.row_ok = m < p.M;
        io.row = io.row_ok ? (uint32_t)m : 0u;
        // One chunk buffer per 32-column chunk of this warp: the tile's stores are issued together at its end, and the
        // wait for the buffers (the previous tile's stores have read them) comes a whole tile after they were issued.
        // (With two buffers per warp, every chunk waited for the store of two chunks earlier: 1100 cycles per chunk.)
        { const long long t0 = clock64(); if (lane == 0) tma_store_wait_read0();
        __syncwarp(); if (warp == 2 && lane == 0) FACC(14, clock64() - t0); }
        uint8_t* my_chunks = epi + (size_t)(warp - 2) * q.chunks_per_warp * kChunkBytes;
        int slot = 0;
        if (p.N <= 8) {                                   // one narrow chunk (cgroup 0 only: four epilogue warps)
          RowEpiIO8 io8{p, q};
          io8.lane = lane; io8.vec_s = vec_s; io8.row_ok = io.row_ok; io8.row = io.row;
          uint32_t raw[8];
          tc_ld8_issue(t_row, raw);
          tc_ld_wait();
#pragma unroll
          for (int j = 0; j < 8; ++j) io8.accv[j] = __uint_as_float(raw[j]);
          for (int r = 1; r < nranges; ++r) {
            tc_ld8_issue(t_row + r * NP, raw);
            tc_ld_wait();
#pragma unroll
            for (int j = 0; j < 8; ++j) io8.accv[j] += __uint_as_float(raw[j]);
          }
          io8.chunk = my_chunks;
          run_program<8, SP, false>(p.prog, io8);
        } else
        for (int c = cgroup * 32; c < p.N; c += cstep, ++slot) {
          uint32_t raw[32];
          const long long t0 = clock64();
          tc_ld32_issue(t_row + c, raw);
          tc_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) io.accv[j] = __uint_as_float(raw[j]);
          for (int r = 1; r < nranges; ++r) {
            tc_ld32_issue(t_row + r * NP + c, raw);
            tc_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) io.accv[j] += __uint_as_float(raw[j]);
          }
          const long long t1 = clock64();
          io.c = c;
          io.chunk = my_chunks + slot * kChunkBytes;
          run_program<32, SP, false>(p.prog, io);
          if (warp == 2 && lane == 0) { FACC(12, t1 - t0); FACC(13, clock64() - t1); }
        }
        // the accumulator stage is free as soon as it has been read
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&tempty_bar[acc]);
        released = true;
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
          slot = 0;
          for (int c = cgroup * 32; c < p.N; c += cstep, ++slot) tma_store_2d(&q.tmD, my_chunks + slot * kChunkBytes, c, tile * BM + sub * 32);
          tma_store_commit();
        }
        (void)nstore;
      } else {
        TcEpiIO io{p};
        uint32_t* stage = stage_area + (warp - 2) * kStageWords;
        io.lane = lane;
        io.m_first = tile * BM + sub * 32;
        const int m = io.m_first + lane;
        const uint32_t mm = m < p.M ? (uint32_t)m : 0u;
#pragma unroll
        for (int k = 0; k < kMaxIn; ++k) {
          io.row_in[k] = 0;
          if (k < p.n_in) io.row_in[k] = (uint32_t)p.in[k].base + tc_digits(p, p.in[k], p.n_nd, p.m_nd, mm);
        }
#pragma unroll
        for (int k = 0; k < kMaxOut; ++k) {
          io.row_out[k] = 0;
          if (k < p.n_out) io.row_out[k] = (uint32_t)p.out[k].base + tc_digits(p, p.out[k], p.n_nd, p.m_nd, mm);
        }
        for (int c = cgroup * 32; c < p.N; c += cstep) {
          uint32_t raw[32];
          tc_ld32_issue(t_row + c, raw);
          tc_ld_wait();
          for (int r = 1; r < nranges; ++r) {
            uint32_t raw2[32];
            tc_ld32_issue(t_row + r * NP + c, raw2);
            tc_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) raw[j] = __float_as_uint(__uint_as_float(raw[j]) + __uint_as_float(raw2[j]));
          }
          // transpose: lane = row  ->  lane = (row group, 4-column piece)
#pragma unroll
          for (int j = 0; j < 32; ++j) stage[lane * 33 + j] = raw[j];
          __syncwarp();
#pragma unroll
          for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) io.accv[i * 4 + e] = __uint_as_float(stage[((lane >> 3) + 4 * i) * 33 + (lane & 7) * 4 + e]);
          __syncwarp();
          io.n0 = (uint32_t)c;
          run_program<32, SP, false>(p.prog, io);
        }
      }
      if (!released) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&tempty_bar[acc]);
      }
      if (warp == 2 && lane == 0) FACC(6, clock64() - t_epi);
    }
    if (kFast && lane == 0) tma_store_wait_all();     // shared memory must outlive the last stores' reads
    (void)nstore;
  } else if (warp >= 2 + n_epi) {
    // ---------------- converters ----------------
    const int sub = warp & 3;                                  // TMEM sub-partition this warp may write
    const int set = (warp - 2 - n_epi) >> 2;                   // this set converts the chunks with ia % conv_sets == set
    const int unit = (sub * 32) / rb;                          // which raw block of the tile holds this warp's rows
    const int row = (sub * 32) % rb + lane;                    // this lane's row inside it
    const int pieces = q.pitch >> 2;                           // 16-byte pieces per shared-memory row
    bool ok = true;
    // raw-block ring position of this warp's block (advances by `units` per tile) and A-stage ring position
    int s = unit % stages; uint32_t rph = (uint32_t)(unit / stages) & 1;
    int as = 0, turn = 0; uint32_t aph = 0;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      // (votes keep the warp together: the tensor-memory stores below are warp-wide)
      { long long t0 = clock64(); if (!__all_sync(0xffffffffu, mbar_wait(&raw_bar[s], rph, abort_flag))) { ok = false; break; } if (warp == 13 && lane == 0) FACC(7, clock64() - t0); }
      const float4* src = reinterpret_cast<const float4*>(ring + (size_t)s * q.unit_stride) + row * pieces;
      for (int kc = 0; kc < k_chunks; ++kc) {
        const bool mine = turn == set;
        if (++turn == conv_sets) turn = 0;
        if (!mine) {
          if (kc == k_chunks - 1) { __syncwarp(); if (lane == 0) mbar_arrive(&empty_bar[s]); }
          if (++as == a_stages) { as = 0; aph ^= 1; }
          continue;
        }
        const long long t_cv = clock64();
        uint32_t hi[32], lo[32];
        if (!(q.debug & 1)) {
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int pc = kc * 8 + j;
            const float4 x = pc < pieces ? src[pc] : make_float4(0.f, 0.f, 0.f, 0.f);
            const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              // hi = x cut to TF32 precision by a mask, lo = x - hi (exact in fp32); the tensor core reads the upper 19
              // bits of lo, i.e. cuts it once more: |a - (hi + lo')| < 2^-20 |a|.  Two full-rate instructions per value
              // instead of two conversions and a subtraction (7 % of the 144 -> 24 block's time).
              const uint32_t hb = __float_as_uint(xs[e]) & 0xffffe000u;
              hi[4 * j + e] = hb;
              lo[4 * j + e] = __float_as_uint(xs[e] - __uint_as_float(hb));
            }
          }
        }
        if (kc == k_chunks - 1) {                                // the raw block is in registers
          __syncwarp();
          if (lane == 0) mbar_arrive(&empty_bar[s]);
        }
        if (!__all_sync(0xffffffffu, mbar_wait(&afree_bar[as], aph ^ 1, abort_flag))) { ok = false; break; }
        if (!(q.debug & 1)) {
          tc_fence_after();
          const uint32_t t_a = tmem_base + ((uint32_t)(sub * 32) << 16) + a_cols0 + (uint32_t)(as * kAStageCols);
          tc_st32(t_a, hi);
          tc_st32(t_a + BK, lo);
          tc_st_wait();
          tc_fence_before();
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&conv_bar[as]);
        if (warp == 13 && lane == 0) FACC(8, clock64() - t_cv);
        if (++as == a_stages) { as = 0; aph ^= 1; }
      }
      s += units;
      while (s >= stages) { s -= stages; rph ^= 1; }
    }
  }

  // ---------------- teardown ----------------
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) FACC(9, clock64() - t_begin);
  if (*abort_flag) {
    if (threadIdx.x == 0 && p.status) { atomicExch(&p.status[0], DNNF_ERR_TIMEOUT); atomicExch(&p.status[1], p.block_index); }
    // give copies that are still in flight time to land before shared memory is released
    if (threadIdx.x == 0) { long long t0 = clock64(); while (clock64() - t0 < 2000000) {} }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

}  // namespace tf32

// ---- host side ------------------------------------------------------------------------------------
static GemmParams& gp_of(Launch& L) { return *reinterpret_cast<GemmParams*>(L.blob.data()); }
static const GemmParams& gp_of(const Launch& L) { return *reinterpret_cast<const GemmParams*>(L.blob.data()); }
// the extras sit behind the parameter blocks of the other tensor-core variants
static tf32::Params& fp_of(Launch& L) { return *reinterpret_cast<tf32::Params*>(L.blob.data() + sizeof(GemmParams) + sizeof(GemmTcParams)); }
static const tf32::Params& fp_of(const Launch& L) { return *reinterpret_cast<const tf32::Params*>(L.blob.data() + sizeof(GemmParams) + sizeof(GemmTcParams)); }

size_t tf32_blob_bytes() { return sizeof(tf32::Params); }

static int tf32_npad(int n) { return (n + 15) / 16 * 16; }
static int tf32_b_bytes_of(int N, int K) { return 2 * tf32_npad(N) * 128 * ((K + tf32::BK - 1) / tf32::BK); }
static int tf32_b_bytes(const GemmParams& gp) { return tf32_b_bytes_of(gp.N, gp.K); }

// The part of the eligibility test that depends on the problem's shape alone (the planner asks it before it
// splits a contraction that is too deep into several that fit).
bool tf32_shape_fits(int64_t M, int64_t N, int64_t K) {
  if (plan_flag(DNNF_PLAN_NO_TF32_GEMM)) return false;
  if (K < 1 || K > 244) return false;                        // a whole row of A (padded) must fit one TMA box of 256 floats
  if (N < 1 || N > 192 || M < 4 * tf32::BM) return false;    // two accumulator stages and two A stages must fit in 512 TMEM columns
  if (tf32_b_bytes_of((int)N, (int)K) > tf32::kMaxBBytes) return false;
  {   // tensor-memory budget (same arithmetic as the plan): never launch with fewer than two A stages
    const int npad = tf32_npad((int)N);
    const bool dual = 4 * npad + 2 * tf32::kAStageCols <= 512;
    if ((512 - 2 * (dual ? 2 : 1) * npad) / tf32::kAStageCols < 2) return false;
  }
  // a whole tile of raw rows must be resident: the converter warps advance chunk by chunk together
  const int kr = ((int)K + 3) / 4 * 4, pitch = kr + ((kr / 4) % 2 == 0 ? 4 : 8);
  if ((tf32::kSmemMax - tf32::kFixedNoEpi - tf32::epi_bytes_for((int)N, (int)K, false) - tf32_b_bytes_of((int)N, (int)K)) / ((32 * pitch * 4 + 1023) / 1024 * 1024) < 4) return false;
  return true;
}

bool tf32_gemm_eligible(const GemmParams& gp) {
  if (gp.A.dtype != DNNF_F32 || gp.B.dtype != DNNF_F32) return false;
  if (gp.batch_ext[0] * gp.batch_ext[1] != 1) return false;
  if (gp.A.stride_col != 1 || gp.A.stride_row % 4 || gp.A.base % 4 || gp.A.stride_row <= 0) return false;
  return tf32_shape_fits(gp.M, gp.N, gp.K);
}

// The fast epilogue form: one dense fp32 output [M x N] (unit stride along n, rows 16-byte aligned),
// every epilogue input either row-invariant (staged in shared memory) or dense like the output.
static bool fast_epilogue(const GemmParams& gp, int8_t* slot) {
  if (gp.n_nd != 1 || gp.m_nd != 1 || gp.n_out != 1 || gp.N % 4) return false;
  auto dense = [](const TensorArg& a) { return a.dtype == DNNF_F32 && a.stride[0] == 1 && a.stride[1] > 0 && a.stride[1] % 4 == 0 && a.base % 4 == 0; };
  if (!dense(gp.out[0])) return false;
  int nslot = 0;
  for (int i = 0; i < gp.n_in; ++i) {
    slot[i] = -1;
    if (gp.in[i].mode == 1) { if (nslot == tf32::kMaxVec) return false; slot[i] = (int8_t)nslot++; }
    else if (!dense(gp.in[i])) return false;
  }
  return true;
}

void tf32_gemm_plan(Launch& L) {
  GemmParams& gp = gp_of(L);
  tf32::Params& q = fp_of(L);
  q.k_chunks = (gp.K + tf32::BK - 1) / tf32::BK;
  q.npad = tf32_npad(gp.N);
  // tensor memory: two accumulator stages (twice as wide in the dual form) and at least two A stages must fit 512 columns
  q.dual = 4 * q.npad + 2 * tf32::kAStageCols <= 512 && !dev_env("DNNF_TF32_NO_DUAL");
  q.fast_epi = fast_epilogue(gp, q.slot) && !dev_env("DNNF_TF32_GENERAL_EPILOGUE");
  q.b_static = gp.static_mask & 1u;
  q.fd_n = make_fastdiv((uint32_t)gp.N); q.fd_npad = make_fastdiv((uint32_t)q.npad); q.fd_kpad = make_fastdiv((uint32_t)(q.k_chunks * tf32::BK));
  q.epi_warps = (gp.N <= 32 && !dev_env("DNNF_TF32_EPI8")) ? 4 : 8;
  q.debug = dev_env("DNNF_TF32_DEBUG") ? atoi(dev_env("DNNF_TF32_DEBUG")) : 0;
  gp.tiles_m = (gp.M + tf32::BM - 1) / tf32::BM;
  gp.tiles_n = 1;
  q.total_tiles = gp.tiles_m;
  L.grid = std::min(q.total_tiles, 148);
  L.threads = tf32::THREADS;
  // shared-memory row of a raw block: K rounded up to 4 floats plus padding that makes the pitch an odd
  // number of 16-byte pieces (conflict-free 128-bit reads down a column of rows)
  const int kr = (gp.K + 3) / 4 * 4;
  q.pitch = kr + ((kr / 4) % 2 == 0 ? 4 : 8);
  q.epi_bytes = tf32::epi_bytes_for(gp.N, gp.K, q.fast_epi != 0);
  { const int chunks = (gp.N + 31) / 32; q.chunks_per_warp = q.epi_warps == 4 ? chunks : (chunks + 1) / 2; }
  const int fixed = tf32::kFixedNoEpi + q.epi_bytes;
  const int ring_budget = tf32::kSmemMax - fixed - tf32_b_bytes(gp);
  q.rb = 32;                                                 // one block per converter warp
  q.unit_stride = (q.rb * q.pitch * 4 + 1023) / 1024 * 1024;
  q.stages = std::min(tf32::kMaxStages, ring_budget / q.unit_stride);
  q.a_stages = std::min(6, (512 - 2 * (q.dual ? 2 : 1) * q.npad) / tf32::kAStageCols);
  L.smem = (size_t)tf32_b_bytes(gp) + (size_t)q.stages * q.unit_stride + fixed;
  q.b_dense = gp.B.stride_col == 1 && gp.B.stride_row == gp.N && gp.N % 4 == 0 && gp.B.base % 4 == 0 &&
              (int64_t)gp.K * gp.N * 4 <= q.epi_bytes && !dev_env("DNNF_TF32_NO_BULK_B");
  L.variant = 4;
  L.static_id = StaticSet<tf32::Static>::find(gp.prog);
}

// fp32 [rows x cols] matrix, unit stride along cols, box = box_cols x box_rows
static bool encode_f32(CUtensorMap* tm, float* base, int64_t cols, int64_t rows, int64_t row_stride, int box_cols, int box_rows,
                       CUtensorMapSwizzle swizzle, std::string& err) {
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)row_stride * 4};
  cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  return tma_encode(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, base, dims, strides, box, swizzle, err);
}

bool tf32_gemm_prepare(Launch& L, std::string& err) {
  GemmParams& gp = gp_of(L);
  tf32::Params& q = fp_of(L);
  float* a = reinterpret_cast<float*>(gp.A.ptr) + gp.A.base;
  if (!encode_f32(&q.tmA, a, gp.K, gp.M, gp.A.stride_row, q.pitch, q.rb, CU_TENSOR_MAP_SWIZZLE_NONE, err)) return false;
  if (q.fast_epi) {
    float* d = reinterpret_cast<float*>(gp.out[0].ptr) + gp.out[0].base;
    if (!encode_f32(&q.tmD, d, gp.N, gp.M, gp.out[0].stride[1], 32, 32, CU_TENSOR_MAP_SWIZZLE_128B, err)) return false;
  }
  return true;
}

template <bool kFast>
struct Tf32Launcher {
  const Launch& L; cudaStream_t st;
  template <class SP> void run() {
    static PerDeviceOnce once;       // per instantiation
    if (once.first_use()) cudaFuncSetAttribute(tf32::gemm_tf32_kernel<SP, kFast>, cudaFuncAttributeMaxDynamicSharedMemorySize, tf32::kSmemMax);
    launch_pdl(tf32::gemm_tf32_kernel<SP, kFast>, L.grid, tf32::THREADS, L.smem, st, gp_of(L), fp_of(L));
  }
};

int tf32_gemm_launch(const Launch& L, cudaStream_t st) {
  if (fp_of(L).fast_epi) {
    Tf32Launcher<true> F{L, st};
    if (!(L.static_id > 0 && StaticSet<tf32::Static>::dispatch(L.static_id, F))) F.run<DynProg>();
  } else {
    Tf32Launcher<false> F{L, st};
    if (!(L.static_id > 0 && StaticSet<tf32::Static>::dispatch(L.static_id, F))) F.run<DynProg>();
  }
  return cudaGetLastError() == cudaSuccess ? 0 : 1;
}

}  // namespace dnnf
