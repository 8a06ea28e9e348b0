// Tensor-core GEMM-anchored blocks for sm_100a: TMA -> 128B-swizzled shared memory ->
// tcgen05.mma (bf16 x bf16 -> fp32 in tensor memory) -> tcgen05.ld epilogue that runs
// the block's micro-op program (bias, GELU, residual, scale, mask ...) on the
// accumulator and stores through the block's output index map.
//
// One persistent CTA per SM, 320 threads, warp-specialised:
//   warp 0      TMA producer (one elected lane)
//   warp 1      TMEM allocation, then MMA issue (one elected lane)
//   warps 2..9  epilogue; warp w reads TMEM lanes 32*(w%4) .. 32*(w%4)+31, warps 2..5 the first
//               half of the tile's columns, warps 6..9 the second half
// A BK=64 shared-memory ring feeds the MMA; two accumulator stages in TMEM let the
// epilogue of tile i overlap the main loop of tile i+1.  Every wait is bounded: when a
// bound runs out the CTA records DNNF_ERR_TIMEOUT in the status words, stops issuing
// work, releases tensor memory and returns.
//
// Every TMA load in this file is a plain per-CTA load; no clusters are used.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdlib>
#include <mutex>

#include "ir.h"
#include "tc_common.cuh"
#include "tma_host.h"

namespace dnnf {

constexpr int TC_BM = 128, TC_BK = 64, TC_EPI_WARPS = 8, TC_THREADS = 64 + 32 * TC_EPI_WARPS;
constexpr int kSmemMax = 227 * 1024;                       // dynamic shared memory per CTA
constexpr int kSmemFixed = 1024 + 256 + TC_EPI_WARPS * kStageWords * 4;   // alignment slack, barriers, staging
constexpr int kSmemBudget = kSmemMax - kSmemFixed;         // left for the operand ring

#ifdef DNNF_TRACE
__device__ __forceinline__ unsigned long long gtime() { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
#define TRACE(slot) do { if (blockIdx.x == 0 && p.status) reinterpret_cast<unsigned long long*>(p.status)[4 + (slot)] = gtime(); } while (0)
#else
#define TRACE(slot) do {} while (0)
#endif

// ---- the kernel ---------------------------------------------------------------------------------
template <class SP>
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ GemmParams p, const __grid_constant__ GemmTcParams q, const __grid_constant__ CUtensorMap tmA,
               const __grid_constant__ CUtensorMap tmB, int stages) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  // carve: [stages][A tile 16 KB][B tile BN*128 B], then barriers
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int BN = q.bn;
  const uint32_t a_bytes = TC_BM * TC_BK * 2, b_bytes = (uint32_t)BN * TC_BK * 2, stage_bytes = a_bytes + b_bytes;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + (size_t)stages * stage_bytes);
  uint64_t* empty_bar = full_bar + stages;
  uint64_t* tfull_bar = empty_bar + stages;      // [2]
  uint64_t* tempty_bar = tfull_bar + 2;          // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty_bar + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  uint32_t* stage_area = tmem_slot + 8;          // TC_EPI_WARPS x kStageWords

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  pdl_launch_dependents();
  if (threadIdx.x == 0) TRACE(0);
  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(&tfull_bar[s], 1); mbar_init(&tempty_bar[s], TC_EPI_WARPS); }
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
  if (threadIdx.x == 0) TRACE(1);
  // set-up above overlaps the previous kernel's tail; nothing below may touch global memory earlier
  pdl_wait();

  const int tiles_mn = p.tiles_m * p.tiles_n;
  const int total_tiles = q.persistent_tiles;
  const int k_tiles = q.k_tiles;

  if (warp == 0) {
    if (lane == 0) {
      // ---------------- TMA producer ----------------
      // (stage index and phase advance by increments: a division by the run-time stage count costs this
      // single thread some 200 cycles of dependent instructions per k-tile)
      int s = 0; uint32_t ph = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const int batch = (int)fd_div((uint32_t)tile, q.fd_tiles_mn), r = tile - batch * tiles_mn;
        const int tm = (int)fd_div((uint32_t)r, q.fd_tiles_n), tn = r - tm * p.tiles_n;
        const int b1 = (int)fd_div((uint32_t)batch, q.fd_batch0), b0 = batch - b1 * p.batch_ext[0];
        // a batch dim an operand is broadcast over has stride 0 and extent 1 in its tensor map
        const int ab0 = p.A.batch_stride[0] ? b0 : 0, ab1 = p.A.batch_stride[1] ? b1 : 0;
        const int bb0 = p.B.batch_stride[0] ? b0 : 0, bb1 = p.B.batch_stride[1] ? b1 : 0;
        for (int kt = 0; kt < k_tiles; ++kt) {
          if (!mbar_wait(&empty_bar[s], ph ^ 1, abort_flag)) { ok = false; break; }
          uint8_t* sa = smem + (size_t)s * stage_bytes;
          uint8_t* sb = sa + a_bytes;
          mbar_expect_tx(&full_bar[s], stage_bytes);
          tma_load_4d(sa, &tmA, &full_bar[s], kt * TC_BK, tm * TC_BM, ab0, ab1);
          if (q.b_kmajor) {
            tma_load_4d(sb, &tmB, &full_bar[s], kt * TC_BK, tn * BN, bb0, bb1);
          } else {
            for (int j = 0; j < BN / 64; ++j)
              tma_load_4d(sb + j * (64 * TC_BK * 2), &tmB, &full_bar[s], tn * BN + j * 64, kt * TC_BK, bb0, bb1);
          }
          if (++s == stages) { s = 0; ph ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---------------- MMA issuer ----------------
      // instruction descriptor: D fp32, A/B bf16, A K-major, B per operand, N, M=128
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((q.b_kmajor ? 0u : 1u) << 16) | ((uint32_t)(BN >> 3) << 17) |
                             ((uint32_t)(TC_BM >> 4) << 24);
      uint32_t tcount = 0;
      int s = 0; uint32_t ph = 0;
      bool ok = true;
      // descriptors of stage 0; a stage further on adds stage_bytes / 16 to the address field, a k-step 2 (32 bytes)
      // or, for an MN-major B, 128 (2048 bytes)
      const uint64_t da0 = make_desc(smem_u32(smem), 16, 1024);
      const uint64_t db0 = q.b_kmajor ? make_desc(smem_u32(smem) + a_bytes, 16, 1024) : make_desc(smem_u32(smem) + a_bytes, 64 * TC_BK * 2, 1024);
      const uint64_t dstage = stage_bytes >> 4, dbk = q.b_kmajor ? 2 : 128;
      uint64_t da_s = da0, db_s = db0;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++tcount) {
        const int acc = tcount & 1;
        const uint32_t aph = (tcount >> 1) & 1;
        if (!mbar_wait(&tempty_bar[acc], aph ^ 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kt = 0; kt < k_tiles; ++kt) {
          if (!mbar_wait(&full_bar[s], ph, abort_flag)) { ok = false; break; }
          // (no tcgen05 fence: TMA wrote the operands and the barrier orders its completion before the MMAs' reads)
#pragma unroll
          for (int kk = 0; kk < TC_BK / 16; ++kk)
            tc_mma_bf16(d_tmem, da_s + 2 * kk, db_s + dbk * kk, idesc, (kt | kk) ? 1u : 0u);
          tc_commit(&empty_bar[s]);          // frees the smem stage once these MMAs have read it
          da_s += dstage; db_s += dstage;
          if (++s == stages) { s = 0; ph ^= 1; da_s = da0; db_s = db0; }
        }
        if (ok) tc_commit(&tfull_bar[acc]);  // accumulator complete
        if (tcount == 0) TRACE(4);
      }
    }
  } else {
    // ---------------- epilogue warps ----------------
    const int sub = warp & 3;                 // TMEM sub-partition this warp may read
    uint32_t tcount = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++tcount) {
      const int batch = (int)fd_div((uint32_t)tile, q.fd_tiles_mn), r = tile - batch * tiles_mn;
      const int tm = (int)fd_div((uint32_t)r, q.fd_tiles_n), tn = r - tm * p.tiles_n;
      const int acc = tcount & 1;
      const uint32_t aph = (tcount >> 1) & 1;
      if (!mbar_wait(&tfull_bar[acc], aph, abort_flag)) { ok = false; break; }
      if (tcount == 0 && warp == 2 && lane == 0) TRACE(5);
      tc_fence_after();
      TcEpiIO io{p};
      uint32_t* stage = stage_area + (warp - 2) * kStageWords;
      io.lane = lane;
      io.m_first = tm * TC_BM + sub * 32;
      const int m = io.m_first + lane;
      const uint32_t mm = m < p.M ? (uint32_t)m : 0u;
      // (fully unrolled with constant indices so that the offset tables stay in registers)
#pragma unroll
      for (int k = 0; k < kMaxIn; ++k) {
        io.row_in[k] = 0;
        if (k < p.n_in)
          io.row_in[k] = (uint32_t)p.in[k].base + tc_digits(p, p.in[k], p.n_nd, p.m_nd, mm) + tc_digits(p, p.in[k], p.n_nd + p.m_nd, p.b_nd, (uint32_t)batch);
      }
#pragma unroll
      for (int k = 0; k < kMaxOut; ++k) {
        io.row_out[k] = 0;
        if (k < p.n_out)
          io.row_out[k] = (uint32_t)p.out[k].base + tc_digits(p, p.out[k], p.n_nd, p.m_nd, mm) + tc_digits(p, p.out[k], p.n_nd + p.m_nd, p.b_nd, (uint32_t)batch);
      }
      const int half = (warp - 2) >> 2;        // which half of the tile's columns
      const int c_begin = half * (BN / 2), c_end = c_begin + BN / 2;
      const uint32_t t_row = tmem_base + ((uint32_t)(sub * 32) << 16) + (uint32_t)(acc * BN);
      for (int c = c_begin; c < c_end; c += 32) {
        const int n0 = tn * BN + c;
        if (n0 >= p.N) break;                  // uniform across the warp
        if (q.debug & 4) continue;
        uint32_t raw[32];
        if (tcount == 0 && warp == 2 && lane == 0 && c == c_begin) TRACE(8);
        tc_ld32_issue(t_row + c, raw);
        tc_ld_wait();
        if (tcount == 0 && warp == 2 && lane == 0 && c == c_begin) TRACE(9);
        // transpose: lane = row  ->  lane = (row group, 4-column piece)
        if (!(q.debug & 2)) {
#pragma unroll
        for (int j = 0; j < 32; ++j) stage[lane * 33 + j] = raw[j];
        __syncwarp();
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
          for (int e = 0; e < 4; ++e) io.accv[i * 4 + e] = __uint_as_float(stage[((lane >> 3) + 4 * i) * 33 + (lane & 7) * 4 + e]);
        __syncwarp();
        }
        if (tcount == 0 && warp == 2 && lane == 0 && c == c_begin) TRACE(10);
        io.n0 = (uint32_t)n0;
        if (!(q.debug & 1)) run_program<32, SP, true>(p.prog, io);
        if (tcount == 0 && warp == 2 && lane == 0 && c == c_begin) TRACE(11);
      }
      tc_fence_before();
      __syncwarp();
      if (tcount == 0 && warp == 2 && lane == 0) TRACE(6);
      if (lane == 0) mbar_arrive(&tempty_bar[acc]);
    }
  }

  // ---------------- teardown ----------------
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) TRACE(7);
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

// ---- static epilogue programs -----------------------------------------------------------------------
#define MO(o, s, i) MicroOp{o, s, i, 0}
DNNF_SP_BEGIN(EP_Store, 2) MO(M_MOV, S_ANCHOR, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(EP_Bias, 3) MO(M_MOV, S_ANCHOR, 0), MO(M_ADD, S_IN, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(EP_BiasGeluTanh, 4) MO(M_MOV, S_ANCHOR, 0), MO(M_ADD, S_IN, 0), MO(M_GELU_TANH, S_NONE, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(EP_BiasResidual, 4) MO(M_MOV, S_ANCHOR, 0), MO(M_ADD, S_IN, 0), MO(M_ADD, S_IN, 1), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(EP_ScaleMask, 4) MO(M_MOV, S_ANCHOR, 0), MO(M_MUL, S_CONST, 0), MO(M_ADD, S_IN, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(EP_BiasGeluPrimitives, 9)
  MO(M_MOV, S_ANCHOR, 0), MO(M_ADD, S_IN, 0), MO(M_SAVE, S_TMP, 0), MO(M_MUL, S_CONST, 0), MO(M_ERF, S_NONE, 0), MO(M_ADD, S_CONST, 1),
  MO(M_MUL, S_TMP, 0), MO(M_MUL, S_CONST, 2), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(EP_BiasGeluTanhPrimitives, 13)
  MO(M_MOV, S_ANCHOR, 0), MO(M_ADD, S_IN, 0), MO(M_SAVE, S_TMP, 0), MO(M_SQUARE, S_NONE, 0), MO(M_MUL, S_TMP, 0), MO(M_MUL, S_CONST, 0),
  MO(M_ADD, S_TMP, 0), MO(M_MUL, S_CONST, 1), MO(M_TANH, S_NONE, 0), MO(M_ADD, S_CONST, 2), MO(M_MUL, S_TMP, 0), MO(M_MUL, S_CONST, 3),
  MO(M_STORE, S_NONE, 0) DNNF_SP_END
#undef MO
using EpiStatic = TypeList<EP_Store, EP_Bias, EP_BiasGeluTanh, EP_BiasResidual, EP_ScaleMask, EP_BiasGeluPrimitives, EP_BiasGeluTanhPrimitives>;

// ---- host side --------------------------------------------------------------------------------------
static GemmParams& gp_of(Launch& L) { return *reinterpret_cast<GemmParams*>(L.blob.data()); }
static const GemmParams& gp_of(const Launch& L) { return *reinterpret_cast<const GemmParams*>(L.blob.data()); }
static GemmTcParams& tc_of(Launch& L) { return *reinterpret_cast<GemmTcParams*>(L.blob.data() + sizeof(GemmParams)); }
static const GemmTcParams& tc_of(const Launch& L) { return *reinterpret_cast<const GemmTcParams*>(L.blob.data() + sizeof(GemmParams)); }

bool tc_gemm_eligible(const GemmParams& gp) {
  if (gp.A.dtype != DNNF_BF16 || gp.B.dtype != DNNF_BF16) return false;
  auto ok8 = [](int64_t v) { return v % 8 == 0; };
  // A: K-major only
  if (gp.A.stride_col != 1 || !ok8(gp.A.stride_row) || !ok8(gp.A.base) || !ok8(gp.A.batch_stride[0]) || !ok8(gp.A.batch_stride[1])) return false;
  bool b_k = gp.B.stride_row == 1, b_n = gp.B.stride_col == 1;
  if (gp.K == 1 && b_n) b_k = false;
  if (!b_k && !b_n) return false;
  int64_t other = b_n ? gp.B.stride_row : gp.B.stride_col;
  if (!ok8(other) || !ok8(gp.B.base) || !ok8(gp.B.batch_stride[0]) || !ok8(gp.B.batch_stride[1])) return false;
  if (gp.A.stride_row <= 0 || other <= 0) return false;
  if (gp.K % 8 || (b_n && gp.N % 8)) return false;       // tensor-map extents in 16-byte units
  return true;
}

void tc_gemm_plan(Launch& L) {
  GemmParams& gp = gp_of(L);
  GemmTcParams& tc = tc_of(L);
  tc.a_kmajor = 1;
  tc.b_kmajor = (gp.B.stride_col != 1) ? 1 : 0;
  tc.k_tiles = (gp.K + TC_BK - 1) / TC_BK;
  int nb = gp.batch_ext[0] * gp.batch_ext[1];
  int tiles_m = (gp.M + TC_BM - 1) / TC_BM;
  // N tile: the candidate with the best SM utilisation over whole waves; larger tiles win ties
  int best_bn = 64; double best = -1;
  for (int bn : {256, 192, 128, 64}) {
    if (bn > 64 && bn / 2 >= gp.N) continue;
    int tiles = tiles_m * ((gp.N + bn - 1) / bn) * nb;
    int waves = (tiles + 147) / 148;
    double useful = (double)gp.N / (((gp.N + bn - 1) / bn) * bn);
    double eff = (double)tiles / (waves * 148.0) * useful * (bn >= 128 ? 1.0 : 0.9);
    if (eff > best + 1e-9) { best = eff; best_bn = bn; }
  }
  tc.bn = best_bn;
  gp.tiles_m = tiles_m;
  gp.tiles_n = (gp.N + tc.bn - 1) / tc.bn;
  tc.persistent_tiles = gp.tiles_m * gp.tiles_n * nb;
  tc.fd_tiles_mn = make_fastdiv((uint32_t)(gp.tiles_m * gp.tiles_n));
  tc.fd_tiles_n = make_fastdiv((uint32_t)gp.tiles_n);
  tc.fd_batch0 = make_fastdiv((uint32_t)gp.batch_ext[0]);
  L.grid = std::min(tc.persistent_tiles, 148);
  L.threads = TC_THREADS;
  int stage_bytes = TC_BM * TC_BK * 2 + tc.bn * TC_BK * 2;
  int stages = std::min(8, kSmemBudget / stage_bytes);
  L.smem = (size_t)stages * stage_bytes + kSmemFixed;
  L.variant = 1;
  L.static_id = StaticSet<EpiStatic>::find(gp.prog);
  tc.debug = dev_env("DNNF_GEMM_DEBUG") ? atoi(dev_env("DNNF_GEMM_DEBUG")) : 0;
}

// dims innermost first: {inner, outer, b0, b1}
static bool encode(CUtensorMap* tm, void* base, int64_t ext_inner, int64_t ext_outer, int64_t stride_outer, const int32_t* bext,
                   const int64_t* bstride, int box_inner, int box_outer, std::string& err) {
  cuuint64_t dims[4] = {(cuuint64_t)ext_inner, (cuuint64_t)ext_outer, (cuuint64_t)bext[0], (cuuint64_t)bext[1]};
  // a broadcast (stride 0) batch dim is addressed with coordinate 0 only; give it extent 1 and any legal stride
  cuuint64_t s1 = (cuuint64_t)stride_outer * 2;
  cuuint64_t s2 = bstride[0] ? (cuuint64_t)bstride[0] * 2 : s1 * ext_outer;
  cuuint64_t s3 = bstride[1] ? (cuuint64_t)bstride[1] * 2 : s2 * bext[0];
  if (!bstride[0]) dims[2] = 1;
  if (!bstride[1]) dims[3] = 1;
  cuuint64_t strides[3] = {s1, s2, s3};
  cuuint32_t box[4] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer, 1, 1};
  return tma_encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B, err);
}

bool tc_gemm_prepare(Launch& L, std::string& err) {
  GemmParams& gp = gp_of(L);
  GemmTcParams& tc = tc_of(L);
  uint16_t* a = reinterpret_cast<uint16_t*>(gp.A.ptr) + gp.A.base;
  uint16_t* b = reinterpret_cast<uint16_t*>(gp.B.ptr) + gp.B.base;
  if (((uintptr_t)a & 15) || ((uintptr_t)b & 15)) { err = "GEMM operand is not 16-byte aligned"; return false; }
  if (!encode(&tc.tmA, a, gp.K, gp.M, gp.A.stride_row, gp.batch_ext, gp.A.batch_stride, TC_BK, TC_BM, err)) return false;
  if (tc.b_kmajor) {
    if (!encode(&tc.tmB, b, gp.K, gp.N, gp.B.stride_col, gp.batch_ext, gp.B.batch_stride, TC_BK, tc.bn, err)) return false;
  } else {
    if (!encode(&tc.tmB, b, gp.N, gp.K, gp.B.stride_row, gp.batch_ext, gp.B.batch_stride, 64, TC_BK, err)) return false;
  }
  return true;
}

struct TcLauncher {
  const Launch& L; cudaStream_t st; int stages;
  template <class SP> void run() {
    static PerDeviceOnce once;       // per instantiation
    if (once.first_use()) cudaFuncSetAttribute(gemm_tc_kernel<SP>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax);
    launch_pdl(gemm_tc_kernel<SP>, L.grid, TC_THREADS, L.smem, st, gp_of(L), tc_of(L), tc_of(L).tmA, tc_of(L).tmB, stages);
  }
};

int tc_gemm_launch(const Launch& L, cudaStream_t st) {
  const GemmTcParams& tc = tc_of(L);
  int stage_bytes = TC_BM * TC_BK * 2 + tc.bn * TC_BK * 2;
  int stages = (int)((L.smem - kSmemFixed) / stage_bytes);
  TcLauncher F{L, st, stages};
  if (!(L.static_id > 0 && StaticSet<EpiStatic>::dispatch(L.static_id, F))) F.run<DynProg>();
  return cudaGetLastError() == cudaSuccess ? 0 : 1;
}

}  // namespace dnnf
