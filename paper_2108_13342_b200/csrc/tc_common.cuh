// Pieces shared by the single-CTA tensor-core kernels (sm_100a): PTX wrappers for mbarriers,
// TMA loads and tcgen05, the shared-memory matrix descriptor, and the epilogue IO that maps
// a warp's 32 x 32 accumulator chunk onto the block's input/output index maps.
//
// Every TMA load in this file is a plain per-CTA load; no clusters are used.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "chain.cuh"
#include "gemm_params.h"

namespace dnnf {

constexpr unsigned long long kWaitLimitNs = 1000000000ull;   // 1 s
constexpr int kStageWords = 32 * 33;                       // per epilogue warp: 32 rows x (32 + 1 pad) words

// ---- PTX wrappers -------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the bound ran out or another role already gave up.
__device__ __forceinline__ unsigned long long wall_ns() { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
// Bounded wait: gives up after kWaitLimitNs of wall-clock time (or as soon as another role of the
// CTA gave up), sets the CTA's abort flag and returns false.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, unsigned long long limit_ns = kWaitLimitNs) {
  if (mbar_try(bar, parity)) return true;
  const unsigned long long t0 = wall_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i) if (mbar_try(bar, parity)) return true;
    if (*abort_flag) return false;
    if (wall_ns() - t0 > limit_ns) { *abort_flag = 1; return false; }
  }
}
__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* tm, uint64_t* bar, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
               ::"r"(smem_u32(dst)), "l"(tm), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
               ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_ld16_issue(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
                 "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
               : "r"(taddr));
}
__device__ __forceinline__ void tc_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
                 "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]),
                 "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]),
                 "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
               : "r"(taddr));
}
__device__ __forceinline__ void tc_ld8_issue(uint32_t taddr, uint32_t (&r)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]) : "r"(taddr));
}
__device__ __forceinline__ void tc_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor (sm_100 format: version 1, 128-byte swizzle).
//  K-major tile  [rows][64 bf16]: rows 128 B apart, 8-row groups 1024 B apart (SBO); LBO unused.
//  MN-major tile [64 k][64 n] blocks: k rows 128 B apart, 8-row groups 1024 B apart (SBO),
//                next 64-wide n block `lbo_bytes` further (LBO).
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= 1ull << 46;          // descriptor version
  d |= 2ull << 61;          // SWIZZLE_128B
  return d;
}

// ---- epilogue IO ------------------------------------------------------------------------------
// After the transpose through shared memory a lane owns, for each of 8 row groups i, four
// consecutive columns of row (lane/8 + 4i) of the warp's 32 x 32 chunk: value index i*4 + v.
// Neighbouring lanes sit on neighbouring columns, so epilogue loads and stores are coalesced
// and all of a chunk's loads are in flight together.
struct TcEpiIO {
  static constexpr int VV = 32;
  const GemmParams& p;
  float accv[32];                                 // the 32 accumulator values of this lane (by value: stays in registers)
  uint32_t row_in[kMaxIn], row_out[kMaxOut];      // offsets of the row this lane owns in TMEM layout (lane = row)
  int m_first;                                    // global row of the warp's first row
  uint32_t n0;                                    // first column of the chunk
  int lane;
  __device__ __forceinline__ uint32_t n_offset(const TensorArg& a, uint32_t n) const {
    if (p.n_nd == 1) return n * (uint32_t)a.stride[0];
    uint32_t off = 0, lin = n;
#pragma unroll
    for (int d = 0; d < 3; ++d) {
      if (d < p.n_nd) {
        uint32_t e = p.it.extent[d];
        uint32_t q = (d == p.n_nd - 1) ? 0u : (__umulhi(lin, p.it.div_m[d]) >> p.it.div_s[d]);
        if (d != p.n_nd - 1 && e == 1) q = lin;
        off += (lin - q * e) * (uint32_t)a.stride[d];
        lin = q;
      }
    }
    return off;
  }
  __device__ __forceinline__ void load(int idx, float (&dst)[VV]) const {
    const TensorArg& a = p.in[idx];
    const uint32_t nn = n0 + (uint32_t)(lane & 7) * 4;
    const uint32_t mine = row_in[idx];
    const bool vec = p.vec_ok && (int)nn + 4 <= p.N;
    const uint32_t noff = vec ? n_offset(a, nn) : 0u;
    if (a.mode == 1) {                          // the same for every row (a bias): load once.
      // (a.mode is uniform over the warp: no lane may leave before the shuffles of the general path)
      float x[4];
      if (vec) {
        if (a.stride[0] == 0) { x[0] = x[1] = x[2] = x[3] = load_scalar<false>(a, mine + noff); }
        else load_vec4<false>(a, mine + noff, x);
      } else {
#pragma unroll
        for (int v = 0; v < 4; ++v) x[v] = ((int)nn + v < p.N) ? load_scalar<false>(a, mine + n_offset(a, nn + v)) : 0.0f;
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) { dst[i * 4] = x[0]; dst[i * 4 + 1] = x[1]; dst[i * 4 + 2] = x[2]; dst[i * 4 + 3] = x[3]; }
      return;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int r = (lane >> 3) + 4 * i;
      const uint32_t ro = __shfl_sync(0xffffffffu, mine, r);
      float* d = &dst[i * 4];
      if (m_first + r >= p.M || (int)nn >= p.N) { d[0] = d[1] = d[2] = d[3] = 0.0f; continue; }
      if (vec) {
        if (a.stride[0] == 0) { float x = load_scalar<false>(a, ro + noff); d[0] = d[1] = d[2] = d[3] = x; }
        else load_vec4<false>(a, ro + noff, d);
      } else {
#pragma unroll
        for (int v = 0; v < 4; ++v) d[v] = ((int)nn + v < p.N) ? load_scalar<false>(a, ro + n_offset(a, nn + v)) : 0.0f;
      }
    }
  }
  __device__ __forceinline__ void anchor(float (&dst)[VV]) const {
#pragma unroll
    for (int v = 0; v < VV; ++v) dst[v] = accv[v];
  }
  __device__ __forceinline__ void store(int idx, const float (&val)[VV]) const {
    const TensorArg& a = p.out[idx];
    const uint32_t nn = n0 + (uint32_t)(lane & 7) * 4;
    const uint32_t mine = row_out[idx];
    const bool vec = p.vec_ok && (int)nn + 4 <= p.N;
    const uint32_t noff = vec ? n_offset(a, nn) : 0u;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int r = (lane >> 3) + 4 * i;
      const uint32_t ro = __shfl_sync(0xffffffffu, mine, r);
      if (m_first + r >= p.M || (int)nn >= p.N) continue;
      if (vec) store_vec4<false>(a, ro + noff, &val[i * 4], false);
      else {
#pragma unroll
        for (int v = 0; v < 4; ++v)
          if ((int)nn + v < p.N) store_scalar<false>(a, ro + n_offset(a, nn + v), val[i * 4 + v], false);
      }
    }
  }
  __device__ __forceinline__ void row_reduce(int, float (&)[VV]) const {}
};

__device__ __forceinline__ uint32_t tc_digits(const GemmParams& p, const TensorArg& a, int first, int count, uint32_t lin) {
  uint32_t off = 0;
  for (int d = first; d < first + count; ++d) {
    const uint32_t e = p.it.extent[d];
    // (multiply-shift division: a run-time divide is some 40 dependent instructions)
    const uint32_t q = (d == first + count - 1) ? 0u : (e == 1 ? lin : (__umulhi(lin, p.it.div_m[d]) >> p.it.div_s[d]));
    off += (lin - q * e) * (uint32_t)a.stride[d];
    lin = q;
  }
  return off;
}

}  // namespace dnnf
