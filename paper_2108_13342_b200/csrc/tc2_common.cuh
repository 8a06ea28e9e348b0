// Pieces shared by the bf16 GEMM kernels that store through TMA (the CTA-pair kernel and the one-tile-per-CTA
// kernel): PTX wrappers, the shared-memory matrix descriptor, the epilogue IO on 32 x 64 bf16 chunk buffers and the
// compile-time epilogue programs.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdlib>

#include "chain.cuh"
#include "gemm_params.h"
#include "ir.h"
#include "tma_host.h"

namespace dnnf {

namespace tc2 {

#ifdef DNNF_TRACE
#define TR(...) __VA_ARGS__
#else
#define TR(...)
#endif
#ifdef DNNF_TRACE
#define T2ACC(slot, v) do { if (blockIdx.x == 0 && p.status) atomicAdd(reinterpret_cast<unsigned long long*>(p.status) + 4 + (slot), (unsigned long long)(v)); } while (0)
#else
#define T2ACC(slot, v) do {} while (0)
#endif

constexpr int BM = 128, BK = 64, EPI_WARPS = 8, THREADS = 64 + 32 * EPI_WARPS;
constexpr unsigned long long kWaitLimitNs = 1000000000ull;   // 1 s
constexpr int kFastPolls = 2048;                             // polls of a barrier before the wall clock is consulted
constexpr int kSmemMax = 227 * 1024;
constexpr int kChunkBytes = 32 * 128;                        // 32 rows x 64 bf16
constexpr int kBiasFloats = 128;                             // per warp, per row-invariant operand
constexpr int kMaxVec = 2;                                   // row-invariant operands staged in shared memory
constexpr int kEpiBytes = EPI_WARPS * (2 * kChunkBytes + kMaxVec * kBiasFloats * 4);
constexpr int kFixed = 1024 + 512 + kEpiBytes;               // alignment slack + barriers + epilogue buffers
constexpr int kRingBudget = kSmemMax - kFixed;


__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t cluster_rank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t mapa(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// arrive on a barrier that lives in another CTA of the cluster (address from mapa)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long wall_ns() { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
// Bounded wait: gives up after kWaitLimitNs of wall-clock time (or as soon as another role of the
// CTA gave up), sets the CTA's abort flag and returns false.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try(bar, parity)) return true;
  // Fast phase: the common case is a wait of well under a microsecond.  Reading the global timer costs about as much
  // as a whole pipeline step of the issuing threads, so the clock is consulted only after this many polls.
#pragma unroll 1
  for (int i = 0; i < kFastPolls; ++i) if (mbar_try(bar, parity)) return true;
  const unsigned long long t0 = wall_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i) if (mbar_try(bar, parity)) return true;
    if (*abort_flag) return false;
    if (wall_ns() - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
  }
}
// Operand load of a CTA pair: the bytes land in THIS CTA's shared memory, the completion is
// counted on the LEADER's barrier (cluster address), so the MMA thread waits on one barrier only.
__device__ __forceinline__ void tma_load_2d_pair(void* dst, const CUtensorMap* tm, uint32_t leader_bar, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(smem_u32(dst)), "l"(tm), "r"(leader_bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* tm, uint64_t* bar, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(smem_u32(dst)), "l"(tm), "r"(smem_u32(bar)), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tm, const void* src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(tm), "r"(smem_u32(src)), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// completion of all MMAs issued so far arrives on one barrier, given by its cluster address
__device__ __forceinline__ void tc_commit2(uint32_t cluster_addr) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(cluster_addr) : "memory");
}
// the same completion delivered to the barrier at the same shared-memory offset in both CTAs of the pair (ranks 0 and 1)
__device__ __forceinline__ void tc_commit2_both(uint32_t local_addr) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(local_addr), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void tc_mma2(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
               ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
                 "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]),
                 "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]),
                 "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
               : "r"(taddr));
}
__device__ __forceinline__ void tc_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= 1ull << 46;
  d |= 2ull << 61;          // SWIZZLE_128B
  return d;
}

// Epilogue IO on 32 consecutive columns of the thread's own row (TMEM layout: lane = row).
// Chunk buffer: 32 rows x 128 B, 128-byte swizzle: the 16-byte piece j of row r sits at
// r*128 + ((j ^ (r & 7)) * 16).
struct EpiIO {
  static constexpr int VV = 32;
  const GemmParams& p;
  float accv[32];
  uint8_t* chunk;            // this warp's current chunk buffer
  const float* vec_s;        // staged row-invariant operands: [kMaxVec][kBiasFloats]
  int lane;
  int col_in_chunk;          // 0 or 32: which half of the 64-column chunk
  int col_in_half;           // column offset inside this warp's half of the tile (for vec_s)
  int c_input;
  __device__ __forceinline__ void load(int idx, float (&dst)[VV]) const {
    const TensorArg& a = p.in[idx];
    if (idx == c_input) {                      // full-tile operand, prefetched by TMA into the chunk buffer
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int piece = (col_in_chunk >> 3) + j;
        uint4 w = *reinterpret_cast<const uint4*>(chunk + lane * 128 + ((piece ^ (lane & 7)) << 4));
        float* d = &dst[8 * j];
        d[0] = __uint_as_float(w.x << 16); d[1] = __uint_as_float(w.x & 0xffff0000u);
        d[2] = __uint_as_float(w.y << 16); d[3] = __uint_as_float(w.y & 0xffff0000u);
        d[4] = __uint_as_float(w.z << 16); d[5] = __uint_as_float(w.z & 0xffff0000u);
        d[6] = __uint_as_float(w.w << 16); d[7] = __uint_as_float(w.w & 0xffff0000u);
      }
      return;
    }
    // row-invariant operand from shared memory (every lane reads the same words: broadcast)
    const float* s = vec_s + a.mode * kBiasFloats + col_in_half;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      float4 w = *reinterpret_cast<const float4*>(s + 4 * j);
      dst[4 * j] = w.x; dst[4 * j + 1] = w.y; dst[4 * j + 2] = w.z; dst[4 * j + 3] = w.w;
    }
  }
  __device__ __forceinline__ void anchor(float (&dst)[VV]) const {
#pragma unroll
    for (int v = 0; v < VV; ++v) dst[v] = accv[v];
  }
  __device__ __forceinline__ void store(int, const float (&val)[VV]) const {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int piece = (col_in_chunk >> 3) + j;
      __nv_bfloat162 a0 = __floats2bfloat162_rn(val[8 * j], val[8 * j + 1]), a1 = __floats2bfloat162_rn(val[8 * j + 2], val[8 * j + 3]);
      __nv_bfloat162 a2 = __floats2bfloat162_rn(val[8 * j + 4], val[8 * j + 5]), a3 = __floats2bfloat162_rn(val[8 * j + 6], val[8 * j + 7]);
      uint4 w = make_uint4(*reinterpret_cast<uint32_t*>(&a0), *reinterpret_cast<uint32_t*>(&a1), *reinterpret_cast<uint32_t*>(&a2),
                           *reinterpret_cast<uint32_t*>(&a3));
      *reinterpret_cast<uint4*>(chunk + lane * 128 + ((piece ^ (lane & 7)) << 4)) = w;
    }
  }
  __device__ __forceinline__ void row_reduce(int, float (&)[VV]) const {}
};


}  // namespace tc2

// ---- static epilogue programs (same tables as the single-CTA kernel) -------------------------------
#define MO(o, s, i) MicroOp{o, s, i, 0}
DNNF_SP_BEGIN(E2_Store, 2) MO(M_MOV, S_ANCHOR, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(E2_Bias, 3) MO(M_MOV, S_ANCHOR, 0), MO(M_ADD, S_IN, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(E2_BiasGeluTanh, 4) MO(M_MOV, S_ANCHOR, 0), MO(M_ADD, S_IN, 0), MO(M_GELU_TANH, S_NONE, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(E2_BiasResidual, 4) MO(M_MOV, S_ANCHOR, 0), MO(M_ADD, S_IN, 0), MO(M_ADD, S_IN, 1), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(E2_BiasGeluPrimitives, 9)
  MO(M_MOV, S_ANCHOR, 0), MO(M_ADD, S_IN, 0), MO(M_SAVE, S_TMP, 0), MO(M_MUL, S_CONST, 0), MO(M_ERF, S_NONE, 0), MO(M_ADD, S_CONST, 1),
  MO(M_MUL, S_TMP, 0), MO(M_MUL, S_CONST, 2), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(E2_BiasGeluTanhPrimitives, 13)
  MO(M_MOV, S_ANCHOR, 0), MO(M_ADD, S_IN, 0), MO(M_SAVE, S_TMP, 0), MO(M_SQUARE, S_NONE, 0), MO(M_MUL, S_TMP, 0), MO(M_MUL, S_CONST, 0),
  MO(M_ADD, S_TMP, 0), MO(M_MUL, S_CONST, 1), MO(M_TANH, S_NONE, 0), MO(M_ADD, S_CONST, 2), MO(M_MUL, S_TMP, 0), MO(M_MUL, S_CONST, 3),
  MO(M_STORE, S_NONE, 0) DNNF_SP_END
#undef MO
using Epi2Static = TypeList<E2_Store, E2_Bias, E2_BiasGeluTanh, E2_BiasResidual, E2_BiasGeluPrimitives, E2_BiasGeluTanhPrimitives>;


}  // namespace dnnf
