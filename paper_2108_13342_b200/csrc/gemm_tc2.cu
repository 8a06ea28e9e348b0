// Tensor-core GEMM-anchored blocks, CTA-pair version (sm_100a).
//
// Two CTAs on neighbouring SMs form a cluster and compute one 256 x BN tile with
// tcgen05.mma.cta_group::2: each CTA loads its own 128 rows of A and only HALF of the B
// tile, so per-SM L2->shared-memory traffic and shared-memory read traffic per flop drop
// by a third against the single-CTA kernel, which is bound by exactly those.  Each CTA's
// tensor memory receives its own 128 accumulator rows.
//
// Epilogue, per warp on a 32-row x 64-column chunk: tcgen05.ld -> registers -> the block's
// micro-op program -> bf16 -> swizzled shared memory -> TMA store.  A full-tile epilogue
// operand (a residual) is prefetched by TMA into the same shared-memory chunk buffer while
// the main loop still runs, and is overwritten in place by the result; row-invariant operands
// (a bias) are staged once per tile.  No per-element index arithmetic, no shuffles.
//
// Both CTAs' operand loads count their bytes on the leader's barrier (cta_group::2 form of the
// TMA load, single destination); stage release and accumulator hand-over use single-target
// tcgen05.commit / mbarrier arrives on cluster shared-memory addresses.
// Split-K (few output tiles, long K): `ksplit` CTA pairs each accumulate a slice of K for the same tile.  Per
// 32 x 64 chunk a warp writes its partial accumulators to scratch and bumps the chunk's counter; the warp whose
// bump is the last adds the other partials to its own (L2 reads), runs the epilogue program and stores.
// Nobody waits for anybody, and the last warp puts the counter back to zero.
// Every wait is bounded; on expiry the CTA pair records DNNF_ERR_TIMEOUT, stops and releases
// tensor memory.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdlib>
#include <mutex>

#include "chain.cuh"
#include "gemm_params.h"
#include "ir.h"
#include "tma_host.h"

namespace dnnf {

namespace tc2 {

#ifdef DNNF_TRACE
#define T2ACC(slot, v) do { if (blockIdx.x == 0 && p.status) atomicAdd(reinterpret_cast<unsigned long long*>(p.status) + 4 + (slot), (unsigned long long)(v)); } while (0)
#else
#define T2ACC(slot, v) do {} while (0)
#endif

constexpr int BM = 128, BK = 64, EPI_WARPS = 8, THREADS = 64 + 32 * EPI_WARPS;
constexpr unsigned long long kWaitLimitNs = 1000000000ull;   // 1 s
constexpr int kSmemMax = 227 * 1024;
constexpr int kChunkBytes = 32 * 128;                        // 32 rows x 64 bf16
constexpr int kBiasFloats = 128;                             // per warp, per row-invariant operand
constexpr int kMaxVec = 2;                                   // row-invariant operands staged in shared memory
constexpr int kEpiBytes = EPI_WARPS * (2 * kChunkBytes + kMaxVec * kBiasFloats * 4);
constexpr int kFixed = 1024 + 512 + kEpiBytes;               // alignment slack + barriers + epilogue buffers
constexpr int kRingBudget = kSmemMax - kFixed;

struct Params {
  CUtensorMap tmA, tmB, tmD, tmC;
  int32_t b_kmajor, k_tiles, bn, total_tiles, tiles_n;
  int32_t c_input;           // index of the epilogue input that is a full tile (TMA-loaded), or -1
  int32_t stages;
  int32_t kpack;             // 64-wide k-tiles per ring stage (1 or 2): one wait, one pair of commits per stage
  int32_t ksplit;            // CTA pairs that share one output tile, each with kt_per k-tiles of the K range (1: no split)
  int32_t kt_per;
  FastDiv fd_tiles, fd_tiles_n;   // item -> (K slice, tile), tile -> (tile row, tile column)
  float* scratch;            // split-K partial accumulators: [unit][ksplit][64 cols][32 rows] fp32
  int32_t* counters;         // split-K arrival counters, one per unit (a warp's 32 x 64 chunk); zero between runs
};

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

template <class SP>
__global__ void __launch_bounds__(THREADS, 1)
gemm_tc2_kernel(const __grid_constant__ GemmParams p, const __grid_constant__ Params q) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int BN = q.bn, HB = BN / 2, stages = q.stages, kpack = q.kpack;
  const uint32_t a_bytes = BM * BK * 2, b_bytes = (uint32_t)HB * BK * 2, sub_bytes = a_bytes + b_bytes, stage_bytes = sub_bytes * (uint32_t)kpack;
  uint8_t* epi = smem + (size_t)stages * stage_bytes;                  // 1024-aligned (stage_bytes is a multiple of 1024)
  uint64_t* bars = reinterpret_cast<uint64_t*>(epi + kEpiBytes);
  uint64_t* full_bar = bars;                  // [stages]  used in the leader only: 1 arrival + the bytes of BOTH CTAs
  uint64_t* empty_bar = full_bar + 8;         // [stages]  1 arrival (commit from the leader)
  uint64_t* tfull_bar = empty_bar + 8;        // [2]       1 arrival (commit from the leader)
  uint64_t* tempty_bar = tfull_bar + 2;       // [2]       leader only: 2 * EPI_WARPS arrivals
  uint64_t* c_bar = tempty_bar + 2;           // [EPI_WARPS][2] residual chunk landed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(c_bar + 2 * EPI_WARPS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();
  const bool leader = rank == 0;
  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(&tfull_bar[s], 1); mbar_init(&tempty_bar[s], 2 * EPI_WARPS); }
    for (int s = 0; s < 2 * EPI_WARPS; ++s) mbar_init(&c_bar[s], 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync();                              // both CTAs: barriers initialised, tensor memory allocated
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();
  const long long t_begin = clock64();

  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int n_tiles = q.total_tiles, k_tiles = q.k_tiles, tiles_n = q.tiles_n;
  const int total = n_tiles * q.ksplit;        // work items: (tile, K slice); item = slice * n_tiles + tile

  if (warp == 0) {
    if (lane == 0) {
      // ---------------- TMA producer (both CTAs): own 128 rows of A, own half of B ----------------
      // (stage index and phase advance by increments: a division by the run-time stage count costs this
      // single thread some 200 cycles of dependent instructions per k-tile)
      int s = 0; uint32_t ph = 0;
      bool ok = true;
      for (int item = pair; item < total && ok; item += n_pairs) {
        const int ks = (int)fd_div((uint32_t)item, q.fd_tiles), tile = item - ks * n_tiles;
        const int tm = (int)fd_div((uint32_t)tile, q.fd_tiles_n), tn = tile - tm * tiles_n;
        const int m0 = tm * 256 + (int)rank * BM, n0 = tn * BN + (int)rank * HB;
        const int kt_end = min(k_tiles, (ks + 1) * q.kt_per);
        for (int kt = ks * q.kt_per; kt < kt_end; kt += kpack) {
          { long long t0 = clock64(); if (!mbar_wait(&empty_bar[s], ph ^ 1, abort_flag)) { ok = false; break; } T2ACC(0, clock64() - t0); }
          const uint32_t lbar = mapa(smem_u32(&full_bar[s]), 0);
          if (leader) mbar_expect_tx(&full_bar[s], 2 * stage_bytes);
          // (a k-tile past K, when k_tiles is odd and kpack is 2, arrives as zeros: its MMAs add nothing)
          for (int u = 0; u < kpack; ++u) {
            uint8_t* sa = smem + (size_t)s * stage_bytes + (size_t)u * sub_bytes;
            uint8_t* sb = sa + a_bytes;
            const int k0 = (kt + u) * BK;
            tma_load_2d_pair(sa, &q.tmA, lbar, k0, m0);
            if (q.b_kmajor) {
              tma_load_2d_pair(sb, &q.tmB, lbar, k0, n0);
            } else {
              for (int j = 0; j < HB / 64; ++j) tma_load_2d_pair(sb + j * (64 * BK * 2), &q.tmB, lbar, n0 + j * 64, k0);
            }
          }
          if (++s == stages) { s = 0; ph ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      if (leader) {
        // ---------------- MMA issuer (leader CTA only) ----------------
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((q.b_kmajor ? 0u : 1u) << 16) | ((uint32_t)(BN >> 3) << 17) |
                               ((uint32_t)(256 >> 4) << 24);
        uint32_t tcount = 0;
        int s = 0; uint32_t ph = 0;
        bool ok = true;
        // descriptors of stage 0; a stage further on adds stage_bytes / 16 to the address field, a k-step 2 (32 bytes)
        // or, for an MN-major B, 128 (2048 bytes); the barriers' cluster addresses are 8 bytes apart
        const uint64_t da0 = make_desc(smem_u32(smem), 16, 1024);
        const uint64_t db0 = q.b_kmajor ? make_desc(smem_u32(smem) + a_bytes, 16, 1024) : make_desc(smem_u32(smem) + a_bytes, 64 * BK * 2, 1024);
        const uint64_t dstage = stage_bytes >> 4, dsub = sub_bytes >> 4, dbk = q.b_kmajor ? 2 : 128;
        const uint32_t e0 = mapa(smem_u32(&empty_bar[0]), 0), e1 = mapa(smem_u32(&empty_bar[0]), 1);
        uint64_t da_s = da0, db_s = db0;
        for (int item = pair; item < total && ok; item += n_pairs, ++tcount) {
          const int acc = tcount & 1;
          const uint32_t aph = (tcount >> 1) & 1;
          { long long t0 = clock64(); if (!mbar_wait(&tempty_bar[acc], aph ^ 1, abort_flag)) { ok = false; break; } T2ACC(1, clock64() - t0); }
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
          const int ks = (int)fd_div((uint32_t)item, q.fd_tiles);
          const int kt_begin = ks * q.kt_per, kt_end = min(k_tiles, kt_begin + q.kt_per);
          for (int kt = kt_begin; kt < kt_end; kt += kpack) {
            { long long t0 = clock64(); if (!mbar_wait(&full_bar[s], ph, abort_flag)) { ok = false; break; } T2ACC(2, clock64() - t0); T2ACC(3, 1); }
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < BK / 16; ++kk)
              tc_mma2(d_tmem, da_s + 2 * kk, db_s + dbk * kk, idesc, ((kt - kt_begin) | kk) ? 1u : 0u);
            if (kpack == 2) {
#pragma unroll
              for (int kk = 0; kk < BK / 16; ++kk)
                tc_mma2(d_tmem, da_s + dsub + 2 * kk, db_s + dsub + dbk * kk, idesc, 1u);
            }
            // stage free in both CTAs once these MMAs have read it.  (Relaying the peer's signal through a helper
            // warp instead of a second commit was measured: the extra hop starves the peer's producer, 40 % slower.)
            tc_commit2(e0 + 8u * (uint32_t)s);
            tc_commit2(e1 + 8u * (uint32_t)s);
            da_s += dstage; db_s += dstage;
            if (++s == stages) { s = 0; ph ^= 1; da_s = da0; db_s = db0; }
          }
          if (ok) { tc_commit2(mapa(smem_u32(&tfull_bar[acc]), 0)); tc_commit2(mapa(smem_u32(&tfull_bar[acc]), 1)); }
        }
      }
    }
  } else {
    // ---------------- epilogue warps (both CTAs) ----------------
    const int ew = warp - 2, sub = warp & 3, half = ew >> 2;
    uint8_t* cbuf = epi + ew * (2 * kChunkBytes);
    float* vec_s = reinterpret_cast<float*>(epi + EPI_WARPS * 2 * kChunkBytes) + ew * (kMaxVec * kBiasFloats);
    uint64_t* my_cbar = c_bar + 2 * ew;
    const int chunks = HB / 64 > 0 ? HB / 64 : 1;                  // 64-column chunks per warp per tile
    const int cols_per_warp = HB;                                   // this warp's share of the tile's columns
    EpiIO io{p};
    io.lane = lane; io.c_input = q.c_input; io.vec_s = vec_s;
    uint32_t tcount = 0, ccount = 0;                                // tiles and chunks processed by this warp
    bool ok = true;
    // prefetch of the residual chunk `g` (global chunk counter of this warp) into buffer g & 1
    auto prefetch = [&](int item, int c, uint32_t g) {
      if (q.c_input < 0 || lane != 0) return;
      const int tile = item - (int)fd_div((uint32_t)item, q.fd_tiles) * n_tiles;
      const int tm = (int)fd_div((uint32_t)tile, q.fd_tiles_n), tn = tile - tm * tiles_n;
      const int m0 = tm * 256 + (int)rank * BM + sub * 32, n0 = tn * BN + half * cols_per_warp + c * 64;
      mbar_expect_tx(&my_cbar[g & 1], kChunkBytes);
      tma_load_2d(cbuf + (g & 1) * kChunkBytes, &q.tmC, &my_cbar[g & 1], n0, m0);
    };
    const int S = q.ksplit;
    if (pair < total) prefetch(pair, 0, 0);
    for (int item = pair; item < total && ok; item += n_pairs, ++tcount) {
      const int ks = (int)fd_div((uint32_t)item, q.fd_tiles), tile = item - ks * n_tiles;
      const int tm = (int)fd_div((uint32_t)tile, q.fd_tiles_n), tn = tile - tm * tiles_n;
      const int m0 = tm * 256 + (int)rank * BM + sub * 32;
      const int nw0 = tn * BN + half * cols_per_warp;
      // stage this tile's row-invariant operands (this warp's columns)
      for (int k = 0; k < p.n_in; ++k) {
        const TensorArg& a = p.in[k];
        if (k == q.c_input) continue;
        for (int c = lane; c < cols_per_warp; c += 32) {
          const int n = nw0 + c;
          vec_s[a.mode * kBiasFloats + c] = n < p.N ? load_scalar<false>(a, (uint32_t)a.base + (uint32_t)n * (uint32_t)a.stride[0]) : 0.0f;
        }
      }
      __syncwarp();
      const int acc = tcount & 1;
      const uint32_t aph = (tcount >> 1) & 1;
      { long long t0 = clock64(); if (!mbar_wait(&tfull_bar[acc], aph, abort_flag)) { ok = false; break; } if (warp == 2 && lane == 0) T2ACC(4, clock64() - t0); }
      tc_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(sub * 32) << 16) + (uint32_t)(acc * BN + half * cols_per_warp);
      for (int c = 0; c < chunks && ok; ++c, ++ccount) {
        const int buf = ccount & 1;
        io.chunk = cbuf + buf * kChunkBytes;
        // This chunk's buffer is free once the store issued from it two chunks ago has been read out: one store
        // may stay in flight.  With a residual operand the OTHER buffer is about to be overwritten by the prefetch
        // below, so the store issued from it one chunk ago has to be read out as well.
#ifdef DNNF_TRACE
        const long long tw0 = clock64();
#endif
        if (lane == 0) { if (q.c_input >= 0) tma_store_wait_read(); else tma_store_wait_read1(); }
        __syncwarp();
#ifdef DNNF_TRACE
        if (warp == 2 && lane == 0) T2ACC(9, clock64() - tw0);
#endif
        {   // prefetch the next residual chunk (possibly of the next item) into the other buffer
          int nt = item, nc = c + 1;
          if (nc == chunks) { nt = item + n_pairs; nc = 0; }
          if (nt < total) prefetch(nt, nc, ccount + 1);
        }
        if (q.c_input >= 0) { if (!mbar_wait(&my_cbar[buf], (ccount >> 1) & 1, abort_flag)) { ok = false; break; } }
        // ---- split-K: hand in this slice's partial chunk; only the last slice to arrive carries on ----
        const float* others = nullptr;
        if (S > 1) {
          const uint32_t unit = (((uint32_t)tile * 2u + rank) * EPI_WARPS + (uint32_t)ew) * (uint32_t)chunks + (uint32_t)c;
          float* mine = q.scratch + ((size_t)unit * S + ks) * 2048;
#pragma unroll 1
          for (int h = 0; h < 2; ++h) {
            uint32_t raw[32];
            tc_ld32(t_row + c * 64 + h * 32, raw);
            tc_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) mine[(h * 32 + i) * 32 + lane] = __uint_as_float(raw[i]);     // a 128-byte line per instruction
          }
          __threadfence();                       // this lane's partials are visible before the counter moves
          __syncwarp();
          int old = 0;
          if (lane == 0) old = atomicAdd(&q.counters[unit], 1);
          old = __shfl_sync(0xffffffffu, old, 0);
          if (old != S - 1) continue;            // somebody else finishes this chunk (uniform over the warp)
          if (lane == 0) q.counters[unit] = 0;   // all S slices have arrived: ready for the next run
          __threadfence();
          others = q.scratch + (size_t)unit * S * 2048;
        }
#pragma unroll 1
        for (int h = 0; h < 2; ++h) {
          uint32_t raw[32];
#ifdef DNNF_TRACE
          const long long tl0 = clock64();
#endif
          tc_ld32(t_row + c * 64 + h * 32, raw);
          tc_ld_wait();
#ifdef DNNF_TRACE
          const long long tl1 = clock64();
          if (warp == 2 && lane == 0) T2ACC(6, tl1 - tl0);
#endif
#pragma unroll
          for (int i = 0; i < 32; ++i) io.accv[i] = __uint_as_float(raw[i]);
          if (others) {
            for (int s2 = 0; s2 < S; ++s2) {
              if (s2 == ks) continue;
              const float* o = others + (size_t)s2 * 2048 + (h * 32) * 32 + lane;
#pragma unroll
              for (int i = 0; i < 32; ++i) io.accv[i] += __ldcg(o + i * 32);       // written by another SM: read from L2
            }
          }
          io.col_in_chunk = h * 32;
          io.col_in_half = c * 64 + h * 32;
          run_program<32, SP, true>(p.prog, io);
#ifdef DNNF_TRACE
          if (warp == 2 && lane == 0) T2ACC(7, clock64() - tl1);
#endif
        }
#ifdef DNNF_TRACE
        const long long ts0 = clock64();
#endif
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_2d(&q.tmD, io.chunk, nw0 + c * 64, m0);
          tma_store_commit();
        }
#ifdef DNNF_TRACE
        if (warp == 2 && lane == 0) T2ACC(8, clock64() - ts0);
#endif
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mapa(smem_u32(&tempty_bar[acc]), 0));   // accumulator drained (leader counts both CTAs)
    }
    if (lane == 0) tma_store_wait_all();
  }

  // ---------------- teardown ----------------
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) T2ACC(5, clock64() - t_begin);
  cluster_sync();                              // the peer may still be signalling our barriers / reading our shared memory
  if (*abort_flag) {
    if (threadIdx.x == 0 && p.status) { atomicExch(&p.status[0], DNNF_ERR_TIMEOUT); atomicExch(&p.status[1], p.block_index); }
    if (threadIdx.x == 0) { long long t0 = clock64(); while (clock64() - t0 < 2000000) {} }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

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

// ---- host side --------------------------------------------------------------------------------------
static GemmParams& gp_of(Launch& L) { return *reinterpret_cast<GemmParams*>(L.blob.data()); }
static const GemmParams& gp_of(const Launch& L) { return *reinterpret_cast<const GemmParams*>(L.blob.data()); }
static tc2::Params& t2_of(Launch& L) { return *reinterpret_cast<tc2::Params*>(L.blob.data() + sizeof(GemmParams) + sizeof(GemmTcParams)); }
static const tc2::Params& t2_of(const Launch& L) { return *reinterpret_cast<const tc2::Params*>(L.blob.data() + sizeof(GemmParams) + sizeof(GemmTcParams)); }

size_t tc2_blob_bytes() { return sizeof(tc2::Params); }

bool tc_gemm_eligible(const GemmParams& gp);

// The pair kernel takes plain 2-D problems whose epilogue operands and result are row-major
// matrices over (m, n): one bf16 output, at most one bf16 full-tile input, row-invariant others.
bool tc2_gemm_eligible(const GemmParams& gp) {
  if (getenv("DNNF_NO_PAIR_GEMM")) return false;
  if (!tc_gemm_eligible(gp)) return false;
  if (gp.batch_ext[0] * gp.batch_ext[1] != 1) return false;
  if (gp.M < 256 || gp.N < 128) return false;
  if (gp.n_nd != 1 || gp.m_nd != 1 || gp.n_out != 1 || !gp.vec_ok) return false;
  const TensorArg& o = gp.out[0];
  if (o.dtype != DNNF_BF16 || o.stride[0] != 1 || o.stride[1] % 8 || o.base % 8 || o.stride[1] <= 0) return false;
  int full = 0, vec = 0;
  for (int i = 0; i < gp.n_in; ++i) {
    const TensorArg& a = gp.in[i];
    if (a.mode == 1) { if (a.stride[0] != 1) return false; vec++; }
    else { if (a.dtype != DNNF_BF16 || a.stride[0] != 1 || a.stride[1] % 8 || a.base % 8 || a.stride[1] <= 0) return false; full++; }
  }
  if (full > 1 || vec > tc2::kMaxVec) return false;
  const bool b_n = gp.B.stride_col == 1 && !(gp.B.stride_row == 1 && gp.K == 1);
  (void)b_n;
  return true;
}

void tc2_gemm_plan(Launch& L) {
  GemmParams& gp = gp_of(L);
  tc2::Params& q = t2_of(L);
  q.b_kmajor = (gp.B.stride_col != 1) ? 1 : 0;
  q.k_tiles = (gp.K + tc2::BK - 1) / tc2::BK;
  const int tiles_m = (gp.M + 255) / 256;
  int best_bn = 128; double best = -1;
  for (int bn : {256, 128}) {
    if (bn / 2 >= gp.N && bn > 128) continue;
    int tiles = tiles_m * ((gp.N + bn - 1) / bn);
    int waves = (tiles + 73) / 74;
    double useful = (double)gp.N / (((gp.N + bn - 1) / bn) * bn);
    double eff = (double)tiles / (waves * 74.0) * useful;
    if (eff > best + 1e-9) { best = eff; best_bn = bn; }
  }
  if (getenv("DNNF_PAIR_BN")) best_bn = atoi(getenv("DNNF_PAIR_BN"));      // development switch
  q.bn = best_bn;
  q.tiles_n = (gp.N + q.bn - 1) / q.bn;
  q.total_tiles = tiles_m * q.tiles_n;
  q.fd_tiles = make_fastdiv((uint32_t)q.total_tiles);
  q.fd_tiles_n = make_fastdiv((uint32_t)q.tiles_n);
  gp.tiles_m = tiles_m; gp.tiles_n = q.tiles_n;
  const int sub_bytes = tc2::BM * tc2::BK * 2 + (q.bn / 2) * tc2::BK * 2;
  // two k-tiles per stage halve the issuing thread's per-stage cost (wait, fence, two commits); worth it when its
  // MMAs are short (BN = 128) or the k loop is long, as long as three stages still fit
  q.kpack = (q.k_tiles >= 4 && tc2::kRingBudget / (2 * sub_bytes) >= 3) ? 2 : 1;
  if (getenv("DNNF_PAIR_KPACK")) q.kpack = atoi(getenv("DNNF_PAIR_KPACK")) == 2 ? 2 : 1;
  const int stage_bytes = sub_bytes * q.kpack;
  q.stages = std::min(8, tc2::kRingBudget / stage_bytes);
  // split-K when fewer than half of the 74 CTA pairs would have a tile and the k loop is long.  Handing partial
  // tiles over through L2 costs about 3 us (measured), a k-tile about 0.22 us: it pays from 32 k-tiles up, with
  // two or three slices (1024 x 768 x 3072: 15.7 -> 13.2 us; 1024 x 768 x 768: 7.2 -> 9.2 us, so not there).
  q.ksplit = 1; q.kt_per = q.k_tiles;
  if (q.total_tiles * 2 <= 74 && q.k_tiles >= 32 && !getenv("DNNF_NO_SPLIT_K")) {
    int want = std::min(3, 74 / q.total_tiles);
    if (getenv("DNNF_SPLIT_K")) want = std::max(1, std::min(8, atoi(getenv("DNNF_SPLIT_K"))));
    if (want > 1) {
      int per = (q.k_tiles + want - 1) / want;
      per = (per + q.kpack - 1) / q.kpack * q.kpack;
      q.kt_per = per;
      q.ksplit = (q.k_tiles + per - 1) / per;
    }
  }
  if (q.ksplit > 1) {
    const int64_t units = (int64_t)q.total_tiles * 2 * tc2::EPI_WARPS * std::max(1, q.bn / 2 / 64);
    L.counter_bytes = units * 4;
    L.scratch_bytes = units * q.ksplit * 2048 * 4;
  } else {
    L.counter_bytes = L.scratch_bytes = 0;
  }
  q.c_input = -1;
  int vec_slot = 0;
  for (int i = 0; i < gp.n_in; ++i) {
    if (gp.in[i].mode == 1) gp.in[i].mode = vec_slot++;      // from here on: slot in the staged-vector area
    else { q.c_input = i; gp.in[i].mode = 0; }
  }
  L.grid = 2 * std::min(q.total_tiles * q.ksplit, 74);
  L.threads = tc2::THREADS;
  L.smem = (size_t)q.stages * stage_bytes + tc2::kFixed;
  L.variant = 3;
  L.static_id = StaticSet<Epi2Static>::find(gp.prog);
}

static bool encode2d(CUtensorMap* tm, void* base, int64_t ext_inner, int64_t ext_outer, int64_t stride_outer_elems, int box_inner, int box_outer,
                     std::string& err) {
  cuuint64_t dims[2] = {(cuuint64_t)ext_inner, (cuuint64_t)ext_outer};
  cuuint64_t strides[1] = {(cuuint64_t)stride_outer_elems * 2};
  cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
  return tma_encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B, err);
}

bool tc2_gemm_prepare(Launch& L, std::string& err) {
  GemmParams& gp = gp_of(L);
  tc2::Params& q = t2_of(L);
  uint16_t* a = reinterpret_cast<uint16_t*>(gp.A.ptr) + gp.A.base;
  uint16_t* b = reinterpret_cast<uint16_t*>(gp.B.ptr) + gp.B.base;
  uint16_t* d = reinterpret_cast<uint16_t*>(gp.out[0].ptr) + gp.out[0].base;
  if (((uintptr_t)a & 15) || ((uintptr_t)b & 15) || ((uintptr_t)d & 15)) { err = "GEMM operand is not 16-byte aligned"; return false; }
  if (!encode2d(&q.tmA, a, gp.K, gp.M, gp.A.stride_row, tc2::BK, tc2::BM, err)) return false;
  if (q.b_kmajor) { if (!encode2d(&q.tmB, b, gp.K, gp.N, gp.B.stride_col, tc2::BK, q.bn / 2, err)) return false; }
  else { if (!encode2d(&q.tmB, b, gp.N, gp.K, gp.B.stride_row, 64, tc2::BK, err)) return false; }
  if (!encode2d(&q.tmD, d, gp.N, gp.M, gp.out[0].stride[1], 64, 32, err)) return false;
  if (q.c_input >= 0) {
    const TensorArg& c = gp.in[q.c_input];
    uint16_t* cp = reinterpret_cast<uint16_t*>(c.ptr) + c.base;
    if ((uintptr_t)cp & 15) { err = "epilogue operand is not 16-byte aligned"; return false; }
    if (!encode2d(&q.tmC, cp, gp.N, gp.M, c.stride[1], 64, 32, err)) return false;
  } else {
    q.tmC = q.tmD;
  }
  return true;
}

struct Tc2Launcher {
  const Launch& L; cudaStream_t st; cudaError_t rc;
  template <class SP> void run() {
    static PerDeviceOnce once;       // per instantiation
    if (once.first_use()) cudaFuncSetAttribute(tc2::gemm_tc2_kernel<SP>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc2::kSmemMax);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(L.grid); cfg.blockDim = dim3(tc2::THREADS); cfg.dynamicSmemBytes = L.smem; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 2;
    rc = cudaLaunchKernelEx(&cfg, tc2::gemm_tc2_kernel<SP>, gp_of(L), t2_of(L));
  }
};

// split-K scratch and counters live in the bound workspace at the offsets the planner chose
void tc2_set_scratch(Launch& L, void* ws_base) {
  tc2::Params& q = t2_of(L);
  q.scratch = L.scratch_off >= 0 ? reinterpret_cast<float*>(reinterpret_cast<char*>(ws_base) + L.scratch_off) : nullptr;
  q.counters = L.counter_off >= 0 ? reinterpret_cast<int32_t*>(reinterpret_cast<char*>(ws_base) + L.counter_off) : nullptr;
}

int tc2_gemm_launch(const Launch& L, cudaStream_t st) {
  Tc2Launcher F{L, st, cudaSuccess};
  if (!(L.static_id > 0 && StaticSet<Epi2Static>::dispatch(L.static_id, F))) F.run<DynProg>();
  return (F.rc == cudaSuccess && cudaGetLastError() == cudaSuccess) ? 0 : 1;
}

}  // namespace dnnf
