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

#include "ir.h"
#include "tc2_common.cuh"
#include "tma_host.h"

namespace dnnf {

namespace tc2 {

constexpr int kProducer2 = 2 + EPI_WARPS;       // the second producer warp sits behind the epilogue warps
constexpr int kThreads2 = THREADS + 32;

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

template <class SP>
__global__ void __launch_bounds__(kThreads2, 1)
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

  if (warp == 0 || warp == kProducer2) {
    if (lane == 0) {
      // ---------------- TMA producers (both CTAs): own 128 rows of A, own half of B ----------------
      // Two producer threads take alternate ring stages: a stage costs its producer a wait, an expect and three or four
      // TMA requests at 50 to 80 ns each, more than the MMA thread spends on it.
      // (stage index and phase advance by increments: a division by the run-time stage count costs this
      // single thread some 200 cycles of dependent instructions per k-tile)
      const uint32_t mine = warp == 0 ? 0u : 1u;
      uint32_t turn = 0;
      int s = 0; uint32_t ph = 0;
      bool ok = true;
      for (int item = pair; item < total && ok; item += n_pairs) {
        const int ks = (int)fd_div((uint32_t)item, q.fd_tiles), tile = item - ks * n_tiles;
        const int tm = (int)fd_div((uint32_t)tile, q.fd_tiles_n), tn = tile - tm * tiles_n;
        const int m0 = tm * 256 + (int)rank * BM, n0 = tn * BN + (int)rank * HB;
        const int kt_end = min(k_tiles, (ks + 1) * q.kt_per);
        for (int kt = ks * q.kt_per; kt < kt_end; kt += kpack, turn ^= 1u) {
          if (turn == mine) {
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
        TR(long long r_tempty = 0, r_wait = 0, r_mma = 0, r_commit = 0, r_n = 0);
        // descriptors of stage 0; a stage further on adds stage_bytes / 16 to the address field, a k-step 2 (32 bytes)
        // or, for an MN-major B, 128 (2048 bytes); the barriers' cluster addresses are 8 bytes apart
        const uint64_t da0 = make_desc(smem_u32(smem), 16, 1024);
        const uint64_t db0 = q.b_kmajor ? make_desc(smem_u32(smem) + a_bytes, 16, 1024) : make_desc(smem_u32(smem) + a_bytes, 64 * BK * 2, 1024);
        const uint64_t dstage = stage_bytes >> 4, dsub = sub_bytes >> 4, dbk = q.b_kmajor ? 2 : 128;
        const uint32_t e_local = smem_u32(&empty_bar[0]);
        uint64_t da_s = da0, db_s = db0;
        for (int item = pair; item < total && ok; item += n_pairs, ++tcount) {
          const int acc = tcount & 1;
          const uint32_t aph = (tcount >> 1) & 1;
          { long long t0 = clock64(); if (!mbar_wait(&tempty_bar[acc], aph ^ 1, abort_flag)) { ok = false; break; } TR(r_tempty += clock64() - t0); }
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
          const int ks = (int)fd_div((uint32_t)item, q.fd_tiles);
          const int kt_begin = ks * q.kt_per, kt_end = min(k_tiles, kt_begin + q.kt_per);
          for (int kt = kt_begin; kt < kt_end; kt += kpack) {
            TR(const long long t0 = clock64());
            if (!mbar_wait(&full_bar[s], ph, abort_flag)) { ok = false; break; }
            TR(const long long t1 = clock64());
            // (no tcgen05 fence here: the operands were written by TMA, and the barrier orders its completion before
            // the MMAs' reads.  Every instruction of this thread that goes to an asynchronous unit costs 50 to 80 ns.)
#pragma unroll
            for (int kk = 0; kk < BK / 16; ++kk)
              tc_mma2(d_tmem, da_s + 2 * kk, db_s + dbk * kk, idesc, ((kt - kt_begin) | kk) ? 1u : 0u);
            if (kpack == 2) {
#pragma unroll
              for (int kk = 0; kk < BK / 16; ++kk)
                tc_mma2(d_tmem, da_s + dsub + 2 * kk, db_s + dsub + dbk * kk, idesc, 1u);
            }
            // stage free in both CTAs once these MMAs have read it: ONE commit, delivered to the barrier at this offset
            // in both CTAs of the pair.
            TR(const long long t2 = clock64());
            tc_commit2_both(e_local + 8u * (uint32_t)s);
            TR(const long long t3 = clock64(); r_wait += t1 - t0; r_mma += t2 - t1; r_commit += t3 - t2; r_n += 1);
            da_s += dstage; db_s += dstage;
            if (++s == stages) { s = 0; ph ^= 1; da_s = da0; db_s = db0; }
          }
          if (ok) tc_commit2_both(smem_u32(&tfull_bar[acc]));
        }
        TR(if (blockIdx.x == 0 && p.status) { long long* t = reinterpret_cast<long long*>(p.status) + 4; t[10] = r_tempty; t[11] = r_wait; t[12] = r_mma; t[13] = r_commit; t[14] = r_n; t[15] = clock64() - t_begin; });
      }
    }
  } else if (warp < 2 + EPI_WARPS) {
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
  if (plan_flag(DNNF_PLAN_NO_PAIR_GEMM)) return false;
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
  if (dev_env("DNNF_PAIR_BN")) best_bn = atoi(dev_env("DNNF_PAIR_BN"));      // development switch
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
  if (dev_env("DNNF_PAIR_KPACK")) q.kpack = atoi(dev_env("DNNF_PAIR_KPACK")) == 2 ? 2 : 1;
  const int stage_bytes = sub_bytes * q.kpack;
  q.stages = std::min(8, tc2::kRingBudget / stage_bytes);
  // split-K when fewer than half of the 74 CTA pairs would have a tile and the k loop is long.  Handing partial
  // tiles over through L2 costs about 3 us (measured), a k-tile about 0.22 us: it pays from 32 k-tiles up, with
  // two or three slices (1024 x 768 x 3072: 15.7 -> 13.2 us; 1024 x 768 x 768: 7.2 -> 9.2 us, so not there).
  q.ksplit = 1; q.kt_per = q.k_tiles;
  {
    int want = 1;
    if (q.total_tiles * 2 <= 74 && q.k_tiles >= 32 && !plan_flag(DNNF_PLAN_NO_SPLIT_K)) want = std::min(3, 74 / q.total_tiles);
    if (dev_env("DNNF_SPLIT_K")) want = std::max(1, std::min(8, atoi(dev_env("DNNF_SPLIT_K"))));
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
  L.threads = tc2::kThreads2;
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
    cfg.gridDim = dim3(L.grid); cfg.blockDim = dim3(tc2::kThreads2); cfg.dynamicSmemBytes = L.smem; cfg.stream = st;
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
