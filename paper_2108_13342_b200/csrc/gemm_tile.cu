// Tensor-core GEMM-anchored blocks, one output tile per CTA (sm_100a).
//
// For problems with too few 256-row tiles to fill the machine with the persistent CTA-pair kernel
// (the projection and feed-forward GEMMs of a 1024-token encoder layer): every CTA computes ONE
// 128 x BN tile (BN = 64 or 128) and leaves.  The kernel is built for latency and for overlap
// between CTAs instead of a long steady state:
//   * at most ~106 KB of shared memory and BN tensor-memory columns per CTA, so two CTAs share an
//     SM: while one runs its epilogue the other's MMAs use the tensor cores, and the CTAs of the
//     NEXT kernel on the stream (programmatic dependent launch) become resident, set up and fetch
//     their weights while this kernel drains;
//   * the B operand of a block is normally a weight, which no kernel of the graph writes: its
//     first ring stages are requested BEFORE the wait on the previous kernel, as are the bias
//     vectors; only the loads of A (and of a residual tile) wait;
//   * the chunk buffers of the epilogue reuse the operand ring, which is idle by then, unless a
//     residual tile has to be prefetched into them while the main loop runs.
// Roles: warps 0, 1 TMA producers (one lane each; producer j loads the k-tiles j, j+2, ...), warp 2 tensor-memory
// allocation and MMA issue (one lane), warps 3..6 epilogue: tcgen05.ld -> micro-op program -> bf16 ->
// swizzled 32 x 64 chunk -> TMA store.
// Every wait is bounded; on expiry the CTA records DNNF_ERR_TIMEOUT and releases tensor memory.
//
// Every TMA load in this file is a plain per-CTA load; no clusters are used.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdlib>

#include "ir.h"
#include "tc2_common.cuh"
#include "tma_host.h"

namespace dnnf {

namespace tile {

using namespace tc2;

constexpr int kEpiWarps = 4, kThreads = 96 + 32 * kEpiWarps;         // 2 producer warps, 1 issuer warp, 4 epilogue warps
constexpr int kVecBytes = kEpiWarps * kMaxVec * kBiasFloats * 4;     // staged row-invariant operands, per warp
constexpr int kBarBytes = 256;
constexpr int kSmemTwoPerSm = 112 * 1024;                            // two CTAs of this size fit one SM

struct Params {
  CUtensorMap tmA, tmB, tmD, tmC;
  int32_t b_kmajor, k_tiles, bn, tiles_n;
  int32_t c_input;           // index of the epilogue input that is a full tile (TMA-loaded), or -1
  int32_t stages;
  int32_t cbuf_off;          // chunk buffers, bytes from the ring's start: 0 (they reuse the ring) or behind the ring
  int32_t tail_off;          // staged vectors, then barriers
  int32_t b_static;          // B is never written by a kernel of the graph
  int32_t tmem_cols;
  int32_t ksplit, kt_per;    // CTAs of a cluster that share a tile (1, 2 or 4) and the k-tiles each of them takes
  FastDiv fd_tiles_n;
};

__device__ __forceinline__ void tc_commit1(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_mma1(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
               ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}
// CTA-scope barrier waits (this kernel has no cluster: the cluster-scope acquire of the pair kernel's wait is not needed).
__device__ __forceinline__ bool mbar_try_cta(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_cta(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_cta(bar, parity)) return true;
#pragma unroll 1
  for (int i = 0; i < kFastPolls; ++i) if (mbar_try_cta(bar, parity)) return true;
  const unsigned long long t0 = wall_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i) if (mbar_try_cta(bar, parity)) return true;
    if (*abort_flag) return false;
    if (wall_ns() - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
  }
}
// One lane of a converged warp.  The role loops below run in ALL lanes of their warp with identical values and only
// the issuing instruction sits under this predicate: the compiler then keeps descriptors, coordinates and barrier
// addresses in uniform registers instead of moving them there, lane by lane, in front of every TMA / MMA instruction.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n.reg .pred p;\nelect.sync _|p, 0xffffffff;\nselp.u32 %0, 1, 0, p;\n}" : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* tm) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(tm) : "memory");
}

// Epilogue IO of the split-K form: a thread owns 32 consecutive columns of its row of the CTA's column slice, reads a
// full-tile operand (a residual) and writes the result straight from / to global memory with 16-byte accesses.
struct SliceIO {
  static constexpr int VV = 32;
  const GemmParams& p;
  float accv[32];
  const float* vec_s;        // staged row-invariant operands of this warp: [kMaxVec][kBiasFloats], indexed by tile column
  int c_input;
  int col;                   // first tile column of the 32
  int n;                     // its global column
  uint32_t res_off, out_off; // element offsets of (row, column 0) in the residual and in the result
  bool row_ok;
  __device__ __forceinline__ void load(int idx, float (&dst)[VV]) const {
    const TensorArg& a = p.in[idx];
    if (idx == c_input) {
      const __nv_bfloat16* src = reinterpret_cast<const __nv_bfloat16*>(a.ptr) + res_off + n;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        uint4 w = make_uint4(0u, 0u, 0u, 0u);
        if (row_ok && n + 8 * j < p.N) w = __ldg(reinterpret_cast<const uint4*>(src + 8 * j));
        float* d = &dst[8 * j];
        d[0] = __uint_as_float(w.x << 16); d[1] = __uint_as_float(w.x & 0xffff0000u);
        d[2] = __uint_as_float(w.y << 16); d[3] = __uint_as_float(w.y & 0xffff0000u);
        d[4] = __uint_as_float(w.z << 16); d[5] = __uint_as_float(w.z & 0xffff0000u);
        d[6] = __uint_as_float(w.w << 16); d[7] = __uint_as_float(w.w & 0xffff0000u);
      }
      return;
    }
    const float* s = vec_s + a.mode * kBiasFloats + col;
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
    __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.out[0].ptr) + out_off + n;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      __nv_bfloat162 a0 = __floats2bfloat162_rn(val[8 * j], val[8 * j + 1]), a1 = __floats2bfloat162_rn(val[8 * j + 2], val[8 * j + 3]);
      __nv_bfloat162 a2 = __floats2bfloat162_rn(val[8 * j + 4], val[8 * j + 5]), a3 = __floats2bfloat162_rn(val[8 * j + 6], val[8 * j + 7]);
      if (row_ok && n + 8 * j < p.N)
        *reinterpret_cast<uint4*>(dst + 8 * j) = make_uint4(*reinterpret_cast<uint32_t*>(&a0), *reinterpret_cast<uint32_t*>(&a1),
                                                            *reinterpret_cast<uint32_t*>(&a2), *reinterpret_cast<uint32_t*>(&a3));
    }
  }
  __device__ __forceinline__ void row_reduce(int, float (&)[VV]) const {}
};

__device__ __forceinline__ void st_cluster_f4(uint32_t cluster_addr, float4 v) {
  asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}

#ifdef DNNF_TRACE
#define TSTAMP(slot) do { if (blockIdx.x == 0 && p.status) reinterpret_cast<unsigned long long*>(p.status)[4 + (slot)] = wall_ns(); } while (0)
#else
#define TSTAMP(slot) do {} while (0)
#endif

// kSplit: the CTAs of a cluster (2 or 4 of them) share one output tile, each accumulates a contiguous range of the
// k-tiles.  The partial sums meet through distributed shared memory as a reduce-scatter: CTA j of the cluster owns
// the columns [j BN / S, (j + 1) BN / S) of the tile, every other CTA writes its partial values of those columns
// into CTA j's operand ring (idle by then), and CTA j adds them to its own accumulator, runs the epilogue program on
// its slice and stores it.  Two cluster barriers frame the exchange: all main loops done (the rings are free), all
// partial sums written.  The main loop shrinks S-fold, and so does each CTA's epilogue.
template <class SP, bool kSplit>
__global__ void __launch_bounds__(kThreads, 2)
gemm_tile_kernel(const __grid_constant__ GemmParams p, const __grid_constant__ Params q) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int BN = q.bn, stages = q.stages;
  const uint32_t a_bytes = BM * BK * 2, b_bytes = (uint32_t)BN * BK * 2, stage_bytes = a_bytes + b_bytes;
  uint8_t* tail = smem + q.tail_off;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(tail + kVecBytes);   // [stages] bytes of one stage
  uint64_t* empty_bar = full_bar + 8;         // [stages] 1 arrival (commit)
  uint64_t* tfull_bar = empty_bar + 8;        // accumulator complete
  uint64_t* c_bar = tfull_bar + 1;            // [kEpiWarps] residual chunks landed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(c_bar + kEpiWarps);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  pdl_launch_dependents();
  if (threadIdx.x == 0) TSTAMP(0);
  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    mbar_init(tfull_bar, 1);
    for (int s = 0; s < kEpiWarps; ++s) mbar_init(&c_bar[s], 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 2) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)q.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  } else if (warp == 0 && lane == 0) {
    prefetch_tmap(&q.tmA); prefetch_tmap(&q.tmB); prefetch_tmap(&q.tmD);
    if (q.c_input >= 0) prefetch_tmap(&q.tmC);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (threadIdx.x == 0) TSTAMP(1);

  const int S = kSplit ? q.ksplit : 1;
  const int rank = kSplit ? (int)cluster_rank() : 0;
  const int tile = kSplit ? (int)(blockIdx.x / (unsigned)S) : (int)blockIdx.x;
  const int tm = (int)fd_div((uint32_t)tile, q.fd_tiles_n), tn = tile - tm * q.tiles_n;
  const int m0 = tm * BM, n0 = tn * BN;
  // this CTA's k-tiles
  const int kt0 = kSplit ? rank * q.kt_per : 0;
  const int k_tiles = kSplit ? min(q.k_tiles - kt0, q.kt_per) : q.k_tiles;

  if (warp < 2) {
    // ---------------- TMA producers: warp j loads the k-tiles j, j+2, j+4, ... ----------------
    // Each instruction that goes to an asynchronous unit (a barrier wait, a TMA request, an MMA, a commit) costs its
    // issuing thread 50 to 80 ns, whatever the size of the operation (measured: a ring that only passes barriers back
    // and forth, without loads or MMAs, still takes 210 ns per k-tile).  Two producers on alternate k-tiles keep the
    // loads off the critical path; the issuer's own instructions (a wait, four MMAs, a commit) then set the pace.
    if (lane == 0) {
      auto load_b = [&](int s, int kt) {
        uint8_t* sb = smem + (size_t)s * stage_bytes + a_bytes;
        if (q.b_kmajor) {
          tma_load_2d(sb, &q.tmB, &full_bar[s], (kt0 + kt) * BK, n0);
        } else {
          for (int j = 0; j < BN / 64; ++j) tma_load_2d(sb + j * (64 * BK * 2), &q.tmB, &full_bar[s], n0 + j * 64, (kt0 + kt) * BK);
        }
      };
      auto load_a = [&](int s, int kt) { tma_load_2d(smem + (size_t)s * stage_bytes, &q.tmA, &full_bar[s], (kt0 + kt) * BK, m0); };
      const int npre = min(stages, k_tiles);
      // a weight operand is written by no kernel: its first stages are requested while the previous kernel still runs
      if (q.b_static)
        for (int kt = warp; kt < npre; kt += 2) { mbar_expect_tx(&full_bar[kt], stage_bytes); load_b(kt, kt); }
      pdl_wait();
      if (warp == 0) TSTAMP(2);
      for (int kt = warp; kt < npre; kt += 2) {
        if (!q.b_static) { mbar_expect_tx(&full_bar[kt], stage_bytes); load_b(kt, kt); }
        load_a(kt, kt);
      }
      // first k-tile of this warp at or beyond the pre-issued ones
      int kt = npre + ((npre ^ warp) & 1);
      int s = kt - stages; uint32_t ph = 0;
      while (s >= stages) { s -= stages; ph ^= 1; }
      for (; kt < k_tiles; kt += 2) {
        if (!mbar_wait_cta(&empty_bar[s], ph, abort_flag)) break;
        mbar_expect_tx(&full_bar[s], stage_bytes);
        load_a(s, kt);
        load_b(s, kt);
        s += 2;
        if (s >= stages) { s -= stages; ph ^= 1; }
      }
    }
    if (kSplit) { __syncwarp(); cluster_sync(); cluster_sync(); }
  } else if (warp == 2) {
    // ---------------- MMA issuer ----------------
    // (No tcgen05 fence inside the loop: the operands were written by TMA, whose completion the barrier itself orders
    // before the MMAs' reads; an instruction saved per k-tile is 50 ns saved.)
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((q.b_kmajor ? 0u : 1u) << 16) | ((uint32_t)(BN >> 3) << 17) |
                             ((uint32_t)(BM >> 4) << 24);
      const uint64_t da0 = make_desc(smem_u32(smem), 16, 1024);
      const uint64_t db0 = q.b_kmajor ? make_desc(smem_u32(smem) + a_bytes, 16, 1024) : make_desc(smem_u32(smem) + a_bytes, 64 * BK * 2, 1024);
      const uint64_t dstage = stage_bytes >> 4, dbk = q.b_kmajor ? 2 : 128;
      uint64_t da_s = da0, db_s = db0;
      int s = 0; uint32_t ph = 0;
      bool ok = true;
      for (int kt = 0; kt < k_tiles; ++kt) {
        if (!mbar_wait_cta(&full_bar[s], ph, abort_flag)) { ok = false; break; }
        if (kt == 0) TSTAMP(3);
        if (kt == k_tiles - 1) TSTAMP(4);
#pragma unroll
        for (int kk = 0; kk < BK / 16; ++kk) tc_mma1(tmem_base, da_s + 2 * kk, db_s + dbk * kk, idesc, (kt | kk) ? 1u : 0u);
        if (kt + stages < k_tiles) tc_commit1(&empty_bar[s]);     // only a stage that is refilled needs the signal
        da_s += dstage; db_s += dstage;
        if (++s == stages) { s = 0; ph ^= 1; da_s = da0; db_s = db0; }
      }
      if (ok) tc_commit1(tfull_bar);         // accumulator complete
    }
    if (kSplit) { __syncwarp(); cluster_sync(); cluster_sync(); }
  } else {
    // ---------------- epilogue warps 3..6: a warp may read the tensor-memory lanes 32 (warp % 4) .. + 31 ----------------
    const int ew = warp - 3, sub = warp & 3;
    const int chunks = BN / 64;
    uint8_t* cbuf = smem + q.cbuf_off + (size_t)ew * chunks * kChunkBytes;
    float* vec_s = reinterpret_cast<float*>(tail) + ew * (kMaxVec * kBiasFloats);
    const int mw0 = m0 + sub * 32;
    auto stage_vectors = [&](bool want_static) {
      for (int k = 0; k < p.n_in; ++k) {
        const TensorArg& a = p.in[k];
        if (k == q.c_input || (((p.static_mask >> (1 + k)) & 1u) != 0) != want_static) continue;
        for (int c = lane; c < BN; c += 32) {
          const int n = n0 + c;
          vec_s[a.mode * kBiasFloats + c] = n < p.N ? load_scalar<false>(a, (uint32_t)a.base + (uint32_t)n * (uint32_t)a.stride[0]) : 0.0f;
        }
      }
    };
    stage_vectors(true);
    pdl_wait();
    if (!kSplit && q.c_input >= 0 && lane == 0) {                 // the residual tile of this warp: all chunks at once
      mbar_expect_tx(&c_bar[ew], (uint32_t)(chunks * kChunkBytes));
      for (int c = 0; c < chunks; ++c) tma_load_2d(cbuf + c * kChunkBytes, &q.tmC, &c_bar[ew], n0 + c * 64, mw0);
    }
    stage_vectors(false);
    __syncwarp();
    bool ok = mbar_wait_cta(tfull_bar, 0, abort_flag);
    if (!kSplit && ok && q.c_input >= 0) ok = mbar_wait_cta(&c_bar[ew], 0, abort_flag);
    ok = __all_sync(0xffffffffu, ok);        // the tensor-memory loads below are warp-wide
    if (ew == 0 && lane == 0) TSTAMP(5);
    const uint32_t t_row = tmem_base + ((uint32_t)(sub * 32) << 16);
    if (kSplit) {
      const int slice = BN / S;                                    // 64 or 32 columns per owner
      const int pieces = slice >> 2;                               // 16-byte pieces of a row of a slice
      const int row = sub * 32 + lane;
      tc_fence_after();
      cluster_sync();                                              // every CTA of the cluster is through its main loop
      if (ew == 0 && lane == 0) TSTAMP(6);
      if (ok) {
        // hand the partial sums of the other CTAs' slices over: receive buffer [sender][piece][row] of float4
        for (int j = 0; j < S; ++j) {
          if (j == rank) continue;
          const int slot = rank < j ? rank : rank - 1;
          const uint32_t remote = mapa(smem_u32(smem), (uint32_t)j) + (uint32_t)((slot * pieces) * BM + row) * 16u;
          for (int c = 0; c < slice; c += 32) {
            uint32_t raw[32];
            tc_ld32(t_row + j * slice + c, raw);
            tc_ld_wait();
#pragma unroll
            for (int v = 0; v < 8; ++v)
              st_cluster_f4(remote + (uint32_t)(((c >> 2) + v) * BM) * 16u,
                            make_float4(__uint_as_float(raw[4 * v]), __uint_as_float(raw[4 * v + 1]), __uint_as_float(raw[4 * v + 2]), __uint_as_float(raw[4 * v + 3])));
          }
        }
      }
      if (ew == 0 && lane == 0) TSTAMP(7);
      cluster_sync();                                              // all partial sums have arrived
      if (ew == 0 && lane == 0) TSTAMP(8);
      if (ok) {
        SliceIO io{p};
        io.vec_s = vec_s; io.c_input = q.c_input;
        const int m = mw0 + lane;
        io.row_ok = m < p.M;
        const uint32_t mm = io.row_ok ? (uint32_t)m : 0u;
        io.out_off = (uint32_t)p.out[0].base + mm * (uint32_t)p.out[0].stride[1];
        io.res_off = q.c_input >= 0 ? (uint32_t)p.in[q.c_input].base + mm * (uint32_t)p.in[q.c_input].stride[1] : 0u;
        const float4* rcv = reinterpret_cast<const float4*>(smem);
        for (int c = 0; c < slice; c += 32) {
          uint32_t raw[32];
          tc_ld32(t_row + rank * slice + c, raw);
          tc_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) io.accv[i] = __uint_as_float(raw[i]);
          for (int sl = 0; sl < S - 1; ++sl) {
#pragma unroll
            for (int v = 0; v < 8; ++v) {
              const float4 w = rcv[(sl * pieces + (c >> 2) + v) * BM + row];
              io.accv[4 * v] += w.x; io.accv[4 * v + 1] += w.y; io.accv[4 * v + 2] += w.z; io.accv[4 * v + 3] += w.w;
            }
          }
          io.col = rank * slice + c;
          io.n = n0 + io.col;
          run_program<32, SP, true>(p.prog, io);
        }
      }
      if (ew == 0 && lane == 0) TSTAMP(9);
    } else if (ok) {
      EpiIO io{p};
      io.lane = lane; io.c_input = q.c_input; io.vec_s = vec_s;
      tc_fence_after();
      for (int c = 0; c < chunks; ++c) {
        io.chunk = cbuf + c * kChunkBytes;
#pragma unroll 1
        for (int h = 0; h < 2; ++h) {
          uint32_t raw[32];
          tc_ld32(t_row + c * 64 + h * 32, raw);
          tc_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) io.accv[i] = __uint_as_float(raw[i]);
          io.col_in_chunk = h * 32;
          io.col_in_half = c * 64 + h * 32;
          run_program<32, SP, true>(p.prog, io);
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) { tma_store_2d(&q.tmD, io.chunk, n0 + c * 64, mw0); tma_store_commit(); }
      }
      if (ew == 0 && lane == 0) TSTAMP(6);
      if (lane == 0) tma_store_wait_all();
      if (ew == 0 && lane == 0) TSTAMP(7);
    }
  }

  // ---------------- teardown ----------------
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0 && p.status) { atomicExch(&p.status[0], DNNF_ERR_TIMEOUT); atomicExch(&p.status[1], p.block_index); }
    // give copies that are still in flight time to land before shared memory is released
    if (threadIdx.x == 0) { long long t0 = clock64(); while (clock64() - t0 < 2000000) {} }
    __syncthreads();
  }
  if (warp == 2) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)q.tmem_cols) : "memory");
  }
}

}  // namespace tile

// ---- host side --------------------------------------------------------------------------------------
static GemmParams& gp_of(Launch& L) { return *reinterpret_cast<GemmParams*>(L.blob.data()); }
static const GemmParams& gp_of(const Launch& L) { return *reinterpret_cast<const GemmParams*>(L.blob.data()); }
static tile::Params& tl_of(Launch& L) { return *reinterpret_cast<tile::Params*>(L.blob.data() + sizeof(GemmParams) + sizeof(GemmTcParams)); }
static const tile::Params& tl_of(const Launch& L) { return *reinterpret_cast<const tile::Params*>(L.blob.data() + sizeof(GemmParams) + sizeof(GemmTcParams)); }

size_t tile_blob_bytes() { return sizeof(tile::Params); }

bool tc_gemm_eligible(const GemmParams& gp);

// Same operand and epilogue forms as the CTA-pair kernel (plain 2-D problem, one bf16 row-major output, at most one
// bf16 full-tile input, row-invariant others), without its lower bounds on M and N.
bool tile_gemm_eligible(const GemmParams& gp) {
  if (!tc_gemm_eligible(gp)) return false;
  if (gp.batch_ext[0] * gp.batch_ext[1] != 1) return false;
  if (gp.N < 32 || gp.N % 8) return false;
  if (gp.n_nd != 1 || gp.m_nd != 1 || gp.n_out != 1 || !gp.vec_ok) return false;
  const TensorArg& o = gp.out[0];
  if (o.dtype != DNNF_BF16 || o.stride[0] != 1 || o.stride[1] % 8 || o.base % 8 || o.stride[1] <= 0) return false;
  int full = 0, vec = 0;
  for (int i = 0; i < gp.n_in; ++i) {
    const TensorArg& a = gp.in[i];
    if (a.mode == 1) { if (a.stride[0] != 1) return false; vec++; }
    else { if (a.dtype != DNNF_BF16 || a.stride[0] != 1 || a.stride[1] % 8 || a.base % 8 || a.stride[1] <= 0) return false; full++; }
  }
  return full <= 1 && vec <= tc2::kMaxVec;
}

// Measured on the projection and feed-forward shapes of a 1024-token encoder layer: a k-tile costs a CTA about 0.35 us
// whatever the tile's size, so a problem with few 256 x 256 tiles and a short K finishes sooner as many small tiles
// (1024 x 768 x 768: 7.2 against 7.8 us; 1024 x 2304 x 768: 7.4 against 8.1; 1024 x 3072 x 768: 9.7 against 11.1), while a
// long K is better off with the CTA-pair kernel and its split over K (1024 x 768 x 3072: 14.2 against 18.5 us).
bool tile_gemm_preferred(const GemmParams& gp) {
  if (plan_flag(DNNF_PLAN_NO_TILE_GEMM)) return false;
  if (dev_env("DNNF_GEMM_TILE")) return atoi(dev_env("DNNF_GEMM_TILE")) != 0;
  const int64_t pair_tiles = (int64_t)((gp.M + 255) / 256) * ((gp.N + 255) / 256);
  const int k_tiles = (gp.K + tc2::BK - 1) / tc2::BK;
  // a long K is better off with the CTA-pair kernel and its split over K (1024 x 768 x 3072: 14.2 us against 22.6 us
  // here without a split and 15.5 us with the cluster split below)
  return pair_tiles < sm_count() / 2 && (k_tiles <= 16 || plan_flag(DNNF_PLAN_CLUSTER_SPLIT_K));
}

void tile_gemm_plan(Launch& L) {
  GemmParams& gp = gp_of(L);
  tile::Params& q = tl_of(L);
  q.b_kmajor = (gp.B.stride_col != 1) ? 1 : 0;
  q.k_tiles = (gp.K + tc2::BK - 1) / tc2::BK;
  const int tiles_m = (gp.M + tc2::BM - 1) / tc2::BM;
  const int sms = sm_count();
  // N tile: 128 columns unless that leaves most of the machine without a CTA (an MMA costs its issuer the same 60
  // cycles whatever its width); with the cluster split the CTAs come from the split instead
  int best_bn = (gp.N > 64 && (plan_flag(DNNF_PLAN_CLUSTER_SPLIT_K) || (int64_t)tiles_m * ((gp.N + 127) / 128) >= 96)) ? 128 : 64;
  if (dev_env("DNNF_TILE_BN")) best_bn = atoi(dev_env("DNNF_TILE_BN")) == 128 ? 128 : 64;
  q.bn = best_bn;
  q.tiles_n = (gp.N + q.bn - 1) / q.bn;
  q.fd_tiles_n = make_fastdiv((uint32_t)q.tiles_n);
  gp.tiles_m = tiles_m; gp.tiles_n = q.tiles_n;
  // Split over K through a cluster (DNNF_PLAN_CLUSTER_SPLIT_K only): a k-tile costs a CTA about 0.35 us whatever the
  // tile's size, so the k-tiles of a tile are shared by a cluster of 4 or 2 CTAs as long as two CTAs per SM hold the
  // whole grid and every CTA keeps at least three k-tiles.  Measured, it does not pay at these sizes: the main loop of
  // 1024 x 768 x 768 ends after 2.6 instead of 5.9 us, but the hand-over (0.6 us barrier, 1.2 us of remote stores, 2 us
  // until every CTA's stores have arrived) and 2.5 us more per launch of a cluster in a chain of dependent kernels eat
  // all of it (11.5 against 8.5 us per launch), hence off by default.
  const int64_t tiles = (int64_t)tiles_m * q.tiles_n;
  int S = 1;
  if (plan_flag(DNNF_PLAN_CLUSTER_SPLIT_K) && !plan_flag(DNNF_PLAN_NO_SPLIT_K)) {
    for (int cand : {4, 2}) {
      if (q.bn / cand < 32) continue;
      if (tiles * cand <= 2 * sms && q.k_tiles >= 3 * cand) { S = cand; break; }
    }
  }
  if (dev_env("DNNF_TILE_SPLIT")) { const int v = atoi(dev_env("DNNF_TILE_SPLIT")); if ((v == 1 || v == 2 || v == 4) && q.bn / v >= 32 && q.k_tiles >= v) S = v; }
  q.ksplit = S;
  q.kt_per = (q.k_tiles + S - 1) / S;
  if ((S - 1) * q.kt_per >= q.k_tiles) { q.ksplit = S = 1; q.kt_per = q.k_tiles; }     // every CTA of the cluster needs a k-tile
  q.c_input = -1;
  int vec_slot = 0;
  for (int i = 0; i < gp.n_in; ++i) {
    if (gp.in[i].mode == 1) gp.in[i].mode = vec_slot++;      // from here on: slot in the staged-vector area
    else { q.c_input = i; gp.in[i].mode = 0; }
  }
  q.b_static = (gp.static_mask & 1u) ? 1 : 0;
  const int stage_bytes = tc2::BM * tc2::BK * 2 + q.bn * tc2::BK * 2;
  // chunk buffers: a residual tile is prefetched into its own ones; without one they reuse the ring; the split form
  // reads and writes global memory directly and needs none
  const bool own_cbuf = q.c_input >= 0 && S == 1;
  const int cbuf_bytes = tc2::BM * q.bn * 2;
  const int fixed = 1024 + tile::kVecBytes + tile::kBarBytes + (own_cbuf ? cbuf_bytes : 0);
  int budget = tile::kSmemTwoPerSm;
  if (dev_env("DNNF_TILE_SMEM")) budget = atoi(dev_env("DNNF_TILE_SMEM")) * 1024;
  q.stages = std::max(2, std::min({8, q.kt_per, (budget - fixed) / stage_bytes}));
  int ring = q.stages * stage_bytes;
  if (S > 1) ring = std::max(ring, (S - 1) * (q.bn / S / 4) * tc2::BM * 16);          // the ring doubles as the receive buffer
  q.cbuf_off = own_cbuf ? ring : 0;
  q.tail_off = own_cbuf ? ring + cbuf_bytes : (S > 1 ? ring : std::max(ring, cbuf_bytes));
  q.tmem_cols = q.bn < 32 ? 32 : q.bn;
  L.counter_bytes = L.scratch_bytes = 0;
  L.grid = (int)(tiles * S);
  L.threads = tile::kThreads;
  L.smem = (size_t)q.tail_off + tile::kVecBytes + tile::kBarBytes + 1024;
  L.variant = 5;
  L.static_id = StaticSet<Epi2Static>::find(gp.prog);
}

static bool encode2d(CUtensorMap* tm, void* base, int64_t ext_inner, int64_t ext_outer, int64_t stride_outer_elems, int box_inner, int box_outer,
                     std::string& err) {
  cuuint64_t dims[2] = {(cuuint64_t)ext_inner, (cuuint64_t)ext_outer};
  cuuint64_t strides[1] = {(cuuint64_t)stride_outer_elems * 2};
  cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
  return tma_encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B, err);
}

bool tile_gemm_prepare(Launch& L, std::string& err) {
  GemmParams& gp = gp_of(L);
  tile::Params& q = tl_of(L);
  uint16_t* a = reinterpret_cast<uint16_t*>(gp.A.ptr) + gp.A.base;
  uint16_t* b = reinterpret_cast<uint16_t*>(gp.B.ptr) + gp.B.base;
  uint16_t* d = reinterpret_cast<uint16_t*>(gp.out[0].ptr) + gp.out[0].base;
  if (((uintptr_t)a & 15) || ((uintptr_t)b & 15) || ((uintptr_t)d & 15)) { err = "GEMM operand is not 16-byte aligned"; return false; }
  if (!encode2d(&q.tmA, a, gp.K, gp.M, gp.A.stride_row, tc2::BK, tc2::BM, err)) return false;
  if (q.b_kmajor) { if (!encode2d(&q.tmB, b, gp.K, gp.N, gp.B.stride_col, tc2::BK, q.bn, err)) return false; }
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

struct TileLauncher {
  const Launch& L; cudaStream_t st; cudaError_t rc;
  template <class SP> void run() {
    const int S = tl_of(L).ksplit;
    if (S <= 1) {
      static PerDeviceOnce once;       // per instantiation
      if (once.first_use()) cudaFuncSetAttribute(tile::gemm_tile_kernel<SP, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
      rc = launch_pdl(tile::gemm_tile_kernel<SP, false>, dim3(L.grid), dim3(tile::kThreads), L.smem, st, gp_of(L), tl_of(L));
      return;
    }
    static PerDeviceOnce once;
    if (once.first_use()) cudaFuncSetAttribute(tile::gemm_tile_kernel<SP, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(L.grid); cfg.blockDim = dim3(tile::kThreads); cfg.dynamicSmemBytes = L.smem; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)S; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 2;
    rc = cudaLaunchKernelEx(&cfg, tile::gemm_tile_kernel<SP, true>, gp_of(L), tl_of(L));
  }
};

int tile_gemm_launch(const Launch& L, cudaStream_t st) {
  TileLauncher F{L, st, cudaSuccess};
  if (!(L.static_id > 0 && StaticSet<Epi2Static>::dispatch(L.static_id, F))) F.run<DynProg>();
  return (F.rc == cudaSuccess && cudaGetLastError() == cudaSuccess) ? 0 : 1;
}

}  // namespace dnnf
