// Single-kernel attention block: scores = Q K^T [* c] [+ mask] -> row softmax -> P V, one launch.
//
// Table 3 forbids this fusion (Many-to-Many followed by Many-to-Many is a red cell), so it is
// never part of a plan made by the paper's rules; dnnf_plan forms it only under
// DNNF_PLAN_BEYOND_TABLE3, from three blocks the normal plan already holds: a batched GEMM
// block whose epilogue is the scale / mask chain, the Softmax row block, and the batched GEMM
// block that multiplies by V (with its permuted store).  The scores and the probabilities then
// never leave the SM: the scores stay in tensor memory as fp32, the probabilities go through
// shared memory as the bf16 A operand of the second MMA.
//
// One CTA per (batch element, head, 128 query rows); all keys of a head at once (at most 256):
//   warp 0      TMA: Q and K tiles, then V (plain per-CTA loads, 4-D maps over the strided head views)
//   warp 1      tensor-memory allocation; MMA 1: S[128 x Sk] = Q K^T; after the softmax MMA 2: O[128 x D] = P V
//   warps 2..9  two threads share a query row (tensor-memory lane), half of the keys each, kept in registers:
//               x = c * s + mask, row maximum, e = exp(x - max) summed in fp32 and written as bf16 into the
//               swizzled P tile; after MMA 2: O / sum -> bf16 -> the block's output index map (the head
//               transpose is a store pattern)
// Every wait is bounded; on expiry the CTA records DNNF_ERR_TIMEOUT and releases tensor memory.
//
// Every TMA load in this file is a plain per-CTA load; no clusters are used.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <set>

#include "ir.h"
#include "lower.h"
#include "tc_common.cuh"
#include "tma_host.h"

namespace dnnf {

int lower_contraction(const Graph& g, const std::vector<int>& ops, uint32_t flags, int anchor, Block& out, std::string& why);

namespace attn {

constexpr int BM = 128, THREADS = 320;
constexpr int kSmemMax = 227 * 1024;

struct Params {
  CUtensorMap tmQ, tmK, tmV;
  int32_t Sq, Sk, D;
  int32_t sk16;              // Sk rounded up to the MMA's N granularity
  int32_t q_tiles;
  int32_t mask_in;           // index of the additive mask among the first GEMM's epilogue inputs, or -1
  float scale;               // 1 when the chain has no scalar factor
  int32_t tmem_cols, o_col;  // allocation and the first column of O
  int32_t q_batch[2], k_batch[2], v_batch[2];   // 1 where the operand has that batch digit (0: broadcast)
  int32_t off_k, off_v, off_p, off_bar;         // shared-memory carve-up, bytes from the 1024-aligned base
  int32_t off_mask;          // the query tile's mask rows staged in shared memory, or -1 (read from global memory)
  int32_t mask_static;       // the mask is written by no kernel of the graph: staged before the wait on the previous kernel
  int32_t mask_pitch4;       // 16-byte pieces per staged mask row (a multiple of 8)
  FastDiv fd_qtiles, fd_b0, fd_pitch4;
};

__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// Wait for the tensor-memory loads issued so far.  The loaded registers are named as read-write operands: without that
// the compiler sees no dependence between the wait and later arithmetic on them, and may schedule that arithmetic
// ahead of the wait when other work (the mask loads) sits between the load's issue and the wait.
__device__ __forceinline__ void tc_ld_wait32(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]), "+r"(r[9]),
                 "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]), "+r"(r[17]), "+r"(r[18]),
                 "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]),
                 "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :: "memory");
}

__device__ __forceinline__ float fast_exp2(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }

template <int NC>
__global__ void __launch_bounds__(THREADS, 1)
attention_kernel(const __grid_constant__ GemmParams pA, const __grid_constant__ GemmParams pC, const __grid_constant__ Params q) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sK = smem + q.off_k;
  uint8_t* sV = smem + q.off_v;
  uint8_t* sP = smem + q.off_p;
  uint64_t* bar_qk = reinterpret_cast<uint64_t*>(smem + q.off_bar);
  uint64_t* bar_v = bar_qk + 1;
  uint64_t* bar_s = bar_qk + 2;      // scores complete
  uint64_t* bar_p = bar_qk + 3;      // probabilities written (8 warps)
  uint64_t* bar_o = bar_qk + 4;      // output accumulator complete
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_qk + 5);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int D = q.D, Sk = q.Sk, sk16 = q.sk16;
  const int d_tiles = D >> 6, s_tiles = (sk16 + 63) >> 6;
  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    mbar_init(bar_qk, 1); mbar_init(bar_v, 1); mbar_init(bar_s, 1); mbar_init(bar_p, 8); mbar_init(bar_o, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)q.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int item = blockIdx.x;
  const int batch = (int)fd_div((uint32_t)item, q.fd_qtiles), qt = item - batch * q.q_tiles;
  const int b1 = (int)fd_div((uint32_t)batch, q.fd_b0), b0 = batch - b1 * pA.batch_ext[0];

  // The mask rows of this query tile, staged in shared memory by the softmax warps with coalesced loads (a thread
  // later reads ITS row: from global memory that is one cache line per lane and instruction).  16-byte pieces are
  // XOR-swizzled by the row so that eight neighbouring rows read eight different bank groups.
  const bool stage_mask = q.off_mask >= 0 && (reinterpret_cast<uintptr_t>(pA.in[q.mask_in >= 0 ? q.mask_in : 0].ptr) & 15) == 0;
  auto load_mask_tile = [&]() {
    const TensorArg& ma = pA.in[q.mask_in];
    const uint32_t tile_off = (uint32_t)ma.base + tc_digits(pA, ma, pA.n_nd + pA.m_nd, pA.b_nd, (uint32_t)batch);
    float4* sM = reinterpret_cast<float4*>(smem + q.off_mask);
    const int p4 = q.mask_pitch4;
    for (int i = (int)threadIdx.x - 64; i < BM * p4; i += THREADS - 64) {
      const int r = (int)fd_div((uint32_t)i, q.fd_pitch4), c4 = i - r * p4;
      const int m = qt * BM + r;
      float4 w = make_float4(0.f, 0.f, 0.f, 0.f);
      if (m < q.Sq && 4 * c4 < q.Sk) w = __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(ma.ptr) + tile_off + (uint32_t)m * (uint32_t)ma.stride[1]) + c4);
      sM[r * p4 + (c4 ^ (r & 7))] = w;
    }
  };
  if (stage_mask && q.mask_static && warp >= 2) load_mask_tile();      // a weight: no need to wait for the previous kernel
  pdl_wait();
  if (stage_mask && !q.mask_static && warp >= 2) load_mask_tile();

  if (warp == 0) {
    if (lane == 0) {
      // ---------------- loads: the whole head at once ----------------
      mbar_expect_tx(bar_qk, (uint32_t)(d_tiles * (BM + sk16) * 128));
      for (int kt = 0; kt < d_tiles; ++kt) {
        tma_load_4d(sQ + kt * (BM * 128), &q.tmQ, bar_qk, kt * 64, qt * BM, q.q_batch[0] ? b0 : 0, q.q_batch[1] ? b1 : 0);
        tma_load_4d(sK + kt * (sk16 * 128), &q.tmK, bar_qk, kt * 64, 0, q.k_batch[0] ? b0 : 0, q.k_batch[1] ? b1 : 0);
      }
      mbar_expect_tx(bar_v, (uint32_t)(s_tiles * d_tiles * 8192));
      for (int kt = 0; kt < s_tiles; ++kt)
        for (int j = 0; j < d_tiles; ++j)
          tma_load_4d(sV + (kt * d_tiles + j) * 8192, &q.tmV, bar_v, j * 64, kt * 64, q.v_batch[0] ? b0 : 0, q.v_batch[1] ? b1 : 0);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---------------- MMA issuer ----------------
      const uint32_t idesc0 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BM >> 4) << 24);
      const uint32_t idesc_s = idesc0 | ((uint32_t)(sk16 >> 3) << 17);                       // B = K, K-major
      const uint32_t idesc_o = idesc0 | (1u << 16) | ((uint32_t)(D >> 3) << 17);             // B = V, MN-major
      bool ok = mbar_wait(bar_qk, 0, abort_flag);
      if (ok) {
        for (int kt = 0; kt < d_tiles; ++kt) {
          const uint64_t da = make_desc(smem_u32(sQ) + kt * (BM * 128), 16, 1024);
          const uint64_t db = make_desc(smem_u32(sK) + kt * (sk16 * 128), 16, 1024);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) tc_mma_bf16(tmem_base, da + 2 * kk, db + 2 * kk, idesc_s, (kt | kk) ? 1u : 0u);
        }
        tc_commit(bar_s);
        ok = mbar_wait(bar_p, 0, abort_flag) && mbar_wait(bar_v, 0, abort_flag);
      }
      if (ok) {
        tc_fence_after();
        const uint32_t d_o = tmem_base + (uint32_t)q.o_col;
        for (int kt = 0; kt < s_tiles; ++kt) {
          const uint64_t da = make_desc(smem_u32(sP) + kt * (BM * 128), 16, 1024);
          const uint64_t db = make_desc(smem_u32(sV) + kt * d_tiles * 8192, 8192, 1024);
          const int ksteps = min(4, (sk16 - kt * 64) >> 4);
          for (int kk = 0; kk < ksteps; ++kk) tc_mma_bf16(d_o, da + 2 * kk, db + 128 * kk, idesc_o, (kt | kk) ? 1u : 0u);
        }
        tc_commit(bar_o);
      }
    }
  } else {
    // ---------------- softmax and output: two threads share a query row ----------------
    // warp 2 + 4 h + s: tensor-memory lanes 32 ((2 + s) % 4) .., column half h.  A thread keeps its NC x 32 scores in
    // registers from the tensor-memory load to the bf16 store: one pass, the mask read once, all loads in flight
    // together; the two halves of a row exchange maximum and sum through shared memory.
    const int sub = warp & 3, half = (warp - 2) >> 2;
    const int row = sub * 32 + lane;
    const int m = qt * BM + row;
    const bool row_ok = m < q.Sq;
    const uint32_t mm = row_ok ? (uint32_t)m : 0u;
    const uint32_t t_row = tmem_base + ((uint32_t)(sub * 32) << 16);
    const float c = q.scale;
    const int col0 = half * NC * 32;                       // this thread's first column
    float* xch = reinterpret_cast<float*>(smem + q.off_bar + 128);   // [2 values][2 halves][128 rows]
    const bool has_mask = q.mask_in >= 0;
    const TensorArg& ma = pA.in[has_mask ? q.mask_in : 0];
    uint32_t moff = 0;
    if (has_mask) moff = (uint32_t)ma.base + tc_digits(pA, ma, pA.n_nd, pA.m_nd, mm) + tc_digits(pA, ma, pA.n_nd + pA.m_nd, pA.b_nd, (uint32_t)batch);
    const bool mask_vec = has_mask && ma.dtype == DNNF_F32 && ma.stride[0] == 1 && (moff & 3u) == 0 && (Sk & 3) == 0 &&
                          (reinterpret_cast<uintptr_t>(ma.ptr) & 15) == 0;
    // the mask values of this thread's columns (requested before the scores are waited for)
    float x[NC * 32];
    if (stage_mask) {
      asm volatile("bar.sync 1, 256;" ::: "memory");       // the tile is complete
      const float4* srow = reinterpret_cast<const float4*>(smem + q.off_mask) + row * q.mask_pitch4;
#pragma unroll
      for (int j = 0; j < NC * 8; ++j) {
        float4 w = make_float4(0.f, 0.f, 0.f, 0.f);
        if (col0 + 4 * j < sk16) w = srow[((col0 >> 2) + j) ^ (row & 7)];
        x[4 * j] = w.x; x[4 * j + 1] = w.y; x[4 * j + 2] = w.z; x[4 * j + 3] = w.w;
      }
    } else if (!has_mask) {
#pragma unroll
      for (int j = 0; j < NC * 32; ++j) x[j] = 0.0f;
    } else if (mask_vec) {
      const float4* src = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(ma.ptr) + moff + col0);
#pragma unroll
      for (int j = 0; j < NC * 8; ++j) {
        float4 w = make_float4(0.f, 0.f, 0.f, 0.f);
        if (col0 + 4 * j < Sk) w = __ldg(src + j);
        x[4 * j] = w.x; x[4 * j + 1] = w.y; x[4 * j + 2] = w.z; x[4 * j + 3] = w.w;
      }
    } else {
#pragma unroll
      for (int j = 0; j < NC * 32; ++j) x[j] = (col0 + j < Sk) ? load_scalar<false>(ma, moff + (uint32_t)(col0 + j) * (uint32_t)ma.stride[0]) : 0.0f;
    }
    bool ok = __all_sync(0xffffffffu, mbar_wait(bar_s, 0, abort_flag));
    float inv_sum = 0.0f;
    if (ok) {
      tc_fence_after();
      float mx = -3.0e38f;
#pragma unroll
      for (int ch = 0; ch < NC; ++ch) {
        uint32_t raw[32];
        if (col0 + ch * 32 < sk16) {                       // (uniform over the warp)
          tc_ld32_issue(t_row + col0 + ch * 32, raw);
          tc_ld_wait32(raw);
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float v = fmaf(__uint_as_float(raw[j]), c, x[ch * 32 + j]);
            x[ch * 32 + j] = v;
            if (col0 + ch * 32 + j < Sk) mx = fmaxf(mx, v);
          }
        }
      }
      xch[half * BM + row] = mx;
      asm volatile("bar.sync 1, 256;" ::: "memory");
      mx = fmaxf(mx, xch[(half ^ 1) * BM + row]);
      // exponentials, their sum, the bf16 P tile (K-major, 128-byte swizzle; columns past Sk are zero)
      float sum = 0.0f;
      const float l2e = 1.4426950408889634f;
      const float mxl = mx * l2e;
#pragma unroll
      for (int ch = 0; ch < NC; ++ch) {
        const int c0 = col0 + ch * 32;
        if (c0 < sk16) {
          uint8_t* prow = sP + (c0 >> 6) * (BM * 128) + row * 128;
#pragma unroll
          for (int pc = 0; pc < 4; ++pc) {
            uint32_t w[4];
#pragma unroll
            for (int h = 0; h < 4; ++h) {
              float e[2];
#pragma unroll
              for (int u = 0; u < 2; ++u) {
                const int j = pc * 8 + h * 2 + u;
                e[u] = (c0 + j < Sk) ? fast_exp2(fmaf(x[ch * 32 + j], l2e, -mxl)) : 0.0f;
              }
              // the sum runs over the values the MMA will see
              __nv_bfloat162 b = __floats2bfloat162_rn(e[0], e[1]);
              sum += __low2float(b) + __high2float(b);
              w[h] = *reinterpret_cast<uint32_t*>(&b);
            }
            const int piece = ((c0 & 63) >> 3) + pc;
            *reinterpret_cast<uint4*>(prow + ((piece ^ (row & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
      xch[2 * BM + half * BM + row] = sum;
      fence_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_p);
      asm volatile("bar.sync 1, 256;" ::: "memory");
      inv_sum = 1.0f / (sum + xch[2 * BM + (half ^ 1) * BM + row]);
      ok = __all_sync(0xffffffffu, mbar_wait(bar_o, 0, abort_flag));
    }
    if (ok) {
      tc_fence_after();
      const TensorArg& oa = pC.out[0];
      const uint32_t ooff = (uint32_t)oa.base + tc_digits(pC, oa, pC.n_nd, pC.m_nd, mm) + tc_digits(pC, oa, pC.n_nd + pC.m_nd, pC.b_nd, (uint32_t)batch);
      __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(oa.ptr) + ooff;
      for (int c0 = half * (D >> 1); c0 < (half + 1) * (D >> 1); c0 += 32) {
        uint32_t raw[32];
        tc_ld32_issue(t_row + q.o_col + c0, raw);
        tc_ld_wait32(raw);
        if (row_ok) {
#pragma unroll
          for (int pc = 0; pc < 4; ++pc) {
            uint32_t w[4];
#pragma unroll
            for (int h = 0; h < 4; ++h) {
              __nv_bfloat162 b = __floats2bfloat162_rn(__uint_as_float(raw[pc * 8 + 2 * h]) * inv_sum, __uint_as_float(raw[pc * 8 + 2 * h + 1]) * inv_sum);
              w[h] = *reinterpret_cast<uint32_t*>(&b);
            }
            *reinterpret_cast<uint4*>(dst + c0 + pc * 8) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
    }
  }

  // ---------------- teardown ----------------
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0 && pA.status) { atomicExch(&pA.status[0], DNNF_ERR_TIMEOUT); atomicExch(&pA.status[1], pA.block_index); }
    // give copies that are still in flight time to land before shared memory is released
    if (threadIdx.x == 0) { long long t0 = clock64(); while (clock64() - t0 < 2000000) {} }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)q.tmem_cols) : "memory");
  }
}

}  // namespace attn

// ---- host side --------------------------------------------------------------------------------------
namespace {
struct AttnBlob { GemmParams a, c; attn::Params q; };
AttnBlob& ab_of(Launch& L) { return *reinterpret_cast<AttnBlob*>(L.blob.data()); }
const AttnBlob& ab_of(const Launch& L) { return *reinterpret_cast<const AttnBlob*>(L.blob.data()); }
const GemmParams& gemm_of(const Launch& L) { return *reinterpret_cast<const GemmParams*>(L.blob.data()); }

// dims innermost first: {inner, rows, b0, b1}; a batch digit the operand is broadcast over gets extent 1
bool encode4(CUtensorMap* tm, void* base, int64_t ext_inner, int64_t ext_rows, int64_t row_stride, const int32_t* bext, const int64_t* bstride,
             int box_inner, int box_rows, std::string& err) {
  cuuint64_t dims[4] = {(cuuint64_t)ext_inner, (cuuint64_t)ext_rows, (cuuint64_t)bext[0], (cuuint64_t)bext[1]};
  cuuint64_t s1 = (cuuint64_t)row_stride * 2;
  cuuint64_t s2 = bstride[0] ? (cuuint64_t)bstride[0] * 2 : s1 * ext_rows;
  cuuint64_t s3 = bstride[1] ? (cuuint64_t)bstride[1] * 2 : s2 * bext[0];
  if (!bstride[0]) dims[2] = 1;
  if (!bstride[1]) dims[3] = 1;
  cuuint64_t strides[3] = {s1, s2, s3};
  cuuint32_t box[4] = {(cuuint32_t)box_inner, (cuuint32_t)box_rows, 1, 1};
  return tma_encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B, err);
}
}  // namespace

// MatMul -> [MulC] -> [Add mask] -> Softmax -> MatMul, with index-only operators on the operands and behind the
// second product.  `ops` is the union of the three blocks of the normal plan, in topological order.
int lower_attention(const Graph& g, const std::vector<int>& ops, uint32_t flags, Block& out, std::string& why) {
  std::vector<int> anchors;
  for (int o : ops) { const int k = g.ops[o].kind; if (is_row_anchor(k) || is_contraction(k)) anchors.push_back(o); }
  if (anchors.size() != 3 || g.ops[anchors[0]].kind != DNNF_OP_MATMUL || g.ops[anchors[1]].kind != DNNF_OP_SOFTMAX ||
      g.ops[anchors[2]].kind != DNNF_OP_MATMUL) { why = "not a MatMul - Softmax - MatMul block"; return DNNF_ERR_UNSUPPORTED_OP; }
  const Op& SM = g.ops[anchors[1]];
  const Op& MM2 = g.ops[anchors[2]];
  const int t_scores = SM.in[0], t_prob = SM.out[0];
  if (MM2.in[0] != t_prob) { why = "the probabilities are not the left operand of the second product"; return DNNF_ERR_UNSUPPORTED_OP; }
  for (int t : {t_scores, t_prob}) {
    if (g.tensors[t].is_output || g.tensors[t].consumers.size() != 1) { why = "scores or probabilities are needed elsewhere"; return DNNF_ERR_UNSUPPORTED_OP; }
  }
  std::set<int> in_block(ops.begin(), ops.end());
  // the V side: index-only operators in front of the second product's right operand
  std::set<int> v_side;
  for (int t = MM2.in[1];;) { const int p = g.tensors[t].producer; if (p < 0 || !in_block.count(p)) break; v_side.insert(p); t = g.ops[p].in[0]; }
  std::vector<int> g1, g3;
  bool after_sm = false;
  for (int o : ops) {
    if (o == anchors[1]) { after_sm = true; continue; }
    if (v_side.count(o) || after_sm) g3.push_back(o); else g1.push_back(o);
  }
  Block bA, bC;
  int rc = lower_contraction(g, g1, flags, anchors[0], bA, why);
  if (rc != DNNF_OK) return rc;
  rc = lower_contraction(g, g3, flags, anchors[2], bC, why);
  if (rc != DNNF_OK) return rc;
  // any of the bf16 tensor-core kernels taking both products means: bf16 operands, 16-byte aligned strides
  auto tensor_core = [](int v) { return v == 1 || v == 3 || v == 5; };
  if (!tensor_core(bA.launch.variant) || !tensor_core(bC.launch.variant)) { why = "attention operands do not fit the tensor-core form"; return DNNF_ERR_UNSUPPORTED_OP; }
  const GemmParams& ga = gemm_of(bA.launch);
  const GemmParams& gc = gemm_of(bC.launch);
  auto refuse = [&](const char* m) { why = m; return DNNF_ERR_UNSUPPORTED_OP; };
  if (bA.launch.out_tensors.size() != 1 || bA.launch.out_tensors[0] != t_scores) return refuse("the first product's block stores something else than the scores");
  if (ga.batch_ext[0] != gc.batch_ext[0] || ga.batch_ext[1] != gc.batch_ext[1]) return refuse("batch layouts of the two products differ");
  if (gc.M != ga.M || gc.K != ga.N || gc.N != ga.K) return refuse("shapes of the two products do not chain");
  const int Sq = ga.M, Sk = ga.N, D = ga.K;
  if (D % 64 || D > 128 || Sk > 256 || Sk < 16 || Sk % 8) return refuse("head size or key count outside the single-kernel form");
  if (ga.A.stride_col != 1 || ga.B.stride_row != 1 || gc.B.stride_col != 1) return refuse("operand layouts outside the single-kernel form");
  if (ga.n_nd != 1 || gc.n_nd != 1 || gc.n_out != 1 || gc.n_in != 0) return refuse("index maps outside the single-kernel form");
  const TensorArg& oa = gc.out[0];
  if (oa.dtype != DNNF_BF16 || oa.stride[0] != 1 || !gc.vec_ok || oa.base % 8) return refuse("output is not bf16 with 16-byte aligned rows");
  for (int d = 1; d < gc.it.ndim; ++d) if (oa.stride[d] % 8) return refuse("output is not bf16 with 16-byte aligned rows");
  // the chains: [* c] [+ mask] behind the first product, nothing behind the second
  float scale = 1.0f; int mask_in = -1;
  {
    const Program& pr = ga.prog;
    int i = 0;
    if (pr.n < 2 || pr.ops[i].op != M_MOV || pr.ops[i].src != S_ANCHOR) return refuse("unexpected chain behind the first product");
    ++i;
    if (i < pr.n && pr.ops[i].op == M_MUL && pr.ops[i].src == S_CONST) { scale = pr.consts[pr.ops[i].idx]; ++i; }
    if (i < pr.n && pr.ops[i].op == M_ADD && pr.ops[i].src == S_IN) { mask_in = pr.ops[i].idx; ++i; }
    if (i >= pr.n || pr.ops[i].op != M_STORE) return refuse("unexpected chain behind the first product");
    ++i;
    if (i != pr.n && pr.ops[i].op != M_END) return refuse("unexpected chain behind the first product");
    if (ga.n_in != (mask_in >= 0 ? 1 : 0)) return refuse("unexpected operands behind the first product");
    const Program& pc = gc.prog;
    if (pc.n < 2 || pc.ops[0].op != M_MOV || pc.ops[0].src != S_ANCHOR || pc.ops[1].op != M_STORE || (pc.n > 2 && pc.ops[2].op != M_END))
      return refuse("operators behind the second product");
  }
  Launch& L = out.launch;
  L = Launch{};
  L.blob.assign(sizeof(AttnBlob), 0);
  AttnBlob& ab = ab_of(L);
  ab.a = ga; ab.c = gc;
  attn::Params& q = ab.q;
  q.Sq = Sq; q.Sk = Sk; q.D = D;
  q.sk16 = (Sk + 15) / 16 * 16;
  q.q_tiles = (Sq + attn::BM - 1) / attn::BM;
  q.mask_in = mask_in; q.scale = scale;
  q.o_col = (q.sk16 + 31) / 32 * 32;
  int cols = 32;
  while (cols < q.o_col + D) cols *= 2;
  q.tmem_cols = cols;
  for (int i = 0; i < 2; ++i) {
    q.q_batch[i] = ga.A.batch_stride[i] != 0; q.k_batch[i] = ga.B.batch_stride[i] != 0; q.v_batch[i] = gc.B.batch_stride[i] != 0;
  }
  const int d_tiles = D / 64, s_tiles = (q.sk16 + 63) / 64;
  q.off_k = d_tiles * attn::BM * 128;
  q.off_v = (q.off_k + d_tiles * q.sk16 * 128 + 1023) / 1024 * 1024;
  q.off_p = q.off_v + s_tiles * d_tiles * 8192;
  q.off_bar = q.off_p + s_tiles * attn::BM * 128;
  q.fd_qtiles = make_fastdiv((uint32_t)q.q_tiles);
  q.fd_b0 = make_fastdiv((uint32_t)ga.batch_ext[0]);
  size_t smem = (size_t)q.off_bar + 128 + 4 * attn::BM * 4;        // barriers, the halves' exchange area
  if (smem + 1024 > (size_t)attn::kSmemMax) return refuse("head does not fit shared memory");
  // the mask tile goes to shared memory when it is fp32 with unit column stride, one row digit, 16-byte aligned rows, and fits
  q.off_mask = -1; q.mask_pitch4 = 8; q.mask_static = 0;
  if (mask_in >= 0) {
    const TensorArg& ma = ga.in[mask_in];
    bool ok4 = ma.dtype == DNNF_F32 && ma.stride[0] == 1 && ga.m_nd == 1 && ma.base % 4 == 0 && Sk % 4 == 0;
    for (int d = 1; d < ga.it.ndim; ++d) if (ma.stride[d] % 4) ok4 = false;
    const int pitch4 = (q.sk16 + 31) / 32 * 8;
    const size_t bytes = (size_t)attn::BM * pitch4 * 16;
    if (ok4 && smem + bytes + 1024 <= (size_t)attn::kSmemMax) {
      q.off_mask = (int32_t)smem; q.mask_pitch4 = pitch4; smem += bytes;
      q.mask_static = (ga.static_mask >> (1 + mask_in)) & 1u;
    }
  }
  q.fd_pitch4 = make_fastdiv((uint32_t)q.mask_pitch4);
  L.smem = smem + 1024;                                              // alignment slack
  const int64_t nbatch = (int64_t)ga.batch_ext[0] * ga.batch_ext[1];
  if (nbatch * q.q_tiles >= (1ll << 31)) return refuse("too many tiles");
  L.grid = (int)(nbatch * q.q_tiles);
  L.threads = attn::THREADS;
  L.family = DNNF_FAMILY_ATTENTION;
  L.variant = 0;
  L.flops = bA.launch.flops + bC.launch.flops;
  L.ew.prog = ga.prog;                 // introspection (dnnf_block_program): the chain in front of the softmax
  // tensors: Q, K, [mask], V in; the second product's result out
  L.in_tensors = bA.launch.in_tensors;
  L.in_tensors.push_back(bC.launch.in_tensors[1]);
  L.out_tensors = bC.launch.out_tensors;
  out.inputs.clear();
  for (int t : L.in_tensors) if (std::find(out.inputs.begin(), out.inputs.end(), t) == out.inputs.end()) out.inputs.push_back(t);
  out.outputs = L.out_tensors;
  out.lowered = true;
  return DNNF_OK;
}

void attention_patch(Launch& L, const std::vector<void*>& ip, const std::vector<void*>& op, std::string& err) {
  AttnBlob& ab = ab_of(L);
  std::vector<void*> now(ip);
  now.insert(now.end(), op.begin(), op.end());
  if (L.tc_ready && now == L.encoded_ptrs) return;
  L.tc_ready = false;
  ab.a.A.ptr = ip[0]; ab.a.B.ptr = ip[1];
  for (int i = 0; i < ab.a.n_in; ++i) ab.a.in[i].ptr = ip[2 + i];
  ab.c.B.ptr = ip[2 + ab.a.n_in];
  ab.c.out[0].ptr = op[0];
  const attn::Params& q = ab.q;
  uint16_t* qp = reinterpret_cast<uint16_t*>(ab.a.A.ptr) + ab.a.A.base;
  uint16_t* kp = reinterpret_cast<uint16_t*>(ab.a.B.ptr) + ab.a.B.base;
  uint16_t* vp = reinterpret_cast<uint16_t*>(ab.c.B.ptr) + ab.c.B.base;
  if (((uintptr_t)qp & 15) || ((uintptr_t)kp & 15) || ((uintptr_t)vp & 15) || ((uintptr_t)op[0] & 15)) { err = "attention operand is not 16-byte aligned"; return; }
  if (!encode4(&ab.q.tmQ, qp, q.D, q.Sq, ab.a.A.stride_row, ab.a.batch_ext, ab.a.A.batch_stride, 64, attn::BM, err)) return;
  if (!encode4(&ab.q.tmK, kp, q.D, q.Sk, ab.a.B.stride_col, ab.a.batch_ext, ab.a.B.batch_stride, 64, q.sk16, err)) return;
  if (!encode4(&ab.q.tmV, vp, q.D, q.Sk, ab.c.B.stride_row, ab.c.batch_ext, ab.c.B.batch_stride, 64, 64, err)) return;
  L.tc_ready = true;
  L.encoded_ptrs = now;
}

int attention_launch(const Launch& L, void* status_words, int block_index, cudaStream_t st) {
  if (!L.tc_ready) return 1;
  Launch& M = const_cast<Launch&>(L);
  ab_of(M).a.status = reinterpret_cast<int32_t*>(status_words);
  ab_of(M).a.block_index = block_index;
  const AttnBlob& ab = ab_of(L);
  cudaError_t rc = cudaSuccess;
  auto go = [&](auto kernel, PerDeviceOnce& once) {
    if (once.first_use()) cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, attn::kSmemMax);
    rc = launch_pdl(kernel, dim3(L.grid), dim3(attn::THREADS), L.smem, st, ab.a, ab.c, ab.q);
  };
  static PerDeviceOnce once1, once2, once3, once4;
  // columns per thread: two threads share a row, each takes NC chunks of 32 keys
  const int nc = (ab.q.sk16 + 63) / 64;
  if (nc <= 1) go(attn::attention_kernel<1>, once1);
  else if (nc == 2) go(attn::attention_kernel<2>, once2);
  else if (nc == 3) go(attn::attention_kernel<3>, once3);
  else go(attn::attention_kernel<4>, once4);
  return (rc == cudaSuccess && cudaGetLastError() == cudaSuccess) ? 0 : 1;
}

}  // namespace dnnf
