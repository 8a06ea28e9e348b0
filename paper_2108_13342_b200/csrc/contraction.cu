// Contraction-anchored blocks: lowering (host) and the CUDA-core fallback kernel.
//
// A Many-to-Many anchor that is a dense contraction (MatMul, pointwise convolution)
// keeps its result in the accumulator and runs the block's One-to-One successors on
// it before anything is stored ("the output elements of GEMM are mapped to the
// destination decided by the [fused] operator", Section 4.4).  Reorganize / Shuffle /
// Slice operators in front of the anchor become operand strides; behind it they become
// the store's index map.  Arithmetic in FRONT of the anchor is refused: it would have
// to be recomputed per output tile (the constraint check of Listing 1, Step 2.2).
#include <cuda_runtime.h>

#include <algorithm>
#include <cstring>

#include "chain.cuh"
#include "gemm_params.h"
#include "lower.h"

namespace dnnf {

bool tc_gemm_eligible(const GemmParams& gp);
bool tc_gemm_prepare(Launch& L, std::string& err);                  // encode tensor maps after pointers are known
int tc_gemm_launch(const Launch& L, cudaStream_t st);
void tc_gemm_plan(Launch& L);                                        // choose tiles / grid
size_t tc2_blob_bytes();
bool tc2_gemm_eligible(const GemmParams& gp);
void tc2_gemm_plan(Launch& L);
bool tc2_gemm_prepare(Launch& L, std::string& err);
int tc2_gemm_launch(const Launch& L, cudaStream_t st);
void tc2_set_scratch(Launch& L, void* ws_base);
size_t tile_blob_bytes();
bool tile_gemm_eligible(const GemmParams& gp);
bool tile_gemm_preferred(const GemmParams& gp);
void tile_gemm_plan(Launch& L);
bool tile_gemm_prepare(Launch& L, std::string& err);
int tile_gemm_launch(const Launch& L, cudaStream_t st);
void attention_patch(Launch& L, const std::vector<void*>& ip, const std::vector<void*>& op, std::string& err);
void mbconv_patch(Launch& L, const std::vector<void*>& ip, const std::vector<void*>& op);
int mbconv_launch(const Launch& L, cudaStream_t st);
int attention_launch(const Launch& L, void* status_words, int block_index, cudaStream_t st);
size_t tf32_blob_bytes();
bool tf32_gemm_eligible(const GemmParams& gp);
void tf32_gemm_plan(Launch& L);
bool tf32_gemm_prepare(Launch& L, std::string& err);
int tf32_gemm_launch(const Launch& L, cudaStream_t st);
bool conv_small_eligible(const GemmParams& gp);
void conv_small_plan(Launch& L);
int conv_small_launch(const Launch& L, cudaStream_t st);
bool conv1x1_direct_eligible(const GemmParams& gp);
void conv1x1_direct_plan(Launch& L);
int conv1x1_direct_launch(const Launch& L, cudaStream_t st);
int lower_dwconv(const Graph& g, const std::vector<int>& ops, int anchor, Block& out, std::string& why);
int dwconv_launch(const Launch& L, void* status_words, int block_index, cudaStream_t st);
void dwconv_patch(Launch& L, const std::vector<void*>& ip, const std::vector<void*>& op, std::string& err);
int lower_gather(const Graph& g, const std::vector<int>& ops, int anchor, Block& out, std::string& why);
int gather_launch(const Launch& L, cudaStream_t st);
void gather_patch(Launch& L, const std::vector<void*>& ip, const std::vector<void*>& op);
int lower_pool(const Graph& g, const std::vector<int>& ops, int anchor, Block& out, std::string& why);
int lower_instnorm(const Graph& g, const std::vector<int>& ops, int anchor, Block& out, std::string& why);
int instnorm_launch(const Launch& L, cudaStream_t st);
void instnorm_patch(Launch& L, const std::vector<void*>& ip, const std::vector<void*>& op);
int pool_launch(const Launch& L, void* ws_base, cudaStream_t st);
void pool_patch(Launch& L, const std::vector<void*>& ip, const std::vector<void*>& op);

static GemmParams& gp_of(Launch& L) { return *reinterpret_cast<GemmParams*>(L.blob.data()); }
static const GemmParams& gp_of(const Launch& L) { return *reinterpret_cast<const GemmParams*>(L.blob.data()); }

// ---------------------------------------------------------------------------
// Fallback kernel: 64x64 tile, 256 threads, 4x4 outputs per thread, fp32 FMA.
// Handles any dtype and any operand strides; used when the tensor-core path's
// alignment rules do not hold (and for fp32 MatMul).
// ---------------------------------------------------------------------------
constexpr int FB_T = 64, FB_K = 32;

__device__ __forceinline__ float ld_operand(const GemmOperand& o, int64_t off) {
  if (o.dtype == 0) return __ldg(reinterpret_cast<const float*>(o.ptr) + off);
  return bf16_bits_to_float(__ldg(reinterpret_cast<const uint16_t*>(o.ptr) + off));
}

struct FbEpiIO {
  const GemmParams& p;
  const float* accrow;       // 4 accumulators of this row
  uint32_t row_off_in[kMaxIn], row_off_out[kMaxOut];   // batch + m digits already folded in
  uint32_t n0;               // first column
  int ncols;                 // valid columns (1..4)
  __device__ __forceinline__ uint32_t n_offset(const TensorArg& a, uint32_t n) const {
    uint32_t off = 0, lin = n;
#pragma unroll
    for (int d = 0; d < 3; ++d) {
      if (d < p.n_nd) {
        uint32_t e = p.it.extent[d];
        uint32_t q = (d == p.n_nd - 1) ? 0u : lin / e;
        uint32_t c = (d == p.n_nd - 1) ? lin : lin - q * e;
        off += c * (uint32_t)a.stride[d];
        lin = q;
      }
    }
    return off;
  }
  __device__ __forceinline__ void load(int idx, float (&dst)[4]) const {
    const TensorArg& a = p.in[idx];
#pragma unroll
    for (int v = 0; v < 4; ++v) dst[v] = v < ncols ? load_scalar<false>(a, (uint32_t)a.base + row_off_in[idx] + n_offset(a, n0 + v)) : 0.0f;
  }
  __device__ __forceinline__ void anchor(float (&dst)[4]) const {
#pragma unroll
    for (int v = 0; v < 4; ++v) dst[v] = accrow[v];
  }
  __device__ __forceinline__ void store(int idx, const float (&val)[4]) const {
    const TensorArg& a = p.out[idx];
#pragma unroll
    for (int v = 0; v < 4; ++v)
      if (v < ncols) store_scalar<false>(a, (uint32_t)a.base + row_off_out[idx] + n_offset(a, n0 + v), val[v], false);
  }
  __device__ __forceinline__ void row_reduce(int, float (&)[4]) const {}
};

__device__ __forceinline__ uint32_t digits_offset(const GemmParams& p, const TensorArg& a, int first, int count, uint32_t lin) {
  uint32_t off = 0;
  for (int d = first; d < first + count; ++d) {
    uint32_t e = p.it.extent[d];
    uint32_t q = (d == first + count - 1) ? 0u : lin / e;
    uint32_t c = (d == first + count - 1) ? lin : lin - q * e;
    off += c * (uint32_t)a.stride[d];
    lin = q;
  }
  return off;
}

__global__ void __launch_bounds__(256) gemm_fallback_kernel(const __grid_constant__ GemmParams p) {
  __shared__ float As[FB_K][FB_T + 1];
  __shared__ float Bs[FB_K][FB_T + 1];
  pdl_launch_dependents();
  pdl_wait();
  const int tile_n = blockIdx.x % p.tiles_n, tile_m = blockIdx.x / p.tiles_n;
  const int batch = blockIdx.y;
  const int b0 = batch % p.batch_ext[0], b1 = batch / p.batch_ext[0];
  const int64_t a_base = p.A.base + b0 * p.A.batch_stride[0] + b1 * p.A.batch_stride[1];
  const int64_t b_base = p.B.base + b0 * p.B.batch_stride[0] + b1 * p.B.batch_stride[1];
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < p.K; k0 += FB_K) {
    // All of a chunk's loads are issued before the first store to shared memory (the operand pointers are generic,
    // so a load placed after a store would have to wait for it): small problems are bound by this latency.
    constexpr int kLoads = FB_T * FB_K / 256;
    float va[kLoads], vb[kLoads];
#pragma unroll
    for (int u = 0; u < kLoads; ++u) {
      const int i = threadIdx.x + u * 256;
      int kk, mm;
      if (p.A.stride_col == 1) { kk = i % FB_K; mm = i / FB_K; } else { mm = i % FB_T; kk = i / FB_T; }
      int m = tile_m * FB_T + mm, k = k0 + kk;
      va[u] = (m < p.M && k < p.K) ? ld_operand(p.A, a_base + (int64_t)m * p.A.stride_row + (int64_t)k * p.A.stride_col) : 0.0f;
      int nn;
      if (p.B.stride_col == 1) { nn = i % FB_T; kk = i / FB_T; } else { kk = i % FB_K; nn = i / FB_K; }
      int n = tile_n * FB_T + nn; k = k0 + kk;
      vb[u] = (n < p.N && k < p.K) ? ld_operand(p.B, b_base + (int64_t)k * p.B.stride_row + (int64_t)n * p.B.stride_col) : 0.0f;
    }
#pragma unroll
    for (int u = 0; u < kLoads; ++u) {
      const int i = threadIdx.x + u * 256;
      int kk, mm, nn;
      if (p.A.stride_col == 1) { kk = i % FB_K; mm = i / FB_K; } else { mm = i % FB_T; kk = i / FB_T; }
      As[kk][mm] = va[u];
      if (p.B.stride_col == 1) { nn = i % FB_T; kk = i / FB_T; } else { kk = i % FB_K; nn = i / FB_K; }
      Bs[kk][nn] = vb[u];
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < FB_K; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[kk][ty * 4 + i]; b[i] = Bs[kk][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
  FbEpiIO io{p};
  io.n0 = tile_n * FB_T + tx * 4;
  if ((int)io.n0 >= p.N) return;
  io.ncols = min(4, p.N - (int)io.n0);
  for (int i = 0; i < 4; ++i) {
    int m = tile_m * FB_T + ty * 4 + i;
    if (m >= p.M) break;
    for (int k = 0; k < p.n_in; ++k)
      io.row_off_in[k] = digits_offset(p, p.in[k], p.n_nd, p.m_nd, (uint32_t)m) + digits_offset(p, p.in[k], p.n_nd + p.m_nd, p.b_nd, (uint32_t)batch);
    for (int k = 0; k < p.n_out; ++k)
      io.row_off_out[k] = digits_offset(p, p.out[k], p.n_nd, p.m_nd, (uint32_t)m) + digits_offset(p, p.out[k], p.n_nd + p.m_nd, p.b_nd, (uint32_t)batch);
    io.accrow = acc[i];
    run_program<4, DynProg>(p.prog, io);
  }
}

// ---------------------------------------------------------------------------
// Lowering
// ---------------------------------------------------------------------------
namespace {

// Walk from a MatMul operand back through index-only operators of the block to the
// external tensor that is actually read; express it over the operand's own dims.
bool operand_view(const Graph& g, const std::set<int>& in_block, int tensor, std::vector<int64_t>& ext_out, int& src_tensor,
                  View& view, std::string& why) {
  LowerCtx cx(g);
  cx.in_block = in_block;
  cx.ext = g.tensors[tensor].dims;
  for (int iter = 0; iter < 16; ++iter) {
    cx.split = SplitRequest{};
    cx.why.clear();
    View v; v.coef = contiguous_strides(cx.ext);
    int t = tensor;
    bool ok = true;
    while (true) {
      int p = g.tensors[t].producer;
      if (p < 0 || !in_block.count(p)) break;
      const Op& op = g.ops[p];
      if (!is_index_only(op.kind)) { why = "arithmetic in front of a contraction anchor (no prologue fusion)"; return false; }
      std::vector<View> vin;
      if (!backward_views(cx, op, v, vin)) { ok = false; break; }
      v = vin[0];
      t = op.in[0];
    }
    if (ok) { ext_out = cx.ext; src_tensor = t; view = v; return true; }
    if (cx.split.dim < 0) { why = cx.why; return false; }
    int d = cx.split.dim; int64_t q = cx.split.inner;
    int64_t e = cx.ext[d];
    cx.ext[d] = e / q;
    cx.ext.insert(cx.ext.begin() + d + 1, q);
  }
  why = "operand refinement did not converge";
  return false;
}

// Map the refined dims of an operand view back onto (batch dims..., row, col): every
// original dim must stay a single refined dim for row/col; batch dims may be refined
// as long as at most two remain after dropping extent-1 dims.
bool pack_operand(const Graph& g, const std::vector<int64_t>& orig_dims, const std::vector<int64_t>& ext, int src, const View& v,
                  GemmOperand& o, std::vector<int64_t>& batch_exts, std::vector<int64_t>& batch_strides, std::string& why) {
  size_t r = orig_dims.size();
  // group refined dims by original dim
  std::vector<std::vector<int>> grp(r);
  size_t d = 0;
  for (size_t k = 0; k < r; ++k) {
    int64_t prod = 1;
    while (prod < orig_dims[k] || (d < ext.size() && ext[d] == 1 && prod == orig_dims[k] && grp[k].empty())) {
      if (d >= ext.size()) { why = "internal: refinement mismatch"; return false; }
      prod *= ext[d]; grp[k].push_back((int)d); ++d;
    }
    if (prod != orig_dims[k]) { why = "internal: refinement mismatch"; return false; }
  }
  auto single = [&](size_t k, int64_t& stride) {
    std::vector<int> nz;
    for (int x : grp[k]) if (ext[x] > 1) nz.push_back(x);
    if (nz.size() > 1) return false;
    stride = nz.empty() ? 0 : v.coef[nz[0]];
    return true;
  };
  if (!single(r - 2, o.stride_row) || !single(r - 1, o.stride_col)) { why = "contraction operand dim is split by a reshape"; return false; }
  // batch digits, outermost first, unmerged: the caller merges them jointly for both operands
  batch_exts.clear(); batch_strides.clear();
  for (size_t k = 0; k + 2 < r; ++k) for (int x : grp[k]) if (ext[x] > 1) { batch_exts.push_back(ext[x]); batch_strides.push_back(v.coef[x]); }
  o.batch_stride[0] = o.batch_stride[1] = 0;
  o.base = v.c0;
  o.dtype = g.tensors[src].dtype;
  o.ptr = nullptr;
  return true;
}

}  // namespace

// Up to this many rows an fp32 contraction goes to the one-tile-per-CTA kernel even where the tall-and-skinny tensor-core
// kernel would take it: that kernel has one 128-row tile per CTA and nothing to spread over the GPU.  (Where the
// tensor-core kernel does not apply, the one-tile-per-CTA kernel is taken up to 65536 rows.)
static int small_m_limit() { const char* e = dev_env("DNNF_SMALL_M"); return e ? atoi(e) : 1024; }

int lower_contraction(const Graph& g, const std::vector<int>& ops, uint32_t flags, int anchor, Block& out, std::string& why) {
  (void)flags;
  const Op& A = g.ops[anchor];
  if (A.kind == DNNF_OP_DWCONV3X3) return lower_dwconv(g, ops, anchor, out, why);
  if (A.kind == DNNF_OP_MAXPOOL || A.kind == DNNF_OP_AVGPOOL || A.kind == DNNF_OP_COL2IM) return lower_pool(g, ops, anchor, out, why);
  if (A.kind == DNNF_OP_INSTANCENORM) return lower_instnorm(g, ops, anchor, out, why);
  if (A.kind == DNNF_OP_GATHER) return lower_gather(g, ops, anchor, out, why);
  std::set<int> in_block(ops.begin(), ops.end());
  const Tensor& C = g.tensors[A.out[0]];
  const Tensor& TA = g.tensors[A.in[0]];
  const Tensor& TB = g.tensors[A.in[1]];

  Launch& L = out.launch;
  L = Launch{};
  L.blob.assign(sizeof(GemmParams) + sizeof(GemmTcParams) + std::max({tc2_blob_bytes(), tf32_blob_bytes(), tile_blob_bytes()}), 0);
  GemmParams& gp = gp_of(L);

  // ---- operands ----------------------------------------------------------------
  std::vector<int64_t> a_dims, b_dims, c_dims;
  if (A.kind == DNNF_OP_CONV1X1) {
    int64_t px = TA.dims[0] * TA.dims[1] * TA.dims[2];
    a_dims = {px, TA.dims[3]}; b_dims = TB.dims; c_dims = {px, TB.dims[1]};
  } else {
    a_dims = TA.dims; b_dims = TB.dims; c_dims = C.dims;
  }
  gp.M = (int)c_dims[c_dims.size() - 2]; gp.N = (int)c_dims.back(); gp.K = (int)a_dims.back();
  int srcA = -1, srcB = -1;
  View vA, vB;
  std::vector<int64_t> extA, extB, batchA, batchB;
  if (A.kind == DNNF_OP_CONV1X1) {
    // NHWC activations are already a [pixels, C] matrix
    if (in_block.count(TA.producer) || in_block.count(TB.producer)) { why = "operators in front of a convolution anchor"; return DNNF_ERR_UNSUPPORTED_OP; }
    srcA = A.in[0]; srcB = A.in[1];
    extA = a_dims; extB = b_dims;
    vA.coef = contiguous_strides(a_dims); vB.coef = contiguous_strides(b_dims);
  } else {
    if (!operand_view(g, in_block, A.in[0], extA, srcA, vA, why)) return DNNF_ERR_UNSUPPORTED_OP;
    if (!operand_view(g, in_block, A.in[1], extB, srcB, vB, why)) return DNNF_ERR_UNSUPPORTED_OP;
  }
  std::vector<int64_t> strA, strB;
  if (!pack_operand(g, a_dims, extA, srcA, vA, gp.A, batchA, strA, why)) return DNNF_ERR_UNSUPPORTED_OP;
  if (!pack_operand(g, b_dims, extB, srcB, vB, gp.B, batchB, strB, why)) return DNNF_ERR_UNSUPPORTED_OP;
  int64_t nbatch = 1;
  for (size_t k = 0; k + 2 < c_dims.size(); ++k) nbatch *= c_dims[k];
  // Batch digits (outermost first) come from whichever operand has them; the other either
  // has the same digits or none (broadcast).  Refine both to a common digit list.
  std::vector<int64_t> bext = batchA.empty() ? batchB : batchA;
  {
    int64_t p = 1;
    for (auto e : bext) p *= e;
    if (p != nbatch) { why = "batch layout of the operands does not match the result"; return DNNF_ERR_UNSUPPORTED_OP; }
  }
  auto conform = [&](std::vector<int64_t>& ex, std::vector<int64_t>& st) {
    if (ex.empty()) { st.assign(bext.size(), 0); ex = bext; return true; }
    if (ex == bext) return true;
    // split this operand's digits to match bext where bext is finer
    std::vector<int64_t> ne, ns;
    size_t j = 0;
    for (size_t i = 0; i < ex.size(); ++i) {
      int64_t rem = ex[i];
      std::vector<int64_t> part;
      while (rem > 1 && j < bext.size() && rem % bext[j] == 0) { part.push_back(bext[j]); rem /= bext[j]; ++j; }
      if (rem != 1) return false;
      int64_t mult = 1;
      for (auto e : part) mult *= e;
      for (auto e : part) { mult /= e; ne.push_back(e); ns.push_back(st[i] * mult); }
    }
    if (ne != bext) return false;
    ex = ne; st = ns;
    return true;
  };
  if (!conform(batchA, strA)) {
    // maybe A is the coarser one: use B's digits as the reference
    bext = batchB;
    batchA.clear(); strA.clear();
    std::vector<int64_t> tmp;
    if (!pack_operand(g, a_dims, extA, srcA, vA, gp.A, batchA, strA, why) || !conform(batchA, strA)) { why = "batch dims of the two operands differ"; return DNNF_ERR_UNSUPPORTED_OP; }
  }
  if (!conform(batchB, strB)) { why = "batch dims of the two operands differ"; return DNNF_ERR_UNSUPPORTED_OP; }
  // merge adjacent digits that are contiguous in both operands
  for (size_t i = 0; i + 1 < bext.size();) {
    if (strA[i] == strA[i + 1] * bext[i + 1] && strB[i] == strB[i + 1] * bext[i + 1]) {
      bext[i + 1] *= bext[i];
      bext.erase(bext.begin() + i); strA.erase(strA.begin() + i); strB.erase(strB.begin() + i);
    } else ++i;
  }
  if (bext.size() > 2) { why = "more than two batch dims"; return DNNF_ERR_UNSUPPORTED_OP; }
  for (size_t i = 0; i < bext.size(); ++i) {       // innermost batch digit is index 0
    gp.A.batch_stride[i] = strA[bext.size() - 1 - i];
    gp.B.batch_stride[i] = strB[bext.size() - 1 - i];
  }
  gp.batch_ext[0] = bext.size() > 0 ? (int)bext[bext.size() - 1] : 1;
  gp.batch_ext[1] = bext.size() > 1 ? (int)bext[0] : 1;
  // A weight shared by every batch and an activation whose batches follow each other row after row
  // is one tall 2-D GEMM: fold the batch dims into M (one wave of large tiles instead of many small ones).
  bool fold_batch = false;
  if (A.kind == DNNF_OP_MATMUL && nbatch > 1 && gp.B.batch_stride[0] == 0 && gp.B.batch_stride[1] == 0 &&
      gp.A.batch_stride[0] == (int64_t)gp.M * gp.A.stride_row &&
      (bext.size() < 2 || gp.A.batch_stride[1] == gp.batch_ext[0] * gp.A.batch_stride[0]) && (int64_t)gp.M * nbatch < (1ll << 31)) {
    fold_batch = true;
    gp.M = (int)(gp.M * nbatch);
    gp.batch_ext[0] = gp.batch_ext[1] = 1;
    gp.A.batch_stride[0] = gp.A.batch_stride[1] = 0;
  }

  // ---- epilogue ------------------------------------------------------------------
  LowerCtx cx(g);
  cx.ops = ops;
  cx.in_block = in_block;
  // operand-side index ops are not part of the epilogue walk
  std::vector<int> epi_ops;
  {
    std::set<int> operand_side;
    for (int s = 0; s < 2; ++s) {
      int t = A.in[s];
      while (true) { int p = g.tensors[t].producer; if (p < 0 || !in_block.count(p)) break; operand_side.insert(p); t = g.ops[p].in[0]; }
    }
    for (int o : ops) if (!operand_side.count(o)) epi_ops.push_back(o);
    for (int o : operand_side) {
      // an operand-side value must not be needed elsewhere in the block or outside it
      for (int t : g.ops[o].out) {
        if (g.tensors[t].is_output) { why = "operand-side intermediate is a graph output"; return DNNF_ERR_UNSUPPORTED_OP; }
        for (int c : g.tensors[t].consumers) if (!in_block.count(c)) { why = "operand-side intermediate has an outside consumer"; return DNNF_ERR_UNSUPPORTED_OP; }
      }
    }
  }
  cx.ops = epi_ops;
  cx.in_block = std::set<int>(epi_ops.begin(), epi_ops.end());
  cx.ext = C.dims;
  if (!derive_views(cx, A.out[0], {anchor})) { why = cx.why; return DNNF_ERR_UNSUPPORTED_OP; }
  if (!emit_program(cx, A.out[0], 2)) { why = cx.why; return DNNF_ERR_UNSUPPORTED_OP; }

  // group refined dims by C dim: [batch dims][m][n]
  std::vector<int> group(cx.ext.size(), 0);     // 0 batch, 1 m, 2 n
  {
    size_t d = 0;
    for (size_t k = 0; k < C.dims.size(); ++k) {
      int64_t p = 1;
      int gk;
      if (A.kind == DNNF_OP_CONV1X1) gk = k < 3 ? 1 : 2;
      else gk = k + 2 < C.dims.size() ? (fold_batch ? 1 : 0) : (k + 2 == C.dims.size() ? 1 : 2);
      bool first = true;
      while (p < C.dims[k] || (first && d < cx.ext.size() && cx.ext[d] == 1 && C.dims[k] == 1)) {
        if (d >= cx.ext.size()) { why = "internal: refinement mismatch"; return DNNF_ERR_UNSUPPORTED_OP; }
        p *= cx.ext[d]; group[d] = gk; ++d; first = false;
      }
    }
  }
  // collapse within groups
  struct Dim { int64_t e; int grp; std::vector<int64_t> coef; };
  std::vector<Dim> dims;
  size_t nargs = cx.ins.size() + cx.outs.size();
  auto coef_of = [&](size_t a, size_t d) { return a < cx.ins.size() ? cx.ins[a].view.coef[d] : cx.outs[a - cx.ins.size()].view.coef[d]; };
  for (size_t d = 0; d < cx.ext.size(); ++d) {
    if (cx.ext[d] == 1) continue;
    Dim x{cx.ext[d], group[d], {}};
    for (size_t a = 0; a < nargs; ++a) x.coef.push_back(coef_of(a, d));
    if (!dims.empty() && dims.back().grp == x.grp) {
      bool ok = true;
      for (size_t a = 0; a < nargs; ++a) if (dims.back().coef[a] != x.coef[a] * x.e) ok = false;
      if (ok) { dims.back().e *= x.e; dims.back().coef = x.coef; continue; }
    }
    dims.push_back(x);
  }
  int n_nd = 0, m_nd = 0, b_nd = 0;
  for (auto& x : dims) (x.grp == 2 ? n_nd : x.grp == 1 ? m_nd : b_nd)++;
  if (n_nd == 0) { dims.push_back({1, 2, std::vector<int64_t>(nargs, 0)}); n_nd = 1; }
  if (m_nd == 0) { dims.insert(dims.begin() + b_nd, Dim{1, 1, std::vector<int64_t>(nargs, 0)}); m_nd = 1; }
  if (b_nd == 0) { dims.insert(dims.begin(), Dim{1, 0, std::vector<int64_t>(nargs, 0)}); b_nd = 1; }
  if (n_nd > 3 || m_nd > 3 || (int)dims.size() > kMaxDims) { why = "epilogue index map has too many digits"; return DNNF_ERR_UNSUPPORTED_OP; }
  // the epilogue's batch digits must enumerate batches in the operands' (b1, b0) order: they do, both are row-major over C's batch dims
  int nd = (int)dims.size();
  gp.it.ndim = nd;
  gp.n_nd = n_nd; gp.m_nd = m_nd; gp.b_nd = b_nd;
  for (int d = 0; d < nd; ++d) gp.it.extent[d] = (uint32_t)dims[nd - 1 - d].e;       // innermost first
  set_fastdiv(gp.it);
  gp.n_in = (int)cx.ins.size(); gp.n_out = (int)cx.outs.size();
  bool vec_ok = true;
  auto fill = [&](TensorArg& a, const ExtArg& e, size_t ai) {
    a.ptr = nullptr; a.base = (int32_t)e.view.c0; a.dtype = g.tensors[e.tensor].dtype; a.mode = 0;
    for (int d = 0; d < kMaxDims; ++d) a.stride[d] = d < nd ? (int32_t)dims[nd - 1 - d].coef[ai] : 0;
    if (g.tensors[e.tensor].numel() >= (1ll << 31)) return false;
    bool is_out = ai >= cx.ins.size();
    // mode 1: the operand does not depend on the row or the batch (a bias vector)
    bool row_invariant = !is_out;
    for (int d = n_nd; d < nd; ++d) if (a.stride[d] != 0) row_invariant = false;
    a.mode = row_invariant ? 1 : 0;
    if (a.stride[0] != 1 && !(a.stride[0] == 0 && !is_out)) vec_ok = false;
    if (a.stride[0] == 1) { if (a.base % 8) vec_ok = false; for (int d = 1; d < nd; ++d) if (a.stride[d] % 8) vec_ok = false; }
    return true;
  };
  for (size_t i = 0; i < cx.ins.size(); ++i) if (!fill(gp.in[i], cx.ins[i], i)) { why = "tensor too large"; return DNNF_ERR_UNSUPPORTED_OP; }
  for (size_t i = 0; i < cx.outs.size(); ++i) if (!fill(gp.out[i], cx.outs[i], cx.ins.size() + i)) { why = "tensor too large"; return DNNF_ERR_UNSUPPORTED_OP; }
  if (gp.it.extent[0] % 8) vec_ok = false;
  gp.vec_ok = vec_ok;
  auto is_static = [&](int t) { return g.tensors[t].external && g.tensors[t].producer < 0 && !g.tensors[t].is_output; };
  gp.static_mask = is_static(srcB) ? 1u : 0u;
  for (size_t i = 0; i < cx.ins.size(); ++i) if (is_static(cx.ins[i].tensor)) gp.static_mask |= 2u << i;
  gp.prog = cx.prog;
  L.ew.prog = cx.prog;            // introspection (dnnf_block_program)

  out.inputs.clear(); out.outputs.clear();
  L.in_tensors = {srcA, srcB};
  out.inputs = {srcA, srcB};
  for (auto& a : cx.ins) { L.in_tensors.push_back(a.tensor); if (std::find(out.inputs.begin(), out.inputs.end(), a.tensor) == out.inputs.end()) out.inputs.push_back(a.tensor); }
  for (auto& a : cx.outs) { L.out_tensors.push_back(a.tensor); out.outputs.push_back(a.tensor); }
  L.flops = 2ll * gp.M * gp.N * gp.K * (fold_batch ? 1 : nbatch);
  L.family = A.kind == DNNF_OP_CONV1X1 ? DNNF_FAMILY_CONV1X1 : DNNF_FAMILY_GEMM;

  if (tile_gemm_eligible(gp) && (tile_gemm_preferred(gp) || !tc2_gemm_eligible(gp))) {
    tile_gemm_plan(L);
  } else if (tc2_gemm_eligible(gp)) {
    tc2_gemm_plan(L);
  } else if (tc_gemm_eligible(gp)) {
    L.variant = 1;
    tc_gemm_plan(L);
  } else if (conv_small_eligible(gp) && (gp.M <= small_m_limit() || !tf32_gemm_eligible(gp))) {
    conv_small_plan(L);
  } else if (tf32_gemm_eligible(gp)) {
    tf32_gemm_plan(L);
  } else if (A.kind == DNNF_OP_CONV1X1 && conv1x1_direct_eligible(gp)) {
    conv1x1_direct_plan(L);
  } else {
    L.variant = 0;
    gp.tiles_m = (gp.M + FB_T - 1) / FB_T; gp.tiles_n = (gp.N + FB_T - 1) / FB_T;
    L.grid = gp.tiles_m * gp.tiles_n; L.threads = 256;
  }
  out.lowered = true;
  return DNNF_OK;
}

void patch_contraction(Launch& L, const std::vector<void*>& ip, const std::vector<void*>& op, std::string& err) {
  if (L.family == DNNF_FAMILY_DWCONV) { dwconv_patch(L, ip, op, err); return; }
  if (L.family == DNNF_FAMILY_POOL) { pool_patch(L, ip, op); return; }
  if (L.family == DNNF_FAMILY_INSTNORM) { instnorm_patch(L, ip, op); return; }
  if (L.family == DNNF_FAMILY_GATHER) { gather_patch(L, ip, op); return; }
  if (L.family == DNNF_FAMILY_MBCONV) { mbconv_patch(L, ip, op); return; }
  if (L.family == DNNF_FAMILY_ATTENTION) { attention_patch(L, ip, op, err); if (!L.tc_ready && err.empty()) err = "cannot encode the tensor maps of an attention block"; return; }
  GemmParams& gp = gp_of(L);
  gp.A.ptr = ip[0]; gp.B.ptr = ip[1];
  for (int i = 0; i < gp.n_in; ++i) gp.in[i].ptr = ip[2 + i];
  for (int i = 0; i < gp.n_out; ++i) gp.out[i].ptr = op[i];
  if (L.variant != 1 && L.variant != 3 && L.variant != 4 && L.variant != 5) return;
  // The tensor maps embed addresses: encode them again whenever ANY pointer of the block differs from the
  // ones they were made for (an epilogue operand in any position may be read through a map).
  std::vector<void*> now(ip);
  now.insert(now.end(), op.begin(), op.end());
  if (L.tc_ready && now == L.encoded_ptrs) return;
  L.tc_ready = false;
  bool ok = L.variant == 1 ? tc_gemm_prepare(L, err) : L.variant == 3 ? tc2_gemm_prepare(L, err) : L.variant == 5 ? tile_gemm_prepare(L, err) : tf32_gemm_prepare(L, err);
  if (ok) { L.tc_ready = true; L.encoded_ptrs = now; }
  else if (err.empty()) err = "cannot encode the tensor maps of a contraction block";
}

int launch_contraction(const Launch& L, void* status_words, int block_index, cudaStream_t st, std::string& err) {
  if (L.family == DNNF_FAMILY_MBCONV) { int rc = mbconv_launch(L, st); if (rc) err = "inverted-residual block launch failed"; return rc; }
  if (L.family == DNNF_FAMILY_ATTENTION) { int rc = attention_launch(L, status_words, block_index, st); if (rc) err = "attention launch failed"; return rc; }
  if (L.family == DNNF_FAMILY_GATHER) { int rc = gather_launch(L, st); if (rc) err = "gather launch failed"; return rc; }
  if (L.family == DNNF_FAMILY_POOL) { int rc = pool_launch(L, status_words, st); if (rc) err = "pooling launch failed"; return rc; }
  if (L.family == DNNF_FAMILY_INSTNORM) { int rc = instnorm_launch(L, st); if (rc) err = "instance normalisation launch failed"; return rc; }
  if (L.family == DNNF_FAMILY_DWCONV) { int rc = dwconv_launch(L, status_words, block_index, st); if (rc) err = "depthwise convolution launch failed"; return rc; }
  if (L.variant == 2) { int rc = conv1x1_direct_launch(L, st); if (rc) err = "pointwise convolution launch failed"; return rc; }
  if (L.variant == 7) { int rc = conv_small_launch(L, st); if (rc) err = "pointwise convolution launch failed"; return rc; }
  if ((L.variant == 1 || L.variant == 3 || L.variant == 4 || L.variant == 5) && !L.tc_ready) { err = "tensor maps of the block are not encoded"; return 1; }
  GemmParams gp = gp_of(L);
  gp.status = reinterpret_cast<int32_t*>(status_words);
  gp.block_index = block_index;
  if (L.variant == 3) {
    Launch& M = const_cast<Launch&>(L);
    gp_of(M).status = gp.status; gp_of(M).block_index = block_index;
    tc2_set_scratch(M, status_words);
    int rc = tc2_gemm_launch(L, st);
    if (rc) err = "tensor-core pair GEMM launch failed";
    return rc;
  }
  if (L.variant == 5) {
    Launch& M = const_cast<Launch&>(L);
    gp_of(M).status = gp.status; gp_of(M).block_index = block_index;
    int rc = tile_gemm_launch(L, st);
    if (rc) err = "tensor-core tile GEMM launch failed";
    return rc;
  }
  if (L.variant == 4) {
    Launch& M = const_cast<Launch&>(L);
    gp_of(M).status = gp.status; gp_of(M).block_index = block_index;
    int rc = tf32_gemm_launch(L, st);
    if (rc) err = "tensor-core fp32 GEMM launch failed";
    return rc;
  }
  if (L.variant == 1) {
    Launch& M = const_cast<Launch&>(L);
    gp_of(M).status = gp.status; gp_of(M).block_index = block_index;
    int rc = tc_gemm_launch(L, st);
    if (rc) err = "tensor-core GEMM launch failed";
    return rc;
  }
  dim3 grid(L.grid, gp.batch_ext[0] * gp.batch_ext[1]);
  launch_pdl(gemm_fallback_kernel, grid, 256, 0, st, gp);
  if (cudaGetLastError() != cudaSuccess) { err = "fallback GEMM launch failed"; return 1; }
  return 0;
}

}  // namespace dnnf
