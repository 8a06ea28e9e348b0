// dnnf_run: resolve device pointers and launch one kernel per block on the
// caller's stream.  Nothing here allocates or synchronises.
#include <cuda_runtime.h>

#include <algorithm>
#include <map>

#include "ir.h"
#include "tc_common.cuh"

namespace dnnf {

int launch_ew(const Launch& L, cudaStream_t st);
int launch_row(const Launch& L, cudaStream_t st);
int launch_contraction(const Launch& L, void* status_words, int block_index, cudaStream_t st, std::string& err);
void patch_contraction(Launch& L, const std::vector<void*>& in_ptrs, const std::vector<void*>& out_ptrs, std::string& err);

static void* resolve(Graph& g, int t) {
  while (g.tensors[t].alias_of >= 0) t = g.tensors[t].alias_of;
  Tensor& T = g.tensors[t];
  if (T.external || T.is_output) return T.bound;
  if (T.ws_offset < 0 || !g.ws_ptr) return nullptr;
  return (char*)g.ws_ptr + T.ws_offset;
}

int run_blocks(Graph& g, int only, void* stream) {
  if (!g.planned) { g.err = "graph is not planned (or the plan is not runnable)"; return DNNF_ERR_STATE; }
  if (g.ws_bytes > 256 && !g.ws_ptr) { g.err = "workspace not bound"; return DNNF_ERR_WORKSPACE; }
  cudaStream_t st = (cudaStream_t)stream;
  g.last_status_base = g.ws_ptr;
  // Resolve every pointer first so that a failure launches nothing.
  for (int bi : g.run_order) {
    if (only >= 0 && bi != only) continue;
    Block& b = g.blocks[bi];
    Launch& L = b.launch;
    if (L.family == DNNF_FAMILY_ALIAS) continue;
    std::vector<void*> ip, op;
    for (int t : L.in_tensors) { void* p = resolve(g, t); if (!p) { g.err = "tensor '" + g.tensors[t].name + "' is not bound"; return DNNF_ERR_UNBOUND; } ip.push_back(p); }
    for (int t : L.out_tensors) { void* p = resolve(g, t); if (!p) { g.err = "output tensor is not bound"; return DNNF_ERR_UNBOUND; } op.push_back(p); }
    if (L.family == DNNF_FAMILY_ROW) {
      for (size_t i = 0; i < ip.size(); ++i) L.row.in[i].ptr = ip[i];
      for (size_t i = 0; i < op.size(); ++i) L.row.out[i].ptr = op[i];
    } else if (L.family == DNNF_FAMILY_ELEMENTWISE || L.family == DNNF_FAMILY_TRANSPOSE) {
      for (size_t i = 0; i < ip.size(); ++i) L.ew.in[i].ptr = ip[i];
      for (size_t i = 0; i < op.size(); ++i) L.ew.out[i].ptr = op[i];
    } else {
      std::string err;
      patch_contraction(L, ip, op, err);
      if (!err.empty()) { g.err = err; return DNNF_ERR_CUDA; }
    }
  }
  for (int bi : g.run_order) {
    if (only >= 0 && bi != only) continue;
    Block& b = g.blocks[bi];
    Launch& L = b.launch;
    int rc = 0;
    switch (L.family) {
      case DNNF_FAMILY_ALIAS: break;
      case DNNF_FAMILY_ELEMENTWISE: case DNNF_FAMILY_TRANSPOSE: rc = launch_ew(L, st); break;
      case DNNF_FAMILY_ROW: rc = launch_row(L, st); break;
      default: { std::string err; rc = launch_contraction(L, g.ws_ptr, bi, st, err); if (rc) g.err = err; break; }
    }
    if (rc) {
      if (g.err.empty()) g.err = "kernel launch failed";
      g.err += std::string(" (") + cudaGetErrorString(cudaGetLastError()) + ")";
      return DNNF_ERR_CUDA;
    }
  }
  return DNNF_OK;
}

// Fills the profiling database: every candidate block the last plan asked about and did not find is lowered
// again, given device memory from the caller's scratch area, launched and timed with CUDA events.
int profile_measure(Graph& g, void* scratch, size_t scratch_bytes, void* stream, int iters, int* n_measured) {
  cudaStream_t st = (cudaStream_t)stream;
  if (n_measured) *n_measured = 0;
  if (!scratch || ((uintptr_t)scratch & 255)) { g.err = "scratch must be non-null and 256-byte aligned"; return DNNF_ERR_INVALID_ARG; }
  if (iters < 1) iters = 1;
  cudaEvent_t e0, e1;
  if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) { g.err = "cannot create events"; return DNNF_ERR_CUDA; }
  int rc_all = DNNF_OK, done = 0;
  for (const ProfileMiss& miss : g.profile_misses) {
    Block b; std::string why;
    if (lower_block(g, miss.ops, g.plan_flags, b, why) != DNNF_OK) continue;
    b.ops = miss.ops;
    Launch& L = b.launch;
    if (L.family == DNNF_FAMILY_ALIAS) continue;
    // arena: status words, arrival counters (both zero), the block's tensors, the kernel's own scratch
    size_t off = 256;
    if (L.counter_bytes > 0) { L.counter_off = (int64_t)off; off += (size_t)(L.counter_bytes + 255) / 256 * 256; }
    const size_t zero_bytes = off;
    std::map<int, size_t> place;
    auto put = [&](int t) { if (!place.count(t)) { place[t] = off; off += ((size_t)g.tensors[t].bytes() + 255) / 256 * 256; } };
    for (int t : L.in_tensors) put(t);
    for (int t : L.out_tensors) put(t);
    if (L.scratch_bytes > 0) { L.scratch_off = (int64_t)off; off += (size_t)(L.scratch_bytes + 255) / 256 * 256; }
    if (off > scratch_bytes) continue;                       // does not fit: stays a miss
    std::vector<void*> ip, op;
    for (int t : L.in_tensors) ip.push_back((char*)scratch + place[t]);
    for (int t : L.out_tensors) op.push_back((char*)scratch + place[t]);
    if (L.family == DNNF_FAMILY_ROW) {
      for (size_t i = 0; i < ip.size(); ++i) L.row.in[i].ptr = ip[i];
      for (size_t i = 0; i < op.size(); ++i) L.row.out[i].ptr = op[i];
    } else if (L.family == DNNF_FAMILY_ELEMENTWISE || L.family == DNNF_FAMILY_TRANSPOSE) {
      for (size_t i = 0; i < ip.size(); ++i) L.ew.in[i].ptr = ip[i];
      for (size_t i = 0; i < op.size(); ++i) L.ew.out[i].ptr = op[i];
    } else {
      std::string err;
      patch_contraction(L, ip, op, err);
      if (!err.empty()) continue;
    }
    if (cudaMemsetAsync(scratch, 0, zero_bytes, st) != cudaSuccess) { rc_all = DNNF_ERR_CUDA; break; }
    auto launch = [&]() -> int {
      switch (L.family) {
        case DNNF_FAMILY_ELEMENTWISE: case DNNF_FAMILY_TRANSPOSE: return launch_ew(L, st);
        case DNNF_FAMILY_ROW: return launch_row(L, st);
        default: { std::string err; return launch_contraction(L, scratch, -1, st, err); }
      }
    };
    bool ok = true;
    for (int i = 0; i < 2 && ok; ++i) ok = launch() == 0;
    // `iters` launches back to back between two events (what a graph of blocks looks like to the GPU: the next
    // launch is queued while this one runs), three times; the best per-launch time is kept.
    std::vector<float> ms;
    for (int rep = 0; rep < 3 && ok; ++rep) {
      cudaEventRecord(e0, st);
      for (int i = 0; i < iters && ok; ++i) ok = launch() == 0;
      cudaEventRecord(e1, st);
      if (cudaEventSynchronize(e1) != cudaSuccess) { ok = false; break; }
      float t = 0.f;
      cudaEventElapsedTime(&t, e0, e1);
      ms.push_back(t / (float)iters);
    }
    if (!ok || ms.empty()) { cudaGetLastError(); continue; }
    std::sort(ms.begin(), ms.end());
    profile_db_set(miss.signature, (double)ms[0] * 1000.0);
    ++done;
  }
  cudaStreamSynchronize(st);
  cudaEventDestroy(e0); cudaEventDestroy(e1);
  if (n_measured) *n_measured = done;
  if (rc_all != DNNF_OK) g.err = "profiling run failed";
  return rc_all;
}

// Self-test of the bounded waits: one CTA waits, with the kernels' own wait routine, on a barrier that nothing will
// ever signal.  The wait has to give up after `limit_ns`, raise the CTA's abort flag and come back; the kernel then
// records DNNF_ERR_TIMEOUT in the status words the way every tensor-core kernel's tear-down does.  Nothing faults and
// nothing hangs: this is the path a lost TMA completion or a missing commit would take.
__global__ void wait_expiry_kernel(int32_t* status, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  bool ok = true;
  if (threadIdx.x == 0) ok = mbar_wait(&bar, 0, &abort_flag, limit_ns);
  __syncthreads();
  if (threadIdx.x == 0 && abort_flag && !ok && status) { atomicExch(&status[0], DNNF_ERR_TIMEOUT); atomicExch(&status[1], -2); }
}

int selftest_wait_expiry(Graph& g, unsigned long long limit_ns, void* stream) {
  if (!g.ws_ptr) { g.err = "bind a workspace first: the status words live in it"; return DNNF_ERR_WORKSPACE; }
  if (limit_ns == 0 || limit_ns > 100000000ull) { g.err = "limit must be between 1 ns and 100 ms"; return DNNF_ERR_INVALID_ARG; }
  g.last_status_base = g.ws_ptr;
  wait_expiry_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(reinterpret_cast<int32_t*>(g.ws_ptr), limit_ns);
  if (cudaGetLastError() != cudaSuccess) { g.err = "self-test launch failed"; return DNNF_ERR_CUDA; }
  return DNNF_OK;
}

int read_status(Graph& g, int* status, int* block) {
  *status = 0;
  if (block) *block = -1;
  void* base = g.last_status_base ? g.last_status_base : g.ws_ptr;
  if (!base) return DNNF_OK;
  int words[2] = {0, 0};
  if (cudaMemcpy(words, base, sizeof words, cudaMemcpyDeviceToHost) != cudaSuccess) { g.err = "status read failed"; return DNNF_ERR_CUDA; }
  *status = words[0];
  if (block) *block = words[0] ? words[1] : -1;
  return DNNF_OK;
}

}  // namespace dnnf
