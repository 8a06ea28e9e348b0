// Extended Computational Graph (Section 3.2): operators, tensors, data-flow, plus
// mapping type per operator, IR_removable per tensor and mathematical-property
// flags; fusion blocks and their lowered launches.
#pragma once
#include <cstdlib>
#include <cstdint>
#include <map>
#include <string>
#include <vector>

#include "../../include/dnnf.h"
#include "microop.h"

namespace dnnf {

// Plan flags of the dnnf_plan call that is being served on this thread (kernel-selection overrides, see dnnf.h).
extern thread_local uint32_t tl_plan_flags;
inline bool plan_flag(uint32_t f) { return (tl_plan_flags & f) != 0; }

// Development switches: environment variables that tune or ablate a kernel.  They exist only in libraries built with
// -DDNNF_DEV_SWITCHES; a normal build never reads the environment.
inline const char* dev_env(const char* name) {
#ifdef DNNF_DEV_SWITCHES
  return getenv(name);
#else
  (void)name;
  return nullptr;
#endif
}

struct Attrs {
  double c = 0, lo = 0, hi = 0, p = 0, eps = 1e-5;
  int64_t approx = 0, axis = -1, keepdims = 1, start = 0, end = 0, bits = 0, block = 0, scale = 0, kernel = 0, stride = 1, pad = 0;
  int64_t to = 0, exclusive = 0, reverse = 0;
  std::vector<int64_t> perm, shape, sizes, axes;
};

struct Tensor {
  int id = -1;
  std::string name;
  int dtype = DNNF_F32;
  std::vector<int64_t> dims;
  bool external = false;       // declared by dnnf_add_tensor
  bool weight = false;
  bool is_output = false;      // marked by the caller
  int producer = -1;           // op id, -1 for externals
  std::vector<int> consumers;  // op ids (alive ops only; rebuilt by Graph::relink)
  bool removable = false;      // IR_removable: all consumers sit in the producer's block
  int64_t ws_offset = -1;      // workspace offset (bytes) when materialised between blocks
  int alias_of = -1;           // zero-copy Reorganize result: shares storage with this tensor
  void* bound = nullptr;       // caller-bound device pointer (externals and outputs)
  int64_t numel() const { int64_t n = 1; for (auto d : dims) n *= d; return n; }
  int64_t bytes() const { return numel() * (dtype == DNNF_BF16 ? 2 : 4); }
};

enum MathProp : uint32_t { P_ASSOC = 1, P_COMM = 2, P_DIST = 4 };

struct Op {
  int id = -1;
  int kind = 0;
  int source_id = -1;          // original operator this came from (a Split expands to Slices)
  std::vector<int> in, out;
  Attrs at;
  int mapping = DNNF_ONE_TO_ONE;
  uint32_t props = 0;
  bool alive = true;
  int block = -1;
};

// A lowered block = one kernel launch (or none for a zero-copy alias).
struct ArgRef { int tensor; };   // which tensor supplies TensorArg.ptr at bind time

struct GemmLaunch;   // defined in gemm_host.h
struct ConvLaunch;

struct Launch {
  int family = DNNF_FAMILY_ALIAS;
  int variant = 0;
  bool tc_ready = false;      // tensor maps encoded for the currently bound pointers
  std::vector<void*> encoded_ptrs;   // the pointers (operands, epilogue inputs, outputs) the tensor maps were encoded for
  int static_id = 0;          // compile-time program table the block runs on (0: interpreted)
  int grid = 0, threads = 0;
  size_t smem = 0;
  EwParams ew{};
  RowParams row{};
  std::vector<int> in_tensors, out_tensors;     // parallel to params.in[] / out[]
  std::vector<uint8_t> blob;                    // family-specific parameter block (GEMM / conv)
  int64_t flops = 0;
  // device scratch of the kernel itself, placed in the workspace by the planner: `counter_bytes` sit in the
  // workspace's zeroed header, `scratch_bytes` behind the tensors
  int64_t scratch_bytes = 0, counter_bytes = 0, scratch_off = -1, counter_off = -1;
};

struct Block {
  std::vector<int> ops;        // op ids, topological
  int mapping = DNNF_ONE_TO_ONE;
  std::vector<int> inputs, outputs;   // external tensor ids of the block
  Launch launch;
  bool lowered = false;
};

// A candidate block whose cost the planner wanted from the profiling database and did not find.
struct ProfileMiss { std::string signature; std::vector<int> ops; };

struct Graph {
  std::vector<Tensor> tensors;
  std::vector<Op> ops;
  std::vector<Block> blocks;
  std::vector<int> run_order;            // block indices in execution order
  int n_source_ops = 0;
  bool planned = false;
  uint32_t plan_flags = 0;
  size_t ws_bytes = 0;
  size_t ws_zero_bytes = 256;            // leading bytes of the workspace that must be zero when a run starts
  void* ws_ptr = nullptr;
  size_t ws_bound_bytes = 0;
  void* last_status_base = nullptr;   // workspace whose status words the most recent run used (dnnf_status reads these)
  dnnf_plan_stats pstats{};
  std::vector<ProfileMiss> profile_misses;   // of the last dnnf_plan, one per distinct signature
  int profile_hits = 0;
  std::string err;

  int add_tensor(const std::string& name, int dtype, const std::vector<int64_t>& dims);
  void relink();                          // rebuild producer/consumer lists over alive ops
  std::vector<int> topo_order() const;    // alive ops in topological order
};

// ---- mapping types (ir.cpp) ----
int node_mapping(const Graph& g, const Op& op);                 // Table 2 + most-complex-pair rule
int edge_mapping(const Graph& g, const Op& op, int in_slot);    // mapping of one (input, output) pair
uint32_t math_props(int kind);
void table3(int first, int second, int* fused, int* colour);
bool is_index_only(int kind);       // Reorganize / Shuffle / Slice: no arithmetic
bool is_elementwise(int kind);
bool is_row_anchor(int kind);
bool is_contraction(int kind);
bool is_binary_elementwise(int kind);   // two operands with multidirectional broadcasting
bool is_broadcasting_elementwise(int kind);   // the binary ones and the ternary Where
const char* op_name(int kind);
// Bytes a block stores when tensor t is one of its outputs: the whole tensor, except for a Concat's part, which
// fills only its own range of the shared result.
inline int64_t written_bytes(const Graph& g, int t) {
  const Tensor& T = g.tensors[t];
  if (T.producer >= 0 && g.ops[T.producer].kind == DNNF_OP_CONCATPART) return g.tensors[g.ops[T.producer].in[0]].bytes();
  return T.bytes();
}
int infer_shapes(Graph& g, Op& op, std::string& err);           // creates output tensors

// ---- rewrite.cpp ----
int rewrite_graph(Graph& g, uint32_t flags, dnnf_rewrite_stats* st);
int64_t graph_flops(const Graph& g);

// ---- plan.cpp ----
int plan_graph(Graph& g, uint32_t flags);

// ---- lower.cpp ----
// Lowers `ops` (a candidate block) into a launch.  Returns DNNF_OK or an error;
// `why` explains a refusal (used as the constraint check of Listing 1, Step 2.2).
int lower_block(const Graph& g, const std::vector<int>& ops, uint32_t flags, Block& out, std::string& why);

// ---- profiling database (profile_db.cpp) ----
std::string block_signature(const Graph& g, const Block& b);
bool profile_db_get(const std::string& sig, double* us);
void profile_db_set(const std::string& sig, double us);
size_t profile_db_size();
void profile_db_clear();
int profile_db_save(const char* path);
int profile_db_load(const char* path, int* n_loaded);
double block_cost_us(const Graph& g, const Block& b);

const Program* program_of(const Launch& L);     // the block's micro-op program, wherever the family keeps it

// ---- launch (kernels_*.cu) ----
int launch_block(Graph& g, Block& b, void* stream, std::string& err);

}  // namespace dnnf

struct dnnf_graph {
  dnnf::Graph g;
};
