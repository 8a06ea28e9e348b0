// Profiling database for the fusion-plan generator (Section 4.3, Step 2.3): measured latencies of
// lowered blocks, keyed by a signature of the block (kernel family, operator sequence, data types,
// problem shape).  The planner asks it for the cost of a candidate block before it falls back to the
// analytic model; signatures it asked for and did not find are remembered per graph, so that a
// measuring pass can run exactly those candidates on the device and fill the database.
#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <sstream>

#include "gemm_params.h"
#include "ir.h"

namespace dnnf {

static std::mutex& db_mutex() { static std::mutex m; return m; }
static std::map<std::string, double>& db() { static std::map<std::string, double> d; return d; }

static const char* dtype_tag(int dt) { return dt == DNNF_BF16 ? "bf16" : "f32"; }

// family | operators | dtypes of the block's external tensors | shape key
std::string block_signature(const Graph& g, const Block& b) {
  const Launch& L = b.launch;
  std::ostringstream s;
  static const char* fam[] = {"alias", "ew", "transpose", "row", "gemm", "conv1x1", "dwconv", "pool", "gather"};
  s << fam[L.family] << '|';
  std::vector<int> ops = b.ops;                 // canonical order: the same operator set gives the same signature
  std::sort(ops.begin(), ops.end());
  for (size_t i = 0; i < ops.size(); ++i) s << (i ? "+" : "") << op_name(g.ops[ops[i]].kind);
  s << '|';
  for (int t : L.in_tensors) s << dtype_tag(g.tensors[t].dtype) << ',';
  s << "->";
  for (int t : L.out_tensors) s << dtype_tag(g.tensors[t].dtype) << ',';
  s << '|';
  if (L.family == DNNF_FAMILY_GEMM || L.family == DNNF_FAMILY_CONV1X1) {
    const GemmParams& gp = *reinterpret_cast<const GemmParams*>(L.blob.data());
    s << "M" << gp.M << "N" << gp.N << "K" << gp.K << "B" << gp.batch_ext[0] * gp.batch_ext[1] << "v" << L.variant;
  } else if (L.family == DNNF_FAMILY_ROW) {
    s << "rows" << L.row.rows << "L" << L.row.L;
  } else if (L.family == DNNF_FAMILY_ELEMENTWISE || L.family == DNNF_FAMILY_TRANSPOSE) {
    s << "n" << L.ew.total;
  } else {
    for (int t : L.out_tensors) { for (auto d : g.tensors[t].dims) s << d << 'x'; s << ';'; }
  }
  // bytes of the external tensors, each once: separates broadcast / strided variants of one shape
  int64_t bytes = 0;
  for (int t : b.inputs) bytes += g.tensors[t].bytes();
  for (int t : b.outputs) bytes += g.tensors[t].bytes();
  s << "|bytes" << bytes;
  return s.str();
}

bool profile_db_get(const std::string& sig, double* us) {
  std::lock_guard<std::mutex> lk(db_mutex());
  auto it = db().find(sig);
  if (it == db().end()) return false;
  *us = it->second;
  return true;
}
void profile_db_set(const std::string& sig, double us) {
  std::lock_guard<std::mutex> lk(db_mutex());
  db()[sig] = us;
}
size_t profile_db_size() { std::lock_guard<std::mutex> lk(db_mutex()); return db().size(); }
void profile_db_clear() { std::lock_guard<std::mutex> lk(db_mutex()); db().clear(); }

// one "signature<TAB>microseconds" line per entry
int profile_db_save(const char* path) {
  std::lock_guard<std::mutex> lk(db_mutex());
  FILE* f = fopen(path, "w");
  if (!f) return DNNF_ERR_INVALID_ARG;
  for (auto& kv : db()) fprintf(f, "%s\t%.4f\n", kv.first.c_str(), kv.second);
  fclose(f);
  return DNNF_OK;
}
int profile_db_load(const char* path, int* n_loaded) {
  FILE* f = fopen(path, "r");
  if (!f) return DNNF_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(db_mutex());
  char line[4096];
  int n = 0;
  while (fgets(line, sizeof line, f)) {
    char* tab = strrchr(line, '\t');
    if (!tab) continue;
    *tab = 0;
    double us = atof(tab + 1);
    if (us > 0) { db()[line] = us; ++n; }
  }
  fclose(f);
  if (n_loaded) *n_loaded = n;
  return DNNF_OK;
}

}  // namespace dnnf
