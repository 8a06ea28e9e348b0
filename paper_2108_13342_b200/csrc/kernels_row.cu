// Row family: variant selection and dispatch to the per-variant translation units.
#include <cstdlib>

#include "kernels_row.cuh"

namespace dnnf {

int launch_row_a(const Launch& L, cudaStream_t st);
int launch_row_b(const Launch& L, cudaStream_t st);
int launch_row_c(const Launch& L, cudaStream_t st);
int launch_row_d(const Launch& L, cudaStream_t st);
int launch_row_e(const Launch& L, cudaStream_t st);
int launch_row_f(const Launch& L, cudaStream_t st);
int launch_row_g(const Launch& L, cudaStream_t st);
int launch_row_h(const Launch& L, cudaStream_t st);

// variant encoding: V * 100000 + NV * 1000 + WPR * 10 + RPW
int launch_row(const Launch& L, cudaStream_t st) {
  int rc = 2;
  if (rc == 2) rc = launch_row_a(L, st);
  if (rc == 2) rc = launch_row_b(L, st);
  if (rc == 2) rc = launch_row_c(L, st);
  if (rc == 2) rc = launch_row_d(L, st);
  if (rc == 2) rc = launch_row_e(L, st);
  if (rc == 2) rc = launch_row_f(L, st);
  if (rc == 2) rc = launch_row_g(L, st);
  if (rc == 2) rc = launch_row_h(L, st);
  return rc;
}

bool finalize_row(Launch& L) {
  RowParams& p = L.row;
  int nd = p.it.ndim;
  auto rev = [&](auto* arr) { for (int a = 0, b = nd - 1; a < b; ++a, --b) { auto t = arr[a]; arr[a] = arr[b]; arr[b] = t; } };
  rev(p.it.extent);
  for (int i = 0; i < p.n_in; ++i) rev(p.in[i].stride);
  for (int i = 0; i < p.n_out; ++i) rev(p.out[i].stride);
  const int V = p.vec, Lr = p.L;
  p.inv_L = 1.0f / (float)p.L;
  int nv = 0, wpr = 1, rpw = 1;
  // Enough warps to keep every scheduler busy: with few rows a row is split over several warps
  // (shorter per-thread chains), with many short rows a warp takes several rows (more loads in flight).
  // 4000 (27 warps per SM): measured best when independent blocks overlap on the GPU, 6 % slower than
  // 148 * 32 for a lone 1024-row launch.
  static const long target = dev_env("DNNF_ROW_TARGET_WARPS") ? atol(dev_env("DNNF_ROW_TARGET_WARPS")) : 4000L;
  static const long split_target = dev_env("DNNF_ROW_SPLIT_TARGET") ? atol(dev_env("DNNF_ROW_SPLIT_TARGET")) : 4000L;   // (2000 is 3 % better when independent blocks overlap, 20 % worse for a lone 1024-row launch)
  if (V == 4) {
    const int vectors = (Lr + 3) / 4;
    auto fit = [&](int w) { int need = (vectors + 32 * w - 1) / (32 * w); return need; };   // vectors per lane with w warps per row
    int need = fit(1);
    if (need <= 8) {
      wpr = 1;
      while (wpr < 8 && p.rows * wpr < split_target && fit(wpr) > 1) wpr *= 2;
      need = fit(wpr);
      if (wpr == 1) { nv = need <= 1 ? 1 : need <= 2 ? 2 : need <= 4 ? 4 : need <= 6 ? 6 : 8; }
      else if (wpr == 2) { nv = need <= 1 ? 1 : need <= 2 ? 2 : need <= 3 ? 3 : 4; }
      else if (wpr == 4) { nv = need <= 1 ? 1 : 2; if (need > 2) { wpr = 2; nv = fit(2) <= 3 ? 3 : 4; if (fit(2) > 4) { wpr = 1; nv = fit(1) <= 4 ? 4 : fit(1) <= 6 ? 6 : 8; } } }
      else { nv = need <= 1 ? 1 : need <= 2 ? 2 : need <= 4 ? 4 : 8; }
      if (wpr == 1 && nv <= 2) { rpw = nv == 1 ? 4 : 2; while (rpw > 1 && (p.rows + rpw - 1) / rpw < target) rpw /= 2; }
    } else {
      wpr = 8; int n8 = fit(8); nv = n8 <= 2 ? 2 : n8 <= 4 ? 4 : 8; if (n8 > 8) return false;
    }
  } else {
    int need = (Lr + 31) / 32;
    if (need <= 1) { nv = 1; rpw = 4; }
    else if (need <= 16) nv = need <= 4 ? 4 : 16;
    else { wpr = 8; int n8 = (Lr + 255) / 256; nv = n8 <= 8 ? 8 : 32; if (n8 > 32) return false; }
  }
  // a warp's rows are consecutive along outer dim 1: they must not straddle it
  if (rpw > 1 && nd > 2 && p.it.extent[1] % rpw != 0) rpw = 1;
  L.variant = V * 100000 + nv * 1000 + wpr * 10 + rpw;
  int64_t warps = (p.rows + rpw - 1) / rpw;
  L.grid = wpr > 1 ? (int)p.rows : (int)((warps + kRowWarpsPerCta - 1) / kRowWarpsPerCta);
  L.threads = wpr > 1 ? 32 * wpr : 32 * kRowWarpsPerCta;
  L.static_id = (V == 4 && (wpr < 8 || nv == 1)) ? StaticSet<RowStatic>::find(p.prog) : 0;
  set_fastdiv(p.it);
  return true;
}

}  // namespace dnnf
