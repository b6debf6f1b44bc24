// extern "C" entry points of include/mohge.h: argument validation, workspace carving and the
// launch sequence of every step.  No allocation, no synchronisation (except the status read).

#include <stdarg.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <mutex>

#include "common.cuh"

namespace mohge {

static thread_local char g_err[512] = "";
unsigned long long g_launches = 0;

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
}

int32_t cuda_fail(cudaError_t e, const char* what) {
  set_error("CUDA error %d (%s) at %s", (int)e, cudaGetErrorString(e), what);
  return MOHGE_ERR_CUDA;
}

int32_t make_dims(const mohge_config* c, int64_t T, Dims* D) {
  MOHGE_CHECK_ARG(c != nullptr, "config is NULL");
  MOHGE_CHECK_ARG(T >= 0 && T <= (1 << 24), "T = %lld out of range [0, 2^24]", (long long)T);
  MOHGE_CHECK_ARG(c->n_groups >= 1 && c->n_groups <= MOHGE_MAX_GROUPS, "n_groups = %d not in 1..%d",
                  c->n_groups, MOHGE_MAX_GROUPS);
  MOHGE_CHECK_ARG(c->experts_per_group >= 1 && c->experts_per_group <= MOHGE_MAX_EXPERTS_PER_GROUP,
                  "experts_per_group = %d not in 1..%d", c->experts_per_group,
                  MOHGE_MAX_EXPERTS_PER_GROUP);
  MOHGE_CHECK_ARG(c->k_groups >= 1 && c->k_groups <= c->n_groups, "k_groups = %d not in 1..n_groups",
                  c->k_groups);
  MOHGE_CHECK_ARG(c->k_experts >= 1 && c->k_experts <= MOHGE_MAX_K_EXPERTS &&
                      c->k_experts <= c->k_groups * c->experts_per_group,
                  "k_experts = %d must be in 1..min(%d, k_groups*experts_per_group): Eq. 5 can only "
                  "pick experts of selected groups",
                  c->k_experts, MOHGE_MAX_K_EXPERTS);
  MOHGE_CHECK_ARG(c->dtype == MOHGE_BF16 || c->dtype == MOHGE_F32, "unknown dtype %d", c->dtype);
  MOHGE_CHECK_ARG(c->d_model >= 8 && c->d_model % 8 == 0, "d_model = %d must be a positive multiple of 8",
                  c->d_model);
  MOHGE_CHECK_ARG(c->row_align == 1 || c->row_align == 128, "row_align = %d must be 1 or 128",
                  c->row_align);
  MOHGE_CHECK_ARG(c->eps >= 0.0f, "eps must be >= 0");
  D->d = c->d_model; D->Ng = c->n_groups; D->N = c->experts_per_group;
  D->P = 1;
  while (D->P < D->N) D->P *= 2;
  D->Ne = D->Ng * D->N; D->NL = D->Ng + D->Ne; D->Kg = c->k_groups; D->Ke = c->k_experts;
  D->Wmax = 0;
  for (int g = 0; g < MOHGE_MAX_GROUPS; ++g) {
    D->W[g] = 0;
    if (g < D->Ng) {
      MOHGE_CHECK_ARG(c->group_width[g] >= 8 && c->group_width[g] % 8 == 0,
                      "group_width[%d] = %d must be a positive multiple of 8", g, c->group_width[g]);
      D->W[g] = c->group_width[g];
      if (D->W[g] > D->Wmax) D->Wmax = D->W[g];
    }
  }
  D->align = c->row_align;
  D->T = T; D->R = T * D->Ke;
  D->Rcap = (D->R + (int64_t)D->Ne * (D->align - 1) + D->align - 1) / D->align * D->align;
  D->bf16 = c->dtype == MOHGE_BF16;
  MOHGE_CHECK_ARG(D->Rcap < (1LL << 31) / 2, "too many routed rows (%lld)", (long long)D->Rcap);
  return MOHGE_OK;
}

// ---------------------------------------------------------------- switches
static const char* const kSwitchName[SW_COUNT] = {"pdl", "tc_cg", "tc_wide", "force_simt", "route_fused"};
static const char* const kSwitchEnv[SW_COUNT] = {"MOHGE_PDL", "MOHGE_TC_CG", "MOHGE_TC_WIDE", "MOHGE_FORCE_SIMT",
                                                   "MOHGE_ROUTE_FUSED"};
static std::atomic<int> g_switch[SW_COUNT];
static std::once_flag g_switch_once;

static void read_switches_from_env() {
  for (int i = 0; i < SW_COUNT; ++i) {
    const char* e = getenv(kSwitchEnv[i]);
    g_switch[i].store((e && e[0]) ? atoi(e) : -1);
  }
}
static int switch_index(const char* name) {
  for (int i = 0; name && i < SW_COUNT; ++i)
    if (strcmp(name, kSwitchName[i]) == 0) return i;
  return -1;
}

int switch_value(int which) {
  std::call_once(g_switch_once, read_switches_from_env);
  return g_switch[which].load(std::memory_order_relaxed);
}

// Programmatic dependent launch (see common.cuh): on unless the switch is 0.  Measured 1.5-2.5 %
// of the step at the 8k- and 16k-token workloads, nothing at the large one.
bool dependent_launch() { return switch_value(SW_PDL) != 0; }

// ---------------------------------------------------------------- per-device facts
int32_t current_device(DeviceInfo* out) {
  static DeviceInfo table[kMaxDevices];
  static std::atomic<bool> known[kMaxDevices];
  static std::mutex mu;
  int dev = 0;
  MOHGE_CUDA(cudaGetDevice(&dev));
  MOHGE_CHECK_ARG(dev >= 0 && dev < kMaxDevices, "device ordinal %d is not supported (at most %d devices)",
                  dev, kMaxDevices);
  if (!known[dev].load(std::memory_order_acquire)) {
    std::lock_guard<std::mutex> lock(mu);
    if (!known[dev].load(std::memory_order_relaxed)) {
      DeviceInfo di;
      di.ordinal = dev;
      MOHGE_CUDA(cudaDeviceGetAttribute(&di.sm_count, cudaDevAttrMultiProcessorCount, dev));
      MOHGE_CUDA(cudaDeviceGetAttribute(&di.cc_major, cudaDevAttrComputeCapabilityMajor, dev));
      MOHGE_CUDA(cudaDeviceGetAttribute(&di.cc_minor, cudaDevAttrComputeCapabilityMinor, dev));
      table[dev] = di;
      known[dev].store(true, std::memory_order_release);
    }
  }
  *out = table[dev];
  return MOHGE_OK;
}

static int64_t up256(int64_t v) { return (v + 255) / 256 * 256; }

int router_dw_splits(const Dims& D) {
  const int m_tiles = (D.d + 127) / 128;
  const int64_t k_blocks = (D.T + 63) / 64;
  int64_t s = 148 / m_tiles;
  if (s > 32) s = 32;
  if (s > k_blocks) s = k_blocks;
  if (s < 1) s = 1;
  const int64_t chunk = (k_blocks + s - 1) / s;          // k-blocks per split
  return chunk > 0 ? (int)((k_blocks + chunk - 1) / chunk) : 1;   // no split is empty
}

WsLayout ws_layout(const Dims& D) {
  WsLayout L;
  L.chunks = ceil_div(D.T, kDispatchChunk);
  L.status_off = 0;
  L.stats_off = 256;
  L.hist_off = L.stats_off + up256((int64_t)kStatsBlocks * D.NL * 8);
  L.base_off = L.hist_off + up256((int64_t)(L.chunks + 1) * D.Ne * 4);
  L.dl16_off = L.base_off + up256((int64_t)(L.chunks + 1) * D.Ne * 4);
  L.rdw_off = L.dl16_off + up256((D.T + 1) * (int64_t)((D.NL + 7) / 8 * 8) * 2);
  L.tiles_off = L.rdw_off + up256((int64_t)router_dw_splits(D) * D.NL * D.d * 4);
  // tile capacity: the smallest tile either path uses is 64 x 64
  const int64_t mt = D.Rcap / 64 + D.Ne + 1;
  const int64_t wide = (D.d > 2 * D.Wmax ? D.d : 2 * D.Wmax);
  const int64_t row_tiled = mt * ((wide + 63) / 64);
  const int64_t wgrad = (int64_t)D.Ne * ((2 * D.Wmax + 63) / 64) * ((D.d + 63) / 64);
  L.tiles_cap = row_tiled > wgrad ? row_tiled : wgrad;
  L.dgp_off = L.tiles_off + 1024 + (int64_t)kMaxLists * up256(L.tiles_cap * (int64_t)sizeof(Tile));
  // gate-gradient partial sums of the experts' backward: one float per physical row and
  // 128-column slot of the hidden axis
  L.dgate_slots = (D.Wmax + 127) / 128;
  L.total = L.dgp_off + up256(D.Rcap * (int64_t)L.dgate_slots * 4);
  return L;
}

struct Ws {
  int32_t* status;
  double* stats;
  int32_t* hist;
  int32_t* base;
  __nv_bfloat16* dl16;
  float* rdw;
  int32_t* tile_count;
  Tile* tiles;
  int64_t tiles_cap;
  float* dgp;
  int dgate_slots;
};

static Ws carve(const Dims& D, void* ws) {
  const WsLayout L = ws_layout(D);
  char* p = (char*)ws;
  Ws w;
  w.status = (int32_t*)(p + L.status_off);
  w.stats = (double*)(p + L.stats_off);
  w.hist = (int32_t*)(p + L.hist_off);
  w.base = (int32_t*)(p + L.base_off);
  w.dl16 = (__nv_bfloat16*)(p + L.dl16_off);
  w.rdw = (float*)(p + L.rdw_off);
  w.tile_count = (int32_t*)(p + L.tiles_off);
  w.tiles = (Tile*)(p + L.tiles_off + 1024);   // kMaxLists lists, tiles_cap entries apart
  w.tiles_cap = L.tiles_cap;
  w.dgp = (float*)(p + L.dgp_off);
  w.dgate_slots = L.dgate_slots;
  return w;
}

static bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

#define REQ_PTR(p) MOHGE_CHECK_ARG((p) != nullptr && aligned16(p), #p " must be a non-NULL 16-byte aligned device pointer")
#define OPT_PTR(p) MOHGE_CHECK_ARG(aligned16(p), #p " must be 16-byte aligned")

static bool force_simt() { return switch_value(SW_FORCE_SIMT) == 1; }

static int32_t group_ptrs(const Dims& D, const void* const* w13, const void* const* w2,
                          float* const* dw13, float* const* dw2, GroupPtrs* P) {
  memset(P, 0, sizeof(*P));
  for (int g = 0; g < D.Ng; ++g) {
    if (w13) { REQ_PTR(w13[g]); P->w13[g] = w13[g]; }
    if (w2) { REQ_PTR(w2[g]); P->w2[g] = w2[g]; }
    if (dw13) { REQ_PTR(dw13[g]); P->dw13[g] = dw13[g]; }
    if (dw2) { REQ_PTR(dw2[g]); P->dw2[g] = dw2[g]; }
  }
  return MOHGE_OK;
}

}  // namespace mohge

using namespace mohge;

extern "C" {

const char* mohge_last_error(void) { return g_err; }

int64_t mohge_launch_count(void) { return (int64_t)g_launches; }

int64_t mohge_workspace_bytes(const mohge_config* cfg, int64_t T) {
  Dims D;
  if (make_dims(cfg, T, &D) != MOHGE_OK) return 0;
  return ws_layout(D).total;
}

int64_t mohge_perm_rows(const mohge_config* cfg, int64_t T) {
  Dims D;
  if (make_dims(cfg, T, &D) != MOHGE_OK) return 0;
  return D.Rcap;
}

int32_t mohge_get_switch(const char* name) {
  const int i = switch_index(name);
  if (i < 0) {
    set_error("unknown switch '%s' (pdl, tc_cg, tc_wide, force_simt)", name ? name : "(null)");
    return INT32_MIN;
  }
  return switch_value(i);
}

int32_t mohge_set_switch(const char* name, int32_t value) {
  const int i = switch_index(name);
  MOHGE_CHECK_ARG(i >= 0, "unknown switch '%s' (pdl, tc_cg, tc_wide, force_simt)", name ? name : "(null)");
  MOHGE_CHECK_ARG(value >= -1, "switch value %d: -1 (library's rule) or a non-negative value", value);
  (void)switch_value(i);          // the environment is consulted first, once, and never again
  g_switch[i].store(value);
  return MOHGE_OK;
}

int32_t mohge_workspace_init(const mohge_config* cfg, int64_t T, void* ws, int64_t ws_bytes, void* stream) {
  Dims D;
  int32_t rc = make_dims(cfg, T, &D);
  if (rc) return rc;
  REQ_PTR(ws);
  const int64_t need = ws_layout(D).total;
  if (ws_bytes < need) {
    set_error("workspace of %lld bytes is too small: this configuration and T = %lld need %lld",
              (long long)ws_bytes, (long long)T, (long long)need);
    return MOHGE_ERR_WORKSPACE;
  }
  MOHGE_CUDA(cudaMemsetAsync(ws, 0, 256, (cudaStream_t)stream));
  return MOHGE_OK;
}

int32_t mohge_get_device_status(const void* ws, int32_t* host_out, void* stream) {
  MOHGE_CHECK_ARG(ws != nullptr && host_out != nullptr, "ws and host_out must be non-NULL");
  MOHGE_CUDA(cudaMemcpyAsync(host_out, ws, sizeof(int32_t), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
  MOHGE_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
  const int32_t word = *host_out, code = word >> 24, site = word & 0xffffff;
  if (word == 0) return MOHGE_OK;
  if (code == 1) {
    set_error("a device-side wait gave up after its time budget (site %d of the grouped GEMM kernel)", site);
    return MOHGE_ERR_TIMEOUT;
  }
  set_error(code == 2 ? "a device-side index check failed (site %d): the entry was skipped"
                      : "NaN among the router logits (code %d): ranked below every number", code == 2 ? site : code);
  return MOHGE_ERR_DEVICE_CHECK;
}

int32_t mohge_route(const mohge_config* cfg, int64_t T, const void* x, const void* w_router,
                    const float* logit_bias, const float* logits_in, float* logits_out,
                    int32_t* group_idx, int32_t* expert_idx, float* gate_w, float* gs_saved,
                    float* esp_saved, void* ws, void* stream) {
  Dims D;
  int32_t rc = make_dims(cfg, T, &D);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  REQ_PTR(group_idx); REQ_PTR(expert_idx); REQ_PTR(gate_w); REQ_PTR(gs_saved); REQ_PTR(esp_saved);
  REQ_PTR(ws);
  const float* logits = logits_in;
  if (!logits_in) {
    REQ_PTR(x); REQ_PTR(w_router); REQ_PTR(logits_out); OPT_PTR(logit_bias);
    const int f32 = D.bf16 ? 0 : 1;
    if (D.bf16 && !force_simt()) {
      // the tensor-core launch selects in its epilogue when it can (Eq. 2-6 on the accumulator rows)
      const RouteOut ro = {group_idx, expert_idx, gate_w, gs_saved, esp_saved};
      bool routed = false;
      rc = launch_tc_plain(D, ROLE_LOGITS, x, w_router, 0, logits_out, logit_bias, carve(D, ws).rdw,
                           carve(D, ws).status, st, &ro, &routed);
      if (rc || routed) return rc;
    } else
      rc = launch_simt_plain((int)T, D.NL, D.d, x, f32, D.d, 1, w_router, f32, D.d, 1, logits_out, 1,
                             D.NL, logit_bias, 0, st);
    if (rc) return rc;
    logits = logits_out;
  } else {
    OPT_PTR(logits_in);
    if (logits_out && logits_out != logits_in && T > 0)
      MOHGE_CUDA(cudaMemcpyAsync(logits_out, logits_in, sizeof(float) * T * D.NL,
                                 cudaMemcpyDeviceToDevice, st));
  }
  return launch_router_select(D, logits, group_idx, expert_idx, gate_w, gs_saved, esp_saved,
                              carve(D, ws).status, st);
}

int32_t mohge_aux_stats(const mohge_config* cfg, int64_t T, const float* gs_saved,
                        const float* esp_saved, const int32_t* group_idx,
                        const int32_t* expert_idx, int32_t* group_count, float* group_psum,
                        int32_t* expert_count_routed, int32_t* expert_count_lit,
                        float* expert_psum, float* loss_out, void* ws, void* stream) {
  Dims D;
  int32_t rc = make_dims(cfg, T, &D);
  if (rc) return rc;
  REQ_PTR(gs_saved); REQ_PTR(esp_saved); REQ_PTR(group_idx); REQ_PTR(expert_idx);
  REQ_PTR(group_count); REQ_PTR(group_psum); REQ_PTR(expert_count_routed);
  REQ_PTR(expert_count_lit); REQ_PTR(expert_psum); REQ_PTR(loss_out); REQ_PTR(ws);
  const Ws w = carve(D, ws);
  return launch_aux_stats(D, *cfg, gs_saved, esp_saved, group_idx, expert_idx, group_count,
                          group_psum, expert_count_routed, expert_count_lit, expert_psum, loss_out,
                          w.stats, (cudaStream_t)stream);
}

int32_t mohge_dispatch(const mohge_config* cfg, int64_t T, const void* x,
                       const int32_t* expert_idx, int32_t* counts, int32_t* offsets,
                       int32_t* aligned_offsets, int32_t* row_of, int32_t* prow_of,
                       int32_t* src_of, void* x_perm, void* ws, void* stream) {
  Dims D;
  int32_t rc = make_dims(cfg, T, &D);
  if (rc) return rc;
  REQ_PTR(x); REQ_PTR(expert_idx); REQ_PTR(counts); REQ_PTR(offsets); REQ_PTR(aligned_offsets);
  REQ_PTR(row_of); REQ_PTR(prow_of); REQ_PTR(src_of); REQ_PTR(x_perm); REQ_PTR(ws);
  const Ws w = carve(D, ws);
  return launch_dispatch(D, x, expert_idx, counts, offsets, aligned_offsets, row_of, prow_of, src_of,
                         x_perm, w.hist, w.base, w.status, (cudaStream_t)stream);
}

int32_t mohge_dispatch_indices(const mohge_config* cfg, int64_t T, const int32_t* expert_idx,
                               int32_t* counts, int32_t* offsets, int32_t* aligned_offsets,
                               int32_t* row_of, int32_t* prow_of, int32_t* src_of,
                               int32_t* tok_of_prow, void* ws, void* stream) {
  Dims D;
  int32_t rc = make_dims(cfg, T, &D);
  if (rc) return rc;
  REQ_PTR(expert_idx); REQ_PTR(counts); REQ_PTR(offsets); REQ_PTR(aligned_offsets);
  REQ_PTR(row_of); REQ_PTR(prow_of); REQ_PTR(src_of); REQ_PTR(tok_of_prow); REQ_PTR(ws);
  const Ws w = carve(D, ws);
  return launch_dispatch(D, nullptr, expert_idx, counts, offsets, aligned_offsets, row_of, prow_of, src_of,
                         nullptr, w.hist, w.base, w.status, (cudaStream_t)stream, tok_of_prow);
}

// Forward of the grouped SwiGLU experts for already validated arguments.  Shared by the routed
// experts and by the shared experts (one segment of T rows).
// gather != nullptr: x_perm is x itself and row r of the permuted numbering is row gather[r] of it.
static int32_t expert_fwd_impl(const Dims& D, const GroupPtrs& P, const void* x_perm,
                               const int32_t* counts, const int32_t* aligned_offsets,
                               void* au_saved, void* h_saved, void* y_perm, const Ws& w,
                               cudaStream_t st, const int32_t* gather = nullptr) {
  int32_t rc;
  if (D.bf16 && !force_simt()) {
    MOHGE_CHECK_ARG(D.align == 128, "the BF16 tensor-core path needs row_align = 128");
    // both tile lists with one launch, then the two GEMMs
    const TilePlan plans[2] = {tc_tile_plan(D, ROLE_FWD1), tc_tile_plan(D, ROLE_FWD2)};
    rc = launch_build_tiles_multi(plans, 2, aligned_offsets, w.tile_count, w.tiles, w.tiles_cap,
                                  w.status, st);
    if (rc) return rc;
    rc = launch_tc_grouped(D, ROLE_FWD1, P, x_perm, nullptr, au_saved, h_saved, counts,
                           aligned_offsets, 0, w.tile_count, w.tiles, w.tiles_cap, w.status, st, true,
                           nullptr, 0, gather);
    if (rc) return rc;
    return launch_tc_grouped(D, ROLE_FWD2, P, h_saved, nullptr, y_perm, nullptr, counts,
                             aligned_offsets, 0, w.tile_count + 64, w.tiles + w.tiles_cap,
                             w.tiles_cap, w.status, st, true);
  }
  if (gather) {
    set_error("the row-gathering entry points need the BF16 tensor-core path");
    return MOHGE_ERR_UNSUPPORTED;
  }
  rc = launch_build_tiles(D, ROLE_FWD1, 64, 64, counts, aligned_offsets, w.tile_count, w.tiles,
                          w.tiles_cap, w.status, st);
  if (rc) return rc;
  rc = launch_simt_grouped(D, ROLE_FWD1, P, x_perm, nullptr, au_saved, aligned_offsets, 0,
                           w.tile_count, w.tiles, st);
  if (rc) return rc;
  rc = launch_swiglu_fwd(D, aligned_offsets, au_saved, h_saved, st);
  if (rc) return rc;
  rc = launch_build_tiles(D, ROLE_FWD2, 64, 64, counts, aligned_offsets, w.tile_count, w.tiles,
                          w.tiles_cap, w.status, st);
  if (rc) return rc;
  return launch_simt_grouped(D, ROLE_FWD2, P, h_saved, nullptr, y_perm, aligned_offsets, 0,
                             w.tile_count, w.tiles, st);
}

int32_t mohge_expert_fwd(const mohge_config* cfg, int64_t T, const void* x_perm,
                         const int32_t* counts, const int32_t* aligned_offsets,
                         const void* const* w13, const void* const* w2, void* au_saved,
                         void* h_saved, void* y_perm, void* ws, void* stream) {
  Dims D;
  int32_t rc = make_dims(cfg, T, &D);
  if (rc) return rc;
  REQ_PTR(x_perm); REQ_PTR(counts); REQ_PTR(aligned_offsets); REQ_PTR(au_saved); REQ_PTR(h_saved);
  REQ_PTR(y_perm); REQ_PTR(ws);
  MOHGE_CHECK_ARG(w13 && w2, "w13 and w2 must be host arrays of n_groups device pointers");
  GroupPtrs P;
  rc = group_ptrs(D, w13, w2, nullptr, nullptr, &P);
  if (rc) return rc;
  return expert_fwd_impl(D, P, x_perm, counts, aligned_offsets, au_saved, h_saved, y_perm,
                         carve(D, ws), (cudaStream_t)stream);
}

int32_t mohge_expert_fwd_gather(const mohge_config* cfg, int64_t T, const void* x,
                                const int32_t* tok_of_prow, const int32_t* counts,
                                const int32_t* aligned_offsets, const void* const* w13,
                                const void* const* w2, void* au_saved, void* h_saved, void* y_perm,
                                void* ws, void* stream) {
  Dims D;
  int32_t rc = make_dims(cfg, T, &D);
  if (rc) return rc;
  REQ_PTR(x); REQ_PTR(tok_of_prow); REQ_PTR(counts); REQ_PTR(aligned_offsets); REQ_PTR(au_saved);
  REQ_PTR(h_saved); REQ_PTR(y_perm); REQ_PTR(ws);
  MOHGE_CHECK_ARG(w13 && w2, "w13 and w2 must be host arrays of n_groups device pointers");
  MOHGE_CHECK_ARG(D.d % 8 == 0 && T > 0, "the row-gathering entry points need T > 0");
  GroupPtrs P;
  rc = group_ptrs(D, w13, w2, nullptr, nullptr, &P);
  if (rc) return rc;
  return expert_fwd_impl(D, P, x, counts, aligned_offsets, au_saved, h_saved, y_perm, carve(D, ws),
                         (cudaStream_t)stream, tok_of_prow);
}

int32_t mohge_combine(const mohge_config* cfg, int64_t T, const void* y_perm,
                      const int32_t* prow_of, const float* gate_w, const void* y_add, void* y,
                      void* stream) {
  Dims D;
  int32_t rc = make_dims(cfg, T, &D);
  if (rc) return rc;
  REQ_PTR(y_perm); REQ_PTR(prow_of); REQ_PTR(gate_w); REQ_PTR(y); OPT_PTR(y_add);
  return launch_combine(D, y_perm, prow_of, gate_w, y_add, y, (cudaStream_t)stream);
}

int32_t mohge_combine_bwd(const mohge_config* cfg, int64_t T, const void* dy, const void* y_perm,
                          const int32_t* prow_of, const float* gate_w, const int32_t* counts,
                          const int32_t* aligned_offsets, void* dy_perm, float* dgate_w,
                          void* stream) {
  Dims D;
  int32_t rc = make_dims(cfg, T, &D);
  if (rc) return rc;
  REQ_PTR(dy); REQ_PTR(prow_of); REQ_PTR(gate_w); REQ_PTR(counts);
  REQ_PTR(aligned_offsets); REQ_PTR(dy_perm);
  MOHGE_CHECK_ARG((y_perm == nullptr) == (dgate_w == nullptr),
                  "y_perm and dgate_w must both be given, or both be NULL (scaled rows only)");
  if (y_perm) { REQ_PTR(y_perm); REQ_PTR(dgate_w); }
  return launch_combine_bwd(D, y_perm ? 0 : 1, dy, y_perm, prow_of, gate_w, counts, aligned_offsets,
                            dy_perm, dgate_w, (cudaStream_t)stream);
}

// Backward of the grouped SwiGLU experts for already validated arguments (see expert_fwd_impl).
// Optional by-product of the experts' backward: the gate gradient (see mohge_expert_bwd_dgate).
struct DgateArgs {
  const void* dy;
  const void* y_perm;
  const int32_t* prow_of;
  const float* gate_w;
  float* dgate_w;
};

static int32_t expert_bwd_impl(const Dims& D, const GroupPtrs& P, const void* dy_perm,
                               const void* x_perm, const void* au_saved, const void* h_saved,
                               const int32_t* counts, const int32_t* aligned_offsets, void* dau,
                               void* dx_perm, int32_t accumulate, const Ws& w, cudaStream_t st,
                               const DgateArgs* dg = nullptr, const int32_t* gather = nullptr,
                               const DyFuse* dyf = nullptr) {
  int32_t rc;
  if ((gather || dyf) && !(D.bf16 && !force_simt())) {
    set_error("the row-gathering entry points need the BF16 tensor-core path");
    return MOHGE_ERR_UNSUPPORTED;
  }
  if (!accumulate) {
    rc = launch_zero_empty_wgrad(D, P, counts, st);
    if (rc) return rc;
  }
  if (D.bf16 && !force_simt()) {
    MOHGE_CHECK_ARG(D.align == 128, "the BF16 tensor-core path needs row_align = 128");
    const int roles[4] = {ROLE_DGRAD_DOWN, ROLE_WGRAD_DOWN, ROLE_DGRAD_13, ROLE_WGRAD_13};
    TilePlan plans[4];
    for (int r = 0; r < 4; ++r) plans[r] = tc_tile_plan(D, roles[r]);
    rc = launch_build_tiles_multi(plans, 4, aligned_offsets, w.tile_count, w.tiles, w.tiles_cap,
                                  w.status, st);
    if (rc) return rc;
    for (int r = 0; r < 4; ++r) {
      const void* A = nullptr; const void* B = nullptr; void* C = nullptr; void* C2 = nullptr;
      switch (roles[r]) {
        // dyf: dy_perm is dy [T, d] itself (rows gathered by the kernels), and WGRAD_DOWN reads
        // the gate * H that DGRAD_DOWN has just written instead of H
        case ROLE_DGRAD_DOWN: A = dy_perm; B = au_saved; C = dau; break;
        case ROLE_WGRAD_DOWN: A = dy_perm; B = dyf ? dyf->hs : h_saved; break;
        case ROLE_DGRAD_13: A = dau; C = dx_perm; break;
        default: A = dau; B = x_perm; break;
      }
      rc = launch_tc_grouped(D, roles[r], P, A, B, C, C2, counts, aligned_offsets, accumulate,
                             w.tile_count + 64 * r, w.tiles + w.tiles_cap * r, w.tiles_cap, w.status,
                             st, true, dg ? w.dgp : nullptr, w.dgate_slots, gather, dyf);
      if (rc) return rc;
      if (dg && roles[r] == ROLE_DGRAD_DOWN) {
        int bn[MOHGE_MAX_GROUPS];
        for (int g = 0; g < MOHGE_MAX_GROUPS; ++g) bn[g] = g < D.Ng ? tc_dgrad_down_bn(D, g) : 128;
        rc = launch_dgate_reduce(D, bn, w.dgp, w.dgate_slots, dg->prow_of, dg->gate_w, aligned_offsets,
                                 dg->dy, dg->y_perm, dg->dgate_w, st);
        if (rc) return rc;
      }
    }
    return MOHGE_OK;
  }
  if (dg) {
    // FP32 / FFMA path: the definition, <dy[t], y_perm[row]>
    rc = launch_combine_bwd(D, 2, dg->dy, dg->y_perm, dg->prow_of, dg->gate_w, counts, aligned_offsets,
                            nullptr, dg->dgate_w, st);
    if (rc) return rc;
  }
  struct Step { int role; const void* A; const void* B; void* C; };
  const Step steps[4] = {{ROLE_DGRAD_DOWN, dy_perm, nullptr, dau},
                         {ROLE_WGRAD_DOWN, dy_perm, h_saved, nullptr},
                         {ROLE_DGRAD_13, dau, nullptr, dx_perm},
                         {ROLE_WGRAD_13, dau, x_perm, nullptr}};
  for (int s = 0; s < 4; ++s) {
    rc = launch_build_tiles(D, steps[s].role, 64, 64, counts, aligned_offsets, w.tile_count,
                            w.tiles, w.tiles_cap, w.status, st);
    if (rc) return rc;
    rc = launch_simt_grouped(D, steps[s].role, P, steps[s].A, steps[s].B, steps[s].C,
                             aligned_offsets, accumulate, w.tile_count, w.tiles, st);
    if (rc) return rc;
    if (steps[s].role == ROLE_DGRAD_DOWN) {
      rc = launch_swiglu_bwd(D, aligned_offsets, au_saved, dau, st);
      if (rc) return rc;
    }
  }
  return MOHGE_OK;
}


int32_t mohge_expert_bwd(const mohge_config* cfg, int64_t T, const void* dy_perm,
                         const void* x_perm, const void* au_saved, const void* h_saved,
                         const int32_t* counts, const int32_t* aligned_offsets,
                         const void* const* w13, const void* const* w2, void* dau, void* dx_perm,
                         float* const* dw13, float* const* dw2, int32_t accumulate, void* ws,
                         void* stream) {
  Dims D;
  int32_t rc = make_dims(cfg, T, &D);
  if (rc) return rc;
  REQ_PTR(dy_perm); REQ_PTR(x_perm); REQ_PTR(au_saved); REQ_PTR(h_saved); REQ_PTR(counts);
  REQ_PTR(aligned_offsets); REQ_PTR(dau); REQ_PTR(dx_perm); REQ_PTR(ws);
  MOHGE_CHECK_ARG(w13 && w2 && dw13 && dw2, "w13, w2, dw13, dw2 must be host arrays of n_groups device pointers");
  GroupPtrs P;
  rc = group_ptrs(D, w13, w2, dw13, dw2, &P);
  if (rc) return rc;
  return expert_bwd_impl(D, P, dy_perm, x_perm, au_saved, h_saved, counts, aligned_offsets, dau,
                         dx_perm, accumulate, carve(D, ws), (cudaStream_t)stream);
}

int32_t mohge_expert_bwd_dgate(const mohge_config* cfg, int64_t T, const void* dy_perm,
                               const void* x_perm, const void* au_saved, const void* h_saved,
                               const int32_t* counts, const int32_t* aligned_offsets,
                               const void* const* w13, const void* const* w2, void* dau,
                               void* dx_perm, float* const* dw13, float* const* dw2,
                               int32_t accumulate, const void* dy, const void* y_perm,
                               const int32_t* prow_of, const float* gate_w, float* dgate_w, void* ws,
                               void* stream) {
  Dims D;
  int32_t rc = make_dims(cfg, T, &D);
  if (rc) return rc;
  REQ_PTR(dy_perm); REQ_PTR(x_perm); REQ_PTR(au_saved); REQ_PTR(h_saved); REQ_PTR(counts);
  REQ_PTR(aligned_offsets); REQ_PTR(dau); REQ_PTR(dx_perm); REQ_PTR(ws);
  REQ_PTR(dy); REQ_PTR(y_perm); REQ_PTR(prow_of); REQ_PTR(gate_w); REQ_PTR(dgate_w);
  MOHGE_CHECK_ARG(w13 && w2 && dw13 && dw2, "w13, w2, dw13, dw2 must be host arrays of n_groups device pointers");
  GroupPtrs P;
  rc = group_ptrs(D, w13, w2, dw13, dw2, &P);
  if (rc) return rc;
  const DgateArgs dg = {dy, y_perm, prow_of, gate_w, dgate_w};
  return expert_bwd_impl(D, P, dy_perm, x_perm, au_saved, h_saved, counts, aligned_offsets, dau,
                         dx_perm, accumulate, carve(D, ws), (cudaStream_t)stream, &dg);
}

int32_t mohge_expert_bwd_gather(const mohge_config* cfg, int64_t T, const void* dy_perm,
                                const void* x, const int32_t* tok_of_prow, const void* au_saved,
                                const void* h_saved, const int32_t* counts,
                                const int32_t* aligned_offsets, const void* const* w13,
                                const void* const* w2, void* dau, void* dx_perm, float* const* dw13,
                                float* const* dw2, int32_t accumulate, const void* dy,
                                const void* y_perm, const int32_t* prow_of, const float* gate_w,
                                float* dgate_w, void* ws, void* stream) {
  Dims D;
  int32_t rc = make_dims(cfg, T, &D);
  if (rc) return rc;
  REQ_PTR(dy_perm); REQ_PTR(x); REQ_PTR(tok_of_prow); REQ_PTR(au_saved); REQ_PTR(h_saved); REQ_PTR(counts);
  REQ_PTR(aligned_offsets); REQ_PTR(dau); REQ_PTR(dx_perm); REQ_PTR(ws);
  REQ_PTR(dy); REQ_PTR(y_perm); REQ_PTR(prow_of); REQ_PTR(gate_w); REQ_PTR(dgate_w);
  MOHGE_CHECK_ARG(w13 && w2 && dw13 && dw2, "w13, w2, dw13, dw2 must be host arrays of n_groups device pointers");
  MOHGE_CHECK_ARG(T > 0, "the row-gathering entry points need T > 0");
  GroupPtrs P;
  rc = group_ptrs(D, w13, w2, dw13, dw2, &P);
  if (rc) return rc;
  const DgateArgs dg = {dy, y_perm, prow_of, gate_w, dgate_w};
  return expert_bwd_impl(D, P, dy_perm, x, au_saved, h_saved, counts, aligned_offsets, dau, dx_perm,
                         accumulate, carve(D, ws), (cudaStream_t)stream, &dg, tok_of_prow);
}

int32_t mohge_row_tokens(const mohge_config* cfg, int64_t T, const int32_t* counts,
                         const int32_t* offsets, const int32_t* aligned_offsets,
                         const int32_t* src_of, int32_t* tok_of_prow, void* stream) {
  Dims D;
  int32_t rc = make_dims(cfg, T, &D);
  if (rc) return rc;
  REQ_PTR(counts); REQ_PTR(offsets); REQ_PTR(aligned_offsets); REQ_PTR(src_of); REQ_PTR(tok_of_prow);
  return launch_token_of_row(D, counts, offsets, aligned_offsets, src_of, tok_of_prow, (cudaStream_t)stream);
}

int32_t mohge_expert_bwd_dy(const mohge_config* cfg, int64_t T, const void* dy,
                            const int32_t* tok_of_prow, const void* x_perm, const void* au_saved,
                            const void* h_saved, const int32_t* counts,
                            const int32_t* aligned_offsets, const void* const* w13,
                            const void* const* w2, void* dau, void* dx_perm, float* const* dw13,
                            float* const* dw2, int32_t accumulate, const void* y_perm,
                            const int32_t* prow_of, const float* gate_w, float* dgate_w, void* hs,
                            float* row_gate, void* ws, void* stream) {
  Dims D;
  int32_t rc = make_dims(cfg, T, &D);
  if (rc) return rc;
  REQ_PTR(dy); REQ_PTR(tok_of_prow); REQ_PTR(x_perm); REQ_PTR(au_saved); REQ_PTR(h_saved); REQ_PTR(counts);
  REQ_PTR(aligned_offsets); REQ_PTR(dau); REQ_PTR(dx_perm); REQ_PTR(ws);
  REQ_PTR(y_perm); REQ_PTR(prow_of); REQ_PTR(gate_w); REQ_PTR(dgate_w); REQ_PTR(hs); REQ_PTR(row_gate);
  MOHGE_CHECK_ARG(w13 && w2 && dw13 && dw2, "w13, w2, dw13, dw2 must be host arrays of n_groups device pointers");
  MOHGE_CHECK_ARG(T > 0, "the row-gathering entry points need T > 0");
  GroupPtrs P;
  rc = group_ptrs(D, w13, w2, dw13, dw2, &P);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  rc = launch_row_gate(D, prow_of, gate_w, row_gate, st);
  if (rc) return rc;
  const DgateArgs dg = {dy, y_perm, prow_of, gate_w, dgate_w};
  const DyFuse dyf = {tok_of_prow, row_gate, hs};
  return expert_bwd_impl(D, P, dy, x_perm, au_saved, h_saved, counts, aligned_offsets, dau, dx_perm,
                         accumulate, carve(D, ws), st, &dg, nullptr, &dyf);
}

int32_t mohge_dispatch_bwd(const mohge_config* cfg, int64_t T, const void* dx_perm,
                           const int32_t* prow_of, const void* dx_add, void* dx, void* stream) {
  Dims D;
  int32_t rc = make_dims(cfg, T, &D);
  if (rc) return rc;
  REQ_PTR(dx_perm); REQ_PTR(prow_of); REQ_PTR(dx); OPT_PTR(dx_add);
  return launch_unpermute_sum(D, dx_perm, prow_of, dx_add, dx, (cudaStream_t)stream);
}

// ---------------------------------------------------------------- shared experts
// The shared experts are one dense SwiGLU FFN over all T tokens.  They run through the grouped
// kernels as a single group with a single expert whose segment is x itself: the segment table
// {0, T rounded up to row_align} and the count {T} live in the workspace header, and the
// tensor maps end at row T, so tiles that reach past T read zeros and store nothing.
namespace {
__global__ void shared_segment_kernel(int32_t* hdr, int T, int align) {
  pdl_enter();
  hdr[0] = 0;
  hdr[1] = (T + align - 1) / align * align;
  hdr[2] = T;
}

struct SharedCtx {
  Dims Dm, Ds;          // the layer's dimensions (workspace layout) and the one-expert view
  Ws w;
  int32_t* aligned;     // {0, padded T}
  int32_t* counts;      // {T}
};

int32_t shared_ctx(const mohge_config* cfg, int64_t T, int32_t width, void* ws, SharedCtx* c) {
  int32_t rc = make_dims(cfg, T, &c->Dm);
  if (rc) return rc;
  MOHGE_CHECK_ARG(width >= 8 && width % 8 == 0, "shared_width = %d must be a positive multiple of 8", width);
  MOHGE_CHECK_ARG(ws != nullptr && aligned16(ws), "ws must be a non-NULL 16-byte aligned device pointer");
  mohge_config one = *cfg;
  one.n_groups = 1; one.experts_per_group = 1; one.k_groups = 1; one.k_experts = 1;
  for (int g = 0; g < MOHGE_MAX_GROUPS; ++g) one.group_width[g] = g == 0 ? width : 0;
  rc = make_dims(&one, T, &c->Ds);
  if (rc) return rc;
  c->Ds.Rcap = T > 0 ? T : 1;                       // rows that exist in x, dy and the saved tensors
  c->w = carve(c->Dm, ws);
  MOHGE_CHECK_ARG(ws_layout(c->Ds).tiles_cap <= c->w.tiles_cap,
                  "shared_width = %d needs a larger tile list than this layer's workspace holds", width);
  c->aligned = c->w.status + 16;                    // bytes 64..75 of the workspace header
  c->counts = c->w.status + 18;
  return MOHGE_OK;
}
}  // namespace

int32_t mohge_shared_fwd(const mohge_config* cfg, int64_t T, int32_t shared_width, const void* x,
                         const void* w13_shared, const void* w2_shared, void* au_shared,
                         void* h_shared, void* y_shared, void* ws, void* stream) {
  SharedCtx c;
  int32_t rc = shared_ctx(cfg, T, shared_width, ws, &c);
  if (rc) return rc;
  REQ_PTR(x); REQ_PTR(w13_shared); REQ_PTR(w2_shared); REQ_PTR(au_shared); REQ_PTR(h_shared);
  REQ_PTR(y_shared);
  cudaStream_t st = (cudaStream_t)stream;
  launch_dep(shared_segment_kernel, dim3(1), dim3(1), st, c.aligned, (int)T, c.Ds.align);
  MOHGE_LAUNCH_CHECK("shared_segment_kernel");
  GroupPtrs P;
  memset(&P, 0, sizeof(P));
  P.w13[0] = w13_shared; P.w2[0] = w2_shared;
  return expert_fwd_impl(c.Ds, P, x, c.counts, c.aligned, au_shared, h_shared, y_shared, c.w, st);
}

int32_t mohge_shared_bwd(const mohge_config* cfg, int64_t T, int32_t shared_width, const void* dy,
                         const void* x, const void* au_shared, const void* h_shared,
                         const void* w13_shared, const void* w2_shared, void* dau_shared,
                         void* dx_shared, float* dw13_shared, float* dw2_shared,
                         int32_t accumulate, void* ws, void* stream) {
  SharedCtx c;
  int32_t rc = shared_ctx(cfg, T, shared_width, ws, &c);
  if (rc) return rc;
  REQ_PTR(dy); REQ_PTR(x); REQ_PTR(au_shared); REQ_PTR(h_shared); REQ_PTR(w13_shared);
  REQ_PTR(w2_shared); REQ_PTR(dau_shared); REQ_PTR(dx_shared); REQ_PTR(dw13_shared);
  REQ_PTR(dw2_shared);
  cudaStream_t st = (cudaStream_t)stream;
  launch_dep(shared_segment_kernel, dim3(1), dim3(1), st, c.aligned, (int)T, c.Ds.align);
  MOHGE_LAUNCH_CHECK("shared_segment_kernel");
  GroupPtrs P;
  memset(&P, 0, sizeof(P));
  P.w13[0] = w13_shared; P.w2[0] = w2_shared; P.dw13[0] = dw13_shared; P.dw2[0] = dw2_shared;
  return expert_bwd_impl(c.Ds, P, dy, x, au_shared, h_shared, c.counts, c.aligned, dau_shared,
                         dx_shared, accumulate, c.w, st);
}

int32_t mohge_route_bwd(const mohge_config* cfg, int64_t T, const void* x, const void* w_router,
                        const float* dgate_w, const float* gs_saved, const float* esp_saved,
                        const int32_t* group_idx, const int32_t* expert_idx,
                        const int32_t* group_count, const int32_t* expert_count, float* dlogits,
                        void* dx, float* dw_router, void* ws, void* stream) {
  Dims D;
  int32_t rc = make_dims(cfg, T, &D);
  if (rc) return rc;
  REQ_PTR(x); REQ_PTR(w_router); REQ_PTR(dgate_w); REQ_PTR(gs_saved); REQ_PTR(esp_saved);
  REQ_PTR(group_idx); REQ_PTR(expert_idx); REQ_PTR(dlogits); REQ_PTR(dx); REQ_PTR(dw_router);
  REQ_PTR(ws);
  MOHGE_CHECK_ARG((group_count == nullptr) == (expert_count == nullptr),
                  "group_count and expert_count must both be given or both be NULL");
  cudaStream_t st = (cudaStream_t)stream;
  const bool tc = D.bf16 && !force_simt();
  const Ws w = carve(D, ws);
  const int pitch16 = (D.NL + 7) / 8 * 8;
  rc = launch_router_bwd_elementwise(D, *cfg, dgate_w, nullptr, gs_saved, esp_saved, group_idx,
                                     expert_idx, group_count, expert_count, dlogits,
                                     tc ? w.dl16 : nullptr, pitch16, st);
  if (rc) return rc;
  const int f32 = D.bf16 ? 0 : 1;
  if (T == 0) {
    MOHGE_CUDA(cudaMemsetAsync(dw_router, 0, sizeof(float) * D.NL * D.d, st));
    return MOHGE_OK;
  }
  if (tc) {
    // BF16 copy of dlogits feeds both router-backward GEMMs on the tensor cores
    rc = launch_tc_plain(D, ROLE_ROUTER_DW, x, w.dl16, pitch16, dw_router, nullptr, w.rdw, w.status, st);
    if (rc) return rc;
    return launch_tc_plain(D, ROLE_ROUTER_DX, w.dl16, w_router, pitch16, dx, nullptr, nullptr, w.status, st);
  }
  // dw_router[NL, d] = dlogits^T . x
  rc = launch_simt_plain(D.NL, D.d, (int)T, dlogits, 1, 1, D.NL, x, f32, 1, D.d, dw_router, 1, D.d,
                         nullptr, 0, st);
  if (rc) return rc;
  // dx[T, d] += dlogits . W_r
  return launch_simt_plain((int)T, D.d, D.NL, dlogits, 1, D.NL, 1, w_router, f32, 1, D.d, dx, f32,
                           D.d, nullptr, 1, st);
}

}  // extern "C"
