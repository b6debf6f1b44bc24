// Shared host/device declarations of the MoHGE library (internal; the public ABI is include/mohge.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "mohge.h"

namespace mohge {

// ---------------------------------------------------------------- errors
void set_error(const char* fmt, ...);
int32_t cuda_fail(cudaError_t e, const char* what);

#define MOHGE_CHECK_ARG(cond, ...)          \
  do {                                      \
    if (!(cond)) {                          \
      ::mohge::set_error(__VA_ARGS__);      \
      return MOHGE_ERR_INVALID_ARG;         \
    }                                       \
  } while (0)

#define MOHGE_CUDA(call)                                        \
  do {                                                          \
    cudaError_t e__ = (call);                                   \
    if (e__ != cudaSuccess) return ::mohge::cuda_fail(e__, #call); \
  } while (0)

extern unsigned long long g_launches;   // kernels launched by this library (host-side count)

#define MOHGE_LAUNCH_CHECK(name)                                   \
  do {                                                             \
    cudaError_t e__ = cudaGetLastError();                          \
    if (e__ != cudaSuccess) return ::mohge::cuda_fail(e__, name);  \
    ++::mohge::g_launches;                                         \
  } while (0)

// ---------------------------------------------------------------- dependent launches
// Every kernel of the library is launched with the programmatic-stream-serialization attribute
// (unless MOHGE_PDL=0) and starts with pdl_enter(): the block lets the next kernel of the stream
// be scheduled as soon as SM resources allow, then waits until the previous kernel has completed
// and its writes are visible.  The wait is the first thing a block does, so the order of all
// memory effects is that of ordinary stream launches; what overlaps is launch latency and block
// scheduling.  (The tensor-core GEMM kernel places the wait after its own set-up instead.)
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_enter() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
#endif
bool dependent_launch();   // false when the "pdl" switch is 0

// ---------------------------------------------------------------- switches and per-device facts
// Debugging switches.  Each is read ONCE from its environment variable, the first time any
// switch is asked for, and can afterwards be changed only through mohge_set_switch(); -1 means
// "not set: the library's own rule decides".
enum Switch { SW_PDL = 0, SW_TC_CG = 1, SW_TC_WIDE = 2, SW_FORCE_SIMT = 3, SW_ROUTE_FUSED = 4, SW_COUNT = 5 };
int switch_value(int which);
// What the launchers need to know about the current device, looked up once per device ordinal
// (a process may drive several GPUs; kernel attributes such as the dynamic shared-memory limit
// are per device too, see launch_role in gemm_tc.cu).
constexpr int kMaxDevices = 64;
struct DeviceInfo {
  int ordinal, sm_count, cc_major, cc_minor;
};
int32_t current_device(DeviceInfo* out);

template <typename... KArgs, typename... Args>
inline void launch_dep(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = dependent_launch() ? 1 : 0;
  (void)cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);   // error read by MOHGE_LAUNCH_CHECK
}

// ---------------------------------------------------------------- derived sizes
struct Dims {
  int d, Ng, N, P, Ne, NL, Kg, Ke, Wmax, align;
  int W[MOHGE_MAX_GROUPS];
  int64_t T, R, Rcap;
  bool bf16;
};

int32_t make_dims(const mohge_config* cfg, int64_t T, Dims* out);  // validates the config

static inline int ceil_div(int64_t a, int64_t b) { return (int)((a + b - 1) / b); }

// ---------------------------------------------------------------- workspace layout
// [0, 256)            device status word (int32) and padding
// stats partials      double [kStatsBlocks][NL]
// dispatch histogram  int32 [chunks][Ne] (per-chunk counts) and the same size of chunk bases
// dlogits (BF16)      [T][NLp], NLp = NL rounded up to 8 (operand of the router-backward GEMMs)
// router dW partials  float [splits][NL][d]: split-K partial sums of dw_router (BF16 path)
// tile list           int32 count (+pad to 16 B) followed by int4 entries
constexpr int kStatsBlocks = 296;
constexpr int kDispatchChunk = 256;  // tokens per dispatch block

struct WsLayout {
  int64_t status_off, stats_off, hist_off, base_off, dl16_off, rdw_off, tiles_off, dgp_off, total;
  int dgate_slots;       // 128-column slots per row of the gate-gradient partial sums
  int64_t tiles_cap;
  int chunks;
};
WsLayout ws_layout(const Dims& D);
// Split-K factor of the router weight-gradient GEMM: its output has only d/128 tiles, so the
// token dimension is cut into this many ranges to occupy the SMs (partials summed in fixed order).
int router_dw_splits(const Dims& D);

// One unit of GEMM work: expert e, output tile origin (m0, n0), and a role-specific extent.
struct __align__(16) Tile {
  int32_t e, m0, n0, ext;
};

struct GroupPtrs {
  const void* w13[MOHGE_MAX_GROUPS];
  const void* w2[MOHGE_MAX_GROUPS];
  float* dw13[MOHGE_MAX_GROUPS];
  float* dw2[MOHGE_MAX_GROUPS];
};

struct GroupShape {
  int W[MOHGE_MAX_GROUPS];
  int Ng, N, d, Wmax;
};

enum GemmRole {
  ROLE_FWD1 = 0,        // AU[rows, 2W]   = Xp[rows, d]    . W13^T
  ROLE_FWD2 = 1,        // Yp[rows, d]    = H[rows, W]     . W2^T
  ROLE_DGRAD_DOWN = 2,  // dH[rows, W]    = dYp[rows, d]   . W2
  ROLE_DGRAD_13 = 3,    // dXp[rows, d]   = dAU[rows, 2W]  . W13
  ROLE_WGRAD_DOWN = 4,  // dW2[d, W]      = dYp^T . H      (contraction over the expert's rows)
  ROLE_WGRAD_13 = 5,    // dW13[2W, d]    = dAU^T . Xp
  ROLE_LOGITS = 6,      // logits[T, NL]  = x . W_r^T            (router, single problem)
  ROLE_ROUTER_DW = 7,   // dW_r[NL, d]    = dlogits^T . x
  ROLE_ROUTER_DX = 8,   // dx[T, d]      += dlogits . W_r
};

// Parameters of the device-side tile scheduler (build_tiles_kernel).
struct TilePlan {
  int role, BM, Ng, N, Ne, d;
  int BN[MOHGE_MAX_GROUPS];     // tile width per group
  int Mext[MOHGE_MAX_GROUPS];   // wgrad only: rows of the output (d or 2W)
  int Next[MOHGE_MAX_GROUPS];   // columns of the output
  int Kcost[MOHGE_MAX_GROUPS];  // row-tiled roles: contraction length (cost of one tile)
  int wide;                     // 1: pair neighbouring n-tiles into double-width entries (kTileWide)
};
// A tile-list entry with this bit set in n0 covers TWO neighbouring n-tiles (n0 and n0 + BN):
// the CTA pair computes both from one pass over A (the tensor-core path only).
constexpr int32_t kTileWide = 1 << 30;
TilePlan make_plan(const Dims& D, int role, int BM, const int* BN, bool fused_swiglu);
int32_t launch_build_tiles_plan(const TilePlan& p, const int32_t* aligned, int32_t* tile_count,
                                Tile* tiles, int64_t tiles_cap, int32_t* status, cudaStream_t st);
GroupShape make_group_shape(const Dims& D);

// ---------------------------------------------------------------- launchers (each enqueues on `st`)
// router.cu
int32_t launch_router_select(const Dims& D, const float* logits, int32_t* group_idx,
                             int32_t* expert_idx, float* gate_w, float* gs, float* esp,
                             int32_t* status, cudaStream_t st);
int32_t launch_aux_stats(const Dims& D, const mohge_config& cfg, const float* gs, const float* esp,
                         const int32_t* group_idx, const int32_t* expert_idx, int32_t* group_count,
                         float* group_psum, int32_t* cnt_routed, int32_t* cnt_lit,
                         float* expert_psum, float* loss_out, double* partials, cudaStream_t st);
int32_t launch_router_bwd_elementwise(const Dims& D, const mohge_config& cfg, const float* dgate,
                                      const float* gate_unused, const float* gs, const float* esp,
                                      const int32_t* group_idx, const int32_t* expert_idx,
                                      const int32_t* group_count, const int32_t* expert_count,
                                      float* dlogits, __nv_bfloat16* dl16, int dl16_pitch,
                                      cudaStream_t st);

// dispatch.cu
constexpr int kGatherSlack = 128;   // rows of the gather map past mohge_perm_rows (a pair's tile may reach them)
int32_t launch_dispatch(const Dims& D, const void* x, const int32_t* expert_idx, int32_t* counts,
                        int32_t* offsets, int32_t* aligned, int32_t* row_of, int32_t* prow_of,
                        int32_t* src_of, void* x_perm, int32_t* hist, int32_t* base,
                        int32_t* status, cudaStream_t st, int32_t* tok_of_prow = nullptr);
int32_t launch_combine(const Dims& D, const void* y_perm, const int32_t* prow_of,
                       const float* gate_w, const void* add, void* y, cudaStream_t st);
int32_t launch_combine_bwd(const Dims& D, int mode, const void* dy, const void* y_perm,
                           const int32_t* prow_of, const float* gate_w, const int32_t* counts,
                           const int32_t* aligned, void* dy_perm, float* dgate_w, cudaStream_t st);
// tok_of_prow[r] = token whose row sits at physical row r, T for padding rows and the 128 rows
// past the last segment
int32_t launch_token_of_row(const Dims& D, const int32_t* counts, const int32_t* offsets,
                            const int32_t* aligned, const int32_t* src_of, int32_t* tok_of_prow,
                            cudaStream_t st);
// row_gate[prow_of[t, k]] = gate_w[t, k], 0 at every other physical row (padding)
int32_t launch_row_gate(const Dims& D, const int32_t* prow_of, const float* gate_w, float* row_gate,
                        cudaStream_t st);
int32_t launch_dgate_reduce(const Dims& D, const int* bn, const float* part, int slots,
                            const int32_t* prow_of, const float* gate_w, const int32_t* aligned,
                            const void* dy, const void* y_perm, float* dgate_w, cudaStream_t st);
int32_t launch_unpermute_sum(const Dims& D, const void* dx_perm, const int32_t* prow_of,
                             const void* add, void* dx, cudaStream_t st);

// gemm_simt.cu
int32_t launch_build_tiles(const Dims& D, int role, int BM, int BN, const int32_t* counts,
                           const int32_t* aligned, int32_t* tile_count, Tile* tiles,
                           int64_t tiles_cap, int32_t* status, cudaStream_t st);
int32_t launch_simt_grouped(const Dims& D, int role, const GroupPtrs& P, const void* A,
                            const void* B, void* C, const int32_t* aligned, int accumulate,
                            const int32_t* tile_count, const Tile* tiles, cudaStream_t st);
int32_t launch_swiglu_fwd(const Dims& D, const int32_t* aligned, void* au, void* h,
                          cudaStream_t st);
int32_t launch_swiglu_bwd(const Dims& D, const int32_t* aligned, const void* au, void* dau,
                          cudaStream_t st);
int32_t launch_zero_empty_wgrad(const Dims& D, const GroupPtrs& P, const int32_t* counts,
                                cudaStream_t st);
// plain (single problem) GEMMs of the router:  C[M,N] (+)= A . B^T forms with generic strides
int32_t launch_simt_plain(int M, int N, int K, const void* A, int a_f32, int64_t sAm, int64_t sAk,
                          const void* B, int b_f32, int64_t sBn, int64_t sBk, void* C, int c_f32,
                          int64_t sCm, const float* bias, int accumulate, cudaStream_t st);

// gemm_tc.cu (tcgen05 path, BF16)
// gather != nullptr (FWD1, WGRAD_13 only): the x_perm operand (A of FWD1, B of WGRAD_13) is x
// itself, [T, d], and row r of the permuted numbering is row gather[r] of it (>= T: zeros)
// The experts' backward without dy_perm: DGRAD_DOWN and WGRAD_DOWN gather the rows of dy [T, d]
// (A operand) through tok_of_prow; DGRAD_DOWN scales by row_gate and writes hs = gate * H.
struct DyFuse {
  const int32_t* tok_of_prow;    // [mohge_perm_rows + 128]
  const float* row_gate;         // [mohge_perm_rows]: gate of the pair at a physical row, 0 for padding
  void* hs;                      // layout of h_saved
};
int32_t launch_tc_grouped(const Dims& D, int role, const GroupPtrs& P, const void* A,
                          const void* B, void* C, void* C2, const int32_t* counts,
                          const int32_t* aligned, int accumulate, int32_t* tile_count, Tile* tiles,
                          int64_t tiles_cap, int32_t* status, cudaStream_t st, bool list_prebuilt = false,
                          float* dgate_part = nullptr, int dgate_slots = 0,
                          const int32_t* gather = nullptr, const struct DyFuse* dyf = nullptr);
// UMMA N of a group in ROLE_DGRAD_DOWN (128 or 256): which 128-column slots of dgate_part are written
int tc_dgrad_down_bn(const Dims& D, int g);
TilePlan tc_tile_plan(const Dims& D, int role);
// builds up to four tile lists with one launch; list i goes to tile_count + 64 * i (ints) and
// tiles + i * tiles_cap
constexpr int kMaxLists = 4;
int32_t launch_build_tiles_multi(const TilePlan* plans, int nplans, const int32_t* aligned,
                                 int32_t* tile_count, Tile* tiles, int64_t tiles_cap,
                                 int32_t* status, cudaStream_t st);

// Outputs of the selection (Eq. 2-6) for the LOGITS launch that selects in its epilogue.
struct RouteOut {
  int32_t* group_idx;
  int32_t* expert_idx;
  float* gate_w;
  float* gs;
  float* esp;
};
// route != nullptr (LOGITS only): the launch may also do the selection; *routed says whether it did
// (it does when the shape is covered, the contraction is not split and the switch is not 0).
int32_t launch_tc_plain(const Dims& D, int role, const void* A, const void* B, int64_t b_pitch_elems,
                        void* C, const float* bias, float* partials, int32_t* status, cudaStream_t st,
                        const RouteOut* route = nullptr, bool* routed = nullptr);

}  // namespace mohge
