// Ragged grouped GEMMs of the expert layer on the 5th-generation tensor cores (sm_100a):
// tcgen05.mma kind::f16 (BF16 operands, FP32 accumulators in tensor memory), operands staged in
// shared memory by TMA (cp.async.bulk.tensor, 128-byte swizzle), a multi-stage mbarrier pipeline,
// double-buffered accumulators, and warp-specialised roles:
//   warp 0      TMA producer (one elected lane)
//   warp 1      tensor-memory owner and MMA issuer (one elected lane)
//   warps 2..5  epilogue: tcgen05.ld -> registers -> fused element-wise math -> swizzled staging
//               buffers in shared memory -> TMA stores (every global write of the expert roles is
//               a full 128-byte row piece; the SwiGLU backward also reads A and U through TMA)
//   warp 6      only in the row-gathering form (GATHER = 1, see "gathering form" below): forwards
//               the completion of the producer warp's asynchronous row copies to the MMA issuer
//   warps 6..9  only in the router-logits GEMM whose epilogue also selects (Eq. 2-6): a second
//               epilogue warp for every quarter of the accumulator rows (route_epilogue.cuh)
// One persistent CTA per SM (a CTA pair per two SMs for the expert roles; single CTAs when the
// batch brings 128 rows per expert or fewer) walks the device-built, cost-sorted tile list with a
// fixed stride, in alternating directions when tile costs differ.  The kernel is launched as a
// programmatic dependent of its predecessor: barriers and tensor memory are set up before
// griddepcontrol.wait, every global access comes after it.
//
// Six roles share the kernel (C = A . B^T over a contraction index k):
//   FWD1        [A | U] = Xp . W13^T, fused SwiGLU epilogue writes A, U and H = silu(A) * U.
//               The gate tile and the up tile of the same hidden columns are two TMA boxes (one
//               per CTA of a pair) that form one B operand, so ONE MMA covers both and no weight
//               repacking is needed.
//   FWD2        Yp = H . W2^T
//   DGRAD_DOWN  dH = dYp . W2         (B read MN-major), epilogue turns dH into dA, dU using A, U
//   DGRAD_13    dXp = [dA | dU] . W13 (B read MN-major)
//   WGRAD_DOWN  dW2  = dYp^T . H      (A and B read MN-major, contraction over the expert's rows)
//   WGRAD_13    dW13 = [dA | dU]^T . Xp
// plus three single-problem GEMMs of the router (logits, with the two-level selection in the
// epilogue; router weight gradient; router part of dx).  In the gathering form the rows of an
// operand that the default route reads from a permuted copy (Xp of FWD1 and WGRAD_13, dYp of
// DGRAD_DOWN and WGRAD_DOWN) are fetched from the unpermuted tensor through a row map.
// Expert segments start at multiples of 128 physical rows with zero padding rows, so a 128-row
// tile never straddles two experts and padding contributes exact zeros to the weight gradients.
// Hidden widths that are not multiples of the tile are handled by TMA's out-of-bounds zero fill
// on loads and by the clipping of TMA stores.
//
// Every wait is bounded: after about one second without progress the waiting thread records
// (1 << 24 | site) in the status word, raises a CTA-wide abort flag and every role leaves its
// loop; the CTA then lets copies in flight land, frees its tensor memory and returns.

#include <cuda.h>

#include <atomic>
#include <mutex>

#include "common.cuh"
#include "route_epilogue.cuh"

namespace mohge {
namespace {

constexpr int BM = 128;          // UMMA M (rows of an output tile)
constexpr int BK = 64;           // contraction elements per pipeline stage (128 bytes of BF16)
constexpr int kABytes = BM * BK * 2;          // 16 KiB: 128 rows of A per CTA and stage
constexpr int kThreads = 192;                 // producer, MMA issuer, four epilogue warps
// Row-gathering form (GATHER = 1): kGatherWarps warps copy rows (the producer warp and
// kGatherWarps - 1 more), one more warp relays their completions to the MMA issuer.  More
// gathering warps bring nothing (measured with 1, 2 and 4: 854 / 833 / 833 clocks per k-block in
// FWD1): the copies are bound by what an SM keeps in flight through its load path, not by issue.
#ifndef MOHGE_GATHER_WARPS
#define MOHGE_GATHER_WARPS 1
#endif
constexpr int kGatherWarps = MOHGE_GATHER_WARPS;     // 1, 2 or 4
constexpr int kThreadsGather = kThreads + 32 * kGatherWarps;
// router-logits GEMM in its six-stage form: kRouteSplit epilogue warps per quarter of the rows
constexpr int kThreadsRoute = 64 + 128 * kRouteSplit;
template <int ROLE, int WIDE, int GATHER> __host__ __device__ constexpr int block_threads() {
  return GATHER ? kThreadsGather : (ROLE == ROLE_LOGITS && WIDE == 2) ? kThreadsRoute : kThreads;
}
constexpr int kAccCols = 256;                 // tensor-memory columns per accumulator buffer

// Build-time option -DMOHGE_TC_COUNTERS: every CTA adds, per role, the clocks its MMA issuer spent
// in its loop, waiting for operands (full barriers) and waiting for a free accumulator (the
// exposed part of the epilogue), the clocks per k-block in the middle of long tiles (steady
// state), the clocks its producer waited for a free stage, the clocks the first epilogue warp
// waited for an accumulator, the tiles and k-blocks it processed and its lifetime in
// nanoseconds.  mohge_debug_tc_counters() copies the table to the host.  This is how the balance
// of the tile scheduler over the SMs and the cost of the tile boundaries are measured.  Off in
// the normal build; with it MOHGE_TC_GRID=<n> also limits the persistent grid to n CTAs.
#ifdef MOHGE_TC_COUNTERS
constexpr int kCntRoles = 9, kCntCtas = 160, kCntSlots = 12;
__device__ unsigned long long g_tc_counters[kCntRoles][kCntCtas][kCntSlots];
#define TCC(...) __VA_ARGS__
#else
#define TCC(...)
#endif

// CG = CTAs per MMA (tcgen05 cta_group).  CG = 2 pairs the two CTAs of a cluster on one
// 256 x N tile: each CTA stages its own 128 rows of A and HALF of B, so operand traffic per FLOP
// drops by a third and the smaller stages allow a five-deep pipeline.
// Epilogue staging: each of the four epilogue warps owns a ring of four 4 KiB buffers
// (32 rows x 128 bytes, 128-byte swizzle: the layout a TMA box of 32 rows expects).
constexpr int kStgBufBytes = 4096;
constexpr int kSlots = 4;
constexpr int kStgBytes = 4 * kSlots * kStgBufBytes;         // 64 KiB per CTA

// WIDE = 1 (CTA pairs only): the pair works on double-width entries, 256 x 512 outputs from ONE
// pass over A, the two 256-column halves in the two accumulator buffers.  A stage then holds A
// and the pair's halves of both B tiles (48 KiB per CTA, three stages), which cuts the operand
// bytes per FLOP by a quarter; the price is that the epilogue of an entry no longer overlaps
// the MMAs of the next one.  It pays where the contraction is long (see launch_tc_grouped).
// WIDE = 2 (single CTAs, router logits with at most 160 outputs): a B tile of 20 KiB instead of
// 32 and no staging ring (that epilogue stores from registers), so the shared memory holds six
// stages instead of three.  That GEMM streams x once and is bound by the bytes it keeps in flight
// against the memory latency.
template <int CG, int WIDE = 0> struct Geo {
  static constexpr int kStages = WIDE == 2 ? 6 : (CG == 2 && !WIDE) ? 5 : 3;
  // epilogue staging ring; six-stage form: the lists the epilogue warps of a row quarter exchange
  static constexpr int kStg = WIDE == 2 ? (kRouteSplit - 1) * 128 * 2 * kRouteFuseMaxKe * 4 : kStgBytes;
  static constexpr int kBBytes = WIDE == 2 ? 160 * BK * 2 : 256 / CG * BK * 2;   // one B tile per CTA: 32 KiB or 16 KiB
  static constexpr int kStageBytes = kABytes + kBBytes * (WIDE == 1 ? 2 : 1);
  static constexpr int kSmemBytes = kStages * kStageBytes + kStg + 1024 + 512 + 1088;   // + segment table
  static constexpr int kTileM = BM * CG;
};

enum Epi { EPI_BF16 = 0, EPI_SWIGLU_FWD = 1, EPI_SWIGLU_BWD = 2, EPI_F32 = 3, EPI_LOGITS = 4, EPI_F32_T = 5, EPI_BF16_ACC = 6 };

template <int ROLE> struct RoleTraits;
template <> struct RoleTraits<ROLE_FWD1>       { static constexpr int A_MN = 0, B_MN = 0, EPI = EPI_SWIGLU_FWD; };
template <> struct RoleTraits<ROLE_FWD2>       { static constexpr int A_MN = 0, B_MN = 0, EPI = EPI_BF16; };
template <> struct RoleTraits<ROLE_DGRAD_DOWN> { static constexpr int A_MN = 0, B_MN = 1, EPI = EPI_SWIGLU_BWD; };
template <> struct RoleTraits<ROLE_DGRAD_13>   { static constexpr int A_MN = 0, B_MN = 1, EPI = EPI_BF16; };
template <> struct RoleTraits<ROLE_WGRAD_DOWN> { static constexpr int A_MN = 1, B_MN = 1, EPI = EPI_F32; };
template <> struct RoleTraits<ROLE_WGRAD_13>   { static constexpr int A_MN = 1, B_MN = 1, EPI = EPI_F32; };
// single-problem ("plain") GEMMs of the router: tiles are decoded from the tile index
template <> struct RoleTraits<ROLE_LOGITS>     { static constexpr int A_MN = 0, B_MN = 0, EPI = EPI_LOGITS; };
template <> struct RoleTraits<ROLE_ROUTER_DW>  { static constexpr int A_MN = 1, B_MN = 1, EPI = EPI_F32_T; };
template <> struct RoleTraits<ROLE_ROUTER_DX>  { static constexpr int A_MN = 0, B_MN = 1, EPI = EPI_BF16_ACC; };
template <int ROLE> __host__ __device__ constexpr bool is_plain() { return ROLE >= ROLE_LOGITS; }

struct TcParams {
  CUtensorMap mapA[MOHGE_MAX_GROUPS];
  CUtensorMap mapB[MOHGE_MAX_GROUPS];
  // epilogue outputs, boxes of 32 rows x 128 bytes.  FWD1: A, U, H regions per group;
  // FWD2 / DGRAD_13 / ROUTER_DX: [0][0]; DGRAD_DOWN: dA, dU regions per group; WGRAD: FP32
  // [N, rows, cols]
  CUtensorMap mapO[3][MOHGE_MAX_GROUPS];
  CUtensorMap mapE[2][MOHGE_MAX_GROUPS];   // DGRAD_DOWN epilogue inputs: saved A and U regions
  // Row gather (FWD1: A operand, WGRAD_13: B operand): instead of x_perm the operand is
  // gather_src = x itself, [gather_rows, d], and row r of the permuted numbering is row
  // gather[r] of it; indices >= gather_rows read as zeros (padding rows).
  const int32_t* gather;
  const void* gather_src;
  int gather_rows;
  // Gathering form of the two roles that read dy_perm (DGRAD_DOWN and WGRAD_DOWN: A operand):
  // gather_src = dy [T, d] itself, unscaled.  DGRAD_DOWN then multiplies the accumulator row r by
  // row_gate[r] (the gate of the routed pair at physical row r, 0 for padding rows) and also
  // writes hs = row_gate * H (the layout of h_saved), the B operand WGRAD_DOWN needs instead of H.
  const float* row_gate;
  __nv_bfloat16* hs;
  int hs_pitch;                  // elements per row of hs
  GroupShape gs;
  GroupPtrs gp;
  int BN[MOHGE_MAX_GROUPS];      // UMMA N per group (FWD1: gate half + up half)
  // MN-major operands whose MN extent is a multiple of 64 are mapped with one more dimension
  // (64 elements, k rows, 64-element blocks[, expert]) so that ONE box brings all the 8 KiB
  // swizzle blocks of a stage; otherwise each block is a box of its own
  unsigned char a_blk[MOHGE_MAX_GROUPS], b_blk[MOHGE_MAX_GROUPS];
  const int32_t* aligned;
  const int32_t* tile_count;
  const Tile* tiles;
  __nv_bfloat16* C;              // FWD1: au, FWD2: y_perm, DGRAD_DOWN: dau, DGRAD_13: dx_perm
  __nv_bfloat16* C2;             // FWD1: h
  const __nv_bfloat16* E;        // DGRAD_DOWN: au_saved
  int accumulate;
  int32_t* status;
  // plain roles: C[M, N] over contraction K; tile ti -> (ti / ntn, ti % ntn)
  int plain_total, plain_ntn, plain_M, plain_N, plain_K;
  int plain_splits, plain_kchunk;   // split-K of ROUTER_DW and LOGITS: ranges of plain_kchunk k-blocks
  // LOGITS with more row tiles than CTAs: instead of tiles dealt round robin (512 tiles over 148
  // CTAs leave the last of four rounds half empty) every CTA takes one contiguous range of rows,
  // the same for all, cut into 128-row tiles and, where 64 rows or fewer remain, a last tile
  // whose A box is 64 rows high (mapA[1]); the kernel is bound by streaming x once.
  int plain_balanced;
  float* Cf;                     // LOGITS: logits [T, NL]; ROUTER_DW: dw_router [NL, d]
  RouteFuse rf;                  // LOGITS: selection (Eq. 2-6) in the epilogue; B staged experts first
  const float* bias;             // LOGITS: optional logit bias [NL]
  // DGRAD_DOWN, optional: per physical row and 128-column slot of the hidden axis, the sum over
  // the tile's columns of dH_j * h_j (the gate gradient times the gate, see dgate_reduce_kernel)
  float* dgate_part;
  int dgate_slots;
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

constexpr uint64_t kWaitBudgetNs = 1000ull * 1000ull * 1000ull;

// Bounded wait.  Returns false when the CTA is aborting (this wait or another one gave up).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int32_t* status, int site) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_ns();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 255u) == 0) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > kWaitBudgetNs) {
        atomicCAS(status, 0, (1 << 24) | site);
        *abort_flag = 1;
        return false;
      }
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "l"(pol) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5}], [%2], %6;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "l"(pol) : "memory");
}

// L2 eviction priorities.  Epilogue outputs are written once and not read again by the same
// launch, so they are marked evict-first: left at normal priority they push the operand tiles,
// which every CTA of a wave re-reads, out of L2.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}

__device__ __forceinline__ uint64_t l2_policy_evict_normal() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
  return p;
}
// Operand loads.  An expert's weights (B of the forward and dgrad roles) are needed again by every
// row tile of the expert, i.e. by several waves of CTAs, while 30 MB of outputs and the other
// operand stream through L2 in between; so are both operand slabs of the weight-gradient roles
// (each is shared by the tiles of a whole output row or column).  Marked evict-last they stay:
// measured at the large workload, step 45.5 -> 44.8 ms (four runs each, same GPU); the
// activation operand of the forward and dgrad roles marked evict-first instead cost 1.2 ms, marked
// evict-last it changed nothing.
template <int ROLE> __device__ __forceinline__ uint64_t operand_policy(int operand_b) {
  const bool keep = ROLE == ROLE_WGRAD_DOWN || ROLE == ROLE_WGRAD_13 || (ROLE <= ROLE_DGRAD_13 && operand_b);
  return keep ? l2_policy_evict_last() : l2_policy_evict_normal();
}
// ---- TMA stores from the epilogue staging buffers (bulk async-groups)
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1, uint64_t pol) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group.L2::cache_hint [%0, {%2, %3}], [%1], %4;"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1), "l"(pol) : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2, uint64_t pol) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group.L2::cache_hint [%0, {%2, %3, %4}], [%1], %5;"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2), "l"(pol) : "memory");
}
// element-wise FP32 add into global memory (each output element is touched by exactly one box)
__device__ __forceinline__ void tma_reduce_add_3d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2) {
  asm volatile("cp.reduce.async.bulk.tensor.3d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "l"(pol) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// generic-proxy writes to shared memory become visible to the async proxy (TMA)
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Address of 16-byte piece j of row r in a staging buffer (32 rows x 128 B, 128-byte swizzle)
__device__ __forceinline__ uint32_t stg_addr(uint32_t buf, int r, int j) {
  return buf + (uint32_t)r * 128u + (uint32_t)((j ^ (r & 7)) << 4);
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ void st_shared_u32(uint32_t addr, uint32_t x) {
  asm volatile("st.shared.b32 [%0], %1;" ::"r"(addr), "r"(x) : "memory");
}
__device__ __forceinline__ uint32_t ld_shared_u32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ uint4 ld_shared_v4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
  return v;
}

// ---- CTA-pair (cluster of 2) helpers
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t mapa_rank(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx_cluster(uint32_t bar_cluster, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.relaxed.cluster.shared::cluster.b64 _, [%0], %1;" ::"r"(bar_cluster), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster) {
  asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster) : "memory");
}
// the same with release semantics at cluster scope: what this thread has observed (the landed row
// copies of the gathering form) is visible to whoever acquires the barrier's phase
__device__ __forceinline__ void mbar_arrive_release_cluster(uint32_t bar_cluster) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster) : "memory");
}
// loads of the pair signal the barrier of the leader CTA (cluster address)
__device__ __forceinline__ void tma2_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "l"(pol) : "memory");
}
__device__ __forceinline__ void tma2_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5}], [%2], %6;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "l"(pol) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(pol) : "memory");
}
__device__ __forceinline__ void tma2_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(pol) : "memory");
}
// 16 bytes global -> shared, asynchronously, no registers in between (src_bytes = 0 writes zeros)
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
// the barrier receives one arrival from this thread once all its earlier cp.async have landed
// (.noinc: the arrival is part of the barrier's expected count)
__device__ __forceinline__ void cp_async_arrive(uint32_t bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
template <int CG>
__device__ __forceinline__ void tma_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3, uint64_t pol) {
  if (CG == 2) tma2_load_4d(dst, map, bar, c0, c1, c2, c3, pol); else tma_load_4d(dst, map, bar, c0, c1, c2, c3, pol);
}
template <int CG>
__device__ __forceinline__ void tma_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, uint64_t pol) {
  if (CG == 2) tma2_load_2d(dst, map, bar, c0, c1, pol); else tma_load_2d(dst, map, bar, c0, c1, pol);
}
template <int CG>
__device__ __forceinline__ void tma_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, uint64_t pol) {
  if (CG == 2) tma2_load_3d(dst, map, bar, c0, c1, c2, pol); else tma_load_3d(dst, map, bar, c0, c1, c2, pol);
}
__device__ __forceinline__ void umma2_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// arrives on the same barrier offset in both CTAs of the pair
__device__ __forceinline__ void umma2_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// arrives on the mbarrier once every MMA issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptors (128-byte swizzle, descriptor version of sm_100).
//   K-major  : rows of 64 elements (128 B); 8-row groups 1024 B apart (stride byte offset)
//   MN-major : blocks of 64 MN-elements x 64 k-rows (one TMA box, 8 KiB, leading byte offset);
//              inside a block k-rows are 128 B apart and 8-row groups 1024 B apart
__device__ __forceinline__ uint64_t make_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr & 0x3ffffu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) |
         ((uint64_t)(sbo_bytes >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

// sigmoid and silu from the hardware exp2 and reciprocal approximations (about 2 ulp each):
// the epilogue warps run one per scheduler with nothing to hide latency behind, so the IEEE
// division sequence would cost more than the tile's MMAs.  exp overflow gives 1/inf = 0.
__device__ __forceinline__ float sigmoid_fast(float a) { return __fdividef(1.0f, 1.0f + __expf(-a)); }
__device__ __forceinline__ float silu_fast(float a) { return __fdividef(a, 1.0f + __expf(-a)); }
// Two elements at a time with the packed FP32 instructions of sm_100 (one issue slot for both
// lanes of a multiply, add or fused multiply-add); exp2 and reciprocal stay scalar.
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float rcp_approx(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float2 sigmoid2_fast(float2 a) {
  const float2 t = __fmul2_rn(a, make_float2(-1.4426950408889634f, -1.4426950408889634f));
  const float2 den = __fadd2_rn(make_float2(ex2_approx(t.x), ex2_approx(t.y)), make_float2(1.0f, 1.0f));
  return make_float2(rcp_approx(den.x), rcp_approx(den.y));
}

__device__ __forceinline__ uint32_t pack2(float a, float b) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ float bf_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

// 32 consecutive BF16 of one row; only the first `valid` (multiple of 8) columns exist
__device__ __forceinline__ void store_row32(__nv_bfloat16* p, const float (&v)[32], int valid) {
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    if (q * 8 < valid) {
      uint4 o;
      o.x = pack2(v[q * 8 + 0], v[q * 8 + 1]);
      o.y = pack2(v[q * 8 + 2], v[q * 8 + 3]);
      o.z = pack2(v[q * 8 + 4], v[q * 8 + 5]);
      o.w = pack2(v[q * 8 + 6], v[q * 8 + 7]);
      *reinterpret_cast<uint4*>(p + q * 8) = o;
    }
  }
}
__device__ __forceinline__ void load_row32(const __nv_bfloat16* p, float (&v)[32], int valid) {
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    uint4 o = make_uint4(0, 0, 0, 0);
    if (q * 8 < valid) o = *reinterpret_cast<const uint4*>(p + q * 8);
    v[q * 8 + 0] = bf_lo(o.x); v[q * 8 + 1] = bf_hi(o.x);
    v[q * 8 + 2] = bf_lo(o.y); v[q * 8 + 3] = bf_hi(o.y);
    v[q * 8 + 4] = bf_lo(o.z); v[q * 8 + 5] = bf_hi(o.z);
    v[q * 8 + 6] = bf_lo(o.w); v[q * 8 + 7] = bf_hi(o.w);
  }
}

// Epilogue pacing.  A tile's output leaves while the MMAs of the CTA's next tile run; sent as
// one burst it delays that tile's operand loads (both share the SM's path to L2) by about as
// long as the burst lasts.  The store-heavy roles therefore spread their chunks over
// kPacePct % of the next tile's MMA time (512 clocks per 64-deep k-block at full rate).
#ifndef MOHGE_PACE_PCT
#define MOHGE_PACE_PCT 75
#endif
constexpr int kPacePct = MOHGE_PACE_PCT;      // 0 = no pacing (for measurements)
__device__ __forceinline__ void pace(long long t0, int i, int n, int next_num_kb) {
  const long long target = t0 + (long long)next_num_kb * (512 * kPacePct / 100) * i / n;
  while (clock64() < target) __nanosleep(64);
}

struct TileGeom {
  int e, g, i, W, bn, m0, n0, num_kb, r0, wide;
};

// rows per CTA of the balanced LOGITS form: the same multiple of 64 for every CTA
__device__ __forceinline__ int balanced_rows(int M, int ctas) { return ((M + ctas - 1) / ctas + 63) / 64 * 64; }

template <int ROLE>
__device__ __forceinline__ Tile fetch_tile(const TcParams& p, int ti) {
  if (ROLE == ROLE_LOGITS && p.plain_balanced) {
    Tile t;
    const int ctas = (int)gridDim.x, R = balanced_rows(p.plain_M, ctas);
    const int local = ti / ctas;
    t.e = 0;
    t.n0 = 0;
    t.m0 = (ti % ctas) * R + local * BM;
    int ext = R - local * BM;
    if (ext > BM) ext = BM;
    if (ext > p.plain_M - t.m0) ext = p.plain_M - t.m0;
    t.ext = ext > 0 ? ext : 0;                             // 0: nothing left for this CTA, tile skipped
    return t;
  }
  if (is_plain<ROLE>()) {
    Tile t;
    const int per_m = p.plain_ntn * p.plain_splits;       // tile index = (m, n, split), split fastest
    const int rem = ti % per_m;
    t.e = rem % p.plain_splits;                            // split index
    t.m0 = (ti / per_m) * BM;
    t.n0 = (rem / p.plain_splits) * p.BN[0];
    t.ext = p.plain_M - t.m0 < BM ? p.plain_M - t.m0 : BM;
    return t;
  }
  return p.tiles[ti];
}

template <int ROLE>
__device__ __forceinline__ TileGeom tile_geom(const TcParams& p, const Tile& t, const int32_t* seg) {
  TileGeom q;
  if (is_plain<ROLE>()) {
    q.e = t.e; q.g = 0; q.i = 0; q.W = 0; q.bn = p.BN[0]; q.m0 = t.m0; q.n0 = t.n0; q.wide = 0;
    const int total_kb = (p.plain_K + BK - 1) / BK;
    const int kb0 = t.e * p.plain_kchunk;                  // first k-block of this split
    q.r0 = kb0 * BK;
    q.num_kb = total_kb - kb0 < p.plain_kchunk ? total_kb - kb0 : p.plain_kchunk;
    return q;
  }
  q.e = t.e;
  q.g = t.e / p.gs.N;
  q.i = t.e % p.gs.N;
  q.W = p.gs.W[q.g];
  q.bn = p.BN[q.g];
  q.m0 = t.m0;
  q.n0 = t.n0 & (kTileWide - 1);
  q.wide = (t.n0 & kTileWide) ? 1 : 0;
  q.r0 = 0;
  if (ROLE == ROLE_FWD1 || ROLE == ROLE_DGRAD_DOWN) q.num_kb = (p.gs.d + BK - 1) / BK;
  else if (ROLE == ROLE_FWD2) q.num_kb = (q.W + BK - 1) / BK;
  else if (ROLE == ROLE_DGRAD_13) q.num_kb = (2 * q.W + BK - 1) / BK;
  else {
    q.num_kb = t.ext / BK;
    q.r0 = seg[t.e];          // first physical row of the expert (table staged in shared memory)
  }
  return q;
}

template <int ROLE, int CG, int WIDE, int GATHER = 0>
__global__ void __launch_bounds__(block_threads<ROLE, WIDE, GATHER>(), 1)
tc_grouped_kernel(const __grid_constant__ TcParams p) {
  using RT = RoleTraits<ROLE>;
  using G = Geo<CG, WIDE>;
  constexpr int kStages = G::kStages;
  constexpr int kStageBytes = G::kStageBytes;
  const uint32_t cta_rank = CG == 2 ? cluster_ctarank() : 0u;   // position in the CTA pair
  const int unit = blockIdx.x / CG, unit_stride = gridDim.x / CG;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  // layout: pipeline stages | epilogue staging (4 warps x 4 buffers x 4 KiB) | barriers
  const uint32_t stg0 = smem_base + kStages * kStageBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_gen + kStages * kStageBytes + G::kStg);
  const uint32_t bar0 = stg0 + G::kStg;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kStages + s); };
  auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * kStages + b); };
  auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * kStages + 2 + b); };
  auto ein_bar = [&](int quad, int set) { return bar0 + 8u * (2 * kStages + 4 + quad * 2 + set); };
  auto gath_bar = [&](int s) { return bar0 + 8u * (2 * kStages + 12 + s); };   // row copies of a stage have landed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 12 + kStages);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  // expert segment table (aligned_offsets) staged once, so that no role chases it through global
  // memory between tiles
  int32_t* s_seg = reinterpret_cast<int32_t*>(smem_gen + kStages * kStageBytes + G::kStg + 512);
  // Programmatic dependent launch (when the host asked for it): the next kernel of the stream may
  // be scheduled onto SMs as the CTAs of this one leave, and this kernel may itself have been
  // scheduled while its predecessor was draining.  Nothing before griddep_wait() below touches
  // global memory; without the launch attribute both instructions do nothing.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  TCC(const uint64_t cnt_t0 = global_ns();
      unsigned long long* const cnt = g_tc_counters[ROLE][blockIdx.x < kCntCtas ? blockIdx.x : kCntCtas - 1];)

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      // one arrive.expect_tx per CTA of the pair, plus one relayed arrival per CTA when rows are gathered
      mbar_init(full_bar(s), GATHER ? 2 * CG : CG);
      mbar_init(empty_bar(s), 1);
      mbar_init(gath_bar(s), 32 * kGatherWarps);       // every lane of the gathering warps
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(tfull_bar(b), 1);
      mbar_init(tempty_bar(b), (block_threads<ROLE, WIDE, GATHER>() == kThreadsRoute ? 4 * kRouteSplit : 4) * CG);  // every epilogue warp
    }
    for (int i = 0; i < 8; ++i) mbar_init(ein_bar(i >> 1, i & 1), 1);   // epilogue input loads
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    if (CG == 2) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if (CG == 2) cluster_sync_all();     // the peer's barriers exist before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // barriers and TMEM are set up; from here on the predecessor's results are read
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (!is_plain<ROLE>()) {
    const int ne = p.gs.Ng * p.gs.N;
    for (int i = threadIdx.x; i <= ne; i += blockDim.x) s_seg[i] = p.aligned[i];
    __syncthreads();
  }
  const int total = (ROLE == ROLE_LOGITS && p.plain_balanced)
                        ? (int)gridDim.x * ((balanced_rows(p.plain_M, (int)gridDim.x) + BM - 1) / BM)
                        : is_plain<ROLE>() ? p.plain_total : *p.tile_count;
  // Tile of this CTA (pair) in round i.  The list is sorted by cost, heaviest first.  When the
  // costs differ (zigzag), rounds alternate direction (0..n-1, then n-1..0), so no CTA always gets
  // the heaviest tile of its round; with equal costs the plain order measured slightly faster.  Returns -1 when the round has no tile left for this CTA (last, partial round).
  const bool zigzag = (is_plain<ROLE>() || WIDE) ? false : p.tile_count[1] != 0;   // set by the list builder
  auto tile_of = [&](int i) {
    const int ti = i * unit_stride + ((zigzag && (i & 1)) ? unit_stride - 1 - unit : unit);
    return ti < total ? ti : -1;
  };
  const int rounds = (total + unit_stride - 1) / unit_stride;
  // loop variable: the round when zigzag, else the tile index itself
  const int it0 = zigzag ? 0 : unit, it_step = zigzag ? 1 : unit_stride, it_end = zigzag ? rounds : total;
  // The list entry of the NEXT tile is requested while the current one is worked on: a tile of a
  // short contraction lasts a few thousand clocks, and a dependent global load in front of each
  // one kept the MMA issuer idle for a quarter of that.
  auto prefetch_tile = [&](int it) -> Tile {
    Tile z;
    z.e = 0; z.m0 = 0; z.n0 = 0; z.ext = 0;
    if (it >= it_end) return z;
    const int ti = zigzag ? tile_of(it) : it;
    return ti < 0 ? z : fetch_tile<ROLE>(p, ti);
  };

  if (GATHER && (warp == 0 || (warp >= 6 && warp < 5 + kGatherWarps))) {
    // ================= producer, gathering form =================
    // The x_perm operand (A of FWD1, B of WGRAD_13) is not read from a permuted copy: its rows are
    // rows of x, found through the row map p.gather.  TMA has no efficient row gather (a
    // tile::gather4 copy of four 128-byte rows costs the TMA unit about 77 clocks, 6.6 B per
    // clock), so the whole producer warp brings these rows with 16-byte cp.async copies straight
    // into the swizzled stage (chunk c of row r at r * 128 + ((c ^ (r & 7)) << 4), the layout a
    // TMA box with the 128-byte swizzle produces), while lane 0 of warp 0 still issues the TMA
    // boxes of the other operand.  One warp keeps too few copies in flight against the memory
    // latency (measured: 40-50 clocks per warp-wide copy instruction), so kGatherWarps warps share
    // the rows of a stage: warp gw takes a quarter of the row slots.  Lane l takes chunk l % 8 of
    // the rows l / 8, l / 8 + 4, ...
    //   FWD1      A tile = 128 rows x 128 B per k-block; the 32 row indices of a lane are fixed
    //             for a tile and live in registers
    //   WGRAD_13  B tile = blocks of 64 k-rows x 128 B; the rows are the contraction index, so a
    //             lane's 16 row indices change with every k-block and are fetched one ahead
    //   DGRAD_DOWN, WGRAD_DOWN (the backward without dy_perm): the rows of dy through the same
    //             map, as FWD1 does for its A tile and as WGRAD_13 does for its B tile, here for
    //             the A tile (two 64-column blocks per CTA) with B brought by TMA
    // Each lane's copies of a stage end in cp.async.mbarrier.arrive on the stage's gather
    // barrier; the relay warp waits for that barrier, makes the rows visible to the async proxy
    // and arrives on the pair leader's full barrier.  Row indices >= T (padding rows) and columns
    // past d are written as zeros.
    int stage = 0;
    uint32_t phase = 0;
    bool alive = true;
    const uint64_t polA = operand_policy<ROLE>(0), polB = operand_policy<ROLE>(1);
    const int gw = warp == 0 ? 0 : warp - 5;           // 0 .. kGatherWarps - 1
    const int c16 = lane & 7, r_lo = lane >> 3;
    const char* const xg = reinterpret_cast<const char*>(p.gather_src);
    const size_t pitch = 2 * (size_t)p.gs.d;
    const int n_src = p.gather_rows;
    Tile t_pf = prefetch_tile(it0);
    for (int it = it0; it < it_end && alive; it += it_step) {
      const int ti = zigzag ? tile_of(it) : it;
      const Tile t = t_pf;
      t_pf = prefetch_tile(it + it_step);
      if (ti < 0) continue;
      const TileGeom q = tile_geom<ROLE>(p, t, s_seg);
      const CUtensorMap* mA = &p.mapA[q.g];
      const CUtensorMap* mB = &p.mapB[q.g];
      const int nb = q.bn / CG;
      const int pieces = (WIDE && q.wide) ? 2 : 1;
      const int am0 = q.m0 + BM * (int)cta_rank;
      // which operand is gathered: A with rows = tile rows (K-major: FWD1 gathers x, DGRAD_DOWN dy),
      // B with rows = contraction index (WGRAD_13 gathers x), A with rows = contraction index
      // (WGRAD_DOWN gathers dy)
      constexpr bool kGatherAK = ROLE == ROLE_FWD1 || ROLE == ROLE_DGRAD_DOWN;
      constexpr bool kGatherAMN = ROLE == ROLE_WGRAD_DOWN;
      // bytes TMA brings per stage: the operand that is not gathered
      const uint32_t tx = (kGatherAK || kGatherAMN) ? (uint32_t)pieces * nb * BK * 2 : (uint32_t)kABytes;
      constexpr int kRowsF = 32 / kGatherWarps;         // A, K-major: row slots of this warp's lanes
      // contraction-index gathers: a stage has nblk 64-column blocks of 16 row slots (j) each; the
      // warps share the blocks (or, with fewer blocks than warps, the slots of a block)
      const int nblk = kGatherAMN ? 2 : pieces * (nb / 64);
      int rows[kRowsF > 16 ? kRowsF : 16];             // row of slot j (of this warp, K-major A)
      int rows_next[16];
      if (kGatherAK) {
#pragma unroll
        for (int j = 0; j < kRowsF; ++j) rows[j] = p.gather[am0 + r_lo + 4 * (gw * kRowsF + j)];
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) rows[j] = p.gather[q.r0 + r_lo + 4 * j];
      }
      for (int kb = 0; kb < q.num_kb; ++kb) {
        if (!kGatherAK) {
#pragma unroll
          for (int j = 0; j < 16; ++j)
            rows_next[j] = kb + 1 < q.num_kb ? p.gather[q.r0 + (kb + 1) * BK + r_lo + 4 * j] : 0;
        }
        int ok = 1;
        if (lane == 0) ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 1) ? 1 : 0;
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) { alive = false; break; }
        const uint32_t sA = smem_base + stage * kStageBytes;
        const uint32_t fb = CG == 2 ? mapa_rank(full_bar(stage), 0) : full_bar(stage);
        const int k0 = kb * BK;
        if (lane == 0 && gw == 0) {
          if (CG == 2) mbar_expect_tx_cluster(fb, tx); else mbar_expect_tx(fb, tx);
          if (ROLE == ROLE_FWD1) {
            for (int pc = 0; pc < pieces; ++pc) {
              const uint32_t sB = sA + kABytes + pc * G::kBBytes;
              const int half = q.bn >> 1;
              const int h0 = q.n0 + pc * half;
              if (CG == 2) {
                tma_3d<CG>(sB, mB, fb, k0, h0, 2 * q.i + (int)cta_rank, polB);
              } else {
                tma_3d<CG>(sB, mB, fb, k0, h0, 2 * q.i, polB);
                tma_3d<CG>(sB + half * 128, mB, fb, k0, h0, 2 * q.i + 1, polB);
              }
            }
          } else if (ROLE == ROLE_DGRAD_DOWN) {
            for (int pc = 0; pc < pieces; ++pc) {
              const uint32_t sB = sA + kABytes + pc * G::kBBytes;
              const int bn0 = q.n0 + pc * q.bn + nb * (int)cta_rank;
              if (p.b_blk[q.g]) tma_4d<CG>(sB, mB, fb, 0, k0, bn0 >> 6, q.i, polB);
              else for (int j = 0; j < nb / 64; ++j) tma_3d<CG>(sB + j * 8192, mB, fb, bn0 + 64 * j, k0, q.i, polB);
            }
          } else if (ROLE == ROLE_WGRAD_DOWN) {
            for (int pc = 0; pc < pieces; ++pc) {
              const uint32_t sB = sA + kABytes + pc * G::kBBytes;
              const int bn0 = q.n0 + pc * q.bn + nb * (int)cta_rank;
              if (p.b_blk[q.g]) tma_3d<CG>(sB, mB, fb, 0, q.r0 + k0, bn0 >> 6, polB);
              else for (int j = 0; j < nb / 64; ++j) tma_2d<CG>(sB + j * 8192, mB, fb, bn0 + 64 * j, q.r0 + k0, polB);
            }
          } else {
            if (p.a_blk[q.g]) {
              tma_3d<CG>(sA, mA, fb, 0, q.r0 + k0, am0 >> 6, polA);
            } else {
              tma_2d<CG>(sA, mA, fb, am0, q.r0 + k0, polA);
              tma_2d<CG>(sA + 8192, mA, fb, am0 + 64, q.r0 + k0, polA);
            }
          }
        }
        if (kGatherAK) {
          const int col = k0 + 8 * c16;                  // first of this lane's 8 columns
          const uint32_t col_ok = col < p.gs.d ? 16u : 0u;
          const size_t col_off = col < p.gs.d ? 2 * (size_t)col : 0;
#pragma unroll
          for (int j = 0; j < kRowsF; ++j) {
            const int r = r_lo + 4 * (gw * kRowsF + j), src = rows[j];
            const bool in = src < n_src;
            cp_async_16(sA + (uint32_t)r * 128u + (uint32_t)((c16 ^ (r & 7)) << 4),
                        xg + (in ? (size_t)src * pitch : 0) + col_off, in ? col_ok : 0u);
          }
        } else {
          // blocks of this warp: blk = gw, gw + W, ... when there are at least W = kGatherWarps
          // blocks; else every warp works on block gw % nblk and takes a part of its 16 slots
          const int share = nblk >= kGatherWarps ? 1 : kGatherWarps / nblk;     // warps per block
          const int j_lo = (gw / nblk) * (16 / share) * (share > 1 ? 1 : 0), j_n = 16 / share;
          for (int blk = share > 1 ? gw % nblk : gw; blk < nblk; blk += share > 1 ? nblk : kGatherWarps) {
            // B blocks of the piece's column slice, or (A gathered) the two 64-column blocks of
            // this CTA's 128 tile rows
            const int pc = kGatherAMN ? 0 : blk / (nb / 64), jb = kGatherAMN ? blk : blk % (nb / 64);
            const uint32_t sB = kGatherAMN ? sA : sA + kABytes + pc * G::kBBytes;
            const int col = kGatherAMN ? am0 + 64 * jb + 8 * c16
                                       : q.n0 + pc * q.bn + nb * (int)cta_rank + 64 * jb + 8 * c16;
            const uint32_t col_ok = col < p.gs.d ? 16u : 0u;
            const size_t col_off = col < p.gs.d ? 2 * (size_t)col : 0;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              if (j >= j_lo && j < j_lo + j_n) {
                const int r = r_lo + 4 * j, src = rows[j];
                const bool in = src < n_src;
                cp_async_16(sB + (uint32_t)jb * 8192u + (uint32_t)r * 128u + (uint32_t)((c16 ^ (r & 7)) << 4),
                            xg + (in ? (size_t)src * pitch : 0) + col_off, in ? col_ok : 0u);
              }
            }
          }
#pragma unroll
          for (int j = 0; j < 16; ++j) rows[j] = rows_next[j];
        }
        cp_async_arrive(gath_bar(stage));
        if (++stage == kStages) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 0) {
    // ================= TMA producer =================
    if (lane == 0) {
      const uint64_t polA = operand_policy<ROLE>(0), polB = operand_policy<ROLE>(1);
      int stage = 0;
      uint32_t phase = 0;
      bool alive = true;
      TCC(long long c_empty = 0;)
      Tile t_pf = prefetch_tile(it0);
      for (int it = it0; it < it_end && alive; it += it_step) {
        const int ti = zigzag ? tile_of(it) : it;
        const Tile t = t_pf;
        t_pf = prefetch_tile(it + it_step);
        if (ti < 0) continue;
        if (ROLE == ROLE_LOGITS && t.ext == 0) continue;
        const TileGeom q = tile_geom<ROLE>(p, t, s_seg);
        const bool half_a = ROLE == ROLE_LOGITS && p.plain_balanced && t.ext <= 64;   // 64-row A box
        const CUtensorMap* mA = &p.mapA[half_a ? 1 : q.g];
        const CUtensorMap* mB = &p.mapB[q.g];
        const int nb = q.bn / CG;                          // B rows staged by this CTA per B tile
        const int pieces = (WIDE && q.wide) ? 2 : 1;       // B tiles of this entry
        const uint32_t tx = (half_a ? kABytes / 2 : kABytes) + (uint32_t)pieces * nb * BK * 2;
        const int am0 = q.m0 + BM * (int)cta_rank;         // this CTA's 128 rows of the tile
        for (int kb = 0; kb < q.num_kb; ++kb) {
          TCC(const long long w0 = clock64();)
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 1)) { alive = false; break; }
          TCC(c_empty += clock64() - w0;)
          const uint32_t sA = smem_base + stage * kStageBytes;
          // CG == 2: both CTAs report to the full barrier of the pair's leader (rank 0)
          const uint32_t fb = CG == 2 ? mapa_rank(full_bar(stage), 0) : full_bar(stage);
          if (CG == 2) mbar_expect_tx_cluster(fb, tx); else mbar_expect_tx(fb, tx);
          const int k0 = kb * BK;
          if (RT::A_MN) {
            if (p.a_blk[q.g]) {
              tma_3d<CG>(sA, mA, fb, 0, q.r0 + k0, am0 >> 6, polA);
            } else {
              tma_2d<CG>(sA, mA, fb, am0, q.r0 + k0, polA);
              tma_2d<CG>(sA + 8192, mA, fb, am0 + 64, q.r0 + k0, polA);
            }
          } else {
            tma_2d<CG>(sA, mA, fb, (is_plain<ROLE>() ? q.r0 : 0) + k0, am0, polA);   // r0: split-K offset
          }
          for (int pc = 0; pc < pieces; ++pc) {
            const uint32_t sB = sA + kABytes + pc * G::kBBytes;
            if (ROLE == ROLE_FWD1) {
              const int half = q.bn >> 1;
              const int h0 = q.n0 + pc * half;               // first hidden column of this piece
              if (CG == 2) {          // leader stages the gate rows, its peer the up rows
                tma_3d<CG>(sB, mB, fb, k0, h0, 2 * q.i + (int)cta_rank, polB);
              } else {
                tma_3d<CG>(sB, mB, fb, k0, h0, 2 * q.i, polB);
                tma_3d<CG>(sB + half * 128, mB, fb, k0, h0, 2 * q.i + 1, polB);
              }
            } else {
              const int bn0 = q.n0 + pc * q.bn + nb * (int)cta_rank;   // this CTA's slice of the columns
              if (ROLE == ROLE_LOGITS) {
                if (p.rf.on) {     // expert rows of the router weight first, the group rows behind them
                  const int ne = p.rf.Ng * p.rf.N;
                  tma_2d<CG>(sB, &p.mapB[0], fb, q.r0 + k0, p.rf.Ng, polB);
                  tma_2d<CG>(sB + ne * 128, &p.mapB[1], fb, q.r0 + k0, 0, polB);
                } else {
                  tma_2d<CG>(sB, mB, fb, q.r0 + k0, bn0, polB);
                }
              } else if (ROLE == ROLE_FWD2) {
                tma_3d<CG>(sB, mB, fb, k0, bn0, q.i, polB);
              } else if (ROLE == ROLE_DGRAD_DOWN || ROLE == ROLE_DGRAD_13) {
                if (p.b_blk[q.g]) tma_4d<CG>(sB, mB, fb, 0, k0, bn0 >> 6, q.i, polB);
                else for (int j = 0; j < nb / 64; ++j) tma_3d<CG>(sB + j * 8192, mB, fb, bn0 + 64 * j, k0, q.i, polB);
              } else {
                if (p.b_blk[q.g]) tma_3d<CG>(sB, mB, fb, 0, q.r0 + k0, bn0 >> 6, polB);
                else for (int j = 0; j < nb / 64; ++j) tma_2d<CG>(sB + j * 8192, mB, fb, bn0 + 64 * j, q.r0 + k0, polB);
              }
            }
          }
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      TCC(atomicAdd(&cnt[4], (unsigned long long)c_empty);)
    }
  } else if (warp == 1) {
    // ================= MMA issuer =================
    if (lane == 0 && cta_rank == 0) {      // the leader issues for the pair
      int stage = 0;
      uint32_t phase = 0;
      int buf = 0;
      uint32_t acc_phase = 0;
      bool alive = true;
      TCC(long long c_w0 = 0, c_full = 0, c_tempty = 0, c_tiles = 0, c_kb = 0, c_mid0 = 0, c_mid = 0, c_midn = 0; const long long c_start = clock64();)
      // MMAs of one k-block into accumulator column base d_tmem from the B tile at sB
      auto issue_kblock = [&](uint32_t d_tmem, uint32_t sA, uint32_t sB, uint32_t idesc, bool first) {
#pragma unroll
        for (int kk = 0; kk < BK / 16; ++kk) {
          const uint64_t da = RT::A_MN ? make_desc(sA + kk * 2048, 8192, 1024)
                                       : make_desc(sA + kk * 32, 16, 1024);
          const uint64_t db = RT::B_MN ? make_desc(sB + kk * 2048, 8192, 1024)
                                       : make_desc(sB + kk * 32, 16, 1024);
          const uint32_t acc = (first && kk == 0) ? 0u : 1u;
          if (CG == 2) umma2_bf16(d_tmem, da, db, idesc, acc);
          else umma_bf16(d_tmem, da, db, idesc, acc);
        }
      };
      auto free_stage = [&](int st) { if (CG == 2) umma2_commit(empty_bar(st)); else umma_commit(empty_bar(st)); };
      auto acc_done = [&](int b) { if (CG == 2) umma2_commit(tfull_bar(b)); else umma_commit(tfull_bar(b)); };
      Tile t_pf = prefetch_tile(it0);
      for (int it = it0; it < it_end && alive; it += it_step) {
        const int ti = zigzag ? tile_of(it) : it;
        const Tile t = t_pf;
        t_pf = prefetch_tile(it + it_step);
        if (ti < 0) continue;
        if (ROLE == ROLE_LOGITS && t.ext == 0) continue;
        const TileGeom q = tile_geom<ROLE>(p, t, s_seg);
        TCC(c_tiles += 1; c_kb += q.num_kb * ((WIDE && q.wide) ? 2 : 1);)
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)RT::A_MN << 15) |
                               ((uint32_t)RT::B_MN << 16) | ((uint32_t)(q.bn >> 3) << 17) |
                               ((uint32_t)(G::kTileM >> 4) << 24);
        if (!WIDE || !q.wide) {
          TCC(c_w0 = clock64();)
          if (!mbar_wait(tempty_bar(buf), acc_phase ^ 1u, abort_flag, p.status, 2)) { alive = false; break; }
          TCC(c_tempty += clock64() - c_w0;)
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + buf * kAccCols;
          for (int kb = 0; kb < q.num_kb; ++kb) {
            TCC(c_w0 = clock64();)
            if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status, 3)) { alive = false; break; }
            TCC(c_full += clock64() - c_w0;
                if (q.num_kb >= 32) { if (kb == 8) c_mid0 = clock64(); if (kb == 24) { c_mid += clock64() - c_mid0; c_midn += 16; } })
            tc_fence_after();
            const uint32_t sA = smem_base + stage * kStageBytes;
            issue_kblock(d_tmem, sA, sA + kABytes, idesc, kb == 0);
            free_stage(stage);               // frees the stage (in both CTAs of a pair) once read
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
          if (!alive) break;
          acc_done(buf);
          if (++buf == 2) { buf = 0; acc_phase ^= 1u; }
          continue;
        }
        // ---- double-width entry: accumulators b0 (columns n0..) and b1 (columns n0 + bn..).
        // The epilogue drains b0 first.  The first kDefer k-blocks go to b0 alone while b1 is
        // still being drained, then b1 catches up on the same stages; after that each
        // k-block feeds both.
        const int b0 = buf, b1 = buf ^ 1;
        const uint32_t ph0 = acc_phase, ph1 = (b1 == 0) ? (acc_phase ^ 1u) : acc_phase;
        const uint32_t d0 = tmem_base + b0 * kAccCols, d1 = tmem_base + b1 * kAccCols;
        constexpr int kDefer = 2;
        const int nd = q.num_kb < kDefer ? q.num_kb : kDefer;
        TCC(c_w0 = clock64();)
        if (!mbar_wait(tempty_bar(b0), ph0 ^ 1u, abort_flag, p.status, 2)) { alive = false; break; }
        TCC(c_tempty += clock64() - c_w0;)
        tc_fence_after();
        int st_d[kDefer];
        for (int kb = 0; kb < nd; ++kb) {
          TCC(c_w0 = clock64();)
          if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status, 3)) { alive = false; break; }
          TCC(c_full += clock64() - c_w0;)
          tc_fence_after();
          const uint32_t sA = smem_base + stage * kStageBytes;
          issue_kblock(d0, sA, sA + kABytes, idesc, kb == 0);
          st_d[kb] = stage;
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!alive) break;
        TCC(c_w0 = clock64();)
        if (!mbar_wait(tempty_bar(b1), ph1 ^ 1u, abort_flag, p.status, 6)) { alive = false; break; }
        TCC(c_tempty += clock64() - c_w0;)
        tc_fence_after();
        for (int kb = 0; kb < nd; ++kb) {
          const uint32_t sA = smem_base + st_d[kb] * kStageBytes;
          issue_kblock(d1, sA, sA + kABytes + G::kBBytes, idesc, kb == 0);
          free_stage(st_d[kb]);
        }
        // The last kLead k-blocks feed b0 first and b1 afterwards (from the same stages), so b0
        // is complete, and its epilogue under way, while b1's last MMAs still run.
        constexpr int kLead = 2;
        const int nl = q.num_kb - nd >= kLead ? kLead : 0;
        for (int kb = nd; kb < q.num_kb - nl; ++kb) {
          TCC(c_w0 = clock64();)
          if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status, 3)) { alive = false; break; }
          TCC(c_full += clock64() - c_w0;
              if (q.num_kb >= 32) { if (kb == 8) c_mid0 = clock64(); if (kb == 24) { c_mid += clock64() - c_mid0; c_midn += 32; } })
          tc_fence_after();
          const uint32_t sA = smem_base + stage * kStageBytes;
          issue_kblock(d0, sA, sA + kABytes, idesc, false);
          issue_kblock(d1, sA, sA + kABytes + G::kBBytes, idesc, false);
          free_stage(stage);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!alive) break;
        int st_l[kLead];
        for (int j = 0; j < nl; ++j) {
          TCC(c_w0 = clock64();)
          if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status, 3)) { alive = false; break; }
          TCC(c_full += clock64() - c_w0;)
          tc_fence_after();
          const uint32_t sA = smem_base + stage * kStageBytes;
          issue_kblock(d0, sA, sA + kABytes, idesc, false);
          st_l[j] = stage;
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!alive) break;
        acc_done(b0);
        for (int j = 0; j < nl; ++j) {
          const uint32_t sA = smem_base + st_l[j] * kStageBytes;
          issue_kblock(d1, sA, sA + kABytes + G::kBBytes, idesc, false);
          free_stage(st_l[j]);
        }
        acc_done(b1);
        // two buffers used: the buffer index is unchanged, the phase of both advances
        if (b0 == 0) acc_phase ^= 1u; else { buf = 1; acc_phase ^= 1u; }
      }
      TCC(atomicAdd(&cnt[0], 1ull); atomicAdd(&cnt[1], (unsigned long long)(clock64() - c_start));
          atomicAdd(&cnt[2], (unsigned long long)c_full); atomicAdd(&cnt[3], (unsigned long long)c_tempty);
          atomicAdd(&cnt[8], (unsigned long long)c_tiles); atomicAdd(&cnt[9], (unsigned long long)c_kb);
          atomicAdd(&cnt[10], (unsigned long long)c_mid); atomicAdd(&cnt[11], (unsigned long long)c_midn);)
    }
  } else if (GATHER && warp == 5 + kGatherWarps) {
    // ================= gather relay =================
    // Gathering form only.  For every stage in the producer's order: wait until the 32 lanes'
    // row copies have landed (the stage's gather barrier), make them visible to the async proxy
    // (the MMAs read shared memory through it) and arrive on the full barrier of the pair's leader.
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool alive = true;
      Tile t_pf = prefetch_tile(it0);
      for (int it = it0; it < it_end && alive; it += it_step) {
        const int ti = zigzag ? tile_of(it) : it;
        const Tile t = t_pf;
        t_pf = prefetch_tile(it + it_step);
        if (ti < 0) continue;
        const TileGeom q = tile_geom<ROLE>(p, t, s_seg);
        for (int kb = 0; kb < q.num_kb; ++kb) {
          if (!mbar_wait(gath_bar(stage), phase, abort_flag, p.status, 7)) { alive = false; break; }
          fence_async_smem();
          if (CG == 2) mbar_arrive_release_cluster(mapa_rank(full_bar(stage), 0)); else mbar_arrive(full_bar(stage));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else {
    // ================= epilogue warps =================
    const int quad = warp & 3;                 // tensor-memory lanes [32*quad, 32*quad + 32)
    const int split = (GATHER ? 0 : (warp - 2) >> 2);   // > 0 only with kThreadsRoute threads
    uint32_t list_phase = 0;
    const int row_in_tile = BM * (int)cta_rank + quad * 32 + lane;   // row of the (pair's) tile
    const uint32_t stg = stg0 + (uint32_t)quad * (kSlots * kStgBufBytes);   // this warp's staging ring
    uint32_t n_store = 0;                      // stores issued so far: ring slot = n_store % 4
    uint32_t n_chunk = 0;                      // SwiGLU backward: input chunks consumed so far
    const uint64_t pol_stream = l2_policy_evict_first();
    int buf = 0;
    uint32_t acc_phase = 0;
    bool alive = true;
    TCC(long long c_tfull = 0; const long long c_start = clock64();)
    Tile t_pf = prefetch_tile(it0);
    for (int it = it0; it < it_end && alive; it += it_step) {
      const int ti = zigzag ? tile_of(it) : it;
      const Tile t = t_pf;
      t_pf = prefetch_tile(it + it_step);
      if (ti < 0) continue;
      if (ROLE == ROLE_LOGITS && t.ext == 0) continue;
      TileGeom q = tile_geom<ROLE>(p, t, s_seg);
      // a double-width entry is drained as two pieces, one accumulator buffer each
      const int pieces = (WIDE && q.wide) ? 2 : 1;
      for (int pc = 0; pc < pieces && alive; ++pc) {
      if (pc) q.n0 += RT::EPI == EPI_SWIGLU_FWD ? (q.bn >> 1) : q.bn;
      // row-tiled expert roles: first row of this warp; segments are 128-row aligned, so the
      // rows of one CTA are either all inside the expert's segment or all outside
      const int row0 = q.m0 + BM * (int)cta_rank + quad * 32;
      const bool rows_ok = BM * (int)cta_rank < t.ext;
      int nch_in = 0;
      if (RT::EPI == EPI_SWIGLU_BWD) {
        // A and U of the first 64 columns are fetched while the MMAs of this tile still run
        if (rows_ok) { const int left = q.W - q.n0; nch_in = ((left < q.bn ? left : q.bn) + 63) / 64; }
        if (nch_in > 0 && lane == 0) {
          bulk_wait_read<0>();
          const uint32_t set = n_chunk & 1u, bar = ein_bar(quad, set);
          mbar_expect_tx(bar, 2 * kStgBufBytes);
          tma_load_2d_hint(stg + set * 2 * kStgBufBytes, &p.mapE[0][q.g], bar, q.n0, row0, pol_stream);
          tma_load_2d_hint(stg + (set * 2 + 1) * kStgBufBytes, &p.mapE[1][q.g], bar, q.n0, row0, pol_stream);
        }
      }
      int nch_acc = 0;
      if (RT::EPI == EPI_BF16_ACC) {
        // dx += ...: all (up to four) 64-column chunks of this warp's 32 rows are fetched at once
        // into the staging ring, added to in place and stored from there; rows past T are clipped
        const int left = p.plain_N - q.n0;
        nch_acc = ((left < q.bn ? left : q.bn) + 63) / 64;
        if (q.m0 + BM * (int)cta_rank + quad * 32 >= p.plain_M) nch_acc = 0;
        if (nch_acc > 0 && lane == 0) {
          bulk_wait_read<0>();
          const uint32_t bar = ein_bar(quad, 0);
          mbar_expect_tx(bar, (uint32_t)nch_acc * kStgBufBytes);
          for (int ci = 0; ci < nch_acc; ++ci)
            tma_load_2d_hint(stg + ci * kStgBufBytes, &p.mapO[0][0], bar, q.n0 + ci * 64,
                             q.m0 + quad * 32, pol_stream);
        }
      }
      // the whole warp must agree before the warp-collective tensor-memory loads
      TCC(const long long c_w0 = clock64();)
      const bool got = mbar_wait(tfull_bar(buf), acc_phase, abort_flag, p.status, 4);
      TCC(c_tfull += clock64() - c_w0;)
      if (!__all_sync(0xffffffffu, got)) { alive = false; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + buf * kAccCols;
      const long long d = p.gs.d;
      // pacing reference: now, and the k-blocks of the tile whose MMAs overlap this epilogue
      const long long t_epi = clock64();
      int next_kb = 0;
      if ((RT::EPI == EPI_BF16 || RT::EPI == EPI_F32) && !(WIDE && q.wide) && it + it_step < it_end &&
          (zigzag ? tile_of(it + 1) : it + it_step) >= 0)
        next_kb = tile_geom<ROLE>(p, t_pf, s_seg).num_kb;
      // The accumulator is handed back to the MMA issuer as soon as its last column has left
      // tensor memory, before the arithmetic, the staging and the stores of that data: with
      // double-width entries the next entry's MMAs wait for exactly this.
      bool released = false;
      auto release_acc = [&]() {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (CG == 2) mbar_arrive_cluster(mapa_rank(tempty_bar(buf), 0)); else mbar_arrive(tempty_bar(buf));
        }
        released = true;
      };
      // Staging ring of this warp: kSlots boxes of 4 KiB used in turn; store #n leaves from box
      // n % kSlots.  Before a box is written again the store that last read it (kSlots stores
      // back) must be done reading: with i stores of the current batch not yet issued, at most
      // kSlots - 1 - i of the store groups committed so far may still be pending.
      auto ring_slot = [&](int i) { return stg + ((n_store + (uint32_t)i) % kSlots) * kStgBufBytes; };
      auto ring_wait = [&](int i) {
        const int allowed = kSlots - 1 - i;
        if (lane == 0) {
          if (allowed <= 0) bulk_wait_read<0>();
          else if (allowed == 1) bulk_wait_read<1>();
          else if (allowed == 2) bulk_wait_read<2>();
          else bulk_wait_read<3>();
        }
        __syncwarp();
      };
      if (RT::EPI == EPI_SWIGLU_FWD) {
        const int half = q.bn >> 1;
        for (int c = 0; rows_ok && c < half && q.n0 + c < q.W; c += 64) {
          const bool last_chunk = !(c + 64 < half && q.n0 + c + 64 < q.W);
          ring_wait(2);                                // three boxes of the ring are free
          const uint32_t bA = ring_slot(0), bU = ring_slot(1), bH = ring_slot(2);
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            uint32_t ra[32], ru[32];
            tmem_ld32(taddr + c + 32 * hh, ra);
            tmem_ld32(taddr + half + c + 32 * hh, ru);
            tmem_ld_wait();
            if (last_chunk && hh == 1) release_acc();
            uint32_t pa[4][4], pu[4][4], ph[4][4];       // arithmetic first, then the stores
#pragma unroll
            for (int j4 = 0; j4 < 4; ++j4) {
#pragma unroll
              for (int e2 = 0; e2 < 4; ++e2) {
                const float a0 = __uint_as_float(ra[j4 * 8 + 2 * e2]), a1 = __uint_as_float(ra[j4 * 8 + 2 * e2 + 1]);
                const float u0 = __uint_as_float(ru[j4 * 8 + 2 * e2]), u1 = __uint_as_float(ru[j4 * 8 + 2 * e2 + 1]);
                const float2 a2 = make_float2(a0, a1), u2 = make_float2(u0, u1);
                const float2 h2 = __fmul2_rn(__fmul2_rn(a2, sigmoid2_fast(a2)), u2);   // silu(a) * u
                pa[j4][e2] = pack2(a0, a1); pu[j4][e2] = pack2(u0, u1); ph[j4][e2] = pack2(h2.x, h2.y);
              }
            }
#pragma unroll
            for (int j4 = 0; j4 < 4; ++j4) {
              st_shared_v4(stg_addr(bA, lane, hh * 4 + j4), pa[j4][0], pa[j4][1], pa[j4][2], pa[j4][3]);
              st_shared_v4(stg_addr(bU, lane, hh * 4 + j4), pu[j4][0], pu[j4][1], pu[j4][2], pu[j4][3]);
              st_shared_v4(stg_addr(bH, lane, hh * 4 + j4), ph[j4][0], ph[j4][1], ph[j4][2], ph[j4][3]);
            }
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_store_2d(&p.mapO[0][q.g], bA, q.n0 + c, row0, pol_stream); bulk_commit();
            tma_store_2d(&p.mapO[1][q.g], bU, q.n0 + c, row0, pol_stream); bulk_commit();
            tma_store_2d(&p.mapO[2][q.g], bH, q.n0 + c, row0, pol_stream); bulk_commit();
          }
          n_store += 3;
        }
      } else if (RT::EPI == EPI_BF16) {
        int nch = 0;                                   // 64-column chunks of this piece (at most 4)
        if (rows_ok) { const int left = (int)d - q.n0; nch = ((left < q.bn ? left : q.bn) + 63) >> 6; }
        // Chunks go out in batches of one fence: single chunks while the output is paced against
        // the next tile's MMAs, else as many as the ring holds.
        const int batch = next_kb ? 1 : kSlots;
        for (int c0 = 0; c0 < nch; c0 += batch) {
          const int nb = nch - c0 < batch ? nch - c0 : batch;
          for (int i = 0; i < nb; ++i) {
            const int ci = c0 + i;
            pace(t_epi, ci * 64, q.bn, next_kb);
            ring_wait(i);
            const uint32_t bO = ring_slot(i);
            uint32_t r0[32], r1[32];
            tmem_ld32(taddr + ci * 64, r0);
            tmem_ld32(taddr + ci * 64 + 32, r1);
            tmem_ld_wait();
            if (ci + 1 == nch) release_acc();
#pragma unroll
            for (int j4 = 0; j4 < 4; ++j4) {
              st_shared_v4(stg_addr(bO, lane, j4),
                           pack2(__uint_as_float(r0[j4 * 8 + 0]), __uint_as_float(r0[j4 * 8 + 1])),
                           pack2(__uint_as_float(r0[j4 * 8 + 2]), __uint_as_float(r0[j4 * 8 + 3])),
                           pack2(__uint_as_float(r0[j4 * 8 + 4]), __uint_as_float(r0[j4 * 8 + 5])),
                           pack2(__uint_as_float(r0[j4 * 8 + 6]), __uint_as_float(r0[j4 * 8 + 7])));
              st_shared_v4(stg_addr(bO, lane, 4 + j4),
                           pack2(__uint_as_float(r1[j4 * 8 + 0]), __uint_as_float(r1[j4 * 8 + 1])),
                           pack2(__uint_as_float(r1[j4 * 8 + 2]), __uint_as_float(r1[j4 * 8 + 3])),
                           pack2(__uint_as_float(r1[j4 * 8 + 4]), __uint_as_float(r1[j4 * 8 + 5])),
                           pack2(__uint_as_float(r1[j4 * 8 + 6]), __uint_as_float(r1[j4 * 8 + 7])));
            }
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) {
            for (int i = 0; i < nb; ++i) {
              tma_store_2d(&p.mapO[0][0], ring_slot(i), q.n0 + (c0 + i) * 64, row0, pol_stream);
              bulk_commit();
            }
          }
          n_store += nb;
        }
      } else if (RT::EPI == EPI_SWIGLU_BWD) {
        // per 64-column chunk: A and U arrive by TMA in one of two buffer pairs, dA and dU are
        // written over them in place and leave by TMA; the next chunk's loads fly meanwhile
        float2 dg2 = make_float2(0.0f, 0.0f);          // sum over this tile's columns of dH * h
        // gathering form: the accumulator is dy W2 without the gate; the gate of the row comes in here
        float2 gate2 = make_float2(1.0f, 1.0f);
        if (GATHER && nch_in > 0) { const float gr = p.row_gate[row0 + lane]; gate2 = make_float2(gr, gr); }
        for (int ci = 0; ci < nch_in; ++ci, ++n_chunk) {
          const int c = ci * 64;
          const uint32_t set = n_chunk & 1u;
          if (ci + 1 < nch_in && lane == 0) {
            bulk_wait_read<0>();                       // the other pair's last stores have left
            const uint32_t bar = ein_bar(quad, set ^ 1u);
            mbar_expect_tx(bar, 2 * kStgBufBytes);
            tma_load_2d_hint(stg + (set ^ 1u) * 2 * kStgBufBytes, &p.mapE[0][q.g], bar, q.n0 + c + 64, row0, pol_stream);
            tma_load_2d_hint(stg + ((set ^ 1u) * 2 + 1) * kStgBufBytes, &p.mapE[1][q.g], bar, q.n0 + c + 64, row0, pol_stream);
          }
          const bool in_ok = mbar_wait(ein_bar(quad, set), (n_chunk >> 1) & 1u, abort_flag, p.status, 5);
          if (!__all_sync(0xffffffffu, in_ok)) { alive = false; break; }
          const uint32_t bA = stg + set * 2 * kStgBufBytes, bU = bA + kStgBufBytes;
          // both halves of the chunk leave tensor memory while the shared-memory reads are issued;
          // loads, arithmetic and stores are grouped so that the single warp has independent work
          uint32_t r[2][32];
          tmem_ld32(taddr + c, r[0]);
          tmem_ld32(taddr + c + 32, r[1]);
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            uint4 va[4], vu[4];
#pragma unroll
            for (int j4 = 0; j4 < 4; ++j4) {
              va[j4] = ld_shared_v4(stg_addr(bA, lane, hh * 4 + j4));
              vu[j4] = ld_shared_v4(stg_addr(bU, lane, hh * 4 + j4));
            }
            if (hh == 0) {
              tmem_ld_wait();
              if (ci + 1 == nch_in) release_acc();
            }
            uint32_t oa[4][4], ou[4][4];
            uint32_t oh[GATHER ? 4 : 1][4];           // gathering form: gate * H
#pragma unroll
            for (int j4 = 0; j4 < 4; ++j4) {
              const uint32_t wa[4] = {va[j4].x, va[j4].y, va[j4].z, va[j4].w};
              const uint32_t wu[4] = {vu[j4].x, vu[j4].y, vu[j4].z, vu[j4].w};
#pragma unroll
              for (int e2 = 0; e2 < 4; ++e2) {
                const float2 a2 = make_float2(bf_lo(wa[e2]), bf_hi(wa[e2]));
                const float2 u2 = make_float2(bf_lo(wu[e2]), bf_hi(wu[e2]));
                float2 dh2 = make_float2(__uint_as_float(r[hh][j4 * 8 + 2 * e2]),
                                         __uint_as_float(r[hh][j4 * 8 + 2 * e2 + 1]));
                if (GATHER) dh2 = __fmul2_rn(dh2, gate2);
                const float2 one = make_float2(1.0f, 1.0f);
                const float2 s2 = sigmoid2_fast(a2);
                const float2 oms = __ffma2_rn(s2, make_float2(-1.0f, -1.0f), one);      // 1 - s
                const float2 t2 = __ffma2_rn(a2, oms, one);                             // 1 + a (1 - s)
                const float2 dhs = __fmul2_rn(dh2, s2);
                const float2 du2 = __fmul2_rn(dhs, a2);                                 // dh * silu(a)
                const float2 da2 = __fmul2_rn(__fmul2_rn(dhs, u2), t2);                 // dh * u * silu'(a)
                dg2 = __ffma2_rn(du2, u2, dg2);                                         // dh * h
                oa[j4][e2] = pack2(da2.x, da2.y);
                ou[j4][e2] = pack2(du2.x, du2.y);
                if (GATHER) {
                  const float2 hg2 = __fmul2_rn(__fmul2_rn(__fmul2_rn(a2, s2), u2), gate2);   // gate * silu(a) * u
                  oh[j4][e2] = pack2(hg2.x, hg2.y);
                }
              }
            }
#pragma unroll
            for (int j4 = 0; j4 < 4; ++j4) {
              st_shared_v4(stg_addr(bA, lane, hh * 4 + j4), oa[j4][0], oa[j4][1], oa[j4][2], oa[j4][3]);
              st_shared_v4(stg_addr(bU, lane, hh * 4 + j4), ou[j4][0], ou[j4][1], ou[j4][2], ou[j4][3]);
            }
            if (GATHER) {
              // gate * H of this thread's row, straight from registers (eight columns per store)
              __nv_bfloat16* ph = p.hs + (size_t)(row0 + lane) * p.hs_pitch;
#pragma unroll
              for (int j4 = 0; j4 < 4; ++j4) {
                const int col = q.n0 + c + hh * 32 + j4 * 8;
                if (col < q.W) *reinterpret_cast<uint4*>(ph + col) = make_uint4(oh[j4][0], oh[j4][1], oh[j4][2], oh[j4][3]);
              }
            }
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_store_2d(&p.mapO[0][q.g], bA, q.n0 + c, row0, pol_stream);
            tma_store_2d(&p.mapO[1][q.g], bU, q.n0 + c, row0, pol_stream);
            bulk_commit();
          }
        }
        if (!alive) break;
        // nch_in > 0 only for CTAs whose rows lie inside the expert's segment (padding rows give 0)
        if (p.dgate_part != nullptr && nch_in > 0)
          p.dgate_part[(size_t)(row0 + lane) * p.dgate_slots + (q.n0 >> 7)] = dg2.x + dg2.y;
      } else if (RT::EPI == EPI_F32) {
        // weight gradients: FP32 boxes of 32 rows x 32 columns into [expert, rows, columns]
        const int Mext = ROLE == ROLE_WGRAD_DOWN ? (int)d : 2 * q.W;
        const int Next = ROLE == ROLE_WGRAD_DOWN ? q.W : (int)d;
        int nch = 0;                                   // 32-column chunks of this piece (at most 8)
        if (row0 < Mext) { const int left = Next - q.n0; nch = ((left < q.bn ? left : q.bn) + 31) >> 5; }
        auto send_batch = [&](int c0, int nb) {         // boxes ring_slot(0..nb-1) hold chunks c0..
          fence_async_smem();
          __syncwarp();
          if (lane == 0) {
            for (int i = 0; i < nb; ++i) {
              const int col = q.n0 + (c0 + i) * 32;
              if (p.accumulate) tma_reduce_add_3d(&p.mapO[0][q.g], ring_slot(i), col, row0, q.i);
              else tma_store_3d(&p.mapO[0][q.g], ring_slot(i), col, row0, q.i, pol_stream);
              bulk_commit();
            }
          }
          n_store += nb;
        };
        auto stage_chunk = [&](uint32_t bO, const uint32_t (&r)[32]) {
#pragma unroll
          for (int j = 0; j < 8; ++j)
            st_shared_v4(stg_addr(bO, lane, j), r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
        };
        if (!GATHER && !next_kb && kSlots == 4 && nch > 4) {
          // Nothing to pace against (double-width entries): four chunks go into the ring, the
          // other (up to) four wait in registers, and the accumulator is released at once.
          for (int i = 0; i < 4; ++i) {
            ring_wait(i);
            uint32_t r[32];
            tmem_ld32(taddr + i * 32, r);
            tmem_ld_wait();
            stage_chunk(ring_slot(i), r);
          }
          uint32_t rr[4][32];
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (4 + j < nch) tmem_ld32(taddr + (4 + j) * 32, rr[j]);
          tmem_ld_wait();
          release_acc();
          send_batch(0, 4);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            if (4 + j < nch) {
              ring_wait(j);
              stage_chunk(ring_slot(j), rr[j]);
            }
          }
          send_batch(4, nch - 4);
          nch = 0;                                       // done
        }
        const int batch = next_kb ? 1 : kSlots;
        for (int c0 = 0; c0 < nch; c0 += batch) {
          const int nb = nch - c0 < batch ? nch - c0 : batch;
          for (int i = 0; i < nb; ++i) {
            const int ci = c0 + i;
            pace(t_epi, ci * 32, q.bn, next_kb);
            ring_wait(i);
            const uint32_t bO = ring_slot(i);
            uint32_t r[32];
            tmem_ld32(taddr + ci * 32, r);
            tmem_ld_wait();
            if (ci + 1 == nch) release_acc();
            stage_chunk(bO, r);
          }
          send_batch(c0, nb);
        }
      } else if (RT::EPI == EPI_LOGITS) {
        // logits[t, n] = acc + bias[n]; NL is arbitrary, so stores are scalar and masked.  Under
        // split-K every split writes its partial sum and the bias is added when they are summed.
        const long long row = q.m0 + row_in_tile + (long long)q.e * p.plain_M;
        const bool row_ok = row_in_tile < t.ext;
        const float* bias = p.plain_splits == 1 ? p.bias : nullptr;
        if (p.rf.on) {
          RouteList L;
          bool nan = false;
          switch (p.rf.N) {
            case 4: nan = route_token_groups<4>(p.rf, taddr, row_ok, row, p.Cf, bias, split, L); break;
            case 8: nan = route_token_groups<8>(p.rf, taddr, row_ok, row, p.Cf, bias, split, L); break;
            case 16: nan = route_token_groups<16>(p.rf, taddr, row_ok, row, p.Cf, bias, split, L); break;
            default: nan = route_token_groups<32>(p.rf, taddr, row_ok, row, p.Cf, bias, split, L); break;
          }
          release_acc();
          if (nan && row_ok && p.status != nullptr) atomicCAS(p.status, 0, 3 << 24);
          // The lists of the other warps of this row quarter arrive through shared memory: word
          // (2 k + which) * 128 + row of the area of split s holds entry k of that row.  One
          // barrier says "written" (ein_bar(quad, 0)), one "read" (ein_bar(quad, 1)).
          const uint32_t area = stg0 + (uint32_t)(quad * 32 + lane) * 4u;
          if (split > 0) {
            const bool ok = mbar_wait(ein_bar(quad, 1), list_phase ^ 1u, abort_flag, p.status, 8);
            if (!__all_sync(0xffffffffu, ok)) { alive = false; break; }
#pragma unroll
            for (int k = 0; k < kRouteFuseMaxKe; ++k) {
              st_shared_u32(area + (2 * k) * 512u, __float_as_uint(L.wk[k]));
              st_shared_u32(area + (2 * k + 1) * 512u, (uint32_t)L.we[k]);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(ein_bar(quad, 0));
          } else {
            if (kRouteSplit > 1 && block_threads<ROLE, WIDE, GATHER>() == kThreadsRoute) {
              const bool ok = mbar_wait(ein_bar(quad, 0), list_phase, abort_flag, p.status, 8);
              if (!__all_sync(0xffffffffu, ok)) { alive = false; break; }
              RouteList O;
#pragma unroll
              for (int k = 0; k < kRouteFuseMaxKe; ++k) {
                O.wk[k] = __uint_as_float(ld_shared_u32(area + (2 * k) * 512u));
                O.we[k] = (int)ld_shared_u32(area + (2 * k + 1) * 512u);
              }
              __syncwarp();
              if (lane == 0) mbar_arrive(ein_bar(quad, 1));
              route_list_merge(L, O);
            }
            route_token_finish(p.rf, row_ok, row, L);
          }
          list_phase ^= 1u;
        } else if (split == 0)
        for (int c = 0; c < q.bn; c += 32) {
          uint32_t r[32];
          tmem_ld32(taddr + c, r);
          tmem_ld_wait();
          if (row_ok) {
            float* po = p.Cf + row * p.plain_N;
            if ((p.plain_N & 3) == 0) {          // rows are 16-byte aligned: four columns per store
#pragma unroll
              for (int j = 0; j < 32; j += 4) {
                const int n = q.n0 + c + j;
                if (n < p.plain_N) {
                  float4 v = make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]),
                                         __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
                  if (bias) {
                    const float4 bv = *reinterpret_cast<const float4*>(bias + n);
                    v.x += bv.x; v.y += bv.y; v.z += bv.z; v.w += bv.w;
                  }
                  *reinterpret_cast<float4*>(po + n) = v;
                }
              }
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                const int n = q.n0 + c + j;
                if (n < p.plain_N) po[n] = __uint_as_float(r[j]) + (bias ? bias[n] : 0.0f);
              }
            }
          }
        }
      } else if (RT::EPI == EPI_F32_T) {
        // transposed store: tile rows are the d index, tile columns the router output index
        const int m = q.m0 + row_in_tile;
        const bool row_ok = m < p.plain_M;
        float* cf = p.Cf + (size_t)q.e * p.plain_N * p.plain_M;    // this split's partial sum
        for (int c = 0; c < q.bn; c += 32) {
          uint32_t r[32];
          tmem_ld32(taddr + c, r);
          tmem_ld_wait();
          if (row_ok) {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const int n = q.n0 + c + j;
              if (n < p.plain_N) cf[(size_t)n * p.plain_M + m] = __uint_as_float(r[j]);
            }
          }
        }
      } else if (RT::EPI == EPI_BF16_ACC) {
        if (nch_acc > 0) {
          const bool in_ok = mbar_wait(ein_bar(quad, 0), n_chunk & 1u, abort_flag, p.status, 5);
          if (!__all_sync(0xffffffffu, in_ok)) { alive = false; break; }
          ++n_chunk;                                   // uses of this barrier so far (its phase)
          for (int ci = 0; ci < nch_acc; ++ci) {
            const uint32_t bO = stg + ci * kStgBufBytes;
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
              uint32_t r[32];
              tmem_ld32(taddr + ci * 64 + 32 * hh, r);
              tmem_ld_wait();
#pragma unroll
              for (int j4 = 0; j4 < 4; ++j4) {
                const uint32_t a = stg_addr(bO, lane, hh * 4 + j4);
                const uint4 v = ld_shared_v4(a);
                const uint32_t w[4] = {v.x, v.y, v.z, v.w};
                uint32_t o[4];
#pragma unroll
                for (int e2 = 0; e2 < 4; ++e2)
                  o[e2] = pack2(bf_lo(w[e2]) + __uint_as_float(r[j4 * 8 + 2 * e2]),
                                bf_hi(w[e2]) + __uint_as_float(r[j4 * 8 + 2 * e2 + 1]));
                st_shared_v4(a, o[0], o[1], o[2], o[3]);
              }
            }
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
              tma_store_2d(&p.mapO[0][0], bO, q.n0 + ci * 64, q.m0 + quad * 32, pol_stream);
              bulk_commit();
            }
          }
        }
      }
      if (!released) release_acc();
      if (++buf == 2) { buf = 0; acc_phase ^= 1u; }
      }   // pieces
    }
    if (lane == 0) bulk_wait_all();            // staged stores have left before the CTA retires
    TCC(if (warp == 2 && lane == 0) {
          atomicAdd(&cnt[5], (unsigned long long)c_tfull);
          atomicAdd(&cnt[6], (unsigned long long)(clock64() - c_start));
        })
  }

  // ---- teardown ----
  __syncthreads();
  TCC(if (threadIdx.x == 0) atomicAdd(&cnt[7], (unsigned long long)(global_ns() - cnt_t0));)
  if (*abort_flag) __nanosleep(200000);    // let copies in flight land before the CTA retires
  if (CG == 2) cluster_sync_all();         // the peer may still signal this CTA's barriers until here
  tc_fence_after();
  if (warp == 1) {
    if (CG == 2)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                             const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                             CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                             CUtensorMapFloatOOBfill);

EncodeFn get_encode() {
  static EncodeFn fn = nullptr;
  if (!fn) {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = (EncodeFn)f;
  }
  return fn;
}

// Tensor of `rank` dims (innermost first), BF16 unless `f32`; strides in bytes for dims 1..rank-1
int32_t encode_map(CUtensorMap* m, const void* base, int rank, const uint64_t* dims,
                   const uint64_t* strides, const uint32_t* box, bool f32 = false) {
  EncodeFn fn = get_encode();
  if (!fn) {
    set_error("cuTensorMapEncodeTiled is not available from the driver");
    return MOHGE_ERR_UNSUPPORTED;
  }
  cuuint64_t gd[5], gs[5];
  cuuint32_t bx[5], es[5];
  for (int i = 0; i < rank; ++i) {
    gd[i] = dims[i];
    bx[i] = box[i];
    es[i] = 1;
    if (i > 0) gs[i - 1] = strides[i - 1];
  }
  const CUresult r = fn(m, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                        (cuuint32_t)rank, const_cast<void*>(base), gd, gs,
                        bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_error("cuTensorMapEncodeTiled failed with %d (rank %d, dims %llu x %llu, box %u x %u)", (int)r, rank,
              (unsigned long long)dims[0], (unsigned long long)dims[1], box[0], box[1]);
    return MOHGE_ERR_CUDA;
  }
  return MOHGE_OK;
}

// MN-major operand [k_rows, mn] (mn contiguous, row pitch in bytes), optionally one matrix per
// expert.  `blocks` = 64-element swizzle blocks one stage needs.  When mn is a multiple of 64
// the blocks become a dimension and one box covers them all (*blocked = 1).
int32_t encode_mn_map(CUtensorMap* m, const void* base, uint64_t mn, uint64_t k_rows, uint64_t pitch_bytes,
                      uint64_t n_experts, uint64_t expert_stride_bytes, int blocks, unsigned char* blocked) {
  uint64_t dims[4], str[3];
  uint32_t box[4];
  if (mn % 64 == 0) {
    *blocked = 1;
    dims[0] = 64; dims[1] = k_rows; dims[2] = mn / 64; str[0] = pitch_bytes; str[1] = 128;
    box[0] = 64; box[1] = BK; box[2] = (uint32_t)blocks;
    if (n_experts == 0) return encode_map(m, base, 3, dims, str, box);
    dims[3] = n_experts; str[2] = expert_stride_bytes; box[3] = 1;
    return encode_map(m, base, 4, dims, str, box);
  }
  *blocked = 0;
  dims[0] = mn; dims[1] = k_rows; str[0] = pitch_bytes; box[0] = 64; box[1] = BK;
  if (n_experts == 0) return encode_map(m, base, 2, dims, str, box);
  dims[2] = n_experts; str[1] = expert_stride_bytes; box[2] = 1;
  return encode_map(m, base, 3, dims, str, box);
}

// [cols, rows] BF16 region with a row pitch in bytes, as 32-row x 64-column staging boxes
int32_t encode_stage_map(CUtensorMap* m, const void* base, uint64_t cols, uint64_t rows, uint64_t pitch_bytes) {
  const uint64_t dims[2] = {cols, rows}, str[1] = {pitch_bytes};
  const uint32_t box[2] = {64, 32};
  return encode_map(m, base, 2, dims, str, box);
}
// [cols, rows, experts] FP32 weight-gradient tensor as 32 x 32 staging boxes
int32_t encode_stage_map_f32(CUtensorMap* m, const void* base, uint64_t cols, uint64_t rows, uint64_t n) {
  const uint64_t dims[3] = {cols, rows, n}, str[2] = {cols * 4, cols * rows * 4};
  const uint32_t box[3] = {32, 32, 1};
  return encode_map(m, base, 3, dims, str, box, true);
}

// Encoded tensor maps are kept per (device, role, tile form, operand addresses, shapes): a layer
// that is stepped on the same buffers encodes each map once instead of on every launch (up to
// five cuTensorMapEncodeTiled calls per group and launch, about a hundred per step; host time on
// the critical path of the launch-bound small workloads).  A map depends on nothing but the
// address and the shape, so a hit can never be stale.  Fixed size, oldest entry replaced first.
struct MapKey {
  int32_t role, cg, device, accumulate_unused;
  int32_t d, Ng, N, Wmax, W[MOHGE_MAX_GROUPS];
  int64_t rows, T, b_pitch;
  const void *A, *B, *C, *C2, *gather;
  const void* w[4][MOHGE_MAX_GROUPS];
};
struct MapEntry {
  MapKey key;
  CUtensorMap mapA[MOHGE_MAX_GROUPS], mapB[MOHGE_MAX_GROUPS], mapO[3][MOHGE_MAX_GROUPS], mapE[2][MOHGE_MAX_GROUPS];
  int BN[MOHGE_MAX_GROUPS];
  unsigned char a_blk[MOHGE_MAX_GROUPS], b_blk[MOHGE_MAX_GROUPS];
  bool valid;
};
constexpr int kMapCacheEntries = 64;
MapEntry g_map_cache[kMapCacheEntries];
int g_map_cache_next = 0;
std::mutex g_map_cache_mu;
std::atomic<long long> g_map_hits{0}, g_map_misses{0};

bool map_cache_find(const MapKey& key, TcParams* p) {
  std::lock_guard<std::mutex> lock(g_map_cache_mu);
  for (int i = 0; i < kMapCacheEntries; ++i) {
    const MapEntry& e = g_map_cache[i];
    if (e.valid && memcmp(&e.key, &key, sizeof(MapKey)) == 0) {
      memcpy(p->mapA, e.mapA, sizeof(e.mapA)); memcpy(p->mapB, e.mapB, sizeof(e.mapB));
      memcpy(p->mapO, e.mapO, sizeof(e.mapO)); memcpy(p->mapE, e.mapE, sizeof(e.mapE));
      memcpy(p->BN, e.BN, sizeof(e.BN)); memcpy(p->a_blk, e.a_blk, sizeof(e.a_blk));
      memcpy(p->b_blk, e.b_blk, sizeof(e.b_blk));
      ++g_map_hits;
      return true;
    }
  }
  ++g_map_misses;
  return false;
}
void map_cache_store(const MapKey& key, const TcParams& p) {
  std::lock_guard<std::mutex> lock(g_map_cache_mu);
  MapEntry& e = g_map_cache[g_map_cache_next];
  g_map_cache_next = (g_map_cache_next + 1) % kMapCacheEntries;
  e.key = key;
  memcpy(e.mapA, p.mapA, sizeof(e.mapA)); memcpy(e.mapB, p.mapB, sizeof(e.mapB));
  memcpy(e.mapO, p.mapO, sizeof(e.mapO)); memcpy(e.mapE, p.mapE, sizeof(e.mapE));
  memcpy(e.BN, p.BN, sizeof(e.BN)); memcpy(e.a_blk, p.a_blk, sizeof(e.a_blk));
  memcpy(e.b_blk, p.b_blk, sizeof(e.b_blk));
  e.valid = true;
}

// Tile width per group.  Candidates come widest first.  A narrower tile is taken only when it
// cuts the padded extent by more than a fifth: a 128-wide tile needs half again as many operand
// bytes per FLOP as a 256-wide one, which costs more than a few percent of padded columns
// (measured: hidden width 1408 as 11 x 128 ran 27 % slower than as 6 x 256 with 8 % padding).
int pick_bn(int extent, const int* cand, int ncand) {
  int best = cand[0];
  long long best_pad = (long long)((extent + cand[0] - 1) / cand[0]) * cand[0];
  for (int c = 1; c < ncand; ++c) {
    const long long pad = (long long)((extent + cand[c] - 1) / cand[c]) * cand[c];
    if (pad * 5 < best_pad * 4) {
      best_pad = pad;
      best = cand[c];
    }
  }
  return best;
}

template <int ROLE, int CG, int WIDE = 0, int GATHER = 0>
int32_t launch_role(const TcParams& p, const DeviceInfo& di, cudaStream_t st) {
  // The dynamic shared-memory limit of a kernel and the number of CTA pairs that fit are facts
  // of one device: both are kept per device ordinal (0 = not yet known on that device).
  static std::atomic<int> attr_set[kMaxDevices];
  static std::atomic<int> max_clusters[kMaxDevices];
  const int grid = is_plain<ROLE>() ? (p.plain_total < di.sm_count ? p.plain_total : di.sm_count) : di.sm_count;
  if (!attr_set[di.ordinal].load(std::memory_order_acquire)) {
    MOHGE_CUDA(cudaFuncSetAttribute(tc_grouped_kernel<ROLE, CG, WIDE, GATHER>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    Geo<CG, WIDE>::kSmemBytes));
    attr_set[di.ordinal].store(1, std::memory_order_release);
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(grid / CG * CG);
  cfg.blockDim = dim3(block_threads<ROLE, WIDE, GATHER>());
  cfg.dynamicSmemBytes = Geo<CG, WIDE>::kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CG;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (CG == 2) {
    // Persistent kernel: launch exactly as many CTA pairs as can be resident at once (SMs that
    // cannot be paired stay idle); a pair that had to wait for a free slot would run its whole
    // share of the tile list after everyone else.
    int mc = max_clusters[di.ordinal].load(std::memory_order_acquire);
    if (!mc) {
      MOHGE_CUDA(cudaOccupancyMaxActiveClusters(&mc, tc_grouped_kernel<ROLE, CG, WIDE, GATHER>, &cfg));
      if (mc < 1) mc = 1;
      max_clusters[di.ordinal].store(mc, std::memory_order_release);
    }
    const int want = grid / CG < mc ? grid / CG : mc;
    cfg.gridDim = dim3(want * CG);
  }
  cfg.numAttrs = dependent_launch() ? 2 : 1;
#ifdef MOHGE_TC_COUNTERS
  if (const char* e = getenv("MOHGE_TC_GRID")) {        // measurements with fewer CTAs than SMs
    const int g = atoi(e) / CG * CG;
    if (g >= CG && g < (int)cfg.gridDim.x) cfg.gridDim = dim3(g);
  }
#endif
  MOHGE_CUDA(cudaLaunchKernelEx(&cfg, tc_grouped_kernel<ROLE, CG, WIDE, GATHER>, p));
  MOHGE_LAUNCH_CHECK("tc_grouped_kernel");
  return MOHGE_OK;
}

// Double-width entries for a role of a CTA-pair launch.  Default: where the FLOP-weighted mean
// contraction length of the launch is at least kWideMinK (the exposed epilogue of an entry is
// then a few percent of its MMA time and the saved operand traffic outweighs it).  The debugging
// switch MOHGE_TC_WIDE=<bit mask over roles 0..5> overrides the rule.
constexpr double kWideMinK = 3000.0;
bool wide_tiles(const Dims& D, int role) {
  const int mask = switch_value(SW_TC_WIDE);
  if (mask >= 0) return (mask >> role) & 1;
  // The SwiGLU backward has the longest epilogue of all roles (it also reads A and U) and is the
  // role that gains least: before the operand loads carried L2 priorities it was faster on
  // single-width tiles (step 44.1 -> 43.8 ms at the large workload), with them double-width entries
  // win (45.0-46.0 -> 44.9-45.4 ms, five runs each on two GPUs), so it follows the common rule.
  double num = 0.0, den = 0.0;            // mean contraction length, weighted by the group's width
  for (int g = 0; g < D.Ng; ++g) {
    double k;
    switch (role) {
      case ROLE_FWD1: case ROLE_DGRAD_DOWN: k = D.d; break;
      case ROLE_FWD2: k = D.W[g]; break;
      case ROLE_DGRAD_13: k = 2.0 * D.W[g]; break;
      default: k = (double)D.R / D.Ne; break;            // wgrad: rows of an average expert
    }
    num += k * D.W[g];
    den += D.W[g];
  }
  return den > 0.0 && num / den >= kWideMinK;
}

// CTAs per MMA for the grouped roles.  CTA pairs (256-row tiles, each CTA fetching half of B)
// serve batches whose experts fill such tiles.  When an expert receives 128 rows or fewer on
// average the GEMMs are bound by reading the weights once: a pair would spend half of its MMAs
// and A loads on rows of the next expert, so single CTAs with 128-row tiles run instead (measured
// 5.6 against 4.9 TB/s of weight traffic at 16 rows per expert).  MOHGE_TC_CG=1|2 forces a form.
int cta_group_size(const Dims& D) {
  const int forced = switch_value(SW_TC_CG);
  if (forced == 1 || forced == 2) return forced;
  return D.R <= 128 * (int64_t)D.Ne ? 1 : 2;
}

}  // namespace

// Router GEMMs on the tensor cores (BF16 layer dtype).
//   LOGITS     logits[T, NL]  = x . W_r^T + bias                 A = x,          B = w_router
//   ROUTER_DW  dw_router^T[d, NL] = x^T . dl16  (stored transposed)  A = x,       B = dl16 [T, NLp]
//   ROUTER_DX  dx[T, d]      += dl16 . W_r                       A = dl16,       B = w_router
namespace {
// out[i] = part[0][i] + part[1][i] + ... in this fixed order (run-to-run identical bits)
__global__ void __launch_bounds__(256)
sum_partials_kernel(const float* __restrict__ part, int splits, size_t n, float* __restrict__ out) {
  pdl_enter();
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    float acc = part[i];
#pragma unroll 8
    for (int s = 1; s < splits; ++s) acc += part[(size_t)s * n + i];
    out[i] = acc;
  }
}
// the same for [rows][n_cols] partials of the router logits, plus the bias of the column
__global__ void __launch_bounds__(256)
sum_partials_bias_kernel(const float* __restrict__ part, int splits, size_t n, int n_cols,
                         const float* __restrict__ bias, float* __restrict__ out) {
  pdl_enter();
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    float acc = part[i];
#pragma unroll 8
    for (int s = 1; s < splits; ++s) acc += part[(size_t)s * n + i];
    out[i] = bias ? acc + bias[i % n_cols] : acc;
  }
}

// Split-K factor of the router-logits GEMM: a batch of a few hundred tokens has one or two row
// tiles, so two CTAs would walk the whole contraction alone; the contraction is cut so that about
// one CTA per SM works, as far as the partial-sum buffer (sized for the router weight gradient)
// holds [splits][T][NL] floats.  1 = no split (every batch of a few thousand tokens or more).
int router_logits_splits(const Dims& D, int n_tiles) {
  const int64_t tiles = (int64_t)((D.T + BM - 1) / BM) * n_tiles;
  const int64_t k_blocks = (D.d + BK - 1) / BK;
  int64_t s = 148 / tiles;
  const int64_t fit = (int64_t)router_dw_splits(D) * D.d / D.T;
  if (s > fit) s = fit;
  if (s > 16) s = 16;                                    // the sum of the partials costs too
  if (s > k_blocks) s = k_blocks;
  if (s < 4) return 1;                                   // little to win, one more launch to pay
  const int64_t chunk = (k_blocks + s - 1) / s;
  return (int)((k_blocks + chunk - 1) / chunk);          // no split is empty
}
}  // namespace

int32_t launch_tc_plain(const Dims& D, int role, const void* A, const void* B, int64_t b_pitch_elems,
                        void* C, const float* bias, float* partials, int32_t* status, cudaStream_t st,
                        const RouteOut* route, bool* routed) {
  if (routed) *routed = false;
  if (D.T == 0) return MOHGE_OK;
  DeviceInfo di;
  int32_t rcd = current_device(&di);
  if (rcd) return rcd;
  if (di.cc_major != 10) {
    set_error("the BF16 path needs an sm_100 device (found sm_%d%d)", di.cc_major, di.cc_minor);
    return MOHGE_ERR_UNSUPPORTED;
  }
  TcParams p;
  memset(&p, 0, sizeof(p));
  p.gs = make_group_shape(D);
  p.status = status;
  p.bias = bias;
  const uint64_t d = D.d, T = D.T, NL = D.NL;
  uint64_t dims[2], str[1];
  uint32_t box[2];
  int32_t rc;
  // shapes
  if (role == ROLE_LOGITS) {
    p.plain_M = (int)T; p.plain_N = D.NL; p.plain_K = D.d;
    p.Cf = (float*)C;
  } else if (role == ROLE_ROUTER_DW) {
    p.plain_M = D.d; p.plain_N = D.NL; p.plain_K = (int)T;
    p.Cf = (float*)C;
  } else {  // ROLE_ROUTER_DX
    p.plain_M = (int)T; p.plain_N = D.d; p.plain_K = D.NL;
    p.C = (__nv_bfloat16*)C;
  }
  // LOGITS: selection in the epilogue when the shape is one route_token covers, the logits fit the
  // six-stage form (one column tile of at most 160) and the contraction is not split
  bool fuse = false;
  if (role == ROLE_LOGITS && route != nullptr && switch_value(SW_ROUTE_FUSED) != 0) {
    const int bn = (D.NL + 15) / 16 * 16;
    const bool shape_ok = (D.N == 4 || D.N == 8 || D.N == 16 || D.N == 32) && D.Ne % 8 == 0 && bn <= 160 &&
                          D.Ke <= kRouteFuseMaxKe && D.Ke <= D.Kg * D.N;
    fuse = shape_ok && (partials == nullptr || router_logits_splits(D, 1) == 1);
  }
  // tensor maps: from the cache, or encoded now
  MapKey key;
  memset(&key, 0, sizeof(key));
  key.role = role; key.cg = 1; key.accumulate_unused = fuse ? 1 : 0; key.device = di.ordinal; key.d = D.d; key.Ng = D.Ng; key.N = D.N;
  key.T = D.T; key.b_pitch = b_pitch_elems; key.A = A; key.B = B; key.C = C;
  if (!map_cache_find(key, &p)) {
    if (role == ROLE_LOGITS) {
      p.BN[0] = D.NL >= 256 ? 256 : (D.NL + 15) / 16 * 16;
      dims[0] = d; dims[1] = T; str[0] = d * 2; box[0] = BK; box[1] = BM;
      if ((rc = encode_map(&p.mapA[0], A, 2, dims, str, box))) return rc;
      box[1] = BM / 2;                                     // last tile of a CTA's row range (balanced form)
      if ((rc = encode_map(&p.mapA[1], A, 2, dims, str, box))) return rc;
      dims[0] = d; dims[1] = NL; str[0] = d * 2; box[0] = BK; box[1] = p.BN[0];
      if (fuse) {            // two boxes: the Ne expert rows (from row Ng), then the group rows (from row 0)
        box[1] = D.Ne;
        if ((rc = encode_map(&p.mapB[0], B, 2, dims, str, box))) return rc;
        box[1] = p.BN[0] - D.Ne;
        if ((rc = encode_map(&p.mapB[1], B, 2, dims, str, box))) return rc;
      } else {
        if ((rc = encode_map(&p.mapB[0], B, 2, dims, str, box))) return rc;
      }
    } else if (role == ROLE_ROUTER_DW) {
      p.BN[0] = D.NL >= 256 ? 256 : (D.NL + 63) / 64 * 64;
      dims[0] = d; dims[1] = T; str[0] = d * 2; box[0] = 64; box[1] = BK;
      if ((rc = encode_map(&p.mapA[0], A, 2, dims, str, box))) return rc;
      dims[0] = NL; dims[1] = T; str[0] = (uint64_t)b_pitch_elems * 2; box[0] = 64; box[1] = BK;
      if ((rc = encode_map(&p.mapB[0], B, 2, dims, str, box))) return rc;
    } else {
      p.BN[0] = D.d >= 256 ? 256 : (D.d + 63) / 64 * 64;
      dims[0] = NL; dims[1] = T; str[0] = (uint64_t)b_pitch_elems * 2; box[0] = BK; box[1] = BM;
      if ((rc = encode_map(&p.mapA[0], A, 2, dims, str, box))) return rc;
      dims[0] = d; dims[1] = NL; str[0] = d * 2; box[0] = 64; box[1] = BK;
      if ((rc = encode_map(&p.mapB[0], B, 2, dims, str, box))) return rc;
      if ((rc = encode_stage_map(&p.mapO[0][0], C, d, T, d * 2))) return rc;    // dx, read and written
    }
    map_cache_store(key, p);
  }
  p.plain_ntn = (p.plain_N + p.BN[0] - 1) / p.BN[0];
  const int total_kb = (p.plain_K + BK - 1) / BK;
  p.plain_splits = 1;
  p.plain_kchunk = total_kb;
  if (role == ROLE_ROUTER_DW && partials != nullptr) {
    p.plain_splits = router_dw_splits(D);
    p.plain_kchunk = (total_kb + p.plain_splits - 1) / p.plain_splits;
    if (p.plain_splits > 1) p.Cf = partials;
  }
  if (role == ROLE_LOGITS && partials != nullptr) {
    p.plain_splits = router_logits_splits(D, p.plain_ntn);
    p.plain_kchunk = (total_kb + p.plain_splits - 1) / p.plain_splits;
    if (p.plain_splits > 1) p.Cf = partials;
  }
  p.plain_total = ((p.plain_M + BM - 1) / BM) * p.plain_ntn * p.plain_splits;
  // more row tiles than CTAs and a single column tile: contiguous row ranges of equal length
  p.plain_balanced = (role == ROLE_LOGITS && p.plain_splits == 1 && p.plain_ntn == 1 && p.plain_total > di.sm_count) ? 1 : 0;
  if (fuse) {
    p.rf.on = 1; p.rf.Ng = D.Ng; p.rf.N = D.N; p.rf.Kg = D.Kg; p.rf.Ke = D.Ke;
    p.rf.group_idx = route->group_idx; p.rf.expert_idx = route->expert_idx; p.rf.gate_w = route->gate_w;
    p.rf.gs = route->gs; p.rf.esp = route->esp;
    if (routed) *routed = true;
  }
  switch (role) {
    case ROLE_LOGITS: {
      const int32_t rc2 = p.BN[0] <= 160 ? launch_role<ROLE_LOGITS, 1, 2>(p, di, st)
                                          : launch_role<ROLE_LOGITS, 1>(p, di, st);
      if (rc2 || p.plain_splits == 1) return rc2;
      const size_t n = (size_t)D.T * D.NL;
      launch_dep(sum_partials_bias_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), st, partials, p.plain_splits, n, D.NL,
                                                                           bias, (float*)C);
      MOHGE_LAUNCH_CHECK("sum_partials_bias_kernel");
      return MOHGE_OK;
    }
    case ROLE_ROUTER_DW: {
      const int32_t rc2 = launch_role<ROLE_ROUTER_DW, 1>(p, di, st);
      if (rc2 || p.plain_splits == 1) return rc2;
      const size_t n = (size_t)D.NL * D.d;
      launch_dep(sum_partials_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), st, partials, p.plain_splits, n, (float*)C);
      MOHGE_LAUNCH_CHECK("sum_partials_kernel");
      return MOHGE_OK;
    }
    default: return launch_role<ROLE_ROUTER_DX, 1>(p, di, st);
  }
}

// Activation operands per role:
//   FWD1        A = x_perm               C = au_saved, C2 = h_saved
//   FWD2        A = h_saved              C = y_perm
//   DGRAD_DOWN  A = dy_perm, B = au_saved (epilogue input)   C = dau
//   DGRAD_13    A = dau                  C = dx_perm
//   WGRAD_DOWN  A = dy_perm, B = h_saved     -> dw2
//   WGRAD_13    A = dau,     B = x_perm      -> dw13
// Tile list plan of a grouped role (tile widths per group, pair rows, double-width flag): the same
// choices launch_tc_grouped makes, so that the lists of several roles can be built by one launch
// before the GEMMs run.
int tc_dgrad_down_bn(const Dims& D, int g) {
  const int cand_n[2] = {256, 128};
  return pick_bn(D.W[g], cand_n, 2);
}

TilePlan tc_tile_plan(const Dims& D, int role) {
  const int CG = cta_group_size(D);
  const int cand_n[2] = {256, 128};
  const int cand_h[2] = {128, 64};
  int bn_plan[MOHGE_MAX_GROUPS];
  for (int g = 0; g < MOHGE_MAX_GROUPS; ++g) bn_plan[g] = 128;
  for (int g = 0; g < D.Ng; ++g) {
    switch (role) {
      case ROLE_FWD1: bn_plan[g] = pick_bn(D.W[g], cand_h, CG == 2 ? 1 : 2); break;
      case ROLE_FWD2: case ROLE_DGRAD_13: case ROLE_WGRAD_13: bn_plan[g] = pick_bn(D.d, cand_n, 2); break;
      default: bn_plan[g] = pick_bn(D.W[g], cand_n, 2); break;     // DGRAD_DOWN, WGRAD_DOWN
    }
  }
  TilePlan plan = make_plan(D, role, BM * CG, bn_plan, role == ROLE_FWD1);
  plan.wide = (CG == 2 && wide_tiles(D, role)) ? 1 : 0;
  return plan;
}

int32_t launch_tc_grouped(const Dims& D, int role, const GroupPtrs& P, const void* A,
                          const void* B, void* C, void* C2, const int32_t* /*counts*/,
                          const int32_t* aligned, int accumulate, int32_t* tile_count, Tile* tiles,
                          int64_t tiles_cap, int32_t* status, cudaStream_t st, bool list_prebuilt,
                          float* dgate_part, int dgate_slots, const int32_t* gather, const DyFuse* dyf) {
  DeviceInfo di;
  int32_t rcd = current_device(&di);
  if (rcd) return rcd;
  if (di.cc_major != 10) {
    set_error("the BF16 path needs an sm_100 device (found sm_%d%d)", di.cc_major, di.cc_minor);
    return MOHGE_ERR_UNSUPPORTED;
  }
  TcParams p;
  memset(&p, 0, sizeof(p));
  p.gs = make_group_shape(D);
  p.gp = P;
  p.aligned = aligned; p.tile_count = tile_count; p.tiles = tiles;
  p.C = (__nv_bfloat16*)C; p.C2 = (__nv_bfloat16*)C2; p.E = nullptr;
  p.accumulate = accumulate; p.status = status;
  p.dgate_part = role == ROLE_DGRAD_DOWN ? dgate_part : nullptr;
  p.dgate_slots = dgate_slots;
  p.gather = (role == ROLE_FWD1 || role == ROLE_WGRAD_13) ? gather : nullptr;
  const bool dy_gather = dyf != nullptr && (role == ROLE_DGRAD_DOWN || role == ROLE_WGRAD_DOWN);
  if (dy_gather) p.gather = dyf->tok_of_prow;
  p.gather_src = nullptr;
  p.gather_rows = (int)D.T;
  if (dy_gather && role == ROLE_DGRAD_DOWN) {
    p.row_gate = dyf->row_gate;
    p.hs = (__nv_bfloat16*)dyf->hs;
    p.hs_pitch = D.Wmax;
  }

  const uint64_t d = D.d, rows = D.Rcap, pitchAU = 2ull * D.Wmax * 2, pitchH = (uint64_t)D.Wmax * 2;
  const int CG = cta_group_size(D);
  // UMMA N candidates: multiples of 128 so that a CTA pair's half of an MN-major B stays a
  // multiple of the 64-element swizzle block and the epilogue's 64-column boxes tile the width.
  const int cand_n[2] = {256, 128};
  const int ncand = 2;
  const int cand_h[2] = {128, 64};
  int bn_plan[MOHGE_MAX_GROUPS];
  int32_t rc = MOHGE_OK;
  for (int g = 0; g < MOHGE_MAX_GROUPS; ++g) { p.BN[g] = 128; bn_plan[g] = 128; }
  if (role == ROLE_DGRAD_DOWN) p.E = (const __nv_bfloat16*)B;
  MapKey key;
  memset(&key, 0, sizeof(key));
  key.role = role; key.cg = CG; key.device = di.ordinal;
  key.d = D.d; key.Ng = D.Ng; key.N = D.N; key.Wmax = D.Wmax; key.rows = D.Rcap;
  key.A = A; key.B = B; key.C = C; key.C2 = C2; key.gather = p.gather; key.T = D.T;
  for (int g = 0; g < D.Ng; ++g) {
    key.W[g] = D.W[g];
    key.w[0][g] = P.w13[g]; key.w[1][g] = P.w2[g]; key.w[2][g] = P.dw13[g]; key.w[3][g] = P.dw2[g];
  }
  const bool cached = map_cache_find(key, &p);
  if (p.gather) p.gather_src = (role == ROLE_FWD1 || dy_gather) ? A : B;
  for (int g = 0; g < D.Ng && rc == MOHGE_OK && !cached; ++g) {
    const uint64_t W = D.W[g], N = D.N;
    uint64_t dims[3], str[2];
    uint32_t box[3];
    switch (role) {
      case ROLE_FWD1: {
        const int half = pick_bn(D.W[g], cand_h, CG == 2 ? 1 : 2);
        p.BN[g] = 2 * half; bn_plan[g] = half;
        if (p.gather) {      // A = x [T, d], gathered row by row by the producer warp
          p.gather_src = A;
        } else {
          dims[0] = d; dims[1] = rows; str[0] = d * 2; box[0] = BK; box[1] = BM;
          rc = encode_map(&p.mapA[g], A, 2, dims, str, box);
        }
        if (rc) break;
        dims[0] = d; dims[1] = W; dims[2] = 2 * N; str[0] = d * 2; str[1] = W * d * 2;
        box[0] = BK; box[1] = half; box[2] = 1;
        rc = encode_map(&p.mapB[g], P.w13[g], 3, dims, str, box);
        if (rc) break;
        rc = encode_stage_map(&p.mapO[0][g], C, W, rows, pitchAU);
        if (rc) break;
        rc = encode_stage_map(&p.mapO[1][g], (const char*)C + W * 2, W, rows, pitchAU);
        if (rc) break;
        rc = encode_stage_map(&p.mapO[2][g], C2, W, rows, pitchH);
      } break;
      case ROLE_FWD2: {
        p.BN[g] = bn_plan[g] = pick_bn(D.d, cand_n, ncand);
        dims[0] = W; dims[1] = rows; str[0] = pitchH; box[0] = BK; box[1] = BM;
        rc = encode_map(&p.mapA[g], A, 2, dims, str, box);
        if (rc) break;
        dims[0] = W; dims[1] = d; dims[2] = N; str[0] = W * 2; str[1] = d * W * 2;
        box[0] = BK; box[1] = p.BN[g] / CG; box[2] = 1;
        rc = encode_map(&p.mapB[g], P.w2[g], 3, dims, str, box);
        if (rc || g > 0) break;
        rc = encode_stage_map(&p.mapO[0][0], C, d, rows, d * 2);
      } break;
      case ROLE_DGRAD_DOWN: {
        p.BN[g] = bn_plan[g] = pick_bn(D.W[g], cand_n, ncand);
        if (!dy_gather) {    // else A = dy [T, d], gathered row by row by the producer warp
          dims[0] = d; dims[1] = rows; str[0] = d * 2; box[0] = BK; box[1] = BM;
          rc = encode_map(&p.mapA[g], A, 2, dims, str, box);
        }
        if (rc) break;
        rc = encode_mn_map(&p.mapB[g], P.w2[g], W, d, W * 2, N, d * W * 2, p.BN[g] / CG / 64, &p.b_blk[g]);
        if (rc) break;
        rc = encode_stage_map(&p.mapE[0][g], B, W, rows, pitchAU);
        if (rc) break;
        rc = encode_stage_map(&p.mapE[1][g], (const char*)B + W * 2, W, rows, pitchAU);
        if (rc) break;
        rc = encode_stage_map(&p.mapO[0][g], C, W, rows, pitchAU);
        if (rc) break;
        rc = encode_stage_map(&p.mapO[1][g], (const char*)C + W * 2, W, rows, pitchAU);
      } break;
      case ROLE_DGRAD_13: {
        p.BN[g] = bn_plan[g] = pick_bn(D.d, cand_n, ncand);
        dims[0] = 2 * W; dims[1] = rows; str[0] = pitchAU; box[0] = BK; box[1] = BM;
        rc = encode_map(&p.mapA[g], A, 2, dims, str, box);
        if (rc) break;
        rc = encode_mn_map(&p.mapB[g], P.w13[g], d, 2 * W, d * 2, N, 2 * W * d * 2, p.BN[g] / CG / 64, &p.b_blk[g]);
        if (rc || g > 0) break;
        rc = encode_stage_map(&p.mapO[0][0], C, d, rows, d * 2);
      } break;
      case ROLE_WGRAD_DOWN: {
        p.BN[g] = bn_plan[g] = pick_bn(D.W[g], cand_n, ncand);
        if (!dy_gather) rc = encode_mn_map(&p.mapA[g], A, d, rows, d * 2, 0, 0, 2, &p.a_blk[g]);
        if (rc) break;
        rc = encode_mn_map(&p.mapB[g], B, W, rows, pitchH, 0, 0, p.BN[g] / CG / 64, &p.b_blk[g]);
        if (rc) break;
        rc = encode_stage_map_f32(&p.mapO[0][g], P.dw2[g], W, d, N);
      } break;
      default: {  // ROLE_WGRAD_13
        p.BN[g] = bn_plan[g] = pick_bn(D.d, cand_n, ncand);
        rc = encode_mn_map(&p.mapA[g], A, 2 * W, rows, pitchAU, 0, 0, 2, &p.a_blk[g]);
        if (rc) break;
        if (p.gather) {      // B = x [T, d], gathered row by row by the producer warp
          p.gather_src = B;
        } else {
          rc = encode_mn_map(&p.mapB[g], B, d, rows, d * 2, 0, 0, p.BN[g] / CG / 64, &p.b_blk[g]);
        }
        if (rc) break;
        rc = encode_stage_map_f32(&p.mapO[0][g], P.dw13[g], d, 2 * W, N);
      } break;
    }
  }
  if (rc) return rc;
  if (!cached) map_cache_store(key, p);
  const TilePlan plan = tc_tile_plan(D, role);
  const bool wide = plan.wide != 0;
  if (!list_prebuilt) {
    rc = launch_build_tiles_plan(plan, aligned, tile_count, tiles, tiles_cap, status, st);
    if (rc) return rc;
  }
  if (p.gather && role == ROLE_DGRAD_DOWN) {     // row-gathering forms of the roles that read dy_perm
    if (CG == 2 && wide) return launch_role<ROLE_DGRAD_DOWN, 2, 1, 1>(p, di, st);
    if (CG == 2) return launch_role<ROLE_DGRAD_DOWN, 2, 0, 1>(p, di, st);
    return launch_role<ROLE_DGRAD_DOWN, 1, 0, 1>(p, di, st);
  }
  if (p.gather && role == ROLE_WGRAD_DOWN) {
    if (CG == 2 && wide) return launch_role<ROLE_WGRAD_DOWN, 2, 1, 1>(p, di, st);
    if (CG == 2) return launch_role<ROLE_WGRAD_DOWN, 2, 0, 1>(p, di, st);
    return launch_role<ROLE_WGRAD_DOWN, 1, 0, 1>(p, di, st);
  }
  if (p.gather) {          // row-gathering form of the two roles that read x_perm
    if (role == ROLE_FWD1) {
      if (CG == 2 && wide) return launch_role<ROLE_FWD1, 2, 1, 1>(p, di, st);
      if (CG == 2) return launch_role<ROLE_FWD1, 2, 0, 1>(p, di, st);
      return launch_role<ROLE_FWD1, 1, 0, 1>(p, di, st);
    }
    if (CG == 2 && wide) return launch_role<ROLE_WGRAD_13, 2, 1, 1>(p, di, st);
    if (CG == 2) return launch_role<ROLE_WGRAD_13, 2, 0, 1>(p, di, st);
    return launch_role<ROLE_WGRAD_13, 1, 0, 1>(p, di, st);
  }
  if (CG == 2 && wide) {
    switch (role) {
      case ROLE_FWD1: return launch_role<ROLE_FWD1, 2, 1>(p, di, st);
      case ROLE_FWD2: return launch_role<ROLE_FWD2, 2, 1>(p, di, st);
      case ROLE_DGRAD_DOWN: return launch_role<ROLE_DGRAD_DOWN, 2, 1>(p, di, st);
      case ROLE_DGRAD_13: return launch_role<ROLE_DGRAD_13, 2, 1>(p, di, st);
      case ROLE_WGRAD_DOWN: return launch_role<ROLE_WGRAD_DOWN, 2, 1>(p, di, st);
      default: return launch_role<ROLE_WGRAD_13, 2, 1>(p, di, st);
    }
  }
  if (CG == 2) {
    switch (role) {
      case ROLE_FWD1: return launch_role<ROLE_FWD1, 2>(p, di, st);
      case ROLE_FWD2: return launch_role<ROLE_FWD2, 2>(p, di, st);
      case ROLE_DGRAD_DOWN: return launch_role<ROLE_DGRAD_DOWN, 2>(p, di, st);
      case ROLE_DGRAD_13: return launch_role<ROLE_DGRAD_13, 2>(p, di, st);
      case ROLE_WGRAD_DOWN: return launch_role<ROLE_WGRAD_DOWN, 2>(p, di, st);
      default: return launch_role<ROLE_WGRAD_13, 2>(p, di, st);
    }
  }
  switch (role) {
    case ROLE_FWD1: return launch_role<ROLE_FWD1, 1>(p, di, st);
    case ROLE_FWD2: return launch_role<ROLE_FWD2, 1>(p, di, st);
    case ROLE_DGRAD_DOWN: return launch_role<ROLE_DGRAD_DOWN, 1>(p, di, st);
    case ROLE_DGRAD_13: return launch_role<ROLE_DGRAD_13, 1>(p, di, st);
    case ROLE_WGRAD_DOWN: return launch_role<ROLE_WGRAD_DOWN, 1>(p, di, st);
    default: return launch_role<ROLE_WGRAD_13, 1>(p, di, st);
  }
}

}  // namespace mohge

extern "C" void mohge_map_cache_stats(int64_t* hits, int64_t* misses) {
  if (hits) *hits = (int64_t)mohge::g_map_hits.load();
  if (misses) *misses = (int64_t)mohge::g_map_misses.load();
}

#ifdef MOHGE_TC_COUNTERS
// Copies the counter table [9 roles][160 CTAs][12 slots] (uint64) to `host_out` after a device
// synchronisation; `reset` != 0 clears it afterwards.  Slots: 0 launches, 1 issuer loop clocks,
// 2 issuer waiting for operands, 3 issuer waiting for an accumulator, 4 producer waiting for a
// stage, 5 epilogue warp waiting for an accumulator, 6 epilogue loop clocks, 7 CTA lifetime ns,
// 8 tiles, 9 k-blocks (a double-width entry counts twice), 10 clocks between the 8th and the 24th
// k-block of tiles with 32 k-blocks or more, 11 the k-blocks those clocks cover.
extern "C" int32_t mohge_debug_tc_counters(unsigned long long* host_out, int32_t reset) {
  using namespace mohge;
  MOHGE_CUDA(cudaDeviceSynchronize());
  MOHGE_CUDA(cudaMemcpyFromSymbol(host_out, g_tc_counters, sizeof(g_tc_counters)));
  if (reset) {
    void* p = nullptr;
    MOHGE_CUDA(cudaGetSymbolAddress(&p, g_tc_counters));
    MOHGE_CUDA(cudaMemset(p, 0, sizeof(g_tc_counters)));
  }
  return MOHGE_OK;
}
#endif
