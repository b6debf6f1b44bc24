// Two-level selection (Sec. 3.2, Eq. 2-6) as the epilogue of the router-logits GEMM: one thread
// per token, the token's logits read straight from the accumulator in tensor memory.
//
// The arithmetic is the selection contract of router.cu, operation for operation (same float32
// sequence, same tie rules, same reading of NaN), so the indices and gates are bit-identical to
// those of router_select_kernel on the same logits; only the work is laid out differently:
//   * an epilogue thread owns one accumulator row = one token, so the warp butterflies of the
//     one-warp-per-token kernel become register loops of one thread: the maximum of a group is a
//     running maximum, the balanced tree sum adds neighbours first level by level, the K_e
//     rounds of arg-max become an insertion of each candidate (expert ids ascending) into a list
//     sorted by key, a candidate going above exactly the entries whose key is strictly smaller;
//   * the B operand of the GEMM is staged with the expert rows of the router weight first and
//     the group rows behind them, so that group g's N logits are the accumulator columns
//     [g N, g N + N) (aligned to N, a power of two) and the group logits the columns [Ne, Ne + Ng);
//   * kRouteSplit warps share a quarter of the accumulator rows: warp s of them takes, for each
//     of its tokens, the selected groups of rank s (mod kRouteSplit) and keeps its own sorted list;
//     the lists meet in shared memory and are merged by (key descending, id ascending), which is
//     the order one list would have had.
// Covered shapes: N a power of two from 4 to 32 (then the padded slot count P of the contract
// equals N), Ne a multiple of 8, K_e <= 8.  Everything else takes the two-kernel route.
#pragma once

#include "select_math.cuh"

namespace mohge {

struct RouteFuse {
  int on;                        // 1: LOGITS launch also selects
  int Ng, N, Kg, Ke;
  int32_t* group_idx;            // [T, Kg]
  int32_t* expert_idx;           // [T, Ke]
  float* gate_w;                 // [T, Ke]
  float* gs;                     // [T, Ng]
  float* esp;                    // [T, Ne]
};

constexpr int kRouteFuseMaxKe = 8;

template <int N> __device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, uint32_t (&r)[N]);
template <> __device__ __forceinline__ void tmem_ld_cols<4>(uint32_t taddr, uint32_t (&r)[4]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(taddr) : "memory");
}
template <> __device__ __forceinline__ void tmem_ld_cols<8>(uint32_t taddr, uint32_t (&r)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr) : "memory");
}
template <> __device__ __forceinline__ void tmem_ld_cols<16>(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
template <> __device__ __forceinline__ void tmem_ld_cols<32>(uint32_t taddr, uint32_t (&r)[32]) {
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

constexpr int kRouteSplit = 2;             // epilogue warps per quarter of the accumulator rows

// The K_e best (key, expert id) so far, sorted by (key descending, id ascending); empty = (-1, -1).
struct RouteList {
  float wk[kRouteFuseMaxKe];
  int we[kRouteFuseMaxKe];
};

// Part of one token (row `t` of the batch, accumulator row of this thread at tensor-memory address
// taddr) done by warp `split` of the kRouteSplit that share the row: group logits and Eq. 2 (every
// split computes them, split 0 stores them), then the expert logits (+ bias) of the groups
// g = split (mod kRouteSplit) to memory and, for the token's selected groups of rank = split
// (mod kRouteSplit), Eq. 3-4 and the candidates of Eq. 5 into L.  Every lane of the warp
// must call (the tensor-memory loads are warp-collective); lanes with !row_ok store nothing.
// Returns true when a NaN logit was met.
template <int N>
__device__ __forceinline__ bool route_token_groups(const RouteFuse& f, uint32_t taddr, bool row_ok, long long t,
                                                   float* __restrict__ logits, const float* __restrict__ bias,
                                                   int split, RouteList& L) {
  const int Ng = f.Ng, Ne = f.Ng * N, NL = Ng + Ne;
  bool saw_nan = false;
  auto clean = [&](float v) {                  // NaN logits rank below every number
    if (v != v) { saw_nan = true; return -3.402823466e+38f; }
    return v;
  };
  float* const po = logits + t * NL;
  const bool vec = ((NL | Ng) & 3) == 0;       // 16-byte aligned rows and expert columns
  const bool lead = row_ok && split == 0;
  // ---- group logits, Eq. 2: K_g rounds of arg-max over the raw logits, ties to the lowest g
  float lg[MOHGE_MAX_GROUPS];
  {
    uint32_t r[8];
    tmem_ld_cols<8>(taddr + Ne, r);
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int g = 0; g < MOHGE_MAX_GROUPS; ++g) {
      float v = 0.0f;
      if (g < Ng) {
        v = __uint_as_float(r[g]);
        if (bias) v += bias[g];
        if (lead) po[g] = v;
        v = clean(v);
      }
      lg[g] = v;
    }
  }
  unsigned gmask = 0;
  for (int k = 0; k < f.Kg; ++k) {
    int best = -1;
    float bv = 0.0f;
#pragma unroll
    for (int g = 0; g < MOHGE_MAX_GROUPS; ++g) {
      if (g < Ng && !((gmask >> g) & 1u) && (best < 0 || lg[g] > bv)) {
        best = g;
        bv = lg[g];
      }
    }
    gmask |= 1u << best;
    if (lead) f.group_idx[t * f.Kg + k] = best;
  }
  if (lead) {
#pragma unroll
    for (int g = 0; g < MOHGE_MAX_GROUPS; ++g)
      if (g < Ng) f.gs[t * Ng + g] = sig_s(lg[g]);
  }
  // ---- Eq. 3-5: this split takes the selected groups of rank split, split + kRouteSplit, ...
  // (ascending group order).  Which group that is differs from thread to thread while tensor
  // memory is read with one column address per warp, so the warp reads every group and a thread
  // keeps the logits of its own; after that no thread works on a group it did not select.
#pragma unroll
  for (int k = 0; k < kRouteFuseMaxKe; ++k) { L.wk[k] = -1.0f; L.we[k] = -1; }
  float* const pe = f.esp + t * Ne;
  if (split >= f.Kg) {          // no selected group falls to this split: only its share of the logits
    for (int g = split; g < Ng; g += kRouteSplit) {
      uint32_t r[N];
      tmem_ld_cols<N>(taddr + g * N, r);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      const float* bg = bias ? bias + Ng + g * N : nullptr;
      if (row_ok) {
        float* pl = po + Ng + g * N;
#pragma unroll
        for (int i = 0; i < N; ++i) {
          float v = __uint_as_float(r[i]);
          if (bg) v += bg[i];
          pl[i] = v;
        }
      }
    }
  }
  for (int rk = split; rk < f.Kg; rk += kRouteSplit) {
    const int gt = (int)__fns(gmask, 0, rk + 1);       // position of the (rk + 1)-th set bit
    float l[N];
#pragma unroll
    for (int i = 0; i < N; ++i) l[i] = 0.0f;
    float lgg = 0.0f;                                   // group logit of gt
    for (int g = 0; g < Ng; ++g) {
      uint32_t r[N];
      tmem_ld_cols<N>(taddr + g * N, r);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      const float* bg = bias ? bias + Ng + g * N : nullptr;
      float v[N];
#pragma unroll
      for (int i = 0; i < N; ++i) {
        v[i] = __uint_as_float(r[i]);
        if (bg) v[i] += bg[i];
      }
      // the logits of group g are stored once: by the split g falls to, in its first pass
      if (row_ok && rk == split && (g % kRouteSplit) == split) {
        float* pl = po + Ng + g * N;
        if (vec) {
#pragma unroll
          for (int i = 0; i < N; i += 4) *reinterpret_cast<float4*>(pl + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
        } else {
#pragma unroll
          for (int i = 0; i < N; ++i) pl[i] = v[i];
        }
      }
      const bool mine = g == gt;
#pragma unroll
      for (int i = 0; i < N; ++i) l[i] = mine ? v[i] : l[i];
#pragma unroll
      for (int gg = 0; gg < MOHGE_MAX_GROUPS; ++gg) lgg = (mine && gg == g) ? lg[gg] : lgg;
    }
    const float sgv = sig_s(lgg);
    float m = -INFINITY;
#pragma unroll
    for (int i = 0; i < N; ++i) { l[i] = clean(l[i]); m = fmaxf(m, l[i]); }
    float pr[N], tr[N];
#pragma unroll
    for (int i = 0; i < N; ++i) { pr[i] = exp_s(__fsub_rn(l[i], m)); tr[i] = pr[i]; }
    // balanced binary tree, neighbours first
#pragma unroll
    for (int w = N; w > 1; w >>= 1) {
#pragma unroll
      for (int i = 0; i < (w >> 1); ++i) tr[i] = __fadd_rn(tr[2 * i], tr[2 * i + 1]);
    }
    const float S = tr[0];
    const float rr = __fdiv_rn(sgv, S);
    float es[N];
#pragma unroll
    for (int i = 0; i < N; ++i) {
      es[i] = __fdiv_rn(pr[i], S);
      const float ck = __fmul_rn(pr[i], rr);
      const int ce = gt * N + i;
      // ids ascend inside a split's walk, so a strict comparison keeps ties in id order
#pragma unroll
      for (int k = kRouteFuseMaxKe - 1; k >= 0; --k) {
        const bool gt_k = ck > L.wk[k];
        if (k + 1 < kRouteFuseMaxKe) {
          L.wk[k + 1] = gt_k ? L.wk[k] : L.wk[k + 1];
          L.we[k + 1] = gt_k ? L.we[k] : L.we[k + 1];
        }
        L.wk[k] = gt_k ? ck : L.wk[k];
        L.we[k] = gt_k ? ce : L.we[k];
      }
    }
    if (row_ok) {
      float* ps = pe + gt * N;
#pragma unroll
      for (int i = 0; i < N; i += 4) *reinterpret_cast<float4*>(ps + i) = make_float4(es[i], es[i + 1], es[i + 2], es[i + 3]);
    }
  }
  // ES' of the experts of unselected groups is 0 (Eq. 3): the splits share those groups too
  if (row_ok) {
    const unsigned zmask = ~gmask & ((1u << Ng) - 1u);
    for (int j = split; j < Ng - f.Kg; j += kRouteSplit) {
      float* ps = pe + (int)__fns(zmask, 0, j + 1) * N;
#pragma unroll
      for (int i = 0; i < N; i += 4) *reinterpret_cast<float4*>(ps + i) = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    }
  }
  return saw_nan;
}

// The entries of O go into L: an entry goes above exactly the entries after which it sorts in
// (key descending, id ascending); empty entries (-1, -1) change nothing.
__device__ __forceinline__ void route_list_merge(RouteList& L, const RouteList& O) {
#pragma unroll
  for (int j = 0; j < kRouteFuseMaxKe; ++j) {
    const float ck = O.wk[j];
    const int ce = O.we[j];
#pragma unroll
    for (int k = kRouteFuseMaxKe - 1; k >= 0; --k) {
      const bool gt = ck > L.wk[k] || (ck == L.wk[k] && ce < L.we[k]);
      if (k + 1 < kRouteFuseMaxKe) {
        L.wk[k + 1] = gt ? L.wk[k] : L.wk[k + 1];
        L.we[k + 1] = gt ? L.we[k] : L.we[k + 1];
      }
      L.wk[k] = gt ? ck : L.wk[k];
      L.we[k] = gt ? ce : L.we[k];
    }
  }
}

// Eq. 6: gate_k = key_k / (left-to-right sum of the K_e selected keys); indices and gates to memory
__device__ __forceinline__ void route_token_finish(const RouteFuse& f, bool row_ok, long long t, const RouteList& L) {
  float sum = L.wk[0];
#pragma unroll
  for (int k = 1; k < kRouteFuseMaxKe; ++k)
    if (k < f.Ke) sum = __fadd_rn(sum, L.wk[k]);
  if (row_ok) {
#pragma unroll
    for (int k = 0; k < kRouteFuseMaxKe; ++k) {
      if (k < f.Ke) {
        f.expert_idx[t * f.Ke + k] = L.we[k];
        f.gate_w[t * f.Ke + k] = __fdiv_rn(L.wk[k], sum);
      }
    }
  }
}

}  // namespace mohge
