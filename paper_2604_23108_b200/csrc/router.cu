// Two-level router (Sec. 3.2, Eq. 2-6), auxiliary-loss statistics (Eq. 7-14) and the
// element-wise part of the router backward.  One warp per token.
//
// This translation unit is compiled with -fmad=false and every float operation that decides
// an index is written with an explicit round-to-nearest intrinsic, because the selection is a
// contract: given the float32 logits, the indices are reproducible bit for bit.
//
// Selection arithmetic (IEEE-754 binary32, round to nearest even, no fused multiply-add):
//   groups   K_g rounds of arg-max over the raw group logits (sigmoid is monotone), ties to
//            the lowest g
//   exp_s(z) for z <= 0:  zc = max(z, -100); n = rint(zc * 0x1.715476p+0);
//            r = zc - n * 0x1.62e4p-1;  r = r - n * 0x1.7f7d1cp-20;
//            p = Horner (separate multiply, add) with 1/7!, 1/6!, ..., 1/2!, 1, 1 rounded to
//            float32;  result p * 2^n;  z < -87 gives +0
//   sig_s(z) e = exp_s(-|z|);  z >= 0 ? 1/(1+e) : e/(1+e)
//   per selected group g: m = max_i l_i; p_i = exp_s(l_i - m); S = balanced binary tree sum
//            of p (neighbours first, padded with +0 to a power of two); r = sig_s(l_g) / S;
//            key_i = p_i * r; ES'_i = p_i / S.  Experts of unselected groups: key = -1.
//   experts  K_e rounds of arg-max over (key descending, e ascending)
//   gate_k = key_k / (left-to-right sum of the K_e selected keys)
//   NaN      a NaN logit is invalid input: it is read as -FLT_MAX (the most negative finite
//            float32), i.e. it ranks below every number, ties among such entries go to the lowest
//            index as everywhere else, and the device status word records (3 << 24)
//
// Slot layout inside a warp: group g owns P = next_pow2(N) consecutive slots, slot s = g*P + i
// lives in lane s % 32, register s / 32; a group never straddles a register because P | 32.
// Only the K_g selected groups take part in Eq. 3-5 (experts of the others can never be picked,
// their ES' is 0), so the selection and the router backward work on a COMPACT layout: the
// selected groups in ascending order, slot c = (rank of the group among the selected) * P + i,
// K_g * P slots instead of N_g * P.  Expert ids stay ascending in c, so ties still go to the
// lowest expert id.

#include "common.cuh"
#include "select_math.cuh"

namespace mohge {
namespace {

constexpr unsigned kFull = 0xffffffffu;

// Order-preserving map float -> unsigned (a < b  <=>  ord_key(a) < ord_key(b), no NaNs here) and
// its inverse, so that one integer warp reduction finds the largest key.
__device__ __forceinline__ unsigned ord_key(float k) {
  const unsigned b = __float_as_uint(k);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float ord_key_inv(unsigned u) {
  return __uint_as_float((u & 0x80000000u) ? (u & 0x7fffffffu) : ~u);
}

// K rounds of warp arg-max over (key descending, index ascending).  key[j] belongs to expert
// eid[j] (ascending in j inside a lane).  Winner of round k is left in lane k (win_e, win_key).
// A round is one max-reduction over the ordered keys and one min-reduction over the indices of
// the lanes that hold the maximum; taken experts drop to the key -3.
template <int J>
__device__ __forceinline__ void warp_topk(float (&key)[J], const int (&eid)[J], int K, int lane,
                                          int& win_e, float& win_key) {
  win_e = -1;
  win_key = 0.0f;
  unsigned uk[J];
#pragma unroll
  for (int j = 0; j < J; ++j) uk[j] = ord_key(key[j]);
  const unsigned taken = ord_key(-3.0f);
  for (int k = 0; k < K; ++k) {
    unsigned bu = 0;                     // below every ordered key
    int be = 0x7fffffff;
#pragma unroll
    for (int j = 0; j < J; ++j) {
      if (uk[j] > bu) {
        bu = uk[j];
        be = eid[j];
      }
    }
    const unsigned m = __reduce_max_sync(kFull, bu);
    const int we = __reduce_min_sync(kFull, bu == m ? be : 0x7fffffff);
#pragma unroll
    for (int j = 0; j < J; ++j)
      if (eid[j] == we) uk[j] = taken;
    if (lane == k) {
      win_e = we;
      win_key = ord_key_inv(m);
    }
  }
}

struct RouterShape {
  int T, Ng, N, P, logP, NL, Ne, Kg, Ke;
};

// Compact slot c of a token whose selected groups are the set bits of gmask: the group (the
// (c >> logP)-th set bit, ascending), the expert inside it, the flat expert id; valid = false for
// slots past the K_g selected groups or past the N experts of a group.
struct CompactSlot {
  int g, i, e;
  bool valid;
};
__device__ __forceinline__ CompactSlot compact_slot(const RouterShape& s, unsigned gmask, int c) {
  CompactSlot q;
  const int rank = c >> s.logP;
  q.i = c & (s.P - 1);
  q.valid = rank < s.Kg && q.i < s.N;
  q.g = q.valid ? (int)__fns(gmask, 0, rank + 1) : 0;      // position of the (rank + 1)-th set bit
  q.e = q.g * s.N + q.i;
  return q;
}

template <int J, int JC>
__global__ void __launch_bounds__(256)
router_select_kernel(RouterShape s, const float* __restrict__ logits, int32_t* __restrict__ group_idx,
                     int32_t* __restrict__ expert_idx, float* __restrict__ gate_w,
                     float* __restrict__ gs_saved, float* __restrict__ esp_saved, int32_t* status) {
  pdl_enter();
  const int lane = threadIdx.x & 31;
  bool saw_nan = false;
  auto clean = [&](float v) {                 // NaN logits rank below every number
    if (v != v) { saw_nan = true; return -3.402823466e+38f; }
    return v;
  };
  const int warps_total = (gridDim.x * blockDim.x) >> 5;
  for (int t = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; t < s.T; t += warps_total) {
    const float* L = logits + (size_t)t * s.NL;
    // ---- Eq. 2: top-K_g groups by raw logit ----
    float lg[MOHGE_MAX_GROUPS];
#pragma unroll
    for (int g = 0; g < MOHGE_MAX_GROUPS; ++g) lg[g] = g < s.Ng ? clean(L[g]) : 0.0f;
    unsigned gmask = 0;
    for (int k = 0; k < s.Kg; ++k) {
      int best = -1;
      float bv = 0.0f;
#pragma unroll
      for (int g = 0; g < MOHGE_MAX_GROUPS; ++g) {
        if (g < s.Ng && !((gmask >> g) & 1u) && (best < 0 || lg[g] > bv)) {
          best = g;
          bv = lg[g];
        }
      }
      gmask |= 1u << best;
      if (lane == 0) group_idx[(size_t)t * s.Kg + k] = best;
    }
    const float gsv = lane < s.Ng ? sig_s(clean(L[lane])) : 0.0f;      // GS of group `lane`
    if (lane < s.Ng) gs_saved[(size_t)t * s.Ng + lane] = gsv;
    // ES' of the experts of unselected groups is 0 (Eq. 3)
#pragma unroll
    for (int j = 0; j < J; ++j) {
      const int sl = lane + 32 * j;
      const int g = sl >> s.logP, i = sl & (s.P - 1);
      if (g < s.Ng && i < s.N && !((gmask >> g) & 1u)) esp_saved[(size_t)t * s.Ne + g * s.N + i] = 0.0f;
    }
    // ---- Eq. 3, 4: keys of the lane's compact slots (selected groups only) ----
    float key[JC];
    int eid[JC];
#pragma unroll
    for (int j = 0; j < JC; ++j) {
      const CompactSlot q = compact_slot(s, gmask, lane + 32 * j);
      const float l = q.valid ? clean(L[s.Ng + q.e]) : -INFINITY;
      float m = l;
      for (int mask = s.P >> 1; mask > 0; mask >>= 1) m = fmaxf(m, __shfl_xor_sync(kFull, m, mask));
      const float p = q.valid ? exp_s(__fsub_rn(l, m)) : 0.0f;
      float S = p;
      for (int mask = 1; mask < s.P; mask <<= 1) S = __fadd_rn(S, __shfl_xor_sync(kFull, S, mask));
      const float sg = __shfl_sync(kFull, gsv, q.g & 31);          // GS of this slot's group
      float kv = -2.0f;
      if (q.valid) {
        kv = __fmul_rn(p, __fdiv_rn(sg, S));
        esp_saved[(size_t)t * s.Ne + q.e] = __fdiv_rn(p, S);
      }
      key[j] = kv;
      eid[j] = q.valid ? q.e : (0x7ffffff0 + j);
    }
    // ---- Eq. 5: top-K_e experts, Eq. 6: normalise ----
    int we;
    float wk;
    warp_topk<JC>(key, eid, s.Ke, lane, we, wk);
    float sum = __shfl_sync(kFull, wk, 0);
    for (int k = 1; k < s.Ke; ++k) sum = __fadd_rn(sum, __shfl_sync(kFull, wk, k));
    if (lane < s.Ke) {
      expert_idx[(size_t)t * s.Ke + lane] = we;
      gate_w[(size_t)t * s.Ke + lane] = __fdiv_rn(wk, sum);
    }
  }
  if (saw_nan && status != nullptr) atomicCAS(status, 0, 3 << 24);
}


// the three count arrays start at zero (one launch instead of three memsets)
__global__ void zero_counts_kernel(int32_t* group_count, int Ng, int32_t* cnt_routed, int32_t* cnt_lit,
                                   int Ne) {
  pdl_enter();
  for (int i = threadIdx.x; i < Ne; i += blockDim.x) {
    cnt_routed[i] = 0;
    cnt_lit[i] = 0;
    if (i < Ng) group_count[i] = 0;
  }
  for (int i = Ne + threadIdx.x; i < Ng; i += blockDim.x) group_count[i] = 0;
}

// ---------------------------------------------------------------- statistics (Eq. 7-14)
constexpr int kStatsThreads = 512;
constexpr int kStatsWarps = kStatsThreads / 32;

template <int J, int JC>
__global__ void __launch_bounds__(kStatsThreads)
aux_stats_kernel(RouterShape s, float eps, const float* __restrict__ gs, const float* __restrict__ esp,
                 const int32_t* __restrict__ group_idx, const int32_t* __restrict__ expert_idx,
                 int32_t* __restrict__ group_count, int32_t* __restrict__ cnt_routed,
                 int32_t* __restrict__ cnt_lit, double* __restrict__ partials) {
  pdl_enter();
  __shared__ int s_cg[MOHGE_MAX_GROUPS];
  __shared__ int s_cr[256];
  __shared__ int s_cl[256];
  __shared__ double s_sum[kStatsWarps][256 + MOHGE_MAX_GROUPS];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int i = threadIdx.x; i < 256; i += blockDim.x) {
    s_cr[i] = 0;
    s_cl[i] = 0;
    if (i < MOHGE_MAX_GROUPS) s_cg[i] = 0;
  }
  __syncthreads();
  double accE[J];
#pragma unroll
  for (int j = 0; j < J; ++j) accE[j] = 0.0;
  double accG = 0.0;
  const int warps_total = gridDim.x * kStatsWarps;
  for (int t = blockIdx.x * kStatsWarps + warp; t < s.T; t += warps_total) {
    int myg = lane < s.Kg ? group_idx[(size_t)t * s.Kg + lane] : -1;
    const unsigned gmask = __reduce_or_sync(kFull, myg >= 0 ? (1u << myg) : 0u);
    if (myg >= 0) atomicAdd(&s_cg[myg], 1);
    if (lane < s.Ke) atomicAdd(&s_cr[expert_idx[(size_t)t * s.Ke + lane]], 1);
    // Eq. 10: s'_g = GS_g / sum_j GS_j
    const float gv = lane < s.Ng ? gs[(size_t)t * s.Ng + lane] : 0.0f;
    float gsum = gv;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) gsum += __shfl_xor_sync(kFull, gsum, off);
    if (lane < s.Ng) accG += (double)(gv / gsum);
    // Eq. 14: S_e = ES'_e / (sum over the group + eps); ES' of unselected groups is 0
#pragma unroll
    for (int j = 0; j < J; ++j) {
      const int sl = lane + 32 * j;
      const int g = sl >> s.logP;
      const int i = sl & (s.P - 1);
      const bool valid = g < s.Ng && i < s.N;
      const float ev = valid ? esp[(size_t)t * s.Ne + g * s.N + i] : 0.0f;
      float grp = ev;
      for (int mask = 1; mask < s.P; mask <<= 1) grp += __shfl_xor_sync(kFull, grp, mask);
      if (valid) accE[j] += (double)(ev / (grp + eps));
    }
    // Eq. 12 indicator: top-K_e of ES' over the experts of the selected groups (compact slots)
    float key[JC];
    int eid[JC];
#pragma unroll
    for (int j = 0; j < JC; ++j) {
      const CompactSlot q = compact_slot(s, gmask, lane + 32 * j);
      key[j] = q.valid ? esp[(size_t)t * s.Ne + q.e] : -2.0f;
      eid[j] = q.valid ? q.e : (0x7ffffff0 + j);
    }
    int we;
    float wk;
    warp_topk<JC>(key, eid, s.Ke, lane, we, wk);
    if (lane < s.Ke) atomicAdd(&s_cl[we], 1);
  }
  // fixed-order reduction over the warps of the block, then one partial row per block
#pragma unroll
  for (int j = 0; j < J; ++j) {
    const int sl = lane + 32 * j;
    const int g = sl >> s.logP, i = sl & (s.P - 1);
    if (g < s.Ng && i < s.N) s_sum[warp][g * s.N + i] = accE[j];
  }
  if (lane < s.Ng) s_sum[warp][256 + lane] = accG;
  __syncthreads();
  for (int c = threadIdx.x; c < s.Ne + s.Ng; c += blockDim.x) {
    const int col = c < s.Ne ? c : 256 + (c - s.Ne);
    double v = 0.0;
    for (int w = 0; w < kStatsWarps; ++w) v += s_sum[w][col];
    partials[(size_t)blockIdx.x * s.NL + c] = v;     // columns: experts first, then groups
  }
  for (int i = threadIdx.x; i < s.Ne; i += blockDim.x) {
    if (s_cr[i]) atomicAdd(&cnt_routed[i], s_cr[i]);
    if (s_cl[i]) atomicAdd(&cnt_lit[i], s_cl[i]);
  }
  if (threadIdx.x < s.Ng && s_cg[threadIdx.x]) atomicAdd(&group_count[threadIdx.x], s_cg[threadIdx.x]);
}

struct LossParams {
  float alpha_g, alpha_e;
  int f_norm_by_T, fe_mode;
  float w_over_wmax[MOHGE_MAX_GROUPS];
};

__global__ void aux_finalize_kernel(RouterShape s, LossParams lp, int nblocks,
                                    const double* __restrict__ partials,
                                    const int32_t* __restrict__ group_count,
                                    const int32_t* __restrict__ cnt_routed,
                                    const int32_t* __restrict__ cnt_lit, float* __restrict__ group_psum,
                                    float* __restrict__ expert_psum, float* __restrict__ loss_out) {
  pdl_enter();
  __shared__ double s_tot[256 + MOHGE_MAX_GROUPS];
  // one warp per column: lane l adds the partial rows l, l + 32, ... in that order, then a
  // butterfly adds the 32 lane sums; the order is fixed, so the result is run-to-run identical
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  for (int c = warp; c < s.NL; c += nwarps) {
    double v = 0.0;
    for (int b = lane; b < nblocks; b += 32) v += partials[(size_t)b * s.NL + c];
    for (int m = 16; m > 0; m >>= 1) v += __shfl_xor_sync(kFull, v, m);
    if (lane == 0) {
      s_tot[c] = v;
      if (c < s.Ne) expert_psum[c] = (float)v;
      else group_psum[c - s.Ne] = (float)v;
    }
  }
  __syncthreads();
  if (warp == 0) {
    // losses: lane l adds the terms l, l + 32, ... in that order, then a butterfly (fixed order)
    const double T = (double)s.T;
    const double fn = lp.f_norm_by_T ? 1.0 / T : 1.0;
    double LG = 0.0, LE = 0.0;
    if (lane < s.Ng) {
      const double f = (double)s.Ng / s.Kg * group_count[lane] * fn;   // Eq. 8
      LG = lp.w_over_wmax[lane] * f * (s_tot[s.Ne + lane] / T);        // Eq. 7, 9
    }
    const int32_t* ce = lp.fe_mode == 0 ? cnt_lit : cnt_routed;
    for (int e = lane; e < s.Ne; e += 32) {
      const double f = (double)s.N / s.Ke * ce[e] * fn;                // Eq. 12
      LE += f * (s_tot[e] / T);                                        // Eq. 11, 13
    }
    for (int m = 16; m > 0; m >>= 1) {
      LG += __shfl_xor_sync(kFull, LG, m);
      LE += __shfl_xor_sync(kFull, LE, m);
    }
    if (lane == 0) {
      loss_out[0] = (float)(lp.alpha_g * LG);
      loss_out[1] = (float)(lp.alpha_e * LE);
    }
  }
}

// ---------------------------------------------------------------- router backward (element-wise)
struct BwdParams {
  float alpha_g, alpha_e, eps;
  int f_norm_by_T, with_aux;
  float w_over_wmax[MOHGE_MAX_GROUPS];
};

constexpr int kBwdWarps = 8;

template <int J, int JC>
__global__ void __launch_bounds__(kBwdWarps * 32)
router_bwd_kernel(RouterShape s, BwdParams bp, const float* __restrict__ dgate,
                  const float* __restrict__ gs, const float* __restrict__ esp,
                  const int32_t* __restrict__ group_idx, const int32_t* __restrict__ expert_idx,
                  const int32_t* __restrict__ group_count, const int32_t* __restrict__ expert_count,
                  float* __restrict__ dlogits, __nv_bfloat16* __restrict__ dl16, int dl16_pitch) {
  pdl_enter();
  __shared__ float s_dkey[kBwdWarps][256];
  __shared__ float s_dgs[kBwdWarps][MOHGE_MAX_GROUPS];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const float invT = 1.0f / (float)s.T;
  const float fn = bp.f_norm_by_T ? invT : 1.0f;
  const int warps_total = gridDim.x * kBwdWarps;
  for (int t = blockIdx.x * kBwdWarps + warp; t < s.T; t += warps_total) {
    for (int i = lane; i < 256; i += 32) s_dkey[warp][i] = 0.0f;
    const int myg = lane < s.Kg ? group_idx[(size_t)t * s.Kg + lane] : -1;
    const unsigned gmask = __reduce_or_sync(kFull, myg >= 0 ? (1u << myg) : 0u);
    // Eq. 6 backward: gate_k = key_k / sum key
    int ek = -1;
    float keyk = 0.0f, dgk = 0.0f;
    if (lane < s.Ke) {
      ek = expert_idx[(size_t)t * s.Ke + lane];
      keyk = esp[(size_t)t * s.Ne + ek] * gs[(size_t)t * s.Ng + ek / s.N];
      dgk = dgate[(size_t)t * s.Ke + lane];
    }
    float ssum = keyk;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) ssum += __shfl_xor_sync(kFull, ssum, off);
    float dot = lane < s.Ke ? dgk * (keyk / ssum) : 0.0f;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(kFull, dot, off);
    __syncwarp();
    if (lane < s.Ke) s_dkey[warp][ek] = (dgk - dot) / ssum;
    __syncwarp();
    // experts of unselected groups: ES' is the constant 0, so no gradient reaches their logits
#pragma unroll
    for (int j = 0; j < J; ++j) {
      const int sl = lane + 32 * j;
      const int g = sl >> s.logP, i = sl & (s.P - 1);
      if (g < s.Ng && i < s.N && !((gmask >> g) & 1u)) {
        dlogits[(size_t)t * s.NL + s.Ng + g * s.N + i] = 0.0f;
        if (dl16) dl16[(size_t)t * dl16_pitch + s.Ng + g * s.N + i] = __float2bfloat16(0.0f);
      }
    }
    if (lane < s.Ng) s_dgs[warp][lane] = 0.0f;
    __syncwarp();
    // Eq. 4, 3 backward on the lane's compact slots (selected groups)
#pragma unroll
    for (int j = 0; j < JC; ++j) {
      const CompactSlot q = compact_slot(s, gmask, lane + 32 * j);
      const bool valid = q.valid;
      const int e = q.e, g = q.g;
      const float ev = valid ? esp[(size_t)t * s.Ne + e] : 0.0f;
      const float gv = valid ? gs[(size_t)t * s.Ng + g] : 0.0f;
      const float dpp = valid ? s_dkey[warp][e] : 0.0f;
      float dgs = dpp * ev;                 // dGS_g = sum_i dES''_i ES'_i
      float desp = dpp * gv;                // dES'_i = dES''_i GS_g
      if (bp.with_aux) {
        // L_E: S_e = ES'_e / D, D = sum_j ES'_j + eps (selected groups only; ES' is the constant 0 elsewhere)
        const float fe = valid ? (float)s.N / s.Ke * (float)expert_count[e] * fn : 0.0f;
        float grp = ev, fes = fe * ev;
        for (int mask = 1; mask < s.P; mask <<= 1) {
          grp += __shfl_xor_sync(kFull, grp, mask);
          fes += __shfl_xor_sync(kFull, fes, mask);
        }
        const float Dn = grp + bp.eps;
        if (valid) desp += bp.alpha_e * invT * (fe / Dn - fes / (Dn * Dn));
      }
      float inner = ev * desp;
      for (int mask = 1; mask < s.P; mask <<= 1) {
        inner += __shfl_xor_sync(kFull, inner, mask);
        dgs += __shfl_xor_sync(kFull, dgs, mask);
      }
      if (valid) {
        const float dl = ev * (desp - inner);
        dlogits[(size_t)t * s.NL + s.Ng + e] = dl;
        if (dl16) dl16[(size_t)t * dl16_pitch + s.Ng + e] = __float2bfloat16(dl);
      }
      if (valid && q.i == 0) s_dgs[warp][g] = dgs;
    }
    __syncwarp();
    // Eq. 2 backward (+ L_G through Eq. 10)
    const float gv = lane < s.Ng ? gs[(size_t)t * s.Ng + lane] : 0.0f;
    float dG = lane < s.Ng ? s_dgs[warp][lane] : 0.0f;
    if (bp.with_aux) {
      const float cg = lane < s.Ng ? bp.w_over_wmax[lane] * ((float)s.Ng / s.Kg) *
                                         (float)group_count[lane] * fn
                                   : 0.0f;
      float Ss = gv, cs = cg * gv;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        Ss += __shfl_xor_sync(kFull, Ss, off);
        cs += __shfl_xor_sync(kFull, cs, off);
      }
      dG += bp.alpha_g * invT * (cg / Ss - cs / (Ss * Ss));
    }
    if (lane < s.Ng) {
      const float dl = dG * gv * (1.0f - gv);
      dlogits[(size_t)t * s.NL + lane] = dl;
      if (dl16) dl16[(size_t)t * dl16_pitch + lane] = __float2bfloat16(dl);
    }
    __syncwarp();
  }
}

RouterShape make_shape(const Dims& D) {
  RouterShape s;
  s.T = (int)D.T; s.Ng = D.Ng; s.N = D.N; s.P = D.P; s.NL = D.NL; s.Ne = D.Ne; s.Kg = D.Kg; s.Ke = D.Ke;
  s.logP = 0;
  while ((1 << s.logP) < D.P) ++s.logP;
  return s;
}

int slots_per_lane(const Dims& D) {
  const int slots = D.Ng * D.P;
  int J = 1;
  while (J * 32 < slots) J *= 2;
  return J;
}
int compact_slots_per_lane(const Dims& D) {     // K_g selected groups of P slots each
  const int slots = D.Kg * D.P;
  int J = 1;
  while (J * 32 < slots) J *= 2;
  return J;
}

}  // namespace

// JJ = registers per lane of the full slot layout, JC = of the compact one (JC <= JJ)
#define MOHGE_DISPATCH_JC(JJ_, JC_, ...)                   \
  switch (JC_) {                                           \
    case 1: { constexpr int JJ = JJ_, JC = 1; __VA_ARGS__; } break; \
    case 2: { constexpr int JJ = JJ_, JC = JJ_ < 2 ? JJ_ : 2; __VA_ARGS__; } break; \
    case 4: { constexpr int JJ = JJ_, JC = JJ_ < 4 ? JJ_ : 4; __VA_ARGS__; } break; \
    default: { constexpr int JJ = JJ_, JC = JJ_; __VA_ARGS__; } break; \
  }
#define MOHGE_DISPATCH_J(D_, ...)                                          \
  switch (slots_per_lane(D_)) {                                            \
    case 1: MOHGE_DISPATCH_JC(1, compact_slots_per_lane(D_), __VA_ARGS__); break; \
    case 2: MOHGE_DISPATCH_JC(2, compact_slots_per_lane(D_), __VA_ARGS__); break; \
    case 4: MOHGE_DISPATCH_JC(4, compact_slots_per_lane(D_), __VA_ARGS__); break; \
    default: MOHGE_DISPATCH_JC(8, compact_slots_per_lane(D_), __VA_ARGS__); break; \
  }

int32_t launch_router_select(const Dims& D, const float* logits, int32_t* group_idx,
                             int32_t* expert_idx, float* gate_w, float* gs, float* esp,
                             int32_t* status, cudaStream_t st) {
  if (D.T == 0) return MOHGE_OK;
  const RouterShape s = make_shape(D);
  const int blocks = (int)((D.T + 7) / 8) < 148 * 8 ? (int)((D.T + 7) / 8) : 148 * 8;
  MOHGE_DISPATCH_J(D, (launch_dep(router_select_kernel<JJ, JC>, dim3(blocks), dim3(256), st,
                                          s, logits, group_idx, expert_idx, gate_w, gs, esp, status)));
  MOHGE_LAUNCH_CHECK("router_select_kernel");
  return MOHGE_OK;
}

int32_t launch_aux_stats(const Dims& D, const mohge_config& cfg, const float* gs, const float* esp,
                         const int32_t* group_idx, const int32_t* expert_idx, int32_t* group_count,
                         float* group_psum, int32_t* cnt_routed, int32_t* cnt_lit,
                         float* expert_psum, float* loss_out, double* partials, cudaStream_t st) {
  const RouterShape s = make_shape(D);
  launch_dep(zero_counts_kernel, dim3(1), dim3(256), st, group_count, D.Ng, cnt_routed, cnt_lit, D.Ne);
  MOHGE_LAUNCH_CHECK("zero_counts_kernel");
  int blocks = ceil_div(D.T, kStatsWarps);
  if (blocks > kStatsBlocks) blocks = kStatsBlocks;
  if (blocks > 0) {
    MOHGE_DISPATCH_J(D,
                     (launch_dep(aux_stats_kernel<JJ, JC>, dim3(blocks), dim3(kStatsThreads), st,
                         s, cfg.eps, gs, esp, group_idx, expert_idx, group_count, cnt_routed,
                         cnt_lit, partials)));
    MOHGE_LAUNCH_CHECK("aux_stats_kernel");
  }
  LossParams lp;
  lp.alpha_g = cfg.alpha_g; lp.alpha_e = cfg.alpha_e;
  lp.f_norm_by_T = cfg.f_norm_by_T; lp.fe_mode = cfg.fe_mode;
  for (int g = 0; g < MOHGE_MAX_GROUPS; ++g)
    lp.w_over_wmax[g] = g < D.Ng ? (float)D.W[g] / (float)D.Wmax : 0.0f;
  RouterShape s1 = s;
  if (s1.T == 0) s1.T = 1;   // empty batch: sums are zero, avoid 0/0 in the loss
  launch_dep(aux_finalize_kernel, dim3(1), dim3(1024), st, s1, lp, blocks, partials, group_count, cnt_routed, cnt_lit,
                                         group_psum, expert_psum, loss_out);
  MOHGE_LAUNCH_CHECK("aux_finalize_kernel");
  return MOHGE_OK;
}

int32_t launch_router_bwd_elementwise(const Dims& D, const mohge_config& cfg, const float* dgate,
                                      const float*, const float* gs, const float* esp,
                                      const int32_t* group_idx, const int32_t* expert_idx,
                                      const int32_t* group_count, const int32_t* expert_count,
                                      float* dlogits, __nv_bfloat16* dl16, int dl16_pitch,
                                      cudaStream_t st) {
  if (D.T == 0) return MOHGE_OK;
  const RouterShape s = make_shape(D);
  BwdParams bp;
  bp.alpha_g = cfg.alpha_g; bp.alpha_e = cfg.alpha_e; bp.eps = cfg.eps;
  bp.f_norm_by_T = cfg.f_norm_by_T;
  bp.with_aux = (group_count != nullptr && expert_count != nullptr) ? 1 : 0;
  for (int g = 0; g < MOHGE_MAX_GROUPS; ++g)
    bp.w_over_wmax[g] = g < D.Ng ? (float)D.W[g] / (float)D.Wmax : 0.0f;
  int blocks = ceil_div(D.T, kBwdWarps);
  if (blocks > 148 * 8) blocks = 148 * 8;
  MOHGE_DISPATCH_J(D,
                   (launch_dep(router_bwd_kernel<JJ, JC>, dim3(blocks), dim3(kBwdWarps * 32), st,
                       s, bp, dgate, gs, esp, group_idx, expert_idx, group_count, expert_count,
                       dlogits, dl16, dl16_pitch)));
  MOHGE_LAUNCH_CHECK("router_bwd_kernel");
  return MOHGE_OK;
}

}  // namespace mohge

// ---------------------------------------------------------------- allocation-free statistics
//
// mohge_aux_stats_static is mohge_aux_stats for callers that cannot hand over a workspace
// because they cannot allocate one at that point: code that runs after an inference server or a
// training framework has claimed all device memory for its own pool, or inside a latency-critical
// loop where cudaMalloc's implicit device-wide synchronisation is unacceptable.  The per-block
// partial sums live in the file-scope device array below instead.  Consequences, all documented
// in the header: the array (kStatsBlocks x MOHGE_STATIC_MAX_LOGITS doubles, about 315 KiB) is
// part of the library image on every GPU that loads it until the process exits; all calls on one
// device share it, so two calls that overlap on the GPU race; nothing in it needs to start at
// zero because every partial row that the final reduction reads is rewritten by the same call.
namespace mohge {
namespace {
static __device__ __align__(256) double g_static_partials[kStatsBlocks * MOHGE_STATIC_MAX_LOGITS];
double* g_static_ptr[kMaxDevices] = {nullptr};
}  // namespace
}  // namespace mohge

extern "C" int32_t mohge_aux_stats_static(const mohge_config* cfg, int64_t T, const float* gs_saved,
                                          const float* esp_saved, const int32_t* group_idx,
                                          const int32_t* expert_idx, int32_t* group_count,
                                          float* group_psum, int32_t* expert_count_routed,
                                          int32_t* expert_count_lit, float* expert_psum,
                                          float* loss_out, void* stream) {
  using namespace mohge;
  Dims D;
  const int32_t rc = make_dims(cfg, T, &D);
  if (rc) return rc;
  MOHGE_CHECK_ARG(gs_saved && esp_saved && group_idx && expert_idx && group_count && group_psum &&
                      expert_count_routed && expert_count_lit && expert_psum && loss_out,
                  "mohge_aux_stats_static: every pointer argument must be non-NULL");
  MOHGE_CHECK_ARG(D.NL <= MOHGE_STATIC_MAX_LOGITS,
                  "mohge_aux_stats_static: N_g + N_e = %d router outputs exceed the %d that the built-in "
                  "scratch array holds; use mohge_aux_stats with a caller workspace instead",
                  D.NL, MOHGE_STATIC_MAX_LOGITS);
  int dev = 0;
  MOHGE_CUDA(cudaGetDevice(&dev));
  MOHGE_CHECK_ARG(dev >= 0 && dev < kMaxDevices, "device ordinal %d not supported", dev);
  if (g_static_ptr[dev] == nullptr) {
    // The symbol's name is only a host-side handle; the kernel needs the device address, which
    // is looked up once per device with that device current.
    double* p = nullptr;
    MOHGE_CUDA(cudaGetSymbolAddress((void**)&p, g_static_partials));
    g_static_ptr[dev] = p;
  }
  return launch_aux_stats(D, *cfg, gs_saved, esp_saved, group_idx, expert_idx, group_count,
                          group_psum, expert_count_routed, expert_count_lit, expert_psum, loss_out,
                          g_static_ptr[dev], (cudaStream_t)stream);
}
