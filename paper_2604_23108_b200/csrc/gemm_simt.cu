// Device-side tile scheduler shared by both GEMM paths, and the plain-ALU (FFMA) grouped GEMM
// used by the FP32 layer dtype (TF32 tensor cores would miss the 1e-5 accuracy bar) and as an
// on-GPU cross-check of the tensor-core path.
//
// Tile scheduler: the ragged problem (rows per expert differ, widths differ per group) is cut
// into equal-area output tiles on the device, from aligned_offsets, with no host round trip.
// Experts are ordered by cost per tile, heaviest first (longest-processing-time order), and the
// persistent CTAs walk the list with a fixed stride, so every CTA receives an interleaved sample
// of the sorted costs and the totals differ by at most about one tile.

#include <string.h>

#include "common.cuh"

namespace mohge {

namespace {

#ifndef MOHGE_BAND_TILES
#define MOHGE_BAND_TILES 8
#endif
constexpr int kBandTiles = MOHGE_BAND_TILES;

__device__ __forceinline__ void
build_tiles_body(const TilePlan& p, const int32_t* __restrict__ aligned, int32_t* __restrict__ tile_count,
                 Tile* __restrict__ tiles, long long cap, int32_t* status) {
  __shared__ int s_nt[256], s_mt[256], s_order[256], s_start[257];
  __shared__ long long s_cost[256];
  const int e = threadIdx.x;
  const bool wgrad = p.role >= ROLE_WGRAD_DOWN;
  int rows = 0, g = 0;
  if (e < p.Ne) {
    g = e / p.N;
    rows = aligned[e + 1] - aligned[e];
    int mt, nt = (p.Next[g] + p.BN[g] - 1) / p.BN[g];
    long long cost;
    if (wgrad) {
      mt = rows > 0 ? (p.Mext[g] + p.BM - 1) / p.BM : 0;
      cost = (long long)rows * p.BN[g];
    } else {
      mt = (rows + p.BM - 1) / p.BM;
      cost = (long long)p.Kcost[g] * p.BN[g];
    }
    // with wide entries, n-tiles are taken two at a time (plus a single one when nt is odd)
    const int ne = p.wide ? nt / 2 + (nt & 1) : nt;
    s_mt[e] = mt;
    s_nt[e] = mt * ne;
    s_cost[e] = s_nt[e] > 0 ? cost : -1;
  }
  __syncthreads();
  if (e < p.Ne) {
    int rank = 0;
    for (int o = 0; o < p.Ne; ++o)
      rank += (s_cost[o] > s_cost[e]) || (s_cost[o] == s_cost[e] && o < e);
    s_order[rank] = e;
  }
  __syncthreads();
  if (threadIdx.x < 32) {
    // first tile of every rank (exclusive prefix sum over the sorted experts) and the range of
    // the costs per tile, by one warp: 32 ranks per round, a shuffle scan inside the round
    const int lane = threadIdx.x;
    int run = 0;
    long long lo = -1, hi = -1;
    for (int base = 0; base < p.Ne; base += 32) {
      const int r = base + lane;
      const int v = r < p.Ne ? s_nt[s_order[r]] : 0;
      int inc = v;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, inc, off);
        if (lane >= off) inc += up;
      }
      if (r < p.Ne) s_start[r] = run + inc - v;
      run += __shfl_sync(0xffffffffu, inc, 31);
      const long long c = r < p.Ne ? s_cost[r] : -1;
      if (c > 0) {
        if (lo < 0 || c < lo) lo = c;
        if (c > hi) hi = c;
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const long long olo = __shfl_xor_sync(0xffffffffu, lo, off);
      const long long ohi = __shfl_xor_sync(0xffffffffu, hi, off);
      if (olo > 0 && (lo < 0 || olo < lo)) lo = olo;
      if (ohi > hi) hi = ohi;
    }
    if (lane == 0) {
      s_start[p.Ne] = run;
      if (run > cap) {
        if (blockIdx.x == 0) atomicCAS(status, 0, (2 << 24) | 2);
        s_start[p.Ne] = 0;
      }
      if (blockIdx.x == 0) {
        tile_count[0] = s_start[p.Ne];
        // tile_count[1]: 1 when the costs per tile differ by more than a quarter between experts
        // (skewed routing, or groups of different contraction length): the persistent CTAs then
        // walk the sorted list in alternating directions
        tile_count[1] = (lo > 0 && hi * 4 > lo * 5) ? 1 : 0;
      }
    }
  }
  __syncthreads();
  // every block has built the same per-expert table; the entries are written grid-strided
  const int total = s_start[p.Ne];
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
    int lo = 0, hi = p.Ne - 1;              // last rank whose start <= i
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (s_start[mid] <= i) lo = mid; else hi = mid - 1;
    }
    const int ex = s_order[lo];
    const int gg = ex / p.N;
    const int local = i - s_start[lo];
    // Order inside an expert: bands of kBandTiles m-tiles; inside a band m runs fastest, then n.
    // The CTAs of a wave then work on a near-square block of the output, so the A rows and the
    // B rows they share are both few enough to stay in L2 while the wave needs them (a full
    // column of m-tiles of a large expert would have to survive several waves to be reused).
    const int mt = s_mt[ex];
    const int nt = s_nt[ex] / mt;
    const int band = local / (kBandTiles * nt);
    const int in_band = local - band * kBandTiles * nt;
    const int band_m = mt - band * kBandTiles < kBandTiles ? mt - band * kBandTiles : kBandTiles;
    const int tm = band * kBandTiles + in_band % band_m, tn = in_band / band_m;
    Tile t;
    t.e = ex;
    if (p.wide) {
      const int nt_full = (p.Next[gg] + p.BN[gg] - 1) / p.BN[gg];
      t.n0 = tn < nt_full / 2 ? (2 * tn * p.BN[gg]) | kTileWide : (nt_full - 1) * p.BN[gg];
    } else {
      t.n0 = tn * p.BN[gg];
    }
    if (wgrad) {
      t.m0 = tm * p.BM;
      t.ext = aligned[ex + 1] - aligned[ex];
    } else {
      t.m0 = aligned[ex] + tm * p.BM;
      const int left = aligned[ex + 1] - t.m0;
      t.ext = left < p.BM ? left : p.BM;
    }
    tiles[i] = t;
  }
}

__global__ void __launch_bounds__(256)
build_tiles_kernel(TilePlan p, const int32_t* __restrict__ aligned, int32_t* __restrict__ tile_count,
                   Tile* __restrict__ tiles, long long cap, int32_t* status) {
  pdl_enter();
  build_tiles_body(p, aligned, tile_count, tiles, cap, status);
}

// Several lists with one launch: blockIdx.y picks the plan; list i keeps its count at
// tile_count + 64 * i and its entries at tiles + i * cap.
struct MultiPlan {
  TilePlan p[kMaxLists];
};
__global__ void __launch_bounds__(256)
build_tiles_multi_kernel(MultiPlan mp, const int32_t* __restrict__ aligned, int32_t* __restrict__ tile_count,
                         Tile* __restrict__ tiles, long long cap, int32_t* status) {
  pdl_enter();
  const int i = blockIdx.y;
  build_tiles_body(mp.p[i], aligned, tile_count + 64 * i, tiles + (size_t)cap * i, cap, status);
}

// ---------------------------------------------------------------- FFMA tile core
constexpr int SBM = 64, SBN = 64, SBK = 16;

__device__ __forceinline__ float ld_any(const void* p, bool f32, long long idx) {
  return f32 ? reinterpret_cast<const float*>(p)[idx]
             : __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[idx]);
}

// acc[i][j] += sum_k A(m0+ty*4+i, k) * B(n0+tx*4+j, k),  A(m,k) = A[m*sAm + k*sAk], same for B
__device__ __forceinline__ void simt_tile(const void* A, bool a32, long long sAm, long long sAk,
                                          const void* B, bool b32, long long sBn, long long sBk,
                                          int M, int N, int K, float (&acc)[4][4]) {
  __shared__ float As[SBK][SBM + 4];
  __shared__ float Bs[SBK][SBN + 4];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  for (int k0 = 0; k0 < K; k0 += SBK) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int idx = tid + i * 256;
      int m, k;
      if (sAk == 1) { m = idx >> 4; k = idx & 15; } else { m = idx & 63; k = idx >> 6; }
      As[k][m] = (m < M && k0 + k < K) ? ld_any(A, a32, m * sAm + (k0 + k) * sAk) : 0.0f;
      int n, kb;
      if (sBk == 1) { n = idx >> 4; kb = idx & 15; } else { n = idx & 63; kb = idx >> 6; }
      Bs[kb][n] = (n < N && k0 + kb < K) ? ld_any(B, b32, n * sBn + (k0 + kb) * sBk) : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < SBK; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
}

__device__ __forceinline__ void st_any(void* p, bool f32, long long idx, float v, bool accumulate) {
  if (f32) {
    float* q = reinterpret_cast<float*>(p) + idx;
    *q = accumulate ? *q + v : v;
  } else {
    __nv_bfloat16* q = reinterpret_cast<__nv_bfloat16*>(p) + idx;
    *q = __float2bfloat16(accumulate ? __bfloat162float(*q) + v : v);
  }
}

struct SimtArgs {
  int role, f32, accumulate;
  GroupShape gs;
  GroupPtrs gp;
  const void* A;   // activation operand (see table in launch_simt_grouped)
  const void* B;   // second activation operand (wgrad only)
  void* C;         // activation output (row-tiled roles)
};

__global__ void __launch_bounds__(256)
simt_grouped_kernel(SimtArgs a, const int32_t* __restrict__ aligned,
                    const int32_t* __restrict__ tile_count, const Tile* __restrict__ tiles) {
  pdl_enter();
  const int total = *tile_count;
  const bool f32 = a.f32;
  const long long d = a.gs.d, pitchAU = 2LL * a.gs.Wmax, pitchH = a.gs.Wmax;
  const size_t es = f32 ? 4 : 2;
  for (int ti = blockIdx.x; ti < total; ti += gridDim.x) {
    const Tile t = tiles[ti];
    const int g = t.e / a.gs.N, i = t.e % a.gs.N;
    const long long W = a.gs.W[g];
    const char* A = nullptr;
    const char* B = nullptr;
    char* C = nullptr;
    long long sAm = 0, sAk = 1, sBn = 0, sBk = 1, sCm = 0;
    int M = 0, N = 0, K = 0;
    bool c32 = f32;
    switch (a.role) {
      case ROLE_FWD1:
        A = (const char*)a.A + (size_t)t.m0 * d * es; sAm = d; M = t.ext; K = (int)d;
        B = (const char*)a.gp.w13[g] + ((size_t)i * 2 * W + t.n0) * d * es; sBn = d; N = (int)(2 * W) - t.n0;
        C = (char*)a.C + ((size_t)t.m0 * pitchAU + t.n0) * es; sCm = pitchAU;
        break;
      case ROLE_FWD2:
        A = (const char*)a.A + (size_t)t.m0 * pitchH * es; sAm = pitchH; M = t.ext; K = (int)W;
        B = (const char*)a.gp.w2[g] + ((size_t)i * d + t.n0) * W * es; sBn = W; N = (int)d - t.n0;
        C = (char*)a.C + ((size_t)t.m0 * d + t.n0) * es; sCm = d;
        break;
      case ROLE_DGRAD_DOWN:
        A = (const char*)a.A + (size_t)t.m0 * d * es; sAm = d; M = t.ext; K = (int)d;
        B = (const char*)a.gp.w2[g] + ((size_t)i * d * W + t.n0) * es; sBn = 1; sBk = W; N = (int)W - t.n0;
        C = (char*)a.C + ((size_t)t.m0 * pitchAU + t.n0) * es; sCm = pitchAU;
        break;
      case ROLE_DGRAD_13:
        A = (const char*)a.A + (size_t)t.m0 * pitchAU * es; sAm = pitchAU; M = t.ext; K = (int)(2 * W);
        B = (const char*)a.gp.w13[g] + ((size_t)i * 2 * W * d + t.n0) * es; sBn = 1; sBk = d; N = (int)d - t.n0;
        C = (char*)a.C + ((size_t)t.m0 * d + t.n0) * es; sCm = d;
        break;
      case ROLE_WGRAD_DOWN: {
        const size_t r0 = aligned[t.e];
        A = (const char*)a.A + (r0 * d + t.m0) * es; sAm = 1; sAk = d; M = (int)d - t.m0; K = t.ext;
        B = (const char*)a.B + (r0 * pitchH + t.n0) * es; sBn = 1; sBk = pitchH; N = (int)W - t.n0;
        C = (char*)(a.gp.dw2[g] + ((size_t)i * d + t.m0) * W + t.n0); sCm = W; c32 = true;
      } break;
      default: {  // ROLE_WGRAD_13
        const size_t r0 = aligned[t.e];
        A = (const char*)a.A + (r0 * pitchAU + t.m0) * es; sAm = 1; sAk = pitchAU; M = (int)(2 * W) - t.m0; K = t.ext;
        B = (const char*)a.B + (r0 * d + t.n0) * es; sBn = 1; sBk = d; N = (int)d - t.n0;
        C = (char*)(a.gp.dw13[g] + ((size_t)i * 2 * W + t.m0) * d + t.n0); sCm = d; c32 = true;
      } break;
    }
    if (M > SBM) M = SBM;
    if (N > SBN) N = SBN;
    float acc[4][4];
#pragma unroll
    for (int ii = 0; ii < 4; ++ii)
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) acc[ii][jj] = 0.0f;
    simt_tile(A, f32, sAm, sAk, B, f32, sBn, sBk, M, N, K, acc);
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const bool accum = a.accumulate && a.role >= ROLE_WGRAD_DOWN;
#pragma unroll
    for (int ii = 0; ii < 4; ++ii)
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        const int m = ty * 4 + ii, n = tx * 4 + jj;
        if (m < M && n < N) st_any(C, c32, m * sCm + n, acc[ii][jj], accum);
      }
  }
}

__global__ void __launch_bounds__(256)
simt_plain_kernel(int M, int N, int K, const void* A, int a32, long long sAm, long long sAk,
                  const void* B, int b32, long long sBn, long long sBk, void* C, int c32,
                  long long sCm, const float* __restrict__ bias, int accumulate) {
  pdl_enter();
  const int m0 = blockIdx.y * SBM, n0 = blockIdx.x * SBN;
  const size_t ea = a32 ? 4 : 2, eb = b32 ? 4 : 2;
  float acc[4][4];
#pragma unroll
  for (int ii = 0; ii < 4; ++ii)
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) acc[ii][jj] = 0.0f;
  const int Mt = M - m0 < SBM ? M - m0 : SBM, Nt = N - n0 < SBN ? N - n0 : SBN;
  simt_tile((const char*)A + (size_t)m0 * sAm * ea, a32, sAm, sAk,
            (const char*)B + (size_t)n0 * sBn * eb, b32, sBn, sBk, Mt, Nt, K, acc);
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
  for (int ii = 0; ii < 4; ++ii)
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      const int m = ty * 4 + ii, n = tx * 4 + jj;
      if (m < Mt && n < Nt) {
        const float v = acc[ii][jj] + (bias ? bias[n0 + n] : 0.0f);
        st_any(C, c32, (long long)(m0 + m) * sCm + n0 + n, v, accumulate);
      }
    }
}

// ---------------------------------------------------------------- SwiGLU element-wise (FFMA path)
template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16(v); }

// H = silu(A) * U over the rows of expert blockIdx.x
template <typename T>
__global__ void __launch_bounds__(256)
swiglu_fwd_kernel(GroupShape gs, const int32_t* __restrict__ aligned, const T* __restrict__ au,
                  T* __restrict__ h) {
  pdl_enter();
  const int e = blockIdx.x, W = gs.W[e / gs.N];
  const long long r0 = aligned[e], n = (long long)(aligned[e + 1] - aligned[e]) * W;
  for (long long i = (long long)blockIdx.y * blockDim.x + threadIdx.x; i < n;
       i += (long long)gridDim.y * blockDim.x) {
    const long long r = r0 + i / W, c = i % W;
    const float a = to_f(au[r * 2 * gs.Wmax + c]), u = to_f(au[r * 2 * gs.Wmax + W + c]);
    h[r * gs.Wmax + c] = from_f<T>(a / (1.0f + expf(-a)) * u);
  }
}

// in place: dau[:, c] holds dH on entry; writes dA to [:, c] and dU to [:, W + c]
template <typename T>
__global__ void __launch_bounds__(256)
swiglu_bwd_kernel(GroupShape gs, const int32_t* __restrict__ aligned, const T* __restrict__ au,
                  T* __restrict__ dau) {
  pdl_enter();
  const int e = blockIdx.x, W = gs.W[e / gs.N];
  const long long r0 = aligned[e], n = (long long)(aligned[e + 1] - aligned[e]) * W;
  for (long long i = (long long)blockIdx.y * blockDim.x + threadIdx.x; i < n;
       i += (long long)gridDim.y * blockDim.x) {
    const long long r = r0 + i / W, c = i % W;
    const long long o = r * 2 * gs.Wmax + c;
    const float a = to_f(au[o]), u = to_f(au[o + W]), dh = to_f(dau[o]);
    const float sg = 1.0f / (1.0f + expf(-a));
    dau[o] = from_f<T>(dh * u * sg * (1.0f + a * (1.0f - sg)));
    dau[o + W] = from_f<T>(dh * a * sg);
  }
}

// experts without tokens: their weight gradients are exactly zero
__global__ void __launch_bounds__(256)
zero_empty_wgrad_kernel(GroupShape gs, GroupPtrs gp, const int32_t* __restrict__ counts) {
  pdl_enter();
  const int e = blockIdx.x;
  if (counts[e] != 0) return;
  const int g = e / gs.N, i = e % gs.N;
  const size_t n13 = (size_t)2 * gs.W[g] * gs.d, n2 = (size_t)gs.d * gs.W[g];
  float* p13 = gp.dw13[g] + (size_t)i * n13;
  float* p2 = gp.dw2[g] + (size_t)i * n2;
  for (size_t k = (size_t)blockIdx.y * blockDim.x + threadIdx.x; k < n13; k += (size_t)gridDim.y * blockDim.x) p13[k] = 0.0f;
  for (size_t k = (size_t)blockIdx.y * blockDim.x + threadIdx.x; k < n2; k += (size_t)gridDim.y * blockDim.x) p2[k] = 0.0f;
}

}  // namespace

GroupShape make_group_shape(const Dims& D) {
  GroupShape gs;
  for (int g = 0; g < MOHGE_MAX_GROUPS; ++g) gs.W[g] = g < D.Ng ? D.W[g] : 0;
  gs.Ng = D.Ng; gs.N = D.N; gs.d = D.d; gs.Wmax = D.Wmax;
  return gs;
}

int32_t launch_build_tiles_multi(const TilePlan* plans, int nplans, const int32_t* aligned,
                                 int32_t* tile_count, Tile* tiles, int64_t tiles_cap,
                                 int32_t* status, cudaStream_t st) {
  MultiPlan mp;
  memset(&mp, 0, sizeof(mp));
  for (int i = 0; i < nplans && i < kMaxLists; ++i) mp.p[i] = plans[i];
  launch_dep(build_tiles_multi_kernel, dim3(32, nplans), dim3(256), st, mp, aligned, tile_count, tiles,
                                                           (long long)tiles_cap, status);
  MOHGE_LAUNCH_CHECK("build_tiles_multi_kernel");
  return MOHGE_OK;
}

int32_t launch_build_tiles_plan(const TilePlan& p, const int32_t* aligned, int32_t* tile_count,
                                Tile* tiles, int64_t tiles_cap, int32_t* status, cudaStream_t st) {
  launch_dep(build_tiles_kernel, dim3(32), dim3(256), st, p, aligned, tile_count, tiles, (long long)tiles_cap, status);
  MOHGE_LAUNCH_CHECK("build_tiles_kernel");
  return MOHGE_OK;
}

// Row-tiled roles: output [rows, Next]; wgrad roles: output [Mext, Next] per expert.
TilePlan make_plan(const Dims& D, int role, int BM, const int* BN /*per group*/, bool fused_swiglu) {
  TilePlan p;
  p.role = role; p.BM = BM; p.Ng = D.Ng; p.N = D.N; p.Ne = D.Ne; p.d = D.d; p.wide = 0;
  for (int g = 0; g < MOHGE_MAX_GROUPS; ++g) {
    const int W = g < D.Ng ? D.W[g] : 0;
    p.BN[g] = BN[g];
    p.Mext[g] = 0;
    switch (role) {
      case ROLE_FWD1: p.Next[g] = fused_swiglu ? W : 2 * W; p.Kcost[g] = D.d * (fused_swiglu ? 2 : 1); break;
      case ROLE_FWD2: p.Next[g] = D.d; p.Kcost[g] = W; break;
      case ROLE_DGRAD_DOWN: p.Next[g] = W; p.Kcost[g] = D.d; break;
      case ROLE_DGRAD_13: p.Next[g] = D.d; p.Kcost[g] = 2 * W; break;
      case ROLE_WGRAD_DOWN: p.Mext[g] = D.d; p.Next[g] = W; p.Kcost[g] = 0; break;
      default: p.Mext[g] = 2 * W; p.Next[g] = D.d; p.Kcost[g] = 0; break;
    }
    if (g >= D.Ng) { p.Next[g] = 0; p.BN[g] = 1; }
  }
  return p;
}

int32_t launch_build_tiles(const Dims& D, int role, int BM, int BN, const int32_t* /*counts*/,
                           const int32_t* aligned, int32_t* tile_count, Tile* tiles,
                           int64_t tiles_cap, int32_t* status, cudaStream_t st) {
  int bn[MOHGE_MAX_GROUPS];
  for (int g = 0; g < MOHGE_MAX_GROUPS; ++g) bn[g] = BN;
  return launch_build_tiles_plan(make_plan(D, role, BM, bn, false), aligned, tile_count, tiles,
                                 tiles_cap, status, st);
}

// Operands per role (activation buffers; weights come from GroupPtrs):
//   FWD1        A = x_perm            C = au        |  DGRAD_DOWN  A = dy_perm   C = dau (dH in cols [0,W))
//   FWD2        A = h                 C = y_perm    |  DGRAD_13    A = dau       C = dx_perm
//   WGRAD_DOWN  A = dy_perm, B = h    -> dw2        |  WGRAD_13    A = dau, B = x_perm -> dw13
int32_t launch_simt_grouped(const Dims& D, int role, const GroupPtrs& P, const void* A,
                            const void* B, void* C, const int32_t* aligned, int accumulate,
                            const int32_t* tile_count, const Tile* tiles, cudaStream_t st) {
  SimtArgs a;
  a.role = role; a.f32 = D.bf16 ? 0 : 1; a.accumulate = accumulate;
  a.gs = make_group_shape(D); a.gp = P; a.A = A; a.B = B; a.C = C;
  launch_dep(simt_grouped_kernel, dim3(148 * 4), dim3(256), st, a, aligned, tile_count, tiles);
  MOHGE_LAUNCH_CHECK("simt_grouped_kernel");
  return MOHGE_OK;
}

int32_t launch_swiglu_fwd(const Dims& D, const int32_t* aligned, void* au, void* h, cudaStream_t st) {
  const GroupShape gs = make_group_shape(D);
  if (D.bf16)
    launch_dep(swiglu_fwd_kernel<__nv_bfloat16>, dim3(D.Ne, 32), dim3(256), st, gs, aligned, (const __nv_bfloat16*)au, (__nv_bfloat16*)h);
  else
    launch_dep(swiglu_fwd_kernel<float>, dim3(D.Ne, 32), dim3(256), st, gs, aligned, (const float*)au, (float*)h);
  MOHGE_LAUNCH_CHECK("swiglu_fwd_kernel");
  return MOHGE_OK;
}

int32_t launch_swiglu_bwd(const Dims& D, const int32_t* aligned, const void* au, void* dau, cudaStream_t st) {
  const GroupShape gs = make_group_shape(D);
  if (D.bf16)
    launch_dep(swiglu_bwd_kernel<__nv_bfloat16>, dim3(D.Ne, 32), dim3(256), st, gs, aligned, (const __nv_bfloat16*)au, (__nv_bfloat16*)dau);
  else
    launch_dep(swiglu_bwd_kernel<float>, dim3(D.Ne, 32), dim3(256), st, gs, aligned, (const float*)au, (float*)dau);
  MOHGE_LAUNCH_CHECK("swiglu_bwd_kernel");
  return MOHGE_OK;
}

int32_t launch_zero_empty_wgrad(const Dims& D, const GroupPtrs& P, const int32_t* counts, cudaStream_t st) {
  launch_dep(zero_empty_wgrad_kernel, dim3(D.Ne, 16), dim3(256), st, make_group_shape(D), P, counts);
  MOHGE_LAUNCH_CHECK("zero_empty_wgrad_kernel");
  return MOHGE_OK;
}

int32_t launch_simt_plain(int M, int N, int K, const void* A, int a_f32, int64_t sAm, int64_t sAk,
                          const void* B, int b_f32, int64_t sBn, int64_t sBk, void* C, int c_f32,
                          int64_t sCm, const float* bias, int accumulate, cudaStream_t st) {
  if (M == 0 || N == 0) return MOHGE_OK;
  dim3 grid((N + SBN - 1) / SBN, (M + SBM - 1) / SBM);
  launch_dep(simt_plain_kernel, dim3(grid), dim3(256), st, M, N, K, A, a_f32, sAm, sAk, B, b_f32, sBn, sBk, C, c_f32,
                                          sCm, bias, accumulate);
  MOHGE_LAUNCH_CHECK("simt_plain_kernel");
  return MOHGE_OK;
}

}  // namespace mohge
