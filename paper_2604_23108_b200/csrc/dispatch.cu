// Token permutation (stable counting sort by expert, then token), row gather, weighted combine
// and their backward kernels.  All HBM-bound: 16-byte vector accesses, one block per token row.
//
// Counting sort, deterministic and bit-exact:
//   pass 1  every block takes kDispatchChunk consecutive tokens and counts, per expert, how
//           many of them are routed to it (warp ballots, no atomics)
//   pass 2  one block scans the per-chunk counts per expert (chunk bases), the totals (counts)
//           and the exclusive prefix sums over experts (offsets, aligned_offsets)
//   pass 3  every block recomputes its ballots; the rank of token t for expert e is
//           chunk base + tokens of earlier warps + earlier lanes, i.e. ascending token order

#include "common.cuh"

namespace mohge {
namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr int kChunkWarps = kDispatchChunk / 32;

// bit e of the lane's 256-bit set <=> the lane's token is routed to expert e
struct ExpertSet {
  unsigned w[8];
};

__device__ __forceinline__ ExpertSet load_set(const int32_t* __restrict__ expert_idx, int t, int T,
                                              int Ke, int Ne, int32_t* status) {
  ExpertSet s;
#pragma unroll
  for (int i = 0; i < 8; ++i) s.w[i] = 0;
  if (t < T) {
    for (int k = 0; k < Ke; ++k) {
      const int e = expert_idx[(size_t)t * Ke + k];
      if (e < 0 || e >= Ne) {                // index check: record and skip
        atomicCAS(status, 0, (2 << 24) | 1);
        continue;
      }
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if ((e >> 5) == i) s.w[i] |= 1u << (e & 31);
    }
  }
  return s;
}

// per-warp counts of every expert -> s_wcnt[warp][e]
__device__ __forceinline__ void warp_counts(const ExpertSet& s, int Ne, int lane, int* wcnt) {
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    if (i * 32 < Ne) {
#pragma unroll 8
      for (int b = 0; b < 32; ++b) {
        const unsigned bal = __ballot_sync(kFull, (s.w[i] >> b) & 1u);
        if (lane == b) wcnt[i * 32 + b] = __popc(bal);
      }
    }
  }
}

__global__ void __launch_bounds__(kDispatchChunk)
dispatch_hist_kernel(const int32_t* __restrict__ expert_idx, int T, int Ke, int Ne,
                     int32_t* __restrict__ hist, int32_t* status) {
  pdl_enter();
  __shared__ int s_wcnt[kChunkWarps][256];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int t = blockIdx.x * kDispatchChunk + threadIdx.x;
  const ExpertSet s = load_set(expert_idx, t, T, Ke, Ne, status);
  warp_counts(s, Ne, lane, s_wcnt[warp]);
  __syncthreads();
  for (int e = threadIdx.x; e < Ne; e += blockDim.x) {
    int c = 0;
#pragma unroll
    for (int w = 0; w < kChunkWarps; ++w) c += s_wcnt[w][e];
    hist[(size_t)blockIdx.x * Ne + e] = c;
  }
}

__global__ void __launch_bounds__(256)
dispatch_scan_kernel(int chunks, int Ne, int align, const int32_t* __restrict__ hist,
                     int32_t* __restrict__ base, int32_t* __restrict__ counts,
                     int32_t* __restrict__ offsets, int32_t* __restrict__ aligned) {
  pdl_enter();
  __shared__ int s_cnt[256];
  const int e = threadIdx.x;
  if (e < Ne) {
    int run = 0;
    // sixteen counts are requested before the first is used: one dependent load per chunk kept
    // this single block at a memory round trip per chunk (22 us for 256 chunks)
    for (int b0 = 0; b0 < chunks; b0 += 16) {
      int h[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) h[j] = b0 + j < chunks ? hist[(size_t)(b0 + j) * Ne + e] : 0;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        if (b0 + j < chunks) base[(size_t)(b0 + j) * Ne + e] = run;
        run += h[j];
      }
    }
    counts[e] = run;
    s_cnt[e] = run;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int o = 0, a = 0;
    for (int i = 0; i < Ne; ++i) {
      offsets[i] = o;
      aligned[i] = a;
      o += s_cnt[i];
      a += (s_cnt[i] + align - 1) / align * align;
    }
    offsets[Ne] = o;
    aligned[Ne] = a;
  }
}

__global__ void __launch_bounds__(kDispatchChunk)
dispatch_scatter_kernel(const int32_t* __restrict__ expert_idx, int T, int Ke, int Ne,
                        const int32_t* __restrict__ base, const int32_t* __restrict__ offsets,
                        const int32_t* __restrict__ aligned, int32_t* __restrict__ row_of,
                        int32_t* __restrict__ prow_of, int32_t* __restrict__ src_of,
                        int32_t* status) {
  pdl_enter();
  __shared__ int s_wcnt[kChunkWarps][256];
  __shared__ int s_start[256];     // dense row of the chunk's first token for expert e
  __shared__ int s_pstart[256];    // same in physical numbering
  __shared__ unsigned s_set[kChunkWarps][32][8];   // expert set of every token of the chunk
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int t = blockIdx.x * kDispatchChunk + threadIdx.x;
  const ExpertSet s = load_set(expert_idx, t, T, Ke, Ne, status);
#pragma unroll
  for (int i = 0; i < 8; ++i) s_set[warp][lane][i] = s.w[i];
  warp_counts(s, Ne, lane, s_wcnt[warp]);
  __syncthreads();
  for (int e = threadIdx.x; e < Ne; e += blockDim.x) {
    int run = 0;                   // exclusive scan over the warps of the chunk
#pragma unroll
    for (int w = 0; w < kChunkWarps; ++w) {
      const int c = s_wcnt[w][e];
      s_wcnt[w][e] = run;
      run += c;
    }
    const int b = base[(size_t)blockIdx.x * Ne + e];
    s_start[e] = offsets[e] + b;
    s_pstart[e] = aligned[e] + b;
  }
  __syncthreads();
  // Rank inside the warp: the lanes below this one whose token is also routed to e (in any
  // slot) come first; their membership bits are read from the sets the warp left in shared
  // memory (lanes past T left empty sets).
  for (int k = 0; k < Ke; ++k) {
    int e = t < T ? expert_idx[(size_t)t * Ke + k] : -1;
    if (e >= Ne) e = -1;
    int below = 0;
    if (e >= 0) {
      const int wi = e >> 5, bi = e & 31;
#pragma unroll 8
      for (int l = 0; l < 31; ++l) below += l < lane ? (int)((s_set[warp][l][wi] >> bi) & 1u) : 0;
    }
    if (e >= 0) {
      const int rank = s_wcnt[warp][e] + below;
      const int row = s_start[e] + rank;
      row_of[(size_t)t * Ke + k] = row;
      prow_of[(size_t)t * Ke + k] = s_pstart[e] + rank;
      src_of[row] = t * Ke + k;
    } else if (t < T) {
      row_of[(size_t)t * Ke + k] = -1;         // not an expert: no row (also reported in status)
      prow_of[(size_t)t * Ke + k] = -1;
    }
  }
}

// ---------------------------------------------------------------- row movers
struct alignas(16) Vec16 {
  uint32_t v[4];
};

__device__ __forceinline__ void unpack(const Vec16& a, float (&f)[8], __nv_bfloat16) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(a.v[i] << 16);
    f[2 * i + 1] = __uint_as_float(a.v[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ Vec16 pack(const float (&f)[8], __nv_bfloat16) {
  Vec16 a;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
    a.v[i] = *reinterpret_cast<const uint32_t*>(&h);
  }
  return a;
}
__device__ __forceinline__ void unpack(const Vec16& a, float (&f)[8], float) {
#pragma unroll
  for (int i = 0; i < 4; ++i) f[i] = __uint_as_float(a.v[i]);
#pragma unroll
  for (int i = 4; i < 8; ++i) f[i] = 0.0f;
}
__device__ __forceinline__ Vec16 pack(const float (&f)[8], float) {
  Vec16 a;
#pragma unroll
  for (int i = 0; i < 4; ++i) a.v[i] = __float_as_uint(f[i]);
  return a;
}

// Zeroes a quarter (`part` of 4) of the padding rows [aligned[e] + counts[e], aligned[e+1]) of a
// permuted buffer.  The row movers run 4 * N_e extra blocks that do this, so no launch of its own.
__device__ __forceinline__ void zero_pad_part(const int32_t* __restrict__ counts,
                                              const int32_t* __restrict__ aligned, int e, int part,
                                              int row_vecs, Vec16* __restrict__ buf) {
  const int r0 = aligned[e] + counts[e], r1 = aligned[e + 1];
  const Vec16 z = {{0, 0, 0, 0}};
  const size_t n = (size_t)(r1 - r0) * row_vecs;
  Vec16* p = buf + (size_t)r0 * row_vecs;
  for (size_t i = (size_t)part * blockDim.x + threadIdx.x; i < n; i += (size_t)4 * blockDim.x) p[i] = z;
}

// Row stores of the write-dominated movers (K_e rows written per row read): streaming stores
// (evict-first in L2), measured 2 % faster than plain stores on the row gather at the large workload.
__device__ __forceinline__ void store_streaming(Vec16* dst, const Vec16& v) {
  __stcs(reinterpret_cast<int4*>(dst), *reinterpret_cast<const int4*>(&v));
}

// x_perm[prow_of[t,k], :] = x[t, :]   (row_vecs 16-byte vectors per row)
__global__ void __launch_bounds__(256)
permute_rows_kernel(const Vec16* __restrict__ x, const int32_t* __restrict__ prow_of, int T, int Ke,
                    int row_vecs, int rows_cap, Vec16* __restrict__ x_perm, int nb_tok,
                    const int32_t* __restrict__ counts, const int32_t* __restrict__ aligned) {
  pdl_enter();
  __shared__ int s_row[MOHGE_MAX_K_EXPERTS];
  if ((int)blockIdx.x >= nb_tok) {      // padding rows (launched only when segments are aligned)
    const int j = blockIdx.x - nb_tok;
    zero_pad_part(counts, aligned, j >> 2, j & 3, row_vecs, x_perm);
    return;
  }
  for (int t = blockIdx.x; t < T; t += nb_tok) {
    __syncthreads();
    if (threadIdx.x < Ke) s_row[threadIdx.x] = prow_of[(size_t)t * Ke + threadIdx.x];
    __syncthreads();
    for (int c = threadIdx.x; c < row_vecs; c += blockDim.x) {
      const Vec16 v = x[(size_t)t * row_vecs + c];
      for (int k = 0; k < Ke; ++k)
        if ((unsigned)s_row[k] < (unsigned)rows_cap) store_streaming(x_perm + (size_t)s_row[k] * row_vecs + c, v);
    }
  }
}

// zero the padding rows [aligned[e] + counts[e], aligned[e+1]) of a permuted buffer
__global__ void __launch_bounds__(256)
zero_pad_rows_kernel(const int32_t* __restrict__ counts, const int32_t* __restrict__ aligned,
                     int row_vecs, Vec16* __restrict__ buf) {
  pdl_enter();
  const int e = blockIdx.x;
  const int r0 = aligned[e] + counts[e], r1 = aligned[e + 1];
  const Vec16 z = {{0, 0, 0, 0}};
  const size_t n = (size_t)(r1 - r0) * row_vecs;
  Vec16* p = buf + (size_t)r0 * row_vecs;
  for (size_t i = (size_t)blockIdx.y * blockDim.x + threadIdx.x; i < n;
       i += (size_t)gridDim.y * blockDim.x)
    p[i] = z;
}

// y[t] = sum_k gate[t,k] * y_perm[prow[t,k]] (+ add[t])   (gate == nullptr: plain sum)
template <typename T>
__global__ void __launch_bounds__(256)
combine_kernel(const Vec16* __restrict__ y_perm, const int32_t* __restrict__ prow_of,
               const float* __restrict__ gate_w, const Vec16* __restrict__ add, int Tn, int Ke,
               int row_vecs, int rows_cap, Vec16* __restrict__ y) {
  pdl_enter();
  __shared__ int s_row[MOHGE_MAX_K_EXPERTS];
  __shared__ float s_g[MOHGE_MAX_K_EXPERTS];
  for (int t = blockIdx.x; t < Tn; t += gridDim.x) {
    __syncthreads();
    if (threadIdx.x < Ke) {
      s_row[threadIdx.x] = prow_of[(size_t)t * Ke + threadIdx.x];
      s_g[threadIdx.x] = gate_w ? gate_w[(size_t)t * Ke + threadIdx.x] : 1.0f;
    }
    __syncthreads();
    for (int c = threadIdx.x; c < row_vecs; c += blockDim.x) {
      float acc[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[i] = 0.0f;
      if (add) unpack(add[(size_t)t * row_vecs + c], acc, T());   // e.g. the shared experts' output
#pragma unroll 4
      for (int k = 0; k < Ke; ++k) {
        if ((unsigned)s_row[k] >= (unsigned)rows_cap) continue;   // invalid slot: contributes nothing
        const Vec16 v = y_perm[(size_t)s_row[k] * row_vecs + c];
        float f[8];
        unpack(v, f, T());
        const float g = s_g[k];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = fmaf(g, f[i], acc[i]);
      }
      y[(size_t)t * row_vecs + c] = pack(acc, T());
    }
  }
}

// dgate[t,k] = <dy[t], y_perm[prow[t,k]]>,  dy_perm[prow[t,k]] = gate[t,k] * dy[t]
// MODE 0: both; MODE 1: only the scaled rows (the gate gradient then comes out of the experts'
// backward, and y_perm is not read); MODE 2: only the gate gradient.
template <typename T, int MODE>
__global__ void __launch_bounds__(256)
combine_bwd_kernel(const Vec16* __restrict__ dy, const Vec16* __restrict__ y_perm,
                   const int32_t* __restrict__ prow_of, const float* __restrict__ gate_w, int Tn,
                   int Ke, int row_vecs, int rows_cap, Vec16* __restrict__ dy_perm,
                   float* __restrict__ dgate_w, int nb_tok, const int32_t* __restrict__ counts,
                   const int32_t* __restrict__ aligned) {
  pdl_enter();
  __shared__ int s_row[MOHGE_MAX_K_EXPERTS];
  __shared__ float s_g[MOHGE_MAX_K_EXPERTS];
  __shared__ float s_red[MOHGE_MAX_K_EXPERTS][8];
  if ((int)blockIdx.x >= nb_tok) {      // padding rows of dy_perm
    const int j = blockIdx.x - nb_tok;
    if (MODE != 2) zero_pad_part(counts, aligned, j >> 2, j & 3, row_vecs, dy_perm);
    return;
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  for (int t = blockIdx.x; t < Tn; t += nb_tok) {
    __syncthreads();
    if (threadIdx.x < Ke) {
      s_row[threadIdx.x] = prow_of[(size_t)t * Ke + threadIdx.x];
      s_g[threadIdx.x] = gate_w[(size_t)t * Ke + threadIdx.x];
    }
    __syncthreads();
    if (MODE == 1) {
      // one read of dy[t], K_e scaled copies
      for (int c = threadIdx.x; c < row_vecs; c += blockDim.x) {
        float a[8], o[8];
        unpack(dy[(size_t)t * row_vecs + c], a, T());
        for (int k = 0; k < Ke; ++k) {
          if ((unsigned)s_row[k] >= (unsigned)rows_cap) continue;
          const float g = s_g[k];
#pragma unroll
          for (int i = 0; i < 8; ++i) o[i] = g * a[i];
          store_streaming(dy_perm + (size_t)s_row[k] * row_vecs + c, pack(o, T()));
        }
      }
      continue;
    }
    for (int k = 0; k < Ke; ++k) {
      float part = 0.0f;
      const float g = s_g[k];
      const size_t rbase = (size_t)s_row[k] * row_vecs;
      const bool ok = (unsigned)s_row[k] < (unsigned)rows_cap;
      for (int c = threadIdx.x; ok && c < row_vecs; c += blockDim.x) {
        const Vec16 dv = dy[(size_t)t * row_vecs + c];
        const Vec16 yv = y_perm[rbase + c];
        float a[8], b[8], o[8];
        unpack(dv, a, T());
        unpack(yv, b, T());
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          part = fmaf(a[i], b[i], part);
          o[i] = g * a[i];
        }
        if (MODE == 0) dy_perm[rbase + c] = pack(o, T());
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(kFull, part, off);
      if (lane == 0) s_red[k][warp] = part;
    }
    __syncthreads();
    if (threadIdx.x < Ke) {
      float v = 0.0f;
      for (int w = 0; w < nwarps; ++w) v += s_red[threadIdx.x][w];
      dgate_w[(size_t)t * Ke + threadIdx.x] = v;
    }
  }
}

// Gate gradient from the partial sums the SwiGLU-backward epilogue leaves per physical row and
// 128-column slot: sum_j dH_j h_j with dH = (gate * dy) W2, i.e. gate * <dy, Y>; the slots are
// added in ascending order (fixed) and the sum is divided by the gate.  A gate that is exactly
// zero left a zero row in dy_perm; such a pair takes the definition <dy[t], y_perm[row]> instead.
struct DgateShape {
  int N, Ne, Ke, slots, d;
  int W[MOHGE_MAX_GROUPS];
  int step[MOHGE_MAX_GROUPS];      // tile width of the group / 128: every step-th slot is written
};

template <typename T>
__device__ __forceinline__ float as_float(T v);
template <>
__device__ __forceinline__ float as_float<float>(float v) { return v; }
template <>
__device__ __forceinline__ float as_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T>
__global__ void __launch_bounds__(256)
dgate_reduce_kernel(DgateShape s, int n, const float* __restrict__ part,
                    const int32_t* __restrict__ prow_of, const float* __restrict__ gate_w,
                    const int32_t* __restrict__ aligned, const T* __restrict__ dy,
                    const T* __restrict__ y_perm, int rows_cap, float* __restrict__ dgate_w) {
  pdl_enter();
  for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < n; idx += gridDim.x * blockDim.x) {
    const int r = prow_of[idx];
    float v = 0.0f;
    if ((unsigned)r < (unsigned)rows_cap) {
      const float gate = gate_w[idx];
      if (gate != 0.0f) {
        int lo = 0, hi = s.Ne;           // aligned[lo] <= r < aligned[hi]: lo ends at the row's expert
        while (hi - lo > 1) {
          const int mid = (lo + hi) >> 1;
          if (aligned[mid] <= r) lo = mid; else hi = mid;
        }
        const int g = lo / s.N;
        const float* pr = part + (size_t)r * s.slots;
        const int ns = (s.W[g] + 127) >> 7;
        float acc = 0.0f;
        for (int j = 0; j < ns; j += s.step[g]) acc += pr[j];
        v = acc / gate;
      } else {
        const size_t t = (size_t)(idx / s.Ke);
        float acc = 0.0f;
        for (int c = 0; c < s.d; ++c)
          acc = fmaf(as_float<T>(dy[t * s.d + c]), as_float<T>(y_perm[(size_t)r * s.d + c]), acc);
        v = acc;
      }
    }
    dgate_w[idx] = v;
  }
}

// Source token of every physical row of the permuted numbering (T, which is out of range, for
// padding rows and for the 128 rows past the last segment that a CTA pair's tile may touch):
// the row map the experts' GEMMs use to gather rows of x themselves instead of reading x_perm.
__global__ void __launch_bounds__(256)
token_of_row_kernel(int n_rows, int T, int Ke, int Ne, const int32_t* __restrict__ counts,
                    const int32_t* __restrict__ offsets, const int32_t* __restrict__ aligned,
                    const int32_t* __restrict__ src_of, int32_t* __restrict__ tok_of_prow) {
  pdl_enter();
  for (int r = blockIdx.x * blockDim.x + threadIdx.x; r < n_rows; r += gridDim.x * blockDim.x) {
    int tok = T;
    if (r < aligned[Ne]) {
      int lo = 0, hi = Ne;               // aligned[lo] <= r < aligned[hi]
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (aligned[mid] <= r) lo = mid; else hi = mid;
      }
      const int j = r - aligned[lo];
      if (j < counts[lo]) tok = src_of[offsets[lo] + j] / Ke;
    }
    tok_of_prow[r] = tok;
  }
}

int block_for(int row_vecs) {
  int b = (row_vecs + 31) / 32 * 32;
  if (b > 256) b = 256;
  if (b < 32) b = 32;
  return b;
}

}  // namespace

int32_t launch_token_of_row(const Dims& D, const int32_t* counts, const int32_t* offsets,
                            const int32_t* aligned, const int32_t* src_of, int32_t* tok_of_prow,
                            cudaStream_t st) {
  const int n_rows = (int)D.Rcap + kGatherSlack;
  launch_dep(token_of_row_kernel, dim3((n_rows + 255) / 256 < 1184 ? (n_rows + 255) / 256 : 1184), dim3(256), st,
             n_rows, (int)D.T, D.Ke, D.Ne, counts, offsets, aligned, src_of, tok_of_prow);
  MOHGE_LAUNCH_CHECK("token_of_row_kernel");
  return MOHGE_OK;
}

// x != nullptr: rows of x are copied into x_perm; tok_of_prow != nullptr: the row map for the
// gathering GEMMs is written instead (kGatherSlack rows past mohge_perm_rows included).
int32_t launch_dispatch(const Dims& D, const void* x, const int32_t* expert_idx, int32_t* counts,
                        int32_t* offsets, int32_t* aligned, int32_t* row_of, int32_t* prow_of,
                        int32_t* src_of, void* x_perm, int32_t* hist, int32_t* base,
                        int32_t* status, cudaStream_t st, int32_t* tok_of_prow) {
  const int chunks = ceil_div(D.T, kDispatchChunk);
  const int T = (int)D.T;
  if (chunks > 0) {
    launch_dep(dispatch_hist_kernel, dim3(chunks), dim3(kDispatchChunk), st, expert_idx, T, D.Ke, D.Ne, hist, status);
    MOHGE_LAUNCH_CHECK("dispatch_hist_kernel");
  }
  launch_dep(dispatch_scan_kernel, dim3(1), dim3(256), st, chunks, D.Ne, D.align, hist, base, counts, offsets, aligned);
  MOHGE_LAUNCH_CHECK("dispatch_scan_kernel");
  if (chunks > 0) {
    launch_dep(dispatch_scatter_kernel, dim3(chunks), dim3(kDispatchChunk), st, expert_idx, T, D.Ke, D.Ne, base, offsets,
                                                              aligned, row_of, prow_of, src_of, status);
    MOHGE_LAUNCH_CHECK("dispatch_scatter_kernel");
  }
  if (tok_of_prow != nullptr) {
    const int32_t rc = launch_token_of_row(D, counts, offsets, aligned, src_of, tok_of_prow, st);
    if (rc) return rc;
  }
  if (chunks == 0 || x == nullptr) return MOHGE_OK;
  const int row_vecs = D.d * (D.bf16 ? 2 : 4) / 16;
  const int blocks = T < 148 * 16 ? T : 148 * 16;
  const int pad_blocks = D.align > 1 ? 4 * D.Ne : 0;
  launch_dep(permute_rows_kernel, dim3(blocks + pad_blocks), dim3(block_for(row_vecs)), st,
      (const Vec16*)x, prow_of, T, D.Ke, row_vecs, (int)D.Rcap, (Vec16*)x_perm, blocks, counts, aligned);
  MOHGE_LAUNCH_CHECK("permute_rows_kernel");
  return MOHGE_OK;
}

namespace {
__global__ void __launch_bounds__(256)
row_gate_kernel(int n_rows, int n_slots, const int32_t* __restrict__ prow_of,
                const float* __restrict__ gate_w, float* __restrict__ row_gate, int phase) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (phase == 0) {
    if (i < n_rows) row_gate[i] = 0.0f;
  } else if (i < n_slots) {
    const int r = prow_of[i];
    if ((unsigned)r < (unsigned)n_rows) row_gate[r] = gate_w[i];
  }
}
}  // namespace

int32_t launch_row_gate(const Dims& D, const int32_t* prow_of, const float* gate_w, float* row_gate,
                        cudaStream_t st) {
  const int n_rows = (int)D.Rcap, n_slots = (int)(D.T * D.Ke);
  if (n_rows > 0) {
    row_gate_kernel<<<(n_rows + 255) / 256, 256, 0, st>>>(n_rows, n_slots, prow_of, gate_w, row_gate, 0);
    MOHGE_LAUNCH_CHECK("row_gate_kernel");
  }
  if (n_slots > 0) {
    row_gate_kernel<<<(n_slots + 255) / 256, 256, 0, st>>>(n_rows, n_slots, prow_of, gate_w, row_gate, 1);
    MOHGE_LAUNCH_CHECK("row_gate_kernel");
  }
  return MOHGE_OK;
}

int32_t launch_combine(const Dims& D, const void* y_perm, const int32_t* prow_of,
                       const float* gate_w, const void* add, void* y, cudaStream_t st) {
  if (D.T == 0) return MOHGE_OK;
  const int T = (int)D.T;
  const int row_vecs = D.d * (D.bf16 ? 2 : 4) / 16;
  const int blocks = T < 148 * 16 ? T : 148 * 16;
  if (D.bf16)
    launch_dep(combine_kernel<__nv_bfloat16>, dim3(blocks), dim3(block_for(row_vecs)), st,
        (const Vec16*)y_perm, prow_of, gate_w, (const Vec16*)add, T, D.Ke, row_vecs, (int)D.Rcap,
        (Vec16*)y);
  else
    launch_dep(combine_kernel<float>, dim3(blocks), dim3(block_for(row_vecs)), st,
        (const Vec16*)y_perm, prow_of, gate_w, (const Vec16*)add, T, D.Ke, row_vecs, (int)D.Rcap,
        (Vec16*)y);
  MOHGE_LAUNCH_CHECK("combine_kernel");
  return MOHGE_OK;
}

int32_t launch_unpermute_sum(const Dims& D, const void* dx_perm, const int32_t* prow_of,
                             const void* add, void* dx, cudaStream_t st) {
  return launch_combine(D, dx_perm, prow_of, nullptr, add, dx, st);
}

int32_t launch_dgate_reduce(const Dims& D, const int* bn, const float* part, int slots,
                            const int32_t* prow_of, const float* gate_w, const int32_t* aligned,
                            const void* dy, const void* y_perm, float* dgate_w, cudaStream_t st) {
  if (D.T == 0) return MOHGE_OK;
  DgateShape s;
  s.N = D.N; s.Ne = D.Ne; s.Ke = D.Ke; s.slots = slots; s.d = D.d;
  for (int g = 0; g < MOHGE_MAX_GROUPS; ++g) {
    s.W[g] = g < D.Ng ? D.W[g] : 0;
    s.step[g] = g < D.Ng ? bn[g] / 128 : 1;
  }
  const int n = (int)(D.T * D.Ke);
  const int blocks = (n + 255) / 256 < 148 * 8 ? (n + 255) / 256 : 148 * 8;
  if (D.bf16)
    launch_dep(dgate_reduce_kernel<__nv_bfloat16>, dim3(blocks), dim3(256), st, s, n, part, prow_of, gate_w,
               aligned, (const __nv_bfloat16*)dy, (const __nv_bfloat16*)y_perm, (int)D.Rcap, dgate_w);
  else
    launch_dep(dgate_reduce_kernel<float>, dim3(blocks), dim3(256), st, s, n, part, prow_of, gate_w, aligned,
               (const float*)dy, (const float*)y_perm, (int)D.Rcap, dgate_w);
  MOHGE_LAUNCH_CHECK("dgate_reduce_kernel");
  return MOHGE_OK;
}

template <typename T, int MODE>
static void launch_combine_bwd_mode(const Dims& D, int blocks, int pad_blocks, int row_vecs, const void* dy,
                                    const void* y_perm, const int32_t* prow_of, const float* gate_w,
                                    const int32_t* counts, const int32_t* aligned, void* dy_perm,
                                    float* dgate_w, cudaStream_t st) {
  launch_dep(combine_bwd_kernel<T, MODE>, dim3(blocks + pad_blocks), dim3(block_for(row_vecs)), st,
             (const Vec16*)dy, (const Vec16*)y_perm, prow_of, gate_w, (int)D.T, D.Ke, row_vecs, (int)D.Rcap,
             (Vec16*)dy_perm, dgate_w, blocks, counts, aligned);
}

// mode 0: dy_perm and dgate_w; 1: dy_perm only (y_perm, dgate_w unused); 2: dgate_w only
int32_t launch_combine_bwd(const Dims& D, int mode, const void* dy, const void* y_perm,
                           const int32_t* prow_of, const float* gate_w, const int32_t* counts,
                           const int32_t* aligned, void* dy_perm, float* dgate_w, cudaStream_t st) {
  const int T = (int)D.T;
  const int row_vecs = D.d * (D.bf16 ? 2 : 4) / 16;
  const int pad_blocks = (D.align > 1 && mode != 2) ? 4 * D.Ne : 0;
  if (T > 0) {
    const int blocks = T < 148 * 16 ? T : 148 * 16;
#define MOHGE_CB(TT, MM) launch_combine_bwd_mode<TT, MM>(D, blocks, pad_blocks, row_vecs, dy, y_perm, prow_of, \
                                                        gate_w, counts, aligned, dy_perm, dgate_w, st)
    if (D.bf16) {
      if (mode == 0) MOHGE_CB(__nv_bfloat16, 0); else if (mode == 1) MOHGE_CB(__nv_bfloat16, 1); else MOHGE_CB(__nv_bfloat16, 2);
    } else {
      if (mode == 0) MOHGE_CB(float, 0); else if (mode == 1) MOHGE_CB(float, 1); else MOHGE_CB(float, 2);
    }
#undef MOHGE_CB
    MOHGE_LAUNCH_CHECK("combine_bwd_kernel");
  }
  if (D.align > 1 && T == 0 && mode != 2) {
    launch_dep(zero_pad_rows_kernel, dim3(D.Ne, 4), dim3(256), st, counts, aligned, row_vecs, (Vec16*)dy_perm);
    MOHGE_LAUNCH_CHECK("zero_pad_rows_kernel");
  }
  return MOHGE_OK;
}

}  // namespace mohge
