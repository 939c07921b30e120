// Deterministic sums, base-sample statistics and the sample budget.
//
// For each (batch row, query head) the rows of I_f = sink + I_t + window and of the base sample I_bs
// are gathered (K and V), rescored in fp64 and reduced:
//     D_f = sum_{I_f} w_i,  N_f = sum_{I_f} w_i V[i]                       (Sec. 4.1, N_f and D_f)
//     sum w, sum w^2, sum r, sum r.r over I_bs with r_i = w_i V[i]           (Algorithm 2, get-stats)
// with w_i = exp(s_i - m).  Every CTA leaves one partial; the budget kernel behind this one adds them in a
// fixed order and evaluates the budgets of Corollaries D.2 and Theorem 4.3.
//
// Everything that decides the integer budget is fp64: the same inputs must give the same ceil() as a
// plain fp64 evaluation.  Variances are accumulated around a pivot (the first base-sample row), which
// removes the cancellation of the one-pass formula and makes a constant population give exactly 0.
//
// Grid: per head, `stat_splits` CTAs take the deterministic rows and `stat_splits` CTAs the base-sample
// rows (two code paths with disjoint accumulators, which halves the register footprint of either).
// A row group (LPR lanes) works in batches of UN rows and keeps two batches in flight: the 16-byte row
// slices of batch k + 1 and the indices of batch k + 2 are requested before batch k is reduced, so the
// fp64 arithmetic of one batch hides the memory round trip of the next.
#include "vattn_internal.cuh"
#include <math_constants.h>

namespace {

constexpr int NT = 128;
constexpr int NWARP = NT / 32;
constexpr int UN = 2;            // rows per batch of a row group; two batches are in flight (double buffer)
constexpr int MAXS = VATTN_STAT_MAXS;   // most split CTAs per head and kind

// 16-byte row slices, fetched with streaming loads: a row is read once, so it should be the first to leave the
// caches (the scores, index lists and partials that the step re-reads stay in L2)
template <typename T> struct Raw;
template <> struct Raw<float> {
  float4 v;
  __device__ __forceinline__ void ld(const float* p) { v = __ldcs(reinterpret_cast<const float4*>(p)); }
  __device__ __forceinline__ float get(int e) const { return e == 0 ? v.x : e == 1 ? v.y : e == 2 ? v.z : v.w; }
};
template <> struct Raw<bf16_t> {
  uint4 v;
  __device__ __forceinline__ void ld(const bf16_t* p) { v = __ldcs(reinterpret_cast<const uint4*>(p)); }
  __device__ __forceinline__ float get(int e) const {
    const unsigned w = (e >> 1) == 0 ? v.x : (e >> 1) == 1 ? v.y : (e >> 1) == 2 ? v.z : v.w;
    return __uint_as_float((e & 1) ? (w & 0xFFFF0000u) : (w << 16));
  }
};

template <typename T>
struct RowRegs { Raw<T> k, v; };

// K and V slices of the row in physical slot `ph` (= page * 16 + token % 16)
template <typename T, int D>
__device__ __forceinline__ void load_row(const Prob& p, int g, int ph, int j, RowRegs<T>& r) {
  constexpr int EPL = Elem<T>::EPL;
  const long long off = (long long)(ph >> 4) * p.sb + (long long)g * p.sh + (long long)(ph & 15) * p.st + j * EPL;
  r.k.ld(reinterpret_cast<const T*>(p.kc) + off);
  r.v.ld(reinterpret_cast<const T*>(p.vc) + off);
}
__device__ __forceinline__ int phys_of(const Prob& p, int b, int tok) { return page_of(p, b, tok >> 4) * VATTN_BLOCK + (tok & 15); }
// fp64 inner product <q, K[row]> computed by the LPR lanes of a row group from their K slices
template <typename T, int D>
__device__ __forceinline__ double dot64(const double* qs, const RowRegs<T>& r) {
  constexpr int EPL = Elem<T>::EPL, LPR = D / EPL;
  double acc = 0.0;
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc = fma(qs[e * LPR], (double)r.k.get(e), acc);
#pragma unroll
  for (int mask = LPR / 2; mask >= 1; mask >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, mask);
  return acc;
}
// fp64 weight of one token
template <typename T, int D>
__device__ __forceinline__ double weight64(const Prob& p, const double* qs, const RowRegs<T>& r, double m) {
  return exp(dot64<T, D>(qs, r) * (double)p.scale - m);
}
// weights of the UN rows of a batch with ONE exp per lane: lane j of the row group evaluates the row
// j % UN, the results are handed round with shuffles (every lane of a group holds all UN inner products)
template <typename T, int D>
__device__ __forceinline__ void weights64(const Prob& p, const double* qs, const RowRegs<T> (&row)[UN],
                                          double m, int j, double (&w)[UN]) {
  constexpr int LPR = D / Elem<T>::EPL;
  static_assert((UN == 2 || UN == 4) && LPR >= UN, "one lane per row of the batch");
  double d[UN];
#pragma unroll
  for (int u = 0; u < UN; ++u) d[u] = dot64<T, D>(qs, row[u]);
  const int mu = j & (UN - 1);
  double mine = d[0];
#pragma unroll
  for (int u = 1; u < UN; ++u) mine = (mu == u) ? d[u] : mine;
  const double wm = exp(mine * (double)p.scale - m);
#pragma unroll
  for (int u = 0; u < UN; ++u) w[u] = __shfl_sync(0xFFFFFFFFu, wm, u, LPR);
}

template <typename T, int D>
__global__ void __launch_bounds__(NT, 5) k_stats(const Prob p) {
  constexpr int EPL = Elem<T>::EPL, LPR = D / EPL, RPI = 32 / LPR;
  constexpr int NE = D + 3;               // det CTA: N_f[D], D_f;  base CTA: Sr[D], Sw, Sww, Srr
  constexpr int RG = NWARP * RPI;         // row groups per CTA
  __shared__ double part[NWARP][NE];
  __shared__ double piv[D + 1];
  __shared__ double pivT[D];             // the pivot's w*V, element-major per lane: pivT[e * LPR + j]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // grid (S, Hq, 2 B): the deterministic-row CTAs of every head come first in dispatch order, so they take
  // the SMs that are free while the select kernels still run; the base-row CTAs follow
  const bool base_cta = (int)blockIdx.z >= p.B;
  const int h = blockIdx.y, b = base_cta ? blockIdx.z - p.B : blockIdx.z, g = h / p.G;
  const int bh = b * p.Hq + h;
  const int S = base_cta ? p.stat_splits_base : p.stat_splits;   // CTAs of this kind per head
  const int split = blockIdx.x;
  const int vx = (base_cta ? MAXS : 0) + split;    // position among the head's 2 MAXS partial slots
  if (split >= S) {                                // the grid is as wide as the larger of the two split counts
    if (base_cta) pdl_wait();                      // (every base-row CTA waits, see below)
    return;
  }
  TICK_BEGIN(p, VATTN_K_STATS);
  pdl_trigger();
  // What k_select_topk wrote (meta, I_t) is complete before this grid can start: the grid before this one
  // lets its dependents go only after its own wait on k_select_topk.  Only the base-row CTAs need the
  // grid before this one itself (I_bs), and they wait for it as late as possible.
  const HeadMeta mt = ld_meta(p.meta + bh);
  const int n = mt.n, s0 = mt.s0, l_start = mt.l_start, kk = mt.kk, b0 = mt.b0;
  if (n == 0) {
    if (base_cta) pdl_wait();                      // every base-row CTA waits: "this grid done" implies "the one before done"
    return;
  }
  const int n_f = s0 + kk + (n - l_start);
  const int total = base_cta ? b0 : n_f;
  const int chunk = (total + S - 1) / S;
  const int r_begin = min(total, split * chunk), r_end = min(total, r_begin + chunk);
  const int* tkph = p.topk_idx + (long long)bh * p.npad + p.phys_delta;     // physical slots of I_t
  const int* bsph = p.base_idx + (long long)bh * p.npad + p.phys_delta;     // physical slots of I_bs
  const int ph0 = phys_of(p, b, 0);
  const double m = (double)mt.m;
  const int rsub = lane / LPR, j = lane % LPR;
  const int rg = warp * RPI + rsub;
  const int iters = (r_end - r_begin + RG - 1) / RG;      // uniform over the CTA

  // q in fp64, element-major per lane (qT[e * LPR + j]): read from shared memory where it is used instead of
  // living in 16 registers
  __shared__ double qT[D];
  if (warp == 0 && rsub == 0) {
    float qf[EPL];
    Elem<T>::load(reinterpret_cast<const T*>(p.q) + (long long)bh * D + j * EPL, qf);
#pragma unroll
    for (int e = 0; e < EPL; ++e) qT[e * LPR + j] = (double)qf[e];
  }
  __syncthreads();
  const double* qs = qT + j;

  double acc[EPL], s1 = 0.0, s2 = 0.0, s3 = 0.0;           // det: N_f slice, D_f;  base: Sr slice, Sw, Sww, Srr
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc[e] = 0.0;

  if (!base_cta) {
    // ---------------------------------------------------------------- deterministic rows: sink, I_t, window
    // physical slots of the next batch are requested while the current rows are in flight
    int ph_n[UN];
    bool act_n[UN];
    auto fetch = [&](int k0) {
#pragma unroll
      for (int u = 0; u < UN; ++u) {
        const int r = r_begin + rg + (k0 + u) * RG;
        act_n[u] = (k0 + u < iters) && (r < r_end);
        ph_n[u] = ph0;                                       // idle slots re-read the first row
        if (act_n[u])
          ph_n[u] = r < s0 ? phys_of(p, b, r) : (r < s0 + kk ? __ldg(tkph + r - s0) : phys_of(p, b, l_start + (r - s0 - kk)));
      }
    };
    auto issue = [&](RowRegs<T> (&row)[UN], bool (&act)[UN]) {
#pragma unroll
      for (int u = 0; u < UN; ++u) { act[u] = act_n[u]; load_row<T, D>(p, g, ph_n[u], j, row[u]); }
    };
    auto reduce = [&](const RowRegs<T> (&row)[UN], const bool (&act)[UN]) {
      double wv[UN];
      weights64<T, D>(p, qs, row, m, j, wv);                   // every lane takes part in the shuffles
#pragma unroll
      for (int u = 0; u < UN; ++u) {
        const double w = wv[u];
        if (act[u]) {
          s1 += w;
#pragma unroll
          for (int e = 0; e < EPL; ++e) acc[e] = fma(w, (double)row[u].v.get(e), acc[e]);
        }
      }
    };
    RowRegs<T> rowA[UN], rowB[UN];
    bool actA[UN], actB[UN];
    fetch(0);
    issue(rowA, actA);
    fetch(UN);
    for (int k0 = 0; k0 < iters; k0 += 2 * UN) {
      issue(rowB, actB);
      fetch(k0 + 2 * UN);
      reduce(rowA, actA);
      if (k0 + UN >= iters) break;                             // uniform over the CTA
      issue(rowA, actA);
      fetch(k0 + 3 * UN);
      reduce(rowB, actB);
    }
  } else {
    pdl_wait();
  }
  if (base_cta && b0 > 0) {
    // ---------------------------------------------------------------- base-sample rows, shifted by the pivot
    RowRegs<T> prow;
    const int piv_ph = __ldg(bsph);                          // pivot = first base-sample row
    int ph_n[UN];
    bool act_n[UN];
    auto fetch = [&](int k0) {
#pragma unroll
      for (int u = 0; u < UN; ++u) {
        const int r = r_begin + rg + (k0 + u) * RG;
        act_n[u] = (k0 + u < iters) && (r < r_end);
        ph_n[u] = act_n[u] ? __ldg(bsph + r) : piv_ph;
      }
    };
    auto issue = [&](RowRegs<T> (&row)[UN], bool (&act)[UN]) {
#pragma unroll
      for (int u = 0; u < UN; ++u) { act[u] = act_n[u]; load_row<T, D>(p, g, ph_n[u], j, row[u]); }
    };
    double cw = 0.0;
    auto reduce = [&](const RowRegs<T> (&row)[UN], const bool (&act)[UN]) {
      double wv[UN];
      weights64<T, D>(p, qs, row, m, j, wv);
#pragma unroll
      for (int u = 0; u < UN; ++u) {
        const double w = wv[u];
        if (act[u]) {
          const double dw = w - cw;
          s1 += dw;
          s2 = fma(dw, dw, s2);
#pragma unroll
          for (int e = 0; e < EPL; ++e) {
            const double dr = w * (double)row[u].v.get(e) - pivT[e * LPR + j];
            acc[e] += dr;
            s3 = fma(dr, dr, s3);
          }
        }
      }
    };
    RowRegs<T> rowA[UN], rowB[UN];
    bool actA[UN], actB[UN];
    fetch(0);
    load_row<T, D>(p, g, piv_ph, j, prow);
    issue(rowA, actA);
    fetch(UN);
    issue(rowB, actB);
    fetch(2 * UN);
    cw = weight64<T, D>(p, qs, prow, m);
    if (warp == 0 && rsub == 0) {                     // every row group holds the same pivot: one of them shares it
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        const double c = cw * (double)prow.v.get(e);
        piv[j * EPL + e] = c;
        pivT[e * LPR + j] = c;
      }
      if (j == 0) piv[D] = cw;
    }
    __syncthreads();
    for (int k0 = 0; k0 < max(iters, 1); k0 += 2 * UN) {
      if (k0 > 0) { issue(rowB, actB); fetch(k0 + 2 * UN); }
      reduce(rowA, actA);
      if (k0 + UN >= iters) break;                             // uniform over the CTA
      issue(rowA, actA);
      fetch(k0 + 3 * UN);
      reduce(rowB, actB);
    }
  }
  // across the row groups of the warp
#pragma unroll
  for (int mask = LPR; mask < 32; mask <<= 1) {
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] += __shfl_xor_sync(0xFFFFFFFFu, acc[e], mask);
    s1 += __shfl_xor_sync(0xFFFFFFFFu, s1, mask);
    s2 += __shfl_xor_sync(0xFFFFFFFFu, s2, mask);
  }
#pragma unroll
  for (int mask = 1; mask < 32; mask <<= 1) s3 += __shfl_xor_sync(0xFFFFFFFFu, s3, mask);
  if (rsub == 0) {
#pragma unroll
    for (int e = 0; e < EPL; ++e) part[warp][j * EPL + e] = acc[e];
    if (j == 0) { part[warp][D] = s1; part[warp][D + 1] = s2; part[warp][D + 2] = s3; }
  }
  __syncthreads();
  double* gpart = p.stat_part + ((long long)bh * 2 * MAXS + vx) * NE;
  for (int e = tid; e < NE; e += NT) {
    double s = 0.0;
#pragma unroll
    for (int w = 0; w < NWARP; ++w) s += part[w][e];
    gpart[e] = s;
  }
  if (base_cta && split == 0 && b0 > 0)              // the pivot travels with this CTA's partial
    for (int e = tid; e <= D; e += NT) p.stat_piv[(long long)bh * (D + 1) + e] = piv[e];
  TICK_END(p, VATTN_K_STATS);
}

}  // namespace

cudaError_t launch_stats(const Prob& p, cudaStream_t s) {
  if (p.stat_splits < 1 || p.stat_splits > MAXS || p.stat_splits_base < 1 || p.stat_splits_base > MAXS) return cudaErrorInvalidValue;
  dim3 grid(p.stat_splits > p.stat_splits_base ? p.stat_splits : p.stat_splits_base, p.Hq, 2 * p.B), block(NT);
  if (p.dtype == VATTN_DTYPE_BF16) {
    if (p.D == 128) return launch_pdl(k_stats<bf16_t, 128>, grid, block, 0, s, p);
    else return launch_pdl(k_stats<bf16_t, 64>, grid, block, 0, s, p);
  } else {
    if (p.D == 128) return launch_pdl(k_stats<float, 128>, grid, block, 0, s, p);
    else return launch_pdl(k_stats<float, 64>, grid, block, 0, s, p);
  }
  return cudaGetLastError();
}
