// Deterministic sums, base-sample statistics and the sample budget.
//
// For each (batch row, query head) the rows of I_f = sink + I_t + window and of the base sample I_bs
// are gathered (K and V), rescored in fp64 and reduced:
//     D_f = sum_{I_f} w_i,  N_f = sum_{I_f} w_i V[i]                       (Sec. 4.1, N_f and D_f)
//     sum w, sum w^2, sum r, sum r.r over I_bs with r_i = w_i V[i]           (Algorithm 2, get-stats)
// with w_i = exp(s_i - m).  The last CTA of a head ("ticket") adds the partials in a fixed order and
// evaluates the budgets of Corollaries D.2 and Theorem 4.3, b = clamp(ceil(b_X), b0, n_s).
//
// Everything that decides the integer budget is fp64: the same inputs must give the same ceil() as a
// plain fp64 evaluation.  Variances are accumulated around a pivot (the first base-sample row), which
// removes the cancellation of the one-pass formula and makes a constant population give exactly 0.
#include "vattn_internal.cuh"
#include <math_constants.h>

namespace {

constexpr int NT = ROW_THREADS;
constexpr int NWARP = NT / 32;

template <typename T, int D>
struct RowLayout {
  static constexpr int EPL = Elem<T>::EPL;
  static constexpr int LPR = D / EPL;
  static constexpr int RPI = 32 / LPR;
};

// fp64 weight of one token and its value slice, computed by the LPR lanes of a row group
template <typename T, int D>
__device__ __forceinline__ double row_weight(const Prob& p, int b, int g, const float (&qf)[Elem<T>::EPL], int tok,
                                             int j, double m, float (&v)[Elem<T>::EPL]) {
  constexpr int EPL = Elem<T>::EPL, LPR = D / EPL;
  const T* krow = row_ptr<T>(p, p.kc, b, g, tok);
  const T* vrow = row_ptr<T>(p, p.vc, b, g, tok);
  float kx[EPL];
  Elem<T>::load(krow + j * EPL, kx);
  Elem<T>::load(vrow + j * EPL, v);
  double acc = 0.0;
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc = fma((double)qf[e], (double)kx[e], acc);
#pragma unroll
  for (int mask = LPR / 2; mask >= 1; mask >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, mask);
  return exp(acc * (double)p.scale - m);
}

__device__ __forceinline__ int ceil_sat(double x) {
  if (!isfinite(x) || x >= 2147483647.0) return 2147483647;
  return (int)ceil(x);
}

template <typename T, int D>
__global__ void __launch_bounds__(NT) k_stats(const Prob p) {
  using L = RowLayout<T, D>;
  constexpr int EPL = L::EPL, LPR = L::LPR, RPI = L::RPI;
  constexpr int NE = 2 * D + 4;           // N_f[D], D_f, Sw, Sww, Sr[D], Srr
  __shared__ double part[NWARP][NE];
  __shared__ double tot[NE];
  __shared__ double piv[D + 1];
  __shared__ int is_last;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z, g = h / p.G;
  const int bh = b * p.Hq + h;
  const int S = p.stat_splits;
  HeadMeta& meta = p.meta[bh];
  const int n = meta.n, s0 = meta.s0, l_start = meta.l_start, kk = meta.kk, n_s = meta.n_s, b0 = meta.b0;
  if (n == 0) {
    if (split == 0 && tid == 0) {
      meta.b = 0;
      if (p.dbg.budgets) for (int e = 0; e < 4; ++e) p.dbg.budgets[bh * 4 + e] = 0;
      if (p.dbg.stats) for (int e = 0; e < 8; ++e) p.dbg.stats[bh * 8 + e] = 0.0;
    }
    return;
  }
  const int n_f = s0 + kk + (n - l_start);
  const int total = n_f + b0;
  const int chunk = (total + S - 1) / S;
  const int r_begin = min(total, split * chunk), r_end = min(total, r_begin + chunk);
  const int* tk = p.topk_idx + (long long)bh * p.npad;
  const int* bs = p.base_idx + (long long)bh * p.npad;
  const double m = (double)meta.m;
  const int rsub = lane / LPR, j = lane % LPR;

  float qf[EPL];
  Elem<T>::load(reinterpret_cast<const T*>(p.q) + (long long)bh * D + j * EPL, qf);

  // pivot = first base-sample row (every row group computes the same numbers)
  double cw = 0.0, cr[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) cr[e] = 0.0;
  if (b0 > 0) {
    float v[EPL];
    cw = row_weight<T, D>(p, b, g, qf, bs[0], j, m, v);
#pragma unroll
    for (int e = 0; e < EPL; ++e) cr[e] = cw * (double)v[e];
    if (warp == 0 && rsub == 0) {
#pragma unroll
      for (int e = 0; e < EPL; ++e) piv[j * EPL + e] = cr[e];
      if (j == 0) piv[D] = cw;
    }
  } else {
    for (int e = tid; e <= D; e += NT) piv[e] = 0.0;
  }

  double Nf[EPL], Sr[EPL], Df = 0.0, Sw = 0.0, Sww = 0.0, Srr = 0.0;
#pragma unroll
  for (int e = 0; e < EPL; ++e) { Nf[e] = 0.0; Sr[e] = 0.0; }

  for (int r0 = r_begin + warp * RPI; r0 < r_end; r0 += NWARP * RPI) {
    const int r = r0 + rsub;
    const bool active = r < r_end;
    int tok = 0;
    bool is_base = false;
    if (active) {
      if (r < s0) tok = r;
      else if (r < s0 + kk) tok = tk[r - s0];
      else if (r < n_f) tok = l_start + (r - s0 - kk);
      else { tok = bs[r - n_f]; is_base = true; }
    }
    float v[EPL];
    // inactive row groups still take part in the shuffles (they recompute token 0 and drop it)
    const double w = row_weight<T, D>(p, b, g, qf, tok, j, m, v);
    if (active) {
      if (!is_base) {
        Df += w;
#pragma unroll
        for (int e = 0; e < EPL; ++e) Nf[e] = fma(w, (double)v[e], Nf[e]);
      } else {
        const double dw = w - cw;
        Sw += dw;
        Sww = fma(dw, dw, Sww);
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
          const double dr = w * (double)v[e] - cr[e];
          Sr[e] += dr;
          Srr = fma(dr, dr, Srr);
        }
      }
    }
  }
  // across the row groups of the warp
#pragma unroll
  for (int mask = LPR; mask < 32; mask <<= 1) {
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      Nf[e] += __shfl_xor_sync(0xFFFFFFFFu, Nf[e], mask);
      Sr[e] += __shfl_xor_sync(0xFFFFFFFFu, Sr[e], mask);
    }
    Df += __shfl_xor_sync(0xFFFFFFFFu, Df, mask);
    Sw += __shfl_xor_sync(0xFFFFFFFFu, Sw, mask);
    Sww += __shfl_xor_sync(0xFFFFFFFFu, Sww, mask);
  }
#pragma unroll
  for (int mask = 1; mask < 32; mask <<= 1) Srr += __shfl_xor_sync(0xFFFFFFFFu, Srr, mask);
  if (rsub == 0) {
#pragma unroll
    for (int e = 0; e < EPL; ++e) { part[warp][j * EPL + e] = Nf[e]; part[warp][D + 3 + j * EPL + e] = Sr[e]; }
    if (j == 0) { part[warp][D] = Df; part[warp][D + 1] = Sw; part[warp][D + 2] = Sww; part[warp][2 * D + 3] = Srr; }
  }
  __syncthreads();
  double* gpart = p.stat_part + ((long long)bh * S + split) * NE;
  for (int e = tid; e < NE; e += NT) {
    double s = 0.0;
#pragma unroll
    for (int w = 0; w < NWARP; ++w) s += part[w][e];
    gpart[e] = s;
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) is_last = (atomicAdd(&p.tickets[bh], 1u) == (unsigned)(S - 1));
  __syncthreads();
  if (!is_last) return;
  __threadfence();

  // ------------------------------------------------------------------ last CTA of this head
  for (int e = tid; e < NE; e += NT) {
    double s = 0.0;
    for (int sp = 0; sp < S; ++sp) s += __ldcg(p.stat_part + ((long long)bh * S + sp) * NE + e);
    tot[e] = s;
  }
  __syncthreads();
  double* det = p.det_sums + (long long)bh * (D + 1);
  for (int e = tid; e <= D; e += NT) det[e] = tot[e];
  if (warp != 0) return;

  const double Dfv = tot[D];
  const double ratio = (b0 > 0) ? (double)n_s / (double)b0 : 0.0;
  double nn = 0.0, sr2 = 0.0;                 // |N_hat|^2 and sum_j (sum_i r'_ij)^2
  for (int e = lane; e < D; e += 32) {
    const double srj = tot[D + 3 + e];
    const double nh = tot[e] + ratio * (srj + (double)b0 * piv[e]);
    nn = fma(nh, nh, nn);
    sr2 = fma(srj, srj, sr2);
  }
#pragma unroll
  for (int mask = 16; mask >= 1; mask >>= 1) {
    nn += __shfl_xor_sync(0xFFFFFFFFu, nn, mask);
    sr2 += __shfl_xor_sync(0xFFFFFFFFu, sr2, mask);
  }
  if (lane != 0) return;

  const double Nnorm = sqrt(nn);
  double sigma2 = 0.0, trace = 0.0, Dhat = Dfv;
  int bD = 0, bN = 0, bS = 0, bfin = 0;
  if (n_s > 0) {
    const double Swv = tot[D + 1], Swwv = tot[D + 2], Srrv = tot[2 * D + 3];
    if (b0 >= 2) {
      sigma2 = fmax(0.0, (Swwv - Swv * Swv / (double)b0) / (double)(b0 - 1));
      trace = fmax(0.0, (Srrv - sr2 / (double)b0) / (double)(b0 - 1));
    }
    Dhat = Dfv + ratio * (Swv + (double)b0 * piv[D]);
    const double A = (double)n_s * sqrt(sigma2) / Dhat;
    const double Bn = (double)n_s * sqrt(trace) / Nnorm;
    double t = p.z_delta * A / p.eps;
    const double b_D = t * t;
    t = p.z_delta * Bn / p.eps;
    const double b_N = t * t;
    double mn = CUDART_INF;
    bool nan = false;
#pragma unroll
    for (int jj = 0; jj < 15; ++jj) {
      const double c = p.z1[jj] * A + p.z2[jj] * Bn;
      const double c2 = c * c;
      if (c2 != c2) nan = true;
      mn = fmin(mn, c2);
    }
    const double b_S = nan ? CUDART_NAN : 4.0 / (p.eps * p.eps) * mn;
    bD = ceil_sat(b_D); bN = ceil_sat(b_N); bS = ceil_sat(b_S);
    const double bx = p.mode == 1 ? b_D : (p.mode == 2 ? b_N : b_S);
    if (p.force_budget >= 0) bfin = min(p.force_budget, n_s);
    else {
      if (!isfinite(bx)) atomicOr(p.status, VATTN_STATUS_NONFINITE);
      bfin = min(max(ceil_sat(bx), b0), n_s);
    }
  }
  meta.b = bfin;
  if (p.dbg.budgets) {
    int* o = p.dbg.budgets + bh * 4;
    o[0] = bD; o[1] = bN; o[2] = bS; o[3] = bfin;
  }
  if (p.dbg.stats) {
    double* o = p.dbg.stats + bh * 8;
    o[0] = Dfv; o[1] = sigma2; o[2] = trace; o[3] = Dhat; o[4] = Nnorm; o[5] = (double)n_s; o[6] = (double)b0; o[7] = m;
  }
}

}  // namespace

cudaError_t launch_stats(const Prob& p, cudaStream_t s) {
  dim3 grid(p.stat_splits, p.Hq, p.B), block(NT);
  if (p.dtype == VATTN_DTYPE_BF16) {
    if (p.D == 128) k_stats<bf16_t, 128><<<grid, block, 0, s>>>(p);
    else k_stats<bf16_t, 64><<<grid, block, 0, s>>>(p);
  } else {
    if (p.D == 128) k_stats<float, 128><<<grid, block, 0, s>>>(p);
    else k_stats<float, 64><<<grid, block, 0, s>>>(p);
  }
  return cudaGetLastError();
}
