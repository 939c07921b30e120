// The row kernels: everything that reads K/V rows of the paged cache.
//
//  k_stats  D_f = sum_{I_f} w_i, N_f = sum_{I_f} w_i V[i]                             (Sec. 4.1, N_f and D_f)
//           sum w, sum w^2, sum r, sum r.r over I_bs with r_i = w_i V[i]               (Algorithm 2, get-stats)
//           with w_i = exp(s_i - m) and s_i rescored in fp64 from the K row: everything that decides the integer
//           budget is fp64, so that the same inputs give the same ceil() as a plain fp64 evaluation.  Variances
//           are accumulated around a pivot (the first base-sample row), which removes the cancellation of the
//           one-pass formula and makes a constant population give exactly 0.
//           The last CTA of a head to finish adds the head's partial sums in a fixed order and evaluates the budget
//           b_D, b_N (Corollaries D.2), b_SDPA (Theorem 4.3), b = clamp(ceil(b_X), b0, n_s).
//  k_final  the sampled part of the estimator
//               N = N_f + (n_s/b) sum_{I_dyn} w_i V[i],   D = D_f + (n_s/b) sum_{I_dyn} w_i,   out = N / D
//           (Sec. 4.1; SDPA_{S,p} of Sec. 3 with p = 1 on I_f and p = b/n_s on I_dyn).  I_dyn = the first b residual
//           tokens of the final sample's walk: the part the selection kernel listed, and, for larger budgets,
//           further walk positions evaluated here (or, when b is the whole residual, every residual token).
//
// Both kernels: S CTAs of 8 warps per head.  K/V rows travel global -> shared memory as bulk asynchronous
// copies (cp.async.bulk, one per row, completing on an mbarrier), two 4 KB stages per warp: a warp keeps 8 KB in
// flight, an SM 128 KB or more, without holding rows in registers.  Sums are added in a fixed order (rows of a
// warp, warps of a CTA, CTAs of a head): results are reproducible bit for bit.
#include "vattn_internal.cuh"
#include <math_constants.h>

#ifdef VATTN_PHASE_TICKS
#define DBGT(k) do { TICK_BEGIN(p, 24 + (k)); TICK_END(p, 24 + (k)); } while (0)
#else
#define DBGT(k) do { } while (0)
#endif

namespace {

constexpr int NT = ROW_THREADS;
constexpr int NWARP = NT / 32;
constexpr int STAGE_BYTES = 4096;      // one stage of a warp's row ring
constexpr int WPT = 8;                 // walk positions (or tokens) per thread and round of the final kernel
constexpr int LCAP = NT * WPT;         // rows a CTA of the final kernel lists before its warps stream them
constexpr int STAT_WL = 128;           // rows a warp of the statistics kernel lists before it streams them
constexpr unsigned FULL = 0xFFFFFFFFu;
__host__ __device__ constexpr size_t up16(size_t x) { return (x + 15) / 16 * 16; }

// 16-byte slices of a row held in shared memory
template <typename T> struct Raw;
template <> struct Raw<float> {
  float4 v;
  __device__ __forceinline__ void ld(const void* p) { v = *reinterpret_cast<const float4*>(p); }
  __device__ __forceinline__ float get(int e) const { return e == 0 ? v.x : e == 1 ? v.y : e == 2 ? v.z : v.w; }
};
template <> struct Raw<bf16_t> {
  uint4 v;
  __device__ __forceinline__ void ld(const void* p) { v = *reinterpret_cast<const uint4*>(p); }
  __device__ __forceinline__ float get(int e) const {
    const unsigned w = (e >> 1) == 0 ? v.x : (e >> 1) == 1 ? v.y : (e >> 1) == 2 ? v.z : v.w;
    return __uint_as_float((e & 1) ? (w & 0xFFFF0000u) : (w << 16));
  }
};

__device__ __forceinline__ int ceil_sat(double x) {
  if (!isfinite(x) || x >= 2147483647.0) return 2147483647;
  return (int)ceil(x);
}

// exclusive prefix sum over the CTA of one value per thread; `wtot`: NWARP words nobody touches until the caller's
// next barrier
__device__ __forceinline__ int block_scan_reg_rows(int val, int* wtot, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = val;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int v = __shfl_up_sync(FULL, incl, off);
    if (lane >= off) incl += v;
  }
  if (lane == 31) wtot[warp] = incl;
  __syncthreads();
  const int mine = (lane < NWARP) ? wtot[lane] : 0;
  int winc = mine;
#pragma unroll
  for (int off = 1; off < NWARP; off <<= 1) {
    const int v = __shfl_up_sync(FULL, winc, off);
    if (lane >= off) winc += v;
  }
  total = __shfl_sync(FULL, winc, NWARP - 1);
  const int before = __shfl_sync(FULL, winc - mine, warp);
  return before + incl - val;
}

// per-warp row ring
struct Ring {
  unsigned long long* bar;     // [2]
  unsigned char* stg;          // [2][STAGE_BYTES]
  unsigned issued, consumed;
};

template <typename T, int D>
struct Rows {
  static constexpr int ES = (int)sizeof(T) == 2 ? 2 : 4;
  static constexpr int EPL = Elem<T>::EPL, LPR = D / EPL, RPI = 32 / LPR;
  static constexpr int RWB = D * ES;                    // bytes per row
  static constexpr int RB_KV = STAGE_BYTES / (2 * RWB); // rows per batch when K and V rows travel
  static constexpr int RB_V = STAGE_BYTES / RWB;        // rows per batch of V rows
  static_assert(RB_KV / RPI == 4 && RB_V / RPI == 8 && LPR >= 8, "row-group shapes");

  // request the rows whose physical slots are lph[0..nr) into the next stage
  template <bool WITHK>
  static __device__ __forceinline__ void issue(const Prob& p, Ring& rg, int g, const int* lph, int nr) {
    constexpr int RB = WITHK ? RB_KV : RB_V;
    const int lane = threadIdx.x & 31;
    const unsigned st = rg.issued & 1u;
    unsigned char* dst = rg.stg + st * STAGE_BYTES;
    // the stage was read with ordinary loads a moment ago: order them before the copies that overwrite it
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (lane == 0) mbar_expect_tx(&rg.bar[st], (unsigned)(nr * RWB * (WITHK ? 2 : 1)));
    __syncwarp();
    if (lane < nr) {
      const int ph = lph[lane];
      const long long off = (long long)(ph >> 4) * p.sb + (long long)g * p.sh + (long long)(ph & 15) * p.st;
      if (WITHK) {
        bulk_g2s(dst + lane * RWB, reinterpret_cast<const T*>(p.kc) + off, RWB, &rg.bar[st]);
        bulk_g2s(dst + (RB + lane) * RWB, reinterpret_cast<const T*>(p.vc) + off, RWB, &rg.bar[st]);
      } else {
        bulk_g2s(dst + lane * RWB, reinterpret_cast<const T*>(p.vc) + off, RWB, &rg.bar[st]);
      }
    }
    rg.issued++;
  }
  // wait for the oldest batch in flight; returns its stage (nullptr: the bounded wait ran out)
  static __device__ __forceinline__ const unsigned char* arrive(const Prob& p, Ring& rg) {
    const unsigned st = rg.consumed & 1u, par = (rg.consumed >> 1) & 1u;
    const bool ok = __all_sync(FULL, mbar_wait(&rg.bar[st], par));
    rg.consumed++;
    if (!ok) { if ((threadIdx.x & 31) == 0) atomicOr(p.status, VATTN_STATUS_WAIT_TIMEOUT); return nullptr; }
    return rg.stg + st * STAGE_BYTES;
  }
};

// ---------------------------------------------------------------------------------------------
// k_stats
template <int D>
constexpr size_t stats_smem() {
  return up16((size_t)NWARP * 2 * STAGE_BYTES) + up16((size_t)NWARP * (D + 3) * 8) + up16(D * 8) + up16((D + 1) * 8) +
         up16(2 * D * 4) + up16((NWARP * 2 + 2) * 8) + up16(NWARP * STAT_WL * 4) + 128;
}

template <typename T, int D>
__global__ void __launch_bounds__(NT, 2) k_stats(const Prob p) {
  using R_ = Rows<T, D>;
  constexpr int EPL = R_::EPL, LPR = R_::LPR, RPI = R_::RPI, RWB = R_::RWB, RB = R_::RB_KV;
  constexpr int NE = D + 3;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  unsigned char* sp_ = smem_raw;
  unsigned char* stage = sp_;                                           sp_ += up16((size_t)NWARP * 2 * STAGE_BYTES);
  double* wpart = reinterpret_cast<double*>(sp_);                       sp_ += up16((size_t)NWARP * NE * 8);
  double* qT = reinterpret_cast<double*>(sp_);                          sp_ += up16(D * 8);
  double* piv = reinterpret_cast<double*>(sp_);                         sp_ += up16((D + 1) * 8);
  unsigned char* pivrow = sp_;                                          sp_ += up16(2 * D * 4);
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(sp_); sp_ += up16((NWARP * 2 + 2) * 8);
  int* lph_all = reinterpret_cast<int*>(sp_);                           // [NWARP][STAT_WL] physical slots per warp
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int S = (int)gridDim.x, s = (int)blockIdx.x, bh = (int)blockIdx.y;
  const int b = bh / p.Hq, h = bh % p.Hq, g = h / p.G;
  const int GW = S * NWARP, gw = s * NWARP + warp;
  TICK_BEGIN(p, VATTN_K_STATS);

  // before the wait: the step's inputs only
  const T* qrow = reinterpret_cast<const T*>(p.q) + (long long)bh * D;
  for (int e = tid; e < D; e += NT) qT[(e % EPL) * LPR + e / EPL] = (double)Elem<T>::to_float(qrow[e]);   // element-major per lane
  if (tid < NWARP * 2 + 1) mbar_init(&bars[tid], 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();
  pdl_wait();                                          // the selection kernel is complete: lists, meta
  pdl_trigger();
  DBGT(0);
  const HeadMeta mt = p.meta[bh];
  const int n = mt.n, s0 = mt.s0, l_start = mt.l_start, kk = mt.kk, b0 = mt.b0;
  double* gpart = p.stat_part + ((long long)bh * S + s) * 2 * NE;
  if (n == 0) {
    if (s == 0 && tid == 0) {
      p.budget[bh] = 0;
      if (p.dbg.dyn_cnt) p.dbg.dyn_cnt[bh] = 0;
      if (p.dbg.budgets) for (int e = 0; e < 4; ++e) p.dbg.budgets[bh * 4 + e] = 0;
      if (p.dbg.stats) for (int e = 0; e < 8; ++e) p.dbg.stats[bh * 8 + e] = 0.0;
    }
    return;
  }
  const int n_f = s0 + kk + (n - l_start);
  const int* tkph = p.topk_idx + (long long)bh * 2 * p.npad + p.npad;      // physical slots of I_t
  const int* bsph = p.base_idx + (long long)bh * 2 * p.npad + p.npad;      // physical slots of I_bs
  // pivot of the base-sample sums = the first base-sample row: requested now, used after the deterministic rows
  if (b0 > 0 && tid == 0) {
    const int ph = bsph[0];
    const long long off = (long long)(ph >> 4) * p.sb + (long long)g * p.sh + (long long)(ph & 15) * p.st;
    mbar_expect_tx(&bars[NWARP * 2], 2 * RWB);
    bulk_g2s(pivrow, reinterpret_cast<const T*>(p.kc) + off, RWB, &bars[NWARP * 2]);
    bulk_g2s(pivrow + RWB, reinterpret_cast<const T*>(p.vc) + off, RWB, &bars[NWARP * 2]);
  }
  Ring rg;
  rg.bar = bars + warp * 2;
  rg.stg = stage + (size_t)warp * 2 * STAGE_BYTES;
  rg.issued = rg.consumed = 0;
  int* lph = lph_all + warp * STAT_WL;
  constexpr int WL = STAT_WL;
  const int rsub = lane / LPR, j = lane % LPR;
  const double* qs = qT + j;
  const double md = (double)mt.m;
  // The warps of a CTA are split between the two kinds of rows in proportion to their numbers, so that both kinds
  // stream at the same time (a warp's batches follow each other through its two-stage ring; fewer, longer chains
  // beat two rounds that each pay the first fetch).  Warps [0, wd) take the deterministic rows (sink, I_t, window),
  // warps [wd, 8) the base sample.
  int wd = NWARP;
  if (b0 > 0) {
    wd = (NWARP * n_f + (n_f + b0) / 2) / (n_f + b0);
    wd = wd < 1 ? 1 : (wd > NWARP - 1 ? NWARP - 1 : wd);
  }
  const bool base_w = warp >= wd;
  const int total = base_w ? b0 : n_f;
  const int GWk = S * (base_w ? NWARP - wd : wd), gwk = s * (base_w ? NWARP - wd : wd) + (base_w ? warp - wd : warp);

  double acc[EPL], s1 = 0.0, s2 = 0.0, s3 = 0.0;
  double cw = 0.0, pv[EPL];                            // pivot of the base-sample sums; zero for the deterministic rows
#pragma unroll
  for (int e = 0; e < EPL; ++e) { acc[e] = 0.0; pv[e] = 0.0; }
  bool have_piv = !base_w;

  {
    const int nbat_all = (total + RB - 1) / RB;
    int beta = gwk;                                    // this warp's batches: beta, beta + GWk, ...
#pragma unroll 1
    while (beta < nbat_all) {
      int cnt = 0;
      for (int q_ = 0; q_ < WL / RB && beta < nbat_all; ++q_, beta += GWk) {
        const int rho = beta * RB + lane;
        if (lane < RB && rho < total) {
          int ph;
          if (base_w) ph = bsph[rho];
          else if (rho < s0) ph = page_of(p, b, rho >> 4) * VATTN_BLOCK + (rho & 15);
          else if (rho < s0 + kk) ph = tkph[rho - s0];
          else { const int t2 = l_start + (rho - s0 - kk); ph = page_of(p, b, t2 >> 4) * VATTN_BLOCK + (t2 & 15); }
          lph[cnt + lane] = ph;
        }
        cnt += min(RB, total - beta * RB);
      }
      __syncwarp();
      const int nbat = (cnt + RB - 1) / RB;
      R_::template issue<true>(p, rg, g, lph, min(RB, cnt));
      if (nbat > 1) R_::template issue<true>(p, rg, g, lph + RB, min(RB, cnt - RB));
      if (!have_piv) {
        // the pivot: every row group of the base warps evaluates it from the rows requested above (identical numbers)
        const bool ok = __all_sync(FULL, mbar_wait(&bars[NWARP * 2], 0u));
        if (!ok && lane == 0) atomicOr(p.status, VATTN_STATUS_WAIT_TIMEOUT);
        Raw<T> kr, vr;
        kr.ld(pivrow + j * 16);
        vr.ld(pivrow + RWB + j * 16);
        double dd = 0.0;
#pragma unroll
        for (int e = 0; e < EPL; ++e) dd = fma(qs[e * LPR], (double)kr.get(e), dd);
#pragma unroll
        for (int mask = LPR / 2; mask >= 1; mask >>= 1) dd += __shfl_xor_sync(FULL, dd, mask);
        cw = exp(dd * (double)p.scale - md);
#pragma unroll
        for (int e = 0; e < EPL; ++e) pv[e] = cw * (double)vr.get(e);
        if (s == 0 && warp == wd && rsub == 0) {
          double* gp = p.stat_piv + (long long)bh * (D + 1);
#pragma unroll
          for (int e = 0; e < EPL; ++e) gp[j * EPL + e] = pv[e];
          if (j == 0) gp[D] = cw;
        }
        have_piv = true;
      }
#pragma unroll 1
      for (int k = 0; k < nbat; ++k) {
        const unsigned char* stg = R_::arrive(p, rg);
        const int nr = min(RB, cnt - k * RB);
        if (stg) {
          // w_i = exp(s_i - m) from the K rows (fp64), one exp per lane: lane j of a row group takes row j % 4
          double d[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            Raw<T> kr;
            kr.ld(stg + (rsub + RPI * u) * RWB + j * 16);
            double a2 = 0.0;
#pragma unroll
            for (int e = 0; e < EPL; ++e) a2 = fma(qs[e * LPR], (double)kr.get(e), a2);
#pragma unroll
            for (int mask = LPR / 2; mask >= 1; mask >>= 1) a2 += __shfl_xor_sync(FULL, a2, mask);
            d[u] = a2;
          }
          const int mu = j & 3;
          double mine = d[0];
#pragma unroll
          for (int u = 1; u < 4; ++u) mine = (mu == u) ? d[u] : mine;
          const double wm = exp(mine * (double)p.scale - md);
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const double w = __shfl_sync(FULL, wm, u, LPR);
            const int row = rsub + RPI * u;
            if (row < nr) {
              Raw<T> vr;
              vr.ld(stg + (RB + row) * RWB + j * 16);
              const double dw = w - cw;
              s1 += dw;
              s2 = fma(dw, dw, s2);
#pragma unroll
              for (int e = 0; e < EPL; ++e) {
                const double dr = w * (double)vr.get(e) - pv[e];
                acc[e] += dr;
                s3 = fma(dr, dr, s3);
              }
            }
          }
        }
        __syncwarp();
        // the stage just read is free: request the batch after the next one
        if (k + 2 < nbat) R_::template issue<true>(p, rg, g, lph + (k + 2) * RB, min(RB, cnt - (k + 2) * RB));
      }
    }
  }
  // a base warp without rows still has to publish the pivot when it is the one in charge
  if (!have_piv && s == 0 && warp == wd) {
    const bool ok = __all_sync(FULL, mbar_wait(&bars[NWARP * 2], 0u));
    if (!ok && lane == 0) atomicOr(p.status, VATTN_STATUS_WAIT_TIMEOUT);
    Raw<T> kr, vr;
    kr.ld(pivrow + j * 16);
    vr.ld(pivrow + RWB + j * 16);
    double dd = 0.0;
#pragma unroll
    for (int e = 0; e < EPL; ++e) dd = fma(qs[e * LPR], (double)kr.get(e), dd);
#pragma unroll
    for (int mask = LPR / 2; mask >= 1; mask >>= 1) dd += __shfl_xor_sync(FULL, dd, mask);
    cw = exp(dd * (double)p.scale - md);
    if (rsub == 0) {
      double* gp = p.stat_piv + (long long)bh * (D + 1);
#pragma unroll
      for (int e = 0; e < EPL; ++e) gp[j * EPL + e] = cw * (double)vr.get(e);
      if (j == 0) gp[D] = cw;
    }
  }
  DBGT(1);
  // ---- sums: warp, CTA (fixed order: the deterministic warps, the base-sample warps), out
#pragma unroll
  for (int mask = LPR; mask < 32; mask <<= 1) {
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] += __shfl_xor_sync(FULL, acc[e], mask);
    s1 += __shfl_xor_sync(FULL, s1, mask);
    s2 += __shfl_xor_sync(FULL, s2, mask);
  }
#pragma unroll
  for (int mask = 1; mask < 32; mask <<= 1) s3 += __shfl_xor_sync(FULL, s3, mask);
  if (rsub == 0) {
    double* wp = wpart + warp * NE;
#pragma unroll
    for (int e = 0; e < EPL; ++e) wp[j * EPL + e] = acc[e];
    if (j == 0) { wp[D] = s1; wp[D + 1] = s2; wp[D + 2] = s3; }
  }
  __syncthreads();
  for (int item = tid; item < 2 * NE; item += NT) {
    const int kind = item / NE, e = item % NE;
    double sum = 0.0;
    for (int w = kind ? wd : 0; w < (kind ? NWARP : wd); ++w) sum += wpart[w * NE + e];
    gpart[item] = sum;
  }
  DBGT(2);
  // ------------------------------------------------------------------ budget, by the last CTA of the head
  __threadfence();
  __syncthreads();                                     // (also: `wpart` has been read)
  int* flag = reinterpret_cast<int*>(pivrow);
  if (tid == 0) flag[0] = (atomicAdd(&p.tickets[bh], 1u) == (unsigned)(S - 1));
  __syncthreads();
  if (!flag[0]) { TICK_END(p, VATTN_K_STATS); return; }
  __threadfence();
  double* tot = wpart;                                 // [2][NE] sums over the head's CTAs, in CTA order
  {
    const double* gp = p.stat_part + (long long)bh * S * 2 * NE;
    for (int item = tid; item < 2 * NE; item += NT) {
      double v[VATTN_MAX_SPLITS];                      // all partials of the element at once (one memory round trip)
#pragma unroll
      for (int sp = 0; sp < VATTN_MAX_SPLITS; ++sp) v[sp] = sp < S ? __ldcg(gp + (long long)sp * 2 * NE + item) : 0.0;
      double sum = 0.0;
#pragma unroll
      for (int sp = 0; sp < VATTN_MAX_SPLITS; ++sp) sum += v[sp];                             // fixed order
      tot[item] = sum;
    }
    for (int e = tid; e <= D; e += NT) piv[e] = b0 > 0 ? __ldcg(p.stat_piv + (long long)bh * (D + 1) + e) : 0.0;
  }
  __syncthreads();
  {
    double* det = p.det_sums + (long long)bh * (D + 1);       // N_f, D_f for the final combination
    for (int e = tid; e <= D; e += NT) det[e] = tot[e];
  }
  if (warp == 0) {
    const int n_s = mt.n_s;
    const double* t0 = tot;
    const double* t1 = tot + NE;
    const double Dfv = t0[D];
    const double ratio = (b0 > 0) ? (double)n_s / (double)b0 : 0.0;
    double nn = 0.0, sr2 = 0.0;                        // |N_hat|^2 and sum_j (sum_i r'_ij)^2
    for (int e = lane; e < D; e += 32) {
      const double srj = t1[e];
      const double nh = t0[e] + ratio * (srj + (double)b0 * piv[e]);
      nn = fma(nh, nh, nn);
      sr2 = fma(srj, srj, sr2);
    }
#pragma unroll
    for (int mask = 16; mask >= 1; mask >>= 1) {
      nn += __shfl_xor_sync(FULL, nn, mask);
      sr2 += __shfl_xor_sync(FULL, sr2, mask);
    }
    const double Nnorm = sqrt(nn);
    double sigma2 = 0.0, trace = 0.0, Dhat = Dfv, A = 0.0, Bn = 0.0;
    int bD = 0, bN = 0, bS = 0, bf = 0;
    if (n_s > 0) {
      const double Swv = t1[D], Swwv = t1[D + 1], Srrv = t1[D + 2];
      // lane 0: the denominator chain, lane 1: the numerator chain (one body: variance, square root, division)
      const double sq = lane == 0 ? Swwv : Srrv, lin2 = lane == 0 ? Swv * Swv : sr2;
      double var = 0.0;
      if (b0 >= 2) var = fmax(0.0, (sq - lin2 / (double)b0) / (double)(b0 - 1));
      if (lane == 0) Dhat = Dfv + ratio * (Swv + (double)b0 * piv[D]);
      const double ab = (double)n_s * sqrt(var) / (lane == 0 ? Dhat : Nnorm);
      A = __shfl_sync(FULL, ab, 0);
      Bn = __shfl_sync(FULL, ab, 1);
      sigma2 = __shfl_sync(FULL, var, 0);
      trace = __shfl_sync(FULL, var, 1);
      Dhat = __shfl_sync(FULL, Dhat, 0);
      // lanes 0..14: the split points of b_SDPA; lane 15: b_D; lane 16: b_N (one body: (x / eps)^2)
      double x = CUDART_INF;
      if (lane < 15) x = 2.0 * (p.z1[lane] * A + p.z2[lane] * Bn);
      else if (lane == 15) x = p.z_delta * A;
      else if (lane == 16) x = p.z_delta * Bn;
      x = x / p.eps;
      const double x2 = x * x;
      const bool nan = __any_sync(FULL, lane < 15 && x2 != x2);
      double mn = lane < 15 ? x2 : CUDART_INF;
#pragma unroll
      for (int mask = 16; mask >= 1; mask >>= 1) mn = fmin(mn, __shfl_xor_sync(FULL, mn, mask));
      const double b_D = __shfl_sync(FULL, x2, 15), b_N = __shfl_sync(FULL, x2, 16);
      const double b_S = nan ? CUDART_NAN : mn;
      bD = ceil_sat(b_D); bN = ceil_sat(b_N); bS = ceil_sat(b_S);
      const double bx = p.mode == 1 ? b_D : (p.mode == 2 ? b_N : b_S);
      if (p.force_budget >= 0) bf = min(p.force_budget, n_s);
      else {
        if (!isfinite(bx) && lane == 0) atomicOr(p.status, VATTN_STATUS_NONFINITE);
        bf = min(max(ceil_sat(bx), b0), n_s);
      }
    }
    if (lane == 0) {
      p.budget[bh] = bf;
      if (p.dbg.dyn_cnt) p.dbg.dyn_cnt[bh] = bf;
      if (p.dbg.budgets) {
        int* o = p.dbg.budgets + bh * 4;
        o[0] = bD; o[1] = bN; o[2] = bS; o[3] = bf;
      }
      if (p.dbg.stats) {
        double* o = p.dbg.stats + bh * 8;
        o[0] = Dfv; o[1] = sigma2; o[2] = trace; o[3] = Dhat; o[4] = Nnorm; o[5] = (double)n_s; o[6] = (double)b0;
        o[7] = (double)mt.m;
      }
    }
  }
  DBGT(5);
  TICK_END(p, VATTN_K_STATS);
}

// ---------------------------------------------------------------------------------------------
// k_final
constexpr int FLAT_MAX_HEADS = 4096;   // heads whose work units are dealt out over the whole grid
template <int D>
constexpr size_t final_smem() {
  return up16((size_t)NWARP * 2 * STAGE_BYTES) + up16((size_t)NWARP * (D + 1) * 4) + up16(LCAP * 4) * 2 + up16(VATTN_BANDCAP * 4) +
         up16((NWARP * 2 + 2) * 8) + up16(128 * 4) + up16(16 * 4) + up16((FLAT_MAX_HEADS + 1) * 4) + 128;
}

template <typename T, int D>
__global__ void __launch_bounds__(NT, 2) k_final(const Prob p) {
  using R_ = Rows<T, D>;
  constexpr int EPL = R_::EPL, LPR = R_::LPR, RPI = R_::RPI, RWB = R_::RWB;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  unsigned char* sp_ = smem_raw;
  unsigned char* stage = sp_;                                           sp_ += up16((size_t)NWARP * 2 * STAGE_BYTES);
  float* fw = reinterpret_cast<float*>(sp_);                            sp_ += up16((size_t)NWARP * (D + 1) * 4);
  int* cl_ph = reinterpret_cast<int*>(sp_);                             sp_ += up16(LCAP * 4);       // the CTA's listed rows
  int* cl_sc = reinterpret_cast<int*>(sp_);                             sp_ += up16(LCAP * 4);
  int* vt = reinterpret_cast<int*>(sp_);                                sp_ += up16(VATTN_BANDCAP * 4);
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(sp_); sp_ += up16((NWARP * 2 + 2) * 8);
  int* misc = reinterpret_cast<int*>(sp_);                              sp_ += up16(128 * 4);
  unsigned* rkeys = reinterpret_cast<unsigned*>(sp_);                   sp_ += up16(16 * 4);
  int* upref = reinterpret_cast<int*>(sp_);                             // [BH + 1] units before head hh (flat mode)
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int S = (int)gridDim.x, s = (int)blockIdx.x, bh = (int)blockIdx.y;
  const int BH = p.B * p.Hq;
  const int b = bh / p.Hq, h = bh % p.Hq, g = h / p.G;
  TICK_BEGIN(p, VATTN_K_FINAL);
  if (tid < NWARP * 2) mbar_init(&bars[tid], 1);
  if (tid < 2) walk_keys(p, b, p.rng_head_is_kv ? g : h, 1, tid, rkeys);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();
  pdl_wait();                                          // the statistics kernel (and with it the selection) is complete
  pdl_trigger();
  TICK_BEGIN(p, VATTN_T_BUDGET);

  // ------------------------------------------------------------------ work units
  // The rows the selection kernel listed for head hh, ranks [0, lim_hh), lim = min(b, listed) (nothing when b is the
  // whole residual), are cut into units of U rows, one batch per warp.  Budgets differ a lot between heads, so the
  // units of all heads form one list that the CTAs of the grid walk with a stride (up to 4,096 heads; beyond that a
  // head's units stay with its own CTAs).  Rows beyond the listed ones (rare) are done by the head's own CTAs.
  const bool kv = p.gather_kv != 0;
  const int RB = kv ? R_::RB_KV : R_::RB_V;
  const int U = RB * NWARP;
  const bool flat = BH <= FLAT_MAX_HEADS;
  // (without the flat list a head's units stay with its S CTAs: units of about a 1/S share)
  constexpr int MAXU = 32;                             // most units (partial slots) of listed rows per head
  int ugoal = U;                                       // rows per unit the grid aims at: about one unit per CTA
  auto unit_rows = [&](int lim) -> int {               // rows per unit of a head: a whole number of U, at most MAXU units
    const int nb = (lim + U - 1) / U;
    const int fit = ((nb + MAXU - 1) / MAXU) * U;
    return fit > ugoal ? fit : ugoal;
  };
  auto units_of = [&](int lim) -> int { const int ur = unit_rows(lim); return (lim + ur - 1) / ur; };
  auto lim_of = [&](int hh) -> int {
    const HeadMeta* mh = p.meta + hh;
    const int nn = __ldcg(&mh->n), ns_ = __ldcg(&mh->n_s), li = __ldcg(&mh->dyn_listed);
    const int bb = __ldcg(p.budget + hh);
    if (nn == 0 || bb <= 0 || bb >= ns_) return 0;
    return min(bb, li);
  };
  if (flat) {
    // exclusive prefix of the unit counts (BH <= 4096: 16 heads per thread at most)
    const int per = (BH + NT - 1) / NT;
    int loc = 0, tot1;
    for (int q_ = 0; q_ < per; ++q_) { const int hh = tid * per + q_; if (hh < BH) loc += lim_of(hh); }
    block_scan_reg_rows(loc, misc + 32, tot1);         // listed rows of the whole step
    ugoal = ((tot1 / (S * BH) + U) / U) * U;
    __syncthreads();
    loc = 0;
    for (int q_ = 0; q_ < per; ++q_) { const int hh = tid * per + q_; if (hh < BH) loc += units_of(lim_of(hh)); }
    int run = block_scan_reg_rows(loc, misc + 32, tot1);
    for (int q_ = 0; q_ < per; ++q_) {
      const int hh = tid * per + q_;
      if (hh < BH) { upref[hh] = run; run += units_of(lim_of(hh)); }
    }
    if (tid == 0) upref[BH] = tot1;
    __syncthreads();
  }
  const HeadMeta mt = p.meta[bh];
  const int bfin = __ldcg(p.budget + bh);
  if (!flat) ugoal = (((bfin < mt.dyn_listed ? bfin : mt.dyn_listed) / S + U) / U) * U;
  TICK_END(p, VATTN_T_BUDGET);
  DBGT(8);
  const int my_lim = (mt.n == 0 || bfin <= 0 || bfin >= mt.n_s) ? 0 : min(bfin, mt.dyn_listed);
  const bool whole = mt.n > 0 && bfin > 0 && bfin >= mt.n_s;          // this head's sample is its whole residual
  const bool extend = mt.n > 0 && bfin > my_lim && !whole;            // this head's walk goes on beyond the list
  // partial slots of head hh: one per unit, then one per CTA of the head when it has rows beyond the list
  auto parts_of = [&](int hh_units, bool extra) { return hh_units + (extra ? S : 0); };

  Ring rg;
  rg.bar = bars + warp * 2;
  rg.stg = stage + (size_t)warp * 2 * STAGE_BYTES;
  rg.issued = rg.consumed = 0;
  const int rsub = lane / LPR, j = lane % LPR;
  float facc[EPL], fd = 0.f, qf[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) { facc[e] = 0.f; qf[e] = 0.f; }

  // one partial slot is complete: CTA sums in warp order, the slot, the head's ticket; the last finisher of the head
  // adds the slots in order, scales by n_s/b, adds N_f and D_f and divides
  auto finish_part = [&](int hh, int slot, int nparts) {
#pragma unroll
    for (int mask = LPR; mask < 32; mask <<= 1) {
#pragma unroll
      for (int e = 0; e < EPL; ++e) facc[e] += __shfl_xor_sync(FULL, facc[e], mask);
      fd += __shfl_xor_sync(FULL, fd, mask);
    }
    if (rsub == 0) {
#pragma unroll
      for (int e = 0; e < EPL; ++e) fw[warp * (D + 1) + j * EPL + e] = facc[e];
      if (j == 0) fw[warp * (D + 1) + D] = fd;
    }
#pragma unroll
    for (int e = 0; e < EPL; ++e) facc[e] = 0.f;
    fd = 0.f;
    __syncthreads();
    float* gpart = p.gat_part + ((long long)hh * p.gat_slots + slot) * (D + 1);
    for (int e = tid; e <= D; e += NT) {
      float sum = 0.f;
#pragma unroll
      for (int w = 0; w < NWARP; ++w) sum += fw[w * (D + 1) + e];
      gpart[e] = sum;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) misc[0] = (atomicAdd(&p.tickets[(long long)BH + hh], 1u) == (unsigned)(nparts - 1));
    __syncthreads();
    if (misc[0]) {
      __threadfence();
      const int ns_ = __ldcg(&p.meta[hh].n_s), bb = __ldcg(p.budget + hh);
      const double f = (bb > 0) ? (double)ns_ / (double)bb : 0.0;
      const float* src0 = p.gat_part + (long long)hh * p.gat_slots * (D + 1);
      const double* det = p.det_sums + (long long)hh * (D + 1);
      // every thread requests the partials of its element 16 at a time (one memory round trip each), adds in slot order
      T* o = reinterpret_cast<T*>(p.out) + (long long)hh * D;
      for (int e = tid; e <= D; e += NT) {
        float sum = 0.f;
        for (int sp0 = 0; sp0 < nparts; sp0 += 16) {
          float v[16];
#pragma unroll
          for (int q_ = 0; q_ < 16; ++q_) v[q_] = sp0 + q_ < nparts ? __ldcg(src0 + (long long)(sp0 + q_) * (D + 1) + e) : 0.f;
#pragma unroll
          for (int q_ = 0; q_ < 16; ++q_) sum += v[q_];
        }
        fw[e] = sum;
      }
      __syncthreads();
      const double den = __ldcg(det + D) + f * (double)fw[D];        // D_f + n_s/b * sum w
      for (int e = tid; e < D; e += NT) o[e] = Elem<T>::from_float((float)((__ldcg(det + e) + f * (double)fw[e]) / den));
    }
    __syncthreads();
  };
  // the warps stream the CTA's `cnt` listed rows (cl_ph, cl_sc) of head hh: warp w takes the batches w, w + NWARP, ...
  auto stream_rows = [&](int hh, int cnt) {
    const int gh = (hh % p.Hq) / p.G;
    const float m = __ldcg(&p.meta[hh].m);
    if (kv) Elem<T>::load(reinterpret_cast<const T*>(p.q) + (long long)hh * D + j * EPL, qf);
    const int nbat_all = (cnt + RB - 1) / RB;
    int k = warp;
    if (k < nbat_all) {
      if (kv) R_::template issue<true>(p, rg, gh, cl_ph + k * RB, min(RB, cnt - k * RB));
      else R_::template issue<false>(p, rg, gh, cl_ph + k * RB, min(RB, cnt - k * RB));
    }
#pragma unroll 1
    for (; k < nbat_all; k += NWARP) {
      const int kn = k + NWARP;
      if (kn < nbat_all) {
        if (kv) R_::template issue<true>(p, rg, gh, cl_ph + kn * RB, min(RB, cnt - kn * RB));
        else R_::template issue<false>(p, rg, gh, cl_ph + kn * RB, min(RB, cnt - kn * RB));
      }
      const unsigned char* stg = R_::arrive(p, rg);
      const int nr = min(RB, cnt - k * RB);
      if (stg) {
        if (kv) {
          // K and V rows: the weight of a sampled token is recomputed in fp32 from its K row
          float wmine = 0.f;
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            Raw<T> kr;
            kr.ld(stg + (rsub + RPI * u) * RWB + j * 16);
            float dot = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) dot = fmaf(qf[e], kr.get(e), dot);
#pragma unroll
            for (int mask = LPR / 2; mask >= 1; mask >>= 1) dot += __shfl_xor_sync(FULL, dot, mask);
            if ((j & 3) == u) wmine = dot;
          }
          const float em = expf(p.scale * wmine - m);
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const float ww = __shfl_sync(FULL, em, u, LPR);
            const int row = rsub + RPI * u;
            if (row < nr) {
              Raw<T> vr;
              vr.ld(stg + (R_::RB_KV + row) * RWB + j * 16);
              fd += ww;
#pragma unroll
              for (int e = 0; e < EPL; ++e) facc[e] = fmaf(ww, vr.get(e), facc[e]);
            }
          }
        } else {
          // V rows only; weights from the stored scores (listed with the rows), one exp per lane
          const int myrow = rsub + RPI * (j & 7);
          const float em = (myrow < nr) ? expf(__int_as_float(cl_sc[k * RB + myrow]) - m) : 0.f;
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const float ww = __shfl_sync(FULL, em, u, LPR);
            const int row = rsub + RPI * u;
            if (row < nr) {
              Raw<T> vr;
              vr.ld(stg + row * RWB + j * 16);
              fd += ww;
#pragma unroll
              for (int e = 0; e < EPL; ++e) facc[e] = fmaf(ww, vr.get(e), facc[e]);
            }
          }
        }
      }
      __syncwarp();
    }
  };

  // ------------------------------------------------------------------ (1) the listed rows, unit by unit
  {
    const int ncta = S * BH, cid = bh * S + s;
    const int total_units = flat ? upref[BH] : units_of(my_lim);
#pragma unroll 1
    for (int gu = flat ? cid : s; gu < total_units; gu += flat ? ncta : S) {
      int hh = bh, u = gu;
      if (flat) {
        int lo = 0, hi2 = BH - 1;                      // last head whose first unit is <= gu
        while (lo < hi2) { const int mid = (lo + hi2 + 1) >> 1; if (upref[mid] <= gu) lo = mid; else hi2 = mid - 1; }
        hh = lo; u = gu - upref[hh];
      }
      const int lim = flat ? lim_of(hh) : my_lim;
      const int units = units_of(lim), urows = unit_rows(lim);
      const int bb = __ldcg(p.budget + hh);
      const bool extra = bb > lim;                     // that head also has rows beyond its list (its own CTAs' slots)
      const int* dl = p.dyn_idx + (long long)hh * 3 * p.npad;
      int* ddbg = p.dbg.dyn_idx ? p.dbg.dyn_idx + (long long)hh * p.max_seq_len : nullptr;
      const int r_end = min(lim, (u + 1) * urows);
#pragma unroll 1
      for (int r0 = u * urows; r0 < r_end; r0 += LCAP) {         // rounds of up to LCAP rows
        const int cnt = min(LCAP, r_end - r0);
        for (int x = tid; x < cnt; x += NT) {
          cl_ph[x] = dl[p.npad + r0 + x];
          cl_sc[x] = dl[2 * p.npad + r0 + x];
          if (ddbg) ddbg[r0 + x] = dl[r0 + x];
        }
        __syncthreads();
        DBGT(9);
        stream_rows(hh, cnt);
        __syncthreads();
        DBGT(10);
      }
      finish_part(hh, u, parts_of(units, extra));
      DBGT(11);
    }
  }
  DBGT(12);
  if (mt.n == 0) {
    if (s == 0) {
      T* o = reinterpret_cast<T*>(p.out) + (long long)bh * D;
      for (int e = tid; e < D; e += NT) o[e] = Elem<T>::from_float(0.f);
    }
    TICK_END(p, VATTN_K_FINAL);
    return;
  }
  // ------------------------------------------------------------------ (2) rows beyond the list, by the head's own CTAs
  //   further walk positions, evaluated by all threads (listed <= rank < b < n_s), or every residual token in token
  //   order (b = n_s: no walk needed; every CTA passes over all tokens, so the rank of a token is known everywhere)
  const int my_units = units_of(my_lim);
  if (whole || extend) {
    const int s0 = mt.s0, l_start = mt.l_start;
    for (int c = tid; c < mt.nbt; c += NT) vt[c] = __ldcg(p.vtab + (long long)bh * VATTN_BANDCAP + c);
    __syncthreads();
    const float* sc = p.scores + (long long)bh * p.npad;
    const unsigned* gbitmap = p.bitmap + (long long)bh * p.nwords;
    int* ddbg = p.dbg.dyn_idx ? p.dbg.dyn_idx + (long long)bh * p.max_seq_len : nullptr;
    const Walk wk = make_walk(rkeys, l_start - s0);
    int J = mt.dyn_J, have = whole ? 0 : mt.dyn_listed;
    int tcur = s0;
    bool more = true;
#pragma unroll 1
    while (more) {
      int tokc[WPT]; float svc[WPT];
      int nres = 0;
      const int base = whole ? tcur : J;
      const int end = whole ? l_start : (l_start - s0);
#pragma unroll
      for (int q_ = 0; q_ < WPT; ++q_) {
        tokc[q_] = -1; svc[q_] = 0.f;
        const int x = base + tid * WPT + q_;
        if (x < end) {
          const int tok = whole ? x : s0 + walk_at(wk, x);
          const float sv = __ldg(sc + tok);
          if (!in_topk(mt, vt, gbitmap, tok, sv)) { tokc[q_] = tok; svc[q_] = sv; ++nres; }
        }
      }
      int tot1;
      int rank = have + block_scan_reg_rows(nres, misc + 32, tot1);
      int own = 0;
      unsigned ownm = 0u;
#pragma unroll
      for (int q_ = 0; q_ < WPT; ++q_) {
        if (tokc[q_] >= 0) {
          const bool mine = whole ? ((tokc[q_] >> 7) % S == s) : (rank < bfin && (rank / U) % S == s);   // U rows per CTA in turn
          if (mine) { ownm |= 1u << q_; ++own; if (ddbg) ddbg[rank] = tokc[q_]; }
          ++rank;
        }
      }
      __syncthreads();
      int tot2;
      int pos = block_scan_reg_rows(own, misc + 32, tot2);
#pragma unroll
      for (int q_ = 0; q_ < WPT; ++q_) {
        if ((ownm >> q_) & 1u) {
          const int tok = tokc[q_];
          cl_ph[pos] = page_of(p, b, tok >> 4) * VATTN_BLOCK + (tok & 15);
          cl_sc[pos] = __float_as_int(svc[q_]);
          ++pos;
        }
      }
      have += tot1;
      if (whole) { tcur += NT * WPT; more = tcur < l_start; }
      else { J += NT * WPT; more = have < bfin && J < l_start - s0; }
      __syncthreads();
      stream_rows(bh, tot2);
      __syncthreads();                                 // the CTA's list is free for the next round
    }
    finish_part(bh, my_units + s, parts_of(my_units, true));
  } else if (my_units == 0 && s == 0) {
    // nothing sampled (no residual): the output is the deterministic part alone; one empty slot triggers the division
    finish_part(bh, 0, 1);
  }
  DBGT(13);
  TICK_END(p, VATTN_K_FINAL);
}

}  // namespace

template <typename T, int D>
static cudaError_t launch_rows_t(const Prob& p, cudaStream_t s, bool final_kernel) {
  static size_t have[2][VATTN_MAXDEV];
  if (p.splits < 1 || p.splits > VATTN_MAX_SPLITS) return cudaErrorInvalidValue;
  dim3 grid((unsigned)p.splits, (unsigned)(p.B * p.Hq));
  if (final_kernel) {
    cudaError_t e = optin_smem(k_final<T, D>, final_smem<D>(), have[1]);
    if (e != cudaSuccess) return e;
    return launch_pdl(k_final<T, D>, grid, dim3(NT), final_smem<D>(), s, p);
  }
  cudaError_t e = optin_smem(k_stats<T, D>, stats_smem<D>(), have[0]);
  if (e != cudaSuccess) return e;
  return launch_pdl(k_stats<T, D>, grid, dim3(NT), stats_smem<D>(), s, p);
}
static cudaError_t launch_rows(const Prob& p, cudaStream_t s, bool final_kernel) {
  if (p.dtype == VATTN_DTYPE_BF16) {
    if (p.D == 128) return launch_rows_t<bf16_t, 128>(p, s, final_kernel);
    return launch_rows_t<bf16_t, 64>(p, s, final_kernel);
  }
  if (p.D == 128) return launch_rows_t<float, 128>(p, s, final_kernel);
  return launch_rows_t<float, 64>(p, s, final_kernel);
}
cudaError_t launch_stats(const Prob& p, cudaStream_t s) { return launch_rows(p, s, false); }
cudaError_t launch_final(const Prob& p, cudaStream_t s) { return launch_rows(p, s, true); }
