// Deterministic sums and base-sample statistics.
//
// For each (batch row, query head) the rows of I_f = sink + I_t + window and of the base sample I_bs
// are gathered (K and V), rescored in fp64 and reduced:
//     D_f = sum_{I_f} w_i,  N_f = sum_{I_f} w_i V[i]                       (Sec. 4.1, N_f and D_f)
//     sum w, sum w^2, sum r, sum r.r over I_bs with r_i = w_i V[i]           (Algorithm 2, get-stats)
// with w_i = exp(s_i - m).  Every CTA leaves one partial; the last CTA of a head to finish (a counter) adds them in
// split order and evaluates the budget (Algorithm 2, Theorem 4.3 / Corollaries D.2):
//     sigma^2, Tr(Sigma), D_hat, |N_hat|,  b_D, b_N, b_SDPA,  b = clamp(ceil(b_X), b0, n_s)
// in fp64 (the two square-root / division chains on two lanes, the 15 split points of b_SDPA on 15 lanes).  Heads
// whose I_dyn is a prefix of the part of the walk that the selection kernel listed (the usual case) are then done;
// for the others the same CTA lists the rest of the final sample (Algorithm 1 line 7): it continues the walk from
// where the list ends, or, when b is the whole residual, lists every residual token in token order.
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
  CHECK_SLOT(p, ph, 1);
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


constexpr unsigned FULLMASK = 0xFFFFFFFFu;
constexpr int WPT = 8;                 // walk positions (or tokens) per thread and round of the list extension

__device__ __forceinline__ int ceil_sat(double x) {
  if (!isfinite(x) || x >= 2147483647.0) return 2147483647;
  return (int)ceil(x);
}
__device__ __forceinline__ int block_scan_reg(int val, int* wtot, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = val;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int v = __shfl_up_sync(FULLMASK, incl, off);
    if (lane >= off) incl += v;
  }
  if (lane == 31) wtot[warp] = incl;
  __syncthreads();
  int before = 0;
  total = 0;
#pragma unroll
  for (int w = 0; w < NWARP; ++w) {
    const int t = wtot[w];
    if (w < warp) before += t;
    total += t;
  }
  __syncthreads();
  return before + incl - val;
}

// Budget of head bh from the partials of its CTAs, by the last of them.  tot: [2][D + 3] doubles, piv: [D + 1]
// doubles, scal: [4][MAXS] doubles, misc: [8] ints (shared memory).
__device__ __noinline__ void head_budget(const Prob& p, int b, int h, int bh, double* tot, double* piv, double* scal, int* misc) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int D = p.D, NE = D + 3;
  // ---- everything this function reads from memory is requested up front (one round trip): the head's record,
  //      the pivot, and the partials: thread e adds element e of both kinds in split order, threads 0..3 the scalar
  //      sums (kind 0 = deterministic rows: [D] = D_f; kind 1 = base-sample rows: [D] = Sw, [D+1] = Sww, [D+2] = Srr)
  HeadMeta mt = ld_meta(p.meta + bh);
  const double* src = p.stat_part + (long long)bh * 2 * MAXS * NE;
  const int S0 = p.stat_splits, S1 = p.stat_splits_base;
  double pv = 0.0, pvD = 0.0;
  if (tid < D) pv = __ldcg(p.stat_piv + (long long)bh * (D + 1) + tid);
  if (tid == 0) pvD = __ldcg(p.stat_piv + (long long)bh * (D + 1) + D);
  if (tid < D) {
    double v0[MAXS], v1[MAXS];
#pragma unroll
    for (int sp = 0; sp < MAXS; ++sp) {
      v0[sp] = (sp < S0) ? __ldcg(src + (long long)sp * NE + tid) : 0.0;
      v1[sp] = (sp < S1) ? __ldcg(src + (long long)(MAXS + sp) * NE + tid) : 0.0;
    }
    double a0 = 0.0, a1 = 0.0;
#pragma unroll
    for (int sp = 0; sp < MAXS; ++sp) { a0 += v0[sp]; a1 += v1[sp]; }
    tot[tid] = a0; tot[NE + tid] = a1;
  }
  {                                                  // one scalar partial per thread: D_f of split t, then Sw, Sww, Srr
    const int t1 = tid - S0;
    double v = 0.0;
    if (tid < S0) v = __ldcg(src + (long long)tid * NE + D);
    else if (t1 < 3 * S1) v = __ldcg(src + (long long)(MAXS + t1 / 3) * NE + D + t1 % 3);
    if (tid < S0) scal[tid] = v;
    else if (t1 < 3 * S1) scal[MAXS * (1 + t1 % 3) + t1 / 3] = v;
  }
  // (warp 0) the first 256 marked positions of the final sample's walk array, eight per lane; INT_MAX where none
  int hp[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) hp[i] = warp == 0 ? __ldcg(p.hole_pos + (long long)bh * 2 * VATTN_BANDCAP + i * 32 + lane) : 0;
  const int n_s = mt.n_s, b0 = mt.b0;
  // what does not depend on the sums, computed while they are on their way
  const double ratio = (b0 > 0) ? (double)n_s / (double)b0 : 0.0;
  const double rb0 = b0 > 0 ? 1.0 / (double)b0 : 0.0, rb1 = b0 > 1 ? 1.0 / (double)(b0 - 1) : 0.0;
  double c1 = 0.0, c2 = 0.0;                           // lane's coefficients of A and B
  if (lane < 15) { c1 = 2.0 * p.z1[lane] / p.eps; c2 = 2.0 * p.z2[lane] / p.eps; }
  else if (lane == 15) c1 = p.z_delta / p.eps;
  else if (lane == 16) c2 = p.z_delta / p.eps;
  // the pivot the base-row CTAs used (all of them computed the same numbers; split 0 published them)
  if (tid < D) piv[tid] = b0 > 0 ? pv : 0.0;
  if (tid == 0) piv[D] = b0 > 0 ? pvD : 0.0;
  __syncthreads();
  DBGT(30);
  double* det = p.det_sums + (long long)bh * (D + 1);
  if (warp == 0) {
    const double* t0 = tot;
    const double* t1 = tot + NE;
    double sv = 0.0;                                   // lane k < 4: scalar sum k in split order
    if (lane < 4) {
      const int S = lane == 0 ? S0 : S1;
      for (int sp = 0; sp < S; ++sp) sv += scal[MAXS * lane + sp];
    }
    const double Dfv = __shfl_sync(FULLMASK, sv, 0), sv1 = __shfl_sync(FULLMASK, sv, 1);
    double nn = 0.0, sr2 = 0.0;                        // |N_hat|^2 and sum_j (sum_i r'_ij)^2
    for (int e = lane; e < D; e += 32) {
      const double srj = t1[e];
      const double nh = t0[e] + ratio * (srj + (double)b0 * piv[e]);
      nn = fma(nh, nh, nn);
      sr2 = fma(srj, srj, sr2);
    }
#pragma unroll
    for (int mask = 16; mask >= 1; mask >>= 1) {
      nn += __shfl_xor_sync(FULLMASK, nn, mask);
      sr2 += __shfl_xor_sync(FULLMASK, sr2, mask);
    }
    double sigma2 = 0.0, trace = 0.0, Dhat = Dfv;
    int bD = 0, bN = 0, bS = 0, bf = 0;
    if (n_s > 0) {
      const double Swv = __shfl_sync(FULLMASK, sv, 1), Swwv = __shfl_sync(FULLMASK, sv, 2), Srrv = __shfl_sync(FULLMASK, sv, 3);
      // lane 0: the denominator chain A = n_s sigma / D_hat, lane 1: the numerator chain B = n_s sqrt(Tr) / |N_hat|,
      // both as n_s sqrt(variance / squared norm): one division and one square root deep
      const double sq = lane == 0 ? Swwv : Srrv, lin2 = lane == 0 ? Swv * Swv : sr2;
      double var = 0.0;
      if (b0 >= 2) var = fmax(0.0, (sq - lin2 * rb0) * rb1);
      Dhat = Dfv + ratio * (Swv + (double)b0 * piv[D]);
      const double den2 = lane == 0 ? Dhat * Dhat : nn;
      const double ab = (double)n_s * sqrt(var / den2);
      const double A = __shfl_sync(FULLMASK, ab, 0), Bn = __shfl_sync(FULLMASK, ab, 1);
      sigma2 = __shfl_sync(FULLMASK, var, 0);
      trace = __shfl_sync(FULLMASK, var, 1);
      // lanes 0..14: the split points of b_SDPA; lane 15: b_D; lane 16: b_N (one body: (c1 A + c2 B)^2, the
      // coefficients z / eps prepared while the partials were on their way)
      const double x = c1 * A + c2 * Bn;
      const double x2 = lane <= 16 ? x * x : CUDART_INF;
      const bool nan = __any_sync(FULLMASK, lane < 15 && x2 != x2);
      double mn = lane < 15 ? x2 : CUDART_INF;
#pragma unroll
      for (int mask = 16; mask >= 1; mask >>= 1) mn = fmin(mn, __shfl_xor_sync(FULLMASK, mn, mask));
      const double b_D = __shfl_sync(FULLMASK, x2, 15), b_N = __shfl_sync(FULLMASK, x2, 16);
      const double b_S = nan ? CUDART_NAN : mn;
      bD = ceil_sat(b_D); bN = ceil_sat(b_N); bS = ceil_sat(b_S);
      const double bx = p.mode == 1 ? b_D : (p.mode == 2 ? b_N : b_S);
      if (p.force_budget >= 0) bf = min(p.force_budget, n_s);
      else {
        if (!isfinite(bx) && lane == 0) atomicOr(p.status, VATTN_STATUS_NONFINITE);
        bf = min(max(ceil_sat(bx), b0), n_s);
      }
    }
    // I_dyn = the unmarked entries among the first J of the final sample's walk array, J = b + the marked
    // positions below J (a fixed point, reached in a few steps); budgets beyond the array take a list (below)
    const bool listed = bf > mt.dyn_listed;
    const int nholes = min(max(mt.holes1, 0), VATTN_BANDCAP), nholes2 = min(max(mt.holes2, 0), VATTN_BANDCAP);
    int J = bf;
    if (!listed) {
      const int* hd = p.hole_pos + (long long)bh * 2 * VATTN_BANDCAP;
      const bool far = bf > mt.dyn_J - nholes;           // reaches beyond the walk array: the members there count too
      auto marked_below = [&](int Jq) {                   // (uniform over the warp)
        int c = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) c += __popc(__ballot_sync(FULLMASK, hp[i] < Jq));
        for (int i0 = 256; i0 < nholes; i0 += 32) {
          const int v = i0 + lane < nholes ? __ldcg(hd + i0 + lane) : 0x7FFFFFFF;
          c += __popc(__ballot_sync(FULLMASK, v < Jq));
        }
        if (far)
          for (int i0 = 0; i0 < nholes2; i0 += 32) {
            const int v = i0 + lane < nholes2 ? __ldcg(hd + VATTN_BANDCAP + i0 + lane) : 0x7FFFFFFF;
            c += __popc(__ballot_sync(FULLMASK, v < Jq));
          }
        return c;
      };
      // the least fixed point of J -> b + #{marked < J}: a few steps in the usual case; with nearly every position
      // marked the steps are as short as the runs of marked positions, so after eight a bisection takes over
      bool conv = false;
      for (int it = 0; it < 8; ++it) {
        const int c = marked_below(J);
        if (bf + c == J) { conv = true; break; }
        J = bf + c;
      }
      if (!conv) {
        int lo_ = J, hi_ = far ? mt.l_start - mt.s0 : mt.dyn_J;
        lo_ = min(lo_, hi_);
        while (lo_ < hi_) {
          const int mid = (lo_ + hi_) >> 1;
          if (mid - marked_below(mid) >= bf) hi_ = mid; else lo_ = mid + 1;
        }
        J = lo_;
      }
    }
    if (lane == 0) {
      // the whole residual: every middle token is visited (in token order), members of I_t weigh nothing
      if (!listed && bf >= n_s) J = mt.l_start - mt.s0;
      // nested samples: the base sample's rows are the first b0 rows of I_dyn and their sums are known here (in
      // fp64, from rescored weights): they are folded into the deterministic sums (scaled like the sample), and the
      // gather kernel starts behind them.  Not for lists, nor when the whole residual is visited in token order.
      const bool fold = p.nested_base && !listed && !mt.base_list && bf < n_s && b0 > 0 && mt.base_J <= J;
      misc[4] = bf; misc[5] = listed ? 1 : 0; misc[6] = J; misc[7] = fold ? mt.base_J : 0;
      tot[D] = Dfv; tot[NE + D] = sv1;                 // D_f and the base sample's shifted sum of weights, for the sums below
      p.meta[bh].b = bf;
      if (p.dbg.dyn_cnt) p.dbg.dyn_cnt[bh] = bf;
      if (p.dbg.budgets) {
        int* o = p.dbg.budgets + bh * 4;
        o[0] = bD; o[1] = bN; o[2] = bS; o[3] = bf;
      }
      if (p.dbg.stats) {
        double* o = p.dbg.stats + bh * 8;
        o[0] = Dfv; o[1] = sigma2; o[2] = trace; o[3] = Dhat; o[4] = sqrt(nn); o[5] = (double)n_s; o[6] = (double)b0;
        o[7] = (double)mt.m;
      }
    }
  }
  DBGT(32);
  __syncthreads();
  const int bfin = misc[4];
  {
    // N_f and D_f for the gather kernel's last finisher (with the base sample's share when it is folded in), then
    // the head's record for the gather kernel, then "the budget is known".  The barrier orders every thread's
    // writes before thread 0's release, which is cumulative.
    const int start = misc[7];
    const double f = (start > 0) ? (double)n_s / (double)bfin : 0.0;
    for (int e = tid; e <= D; e += NT)
      det[e] = tot[e] + (start > 0 ? f * (tot[NE + e] + (double)b0 * piv[e]) : 0.0);
    __syncthreads();
    if (tid == 0) {
      p.gat_meta[2 * bh] = make_int4(bfin, n_s, __float_as_int(mt.m), (misc[6] << 1) | misc[5]);
      p.gat_meta[2 * bh + 1] = make_int4(mt.dyn_J, start, 0, 0);
      if (!misc[5])                                    // (a listed head publishes when its list is complete)
        asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p.tickets + bh), "r"(1u) : "memory");
    }
  }
  int* dl = p.dyn_idx + (long long)bh * 3 * p.npad;
  // ---- I_dyn as a list: budgets beyond the walk array (unusual: saturated budgets), and for the debug buffer
  if (bfin > mt.dyn_listed || (p.dbg.dyn_idx && bfin > 0)) {
    __shared__ unsigned rkeys[8];
    if (tid < 2) walk_keys(p, b, h, 1, tid, rkeys);
    __syncthreads();
    const int s0 = mt.s0, l_start = mt.l_start;
    const int* vt = p.vtab + (long long)bh * VATTN_BANDCAP;
    const float* sc = p.scores + (long long)bh * p.npad;
    const unsigned* gbitmap = p.bitmap + (long long)bh * p.nwords;
    const bool whole = bfin >= n_s;                    // every residual token, in token order
    const Walk wk = make_walk(rkeys, l_start - s0);
    int have = 0;
    int cur = whole ? s0 : 0;
    const int end = whole ? l_start : (l_start - s0);
#pragma unroll 1
    while (have < bfin && cur < end) {
      int tokc[WPT];
      int nres = 0;
#pragma unroll
      for (int q_ = 0; q_ < WPT; ++q_) {
        tokc[q_] = -1;
        const int x = cur + tid * WPT + q_;
        if (x < end) {
          const int tok = whole ? x : s0 + walk_at(wk, x);
          if (!in_topk(mt, vt, gbitmap, tok, __ldg(sc + tok))) { tokc[q_] = tok; ++nres; }
        }
      }
      int tot1;
      int rank = have + block_scan_reg(nres, misc, tot1);
#pragma unroll
      for (int q_ = 0; q_ < WPT; ++q_) {
        if (tokc[q_] >= 0) {
          if (rank < bfin) { dl[rank] = tokc[q_]; dl[p.npad + rank] = phys_of(p, b, tokc[q_]); }
          ++rank;
        }
      }
      have += tot1;
      cur += NT * WPT;
    }
  }
  if (misc[5]) {                                       // a listed head: its list is complete now
    __syncthreads();
    if (tid == 0) {
      __threadfence();
      asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p.tickets + bh), "r"(1u) : "memory");
    }
  }
  if (p.dbg.dyn_idx) {
    __syncthreads();
    int* dbg = p.dbg.dyn_idx + (long long)bh * p.max_seq_len;
    for (int i = tid; i < bfin; i += NT) dbg[i] = __ldcg(dl + i);
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(NT, 5) k_stats(const __grid_constant__ Prob p) {
  constexpr int EPL = Elem<T>::EPL, LPR = D / EPL, RPI = 32 / LPR;
  constexpr int NE = D + 3;               // det CTA: N_f[D], D_f;  base CTA: Sr[D], Sw, Sww, Srr
  constexpr int RG = NWARP * RPI;         // row groups per CTA
  __shared__ double part[NWARP][NE];
  __shared__ double piv[D + 1];
  __shared__ double pivT[D];             // the pivot's w*V, element-major per lane: pivT[e * LPR + j]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // grid (S, Hq, 2 B): the deterministic-row CTAs of every head come first in dispatch order (their word is
  // published first), the base-row CTAs follow
  const bool base_cta = (int)blockIdx.z >= p.B;
  const int h = blockIdx.y, b = base_cta ? blockIdx.z - p.B : blockIdx.z, g = h / p.G;
  const int bh = b * p.Hq + h;
  const int S = base_cta ? p.stat_splits_base : p.stat_splits;   // CTAs of this kind per head
  const int split = blockIdx.x;
  const int vx = (base_cta ? MAXS : 0) + split;    // position among the head's 2 MAXS partial slots
  if (split >= S) return;                          // the grid is as wide as the larger of the two split counts
  TICK_BEGIN(p, VATTN_K_STATS);
  pdl_trigger();
  // What a CTA needs of its head comes from the step's inputs (the head's geometry), from the score pass (the
  // largest score) and, for the base sample, from one 64-bit word that the selection kernel publishes when I_t is
  // written and marked in the walk arrays: 2 | base_list << 2 | base_J << 3 | the pivot row's physical slot << 32.  This grid's CTAs
  // were launched after every CTA of that kernel had started (programmatic dependent launch), so the producer of a
  // word is running or done when a CTA here polls it: the wait cannot starve.  It is bounded all the same; when it
  // runs out the CTA falls back to the grid-level dependency wait, which is always sufficient.
  __shared__ unsigned long long s_word;
  __shared__ int s_flag;
  __shared__ int s_misc[8];
  // deterministic-row CTAs wait for "the list of I_t is written" (a 32-bit word, published first), base-row CTAs
  // for the 64-bit word
  const unsigned* fl32 = p.tickets + 4 * p.B * p.Hq + bh;
  if (tid == 0) {
    const unsigned long long v = base_cta ? wait_word64(p.flags64 + bh, VATTN_WORD_SPINS)
                                          : (unsigned long long)wait_word32(fl32, VATTN_WORD_SPINS);
    s_word = v;
  }
  const int n = head_len(p, b, h);
  const Geo geo = head_geometry(p, n);
  const int s0 = geo.s0, l_start = geo.l_start, kk = geo.kk, b0 = geo.b0;
  const float m_f = unord_f32(__ldcg(p.m_ord + bh));
  __syncthreads();
  if (s_word == 0ull) {                            // the bounded wait ran out
    pdl_wait();
    if (tid == 0) s_word = base_cta ? __ldcg(p.flags64 + bh) : 1ull;
    __syncthreads();
  }
  const unsigned long long word = s_word;
  if (base_cta) DBGT(36);
  if (base_cta && split == 0) DBGH(bh, 6);
  const int base_list = (int)((word >> 2) & 1ull), base_J = (int)((word >> 3) & 0x3FFFFFull), word_piv = (int)(word >> 32);
  if (n == 0) {                                    // an empty row: no sums, budget 0
    if (base_cta && split == 0) {
      pdl_wait();
      if (tid == 0) {
        p.gat_meta[2 * bh] = make_int4(0, 0, 0, -1);
        p.gat_meta[2 * bh + 1] = make_int4(0, 0, 0, 0);
        __threadfence();
        asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p.tickets + bh), "r"(1u) : "memory");
        if (p.dbg.dyn_cnt) p.dbg.dyn_cnt[bh] = 0;
        if (p.dbg.budgets) for (int e = 0; e < 4; ++e) p.dbg.budgets[bh * 4 + e] = 0;
        if (p.dbg.stats) for (int e = 0; e < 8; ++e) p.dbg.stats[bh * 8 + e] = 0.0;
      }
    }
    return;
  }
  const int n_f = s0 + kk + (n - l_start);
  // base sample: the unmarked entries among the first base_J of its walk array, or a list of b0 entries
  const int total = base_cta ? (base_list ? b0 : base_J) : n_f;
  const int chunk = (total + S - 1) / S;
  const int r_begin = min(total, split * chunk), r_end = min(total, r_begin + chunk);
  const int* tkph = p.topk_idx + (long long)bh * 2 * p.npad + p.npad;       // physical slots of I_t
  const int* bstok = base_list ? p.base_idx + (long long)bh * 2 * p.npad : p.walk_tok + (long long)bh * 4 * p.npad;
  const int* bsph = bstok + p.npad;                                           // physical slots of the entries
  const int ph0 = phys_of(p, b, 0);
  const double m = (double)m_f;
  const int rsub = lane / LPR, j = lane % LPR;
  const int rg = warp * RPI + rsub;
  const int iters = (r_end - r_begin + RG - 1) / RG;      // uniform over the CTA

  // q in fp64, element-major per lane (qT[e * LPR + j]): read from shared memory where it is used instead of
  // living in 16 registers
  __shared__ double qT[D];
  if (warp == 0 && rsub == 0) {
    float qf[EPL];
    Elem<T>::load(reinterpret_cast<const T*>(p.q) + q_row(p, b, h) + j * EPL, qf);
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
  }
  if (base_cta && b0 > 0) {
    // ---------------------------------------------------------------- base-sample rows, shifted by the pivot
    RowRegs<T> prow;
    const int piv_ph = base_list ? __ldcg(bsph) : word_piv;      // pivot = first base-sample row
    // (the entries are only requested here and looked at one batch later, when the rows are requested: a marked
    // entry, token -1, is a member of I_t, not a sample; its slot is valid all the same)
    int ph_n[UN], tok_n[UN];
    auto fetch = [&](int k0) {
#pragma unroll
      for (int u = 0; u < UN; ++u) {
        const int r = r_begin + rg + (k0 + u) * RG;
        const bool in = (k0 + u < iters) && (r < r_end);
        ph_n[u] = in ? __ldg(bsph + r) : piv_ph;
        tok_n[u] = in ? __ldg(bstok + r) : -1;
      }
    };
    auto issue = [&](RowRegs<T> (&row)[UN], bool (&act)[UN]) {
#pragma unroll
      for (int u = 0; u < UN; ++u) { act[u] = tok_n[u] >= 0; load_row<T, D>(p, g, ph_n[u], j, row[u]); }
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
    DBGT(37);
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
  // ---- the last CTA of the head to arrive here evaluates the budget
  // (the barrier orders every thread's writes before thread 0's fence, which is cumulative; likewise on the way in)
  __syncthreads();
  DBGT(34);
  if (tid == 0) {
    __threadfence();
    s_flag = (atomicAdd(&p.tickets[3 * p.B * p.Hq + bh], 1u) == (unsigned)(p.stat_splits + p.stat_splits_base - 1));
    __threadfence();
  }
  __syncthreads();
  if (base_cta && split == 0) DBGH(bh, 2);              // (one base CTA's rows are done)
  if (s_flag) {
    DBGH(bh, 3);
    // the rest of the list needs the selection kernel's last words (how far it listed the walk): wait for that
    // grid as a whole, which also makes "this grid has completed" imply "the selection kernel has" for the gather
    // kernel behind
    pdl_wait();
    DBGT(35);
    TICK_BEGIN(p, VATTN_T_BUDGET);
    head_budget(p, b, h, bh, &part[0][0], piv, pivT, s_misc);
    DBGH(bh, 4);
    TICK_END(p, VATTN_T_BUDGET);
  }
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
