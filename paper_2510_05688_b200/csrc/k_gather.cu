// Sampled part of the estimator and the final combination (Sec. 4.1 of the paper):
//     N = N_f + (n_s/b) * sum_{I_dyn} w_i V[i],   D = D_f + (n_s/b) * sum_{I_dyn} w_i,   out = N / D
// which is SDPA_{S,p} of Sec. 3 with p = 1 on I_f and p = b/n_s on I_dyn.
//
// HBM-bound row gather: the b sampled V rows of a head (ascending token order, so rows of one page sit
// next to each other) are split over `gat_splits` CTAs; LPR lanes fetch one row with one 16-byte load
// each, several rows in flight per warp.  Weights come from the stored fp32 scores (no K re-read).
// Partials are added in a fixed order by the last CTA of the head, so results are reproducible.
#include "vattn_internal.cuh"

namespace {

constexpr int NT = 128;
constexpr int NWARP = NT / 32;
constexpr int UNROLL = 4;
constexpr int MAXS = 32;         // most split CTAs per head

template <typename T, int D>
__global__ void __launch_bounds__(NT) k_gather(const Prob p) {
  constexpr int EPL = Elem<T>::EPL, LPR = D / EPL, RPI = 32 / LPR;
  constexpr int NE = D + 1;
  __shared__ float part[NWARP][NE];
  __shared__ int is_last;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z, g = h / p.G;
  const int bh = b * p.Hq + h;
  const int S = p.gat_splits;
  DEV_BEGIN(p, 5);
  const HeadMeta meta = p.meta[bh];
  T* out = reinterpret_cast<T*>(p.out) + (long long)bh * D;
  if (meta.n == 0) {
    if (split == 0) for (int e = tid; e < D; e += NT) out[e] = Elem<T>::from_float(0.f);
    return;
  }
  const int nb = meta.b;
  const int chunk = (nb + S - 1) / S;
  const int r_begin = min(nb, split * chunk), r_end = min(nb, r_begin + chunk);
  const int* dyn = p.dyn_idx + (long long)bh * p.npad;
  const float* sc = p.scores + (long long)bh * p.npad;
  const float m = meta.m;
  const int rsub = lane / LPR, j = lane % LPR;

  float acc[EPL], dd = 0.f;
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc[e] = 0.f;

  DEV_MARK(p, 5, 2, bh == 0 && split == 0);
  constexpr int RG = NWARP * RPI;                         // row groups per CTA
  const int rg = warp * RPI + rsub;
  const int iters = (r_end - r_begin + RG - 1) / RG;
  for (int k0 = 0; k0 < iters; k0 += UNROLL) {
    int tok[UNROLL];
    float w[UNROLL];
    float v[UNROLL][EPL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const int r = r_begin + rg + (k0 + u) * RG;
      tok[u] = (k0 + u < iters && r < r_end) ? __ldg(dyn + r) : -1;
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      if (tok[u] >= 0) {
        Elem<T>::load(row_ptr<T>(p, p.vc, b, g, tok[u]) + j * EPL, v[u]);
        w[u] = __ldg(sc + tok[u]);
      } else {
        w[u] = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) v[u][e] = 0.f;
      }
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const float ww = (tok[u] >= 0) ? expf(w[u] - m) : 0.f;
      dd += ww;
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc[e] = fmaf(ww, v[u][e], acc[e]);
    }
  }
  DEV_MARK(p, 5, 3, bh == 0 && split == 0);
#pragma unroll
  for (int mask = LPR; mask < 32; mask <<= 1) {
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] += __shfl_xor_sync(0xFFFFFFFFu, acc[e], mask);
    dd += __shfl_xor_sync(0xFFFFFFFFu, dd, mask);
  }
  if (rsub == 0) {
#pragma unroll
    for (int e = 0; e < EPL; ++e) part[warp][j * EPL + e] = acc[e];
    if (j == 0) part[warp][D] = dd;
  }
  __syncthreads();
  float* gpart = p.gat_part + ((long long)bh * S + split) * NE;
  for (int e = tid; e < NE; e += NT) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < NWARP; ++w) s += part[w][e];
    gpart[e] = s;
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) is_last = (atomicAdd(&p.tickets[p.B * p.Hq + bh], 1u) == (unsigned)(S - 1));
  __syncthreads();
  DEV_MARK(p, 5, 5, bh == 0 && split == 0);
  if (!is_last) { DEV_END(p, 5); return; }
  __threadfence();
  DEV_MARK(p, 5, 6, bh == 0);
#ifdef VATTN_DEV_TIMING
  if (p.devt && tid == 0) atomicMax(&p.devt[5 * 32 + 9], dev_gtime());
#endif

  // last CTA of the head: every thread requests all partials of its element at once (one memory
  // round trip), adds them in split order, scales by n_s/b and divides
  __shared__ float s_den;
  const double* det = p.det_sums + (long long)bh * (D + 1);
  const double f = (nb > 0) ? (double)meta.n_s / (double)nb : 0.0;
  const float* src0 = p.gat_part + (long long)bh * S * NE;
  float num_s[(D + NT - 1) / NT];
#pragma unroll
  for (int it = 0; it < (D + NT - 1) / NT; ++it) {
    const int e = tid + it * NT;
    float v[MAXS];
#pragma unroll
    for (int sp = 0; sp < MAXS; ++sp) v[sp] = (sp < S && e < D) ? __ldcg(src0 + (long long)sp * NE + e) : 0.f;
    float s = 0.f;
#pragma unroll
    for (int sp = 0; sp < MAXS; ++sp) s += v[sp];
    num_s[it] = s;
  }
  if (warp == 0) {                                            // the denominator: lane sp holds split sp
    float v = (lane < S) ? __ldcg(src0 + (long long)lane * NE + D) : 0.f;
    float s = 0.f;
#pragma unroll
    for (int sp = 0; sp < MAXS; ++sp) s += __shfl_sync(0xFFFFFFFFu, v, sp);
    if (lane == 0) s_den = s;
  }
  __syncthreads();
  DEV_MARK(p, 5, 7, bh == 0);
#ifdef VATTN_DEV_TIMING
  if (p.devt && tid == 0) atomicMax(&p.devt[5 * 32 + 8], dev_gtime());
#endif
  const double den = det[D] + f * (double)s_den;
#pragma unroll
  for (int it = 0; it < (D + NT - 1) / NT; ++it) {
    const int e = tid + it * NT;
    if (e < D) out[e] = Elem<T>::from_float((float)((det[e] + f * (double)num_s[it]) / den));
  }
  DEV_END(p, 5);
}

}  // namespace

cudaError_t launch_gather(const Prob& p, cudaStream_t s) {
  dim3 grid(p.gat_splits, p.Hq, p.B), block(NT);
  if (p.gat_splits < 1 || p.gat_splits > MAXS) return cudaErrorInvalidValue;
  if (p.dtype == VATTN_DTYPE_BF16) {
    if (p.D == 128) k_gather<bf16_t, 128><<<grid, block, 0, s>>>(p);
    else k_gather<bf16_t, 64><<<grid, block, 0, s>>>(p);
  } else {
    if (p.D == 128) k_gather<float, 128><<<grid, block, 0, s>>>(p);
    else k_gather<float, 64><<<grid, block, 0, s>>>(p);
  }
  return cudaGetLastError();
}
