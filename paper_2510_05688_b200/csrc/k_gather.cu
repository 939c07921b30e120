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

constexpr int NT = ROW_THREADS;
constexpr int NWARP = NT / 32;
constexpr int UNROLL = 4;

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

  for (int r0 = r_begin + warp * RPI; r0 < r_end; r0 += NWARP * RPI * UNROLL) {
    int tok[UNROLL];
    float w[UNROLL];
    float v[UNROLL][EPL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const int r = r0 + u * NWARP * RPI + rsub;
      tok[u] = (r < r_end) ? dyn[r] : -1;
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      if (tok[u] >= 0) {
        Elem<T>::load(row_ptr<T>(p, p.vc, b, g, tok[u]) + j * EPL, v[u]);
        w[u] = sc[tok[u]];
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
  if (!is_last) return;
  __threadfence();

  // last CTA of the head: fixed-order sum of the partials, scale by n_s/b, divide
  const double* det = p.det_sums + (long long)bh * (D + 1);
  const double f = (nb > 0) ? (double)meta.n_s / (double)nb : 0.0;
  double den = det[D];
  {
    float s = 0.f;
    for (int sp = 0; sp < S; ++sp) s += __ldcg(p.gat_part + ((long long)bh * S + sp) * NE + D);
    den += f * (double)s;
  }
  for (int e = tid; e < D; e += NT) {
    float s = 0.f;
    for (int sp = 0; sp < S; ++sp) s += __ldcg(p.gat_part + ((long long)bh * S + sp) * NE + e);
    const double num = det[e] + f * (double)s;
    out[e] = Elem<T>::from_float((float)(num / den));
  }
}

}  // namespace

cudaError_t launch_gather(const Prob& p, cudaStream_t s) {
  dim3 grid(p.gat_splits, p.Hq, p.B), block(NT);
  if (p.dtype == VATTN_DTYPE_BF16) {
    if (p.D == 128) k_gather<bf16_t, 128><<<grid, block, 0, s>>>(p);
    else k_gather<bf16_t, 64><<<grid, block, 0, s>>>(p);
  } else {
    if (p.D == 128) k_gather<float, 128><<<grid, block, 0, s>>>(p);
    else k_gather<float, 64><<<grid, block, 0, s>>>(p);
  }
  return cudaGetLastError();
}
