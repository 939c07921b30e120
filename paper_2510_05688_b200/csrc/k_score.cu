// Score pass: s[b,h,i] = scale * <q[b,h], K[b,g,i]> for every token of the paged cache, the (up to 4)
// query heads of a KV-head group together (the inner products of the SDPA definition, Sec. 3 of the
// paper; Algorithm 1 line 3 ranks tokens by them).  Also keeps, per query head, the running maximum
// score (softmax stabiliser) and, per KV head, max |K element| (used for the rounding-error bound of
// these fp32 scores).
//
// HBM-bound stream over K: a warp owns whole 16-token pages; LPR lanes cover one row with one 16-byte
// load each, so a warp instruction fetches 512 contiguous bytes.  Summation structure (this fixes the
// error bound the select kernel uses): EPL sequential fp32 FMAs per lane, then a log2(LPR)-level
// butterfly that halves the number of live partial sums at every level ("reduce-scatter"), one
// multiply by `scale`: at most 13 roundings.
#include "vattn_internal.cuh"

namespace {

constexpr int PPW = 4;      // pages per warp
constexpr int WARPS = 4;    // warps per CTA
constexpr int TILE = PPW * WARPS * VATTN_BLOCK;

template <typename T, int D>
__global__ void __launch_bounds__(WARPS * 32) k_score(const Prob p) {
  constexpr int EPL = Elem<T>::EPL;
  constexpr int LPR = D / EPL;       // lanes per row
  constexpr int RPI = 32 / LPR;      // rows per warp instruction
  constexpr int ITERS = 16 / RPI;    // instructions per page
  constexpr int NV = ITERS * 4;      // partial sums per lane per page (4 heads)

  const int b = blockIdx.z;
  const int n = clamped_len(p, b);
  const int tile0 = blockIdx.x * TILE;
  if (tile0 >= n) return;
  const int GC = (p.G + 3) >> 2;
  const int g = blockIdx.y / GC, hc = blockIdx.y % GC;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = lane / LPR, j = lane % LPR;

  float qv[4][EPL];
#pragma unroll
  for (int hh = 0; hh < 4; ++hh) {
    const int hl = hc * 4 + hh;
    if (hl < p.G) {
      Elem<T>::load(reinterpret_cast<const T*>(p.q) + ((long long)b * p.Hq + g * p.G + hl) * D + j * EPL, qv[hh]);
    } else {
#pragma unroll
      for (int e = 0; e < EPL; ++e) qv[hh][e] = 0.f;
    }
  }
  float runmax[2] = {-INFINITY, -INFINITY};
  float kmax = 0.f;

  for (int pp = 0; pp < PPW; ++pp) {
    const int tok0 = tile0 + (warp * PPW + pp) * VATTN_BLOCK;
    if (tok0 >= n) break;
    const T* base = row_ptr<T>(p, p.kc, b, g, tok0);
    float acc[NV];
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
      const int t = it * RPI + r;
      float x[EPL];
      Elem<T>::load(base + (long long)t * p.st + j * EPL, x);
      if (tok0 + t < n) {
#pragma unroll
        for (int e = 0; e < EPL; ++e) kmax = fmaxf(kmax, fabsf(x[e]));
      }
#pragma unroll
      for (int hh = 0; hh < 4; ++hh) {
        float a = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) a = fmaf(qv[hh][e], x[e], a);
        acc[it * 4 + hh] = a;
      }
    }
    // butterfly over the LPR lanes of a row; every level halves the live values
    int width = NV;
#pragma unroll
    for (int mask = LPR / 2; mask >= 1; mask >>= 1) {
      const int half = width >> 1;
      const bool upper = (j & mask) != 0;
#pragma unroll
      for (int v = 0; v < NV / 2; ++v) {
        if (v < half) {
          const float send = upper ? acc[v] : acc[v + half];
          const float keep = upper ? acc[v + half] : acc[v];
          acc[v] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, mask);
        }
      }
      width = half;
    }
    // lane (r, j) now holds partial-sum index v = 2j + e: instruction it = j/2, head 2(j&1)+e
    const int tok = tok0 + (j >> 1) * RPI + r;
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int hl = hc * 4 + 2 * (j & 1) + e;
      const float sc = p.scale * acc[e];
      if (tok < n && hl < p.G) {
        p.scores[((long long)b * p.Hq + g * p.G + hl) * p.npad + tok] = sc;
        runmax[e] = fmaxf(runmax[e], sc);
      }
    }
  }
#pragma unroll
  for (int mask = 2; mask < 32; mask <<= 1) {
    runmax[0] = fmaxf(runmax[0], __shfl_xor_sync(0xFFFFFFFFu, runmax[0], mask));
    runmax[1] = fmaxf(runmax[1], __shfl_xor_sync(0xFFFFFFFFu, runmax[1], mask));
  }
#pragma unroll
  for (int mask = 1; mask < 32; mask <<= 1) kmax = fmaxf(kmax, __shfl_xor_sync(0xFFFFFFFFu, kmax, mask));
  if (lane < 2) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int hl = hc * 4 + 2 * lane + e;
      if (hl < p.G && runmax[e] > -INFINITY)
        atomicMax(&p.m_ord[b * p.Hq + g * p.G + hl], ord_f32(runmax[e]));
    }
  }
  if (lane == 0) atomicMax(&p.kabsmax[b * p.Hkv + g], __float_as_uint(kmax));
}

}  // namespace

cudaError_t launch_score(const Prob& p, cudaStream_t s) {
  const int GC = (p.G + 3) / 4;
  dim3 grid((p.max_seq_len + TILE - 1) / TILE, p.Hkv * GC, p.B), block(WARPS * 32);
  if (p.dtype == VATTN_DTYPE_BF16) {
    if (p.D == 128) k_score<bf16_t, 128><<<grid, block, 0, s>>>(p);
    else k_score<bf16_t, 64><<<grid, block, 0, s>>>(p);
  } else {
    if (p.D == 128) k_score<float, 128><<<grid, block, 0, s>>>(p);
    else k_score<float, 64><<<grid, block, 0, s>>>(p);
  }
  return cudaGetLastError();
}
