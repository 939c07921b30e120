// Dense attention over the paged cache (full SDPA, Sec. 3 of the paper), FlashDecoding style: the
// context is split over CTAs, every CTA keeps an online softmax for the (up to 4) query heads of a
// KV-head group, and the last CTA of a group merges the split partials in a fixed order.
// This is the comparison kernel: the latency the sparse step has to beat on the same cache.
#include <math.h>
#include <string.h>
#include "vattn_internal.cuh"

namespace {

constexpr int WARPS = 4;
constexpr int NT = WARPS * 32;

template <typename T, int D>
__global__ void __launch_bounds__(NT) k_dense(const Prob p) {
  constexpr int EPL = Elem<T>::EPL, LPR = D / EPL, RPI = 32 / LPR, ITERS = 16 / RPI, NV = ITERS * 4;
  __shared__ float s_acc[WARPS][4][D];
  __shared__ float s_m[WARPS][4], s_l[WARPS][4];
  __shared__ int is_last;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int split = blockIdx.x, b = blockIdx.z;
  const int GC = (p.G + 3) >> 2;
  const int g = blockIdx.y / GC, hc = blockIdx.y % GC;
  const int S = p.dense_splits;
  const int n = clamped_len(p, b);
  const int r = lane / LPR, j = lane % LPR;
  const int npages = (n + 15) >> 4;
  const int pps = (npages + S - 1) / S;
  const int pg_begin = min(npages, split * pps), pg_end = min(npages, pg_begin + pps);

  float qv[4][EPL];
#pragma unroll
  for (int hh = 0; hh < 4; ++hh) {
    const int hl = hc * 4 + hh;
    if (hl < p.G) Elem<T>::load(reinterpret_cast<const T*>(p.q) + q_row(p, b, g * p.G + hl) + j * EPL, qv[hh]);
    else {
#pragma unroll
      for (int e = 0; e < EPL; ++e) qv[hh][e] = 0.f;
    }
  }
  int nh2[2];                                  // tokens that this lane's two heads see (query tokens of one call differ)
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const int hl = hc * 4 + 2 * (j & 1) + e;
    nh2[e] = hl < p.G ? head_len(p, b, g * p.G + hl) : n;
  }
  float m_run[4], l_lane[2] = {0.f, 0.f}, acc[4][EPL];
#pragma unroll
  for (int hh = 0; hh < 4; ++hh) {
    m_run[hh] = -INFINITY;
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[hh][e] = 0.f;
  }

  for (int pg = pg_begin + warp; pg < pg_end; pg += WARPS) {
    const int tok0 = pg << 4;
    const T* kbase = row_ptr<T>(p, p.kc, b, g, tok0);
    const T* vbase = row_ptr<T>(p, p.vc, b, g, tok0);
    float sacc[NV];
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
      float x[EPL];
      Elem<T>::load(kbase + (long long)(it * RPI + r) * p.st + j * EPL, x);
#pragma unroll
      for (int hh = 0; hh < 4; ++hh) {
        float a = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) a = fmaf(qv[hh][e], x[e], a);
        sacc[it * 4 + hh] = a;
      }
    }
    int width = NV;
#pragma unroll
    for (int mask = LPR / 2; mask >= 1; mask >>= 1) {
      const int half = width >> 1;
      const bool upper = (j & mask) != 0;
#pragma unroll
      for (int v = 0; v < NV / 2; ++v) {
        if (v < half) {
          const float send = upper ? sacc[v] : sacc[v + half];
          const float keep = upper ? sacc[v + half] : sacc[v];
          sacc[v] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, mask);
        }
      }
      width = half;
    }
    // lane (r, j): token (j>>1)*RPI + r, heads 2(j&1)+{0,1}
    const int tok_l = tok0 + (j >> 1) * RPI + r;
    float sv[2], pm[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) { sv[e] = tok_l < nh2[e] ? p.scale * sacc[e] : -INFINITY; pm[e] = sv[e]; }
#pragma unroll
    for (int mask = 2; mask < 32; mask <<= 1) {
      pm[0] = fmaxf(pm[0], __shfl_xor_sync(0xFFFFFFFFu, pm[0], mask));
      pm[1] = fmaxf(pm[1], __shfl_xor_sync(0xFFFFFFFFu, pm[1], mask));
    }
    const float o0 = __shfl_xor_sync(0xFFFFFFFFu, pm[0], 1), o1 = __shfl_xor_sync(0xFFFFFFFFu, pm[1], 1);
    float pmax[4];
    pmax[0] = (j & 1) ? o0 : pm[0]; pmax[1] = (j & 1) ? o1 : pm[1];
    pmax[2] = (j & 1) ? pm[0] : o0; pmax[3] = (j & 1) ? pm[1] : o1;
    float m_new[4];
#pragma unroll
    for (int hh = 0; hh < 4; ++hh) {
      m_new[hh] = fmaxf(m_run[hh], pmax[hh]);
      const float alpha = (m_run[hh] == -INFINITY) ? 0.f : __expf(m_run[hh] - m_new[hh]);
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc[hh][e] *= alpha;
      if ((hh >> 1) == (j & 1)) l_lane[hh & 1] *= alpha;
      m_run[hh] = m_new[hh];
    }
    float pv[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      pv[e] = sv[e] == -INFINITY ? 0.f : __expf(sv[e] - m_new[2 * (j & 1) + e]);
      l_lane[e] += pv[e];
    }
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
      float x[EPL];
      Elem<T>::load(vbase + (long long)(it * RPI + r) * p.st + j * EPL, x);
      if (tok0 + it * RPI + r >= n) {            // tail of the last page: whatever it holds must not count
#pragma unroll
        for (int e = 0; e < EPL; ++e) x[e] = 0.f;
      }
#pragma unroll
      for (int hh = 0; hh < 4; ++hh) {
        const float pw = __shfl_sync(0xFFFFFFFFu, pv[hh & 1], r * LPR + 2 * it + (hh >> 1));
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[hh][e] = fmaf(pw, x[e], acc[hh][e]);
      }
    }
  }
  // warp partial: rows of the different row groups, l over the lanes that hold the same heads
#pragma unroll
  for (int mask = LPR; mask < 32; mask <<= 1)
#pragma unroll
    for (int hh = 0; hh < 4; ++hh)
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc[hh][e] += __shfl_xor_sync(0xFFFFFFFFu, acc[hh][e], mask);
#pragma unroll
  for (int mask = 2; mask < 32; mask <<= 1) {
    l_lane[0] += __shfl_xor_sync(0xFFFFFFFFu, l_lane[0], mask);
    l_lane[1] += __shfl_xor_sync(0xFFFFFFFFu, l_lane[1], mask);
  }
  if (r == 0) {
#pragma unroll
    for (int hh = 0; hh < 4; ++hh)
#pragma unroll
      for (int e = 0; e < EPL; ++e) s_acc[warp][hh][j * EPL + e] = acc[hh][e];
  }
  if (lane < 2) {
    s_l[warp][2 * lane] = l_lane[0]; s_l[warp][2 * lane + 1] = l_lane[1];
    s_m[warp][2 * lane] = lane ? m_run[2] : m_run[0]; s_m[warp][2 * lane + 1] = lane ? m_run[3] : m_run[1];
  }
  __syncthreads();
  // CTA partial -> global: [D] unnormalised sum, m, l per head
  constexpr int NE = dense_rec(D);
  for (int idx = tid; idx < 4 * NE; idx += NT) {
    const int hh = idx / NE, e = idx % NE;
    const int hl = hc * 4 + hh;
    if (hl >= p.G) continue;
    float mc = -INFINITY;
#pragma unroll
    for (int w = 0; w < WARPS; ++w) mc = fmaxf(mc, s_m[w][hh]);
    float val;
    if (e == D) val = mc;
    else {
      val = 0.f;
#pragma unroll
      for (int w = 0; w < WARPS; ++w) {
        const float sc = (s_m[w][hh] == -INFINITY) ? 0.f : __expf(s_m[w][hh] - mc);
        val += sc * (e < D ? s_acc[w][hh][e] : s_l[w][hh]);
      }
    }
    p.dense_part[(((long long)b * p.Hq + g * p.G + hl) * S + split) * NE + e] = val;
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    unsigned* ticket = &p.tickets[2 * p.B * p.Hq + b * p.Hq + blockIdx.y];
    is_last = (atomicAdd(ticket, 1u) == (unsigned)(S - 1));
    if (is_last) *ticket = 0u;                 // every CTA of the group has drawn: ready for the next call
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  for (int idx = tid; idx < 4 * D; idx += NT) {
    const int hh = idx / D, e = idx % D;
    const int hl = hc * 4 + hh;
    if (hl >= p.G) continue;
    const long long bh = (long long)b * p.Hq + g * p.G + hl;
    const float* base = p.dense_part + bh * S * NE;
    float mg = -INFINITY;
    for (int sp = 0; sp < S; ++sp) mg = fmaxf(mg, __ldcg(base + sp * NE + D));
    float num = 0.f, den = 0.f;
    for (int sp = 0; sp < S; ++sp) {
      const float ms = __ldcg(base + sp * NE + D);
      const float sc = (ms == -INFINITY) ? 0.f : __expf(ms - mg);
      num += sc * __ldcg(base + sp * NE + e);
      den += sc * __ldcg(base + sp * NE + D + 1);
    }
    reinterpret_cast<T*>(p.out)[q_row(p, b, g * p.G + hl) + e] = Elem<T>::from_float(den > 0.f ? num / den : 0.f);
  }
}


// ---------------------------------------------------------------------------------------------
// bf16 tensor-core variant.  Same split-KV structure, but every warp streams pages through a ring of
// shared-memory stages (bulk asynchronous copies, mbarrier transaction counts) and both contractions of
// a page run on the tensor cores (mma.sync m16n8k16, fp32 accumulate):
//     S^T[head, token] = q K^T     A = q fragments (heads as M, zero rows above the group size),
//                                  B = K rows read with 16-byte shared loads (k-slots mapped onto d so
//                                      that a thread owns 8 consecutive elements of a row)
//     out[head, dim]  += P V       A = exp(S - m) packed to bf16 straight from the S^T accumulators,
//                                  B = V read with 16-byte shared loads from the page as it lies in the cache
//                                      (one copy per page): a thread takes 8 consecutive dims of its four
//                                      tokens and pairs them up with byte permutes, so column slot (block e,
//                                      column gr) of a 64-dim half stands for dim 8 gr + e and a thread's
//                                      accumulators are 16 consecutive dims (no transposing loads, no padding)
constexpr int DN_WARPS = 6;
constexpr int DN_NST = 2;

__device__ __forceinline__ unsigned prmt(unsigned a, unsigned b, unsigned sel) {
  unsigned r;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}
__device__ __forceinline__ unsigned pack_bf16x2(float lo, float hi) {      // round to nearest even, lo in bits 0..15
  unsigned r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// WIDE: up to 16 heads per CTA (rows 8..15 of the tiles carry heads 8..15: groups of more than 8 heads, as calls
// with several query tokens make them), one CTA per SM with four stages per warp; otherwise 8 heads, two CTAs per
// SM, two stages
template <int D, bool WIDE>
__global__ void __launch_bounds__((WIDE ? 2 : 1) * DN_WARPS * 32) k_dense_mma(const Prob p) {
  constexpr int HS = WIDE ? 16 : 8;            // heads per CTA
  constexpr int NW = (WIDE ? 2 : 1) * DN_WARPS; // warps per CTA
  constexpr int NST = DN_NST;
  constexpr int NC = D / 32;                   // 32-element chunks of a K row
  constexpr int ROWB = D * 2, KPAGE = 16 * ROWB;
  constexpr int STAGE = 2 * KPAGE;             // a K page and a V page
  constexpr int NH = D / 64;                   // 64-dim halves of a V row
  constexpr int NB = D / 8;                    // 8-dim column blocks of the output
  constexpr int NE = dense_rec(D);
  extern __shared__ __align__(128) unsigned char smem_dyn[];
  __shared__ float s_m[NW][HS], s_l[NW][HS];
  __shared__ int is_last;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
  const int gr = lane >> 2, t = lane & 3;
  unsigned char* ring = smem_dyn + (size_t)warp * NST * STAGE;
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem_dyn + (size_t)NW * NST * STAGE) + warp * NST;
  float* s_acc = reinterpret_cast<float*>(smem_dyn);          // [NW][HS][D], reuses the rings after the main loop
  float* g_m = s_acc + NW * HS * D;                     // [HS][128] the merge's split maxima, [HS][128] weights,
  float* g_sc = g_m + HS * 128;                               // [HS] denominators: behind the partials, also in the rings
  float* g_den = g_sc + HS * 128;

  const int split = blockIdx.x, b = blockIdx.z, SG = gridDim.x;
  const int GC = (p.G + HS - 1) / HS;
  const int g = blockIdx.y / GC, hc = blockIdx.y % GC;
  const int h0 = g * p.G + hc * HS, nh = min(HS, p.G - hc * HS);
  const int n = clamped_len(p, b);
  const int npages = (n + 15) >> 4;
  // a sequence takes the share of the SG splits that its length has of the longest possible one, so every
  // CTA that works gets about the same number of pages whatever the mix of lengths; the others leave
  const int npages_max = max(1, (p.max_seq_len + 15) >> 4);
  const int S = min(SG, max(1, (int)(((long long)SG * npages + npages_max - 1) / npages_max)));
  if (split >= S) return;
  const int wglob = split * NW + warp, wtot = S * NW;
  const int mine = wglob < npages ? (npages - 1 - wglob) / wtot + 1 : 0;
  const bf16_t* kc = reinterpret_cast<const bf16_t*>(p.kc);
  const bf16_t* vc = reinterpret_cast<const bf16_t*>(p.vc);

  if (lane < NST) mbar_init(&bars[lane], 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncwarp();

  int pg_ids = 0;
  auto load_ids = [&](int k_base) {
    const int k = k_base + lane;
    pg_ids = (k < mine) ? page_of(p, b, wglob + k * wtot) : 0;
  };
  const unsigned long long stream_policy = l2_evict_first_policy();
  // whole warp: lane 0 arms the barrier, then one copy per page (lanes 0 and 16), or, when the rows of a
  // page are not contiguous, lanes 0..15 copy one V row each and lanes 16..31 one K row each
  auto issue = [&](int k, int pg) {
    unsigned long long* bar = &bars[k % NST];
    unsigned char* dst = ring + (size_t)(k % NST) * STAGE;
    const long long off = (long long)pg * p.sb + (long long)g * p.sh;
    if (lane == 0) {
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_expect_tx(bar, 2 * KPAGE);
    }
    __syncwarp();
    // K and V are read once: evict-first in L2
    if (p.st == D) {
      if (lane == 0) bulk_g2s_stream(dst + KPAGE, vc + off, KPAGE, bar, stream_policy);
      else if (lane == 16) bulk_g2s_stream(dst, kc + off, KPAGE, bar, stream_policy);
    } else if (lane < 16) bulk_g2s_stream(dst + KPAGE + lane * ROWB, vc + off + (long long)lane * p.st, ROWB, bar, stream_policy);
    else bulk_g2s_stream(dst + (lane - 16) * ROWB, kc + off + (long long)(lane - 16) * p.st, ROWB, bar, stream_policy);
  };
  load_ids(0);
  for (int k = 0; k < min(NST, mine); ++k) issue(k, __shfl_sync(0xFFFFFFFFu, pg_ids, k));
  // q as the A operand: head (h0 + gr) in rows 0..7; rows 8..15 zero, or heads h0 + 8 + gr (WIDE)
  uint4 aq[NC], aq2[WIDE ? NC : 1];
#pragma unroll
  for (int c = 0; c < NC; ++c) {
    aq[c] = make_uint4(0u, 0u, 0u, 0u);
    if (gr < nh)
      aq[c] = *reinterpret_cast<const uint4*>(reinterpret_cast<const bf16_t*>(p.q) + q_row(p, b, h0 + gr) + c * 32 + t * 8);
    if (WIDE) {
      aq2[c] = make_uint4(0u, 0u, 0u, 0u);
      if (8 + gr < nh)
        aq2[c] = *reinterpret_cast<const uint4*>(reinterpret_cast<const bf16_t*>(p.q) + q_row(p, b, h0 + 8 + gr) + c * 32 + t * 8);
    }
  }
  constexpr int NHT = WIDE ? 2 : 1;            // heads per thread: gr, and 8 + gr
  int n_h[NHT];                                // tokens that the head sees (query tokens of one call differ)
  float m_run[NHT], l_run[NHT];                // l is this lane's share
  float acc[NHT][NB][2];
#pragma unroll
  for (int x = 0; x < NHT; ++x) {
    n_h[x] = 8 * x + gr < nh ? head_len(p, b, h0 + 8 * x + gr) : n;
    m_run[x] = -INFINITY; l_run[x] = 0.f;
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) { acc[x][nb][0] = 0.f; acc[x][nb][1] = 0.f; }
  }
  bool failed = false;

  for (int k = 0; k < mine; ++k) {
    const int s = k % NST;
    if (!mbar_wait(&bars[s], (unsigned)(k / NST) & 1u)) { failed = true; break; }
    unsigned char* stg = ring + (size_t)s * STAGE;
    const int tok0 = (wglob + k * wtot) << 4;
    if (tok0 + 16 > n) {                       // last page: rows beyond n may hold anything; clear their V
      for (int r = n - tok0; r < 16; ++r)
        for (int c = lane; c < ROWB / 4; c += 32) reinterpret_cast<unsigned*>(stg + KPAGE + r * ROWB)[c] = 0u;
      __syncwarp();
    }
    // S^T for tokens 0..7 (sa) and 8..15 (sb): c[0], c[1] are head gr, c[2], c[3] head 8 + gr (WIDE)
    float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      const uint4 klo = *reinterpret_cast<const uint4*>(stg + gr * ROWB + c * 64 + t * 16);
      const uint4 khi = *reinterpret_cast<const uint4*>(stg + (gr + 8) * ROWB + c * 64 + t * 16);
      mma_bf16_16816(sa, aq[c].x, WIDE ? aq2[WIDE ? c : 0].x : 0u, aq[c].y, WIDE ? aq2[WIDE ? c : 0].y : 0u, klo.x, klo.y);
      mma_bf16_16816(sa, aq[c].z, WIDE ? aq2[WIDE ? c : 0].z : 0u, aq[c].w, WIDE ? aq2[WIDE ? c : 0].w : 0u, klo.z, klo.w);
      mma_bf16_16816(sb, aq[c].x, WIDE ? aq2[WIDE ? c : 0].x : 0u, aq[c].y, WIDE ? aq2[WIDE ? c : 0].y : 0u, khi.x, khi.y);
      mma_bf16_16816(sb, aq[c].z, WIDE ? aq2[WIDE ? c : 0].z : 0u, aq[c].w, WIDE ? aq2[WIDE ? c : 0].w : 0u, khi.z, khi.w);
    }
    // this thread: heads gr (and 8 + gr), tokens tok0 + {2t, 2t+1, 8+2t, 9+2t}
    const int tk[4] = {tok0 + 2 * t, tok0 + 2 * t + 1, tok0 + 8 + 2 * t, tok0 + 9 + 2 * t};
    float alpha[NHT];
    unsigned pa[NHT][2];                       // exp(S - m) of tokens 2t, 2t+1 and of 8+2t, 9+2t, packed
#pragma unroll
    for (int x = 0; x < NHT; ++x) {
      float sc[4] = {sa[2 * x], sa[2 * x + 1], sb[2 * x], sb[2 * x + 1]};
      float mx = -INFINITY;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        sc[e] = (tk[e] < n_h[x]) ? p.scale * sc[e] : -INFINITY;
        mx = fmaxf(mx, sc[e]);
      }
      mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 2));
      const float m_new = fmaxf(m_run[x], mx);   // (-inf while the head has seen none of its tokens)
      alpha[x] = (m_run[x] == -INFINITY) ? 0.f : __expf(m_run[x] - m_new);
      float pr[4], psum = 0.f;
#pragma unroll
      for (int e = 0; e < 4; ++e) { pr[e] = sc[e] == -INFINITY ? 0.f : __expf(sc[e] - m_new); psum += pr[e]; }
      l_run[x] = l_run[x] * alpha[x] + psum;
      m_run[x] = m_new;
      pa[x][0] = pack_bf16x2(pr[0], pr[1]); pa[x][1] = pack_bf16x2(pr[2], pr[3]);
    }
    // out += P V: this thread's tokens 2t, 2t+1 (k slots of pa[.][0]) and 8+2t, 9+2t (pa[.][1]), 8 dims at a time
    const unsigned char* vrow = stg + KPAGE + (2 * t) * ROWB + gr * 16;
#pragma unroll
    for (int hf = 0; hf < NH; ++hf) {
      const uint4 v0 = *reinterpret_cast<const uint4*>(vrow + hf * 128);
      const uint4 v1 = *reinterpret_cast<const uint4*>(vrow + ROWB + hf * 128);
      const uint4 v2 = *reinterpret_cast<const uint4*>(vrow + 8 * ROWB + hf * 128);
      const uint4 v3 = *reinterpret_cast<const uint4*>(vrow + 9 * ROWB + hf * 128);
      const unsigned w0[4] = {v0.x, v0.y, v0.z, v0.w}, w1[4] = {v1.x, v1.y, v1.z, v1.w};
      const unsigned w2[4] = {v2.x, v2.y, v2.z, v2.w}, w3[4] = {v3.x, v3.y, v3.z, v3.w};
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const unsigned sel = (e & 1) ? 0x7632u : 0x5410u;
        const unsigned b0 = prmt(w0[e >> 1], w1[e >> 1], sel), b1 = prmt(w2[e >> 1], w3[e >> 1], sel);
        const int nb = hf * 8 + e;
        float c0[4] = {acc[0][nb][0] * alpha[0], acc[0][nb][1] * alpha[0], WIDE ? acc[NHT - 1][nb][0] * alpha[NHT - 1] : 0.f,
                       WIDE ? acc[NHT - 1][nb][1] * alpha[NHT - 1] : 0.f};
        mma_bf16_16816(c0, pa[0][0], WIDE ? pa[NHT - 1][0] : 0u, pa[0][1], WIDE ? pa[NHT - 1][1] : 0u, b0, b1);
        acc[0][nb][0] = c0[0]; acc[0][nb][1] = c0[1];
        if (WIDE) { acc[NHT - 1][nb][0] = c0[2]; acc[NHT - 1][nb][1] = c0[3]; }
      }
    }
    __syncwarp();
    if (k + NST < mine) {
      if (((k + NST) & 31) == 0) load_ids(k + NST);
      issue(k + NST, __shfl_sync(0xFFFFFFFFu, pg_ids, (k + NST) & 31));
    }
  }
  if (failed) {
    if (lane == 0) atomicOr(p.status, VATTN_STATUS_WAIT_TIMEOUT);
    for (int s = 0; s < NST; ++s) mbar_wait(&bars[s], 0u) || mbar_wait(&bars[s], 1u);
  }
#pragma unroll
  for (int x = 0; x < NHT; ++x) {
    l_run[x] += __shfl_xor_sync(0xFFFFFFFFu, l_run[x], 1);
    l_run[x] += __shfl_xor_sync(0xFFFFFFFFu, l_run[x], 2);
  }
  __syncthreads();                             // every warp is done with its ring: reuse it for the partials
  // accumulator (block 8 hf + e, columns 2t and 2t+1) is dim 64 hf + 8 (2t) + e and 64 hf + 8 (2t+1) + e
#pragma unroll
  for (int x = 0; x < NHT; ++x) {
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
      s_acc[(warp * HS + 8 * x + gr) * D + (nb >> 3) * 64 + 16 * t + (nb & 7)] = acc[x][nb][0];
      s_acc[(warp * HS + 8 * x + gr) * D + (nb >> 3) * 64 + 16 * t + 8 + (nb & 7)] = acc[x][nb][1];
    }
    if (t == 0) { s_m[warp][8 * x + gr] = m_run[x]; s_l[warp][8 * x + gr] = l_run[x]; }
  }
  __syncthreads();
  // CTA partial -> global: [D] unnormalised sums, then m and l, per head; warps in a fixed order
  __shared__ float s_w[NW][HS];          // weight of warp w's partial inside the CTA's
  if (tid < HS) {
    float mc = -INFINITY;
#pragma unroll
    for (int w = 0; w < NW; ++w) mc = fmaxf(mc, s_m[w][tid]);
    float lc = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
      const float sc = (s_m[w][tid] == -INFINITY) ? 0.f : __expf(s_m[w][tid] - mc);
      s_w[w][tid] = sc;
      lc += sc * s_l[w][tid];
    }
    if (tid < nh)
      *reinterpret_cast<float4*>(p.dense_part + (((long long)b * p.Hq + h0 + tid) * SG + split) * NE + D) = make_float4(mc, lc, 0.f, 0.f);
  }
  __syncthreads();
  for (int idx = tid; idx < nh * (D / 4); idx += NW * 32) {
    const int hh = idx / (D / 4), e = (idx % (D / 4)) * 4;
    float4 val = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int w = 0; w < NW; ++w) {
      const float sc = s_w[w][hh];
      const float4 x = *reinterpret_cast<const float4*>(&s_acc[(w * HS + hh) * D + e]);
      val.x += sc * x.x; val.y += sc * x.y; val.z += sc * x.z; val.w += sc * x.w;
    }
    *reinterpret_cast<float4*>(p.dense_part + (((long long)b * p.Hq + h0 + hh) * SG + split) * NE + e) = val;
  }
  // release: the barrier orders every thread's stores before thread 0's fence (cumulative), which orders
  // them before the ticket; acquire: the ticket, a fence, and the barrier before anyone reads the partials
  __syncthreads();
  if (tid == 0) {
    __threadfence();
    unsigned* ticket = &p.tickets[2 * p.B * p.Hq + b * p.Hq + blockIdx.y];
    is_last = (atomicAdd(ticket, 1u) == (unsigned)(S - 1));
    if (is_last) *ticket = 0u;                 // every CTA of the group has drawn: ready for the next call
    __threadfence();
  }
  __syncthreads();
  if (!is_last) return;
  // last CTA of the group.  Two rounds of loads: every split's (m, l) pair; then, per four output
  // elements, the S partials with up to MB of them in flight, added in split order
  constexpr int MB = 20;
  __syncthreads();                             // (the partials in shared memory have been read)
  for (int idx = tid; idx < HS * S; idx += NW * 32) {
    const int hh = idx / S, sp = idx % S;
    if (hh < nh) {
      const float2 ml = __ldcg(reinterpret_cast<const float2*>(p.dense_part + (((long long)b * p.Hq + h0 + hh) * SG + sp) * NE + D));
      g_m[hh * 128 + sp] = ml.x; g_sc[hh * 128 + sp] = ml.y;
    }
  }
  __syncthreads();
  for (int hh = warp; hh < nh; hh += NW) {
    float mg = -INFINITY;
    for (int sp = lane; sp < S; sp += 32) mg = fmaxf(mg, g_m[hh * 128 + sp]);
#pragma unroll
    for (int mk = 16; mk >= 1; mk >>= 1) mg = fmaxf(mg, __shfl_xor_sync(0xFFFFFFFFu, mg, mk));
    float den = 0.f;
    for (int sp0 = 0; sp0 < S; sp0 += 32) {          // fixed order: chunks of 32 splits, lanes in a shuffle tree
      const int sp = sp0 + lane;
      float lv = 0.f;
      if (sp < S) {
        const float ms = g_m[hh * 128 + sp];
        const float scv = (ms == -INFINITY) ? 0.f : __expf(ms - mg);
        lv = scv * g_sc[hh * 128 + sp];
        g_sc[hh * 128 + sp] = scv;
      }
#pragma unroll
      for (int mk = 16; mk >= 1; mk >>= 1) lv += __shfl_xor_sync(0xFFFFFFFFu, lv, mk);
      den += lv;
    }
    if (lane == 0) g_den[hh] = den;
  }
  __syncthreads();
  for (int idx = tid; idx < nh * (D / 4); idx += NW * 32) {
    const int hh = idx / (D / 4), e = (idx % (D / 4)) * 4;
    const long long bh = (long long)b * p.Hq + h0 + hh;
    const float* base = p.dense_part + bh * SG * NE + e;
    float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int sp0 = 0; sp0 < S; sp0 += MB) {
      float4 v[MB];
#pragma unroll
      for (int u = 0; u < MB; ++u)
        v[u] = (sp0 + u < S) ? __ldcg(reinterpret_cast<const float4*>(base + (long long)(sp0 + u) * NE)) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int u = 0; u < MB; ++u) {
        const float scv = (sp0 + u < S) ? g_sc[hh * 128 + sp0 + u] : 0.f;
        num.x += scv * v[u].x; num.y += scv * v[u].y; num.z += scv * v[u].z; num.w += scv * v[u].w;
      }
    }
    const float den = g_den[hh];                  // zero: the head sees no token
    bf16_t* o = reinterpret_cast<bf16_t*>(p.out) + q_row(p, b, h0 + hh) + e;
    o[0] = Elem<bf16_t>::from_float(den > 0.f ? num.x / den : 0.f);
    o[1] = Elem<bf16_t>::from_float(den > 0.f ? num.y / den : 0.f);
    o[2] = Elem<bf16_t>::from_float(den > 0.f ? num.z / den : 0.f);
    o[3] = Elem<bf16_t>::from_float(den > 0.f ? num.w / den : 0.f);
  }
}

template <int D, bool WIDE>
static cudaError_t launch_dense_mma(const Prob& p, cudaStream_t s) {
  constexpr int STAGE = 2 * 16 * D * 2, HS = WIDE ? 16 : 8, NST = DN_NST, NW = (WIDE ? 2 : 1) * DN_WARPS;
  const size_t ring = (size_t)NW * NST * STAGE;
  const size_t accb = ((size_t)NW * HS * D + 2 * HS * 128 + HS) * sizeof(float);
  const size_t smem = (ring > accb ? ring : accb) + NW * NST * 8;
  static size_t have[VATTN_MAXDEV];
  cudaError_t e = optin_smem(k_dense_mma<D, WIDE>, smem, have);
  if (e != cudaSuccess) return e;
  const int GC = (p.G + HS - 1) / HS;
  const int groups = p.B * p.Hkv * GC;
  // Two CTAs fit an SM (registers and shared memory; one of the 16-head kind).  With few groups: as many splits as
  // fill one wave, rounded down (a second, partly filled wave costs a whole CTA's duration).  With many groups (large
  // batches, whose lengths differ): pieces small enough for four to five waves, so the SMs drain evenly.
  const int slots = (WIDE ? 1 : 2) * device_sm_count();
  int S = slots / groups >= 3 ? slots / groups : (9 * slots / 2 + groups - 1) / groups;
  if (S > p.dense_splits) S = p.dense_splits;
  if (S < 1) S = 1;
  dim3 grid(S, p.Hkv * GC, p.B), block(NW * 32);
  k_dense_mma<D, WIDE><<<grid, block, smem, s>>>(p);
  return cudaGetLastError();
}
}  // namespace

cudaError_t launch_dense(const Prob& p, cudaStream_t s, int* launches) {
  if (p.dtype == VATTN_DTYPE_BF16) {
    if (launches) *launches = 1;
    if (p.G > 8) return p.D == 128 ? launch_dense_mma<128, true>(p, s) : launch_dense_mma<64, true>(p, s);
    return p.D == 128 ? launch_dense_mma<128, false>(p, s) : launch_dense_mma<64, false>(p, s);
  } else {
    const int GC = (p.G + 3) / 4;
    const int groups = p.B * p.Hkv * GC;
    Prob pf = p;                                 // about four CTAs per SM
    pf.dense_splits = min(p.dense_splits, max(1, (4 * device_sm_count() + groups - 1) / groups));
    dim3 grid(pf.dense_splits, p.Hkv * GC, p.B), block(NT);
    if (p.D == 128) k_dense<float, 128><<<grid, block, 0, s>>>(pf);
    else k_dense<float, 64><<<grid, block, 0, s>>>(pf);
  }
  if (launches) *launches = 1;
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Dense decode without any caller-provided scratch.
//
// Some callers cannot hand this library a workspace: a serving engine that claimed the whole GPU
// for its KV-cache pool at start-up has nothing left to carve one from, and code on a latency-
// critical path may not call cudaMalloc at all (it synchronises the device).  For them the split
// partials and the "last CTA" tickets of the dense kernel live in the fixed array below, which
// every GPU that loads this library holds until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[VATTN_NOALLOC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices];       // device address of g_noalloc_scratch, per device ordinal
bool g_scratch_ready[kMaxDevices];

// The array's name is only a host-side handle in host code; the address a kernel can use has to be
// asked for, once per device, with that device current.
cudaError_t noalloc_scratch(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (!g_scratch_ready[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_addr[dev] = ptr;
    g_scratch_ready[dev] = true;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}
inline size_t up256(size_t x) { return (x + 255) / 256 * 256; }
}  // namespace

extern "C" int vattn_dense_decode_noalloc(const vattn_shape* shape, float scale, const void* q, const void* k_cache,
                                          const void* v_cache, const int32_t* block_table, const int32_t* seq_lens,
                                          void* out, void* stream) {
  if (!shape || !q || !k_cache || !v_cache || !block_table || !seq_lens || !out) return VATTN_ERR_INVALID_ARG;
  const vattn_shape& s = *shape;
  if (s.batch <= 0 || s.num_q_heads <= 0 || s.num_kv_heads <= 0 || s.max_blocks_per_seq <= 0 || s.num_blocks <= 0 ||
      s.max_seq_len < 0 || s.num_q_heads % s.num_kv_heads != 0 || s.batch > 65535 || s.num_q_heads > 65535)
    return VATTN_ERR_INVALID_ARG;
  if ((s.head_dim != 64 && s.head_dim != 128) || s.block_size != VATTN_BLOCK ||
      (s.dtype != VATTN_DTYPE_FP32 && s.dtype != VATTN_DTYPE_BF16) || s.num_q_heads / s.num_kv_heads > 64 || s.q_len > 1)
    return VATTN_ERR_UNSUPPORTED;
  if ((long long)s.max_seq_len > (long long)s.max_blocks_per_seq * s.block_size) return VATTN_ERR_INVALID_ARG;
  const uintptr_t bits = reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k_cache) |
                         reinterpret_cast<uintptr_t>(v_cache) | reinterpret_cast<uintptr_t>(out);
  if (bits & 15) return VATTN_ERR_INVALID_ARG;
  if (!(scale == scale) || isinf(scale)) return VATTN_ERR_INVALID_ARG;

  // layout inside the fixed array: status word | tickets (must start at zero) | split partials
  const size_t BH = (size_t)s.batch * s.num_q_heads, D = (size_t)s.head_dim;
  const int G = s.num_q_heads / s.num_kv_heads, GC = (G + 3) / 4;
  const size_t groups = (size_t)s.batch * s.num_kv_heads * GC;
  const size_t head_bytes = 256 + up256(3 * BH * sizeof(unsigned));
  int splits = (int)((4 * (size_t)device_sm_count() + groups - 1) / groups);
  splits = splits < 1 ? 1 : (splits > 128 ? 128 : splits);
  while (splits > 1 && head_bytes + BH * splits * dense_rec((int)D) * sizeof(float) > VATTN_NOALLOC_SCRATCH_BYTES) --splits;
  if (head_bytes + BH * splits * dense_rec((int)D) * sizeof(float) > VATTN_NOALLOC_SCRATCH_BYTES)
    return VATTN_ERR_WORKSPACE;     // batch * heads too large for the built-in scratch

  void* base = nullptr;
  if (noalloc_scratch(&base) != cudaSuccess) return VATTN_ERR_CUDA;
  unsigned char* w = static_cast<unsigned char*>(base);
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  Prob p;
  memset(&p, 0, sizeof(p));
  p.B = s.batch; p.Hq = s.num_q_heads; p.Hkv = s.num_kv_heads; p.G = G; p.D = s.head_dim; p.dtype = s.dtype;
  p.Tq = 1; p.G1 = G;
  p.max_blocks = s.max_blocks_per_seq; p.num_blocks = s.num_blocks; p.max_seq_len = s.max_seq_len;
  if (s.kv_stride_block == 0 && s.kv_stride_head == 0 && s.kv_stride_token == 0) {
    p.st = s.head_dim; p.sh = (long long)s.block_size * s.head_dim; p.sb = (long long)s.num_kv_heads * p.sh;
  } else {
    const int epl = s.dtype == VATTN_DTYPE_BF16 ? 8 : 4;
    if (s.kv_stride_block <= 0 || s.kv_stride_head <= 0 || s.kv_stride_token < s.head_dim ||
        s.kv_stride_block % epl || s.kv_stride_head % epl || s.kv_stride_token % epl)
      return VATTN_ERR_INVALID_ARG;
    p.sb = s.kv_stride_block; p.sh = s.kv_stride_head; p.st = s.kv_stride_token;
  }
  p.q = q; p.kc = k_cache; p.vc = v_cache; p.bt = block_table; p.seq_lens = seq_lens; p.out = out;
  p.scale = scale != 0.f ? scale : (float)(1.0 / sqrt((double)s.head_dim));
  p.status = reinterpret_cast<unsigned*>(w);
  p.tickets = reinterpret_cast<unsigned*>(w + 256);
  p.dense_part = reinterpret_cast<float*>(w + head_bytes);
  p.dense_splits = splits;
  // the array keeps whatever the previous call left: the tickets and the status word must be zero again
  if (cudaMemsetAsync(w, 0, head_bytes, st) != cudaSuccess) return VATTN_ERR_CUDA;
  if (launch_dense(p, st, nullptr) != cudaSuccess) return VATTN_ERR_CUDA;
  return VATTN_OK;
}

// Status bits (VATTN_STATUS_*) that the kernels of the last vattn_dense_decode_noalloc call on the current device
// left in the fixed array's first word; waits for `stream`.
extern "C" int vattn_noalloc_last_status(uint32_t* bits, void* stream) {
  if (!bits) return VATTN_ERR_INVALID_ARG;
  void* base = nullptr;
  if (noalloc_scratch(&base) != cudaSuccess) return VATTN_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(bits, base, sizeof(uint32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess) return VATTN_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return VATTN_ERR_CUDA;
  return VATTN_OK;
}
