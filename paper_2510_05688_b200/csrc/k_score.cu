// Score pass: s[b,h,i] = scale * <q[b,h], K[b,g,i]> for every token of the paged cache, the query heads
// of a KV-head group together (the inner products of the SDPA definition, Sec. 3 of the paper;
// Algorithm 1 line 3 ranks tokens by them).  Also keeps, per query head, the running maximum score
// (softmax stabiliser) and, per KV head, max |K element| (for the rounding-error bound of the scores).
//
// HBM-bound stream over K (every K row is read exactly once).  Two arithmetic paths:
//  * bf16: pages travel into shared memory with bulk asynchronous copies (a 4-stage mbarrier ring per
//    warp) and the [16 tokens x d] x [d x 8 heads] contraction of a page runs on the tensor cores
//    (mma.sync m16n8k16, fp32 accumulate).  A dot product does not care in which order its terms are
//    paired, so the k-slots of the fragment layout are mapped onto d such that each thread owns 8
//    consecutive elements of a row and reads them with one 16-byte shared load.  This removes the
//    CUDA-core FMAs and the cross-lane reduction that made a first version ALU-co-bound.
//  * fp32: CUDA-core FMAs, EPL sequential FMAs per lane and a butterfly that halves the live partial
//    sums at every level (tf32 tensor cores would not keep fp32 accuracy).
//
// The same CTAs also pre-filter the sampling keys: Philox4x32-10 keys of streams 0 and 1 are computed
// for every (token, head) of the tile and tokens whose key is below the stream's bound are appended to
// per-head candidate lists, so the select kernels never run Philox over the whole context
// (uniform-sample of Algorithm 1 line 7 / Algorithm 2 line 1 = the c smallest keys of the residual).
#include "vattn_internal.cuh"

namespace {

constexpr int PPW = 4;      // pages per warp
constexpr int WARPS = 4;    // warps per CTA
constexpr int TILE = PPW * WARPS * VATTN_BLOCK;   // 256 tokens

// ---------------------------------------------------------------------------------------------
// sampling-candidate pre-filter for the tile [tile0, tile0 + TILE) and heads h0 .. h0 + nh - 1
template <int MAXH>
__device__ void emit_candidates(const Prob& p, int b, int g, int h0, int nh, int tile0, int n,
                                uint2 (*s_list)[TILE], unsigned* s_cnt) {
  const int tid = threadIdx.x;
  const Geo geo = head_geometry(p, n);
  if (geo.n_s <= 0) return;                                    // uniform for the CTA
  const unsigned bound0 = cand0_bound(geo);
  for (int i = tid; i < 2 * MAXH; i += WARPS * 32) s_cnt[i] = 0;
  __syncthreads();
  const unsigned c3base = (unsigned)p.step << 1;
  for (int item = tid; item < nh * (TILE / 4); item += WARPS * 32) {
    const int hh = item / (TILE / 4), quad = item % (TILE / 4);
    const int t0 = tile0 + quad * 4;
    if (t0 >= geo.l_start || t0 + 4 <= geo.s0) continue;
    const int hrng = p.rng_head_is_kv ? g : (h0 + hh);
    const unsigned c1 = ((unsigned)b << 16) | (unsigned)hrng;
#pragma unroll
    for (int stream = 0; stream < 2; ++stream) {
      const unsigned bound = stream ? VATTN_CAND1_BOUND : bound0;
      if (bound == 0u) continue;
      const uint4 r = philox4x32_10((unsigned)(t0 >> 2), c1, (unsigned)p.layer, c3base | (unsigned)stream,
                                    p.seed_lo, p.seed_hi);
      const unsigned key[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int tok = t0 + e;
        if (key[e] < bound && tok >= geo.s0 && tok < geo.l_start) {
          const unsigned pos = atomicAdd(&s_cnt[stream * MAXH + hh], 1u);
          s_list[stream * MAXH + hh][pos] = make_uint2(key[e], (unsigned)tok);
        }
      }
    }
  }
  __syncthreads();
  const int warp = tid >> 5, lane = tid & 31;
  for (int l = warp; l < 2 * MAXH; l += WARPS) {
    const int stream = l / MAXH, hh = l % MAXH;
    const unsigned cnt = s_cnt[l];
    if (hh >= nh || cnt == 0) continue;
    const long long bh = (long long)b * p.Hq + h0 + hh;
    unsigned base = 0;
    if (lane == 0) base = atomicAdd(&p.cand_cnt[(long long)stream * p.B * p.Hq + bh], cnt);
    base = __shfl_sync(0xFFFFFFFFu, base, 0);
    uint2* dst = p.cand + ((long long)stream * p.B * p.Hq + bh) * p.cand_cap;
    for (unsigned j = lane; j < cnt; j += 32)
      if (base + j < (unsigned)p.cand_cap) dst[base + j] = s_list[l][j];
  }
}

// ---------------------------------------------------------------------------------------------
// bf16: tensor-core path, up to 8 heads per CTA
// ---------------------------------------------------------------------------------------------
// bf16, streaming variant: every warp owns a ring of NST shared-memory stages and keeps NST pages
// (16 tokens x d, one contiguous slab of the paged cache) in flight with bulk asynchronous copies
// (cp.async.bulk + mbarrier transaction counts); fragments are read back with 16-byte shared loads.
// The copies need no registers while in flight, so an SM holds ~130 KB of outstanding reads with two
// resident CTAs.  A warp walks the pages p = w, w + W, w + 2W, ... of its (batch row, KV head).
constexpr int NST = 4;          // stages per warp
constexpr int CWARPS = 8;       // warps of a CTA that pre-filter sampling keys (two per streaming warp)

// Sampling-candidate pre-filter, run by the CWARPS candidate warps of a CTA: Philox keys of streams 0
// and 1 for every (token, head) of the CTA's pages; tokens whose key is below the stream's bound are
// staged in CTA-wide lists, one per (stream, head), and appended to the global lists every CHUNK pages
// per warp.  Lanes are items (stream, head, token quad); the 4 lanes of a list are adjacent, so the
// positions inside a page come from ballots; one shared-memory atomic per (page, list) reserves the
// range.  Global counters are bumped once per list and flush, which keeps the contended atomics rare.
constexpr int CL = 256;          // staged entries per (stream, head) list of a CTA
constexpr int CHUNK = 4;         // pages per candidate warp between two flushes (CWARPS*CHUNK*16*1/4 = 128 expected)

__device__ __forceinline__ void cand_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(CWARPS * 32) : "memory"); }

__device__ void candidate_warps(const Prob& p, int b, int g, int h0, int nh, int n, int page0, int wtot, int npages,
                                int cw, uint2* clist, unsigned* s_cnt) {
  const int lane = threadIdx.x & 31;
  const Geo geo = head_geometry(p, n);
  if (geo.n_s <= 0) return;                                   // uniform over the CTA
  const unsigned bound0 = cand0_bound(geo);
  const int nitems = 8 * nh, nrounds = (nitems + 31) >> 5;
  const unsigned lmask = 0xFu << (lane & ~3), lt = (1u << lane) - 1u;
  // pages of this CTA: page0 + j * wtot for the streaming warp j % WARPS; candidate warp cw takes the
  // CTA-local page slots cw, cw + CWARPS, ...   (slot s = page page0_cta + (s % WARPS) + (s / WARPS) * wtot)
  const int slots = (npages > page0) ? ((npages - 1 - page0) / wtot + 1) * WARPS : 0;   // upper bound, CTA-uniform
  const int nchunks = (slots + CWARPS * CHUNK - 1) / (CWARPS * CHUNK);
  if (cw * 32 + lane < 16) s_cnt[cw * 32 + lane] = 0u;
  cand_barrier();
  for (int c = 0; c < nchunks; ++c) {
    for (int kk = 0; kk < CHUNK; ++kk) {
      const int slot = (c * CHUNK + kk) * CWARPS + cw;
      const int page = page0 + (slot % WARPS) + (slot / WARPS) * wtot;
      const int tok0 = page << 4;
      if (page >= npages || tok0 >= geo.l_start || tok0 + 16 <= geo.s0) continue;
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        if (r >= nrounds) break;
        const int item = 32 * r + lane;
        const int L = item >> 2, quad = item & 3;
        const int stream = L / nh, hh = L % nh;
        const unsigned bound = (item < nitems) ? (stream ? VATTN_CAND1_BOUND : bound0) : 0u;
        const int t0 = tok0 + quad * 4;
        unsigned key[4] = {0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu};
        if (bound) {
          const int hrng = p.rng_head_is_kv ? g : (h0 + hh);
          const uint4 rr = philox4x32_10((unsigned)(t0 >> 2), ((unsigned)b << 16) | (unsigned)hrng, (unsigned)p.layer,
                                         ((unsigned)p.step << 1) | (unsigned)stream, p.seed_lo, p.seed_hi);
          key[0] = rr.x; key[1] = rr.y; key[2] = rr.z; key[3] = rr.w;
        }
        unsigned bal[4], total = 0u;
        bool hit[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int tok = t0 + e;
          hit[e] = key[e] < bound && tok >= geo.s0 && tok < geo.l_start;
          bal[e] = __ballot_sync(0xFFFFFFFFu, hit[e]) & lmask;
          total += __popc(bal[e]);
        }
        unsigned base = 0u;
        if ((lane & 3) == 0 && total) base = atomicAdd(&s_cnt[L], total);
        base = __shfl_sync(0xFFFFFFFFu, base, lane & ~3);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const unsigned pos = base + __popc(bal[e] & lt);
          if (hit[e] && pos < (unsigned)CL) clist[L * CL + pos] = make_uint2(key[e], (unsigned)(t0 + e));
          base += __popc(bal[e]);
        }
      }
    }
    cand_barrier();
    // flush: candidate warp cw owns lists cw and cw + CWARPS
    for (int L = cw; L < 2 * nh; L += CWARPS) {
      const unsigned raw = s_cnt[L];
      const unsigned cnt = raw < (unsigned)CL ? raw : (unsigned)CL;
      if (raw == 0u) continue;
      const long long slot_g = (long long)(L / nh) * p.B * p.Hq + (long long)b * p.Hq + h0 + (L % nh);
      unsigned gbase = 0u;
      // a list that overflowed its staging area is incomplete: poison the global count so that the select
      // kernels draw from the full context instead
      if (lane == 0) {
        if (raw > (unsigned)CL) { atomicOr(&p.cand_cnt[slot_g], 0x80000000u); gbase = (unsigned)p.cand_cap; }
        else gbase = atomicAdd(&p.cand_cnt[slot_g], cnt);
      }
      gbase = __shfl_sync(0xFFFFFFFFu, gbase, 0);
      uint2* dst = p.cand + slot_g * p.cand_cap;
      for (unsigned j = lane; j < cnt; j += 32)
        if (gbase + j < (unsigned)p.cand_cap) dst[gbase + j] = clist[L * CL + j];
      __syncwarp();
      if (lane == 0) s_cnt[L] = 0u;
    }
    cand_barrier();
  }
}

template <int D>
__global__ void __launch_bounds__((WARPS + CWARPS) * 32) k_score_stream(const Prob p) {
  constexpr int NC = D / 32;
  constexpr int ROWB = D * 2;                 // bytes per row
  constexpr int PAGEB = VATTN_BLOCK * ROWB;   // bytes per (page, KV head) slab
  extern __shared__ __align__(128) unsigned char smem_dyn[];
  const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int role = wid >= WARPS;              // warps 0..3 stream K, warps 4..11 pre-filter sampling keys
  const int cw = wid - WARPS;                 // candidate warp index (role 1)
  const int warp = role ? (cw & (WARPS - 1)) : wid;      // the streaming warp whose pages this warp works on
  unsigned char* ring = smem_dyn + (size_t)warp * NST * PAGEB;
  uint2* clist = reinterpret_cast<uint2*>(smem_dyn + (size_t)WARPS * NST * PAGEB);
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem_dyn + (size_t)WARPS * NST * PAGEB +
                                                                   (size_t)16 * CL * sizeof(uint2)) + warp * NST;
  unsigned* s_cnt = reinterpret_cast<unsigned*>(smem_dyn + (size_t)WARPS * NST * PAGEB + (size_t)16 * CL * sizeof(uint2) +
                                                (size_t)WARPS * NST * 8);
  DEV_BEGIN(p, 1);
  pdl_trigger();
  const int b = blockIdx.z;
  const int n = clamped_len(p, b);
  const int npages = (n + 15) >> 4;
  const int GC = (p.G + 7) >> 3;
  const int g = blockIdx.y / GC, hc = blockIdx.y % GC;
  const int gr = lane >> 2, t = lane & 3;
  const int h0 = g * p.G + hc * 8;
  const int nh = min(8, p.G - hc * 8);
  const int wglob = blockIdx.x * WARPS + warp, wtot = gridDim.x * WARPS;
  const int mine = wglob < npages ? (npages - 1 - wglob) / wtot + 1 : 0;    // pages this warp owns
  if (role == 1) {
#ifdef VATTN_DEV_TIMING
    if (p.devt && lane == 0 && wglob == 0 && blockIdx.y == 0) p.devt[32 + 4] = dev_gtime();
#endif
    candidate_warps(p, b, g, h0, nh, n, blockIdx.x * WARPS, wtot, npages, cw, clist, s_cnt);
#ifdef VATTN_DEV_TIMING
    if (p.devt && lane == 0 && wglob == 0 && blockIdx.y == 0) p.devt[32 + 5] = dev_gtime();
    if (p.devt && lane == 0) atomicMax(&p.devt[32 + 6], dev_gtime());
#endif
    return;
  }
  if (mine == 0) return;                      // streaming warps use no CTA-wide barrier
  const bf16_t* kc = reinterpret_cast<const bf16_t*>(p.kc);

  if (lane < NST) mbar_init(&bars[lane], 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncwarp();

  // page ids of this warp's first 32 pages (lane l holds the l-th); refreshed every 32 pages
  int pg_ids = 0;
  auto load_ids = [&](int k_base) {
    const int k = k_base + lane;
    pg_ids = (k < mine) ? page_of(p, b, wglob + k * wtot) : 0;
  };
  auto issue = [&](int k, int pg) {       // lane 0 only
    unsigned long long* bar = &bars[k % NST];
    unsigned char* dst = ring + (size_t)(k % NST) * PAGEB;
    const bf16_t* src = kc + (long long)pg * p.sb + (long long)g * p.sh;
    mbar_expect_tx(bar, PAGEB);
    if (p.st == D) bulk_g2s(dst, src, PAGEB, bar);
    else
      for (int r = 0; r < VATTN_BLOCK; ++r) bulk_g2s(dst + r * ROWB, src + (long long)r * p.st, ROWB, bar);
  };
  load_ids(0);
  for (int k = 0; k < min(NST, mine); ++k) {
    const int pg = __shfl_sync(0xFFFFFFFFu, pg_ids, k);
    if (lane == 0) issue(k, pg);
  }

  uint4 bq[NC];
#pragma unroll
  for (int c = 0; c < NC; ++c) {
    bq[c] = make_uint4(0u, 0u, 0u, 0u);
    if (gr < nh)
      bq[c] = *reinterpret_cast<const uint4*>(reinterpret_cast<const bf16_t*>(p.q) +
                                              ((long long)b * p.Hq + h0 + gr) * D + c * 32 + t * 8);
  }
  float runmax[2] = {-INFINITY, -INFINITY};
  unsigned kabs = 0u;
  bool failed = false;

  for (int k = 0; k < mine; ++k) {
    const int s = k % NST;
    if (!mbar_wait(&bars[s], (unsigned)(k / NST) & 1u)) { failed = true; break; }
    const unsigned char* stg = ring + (size_t)s * PAGEB;
    const int tok0 = (wglob + k * wtot) << 4;
    float acc[4] = {0.f, 0.f, 0.f, 0.f}, acc1[4] = {0.f, 0.f, 0.f, 0.f};   // two independent MMA chains
    unsigned klo = 0u, khi = 0u;
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      const uint4 alo = *reinterpret_cast<const uint4*>(stg + gr * ROWB + c * 64 + t * 16);
      const uint4 ahi = *reinterpret_cast<const uint4*>(stg + (gr + 8) * ROWB + c * 64 + t * 16);
      mma_bf16_16816(acc, alo.x, ahi.x, alo.y, ahi.y, bq[c].x, bq[c].y);
      mma_bf16_16816(acc1, alo.z, ahi.z, alo.w, ahi.w, bq[c].z, bq[c].w);
      klo = __vimax3_u16x2(klo, alo.x & 0x7FFF7FFFu, alo.y & 0x7FFF7FFFu);
      klo = __vimax3_u16x2(klo, alo.z & 0x7FFF7FFFu, alo.w & 0x7FFF7FFFu);
      khi = __vimax3_u16x2(khi, ahi.x & 0x7FFF7FFFu, ahi.y & 0x7FFF7FFFu);
      khi = __vimax3_u16x2(khi, ahi.z & 0x7FFF7FFFu, ahi.w & 0x7FFF7FFFu);
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[e] += acc1[e];
    // the stage has been read (the MMAs consumed every fragment): refill it with page k + NST
    __syncwarp();
    if (k + NST < mine) {
      if (((k + NST) & 31) == 0) load_ids(k + NST);
      const int pg = __shfl_sync(0xFFFFFFFFu, pg_ids, (k + NST) & 31);
      if (lane == 0) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        issue(k + NST, pg);
      }
    }
    const int tk_lo = tok0 + gr, tk_hi = tok0 + gr + 8;
    if (tk_lo < n) kabs = __vimax3_u16x2(kabs, klo, 0u);
    if (tk_hi < n) kabs = __vimax3_u16x2(kabs, khi, 0u);
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int hl = 2 * t + e;
      if (hl < nh) {
        float* dst = p.scores + ((long long)b * p.Hq + h0 + hl) * p.npad;
        const float s_lo = p.scale * acc[e], s_hi = p.scale * acc[2 + e];
        if (tk_lo < n) { dst[tk_lo] = s_lo; runmax[e] = fmaxf(runmax[e], s_lo); }
        if (tk_hi < n) { dst[tk_hi] = s_hi; runmax[e] = fmaxf(runmax[e], s_hi); }
      }
    }
  }
  if (failed) {
    // give the copies still in flight a bounded chance to land before the shared memory is released
    if (lane == 0) atomicOr(p.status, VATTN_STATUS_WAIT_TIMEOUT);
    for (int s = 0; s < NST; ++s) mbar_wait(&bars[s], 0u) || mbar_wait(&bars[s], 1u);
    return;
  }
#pragma unroll
  for (int mask = 4; mask < 32; mask <<= 1) {
    runmax[0] = fmaxf(runmax[0], __shfl_xor_sync(0xFFFFFFFFu, runmax[0], mask));
    runmax[1] = fmaxf(runmax[1], __shfl_xor_sync(0xFFFFFFFFu, runmax[1], mask));
  }
#pragma unroll
  for (int mask = 1; mask < 32; mask <<= 1) kabs = __vimax3_u16x2(kabs, __shfl_xor_sync(0xFFFFFFFFu, kabs, mask), 0u);
  if (lane < 4) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int hl = 2 * lane + e;
      if (hl < nh && runmax[e] > -INFINITY) atomicMax(&p.m_ord[b * p.Hq + h0 + hl], ord_f32(runmax[e]));
    }
  }
  if (lane == 0) {
    const unsigned mx = max(kabs & 0xFFFFu, kabs >> 16);
    atomicMax(&p.kabsmax[b * p.Hkv + g], mx << 16);
  }
  DEV_END(p, 1);
}

// ---------------------------------------------------------------------------------------------
// fp32 (and generic) CUDA-core path, up to 4 heads per CTA
template <typename T, int D>
__global__ void __launch_bounds__(WARPS * 32) k_score_fma(const Prob p) {
  constexpr int EPL = Elem<T>::EPL;
  constexpr int LPR = D / EPL;       // lanes per row
  constexpr int RPI = 32 / LPR;      // rows per warp instruction
  constexpr int ITERS = 16 / RPI;    // instructions per page
  constexpr int NV = ITERS * 4;      // partial sums per lane per page (4 heads)
  __shared__ uint2 s_list[8][TILE];
  __shared__ unsigned s_cnt[8];

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
  emit_candidates<4>(p, b, g, g * p.G + hc * 4, min(4, p.G - hc * 4), tile0, n, s_list, s_cnt);
}

}  // namespace

template <int D>
static cudaError_t launch_stream(const Prob& p, cudaStream_t s) {
  const size_t smem = (size_t)WARPS * NST * VATTN_BLOCK * D * 2 + (size_t)16 * CL * sizeof(uint2) +
                      (size_t)WARPS * NST * 8 + 16 * sizeof(unsigned);
  static bool attr_done = false;
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(k_score_stream<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_done = true;
  }
  // one wave of two CTAs per SM; a warp walks pages with stride (CTAs along x) * WARPS
  const int groups = p.Hkv * ((p.G + 7) / 8) * p.B;
  const int pages = (p.max_seq_len + VATTN_BLOCK - 1) / VATTN_BLOCK;
  // A single sequence whose groups divide the 2 x 148 resident CTAs (almost) evenly runs as one wave.  Anything
  // else (several sequences, possibly of different lengths; a group count that leaves SMs idle) is cut into
  // about eight waves of CTAs with at least 32 pages each, which the hardware scheduler balances.
  const int slots = 2 * 148;
  int cx = slots / groups;
  if (cx < 1) cx = 1;
  const bool one_wave = p.B == 1 && groups * cx <= slots && (slots - groups * cx) * 20 < slots;
  if (!one_wave) {
    cx = (8 * slots + groups - 1) / groups;
    const int cx_fine = (pages + 31) / 32;
    if (cx > cx_fine) cx = cx_fine;
  }
  const int cx_max = (pages + WARPS - 1) / WARPS;
  if (cx > cx_max) cx = cx_max;
  if (cx < 1) cx = 1;
  dim3 grid(cx, p.Hkv * ((p.G + 7) / 8), p.B), block((WARPS + CWARPS) * 32);
  k_score_stream<D><<<grid, block, smem, s>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_score(const Prob& p, cudaStream_t s) {
  dim3 block(WARPS * 32);
  const int tiles = (p.max_seq_len + TILE - 1) / TILE;
  if (p.dtype == VATTN_DTYPE_BF16) {
    // rows must be 16-byte aligned for the bulk copies (any stride that is a multiple of 8 elements is)
    if (p.D == 128) return launch_stream<128>(p, s);
    return launch_stream<64>(p, s);
  } else {
    dim3 grid(tiles, p.Hkv * ((p.G + 3) / 4), p.B);
    if (p.D == 128) k_score_fma<float, 128><<<grid, block, 0, s>>>(p);
    else k_score_fma<float, 64><<<grid, block, 0, s>>>(p);
  }
  return cudaGetLastError();
}
