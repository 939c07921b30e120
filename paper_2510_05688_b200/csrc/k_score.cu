// Score pass: s[b,h,i] = scale * <q[b,h], K[b,g,i]> for every token of the paged cache, the query heads
// of a KV-head group together (the inner products of the SDPA definition, Sec. 3 of the paper;
// Algorithm 1 line 3 ranks tokens by them).  Also keeps, per query head, the running maximum score
// (softmax stabiliser) and, per KV head, max |K element| (for the rounding-error bound of the scores).
//
// HBM-bound stream over K (every K row is read exactly once).  Two arithmetic paths:
//  * bf16: a persistent grid of two CTAs per SM.  The work is cut into units (batch row, KV-head group,
//    run of consecutive pages) on the device, from the actual sequence lengths; CTAs take their first unit
//    by index and the following ones from an atomic counter, so ragged batches balance themselves.  In a
//    CTA one producer warp walks the CTA's units and keeps a ring of S page-sized stages full with bulk
//    asynchronous copies (cp.async.bulk + mbarrier transaction counts; one 4 KB slab per page, the group's
//    query rows ride along with the first pages of a unit); four consumer warps take the stages in turn
//    (full / empty mbarriers, bounded waits) and run the [16 tokens x d] x [d x 8 heads] contraction of a
//    page on the tensor cores (mma.sync m16n8k16, fp32 accumulate, two independent chains).  A dot product
//    does not care in which order its terms are paired, so the k-slots of the fragment layout are mapped
//    onto d such that each thread owns 8 consecutive elements of a row and reads them with one 16-byte
//    shared load.  The ring never drains between units.
//  * fp32: CUDA-core FMAs, EPL sequential FMAs per lane and a butterfly that halves the live partial
//    sums at every level (tf32 tensor cores would not keep fp32 accuracy).
#include "vattn_internal.cuh"

namespace {

constexpr int PPW = 4;      // pages per warp                         (fp32 path)
constexpr int WARPS = 4;    // warps per CTA                          (fp32 path)
constexpr int TILE = PPW * WARPS * VATTN_BLOCK;   // 256 tokens       (fp32 path)

// ---------------------------------------------------------------------------------------------
// bf16: persistent producer / consumer kernel
constexpr int CWN = 4;                              // consumer warps per CTA
constexpr int SCORE_THREADS = (CWN + 1) * 32;       // + one producer warp
constexpr int MIN_UNIT_PAGES = 16;
constexpr int UNITS_PER_CTA = 8;                    // target for batches (a single sequence gets one unit per CTA)

struct __align__(16) StageMeta {   // written by the producer before it arms the stage's full barrier
  int tok0;             // first token of the page; < 0: no more work for the consumer that owns this stage
  int n;                // tokens of the sequence
  int bh0;              // batch row * Hq + first query head of the group slice
  int nh_unit;          // query heads in the slice (<= 16) | running unit number of the CTA << 5: a change of
};                      // the unit tells the consumer to flush its maxima and reload q

// Clears the per-step counters (running maxima, tickets, list lengths, unit counter).  A kernel rather than a
// memset node so that the score kernel behind it can start its prologue and its first copies meanwhile: it
// lets its dependents go at once and waits for the previous step before it writes.
// (`late`: the grid before this one wrote the step's inputs, which the score kernel reads in its prologue, so
// the dependents may only go once that grid has completed.)
__global__ void __launch_bounds__(256) k_zero(unsigned* z, int words, int late, unsigned long long* ticks) {
  if (ticks && threadIdx.x == 0) atomicMin(ticks + 2 * VATTN_K_ZERO, gtime_ns());
  if (!late) pdl_trigger();
  pdl_wait();
  if (late) pdl_trigger();
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < words; i += gridDim.x * blockDim.x) z[i] = 0u;
  if (ticks && threadIdx.x == 0) atomicMax(ticks + 2 * VATTN_K_ZERO + 1, gtime_ns());
}

__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// WIDE: slices of up to 16 heads (groups of more than 8 heads: calls with several query tokens, or many query heads
// per KV head); otherwise the second half of the slice and its registers are compiled out
template <int D, bool WIDE>
__global__ void __launch_bounds__(SCORE_THREADS, 2) k_score_stream(const Prob p, int qslot_bytes) {
  constexpr int NC = D / 32;
  constexpr int ROWB = D * 2;                 // bytes per row
  constexpr int PAGEB = VATTN_BLOCK * ROWB;   // bytes per (page, KV head) slab
  constexpr int S = 2048 / D;                 // stages: 64 KB of pages in flight per CTA
  extern __shared__ __align__(128) unsigned char smem_dyn[];
  unsigned char* ring = smem_dyn;
  unsigned char* qring = ring + (size_t)S * PAGEB;
  StageMeta* meta = reinterpret_cast<StageMeta*>(qring + (size_t)S * qslot_bytes);
  unsigned long long* full = reinterpret_cast<unsigned long long*>(meta + S);
  unsigned long long* empty = full + S;
  int* s_len = reinterpret_cast<int*>(empty + S);    // [B]   clamped sequence lengths
  int* s_pref = s_len + p.B;                         // [B+1] units before batch row b
  int* s_misc = s_pref + p.B + 1;                    // [16]
  const int tid = threadIdx.x, wid = tid >> 5, lane = tid & 31;
  TICK_BEGIN(p, VATTN_K_SCORE);

  // ---- units: every CTA derives the same decomposition from the sequence lengths
  constexpr int SL = WIDE ? 16 : 8;                   // heads per slice: one pass over K serves a slice
  const int GC = (p.G + SL - 1) / SL;
  const int GPB = p.Hkv * GC;                         // (KV head, head slice) groups per batch row
  int my_pages = 0;
  for (int b = tid; b < p.B; b += SCORE_THREADS) {
    const int n = clamped_len(p, b);
    s_len[b] = n;
    my_pages += (n + 15) >> 4;
  }
#pragma unroll
  for (int mk = 16; mk >= 1; mk >>= 1) my_pages += __shfl_xor_sync(0xFFFFFFFFu, my_pages, mk);
  if (lane == 0) s_misc[wid] = my_pages;
  if (tid < S) { mbar_init(&full[tid], 1); mbar_init(&empty[tid], 1); }
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  __syncthreads();
  long long pages_total = 0;
  for (int w = 0; w <= CWN; ++w) pages_total += s_misc[w];
  const long long want_units = (long long)gridDim.x * (p.B == 1 ? 1 : UNITS_PER_CTA);
  long long ch64 = (pages_total * GPB + want_units - 1) / want_units;
  const int CH = (int)(ch64 < MIN_UNIT_PAGES ? MIN_UNIT_PAGES : ch64);      // pages per unit
  if (wid == 0) {                                     // exclusive prefix of the units per batch row
    int carry = 0;
    for (int b0 = 0; b0 < p.B; b0 += 32) {
      const int b = b0 + lane;
      const int units = (b < p.B) ? GPB * ((((s_len[b] + 15) >> 4) + CH - 1) / CH) : 0;
      int incl = units;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += v;
      }
      if (b < p.B) s_pref[b] = carry + incl - units;
      carry += __shfl_sync(0xFFFFFFFFu, incl, 31);
    }
    if (lane == 0) s_pref[p.B] = carry;
  }
  __syncthreads();
  const int U = s_pref[p.B];
  const bf16_t* kc = reinterpret_cast<const bf16_t*>(p.kc);

  if (wid == CWN) {
    // =============================================================== producer warp
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    const unsigned long long kpolicy = l2_evict_first_policy();
    long long i = 0;                                  // stages armed so far
    int ucount = 0;
    bool failed = false;
    int u = blockIdx.x;
    bool first = true;
    while (u < U && !failed) {
      unsigned nxt = 0u;
      int lo = 0, hi = p.B - 1;                        // last batch row whose first unit is <= u
      while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (s_pref[mid] <= u) lo = mid; else hi = mid - 1;
      }
      const int b = lo, n = s_len[b], np = (n + 15) >> 4;
      const int chunks = (np + CH - 1) / CH;
      const int r = u - s_pref[b];
      const int gc = r / chunks, chunk = r % chunks;
      const int g = gc / GC, hc = gc % GC;
      const int h0 = g * p.G + hc * SL, nh = min(SL, p.G - hc * SL);
      const int pA = chunk * CH, cnt = min(CH, np - pA);
      const bf16_t* qsrc = reinterpret_cast<const bf16_t*>(p.q) + ((long long)b * p.Hq + h0) * D;
      // S lanes arm S stages at a time, each lane its own: wait for the stage to be handed back, describe the
      // page, post the copy.  The page ids of the next round are requested before this round's waits.
      int pid_next = (lane < S && lane < cnt) ? page_of(p, b, pA + lane) : 0;
      for (int k0 = 0; k0 < cnt; k0 += S) {
        const int pid = pid_next;
        pid_next = (lane < S && k0 + S + lane < cnt) ? page_of(p, b, pA + k0 + S + lane) : 0;
        bool ok = true;
        if (lane < S && k0 + lane < cnt) {
          const long long ii = i + lane;
          const int stage = (int)(ii % S);
          if (ii >= S) ok = mbar_wait(&empty[stage], (unsigned)((ii / S) - 1) & 1u);
          if (ok) {
            const int k = k0 + lane;
            StageMeta m;
            m.tok0 = (pA + k) << 4; m.n = n; m.bh0 = b * p.Hq + h0; m.nh_unit = nh | (ucount << 5);
            meta[stage] = m;
            const bool with_q = k < CWN;              // every consumer meets q on its first page of the unit
            const int nq = min(nh, 8);                // the first 8 heads' rows ride with the page; the others are read by the consumers
            const unsigned qbytes = (unsigned)(nq * ROWB);
            unsigned char* dst = ring + (size_t)stage * PAGEB;
            const bf16_t* src = kc + (long long)pid * p.sb + (long long)g * p.sh;
            mbar_expect_tx(&full[stage], PAGEB + (with_q ? qbytes : 0u));
            if (with_q) {
              if (p.Tq == 1) bulk_g2s(qring + (size_t)stage * qslot_bytes, qsrc, qbytes, &full[stage]);
              else                                    // the rows of different query tokens are apart in memory
                for (int rr = 0; rr < nq; ++rr)
                  bulk_g2s(qring + (size_t)stage * qslot_bytes + rr * ROWB,
                           reinterpret_cast<const bf16_t*>(p.q) + q_row(p, b, h0 + rr), ROWB, &full[stage]);
            }
            if (p.st == D) bulk_g2s_stream(dst, src, PAGEB, &full[stage], kpolicy);
            else
              for (int rr = 0; rr < VATTN_BLOCK; ++rr) bulk_g2s_stream(dst + rr * ROWB, src + (long long)rr * p.st, ROWB, &full[stage], kpolicy);
          }
        }
        i += min(S, cnt - k0);
        if (!__all_sync(0xFFFFFFFFu, ok)) { failed = true; break; }
        if (k0 == 0) {
          // The first copies of the CTA are under way; from here on the kernel touches what the grid before
          // it clears (k_zero), so wait for it, and only then let the key pre-filter behind this grid start.
          if (first) { pdl_wait(); pdl_trigger(); first = false; }
          if (lane == 0) nxt = atomicAdd(p.unit_ctr, 1u);  // the unit after this one; the round trip hides behind this unit
        }
      }
      ++ucount;
      u = (int)gridDim.x + (int)__shfl_sync(0xFFFFFFFFu, nxt, 0);
    }
    if (first) { pdl_wait(); pdl_trigger(); }
    // one end mark per consumer (consumer w owns the stages i = w mod CWN)
    if (!failed) {
      bool ok = true;
      if (lane < CWN) {
        const long long ii = i + lane;
        const int stage = (int)(ii % S);
        if (ii >= S) ok = mbar_wait(&empty[stage], (unsigned)((ii / S) - 1) & 1u);
        if (ok) {
          StageMeta m;
          m.tok0 = -1; m.n = 0; m.bh0 = 0; m.nh_unit = 0;
          meta[stage] = m;
          mbar_arrive(&full[stage]);
        }
      }
      i += CWN;
      if (!__all_sync(0xFFFFFFFFu, ok)) failed = true;
    }
    if (failed) {
      // a consumer gave up: report, and give the copies still in flight a bounded chance to land before the
      // shared memory is released
      if (lane == 0) atomicOr(p.status, VATTN_STATUS_WAIT_TIMEOUT);
      // (a stage that was never armed simply runs into the wait limit)
      for (long long j = (i > S ? i - S : 0) + lane; j < i; j += 32) mbar_wait(&full[j % S], (unsigned)(j / S) & 1u);
    }
    TICK_END_IF(p, VATTN_K_SCORE, lane == 0);
    return;
  }

  // ================================================================= consumer warps
  const int gr = lane >> 2, t = lane & 3;
  uint4 bq[NC], bq2[NC];                            // q fragments of heads 0..7 and 8..15 of the slice
#pragma unroll
  for (int c = 0; c < NC; ++c) { bq[c] = make_uint4(0u, 0u, 0u, 0u); bq2[c] = make_uint4(0u, 0u, 0u, 0u); }
  float runmax[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // heads 2t, 2t+1, 8+2t, 9+2t
  unsigned kabs = 0u;
  int cur_unit = -1, cur_bh0 = 0, cur_nh = 0;       // cur_unit holds nh_unit of the unit in progress
  unsigned hide = 0u;                                 // tokens at the end of the sequence that this thread's heads do not see, a byte per head
  auto flush = [&]() {                                // running maxima of the unit just finished
    if (cur_unit < 0) return;
#pragma unroll
    for (int mask = 4; mask < 32; mask <<= 1) {
#pragma unroll
      for (int e = 0; e < (WIDE ? 4 : 2); ++e) runmax[e] = fmaxf(runmax[e], __shfl_xor_sync(0xFFFFFFFFu, runmax[e], mask));
    }
#pragma unroll
    for (int mask = 1; mask < 32; mask <<= 1) kabs = __vimax3_u16x2(kabs, __shfl_xor_sync(0xFFFFFFFFu, kabs, mask), 0u);
    if (lane < 4) {
#pragma unroll
      for (int e = 0; e < (WIDE ? 4 : 2); ++e) {
        const int hl = (e >> 1) * 8 + 2 * lane + (e & 1);
        if (hl < cur_nh && runmax[e] > -INFINITY) atomicMax(&p.m_ord[cur_bh0 + hl], ord_f32(runmax[e]));
      }
    }
    if (lane == 0) {
      const unsigned mx = max(kabs & 0xFFFFu, kabs >> 16);
      const int b = cur_bh0 / p.Hq, g = (cur_bh0 % p.Hq) / p.G;
      atomicMax(&p.kabsmax[b * p.Hkv + g], mx << 16);
    }
    runmax[0] = runmax[1] = runmax[2] = runmax[3] = -INFINITY;
    kabs = 0u;
  };

  pdl_wait();                                         // scores and counters of the previous step are free now
  pdl_trigger();
  for (long long i = wid;; i += CWN) {
    const int stage = (int)(i % S);
    if (!__all_sync(0xFFFFFFFFu, mbar_wait(&full[stage], (unsigned)(i / S) & 1u))) {   // warp-uniform decision
      if (lane == 0) atomicOr(p.status, VATTN_STATUS_WAIT_TIMEOUT);
      break;
    }
    const StageMeta m = meta[stage];
    if (m.tok0 < 0) break;
    const int m_nh = m.nh_unit & 31;
    if (m.nh_unit != cur_unit) {
      flush();
      cur_unit = m.nh_unit; cur_bh0 = m.bh0; cur_nh = m_nh;
      if (p.Tq > 1) {
#pragma unroll
        hide = 0u;
#pragma unroll
        for (int e = 0; e < (WIDE ? 4 : 2); ++e)
          hide |= (unsigned)(p.Tq - 1 - head_tok(p, (m.bh0 + (e >> 1) * 8 + 2 * t + (e & 1)) % p.Hq)) << (8 * e);
      }
      if (WIDE && m_nh > 8) {                          // heads 8..15 of the slice: their rows come straight from q
        const int bb = m.bh0 / p.Hq, hv0 = m.bh0 % p.Hq;
#pragma unroll
        for (int c = 0; c < NC; ++c)
          bq2[c] = (8 + gr < m_nh) ? __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const bf16_t*>(p.q) +
                                                                         q_row(p, bb, hv0 + 8 + gr) + c * 32 + t * 8))
                                   : make_uint4(0u, 0u, 0u, 0u);
      }
      const unsigned char* qs = qring + (size_t)stage * qslot_bytes;
#pragma unroll
      for (int c = 0; c < NC; ++c)
        bq[c] = (gr < m_nh) ? *reinterpret_cast<const uint4*>(qs + gr * ROWB + c * 64 + t * 16) : make_uint4(0u, 0u, 0u, 0u);
    }
    const unsigned char* stg = ring + (size_t)stage * PAGEB;
    float acc[4] = {0.f, 0.f, 0.f, 0.f}, acc1[4] = {0.f, 0.f, 0.f, 0.f};   // two independent MMA chains
    float accB[4] = {0.f, 0.f, 0.f, 0.f}, accB1[4] = {0.f, 0.f, 0.f, 0.f}; // heads 8..15 of the slice, from the same page
    const bool two = WIDE && m_nh > 8;                 // (uniform over the warp)
    unsigned klo = 0u, khi = 0u;
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      const uint4 alo = *reinterpret_cast<const uint4*>(stg + gr * ROWB + c * 64 + t * 16);
      const uint4 ahi = *reinterpret_cast<const uint4*>(stg + (gr + 8) * ROWB + c * 64 + t * 16);
      mma_bf16_16816(acc, alo.x, ahi.x, alo.y, ahi.y, bq[c].x, bq[c].y);
      mma_bf16_16816(acc1, alo.z, ahi.z, alo.w, ahi.w, bq[c].z, bq[c].w);
      if (two) {
        mma_bf16_16816(accB, alo.x, ahi.x, alo.y, ahi.y, bq2[c].x, bq2[c].y);
        mma_bf16_16816(accB1, alo.z, ahi.z, alo.w, ahi.w, bq2[c].z, bq2[c].w);
      }
      klo = __vimax3_u16x2(klo, alo.x & 0x7FFF7FFFu, alo.y & 0x7FFF7FFFu);
      klo = __vimax3_u16x2(klo, alo.z & 0x7FFF7FFFu, alo.w & 0x7FFF7FFFu);
      khi = __vimax3_u16x2(khi, ahi.x & 0x7FFF7FFFu, ahi.y & 0x7FFF7FFFu);
      khi = __vimax3_u16x2(khi, ahi.z & 0x7FFF7FFFu, ahi.w & 0x7FFF7FFFu);
    }
    // the stage (page and query rows) has been read: hand it back to the producer
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty[stage]);
#pragma unroll
    for (int e = 0; e < 4; ++e) { acc[e] += acc1[e]; accB[e] += accB1[e]; }
    const int tk_lo = m.tok0 + gr, tk_hi = m.tok0 + gr + 8;
    if (tk_lo < m.n) kabs = __vimax3_u16x2(kabs, klo, 0u);
    if (tk_hi < m.n) kabs = __vimax3_u16x2(kabs, khi, 0u);
#pragma unroll
    for (int e4 = 0; e4 < (WIDE ? 4 : 2); ++e4) {
      const int e = e4 & 1, hl = (e4 >> 1) * 8 + 2 * t + e;
      if (hl < m_nh) {
        float* dst = p.scores + (long long)(m.bh0 + hl) * p.npad;
        const float s_lo = p.scale * (e4 < 2 ? acc[e] : accB[e]), s_hi = p.scale * (e4 < 2 ? acc[2 + e] : accB[2 + e]);
        const int seen = m.n - (int)((hide >> (8 * e4)) & 0xFFu);
        if (tk_lo < m.n) { dst[tk_lo] = s_lo; if (tk_lo < seen) runmax[e4] = fmaxf(runmax[e4], s_lo); }
        if (tk_hi < m.n) { dst[tk_hi] = s_hi; if (tk_hi < seen) runmax[e4] = fmaxf(runmax[e4], s_hi); }
      }
    }
  }
  flush();
  TICK_END(p, VATTN_K_SCORE);
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
      Elem<T>::load(reinterpret_cast<const T*>(p.q) + q_row(p, b, g * p.G + hl) + j * EPL, qv[hh]);
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
        if (p.Tq == 1 || tok < n - (p.Tq - 1 - head_tok(p, g * p.G + hl))) runmax[e] = fmaxf(runmax[e], sc);
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

template <int D, bool WIDE>
static cudaError_t launch_stream(const Prob& p, cudaStream_t s) {
  constexpr int S = 2048 / D, PAGEB = VATTN_BLOCK * D * 2, SL = WIDE ? 16 : 8;
  const int nh_max = p.G < 8 ? p.G : 8;
  const int qslot_bytes = nh_max * D * 2;
  const size_t smem = (size_t)S * PAGEB + (size_t)S * qslot_bytes + (size_t)S * sizeof(StageMeta) + (size_t)2 * S * 8 +
                      sizeof(int) * ((size_t)2 * p.B + 1 + 16);
  if (smem > 113 * 1024) return cudaErrorInvalidValue;        // two CTAs per SM (plan creation bounds the batch)
  static size_t have[VATTN_MAXDEV];
  cudaError_t e = optin_smem(k_score_stream<D, WIDE>, smem, have, true);
  if (e != cudaSuccess) return e;
  // persistent: two CTAs per SM, fewer when the problem cannot have that many units
  const long long pages = (p.max_seq_len + VATTN_BLOCK - 1) / VATTN_BLOCK;
  const long long units_max = (long long)p.B * p.Hkv * ((p.G + SL - 1) / SL) * ((pages + MIN_UNIT_PAGES - 1) / MIN_UNIT_PAGES);
  const int slots = 2 * device_sm_count();
  const int grid = (int)(units_max < slots ? (units_max < 1 ? 1 : units_max) : slots);
  return launch_pdl(k_score_stream<D, WIDE>, dim3(grid), dim3(SCORE_THREADS), smem, s, p, qslot_bytes);
}

// `pdl`: launch with the programmatic-serialization attribute, i.e. let this grid start while the kernel before it
// in the stream still runs.  Only sound when that kernel is one of this library's own (it then has no stores
// left that the step reads once its CTAs have let their dependents go); against a caller's kernel the launch
// is an ordinary one.
cudaError_t launch_zero(unsigned* z, size_t bytes, bool pdl, bool late, unsigned long long* ticks, cudaStream_t s) {
  const int words = (int)(bytes / sizeof(unsigned));
  int grid = (words + 1023) / 1024;
  if (grid > 148) grid = 148;
  if (grid < 1) grid = 1;
  if (pdl) return launch_pdl(k_zero, dim3(grid), dim3(256), 0, s, z, words, late ? 1 : 0, ticks);
  k_zero<<<grid, 256, 0, s>>>(z, words, 1, ticks);
  return cudaGetLastError();
}

cudaError_t launch_score(const Prob& p, cudaStream_t s) {
  dim3 block(WARPS * 32);
  const int tiles = (p.max_seq_len + TILE - 1) / TILE;
  if (p.dtype == VATTN_DTYPE_BF16) {
    // rows must be 16-byte aligned for the bulk copies (any stride that is a multiple of 8 elements is)
    if (p.G > 8) return p.D == 128 ? launch_stream<128, true>(p, s) : launch_stream<64, true>(p, s);
    return p.D == 128 ? launch_stream<128, false>(p, s) : launch_stream<64, false>(p, s);
  } else {
    dim3 grid(tiles, p.Hkv * ((p.G + 3) / 4), p.B);
    if (p.D == 128) k_score_fma<float, 128><<<grid, block, 0, s>>>(p);
    else k_score_fma<float, 64><<<grid, block, 0, s>>>(p);
  }
  return cudaGetLastError();
}
