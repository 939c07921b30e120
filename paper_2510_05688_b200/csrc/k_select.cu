// Index selection: one CTA per (batch row, query head).
//
//  k_select_topk  : I_t = the k middle tokens with the largest score, ties to the lowest index
//                   (Algorithm 1 line 3, "oracle top-k" of Sec. 3).
//  k_presort      : the base sample I_bs = uniform-sample of b0 residual tokens (Algorithm 2 line 1) and the
//                   residual in the order in which the final sample draws it (Algorithm 1 line 7).
//  k_budget       : the budget b from the statistics partials, then I_dyn = uniform-sample of b residual
//                   tokens for the heads k_presort could not serve.
//
// All selections are "the c smallest (key, index) pairs".  The generic form is an 8-bit-digit radix select
// over 32-bit keys held in shared memory, followed by an ordered compaction through bitmaps, so its lists
// come out ascending.  Keys are the order-reversed score for top-k and Philox4x32-10 words for sampling.
//
// Fast paths (one pass over the context instead of four): the top-k threshold is first estimated from a
// strided sample of the scores (1024 linear bins between the sample minimum and the head maximum), one
// pass collects the few thousand tokens above the estimate, and the exact radix select runs on those
// candidates only.  Sampling sorts the candidate lists the score kernel pre-filtered (tokens whose
// Philox key is below a bound): if the list holds at least c residual tokens, the c smallest keys of
// the residual are its first c residual entries.  Whenever an estimate fails (too few / too many
// candidates, list overflow, near-tie band reaching below the estimate) the generic full-context select
// runs instead.
//
// Exact top-k from fp32 scores: the stored scores differ from the exact inner products by at most
// gamma (a bound from the summation structure of the score kernel).  After the fp32 threshold T is
// known, tokens above T + 2*gamma are certainly selected and tokens below T - 2*gamma certainly not;
// the few in between are rescored in fp64 from their K rows and ranked exactly.
#include "vattn_internal.cuh"
#include <math_constants.h>

namespace {

constexpr int NT = SEL_THREADS;
constexpr int NWARP = NT / 32;

constexpr int CANDCAP = 4096;      // top-k candidates kept by the fast path
constexpr int NBIN = 1024;          // linear bins of the threshold estimate (one per thread)
constexpr int PAIRCAP0 = 4096;      // base-sample candidate pairs staged in shared memory

struct Sm {
  double* band_s;     // [BANDCAP]
  unsigned* keys;     // [bigbytes/4] select keys of the context, or staged (key, token) pairs
  unsigned* w0;       // [nwords] selected / "less than threshold" bitmap
  unsigned* w1;       // [nwords] "equal to threshold" / band bitmap
  unsigned* w2;       // [nwords] I_t bitmap (residual mask) / scratch
  int* scan;          // [nwords]
  unsigned* hist;     // [256]
  int* band_idx;      // [BANDCAP]
  int* lin;           // [NBIN]
  int* cand_idx;      // [CANDCAP]
  unsigned* ckey;     // [CANDCAP] select keys of the candidates
  int* misc;          // [64]
};

__device__ __forceinline__ Sm carve(unsigned char* base, int bigbytes, int nwords) {
  Sm s;
  s.band_s = reinterpret_cast<double*>(base);            base += sizeof(double) * VATTN_BANDCAP;
  s.keys = reinterpret_cast<unsigned*>(base);            base += (size_t)bigbytes;
  s.w0 = reinterpret_cast<unsigned*>(base);              base += sizeof(unsigned) * (size_t)nwords;
  s.w1 = reinterpret_cast<unsigned*>(base);              base += sizeof(unsigned) * (size_t)nwords;
  s.w2 = reinterpret_cast<unsigned*>(base);              base += sizeof(unsigned) * (size_t)nwords;
  s.scan = reinterpret_cast<int*>(base);                 base += sizeof(int) * (size_t)nwords;
  s.hist = reinterpret_cast<unsigned*>(base);            base += sizeof(unsigned) * 256;
  s.band_idx = reinterpret_cast<int*>(base);             base += sizeof(int) * VATTN_BANDCAP;
  s.lin = reinterpret_cast<int*>(base);                  base += sizeof(int) * NBIN;
  s.cand_idx = reinterpret_cast<int*>(base);             base += sizeof(int) * CANDCAP;
  s.ckey = reinterpret_cast<unsigned*>(base);            base += sizeof(unsigned) * CANDCAP;
  s.misc = reinterpret_cast<int*>(base);
  return s;
}

// exclusive prefix sum of a[0..nw) in place; returns the total.  misc[8..40) is scratch.
__device__ int block_excl_scan(int* a, int nw, int* misc) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ipt = (nw + NT - 1) / NT;
  const int start = min(nw, tid * ipt), end = min(nw, start + ipt);
  int local = 0;
  for (int i = start; i < end; ++i) local += a[i];
  int incl = local;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    int v = __shfl_up_sync(0xFFFFFFFFu, incl, off);
    if (lane >= off) incl += v;
  }
  __syncthreads();                       // misc scratch may still be read by an earlier call
  if (lane == 31) misc[8 + warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int v = misc[8 + lane], in2 = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      int u = __shfl_up_sync(0xFFFFFFFFu, in2, off);
      if (lane >= off) in2 += u;
    }
    misc[8 + lane] = in2 - v;
    if (lane == 31) misc[40] = in2;
  }
  __syncthreads();
  int run = incl - local + misc[8 + warp];
  for (int i = start; i < end; ++i) { int v = a[i]; a[i] = run; run += v; }
  const int total = misc[40];
  __syncthreads();
  return total;
}

// Exclusive prefix sum over the CTA of one value per thread, with a single barrier: warp scans, the 32 warp
// totals go through `wtot` (32 ints of shared memory that no thread touches between this call's barrier and
// the next barrier of the caller), and every warp scans the totals itself.  `total` = sum over the CTA.
__device__ __forceinline__ int block_scan_reg(int val, int* wtot, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = val;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int v = __shfl_up_sync(0xFFFFFFFFu, incl, off);
    if (lane >= off) incl += v;
  }
  if (lane == 31) wtot[warp] = incl;
  __syncthreads();
  const int mine = (lane < NWARP) ? wtot[lane] : 0;
  int winc = mine;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int v = __shfl_up_sync(0xFFFFFFFFu, winc, off);
    if (lane >= off) winc += v;
  }
  total = __shfl_sync(0xFFFFFFFFu, winc, 31);
  const int before = __shfl_sync(0xFFFFFFFFu, winc - mine, warp);
  return before + incl - val;
}

// Radix select of the c-th smallest key among the valid tokens of [lo, hi).  1 <= c <= #valid.
// On return every thread knows T (the c-th smallest key) and need_eq (how many keys equal to T are
// selected; all keys < T are).  keyfn(i, key) returns validity.
template <typename KeyT, bool AGG, class F>
__device__ void block_select(F keyfn, int lo, int hi, int c, unsigned* hist, int* misc, KeyT& T, int& need_eq) {
  constexpr int NP = (int)sizeof(KeyT);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  KeyT prefix = 0, mask = 0;
  int rem = c;
  const int lo32 = lo & ~31, hi32 = (hi + 31) & ~31;
  for (int pass = 0; pass < NP; ++pass) {
    const int shift = (NP - 1 - pass) * 8;
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    for (int i = lo32 + tid; i < hi32; i += NT) {
      KeyT key = 0;
      bool ok = (i >= lo) && (i < hi);
      if (ok) ok = keyfn(i, key);
      ok = ok && ((key & mask) == prefix);
      const unsigned digit = (unsigned)((key >> shift) & 0xFF);
      if (AGG) {
        const unsigned peers = __match_any_sync(0xFFFFFFFFu, ok ? digit : 0xFFFFFFFFu);
        if (ok && lane == (__ffs(peers) - 1)) atomicAdd(&hist[digit], (unsigned)__popc(peers));
      } else {
        if (ok) atomicAdd(&hist[digit], 1u);
      }
    }
    __syncthreads();
    if (warp == 0) {
      int cnt[8], s = 0;
#pragma unroll
      for (int e = 0; e < 8; ++e) { cnt[e] = (int)hist[lane * 8 + e]; s += cnt[e]; }
      int incl = s;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        int v = __shfl_up_sync(0xFFFFFFFFu, incl, off);
        if (lane >= off) incl += v;
      }
      const int excl = incl - s;
      if (excl < rem && rem <= incl) {
        int cum = excl;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          if (rem <= cum + cnt[e]) { misc[0] = lane * 8 + e; misc[1] = cum; break; }
          cum += cnt[e];
        }
      }
    }
    __syncthreads();
    prefix |= (KeyT)(unsigned)misc[0] << shift;
    mask |= (KeyT)0xFF << shift;
    rem -= misc[1];
    __syncthreads();
  }
  T = prefix;
  need_eq = rem;
}

__device__ __forceinline__ unsigned lowest_bits(unsigned word, int take) {
  if (take <= 0) return 0u;
  if (take >= __popc(word)) return word;
  unsigned r = 0;
  for (int t = 0; t < take; ++t) { unsigned lsb = word & (0u - word); r |= lsb; word ^= lsb; }
  return r;
}

// sel |= the `need_eq` lowest-index bits of eq; then write the selected token indices ascending to
// out_a (and out_b if non-null).  Returns the number selected.
__device__ int finalize_emit(const Prob& p, int b, unsigned* sel, const unsigned* eq, int need_eq, int nw, int* scan,
                             int* misc, int* out_a, int* out_b) {
  const int tid = threadIdx.x;
  if (need_eq > 0) {
    for (int w = tid; w < nw; w += NT) scan[w] = __popc(eq[w]);
    __syncthreads();
    block_excl_scan(scan, nw, misc);
    for (int w = tid; w < nw; w += NT) sel[w] |= lowest_bits(eq[w], need_eq - scan[w]);
    __syncthreads();
  }
  int total;
  if (nw <= NT) {                                     // one word per thread: prefix in registers, one barrier
    __syncthreads();                                  // sel[] complete; the scratch below is free
    const int mine = (tid < nw) ? __popc(sel[tid]) : 0;
    const int excl = block_scan_reg(mine, misc + 8, total);
    if (tid < nw) scan[tid] = excl;
  } else {
    for (int w = tid; w < nw; w += NT) scan[w] = __popc(sel[w]);
    __syncthreads();
    total = block_excl_scan(scan, nw, misc);
  }
  for (int w = tid; w < nw; w += NT) {
    unsigned bits = sel[w];
    int pos = scan[w];
    // the 32 tokens of a word lie in two pages: both ids are requested before the first is needed
    const int pg_lo = (bits & 0xFFFFu) ? page_of(p, b, 2 * w) : 0;
    const int pg_hi = (bits >> 16) ? page_of(p, b, 2 * w + 1) : 0;
    while (bits) {
      const int bit = __ffs(bits) - 1;
      bits &= bits - 1;
      const int idx = w * 32 + bit;
      out_a[pos] = idx;
      out_a[p.phys_delta + pos] = (bit < 16 ? pg_lo : pg_hi) * VATTN_BLOCK + (idx & 15);   // physical slot for the row kernels
      if (out_b) out_b[pos] = idx;
      ++pos;
    }
  }
  __syncthreads();
  return total;
}

// exact fp64 score of one token, computed by a whole warp (all lanes return it)
template <typename T, int D>
__device__ double score64_warp(const Prob& p, int b, int g, const T* qrow, int tok) {
  const int lane = threadIdx.x & 31;
  const T* krow = row_ptr<T>(p, p.kc, b, g, tok);
  double acc = 0.0;
#pragma unroll
  for (int t = 0; t < D / 32; ++t) {
    const int e = lane + 32 * t;
    acc = fma((double)Elem<T>::to_float(qrow[e]), (double)Elem<T>::to_float(krow[e]), acc);
  }
#pragma unroll
  for (int mask = 16; mask >= 1; mask >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, mask);
  return acc * (double)p.scale;
}
// the same number, by one thread (identical summation tree, so identical bits)
template <typename T, int D>
__device__ double score64_thread(const Prob& p, int b, int g, const T* qrow, int tok) {
  const T* krow = row_ptr<T>(p, p.kc, b, g, tok);
  double part[32];
  for (int l = 0; l < 32; ++l) {
    double acc = 0.0;
    for (int t = 0; t < D / 32; ++t) {
      const int e = l + 32 * t;
      acc = fma((double)Elem<T>::to_float(qrow[e]), (double)Elem<T>::to_float(krow[e]), acc);
    }
    part[l] = acc;
  }
  for (int mask = 16; mask >= 1; mask >>= 1)
    for (int l = 0; l < 32; ++l)
      if (!(l & mask) && (l | mask) < 32 && l < mask) part[l] = part[l] + part[l | mask];
  return part[0] * (double)p.scale;
}

// Philox sampling keys of the middle range into shared memory (one Philox call covers 4 tokens)
__device__ void fill_philox_keys(const Prob& p, unsigned* keys, int lo, int hi, int b, int hrng, int stream) {
  const unsigned c1 = ((unsigned)b << 16) | (unsigned)hrng;
  const unsigned c3 = ((unsigned)p.step << 1) | (unsigned)stream;
  for (int c4 = (lo >> 2) + threadIdx.x; c4 < ((hi + 3) >> 2); c4 += NT) {
    const uint4 r = philox4x32_10((unsigned)c4, c1, (unsigned)p.layer, c3, p.seed_lo, p.seed_hi);
    *reinterpret_cast<uint4*>(&keys[c4 * 4]) = r;
  }
}
__device__ __forceinline__ unsigned philox_key_of(const Prob& p, int i, int b, int hrng, int stream) {
  const uint4 r = philox4x32_10((unsigned)(i >> 2), ((unsigned)b << 16) | (unsigned)hrng, (unsigned)p.layer,
                                ((unsigned)p.step << 1) | (unsigned)stream, p.seed_lo, p.seed_hi);
  const int e = i & 3;
  return e == 0 ? r.x : e == 1 ? r.y : e == 2 ? r.z : r.w;
}

// c residual tokens with the smallest (Philox key, index); residual = [lo,hi) minus the bits of `it`.
// Result bitmap in sm.w0; emitted ascending to out_a/out_b.
template <bool CACHED>
__device__ int sample_select(const Prob& p, const Sm& sm, int lo, int hi, int nw, int c, int n_s, int b, int hrng,
                             int stream, const unsigned* it, int* out_a, int* out_b) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (c <= 0) return 0;
  if (c >= n_s) {                         // the whole residual
    for (int w = tid; w < nw; w += NT) {
      const int i0 = w * 32;
      unsigned m = 0xFFFFFFFFu;
      if (i0 < lo) m &= (lo - i0 >= 32) ? 0u : (0xFFFFFFFFu << (lo - i0));
      if (i0 + 32 > hi) m &= (hi <= i0) ? 0u : (0xFFFFFFFFu >> (i0 + 32 - hi));
      sm.w0[w] = m & ~it[w];
    }
    __syncthreads();
    return finalize_emit(p, b, sm.w0, sm.w1, 0, nw, sm.scan, sm.misc, out_a, out_b);
  }
  if (CACHED) fill_philox_keys(p, sm.keys, lo, hi, b, hrng, stream);
  __syncthreads();
  auto keyfn = [&](int i, unsigned& key) -> bool {
    if ((it[i >> 5] >> (i & 31)) & 1u) return false;
    key = CACHED ? sm.keys[i] : philox_key_of(p, i, b, hrng, stream);
    return true;
  };
  unsigned T; int need_eq;
  block_select<unsigned, false>(keyfn, lo, hi, c, sm.hist, sm.misc, T, need_eq);
  for (int w = warp; w < nw; w += NWARP) {
    const int i = w * 32 + lane;
    unsigned key = 0;
    bool ok = (i >= lo) && (i < hi);
    if (ok) ok = keyfn(i, key);
    const unsigned lt = __ballot_sync(0xFFFFFFFFu, ok && key < T);
    const unsigned eq = __ballot_sync(0xFFFFFFFFu, ok && key == T);
    if (lane == 0) { sm.w0[w] = lt; sm.w1[w] = eq; }
  }
  __syncthreads();
  return finalize_emit(p, b, sm.w0, sm.w1, need_eq, nw, sm.scan, sm.misc, out_a, out_b);
}

// ---------------------------------------------------------------------------------------------
// top-k, fast path: requires the inverted ordered score keys of [s0, l_start) in sm.keys.
//  1. a strided sample of the scores is binned linearly between its minimum and the head maximum; the
//     bin edge below which about kk + margin tokens are expected becomes the candidate threshold U;
//  2. one pass collects the tokens with score >= U (each thread keeps a 32-bit take mask, positions
//     come from one block scan: no atomics in the loop);
//  3. the kk-th largest candidate is located by a second linear-bin histogram over [U, m] and an exact
//     ranking inside its bin;
//  4. candidates above T + 2 gamma are members, those within 2 gamma are rescored in fp64.
// On success the bitmap of I_t is in sm.w0.  Returns false (sm.w0 / sm.w1 undefined) when the generic
// path has to run.
template <typename T, int D>
__device__ bool topk_fast(const Prob& p, const Sm& sm, int b, int g, const T* qrow, const float* sc,
                          unsigned long long* kbar, int& landed, int s0, int l_start, int kk, int nw, float m, float gamma) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int mlen = l_start - s0;
  int* misc = sm.misc;
  float* fmisc = reinterpret_cast<float*>(misc);
  float U = -INFINITY;              // candidates are the tokens with score >= U
  int ncand = 0;
  float range2 = 0.f, inv_w2 = 0.f;  // linear bins of the candidates: bin = (m - score) * inv_w2
  bool have_hist = false;           // the candidate pass has filled the bins already
  if (tid == 0) { misc[2] = NBIN; misc[4] = 0; misc[5] = 0; misc[6] = -1; }
  const float* sf = reinterpret_cast<const float*>(sm.keys);   // raw scores, valid once the bulk copy has landed
  if (mlen <= CANDCAP) {
    landed = __syncthreads_and(mbar_wait(kbar, 0u)) ? 1 : -1;
    if (landed < 0) return false;
    for (int j = tid; j < mlen; j += NT) { sm.cand_idx[j] = s0 + j; sm.ckey[j] = ~ord_f32(sf[s0 + j]); }
    ncand = mlen;
    __syncthreads();
  } else {
    constexpr int SAMPLE = 2048;
    const int stride = (mlen + SAMPLE - 1) / SAMPLE;
    const int ms = (mlen + stride - 1) / stride;
    float smp[2];                                               // this thread's sample scores (ms <= 2048 = 2 NT)
    smp[0] = (tid < ms) ? __ldcg(sc + s0 + tid * stride) : INFINITY;
    smp[1] = (tid + NT < ms) ? __ldcg(sc + s0 + (tid + NT) * stride) : INFINITY;
    float smin = fminf(smp[0], smp[1]);
#pragma unroll
    for (int mk = 16; mk >= 1; mk >>= 1) smin = fminf(smin, __shfl_xor_sync(0xFFFFFFFFu, smin, mk));
    sm.lin[tid] = 0;
    if (lane == 0) fmisc[8 + warp] = smin;
    __syncthreads();
    smin = fmisc[8 + lane];
#pragma unroll
    for (int mk = 16; mk >= 1; mk >>= 1) smin = fminf(smin, __shfl_xor_sync(0xFFFFFFFFu, smin, mk));
    const float range = m - smin;
    const float inv_w = (range > 0.f) ? (float)NBIN / range : 0.f;
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      if (tid + u * NT < ms) {
        const float x = (m - smp[u]) * inv_w;
        atomicAdd(&sm.lin[x >= (float)(NBIN - 1) ? NBIN - 1 : (x > 0.f ? (int)x : 0)], 1);
      }
    }
    __syncthreads();
    const int cnt = sm.lin[tid];
    int tot1;
    const int excl1 = block_scan_reg(cnt, reinterpret_cast<int*>(sm.hist), tot1);
    const double fms = (double)kk * (double)ms / (double)mlen;
    const int r = (int)(fms + 4.0 * sqrt(fms) + 8.0);
    if (excl1 < r && r <= excl1 + cnt) misc[2] = tid;
    sm.lin[tid] = 0;                                            // every thread has read its bin: reuse for pass two
    landed = __syncthreads_and(mbar_wait(kbar, 0u)) ? 1 : -1;  // the scores have had the estimate's time to arrive
    if (landed < 0) return false;
    const int jstar = misc[2];
    if (jstar >= NBIN - 1) return false;                      // the sample cannot place the threshold
    U = m - (float)(jstar + 1) * (range / (float)NBIN);
    // One pass over the context: 32 tokens per thread, take mask in a register (no atomics in the loop);
    // positions come from one scan; the candidates are written and counted in linear bins over [U, m].
    range2 = m - U;
    inv_w2 = (range2 > 0.f) ? (float)NBIN / range2 : 0.f;
    have_hist = true;
    unsigned take = 0u;
    const int base_i = s0 + tid;
#pragma unroll 8
    for (int it = 0; it < 32; ++it) {
      const int i = base_i + it * NT;
      if (i < l_start && sf[i] >= U) take |= 1u << it;
    }
    bool beyond = false;
    for (int it = 32; base_i + it * NT < l_start; ++it)       // contexts longer than 32 * NT tokens
      beyond = beyond || (sf[base_i + it * NT] >= U);
    if (beyond) misc[6] = -2;
    int pos = block_scan_reg(__popc(take), reinterpret_cast<int*>(sm.hist) + 64, ncand);
    if (misc[6] == -2 || ncand < kk || ncand > CANDCAP) return false;     // (misc[6] was written before the barrier)
    while (take) {
      const int it = __ffs(take) - 1;
      take &= take - 1;
      const int i = base_i + it * NT;
      const float sv = sf[i];
      sm.cand_idx[pos] = i;
      sm.ckey[pos] = ~ord_f32(sv);
      const float x = (m - sv) * inv_w2;
      atomicAdd(&sm.lin[x >= (float)(NBIN - 1) ? NBIN - 1 : (x > 0.f ? (int)x : 0)], 1);
      ++pos;
    }
    __syncthreads();
  }
  // ---- the kk-th largest candidate: linear bins over [cmin, m] (or [U, m]), exact ranking inside the bin
  if (!have_hist) {
    float cmin = INFINITY;
    for (int j = tid; j < ncand; j += NT) cmin = fminf(cmin, unord_f32(~sm.ckey[j]));
#pragma unroll
    for (int mk = 16; mk >= 1; mk >>= 1) cmin = fminf(cmin, __shfl_xor_sync(0xFFFFFFFFu, cmin, mk));
    sm.lin[tid] = 0;
    if (lane == 0) fmisc[8 + warp] = cmin;
    __syncthreads();
    cmin = fmisc[8 + lane];
#pragma unroll
    for (int mk = 16; mk >= 1; mk >>= 1) cmin = fminf(cmin, __shfl_xor_sync(0xFFFFFFFFu, cmin, mk));
    range2 = m - cmin;
    inv_w2 = (range2 > 0.f) ? (float)NBIN / range2 : 0.f;
  }
  auto bin2 = [&](unsigned key) -> int {
    const float x = (m - unord_f32(~key)) * inv_w2;
    return x >= (float)(NBIN - 1) ? NBIN - 1 : (x > 0.f ? (int)x : 0);
  };
  if (!have_hist) {
    for (int j = tid; j < ncand; j += NT) atomicAdd(&sm.lin[bin2(sm.ckey[j])], 1);
    __syncthreads();
  }
  const int cnt2 = sm.lin[tid];
  {
    int tot2;
    const int excl = block_scan_reg(cnt2, reinterpret_cast<int*>(sm.hist) + 32, tot2);
    if (excl < kk && kk <= excl + cnt2) { misc[6] = tid; misc[7] = kk - excl; }
  }
  __syncthreads();
  const int jb = misc[6], r_in = misc[7];
  if (jb < 0) return false;
  for (int j = tid; j < ncand; j += NT) {
    if (bin2(sm.ckey[j]) == jb) {
      const int pos = atomicAdd(&misc[4], 1);
      if (pos < VATTN_BANDCAP) sm.band_idx[pos] = j;
    }
  }
  __syncthreads();
  const int nmem = misc[4];
  if (nmem > VATTN_BANDCAP) return false;
  for (int a = tid; a < nmem; a += NT) {                      // r_in-th largest score of the bin (value only)
    const unsigned mine = sm.ckey[sm.band_idx[a]];
    int less = 0, leq = 0;                                    // inverted keys: smaller key = larger score
    for (int u = 0; u < nmem; ++u) {
      const unsigned o = sm.ckey[sm.band_idx[u]];
      less += o < mine;
      leq += o <= mine;
    }
    if (less < r_in && r_in <= leq) misc[3] = (int)mine;      // all writers hold the same key
  }
  __syncthreads();
  const unsigned Tk = (unsigned)misc[3];
  const float Tf = unord_f32(~Tk);
  const float hi = __fadd_ru(Tf, 2.f * gamma), lo = __fadd_rd(Tf, -2.f * gamma);
  // every token that could still enter the top-k (score >= lo) must be a candidate
  if (!(lo >= U)) return false;
  for (int w = tid; w < nw; w += NT) sm.w0[w] = 0u;
  if (tid == 0) { misc[4] = 0; misc[5] = 0; }
  __syncthreads();
  int in_local = 0;
  for (int j = tid; j < ncand; j += NT) {
    const int idx = sm.cand_idx[j];
    const float s = unord_f32(~sm.ckey[j]);
    if (s > hi) { atomicOr(&sm.w0[idx >> 5], 1u << (idx & 31)); ++in_local; }
    else if (s >= lo) {
      const int pos = atomicAdd(&misc[5], 1);
      if (pos < VATTN_BANDCAP) sm.band_idx[pos] = idx;
    }
  }
#pragma unroll
  for (int mk = 16; mk >= 1; mk >>= 1) in_local += __shfl_xor_sync(0xFFFFFFFFu, in_local, mk);
  if (lane == 0 && in_local) atomicAdd(&misc[4], in_local);
  __syncthreads();
  const int n_in = misc[4], n_band = misc[5];
  const int need = kk - n_in;
  if (n_band > VATTN_BANDCAP) return false;
  if (need >= n_band) {
    for (int c = tid; c < n_band; c += NT) { const int idx = sm.band_idx[c]; atomicOr(&sm.w0[idx >> 5], 1u << (idx & 31)); }
  } else {
    for (int c = warp; c < n_band; c += NWARP) {
      const double s64 = score64_warp<T, D>(p, b, g, qrow, sm.band_idx[c]);
      if (lane == 0) sm.band_s[c] = s64;
    }
    __syncthreads();
    for (int c = tid; c < n_band; c += NT) {
      const double mine = sm.band_s[c];
      const int mi = sm.band_idx[c];
      int rank = 0;
      for (int u = 0; u < n_band; ++u) {
        const double o = sm.band_s[u];
        rank += (o > mine) || (o == mine && sm.band_idx[u] < mi);
      }
      if (rank < need) atomicOr(&sm.w0[mi >> 5], 1u << (mi & 31));
    }
  }
  __syncthreads();
  return true;
}

// top-k, generic path: radix select over the whole middle range (any size, any score distribution)
template <typename T, int D, bool CACHED>
__device__ void topk_generic(const Prob& p, const Sm& sm, int b, int g, const T* qrow, const float* sc, int s0,
                             int l_start, int kk, int nw, float gamma) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  auto keyfn = [&](int i, unsigned& key) -> bool { key = CACHED ? sm.keys[i] : ~ord_f32(sc[i]); return true; };
  unsigned Tk; int need_eq;
  block_select<unsigned, true>(keyfn, s0, l_start, kk, sm.hist, sm.misc, Tk, need_eq);
  const float Tf = unord_f32(~Tk);
  const float hi = __fadd_ru(Tf, 2.f * gamma), lo = __fadd_rd(Tf, -2.f * gamma);
  // certain members -> w0, near-tie band -> w1
  for (int w = warp; w < nw; w += NWARP) {
    const int i = w * 32 + lane;
    const bool ok = (i >= s0) && (i < l_start);
    const float s = ok ? (CACHED ? unord_f32(~sm.keys[i]) : sc[i]) : 0.f;
    const unsigned in = __ballot_sync(0xFFFFFFFFu, ok && s > hi);
    const unsigned band = __ballot_sync(0xFFFFFFFFu, ok && !(s > hi) && s >= lo);
    if (lane == 0) { sm.w0[w] = in; sm.w1[w] = band; }
  }
  __syncthreads();
  for (int w = tid; w < nw; w += NT) sm.scan[w] = __popc(sm.w0[w]);
  __syncthreads();
  const int n_in = block_excl_scan(sm.scan, nw, sm.misc);
  for (int w = tid; w < nw; w += NT) sm.scan[w] = __popc(sm.w1[w]);
  __syncthreads();
  const int n_band = block_excl_scan(sm.scan, nw, sm.misc);      // scan[w] = rank of word w's first band bit
  const int need = kk - n_in;                                     // 1 <= need <= n_band
  if (need >= n_band) {
    for (int w = tid; w < nw; w += NT) sm.w0[w] |= sm.w1[w];
    __syncthreads();
  } else if (n_band <= VATTN_BANDCAP) {
    // band list ascending by index, exact scores, O(band^2) ranking by (-score, index)
    for (int w = tid; w < nw; w += NT) {
      unsigned bits = sm.w1[w];
      int pos = sm.scan[w];
      while (bits) { const int bit = __ffs(bits) - 1; bits &= bits - 1; sm.band_idx[pos++] = w * 32 + bit; }
    }
    __syncthreads();
    for (int c = warp; c < n_band; c += NWARP) {
      const double s64 = score64_warp<T, D>(p, b, g, qrow, sm.band_idx[c]);
      if (lane == 0) sm.band_s[c] = s64;
    }
    __syncthreads();
    for (int c = tid; c < n_band; c += NT) {
      const double mine = sm.band_s[c];
      int rank = 0;
      for (int u = 0; u < n_band; ++u) {
        const double o = sm.band_s[u];
        rank += (o > mine) || (o == mine && u < c);
      }
      if (rank < need) { const int idx = sm.band_idx[c]; atomicOr(&sm.w0[idx >> 5], 1u << (idx & 31)); }
    }
    __syncthreads();
  } else {
    // too many near-ties for the list: exact 64-bit radix select over the band, scores recomputed on the fly
    if (tid == 0) atomicOr(p.status, VATTN_STATUS_BAND_OVERFLOW);
    auto key64 = [&](int i, unsigned long long& key) -> bool {
      if (!((sm.w1[i >> 5] >> (i & 31)) & 1u)) return false;
      key = ~ord_f64(score64_thread<T, D>(p, b, g, qrow, i));
      return true;
    };
    unsigned long long T64; int need_eq64;
    block_select<unsigned long long, true>(key64, s0, l_start, need, sm.hist, sm.misc, T64, need_eq64);
    for (int w = warp; w < nw; w += NWARP) {
      const int i = w * 32 + lane;
      unsigned long long key = 0;
      bool ok = (i >= s0) && (i < l_start);
      if (ok) ok = key64(i, key);
      const unsigned lt = __ballot_sync(0xFFFFFFFFu, ok && key < T64);
      const unsigned eq = __ballot_sync(0xFFFFFFFFu, ok && key == T64);
      if (lane == 0) { sm.w0[w] |= lt; sm.w2[w] = eq; }
    }
    __syncthreads();
    for (int w = tid; w < nw; w += NT) sm.scan[w] = __popc(sm.w2[w]);
    __syncthreads();
    block_excl_scan(sm.scan, nw, sm.misc);
    for (int w = tid; w < nw; w += NT) sm.w0[w] |= lowest_bits(sm.w2[w], need_eq64 - sm.scan[w]);
    __syncthreads();
  }
}

template <typename T, int D, bool CACHED>
__global__ void __launch_bounds__(NT, 1) k_select_topk(const Prob p, int bigbytes) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int h = blockIdx.x, b = blockIdx.y, g = h / p.G;
  const int bh = b * p.Hq + h;
  TICK_BEGIN(p, VATTN_K_TOPK);
  __shared__ unsigned long long kbar;         // completion of the bulk copy of the scores
  const Sm sm = carve(smem_raw, bigbytes, p.nwords);
  HeadMeta& meta = p.meta[bh];

  // before the wait: everything that depends on the step's inputs only
  const int n = clamped_len(p, b);
  const Geo geo = head_geometry(p, n);
  const int s0 = geo.s0, l_start = geo.l_start, kk = geo.kk, n_s = geo.n_s, b0 = geo.b0;
  const int mlen = l_start - s0;
  const int nw = (n + 31) >> 5;
  const T* qrow = reinterpret_cast<const T*>(p.q) + (long long)bh * D;
  const float* sc = p.scores + (long long)bh * p.npad;
  double sa = 0.0;                      // sum |q_e| (warp 0)
  if (warp == 0) {
    for (int e = lane; e < D; e += 32) sa += fabs((double)Elem<T>::to_float(qrow[e]));
#pragma unroll
    for (int mk = 16; mk >= 1; mk >>= 1) sa += __shfl_xor_sync(0xFFFFFFFFu, sa, mk);
  }
  for (int w = tid; w < nw; w += NT) { sm.w0[w] = 0u; sm.w1[w] = 0u; }
  pdl_wait();
  pdl_trigger();                      // dependents may read the score kernel's outputs before their own wait
  const float m = (n > 0) ? unord_f32(__ldcg(p.m_ord + bh)) : 0.f;

  // gamma: bound on |fp32 score - exact score|.  fp32 path: at most 13 roundings (x16 = margin).
  // bf16 tensor-core path: at most 8 accumulation steps of 16 exact products each (two chains of 4 and one
  // addition for d = 128), every step assumed to lose up to 17 units of 2^-23 of the running magnitude
  // (truncating adder) -> 8*17*2 = 272, taken as 512.
  if (warp == 0) {
    const double kmax = (double)__uint_as_float(__ldcg(p.kabsmax + b * p.Hkv + g));
    const double roundings = (p.dtype == VATTN_DTYPE_BF16) ? 512.0 : 16.0;
    const double gm = roundings * 5.9604644775390625e-8 * fabs((double)p.scale) * sa * kmax * 1.000001;
    if (lane == 0) reinterpret_cast<float*>(sm.misc)[48] = __double2float_ru(gm);
  }
  const bool staged = CACHED && kk > 0 && kk < mlen;
  if (staged && tid == 0) {
    // the scores of the middle range travel to shared memory as one asynchronous bulk copy (raw fp32, the
    // 16-byte aligned span around [s0, l_start)); the threshold estimate below runs meanwhile on a sample
    // it reads from global memory
    const int a0 = s0 & ~3, a1 = (l_start + 3) & ~3;             // within the padded row: npad is a multiple of 32
    mbar_init(&kbar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    mbar_expect_tx(&kbar, (unsigned)(a1 - a0) * 4u);
    bulk_g2s(sm.keys + a0, sc + a0, (unsigned)(a1 - a0) * 4u, &kbar);
  }
  __syncthreads();
  const float gamma = reinterpret_cast<float*>(sm.misc)[48];
  if (tid == 0) {
    meta.n = n; meta.s0 = s0; meta.l_start = l_start; meta.kk = kk; meta.n_s = n_s; meta.b0 = b0;
    meta.b = 0; meta.m = m; meta.gamma = gamma;
    if (p.dbg.topk_cnt) p.dbg.topk_cnt[bh] = kk;
    if (p.dbg.base_cnt) p.dbg.base_cnt[bh] = b0;
  }
  unsigned* gbitmap = p.bitmap + (long long)bh * p.nwords;
  if (n == 0) { if (p.dbg.paths && tid == 0) p.dbg.paths[bh] = 0; return; }

  int path = 0;
  // ------------------------------------------------------------------ top-k over the middle range
  if (kk > 0 && kk == mlen) {
    for (int w = tid; w < nw; w += NT) {
      const int i0 = w * 32;
      unsigned mk = 0xFFFFFFFFu;
      if (i0 < s0) mk &= (s0 - i0 >= 32) ? 0u : (0xFFFFFFFFu << (s0 - i0));
      if (i0 + 32 > l_start) mk &= (l_start <= i0) ? 0u : (0xFFFFFFFFu >> (i0 + 32 - l_start));
      sm.w0[w] = mk;
    }
    __syncthreads();
  } else if (kk > 0) {
    bool done = false;
    if (CACHED) {
      int landed = 0;                                  // 1: the scores are in shared memory, -1: the copy never arrived
      done = topk_fast<T, D>(p, sm, b, g, qrow, sc, &kbar, landed, s0, l_start, kk, nw, m, gamma);
      if (done) path |= 1;
      if (!done) {
        // the generic select wants order-reversed integer keys: wait for the copy if nobody has yet, convert
        if (landed == 0) landed = __syncthreads_and(mbar_wait(&kbar, 0u)) ? 1 : -1;
        if (landed < 0) {                              // give up on this head: report, leave I_t empty
          if (tid == 0) atomicOr(p.status, VATTN_STATUS_WAIT_TIMEOUT);
          mbar_wait(&kbar, 0u);                        // a second bounded chance before the buffer is released
        } else {
          for (int i = s0 + tid; i < l_start; i += NT) sm.keys[i] = ~ord_f32(__uint_as_float(sm.keys[i]));
        }
      }
    }
    if (!done) {
      __syncthreads();
      for (int w = tid; w < nw; w += NT) { sm.w0[w] = 0u; sm.w1[w] = 0u; }
      __syncthreads();
      topk_generic<T, D, CACHED>(p, sm, b, g, qrow, sc, s0, l_start, kk, nw, gamma);
    }
  }
  // emit I_t ascending, keep its bitmap (shared w2 + global)
  int* tk_out = p.topk_idx + (long long)bh * p.npad;
  int* tk_dbg = p.dbg.topk_idx ? p.dbg.topk_idx + (long long)bh * p.max_seq_len : nullptr;
  finalize_emit(p, b, sm.w0, sm.w1, 0, nw, sm.scan, sm.misc, tk_out, tk_dbg);
  for (int w = tid; w < p.nwords; w += NT) {
    const unsigned v = (w < nw) ? sm.w0[w] : 0u;
    sm.w2[w] = v;
    gbitmap[w] = v;
  }
  __syncthreads();

  if (p.dbg.paths && tid == 0) p.dbg.paths[bh] = path;
  TICK_END(p, VATTN_K_TOPK);
}

// Sampling without a selection on the critical path (Algorithm 2 line 1 and Algorithm 1 line 7).
// grid.z = Philox stream: 0 draws the base sample I_bs, 1 prepares the final sample I_dyn.
//
// "The c smallest (key, token) pairs of the residual" is a prefix of the residual's pairs in sorted order,
// whatever c is.  The pre-filtered candidate list of the score kernel holds every middle token whose key
// is below a bound, so sorting it needs nothing from the top-k selection: it happens BEFORE this grid's
// dependency wait, while k_select_topk still runs on other SMs (counting sort into 4096 buckets by a
// monotone function of the key, then every pair ranks itself inside its bucket).  After the wait only the
// members of I_t are dropped, by an order-preserving compaction: stream 0 keeps the first b0 survivors,
// stream 1 all of them (the gather kernel later reads the first b, once b is known).  Lists that cannot
// serve (overflow, too long for shared memory, fewer than b0 survivors, b0 = whole residual) fall back to
// the full-context select: here for stream 0, in k_budget for stream 1 (sorted_cnt = -1).
constexpr int SORT_BUCKETS = 4096;
constexpr int SORT_BUCKET_MAX = 64;
constexpr size_t SORT_FIXED_BYTES = sizeof(int) * (2 * SORT_BUCKETS + 1 + 64);      // + nwords words
template <bool CACHED>
__global__ void __launch_bounds__(NT, 1) k_presort(const Prob p, int paircap, int bigbytes) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int h = blockIdx.x, b = blockIdx.y, stream = blockIdx.z, g = h / p.G;
  const int bh = b * p.Hq + h;
  TICK_BEGIN(p, VATTN_K_PRESORT);
  uint2* pairs = reinterpret_cast<uint2*>(smem_raw);          // [paircap] bucketed (key, token), later sorted (token, slot)
  int* srt = reinterpret_cast<int*>(pairs + paircap);         // [paircap] tokens in sorted order
  int* off = srt + paircap;                                   // [SORT_BUCKETS + 1] bucket starts
  int* cur = off + SORT_BUCKETS + 1;                          // [SORT_BUCKETS] fill cursors
  int* misc = cur + SORT_BUCKETS;                             // [64]
  unsigned* bits = reinterpret_cast<unsigned*>(misc + 64);    // [nwords] bitmap of I_t

  // ------------------------------------------------ before the wait: step inputs and score-kernel lists only
  const int n = clamped_len(p, b);
  const Geo geo = head_geometry(p, n);
  const long long l = (long long)stream * p.B * p.Hq + bh;
  const unsigned bound = stream ? VATTN_CAND1_BOUND : cand0_bound(geo);
  bool usable = n > 0 && geo.n_s > 0 && bound != 0u && (stream == 1 || geo.b0 < geo.n_s);
  unsigned cnt = 0;
  if (usable) {
    cnt = __ldcg(p.cand_cnt + l);
    usable = cnt <= (unsigned)p.cand_cap && cnt <= (unsigned)paircap;
  }
  int nall = 0;
  if (usable) {
    const uint2* glist = p.cand + l * p.cand_cap;
    const float bscale = (float)SORT_BUCKETS / (float)bound;
    auto bucket_of = [&](unsigned key) -> int {               // monotone in key
      const int x = (int)((float)key * bscale);
      return x > SORT_BUCKETS - 1 ? SORT_BUCKETS - 1 : x;
    };
    for (int j = tid; j <= SORT_BUCKETS; j += NT) off[j] = 0;
    if (tid == 0) misc[0] = 0;
    __syncthreads();
    for (int j0 = tid; j0 < (int)cnt; j0 += 4 * NT) {
      uint2 e[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) e[u] = (j0 + u * NT < (int)cnt) ? __ldcg(glist + j0 + u * NT) : make_uint2(0u, 0xFFFFFFFFu);
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (e[u].y < (unsigned)n) atomicAdd(&off[bucket_of(e[u].x)], 1);
    }
    __syncthreads();
    for (int j = tid; j < SORT_BUCKETS; j += NT)
      if (off[j] > SORT_BUCKET_MAX) misc[0] = 1;
    __syncthreads();
    nall = block_excl_scan(off, SORT_BUCKETS, misc);           // scratch misc[8..40]
    if (misc[0]) usable = false;
    else {
      for (int j = tid; j < SORT_BUCKETS; j += NT) cur[j] = off[j];
      if (tid == 0) off[SORT_BUCKETS] = nall;
      __syncthreads();
      for (int j0 = tid; j0 < (int)cnt; j0 += 4 * NT) {
        uint2 e[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) e[u] = (j0 + u * NT < (int)cnt) ? __ldcg(glist + j0 + u * NT) : make_uint2(0u, 0xFFFFFFFFu);
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (e[u].y < (unsigned)n) pairs[atomicAdd(&cur[bucket_of(e[u].x)], 1)] = e[u];
      }
      __syncthreads();
      // neighbouring threads hold pairs of the same bucket: the reads below are mostly broadcasts
      for (int i = tid; i < nall; i += NT) {
        const uint2 e = pairs[i];
        const int bk = bucket_of(e.x);
        const int lo = off[bk], hi = off[bk + 1];
        int rank = 0;
        for (int v = lo; v < hi; ++v) {
          const uint2 o = pairs[v];
          rank += (o.x < e.x) || (o.x == e.x && o.y < e.y);
        }
        srt[lo + rank] = (int)e.y;
      }
      __syncthreads();
      for (int i = tid; i < nall; i += NT) {                   // the keys are spent: (token, physical slot) in their place
        const int tok = srt[i];
        pairs[i] = make_uint2((unsigned)tok, (unsigned)(page_of(p, b, tok >> 4) * VATTN_BLOCK + (tok & 15)));
      }
    }
  }
  pdl_wait();                         // the bitmap of I_t and meta come from k_select_topk
  pdl_trigger();
  HeadMeta& meta = p.meta[bh];
  if (n == 0 || geo.n_s <= 0) { if (stream == 1 && tid == 0) meta.sorted_cnt = 0; return; }
  if (stream == 0 && geo.b0 <= 0) return;
  const int nw = (n + 31) >> 5;
  const unsigned* gbitmap = p.bitmap + (long long)bh * p.nwords;

  if (usable) {
    for (int w = tid; w < nw; w += NT) bits[w] = __ldcg(gbitmap + w);
    __syncthreads();                                           // also orders the last writes to pairs[]
    // order-preserving compaction: warp w owns the sorted entries [w_lo, w_hi)
    const int seg = ((nall + NWARP - 1) / NWARP + 31) & ~31;
    const int w_lo = min(nall, warp * seg), w_hi = min(nall, w_lo + seg);
    int kept = 0;
    for (int i0 = w_lo; i0 < w_hi; i0 += 32) {
      const int i = i0 + lane;
      bool keep = false;
      if (i < w_hi) { const unsigned tok = pairs[i].x; keep = !((bits[tok >> 5] >> (tok & 31)) & 1u); }
      kept += __popc(__ballot_sync(0xFFFFFFFFu, keep));
    }
    if (lane == 0) misc[8 + warp] = kept;
    __syncthreads();
    if (warp == 0) {
      const int v = misc[8 + lane];
      int incl = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += u;
      }
      misc[8 + lane] = incl - v;
      if (lane == 31) misc[40] = incl;
    }
    __syncthreads();
    const int total = misc[40];
    if (stream == 1 || total >= geo.b0) {
      const int limit = stream ? total : geo.b0;
      int* out = stream ? p.sort_idx + (long long)bh * p.cand_cap : p.base_idx + (long long)bh * p.npad;
      const long long delta = stream ? p.sort_phys_delta : p.phys_delta;
      int* dbg = (stream == 0 && p.dbg.base_idx) ? p.dbg.base_idx + (long long)bh * p.max_seq_len : nullptr;
      int run = misc[8 + warp];
      for (int i0 = w_lo; i0 < w_hi && run < limit; i0 += 32) {
        const int i = i0 + lane;
        bool keep = false;
        uint2 e = make_uint2(0u, 0u);
        if (i < w_hi) { e = pairs[i]; keep = !((bits[e.x >> 5] >> (e.x & 31)) & 1u); }
        const unsigned bal = __ballot_sync(0xFFFFFFFFu, keep);
        const int pos = run + __popc(bal & ((1u << lane) - 1u));
        if (keep && pos < limit) {
          out[pos] = (int)e.x;
          out[delta + pos] = (int)e.y;
          if (dbg) dbg[pos] = (int)e.x;
        }
        run += __popc(bal);
      }
      if (tid == 0) {
        if (stream == 1) meta.sorted_cnt = total;
        else if (p.dbg.paths) atomicOr(&p.dbg.paths[bh], 2);
      }
      TICK_END(p, VATTN_K_PRESORT);
      return;
    }
  }
  if (stream == 1) { if (tid == 0) meta.sorted_cnt = -1; return; }
  // base sample from the full context
  __syncthreads();
  const Sm sm = carve(smem_raw, bigbytes, p.nwords);
  for (int w = tid; w < nw; w += NT) sm.w2[w] = __ldcg(gbitmap + w);
  __syncthreads();
  const int hrng = p.rng_head_is_kv ? g : h;
  int* bs_out = p.base_idx + (long long)bh * p.npad;
  int* bs_dbg = p.dbg.base_idx ? p.dbg.base_idx + (long long)bh * p.max_seq_len : nullptr;
  sample_select<CACHED>(p, sm, geo.s0, geo.l_start, nw, geo.b0, geo.n_s, b, hrng, 0, sm.w2, bs_out, bs_dbg);
  TICK_END(p, VATTN_K_PRESORT);
}

// Budget (Algorithm 2, Theorem 4.3 / Corollaries D.2) and the slow path of the final sample.
//
// One CTA per head.  The partials of the statistics kernel are added in split order (every thread requests
// all partials of its element at once: one memory round trip), then warp 0 evaluates
//     sigma^2, Tr(Sigma), D_hat, |N_hat|,  b_D, b_N, b_SDPA,  b = clamp(ceil(b_X), b0, n_s)
// in fp64 (the two square-root / division chains on two lanes, the 15 split points of b_SDPA on 15 lanes).
// Heads whose I_dyn is a prefix of the pre-sorted list (b < n_s and b <= sorted_cnt) are done: the gather
// kernel reads the prefix (it is copied to the debug buffer when one is registered).  For the others the
// sample is drawn from the full context and written ascending to dyn_idx.
__device__ __forceinline__ int ceil_sat(double x) {
  if (!isfinite(x) || x >= 2147483647.0) return 2147483647;
  return (int)ceil(x);
}

template <bool CACHED>
__global__ void __launch_bounds__(NT, 1) k_budget(const Prob p, int bigbytes) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ double tot[2][128 + 3];
  __shared__ double piv[128 + 1];
  __shared__ int s_b;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int h = blockIdx.x, b = blockIdx.y, g = h / p.G;
  const int bh = b * p.Hq + h;
  TICK_BEGIN(p, VATTN_K_BUDGET);
  pdl_trigger();
  pdl_wait();
  const int D = p.D, NE = D + 3;
  // ---- partial sums in split order; kind 0 = deterministic rows, kind 1 = base-sample rows.  The requests
  // depend on nothing but the head's number: they go out together with the read of the head's meta record.
  double item_sum[(2 * (128 + 3) + NT - 1) / NT];
#pragma unroll
  for (int it = 0; it < (2 * (128 + 3) + NT - 1) / NT; ++it) {
    const int item = tid + it * NT;
    double sum = 0.0;
    if (item < 2 * NE) {
      const int kind = item / NE, e = item % NE;
      const int S = kind ? p.stat_splits_base : p.stat_splits;
      const double* src = p.stat_part + ((long long)bh * 2 * VATTN_STAT_MAXS + kind * VATTN_STAT_MAXS) * NE + e;
      double v[VATTN_STAT_MAXS];
#pragma unroll
      for (int sp = 0; sp < VATTN_STAT_MAXS; ++sp) v[sp] = (sp < S) ? __ldcg(src + (long long)sp * NE) : 0.0;
#pragma unroll
      for (int sp = 0; sp < VATTN_STAT_MAXS; ++sp) sum += v[sp];
    }
    item_sum[it] = sum;
  }
  // the pivot the base-row CTAs used (all of them computed the same numbers; split 0 published them)
  double piv_v[(128 + 1 + NT - 1) / NT];
#pragma unroll
  for (int it = 0; it < (128 + 1 + NT - 1) / NT; ++it) {
    const int e = tid + it * NT;
    piv_v[it] = (e <= D) ? __ldcg(p.stat_piv + (long long)bh * (D + 1) + e) : 0.0;
  }
  HeadMeta meta = p.meta[bh];
  const int n_s = meta.n_s, b0 = meta.b0;
  if (meta.n == 0) {
    if (tid == 0) {
      p.meta[bh].b = 0;
      if (p.dbg.dyn_cnt) p.dbg.dyn_cnt[bh] = 0;
      if (p.dbg.budgets) for (int e = 0; e < 4; ++e) p.dbg.budgets[bh * 4 + e] = 0;
      if (p.dbg.stats) for (int e = 0; e < 8; ++e) p.dbg.stats[bh * 8 + e] = 0.0;
    }
    return;
  }
#pragma unroll
  for (int it = 0; it < (2 * (128 + 3) + NT - 1) / NT; ++it) {
    const int item = tid + it * NT;
    if (item < 2 * NE) tot[item / NE][item % NE] = item_sum[it];
  }
#pragma unroll
  for (int it = 0; it < (128 + 1 + NT - 1) / NT; ++it) {
    const int e = tid + it * NT;
    if (e <= D) piv[e] = (b0 > 0) ? piv_v[it] : 0.0;     // no base sample: the record holds an earlier step's numbers
  }
  __syncthreads();
  double* det = p.det_sums + (long long)bh * (D + 1);
  for (int e = tid; e <= D; e += NT) det[e] = tot[0][e];
  if (warp == 0) {
    const double Dfv = tot[0][D];
    const double ratio = (b0 > 0) ? (double)n_s / (double)b0 : 0.0;
    double nn = 0.0, sr2 = 0.0;                 // |N_hat|^2 and sum_j (sum_i r'_ij)^2
    for (int e = lane; e < D; e += 32) {
      const double srj = tot[1][e];
      const double nh = tot[0][e] + ratio * (srj + (double)b0 * piv[e]);
      nn = fma(nh, nh, nn);
      sr2 = fma(srj, srj, sr2);
    }
#pragma unroll
    for (int mask = 16; mask >= 1; mask >>= 1) {
      nn += __shfl_xor_sync(0xFFFFFFFFu, nn, mask);
      sr2 += __shfl_xor_sync(0xFFFFFFFFu, sr2, mask);
    }
    const double Nnorm = sqrt(nn);
    double sigma2 = 0.0, trace = 0.0, Dhat = Dfv, A = 0.0, Bn = 0.0;
    int bD = 0, bN = 0, bS = 0, bfin = 0;
    if (n_s > 0) {                              // uniform over the warp
      const double Swv = tot[1][D], Swwv = tot[1][D + 1], Srrv = tot[1][D + 2];
      // lane 0: the denominator chain, lane 1: the numerator chain (each: division, square root, division)
      if (lane == 0) {
        if (b0 >= 2) sigma2 = fmax(0.0, (Swwv - Swv * Swv / (double)b0) / (double)(b0 - 1));
        Dhat = Dfv + ratio * (Swv + (double)b0 * piv[D]);
        A = (double)n_s * sqrt(sigma2) / Dhat;
      } else if (lane == 1) {
        if (b0 >= 2) trace = fmax(0.0, (Srrv - sr2 / (double)b0) / (double)(b0 - 1));
        Bn = (double)n_s * sqrt(trace) / Nnorm;
      }
      A = __shfl_sync(0xFFFFFFFFu, A, 0);
      Bn = __shfl_sync(0xFFFFFFFFu, Bn, 1);
      trace = __shfl_sync(0xFFFFFFFFu, trace, 1);
      // b_SDPA: lane jj takes split point jj of the failure probability
      double c2 = CUDART_INF;
      if (lane < 15) {
        const double c = p.z1[lane] * A + p.z2[lane] * Bn;
        c2 = c * c;
      }
      const bool nan = __any_sync(0xFFFFFFFFu, c2 != c2);
      double mn = c2;
#pragma unroll
      for (int mask = 16; mask >= 1; mask >>= 1) mn = fmin(mn, __shfl_xor_sync(0xFFFFFFFFu, mn, mask));
      if (lane == 0) {
        double t = p.z_delta * A / p.eps;
        const double b_D = t * t;
        t = p.z_delta * Bn / p.eps;
        const double b_N = t * t;
        const double b_S = nan ? CUDART_NAN : 4.0 / (p.eps * p.eps) * mn;
        bD = ceil_sat(b_D); bN = ceil_sat(b_N); bS = ceil_sat(b_S);
        const double bx = p.mode == 1 ? b_D : (p.mode == 2 ? b_N : b_S);
        if (p.force_budget >= 0) bfin = min(p.force_budget, n_s);
        else {
          if (!isfinite(bx)) atomicOr(p.status, VATTN_STATUS_NONFINITE);
          bfin = min(max(ceil_sat(bx), b0), n_s);
        }
      }
    }
    if (lane == 0) {
      s_b = bfin;
      p.meta[bh].b = bfin;
      if (p.dbg.dyn_cnt) p.dbg.dyn_cnt[bh] = bfin;
      if (p.dbg.budgets) {
        int* o = p.dbg.budgets + bh * 4;
        o[0] = bD; o[1] = bN; o[2] = bS; o[3] = bfin;
      }
      if (p.dbg.stats) {
        double* o = p.dbg.stats + bh * 8;
        o[0] = Dfv; o[1] = sigma2; o[2] = trace; o[3] = Dhat; o[4] = Nnorm; o[5] = (double)n_s; o[6] = (double)b0;
        o[7] = (double)meta.m;
      }
    }
  }
  __syncthreads();
  meta.b = s_b;
  if (meta.b <= 0) { TICK_END(p, VATTN_K_BUDGET); return; }
  // ---- final sample
  if (meta.b < meta.n_s && meta.sorted_cnt >= meta.b) {
    if (p.dbg.dyn_idx) {
      const int* src = p.sort_idx + (long long)bh * p.cand_cap;
      int* dbg = p.dbg.dyn_idx + (long long)bh * p.max_seq_len;
      for (int i = tid; i < meta.b; i += NT) dbg[i] = src[i];
    }
    if (p.dbg.paths && tid == 0) atomicOr(&p.dbg.paths[bh], 4);
    TICK_END(p, VATTN_K_BUDGET);
    return;
  }
  const Sm sm = carve(smem_raw, bigbytes, p.nwords);
  const int nw = (meta.n + 31) >> 5;
  const unsigned* gbitmap = p.bitmap + (long long)bh * p.nwords;
  for (int w = tid; w < nw; w += NT) sm.w2[w] = gbitmap[w];
  __syncthreads();
  const int hrng = p.rng_head_is_kv ? g : h;
  int* out = p.dyn_idx + (long long)bh * p.npad;
  int* dbg = p.dbg.dyn_idx ? p.dbg.dyn_idx + (long long)bh * p.max_seq_len : nullptr;
  sample_select<CACHED>(p, sm, meta.s0, meta.l_start, nw, meta.b, meta.n_s, b, hrng, 1, sm.w2, out, dbg);
  TICK_END(p, VATTN_K_BUDGET);
}

}  // namespace

static int keycap_of(const Prob& p) { return p.npad <= VATTN_KEYCACHE_MAX ? p.npad : 0; }
// bytes of the shared "big" region: the context's select keys, or staged candidate pairs
static int big_bytes(const Prob& p, bool final_kernel) {
  const size_t keys = sizeof(unsigned) * (size_t)keycap_of(p);
  const size_t pairs = sizeof(uint2) * (size_t)(final_kernel ? p.cand_cap : PAIRCAP0);
  size_t b = keys > pairs ? keys : pairs;
  const size_t fixed = sizeof(double) * VATTN_BANDCAP + 4 * sizeof(unsigned) * (size_t)p.nwords + sizeof(unsigned) * 256 +
                       sizeof(int) * (VATTN_BANDCAP + NBIN + 2 * CANDCAP + 64);
  const size_t limit = 222 * 1024;                            // 227 KB per CTA minus the kernels' static arrays
  if (fixed + b > limit) b = (limit - fixed) / 16 * 16;       // fewer staged pairs: the list path then declines
  return (int)b;
}

// Opt-in to large dynamic shared memory once per kernel and size (a function attribute, not a
// stream operation; done before the first launch so that later launches can be stream-captured).
template <typename KernelT>
static cudaError_t launch_sel(KernelT kern, const Prob& p, cudaStream_t s, bool final_kernel) {
  const int big = big_bytes(p, final_kernel);
  const size_t smem = sizeof(double) * VATTN_BANDCAP + 4 * sizeof(unsigned) * (size_t)p.nwords + sizeof(unsigned) * 256 +
                      sizeof(int) * (VATTN_BANDCAP + NBIN + 2 * CANDCAP + 64) + (size_t)big;
  static const void* seen_fn[32];
  static size_t seen_sz[32];
  static int nseen = 0;
  bool done = false;
  for (int i = 0; i < nseen; ++i) done = done || (seen_fn[i] == (const void*)kern && seen_sz[i] >= smem);
  if (!done) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if (nseen < 32) { seen_fn[nseen] = (const void*)kern; seen_sz[nseen] = smem; ++nseen; }
  }
  dim3 grid(p.Hq, p.B), block(NT);
  return launch_pdl(kern, grid, block, smem, s, p, big);
}

cudaError_t launch_select_topk(const Prob& p, cudaStream_t s) {
  const bool cached = keycap_of(p) > 0;
  if (p.dtype == VATTN_DTYPE_BF16) {
    if (p.D == 128) return cached ? launch_sel(k_select_topk<bf16_t, 128, true>, p, s, false) : launch_sel(k_select_topk<bf16_t, 128, false>, p, s, false);
    return cached ? launch_sel(k_select_topk<bf16_t, 64, true>, p, s, false) : launch_sel(k_select_topk<bf16_t, 64, false>, p, s, false);
  }
  if (p.D == 128) return cached ? launch_sel(k_select_topk<float, 128, true>, p, s, false) : launch_sel(k_select_topk<float, 128, false>, p, s, false);
  return cached ? launch_sel(k_select_topk<float, 64, true>, p, s, false) : launch_sel(k_select_topk<float, 64, false>, p, s, false);
}

static size_t select_smem_bytes(const Prob& p, bool final_kernel) {
  return sizeof(double) * VATTN_BANDCAP + 4 * sizeof(unsigned) * (size_t)p.nwords + sizeof(unsigned) * 256 +
         sizeof(int) * (VATTN_BANDCAP + NBIN + 2 * CANDCAP + 64) + (size_t)big_bytes(p, final_kernel);
}

template <typename KernelT>
static cudaError_t launch_presort_t(KernelT kern, const Prob& p, cudaStream_t s) {
  const size_t fixed = SORT_FIXED_BYTES + sizeof(unsigned) * (size_t)p.nwords;
  const size_t limit = 227 * 1024;
  const size_t per_pair = sizeof(uint2) + sizeof(int);
  size_t paircap = (size_t)p.cand_cap;
  if (fixed + paircap * per_pair > limit) paircap = (limit - fixed) / per_pair;   // longer lists take the slow path
  size_t smem = fixed + paircap * per_pair;
  const size_t sel = select_smem_bytes(p, false);              // the stream-0 fallback reuses the buffer
  if (sel > smem) smem = sel;
  static size_t attr_sz[2] = {0, 0};
  const int which = keycap_of(p) > 0 ? 1 : 0;
  if (attr_sz[which] < smem) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_sz[which] = smem;
  }
  return launch_pdl(kern, dim3(p.Hq, p.B, 2), dim3(NT), smem, s, p, (int)paircap, big_bytes(p, false));
}

cudaError_t launch_presort(const Prob& p, cudaStream_t s) {
  return keycap_of(p) > 0 ? launch_presort_t(k_presort<true>, p, s) : launch_presort_t(k_presort<false>, p, s);
}

cudaError_t launch_budget(const Prob& p, cudaStream_t s) {
  return keycap_of(p) > 0 ? launch_sel(k_budget<true>, p, s, true) : launch_sel(k_budget<false>, p, s, true);
}
