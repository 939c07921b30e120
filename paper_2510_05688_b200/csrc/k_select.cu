// Index selection, one 1024-thread CTA per (batch row, query head):
//
//   I_t   = the k middle tokens with the largest score, ties to the lowest index (Algorithm 1 line 3, the
//           "oracle top-k" of Sec. 3), as a list with physical slots and as a membership rule for the row kernels;
//   I_bs  = uniform-sample of b0 residual tokens (Algorithm 2 line 1), listed in walk order;
//   the head of the final sample's walk (Algorithm 1 line 7): the first residual tokens it meets, with their
//           fp32 scores, so that the final-sample kernel can start fetching rows the moment it knows the budget.
//
// Selection, usual case.  A thread owns whole pages (16 consecutive tokens = one aligned 64-byte read of the score
// row), so "ascending token order" is "thread order" and ordered positions come from one prefix sum per pass.
//   A  histogram of the top 11 bits of the order-reversed score keys; the bin d1 that holds rank k;
//   B  keys before bin d1 - 1 belong to I_t for certain; keys of bins d1 - 1 .. d1 + 1 are candidates (a few
//      hundred to two thousand), compacted in token order;
//   C  the exact rank-k key T among the candidates (three 8-bit radix levels over the candidate list).
// The stored scores differ from the exact inner products by at most gamma (a bound from the summation structure
// of the score kernel), so candidates above T + 2 gamma are certainly selected, candidates below T - 2 gamma
// certainly not, and the few in between are rescored in fp64 from their K rows and ranked exactly.
// Anything unusual (too many candidates or near-ties, a band that leaves the candidate bins, every middle token
// selected) takes the general path: a 32-bit radix select over the whole range with re-read scores, and for more
// than 1,024 near-ties (constant keys, a zero query) an exact 64-bit radix select over fp64 scores.
//
// Sampling.  Walk position j costs a few dozen integer instructions (an 8-round Feistel permutation with cycle
// walking, see vattn_internal.cuh), positions are independent, and "is this token in I_t" is one comparison of
// its score with T + 2 gamma plus a look-up for the near-ties: O(sample size) work, no keys per token, no sort.
// A thread evaluates 8 consecutive walk positions, ranks come from one prefix sum.
#include "vattn_internal.cuh"
#include <math_constants.h>



namespace {

constexpr int NT = SEL_THREADS;
constexpr int NWARP = NT / 32;
constexpr int HBINS = 2048;            // bins of one radix level
constexpr int ALLCAP = 4096;           // candidates of a head
constexpr unsigned FULL = 0xFFFFFFFFu;

struct Sm {
  unsigned char* big;          // 128 KB: the head's score keys (usual case), or the scratch of the general path's scans
  unsigned char* cand;         // 32 KB: candidate list (key, token); with `hist` in front: staging of the sample lists
  int* hist;                   // [HBINS] top key bits of the sample | [2 HBINS] + [2 HBINS] the candidates' two levels
  unsigned char* cv;           // [ALLCAP] candidate verdicts: 0 out, 1 member, 2 near-tie
  int* vback;                  // [BANDCAP] candidate index of a near-tie
  int* vtab;                   // [BANDCAP] near-tie tokens ascending, bit 31 = member of I_t
  double* band_s;              // [BANDCAP] exact scores of the near-ties
  int* bandl;                  // [BANDCAP] near-tie tokens of the general path
  int* misc;                   // [128]
  unsigned* rkeys;             // [2][8] round keys of the two walks
};
__host__ __device__ constexpr size_t up16(size_t x) { return (x + 15) / 16 * 16; }
constexpr int KEYCAP = 32768;          // score keys held in shared memory by the usual case
constexpr size_t BIG_BYTES = (size_t)KEYCAP * 4;
constexpr int LROUND = 4096;           // walk positions per round of the sample listing (4 per thread)
constexpr size_t SMEM_BYTES = BIG_BYTES + up16(5 * HBINS * 4) + up16(ALLCAP * 8) + up16(ALLCAP) + up16(VATTN_BANDCAP * 4) * 3 +
                              up16(VATTN_BANDCAP * 8) + up16(128 * 4) + up16(16 * 4) + 128;
static_assert(5 * HBINS * 4 + ALLCAP * 8 >= LROUND * 12, "the listing's staging lies over the histograms and the candidate list");
// position of key i in the swizzled key array: thread t owns keys [32 t, 32 t + 32) and reads them as eight 16-byte
// chunks; chunk c of thread t lives in slot c ^ (t & 7), so that the eight lanes of a quarter warp hit different banks
__device__ __forceinline__ int key_slot(int i) { return (i & ~31) | ((((i >> 2) ^ (i >> 5)) & 7) << 2) | (i & 3); }
__device__ __forceinline__ Sm carve(unsigned char* base) {
  Sm s;
  s.big = base;                                 base += BIG_BYTES;
  s.hist = reinterpret_cast<int*>(base);        base += up16(5 * HBINS * 4);
  s.cand = base;                                base += up16(ALLCAP * 8);
  s.band_s = reinterpret_cast<double*>(base);   base += up16(VATTN_BANDCAP * 8);
  s.cv = base;                                  base += up16(ALLCAP);
  s.vback = reinterpret_cast<int*>(base);       base += up16(VATTN_BANDCAP * 4);
  s.vtab = reinterpret_cast<int*>(base);        base += up16(VATTN_BANDCAP * 4);
  s.bandl = reinterpret_cast<int*>(base);       base += up16(VATTN_BANDCAP * 4);
  s.misc = reinterpret_cast<int*>(base);        base += up16(128 * 4);
  s.rkeys = reinterpret_cast<unsigned*>(base);  base += up16(16 * 4);
  return s;
}

// ---------------------------------------------------------------------------------------------
// block-level scans (NT threads); `wtot`: NWARP words that no thread touches until the caller's next barrier
__device__ __forceinline__ int block_scan_reg(int val, int* wtot, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = val;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int v = __shfl_up_sync(FULL, incl, off);
    if (lane >= off) incl += v;
  }
  if (lane == 31) wtot[warp] = incl;
  __syncthreads();
  const int mine = wtot[lane];
  int winc = mine;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int v = __shfl_up_sync(FULL, winc, off);
    if (lane >= off) winc += v;
  }
  total = __shfl_sync(FULL, winc, 31);
  const int before = __shfl_sync(FULL, winc - mine, warp);
  return before + incl - val;
}
// two counts per thread, packed in one 64-bit word
__device__ __forceinline__ unsigned long long block_scan2(unsigned long long val, unsigned long long* wtot,
                                                          unsigned long long& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned long long incl = val;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const unsigned long long v = __shfl_up_sync(FULL, incl, off);
    if (lane >= off) incl += v;
  }
  if (lane == 31) wtot[warp] = incl;
  __syncthreads();
  const unsigned long long mine = wtot[lane];
  unsigned long long winc = mine;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const unsigned long long v = __shfl_up_sync(FULL, winc, off);
    if (lane >= off) winc += v;
  }
  total = __shfl_sync(FULL, winc, 31);
  const unsigned long long before = __shfl_sync(FULL, winc - mine, warp);
  return before + incl - val;
}
// exclusive prefix sum of a[0..nw) in place; returns the total.  misc[32..64) is scratch.
__device__ __noinline__ int block_excl_scan(int* a, int nw, int* misc) {
  const int tid = threadIdx.x;
  const int ipt = (nw + NT - 1) / NT;
  const int start = min(nw, tid * ipt), end = min(nw, start + ipt);
  int local = 0;
  for (int i = start; i < end; ++i) local += a[i];
  __syncthreads();                       // the scratch may still be read by an earlier call
  int total;
  int run = block_scan_reg(local, misc + 32, total);
  for (int i = start; i < end; ++i) { const int v = a[i]; a[i] = run; run += v; }
  __syncthreads();
  return total;
}

// The bin that holds rank `rem` (1-based, counted from bin 0) of a histogram of nb <= 2048 bins (thread t adds up
// bins [8t, 8t + 8)).  Returns the bin; misc[1] = keys in the bins before it, misc[3..5] = keys in the bin before
// it, in it, after it.  One body for every call site.
__device__ __noinline__ int pick_bin(const int* h, int nb, int rem, int* misc) {
  const int tid = threadIdx.x;
  int c8[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) c8[e] = 0;
  if (tid * 8 < nb) {
    const int4* src = reinterpret_cast<const int4*>(h) + 2 * tid;
    const int4 a = src[0], b4 = src[1];
    c8[0] = a.x; c8[1] = a.y; c8[2] = a.z; c8[3] = a.w;
    c8[4] = b4.x; c8[5] = b4.y; c8[6] = b4.z; c8[7] = b4.w;
  }
  int sum = 0;
#pragma unroll
  for (int e = 0; e < 8; ++e) sum += c8[e];
  int total;
  const int excl = block_scan_reg(sum, misc + 32, total);
  if (tid == 0) { misc[3] = 0; misc[5] = 0; misc[6] = -1; }
  __syncthreads();
  if (excl < rem && rem <= excl + sum) {
    int cum = excl;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      if (rem <= cum + c8[e]) {
        misc[0] = tid * 8 + e; misc[1] = cum; misc[4] = c8[e];
        if (e > 0) misc[3] = c8[e > 0 ? e - 1 : 0];
        if (e < 7) misc[5] = c8[e < 7 ? e + 1 : 7];
        misc[6] = e;
        break;
      }
      cum += c8[e];
    }
  }
  __syncthreads();
  const int bin = misc[0], e_in = misc[6];
  if (e_in == 0 && tid == (bin >> 3) - 1) misc[3] = c8[7];      // the neighbours in the next thread's range
  if (e_in == 7 && tid == (bin >> 3) + 1) misc[5] = c8[0];
  __syncthreads();
  return bin;
}

// The same with one barrier inside and none of the serial loops: thread t adds up the nb / NT (2 or 4) bins
// [t nb/NT, (t+1) nb/NT).  Writes the bin to out[0] and the keys before it to out[1]; the caller's next barrier
// publishes them.  `wtot`: NWARP words of scratch.
__device__ __forceinline__ void block_pick(const int* h, int nb, int rem, int* wtot, int* out) {
  const int tid = threadIdx.x;
  const int per = nb / NT;                               // 2 or 4
  int c4[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) c4[i] = i < per ? h[tid * per + i] : 0;
  const int sum = c4[0] + c4[1] + c4[2] + c4[3];
  int total;
  const int excl = block_scan_reg(sum, wtot, total);
  if (excl < rem && rem <= excl + sum) {
    int cum = excl;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (i < per && rem <= cum + c4[i]) { out[0] = tid * per + i; out[1] = cum; break; }
      cum += c4[i];
    }
  }
}

// Radix select over the keys `loop` delivers (loop(body) calls body(key) for every key): the rank-th smallest
// key (rank >= 1) and how many keys equal to it are among the rank smallest.
template <typename KeyT, class Loop>
__device__ KeyT radix_select(const Sm& sm, int rank, int& need_eq, Loop loop) {
  constexpr int KB = (int)sizeof(KeyT) * 8;
  constexpr int NLEV = (KB + 10) / 11;
  const int tid = threadIdx.x;
  KeyT prefix = 0;
  int rem = rank, used = 0;
#pragma unroll 1
  for (int l = 0; l < NLEV; ++l) {
    const int bits = (KB - used) < 11 ? KB - used : 11;   // 11 + 11 + 10 bits, or 5 x 11 + 9
    const int shift = KB - used - bits;
    const int nb = 1 << bits;
    int* h = sm.hist;
    for (int i = tid; i < HBINS; i += NT) h[i] = 0;
    __syncthreads();
    loop([&](KeyT key) {
      if (l == 0 || (key >> (shift + bits)) == prefix) atomicAdd(&h[(unsigned)(key >> shift) & (unsigned)(nb - 1)], 1);
    });
    __syncthreads();
    const int bin = pick_bin(h, nb, rem, sm.misc);
    prefix = (prefix << bits) | (KeyT)(unsigned)bin;
    rem -= sm.misc[1];
    used += bits;
    __syncthreads();
  }
  need_eq = rem;
  return prefix;
}

// exact fp64 score of one token, computed by a whole warp from global memory (all lanes return it)
template <typename T, int D>
__device__ __noinline__ double score64_warp(const T* krow, const T* qrow, float scale) {
  const int lane = threadIdx.x & 31;
  double acc = 0.0;
#pragma unroll
  for (int t = 0; t < D / 32; ++t) {
    const int e = lane + 32 * t;
    acc = fma((double)Elem<T>::to_float(qrow[e]), (double)Elem<T>::to_float(krow[e]), acc);
  }
#pragma unroll
  for (int mask = 16; mask >= 1; mask >>= 1) acc += __shfl_xor_sync(FULL, acc, mask);
  return acc * (double)scale;
}
// the same number, by one thread (identical summation tree, so identical bits)
template <typename T, int D>
__device__ __noinline__ double score64_thread(const T* krow, const T* qrow, float scale) {
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
    for (int l = 0; l < mask; ++l) part[l] = part[l] + part[l | mask];
  return part[0] * (double)scale;
}

// ---------------------------------------------------------------------------------------------
template <typename T, int D>
__global__ void __launch_bounds__(NT, 1) k_select(const Prob p) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int bh = blockIdx.x;
  const int b = bh / p.Hq, h = bh % p.Hq, g = h / p.G;
  const unsigned lt = (1u << lane) - 1u;
  const Sm sm = carve(smem_raw);
  TICK_BEGIN(p, VATTN_K_SELECT);

  // ------------------------------------------------------------------ before the wait: the step's inputs only
  const int n = head_len(p, b, h);
  const Geo geo = head_geometry(p, n);
  const int s0 = geo.s0, l_start = geo.l_start, kk = geo.kk, n_s = geo.n_s, b0 = geo.b0;
  const int mlen = l_start - s0;
  const T* qrow = reinterpret_cast<const T*>(p.q) + q_row(p, b, h);
  const float* sc = p.scores + (long long)bh * p.npad;
  int* tk = p.topk_idx + (long long)bh * 2 * p.npad;
  unsigned* gbitmap = p.bitmap + (long long)bh * p.nwords;
  HeadMeta mt;
  mt.n = n; mt.s0 = s0; mt.l_start = l_start; mt.kk = kk; mt.n_s = n_s; mt.b0 = b0;
  mt.nbt = 0; mt.band_mode = 0; mt.m = 0.f; mt.hi = CUDART_INF_F; mt.lo = CUDART_INF_F;
  mt.run1 = 0; mt.dyn_listed = 0; mt.dyn_J = 0; mt.path = 0; mt.b = 0;
  if (n == 0) {
    pdl_wait();
    pdl_trigger();
    if (tid == 0) {
      mt.base_J = 0; mt.holes2 = 0; mt.base_list = 0; mt.holes1 = 0;
      p.meta[bh] = mt;
      __threadfence();
      asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p.flags64 + bh), "l"(2ull) : "memory");
      asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p.tickets + 4 * p.B * p.Hq + bh), "r"(1u) : "memory");
      if (p.dbg.topk_cnt) p.dbg.topk_cnt[bh] = 0;
      if (p.dbg.base_cnt) p.dbg.base_cnt[bh] = 0;
      if (p.dbg.paths) p.dbg.paths[bh] = 0;
    }
    return;
  }
  for (int i = tid; i < 5 * HBINS; i += NT) sm.hist[i] = 0;
  if (tid < 4) walk_keys(p, b, h, tid >> 1, tid & 1, sm.rkeys + (tid >> 1) * 8);
  double sa = 0.0;                                     // sum |q_e| (warp 0), for the rounding bound of the scores
  if (warp == 0) {
    for (int e = lane; e < D; e += 32) sa += fabs((double)Elem<T>::to_float(qrow[e]));
#pragma unroll
    for (int mk = 16; mk >= 1; mk >>= 1) sa += __shfl_xor_sync(FULL, sa, mk);
  }
  for (int w = tid; w < ((n + 31) >> 5); w += NT) gbitmap[w] = 0u;     // only the overflow path sets and reads bits
  // the first entries of the head's list of marked positions are read unconditionally by the budget: "none" until set
  if (tid < 256) p.hole_pos[(long long)bh * 2 * VATTN_BANDCAP + tid] = 0x7FFFFFFF;

  pdl_wait();                                          // the score pass is complete: scores, maxima
  pdl_trigger();
  TICK_BEGIN(p, VATTN_T_TOPK);
  const float m = unord_f32(__ldcg(p.m_ord + bh));
  mt.m = m;
  // gamma: bound on |fp32 score - exact score|.  fp32 path: at most 13 roundings (x16 = margin).  bf16
  // tensor-core path: at most 8 accumulation steps of 16 exact products each, every step assumed to lose up
  // to 17 units of 2^-23 of the running magnitude (truncating adder) -> 8*17*2 = 272, taken as 512.
  if (warp == 0 && lane == 0) {
    const double kmax = (double)__uint_as_float(__ldcg(p.kabsmax + b * p.Hkv + g));
    const double roundings = (p.dtype == VATTN_DTYPE_BF16) ? 512.0 : 16.0;
    const double gm = roundings * 5.9604644775390625e-8 * fabs((double)p.scale) * sa * kmax * 1.000001;
    reinterpret_cast<float*>(sm.misc)[100] = __double2float_ru(gm);
  }
  __syncthreads();
  const float gamma = reinterpret_cast<float*>(sm.misc)[100];
  int path = 0;
  float hi = CUDART_INF_F, lo = CUDART_INF_F;          // members: s > hi; near-tie band: lo <= s <= hi
  int nbt = 0, band_mode = 0, run1 = 0;
  bool general = kk > 0 && kk == mlen;

  // ------------------------------------------------------------------ selection, usual case
  // Block-wide barriers are what this kernel pays for (a 1024-thread barrier costs a few hundred ns): the passes
  // below meet at about a dozen of them.
  const int G16 = (n + 15) >> 4;
  unsigned* keys = reinterpret_cast<unsigned*>(sm.big);       // key of token i at keys[key_slot(i)] (usual case only)
  bool cached = G16 <= KEYCAP / 16;                    // the head's keys are in shared memory (contexts up to 32,768 tokens)
  if (kk > 0 && kk < mlen && !cached) general = true;
  if (cached) {
    // ---- the head's scores into shared memory as order-reversed keys (smaller key = larger score): coalesced
  // 16-byte reads, swizzled 16-byte writes; everything below reads keys from shared memory
  for (int c4 = tid; c4 < G16 * 4; c4 += NT) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(sc) + c4);
    uint4 k4;
    k4.x = v.x ^ (~((int)v.x >> 31) & 0x7FFFFFFFu); k4.y = v.y ^ (~((int)v.y >> 31) & 0x7FFFFFFFu);
    k4.z = v.z ^ (~((int)v.z >> 31) & 0x7FFFFFFFu); k4.w = v.w ^ (~((int)v.w >> 31) & 0x7FFFFFFFu);
    *reinterpret_cast<uint4*>(keys + key_slot(c4 << 2)) = k4;
  }
  }
  unsigned* candk = reinterpret_cast<unsigned*>(sm.cand);
  int* candt = reinterpret_cast<int*>(candk + ALLCAP);
  int below = 0, ncand = 0;
  unsigned kbase = 0u;
  if (kk > 0 && kk < mlen && !general) {
    int* hA = sm.hist, * hB = sm.hist + HBINS, * hC = sm.hist + 3 * HBINS;      // 2048, 4096, 4096 bins
    unsigned long long* wt = reinterpret_cast<unsigned long long*>(sm.misc + 64);
    // physical pages of the thread's two pages (tokens [32 t, 32 t + 32))
    const int pgp0 = 2 * tid < G16 ? page_of(p, b, 2 * tid) : 0, pgp1 = 2 * tid + 1 < G16 ? page_of(p, b, 2 * tid + 1) : 0;
    __syncthreads();
    // ---- A: where is rank k?  A histogram of ALL keys would hammer the handful of bins that hold most scores
    // (shared-memory atomics to one address serialise), so the bin is estimated from a sample: one token per page.
    // The candidate bins are the estimate's neighbourhood, two bins to either side; pass B counts the keys above
    // them exactly and verifies that rank k really falls among the candidates.
    int ns_loc = 0;
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      const int i = ((2 * tid + c) << 4) + (tid & 15);           // a different offset in the page per thread
      if (i >= s0 && i < l_start) { atomicAdd(&hA[keys[key_slot(i)] >> 21], 1); ++ns_loc; }
    }
    int ns_tot;
    // A middle range of a few tokens may hold no sampled token at all (a page's sample sits at one offset): the
    // pick below then finds no bin and writes nothing, so its outputs are preset to bin 0 (the largest scores:
    // pass B verifies that choice like any other and falls back to the general selection when it is wrong).
    if (tid == 0) { sm.misc[0] = 0; sm.misc[1] = 0; }
    block_scan_reg(ns_loc, sm.misc + 32, ns_tot);      // (one barrier: the sample histogram is complete behind it)
    __syncthreads();
    {
      const long long rs = ((long long)kk * ns_tot + mlen - 1) / mlen;          // the rank inside the sample, rounded up
      block_pick(hA, HBINS, (int)max(1ll, min((long long)ns_tot, rs)), sm.misc + 32, sm.misc);
    }
    __syncthreads();
    DBGT(0);
    const int d1 = sm.misc[0];
    const int dlo = max(d1 - 2, 0), dhi = min(d1 + 2, HBINS - 1);           // candidate bins
    kbase = (unsigned)dlo << 21;                       // candidate keys relative to it are below 5 * 2^21 < 2^24
    unsigned kend = dhi == HBINS - 1 ? 0xFFFFFFFFu : (((unsigned)dhi + 1u) << 21) - 1u;    // last candidate key
    {
      // Scores that crowd into a few bins (a near-uniform head: all of them within a factor of two) would make
      // most of the head a candidate.  The sample says how many keys the five bins hold; when that is more than
      // the candidate list takes, the candidates are a narrower key range inside the five bins: the sample's keys
      // of those bins in 5 x 256 finer bins, and the range between the ranks k' - delta and k' + delta of the sample (delta: four
      // standard deviations of the sample's rank and a little more).  Pass B verifies the range like the bins.
      int c5 = 0, cb = 0;                              // sample keys in the five bins; in those of them before d1
      for (int d = dlo; d <= dhi; ++d) { c5 += hA[d]; if (d < d1) cb += hA[d]; }
      const long long rs = max(1ll, min((long long)ns_tot, ((long long)kk * ns_tot + mlen - 1) / mlen));
      if ((long long)c5 * mlen > (long long)(ALLCAP * 7 / 8) * ns_tot) {      // (uniform over the CTA)
        const int before = sm.misc[1] - cb;            // sample keys before bin dlo
        __syncthreads();                               // (misc is written again below)
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          const int i = ((2 * tid + c) << 4) + (tid & 15);
          if (i >= s0 && i < l_start) {
            const unsigned key = keys[key_slot(i)];
            const int d = (int)(key >> 21);
            if (d >= dlo && d <= dhi) atomicAdd(&hC[((d - dlo) << 8) | ((key >> 13) & 0xFFu)], 1);     // 5 x 256 finer bins
          }
        }
        __syncthreads();
        const int r5 = (int)rs - before;               // the rank among the sample keys of the five bins (1-based)
        const int delta = 4 * (int)sqrtf((float)rs) + 8;
        block_pick(hC, HBINS, max(1, min(c5, r5 - delta)), sm.misc + 32, sm.misc + 8);
        __syncthreads();
        block_pick(hC, HBINS, max(1, min(c5, r5 + delta)), sm.misc + 32, sm.misc + 10);
        __syncthreads();
        const unsigned f_lo = (unsigned)sm.misc[8], f_hi = (unsigned)sm.misc[10];
        if (r5 - delta >= 1) kbase = (((unsigned)dlo + (f_lo >> 8)) << 21) | ((f_lo & 0xFFu) << 13);
        if (r5 + delta <= c5) kend = (((unsigned)dlo + (f_hi >> 8)) << 21) | ((f_hi & 0xFFu) << 13) | 0x1FFFu;
        for (int i = tid; i < HBINS; i += NT) hC[i] = 0;       // (the exact selection uses it again)
        path |= 8;
        __syncthreads();
      }
    }
    DBGT(1);
    {
      // ---- B: upper keys' tokens to the list of I_t, candidates to their list, both ascending by token
      unsigned umask[2], cmask[2];
      int nu = 0, nc = 0;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        const int i0 = (2 * tid + c) << 4;
        unsigned vm = 0u;
        {
          const int a_ = max(s0 - i0, 0), z_ = min(l_start - i0, 16);
          if (z_ > a_) vm = ((1u << z_) - 1u) & ~((1u << a_) - 1u);
        }
        unsigned um = 0u, cm = 0u;
        if (vm) {
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            const uint4 k4 = *reinterpret_cast<const uint4*>(keys + key_slot(i0 + 4 * q4));
            const unsigned kq[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              um |= (kq[e] < kbase ? 1u : 0u) << (4 * q4 + e);
              cm |= (kq[e] >= kbase && kq[e] <= kend ? 1u : 0u) << (4 * q4 + e);
            }
          }
        }
        umask[c] = um & vm; cmask[c] = cm & vm;
        nu += __popc(umask[c]); nc += __popc(cmask[c]);
      }
      DBGT(10);
      unsigned long long tot2;
      const unsigned long long ex2 = block_scan2((unsigned long long)nu | ((unsigned long long)nc << 32), wt, tot2);
      DBGT(11);
      int upos = (int)(ex2 & 0xFFFFFFFFull), cpos = (int)(ex2 >> 32);
      below = (int)(tot2 & 0xFFFFFFFFull);             // keys above the candidate bins: members of I_t for certain
      ncand = (int)(tot2 >> 32);
      // rank k must fall among the candidates
      general = !(below < kk && kk <= below + ncand) || ncand > ALLCAP;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        if (!general && (umask[c] | cmask[c])) {
          const int i0 = (2 * tid + c) << 4;
          const int pgp = c ? pgp1 : pgp0;
          unsigned um = umask[c], cm = cmask[c];
          while (um) { const int e = __ffs(um) - 1; um &= um - 1; tk[upos] = i0 + e; tk[p.npad + upos] = pgp * VATTN_BLOCK + e; ++upos; }
          while (cm) {
            const int e = __ffs(cm) - 1; cm &= cm - 1;
            const unsigned key = keys[key_slot(i0 + e)];
            candk[cpos] = key; candt[cpos] = i0 + e; ++cpos;
            atomicAdd(&hB[(key - kbase) >> 12], 1);    // first level of the exact selection among the candidates
          }
        }
      }
      __syncthreads();
      DBGT(2);
    }
    if (!general) {
      // ---- C: the (kk - below)-th smallest candidate key: 11 + 12 bits
      block_pick(hB, 2 * HBINS, kk - below, sm.misc + 32, sm.misc + 3);
      __syncthreads();
      const unsigned pref = (unsigned)sm.misc[3];
      for (int c = tid; c < ncand; c += NT) {
        const unsigned rel = candk[c] - kbase;
        if ((rel >> 12) == pref) atomicAdd(&hC[rel & 0xFFFu], 1);
      }
      __syncthreads();
      block_pick(hC, 2 * HBINS, kk - below - sm.misc[4], sm.misc + 32, sm.misc + 5);
      __syncthreads();
      DBGT(3);
      const float Tf = unord_f32(~(kbase + (pref << 12) + (unsigned)sm.misc[5]));
      hi = __fadd_ru(Tf, 2.f * gamma); lo = __fadd_rd(Tf, -2.f * gamma);
      // the band must stay inside the candidate bins: every upper key is then above it, every other key below it
      const bool up_ok = kbase == 0u || hi <= unord_f32(~kbase);
      const bool dn_ok = kend == 0xFFFFFFFFu || lo >= unord_f32(~kend);
      // classify the candidates: thread t takes a run of consecutive entries, so ordinals are one prefix sum
      const int per = (ncand + NT - 1) / NT;
      const int c_lo = min(ncand, tid * per), c_hi = min(ncand, c_lo + per);
      int na = 0, nbd = 0;
      for (int c = c_lo; c < c_hi; ++c) {
        const float sv = unord_f32(~candk[c]);
        const int code = sv > hi ? 1 : (sv >= lo ? 2 : 0);
        sm.cv[c] = (unsigned char)code;
        na += code == 1; nbd += code == 2;
      }
      unsigned long long tot2;
      const unsigned long long ex3 = block_scan2((unsigned long long)na | ((unsigned long long)nbd << 32), wt, tot2);
      const int n_above = (int)(tot2 & 0xFFFFFFFFull);
      nbt = (int)(tot2 >> 32);
      general = !up_ok || !dn_ok || nbt > VATTN_BANDCAP;
      if (!general) {
        int bo = (int)(ex3 >> 32);
        for (int c = c_lo; c < c_hi; ++c)
          if (sm.cv[c] == 2) { sm.vtab[bo] = candt[c]; sm.vback[bo] = c; ++bo; }
        __syncthreads();
        DBGT(4);
        const int need = kk - below - n_above;         // near-ties that belong to I_t (at least the rank-k key itself)
        if (need >= nbt) {
          for (int c = tid; c < nbt; c += NT) { sm.vtab[c] |= (int)0x80000000; sm.cv[sm.vback[c]] = 1; }
        } else {
          path |= 2;
          for (int c = warp; c < nbt; c += NWARP) {
            const double s64 = score64_warp<T, D>(row_ptr<T>(p, p.kc, b, g, sm.vtab[c]), qrow, p.scale);
            if (lane == 0) sm.band_s[c] = s64;
          }
          __syncthreads();
          for (int c = tid; c < nbt; c += NT) {
            const double mine = sm.band_s[c];
            int rank = 0;
            for (int u = 0; u < nbt; ++u) {
              const double o = sm.band_s[u];
              rank += (o > mine) || (o == mine && u < c);
            }
            if (rank < need) { sm.vtab[c] |= (int)0x80000000; sm.cv[sm.vback[c]] = 1; }
          }
        }
        __syncthreads();
        DBGT(5);
        // the candidates that made it: behind the upper tokens, ascending too
        int nm = 0;
        for (int c = c_lo; c < c_hi; ++c) nm += sm.cv[c] == 1;
        int tot1;
        int pos = below + block_scan_reg(nm, sm.misc + 32, tot1);
        for (int c = c_lo; c < c_hi; ++c)
          if (sm.cv[c] == 1) {
            const int tok = candt[c];
            tk[pos] = tok;
            tk[p.npad + pos] = page_of(p, b, tok >> 4) * VATTN_BLOCK + (tok & 15);
            ++pos;
          }
        run1 = below;
        path |= 1;
      }
      __syncthreads();
    }
  }

  // ------------------------------------------------------------------ selection, general case
  if (kk > 0 && general) {
    const int PT = (mlen + NT - 1) / NT;               // keys per thread
    // every key of the middle range, in token order per thread: f(u, token, valid, key); uniform trip count
    auto for_slice = [&](auto f) {
#pragma unroll 1
      for (int u = 0; u < PT; ++u) {
        const int i = s0 + tid + NT * u;
        const bool v = i < l_start;
        f(u, i, v, v ? ~ord_f32(__ldg(sc + i)) : 0xFFFFFFFFu);
      }
    };
    cached = false;                                    // the scans' scratch below takes the place of the keys
    __syncthreads();
    int* cntM = reinterpret_cast<int*>(sm.big);        // [PT * NWARP] tokens above the band per (u, warp), then its scan
    int* cntB = cntM + PT * NWARP;                     // the same for the band
    hi = CUDART_INF_F; lo = CUDART_INF_F;
    nbt = 0;
    if (kk == mlen) { hi = -CUDART_INF_F; lo = -CUDART_INF_F; }
    else {
      int need_eq;
      const unsigned Tk = radix_select<unsigned>(sm, kk, need_eq, [&](auto body) {
        for_slice([&](int, int, bool v, unsigned key) { if (v) body(key); });
      });
      const float Tf = unord_f32(~Tk);
      hi = __fadd_ru(Tf, 2.f * gamma); lo = __fadd_rd(Tf, -2.f * gamma);
    }
    // ---- classify: above the band (ordered counts per (u, warp)), inside it
    for_slice([&](int u, int, bool v, unsigned key) {
      const float s = unord_f32(~key);
      const unsigned bm = __ballot_sync(FULL, v && s > hi), bb = __ballot_sync(FULL, v && !(s > hi) && s >= lo);
      if (lane == 0) { cntM[u * NWARP + warp] = __popc(bm); cntB[u * NWARP + warp] = __popc(bb); }
    });
    __syncthreads();
    const int n_in = block_excl_scan(cntM, PT * NWARP, sm.misc);
    nbt = block_excl_scan(cntB, PT * NWARP, sm.misc);
    for_slice([&](int u, int i, bool v, unsigned key) {
      const float s = unord_f32(~key);
      const bool mem = v && s > hi, bnd = v && !(s > hi) && s >= lo;
      const unsigned bm = __ballot_sync(FULL, mem), bb = __ballot_sync(FULL, bnd);
      if (mem) {
        const int pos = cntM[u * NWARP + warp] + __popc(bm & lt);
        tk[pos] = i;
        tk[p.npad + pos] = page_of(p, b, i >> 4) * VATTN_BLOCK + (i & 15);
      }
      const int posb = cntB[u * NWARP + warp] + __popc(bb & lt);
      if (bnd && posb < VATTN_BANDCAP) sm.vtab[posb] = i;
    });
    __syncthreads();
    const int need = kk - n_in;
    if (nbt <= VATTN_BANDCAP) {
      if (need >= nbt) {
        for (int c = tid; c < nbt; c += NT) sm.vtab[c] |= (int)0x80000000;
      } else {
        path |= 2;
        for (int c = warp; c < nbt; c += NWARP) {
          const double s64 = score64_warp<T, D>(row_ptr<T>(p, p.kc, b, g, sm.vtab[c]), qrow, p.scale);
          if (lane == 0) sm.band_s[c] = s64;
        }
        __syncthreads();
        for (int c = tid; c < nbt; c += NT) {
          const double mine = sm.band_s[c];
          int rank = 0;
          for (int u = 0; u < nbt; ++u) {
            const double o = sm.band_s[u];
            rank += (o > mine) || (o == mine && u < c);
          }
          if (rank < need) sm.vtab[c] |= (int)0x80000000;
        }
      }
      __syncthreads();
      for (int c = tid; c < nbt; c += NT) {            // the band's members behind the tokens above it, ascending too
        const int e = sm.vtab[c];
        if (e < 0) {
          int ord = 0;
          for (int u = 0; u < c; ++u) ord += sm.vtab[u] < 0;
          const int tok = e & 0x7FFFFFFF;
          tk[n_in + ord] = tok;
          tk[p.npad + n_in + ord] = page_of(p, b, tok >> 4) * VATTN_BLOCK + (tok & 15);
        }
      }
    } else {
      // too many near-ties for a list: exact fp64 scores as ordered 64-bit keys (smaller key = larger score), an
      // exact radix select of the `need` smallest, equal keys to the lowest indices; verdicts go to the bitmap
      path |= 4;
      band_mode = 1;
      if (tid == 0) atomicOr(p.status, VATTN_STATUS_BAND_OVERFLOW);
      unsigned long long* k64 = reinterpret_cast<unsigned long long*>(p.dyn_idx + (long long)bh * 3 * p.npad);
      for_slice([&](int, int i, bool v, unsigned key) {
        const float s = unord_f32(~key);
        if (v && !(s > hi) && s >= lo) k64[i] = ~ord_f64(score64_thread<T, D>(row_ptr<T>(p, p.kc, b, g, i), qrow, p.scale));
      });
      __syncthreads();
      int need_eq;
      const unsigned long long T64 = radix_select<unsigned long long>(sm, need, need_eq, [&](auto body) {
        for_slice([&](int, int i, bool v, unsigned key) {
          const float s = unord_f32(~key);
          if (v && !(s > hi) && s >= lo) body(k64[i]);
        });
      });
      // ordered counts of the keys below T64 and equal to it
      for_slice([&](int u, int i, bool v, unsigned key) {
        const float s = unord_f32(~key);
        const bool bnd = v && !(s > hi) && s >= lo;
        const unsigned long long kx = bnd ? k64[i] : 0ull;
        const unsigned bl = __ballot_sync(FULL, bnd && kx < T64), be = __ballot_sync(FULL, bnd && kx == T64);
        if (lane == 0) { cntM[u * NWARP + warp] = __popc(bl); cntB[u * NWARP + warp] = __popc(be); }
      });
      __syncthreads();
      block_excl_scan(cntM, PT * NWARP, sm.misc);
      block_excl_scan(cntB, PT * NWARP, sm.misc);
      for_slice([&](int u, int i, bool v, unsigned key) {
        const float s = unord_f32(~key);
        const bool bnd = v && !(s > hi) && s >= lo;
        const unsigned long long kx = bnd ? k64[i] : 0ull;
        const bool isl = bnd && kx < T64, ise = bnd && kx == T64;
        const unsigned bl = __ballot_sync(FULL, isl), be = __ballot_sync(FULL, ise);
        const int lt_before = cntM[u * NWARP + warp] + __popc(bl & lt);
        const int eq_before = cntB[u * NWARP + warp] + __popc(be & lt);
        if (isl || (ise && eq_before < need_eq)) {
          const int pos = n_in + lt_before + min(eq_before, need_eq);
          tk[pos] = i;
          tk[p.npad + pos] = page_of(p, b, i >> 4) * VATTN_BLOCK + (i & 15);
          atomicOr(&gbitmap[i >> 5], 1u << (i & 31));
        }
      });
    }
    run1 = n_in;
    __threadfence();                                   // the bitmap's bits are read back below through L2
    __syncthreads();
  }
  mt.hi = hi; mt.lo = lo; mt.nbt = band_mode ? 0 : nbt; mt.band_mode = band_mode; mt.run1 = run1; mt.path = path;
  TICK_END(p, VATTN_T_TOPK);
  DBGH(bh, 0);

  // the final walk's round keys for the gather kernel (it extends the walk array for long budgets)
  if (tid < 8) p.wkeys[(long long)bh * 8 + tid] = sm.rkeys[8 + tid];
  // the near-tie list for the budget's list path
  int* gvtab = p.vtab + (long long)bh * VATTN_BANDCAP;
  for (int c = tid; c < mt.nbt; c += NT) gvtab[c] = sm.vtab[c];
  if (tid == 0) {
    if (p.dbg.topk_cnt) p.dbg.topk_cnt[bh] = kk;
    if (p.dbg.base_cnt) p.dbg.base_cnt[bh] = b0;
    if (p.dbg.paths) p.dbg.paths[bh] = path;
  }
  __syncthreads();                                     // the list of I_t is read back below (through L2: ld.cg)
  // "the list of I_t is written": the statistics kernel's deterministic-row CTAs start while the samples are
  // prepared below (the barrier orders every thread's writes before thread 0's release, which is cumulative)
  if (tid == 0) asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p.tickets + 4 * p.B * p.Hq + bh), "r"(1u) : "memory");
  if (p.dbg.topk_idx) {
    // I_t ascending for the debug buffer: two ascending runs merged by rank
    __threadfence();
    __syncthreads();
    int* dst = p.dbg.topk_idx + (long long)bh * p.max_seq_len;
    for (int a = tid; a < kk; a += NT) {
      const int tok = __ldcg(tk + a);
      int lo_ = a < run1 ? run1 : 0, hi_ = a < run1 ? kk : run1;
      const int base_ = lo_;
      while (lo_ < hi_) { const int mid = (lo_ + hi_) >> 1; if (__ldcg(tk + mid) < tok) lo_ = mid + 1; else hi_ = mid; }
      dst[(a < run1 ? a : a - run1) + (lo_ - base_)] = tok;
    }
  }

  // ------------------------------------------------------------------ the samples
  // uniform-sample(R, c) is the first c residual tokens of a walk of the middle range.  The walk kernel left the
  // first positions of both walks (tokens, physical slots) in the walk arrays; what is missing is which of those
  // tokens are members of I_t.  Each member's walk position is sigma^-1(token): the member is marked there (token =
  // -1), and a sample of c residual tokens becomes "the unmarked entries among the first J", J = c + the number of
  // marked positions below J (a fixed point reached in a few steps).  No list is compacted; the row kernels skip
  // marked entries.  For the final sample (c = the budget, not known yet) the marked positions are left in hole_pos.
  int* wa0 = p.walk_tok + (long long)bh * 4 * p.npad;            // base sample's walk: tokens (slots at + npad)
  int* wa1 = wa0 + 2 * p.npad;                                   // final sample's walk
  const int W0 = walk_region(n_s > 0 ? b0 : 0, n_s, mlen, kk);   // entries the walk kernel wrote
  const int W1 = walk_region(dyn_listed_want(p, n_s, b0), n_s, mlen, kk);
  int* hp0 = sm.hist;                                  // marked positions of the base walk (over the histograms)
  int* cnts = sm.misc + 8;                             // marked positions: [0] base walk, [1] final walk; [2] members beyond its array
  int base_J = 0, base_list = 0, holes1 = 0, holes2 = 0, dyn_J = 0, dyn_listed = 0, piv_ph = 0;
  if (n_s > 0 && kk <= NT * 4) {
    // physical slots of the first entries of the base walk: one of them is the pivot (the first unmarked entry)
    int pvph = 0;
    if (warp == 0 && lane < 4 && lane < W0) pvph = __ldcg(wa0 + p.npad + lane);
    if (tid == 0) { cnts[0] = 0; cnts[1] = 0; cnts[2] = 0; }
    const Walk wk0 = make_walk(sm.rkeys + (p.nested_base ? 8 : 0), mlen);
    __syncthreads();
    DBGT(16);
    // (only the base walk's marks stand between the top-k and the statistics kernel's base rows: the final walk's
    // marks and member positions follow after the word for the base rows has been published)
    for (int a = tid; a < kk; a += NT) {
      const int t = __ldcg(tk + a) - s0;
      const int x0 = walk_inv(wk0, t);
      if (x0 < W0) {
        wa0[x0] = -1;
        const int i0 = atomicAdd(&cnts[0], 1);
        if (i0 < HBINS) hp0[i0] = x0;
      }
    }
    __syncthreads();
    DBGT(17);
    const int H0 = cnts[0];
    if (H0 > HBINS) base_list = 1;
    else if (warp == 0) {
      // J = b0 + #{marked positions < J}; the pivot = the first unmarked position.  "The prefix that holds `want`
      // unmarked entries" is the least fixed point of J -> want + #{marked < J}: a few steps from J = want in the
      // usual case; when nearly every position is marked (top-k sets that take most of the middle range) the steps
      // are as short as the runs of marked positions, so after eight of them a bisection takes over (J minus the
      // marked positions below J never decreases).  W0 + 1: the array holds fewer than `want` unmarked entries.
      auto below = [&](int J) {
        int c = 0;
        for (int i = lane; i < H0; i += 32) c += hp0[i] < J;
#pragma unroll
        for (int mk = 16; mk >= 1; mk >>= 1) c += __shfl_xor_sync(FULL, c, mk);
        return c;
      };
      auto prefix_for = [&](int want) {
        int J = want;
        for (int it = 0; it < 8; ++it) {
          const int c = below(J);
          if (want + c == J) return J;
          J = want + c;
        }
        if (W0 - below(W0) < want) return W0 + 1;
        int lo_ = min(J, W0), hi_ = W0;                  // the steps above never overshoot the fixed point
        while (lo_ < hi_) {
          const int mid = (lo_ + hi_) >> 1;
          if (mid - below(mid) >= want) hi_ = mid; else lo_ = mid + 1;
        }
        return lo_;
      };
      const int J = prefix_for(b0);
      const int pivx = prefix_for(1) - 1;
      int ph = __shfl_sync(FULL, pvph, pivx & 3);
      if (pivx >= 4 && pivx < W0) ph = __ldcg(wa0 + p.npad + pivx);
      if (lane == 0) { sm.misc[4] = J; sm.misc[5] = ph; sm.misc[6] = (J > W0 || pivx >= W0) ? 1 : 0; }
    }
    __syncthreads();
    if (!base_list) { base_J = sm.misc[4]; piv_ph = sm.misc[5]; base_list = sm.misc[6]; }
  } else if (n_s > 0) {
    base_list = 1;
  }
  if (base_J >= (1 << 22)) base_list = 1;              // the published word has 22 bits for it
  mt.base_J = base_J; mt.holes2 = 0; mt.base_list = base_list; mt.holes1 = 0;
  mt.dyn_J = 0; mt.dyn_listed = 0;                     // (the final walk's fields follow below)
  DBGT(6);

  // The base sample as a list: for the debug buffer, and for the row kernels when the walk array fell short.
  // Rounds of 4096 walk positions, four consecutive ones per thread; the rank of a residual token is a prefix sum
  // away.  Listed entries are staged in shared memory in rank order and written out with consecutive threads on
  // consecutive words.
  int* bdbg = p.dbg.base_idx ? p.dbg.base_idx + (long long)bh * p.max_seq_len : nullptr;
  if (n_s > 0 && (base_list || bdbg)) {
    int* bl_tok = p.base_idx + (long long)bh * 2 * p.npad;
    int* st_tok = sm.hist, * st_ph = sm.hist + LROUND;
    __syncthreads();                                   // marks in the walk array are read back below (ld.cg)
    const int want = b0;
    const Walk wk = make_walk(sm.rkeys + (p.nested_base ? 8 : 0), mlen);
    const int* pre = wa0;
    const int Jpre = W0;
    int have = 0, J = 0;
#pragma unroll 1
    while (have < want && J < mlen) {
      // the positions computed ahead first; then further ones, as many as the missing tokens are expected to need
      int Jn = J < Jpre ? Jpre : J + walk_region(want - have, n_s, mlen, kk);
      Jn = min(min(Jn, mlen), J + LROUND);
      const int j0 = J + tid * 4;
      int tokc[4], phc[4];
#pragma unroll
      for (int q_ = 0; q_ < 4; ++q_) {
        const int jj = j0 + q_;
        tokc[q_] = -1; phc[q_] = 0;
        if (jj < Jn) {
          // (a marked entry reads -1; with too many members for marking, none is marked: test them all)
          const int tok = jj < Jpre ? __ldcg(pre + jj) : s0 + walk_at(wk, jj);
          if (tok >= 0) {
            const float sv = cached ? unord_f32(~keys[key_slot(tok)]) : __ldg(sc + tok);
            if (!in_topk(mt, sm.vtab, gbitmap, tok, sv)) tokc[q_] = tok;
          }
          if (tokc[q_] >= 0) phc[q_] = page_of(p, b, tokc[q_] >> 4);
        }
      }
      int cnt = 0;
#pragma unroll
      for (int q_ = 0; q_ < 4; ++q_) cnt += tokc[q_] >= 0;
      int tot1;
      int idx = block_scan_reg(cnt, sm.misc + 32, tot1);          // rank inside the round
      const int nlist = min(tot1, want - have);
#pragma unroll
      for (int q_ = 0; q_ < 4; ++q_) {
        if (tokc[q_] >= 0) {
          if (idx < nlist) { st_tok[idx] = tokc[q_]; st_ph[idx] = phc[q_] * VATTN_BLOCK + (tokc[q_] & 15); }
          ++idx;
        }
      }
      __syncthreads();
      for (int x = tid; x < nlist; x += NT) {
        const int r_ = have + x;
        bl_tok[r_] = st_tok[x]; bl_tok[p.npad + r_] = st_ph[x];
        if (bdbg) bdbg[r_] = st_tok[x];
      }
      have += tot1;
      J = Jn;
      __syncthreads();
    }
  }
  // the head's record, then "I_t is written and marked" for the statistics kernel.  The barrier orders every
  // thread's writes before thread 0's release, which is cumulative: one fence, not one per thread.
  __syncthreads();
  if (tid == 0) {
    p.meta[bh] = mt;
    const unsigned long long word = 2ull | ((unsigned long long)base_list << 2) | ((unsigned long long)(unsigned)base_J << 3) |
                                    ((unsigned long long)(unsigned)piv_ph << 32);
    asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p.flags64 + bh), "l"(word) : "memory");
    DBGH(bh, 1);
  }
  // ---- the final walk: marks in its array, positions of all members (read by the budget code and the gather
  //      kernel, which start after this kernel has completed)
  if (n_s > 0 && kk <= NT * 4) {
    int* hp1 = p.hole_pos + (long long)bh * 2 * VATTN_BANDCAP;     // positions inside the walk array; + BANDCAP: beyond it
    const Walk wk1 = make_walk(sm.rkeys + 8, mlen);
    for (int a = tid; a < kk; a += NT) {
      const int x1 = walk_inv(wk1, __ldcg(tk + a) - s0);
      if (x1 < W1) {
        wa1[x1] = -1;
        const int i1 = atomicAdd(&cnts[1], 1);
        if (i1 < VATTN_BANDCAP) hp1[i1] = x1;
      } else {                                         // (budgets that reach beyond the array need these)
        const int i2 = atomicAdd(&cnts[2], 1);
        if (i2 < VATTN_BANDCAP) hp1[VATTN_BANDCAP + i2] = x1;
      }
    }
    __syncthreads();
    if (tid == 0) {
      holes1 = cnts[1]; holes2 = cnts[2];
      // every member's position is known: any budget can be served as "the non-members among the first J
      // positions" (entries beyond the array are computed by the gather kernel); else only budgets inside the array
      if (holes1 <= VATTN_BANDCAP) { dyn_J = W1; dyn_listed = holes2 <= VATTN_BANDCAP ? n_s : W1 - holes1; }
      HeadMeta* gm = p.meta + bh;
      gm->holes1 = min(holes1, VATTN_BANDCAP); gm->holes2 = min(holes2, VATTN_BANDCAP);
      gm->dyn_J = dyn_J; gm->dyn_listed = dyn_listed;
    }
  }
  TICK_END(p, VATTN_K_SELECT);
}

// The tokens of the first walk positions of both walks, for every head.  sigma depends on (seed, layer, step, batch
// row, head, stream, sequence length) only, not on K or the scores, so it is evaluated here, beside the score pass
// (which is bound by HBM and leaves the integer pipes idle); the selection kernel then only looks tokens up.
__global__ void __launch_bounds__(256) k_walk(const Prob p) {
  __shared__ unsigned keys[16];
  pdl_trigger();
  TICK_BEGIN(p, VATTN_K_WALK);
  const int tid = threadIdx.x, bh = blockIdx.y;
  const int b = bh / p.Hq, h = bh % p.Hq;
  const int n = head_len(p, b, h);
  const Geo geo = head_geometry(p, n);
  const int mlen = geo.l_start - geo.s0;
  const int J0 = walk_region(geo.b0, geo.n_s, mlen, geo.kk);
  const int J1 = walk_region(dyn_listed_want(p, geo.n_s, geo.b0), geo.n_s, mlen, geo.kk);
  // (the grid is sized for the longest sequence a plan takes: a CTA without positions leaves before the round keys)
  // CTA x takes positions [1024 x, 1024 x + 1024) of the two walks laid end to end.  Cycle walking repeats the
  // network until the value falls below |M|; with |M| just above a power of two that is two passes on average and
  // four or five for the slowest lane of a warp, so a lane does not wait for its neighbours: it has several
  // positions to do and goes on to its next one as soon as one is finished (one pass per loop iteration).
  constexpr int PER = 1024;
  if (geo.n_s > 0 && (int)blockIdx.x * PER < J0 + J1) {
    if (tid < 4) walk_keys(p, b, h, tid >> 1, tid & 1, keys + (tid >> 1) * 8);
    __syncthreads();
    int* out0 = p.walk_tok + (long long)bh * 4 * p.npad;       // [walk][tokens, physical slots][npad]
#pragma unroll 1
    for (int x_lo = (int)blockIdx.x * PER; x_lo < J0 + J1; x_lo += (int)gridDim.x * PER) {     // (the grid normally covers the range once)
    const int x_hi = min(x_lo + PER, J0 + J1);
#pragma unroll 1
    for (int which = 0; which < 2; ++which) {          // the part of this CTA's range in the base walk, then in the final walk
      const int a = which == 0 ? x_lo : max(x_lo, J0), e = which == 0 ? min(x_hi, J0) : x_hi;
      if (a >= e) continue;
      const Walk w = make_walk(keys + ((which == 1 || p.nested_base) ? 8 : 0), mlen);
      const int off = which == 0 ? 0 : J0;
      int* dst = out0 + (which == 0 ? 0 : 2 * p.npad);
      int x = a + tid;
      unsigned cur = (unsigned)(x - off);
      while (x < e) {
        cur = walk_pass(w, cur);
        if (cur < w.mlen) {
          const int tok = geo.s0 + (int)cur;
          dst[x - off] = tok;
          dst[p.npad + x - off] = page_of(p, b, tok >> 4) * VATTN_BLOCK + (tok & 15);
          x += 256;
          cur = (unsigned)(x - off);
        }
      }
    }
    }
  }
  TICK_END(p, VATTN_K_WALK);
  // This grid does not wait for the score kernel before it, so one of its CTAs does at the end: "this grid has
  // completed" then implies "the score kernel has completed" for the selection kernel behind it.
  if (blockIdx.x == 0 && blockIdx.y == 0) pdl_wait();
}

}  // namespace

cudaError_t launch_walk(const Prob& p, cudaStream_t s) {
  // positions per head: about 1.03 (b0 + 8 b0), or the whole middle range under a forced budget
  const double b0max = (double)p.base_rate * (double)p.max_seq_len + 2.0;
  double pos = p.force_budget >= 0 ? (double)p.max_seq_len + 1.1 * b0max : (1.2 + 1.05 * VATTN_WALK_B0S) * b0max + 64.0;
  if (pos > 2.0 * p.max_seq_len) pos = 2.0 * p.max_seq_len;
  int gx = (int)(pos / 1024.0) + 1;                    // 1024 positions per CTA
  if (gx > 65535) gx = 65535;
  return launch_pdl(k_walk, dim3((unsigned)gx, (unsigned)(p.B * p.Hq)), dim3(256), 0, s, p);
}

template <typename T, int D>
static cudaError_t launch_select_t(const Prob& p, cudaStream_t s) {
  static size_t have[VATTN_MAXDEV];
  cudaError_t e = optin_smem(k_select<T, D>, SMEM_BYTES, have);
  if (e != cudaSuccess) return e;
  return launch_pdl(k_select<T, D>, dim3((unsigned)(p.B * p.Hq)), dim3(NT), SMEM_BYTES, s, p);
}

cudaError_t launch_select(const Prob& p, cudaStream_t s) {
  if (p.dtype == VATTN_DTYPE_BF16) {
    if (p.D == 128) return launch_select_t<bf16_t, 128>(p, s);
    return launch_select_t<bf16_t, 64>(p, s);
  }
  if (p.D == 128) return launch_select_t<float, 128>(p, s);
  return launch_select_t<float, 64>(p, s);
}
