// Index selection: one CTA per (batch row, query head).
//
//  k_select_topk_base : I_t = the k middle tokens with the largest score, ties to the lowest index
//                       (Algorithm 1 line 3, "oracle top-k" of Sec. 3), then the base sample
//                       I_bs = uniform-sample of b0 residual tokens (Algorithm 2 line 1).
//  k_select_final     : I_dyn = uniform-sample of b residual tokens (Algorithm 1 line 7).
//
// Both selections are "the c smallest (key, index) pairs": an 8-bit-digit radix select over 32-bit
// keys held in shared memory, followed by an ordered compaction through bitmaps, so every list comes
// out ascending.  Keys are the order-reversed score for top-k and Philox4x32-10 words for sampling.
//
// Exact top-k from fp32 scores: the stored scores differ from the exact inner products by at most
// gamma (a bound from the summation structure of the score kernel).  After the fp32 threshold T is
// known, tokens above T + 2*gamma are certainly selected and tokens below T - 2*gamma certainly not;
// the few in between are rescored in fp64 from their K rows and ranked exactly.
#include "vattn_internal.cuh"

namespace {

constexpr int NT = SEL_THREADS;
constexpr int NWARP = NT / 32;

struct Sm {
  double* band_s;     // [BANDCAP]
  unsigned* keys;     // [keycap]
  unsigned* w0;       // [nwords] selected / "less than threshold" bitmap
  unsigned* w1;       // [nwords] "equal to threshold" / band bitmap
  unsigned* w2;       // [nwords] I_t bitmap (residual mask) / scratch
  int* scan;          // [nwords]
  unsigned* hist;     // [256]
  int* band_idx;      // [BANDCAP]
  int* misc;          // [64]
};

__device__ __forceinline__ Sm carve(unsigned char* base, int keycap, int nwords) {
  Sm s;
  s.band_s = reinterpret_cast<double*>(base);            base += sizeof(double) * VATTN_BANDCAP;
  s.keys = reinterpret_cast<unsigned*>(base);            base += sizeof(unsigned) * (size_t)keycap;
  s.w0 = reinterpret_cast<unsigned*>(base);              base += sizeof(unsigned) * (size_t)nwords;
  s.w1 = reinterpret_cast<unsigned*>(base);              base += sizeof(unsigned) * (size_t)nwords;
  s.w2 = reinterpret_cast<unsigned*>(base);              base += sizeof(unsigned) * (size_t)nwords;
  s.scan = reinterpret_cast<int*>(base);                 base += sizeof(int) * (size_t)nwords;
  s.hist = reinterpret_cast<unsigned*>(base);            base += sizeof(unsigned) * 256;
  s.band_idx = reinterpret_cast<int*>(base);             base += sizeof(int) * VATTN_BANDCAP;
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
__device__ int finalize_emit(unsigned* sel, const unsigned* eq, int need_eq, int nw, int* scan, int* misc,
                             int* out_a, int* out_b) {
  const int tid = threadIdx.x;
  if (need_eq > 0) {
    for (int w = tid; w < nw; w += NT) scan[w] = __popc(eq[w]);
    __syncthreads();
    block_excl_scan(scan, nw, misc);
    for (int w = tid; w < nw; w += NT) sel[w] |= lowest_bits(eq[w], need_eq - scan[w]);
    __syncthreads();
  }
  for (int w = tid; w < nw; w += NT) scan[w] = __popc(sel[w]);
  __syncthreads();
  const int total = block_excl_scan(scan, nw, misc);
  for (int w = tid; w < nw; w += NT) {
    unsigned bits = sel[w];
    int pos = scan[w];
    while (bits) {
      const int bit = __ffs(bits) - 1;
      bits &= bits - 1;
      const int idx = w * 32 + bit;
      out_a[pos] = idx;
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
    return finalize_emit(sm.w0, sm.w1, 0, nw, sm.scan, sm.misc, out_a, out_b);
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
  return finalize_emit(sm.w0, sm.w1, need_eq, nw, sm.scan, sm.misc, out_a, out_b);
}

template <typename T, int D, bool CACHED>
__global__ void __launch_bounds__(NT, 1) k_select_topk_base(const Prob p, int keycap) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int h = blockIdx.x, b = blockIdx.y, g = h / p.G;
  const int bh = b * p.Hq + h;
  const Sm sm = carve(smem_raw, keycap, p.nwords);
  HeadMeta& meta = p.meta[bh];

  const int n = clamped_len(p, b);
  const int s0 = min(p.sink, n);
  const int l_start = max(n - p.window, s0);
  const int mlen = l_start - s0;
  int kb = p.k;
  if (p.topk_frac > 0.f) kb = (int)floor((double)p.topk_frac * (double)n);
  const int kk = min(kb, mlen);
  const int n_s = mlen - kk;
  int b0 = 0;
  if (n_s > 0) b0 = min(n_s, max(2, (int)floor((double)p.base_rate * (double)n_s)));
  const int nw = (n + 31) >> 5;
  const T* qrow = reinterpret_cast<const T*>(p.q) + (long long)bh * D;
  const float* sc = p.scores + (long long)bh * p.npad;
  const float m = (n > 0) ? unord_f32(p.m_ord[bh]) : 0.f;

  // gamma: bound on |fp32 score - exact score| (13 roundings, see the score kernel)
  if (warp == 0) {
    double sa = 0.0;
    for (int e = lane; e < D; e += 32) sa += fabs((double)Elem<T>::to_float(qrow[e]));
#pragma unroll
    for (int mk = 16; mk >= 1; mk >>= 1) sa += __shfl_xor_sync(0xFFFFFFFFu, sa, mk);
    const double kmax = (double)__uint_as_float(p.kabsmax[b * p.Hkv + g]);
    const double gm = 16.0 * 5.9604644775390625e-8 * fabs((double)p.scale) * sa * kmax * 1.000001;
    if (lane == 0) reinterpret_cast<float*>(sm.misc)[48] = __double2float_ru(gm);
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
  if (n == 0) return;

  // ------------------------------------------------------------------ top-k over the middle range
  for (int w = tid; w < nw; w += NT) { sm.w0[w] = 0u; sm.w1[w] = 0u; }
  __syncthreads();
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
    if (CACHED) {
      for (int i = s0 + tid; i < l_start; i += NT) sm.keys[i] = ~ord_f32(sc[i]);
      __syncthreads();
    }
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
  // emit I_t ascending, keep its bitmap (shared w2 + global)
  int* tk_out = p.topk_idx + (long long)bh * p.npad;
  int* tk_dbg = p.dbg.topk_idx ? p.dbg.topk_idx + (long long)bh * p.max_seq_len : nullptr;
  finalize_emit(sm.w0, sm.w1, 0, nw, sm.scan, sm.misc, tk_out, tk_dbg);
  for (int w = tid; w < p.nwords; w += NT) {
    const unsigned v = (w < nw) ? sm.w0[w] : 0u;
    sm.w2[w] = v;
    gbitmap[w] = v;
  }
  __syncthreads();

  // ------------------------------------------------------------------ base sample (Philox stream 0)
  const int hrng = p.rng_head_is_kv ? g : h;
  int* bs_out = p.base_idx + (long long)bh * p.npad;
  int* bs_dbg = p.dbg.base_idx ? p.dbg.base_idx + (long long)bh * p.max_seq_len : nullptr;
  sample_select<CACHED>(p, sm, s0, l_start, nw, b0, n_s, b, hrng, 0, sm.w2, bs_out, bs_dbg);
}

template <bool CACHED>
__global__ void __launch_bounds__(NT, 1) k_select_final(const Prob p, int keycap) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int tid = threadIdx.x;
  const int h = blockIdx.x, b = blockIdx.y, g = h / p.G;
  const int bh = b * p.Hq + h;
  const Sm sm = carve(smem_raw, keycap, p.nwords);
  const HeadMeta meta = p.meta[bh];
  if (p.dbg.dyn_cnt && tid == 0) p.dbg.dyn_cnt[bh] = meta.b;
  if (meta.n == 0 || meta.b <= 0) return;
  const int nw = (meta.n + 31) >> 5;
  const unsigned* gbitmap = p.bitmap + (long long)bh * p.nwords;
  for (int w = tid; w < nw; w += NT) sm.w2[w] = gbitmap[w];
  __syncthreads();
  const int hrng = p.rng_head_is_kv ? g : h;
  int* out = p.dyn_idx + (long long)bh * p.npad;
  int* dbg = p.dbg.dyn_idx ? p.dbg.dyn_idx + (long long)bh * p.max_seq_len : nullptr;
  sample_select<CACHED>(p, sm, meta.s0, meta.l_start, nw, meta.b, meta.n_s, b, hrng, 1, sm.w2, out, dbg);
}

}  // namespace

static int keycap_of(const Prob& p) { return p.npad <= VATTN_KEYCACHE_MAX ? p.npad : 0; }

size_t select_smem_bytes(const Prob& p) {
  return sizeof(double) * VATTN_BANDCAP + sizeof(unsigned) * (size_t)keycap_of(p) + 4 * sizeof(unsigned) * (size_t)p.nwords +
         sizeof(unsigned) * 256 + sizeof(int) * VATTN_BANDCAP + sizeof(int) * 64;
}

// Opt-in to large dynamic shared memory once per kernel and size (a function attribute, not a
// stream operation; done before the first launch so that later launches can be stream-captured).
template <typename KernelT>
static cudaError_t launch_sel(KernelT kern, const Prob& p, cudaStream_t s) {
  const size_t smem = select_smem_bytes(p);
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
  kern<<<grid, block, smem, s>>>(p, keycap_of(p));
  return cudaGetLastError();
}

cudaError_t launch_select_topk_base(const Prob& p, cudaStream_t s) {
  const bool cached = keycap_of(p) > 0;
  if (p.dtype == VATTN_DTYPE_BF16) {
    if (p.D == 128) return cached ? launch_sel(k_select_topk_base<bf16_t, 128, true>, p, s) : launch_sel(k_select_topk_base<bf16_t, 128, false>, p, s);
    return cached ? launch_sel(k_select_topk_base<bf16_t, 64, true>, p, s) : launch_sel(k_select_topk_base<bf16_t, 64, false>, p, s);
  }
  if (p.D == 128) return cached ? launch_sel(k_select_topk_base<float, 128, true>, p, s) : launch_sel(k_select_topk_base<float, 128, false>, p, s);
  return cached ? launch_sel(k_select_topk_base<float, 64, true>, p, s) : launch_sel(k_select_topk_base<float, 64, false>, p, s);
}

cudaError_t launch_select_final(const Prob& p, cudaStream_t s) {
  return keycap_of(p) > 0 ? launch_sel(k_select_final<true>, p, s) : launch_sel(k_select_final<false>, p, s);
}
