// Sampled part of the estimator and the final combination (Sec. 4.1 of the paper):
//     N = N_f + (n_s/b) * sum_{I_dyn} w_i V[i],   D = D_f + (n_s/b) * sum_{I_dyn} w_i,   out = N / D
// which is SDPA_{S,p} of Sec. 3 with p = 1 on I_f and p = b/n_s on I_dyn.
//
// HBM-bound row gather.  Work unit = a chunk of consecutive entries of one head's I_dyn list.  LPR lanes
// fetch one V row with one 16-byte load each; a row group keeps 4 rows in flight and requests the next
// batch's indices (token + physical slot, written by the select kernels) while the current rows arrive.
// Rows are fetched with streaming loads (read once: first to leave the caches, so that the scores and index
// lists stay in L2).  Weights come from the stored fp32 scores (no K re-read).  Partials are added in chunk order by the
// last CTA of the head ("ticket"), so results are reproducible.
//
// Two decompositions:
//  * flat (batch * heads <= 128): budgets differ a lot between heads, so the chunks of all heads form one
//    list (a prefix sum over the heads' chunk counts, recomputed by every CTA) that the CTAs walk with a
//    grid stride.  A chunk is a whole number of batches (a batch = what one CTA keeps in flight at once:
//    32 rows of 128 bf16) and a head uses up to 32 chunks (64 to 128 when no more than 18 heads share the
//    grid): lists of more batches than that get chunks of
//    two, three, ... batches, whose index loads overlap the previous batch's rows.  (With up to 128
//    single-batch chunks per head the last finisher needed three dependent rounds of partial loads and
//    long lists overflowed the grid: 92 -> 76 us per step at 5x density, 73.0 -> 72.4 us at 10x.);
//  * per head (larger problems): grid (32, heads, batch); a head with budget b uses ceil(b / chunk) of its
//    32 CTAs, chunk = max(256, ceil(b / 32)) rows, the others exit at once.
#include "vattn_internal.cuh"
#include <type_traits>

namespace {

// what this kernel needs of a head, as the statistics kernel left it (16 bytes: the table of all heads is four cache
// lines at 32 heads, and every CTA reads all of it)
// b: the budget; L: entries to visit (a prefix of the final sample's walk array, members of I_t marked, or the b
// entries of the head's list when `list` is set); n = 0: an empty row
// W1: entries of the walk array (the gather computes the ones beyond it)
// start: entries before it are accounted for already (nested samples: the base sample's rows)
struct GMeta { int b, n_s; float m; int n, L, list, W1, start; };
__device__ __forceinline__ GMeta ld_gmeta(const int4* g) {
  const int4 v = __ldcg(g);
  GMeta r; r.b = v.x; r.n_s = v.y; r.m = __int_as_float(v.z);
  r.n = v.w < 0 ? 0 : 1; r.L = v.w < 0 ? 0 : (v.w >> 1); r.list = v.w < 0 ? 0 : (v.w & 1);
  const int2 w = __ldcg(reinterpret_cast<const int2*>(g + 1));
  r.W1 = w.x; r.start = w.y;
  return r;
}

constexpr int NT = 128;
constexpr int NWARP = NT / 32;
constexpr int UNROLL = 4;         // rows in flight per row group (16-byte slices kept raw until used); 8 and 2 are slower
constexpr int MAXS = 32;           // most chunks (partials) per head, per-head decomposition
constexpr int FLAT_MAX_HEADS = VATTN_GATHER_FLAT_HEADS;
constexpr int MIN_CHUNK = 64;      // rows of a chunk in the per-head decomposition are >= 4 * MIN_CHUNK (8 * from 512 heads on)

template <typename T, int D, bool KV>
struct Gather {
  static constexpr int EPL = Elem<T>::EPL, LPR = D / EPL, RPI = 32 / LPR, NE = D + 1, RG = NWARP * RPI;
  static_assert(LPR >= UNROLL, "each row of a batch needs a lane of its row group to own its weight");

  static __device__ __forceinline__ void unpack(const uint4& r, float (&v)[EPL]) {
    if (EPL == 8) {
      v[0] = __uint_as_float(r.x << 16); v[1] = __uint_as_float(r.x & 0xFFFF0000u);
      v[2] = __uint_as_float(r.y << 16); v[3] = __uint_as_float(r.y & 0xFFFF0000u);
      v[4 % EPL] = __uint_as_float(r.z << 16); v[5 % EPL] = __uint_as_float(r.z & 0xFFFF0000u);
      v[6 % EPL] = __uint_as_float(r.w << 16); v[7 % EPL] = __uint_as_float(r.w & 0xFFFF0000u);
    } else {
      v[0] = __uint_as_float(r.x); v[1] = __uint_as_float(r.y); v[2] = __uint_as_float(r.z); v[3] = __uint_as_float(r.w);
    }
  }
  // Entries of the final sample's walk beyond its array (budgets of more than about eight base budgets): the token
  // of such a position is computed here (sigma), its membership in I_t decided from its score like the selection
  // kernel would.  keys: the walk's round keys, mt: the head's record (both in shared memory).
  // ident: the budget is the whole residual; every middle token is visited, in token order (no walk needed).
  struct Far { bool on, ident; int W1, s0, mlen; const unsigned* keys; const HeadMeta* mt; };
  // rows [r_begin, r_end) of head bh -> partial `slot`; the last of `nslots` finishers combines
  template <bool FAR>
  static __device__ void run(const Prob& p, int bh, const GMeta& meta, int r_begin, int r_end, const Far& far, int slot, int nslots,
                             float (*part)[NE], int* is_last, float* s_den) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int h = bh % p.Hq, g = h / p.G;
    T* out = reinterpret_cast<T*>(p.out) + q_row(p, bh / p.Hq, h);
    if (meta.n == 0) {
      if (slot == 0) for (int e = tid; e < D; e += NT) out[e] = Elem<T>::from_float(0.f);
      return;
    }
    // I_dyn: the unmarked entries of a prefix of the final sample's walk array (a marked entry, token -1, is a
    // member of I_t: its row is fetched like the others and weighs nothing), or the head's list
    const int* dyn = meta.list ? p.dyn_idx + (long long)bh * 3 * p.npad : p.walk_tok + ((long long)bh * 4 + 2) * p.npad;
    const int* dph = dyn + p.npad;
    const float* sc = p.scores + (long long)bh * p.npad;
    const T* vc = reinterpret_cast<const T*>(p.vc) + (long long)g * p.sh;
    const float m = meta.m;
    const int rsub = lane / LPR, j = lane % LPR;
    const int rg = warp * RPI + rsub;
    const int iters = (r_end - r_begin + RG - 1) / RG;

    float acc[EPL], dd = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = 0.f;

    // A batch = UNROLL rows per row group.  Batches whose rows all exist (every one but a chunk's last) run a
    // body without per-row validity tests; FULL is a compile-time tag.
    const int full_iters = ((r_end - r_begin) / (RG * UNROLL)) * UNROLL;
    int tok_n[UNROLL], ph_n[UNROLL];
    auto fetch_idx = [&](int k0, auto full_tag) {
      constexpr bool FULL = decltype(full_tag)::value;
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
        const int r = r_begin + rg + (k0 + u) * RG;
        const bool ok = (FULL || ((k0 + u < iters) && (r < r_end))) && !(FAR && far.ident);
        // (FAR, not ident: this CTA has just extended the array over its entries: they are read back through L2)
        tok_n[u] = ok ? (FAR ? __ldcg(dyn + r) : __ldg(dyn + r)) : -1;
        ph_n[u] = ok ? (FAR ? __ldcg(dph + r) : __ldg(dph + r)) : 0;
      }
      if (FAR && far.ident) {                           // the whole residual: entry r is middle token r
        int cph = 0;                                    // lane u of a row group looks up row u's page
        if (j < UNROLL) {
          const int r = r_begin + rg + (k0 + j) * RG;
          if (FULL || ((k0 + j < iters) && (r < r_end))) {
            const int tok = far.s0 + r;
            cph = page_of(p, bh / p.Hq, tok >> 4) * VATTN_BLOCK + (tok & 15);
          }
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
          const int r = r_begin + rg + (k0 + u) * RG;
          const bool ok = FULL || ((k0 + u < iters) && (r < r_end));
          tok_n[u] = ok ? far.s0 + r : -1;
          ph_n[u] = __shfl_sync(0xFFFFFFFFu, cph, u, LPR);
        }
      }
    };
    auto fetch_next = [&](int k0) {                   // indices of the batch that starts at iteration k0, if any
      if (k0 >= iters) return;
      if (k0 + UNROLL <= full_iters) fetch_idx(k0, std::true_type{});
      else fetch_idx(k0, std::false_type{});
    };
    // a computed entry's token may be a member of I_t (nothing marked it): its score s decides
    auto far_member = [&](int k0, int u, int tok, float s) -> bool {
      if (!FAR || !far.ident || tok < 0) return false;
      return in_topk(*far.mt, p.vtab + (long long)bh * VATTN_BANDCAP, p.bitmap + (long long)bh * p.nwords, tok, s);
    };
    // K+V variant: the score of a sampled token is recomputed from its K row (what a selector that leaves no
    // scores for the whole context behind would need); the K slices of a batch come first, then its V slices
    float qf[EPL];
    const T* kcg = reinterpret_cast<const T*>(p.kc) + (long long)g * p.sh;
    if (KV) Elem<T>::load(reinterpret_cast<const T*>(p.q) + q_row(p, bh / p.Hq, h) + j * EPL, qf);
    auto batch = [&](int k0, auto full_tag) {
      constexpr bool FULL = decltype(full_tag)::value;
      // lane u of a row group owns row u's weight: one score load and one exp per row instead of LPR
      int tok[UNROLL], tok_mine = -1;
      float w_mine = 0.f;
      uint4 raw[UNROLL];
      if (KV) {
        long long off[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
          tok[u] = tok_n[u];
          int ph = ph_n[u];
          CHECK_SLOT(p, ph, 2);
          off[u] = (long long)(ph >> 4) * p.sb + (long long)(ph & 15) * p.st + j * EPL;
          if (!FULL) raw[u] = make_uint4(0u, 0u, 0u, 0u);
          if (FULL || tok[u] >= 0) raw[u] = __ldcs(reinterpret_cast<const uint4*>(kcg + off[u]));
        }
        fetch_next(k0 + UNROLL);
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
          float kv[EPL], dot = 0.f;
          unpack(raw[u], kv);
#pragma unroll
          for (int e = 0; e < EPL; ++e) dot = fmaf(qf[e], kv[e], dot);
#pragma unroll
          for (int mask = LPR / 2; mask >= 1; mask >>= 1) dot += __shfl_xor_sync(0xFFFFFFFFu, dot, mask);
          if (j == u) {
            w_mine = p.scale * dot;
            tok_mine = (FAR && tok[u] >= 0 && far_member(k0, u, tok[u], __ldg(sc + tok[u]))) ? -1 : tok[u];
          }
          if (!FULL) raw[u] = make_uint4(0u, 0u, 0u, 0u);
          if (FULL || tok[u] >= 0) raw[u] = __ldcs(reinterpret_cast<const uint4*>(vc + off[u]));
        }
      } else {
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
          tok[u] = tok_n[u];
          if (!FULL) raw[u] = make_uint4(0u, 0u, 0u, 0u);
          if (j == u) tok_mine = tok[u];
          if (FULL || tok[u] >= 0) {
            int ph = ph_n[u];
            CHECK_SLOT(p, ph, 3);
            raw[u] = __ldcs(reinterpret_cast<const uint4*>(vc + (long long)(ph >> 4) * p.sb + (long long)(ph & 15) * p.st + j * EPL));
          }
        }
        CHECK_TOK(p, tok_mine, 5);
        if (tok_mine >= 0) w_mine = __ldg(sc + tok_mine);
        fetch_next(k0 + UNROLL);
        if (FAR && j < UNROLL && far_member(k0, j, tok_mine, w_mine)) tok_mine = -1;                        // next batch's indices travel with this batch's rows
      }
      const float e_mine = (tok_mine >= 0) ? expf(w_mine - m) : 0.f;
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
        const float ww = __shfl_sync(0xFFFFFFFFu, e_mine, u, LPR);
        dd += ww;
        float v[EPL];
        unpack(raw[u], v);
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] = fmaf(ww, v[e], acc[e]);
      }
    };
    fetch_next(0);
    for (int k0 = 0; k0 < iters; k0 += UNROLL) {
      if (k0 + UNROLL <= full_iters) batch(k0, std::true_type{});   // uniform over the CTA
      else batch(k0, std::false_type{});
    }
#pragma unroll
    for (int mask = LPR; mask < 32; mask <<= 1) {
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc[e] += __shfl_xor_sync(0xFFFFFFFFu, acc[e], mask);
      dd += __shfl_xor_sync(0xFFFFFFFFu, dd, mask);
    }
    __syncthreads();                                  // `part` may still be read by the previous chunk
    DBGT(22);
    if (rsub == 0) {
#pragma unroll
      for (int e = 0; e < EPL; ++e) part[warp][j * EPL + e] = acc[e];
      if (j == 0) part[warp][D] = dd;
    }
    __syncthreads();
    float* gpart = p.gat_part + ((long long)bh * p.gat_slots + slot) * NE;
    for (int e = tid; e < NE; e += NT) {
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < NWARP; ++w) s += part[w][e];
      gpart[e] = s;
    }
    // (the barrier orders every thread's writes before thread 0's fence, which is cumulative; likewise on the way in)
    __syncthreads();
    if (tid == 0) {
      __threadfence();
      *is_last = (atomicAdd(&p.tickets[p.B * p.Hq + bh], 1u) == (unsigned)(nslots - 1));
      __threadfence();
    }
    __syncthreads();
    DBGT(23);
    if (!*is_last) return;
    DBGH(bh, 5);

    // last finisher of the head: every thread requests all partials of its element at once (one memory
    // round trip), adds them in slot order, scales by n_s/b and divides
    const int nb = meta.b;
    const double* det = p.det_sums + (long long)bh * (D + 1);
    const double f = (nb > 0) ? (double)meta.n_s / (double)nb : 0.0;
    const float* src0 = p.gat_part + (long long)bh * p.gat_slots * NE;
    float num_s[(D + NT - 1) / NT];
    double det_e[(D + NT - 1) / NT];
    const double det_d = __ldcg(det + D);             // N_f, D_f of the statistics kernel, requested with the partials
#pragma unroll
    for (int it = 0; it < (D + NT - 1) / NT; ++it) det_e[it] = (tid + it * NT < D) ? __ldcg(det + tid + it * NT) : 0.0;
#pragma unroll
    for (int it = 0; it < (D + NT - 1) / NT; ++it) {
      const int e = tid + it * NT;
      float s = 0.f;
      for (int s0 = 0; s0 < nslots; s0 += 32) {       // 32 partials per round trip, added in slot order
        float vv[32];
#pragma unroll
        for (int sp = 0; sp < 32; ++sp) vv[sp] = (s0 + sp < nslots && e < D) ? __ldcg(src0 + (long long)(s0 + sp) * NE + e) : 0.f;
#pragma unroll
        for (int sp = 0; sp < 32; ++sp) s += vv[sp];
      }
      num_s[it] = s;
    }
    if (warp == 0) {                                  // the denominator: lane sp holds slot s0 + sp
      float s = 0.f;
      for (int s0 = 0; s0 < nslots; s0 += 32) {
        const float vd = (s0 + lane < nslots) ? __ldcg(src0 + (long long)(s0 + lane) * NE + D) : 0.f;
#pragma unroll
        for (int sp = 0; sp < 32; ++sp) s += __shfl_sync(0xFFFFFFFFu, vd, sp);
      }
      if (lane == 0) *s_den = s;
    }
    __syncthreads();
    const double den = det_d + f * (double)(*s_den);
#pragma unroll
    for (int it = 0; it < (D + NT - 1) / NT; ++it) {
      const int e = tid + it * NT;
      if (e < D) out[e] = Elem<T>::from_float((float)((det_e[it] + f * (double)num_s[it]) / den));
    }
  }
};


// Entries [x_lo, x_hi) of head bh's final walk beyond what the walk kernel laid out (budgets of more than about eight
// base budgets): the CTA that will gather them writes them into the walk array first.  Pass 1: positions -> tokens,
// a thread going on to its next position as soon as one cycle walk ends; pass 2: the tokens' scores decide membership
// in I_t as the selection kernel would (marked: token -1), slots from the block table; four entries per thread and
// round trip.  keys: the walk's round keys, mt: the head's record (both in shared memory).
__device__ void extend_walk_array(const Prob& p, int bh, const unsigned* keys, const HeadMeta* mt, int x_lo, int x_hi) {
  const int tid = threadIdx.x, b = bh / p.Hq;
  int* wt = p.walk_tok + ((long long)bh * 4 + 2) * p.npad;
  int* wp = wt + p.npad;
  const Walk wk = make_walk(keys, mt->l_start - mt->s0);
  {
    int x = x_lo + tid;
    unsigned cur = (unsigned)x;
    while (x < x_hi) {
      cur = walk_pass(wk, cur);
      if (cur < wk.mlen) { wt[x] = mt->s0 + (int)cur; x += NT; cur = (unsigned)x; }
    }
  }
  __syncthreads();
  const int* vt = p.vtab + (long long)bh * VATTN_BANDCAP;
  const float* sc = p.scores + (long long)bh * p.npad;
  const unsigned* gbitmap = p.bitmap + (long long)bh * p.nwords;
  for (int x0 = x_lo; x0 < x_hi; x0 += 4 * NT) {
    int tk4[4], pg4[4];
    float s4[4];
#pragma unroll
    for (int q_ = 0; q_ < 4; ++q_) { const int x = x0 + q_ * NT + tid; tk4[q_] = x < x_hi ? __ldcg(wt + x) : -1; }
#pragma unroll
    for (int q_ = 0; q_ < 4; ++q_) {
      s4[q_] = tk4[q_] >= 0 ? __ldg(sc + tk4[q_]) : 0.f;
      pg4[q_] = tk4[q_] >= 0 ? page_of(p, b, tk4[q_] >> 4) : 0;
    }
#pragma unroll
    for (int q_ = 0; q_ < 4; ++q_) {
      const int x = x0 + q_ * NT + tid;
      if (tk4[q_] >= 0) {
        if (in_topk(*mt, vt, gbitmap, tk4[q_], s4[q_])) wt[x] = -1;
        wp[x] = pg4[q_] * VATTN_BLOCK + (tk4[q_] & 15);
      }
    }
  }
  __syncthreads();
}

// what a unit needs for entries beyond the walk array (see Gather::Far); uniform over the CTA
template <typename G>
__device__ __forceinline__ typename G::Far far_setup(const Prob& p, int bh, const GMeta& meta, int nb, unsigned* s_keys, HeadMeta* s_mt) {
  typename G::Far far;
  far.ident = meta.n > 0 && !meta.list && meta.b >= meta.n_s && meta.b > 0;
  far.W1 = far.ident ? 0 : meta.W1;
  far.on = meta.n > 0 && !meta.list && meta.L > far.W1;
  far.s0 = 0; far.mlen = 1; far.keys = s_keys; far.mt = s_mt;
  if (far.on) {                                        // the head's record and its walk's round keys, as the selection kernel left them
    if (threadIdx.x < 8) s_keys[threadIdx.x] = __ldcg(p.wkeys + (long long)bh * 8 + threadIdx.x);
    if (threadIdx.x == 32) *s_mt = ld_meta(p.meta + bh);
    __syncthreads();
    far.s0 = s_mt->s0; far.mlen = s_mt->l_start - s_mt->s0;
  }
  return far;
}

template <typename T, int D, bool KV>
__global__ void __launch_bounds__(NT, 8) k_gather(const Prob p) {
  using G = Gather<T, D, KV>;
  __shared__ float part[NWARP][G::NE];
  __shared__ int is_last;
  __shared__ float s_den;
  __shared__ unsigned s_keys[8];
  __shared__ HeadMeta s_mt;
  __shared__ unsigned s_ready;
  TICK_BEGIN(p, VATTN_K_GATHER);
  const int bh = blockIdx.z * p.Hq + blockIdx.y;
  // A head's CTAs start when that head's budget is published (the statistics kernel's last CTA of the head
  // releases a word), not when the whole statistics kernel has completed: heads finish over tens of microseconds
  // at large batch.  Every CTA of the statistics kernel had started before this grid was launched, so the wait
  // cannot starve; it is bounded and falls back to the grid-level wait.  CTAs leave as soon as they are done (a CTA
  // that waited for the grid at its end would hold its slot against the CTAs behind it); one CTA does wait, so
  // that "this grid has completed" implies "the statistics kernel has".
  const bool anchor = blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0;
  if (threadIdx.x == 0) s_ready = wait_word32(p.tickets + bh, VATTN_WORD_SPINS);
  __syncthreads();
  const bool waited = s_ready == 0u;
  if (waited) pdl_wait();                               // uniform over the CTA
  const GMeta meta = ld_gmeta(p.gat_meta + 2 * bh);
  const int nb = meta.n > 0 ? meta.L - meta.start : 0; // entries to visit: [start, L)
  // chunks of at least MIN_CHUNK rows, at most MAXS of them; CTAs beyond the head's chunk count leave at once
  // (with this many heads the kernel is throughput-bound: 4 batches per row group amortise the fixed hops; from 512
  // heads on, twice that: 285 instead of 303 us at batch 32, while at batch 8 it would cost 3 us)
  const int chunk = max((p.B * p.Hq >= 512 ? 8 : 4) * MIN_CHUNK, (nb + MAXS - 1) / MAXS);
  const int nslots = max(1, (nb + chunk - 1) / chunk);
  if ((int)blockIdx.x < nslots) {
    const int r_begin = meta.start + min(nb, (int)blockIdx.x * chunk), r_end = min(meta.L, r_begin + chunk);
    const typename G::Far far = far_setup<G>(p, bh, meta, nb, s_keys, &s_mt);
    if (far.on && !far.ident && r_end > far.W1) extend_walk_array(p, bh, s_keys, &s_mt, max(r_begin, far.W1), r_end);
    if (far.on) G::template run<true>(p, bh, meta, r_begin, r_end, far, blockIdx.x, nslots, part, &is_last, &s_den);
    else G::template run<false>(p, bh, meta, r_begin, r_end, far, blockIdx.x, nslots, part, &is_last, &s_den);
    TICK_END(p, VATTN_K_GATHER);
  }
  if (anchor && !waited) pdl_wait();
}

template <typename T, int D, bool KV>
__global__ void __launch_bounds__(NT, 8) k_gather_flat(const Prob p) {
  using G = Gather<T, D, KV>;
  __shared__ float part[NWARP][G::NE];
  __shared__ int is_last;
  __shared__ float s_den;
  __shared__ unsigned s_keys[8];
  __shared__ HeadMeta s_mt;
  __shared__ unsigned s_ready;
  TICK_BEGIN(p, VATTN_K_GATHER);
  const int tid = threadIdx.x;
  const int BH = p.B * p.Hq;
  constexpr int BATCH = G::RG * UNROLL;               // rows a CTA keeps in flight at once
  // Work unit u = chunk u / BH of head u % BH: neighbouring CTAs (which tend to share an SM) serve different heads,
  // whose chunks differ in length.  A head's units start as soon as its budget is published (a per-head word that
  // the statistics kernel's last CTA of the head releases), not when all budgets are known.  Every CTA of the
  // statistics kernel had started before this grid was launched (programmatic dependent launch), so the wait
  // cannot starve; it is bounded all the same and falls back to the grid-level dependency wait.
  bool waited = false;
  for (int u = blockIdx.x; u < BH * p.gat_slots; u += gridDim.x) {
    const int bh = u % BH, ci = u / BH;
    if (tid == 0) {
      const unsigned v = waited ? 0u : wait_word32(p.tickets + bh, VATTN_WORD_SPINS);
      s_ready = v;
    }
    __syncthreads();
    if (!waited && s_ready == 0u) { pdl_wait(); waited = true; }      // uniform over the CTA
    DBGT(21);
    const GMeta meta = ld_gmeta(p.gat_meta + 2 * bh);
    const int nb = meta.n > 0 ? meta.L - meta.start : 0;       // entries to visit: [start, L)
    const int batches = (nb + BATCH - 1) / BATCH;
    const int rows = BATCH * max(1, (batches + p.gat_slots - 1) / p.gat_slots);
    const int nslots = max(1, (nb + rows - 1) / rows); // a head without samples still writes its output
    if (ci < nslots) {
      const int r_begin = meta.start + min(nb, ci * rows), r_end = min(meta.L, r_begin + rows);
      const typename G::Far far = far_setup<G>(p, bh, meta, nb, s_keys, &s_mt);
      if (far.on && !far.ident && r_end > far.W1) extend_walk_array(p, bh, s_keys, &s_mt, max(r_begin, far.W1), r_end);
      if (far.on) G::template run<true>(p, bh, meta, r_begin, r_end, far, ci, nslots, part, &is_last, &s_den);
      else G::template run<false>(p, bh, meta, r_begin, r_end, far, ci, nslots, part, &is_last, &s_den);
    }
    __syncthreads();
  }
  TICK_END(p, VATTN_K_GATHER);
  if (!waited) pdl_wait();                             // "this grid has completed" implies "the one before has"
}

}  // namespace

template <typename T, int D, bool KV>
static cudaError_t launch_gather_t(const Prob& p, cudaStream_t s) {
  const int BH = p.B * p.Hq;
  if (BH <= FLAT_MAX_HEADS) {
    // at most gat_slots chunks per head; 8 CTAs per SM walk them with a grid stride
    if (p.gat_slots < VATTN_GATHER_FLAT_SLOTS) return cudaErrorInvalidValue;
    const long long most = (long long)BH * p.gat_slots;
    const long long cap = 8ll * device_sm_count();
    const int grid = (int)(most < cap ? most : cap);
    return launch_pdl(k_gather_flat<T, D, KV>, dim3(grid), dim3(NT), 0, s, p);
  }
  if (p.gat_slots < MAXS) return cudaErrorInvalidValue;
  return launch_pdl(k_gather<T, D, KV>, dim3(MAXS, p.Hq, p.B), dim3(NT), 0, s, p);
}

cudaError_t launch_gather(const Prob& p, cudaStream_t s) {
  if (p.dtype == VATTN_DTYPE_BF16) {
    if (p.D == 128) return p.gather_kv ? launch_gather_t<bf16_t, 128, true>(p, s) : launch_gather_t<bf16_t, 128, false>(p, s);
    return p.gather_kv ? launch_gather_t<bf16_t, 64, true>(p, s) : launch_gather_t<bf16_t, 64, false>(p, s);
  }
  if (p.D == 128) return p.gather_kv ? launch_gather_t<float, 128, true>(p, s) : launch_gather_t<float, 128, false>(p, s);
  return p.gather_kv ? launch_gather_t<float, 64, true>(p, s) : launch_gather_t<float, 64, false>(p, s);
}
