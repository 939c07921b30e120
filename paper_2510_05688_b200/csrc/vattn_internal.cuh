// Internal declarations shared by the kernels of libvattn (sm_100a).  Not part of the ABI.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "vattn.h"

#define VATTN_BLOCK 16                 // tokens per KV page
#define VATTN_MAX_SEQ (1 << 18)        // longest sequence a plan accepts
#define VATTN_BANDCAP 1024             // near-tie top-k candidates ranked from a list (more: exact radix select)
#define SEL_THREADS 1024               // threads of the selection kernel (one CTA per head)
#ifndef VATTN_WALK_B0S
#define VATTN_WALK_B0S 8                 // base budgets of the final walk that the walk kernel lays out ahead
#endif
#define VATTN_STAT_MAXS 16             // most split CTAs per head and row kind of the statistics kernel
#define VATTN_GATHER_FLAT_HEADS 128    // the gather kernel's flat decomposition serves up to this many heads ...
#define VATTN_GATHER_FLAT_SLOTS 32     // ... with up to this many chunks (partials) each

// Per (batch row, query head) record, written by the selection kernel for the row kernels.
struct HeadMeta {
  int n;            // tokens in the sequence (clamped to [0, max_seq_len])
  int s0;           // |I_s| = min(sink, n)
  int l_start;      // first token of the local window; middle range M = [s0, l_start)
  int kk;           // |I_t| = min(k, |M|)
  int n_s;          // residual size |M| - kk
  int b0;           // base-sample size
  int nbt;          // near-tie tokens of the top-k threshold (listed in vtab unless band_mode is set)
  int band_mode;    // 1: the near-ties were too many for the list; their verdicts are bits of the bitmap
  float m;          // largest fp32 score of the head (softmax stabiliser)
  float hi, lo;     // a middle token is in I_t if its score is above hi; scores in [lo, hi] are near-ties
  int run1;         // the list of I_t is two ascending runs: [0, run1) and [run1, kk)
  int dyn_listed;   // budgets up to this many are served as "the non-members among the first J positions of the final
  int dyn_J;        //   sample's walk" (dyn_J positions are in the walk array, members marked), larger ones from a list
  int path;         // code path of the selection (vattn_debug.paths)
  int b;            // final budget |I_dyn| (written by the statistics kernel)
  int base_J;       // the base sample = the unmarked entries among the first base_J of its walk array ...
  int holes2;       //   members of I_t at positions of the final sample's walk beyond its array (hole_pos + BANDCAP)
                    //   base_list = 1: the base sample is in base_idx instead
  int base_list;    //   (b0 entries, none marked)
  int holes1;       // marked entries among the first dyn_J of the final sample's walk (their positions in hole_pos)
};

// Everything a kernel needs, passed by value.
// floats in one split partial of the dense kernel: D unnormalised sums, the split's maximum, its sum of
// weights, and two floats of padding (records stay 16-byte aligned)
__host__ __device__ constexpr int dense_rec(int D) { return D + 4; }

struct Prob {
  int B, Hq, Hkv, G, D, dtype;   // Hq, G count (query token, head) pairs when a call carries several query tokens
  int Tq, G1;                    // query tokens per sequence (>= 1) and real query heads per KV head (G = Tq * G1)
  int max_blocks, num_blocks, max_seq_len, npad, nwords;   // npad: max_seq_len rounded up to 32; nwords = npad/32
  long long sb, sh, st;                                      // KV strides in elements
  const void* q; const void* kc; const void* vc; const int* bt; const int* seq_lens; void* out;
  int sink, window, k;
  float topk_frac, base_rate, scale;
  int mode, layer, step, rng_head_is_kv, force_budget;       // force_budget < 0: off
  int nested_base;        // 1: the base sample is the head of the final sample's walk
  int gather_kv;          // 1: the weights of the sampled tokens are recomputed from their K rows
  unsigned seed_lo, seed_hi;
  double eps, delta, z_delta;
  double z1[15], z2[15];                                     // z(delta*j/16), z(delta*(16-j)/16), j = 1..15
  // workspace
  float* scores;          // [B,Hq,npad]
  unsigned* m_ord;        // [B,Hq]  order-preserving encoding of the running max score
  unsigned* kabsmax;      // [B,Hkv] bits of max |K element| over the sequence
  unsigned* unit_ctr;     // [1] work-unit counter of the persistent score kernel
  unsigned long long* flags64;   // [B,Hq] word the selection kernel publishes per head when I_t is written and marked in
                          //   the walk arrays: 2 | base_list << 2 | base_J << 3 | pivot's physical slot << 32 (zero: not yet)
  unsigned* tickets;      // [5,B,Hq] [0] "the head's budget is published" (statistics kernel -> gather kernel);
                          //          "last CTA done" counters of [1] the gather kernel, [2] the dense kernel and [3] the
                          //          statistics kernel; [4] "the list of I_t is written" (selection -> statistics kernel)
  unsigned* status;       // [1]
  unsigned* bitmap;       // [B,Hq,nwords] near-tie tokens that made it into I_t (used when they are too many for a list)
  int* vtab;              // [B,Hq,BANDCAP] near-tie tokens ascending, bit 31 = member of I_t
  int* topk_idx;          // [B,Hq,2,npad] I_t as two ascending runs, then the physical slot (page * 16 + token % 16) of
                          //               every entry
  int* base_idx;          // [B,Hq,2,npad] I_bs in walk order: tokens, physical slots
  int* walk_tok;          // [B,Hq,2,2,npad] the first positions of both walks (computed beside the score pass): per
                          //   walk the tokens, then their physical slots.  The selection kernel marks the members
                          //   of I_t (token = -1; the slot stays valid): a sample is the unmarked entries of a prefix
  unsigned* wkeys;        // [B,Hq,8] round keys of the final sample's walk (for the gather kernel's array extension)
  int* hole_pos;          // [B,Hq,2,VATTN_BANDCAP] positions of the marked entries of the final sample's walk array, in
                          //   no particular order (the first 256 words read INT_MAX where there is none); then the
                          //   positions of the members of I_t beyond the array
  int* dyn_idx;           // [B,Hq,3,npad] I_dyn as a list (tokens, physical slots) for budgets beyond the walk arrays
                          //               (scratch of the near-tie overflow path while the selection runs)
  HeadMeta* meta;         // [B,Hq]
  double* stat_part;      // [B,Hq,2*16,D+3]  partials of the statistics kernel (deterministic-row CTAs, then base-row CTAs)
  double* stat_piv;       // [B,Hq,D+1] pivot row of the base-sample sums: w*V then w
  double* det_sums;       // [B,Hq,D+1] N_f then D_f
  int4* gat_meta;         // [B,Hq,2] what the gather kernel needs of a head: b, n_s, bits of m, entries to visit << 1 |
                          //   list (-1: an empty row); entries of the final sample's walk array
  float* gat_part;        // [B,Hq,gat_slots,D+1]  partials of the gather kernel, one per chunk
  int gat_slots;          // partial slots (chunks) per head: 32; 64 to 128 when at most 18 heads share the grid
  int stat_splits, stat_splits_base;   // statistics CTAs per head: deterministic rows, base-sample rows
  float* dense_part;      // [B,Hq,dense_splits,dense_rec(D)]
  int dense_splits;
  vattn_debug dbg;
};

// Optional device-side kernel time stamps (vattn_debug.kernel_ticks): thread 0 of every CTA folds
// %globaltimer into [k][0] = earliest start and [k][1] = latest end of kernel k.  Unlike events between the
// kernels this does not serialise the step: it shows the overlapped timeline of a real (graph-replayed) step.
__device__ __forceinline__ unsigned long long gtime_ns() { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
#define TICK_BEGIN(p, k) do { if ((p).dbg.kernel_ticks && threadIdx.x == 0) atomicMin((p).dbg.kernel_ticks + 2 * (k), gtime_ns()); } while (0)
#define TICK_END(p, k) do { if ((p).dbg.kernel_ticks && threadIdx.x == 0) atomicMax((p).dbg.kernel_ticks + 2 * (k) + 1, gtime_ns()); } while (0)
#define TICK_END_IF(p, k, cond) do { if ((p).dbg.kernel_ticks && (cond)) atomicMax((p).dbg.kernel_ticks + 2 * (k) + 1, gtime_ns()); } while (0)
// measurement builds (-DVATTN_PHASE_TICKS): stamps of phases inside the kernels, rows 8 + k of a larger tick buffer
#ifdef VATTN_PHASE_TICKS
#define DBGT(k) do { TICK_BEGIN(p, 8 + (k)); TICK_END(p, 8 + (k)); } while (0)
// per-head stamps: row 64 + 4 * bh + (k >> 1), column k & 1
#define DBGH(bh, k) do { if ((p).dbg.kernel_ticks && threadIdx.x == 0) (p).dbg.kernel_ticks[2 * (64 + 4 * (bh) + ((k) >> 1)) + ((k) & 1)] = gtime_ns(); } while (0)
#else
#define DBGT(k) do { } while (0)
#define DBGH(bh, k) do { } while (0)
#endif
// rows of kernel_ticks
#define VATTN_K_ZERO 0
#define VATTN_K_SCORE 1
#define VATTN_K_WALK 2
#define VATTN_K_SELECT 3
#define VATTN_K_STATS 4
#define VATTN_K_GATHER 5
#define VATTN_T_TOPK 6       // [0]: first selection CTA past its dependency wait, [1]: last CTA with I_t complete
#define VATTN_T_BUDGET 7     // [0]: first head whose statistics are complete, [1]: last head that knows its budget

// Programmatic dependent launch: a kernel launched with launch_pdl may start while its predecessor in the
// stream is still running; it must call pdl_wait() before touching anything the predecessor writes (the
// wait returns once the predecessor has completed and its writes are visible).  pdl_trigger() in the
// predecessor lets the dependent grid start launching early; the dependent still waits for completion.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, args...);
}

// ---------------------------------------------------------------------------------------------
// small device helpers
__device__ __forceinline__ unsigned ord_f32(float f) {          // order-preserving float -> uint
  unsigned u = __float_as_uint(f);
  return u ^ ((u >> 31) ? 0xFFFFFFFFu : 0x80000000u);
}
__device__ __forceinline__ float unord_f32(unsigned o) {
  unsigned u = (o & 0x80000000u) ? (o ^ 0x80000000u) : ~o;
  return __uint_as_float(u);
}
__device__ __forceinline__ unsigned long long ord_f64(double f) {
  unsigned long long u = (unsigned long long)__double_as_longlong(f);
  return u ^ ((u >> 63) ? 0xFFFFFFFFFFFFFFFFull : 0x8000000000000000ull);
}

struct bf16x8 { uint4 v; };

template <typename T> struct Elem;
template <> struct Elem<float> {
  static constexpr int EPL = 4;                                  // elements per 16-byte load
  __device__ static __forceinline__ void load(const float* p, float (&x)[4]) {
    float4 v = *reinterpret_cast<const float4*>(p);
    x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
  }
  __device__ static __forceinline__ float to_float(float v) { return v; }
  __device__ static __forceinline__ float from_float(float v) { return v; }
};
struct bf16_t { unsigned short bits; };
template <> struct Elem<bf16_t> {
  static constexpr int EPL = 8;
  __device__ static __forceinline__ void load(const bf16_t* p, float (&x)[8]) {
    uint4 v = *reinterpret_cast<const uint4*>(p);
    x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xFFFF0000u);
    x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xFFFF0000u);
    x[4] = __uint_as_float(v.z << 16); x[5] = __uint_as_float(v.z & 0xFFFF0000u);
    x[6] = __uint_as_float(v.w << 16); x[7] = __uint_as_float(v.w & 0xFFFF0000u);
  }
  __device__ static __forceinline__ float to_float(bf16_t v) { return __uint_as_float(((unsigned)v.bits) << 16); }
  __device__ static __forceinline__ bf16_t from_float(float f) {    // round to nearest even
    unsigned u = __float_as_uint(f);
    bf16_t r;
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) { r.bits = (unsigned short)((u >> 16) | 0x40); return r; }   // NaN
    u += 0x7FFFu + ((u >> 16) & 1u);
    r.bits = (unsigned short)(u >> 16);
    return r;
  }
};

// physical page of logical page `lp` of batch row b (bounds-checked; a bad entry raises a status bit)
// Diagnosis builds (-DVATTN_CHECK_SLOTS): a physical slot (page * 16 + token % 16) is checked before it becomes an
// address; a slot outside the cache is recorded (status bit, first offender's value and site) and replaced by slot 0.
#ifdef VATTN_CHECK_SLOTS
#define CHECK_SLOT(p, ph, site) do { if ((unsigned)((ph) >> 4) >= (unsigned)(p).num_blocks) { \
    atomicOr((p).status, VATTN_STATUS_BAD_BLOCK); \
    if ((p).dbg.paths) { (p).dbg.paths[0] = 0x40000000 | (site); (p).dbg.paths[1] = (ph); (p).dbg.paths[2] = blockIdx.x | (blockIdx.y << 12) | (blockIdx.z << 24); } \
    (ph) = 0; } } while (0)
#define CHECK_TOK(p, tok, site) do { if ((tok) >= (p).npad) { \
    atomicOr((p).status, VATTN_STATUS_BAD_BLOCK); \
    if ((p).dbg.paths) { (p).dbg.paths[0] = 0x40000000 | (site); (p).dbg.paths[1] = (tok); (p).dbg.paths[2] = blockIdx.x | (blockIdx.y << 12) | (blockIdx.z << 24); } \
    (tok) = -1; } } while (0)
#else
#define CHECK_SLOT(p, ph, site) do { } while (0)
#define CHECK_TOK(p, tok, site) do { } while (0)
#endif
__device__ __forceinline__ int page_of(const Prob& p, int b, int lp) {
  int pg = p.bt[(long long)b * p.max_blocks + lp];
  if ((unsigned)pg >= (unsigned)p.num_blocks) { atomicOr(p.status, VATTN_STATUS_BAD_BLOCK); pg = 0; }
  return pg;
}
template <typename T>
__device__ __forceinline__ const T* row_ptr(const Prob& p, const void* cache, int b, int g, int tok) {
  int pg = page_of(p, b, tok >> 4);
  return reinterpret_cast<const T*>(cache) + (long long)pg * p.sb + (long long)g * p.sh + (long long)(tok & 15) * p.st;
}
__device__ __forceinline__ int clamped_len(const Prob& p, int b) {
  int n = p.seq_lens[b];
  if (n < 0 || n > p.max_seq_len) { atomicOr(p.status, VATTN_STATUS_BAD_SEQLEN); n = n < 0 ? 0 : p.max_seq_len; }
  return n;
}

// Calls with several query tokens per sequence (a question, speculative tokens).  The cache already holds their
// K and V rows; query token t of Tq sees the first n - (Tq - 1 - t) tokens (causal).  Inside the kernels every
// (query token, head) pair is a head of its own: head index hv = g * G + t * G1 + i stands for query token t and
// real head g * G1 + i, so the heads that share KV head g stay contiguous (one pass over K serves all of them).
// q and out are [B, Tq, Hkv * G1, D] in memory.
__device__ __forceinline__ int head_tok(const Prob& p, int hv) { return (hv % p.G) / p.G1; }
__device__ __forceinline__ int head_real(const Prob& p, int hv) { return (hv / p.G) * p.G1 + (hv % p.G1); }
// element offset of head hv's row in q and out
__device__ __forceinline__ long long q_row(const Prob& p, int b, int hv) {
  if (p.Tq == 1) return ((long long)b * p.Hq + hv) * p.D;
  return (((long long)b * p.Tq + head_tok(p, hv)) * (p.Hkv * p.G1) + head_real(p, hv)) * p.D;
}
// tokens that head hv of batch row b sees
__device__ __forceinline__ int head_len(const Prob& p, int b, int hv) {
  const int n = clamped_len(p, b);
  return p.Tq == 1 ? n : max(0, n - (p.Tq - 1 - head_tok(p, hv)));
}

// Index-set geometry of one sequence (Algorithm 1 lines 1-5 with absolute sink/window counts):
// sink range [0,s0), window [l_start,n), middle M = [s0,l_start), kk = |I_t|, n_s = |M| - kk, b0.
struct Geo { int s0, l_start, kk, n_s, b0; };
__device__ __forceinline__ Geo head_geometry(const Prob& p, int n) {
  Geo g;
  g.s0 = min(p.sink, n);
  g.l_start = max(n - p.window, g.s0);
  const int mlen = g.l_start - g.s0;
  int kb = p.k;
  if (p.topk_frac > 0.f) kb = (int)floor((double)p.topk_frac * (double)n);
  g.kk = min(kb, mlen);
  g.n_s = mlen - g.kk;
  g.b0 = 0;
  if (g.n_s > 0) g.b0 = min(g.n_s, max(2, (int)floor((double)p.base_rate * (double)g.n_s)));
  return g;
}
#define VATTN_MAX_BATCH_BF16 1536     // batch rows a bf16 plan accepts (12 bytes of shared memory per row in k_score)

// Philox4x32-10 (Salmon et al., SC'11): counter (c0..c3), key (k0,k1)
__device__ __forceinline__ uint4 philox4x32_10(unsigned c0, unsigned c1, unsigned c2, unsigned c3,
                                               unsigned k0, unsigned k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const unsigned long long p0 = (unsigned long long)c0 * 0xD2511F53ull;      // one widening multiply each
    const unsigned long long p1 = (unsigned long long)c2 * 0xCD9E8D57ull;
    const unsigned hi0 = (unsigned)(p0 >> 32), lo0 = (unsigned)p0, hi1 = (unsigned)(p1 >> 32), lo1 = (unsigned)p1;
    unsigned n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  return make_uint4(c0, c1, c2, c3);
}

// ---------------------------------------------------------------------------------------------
// uniform-sample (Algorithm 1 line 7, Algorithm 2 line 1) = the first c residual tokens met when the middle range
// is walked in the order s0 + sigma(0), s0 + sigma(1), ...; sigma is a keyed permutation of [0, mlen): an 8-round
// alternating Feistel network on the smallest domain 2^w >= mlen (w >= 2) with cycle walking.  Round keys: the
// eight words of Philox4x32-10(key = seed, counter = (c, batch << 16 | head, layer, step << 1 | stream)), c = 0, 1.
__device__ __forceinline__ unsigned mix32(unsigned x, unsigned key) {
  unsigned v = (x ^ key) * 0x9E3779B1u;
  v ^= v >> 15; v *= 0x85EBCA77u;
  v ^= v >> 13; v *= 0xC2B2AE3Du;
  v ^= v >> 16;
  return v;
}
struct Walk { unsigned k[8]; int lw, rw; unsigned mlen; };
__device__ __forceinline__ Walk make_walk(const unsigned* keys, int mlen) {
  Walk w;
#pragma unroll
  for (int i = 0; i < 8; ++i) w.k[i] = keys[i];
  const int wbits = max(2, 32 - __clz(max(mlen - 1, 0)));
  w.lw = wbits >> 1; w.rw = wbits - w.lw; w.mlen = (unsigned)max(mlen, 1);
  return w;
}
// one pass of the network over the domain 2^(lw + rw) (cycle walking repeats it until the value is below mlen)
__device__ __forceinline__ unsigned walk_pass(const Walk& w, unsigned x) {
  const unsigned ml = (1u << w.lw) - 1u, mr = (1u << w.rw) - 1u;
  unsigned L = x >> w.rw, R = x & mr;
#pragma unroll
  for (int i = 0; i < 8; i += 2) {
    L ^= mix32(R, w.k[i]) & ml;
    R ^= mix32(L, w.k[i + 1]) & mr;
  }
  return (L << w.rw) | R;
}
__device__ __forceinline__ int walk_at(const Walk& w, int j) {
  unsigned x = (unsigned)j;
  do { x = walk_pass(w, x); } while (x >= w.mlen);
  return (int)x;
}
// sigma^-1: the walk position at which middle token t (relative to s0) is met
__device__ __forceinline__ int walk_inv(const Walk& w, int t) {
  const unsigned ml = (1u << w.lw) - 1u, mr = (1u << w.rw) - 1u;
  unsigned x = (unsigned)t;
  do {
    unsigned L = x >> w.rw, R = x & mr;
#pragma unroll
    for (int i = 6; i >= 0; i -= 2) {
      R ^= mix32(L, w.k[i + 1]) & mr;
      L ^= mix32(R, w.k[i]) & ml;
    }
    x = (L << w.rw) | R;
  } while (x >= w.mlen);
  return (int)x;
}
// Walk positions expected to hold the first `want` residual tokens, with a margin of four standard deviations
// (the selection kernel walks on if the margin was not enough).
__device__ __forceinline__ int walk_region(int want, int n_s, int mlen, int kk) {
  if (want <= 0 || n_s <= 0) return 0;
  if (want >= n_s) return mlen;
  const double miss = (double)want * (double)mlen / (double)n_s;
  const long long span = (long long)(miss + 4.0 * sqrt(miss * (double)kk / (double)mlen + 1.0) + 8.0);
  return (int)(span < (long long)mlen ? span : (long long)mlen);
}
// residual tokens of the final sample's walk that are listed ahead of the budget: eight base budgets (budgets beyond
// that make the final-sample kernel walk on), or the forced budget
__device__ __forceinline__ int dyn_listed_want(const Prob& p, int n_s, int b0) {
  if (n_s <= 0) return 0;
  return min(n_s, p.force_budget >= 0 ? p.force_budget : VATTN_WALK_B0S * b0);
}
// round keys of one (batch row, head, stream) into keys[0..8): two threads, one Philox call each.  The head word is
// the real query head (or the KV head with rng_head_is_kv); query token t of a call draws as decode step `step + t`
__device__ __forceinline__ void walk_keys(const Prob& p, int b, int hv, int stream, int half, unsigned* keys) {
  const int hrng = p.rng_head_is_kv ? hv / p.G : head_real(p, hv);
  const unsigned step = (unsigned)p.step + (unsigned)head_tok(p, hv);
  const uint4 w4 = philox4x32_10((unsigned)half, ((unsigned)b << 16) | (unsigned)hrng, (unsigned)p.layer,
                                 (step << 1) | (unsigned)stream, p.seed_lo, p.seed_hi);
  keys[half * 4 + 0] = w4.x; keys[half * 4 + 1] = w4.y; keys[half * 4 + 2] = w4.z; keys[half * 4 + 3] = w4.w;
}
// is middle token `tok` (fp32 score s) a member of I_t?  vt: the head's near-tie list (shared or global memory)
__device__ __forceinline__ bool in_topk(const HeadMeta& mt, const int* vt, const unsigned* bitmap, int tok, float s) {
  if (s > mt.hi) return true;
  if (!(s >= mt.lo)) return false;
  if (mt.band_mode) return (__ldcg(bitmap + (tok >> 5)) >> (tok & 31)) & 1u;
  for (int c = 0; c < mt.nbt; ++c) {
    const int e = vt[c];
    if ((e & 0x7FFFFFFF) == tok) return e < 0;
  }
  return false;
}

// ---------------------------------------------------------------------------------------------
// asynchronous bulk copies (global -> shared) completing on an mbarrier, and the bf16 tensor-core MMA
constexpr unsigned WAIT_SPINS = 1u << 20;      // polls of a bounded mbarrier wait
__device__ __forceinline__ unsigned smem_u32(const void* ptr) { return (unsigned)__cvta_generic_to_shared(ptr); }
__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, unsigned parity) {
  unsigned ok;
  asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
               : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// bounded wait: gives up after WAIT_SPINS polls and reports it
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, unsigned parity) {
  if (mbar_try_wait(bar, parity)) return true;
  for (unsigned it = 0; it < WAIT_SPINS; ++it) {
    __nanosleep(64);                      // leave the issue slots to the warps that have work
    if (mbar_try_wait(bar, parity)) return true;
  }
  return false;
}
// the same copy for data that is read once (the K stream of the score pass): its lines are the first to leave
// L2, so that what the step re-reads (scores, candidate lists, index lists) stays there
__device__ __forceinline__ unsigned long long l2_evict_first_policy() {
  unsigned long long pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_g2s_stream(void* dst, const void* src, unsigned bytes, unsigned long long* bar,
                                                unsigned long long policy) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy) : "memory");
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, unsigned bytes, unsigned long long* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3,
                                               unsigned b0, unsigned b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}


// The opt-in to more than 48 KB of dynamic shared memory (and the carve-out preference) is a property of a
// kernel in ONE device's context: it is made once per device ordinal (`have` = bytes already granted there).
constexpr int VATTN_MAXDEV = 64;
template <typename KernelT>
inline cudaError_t optin_smem(KernelT kern, size_t smem, size_t* have, bool prefer_max_carveout = false) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= VATTN_MAXDEV) return cudaErrorInvalidDevice;
  if (__atomic_load_n(&have[dev], __ATOMIC_ACQUIRE) >= smem + 1) return cudaSuccess;
  if (smem > 48 * 1024) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  if (prefer_max_carveout) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
  }
  __atomic_store_n(&have[dev], smem + 1, __ATOMIC_RELEASE);
  return cudaSuccess;
}

// HeadMeta through L2 (ld.cg): for kernels that read it before their stream predecessor has completed (after a
// flag) and therefore cannot count on the launch-boundary L1 invalidation.
static_assert(sizeof(HeadMeta) == 80, "HeadMeta is read as five 16-byte words");
__device__ __forceinline__ HeadMeta ld_meta(const HeadMeta* g) {
  union U { HeadMeta m; int4 v[5]; __device__ U() {} } u;
  const int4* src = reinterpret_cast<const int4*>(g);
  u.v[0] = __ldcg(src); u.v[1] = __ldcg(src + 1); u.v[2] = __ldcg(src + 2); u.v[3] = __ldcg(src + 3);
  u.v[4] = __ldcg(src + 4);
  return u.m;
}

// Bounded waits for a word that another kernel's CTA publishes with a release store (zero = not yet).  Relaxed polls
// (an acquire per poll would cost the SM an L1 invalidation each time, for every waiting CTA), one acquire fence
// at the end.  Returns the word, or zero when `spins` polls saw nothing: the caller then falls back to the
// grid-level dependency wait (or reports it); no wait in this library is unbounded.
__device__ __forceinline__ unsigned wait_word32(const unsigned* w, unsigned spins) {
  unsigned v = 0u;
  for (unsigned it = 0; it < spins; ++it) {
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(w) : "memory");
    if (v != 0u) break;
    __nanosleep(128);
  }
  asm volatile("fence.acq_rel.gpu;" ::: "memory");
  return v;
}
__device__ __forceinline__ unsigned long long wait_word64(const unsigned long long* w, unsigned spins) {
  unsigned long long v = 0ull;
  for (unsigned it = 0; it < spins; ++it) {
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(w) : "memory");
    if (v != 0ull) break;
    __nanosleep(128);
  }
  asm volatile("fence.acq_rel.gpu;" ::: "memory");
  return v;
}
constexpr unsigned VATTN_WORD_SPINS = 1u << 16;   // polls of a published word (about 10 ms) before the fallback

// launchers (one per translation unit)
cudaError_t launch_zero(unsigned* z, size_t bytes, bool pdl, bool late, unsigned long long* ticks, cudaStream_t s);
cudaError_t launch_score(const Prob& p, cudaStream_t s);
cudaError_t launch_walk(const Prob& p, cudaStream_t s);
cudaError_t launch_select(const Prob& p, cudaStream_t s);
cudaError_t launch_stats(const Prob& p, cudaStream_t s);
cudaError_t launch_gather(const Prob& p, cudaStream_t s);
cudaError_t launch_dense(const Prob& p, cudaStream_t s, int* launches);
int device_sm_count();                                   // SMs of the current device (cached per device)
