// Sampling-candidate pre-filter (uniform-sample of Algorithm 1 line 7 and Algorithm 2 line 1, first half).
//
// "Draw c residual tokens uniformly without replacement" is implemented as "the c smallest Philox4x32-10
// keys of the residual".  The keys depend on (seed, layer, step, batch row, head, token, stream) only, not
// on K or on the scores, so they are generated here, concurrently with the score kernel (which is bound by
// HBM and leaves the integer pipes idle): for every (token, query head) of the middle range and both
// streams, a token whose key is below the stream's bound is appended to that (stream, head)'s candidate
// list.  Stream 1 keeps a quarter of the tokens; stream 0 keeps b0 + 6 sqrt(b0) + 16 expected tokens.  The
// lists come out in no particular order; k_presort sorts them.
//
// One CTA = 2048 consecutive tokens of one head: hits are compacted with warp ballots into two staged
// lists in shared memory, then appended to the global lists with one atomic per list.  A staged list that
// overflows (it holds twice the expected quarter) poisons the global count, which sends the consumers of
// that list to their full-context path.
#include "vattn_internal.cuh"

namespace {

constexpr int CT = 256;            // threads
constexpr int CTILE = 2048;        // tokens per CTA
constexpr int CCAP = 1024;         // staged entries per stream

__global__ void __launch_bounds__(CT, 4) k_cand(const Prob p) {
  __shared__ uint2 lst[2][CCAP];
  __shared__ unsigned cnt[2], gbase[2];
  pdl_trigger();
  TICK_BEGIN(p, VATTN_K_CAND);
  const int tid = threadIdx.x, lane = tid & 31;
  const int b = blockIdx.z, h = blockIdx.y, tile0 = blockIdx.x * CTILE;
  const int bh = b * p.Hq + h;
  const int n = clamped_len(p, b);
  const Geo geo = head_geometry(p, n);
  const int lo = max(tile0, geo.s0), hi = min(tile0 + CTILE, geo.l_start);
  const bool work = geo.n_s > 0 && lo < hi;                   // uniform over the CTA
  if (work) {
    const unsigned bound0 = cand0_bound(geo);
    if (tid < 2) cnt[tid] = 0u;
    __syncthreads();
    const int hrng = p.rng_head_is_kv ? h / p.G : h;
    const unsigned c1 = ((unsigned)b << 16) | (unsigned)hrng;
    const unsigned lt = (1u << lane) - 1u;
    // the CTA's (quad, stream) Philox calls of a thread are independent chains: all of them first (the
    // integer-multiply latency of one hides behind the others), then the compaction
    constexpr int QPT = CTILE / 4 / CT;                         // quads per thread
    unsigned key[QPT][2][4];
    bool active[QPT];
#pragma unroll
    for (int qi = 0; qi < QPT; ++qi) {
      const int t0 = tile0 + (tid + qi * CT) * 4;
      active[qi] = t0 < hi && t0 + 4 > lo;
#pragma unroll
      for (int stream = 0; stream < 2; ++stream) {
        const uint4 r = philox4x32_10((unsigned)(t0 >> 2), c1, (unsigned)p.layer, ((unsigned)p.step << 1) | (unsigned)stream,
                                      p.seed_lo, p.seed_hi);
        key[qi][stream][0] = r.x; key[qi][stream][1] = r.y; key[qi][stream][2] = r.z; key[qi][stream][3] = r.w;
      }
    }
#pragma unroll
    for (int qi = 0; qi < QPT; ++qi) {
      const int t0 = tile0 + (tid + qi * CT) * 4;
#pragma unroll
      for (int stream = 0; stream < 2; ++stream) {
        const unsigned bound = stream ? VATTN_CAND1_BOUND : bound0;
        if (bound == 0u) continue;                             // uniform
        unsigned bal[4], total = 0u;
        bool hit[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int tok = t0 + e;
          hit[e] = active[qi] && key[qi][stream][e] < bound && tok >= lo && tok < hi;
          bal[e] = __ballot_sync(0xFFFFFFFFu, hit[e]);
          total += __popc(bal[e]);
        }
        unsigned base = 0u;
        if (lane == 0 && total) base = atomicAdd(&cnt[stream], total);
        base = __shfl_sync(0xFFFFFFFFu, base, 0);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const unsigned pos = base + __popc(bal[e] & lt);
          if (hit[e] && pos < (unsigned)CCAP) lst[stream][pos] = make_uint2(key[qi][stream][e], (unsigned)(t0 + e));
          base += __popc(bal[e]);
        }
      }
    }
    __syncthreads();
    if (tid < 2) {
      const unsigned raw = cnt[tid];
      unsigned gb = 0u;
      if (raw) {
        unsigned* gcnt = p.cand_cnt + (long long)tid * p.B * p.Hq + bh;
        if (raw > (unsigned)CCAP) { atomicOr(gcnt, 0x80000000u); gb = (unsigned)p.cand_cap; }   // incomplete list
        else gb = atomicAdd(gcnt, raw);
      }
      gbase[tid] = gb;
    }
    __syncthreads();
#pragma unroll
    for (int stream = 0; stream < 2; ++stream) {
      const unsigned raw = cnt[stream];
      const unsigned c = raw < (unsigned)CCAP ? raw : (unsigned)CCAP;
      const unsigned gb = gbase[stream];
      uint2* dst = p.cand + ((long long)stream * p.B * p.Hq + bh) * p.cand_cap;
      for (unsigned j = tid; j < c; j += CT)
        if (gb + j < (unsigned)p.cand_cap) dst[gb + j] = lst[stream][j];
    }
  }
  // This grid does not wait for the score kernel before it, so one of its CTAs does at the end: "this grid
  // has completed" then implies "the score kernel has completed" for the kernels behind it.
  TICK_END(p, VATTN_K_CAND);
  if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0) pdl_wait();
}

}  // namespace

cudaError_t launch_cand(const Prob& p, cudaStream_t s) {
  const int tiles = (p.max_seq_len + CTILE - 1) / CTILE;
  // this kernel shares SMs with the score kernel: ask for the same (largest) shared-memory carve-out
  static bool attr_done = false;
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(k_cand, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    attr_done = true;
  }
  return launch_pdl(k_cand, dim3(tiles < 1 ? 1 : tiles, p.Hq, p.B), dim3(CT), 0, s, p);
}
