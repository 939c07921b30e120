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
    if (hl < p.G) Elem<T>::load(reinterpret_cast<const T*>(p.q) + ((long long)b * p.Hq + g * p.G + hl) * D + j * EPL, qv[hh]);
    else {
#pragma unroll
      for (int e = 0; e < EPL; ++e) qv[hh][e] = 0.f;
    }
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
    const bool tok_ok = (tok0 + (j >> 1) * RPI + r) < n;
    float sv[2], pm[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) { sv[e] = tok_ok ? p.scale * sacc[e] : -INFINITY; pm[e] = sv[e]; }
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
      pv[e] = __expf(sv[e] - m_new[2 * (j & 1) + e]);
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
  constexpr int NE = D + 2;
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
  if (tid == 0) is_last = (atomicAdd(&p.tickets[2 * p.B * p.Hq + b * p.Hq + blockIdx.y], 1u) == (unsigned)(S - 1));
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
    reinterpret_cast<T*>(p.out)[bh * D + e] = Elem<T>::from_float(n > 0 ? num / den : 0.f);
  }
}

}  // namespace

cudaError_t launch_dense(const Prob& p, cudaStream_t s, int* launches) {
  const int GC = (p.G + 3) / 4;
  dim3 grid(p.dense_splits, p.Hkv * GC, p.B), block(NT);
  if (p.dtype == VATTN_DTYPE_BF16) {
    if (p.D == 128) k_dense<bf16_t, 128><<<grid, block, 0, s>>>(p);
    else k_dense<bf16_t, 64><<<grid, block, 0, s>>>(p);
  } else {
    if (p.D == 128) k_dense<float, 128><<<grid, block, 0, s>>>(p);
    else k_dense<float, 64><<<grid, block, 0, s>>>(p);
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
      (s.dtype != VATTN_DTYPE_FP32 && s.dtype != VATTN_DTYPE_BF16) || s.num_q_heads / s.num_kv_heads > 64)
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
  int splits = (int)((4 * 148 + groups - 1) / groups);
  splits = splits < 1 ? 1 : (splits > 128 ? 128 : splits);
  while (splits > 1 && head_bytes + BH * splits * (D + 2) * sizeof(float) > VATTN_NOALLOC_SCRATCH_BYTES) --splits;
  if (head_bytes + BH * splits * (D + 2) * sizeof(float) > VATTN_NOALLOC_SCRATCH_BYTES)
    return VATTN_ERR_WORKSPACE;     // batch * heads too large for the built-in scratch

  void* base = nullptr;
  if (noalloc_scratch(&base) != cudaSuccess) return VATTN_ERR_CUDA;
  unsigned char* w = static_cast<unsigned char*>(base);
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  Prob p;
  memset(&p, 0, sizeof(p));
  p.B = s.batch; p.Hq = s.num_q_heads; p.Hkv = s.num_kv_heads; p.G = G; p.D = s.head_dim; p.dtype = s.dtype;
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
