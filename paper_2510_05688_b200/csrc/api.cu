// C ABI of libvattn: plan objects, argument checks, workspace layout and the launch sequence of one
// decode step.  Host code only; no device memory is allocated or freed here.
#include <math.h>
#include <new>
#include <string.h>
#include "vattn_internal.cuh"

struct vattn_plan {
  vattn_shape shape;
  vattn_params params;
  vattn_debug dbg;
  void* ws;
  size_t ws_bytes;
  bool status_ready;
  bool dense_ready;       // the dense kernel's tickets are known to be zero (its last CTAs put them back)
  int last_launches;
  // optional per-kernel timing (events are created on first use; no device memory involved)
  bool profiling;
  int stop_after;           // measurement aid: enqueue only the first stop_after kernels of a step (0 = all)
  cudaEvent_t* ev;          // [kProfCalls][kProfEvents]
  int prof_calls;           // calls recorded since the last read
  // derived
  int G, npad, nwords, dense_splits, stat_splits, stat_splits_base;
  size_t off_scores, off_zero, zero_bytes, off_status, off_bitmap, off_vtab, off_topk, off_base, off_walk, off_holes, off_wkeys, off_dyn, off_meta, off_stat,
      off_piv, off_det, off_gmeta, off_probe, off_gat, off_dense, total;
  int gat_slots;
  // vattn_decode_host: CUDA graphs of whole host steps, one per distinct argument set (see there)
  struct HostStep {
    bool used, pinned, mapped;
    void *q_dev, *bt_dev, *sl_dev, *out_dev;   // device addresses of the host buffers when they are mapped
    int hits, launches;
    cudaGraphExec_t exec;
    const void *q, *kc, *vc, *bt, *sl, *out, *staging, *stream;
    int sink, window, k;
    float eps, delta;
    uint64_t seed;
    unsigned long long gen;
  } host_steps[8];
  int host_next;
  bool inputs_just_staged;     // set around the step of a host call whose inputs a kernel has just copied in
  unsigned long long gen;      // bumped by every setter: steps captured under older settings are dropped
};

namespace {

constexpr int kProfCalls = 256;      // calls whose events are kept between two reads of the profile
constexpr int kProfEvents = VATTN_NUM_KERNELS + 1;

inline void prof_mark(vattn_plan* pl, int slot, cudaStream_t st) {
  if (pl->profiling && pl->ev && pl->prof_calls < kProfCalls) cudaEventRecord(pl->ev[pl->prof_calls * kProfEvents + slot], st);
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Upper-tail standard-normal quantile: the z with P(Z > z) = t, 0 < t < 1.  The Lemma's
// Phi^{-1}(1 - delta/2) is upper_quantile(delta/2).  Rational first guess (Abramowitz & Stegun 26.2.23),
// then Newton steps on erfc, which converge to the last bit or two of a double.
double upper_quantile(double t) {
  if (!(t > 0.0) || !(t < 1.0)) return NAN;
  const bool flip = t > 0.5;
  const double pp = flip ? 1.0 - t : t;
  const double u = sqrt(-2.0 * log(pp));
  double z = u - (2.515517 + u * (0.802853 + u * 0.010328)) / (1.0 + u * (1.432788 + u * (0.189269 + u * 0.001308)));
  for (int it = 0; it < 8; ++it) {
    const double f = 0.5 * erfc(z * M_SQRT1_2) - pp;
    const double pdf = exp(-0.5 * z * z) * 0.3989422804014326779;
    const double step = f / pdf;
    z += step;
    if (fabs(step) <= 1e-16 * fabs(z)) break;
  }
  return flip ? -z : z;
}

// (query token, head) pairs per batch row: the kernels treat each as a head of its own
inline int q_tokens(const vattn_shape& s) { return s.q_len > 1 ? s.q_len : 1; }
inline int heads_v(const vattn_shape& s) { return s.num_q_heads * q_tokens(s); }

void derive(vattn_plan* pl) {
  const vattn_shape& s = pl->shape;
  pl->G = heads_v(s) / s.num_kv_heads;
  pl->npad = (s.max_seq_len + 31) / 32 * 32;
  if (pl->npad == 0) pl->npad = 32;
  pl->nwords = pl->npad / 32;
  const int heads = s.batch * heads_v(s);
  const int GC = (pl->G + 3) / 4;
  const int groups = s.batch * s.num_kv_heads * GC;
  const int sp = (8 * device_sm_count() + groups - 1) / groups;
  pl->dense_splits = sp < 1 ? 1 : (sp > 128 ? 128 : sp);
  // statistics kernel (128-thread CTAs, 5 per SM): one wave for both kinds of CTA.  The base-sample rows are on
  // the step's critical path (they wait for the sample's list), the deterministic rows start earlier: three fifths
  // of the wave go to the former.  (When even four CTAs per kind and head overfill the wave the kernel is
  // throughput-bound: split freely.)
  {
    const int wave = (5 * device_sm_count()) / heads;
    if (wave < 8) {
      pl->stat_splits = pl->stat_splits_base = 4;
    } else {
      const int sb = (3 * wave + 2) / 5;
      pl->stat_splits_base = sb > VATTN_STAT_MAXS ? VATTN_STAT_MAXS : sb;
      const int sd = wave - pl->stat_splits_base;
      pl->stat_splits = sd < 4 ? 4 : (sd > VATTN_STAT_MAXS ? VATTN_STAT_MAXS : sd);
    }
  }
  const size_t BH = (size_t)heads, D = (size_t)s.head_dim;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  pl->off_scores = take(BH * pl->npad * sizeof(float));
  // cleared every step: running maxima [BH], max |K| [B*Hkv], tickets [5*BH], the score kernel's unit counter
  pl->zero_bytes = align_up((BH + (size_t)s.batch * s.num_kv_heads + 5 * BH + 4) * sizeof(unsigned), 8) + BH * 8;   // ... and the 64-bit words [BH]
  pl->off_zero = take(pl->zero_bytes);
  pl->off_status = take(sizeof(unsigned));
  pl->off_bitmap = take(BH * pl->nwords * sizeof(unsigned));
  pl->off_vtab = take(BH * VATTN_BANDCAP * sizeof(int));
  pl->off_topk = take(2 * BH * pl->npad * sizeof(int));     // token indices, then physical slots
  pl->off_base = take(2 * BH * pl->npad * sizeof(int));
  pl->off_walk = take(4 * BH * pl->npad * sizeof(int));     // first walk positions of both walks: tokens, physical slots
  pl->off_holes = take(2 * BH * VATTN_BANDCAP * sizeof(int));
  pl->off_wkeys = take(BH * 8 * sizeof(unsigned));
  pl->off_dyn = take(3 * BH * pl->npad * sizeof(int));      // tokens, physical slots, score bits
  pl->off_meta = take(BH * sizeof(HeadMeta));
  pl->off_stat = take(BH * 2 * VATTN_STAT_MAXS * (D + 3) * sizeof(double));
  pl->off_piv = take(BH * (D + 1) * sizeof(double));
  pl->off_det = take(BH * (D + 1) * sizeof(double));
  pl->off_gmeta = take(2 * BH * sizeof(int4));
  pl->off_probe = take(4 * sizeof(unsigned));
  // partial slots (chunks) per head of the gather kernel: 32, except that a handful of heads may use more of
  // the 8 CTAs per SM (64 to 128 chunks each when that many fit the grid at once)
  {
    const size_t fit = (size_t)(8 * device_sm_count()) / BH;
    const size_t flat = fit >= 2 * VATTN_GATHER_FLAT_SLOTS ? (fit > 128 ? 128 : fit) : VATTN_GATHER_FLAT_SLOTS;
    pl->gat_slots = BH <= VATTN_GATHER_FLAT_HEADS ? (int)flat : 32;   // per-head decomposition: up to 32 chunks
  }
  pl->off_gat = take(BH * (size_t)pl->gat_slots * (D + 1) * sizeof(float));
  pl->off_dense = take(BH * pl->dense_splits * dense_rec((int)D) * sizeof(float));
  pl->total = off;
}

int fill_prob(const vattn_plan* pl, Prob& p, const void* q, const void* kc, const void* vc, const int32_t* bt,
              const int32_t* sl, void* out) {
  const vattn_shape& s = pl->shape;
  const vattn_params& pr = pl->params;
  memset(&p, 0, sizeof(p));
  p.B = s.batch; p.Hq = heads_v(s); p.Hkv = s.num_kv_heads; p.G = pl->G; p.D = s.head_dim; p.dtype = s.dtype;
  p.Tq = q_tokens(s); p.G1 = s.num_q_heads / s.num_kv_heads;
  p.max_blocks = s.max_blocks_per_seq; p.num_blocks = s.num_blocks; p.max_seq_len = s.max_seq_len;
  p.npad = pl->npad; p.nwords = pl->nwords;
  if (s.kv_stride_block == 0 && s.kv_stride_head == 0 && s.kv_stride_token == 0) {
    p.st = s.head_dim; p.sh = (long long)s.block_size * s.head_dim; p.sb = (long long)s.num_kv_heads * p.sh;
  } else {
    p.sb = s.kv_stride_block; p.sh = s.kv_stride_head; p.st = s.kv_stride_token;
  }
  p.q = q; p.kc = kc; p.vc = vc; p.bt = bt; p.seq_lens = sl; p.out = out;
  p.topk_frac = pr.topk_frac;
  p.base_rate = pr.base_rate > 0.f ? pr.base_rate : 0.025f;
  p.scale = pr.scale != 0.f ? pr.scale : (float)(1.0 / sqrt((double)s.head_dim));
  p.mode = pr.mode; p.layer = pr.layer; p.step = pr.step; p.rng_head_is_kv = pr.rng_head_is_kv;
  p.gather_kv = pr.gather_mode == 1;
  p.force_budget = (pr.force_budget_on || pr.force_budget > 0) ? (pr.force_budget < 0 ? -1 : pr.force_budget) : -1;
  p.nested_base = pr.nested_base ? 1 : 0;
  unsigned char* w = static_cast<unsigned char*>(pl->ws);
  p.scores = reinterpret_cast<float*>(w + pl->off_scores);
  unsigned* z = reinterpret_cast<unsigned*>(w + pl->off_zero);
  const size_t BH = (size_t)s.batch * heads_v(s);
  p.m_ord = z; p.kabsmax = z + BH; p.tickets = z + BH + (size_t)s.batch * s.num_kv_heads;
  p.unit_ctr = p.tickets + 5 * BH;
  p.flags64 = reinterpret_cast<unsigned long long*>(w + pl->off_zero + pl->zero_bytes - BH * 8);
  p.status = reinterpret_cast<unsigned*>(w + pl->off_status);
  p.bitmap = reinterpret_cast<unsigned*>(w + pl->off_bitmap);
  p.vtab = reinterpret_cast<int*>(w + pl->off_vtab);
  p.topk_idx = reinterpret_cast<int*>(w + pl->off_topk);
  p.base_idx = reinterpret_cast<int*>(w + pl->off_base);
  p.walk_tok = reinterpret_cast<int*>(w + pl->off_walk);
  p.hole_pos = reinterpret_cast<int*>(w + pl->off_holes);
  p.wkeys = reinterpret_cast<unsigned*>(w + pl->off_wkeys);
  p.dyn_idx = reinterpret_cast<int*>(w + pl->off_dyn);
  p.meta = reinterpret_cast<HeadMeta*>(w + pl->off_meta);
  p.stat_part = reinterpret_cast<double*>(w + pl->off_stat);
  p.stat_piv = reinterpret_cast<double*>(w + pl->off_piv);
  p.det_sums = reinterpret_cast<double*>(w + pl->off_det);
  p.gat_meta = reinterpret_cast<int4*>(w + pl->off_gmeta);
  p.gat_part = reinterpret_cast<float*>(w + pl->off_gat);
  p.gat_slots = pl->gat_slots;
  p.dense_part = reinterpret_cast<float*>(w + pl->off_dense);
  p.dense_splits = pl->dense_splits;
  p.stat_splits = pl->stat_splits; p.stat_splits_base = pl->stat_splits_base;
  p.dbg = pl->dbg;
  return VATTN_OK;
}

inline bool misaligned(const void* ptr, size_t a) { return (reinterpret_cast<uintptr_t>(ptr) & (a - 1)) != 0; }

int check_common(const vattn_plan* pl, const void* q, const void* kc, const void* vc, const int32_t* bt,
                 const int32_t* sl, const void* out) {
  if (!pl || !q || !kc || !vc || !bt || !sl || !out) return VATTN_ERR_INVALID_ARG;
  if (misaligned(q, 16) || misaligned(kc, 16) || misaligned(vc, 16) || misaligned(out, 16) || misaligned(bt, 4) ||
      misaligned(sl, 4))
    return VATTN_ERR_INVALID_ARG;
  if (!pl->ws || pl->ws_bytes < pl->total) return VATTN_ERR_WORKSPACE;
  return VATTN_OK;
}

#define CU(x) do { if ((x) != cudaSuccess) return VATTN_ERR_CUDA; } while (0)

// clears the per-step counters: with a kernel for the sparse step (the score kernel overlaps it), with a
// memset node otherwise
int prepare_stream(vattn_plan* pl, const Prob& p, cudaStream_t st, bool with_kernel) {
  if (!pl->status_ready) {
    CU(cudaMemsetAsync(p.status, 0, sizeof(unsigned), st));
    pl->status_ready = true;
  }
  // The clearing kernel may run ahead of its stream predecessor only when that is this library's own input
  // staging kernel; a caller's kernel (a GEMM, RoPE, a KV append that writes what this step reads) is waited for.
  if (with_kernel) CU(launch_zero(p.m_ord, pl->zero_bytes, pl->inputs_just_staged, pl->inputs_just_staged, p.dbg.kernel_ticks, st));
  else if (!pl->dense_ready) {
    // the dense kernel only needs its tickets at zero, and the last CTA of every group puts its ticket back:
    // one memset after the workspace is bound, none afterwards
    CU(cudaMemsetAsync(p.m_ord, 0, pl->zero_bytes, st));
    pl->dense_ready = true;
  }
  return VATTN_OK;
}

}  // namespace

int device_sm_count() {
  static int cached[VATTN_MAXDEV];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= VATTN_MAXDEV) { cudaGetLastError(); return 148; }
  int n = __atomic_load_n(&cached[dev], __ATOMIC_ACQUIRE);
  if (n > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) { cudaGetLastError(); return 148; }
  __atomic_store_n(&cached[dev], n, __ATOMIC_RELEASE);
  return n;
}

extern "C" {

double vattn_normal_quantile(double x) { return upper_quantile(0.5 * x); }

int vattn_plan_create(const vattn_shape* shape, vattn_plan** out) {
  if (!shape || !out) return VATTN_ERR_INVALID_ARG;
  const vattn_shape& s = *shape;
  if (s.batch <= 0 || s.num_q_heads <= 0 || s.num_kv_heads <= 0 || s.max_blocks_per_seq <= 0 || s.num_blocks <= 0 ||
      s.max_seq_len < 0 || s.q_len < 0)
    return VATTN_ERR_INVALID_ARG;
  if (s.num_q_heads % s.num_kv_heads != 0) return VATTN_ERR_INVALID_ARG;
  if (s.batch > 65535 || s.num_q_heads > 65535) return VATTN_ERR_INVALID_ARG;
  // grid dimensions y and z hold (batch row, head) pairs and twice the batch
  if (s.q_len > 64) return VATTN_ERR_UNSUPPORTED;
  if (s.batch > 32767 || (long long)s.batch * heads_v(s) > 65535) return VATTN_ERR_UNSUPPORTED;
  // the bf16 score kernel keeps two per-row tables of the batch in shared memory beside its page ring
  if (s.dtype == VATTN_DTYPE_BF16 && s.batch > VATTN_MAX_BATCH_BF16) return VATTN_ERR_UNSUPPORTED;
  if (s.head_dim != 64 && s.head_dim != 128) return VATTN_ERR_UNSUPPORTED;
  if (s.block_size != VATTN_BLOCK) return VATTN_ERR_UNSUPPORTED;
  if (s.dtype != VATTN_DTYPE_FP32 && s.dtype != VATTN_DTYPE_BF16) return VATTN_ERR_UNSUPPORTED;
  if (heads_v(s) / s.num_kv_heads > 64) return VATTN_ERR_UNSUPPORTED;
  if (s.max_seq_len > VATTN_MAX_SEQ) return VATTN_ERR_UNSUPPORTED;
  if ((long long)s.max_seq_len > (long long)s.max_blocks_per_seq * s.block_size) return VATTN_ERR_INVALID_ARG;
  const bool custom = s.kv_stride_block || s.kv_stride_head || s.kv_stride_token;
  if (custom) {
    const int epl = s.dtype == VATTN_DTYPE_BF16 ? 8 : 4;
    if (s.kv_stride_block <= 0 || s.kv_stride_head <= 0 || s.kv_stride_token < s.head_dim) return VATTN_ERR_INVALID_ARG;
    if (s.kv_stride_block % epl || s.kv_stride_head % epl || s.kv_stride_token % epl) return VATTN_ERR_INVALID_ARG;
  }
  vattn_plan* pl = new (std::nothrow) vattn_plan();
  if (!pl) return VATTN_ERR_INVALID_ARG;
  memset(pl, 0, sizeof(*pl));
  pl->shape = s;
  pl->params.force_budget = -1;
  derive(pl);
  *out = pl;
  return VATTN_OK;
}

void vattn_plan_destroy(vattn_plan* plan) {
  if (!plan) return;
  for (auto& e : plan->host_steps)
    if (e.used && e.exec) cudaGraphExecDestroy(e.exec);
  if (plan->ev) {
    for (int i = 0; i < kProfCalls * kProfEvents; ++i) cudaEventDestroy(plan->ev[i]);
    delete[] plan->ev;
  }
  delete plan;
}

int vattn_set_stop_after(vattn_plan* plan, int kernels) {
  if (!plan || kernels < 0 || kernels > VATTN_NUM_KERNELS) return VATTN_ERR_INVALID_ARG;
  plan->stop_after = kernels;
  plan->gen++;
  return VATTN_OK;
}

int vattn_set_profiling(vattn_plan* plan, int enable) {
  if (!plan) return VATTN_ERR_INVALID_ARG;
  if (enable && !plan->ev) {
    plan->ev = new (std::nothrow) cudaEvent_t[kProfCalls * kProfEvents];
    if (!plan->ev) return VATTN_ERR_INVALID_ARG;
    for (int i = 0; i < kProfCalls * kProfEvents; ++i)
      if (cudaEventCreate(&plan->ev[i]) != cudaSuccess) return VATTN_ERR_CUDA;
  }
  plan->profiling = enable != 0;
  plan->gen++;
  plan->prof_calls = 0;
  return VATTN_OK;
}

int vattn_read_profile(vattn_plan* plan, float* ms_sum, int* calls) {
  if (!plan || !ms_sum || !calls) return VATTN_ERR_INVALID_ARG;
  for (int k = 0; k < VATTN_NUM_KERNELS; ++k) ms_sum[k] = 0.f;
  *calls = plan->prof_calls;
  if (!plan->ev || plan->prof_calls == 0) return VATTN_OK;
  CU(cudaEventSynchronize(plan->ev[(plan->prof_calls - 1) * kProfEvents + VATTN_NUM_KERNELS]));
  for (int c = 0; c < plan->prof_calls; ++c)
    for (int k = 0; k < VATTN_NUM_KERNELS; ++k) {
      float ms = 0.f;
      CU(cudaEventElapsedTime(&ms, plan->ev[c * kProfEvents + k], plan->ev[c * kProfEvents + k + 1]));
      ms_sum[k] += ms;
    }
  plan->prof_calls = 0;
  return VATTN_OK;
}

size_t vattn_workspace_bytes(const vattn_plan* plan) { return plan ? plan->total : 0; }

int vattn_set_workspace(vattn_plan* plan, void* dev_ptr, size_t bytes) {
  if (!plan) return VATTN_ERR_INVALID_ARG;
  if (!dev_ptr || misaligned(dev_ptr, 256) || bytes < plan->total) return VATTN_ERR_WORKSPACE;
  plan->ws = dev_ptr;
  plan->ws_bytes = bytes;
  plan->status_ready = false;
  plan->dense_ready = false;
  plan->gen++;
  return VATTN_OK;
}

int vattn_set_params(vattn_plan* plan, const vattn_params* params) {
  if (!plan) return VATTN_ERR_INVALID_ARG;
  plan->gen++;
  if (!params) { memset(&plan->params, 0, sizeof(plan->params)); plan->params.force_budget = -1; return VATTN_OK; }
  const vattn_params& p = *params;
  if (p.base_rate < 0.f || p.base_rate > 1.f || p.topk_frac < 0.f || p.topk_frac > 1.f) return VATTN_ERR_INVALID_ARG;
  if (p.mode < 0 || p.mode > 2 || p.step < 0 || !(p.scale == p.scale) || isinf(p.scale)) return VATTN_ERR_INVALID_ARG;
  if (p.gather_mode < 0 || p.gather_mode > 1 || p.nested_base < 0 || p.nested_base > 1) return VATTN_ERR_INVALID_ARG;
  plan->params = p;
  return VATTN_OK;
}

int vattn_set_debug(vattn_plan* plan, const vattn_debug* debug) {
  if (!plan) return VATTN_ERR_INVALID_ARG;
  if (debug) plan->dbg = *debug; else memset(&plan->dbg, 0, sizeof(plan->dbg));
  plan->gen++;
  return VATTN_OK;
}

int vattn_decode(vattn_plan* plan, const void* q, const void* k_cache, const void* v_cache,
                 const int32_t* block_table, const int32_t* seq_lens, int sink, int window, int k, float eps,
                 float delta, uint64_t seed, void* out, void* stream) {
  int rc = check_common(plan, q, k_cache, v_cache, block_table, seq_lens, out);
  if (rc != VATTN_OK) return rc;
  if (!(eps > 0.f && eps < 1.f) || !(delta > 0.f && delta < 1.f) || sink < 0 || window < 0 || k < 0)
    return VATTN_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  Prob p;
  fill_prob(plan, p, q, k_cache, v_cache, block_table, seq_lens, out);
  p.sink = sink; p.window = window; p.k = k;
  {
    // statistics kernel: never more CTAs than rows warrant (about 64 deterministic, 48 base-sample rows each)
    const double msl = (double)plan->shape.max_seq_len;
    double kmax = plan->params.topk_frac > 0.f ? floor((double)plan->params.topk_frac * msl) : (double)k;
    double rows = (double)sink + (double)window + kmax;
    if (rows > msl) rows = msl;
    int want = (int)((rows + 127.0) / 128.0) * 2;
    if (want < 1) want = 1;
    if (want < p.stat_splits) p.stat_splits = want;
    const double brows = (double)p.base_rate * msl;
    want = (int)((brows + 95.0) / 96.0) * 2;
    if (want < 1) want = 1;
    if (want < p.stat_splits_base) p.stat_splits_base = want;
  }
  p.seed_lo = (unsigned)(seed & 0xFFFFFFFFull); p.seed_hi = (unsigned)(seed >> 32);
  p.eps = (double)eps; p.delta = (double)delta;
  p.z_delta = upper_quantile(0.5 * p.delta);
  for (int j = 1; j <= 15; ++j) {
    p.z1[j - 1] = upper_quantile(0.5 * (p.delta * j / 16.0));
    p.z2[j - 1] = upper_quantile(0.5 * (p.delta * (16 - j) / 16.0));
  }
  plan->last_launches = 0;
  rc = prepare_stream(plan, p, st, true);
  if (rc != VATTN_OK) return rc;
  plan->last_launches++;                      // the counter-clearing kernel
  prof_mark(plan, 0, st);
  // score pass (walk tokens beside it) -> selection and sample lists (one CTA per head) -> deterministic and
  // base-sample rows (started per head by flags of the selection kernel), budget by the last CTA of a head -> final
  // sample, combination.  Every kernel is launched with programmatic dependent launch: its prologue
  // runs while its predecessor drains.
  CU(launch_score(p, st));            plan->last_launches++;
  prof_mark(plan, 1, st);
  if (plan->stop_after == 1) return VATTN_OK;
  if (p.dbg.scores)
    CU(cudaMemcpy2DAsync(p.dbg.scores, sizeof(float) * (size_t)p.max_seq_len, p.scores, sizeof(float) * (size_t)p.npad,
                         sizeof(float) * (size_t)p.max_seq_len, (size_t)p.B * p.Hq, cudaMemcpyDeviceToDevice, st));
  CU(launch_walk(p, st));             plan->last_launches++;
  prof_mark(plan, 2, st);
  if (plan->stop_after == 2) return VATTN_OK;
  CU(launch_select(p, st));           plan->last_launches++;
  prof_mark(plan, 3, st);
  if (plan->stop_after == 3) return VATTN_OK;
  CU(launch_stats(p, st));            plan->last_launches++;
  prof_mark(plan, 4, st);
  if (plan->stop_after == 4) return VATTN_OK;
  CU(launch_gather(p, st));           plan->last_launches++;
  prof_mark(plan, 5, st);
  if (plan->profiling && plan->prof_calls < kProfCalls) plan->prof_calls++;
  return VATTN_OK;
}

int vattn_dense_decode(vattn_plan* plan, const void* q, const void* k_cache, const void* v_cache,
                       const int32_t* block_table, const int32_t* seq_lens, void* out, void* stream) {
  int rc = check_common(plan, q, k_cache, v_cache, block_table, seq_lens, out);
  if (rc != VATTN_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  Prob p;
  fill_prob(plan, p, q, k_cache, v_cache, block_table, seq_lens, out);
  plan->last_launches = 0;
  rc = prepare_stream(plan, p, st, false);
  if (rc != VATTN_OK) return rc;
  int launches = 0;
  CU(launch_dense(p, st, &launches));
  plan->last_launches = launches;
  return VATTN_OK;
}

size_t vattn_host_staging_bytes(const vattn_plan* plan) {
  if (!plan) return 0;
  const vattn_shape& s = plan->shape;
  const size_t es = s.dtype == VATTN_DTYPE_BF16 ? 2 : 4;
  const size_t qb = align_up((size_t)s.batch * heads_v(s) * s.head_dim * es, 256);
  return 2 * qb + align_up((size_t)s.batch * s.max_blocks_per_seq * 4, 256) + align_up((size_t)s.batch * 4, 256);
}

// Host buffers that are page-locked and mapped are read and written by kernels directly: one small kernel
// copies q, block_table and seq_lens into the staging buffer (three DMA copies of a few KB cost about 6 us
// each; this costs one PCIe round trip), and the step writes `out` straight into the host buffer.
__global__ void __launch_bounds__(256) k_stage_in(unsigned* dst0, const unsigned* src0, int n0, unsigned* dst1,
                                                  const unsigned* src1, int n1, unsigned* dst2, const unsigned* src2, int n2) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x, nt = gridDim.x * blockDim.x;
  for (int i = t; i < n0; i += nt) dst0[i] = src0[i];
  for (int i = t; i < n1; i += nt) dst1[i] = src1[i];
  for (int i = t; i < n2; i += nt) dst2[i] = src2[i];
}

// copies in, step, copy out: the stream work of one host step (no synchronisation)
static int enqueue_host_step(vattn_plan* plan, const void* q_host, const void* k_cache, const void* v_cache,
                             const int32_t* block_table_host, const int32_t* seq_lens_host, int sink, int window, int k,
                             float eps, float delta, uint64_t seed, void* out_host, void* staging, cudaStream_t st,
                             const vattn_plan::HostStep* mapped) {
  const vattn_shape& s = plan->shape;
  const size_t es = s.dtype == VATTN_DTYPE_BF16 ? 2 : 4;
  const size_t qbytes = (size_t)s.batch * heads_v(s) * s.head_dim * es, qb = align_up(qbytes, 256);
  const size_t btbytes = (size_t)s.batch * s.max_blocks_per_seq * 4, slbytes = (size_t)s.batch * 4;
  unsigned char* d = static_cast<unsigned char*>(staging);
  void* dq = d; void* dout = d + qb; int32_t* dbt = reinterpret_cast<int32_t*>(d + 2 * qb);
  int32_t* dsl = reinterpret_cast<int32_t*>(d + 2 * qb + align_up(btbytes, 256));
  if (mapped) {
    const int words = (int)((qbytes + btbytes + slbytes) / 4);
    int grid = (words + 255) / 256;                 // one word per thread: a single PCIe round trip
    if (grid > 296) grid = 296;
    if (grid < 1) grid = 1;
    k_stage_in<<<grid, 256, 0, st>>>(static_cast<unsigned*>(dq), static_cast<const unsigned*>(mapped->q_dev), (int)(qbytes / 4),
                                     reinterpret_cast<unsigned*>(dbt), static_cast<const unsigned*>(mapped->bt_dev),
                                     (int)(btbytes / 4), reinterpret_cast<unsigned*>(dsl),
                                     static_cast<const unsigned*>(mapped->sl_dev), (int)(slbytes / 4));
    CU(cudaGetLastError());
    plan->inputs_just_staged = true;
    const int rc = vattn_decode(plan, dq, k_cache, v_cache, dbt, dsl, sink, window, k, eps, delta, seed, mapped->out_dev, st);
    plan->inputs_just_staged = false;
    if (rc == VATTN_OK) plan->last_launches++;
    return rc;
  }
  CU(cudaMemcpyAsync(dq, q_host, qbytes, cudaMemcpyHostToDevice, st));
  CU(cudaMemcpyAsync(dbt, block_table_host, btbytes, cudaMemcpyHostToDevice, st));
  CU(cudaMemcpyAsync(dsl, seq_lens_host, slbytes, cudaMemcpyHostToDevice, st));
  int rc = vattn_decode(plan, dq, k_cache, v_cache, dbt, dsl, sink, window, k, eps, delta, seed, dout, st);
  if (rc != VATTN_OK) return rc;
  CU(cudaMemcpyAsync(out_host, dout, qbytes, cudaMemcpyDeviceToHost, st));
  return VATTN_OK;
}

static bool is_pinned_host(const void* ptr) {
  cudaPointerAttributes a;
  if (cudaPointerGetAttributes(&a, ptr) != cudaSuccess) { cudaGetLastError(); return false; }
  return a.type == cudaMemoryTypeHost;
}

static void* mapped_device_pointer(const void* host) {
  void* dev = nullptr;
  if (cudaHostGetDevicePointer(&dev, const_cast<void*>(host), 0) != cudaSuccess) { cudaGetLastError(); return nullptr; }
  return dev;
}

int vattn_decode_host(vattn_plan* plan, const void* q_host, const void* k_cache, const void* v_cache,
                      const int32_t* block_table_host, const int32_t* seq_lens_host, int sink, int window, int k,
                      float eps, float delta, uint64_t seed, void* out_host, void* staging, void* stream) {
  if (!plan || !q_host || !block_table_host || !seq_lens_host || !out_host || !staging || misaligned(staging, 256))
    return VATTN_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // A caller that repeats a step with the same buffers (a decode loop) gets it as one CUDA graph from the
  // third call on: the second call with an argument set records it, later ones replay it.  Only with
  // page-locked host buffers, outside any capture of the caller, and with no introspection switched on.
  vattn_plan::HostStep* e = nullptr;
  const vattn_debug& dg = plan->dbg;
  const bool plain_only = plan->profiling || plan->stop_after != 0 || dg.kernel_ticks || dg.topk_idx || dg.topk_cnt ||
                          dg.base_idx || dg.base_cnt || dg.dyn_idx || dg.dyn_cnt || dg.budgets || dg.stats || dg.scores ||
                          dg.paths;
  if (!plain_only) {
    for (auto& c : plan->host_steps)
      if (c.used && c.gen == plan->gen && c.q == q_host && c.kc == k_cache && c.vc == v_cache && c.bt == block_table_host &&
          c.sl == seq_lens_host && c.out == out_host && c.staging == staging && c.stream == stream && c.sink == sink &&
          c.window == window && c.k == k && c.eps == eps && c.delta == delta && c.seed == seed) { e = &c; break; }
    if (!e) {
      e = &plan->host_steps[plan->host_next];
      plan->host_next = (plan->host_next + 1) % 8;
      if (e->used && e->exec) cudaGraphExecDestroy(e->exec);
      *e = vattn_plan::HostStep{};
      e->used = true; e->gen = plan->gen;
      e->q = q_host; e->kc = k_cache; e->vc = v_cache; e->bt = block_table_host; e->sl = seq_lens_host; e->out = out_host;
      e->staging = staging; e->stream = stream; e->sink = sink; e->window = window; e->k = k; e->eps = eps; e->delta = delta;
      e->seed = seed;
      e->pinned = is_pinned_host(q_host) && is_pinned_host(block_table_host) && is_pinned_host(seq_lens_host) &&
                  is_pinned_host(out_host);
      if (e->pinned) {
        e->q_dev = mapped_device_pointer(q_host);
        e->bt_dev = mapped_device_pointer(block_table_host);
        e->sl_dev = mapped_device_pointer(seq_lens_host);
        e->out_dev = mapped_device_pointer(out_host);
        e->mapped = e->q_dev && e->bt_dev && e->sl_dev && e->out_dev && !misaligned(e->out_dev, 16) && !misaligned(e->q_dev, 4);
      }
    }
    if (e->exec) {
      CU(cudaGraphLaunch(e->exec, st));
      CU(cudaStreamSynchronize(st));
      plan->last_launches = e->launches;
      return VATTN_OK;
    }
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    const bool capturable_stream = st != nullptr && st != cudaStreamLegacy && st != cudaStreamPerThread;   // not the default streams
    if (e->pinned && e->hits >= 1 && capturable_stream && cudaStreamIsCapturing(st, &cs) == cudaSuccess &&
        cs == cudaStreamCaptureStatusNone) {
      cudaGraph_t graph = nullptr;
      if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) != cudaSuccess) { cudaGetLastError(); e->pinned = false; goto plain; }
      const int rc = enqueue_host_step(plan, q_host, k_cache, v_cache, block_table_host, seq_lens_host, sink, window, k, eps,
                                       delta, seed, out_host, staging, st, e->mapped ? e : nullptr);
      const cudaError_t ce = cudaStreamEndCapture(st, &graph);
      if (rc != VATTN_OK || ce != cudaSuccess || !graph) {
        if (graph) cudaGraphDestroy(graph);
        cudaGetLastError();
        e->pinned = false;                              // do not try again with this argument set
        if (rc != VATTN_OK) return rc;
      } else {
        cudaGraphExec_t exec = nullptr;
        const cudaError_t ie = cudaGraphInstantiate(&exec, graph, 0);
        cudaGraphDestroy(graph);
        if (ie == cudaSuccess) {
          e->exec = exec;
          e->launches = plan->last_launches;
          CU(cudaGraphLaunch(e->exec, st));
          CU(cudaStreamSynchronize(st));
          return VATTN_OK;
        }
        cudaGetLastError();
        e->pinned = false;
      }
    }
  plain:
    e->hits++;
  }
  {
    const int rc = enqueue_host_step(plan, q_host, k_cache, v_cache, block_table_host, seq_lens_host, sink, window, k, eps,
                                     delta, seed, out_host, staging, st, (e && e->mapped) ? e : nullptr);
    if (rc != VATTN_OK) return rc;
    CU(cudaStreamSynchronize(st));
  }
  return VATTN_OK;
}

int vattn_last_status(vattn_plan* plan, void* stream, uint32_t* bits) {
  if (!plan || !bits) return VATTN_ERR_INVALID_ARG;
  if (!plan->ws) return VATTN_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  unsigned* dev = reinterpret_cast<unsigned*>(static_cast<unsigned char*>(plan->ws) + plan->off_status);
  if (!plan->status_ready) { *bits = 0; return VATTN_OK; }
  CU(cudaMemcpyAsync(bits, dev, sizeof(unsigned), cudaMemcpyDeviceToHost, st));
  CU(cudaMemsetAsync(dev, 0, sizeof(unsigned), st));
  CU(cudaStreamSynchronize(st));
  return VATTN_OK;
}

// ---------------------------------------------------------------------------------------------
// The bounded wait on its own: a kernel polls a word of the workspace that nothing publishes, with the given poll
// limit, and reports how the wait ended.  No other kernel is involved: what the caller sees is what a CTA of the
// step sees when its producer never publishes (it then falls back to the grid-level dependency wait).
__global__ void k_probe_wait(const unsigned* word, unsigned spins, unsigned* result) {
  if (threadIdx.x == 0) {
    const unsigned long long t0 = gtime_ns();
    const unsigned v = wait_word32(word, spins);
    result[0] = v == 0u ? 1u : 0u;                     // 1: the wait ran out
    result[1] = (unsigned)((gtime_ns() - t0) / 1000ull);      // microseconds spent waiting
  }
}

int vattn_probe_bounded_wait(vattn_plan* plan, uint32_t spins, uint32_t* ran_out, uint32_t* waited_us, void* stream) {
  if (!plan || !ran_out || !waited_us || spins == 0 || spins > (1u << 20)) return VATTN_ERR_INVALID_ARG;
  if (!plan->ws) return VATTN_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  unsigned* dev = reinterpret_cast<unsigned*>(static_cast<unsigned char*>(plan->ws) + plan->off_probe);
  CU(cudaMemsetAsync(dev, 0, 4 * sizeof(unsigned), st));
  k_probe_wait<<<1, 32, 0, st>>>(dev, spins, dev + 2);
  CU(cudaGetLastError());
  unsigned host[2] = {0u, 0u};
  CU(cudaMemcpyAsync(host, dev + 2, 2 * sizeof(unsigned), cudaMemcpyDeviceToHost, st));
  CU(cudaStreamSynchronize(st));
  *ran_out = host[0]; *waited_us = host[1];
  return VATTN_OK;
}

int vattn_last_launch_count(const vattn_plan* plan) { return plan ? plan->last_launches : 0; }

const char* vattn_strerror(int code) {
  switch (code) {
    case VATTN_OK: return "ok";
    case VATTN_ERR_INVALID_ARG: return "invalid argument";
    case VATTN_ERR_UNSUPPORTED: return "unsupported shape or element type";
    case VATTN_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case VATTN_ERR_CUDA: return "CUDA runtime error";
    default: return "unknown error";
  }
}

}  // extern "C"
