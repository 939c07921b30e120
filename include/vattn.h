/*
 * libvattn — verified sparse-attention decode step (vAttention, arXiv 2510.05688) for sm_100a.
 *
 * C ABI.  All tensor arguments are DEVICE pointers unless a comment says "host".  The caller owns
 * every tensor and the workspace; the library never allocates or frees device memory and
 * vattn_decode / vattn_dense_decode never synchronise (they only enqueue work on `stream`).
 * A plan holds host-side descriptors only.  One plan must not be used from two streams at once
 * (its workspace is shared state).
 *
 * Tensor layouts
 *   q, out        [batch, num_q_heads, head_dim], contiguous, 16-byte aligned, element type `dtype`
 *                 ([batch, q_len, num_q_heads, head_dim] for a plan with vattn_shape.q_len > 1)
 *   k_cache,
 *   v_cache       paged: element (block p, kv head g, token t, dim j) at
 *                 p*kv_stride_block + g*kv_stride_head + t*kv_stride_token + j   (element units);
 *                 default "HND" = [num_blocks, num_kv_heads, block_size, head_dim] contiguous.
 *                 Rows must be 16-byte aligned (strides multiples of 8 bf16 / 4 fp32 elements).
 *   block_table   int32 [batch, max_blocks_per_seq]: logical page -> physical page
 *   seq_lens      int32 [batch]: tokens n_b currently in each sequence (0 <= n_b <= max_seq_len)
 * Query head h reads KV head h / (num_q_heads / num_kv_heads); every query head has its own
 * index sets, budget and sample (the paper states its guarantee per attention head: Fig. 3 caption).
 *
 * Return codes: 0 OK; negative = error, nothing was enqueued.
 */
#ifndef VATTN_H_
#define VATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define VATTN_OK               0
#define VATTN_ERR_INVALID_ARG -1   /* null / misaligned pointer, eps or delta outside (0,1), negative sink/window/k, Hq % Hkv != 0 */
#define VATTN_ERR_UNSUPPORTED -2   /* head_dim not in {64,128}, block_size != 16, unknown dtype, GQA ratio > 64 */
#define VATTN_ERR_WORKSPACE   -3   /* workspace missing, misaligned or too small */
#define VATTN_ERR_CUDA        -4   /* a CUDA runtime call or kernel launch failed */

#define VATTN_DTYPE_FP32 0
#define VATTN_DTYPE_BF16 1

/* bits of the device status word (vattn_last_status) */
#define VATTN_STATUS_BAD_BLOCK      1u   /* a block_table entry was outside [0, num_blocks): page treated as page 0 */
#define VATTN_STATUS_BAD_SEQLEN     2u   /* a seq_len was outside [0, max_seq_len]: clamped */
#define VATTN_STATUS_BAND_OVERFLOW  4u   /* more near-tie top-k candidates than the fast list holds: exact slow path ran */
#define VATTN_STATUS_NONFINITE      8u   /* a budget statistic was not finite: that head used the whole residual */
#define VATTN_STATUS_WAIT_TIMEOUT  16u   /* a bounded wait for an asynchronous copy ran out: the step's output is invalid */

typedef struct vattn_plan vattn_plan;    /* opaque; host memory */

typedef struct {
  int32_t batch, num_q_heads, num_kv_heads, head_dim;     /* head_dim in {64,128}; num_q_heads % num_kv_heads == 0 */
  int32_t block_size;                                     /* tokens per page: 16 */
  int32_t max_blocks_per_seq, num_blocks, max_seq_len;    /* max_seq_len <= max_blocks_per_seq * block_size */
  int32_t dtype;                                          /* VATTN_DTYPE_*: element type of q, k_cache, v_cache, out */
  int64_t kv_stride_block, kv_stride_head, kv_stride_token; /* elements; all zero = contiguous HND */
  int32_t q_len;                                          /* query tokens per sequence in one call; 0 or 1 = one (plain
                                                             decoding).  With q_len = T > 1 (a question, or speculative
                                                             tokens: the split-prompt setup of App. C, where everything
                                                             after the context runs through sparse attention) q and out
                                                             are [batch, T, num_q_heads, head_dim], the cache already
                                                             holds the T tokens' K and V rows, seq_lens counts them, and
                                                             query token t attends to the first seq_len - (T - 1 - t)
                                                             tokens (causal).  Every (token, head) pair is treated as a
                                                             head of its own -- own index sets, statistics, budget and
                                                             samples, drawn as decode step `step + t` -- and the pairs
                                                             that share a KV head share one pass over its K rows.
                                                             T * num_q_heads / num_kv_heads <= 64.  Introspection arrays
                                                             then have the head axis [KV head, t, head within the group] */
} vattn_shape;

/* Everything Algorithm 1/2 need beyond the short argument list of vattn_decode.  Zero = default. */
typedef struct {
  float   base_rate;       /* f_b: fraction of the residual n_s drawn as the base sample (Sec. 4.2, last paragraph);
                              default 0.025.  b0 = min(n_s, max(2, floor(f_b * n_s))) */
  float   topk_frac;       /* f_t: if > 0, k_b = floor(topk_frac * n_b) replaces the scalar k (Algorithm 1 line 3) */
  float   scale;           /* softmax scale applied to <K[i], q>; default 1/sqrt(head_dim) rounded to fp32 */
  int32_t mode;            /* which computation is kept verified (Algorithm 2): 0 SDPA (Theorem 4.3),
                              1 denominator only, 2 numerator only (Corollaries D.2) */
  int32_t layer, step;     /* Philox counter words; step < 2^31.  A step is a pure function of
                              (seed, layer, batch row, head, step): nothing is carried between calls */
  int32_t rng_head_is_kv;  /* 0: sampling keys per query head; 1: per KV head (the heads of a group share keys) */
  int32_t force_budget;    /* < 0 (or 0 with force_budget_on == 0): off; else b = min(force_budget, n_s) */
  int32_t force_budget_on; /* set to 1 to apply force_budget (so that a forced budget of 0 is expressible) */
  int32_t gather_mode;     /* 0: the sampled tokens' weights exp(s_i - m) come from the scores of the score pass and
                              only their V rows are read (default); 1: K and V rows are read and the scores are
                              recomputed from the K rows in fp32: the traffic of a pipeline whose selector leaves
                              no scores behind (the paper's composition with an approximate top-k, Sec. 4) */
  int32_t nested_base;     /* 0: base sample and final sample are independent draws (Algorithm 2 line 1 and
                              Algorithm 1 line 7 are separate calls); 1: the base sample is the first b0 tokens of
                              the final sample's walk, so I_bs is a subset of I_dyn (the reuse of the rows read for
                              the budget that the implementation paragraph of Sec. 4.2 describes) */
} vattn_params;

/* Optional per-call introspection.  All DEVICE pointers; NULL = not wanted.  cap = max_seq_len. */
typedef struct {
  int32_t *topk_idx, *topk_cnt;   /* [B,Hq,cap], [B,Hq]  I_t ascending (I_f = sink range + I_t + window range) */
  int32_t *base_idx, *base_cnt;   /* I_bs, b0: in the order of the walk that drew it (compare as a set) */
  int32_t *dyn_idx,  *dyn_cnt;    /* I_dyn, b: likewise */
  int32_t *budgets;               /* [B,Hq,4] ceil(b_D), ceil(b_N), ceil(b_SDPA) (saturating at 2^31-1), b */
  double  *stats;                 /* [B,Hq,8] D_f, sigma^2, Tr(Sigma), D_hat, |N_hat|_2, n_s, b0, m (weights are
                                     exp(s - m) with m the head's largest fp32 score) */
  float   *scores;                /* [B,Hq,cap] fp32 scores s_i = scale * <K[i], q> */
  int32_t *paths;                 /* [B,Hq] which code path the top-k selection took: bit 0 the usual one (one histogram
                                     of the keys' top bits, then an exact selection among the few candidates around
                                     the threshold; clear: the radix select over the whole middle range), bit 1
                                     near-tie tokens were rescored in fp64 and ranked from a list, bit 2 they were
                                     too many for the list and the exact 64-bit radix select ran
                                     (VATTN_STATUS_BAND_OVERFLOW) */
  unsigned long long *kernel_ticks; /* [VATTN_NUM_TICKS][2] device-side time stamps in ns (%globaltimer): rows 0-5 the
                                     counter-clearing kernel, the score kernel, the walk kernel, the selection kernel,
                                     the statistics kernel and the gather kernel ([k][0] = earliest CTA start,
                                     [k][1] = latest end); row 6 the top-k selection proper (first CTA past its
                                     dependency wait .. last CTA with I_t complete); row 7 the budgets (first head
                                     whose statistics are complete .. last head that knows its budget).
                                     Folded with atomic min / max: set [k][0] = UINT64_MAX and [k][1] = 0 before the
                                     step to be observed.  Unlike event profiling this leaves the step as it is */
} vattn_debug;

/* Create / destroy a plan for one problem shape.  `out` receives a host object.  Errors: INVALID_ARG,
 * UNSUPPORTED (head_dim other than 64 / 128, block_size other than 16, more than 64 (query token, query head)
 * pairs per KV head, q_len above 64, max_seq_len above 262,144, a bf16 batch above 1,536 rows, a batch above
 * 32,767 rows or more than 65,535 (batch row, query token, query head) triples: the kernels' grid dimensions). */
int    vattn_plan_create(const vattn_shape* shape, vattn_plan** out);
void   vattn_plan_destroy(vattn_plan* plan);

/* Bytes of device scratch a plan needs (a pure function of the shape), and handing it over.
 * The pointer must be 256-byte aligned and stay valid while the plan is used.  The contents need not
 * be initialised: the library clears what it needs (vattn_decode on every call, vattn_dense_decode on its
 * first call after this one); between calls it expects to find the workspace as it left it. */
size_t vattn_workspace_bytes(const vattn_plan* plan);
int    vattn_set_workspace(vattn_plan* plan, void* dev_ptr, size_t bytes);

/* Copy parameters / debug pointers into the plan (host structs; NULL resets to defaults). */
int    vattn_set_params(vattn_plan* plan, const vattn_params* params);
int    vattn_set_debug(vattn_plan* plan, const vattn_debug* debug);

/*
 * One verified sparse-attention decode step (Algorithm 1 with budget_X of Algorithm 2), for every
 * (batch row, query head):
 *   I_f  = first `sink` tokens + last `window` tokens + the k middle tokens with the largest
 *          scale*<K[i],q> (ties to the lowest index);            n_s = n - |I_f|
 *   I_bs = b0 residual tokens, uniform without replacement (Philox stream 0)
 *   b    = clamp(ceil(b_X(eps, delta; base-sample statistics)), b0, n_s)
 *   I_dyn= b residual tokens, uniform without replacement (Philox stream 1)
 *   out  = (N_f + n_s/b * sum_{I_dyn} w_i V[i]) / (D_f + n_s/b * sum_{I_dyn} w_i),  w_i = exp(s_i - m)
 * (Sec. 4.1 numerator/denominator equations; SDPA_{S,p} of Sec. 3).  A uniform sample of c tokens is
 * "the first c residual tokens met when the middle range [sink, n - window) is walked in the order
 * sink + sigma(0), sink + sigma(1), ...": sigma is a keyed permutation of the middle range, an 8-round
 * alternating Feistel network on ceil(log2(range)) bits (at least 2) with cycle walking, whose round keys are
 * the eight words of Philox4x32-10(key = seed, counter = (c, batch<<16 | head, layer, step<<1 | stream)),
 * c = 0, 1, and whose round function is xor with the round key followed by three multiply / xor-shift steps.
 * Degenerate inputs: n = 0 -> out row = 0; sink+window >= n -> exact attention, budget 0;
 * k larger than the middle range is clipped; sink = window = k = 0 with a forced budget of 0 leaves no token at
 * all and the row is 0/0 (NaN), as the formula gives.
 * eps, delta in (0,1).  Errors: INVALID_ARG, WORKSPACE, CUDA.  The step is several kernel launches: after
 * VATTN_ERR_CUDA some of them may have been enqueued already (they run; `out` is then undefined), and the
 * first kernel waits for whatever the caller enqueued on `stream` before the call.
 */
int vattn_decode(vattn_plan* plan, const void* q, const void* k_cache, const void* v_cache,
                 const int32_t* block_table, const int32_t* seq_lens,
                 int sink, int window, int k, float eps, float delta, uint64_t seed,
                 void* out, void* stream /* cudaStream_t */);

/* Dense attention over the same paged cache (full SDPA of Sec. 3), split over the context with a
 * fixed-order merge: the latency the sparse step is compared with.  Uses the plan's workspace (and relies on
 * the words it leaves there between calls: hand the plan a workspace, then do not write to it).  With
 * q_len > 1 the query tokens of a call are masked causally like vattn_decode's. */
int vattn_dense_decode(vattn_plan* plan, const void* q, const void* k_cache, const void* v_cache,
                       const int32_t* block_table, const int32_t* seq_lens, void* out, void* stream);

/*
 * vattn_dense_decode for callers that cannot give the library a workspace.  (The paper has no
 * counterpart: this is a deployment convenience.)  Who needs it: a serving engine that handed the
 * whole GPU to its KV-cache pool at start-up and has no device memory left to carve a workspace
 * from, or code on a latency-critical path that must not call cudaMalloc (which synchronises the
 * device).  No plan is needed and nothing is allocated, on the host or on the device: the split
 * partials live in a fixed array of VATTN_NOALLOC_SCRATCH_BYTES that is part of the library image, so
 * every GPU that loads the library holds that much memory until the process exits.
 *   - `scale` 0 means 1/sqrt(head_dim).  Arguments and layouts are those of vattn_dense_decode; one query token
 *     per sequence only (q_len > 1: VATTN_ERR_UNSUPPORTED).
 *   - The problem must fit: 256 + 12*batch*num_q_heads (rounded up to 256) +
 *     batch*num_q_heads*(head_dim+4)*4 bytes <= VATTN_NOALLOC_SCRATCH_BYTES (about 8,000 (batch row, query
 *     head) pairs at head_dim 128); larger problems return VATTN_ERR_WORKSPACE.  Fewer context splits are
 *     used when the usual number does not fit, so results can differ from vattn_dense_decode in the
 *     last bits.
 *   - The first call on each device looks up the array's device address (with that device current);
 *     make that first call outside any stream capture.
 *   - All calls, from every thread and stream, share the one array: two calls that overlap on the GPU
 *     race.  Serialise them on one stream or with events.  The part that must start at zero is cleared
 *     on `stream` at the start of every call.
 *   - Block-table entries outside [0, num_blocks) are read as page 0 and sequence lengths are clamped, as in
 *     vattn_dense_decode; the status bits of the last call on the current device (also WAIT_TIMEOUT, after
 *     which `out` is invalid) are read with vattn_noalloc_last_status, which waits for `stream`.
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE (too large), CUDA.
 */
#define VATTN_NOALLOC_SCRATCH_BYTES (4u << 20)
int vattn_dense_decode_noalloc(const vattn_shape* shape, float scale, const void* q, const void* k_cache,
                               const void* v_cache, const int32_t* block_table, const int32_t* seq_lens,
                               void* out, void* stream);
int vattn_noalloc_last_status(uint32_t* bits /* host */, void* stream);

/* Same step as vattn_decode with HOST buffers for q, block_table, seq_lens and out (the caches stay on
 * the device): copies the inputs in, runs the step, copies `out` back and waits for it.  `staging` is a
 * caller-owned device buffer of at least vattn_host_staging_bytes(plan) bytes.  Host buffers that are
 * page-locked and mapped into the device's address space are read by one small kernel and `out` is
 * written to the host buffer by the step itself (no copy-engine transfers, which cost several
 * microseconds each at these sizes); any other host memory goes through cudaMemcpyAsync.
 * A decode loop repeats this call with the same buffers: from the second call with one argument set on
 * (all pointers, scalars and the stream equal; page-locked host buffers; `stream` not being captured by
 * the caller; no debug buffers, profiling or stop-after in effect) the copies and kernels are recorded as
 * one CUDA graph that later calls replay, which reads the host buffers' current contents.  The plan keeps
 * the graphs of the 8 most recent argument sets (host objects; no device memory); every setter drops them. */
size_t vattn_host_staging_bytes(const vattn_plan* plan);
int vattn_decode_host(vattn_plan* plan, const void* q_host, const void* k_cache, const void* v_cache,
                      const int32_t* block_table_host, const int32_t* seq_lens_host,
                      int sink, int window, int k, float eps, float delta, uint64_t seed,
                      void* out_host, void* staging, void* stream);

/* OR of the status bits raised since the last call of this function on this plan.  Synchronises
 * `stream`; not for the hot path.  Errors: INVALID_ARG, WORKSPACE, CUDA. */
int vattn_last_status(vattn_plan* plan, void* stream, uint32_t* bits /* host */);

/* The step's kernels hand work to one another through words in the workspace: a producer CTA publishes a word
 * (release store), consumer CTAs poll it.  Every such wait is bounded: after a fixed number of polls the CTA falls
 * back to the grid-level dependency wait, which is always sufficient (the paper has no counterpart: this is how the
 * implementation overlaps Algorithm 1's stages).  This call runs the wait primitive alone: one thread polls a word
 * that nothing publishes, `spins` times (1 .. 2^20), and reports through *ran_out (host; 1 = the limit ended the
 * wait) and *waited_us (host; device-side microseconds).  It synchronises `stream`.  The context stays usable.
 * Errors: INVALID_ARG (null pointers, spins outside the range), WORKSPACE, CUDA. */
int vattn_probe_bounded_wait(vattn_plan* plan, uint32_t spins, uint32_t* ran_out /* host */,
                             uint32_t* waited_us /* host */, void* stream);

/* Number of kernels the last vattn_decode / vattn_dense_decode call on this plan enqueued. */
int vattn_last_launch_count(const vattn_plan* plan);

/* Measurement aid: while kernels > 0, vattn_decode enqueues only its first `kernels` kernels (in the order
 * listed for vattn_set_profiling below) and leaves `out` untouched; 0 restores the whole step.  Lets a
 * harness time one kernel launched back to back, without the launch gaps that events inside a step see.
 * Errors: INVALID_ARG (kernels outside [0, VATTN_NUM_KERNELS]). */
int vattn_set_stop_after(vattn_plan* plan, int kernels);

/* Optional per-kernel timing of vattn_decode, for measurement harnesses.  While enabled, every call
 * records CUDA events on `stream` around each of its VATTN_NUM_KERNELS kernels (score pass; walk tokens;
 * selection and sample lists; deterministic and base-sample rows with the budget; final sample and combination),
 * for up to 256 calls between two reads.  The events keep a kernel's prologue from running beside its predecessor, so the times add up to
 * more than an unprofiled step takes.  vattn_read_profile waits for the last recorded call, writes the
 * summed elapsed milliseconds per kernel to ms_sum[VATTN_NUM_KERNELS] (host) and the number of calls to
 * *calls (host), and starts a new window.  Events add a little latency: do not enable in production. */
#define VATTN_NUM_KERNELS 5
#define VATTN_NUM_TICKS 8
int vattn_set_profiling(vattn_plan* plan, int enable);
int vattn_read_profile(vattn_plan* plan, float* ms_sum, int* calls);

const char* vattn_strerror(int code);

/* z(x) = Phi^{-1}(1 - x/2), the two-sided standard-normal quantile of Lemma 4.1, as the library
 * evaluates it on the host (fp64) for the budget formulas.  0 < x < 2; NaN otherwise. */
double vattn_normal_quantile(double x);

#ifdef __cplusplus
}
#endif
#endif /* VATTN_H_ */
