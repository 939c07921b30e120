"""CPU oracle for the verified sparse-attention decode step (vAttention, arXiv 2510.05688).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, fp64 restatement of what the
paper's Algorithm 1 and Algorithm 2 compute for one decode step.  Only tests, the smoke
check and the benchmark's CPU-baseline leg may import it; the CUDA library never does,
and this file imports nothing from the CUDA package.

Every function follows a passage of the paper, taken in the paper's order and notation:

  scores            <K[i], q>                                 (Sec. 3, full SDPA equation)
  deterministic_sets I_s, I_l, I_t, I_f, n_s                  (Algorithm 1, lines 1-5)
  walk_order, sample uniform-sample(I_f, ., n)                (Algorithm 1 line 7; Algorithm 2 line 1)
  base_stats        get-stats / compute-stats                 (Algorithm 2; Corollaries D.2)
  budgets           b_D, b_N (Corollaries D.2), b_SDPA (Theorem 4.3), lower cap by the base budget
                    (captions of the epsilon/delta ablation figures in App. F)
  combine           N = N_f + n_s/|I_dyn| * sum, D likewise   (Sec. 4.1 numerator/denominator equations)
                    and SDPA_{S,p} (Sec. 3, importance-weighted equation)
  dense_sdpa        full SDPA                                  (Sec. 3)

Parity status: index sets, budgets and the estimator are pinned by tests/test_oracle_*.py
(dense-limit equality, brute-force subset enumeration, closed-form budgets, published Philox
known-answer vectors, the (eps, delta) definition over 1,000 seeds).  The *exact output values
for a given seed* have no counterpart in the paper (it prints no worked example and fixes no
random generator): for those values parity is unpinned beyond the pins above.

Readings taken where the paper is silent:
  * softmax scale is a parameter (default 1/sqrt(d)); exp is stabilised by the global max m,
    which cancels in N/D and in both budget ratios;
  * sink/window are absolute token counts, top-k is taken over the middle range only, ties go
    to the lowest index;
  * uniform sampling is WITHOUT replacement (so a budget equal to the residual gives dense SDPA);
    it is realised as "the first c residual tokens met when the middle range is walked in the order
    of a keyed pseudorandom permutation" (a Feistel network with cycle walking whose round keys are
    Philox4x32-10 words), with independent keys for the base sample (stream 0) and the final
    sample (stream 1);
  * sample variances use the unbiased (b0 - 1) denominator; tau uses the full estimates
    D_hat = D_f + ..., N_hat = N_f + ... as the corollaries define them;
  * the Theorem's min over (eps', delta') is taken in closed form over eps' and on the grid
    delta' = delta*j/16, j = 1..15, over delta'.
"""
from __future__ import annotations

import numpy as np
from scipy.stats import norm

BLOCK = 16
INT32_MAX = 2**31 - 1

# ----------------------------------------------------------------------------- element types
def _bf16_bits_to_f64(b):
    return (np.asarray(b, np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def to_f64(a, dtype):
    """Read stored elements exactly into fp64 (bf16 arrives as uint16 bit patterns)."""
    return _bf16_bits_to_f64(a) if dtype == "bf16" else np.asarray(a, np.float32).astype(np.float64)


def f64_to_bf16_bits(x):
    """Round fp64 directly to bf16 (nearest, ties to even): one rounding, no fp32 intermediate."""
    x = np.asarray(x, np.float64)
    u = x.view(np.uint64)
    # bf16 keeps 8 significand bits (7 stored); fp64 stores 52.  For the normal range of
    # bf16 (|x| in [2^-126, 2^128)) rounding the fp64 significand to 7 stored bits is exact
    # bf16 rounding; outputs here are attention averages, far inside that range.
    drop = np.uint64(52 - 7)
    lsb = (u >> drop) & np.uint64(1)
    r = (u + (np.uint64(1) << (drop - np.uint64(1))) - np.uint64(1) + lsb) >> drop << drop
    f32 = r.view(np.float64).astype(np.float32)          # exact: only 8 significant bits remain
    return (f32.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def gather_rows(cache, block_row, g, n, dtype):
    """Logical rows 0..n-1 of KV head g: row i lives at cache[block_row[i // 16], g, i % 16, :]."""
    nb = (n + BLOCK - 1) // BLOCK
    pages = np.asarray(block_row[:nb], np.int64)
    rows = to_f64(cache[pages, g], dtype).reshape(nb * BLOCK, cache.shape[-1])
    return rows[:n]


# ----------------------------------------------------------------------------- Philox4x32-10
# Counter-based generator of Salmon, Moraes, Dror, Shaw, "Parallel Random Numbers: As Easy as
# 1, 2, 3" (SC'11): 10 rounds; each round multiplies counter words 0 and 2 by two fixed odd
# constants, xors the high halves with the other counter words and the key, and permutes; the
# key is advanced by two Weyl constants between rounds.
_PHILOX_M0 = np.uint64(0xD2511F53)
_PHILOX_M1 = np.uint64(0xCD9E8D57)
_PHILOX_W0 = 0x9E3779B9
_PHILOX_W1 = 0xBB67AE85
_MASK32 = np.uint64(0xFFFFFFFF)


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Vectorised Philox4x32-10. Counter words are uint32 arrays (broadcastable); key words ints."""
    c0 = np.asarray(c0, np.uint64) & _MASK32
    c1 = np.asarray(c1, np.uint64) & _MASK32
    c2 = np.asarray(c2, np.uint64) & _MASK32
    c3 = np.asarray(c3, np.uint64) & _MASK32
    k0 = int(k0) & 0xFFFFFFFF
    k1 = int(k1) & 0xFFFFFFFF
    for rnd in range(10):
        if rnd > 0:
            k0 = (k0 + _PHILOX_W0) & 0xFFFFFFFF
            k1 = (k1 + _PHILOX_W1) & 0xFFFFFFFF
        p0 = _PHILOX_M0 * c0
        p1 = _PHILOX_M1 * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & _MASK32
        hi1, lo1 = p1 >> np.uint64(32), p1 & _MASK32
        c0, c1, c2, c3 = hi1 ^ c1 ^ np.uint64(k0), lo1, hi0 ^ c3 ^ np.uint64(k1), lo0
    return (c0.astype(np.uint32), c1.astype(np.uint32), c2.astype(np.uint32), c3.astype(np.uint32))


def walk_round_keys(seed, batch_idx, head_idx, layer, step, stream):
    """Eight 32-bit round keys of one (batch row, head, layer, step, stream):

    the words of Philox4x32-10(key = (seed_lo, seed_hi), ctr = (c, (batch << 16) | head, layer,
    (step << 1) | stream)) for c = 0 and c = 1."""
    w1 = ((int(batch_idx) & 0xFFFF) << 16) | (int(head_idx) & 0xFFFF)
    w3 = ((int(step) << 1) | int(stream)) & 0xFFFFFFFF
    out = philox4x32_10(np.arange(2, dtype=np.uint64), np.uint64(w1), np.uint64(int(layer) & 0xFFFFFFFF),
                        np.uint64(w3), int(seed) & 0xFFFFFFFF, (int(seed) >> 32) & 0xFFFFFFFF)
    return [int(out[j][c]) for c in range(2) for j in range(4)]


_MIX_A = np.uint64(0x9E3779B1)
_MIX_B = np.uint64(0x85EBCA77)
_MIX_C = np.uint64(0xC2B2AE3D)


def _mix32(x, key):
    """Round function of the permutation: xor with the round key, then three rounds of
    (multiply by an odd constant mod 2^32, xor-shift right), so that the low output bits depend on
    every input bit."""
    v = (np.asarray(x, np.uint64) ^ np.uint64(key)) & _MASK32
    v = (v * _MIX_A) & _MASK32
    v ^= v >> np.uint64(15)
    v = (v * _MIX_B) & _MASK32
    v ^= v >> np.uint64(13)
    v = (v * _MIX_C) & _MASK32
    v ^= v >> np.uint64(16)
    return v


def walk_bits(mlen):
    """Width of the permutation's domain: the smallest w >= 2 with 2^w >= mlen."""
    return max(2, int(max(int(mlen) - 1, 0)).bit_length())


def feistel(x, w, keys):
    """Keyed bijection of [0, 2^w): an alternating Feistel network of 8 rounds on the halves
    L (high floor(w/2) bits) and R (low ceil(w/2) bits).  Even rounds replace L by
    L xor (mix32(R, key_i) mod 2^|L|), odd rounds R by R xor (mix32(L, key_i) mod 2^|R|); each round is
    invertible whatever mix32 is, so the composition is a permutation."""
    lw = w // 2
    rw = w - lw
    x = np.asarray(x, np.uint64)
    L = x >> np.uint64(rw)
    R = x & np.uint64((1 << rw) - 1)
    for i in range(8):
        if i % 2 == 0:
            L = L ^ (_mix32(R, keys[i]) & np.uint64((1 << lw) - 1))
        else:
            R = R ^ (_mix32(L, keys[i]) & np.uint64((1 << rw) - 1))
    return (L << np.uint64(rw)) | R


def walk_order(mlen, keys):
    """sigma(0), ..., sigma(mlen-1): the keyed permutation of [0, mlen) obtained from `feistel` on
    [0, 2^w) by cycle walking (apply the bijection again while the image is >= mlen)."""
    mlen = int(mlen)
    w = walk_bits(mlen)
    x = feistel(np.arange(mlen, dtype=np.uint64), w, keys)
    while True:
        out = x >= np.uint64(mlen)
        if not out.any():
            return x.astype(np.int64)
        x[out] = feistel(x[out], w, keys)


def sample(in_residual, c, first, order):
    """uniform-sample: walk the middle range [first, first + len(order)) in the order
    first + sigma(0), first + sigma(1), ... and keep the first c tokens that are residual tokens;
    returned ascending.

    sigma is a keyed pseudorandom permutation of the middle range, so the residual tokens appear in
    a uniformly random order and the first c of them are a uniform draw of c residual tokens without
    replacement (Algorithm 1 line 7, Algorithm 2 line 1).  Any prefix of the walk is itself such a
    draw, which is what lets the base sample and the final sample be read off walks of their own."""
    c = int(c)
    if c <= 0 or len(order) == 0:
        return np.zeros(0, np.int64)
    toks = int(first) + np.asarray(order, np.int64)
    toks = toks[np.asarray(in_residual, bool)[toks]]
    return np.sort(toks[:c])


# ----------------------------------------------------------------------------- Algorithm 1, lines 1-5
def scores(q, K, scale):
    """s_i = scale * <K[i], q> in fp64 (Sec. 3).  K: [n,d] fp64, q: [d] fp64."""
    return (K * q[None, :]).sum(axis=1) * float(scale)


def deterministic_sets(s, sink, window, k):
    """I_s, I_l (absolute counts), I_t = top-k of the middle range by score, ties -> lowest index.

    Returns (I_f sorted ascending, I_t sorted ascending, residual R sorted ascending)."""
    n = s.shape[0]
    ns_ = min(int(sink), n)
    l_start = max(n - int(window), ns_)
    I_s = np.arange(0, ns_, dtype=np.int64)
    I_l = np.arange(l_start, n, dtype=np.int64)
    M = np.arange(ns_, l_start, dtype=np.int64)
    kk = min(int(k), M.size)
    if kk > 0:
        order = np.lexsort((M, -s[M]))                  # primary: score descending, secondary: index
        I_t = np.sort(M[order[:kk]])
    else:
        I_t = np.zeros(0, np.int64)
    in_t = np.zeros(n, bool)
    in_t[I_t] = True
    R = M[~in_t[M]]
    I_f = np.concatenate([I_s, I_t, I_l])
    I_f.sort()
    return I_f, I_t, R


# ----------------------------------------------------------------------------- Algorithm 2
def z_of(x):
    """z(x) = Phi^{-1}(1 - x/2), the two-sided normal quantile of the Lemma (computed as the
    upper-tail inverse at x/2, which is the same number without the 1 - x/2 cancellation)."""
    return float(norm.isf(0.5 * float(x)))


def base_size(n_s, base_rate):
    """b0 = floor(f_b * n_s), at least 2 (a variance needs two points), at most n_s."""
    return int(min(n_s, max(2, int(np.floor(float(np.float32(base_rate)) * n_s)))))


def base_stats(w, V, I_f, I_bs, n_s):
    """Statistics of Algorithm 2 from the base sample I_bs (r_i = w_i V[i]):

    sigma2 = sample variance of w over I_bs, trace = sum_j sample variance of r_ij,
    D_hat = D_f + (n_s/b0) sum w, N_hat = N_f + (n_s/b0) sum r   (Corollaries D.2)."""
    b0 = len(I_bs)
    D_f = w[I_f].sum()
    N_f = (w[I_f, None] * V[I_f]).sum(axis=0)
    wb = w[I_bs]
    rb = wb[:, None] * V[I_bs]
    if b0 >= 2:
        sigma2 = ((wb - wb.mean()) ** 2).sum() / (b0 - 1)
        trace = ((rb - rb.mean(axis=0)[None, :]) ** 2).sum() / (b0 - 1)
    else:
        sigma2 = trace = 0.0
    D_hat = D_f + (n_s / b0) * wb.sum()
    N_hat = N_f + (n_s / b0) * rb.sum(axis=0)
    return dict(D_f=float(D_f), N_f=N_f, sigma2=float(sigma2), trace=float(trace),
                D_hat=float(D_hat), N_hat_norm=float(np.sqrt((N_hat ** 2).sum())))


def budgets(st, n_s, eps, delta):
    """Real-valued budgets b_D, b_N (Corollaries D.2) and b_SDPA (Theorem 4.3).

    With A = n_s*sigma/D_hat and Bn = n_s*sqrt(trace)/|N_hat|:  b_D(e,x) = (z(x) A / e)^2 and
    b_N(e,x) = (z(x) Bn / e)^2.  In the Theorem, for fixed delta' the first argument of the max
    falls and the second rises with eps', so the inner optimum is where they are equal:
    4 (z(delta') A + z(delta-delta') Bn)^2 / eps^2; the outer min is taken on delta' = delta*j/16."""
    eps = float(np.float32(eps))
    delta = float(np.float32(delta))
    with np.errstate(all="ignore"):
        A = np.float64(n_s) * np.sqrt(np.float64(st["sigma2"])) / np.float64(st["D_hat"])
        Bn = np.float64(n_s) * np.sqrt(np.float64(st["trace"])) / np.float64(st["N_hat_norm"])
        zd = z_of(delta)
        b_D = (zd * A / eps) ** 2
        b_N = (zd * Bn / eps) ** 2
        cand = [(z_of(delta * j / 16.0) * A + z_of(delta * (16 - j) / 16.0) * Bn) ** 2 for j in range(1, 16)]
        b_S = 4.0 / eps ** 2 * (np.nan if any(np.isnan(c) for c in cand) else min(cand))
    return float(b_D), float(b_N), float(b_S)


def ceil_sat(x):
    """ceil with saturation: non-finite or >= 2^31-1 gives 2^31-1."""
    if not np.isfinite(x) or x >= INT32_MAX:
        return INT32_MAX
    return int(np.ceil(x))


def final_budget(bx, b0, n_s, force_budget=-1):
    """b = clamp(ceil(b_X), b0, n_s); non-finite -> n_s; force_budget >= 0 overrides."""
    if force_budget is not None and force_budget >= 0:
        return int(min(force_budget, n_s))
    return int(min(max(ceil_sat(bx), b0), n_s))


# ----------------------------------------------------------------------------- estimator
def combine(w, V, I_f, I_dyn, n_s):
    """N and D of Sec. 4.1: exact sums over I_f plus n_s/|I_dyn| times the sampled sums."""
    D = w[I_f].sum()
    N = (w[I_f, None] * V[I_f]).sum(axis=0)
    if len(I_dyn) > 0:
        f = n_s / len(I_dyn)
        D = D + f * w[I_dyn].sum()
        N = N + f * (w[I_dyn, None] * V[I_dyn]).sum(axis=0)
    return N, D


def dense_sdpa(q, K, V, scale):
    """Full SDPA of Sec. 3 for one head: sum_i a_i V[i], a = softmax(scale * K q)."""
    s = scores(q, K, scale)
    a = np.exp(s - s.max())
    return (a[:, None] * V).sum(axis=0) / a.sum()


# ----------------------------------------------------------------------------- one head, one step
def decode_head(q, K, V, *, sink, window, k, eps, delta, seed, batch_idx, head_idx, rng_head,
                base_rate=0.025, scale=None, mode=0, layer=0, step=0, force_budget=-1, nested_base=0):
    """Algorithm 1 for one (batch row, query head).  q [d], K,V [n,d] fp64.  Returns a dict.

    nested_base = 1 reads the base sample off the final sample's walk (I_bs = its first b0 residual
    tokens, I_dyn = its first b: I_bs is a subset of I_dyn), the reuse of budget-calculation rows that the
    implementation paragraph of Sec. 4.2 describes; 0 (default) draws the two independently, as the
    separate uniform-sample calls of Algorithm 2 line 1 and Algorithm 1 line 7 read."""
    n, d = K.shape
    if scale is None:
        scale = float(np.float32(1.0 / np.sqrt(d)))
    res = dict(n=n)
    if n == 0:
        res.update(out=np.zeros(d), I_f=np.zeros(0, np.int64), I_t=np.zeros(0, np.int64),
                   I_bs=np.zeros(0, np.int64), I_dyn=np.zeros(0, np.int64), n_s=0, b0=0, b=0,
                   budgets=(0, 0, 0, 0), stats=np.zeros(8), scores=np.zeros(0))
        return res
    s = scores(q, K, scale)
    m = s.max()
    w = np.exp(s - m)
    I_f, I_t, R = deterministic_sets(s, sink, window, k)
    n_s = int(R.size)
    res.update(scores=s, m=float(m), I_f=I_f, I_t=I_t, n_s=n_s)
    if n_s == 0:
        N, D = combine(w, V, I_f, np.zeros(0, np.int64), 0)
        res.update(out=N / D, I_bs=np.zeros(0, np.int64), I_dyn=np.zeros(0, np.int64), b0=0, b=0,
                   budgets=(0, 0, 0, 0),
                   stats=np.array([D, 0.0, 0.0, D, np.sqrt((N ** 2).sum()), 0.0, 0.0, m]))
        return res
    b0 = base_size(n_s, base_rate)
    first = min(int(sink), n)                       # the middle range starts behind the sink tokens
    mlen = max(n - int(window), first) - first
    in_R = np.zeros(n, bool)
    in_R[R] = True
    I_bs = sample(in_R, b0, first,
                  walk_order(mlen, walk_round_keys(seed, batch_idx, rng_head, layer, step, 1 if nested_base else 0)))
    st = base_stats(w, V, I_f, I_bs, n_s)
    b_D, b_N, b_S = budgets(st, n_s, eps, delta)
    bx = (b_S, b_D, b_N)[int(mode)]
    b = final_budget(bx, b0, n_s, force_budget)
    I_dyn = sample(in_R, b, first, walk_order(mlen, walk_round_keys(seed, batch_idx, rng_head, layer, step, 1)))
    N, D = combine(w, V, I_f, I_dyn, n_s)
    res.update(out=N / D, I_bs=I_bs, I_dyn=I_dyn, b0=b0, b=b,
               budgets=(ceil_sat(b_D), ceil_sat(b_N), ceil_sat(b_S), b),
               budgets_real=(b_D, b_N, b_S),
               stats=np.array([st["D_f"], st["sigma2"], st["trace"], st["D_hat"], st["N_hat_norm"],
                               float(n_s), float(b0), m]))
    return res


def resolve_k(k, topk_frac, n):
    """k for a sequence of n tokens: floor(topk_frac * n) when topk_frac > 0, else the scalar k."""
    tf = float(np.float32(topk_frac or 0.0))
    return int(np.floor(tf * n)) if tf > 0.0 else int(k)


def vattn_decode(q, k_cache, v_cache, block_table, seq_lens, sink, window, k, eps, delta, seed, *,
                 dtype, base_rate=0.025, topk_frac=0.0, scale=None, mode=0, layer=0, step=0,
                 rng_head_is_kv=0, force_budget=-1, nested_base=0, heads=None):
    """One decode step over the paged cache.  Returns (out [B,Hq,d] in the storage type, details).

    q [B,Hq,d]; caches [num_blocks,Hkv,16,d]; every query head h uses KV head h // (Hq/Hkv) and
    has its own index sets, budget and sample.  `heads` optionally restricts the work to a list of
    (b, h) pairs (used for sampled checks at large sizes); other rows of `out` stay zero."""
    B, Hq, d = q.shape
    Hkv = k_cache.shape[1]
    G = Hq // Hkv
    base_rate = 0.025 if not base_rate else base_rate
    if not scale:
        scale = float(np.float32(1.0 / np.sqrt(d)))
    else:
        scale = float(np.float32(scale))
    out64 = np.zeros((B, Hq, d))
    details = {}
    todo = heads if heads is not None else [(b, h) for b in range(B) for h in range(Hq)]
    cache_rows = {}
    for (b, h) in todo:
        n = int(seq_lens[b])
        g = h // G
        if (b, g) not in cache_rows:
            cache_rows = {(b, g): (gather_rows(k_cache, block_table[b], g, n, dtype),
                                   gather_rows(v_cache, block_table[b], g, n, dtype))}
        K, V = cache_rows[(b, g)]
        r = decode_head(to_f64(q[b, h], dtype), K, V, sink=sink, window=window,
                        k=resolve_k(k, topk_frac, n), eps=eps, delta=delta, seed=seed, batch_idx=b,
                        head_idx=h, rng_head=(g if rng_head_is_kv else h), base_rate=base_rate,
                        scale=scale, mode=mode, layer=layer, step=step, force_budget=force_budget,
                        nested_base=nested_base)
        out64[b, h] = r["out"]
        details[(b, h)] = r
    out = f64_to_bf16_bits(out64) if dtype == "bf16" else out64.astype(np.float32)
    return out, details


def dense_decode(q, k_cache, v_cache, block_table, seq_lens, *, dtype, scale=None):
    """Dense SDPA over the same paged cache, fp64 (the comparison kernel's reference)."""
    B, Hq, d = q.shape
    Hkv = k_cache.shape[1]
    G = Hq // Hkv
    if not scale:
        scale = float(np.float32(1.0 / np.sqrt(d)))
    out = np.zeros((B, Hq, d))
    for b in range(B):
        n = int(seq_lens[b])
        if n == 0:
            continue
        for g in range(Hkv):
            K = gather_rows(k_cache, block_table[b], g, n, dtype)
            V = gather_rows(v_cache, block_table[b], g, n, dtype)
            for h in range(g * G, (g + 1) * G):
                out[b, h] = dense_sdpa(to_f64(q[b, h], dtype), K, V, scale)
    return out


# ----------------------------------------------------------------------------- several query tokens per call
def _visible_lens(seq_lens, Tq, t):
    """Tokens that query token t of Tq sees: the cache already holds all Tq new rows, attention is causal."""
    return np.maximum(np.asarray(seq_lens, np.int64) - (Tq - 1 - t), 0)


def vattn_decode_multi(q, k_cache, v_cache, block_table, seq_lens, sink, window, k, eps, delta, seed, *,
                       dtype, step=0, heads=None, **params):
    """A call that carries Tq query tokens per sequence (a question, speculative tokens: the split-prompt
    setup of App. C, where everything after the context goes through sparse attention).

    q [B,Tq,Hq,d].  Query token t attends to the first n - (Tq - 1 - t) tokens and is, in every other
    respect, the decode step `step + t` of Algorithm 1 on that prefix: own index sets, statistics, budget
    and samples per (token, head).  `heads` optionally restricts the work to (b, t, h) triples.
    Returns (out [B,Tq,Hq,d] in the storage type, details keyed (b, t, h))."""
    B, Tq, Hq, d = q.shape
    out = np.zeros((B, Tq, Hq, d), np.uint16 if dtype == "bf16" else np.float32)
    details = {}
    for t in range(Tq):
        sel = None if heads is None else [(b, h) for (b, tt, h) in heads if tt == t]
        if sel is not None and not sel:
            continue
        o, det = vattn_decode(np.ascontiguousarray(q[:, t]), k_cache, v_cache, block_table,
                              _visible_lens(seq_lens, Tq, t), sink, window, k, eps, delta, seed, dtype=dtype,
                              step=step + t, heads=sel, **params)
        out[:, t] = o
        for (b, h), r in det.items():
            details[(b, t, h)] = r
    return out, details


def dense_decode_multi(q, k_cache, v_cache, block_table, seq_lens, *, dtype, scale=None):
    """Causal dense SDPA for Tq query tokens per sequence, fp64: q [B,Tq,Hq,d] -> [B,Tq,Hq,d]."""
    B, Tq, Hq, d = q.shape
    out = np.zeros((B, Tq, Hq, d))
    for t in range(Tq):
        out[:, t] = dense_decode(np.ascontiguousarray(q[:, t]), k_cache, v_cache, block_table,
                                 _visible_lens(seq_lens, Tq, t), dtype=dtype, scale=scale)
    return out
