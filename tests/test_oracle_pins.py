"""Pins for the CPU oracle: each test checks it against something other than itself.

P1  a budget equal to the whole residual (or sink+window covering the context) must give dense
    SDPA, computed here independently (explicit de-paging loop + torch fp64 SDPA).
P2  tiny inputs: top-k against a full sort, the residual against a set difference, and the
    estimator averaged over ALL subsets of the residual must equal the exact sums; its variance
    must equal the finite-population formula for sampling without replacement.
P3  the (eps, delta) definition (Definition 4.1 of the paper) over 1,000 seeds.
P4  closed-form budgets (Lemma 4.1, Corollaries D.2, Theorem 4.3) on hand-computable populations.
P5  Philox4x32-10 against the published known-answer vectors; the walk permutation against brute force
    (a bijection, undone by the network run backwards; cycle walking stays inside the middle range).
P6  the sampler is uniform over subsets and over walk positions (chi-square) and never selects outside the
    residual.
"""
import itertools
import math
import os
import statistics

import numpy as np
import pytest
import torch

from oracle import vattn_oracle as O
from paper_2510_05688_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def ZQ(x):
    """Phi^{-1}(1 - x/2) from the Python standard library (not the routine the oracle calls)."""
    return statistics.NormalDist().inv_cdf(1.0 - 0.5 * x)


# ----------------------------------------------------------------------------- helpers (independent of the oracle)
def depage_loop(case, cache, b, g):
    """Token-by-token de-paging, written independently of oracle.gather_rows."""
    vals = case.values(cache).astype(np.float64)
    n = int(case.seq_lens[b])
    rows = np.zeros((n, case.head_dim))
    for i in range(n):
        rows[i] = vals[int(case.block_table[b, i // 16]), g, i % 16]
    return rows


def torch_sdpa(case, b, h, scale):
    G = case.num_q_heads // case.num_kv_heads
    g = h // G
    K = torch.from_numpy(depage_loop(case, case.k_cache, b, g))
    V = torch.from_numpy(depage_loop(case, case.v_cache, b, g))
    q = torch.from_numpy(case.values(case.q)[b, h].astype(np.float64))[None, :]
    o = torch.nn.functional.scaled_dot_product_attention(q[None, None], K[None, None], V[None, None], scale=scale)
    return o[0, 0, 0].numpy()


def small_case(dtype, seq_lens=(70, 33), Hq=4, Hkv=2, d=32, **kw):
    args = dict(dtype=dtype, B=len(seq_lens), Hq=Hq, Hkv=Hkv, d=d, seq_lens=list(seq_lens), sink=3,
                window=5, k=4, eps=0.05, delta=0.05, seed=11, gen_seed=77, rho_v=1.0,
                heavy=dict(R=3, c1=3.0, alpha=(1.0, 1.0)))
    args.update(kw)
    return synth.make_case("small", **args)


def run_oracle(case, **over):
    p = dict(case.params)
    p.update(over)
    return O.vattn_decode(case.q, case.k_cache, case.v_cache, case.block_table, case.seq_lens, case.sink,
                          case.window, case.k, case.eps, case.delta, case.seed, dtype=case.dtype, **p)


# ----------------------------------------------------------------------------- P1
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_p1_full_residual_budget_equals_dense_sdpa(dtype):
    case = small_case(dtype)
    scale = float(np.float32(1.0 / math.sqrt(case.head_dim)))
    out, det = run_oracle(case, force_budget=10**9)
    for (b, h), r in det.items():
        assert r["b"] == r["n_s"] and len(r["I_dyn"]) == r["n_s"]
        ref = torch_sdpa(case, b, h, scale)
        np.testing.assert_allclose(r["out"], ref, rtol=1e-12, atol=1e-13)
    dense = O.dense_decode(case.q, case.k_cache, case.v_cache, case.block_table, case.seq_lens, dtype=dtype)
    for (b, h) in det:
        np.testing.assert_allclose(dense[b, h], torch_sdpa(case, b, h, scale), rtol=1e-12, atol=1e-13)


def test_p1_sink_plus_window_cover_context():
    case = small_case("fp32", sink=40, window=40)
    scale = float(np.float32(1.0 / math.sqrt(case.head_dim)))
    _, det = run_oracle(case)
    for (b, h), r in det.items():
        assert r["n_s"] == 0 and r["b"] == 0 and r["budgets"] == (0, 0, 0, 0)
        assert len(r["I_f"]) == r["n"] and len(r["I_t"]) == 0
        np.testing.assert_allclose(r["out"], torch_sdpa(case, b, h, scale), rtol=1e-12, atol=1e-13)


def test_p1_explicit_scale_and_gqa_mapping():
    # a different scale must change the result exactly as torch's scale= does; heads of one
    # group share K/V but not q
    case = small_case("fp32", seq_lens=(41,), Hq=6, Hkv=2, d=16)
    _, det = run_oracle(case, force_budget=10**9, scale=0.37)
    sc = float(np.float32(0.37))
    for (b, h), r in det.items():
        np.testing.assert_allclose(r["out"], torch_sdpa(case, b, h, sc), rtol=1e-12, atol=1e-13)


def test_bf16_output_rounding_is_single_rne():
    x = np.array([1.0, 1.00390625, 1.01171875, -3.0000001, 0.1, 1.0 + 2**-8 - 2**-30, 65280.0, 1e-3], np.float64)
    got = O.f64_to_bf16_bits(x)
    want = torch.tensor(x, dtype=torch.float64).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert (got == want).all()
    # tie case: exactly halfway between two bf16 values goes to the even one
    assert O.f64_to_bf16_bits(np.array([1.00390625]))[0] == 0x3F80       # 1 + 2^-8 -> 1.0
    assert O.f64_to_bf16_bits(np.array([1.01171875]))[0] == 0x3F82       # 1 + 3*2^-8 -> 1 + 2^-6
    # just above the halfway point must round up (a conversion through fp32 would lose the 2^-30
    # and then break the tie downwards: the oracle rounds once)
    assert O.f64_to_bf16_bits(np.array([1.0 + 2**-8 + 2**-30]))[0] == 0x3F81


# ----------------------------------------------------------------------------- P2
def test_p2_topk_and_residual_bruteforce():
    rng = np.random.default_rng(5)
    for trial in range(50):
        n = int(rng.integers(1, 15))
        s = rng.standard_normal(n).round(1)            # rounding creates ties
        sink, window, k = int(rng.integers(0, 4)), int(rng.integers(0, 4)), int(rng.integers(0, 6))
        I_f, I_t, R = O.deterministic_sets(s, sink, window, k)
        ns_ = min(sink, n)
        ls = max(n - window, ns_)
        M = list(range(ns_, ls))
        ranked = sorted(M, key=lambda i: (-s[i], i))   # full sort, ties -> lowest index
        want_t = sorted(ranked[:min(k, len(M))])
        assert list(I_t) == want_t
        want_f = sorted(set(range(ns_)) | set(range(ls, n)) | set(want_t))
        assert list(I_f) == want_f
        assert list(R) == sorted(set(range(n)) - set(want_f))


def test_p2_estimator_unbiased_over_all_subsets_and_variance():
    rng = np.random.default_rng(9)
    n, d = 12, 3
    s = rng.standard_normal(n)
    V = rng.standard_normal((n, d))
    w = np.exp(s - s.max())
    I_f, I_t, R = O.deterministic_sets(s, 1, 2, 2)
    n_s = len(R)
    assert n_s == 7
    D_exact = w.sum()
    N_exact = (w[:, None] * V).sum(axis=0)
    for b in (1, 3, 7):
        Ds, Ns = [], []
        for sub in itertools.combinations(R.tolist(), b):
            N, D = O.combine(w, V, I_f, np.array(sub), n_s)
            Ds.append(D)
            Ns.append(N)
        Ds, Ns = np.array(Ds), np.array(Ns)
        assert abs(Ds.mean() - D_exact) < 1e-12
        np.testing.assert_allclose(Ns.mean(axis=0), N_exact, atol=1e-12)
        # sampling without replacement: Var = n_s^2 (1 - b/n_s) S^2 / b, S^2 with n_s - 1
        S2 = w[R].var(ddof=1)
        assert abs(Ds.var() - n_s**2 * (1 - b / n_s) * S2 / b) < 1e-12
    # b = n_s has a single subset and is exact
    N, D = O.combine(w, V, I_f, R, n_s)
    assert abs(D - D_exact) < 1e-14


def test_p2_sample_is_first_residual_tokens_of_the_walk():
    # a hand-written walk order over the middle range [2, 10): the sample is its first c residual tokens
    order = np.array([4, 0, 7, 2, 6, 1, 3, 5])                  # sigma(0..7); tokens 6, 2, 9, 4, 8, 3, 5, 7
    in_R = np.zeros(12, bool)
    in_R[[2, 3, 5, 6, 8, 9]] = True                             # tokens 4 and 7 are top-k members
    walk = [6, 2, 9, 8, 3, 5]                                   # the walk with the members struck out
    for c in range(0, 7):
        assert O.sample(in_R, c, 2, order).tolist() == sorted(walk[:c])
    assert O.sample(in_R, 99, 2, order).tolist() == [2, 3, 5, 6, 8, 9]
    assert O.sample(in_R, 3, 2, np.zeros(0, np.int64)).tolist() == []


def test_walk_round_keys_are_the_philox_words_of_counters_0_and_1():
    seed, b, h, layer, step = (0xDEADBEEF << 32) | 0x12345678, 3, 7, 5, 1000
    for stream in (0, 1):
        keys = O.walk_round_keys(seed, b, h, layer, step, stream)
        want = []
        for c in (0, 1):
            out = O.philox4x32_10(np.uint64(c), np.uint64((b << 16) | h), np.uint64(layer),
                                  np.uint64((step << 1) | stream), seed & 0xFFFFFFFF, seed >> 32)
            want += [int(o) for o in out]
        assert keys == want and len(set(keys)) == 8
    assert O.walk_round_keys(seed, b, h, layer, step, 0) != O.walk_round_keys(seed, b, h, layer, step, 1)
    assert O.walk_round_keys(seed, b, h, layer, step, 0) != O.walk_round_keys(seed, b, h + 1, layer, step, 0)


def _unfeistel(y, w, keys):
    """The network run backwards, written out here on Python ints (not the oracle's code): undoing
    round i needs only the half that round i left untouched."""
    lw = w // 2
    rw = w - lw
    L, R = y >> rw, y & ((1 << rw) - 1)

    def mix(x, k):
        v = (x ^ k) & 0xFFFFFFFF
        v = (v * 0x9E3779B1) & 0xFFFFFFFF
        v ^= v >> 15
        v = (v * 0x85EBCA77) & 0xFFFFFFFF
        v ^= v >> 13
        v = (v * 0xC2B2AE3D) & 0xFFFFFFFF
        v ^= v >> 16
        return v
    for i in reversed(range(8)):
        if i % 2 == 0:
            L ^= mix(R, keys[i]) & ((1 << lw) - 1)
        else:
            R ^= mix(L, keys[i]) & ((1 << rw) - 1)
    return (L << rw) | R


def test_feistel_is_a_bijection_and_the_reversed_network_undoes_it():
    rng = np.random.default_rng(12)
    for w in range(2, 14):
        keys = [int(x) for x in rng.integers(0, 2**32, size=8)]
        img = O.feistel(np.arange(1 << w, dtype=np.uint64), w, keys)
        assert sorted(img.tolist()) == list(range(1 << w))
        for x in (0, 1, (1 << w) - 1, (1 << w) // 3):
            assert _unfeistel(int(img[x]), w, keys) == x
    assert [O.walk_bits(m) for m in (0, 1, 2, 4, 5, 8, 9, 1024, 1025, 32512)] == [2, 2, 2, 2, 3, 3, 4, 10, 11, 15]


def test_walk_order_is_a_permutation_of_the_middle_range():
    rng = np.random.default_rng(13)
    for mlen in list(range(0, 70)) + [127, 128, 129, 1000, 4097, 32512]:
        keys = [int(x) for x in rng.integers(0, 2**32, size=8)]
        order = O.walk_order(mlen, keys)
        assert sorted(order.tolist()) == list(range(mlen))
    # cycle walking: the image of j is the first point of the orbit j -> feistel(j) -> ... below mlen
    keys = [int(x) for x in rng.integers(0, 2**32, size=8)]
    mlen, w = 37, 6
    order = O.walk_order(mlen, keys)
    for j in range(mlen):
        y = int(O.feistel(np.array([j], np.uint64), w, keys)[0])
        while y >= mlen:
            y = int(O.feistel(np.array([y], np.uint64), w, keys)[0])
        assert y == int(order[j])


def test_walk_positions_are_uniform_and_streams_are_unrelated():
    # over seeds, sigma(j) is uniform on [0, mlen) for fixed j, and neighbouring images are not tied together
    mlen, T = 13, 26000
    hits = np.zeros((3, mlen))
    gap = np.zeros(mlen)
    same = 0
    for seed in range(T):
        o0 = O.walk_order(mlen, O.walk_round_keys(seed, 2, 5, 1, 9, 0))
        o1 = O.walk_order(mlen, O.walk_round_keys(seed, 2, 5, 1, 9, 1))
        for r, j in enumerate((0, 6, 12)):
            hits[r, o0[j]] += 1
        gap[(o0[1] - o0[0]) % mlen] += 1
        same += int(o0[0] == o1[0])
    exp = T / mlen
    for r in range(3):
        assert ((hits[r] - exp) ** 2 / exp).sum() < 40.0          # 12 dof: P(chi2 > 40) ~ 7e-5
    assert gap[0] == 0
    expg = T / (mlen - 1)
    assert ((gap[1:] - expg) ** 2 / expg).sum() < 38.0            # 11 dof
    assert abs(same / T - 1.0 / mlen) < 4.0 * math.sqrt((1 / mlen) * (1 - 1 / mlen) / T)


def test_resolve_k_and_base_size_by_hand():
    # k = floor(f32(f_t) * n) with the product in fp64: f32(0.02) = 0.0199999995529651..., so 0.02 * 4150 falls
    # just below 83
    assert [O.resolve_k(7, 0.02, n) for n in (4097, 4150, 4151)] == [81, 82, 83]
    assert O.resolve_k(7, 0.0, 4150) == 7 and O.resolve_k(7, None, 10) == 7
    assert O.resolve_k(0, 0.5, 9) == 4 and O.resolve_k(3, 1.0, 9) == 9
    # b0 = min(n_s, max(2, floor(f32(f_b) * n_s))): f32(0.025) = 0.02500000037..., so 0.025 * 80 = 2.00000003 -> 2
    assert [O.base_size(ns, 0.025) for ns in (1, 2, 3, 79, 80, 120)] == [1, 2, 2, 2, 2, 3]
    assert O.base_size(0, 0.025) == 0 and O.base_size(40, 1.0) == 40 and O.base_size(1000, 0.1) == 100


def test_nested_base_sample_is_a_prefix_of_the_final_sample():
    case = small_case("fp32", seq_lens=(300,), Hq=2, Hkv=1, d=16, sink=4, window=4, k=8)
    _, det = run_oracle(case, base_rate=0.1, nested_base=1, force_budget=60)
    _, ind = run_oracle(case, base_rate=0.1, force_budget=60)
    for key, r in det.items():
        assert r["b"] == 60 and r["b0"] == 28 and set(r["I_bs"].tolist()) <= set(r["I_dyn"].tolist())
        # the final sample's walk is the same in both variants; only the base sample moves
        assert not set(ind[key]["I_bs"].tolist()) <= set(ind[key]["I_dyn"].tolist())
        keys1 = O.walk_round_keys(case.seed, key[0], key[1], 0, 0, 1)
        walk = [4 + int(x) for x in O.walk_order(300 - 8, keys1) if (4 + int(x)) not in set(r["I_t"].tolist())]
        assert sorted(walk[:r["b0"]]) == r["I_bs"].tolist() and sorted(walk[:r["b"]]) == r["I_dyn"].tolist()


# ----------------------------------------------------------------------------- P3
def test_p3_eps_delta_definition_over_1000_seeds():
    eps = delta = 0.1
    case = synth.make_case("p3", dtype="fp32", B=1, Hq=1, Hkv=1, d=64, seq_lens=[8192], sink=128, window=128,
                           k=int(0.025 * 8192), eps=eps, delta=delta, seed=0, gen_seed=31337, key_std=0.1,
                           rho_v=2.0, heavy=None, params=dict(base_rate=0.025))
    scale = float(np.float32(1.0 / 8.0))
    ref = torch_sdpa(case, 0, 0, scale)
    T, fails, used = 1000, 0, []
    for seed in range(T):
        case.seed = seed
        _, det = run_oracle(case)
        r = det[(0, 0)]
        used.append(r["b"] / r["n_s"])
        err = np.linalg.norm(r["out"] - ref) / np.linalg.norm(ref)
        fails += err > eps
    # the case must not be vacuous (budget well below the residual)
    assert np.mean(used) < 0.5
    slack = 3.0 * math.sqrt(delta * (1 - delta) / T)
    assert fails / T <= delta + slack


def test_p3_nested_base_sample_failure_rate_is_measured():
    # nested_base = 1: the base sample is the first b0 residual tokens of the final sample's own walk, so the
    # budget depends on rows that are also in the sample.  The (eps, delta) statement is measured, not assumed:
    # 1,000 seeds of the same case as above, failure rate within the same statistical slack.  (Measured when this
    # test was written: independent samples 0 failures, nested 0 failures of 1,000; the bound is delta = 0.1.)
    eps = delta = 0.1
    case = synth.make_case("p3", dtype="fp32", B=1, Hq=1, Hkv=1, d=64, seq_lens=[8192], sink=128, window=128,
                           k=int(0.025 * 8192), eps=eps, delta=delta, seed=0, gen_seed=31337, key_std=0.1,
                           rho_v=2.0, heavy=None, params=dict(base_rate=0.025, nested_base=1))
    scale = float(np.float32(1.0 / 8.0))
    ref = torch_sdpa(case, 0, 0, scale)
    T, fails, used, nested_ok = 1000, 0, [], 0
    for seed in range(T):
        case.seed = seed
        _, det = run_oracle(case)
        r = det[(0, 0)]
        used.append(r["b"] / r["n_s"])
        nested_ok += set(r["I_bs"].tolist()) <= set(r["I_dyn"].tolist())
        err = np.linalg.norm(r["out"] - ref) / np.linalg.norm(ref)
        fails += err > eps
    assert nested_ok == T
    assert np.mean(used) < 0.5
    print("nested P3: failures", fails, "of", T, "mean b/n_s", float(np.mean(used)))
    assert fails / T <= delta + 3.0 * math.sqrt(delta * (1 - delta) / T)


# ----------------------------------------------------------------------------- P4
def test_p4_normal_quantiles_table():
    for line in open(os.path.join(GOLD, "normal_quantiles.txt")):
        if line.startswith("#") or not line.strip():
            continue
        x, z = map(float, line.split())
        assert abs(O.z_of(x) - z) < 6e-7


def _stats(sigma2, trace, D_hat, N_norm):
    return dict(sigma2=sigma2, trace=trace, D_hat=D_hat, N_hat_norm=N_norm)


def test_p4_budget_closed_forms_and_scaling():
    n_s, eps, delta = 1000, 0.125, 0.05          # eps exactly representable in fp32
    st = _stats(0.04, 0.09, 500.0, 50.0)         # sigma = .2, sqrt(trace) = .3
    b_D, b_N, b_S = O.budgets(st, n_s, eps, delta)
    z = ZQ(float(np.float32(delta)))               # stdlib quantile: independent of the oracle's scipy call
    assert abs(b_D - (z * n_s * 0.2 / (eps * 500.0)) ** 2) < 1e-9 * b_D
    assert abs(b_N - (z * n_s * 0.3 / (eps * 50.0)) ** 2) < 1e-9 * b_N
    # b(eps/2) = 4 b(eps) for all three
    h_D, h_N, h_S = O.budgets(st, n_s, eps / 2, delta)
    for a, b in ((h_D, b_D), (h_N, b_N), (h_S, b_S)):
        assert abs(a - 4 * b) < 1e-9 * a
    # Theorem: splitting eps and delta costs more than 4x either single-quantity budget,
    # and the grid minimum is no worse than the midpoint split
    assert b_S > 4 * max(b_D, b_N)
    A, Bn = n_s * 0.2 / 500.0, n_s * 0.3 / 50.0
    mid = 4 / eps**2 * (O.z_of(delta / 2) * (A + Bn)) ** 2
    assert b_S <= mid * (1 + 1e-12)
    # brute force over a fine (eps', delta') grid of the Theorem's min-max never beats the closed form by
    # more than the grid resolution, and never exceeds it
    best = math.inf
    for dj in np.linspace(delta / 16, delta * 15 / 16, 15):
        z1, z2 = O.z_of(dj), O.z_of(delta - dj)
        for e1 in np.linspace(eps * 0.001, eps * 0.999, 4000):
            val = max((z1 * A / (e1 / 2)) ** 2, (z2 * Bn / ((eps - e1) / 2)) ** 2)
            best = min(best, val)
    assert b_S <= best <= b_S * 1.01


def test_p4_equal_residual_weights_give_base_budget():
    # all keys identical -> all residual weights equal -> sigma^2 = 0 -> b_D = 0 -> b = b0 (D mode)
    case = small_case("fp32", seq_lens=(400,), Hq=1, Hkv=1, d=16, heavy=None, sink=4, window=4, k=8)
    vals = case.k_cache.copy()
    vals[...] = vals[case.block_table[0, 0], 0, 0][None, None, None, :]
    case.k_cache = vals
    _, det = run_oracle(case, mode=1, base_rate=0.05)
    r = det[(0, 0)]
    assert r["stats"][1] == 0.0 and r["budgets"][0] == 0
    assert r["b"] == r["b0"] == int(math.floor(float(np.float32(0.05)) * r["n_s"]))
    # ties in the top-k go to the lowest indices of the middle range
    assert r["I_t"].tolist() == list(range(4, 12))


def test_p4_scalar_values_make_numerator_budget_equal_denominator_budget():
    # d = 1 and V == 1: the numerator is the denominator, so b_N == b_D
    rng = np.random.default_rng(3)
    n = 300
    K = rng.standard_normal((n, 1))
    V = np.ones((n, 1))
    r = O.decode_head(np.array([1.3]), K, V, sink=2, window=2, k=5, eps=0.05, delta=0.05, seed=1, batch_idx=0,
                      head_idx=0, rng_head=0, base_rate=0.1, scale=1.0, mode=0)
    b_D, b_N, _ = r["budgets_real"]
    assert abs(b_D - b_N) <= 1e-12 * b_D


def test_p4_two_point_population_by_hand():
    # base sample = whole residual (base_rate 1): m tokens with weight a and m with weight b
    m_, a, b = 20, 1.0, 0.5
    n_s = 2 * m_
    w = np.array([2.0] + [a] * m_ + [b] * m_)           # token 0 is the deterministic set, weight 2
    V = np.ones((n_s + 1, 1))
    st = O.base_stats(w, V, np.array([0]), np.arange(1, n_s + 1), n_s)
    var = (n_s / (n_s - 1)) * ((a - b) / 2) ** 2        # unbiased sample variance of a two-point set
    assert abs(st["sigma2"] - var) < 1e-15
    D = 2.0 + m_ * (a + b)
    assert abs(st["D_hat"] - D) < 1e-12 and abs(st["D_f"] - 2.0) < 1e-15
    b_D, _, _ = O.budgets(st, n_s, 0.25, 0.05)
    assert abs(b_D - (ZQ(float(np.float32(0.05))) * n_s * math.sqrt(var) / (0.25 * D)) ** 2) < 1e-9 * b_D
    assert O.final_budget(b_D, 5, n_s) == min(max(math.ceil(b_D), 5), n_s)
    assert O.final_budget(0.0, 5, n_s) == 5 and O.final_budget(1e30, 5, n_s) == n_s
    assert O.final_budget(float("nan"), 5, n_s) == n_s and O.final_budget(3.2, 5, n_s, force_budget=7) == 7


def test_base_sample_estimates_are_close_to_population_values():
    # the paper's Table 9 reports a few % error for base-sample estimates at f_b = 0.025-0.1
    case = synth.make_case("t9", dtype="fp32", B=1, Hq=1, Hkv=1, d=64, seq_lens=[16384], sink=128, window=128,
                           k=409, eps=0.05, delta=0.05, seed=0, gen_seed=99, key_std=1.0, rho_v=1.0, heavy=None)
    K = O.gather_rows(case.k_cache, case.block_table[0], 0, 16384, "fp32")
    V = O.gather_rows(case.v_cache, case.block_table[0], 0, 16384, "fp32")
    q = O.to_f64(case.q[0, 0], "fp32")
    s = O.scores(q, K, 0.125)
    w = np.exp(s - s.max())
    I_f, I_t, R = O.deterministic_sets(s, 128, 128, 409)
    pop_sigma2 = w[R].var(ddof=1)
    pop_trace = ((w[R, None] * V[R]).var(axis=0, ddof=1)).sum()
    errs = []
    for seed in range(40):
        in_R = np.zeros(16384, bool)
        in_R[R] = True
        I_bs = O.sample(in_R, O.base_size(len(R), 0.1), 128,
                        O.walk_order(16384 - 256, O.walk_round_keys(seed, 0, 0, 0, 0, 0)))
        st = O.base_stats(w, V, I_f, I_bs, len(R))
        errs.append((abs(st["sigma2"] - pop_sigma2) / pop_sigma2, abs(st["trace"] - pop_trace) / pop_trace))
    errs = np.array(errs).mean(axis=0)
    assert errs[0] < 0.15 and errs[1] < 0.15


# ----------------------------------------------------------------------------- P5
def test_p5_philox_known_answer_vectors():
    rows = 0
    for line in open(os.path.join(GOLD, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        v = [int(x, 16) for x in line.split()]
        out = O.philox4x32_10(*[np.array([c], np.uint64) for c in v[:4]], v[4], v[5])
        assert [int(o[0]) for o in out] == v[6:]
        rows += 1
    assert rows == 3


# ----------------------------------------------------------------------------- P6
def test_p6_sampler_uniform_over_subsets():
    n, c = 12, 3
    R = np.array([2, 3, 5, 6, 7, 8, 9, 10])              # residual of size 8: middle range [1, 11) minus {1, 4}
    in_R = np.zeros(n, bool)
    in_R[R] = True
    subsets = {s: 0 for s in itertools.combinations(R.tolist(), c)}
    T = 28000
    incl = np.zeros(n)
    for seed in range(T):
        pick = O.sample(in_R, c, 1, O.walk_order(10, O.walk_round_keys(seed, 0, 1, 2, 3, 1)))
        subsets[tuple(pick.tolist())] += 1               # KeyError if anything outside R is drawn
        incl[pick] += 1
    exp = T / len(subsets)
    chi2 = sum((v - exp) ** 2 / exp for v in subsets.values())
    assert len(subsets) == 56 and chi2 < 105.0            # 55 dof: P(chi2 > 105) ~ 5e-5
    assert np.abs(incl[R] / T - c / len(R)).max() < 0.012


# ----------------------------------------------------------------------------- several query tokens per call
def test_multi_query_full_budget_equals_causal_sdpa():
    """With the whole residual as budget every query token of a call must give causal dense attention: token t
    of Tq sees the first n - (Tq - 1 - t) rows.  The reference is torch's SDPA over all Tq rows at once with an
    explicit mask built here, on independently de-paged K and V."""
    case = small_case("bf16", seq_lens=(70, 33, 2))
    Tq = 3
    q4 = synth.multi_query(case, Tq)
    scale = float(np.float32(1.0 / math.sqrt(case.head_dim)))
    out, det = O.vattn_decode_multi(q4, case.k_cache, case.v_cache, case.block_table, case.seq_lens, case.sink,
                                    case.window, case.k, case.eps, case.delta, case.seed, dtype=case.dtype,
                                    force_budget=10**9)
    dense = O.dense_decode_multi(q4, case.k_cache, case.v_cache, case.block_table, case.seq_lens, dtype=case.dtype)
    G = case.num_q_heads // case.num_kv_heads
    qv = case.values(q4).astype(np.float64)
    for b in range(case.batch):
        n = int(case.seq_lens[b])
        mask = torch.zeros(Tq, n, dtype=torch.bool)
        for t in range(Tq):
            mask[t, :max(0, n - (Tq - 1 - t))] = True
        for h in range(case.num_q_heads):
            K = torch.from_numpy(depage_loop(case, case.k_cache, b, h // G))
            V = torch.from_numpy(depage_loop(case, case.v_cache, b, h // G))
            Q = torch.from_numpy(qv[b, :, h])
            ref = torch.nn.functional.scaled_dot_product_attention(Q[None, None], K[None, None], V[None, None],
                                                                   attn_mask=mask[None, None], scale=scale)[0, 0].numpy()
            for t in range(Tq):
                r = det[(b, t, h)]
                if r["n"] == 0:                              # a query token that sees nothing: zeros by convention
                    assert not r["out"].any() and not dense[b, t, h].any()
                    continue
                assert r["n"] == n - (Tq - 1 - t) and r["b"] == r["n_s"]
                np.testing.assert_allclose(r["out"], ref[t], rtol=1e-12, atol=1e-13)
                np.testing.assert_allclose(dense[b, t, h], ref[t], rtol=1e-12, atol=1e-13)


def test_multi_query_tokens_are_consecutive_decode_steps():
    """Query token t of a call is decode step `step + t` on its prefix: the same index sets, budget and output
    as a single-query call with that step word and that length; one query token is the single-query call."""
    case = small_case("fp32", seq_lens=(90, 41))
    Tq = 2
    q4 = synth.multi_query(case, Tq)
    _, det = O.vattn_decode_multi(q4, case.k_cache, case.v_cache, case.block_table, case.seq_lens, case.sink,
                                  case.window, case.k, case.eps, case.delta, case.seed, dtype=case.dtype, step=5)
    for t in range(Tq):
        lens = np.asarray(case.seq_lens) - (Tq - 1 - t)
        _, one = O.vattn_decode(np.ascontiguousarray(q4[:, t]), case.k_cache, case.v_cache, case.block_table, lens,
                                case.sink, case.window, case.k, case.eps, case.delta, case.seed, dtype=case.dtype,
                                step=5 + t)
        for (b, h), r in one.items():
            m = det[(b, t, h)]
            assert np.array_equal(m["I_dyn"], r["I_dyn"]) and np.array_equal(m["I_bs"], r["I_bs"])
            assert m["budgets"] == r["budgets"] and np.array_equal(m["out"], r["out"])
    # samples of consecutive tokens differ (their step words do)
    assert any(not np.array_equal(det[(0, 0, h)]["I_bs"], det[(0, 1, h)]["I_bs"]) for h in range(case.num_q_heads))
    out1, det1 = O.vattn_decode_multi(case.q[:, None], case.k_cache, case.v_cache, case.block_table, case.seq_lens,
                                      case.sink, case.window, case.k, case.eps, case.delta, case.seed, dtype=case.dtype)
    out0, det0 = run_oracle(case)
    assert np.array_equal(out1[:, 0], out0)
