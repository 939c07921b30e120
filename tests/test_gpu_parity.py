"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded inputs.

Index sets (I_t, I_bs, I_dyn), budgets and counts must be bit-exact; outputs within 1e-5 relative
(fp32) / 2e-2 absolute-or-relative (bf16).  Small cases span several tiles and ragged tails; the
five workload configurations run at full size.
"""
import numpy as np
import pytest

from oracle import vattn_oracle as O
from paper_2510_05688_b200 import synth
from helpers import (assert_out_close, assert_parity, assert_parity_multi, out_values, run_gpu, run_gpu_multi, run_oracle,
                     run_oracle_multi)

pytestmark = pytest.mark.gpu


def small(dtype, seq_lens, Hq=8, Hkv=2, d=128, **kw):
    args = dict(dtype=dtype, B=len(seq_lens), Hq=Hq, Hkv=Hkv, d=d, seq_lens=list(seq_lens), sink=4, window=8, k=16,
                eps=0.05, delta=0.05, seed=1234, gen_seed=42, key_std=1.0, rho_v=1.0,
                heavy=dict(R=12, c1=5.0, alpha=(0.75, 1.25)), params=dict(base_rate=0.05))
    args.update(kw)
    return synth.make_case("small", **args)


def check(case, **over):
    out_ref, det = run_oracle(case, **over)
    out, dbg, plan = run_gpu(case, **over)
    assert_parity(case, out, dbg, det, out_ref)
    return out, dbg, det, plan


# ----------------------------------------------------------------------------- small shapes, ragged tails
@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("bf16", 64), ("fp32", 64), ("fp32", 128)])
def test_small_ragged_batches(dtype, d):
    case = small(dtype, [1, 15, 16, 17, 255, 600, 1000, 2049, 33], d=d)
    check(case)
    check(case, mode=1)
    check(case, mode=2)


@pytest.mark.parametrize("Hq,Hkv", [(4, 4), (8, 1), (6, 2), (10, 2)])
def test_gqa_ratios(Hq, Hkv):
    # G = 1, 8 (two head chunks), 3 and 5 (partial head chunks)
    check(small("bf16", [700, 129], Hq=Hq, Hkv=Hkv))


def test_sixteen_heads_per_kv_head():
    check(small("bf16", [530, 90], Hq=16, Hkv=1))            # G = 16: two chunks of 8 heads in the score pass


def test_context_beyond_the_shared_memory_key_cache():
    # 45,000 tokens on 8 CTAs per head: two pages per thread, so every selection pass re-reads its scores from L2
    case = synth.make_case("long", dtype="bf16", B=1, Hq=2, Hkv=1, d=128, seq_lens=[45000], sink=64, window=64, k=700,
                           eps=0.1, delta=0.1, seed=3, gen_seed=808, rho_v=1.0,
                           heavy=dict(R=64, c1=8.0, alpha=(0.75, 1.25)), params=dict(base_rate=0.02))
    _, dbg, _, _ = check(case)
    assert (dbg["paths"] & 4 == 0).all()


def test_padded_cache_strides():
    # rows 16-byte aligned but not contiguous: token stride d + 8, head stride padded, as a caller's cache may be
    import torch
    from paper_2510_05688_b200 import binding as vb
    case = small("bf16", [700, 129])
    d, Hkv, nblk = case.head_dim, case.num_kv_heads, case.num_blocks
    st, sh = d + 8, 16 * (d + 8) + 24
    sb = Hkv * sh + 40
    dev = vb.case_to_device(case)

    def pad(cache):
        buf = torch.full((nblk * sb,), 7.0, dtype=cache.dtype, device="cuda")
        view = torch.as_strided(buf, (nblk, Hkv, 16, d), (sb, sh, st, 1))
        view.copy_(cache)
        return buf
    kbuf, vbuf = pad(dev["k_cache"]), pad(dev["v_cache"])
    plan = vb.Plan(batch=case.batch, num_q_heads=case.num_q_heads, num_kv_heads=Hkv, head_dim=d,
                   max_blocks_per_seq=case.max_blocks_per_seq, num_blocks=nblk, max_seq_len=case.max_blocks_per_seq * 16,
                   dtype=vb.DTYPE_BF16, kv_strides=(sb, sh, st))
    out_ref, det = run_oracle(case)
    got, dbg, _ = run_gpu(case, plan=plan, dev=dict(dev, k_cache=kbuf, v_cache=vbuf))
    assert_parity(case, got, dbg, det, out_ref)
    out = torch.empty_like(dev["q"])
    plan.dense_decode(dev["q"], kbuf, vbuf, dev["block_table"], dev["seq_lens"], out)
    torch.cuda.synchronize()
    ref = O.dense_decode(case.q, case.k_cache, case.v_cache, case.block_table, case.seq_lens, dtype="bf16")
    assert (np.abs(out.float().cpu().numpy() - ref) <= 2e-2 * np.maximum(1.0, np.abs(ref))).all()


def test_empty_and_covered_sequences():
    case = small("bf16", [0, 5, 12, 300, 0], sink=4, window=8, k=3)
    out, dbg, det, _ = check(case)
    assert (out_values(case, out)[0] == 0).all() and (out_values(case, out)[4] == 0).all()
    # sink + window >= n: exact attention, budget 0
    for h in range(case.num_q_heads):
        assert det[(1, h)]["n_s"] == 0 and dbg["dyn_cnt"][1, h] == 0
    dense = O.dense_decode(case.q, case.k_cache, case.v_cache, case.block_table, case.seq_lens, dtype=case.dtype)
    assert np.abs(out_values(case, out)[1:3] - dense[1:3]).max() < 2e-2


def test_k_zero_and_k_larger_than_middle():
    check(small("fp32", [400, 77], d=64, k=0))
    check(small("fp32", [400, 77], d=64, k=100000))
    check(small("bf16", [400, 77], sink=0, window=0, k=7))


def test_middle_range_without_a_sampled_token():
    """Middle ranges of a few tokens that miss the one token per page which the selection samples for its threshold
    estimate (page 0 is sampled at offset 0, page 1 at offset 0, page 2 at offset 1, ...): the estimate has nothing to
    go on and the selection must still be exact."""
    check(small("bf16", [14, 15, 16, 10, 12, 31, 40], sink=4, window=1, k=1))
    check(small("bf16", [14, 16, 30], sink=4, window=1, k=3, params=dict(base_rate=0.1, nested_base=1)))
    check(small("fp32", [13, 20, 47], d=64, sink=1, window=2, k=2))


def test_topk_takes_almost_the_whole_middle_range():
    """k within a few tokens of the middle range: nearly every walk position is a member of I_t, so the prefix that
    holds the base sample (and the pivot, and the final sample) lies behind long runs of marked positions."""
    case = small("bf16", [202, 300, 150, 1000], sink=0, window=1, k=200, params=dict(base_rate=0.3))
    check(case)                                        # residuals of 1, 99, 0 and 799 tokens
    out_ref, _ = run_oracle(case)
    out, _, _ = run_gpu(case, debug=False)             # (without introspection the samples come off the walk arrays)
    assert_out_close(case, out, out_ref, "k = middle - 1")
    for k in (995, 990, 900):
        case = small("bf16", [1000], sink=2, window=2, k=k, params=dict(base_rate=0.1, nested_base=k % 2))
        check(case)
        out_ref, _ = run_oracle(case)
        out, _, _ = run_gpu(case, debug=False)
        assert_out_close(case, out, out_ref, f"k = {k} of 996")


def test_topk_fraction_and_kv_head_rng():
    check(small("bf16", [900, 350], k=0, params=dict(base_rate=0.05, topk_frac=0.03)))
    check(small("bf16", [900, 350], params=dict(base_rate=0.1, rng_head_is_kv=1, layer=3, step=77)))


def test_full_residual_budget_equals_dense_attention():
    case = small("fp32", [513, 64], d=64)
    out, dbg, det, _ = check(case, force_budget=10**9)
    dense = O.dense_decode(case.q, case.k_cache, case.v_cache, case.block_table, case.seq_lens, dtype=case.dtype)
    ref = np.abs(dense).max(axis=-1, keepdims=True)
    assert (np.abs(out_values(case, out) - dense) / ref).max() < 1e-5
    check(case, force_budget=0)
    check(case, force_budget=37)


def test_explicit_scale():
    check(small("bf16", [300], params=dict(base_rate=0.05, scale=0.2)))


def test_identical_keys_take_the_exact_tie_path():
    # every key row identical: all scores tie, the near-tie band is the whole middle range
    case = small("bf16", [3000], Hq=4, Hkv=2, heavy=None, k=40)
    kc = case.k_cache.copy()
    kc[...] = kc[case.block_table[0, 0], :, 0][None, :, None, :]
    case.k_cache = kc
    out, dbg, det, plan = check(case)
    for h in range(4):
        assert dbg["topk_idx"][0, h, :40].tolist() == list(range(4, 44))      # lowest indices win ties
        assert dbg["stats"][0, h, 1] == 0.0                                     # sigma^2 exactly 0
    assert plan.last_status() & 4                                               # band overflow was reported


def test_zero_query_and_duplicated_rows():
    case = small("bf16", [500], Hq=4, Hkv=2, heavy=None)
    q = case.q.copy()
    q[0, 1] = 0                                                                 # bf16 bit pattern of 0
    case.q = q
    kc = case.k_cache.copy()
    pg = case.block_table[0]
    kc[pg[3], :, 5] = kc[pg[9], :, 2]                                           # two identical rows (tokens 53, 146)
    case.k_cache = kc
    check(case)


def test_bad_block_table_entry_sets_status_without_faulting():
    import torch
    from paper_2510_05688_b200 import binding as vb
    case = small("bf16", [200])
    dev = vb.case_to_device(case)
    dev["block_table"][0, 2] = case.num_blocks + 5
    plan = vb.plan_for_case(case)
    out = torch.empty_like(dev["q"])
    plan.decode(dev["q"], dev["k_cache"], dev["v_cache"], dev["block_table"], dev["seq_lens"], 4, 8, 16, 0.05, 0.05,
                1, out)
    torch.cuda.synchronize()
    assert plan.last_status() & vb.STATUS_BAD_BLOCK
    assert plan.last_status() == 0                                              # reading clears the word


def test_two_calls_are_bitwise_reproducible():
    case = small("bf16", [2049, 700])
    out1, dbg1, plan = run_gpu(case)
    out2, dbg2, _ = run_gpu(case, plan=plan)
    assert np.array_equal(out1, out2)
    assert np.array_equal(dbg1["dyn_idx"], dbg2["dyn_idx"])


def test_dense_kernel_matches_dense_sdpa():
    import torch
    from paper_2510_05688_b200 import binding as vb
    for dtype, d in (("bf16", 128), ("fp32", 64), ("bf16", 64), ("fp32", 128)):
        case = small(dtype, [1, 17, 0, 1000, 2049], d=d)
        dev = vb.case_to_device(case)
        plan = vb.plan_for_case(case)
        out = torch.empty_like(dev["q"])
        plan.dense_decode(dev["q"], dev["k_cache"], dev["v_cache"], dev["block_table"], dev["seq_lens"], out)
        torch.cuda.synchronize()
        got = out.float().cpu().numpy().astype(np.float64)
        ref = O.dense_decode(case.q, case.k_cache, case.v_cache, case.block_table, case.seq_lens, dtype=dtype)
        tol = 2e-2 if dtype == "bf16" else 2e-5
        assert (np.abs(got - ref) <= tol * np.maximum(1.0, np.abs(ref))).all(), (dtype, d, np.abs(got - ref).max())
        assert plan.last_launch_count() == 1
        # the kernel leaves its counters ready for the next call: the same again, and after a sparse step
        out2 = torch.empty_like(out)
        plan.dense_decode(dev["q"], dev["k_cache"], dev["v_cache"], dev["block_table"], dev["seq_lens"], out2)
        torch.cuda.synchronize()
        assert torch.equal(out2.view(torch.int16 if dtype == "bf16" else torch.int32),
                           out.view(torch.int16 if dtype == "bf16" else torch.int32))
        plan.decode(dev["q"], dev["k_cache"], dev["v_cache"], dev["block_table"], dev["seq_lens"], case.sink,
                    case.window, case.k, case.eps, case.delta, case.seed, out2)
        plan.dense_decode(dev["q"], dev["k_cache"], dev["v_cache"], dev["block_table"], dev["seq_lens"], out2)
        torch.cuda.synchronize()
        assert torch.equal(out2.view(torch.int16 if dtype == "bf16" else torch.int32),
                           out.view(torch.int16 if dtype == "bf16" else torch.int32))


@pytest.mark.parametrize("Hq,Hkv", [(8, 8), (8, 1), (12, 1), (6, 2)])
def test_dense_kernel_group_sizes_and_mixed_lengths(Hq, Hkv):
    """Query-head groups of 1, 3, 8 and 12 heads (a group larger than the 8 rows of a tile takes two CTAs), and
    lengths from one page to the longest the cache holds: sequences get splits in proportion to their length."""
    import torch
    from paper_2510_05688_b200 import binding as vb
    case = small("bf16", [16, 5000, 333, 4097, 1, 2500], Hq=Hq, Hkv=Hkv)
    dev = vb.case_to_device(case)
    plan = vb.plan_for_case(case)
    out = torch.empty_like(dev["q"])
    plan.dense_decode(dev["q"], dev["k_cache"], dev["v_cache"], dev["block_table"], dev["seq_lens"], out)
    torch.cuda.synchronize()
    got = out.float().cpu().numpy().astype(np.float64)
    ref = O.dense_decode(case.q, case.k_cache, case.v_cache, case.block_table, case.seq_lens, dtype="bf16")
    assert (np.abs(got - ref) <= 2e-2 * np.maximum(1.0, np.abs(ref))).all(), np.abs(got - ref).max()
    assert plan.last_status() == 0


def test_host_buffer_entry_point_matches_device_entry_point():
    import torch
    from paper_2510_05688_b200 import binding as vb
    case = small("bf16", [900, 350])
    out_dev, _, plan = run_gpu(case, debug=False)
    dev = vb.case_to_device(case)
    qh = dev["q"].cpu().pin_memory()
    bth = dev["block_table"].cpu().pin_memory()
    slh = dev["seq_lens"].cpu().pin_memory()
    outh = torch.empty_like(qh).pin_memory()
    plan.decode_host(qh, dev["k_cache"], dev["v_cache"], bth, slh, case.sink, case.window, case.k, case.eps,
                     case.delta, case.seed, outh)
    assert np.array_equal(outh.view(torch.int16).numpy().view(np.uint16), out_dev)
    # a decode loop: the same buffers again and again (from the third call on the step replays as one CUDA
    # graph), with new contents in the host buffers every time
    rng = np.random.default_rng(5)
    for it in range(5):
        case.q = synth.f32_to_bf16_bits(rng.standard_normal(case.q.shape).astype(np.float32))
        lens = np.array([900 - 7 * it, 350 - it], dtype=np.int32)
        case.seq_lens = lens
        qh.view(torch.int16).copy_(torch.from_numpy(case.q.view(np.int16)))
        slh.copy_(torch.from_numpy(lens))
        outh.zero_()
        plan.decode_host(qh, dev["k_cache"], dev["v_cache"], bth, slh, case.sink, case.window, case.k, case.eps,
                         case.delta, case.seed, outh)
        want, _, _ = run_gpu(case, debug=False)               # a plan of its own: setters would drop the graph
        assert np.array_equal(outh.view(torch.int16).numpy().view(np.uint16), want), f"host step {it}"
    assert plan.last_status() == 0


def test_seeded_random_shapes():
    # odd sizes, sink + window around n, k from 0 to more than the middle range, ragged batches
    rng = np.random.default_rng(2024)
    for trial in range(12):
        B = int(rng.integers(1, 5))
        lens = [int(x) for x in rng.integers(1, 601, size=B)]
        Hkv = int(rng.choice([1, 2, 4]))
        G = int(rng.choice([1, 2, 3, 4, 8]))
        d = int(rng.choice([64, 128]))
        dtype = str(rng.choice(["bf16", "fp32"]))
        case = small(dtype, lens, Hq=Hkv * G, Hkv=Hkv, d=d, sink=int(rng.integers(0, 40)), window=int(rng.integers(0, 40)),
                     k=int(rng.integers(0, 80)), seed=int(rng.integers(0, 2**40)), gen_seed=1000 + trial,
                     eps=float(rng.choice([0.05, 0.1, 0.3])), delta=float(rng.choice([0.05, 0.2])),
                     params=dict(base_rate=float(rng.choice([0.025, 0.1, 0.5])), mode=int(rng.integers(0, 3)),
                                 layer=int(rng.integers(0, 32)), step=int(rng.integers(0, 1000))))
        check(case)


def test_appending_rows_between_steps_reuses_the_plan():
    # reasoning-length decode: one K/V row per sequence is appended between steps, the step word advances,
    # nothing but seq_lens and the new rows changes
    import torch
    from paper_2510_05688_b200 import binding as vb
    B, n0, steps = 2, 1036, 5
    full = synth.make_case("grow", dtype="bf16", B=B, Hq=8, Hkv=2, d=128, seq_lens=[n0 + steps] * B, sink=16, window=16,
                           k=26, eps=0.05, delta=0.05, seed=5, gen_seed=77, rho_v=1.0,
                           heavy=dict(R=16, c1=6.0, alpha=(0.75, 1.25)), params=dict(base_rate=0.05), poison_unused=False)
    dev_full = vb.case_to_device(full)
    # start from caches in which the rows beyond n0 are not written yet
    kc, vc = dev_full["k_cache"].clone(), dev_full["v_cache"].clone()
    bt = full.block_table
    for b in range(B):
        for i in range(n0, n0 + steps):
            kc[bt[b, i // 16], :, i % 16] = 0
            vc[bt[b, i // 16], :, i % 16] = 0
    plan = vb.plan_for_case(full)
    out = torch.empty_like(dev_full["q"])
    for s in range(steps):
        n = n0 + s
        for b in range(B):                       # the harness appends row n-1 of every sequence
            i = n - 1
            kc[bt[b, i // 16], :, i % 16] = dev_full["k_cache"][bt[b, i // 16], :, i % 16]
            vc[bt[b, i // 16], :, i % 16] = dev_full["v_cache"][bt[b, i // 16], :, i % 16]
        case = synth.Case(name="grow", dtype="bf16", q=full.q, k_cache=full.k_cache, v_cache=full.v_cache,
                          block_table=full.block_table, seq_lens=np.array([n] * B, np.int32), sink=16, window=16,
                          k=int(0.025 * n), eps=0.05, delta=0.05, seed=5, params=dict(base_rate=0.05, step=s))
        dev = dict(dev_full, k_cache=kc, v_cache=vc, seq_lens=torch.from_numpy(case.seq_lens).cuda())
        out_ref, det = run_oracle(case)
        got, dbg, _ = run_gpu(case, plan=plan, dev=dev)
        assert_parity(case, got, dbg, det, out_ref)


# ----------------------------------------------------------------------------- fast paths and their fallbacks at size
def mid(**kw):
    args = dict(dtype="bf16", B=1, Hq=8, Hkv=2, d=128, seq_lens=[20000], sink=64, window=64, k=500, eps=0.05,
                delta=0.05, seed=99, gen_seed=4242, key_std=1.0, rho_v=1.0,
                heavy=dict(R=64, c1=8.0, alpha=(0.75, 1.25)), params=dict(base_rate=0.025))
    args.update(kw)
    return synth.make_case("mid", **args)


def test_large_base_rate_and_large_budgets():
    # base sample of half the residual; forced budgets of a fifth, of almost half and of all of it: walks of
    # thousands of positions, several rounds of a warp's row list, the last walk covering the whole middle range
    check(mid(params=dict(base_rate=0.5)))
    check(mid(), force_budget=4000)
    check(mid(), force_budget=9000)
    _, dbg, det, _ = check(mid(), force_budget=10**9)
    assert all(r["b"] == r["n_s"] for r in det.values())


def test_single_huge_outlier_score_defeats_the_threshold_estimate():
    case = mid(heavy=None)
    kc = synth.bf16_bits_to_f32(case.k_cache)
    q = synth.bf16_bits_to_f32(case.q)
    tok = 7777
    pg = case.block_table[0, tok // 16]
    for g in range(2):                        # one key aligned with the group's first query, logit ~ +3000
        kc[pg, g, tok % 16] = 3000.0 * np.sqrt(128.0) * q[0, g * 4] / float(q[0, g * 4] @ q[0, g * 4])
    case.k_cache = synth.f32_to_bf16_bits(kc)
    check(case)                               # heads 0 and 4 see the outlier: a top radix bin with a single key


def test_many_topk_and_fp32_at_size():
    check(mid(k=6000))                        # a third of the context is top-k
    check(mid(dtype="fp32", d=64, seq_lens=[20000, 9000], B=2))


def test_maximum_context_length():
    # 262,144 tokens (the largest context a plan accepts), one head on 8 CTAs: 128 scores per thread re-read from
    # L2 in every selection pass, walks over an 18-bit domain, the score pass walks 16,384 pages
    case = synth.make_case("max", dtype="bf16", B=1, Hq=1, Hkv=1, d=128, seq_lens=[262144], sink=128, window=128, k=3000,
                           eps=0.1, delta=0.1, seed=11, gen_seed=909, rho_v=1.0,
                           heavy=dict(R=128, c1=9.0, alpha=(0.75, 1.25)), params=dict(base_rate=0.01))
    _, dbg, det, _ = check(case)
    assert det[(0, 0)]["b"] < det[(0, 0)]["n_s"]
    assert (dbg["paths"] & 5 == 0).all()


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("bf16", 64), ("fp32", 64), ("fp32", 128)])
def test_gather_that_recomputes_the_weights_from_k_rows(dtype, d):
    check(small(dtype, [1, 17, 600, 2049], d=d), gather_mode=1)


def test_gather_from_k_rows_at_size():
    check(mid(), gather_mode=1)


def test_largest_bf16_batch():
    # 1,536 rows (the most a bf16 plan accepts): the score kernel's per-row tables fill its shared memory
    rng = np.random.default_rng(78)
    lens = [int(x) for x in rng.integers(0, 72, size=1536)]
    check(small("bf16", lens, Hq=2, Hkv=1))


def test_many_short_sequences_in_one_batch():
    # 48 ragged rows, some of them empty: the score pass cuts them into many small work units that its CTAs
    # take from a counter, and every list kernel meets heads without any work
    rng = np.random.default_rng(77)
    lens = [int(x) for x in rng.integers(0, 700, size=48)]
    lens[3] = 0
    lens[17] = 0
    lens[47] = 1
    check(small("bf16", lens, Hq=8, Hkv=2))


@pytest.mark.parametrize("B,Hq,Hkv", [(2, 32, 8), (4, 32, 8), (17, 8, 2)])
def test_head_counts_around_the_decomposition_thresholds(B, Hq, Hkv):
    # 64 heads: statistics CTAs split unevenly between the two row kinds, flat gather with 32 chunks per head;
    # 128 heads: even split (the wave is overfull), the flat gather's largest head count; 136 heads: the
    # per-head gather.  Forced budgets of 3,000 rows give chunks of several batches and a ragged last batch.
    lens = [int(x) for x in np.random.default_rng(5 + B).integers(3500, 5200, size=B)]
    case = small("bf16", lens, Hq=Hq, Hkv=Hkv, sink=16, window=32, k=64)
    check(case)
    check(case, force_budget=3001)


def test_eps_delta_guarantee_holds_on_the_cuda_path():
    # Definition 4.1 of the paper on the product path: over many seeds, the relative error of the sparse
    # output against exact attention exceeds eps with frequency at most delta (plus binomial slack)
    import math
    import torch
    from paper_2510_05688_b200 import binding as vb
    eps = delta = 0.1
    case = synth.make_case("guarantee", dtype="fp32", B=1, Hq=8, Hkv=2, d=64, seq_lens=[8192], sink=128, window=128,
                           k=int(0.025 * 8192), eps=eps, delta=delta, seed=0, gen_seed=31337, key_std=0.1,
                           rho_v=2.0, heavy=None, params=dict(base_rate=0.025))
    ref = O.dense_decode(case.q, case.k_cache, case.v_cache, case.block_table, case.seq_lens, dtype=case.dtype)
    dev = vb.case_to_device(case)
    plan = vb.plan_for_case(case)
    plan.set_params(**case.params)
    dbg = plan.enable_debug()
    out = torch.empty_like(dev["q"])
    seeds, fails, trials, used = 128, 0, 0, []
    for seed in range(seeds):
        plan.decode(dev["q"], dev["k_cache"], dev["v_cache"], dev["block_table"], dev["seq_lens"], case.sink, case.window,
                    case.k, case.eps, case.delta, seed, out)
        torch.cuda.synchronize()
        got = out.cpu().numpy().astype(np.float64)
        err = np.linalg.norm(got[0] - ref[0], axis=-1) / np.linalg.norm(ref[0], axis=-1)
        fails += int((err > eps).sum())
        trials += err.size
        used.append(float(dbg["dyn_cnt"].cpu().numpy().mean()))
    n_s = 8192 - 256 - case.k
    assert np.mean(used) < 0.5 * n_s                       # not vacuous: budgets well below the residual
    assert fails / trials <= delta + 3.0 * math.sqrt(delta * (1 - delta) / trials)
    assert plan.last_status() == 0


# ----------------------------------------------------------------------------- the five workloads
def test_config1_tiny():
    case = synth.config1_tiny()
    out, dbg, det, _ = check(case)                 # SDPA mode: the budget saturates at the residual
    check(case, mode=1)                            # denominator mode: a budget below the residual
    assert det[(0, 0)]["b"] == det[(0, 0)]["n_s"]


def test_config2_llama8b_full_size():
    case = synth.config2_llama8b()
    out, dbg, det, _ = check(case)
    dens = np.mean([(len(r["I_f"]) + r["b"]) / r["n"] for r in det.values()])
    assert 0.09 < dens < 0.11                      # the calibrated ~10x sparsity operating point
    assert (dbg["paths"] & 1 == 1).all() and (dbg["paths"] & 4 == 0).all()   # scores in registers, near-ties from the list


def test_config3_uniform_full_size_and_sparsity_sweep():
    case = synth.config3_uniform()
    check(case)
    n_f = 128 + 128 + case.k
    for S in (5, 10, 20):
        check(case, force_budget=round(32768 / S) - n_f)


def test_config4_serving_all_heads():
    case = synth.config4_serving()                 # 32 rows x 32 heads, every one of them compared
    out_ref, det = run_oracle(case)
    out, dbg, _ = run_gpu(case)
    assert len(det) == 1024
    assert_parity(case, out, dbg, det, out_ref)


@pytest.mark.parametrize("n", [1024, 1025, 1039, 1040, 2048, 9000, 32768])
def test_config5_reasoning_steps(n):
    check(synth.config5_reasoning(n=n, B=8))       # batch 8 at every length, as the benchmark times it


def test_nested_base_sample():
    # the base sample read off the final sample's walk (I_bs a subset of I_dyn)
    _, dbg, det, _ = check(small("bf16", [2049, 700, 33], params=dict(base_rate=0.05, nested_base=1)))
    for (b, h), r in det.items():
        if r["n_s"] > 0:
            assert set(dbg["base_idx"][b, h, :r["b0"]].tolist()) <= set(dbg["dyn_idx"][b, h, :r["b"]].tolist())
    check(mid(params=dict(base_rate=0.025, nested_base=1)))


def test_bad_sequence_length_sets_status_and_is_clamped():
    import torch
    from paper_2510_05688_b200 import binding as vb
    case = small("bf16", [200, 300])
    dev = vb.case_to_device(case)
    plan = vb.plan_for_case(case)
    out = torch.empty_like(dev["q"])
    for bad, as_if in ((-3, 0), (plan.shape.max_seq_len + 1, plan.shape.max_seq_len)):
        sl = dev["seq_lens"].clone()
        sl[0] = bad
        plan.decode(dev["q"], dev["k_cache"], dev["v_cache"], dev["block_table"], sl, 4, 8, 16, 0.05, 0.05, 1, out)
        torch.cuda.synchronize()
        assert plan.last_status() & vb.STATUS_BAD_SEQLEN
        got = out.clone()
        sl[0] = as_if                                 # the clamped length gives the same step, without the bit
        plan.decode(dev["q"], dev["k_cache"], dev["v_cache"], dev["block_table"], sl, 4, 8, 16, 0.05, 0.05, 1, out)
        torch.cuda.synchronize()
        assert plan.last_status() == 0
        assert torch.equal(got.view(torch.int16)[1], out.view(torch.int16)[1])
        if as_if == 0:
            assert (got[0] == 0).all()


def test_non_finite_statistics_fall_back_to_the_whole_residual():
    # an infinite V element in one base-sample row: that head's statistics are not finite, its budget becomes the
    # whole residual, the status word says so; the other heads of the step are untouched
    import torch
    from paper_2510_05688_b200 import binding as vb
    case = small("bf16", [900], Hq=4, Hkv=2)
    _, dbg0, plan = run_gpu(case)
    tok = int(dbg0["base_idx"][0, 0, 0])               # a base-sample token of head 0 (KV head 0)
    vc = case.v_cache.copy()
    vc[case.block_table[0, tok // 16], 0, tok % 16, 5] = 0x7F80          # +inf in bf16
    case.v_cache = vc
    out, dbg, plan = run_gpu(case)
    assert plan.last_status() & vb.STATUS_NONFINITE
    n_s = int(dbg["stats"][0, 0, 5])
    assert int(dbg["dyn_cnt"][0, 0]) == n_s and int(dbg["budgets"][0, 0, 3]) == n_s
    assert np.array_equal(dbg["dyn_idx"][0, 2], dbg0["dyn_idx"][0, 2])
    assert np.array_equal(dbg["budgets"][0, 2:], dbg0["budgets"][0, 2:])    # KV head 1 does not see the row


def test_bounded_wait_runs_out_and_the_context_stays_usable():
    # The step's kernels wait for one another's published words with a poll limit.  Here the wait primitive runs
    # alone on a word that nothing publishes: it must give up at its limit (no hang), report that, and leave the
    # context usable: a whole step afterwards still matches the oracle.
    from paper_2510_05688_b200 import binding as vb
    case = small("bf16", [700, 333], Hq=4, Hkv=2)
    plan = vb.plan_for_case(case)
    plan.set_params(**case.params)
    ran_out, waited_us = plan.probe_bounded_wait(2000)
    assert ran_out == 1
    assert 50 <= waited_us <= 200000, waited_us           # 2,000 polls of at least 128 ns each, far below a second
    ran_out2, waited_us2 = plan.probe_bounded_wait(20000)
    assert ran_out2 == 1 and waited_us2 > waited_us
    with pytest.raises(vb.VattnError):
        plan.probe_bounded_wait(0)
    check(case)


def test_budgets_beyond_the_walk_array_and_up_to_the_whole_residual():
    # A small base rate makes the final sample's walk array (about eight base budgets) short, a small eps makes the
    # budgets long: some heads end between the array's end and the whole residual (their entries beyond the array
    # are computed by the gather kernel), others take the whole residual (token order).
    rng = np.random.default_rng(91)
    lens = [int(x) for x in rng.integers(2500, 6000, size=3)]
    case = small("bf16", lens, Hq=8, Hkv=2, sink=8, window=16, k=48)
    case.params = dict(case.params, base_rate=0.01)
    far, whole = 0, 0
    for eps in (0.2, 0.08, 0.03, 0.01):
        case.eps = eps
        out, dbg, det, plan = check(case)
        b = np.asarray(dbg["budgets"])[..., 3].reshape(-1).astype(np.int64)
        b0 = np.asarray(dbg["base_cnt"]).reshape(-1).astype(np.int64)
        n_s = np.asarray(dbg["stats"])[..., 5].reshape(-1).astype(np.int64)
        far += int(((b > 9 * b0) & (b < n_s)).sum())
        whole += int(((b == n_s) & (n_s > 0)).sum())
    assert far > 0 and whole > 0, (far, whole)
    case32 = small("fp32", lens[:2], Hq=4, Hkv=2, sink=8, window=16, k=48)
    case32.params = dict(case32.params, base_rate=0.01)
    case32.eps = 0.05
    check(case32)


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("fp32", 64), ("fp32", 128), ("bf16", 64)])
def test_sampling_keys_per_kv_head(dtype, d):
    # rng_head_is_kv = 1: the heads of a KV-head group walk the middle range in one order (their budgets, nested
    # base samples and top-k members still differ).  Ragged rows, an empty one, group sizes 2, 3, 4 and 8, the nested
    # variant, budgets beyond the walk array and equal to the whole residual.
    lens = [2300, 0, 777, 1500, 33]
    base = dict(base_rate=0.05, rng_head_is_kv=1)
    check(small(dtype, lens, Hq=8, Hkv=2, d=d, params=base))
    check(small(dtype, lens, Hq=8, Hkv=2, d=d, params=dict(base, nested_base=1)))
    check(small(dtype, lens, Hq=8, Hkv=4, d=d, params=base))                      # groups of two heads
    check(small(dtype, lens, Hq=6, Hkv=2, d=d, params=base))                      # groups of three
    check(small(dtype, lens, Hq=8, Hkv=1, d=d, params=base))                      # groups of eight
    case = small(dtype, [4000, 2500], Hq=8, Hkv=2, d=d, sink=8, window=16, k=48, params=dict(base, base_rate=0.01))
    for eps in (0.2, 0.03, 0.01):
        case.eps = eps
        check(case)


def test_config2_with_sampling_keys_per_kv_head():
    case = synth.config2_llama8b()
    case.params = dict(case.params, rng_head_is_kv=1)
    out, dbg, det, plan = check(case)
    case.params = dict(case.params, nested_base=1)
    check(case)


# ----------------------------------------------------------------------------- several query tokens per call
@pytest.mark.parametrize("dtype,d,Tq", [("bf16", 128, 3), ("fp32", 64, 2), ("bf16", 64, 4), ("fp32", 128, 5)])
def test_multi_query_calls(dtype, d, Tq):
    """A question or speculative tokens in one call (App. C, split-prompt setup): query token t sees the first
    n - (Tq - 1 - t) tokens and is decode step `step + t`; sequences shorter than the call leave tokens that see
    nothing.  Groups of Tq * 4 = 8..20 heads per KV head: whole and partial chunks of the score pass."""
    import torch
    case = small(dtype, [1, 17, 255, 600, 2049, 2, 1000], d=d)
    q4 = synth.multi_query(case, Tq)
    out_ref, det = run_oracle_multi(case, q4)
    out, dbg, plan, dev = run_gpu_multi(case, q4)
    assert_parity_multi(case, Tq, out, dbg, det, out_ref)
    assert plan.last_status() == 0
    # the dense comparison kernel with the same causal offsets
    dn = torch.empty_like(dev["q"])
    plan.dense_decode(dev["q"], dev["k_cache"], dev["v_cache"], dev["block_table"], dev["seq_lens"], dn)
    torch.cuda.synchronize()
    ref = O.dense_decode_multi(q4, case.k_cache, case.v_cache, case.block_table, case.seq_lens, dtype=dtype)
    tol = 2e-2 if dtype == "bf16" else 2e-5
    assert (np.abs(dn.float().cpu().numpy() - ref) <= tol * np.maximum(1.0, np.abs(ref))).all()


def test_multi_query_variants():
    case = small("bf16", [900, 350, 77])
    q4 = synth.multi_query(case, 2)
    for over in (dict(mode=1), dict(mode=2), dict(rng_head_is_kv=1, layer=2, step=40), dict(nested_base=1),
                 dict(gather_mode=1), dict(force_budget=10**9), dict(topk_frac=0.03)):
        out_ref, det = run_oracle_multi(case, q4, **over)
        out, dbg, _, _ = run_gpu_multi(case, q4, **over)
        assert_parity_multi(case, 2, out, dbg, det, out_ref)


def test_multi_query_host_buffer_entry_point():
    import torch
    from paper_2510_05688_b200 import binding as vb
    case = small("bf16", [900, 350])
    q4 = synth.multi_query(case, 3)
    out_dev, _, plan, dev = run_gpu_multi(case, q4, debug=False)
    qh = dev["q"].cpu().pin_memory()
    bth = dev["block_table"].cpu().pin_memory()
    slh = dev["seq_lens"].cpu().pin_memory()
    outh = torch.empty_like(qh).pin_memory()
    for _ in range(3):                                   # the third call replays the recorded step
        outh.zero_()
        plan.decode_host(qh, dev["k_cache"], dev["v_cache"], bth, slh, case.sink, case.window, case.k, case.eps,
                         case.delta, case.seed, outh)
        assert np.array_equal(outh.view(torch.int16).numpy().view(np.uint16), out_dev)


def test_multi_query_limits():
    from paper_2510_05688_b200 import binding as vb
    case = small("bf16", [64])                           # 4 heads per KV head: 16 tokens fill the 64 rows of a group
    vb.plan_for_case(case, q_len=16)
    with pytest.raises(vb.VattnError):
        vb.plan_for_case(case, q_len=17)
    shape = vb.plan_for_case(case, q_len=2).shape
    import torch
    dev = vb.case_to_device(case)
    q = torch.zeros(1, 2, 8, 128, dtype=torch.bfloat16, device="cuda")
    assert vb.dense_decode_noalloc(shape, q, dev["k_cache"], dev["v_cache"], dev["block_table"], dev["seq_lens"],
                                   torch.empty_like(q)) == vb.ERR_UNSUPPORTED


def test_multi_query_one_token_is_the_plain_call():
    case = small("bf16", [700, 129])
    out1, dbg1, _, _ = run_gpu_multi(case, np.ascontiguousarray(case.q[:, None]))
    out0, dbg0, _ = run_gpu(case)
    assert np.array_equal(out1[:, 0], out0)
    for key in ("topk_idx", "dyn_idx", "budgets"):
        assert np.array_equal(dbg1[key], dbg0[key])


def test_multi_query_llama8b_layer_sampled_heads():
    """The benchmark layer with four query tokens per call (128 (token, head) pairs, 16 per KV head): sampled pairs
    against the oracle, every output row finite."""
    case = synth.config2_llama8b()
    Tq = 4
    q4 = synth.multi_query(case, Tq)
    heads = [(0, 0, 0), (0, 1, 5), (0, 2, 17), (0, 3, 31), (0, 3, 12), (0, 0, 26)]
    out_ref, det = run_oracle_multi(case, q4, heads=heads)
    out, dbg, plan, _ = run_gpu_multi(case, q4)
    sel = {k: v for k, v in det.items()}
    # compare only the sampled pairs: rows of the others are zero in the oracle's output
    from helpers import virtual_head
    det_v = {(b, virtual_head(case, Tq, t, h)): r for (b, t, h), r in sel.items()}
    B, Hq, dd = case.batch, case.num_q_heads, case.head_dim
    out_v = np.zeros((B, Tq * Hq, dd), out.dtype); ref_v = np.zeros((B, Tq * Hq, dd), out_ref.dtype)
    for (b, t, h) in heads:
        out_v[b, virtual_head(case, Tq, t, h)] = out[b, t, h]
        ref_v[b, virtual_head(case, Tq, t, h)] = out_ref[b, t, h]
    assert_parity(case, out_v, dbg, det_v, ref_v)
    assert np.isfinite(out_values(case, out)).all() and plan.last_status() == 0
