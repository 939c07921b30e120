"""GPU parity on seeded random small problems: shapes, lengths, index-set sizes, (eps, delta), parameter switches
and the number of query tokens per call drawn at random, each compared with the oracle like the fixed cases.

The fixed tests choose their shapes by hand; this sweep reaches the combinations nobody thought of (the first one
it found: a middle range of nine tokens that held none of the tokens the selection samples for its threshold
estimate).  The plans of one sweep are created one after another in one process, so a kernel that reads scratch
it has not written meets whatever the plan before it left there.
"""
import numpy as np
import pytest

from paper_2510_05688_b200 import synth
from helpers import (assert_out_close, assert_parity, assert_parity_multi, run_gpu, run_gpu_multi, run_oracle,
                     run_oracle_multi)

pytestmark = pytest.mark.gpu

LENGTHS = [0, 1, 2, 15, 16, 17, 31, 33, 64, 100, 255, 256, 257, 500, 777, 1024, 1500, 2049, 3000]


def draw_case(rng):
    dtype = str(rng.choice(["bf16", "fp32"]))
    d = int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 3, 4]))
    G = int(rng.choice([1, 2, 3, 4, 5, 8]))
    B = int(rng.integers(1, 6))
    lens = [int(x) for x in rng.choice(LENGTHS, size=B)]
    params = dict(base_rate=float(rng.choice([0.025, 0.05, 0.1, 0.3])))
    if rng.random() < 0.3:
        params["topk_frac"] = float(rng.choice([0.01, 0.03, 0.1]))
    if rng.random() < 0.3:
        params["mode"] = int(rng.integers(0, 3))
    if rng.random() < 0.3:
        params["rng_head_is_kv"] = 1
    if rng.random() < 0.3:
        params["nested_base"] = 1
    if rng.random() < 0.2:
        params["gather_mode"] = 1
    if rng.random() < 0.3:
        params["step"] = int(rng.integers(0, 100000))
        params["layer"] = int(rng.integers(0, 64))
    if rng.random() < 0.15:
        params["force_budget"] = int(rng.choice([0, 5, 100, 10**9]))
    heavy = None if rng.random() < 0.3 else dict(R=int(rng.integers(1, 20)), c1=float(rng.choice([2.0, 5.0, 9.0])),
                                                 alpha=(0.75, 1.25))
    q_len = int(rng.choice([1, 1, 1, 2, 3, 4]))
    case = synth.make_case("random", dtype=dtype, B=B, Hq=Hkv * G, Hkv=Hkv, d=d, seq_lens=lens,
                           sink=int(rng.choice([0, 1, 4, 16, 128])), window=int(rng.choice([0, 1, 8, 16, 128])),
                           k=int(rng.choice([0, 1, 7, 16, 64, 300, 100000])),
                           eps=float(rng.choice([0.02, 0.05, 0.1, 0.3])), delta=float(rng.choice([0.01, 0.05, 0.2])),
                           seed=int(rng.integers(0, 2**31)), gen_seed=int(rng.integers(0, 2**31)), key_std=1.0,
                           rho_v=1.0, heavy=heavy, params=params)
    return case, q_len


@pytest.mark.parametrize("sweep", [1, 2])
def test_random_problems_with_introspection(sweep):
    """Index sets, budgets, statistics and outputs (the introspection switches on the list-building paths)."""
    for it in range(40):
        case, q_len = draw_case(np.random.default_rng(sweep * 100003 + it))
        if q_len == 1:
            out_ref, det = run_oracle(case)
            out, dbg, plan = run_gpu(case)
            assert_parity(case, out, dbg, det, out_ref)
        else:
            q4 = synth.multi_query(case, q_len)
            out_ref, det = run_oracle_multi(case, q4)
            out, dbg, plan, _ = run_gpu_multi(case, q4)
            assert_parity_multi(case, q_len, out, dbg, det, out_ref)
        assert plan.last_status() & ~4 == 0, (sweep, it)


def test_random_problems_outputs_only():
    """Without introspection the samples are read off the walk arrays (no lists): outputs against the oracle."""
    for it in range(40):
        case, q_len = draw_case(np.random.default_rng(31 * 100003 + it))
        if q_len == 1:
            out_ref, _ = run_oracle(case)
            out, _, plan = run_gpu(case, debug=False)
        else:
            q4 = synth.multi_query(case, q_len)
            out_ref, _ = run_oracle_multi(case, q4)
            out, _, plan, _ = run_gpu_multi(case, q4, debug=False)
        assert_out_close(case, out.reshape(out_ref.shape), out_ref, f"outputs only, case {it}")
        assert plan.last_status() & ~4 == 0, it


def test_random_dense_problems():
    """The dense comparison kernels on random shapes: group sizes 1..16 (both tile widths), batches up to 19 mixed
    lengths, one to four query tokens, twice in a row (the kernel puts its counters back), and the entry point that
    allocates nothing where it applies."""
    import torch
    from oracle import vattn_oracle as O
    from paper_2510_05688_b200 import binding as vb
    lengths = LENGTHS + [5000, 9001]
    for it in range(40):
        rng = np.random.default_rng(7 * 7919 + it)
        dtype = str(rng.choice(["bf16", "bf16", "fp32"]))
        d = int(rng.choice([64, 128]))
        Hkv = int(rng.choice([1, 2, 3, 4, 8]))
        G = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 9, 12, 16]))
        B = int(rng.integers(1, 20))
        lens = [int(x) for x in rng.choice(lengths, size=B)]
        q_len = int(rng.choice([1, 1, 2, 3, 4]))
        case = synth.make_case("random_dense", dtype=dtype, B=B, Hq=Hkv * G, Hkv=Hkv, d=d, seq_lens=lens, sink=4,
                               window=4, k=4, eps=0.1, delta=0.1, seed=1, gen_seed=int(rng.integers(0, 2**31)),
                               key_std=1.0, rho_v=1.0, heavy=None, params={})
        q4 = synth.multi_query(case, q_len)
        dev = vb.case_to_device(case)
        if dtype == "bf16":
            qd = torch.from_numpy(np.ascontiguousarray(q4).view(np.int16)).cuda().view(torch.bfloat16)
        else:
            qd = torch.from_numpy(np.ascontiguousarray(q4)).cuda()
        plan = vb.plan_for_case(case, q_len=q_len)
        ref = O.dense_decode_multi(q4, case.k_cache, case.v_cache, case.block_table, case.seq_lens, dtype=dtype)
        tol = 2e-2 if dtype == "bf16" else 2e-5
        bits = torch.int16 if dtype == "bf16" else torch.int32
        outs = []
        for _ in range(2):
            out = torch.empty_like(qd)
            plan.dense_decode(qd, dev["k_cache"], dev["v_cache"], dev["block_table"], dev["seq_lens"], out)
            torch.cuda.synchronize()
            got = out.float().cpu().numpy().astype(np.float64)
            assert (np.abs(got - ref) <= tol * np.maximum(1.0, np.abs(ref))).all(), (it, np.abs(got - ref).max())
            outs.append(out)
        assert torch.equal(outs[0].view(bits), outs[1].view(bits)) and plan.last_status() == 0, it
        if q_len == 1:
            out = torch.empty_like(dev["q"])
            rc = vb.dense_decode_noalloc(plan.shape, dev["q"], dev["k_cache"], dev["v_cache"], dev["block_table"],
                                         dev["seq_lens"], out)
            torch.cuda.synchronize()
            assert rc in (vb.OK, vb.ERR_WORKSPACE), rc
            if rc == vb.OK:
                got = out.float().cpu().numpy().astype(np.float64)
                assert (np.abs(got - ref[:, 0]) <= tol * np.maximum(1.0, np.abs(ref[:, 0]))).all(), it


def test_random_calls_on_one_plan():
    """A decode loop: one plan and one cache, every call with other lengths (empty sequences included), index-set
    sizes, (eps, delta), seeds and switches.  What a call leaves in the workspace must not reach the next one."""
    import copy
    import torch
    from paper_2510_05688_b200 import binding as vb
    for it in range(12):
        rng = np.random.default_rng(1 * 15485863 + 20 + it)          # (session 27 of this stream found the prefix search's step limit)
        dtype = str(rng.choice(["bf16", "fp32"]))
        d = int(rng.choice([64, 128]))
        Hkv = int(rng.choice([1, 2, 4]))
        G = int(rng.choice([1, 2, 4, 8]))
        B = int(rng.integers(1, 6))
        maxlens = [int(x) for x in rng.choice([64, 300, 1000, 2049, 4000], size=B)]
        base = synth.make_case("one_plan", dtype=dtype, B=B, Hq=Hkv * G, Hkv=Hkv, d=d, seq_lens=maxlens, sink=4,
                               window=8, k=16, eps=0.05, delta=0.05, seed=1, gen_seed=int(rng.integers(0, 2**31)),
                               key_std=1.0, rho_v=1.0, heavy=dict(R=12, c1=5.0, alpha=(0.75, 1.25)),
                               params=dict(base_rate=0.05))
        dev = vb.case_to_device(base)
        plan = vb.plan_for_case(base)
        for step in range(8):
            case = copy.copy(base)
            lens = np.array([int(rng.integers(0, m + 1)) if rng.random() < 0.8 else int(rng.choice([0, 1, 15, 16, 17, m]))
                             for m in maxlens], np.int32)
            case.seq_lens = lens
            case.sink = int(rng.choice([0, 1, 4, 64]))
            case.window = int(rng.choice([0, 1, 8, 64]))
            case.k = int(rng.choice([0, 1, 16, 200, 100000]))
            case.eps = float(rng.choice([0.02, 0.05, 0.3]))
            case.delta = float(rng.choice([0.01, 0.05, 0.2]))
            case.seed = int(rng.integers(0, 2**31))
            params = dict(base_rate=float(rng.choice([0.025, 0.1, 0.3])), step=step)
            if rng.random() < 0.3:
                params["nested_base"] = 1
            if rng.random() < 0.3:
                params["rng_head_is_kv"] = 1
            if rng.random() < 0.2:
                params["gather_mode"] = 1
            if rng.random() < 0.2:
                params["force_budget"] = int(rng.choice([0, 7, 10**9]))
            if rng.random() < 0.3:
                params["topk_frac"] = float(rng.choice([0.01, 0.1]))
            case.params = params
            out_ref, det = run_oracle(case)
            out, dbg, _ = run_gpu(case, plan=plan, dev=dict(dev, seq_lens=torch.from_numpy(lens).cuda()))
            assert_parity(case, out, dbg, det, out_ref)
            assert plan.last_status() & ~4 == 0, (it, step)
