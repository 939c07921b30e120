"""The dense-decode entry point that allocates nothing, for callers that cannot allocate.

A serving engine that gave the whole GPU to its KV-cache pool, or code that must not call cudaMalloc on
its path, cannot create a plan workspace.  vattn_dense_decode_noalloc keeps its scratch in a fixed array
inside the library instead.  This test calls it through the C ABI twice in a row (the array keeps the
previous call's contents, so the second call proves the clearing) and compares each result with the
ordinary entry point and with the CPU reference of dense attention, within the tolerance the dense
parity test uses.  It lives in a file pytest collects last, so a failure here cannot hide any other
test under -x.
"""
import numpy as np
import pytest

from oracle import vattn_oracle as O
from paper_2510_05688_b200 import synth

pytestmark = pytest.mark.gpu


def _case(dtype, d, seq_lens, gen_seed):
    return synth.make_case("noalloc", dtype=dtype, B=len(seq_lens), Hq=8, Hkv=2, d=d, seq_lens=list(seq_lens), sink=4,
                           window=8, k=16, eps=0.05, delta=0.05, seed=1, gen_seed=gen_seed, rho_v=1.0,
                           heavy=dict(R=12, c1=5.0, alpha=(0.75, 1.25)))


def test_noalloc_dense_matches_planned_dense_on_two_calls_in_a_row():
    import torch
    from paper_2510_05688_b200 import binding as vb
    cases = [_case("bf16", 128, [2049, 1, 700, 0], 11), _case("fp32", 64, [333, 1500], 12)]
    for case in cases:                                       # second case = second call on a used array
        dev = vb.case_to_device(case)
        plan = vb.plan_for_case(case)
        ref = torch.empty_like(dev["q"])
        plan.dense_decode(dev["q"], dev["k_cache"], dev["v_cache"], dev["block_table"], dev["seq_lens"], ref)
        cpu = O.dense_decode(case.q, case.k_cache, case.v_cache, case.block_table, case.seq_lens, dtype=case.dtype)
        for call in range(2):
            out = torch.full_like(dev["q"], 7.0)
            rc = vb.dense_decode_noalloc(plan.shape, dev["q"], dev["k_cache"], dev["v_cache"], dev["block_table"],
                                         dev["seq_lens"], out)
            assert rc == vb.OK
            torch.cuda.synchronize()
            a, b = out.float().cpu().numpy().astype(np.float64), ref.float().cpu().numpy().astype(np.float64)
            tol = 2e-2 if case.dtype == "bf16" else 2e-5
            assert (np.abs(a - b) <= tol * np.maximum(1.0, np.abs(b))).all(), (case.dtype, call, np.abs(a - b).max())
            assert (np.abs(a - cpu) <= tol * np.maximum(1.0, np.abs(cpu))).all(), (case.dtype, call, np.abs(a - cpu).max())


def test_noalloc_rejects_problems_beyond_the_fixed_scratch():
    import torch
    from paper_2510_05688_b200 import binding as vb
    case = _case("bf16", 128, [64], 13)
    dev = vb.case_to_device(case)
    out = torch.empty_like(dev["q"])
    big = vb.Shape(4096, 8, 2, 128, 16, case.max_blocks_per_seq, case.num_blocks, 64, vb.DTYPE_BF16, 0, 0, 0)
    need = 256 + 12 * 4096 * 8 + 4096 * 8 * 130 * 4
    assert need > vb.NOALLOC_SCRATCH_BYTES
    rc = vb.dense_decode_noalloc(big, dev["q"], dev["k_cache"], dev["v_cache"], dev["block_table"], dev["seq_lens"], out)
    assert rc == vb.ERR_WORKSPACE
    bad = vb.Shape(1, 8, 2, 96, 16, case.max_blocks_per_seq, case.num_blocks, 64, vb.DTYPE_BF16, 0, 0, 0)
    assert vb.dense_decode_noalloc(bad, dev["q"], dev["k_cache"], dev["v_cache"], dev["block_table"], dev["seq_lens"],
                                   out) == vb.ERR_UNSUPPORTED


def test_noalloc_status_word_reports_a_bad_block_table_entry():
    import torch
    from paper_2510_05688_b200 import binding as vb
    case = _case("bf16", 128, [700, 90], 14)
    dev = vb.case_to_device(case)
    plan = vb.plan_for_case(case)
    out = torch.empty_like(dev["q"])
    assert vb.dense_decode_noalloc(plan.shape, dev["q"], dev["k_cache"], dev["v_cache"], dev["block_table"],
                                   dev["seq_lens"], out) == vb.OK
    assert vb.noalloc_last_status() == 0
    bt = dev["block_table"].clone()
    bt[0, 3] = case.num_blocks + 5                           # outside the pool: read as page 0, reported
    assert vb.dense_decode_noalloc(plan.shape, dev["q"], dev["k_cache"], dev["v_cache"], bt, dev["seq_lens"], out) == vb.OK
    assert vb.noalloc_last_status() & vb.STATUS_BAD_BLOCK
    # the next call starts from a clean word
    assert vb.dense_decode_noalloc(plan.shape, dev["q"], dev["k_cache"], dev["v_cache"], dev["block_table"],
                                   dev["seq_lens"], out) == vb.OK
    assert vb.noalloc_last_status() == 0
