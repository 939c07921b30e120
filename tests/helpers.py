"""Shared test helpers: run the CUDA path through the C ABI and compare it with the oracle."""
import numpy as np

from oracle import vattn_oracle as O

BF16_TOL = 2e-2      # absolute-or-relative, bf16 outputs
FP32_REL = 1e-5      # relative to the head's largest |output|, fp32 outputs


def run_oracle(case, heads=None, **over):
    p = dict(case.params)
    p.update(over)
    p.pop("gather_mode", None)          # where the weights are read from is not part of what is computed
    return O.vattn_decode(case.q, case.k_cache, case.v_cache, case.block_table, case.seq_lens, case.sink,
                          case.window, case.k, case.eps, case.delta, case.seed, dtype=case.dtype, heads=heads, **p)


def run_gpu(case, debug=True, plan=None, dev=None, **over):
    """One vattn_decode call through the C ABI.  Returns (out as numpy, debug dict of numpy arrays, plan)."""
    import torch
    from paper_2510_05688_b200 import binding as vb
    p = dict(case.params)
    p.update(over)
    if dev is None:
        dev = vb.case_to_device(case)
    if plan is None:
        plan = vb.plan_for_case(case)
    plan.set_params(**p)
    dbg = plan.enable_debug() if debug else None
    out = torch.empty_like(dev["q"])
    plan.decode(dev["q"], dev["k_cache"], dev["v_cache"], dev["block_table"], dev["seq_lens"], case.sink, case.window,
                case.k, case.eps, case.delta, case.seed, out)
    torch.cuda.synchronize()
    if case.dtype == "bf16":
        out_np = out.view(torch.int16).cpu().numpy().view(np.uint16)
    else:
        out_np = out.cpu().numpy()
    dbg_np = {k: v.cpu().numpy() for k, v in dbg.items()} if dbg else None
    return out_np, dbg_np, plan


def virtual_head(case, q_len, t, h):
    """Index of (query token t, head h) on the head axis of the introspection arrays of a q_len > 1 plan:
    [KV head, query token, head within the group] flattened."""
    G1 = case.num_q_heads // case.num_kv_heads
    return (h // G1) * (q_len * G1) + t * G1 + (h % G1)


def run_oracle_multi(case, q4, heads=None, **over):
    p = dict(case.params)
    p.update(over)
    p.pop("gather_mode", None)
    return O.vattn_decode_multi(q4, case.k_cache, case.v_cache, case.block_table, case.seq_lens, case.sink, case.window,
                                case.k, case.eps, case.delta, case.seed, dtype=case.dtype, heads=heads, **p)


def run_gpu_multi(case, q4, debug=True, **over):
    """One call with q4 [B,Tq,Hq,d] through the C ABI.  Returns (out [B,Tq,Hq,d] numpy, debug dict, plan)."""
    import torch
    from paper_2510_05688_b200 import binding as vb
    p = dict(case.params)
    p.update(over)
    Tq = q4.shape[1]
    dev = vb.case_to_device(case)
    if case.dtype == "bf16":
        qd = torch.from_numpy(np.ascontiguousarray(q4).view(np.int16)).cuda().view(torch.bfloat16)
    else:
        qd = torch.from_numpy(np.ascontiguousarray(q4)).cuda()
    plan = vb.plan_for_case(case, q_len=Tq)
    plan.set_params(**p)
    dbg = plan.enable_debug() if debug else None
    out = torch.empty_like(qd)
    plan.decode(qd, dev["k_cache"], dev["v_cache"], dev["block_table"], dev["seq_lens"], case.sink, case.window,
                case.k, case.eps, case.delta, case.seed, out)
    torch.cuda.synchronize()
    out_np = out.view(torch.int16).cpu().numpy().view(np.uint16) if case.dtype == "bf16" else out.cpu().numpy()
    dbg_np = {k: v.cpu().numpy() for k, v in dbg.items()} if dbg else None
    return out_np, dbg_np, plan, dict(dev, q=qd)


def assert_parity_multi(case, q_len, out, dbg, det, out_ref, check_scores=True):
    """assert_parity with (b, t, h) mapped onto the plan's head axis."""
    B, Hq, d = case.batch, case.num_q_heads, case.head_dim
    det_v = {(b, virtual_head(case, q_len, t, h)): r for (b, t, h), r in det.items()}
    out_v = np.zeros((B, q_len * Hq, d), out.dtype)
    ref_v = np.zeros((B, q_len * Hq, d), out_ref.dtype)
    for t in range(q_len):
        for h in range(Hq):
            hv = virtual_head(case, q_len, t, h)
            out_v[:, hv] = out[:, t, h]
            ref_v[:, hv] = out_ref[:, t, h]
    assert_parity(case, out_v, dbg, det_v, ref_v, check_scores=check_scores)


def out_values(case, out):
    if case.dtype == "bf16":
        return (np.asarray(out, np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    return np.asarray(out, np.float64)


def assert_out_close(case, got, want, where=""):
    g, w = out_values(case, got), out_values(case, want)
    if case.dtype == "bf16":
        bad = np.abs(g - w) > BF16_TOL * np.maximum(1.0, np.abs(w))
        assert not bad.any(), f"{where}: bf16 output off by {np.abs(g - w).max():.3e}"
    else:
        ref = np.abs(w).max(axis=-1, keepdims=True)
        err = np.abs(g - w) / np.maximum(ref, 1e-30)
        assert err.max() <= FP32_REL, f"{where}: fp32 output rel err {err.max():.3e}"


def assert_parity(case, out, dbg, det, out_ref, check_scores=True):
    """Bit-exact index sets, budgets and samples; outputs within tolerance, for every head in `det`."""
    for (b, h), r in det.items():
        tag = f"{case.name} b={b} h={h}"
        n = r["n"]
        if n == 0:
            assert dbg["topk_cnt"][b, h] == 0 and dbg["dyn_cnt"][b, h] == 0, tag
            continue
        kk = int(dbg["topk_cnt"][b, h])
        assert kk == len(r["I_t"]), f"{tag}: |I_t| {kk} vs {len(r['I_t'])}"
        assert np.array_equal(dbg["topk_idx"][b, h, :kk], r["I_t"]), f"{tag}: I_t differs"
        b0 = int(dbg["base_cnt"][b, h])
        assert b0 == r["b0"], f"{tag}: b0 {b0} vs {r['b0']}"
        assert np.array_equal(np.sort(dbg["base_idx"][b, h, :b0]), r["I_bs"]), f"{tag}: I_bs differs"
        assert tuple(int(x) for x in dbg["budgets"][b, h]) == tuple(r["budgets"]), \
            f"{tag}: budgets {dbg['budgets'][b, h]} vs {r['budgets']}"
        bb = int(dbg["dyn_cnt"][b, h])
        assert bb == r["b"], tag
        # the set is unique; its order is a representation (ascending key or ascending token)
        assert np.array_equal(np.sort(dbg["dyn_idx"][b, h, :bb]), r["I_dyn"]), f"{tag}: I_dyn differs"
        st, sr = dbg["stats"][b, h], r["stats"]
        assert st[5] == sr[5] and st[6] == sr[6], tag
        np.testing.assert_allclose(st[7], sr[7], rtol=2e-6, atol=1e-4, err_msg=tag)     # m is an fp32 score
        # weights are relative to each side's own m: compare the m-free ratios
        sc = np.exp(sr[7] - st[7])
        np.testing.assert_allclose(st[0] * 1.0, sr[0] * sc, rtol=1e-9, err_msg=tag + " D_f")
        np.testing.assert_allclose(st[3], sr[3] * sc, rtol=1e-9, err_msg=tag + " D_hat")
        np.testing.assert_allclose(st[4], sr[4] * sc, rtol=1e-9, atol=1e-300, err_msg=tag + " N_hat")
        np.testing.assert_allclose(st[1], sr[1] * sc * sc, rtol=1e-7, atol=1e-30, err_msg=tag + " sigma2")
        np.testing.assert_allclose(st[2], sr[2] * sc * sc, rtol=1e-7, atol=1e-30, err_msg=tag + " trace")
        if check_scores:
            s32 = dbg["scores"][b, h, :n].astype(np.float64)
            assert np.abs(s32 - r["scores"]).max() <= 2e-5 * max(1.0, np.abs(r["scores"]).max()), tag + " scores"
    idx = sorted(det.keys())
    bs = np.array([i[0] for i in idx]); hs = np.array([i[1] for i in idx])
    assert_out_close(case, np.asarray(out)[bs, hs], np.asarray(out_ref)[bs, hs], case.name)
