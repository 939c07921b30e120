#!/usr/bin/env python
"""Benchmark of the verified sparse-attention decode step (one step = one pass of the whole hot path:
score pass; top-k selection and sample lists; statistics rows; budget, final sample and combination) on
the Llama-3.1-8B-shaped layer
at 32K context and ~10x sparsity.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is microseconds per decode-attention step with inputs resident
in HBM (CUDA-graph replays, rotating over distinct cache pools so no replay sees a warm L2); `e2e`
is the same step through the host-buffer entry point (pinned host q / block table / seq_lens in, out
back); `roofline` is the dominant kernel against the measured HBM copy bandwidth; `cpu_baseline` is the
fp64 CPU oracle timed on this machine.  With --impl reference the oracle itself is the timed program.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np

METRIC = "decode_attention_us_per_step"
UNIT = "us"
POOLS = 4
WORKLOAD = ("cfg2_llama8b: B=1, Hq=32, Hkv=8 (GQA 4), d=128, n=32768, bf16 paged KV (block 16, HND, permuted "
            "block table), sink=window=128, k=819 (2.5%), f_b=0.025, eps=delta=0.05, heavy-hitter strength c1=9.85")


def read_traffic():
    """DRAM bytes per launch (read + write) of each kernel on this workload, from the tracked ncu summary
    profiles/dram_traffic_cfg2.txt (lines `kernel bytes`; the header names the commit it was captured at)."""
    path = os.path.join(ROOT, "profiles", "dram_traffic_cfg2.txt")
    vals, note = {}, "none: no ncu capture of the current kernels has been summarised"
    if os.path.exists(path):
        for ln in open(path):
            if ln.startswith("#"):
                if "captured at" in ln:
                    note = ln.lstrip("# ").strip()
                continue
            parts = ln.split()
            if len(parts) >= 2:
                vals[parts[0]] = float(parts[1])
    return vals, note


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler(threading.Thread):
    """Polls SM clock and throttle reasons through NVML (read-only) while a region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.samples, self.stop_flag, self.mark = index, [], False, None
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.max_mhz = None

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self.stop_flag:
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                try:
                    reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    reasons = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.samples.append((time.perf_counter(), mhz, int(reasons)))
            except Exception:
                pass
            time.sleep(0.002)

    def summary(self, t0, t1):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        sel = [s for s in self.samples if t0 <= s[0] <= t1] or self.samples[-3:]
        names = {0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x10: "sync_boost",
                 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
                 0x100: "display_clock_setting"}
        bits = 0
        for s in sel:
            bits |= s[2]
        return {"sm_mhz": float(np.median([s[1] for s in sel])), "sm_max_mhz": self.max_mhz,
                "reasons": [n for b, n in names.items() if bits & b], "samples": len(sel)}


def oracle_step(case, heads=None):
    from oracle import vattn_oracle as O
    return O.vattn_decode(case.q, case.k_cache, case.v_cache, case.block_table, case.seq_lens, case.sink, case.window,
                          case.k, case.eps, case.delta, case.seed, dtype=case.dtype, heads=heads, **case.params)


def cpu_seconds():
    t = os.times()
    return t.user + t.system


def cores_used(cpu_s, wall_s):
    """Average number of host threads the timed oracle section kept busy (CPU time / wall time)."""
    return round(max(1.0, cpu_s / max(wall_s, 1e-9)), 1)


def run_reference(args, rank, world):
    """The CPU oracle as the timed program: each step is one query head of the workload (1/32 of a
    full step), scaled to a full step; the step count is cut if the run would exceed ~3 minutes."""
    if rank != 0:
        return
    from paper_2510_05688_b200 import synth
    case = synth.config2_llama8b()
    heads_all = [(0, h) for h in range(case.num_q_heads)]
    t0 = time.perf_counter()
    oracle_step(case, heads=[heads_all[0]])
    t_one = time.perf_counter() - t0
    budget_s = 150.0
    steps = max(1, min(args.steps, int(budget_s / max(t_one, 1e-3)) - args.warmup))
    warm = args.warmup
    for i in range(warm):
        oracle_step(case, heads=[heads_all[i % len(heads_all)]])
    t0, c0 = time.perf_counter(), cpu_seconds()
    for i in range(steps):
        oracle_step(case, heads=[heads_all[i % len(heads_all)]])
    dt = time.perf_counter() - t0
    ncores = cores_used(cpu_seconds() - c0, dt)
    us_full = dt / steps * len(heads_all) * 1e6
    sample = (f"each step = 1 of {len(heads_all)} query heads of the workload (K/V de-paging of its KV head "
              f"included), time scaled x{len(heads_all)}; {steps} of the requested {args.steps} steps timed")
    line = {"impl": "reference", "metric": METRIC, "value": us_full, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": warm, "ms_per_step": us_full / 1e3, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": {"workload": WORKLOAD},
            "cpu_baseline": {"value": us_full, "unit": UNIT, "cores": ncores, "host_cores": os.cpu_count(),
                             "kind": "oracle", "sample": sample},
            "e2e": {"value": us_full, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def time_other_configs(vb, synth, torch, steps=40, pools=3):
    """Sparse step and own dense kernel on the other workload configurations (plain launches back to
    back on the current stream, rotating over `pools` copies of the cache so the L2 is not warm)."""
    out = {}

    def run(name, case, **over):
        dev0 = vb.case_to_device(case)
        devs = [dev0] + [dict(dev0, k_cache=dev0["k_cache"].clone(), v_cache=dev0["v_cache"].clone())
                         for _ in range(pools - 1)]
        plan = vb.plan_for_case(case)
        params = dict(case.params)
        params.update(over)
        plan.set_params(**params)
        o = torch.empty_like(dev0["q"])
        dbg = plan.enable_debug()

        def sparse(i):
            d = devs[i % pools]
            plan.decode(d["q"], d["k_cache"], d["v_cache"], d["block_table"], d["seq_lens"], case.sink, case.window,
                        case.k, case.eps, case.delta, case.seed, o)

        def dense(i):
            d = devs[i % pools]
            plan.dense_decode(d["q"], d["k_cache"], d["v_cache"], d["block_table"], d["seq_lens"], o)
        sparse(0)
        torch.cuda.synchronize()
        n = case.seq_lens.astype(np.float64)[:, None]
        dens = float(np.mean((dbg["topk_cnt"].cpu().numpy() + min(case.sink, int(n.max())) + min(case.window, int(n.max()))
                              + dbg["dyn_cnt"].cpu().numpy())[case.seq_lens > 0] / n[case.seq_lens > 0]))
        plan.disable_debug()
        res = {"mean_density": round(dens, 4)}
        for label, fn in (("sparse_us", sparse), ("dense_us", dense)):
            for i in range(3):
                fn(i)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(steps):
                fn(i)
            e1.record()
            torch.cuda.synchronize()
            res[label] = round(e0.elapsed_time(e1) / steps * 1e3, 1)
        plan.set_profiling(True)
        for i in range(10):
            sparse(i)
        torch.cuda.synchronize()
        prof, calls = plan.read_profile()
        plan.set_profiling(False)

        # the score pass alone, launched back to back (no events in between)
        plan.set_stop_after(1)
        for i in range(3):
            sparse(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(steps):
            sparse(i)
        e1.record()
        torch.cuda.synchronize()
        plan.set_stop_after(0)
        res["k_score_alone_us"] = round(e0.elapsed_time(e1) / steps * 1e3, 1)
        res["k_score_alone_gbs"] = round((float(case.seq_lens.sum()) * case.num_kv_heads * case.head_dim *
                                          (2 if case.dtype == "bf16" else 4) + float(case.seq_lens.sum()) *
                                          case.num_q_heads * 4) / (res["k_score_alone_us"] * 1e-6) / 1e9, 1)
        res["kernels_us"] = {k_: round(v / max(calls, 1) * 1e3, 1) for k_, v in prof.items()}
        out[name] = res
        del devs, plan

    run("cfg1_tiny", synth.config1_tiny())
    c3 = synth.config3_uniform()
    n_f = 128 + 128 + c3.k
    run("cfg3_uniform_natural", c3)
    for S in (5, 10, 20):
        run(f"cfg3_uniform_{S}x", c3, force_budget=round(32768 / S) - n_f)
    run("cfg5_reasoning_B8_n32768", synth.config5_reasoning(n=32768, B=8))
    run("cfg4_serving_B32", synth.config4_serving(), )
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing leg")
    ap.add_argument("--flashinfer", action="store_true",
                    help="also time FlashInfer's paged batch decode (third-party dense kernel) as external context")
    ap.add_argument("--all-configs", action="store_true",
                    help="also time the other workload configurations (tiny, near-uniform sweep, batched serving, "
                         "reasoning-length) and add them to the JSON line as `other_configs`")
    ap.add_argument("--profile-only", action="store_true",
                    help="run only warm-up + a few plain (non-graph) steps: the command ncu captures")
    ap.add_argument("--profile-dense", action="store_true",
                    help="with --profile-only: every step is followed by the dense comparison kernel on the same inputs")
    ap.add_argument("--profile-qlen", type=int, default=1,
                    help="with --profile-only: query tokens per sequence and call (vattn_shape.q_len)")
    ap.add_argument("--profile-config", default="cfg2", choices=["cfg2", "cfg5", "cfg4"],
                    help="with --profile-only: the workload to run (cfg5: batch 8 at n=32768; cfg4: batch 32, mixed "
                         "lengths; one cache pool each, 1.1 GB and 2.6 GB)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if not args.profile_only else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import torch
    import torch.distributed as dist
    from paper_2510_05688_b200 import binding as vb
    from paper_2510_05688_b200 import build as vbuild
    from paper_2510_05688_b200 import synth
    from paper_2510_05688_b200.shard import max_over_ranks

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        vbuild.build()
    if world > 1:
        dist.barrier()
    vb.lib()

    # ---- workload: every rank runs its own copy of the layer (weak scaling, no exchange on the path)
    case = synth.config2_llama8b()
    npools = POOLS
    if args.profile_only and args.profile_config != "cfg2":
        case = {"cfg5": synth.config5_reasoning, "cfg4": synth.config4_serving}[args.profile_config]()
        npools = 1                                         # the cache alone is several times the L2
    dev0 = vb.case_to_device(case)
    q_len = args.profile_qlen if args.profile_only else 1
    if q_len > 1:                                          # several query tokens per call: q is [B, q_len, Hq, d]
        dev0["q"] = torch.from_numpy(np.ascontiguousarray(synth.multi_query(case, q_len)).view(np.int16)).cuda().view(
            torch.bfloat16)
    pools = [dev0] + [{k: v.clone() for k, v in dev0.items()} for _ in range(npools - 1)]
    plan = vb.plan_for_case(case, q_len=q_len)
    plan.set_params(**case.params)
    outs = [torch.empty_like(dev0["q"]) for _ in range(POOLS)]
    stream = torch.cuda.Stream()

    def step(i, dense=False):
        d = pools[i % npools]
        if dense:
            plan.dense_decode(d["q"], d["k_cache"], d["v_cache"], d["block_table"], d["seq_lens"], outs[i % POOLS],
                              stream=stream)
        else:
            plan.decode(d["q"], d["k_cache"], d["v_cache"], d["block_table"], d["seq_lens"], case.sink, case.window,
                        case.k, case.eps, case.delta, case.seed, outs[i % POOLS], stream=stream)

    with torch.cuda.stream(stream):
        for i in range(args.warmup):
            step(i)
        stream.synchronize()
        if args.profile_only:
            for i in range(max(1, args.steps)):
                step(i)
                if args.profile_dense:
                    step(i, dense=True)
            stream.synchronize()
            if rank == 0:
                print(json.dumps({"profile_only": True, "steps": args.steps, "launches_per_step": plan.last_launch_count()}))
            return

        # one debug call for budgets / density (not timed)
        dbg = plan.enable_debug()
        step(0)
        stream.synchronize()
        b_dyn = dbg["dyn_cnt"].cpu().numpy().astype(np.int64)
        b0s = dbg["base_cnt"].cpu().numpy().astype(np.int64)
        kks = dbg["topk_cnt"].cpu().numpy().astype(np.int64)
        status = plan.last_status(stream)
        plan.disable_debug()
        launches_per_step = plan.last_launch_count()

        # CUDA graphs: one per pool, for the sparse step and for the dense comparison
        def capture(dense):
            graphs = []
            for i in range(POOLS):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    step(i, dense)
                graphs.append(g)
            return graphs

        def timed(graphs, steps, warm):
            for i in range(warm):
                graphs[i % POOLS].replay()
            stream.synchronize()
            if world > 1:
                dist.barrier()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0 = time.perf_counter()
            e0.record(stream)
            for i in range(steps):
                graphs[i % POOLS].replay()
            e1.record(stream)
            torch.cuda.synchronize()
            t1 = time.perf_counter()
            if world > 1:
                dist.barrier()
            return e0.elapsed_time(e1) / steps, t0, t1

        sparse_graphs = capture(False)
        dense_graphs = capture(True)
        sampler = ClockSampler(local)
        sampler.start()
        ms_step, t0, t1 = timed(sparse_graphs, args.steps, args.warmup)
        sampler.stop_flag = True
        sampler.join(timeout=2.0)
        clocks = sampler.summary(t0, t1)
        ms_dense, _, _ = timed(dense_graphs, min(args.steps, 2000), args.warmup)

        # spread of the step time: 200 replays timed one by one (each pair of events adds a little)
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(200)]
        for i, (a, b_) in enumerate(pairs):
            a.record(stream)
            sparse_graphs[i % POOLS].replay()
            b_.record(stream)
        torch.cuda.synchronize()
        each = np.array([a.elapsed_time(b_) * 1e3 for a, b_ in pairs])
        step_pct = {"p10": round(float(np.percentile(each, 10)), 2), "p50": round(float(np.percentile(each, 50)), 2),
                    "p90": round(float(np.percentile(each, 90)), 2), "n": len(pairs)}

        # the step's real timeline: device-side time stamps of every kernel's first CTA start and last CTA end
        # inside graph-replayed steps (nothing is serialised: overlapping kernels show as overlapping)
        ticks = plan.enable_kernel_ticks()
        tl_graphs = capture(False)
        tl = []
        for i in range(48):
            plan.reset_kernel_ticks()
            tl_graphs[i % POOLS].replay()
            stream.synchronize()
            t = ticks.cpu().numpy().astype(np.float64)
            if i >= 8:
                tl.append((t - t[0, 0]) * 1e-3)
        tl = np.median(np.stack(tl), axis=0)
        plan.disable_debug()
        del tl_graphs
        timeline = {name: [round(float(tl[k_, 0]), 2), round(float(tl[k_, 1]), 2) if tl[k_, 1] > 0 else None]
                    for k_, name in enumerate(vb.TICK_NAMES)}

        # the K+V gather variant (weights recomputed from the K rows of the sampled tokens)
        plan.set_params(**dict(case.params, gather_mode=1))
        kv_graphs = capture(False)
        ms_kv, _, _ = timed(kv_graphs, min(args.steps, 500), args.warmup)
        del kv_graphs
        # sampling keys per KV head: the heads of a group draw nested samples, so their sampled rows coincide
        # (another sample than the default's, hence other budgets: a variant, not the headline)
        plan.set_params(**dict(case.params, rng_head_is_kv=1))
        grp_graphs = capture(False)
        ms_grp, _, _ = timed(grp_graphs, min(args.steps, 500), args.warmup)
        del grp_graphs
        # nested samples: the base sample is the head of the final sample's own walk (I_bs inside I_dyn)
        plan.set_params(**dict(case.params, nested_base=1))
        nst_graphs = capture(False)
        ms_nst, _, _ = timed(nst_graphs, min(args.steps, 500), args.warmup)
        plan.set_params(**case.params)
        del nst_graphs

        # four query tokens per call (a question, speculative tokens): 128 (token, head) pairs share one pass over K
        MQ = 4
        q4 = torch.from_numpy(np.ascontiguousarray(synth.multi_query(case, MQ)).view(np.int16)).cuda().view(torch.bfloat16)
        mq_plan = vb.plan_for_case(case, q_len=MQ)
        mq_plan.set_params(**case.params)
        mq_out = torch.empty_like(q4)

        def mq_capture(dense):
            graphs = []
            for i in range(POOLS):
                d = pools[i % npools]
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    if dense:
                        mq_plan.dense_decode(q4, d["k_cache"], d["v_cache"], d["block_table"], d["seq_lens"], mq_out,
                                             stream=stream)
                    else:
                        mq_plan.decode(q4, d["k_cache"], d["v_cache"], d["block_table"], d["seq_lens"], case.sink,
                                       case.window, case.k, case.eps, case.delta, case.seed, mq_out, stream=stream)
                graphs.append(g)
            return graphs
        for dense_ in (False, True):                       # first calls outside a capture (attributes, lazy loading)
            d = pools[0]
            if dense_:
                mq_plan.dense_decode(q4, d["k_cache"], d["v_cache"], d["block_table"], d["seq_lens"], mq_out, stream=stream)
            else:
                mq_plan.decode(q4, d["k_cache"], d["v_cache"], d["block_table"], d["seq_lens"], case.sink, case.window,
                               case.k, case.eps, case.delta, case.seed, mq_out, stream=stream)
        stream.synchronize()
        mq_graphs = mq_capture(False)
        ms_mq, _, _ = timed(mq_graphs, min(args.steps, 500), args.warmup)
        del mq_graphs
        mq_graphs = mq_capture(True)
        ms_mq_dense, _, _ = timed(mq_graphs, min(args.steps, 500), args.warmup)
        del mq_graphs, mq_plan

        # optional external context: a third-party dense paged-decode kernel on the same cache
        fi_us = None
        if args.flashinfer:
            try:
                import flashinfer
                nb = (int(case.seq_lens[0]) + 15) // 16
                indptr = torch.tensor([0, nb], dtype=torch.int32, device="cuda")
                last = torch.tensor([(int(case.seq_lens[0]) - 1) % 16 + 1], dtype=torch.int32, device="cuda")
                kvs = [torch.stack([d["k_cache"], d["v_cache"]], dim=1).contiguous() for d in pools]
                idx = pools[0]["block_table"][0, :nb].contiguous()
                wsfi = torch.empty(128 << 20, dtype=torch.uint8, device="cuda")
                w = flashinfer.BatchDecodeWithPagedKVCacheWrapper(wsfi, "HND", use_tensor_cores=True)
                w.plan(indptr, idx, last, case.num_q_heads, case.num_kv_heads, case.head_dim, 16,
                       q_data_type=torch.bfloat16, kv_data_type=torch.bfloat16)
                for i in range(5):
                    w.run(pools[0]["q"], kvs[i % POOLS])
                stream.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for i in range(200):
                    w.run(pools[0]["q"], kvs[i % POOLS])
                e1.record(stream)
                torch.cuda.synchronize()
                fi_us = e0.elapsed_time(e1) / 200 * 1e3
                del kvs
            except Exception as ex:          # context only: never fail the bench for it
                fi_us = f"unavailable: {type(ex).__name__}"

        # per-kernel timing (plain launches with events between the kernels)
        plan.set_profiling(True)
        prof_steps = min(args.steps, 200)
        for i in range(prof_steps):
            step(i)
        stream.synchronize()
        prof, calls = plan.read_profile()
        plan.set_profiling(False)

        # the bandwidth kernel alone, launched back to back (16 launches per graph, pools rotating): its
        # duration without the launch gap that the events inside a step include
        plan.set_stop_after(1)
        B2B = 4 * POOLS
        g_score = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_score, stream=stream):
            for i in range(B2B):
                step(i)
        for _ in range(3):
            g_score.replay()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(20):
            g_score.replay()
        e1.record(stream)
        torch.cuda.synchronize()
        us_score_b2b = e0.elapsed_time(e1) / (20 * B2B) * 1e3
        plan.set_stop_after(0)

        # end to end through the host-buffer entry point
        qh = dev0["q"].cpu().pin_memory()
        bth = dev0["block_table"].cpu().pin_memory()
        slh = dev0["seq_lens"].cpu().pin_memory()
        outh = torch.empty_like(qh).pin_memory()
        e2e_steps = min(args.steps, 500)

        def e2e_step(i):
            d = pools[i % POOLS]
            plan.decode_host(qh, d["k_cache"], d["v_cache"], bth, slh, case.sink, case.window, case.k, case.eps,
                             case.delta, case.seed, outh, stream=stream)
        # the entry point records a call's CUDA graph on the second call with one argument set: warm up until every
        # pool's graph exists, so that only replays are timed
        for i in range(max(args.warmup, 2 * POOLS + 1)):
            e2e_step(i)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(e2e_steps):
            e2e_step(i)
        e1.record(stream)
        torch.cuda.synchronize()
        ms_e2e = e0.elapsed_time(e1) / e2e_steps

    other = None
    if args.all_configs and rank == 0:
        other = time_other_configs(vb, synth, torch)

    ms_step_max = max_over_ranks(ms_step, world)
    ms_e2e_max = max_over_ranks(ms_e2e, world)
    ms_dense_max = max_over_ranks(ms_dense, world)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- algorithmic bytes per launch: what each kernel must move.  Score pass: every K row once, 4 bytes written
    # per (token, query head).  Per-head kernel: the scores once (selection), K and V rows of I_f and I_bs (rescored
    # in fp64), V row + 4-byte score of every token of I_dyn.
    es, d, Hq, Hkv = 2, case.head_dim, case.num_q_heads, case.num_kv_heads
    n_tot = int(case.seq_lens.sum())
    n_f = kks.sum() + Hq * (min(case.sink, n_tot) + min(case.window, n_tot))
    # Entries of a walk that hold c residual tokens: c * |M| / n_s (members of I_t sit among them, marked).
    mlen_tot = n_tot - Hq * 0 - (min(case.sink, n_tot) + min(case.window, n_tot))        # middle range of the one row
    infl = mlen_tot / max(1.0, float(mlen_tot - kks.mean()))
    walk_entries = float((b0s * 1.04 + 8).sum() + np.minimum(8.3 * b0s + 8, mlen_tot).sum())   # both walk arrays, all heads
    alg = {
        "k_score": n_tot * Hkv * d * es + n_tot * Hq * 4,
        "k_walk": int(walk_entries * 8),                                   # token + physical slot per entry
        "k_select": n_tot * Hq * 4 + int(kks.sum()) * 16,                  # scores once; I_t written (8 B) and read back, marks
        "k_stats": int(n_f + b0s.sum() * infl) * (d * es * 2 + 8),         # K and V rows of I_f and the base prefix, entries
        "k_gather": int(b_dyn.sum() * infl) * (d * es + 12),               # V row, token, slot, score of every entry visited
    }
    rows_bytes = alg["k_stats"] + alg["k_gather"]
    traffic, traffic_note = read_traffic()
    peak, peak_kind = measured_peaks()
    kern = {}
    for name in vb.KERNEL_NAMES:
        us = prof[name] / max(calls, 1) * 1e3
        kern[name] = {"us": round(us, 2), "alg_bytes": int(alg[name]),
                      "gbs": round(alg[name] / (us * 1e-6) / 1e9, 1) if us > 0 else None}
    # dominant kernel = the one that moves most of the step's bytes
    top = "k_score"
    top_us = prof[top] / max(calls, 1) * 1e3
    achieved = alg[top] / (top_us * 1e-6) / 1e9
    b2b_gbs = alg[top] / (us_score_b2b * 1e-6) / 1e9
    density = float(np.mean((kks + 256 + b_dyn) / n_tot))
    sparse_bytes = alg["k_score"] + rows_bytes
    dense_bytes = 2 * n_tot * Hkv * d * es

    def span(name):
        a, b_ = timeline[name]
        return (b_ - a) if (a is not None and b_ is not None and b_ > a) else None

    def frac_of(bytes_, us):
        if not us:
            return None
        g = bytes_ / (us * 1e-6) / 1e9
        return {"us": round(us, 2), "achieved": round(g, 1), "frac": round(g / peak, 4), "frac_of_8TBs_nominal": round(g / 8000.0, 4)}
    # the row kernels (statistics, final sample): device-side spans inside graph-replayed steps
    # (the row kernels' CTAs are resident, waiting, long before they have work: their spans start when the last head's
    # I_t is complete, the gather's when the last budget is known)
    rows_span = stats_span = None
    if timeline["topk"][1] is not None and timeline["k_gather"][1] is not None:
        rows_span = timeline["k_gather"][1] - timeline["topk"][1]
    if timeline["topk"][1] is not None and timeline["budget"][1] is not None:
        stats_span = timeline["budget"][1] - timeline["topk"][1]

    cpu = None
    if not args.no_cpu_baseline:
        reps, t_cpu0, c_cpu0 = 0, time.perf_counter(), cpu_seconds()
        while reps < 2 or (time.perf_counter() - t_cpu0 < 10.0 and reps < 16):
            oracle_step(case)
            reps += 1
        wall = time.perf_counter() - t_cpu0
        cpu_us = wall / reps * 1e6
        cpu = {"value": cpu_us, "unit": UNIT, "cores": cores_used(cpu_seconds() - c_cpu0, wall),
               "host_cores": os.cpu_count(), "kind": "oracle",
               "sample": f"{reps} full steps of the same workload (all 32 heads, fp64 numpy, one thread)"}

    us_step = ms_step_max * 1e3
    line = {
        "metric": METRIC, "value": us_step / world, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step_max, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD, "l2": f"rotating {POOLS} distinct cache pools (134 MB of K+V each, "
                   "more than the 126 MB L2 together with the previous pool)", "launch": "CUDA graph replay per step",
                   "mean_density": round(density, 4), "sparsity_x": round(1.0 / density, 2),
                   "mean_budget": float(b_dyn.mean()), "status_bits": status, "step_us_percentiles": step_pct,
                   "kv_gather_variant_us_per_step": round(ms_kv * 1e3, 2),
                   "kv_head_sampling_keys_variant_us_per_step": round(ms_grp * 1e3, 2),
                   "nested_base_variant_us_per_step": round(ms_nst * 1e3, 2),
                   "four_query_tokens_per_call": {"sparse_us_per_call": round(ms_mq * 1e3, 2),
                                                  "dense_us_per_call": round(ms_mq_dense * 1e3, 2),
                                                  "sparse_us_per_token": round(ms_mq * 1e3 / 4, 2)},
                   "value_is": "max-over-ranks step time / n_gpus (each rank runs its own layer)"},
        "e2e": {"value": ms_e2e_max * 1e3 / world, "unit": UNIT,
                "h2d_bytes_per_step": int(qh.numel() * 2 + bth.numel() * 4 + slh.numel() * 4),
                "d2h_bytes_per_step": int(outh.numel() * 2)},
        "gpu_launches": launches_per_step * args.steps,
        "roofline": {"bound": "hbm", "kernel": top, "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
                     "frac": round(achieved / peak, 4), "frac_of": peak_kind, "frac_of_8TBs_nominal": round(achieved / 8000.0, 4),
                     "traffic": traffic.get(top), "traffic_source": traffic_note,
                     "alg_bytes_per_launch": int(alg[top]), "us_per_launch": round(top_us, 2),
                     "timing": "CUDA events around the kernel inside plain-launched steps (includes the launch gap)",
                     "back_to_back": {"us_per_launch": round(us_score_b2b, 2), "achieved": round(b2b_gbs, 1),
                                      "frac": round(b2b_gbs / peak, 4),
                                      "timing": "the kernel alone, 16 launches per CUDA graph, pools rotating"},
                     "device_timer": dict(frac_of(alg[top], span("k_score")) or {},
                                          timing="first CTA start to last CTA end (%globaltimer) inside graph-replayed steps")},
        # the gather / reduce part of the step (rows of I_f, I_bs and I_dyn) and the whole step, against the same peak
        "roofline_rows": dict(frac_of(rows_bytes, rows_span) or {}, kernel="k_stats + k_gather", alg_bytes=int(rows_bytes),
                              traffic=(traffic.get("k_stats", 0) + traffic.get("k_gather", 0)) or None,
                              timing="last head's I_t complete to last CTA of k_gather (%globaltimer), graph-replayed steps"),
        "roofline_k_stats": dict(frac_of(alg["k_stats"], stats_span) or {}, alg_bytes=int(alg["k_stats"]),
                                 timing="last head's I_t complete to last budget known (marking, rows, budget)"),
        "roofline_k_gather": dict(frac_of(alg["k_gather"], (timeline["k_gather"][1] - timeline["budget"][1])
                                          if timeline["k_gather"][1] and timeline["budget"][1] else None) or {},
                                  alg_bytes=int(alg["k_gather"]), timing="last budget known to last CTA of k_gather"),
        "roofline_step": dict(frac_of(sparse_bytes, us_step) or {}, alg_bytes=int(sparse_bytes)),
        "kernels": kern,
        "timeline_us": timeline,
        "dense": {"us_per_step": round(ms_dense_max * 1e3, 2), "alg_bytes": int(dense_bytes),
                  "gbs": round(dense_bytes / (ms_dense_max * 1e-3) / 1e9, 1),
                  "sparse_over_dense_time": round(ms_step_max / ms_dense_max, 3),
                  "sparse_alg_bytes": int(sparse_bytes), "flashinfer_us_per_step": fi_us},
        "cpu_baseline": cpu,
        "clocks": clocks,
    }
    if other is not None:
        line["other_configs"] = other
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
