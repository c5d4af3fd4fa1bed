#!/usr/bin/env python
"""Benchmark of the GRPO/AERO hot path: group stage + fused lm_head log-prob/loss
forward + backward, in rollout tokens per second.

    python bench.py --gpus 1 --steps 10 --warmup 3            # CUDA library (default)
    python bench.py --impl reference --steps 2 --warmup 1     # the fp64 CPU oracle, timed

One step = one pass of the whole path over one synthetic batch of the workload
(default: the Qwen2.5-Math-1.5B shaped batch).  Prints one JSON line on rank 0.
With N > 1 ranks (torchrun) every rank runs an independent replica of the step on
its own batch; there is no data-path collective.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "rollout tokens/sec, fused GRPO logprob+loss fwd+bwd"
# dram__bytes_read.sum + dram__bytes_write.sum of one lmhead_kernel<MODE_FWD> launch on the full-size workload,
# from the one-pass ncu captures summarised in profiles/lmhead_fwd_full_size_dram.md (per workload index).
NCU_FWD_TRAFFIC = {1: {"bytes": 6.057e9, "tokens": 204780}, 2: {"bytes": 197.6e9, "tokens": 468700}}
# the same for the launches of lmhead_kernel<MODE_FWD_P> of one step (they also write the chunk blocks)
NCU_FWDP_TRAFFIC = {1: {"bytes": 71.87e9, "tokens": 204780}, 2: {"bytes": 315.6e9, "tokens": 468700}}
NCU_FWD_TRAFFIC_SOURCE = "ncu capture of the full-size launch (dram__bytes_read.sum + dram__bytes_write.sum)"
UNIT = "tokens/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=1, help="workload index 0..4")
    ap.add_argument("--chunk-tokens", type=int, default=4 * 148 * 128)
    ap.add_argument("--prompts", type=int, default=0, help="override the number of prompts (reduced runs for profiling)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-group-leg", action="store_true")
    ap.add_argument("--no-variants-leg", action="store_true",
                    help="skip the timings of the regularised step (KL + entropy) and of the log-prob pass alone")
    ap.add_argument("--only-group-leg", action="store_true",
                    help="run only the large-input group-stage measurement (for profiling that stage alone)")
    return ap.parse_args()


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm=p["hbm_gbs"], burst=p["bf16_tflops"], sustained=p["bf16_tflops_sustained"], src="measured")
    return dict(hbm=6650.0, burst=1590.0, sustained=1400.0, src="fallback")


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index):
        import torch
        self.proc = None
        self.path = tempfile.mktemp(suffix=".csv")
        try:
            uuid = "GPU-" + str(torch.cuda.get_device_properties(device_index).uuid)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", uuid, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 7:
                    continue
                try:
                    sm.append(float(f[0]))
                    mx.append(float(f[1]))
                except ValueError:
                    continue
                for n, v in zip(names, f[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        return out


# ----------------------------------------------------------------------------- oracle legs
def oracle_sample(wl, st, n_tokens):
    """The first n_tokens token rows of the workload as one group (rollouts truncated at the
    sample boundary), as fp64 arrays for the oracle.  Inputs only; no result of the CUDA path."""
    import torch
    from paper_2602_14338_b200 import synth

    n_tokens = int(min(n_tokens, st.cs[-1]))
    R = int(np.searchsorted(st.cs, n_tokens, side="left"))
    cs = np.minimum(st.cs[:R + 1], n_tokens).astype(np.int64)
    go = np.array([0, R], np.int32)
    reward = st.reward[:R].copy()
    if R >= 2:                                   # make sure the sample group is a mixed one
        reward[0], reward[1] = 1.0, 0.0
    H, W = synth.make_tensors(wl, n_tokens, device="cpu")
    return dict(go=go, cs=cs, reward=reward, key=st.key[:R], y=st.y[:n_tokens], noise=st.noise[:n_tokens],
                H=H.double().numpy(), W=W.double().numpy(), T=n_tokens)


def oracle_step(O, s, old):
    cfg = O.Cfg()
    g = O.group_stats(cfg, s["go"], s["reward"], s["cs"], key=s["key"])
    f = O.grpo_loss_fwd(cfg, s["H"], s["W"], s["y"], old, s["cs"], g["adv"], g["w"], g["keep"])
    dH, dW = O.grpo_loss_bwd(s["H"], s["W"], s["y"], s["cs"], g["keep"], f["lse"], f["g"])
    return f["loss"], int(g["counters"][1])


def time_oracle(wl, st, budget_s, steps=1, warmup=0):
    """Time the oracle as it stands on a bounded token sample; returns (tokens/s, cores, sample text, ms/step)."""
    from oracle import aero_oracle as O
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [os.cpu_count() or 1])
    except Exception:
        cores = os.cpu_count() or 1
    # calibrate on 32 tokens, then size the sample for the time budget
    cal = oracle_sample(wl, st, 32)
    t0 = time.perf_counter()
    oracle_step(O, cal, np.full(cal["T"], -12.0))
    per_tok = (time.perf_counter() - t0) / max(cal["T"], 1)
    n = int(budget_s / max(per_tok, 1e-9) / max(steps + warmup, 1))
    n = max(64, min(1024, n, int(st.cs[-1])))
    s = oracle_sample(wl, st, n)
    z = O.logits(s["H"], s["W"])
    lp, _ = O.log_softmax_pick(z, s["y"])
    del z
    old = lp + s["noise"]
    for _ in range(warmup):
        oracle_step(O, s, old)
    t0 = time.perf_counter()
    kept = 0
    for _ in range(steps):
        _, kept = oracle_step(O, s, old)
    dt = (time.perf_counter() - t0) / steps
    sample = (f"first {s['T']} token rows of the workload as one group of {len(s['reward'])} rollouts "
              f"({kept} kept tokens per step), full d={wl.d} and V={wl.V}, fp64 numpy")
    return kept / dt, cores, sample, dt * 1e3


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2602_14338_b200 import synth
    wl = synth.WORKLOADS[args.config]
    st = synth.make_structure(wl)
    val, cores, sample, ms = time_oracle(wl, st, 150.0, steps=max(args.steps, 1), warmup=args.warmup)
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "d": wl.d, "V": wl.V, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- CUDA arm
def run_ours(args):
    import torch
    from paper_2602_14338_b200 import binding as B
    from paper_2602_14338_b200 import dist as D
    from paper_2602_14338_b200 import synth

    rank, world, local = D.init_from_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (the library has no CPU path)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    pk = peaks()
    if args.only_group_leg:
        ctx = B.Context(local)
        print(json.dumps({"group_stage": group_stage_leg(ctx, pk, dev)}), flush=True)
        return

    base = synth.WORKLOADS[args.config]
    wl = synth.scaled(base, seed=base.seed + 100 * rank)      # an independent batch per replica
    if args.prompts > 0:
        wl = synth.scaled(wl, P=args.prompts)
    st = synth.make_structure(wl)
    P, R, T = len(st.go) - 1, len(st.reward), int(st.cs[-1])
    H, W = synth.make_tensors(wl, T, device=dev)
    ctx = B.Context(local)
    over = dict(seed=wl.seed, dtype=B.AERO_BF16 if wl.dtype == "bf16" else B.AERO_FP32)
    if wl.aero:
        over.update(uniform_policy=B.AERO_UNIFORM_BAYES, rejection=1, k_ratio=1)
    cfg = B.cfg_default(**over)

    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    go, reward, cs, key, y = t(st.go), t(st.reward), t(st.cs), t(st.key.view(np.int32)), t(st.y)
    alpha = t(st.alpha) if st.alpha is not None else None
    beta = t(st.beta) if st.beta is not None else None
    noise = t(st.noise)

    gbuf, fbuf = {}, {}
    dH = torch.empty_like(H)
    dW = torch.empty((wl.V, wl.d), dtype=torch.float32, device=dev)
    chunk = min(args.chunk_tokens, (T + 127) // 128 * 128)
    ws_b = torch.empty(max(ctx.bwd_workspace_bytes(T, wl.d, wl.V, R, chunk), ctx.fwd_bwd_workspace_bytes(T, wl.d, wl.V, R, chunk)),
                       dtype=torch.uint8, device=dev)

    # old log-probs: the current policy's own log-probs (the log-prob pass alone) plus seeded noise
    f0 = ctx.logprob_fwd(cfg, H, W, y)
    old = (f0["logp"][:T] + noise).contiguous()
    del f0

    def step():
        # group stage, then forward and backward of stage (b) in one call (no recompute of the logits)
        g = ctx.group_stats(cfg, go, reward, cs, key=key, alpha_in=alpha, beta_in=beta, out=gbuf)
        f, _, _ = ctx.grpo_loss_fwd_bwd(cfg, H, W, y, old, cs, g["adv"], g["w"], g["keep"], out=fbuf, dH=dH, dW=dW,
                                        workspace=ws_b)
        return g, f

    def step_two_calls():
        # the same step through the separate forward and backward calls (the backward recomputes the logits)
        g = ctx.group_stats(cfg, go, reward, cs, key=key, alpha_in=alpha, beta_in=beta, out=gbuf)
        f = ctx.grpo_loss_fwd(cfg, H, W, y, old, cs, g["adv"], g["w"], g["keep"], out=fbuf)
        ctx.grpo_loss_bwd(cfg, H, W, y, cs, g["keep"], f["lse"], f["g"], dH=dH, dW=dW, workspace=ws_b)

    for _ in range(max(args.warmup, 1)):
        g, f = step()
    torch.cuda.synchronize()
    T_kept = int(g["counters"][1].item())
    status = ctx.last_status()

    D.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    l0 = ctx.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    launches = ctx.launch_count() - l0
    D.barrier()
    ms_local = e0.elapsed_time(e1)
    units, ms_total = D.aggregate(T_kept * args.steps, ms_local, device=dev)
    ms_step = ms_total / args.steps
    value = units / (ms_total * 1e-3)

    # dominant kernel of the timed step: lmhead_kernel<MODE_FWD_P> (one launch per chunk), timed with CUDA events
    # that the library records around its launches, over three more steps
    ctx.enable_kernel_timing(True)
    fp_total_ms, fp_launches = 0.0, 0
    for _ in range(3):
        step()
        ms_i, n_i = ctx.kernel_timing_ms()          # read out per step: the library keeps at most 256 pairs of events
        fp_total_ms += ms_i
        fp_launches += n_i
    ctx.enable_kernel_timing(False)
    fwdp_ms_step = fp_total_ms / 3.0
    # the plain forward kernel (MODE_FWD, used by the separate forward call and the log-prob pass), timed over its call
    fw = []
    for _ in range(max(3, min(args.steps, 10))):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        ctx.grpo_loss_fwd(cfg, H, W, y, old, cs, gbuf["adv"], gbuf["w"], gbuf["keep"], out=fbuf)
        b.record()
        torch.cuda.synchronize()
        fw.append(a.elapsed_time(b))
    fwd_ms = float(np.mean(fw))
    clocks = sampler.stop()
    flops_launch = 2.0 * T_kept * wl.d * wl.V
    cap = NCU_FWD_TRAFFIC.get(args.config) if args.prompts == 0 else None
    traffic = cap["bytes"] * T_kept / cap["tokens"] if cap else None
    achieved = flops_launch / (fwdp_ms_step * 1e-3) / 1e12
    capp = NCU_FWDP_TRAFFIC.get(args.config) if args.prompts == 0 else None
    # the kernel is timed inside whole steps, under the power cap they run into: the sustained GEMM rate is its peak
    roofline = {"bound": "tensor", "kernel": "lmhead_kernel<MODE_FWD_P>", "achieved": achieved, "peak": pk["sustained"],
                "unit": "TFLOP/s", "frac": achieved / pk["sustained"],
                "peak_source": pk["src"] + " sustained bf16 (kernel timed inside the step)",
                "frac_of_burst": achieved / pk["burst"], "peak_burst": pk["burst"],
                "traffic": capp["bytes"] * T_kept / capp["tokens"] if capp else None,
                "traffic_source": NCU_FWD_TRAFFIC_SOURCE.replace("launch", "launches of one step") if capp else None,
                "launches_per_step": fp_launches / 3.0, "ms_per_step_all_launches": fwdp_ms_step,
                "plain_forward_kernel": {"kernel": "lmhead_kernel<MODE_FWD>", "ms_per_launch": fwd_ms,
                                         "achieved": flops_launch / (fwd_ms * 1e-3) / 1e12,
                                         "frac": flops_launch / (fwd_ms * 1e-3) / 1e12 / pk["burst"],
                                         "peak_source": pk["src"] + " burst bf16 (kernel timed in a call of its own)",
                                         "frac_of_sustained": flops_launch / (fwd_ms * 1e-3) / 1e12 / pk["sustained"],
                                         "traffic": traffic},
                "step_executed_tflops": 6.0 * T_kept * wl.d * wl.V / (ms_local / args.steps * 1e-3) / 1e12,
                "step_frac_of_sustained": 6.0 * T_kept * wl.d * wl.V / (ms_local / args.steps * 1e-3) / 1e12 / pk["sustained"]}
    # the two-call step (8 d V executed FLOPs per token), for comparison
    step_two_calls()
    torch.cuda.synchronize()
    a2, b2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a2.record()
    for _ in range(2):
        step_two_calls()
    b2.record()
    torch.cuda.synchronize()
    ms2 = a2.elapsed_time(b2) / 2
    roofline["two_call_step"] = {"ms": ms2, "tokens_per_s": T_kept / (ms2 * 1e-3),
                                 "executed_tflops": 8.0 * T_kept * wl.d * wl.V / (ms2 * 1e-3) / 1e12,
                                 "frac_of_sustained": 8.0 * T_kept * wl.d * wl.V / (ms2 * 1e-3) / 1e12 / pk["sustained"]}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 1), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
        "config": {"workload": wl.name, "P": P, "R": R, "T_input": T, "T_kept": T_kept, "d": wl.d, "V": wl.V,
                   "parallelism": f"replicas x{world}", "chunk_tokens": int(chunk),
                   "l2": "inputs larger than L2 (H+W > 1 GB per step)", "tokens_counted": "kept tokens",
                   "input_tokens_per_s": T * world / (ms_step * 1e-3), "status_word": status},
        "clocks": {k: clocks[k] for k in ("sm_mhz", "sm_max_mhz", "reasons")},
        "gpu_launches": int(launches),
        "roofline": roofline,
    }

    if rank == 0 and world == 1 and not args.no_variants_leg:
        line["variants"] = variants_leg(ctx, cfg, wl, H, W, y, old, noise, cs, gbuf, dH, dW, ws_b, T_kept, pk)
    if rank == 0 and world == 1 and not args.no_group_leg:
        line["group_stage"] = group_stage_leg(ctx, pk, dev)
    if rank == 0 and not args.no_e2e:
        line["e2e"] = e2e_leg(ctx, cfg, wl, st, H, W, old, dH, dW, chunk, args, T_kept)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        val, cores, sample, _ = time_oracle(base, synth.make_structure(base), 20.0)
        line["cpu_baseline"] = {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample}
    if rank == 0:
        print(json.dumps(line), flush=True)
    D.barrier()


def variants_leg(ctx, cfg, wl, H, W, y, old, noise, cs, g, dH, dW, ws_b, T_kept, pk):
    """The step with Eq. 2's KL term and the entropy bonus (aero_grpo_loss_reg_fwd/_bwd), the one-call step
    with the KL term (aero_grpo_loss_kl_fwd_bwd), and the log-prob pass alone (aero_logprob_fwd) that produces old / reference log-probs."""
    import copy
    import torch

    T = H.shape[0]
    rcfg = copy.copy(cfg)
    rcfg.kl_beta, rcfg.ent_coef = 0.04, 1e-3
    ref = (old + 0.5 * noise).contiguous()
    fb, lb = {}, {}

    def timed(fn, n=3):
        fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(n):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / n

    def reg_step():
        f = ctx.grpo_loss_reg_fwd(rcfg, H, W, y, old, ref, cs, g["adv"], g["w"], g["keep"], out=fb)
        ctx.grpo_loss_reg_bwd(rcfg, H, W, y, cs, g["keep"], f["lse"], f["g"], f["entropy"], g["w"], dH=dH, dW=dW,
                              workspace=ws_b)

    ms_reg = timed(reg_step)
    kcfg = copy.copy(cfg)
    kcfg.kl_beta = 0.04
    kb = {}
    ms_kl = timed(lambda: ctx.grpo_loss_fwd_bwd(kcfg, H, W, y, old, cs, g["adv"], g["w"], g["keep"], out=kb, dH=dH, dW=dW,
                                                workspace=ws_b, ref_logp=ref))
    ms_lp = timed(lambda: ctx.logprob_fwd(rcfg, H, W, y, out=lb))
    # allocation controller on 2^22 simulated prompts with success rates ~ Beta(0.5, 0.5)
    from paper_2602_14338_b200 import binding as B
    from paper_2602_14338_b200 import synth
    Pn = 1 << 22
    thr = torch.from_numpy(synth.success_thresholds(Pn, 0.5, 0.5, seed=4301).view(np.int32)).to(H.device)
    acfg = B.cfg_default(uniform_policy=B.AERO_UNIFORM_BAYES, rejection=1, k_ratio=1, seed=4302)
    ab = {}
    ms_alloc = timed(lambda: ctx.allocate_sim(acfg, B.alloc_cfg_default(), thr, out=ab), n=5)
    cnt = ab["counters"].cpu().tolist()
    # down-sampling ratio k = 1..4 on the AERO-curated batch (workload 3): what the backward has to process
    st3 = synth.make_structure(synth.WORKLOADS[3])
    t3 = lambda x: torch.from_numpy(np.ascontiguousarray(x)).to(H.device)
    go3, rw3, cs3, key3 = t3(st3.go), t3(st3.reward), t3(st3.cs), t3(st3.key.view(np.int32))
    al3, be3 = t3(st3.alpha), t3(st3.beta)
    ksweep = {}
    for k in (1, 2, 3, 4):
        kc = B.cfg_default(uniform_policy=B.AERO_UNIFORM_BAYES, rejection=1, k_ratio=k, seed=synth.WORKLOADS[3].seed)
        gk = ctx.group_stats(kc, go3, rw3, cs3, key=key3, alpha_in=al3, beta_in=be3)
        ck = gk["counters"].cpu().tolist()
        ksweep[str(k)] = {"kept_rollouts": ck[0], "kept_tokens": ck[1], "kept_token_fraction": ck[1] / max(ck[7], 1)}
    fl = 2.0 * wl.d * wl.V
    return {"allocation_sim": {"prompts": Pn, "ms": ms_alloc, "prompts_per_s": Pn / (ms_alloc * 1e-3),
                               "launches": 23, "mean_rollouts_generated": cnt[0] / Pn, "mean_rollouts_trained": cnt[1] / Pn,
                               "zero_accuracy_before": cnt[2] / Pn, "zero_accuracy_after": cnt[3] / Pn,
                               "iterations": cnt[5]},
            "k_ratio_sweep_workload3": ksweep,
            "regularised_step": {"kl_beta": 0.04, "ent_coef": 1e-3, "ms": ms_reg, "tokens_per_s": T_kept / (ms_reg * 1e-3),
                                 "executed_tflops": 4 * fl * T_kept / (ms_reg * 1e-3) / 1e12,
                                 "frac_of_sustained": 4 * fl * T_kept / (ms_reg * 1e-3) / 1e12 / pk["sustained"]},
            "kl_step_one_call": {"kl_beta": 0.04, "ms": ms_kl, "tokens_per_s": T_kept / (ms_kl * 1e-3),
                                 "executed_tflops": 3 * fl * T_kept / (ms_kl * 1e-3) / 1e12,
                                 "frac_of_sustained": 3 * fl * T_kept / (ms_kl * 1e-3) / 1e12 / pk["sustained"]},
            "logprob_pass": {"rows": T, "ms": ms_lp, "tokens_per_s": T / (ms_lp * 1e-3),
                             "tflops": fl * T / (ms_lp * 1e-3) / 1e12, "frac_of_burst": fl * T / (ms_lp * 1e-3) / 1e12 / pk["burst"]}}


def group_stage_leg(ctx, pk, dev):
    """Stage (a) alone on an input large enough to be bandwidth-bound (2^22 prompts of 2..16 rollouts):
    algorithmic bytes (37 per rollout + 26 per prompt) over the duration of the stage's four launches."""
    import torch
    from paper_2602_14338_b200 import binding as B
    from paper_2602_14338_b200 import synth

    wl = synth.scaled(synth.WORKLOADS[3], P=1 << 22, seed=4222, len_median=64.0, len_cap=256)
    st = synth.make_structure(wl)
    P, R = len(st.go) - 1, len(st.reward)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    go, reward, cs, key = t(st.go), t(st.reward), t(st.cs), t(st.key.view(np.int32))
    alpha, beta = t(st.alpha), t(st.beta)
    cfg = B.cfg_default(uniform_policy=B.AERO_UNIFORM_BAYES, rejection=1, k_ratio=1, seed=wl.seed)
    out = {}
    for _ in range(3):
        ctx.group_stats(cfg, go, reward, cs, key=key, alpha_in=alpha, beta_in=beta, out=out)
    torch.cuda.synchronize()
    times = []
    for _ in range(10):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        ctx.group_stats(cfg, go, reward, cs, key=key, alpha_in=alpha, beta_in=beta, out=out)
        b.record()
        torch.cuda.synchronize()
        times.append(a.elapsed_time(b))
    ms = float(np.median(times))
    nbytes = 37.0 * R + 26.0 * P
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"P": P, "R": R, "ms": ms, "bound": "hbm", "achieved": gbs, "peak": pk["hbm"], "unit": "GB/s",
            "frac": gbs / pk["hbm"], "algorithmic_bytes": nbytes,
            "kept_rollout_frac": float(out["metrics"][2].item())}


def e2e_leg(ctx, cfg, wl, st, H, W, old, dH, dW, chunk, args, T_kept):
    """Same step through the host-buffer entry point: inputs in pinned host memory, copies inside the timed region."""
    import torch

    P, R, T = len(st.go) - 1, len(st.reward), int(st.cs[-1])
    pin = lambda x: x.pin_memory()
    go_h, rw_h, cs_h = pin(torch.from_numpy(st.go)), pin(torch.from_numpy(st.reward)), pin(torch.from_numpy(st.cs))
    key_h = pin(torch.from_numpy(st.key.view(np.int32)))
    al_h = pin(torch.from_numpy(st.alpha)) if st.alpha is not None else None
    be_h = pin(torch.from_numpy(st.beta)) if st.beta is not None else None
    H_h, y_h, old_h = pin(H.cpu()), pin(torch.from_numpy(st.y)), pin(old.cpu())
    ws = torch.empty(ctx.step_workspace_bytes(P, R, T, wl.d, wl.V, chunk, cfg.dtype), dtype=torch.uint8, device=H.device)
    h2d = H_h.numel() * H_h.element_size() + 8 * T + 4 * (P + 1) + 16 * R + 8 + (8 * P if al_h is not None else 0)
    d2h = 4 + 64 + 32
    n = max(2, min(args.steps, 5))
    ctx.grpo_step_host(cfg, go_h, rw_h, cs_h, key_h, al_h, be_h, H_h, y_h, old_h, W, dH, dW, ws)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(n):
        loss, counters, _ = ctx.grpo_step_host(cfg, go_h, rw_h, cs_h, key_h, al_h, be_h, H_h, y_h, old_h, W, dH, dW, ws)
    dt = (time.perf_counter() - t0) / n
    assert int(counters[1]) == T_kept
    return {"value": T_kept / dt, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
            "ms_per_step": dt * 1e3, "loss": float(loss.item())}


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
