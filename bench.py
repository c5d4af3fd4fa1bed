#!/usr/bin/env python
"""Benchmark of the GRPO/AERO hot path: group stage + fused lm_head log-prob/loss
forward + backward, in rollout tokens per second.

    python bench.py --gpus 1 --steps 10 --warmup 3            # CUDA library (default)
    python bench.py --impl reference --steps 2 --warmup 1     # the fp64 CPU oracle, timed

One step = one pass of the whole path over one synthetic batch of the workload.  The
default workload is the largest one that fits one GPU, the stress batch at the Qwen2.5-7B
shape (d = 3584, V = 152064, about 4.5 M input tokens); the three smaller bf16 workloads
are timed with a few steps each and reported as sub-records.  Prints one JSON line on
rank 0.  With N > 1 ranks (torchrun, or `--gpus N`, which starts the ranks itself) every
rank takes its own batch of prompts against a replicated W, and the step includes the
exchange of a data-parallel step: all-reduce of the group counters, weights brought to the
batch-wide denominators, all-reduce of dW and of the loss.
"""
from __future__ import annotations

import argparse
import gc
import json
import os
import socket
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "rollout tokens/sec, fused GRPO logprob+loss fwd+bwd"
UNIT = "tokens/s"
NOMINAL_BF16_TFLOPS = 2250.0          # dense bf16 of the data sheet; the targets are stated against it
TARGET_STAGE_B, TARGET_STAGE_A = 0.60, 0.70


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per token tile of a launch of lmhead_kernel<MODE_FWD_P> at
# d = 3584, V = 152064, from an ncu capture of a reduced case of this program (one wave of 148 token tiles per launch:
# 6.78 GB read + 5.74 GB written, mean of two launches; profiles/one_call_step_full_chunk_dram.md).  The traffic of a
# launch grows with its token tiles (every wave of 74 tiles streams W once and re-reads its H tiles), so a full launch
# is that figure times its tiles.  Valid for this shape and for the kernel as captured; otherwise null.
FWDP_TRAFFIC_PER_TILE = {(3584, 152064): (6.78e9 + 5.74e9) / 148}
FWDP_TRAFFIC_NOTE = ("per launch over a full chunk: the ncu counters of a reduced case (`bench.py --config 2 --prompts 10 "
                     "--chunk-tokens 18944 --only-main --steps 1 --warmup 1`, 148 token tiles per launch, 12.5 GB) scaled by "
                     "the token tiles of a launch; algorithmic 24.7 GB per full launch, the excess being H tiles re-read "
                     "after leaving L2; null for other shapes")


def fwdp_traffic(wl, chunk_tokens):
    per_tile = FWDP_TRAFFIC_PER_TILE.get((wl.d, wl.V))
    return None if per_tile is None else per_tile * (int(chunk_tokens) // 128)


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=4, help="workload index 0..4 of the headline line")
    ap.add_argument("--chunk-tokens", type=int, default=4 * 148 * 128)
    ap.add_argument("--prompts", type=int, default=0, help="override the number of prompts (reduced runs for profiling)")
    ap.add_argument("--sub-workloads", default="1,2,3", help="workloads timed briefly and reported as sub-records")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-group-leg", action="store_true")
    ap.add_argument("--no-variants-leg", action="store_true",
                    help="skip the regularised step, the log-prob pass alone, the allocation simulation and the k sweep")
    ap.add_argument("--only-group-leg", action="store_true",
                    help="run only the large-input group-stage measurement (for profiling that stage alone)")
    ap.add_argument("--only-main", action="store_true", help="only the timed steps of the headline workload")
    ap.add_argument("--gemm-sync", type=int, default=-1,
                    help="meeting points per unit of the backward products' producers (aero_set_tuning); -1: the library's default")
    ap.add_argument("--w-hint", type=int, default=-1,
                    help="lm_head kernel loads W with the evict-first L2 priority (aero_set_tuning); -1: the library's default")
    ap.add_argument("--k-zigzag", type=int, default=-1,
                    help="lm_head kernel walks d forwards and backwards in turn (aero_set_tuning); -1: the library's default")
    ap.add_argument("--gemm-pairs", type=int, default=-1,
                    help="backward products on CTA pairs (1) or single CTAs (0) (aero_set_tuning); -1: the library's default")
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
    """A bounded sample of the workload for the oracle: its first rollouts (up to 8), each cut to its
    first n_tokens / 8 token rows, as one group, in fp64.  Inputs only; no result of the CUDA path."""
    from paper_2602_14338_b200 import synth

    G = int(min(8, len(st.reward)))
    cap = max(1, int(n_tokens) // G)
    lens = np.minimum(st.cs[1:G + 1] - st.cs[:G], cap).astype(np.int64)
    rows = np.concatenate([np.arange(st.cs[i], st.cs[i] + lens[i]) for i in range(G)])
    cs = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    go = np.array([0, G], np.int32)
    reward = st.reward[:G].copy()
    if G >= 2:                                   # make sure the sample group is a mixed one
        reward[0], reward[1] = 1.0, 0.0
    H, W = synth.make_tensors(wl, int(st.cs[G]), device="cpu")
    return dict(go=go, cs=cs, reward=reward, key=st.key[:G], y=st.y[rows], noise=st.noise[rows],
                H=H[rows].double().numpy(), W=W.double().numpy(), T=int(cs[-1]))


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
    sample = (f"the workload's first {len(s['reward'])} rollouts, each cut to its first {int(s['cs'][1:].max() if s['T'] else 0)} "
              f"token rows at most, as one group: {s['T']} rows, {kept} kept tokens per step, full d={wl.d} and V={wl.V}, "
              f"fp64 numpy")
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
class Prepared:
    """One workload resident on the device: inputs, outputs and the workspace of the step."""

    def __init__(self, ctx, dev, idx, rank, chunk_tokens, prompts=0):
        import torch
        from paper_2602_14338_b200 import binding as B
        from paper_2602_14338_b200 import synth

        self.ctx, self.dev = ctx, dev
        self.base = synth.WORKLOADS[idx]
        wl = synth.scaled(self.base, seed=self.base.seed + 100 * rank)      # an independent batch of prompts per rank
        if prompts > 0:
            wl = synth.scaled(wl, P=prompts)
        self.wl = wl
        self.st = st = synth.make_structure(wl)
        self.P, self.R, self.T = len(st.go) - 1, len(st.reward), int(st.cs[-1])
        self.H, self.W = synth.make_tensors(wl, self.T, device=dev)
        over = dict(seed=wl.seed, dtype=B.AERO_BF16 if wl.dtype == "bf16" else B.AERO_FP32)
        if wl.aero:
            over.update(uniform_policy=B.AERO_UNIFORM_BAYES, rejection=1, k_ratio=1)
        self.cfg_over = over
        self.cfg = B.cfg_default(**over)
        t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
        self.go, self.reward, self.cs, self.key, self.y = t(st.go), t(st.reward), t(st.cs), t(st.key.view(np.int32)), t(st.y)
        self.alpha = t(st.alpha) if st.alpha is not None else None
        self.beta = t(st.beta) if st.beta is not None else None
        self.noise = t(st.noise)
        self.gbuf, self.fbuf = {}, {}
        self.dH = torch.empty_like(self.H)
        self.dW = torch.empty((wl.V, wl.d), dtype=torch.float32, device=dev)
        self.chunk = min(chunk_tokens, (self.T + 127) // 128 * 128)
        T, R = self.T, self.R
        self.ws = torch.empty(max(ctx.bwd_workspace_bytes(T, wl.d, wl.V, R, self.chunk),
                                  ctx.fwd_bwd_workspace_bytes(T, wl.d, wl.V, R, self.chunk)), dtype=torch.uint8, device=dev)
        # old log-probs: the current policy's own log-probs (the log-prob pass alone) plus seeded noise
        f0 = ctx.logprob_fwd(self.cfg, self.H, self.W, self.y)
        self.old = (f0["logp"][:T] + self.noise).contiguous()
        del f0

    def step(self, cfg=None):
        """Group stage, then forward and backward of stage (b) in one call (no recompute of the logits)."""
        cfg = cfg or self.cfg
        g = self.ctx.group_stats(cfg, self.go, self.reward, self.cs, key=self.key, alpha_in=self.alpha, beta_in=self.beta,
                                 out=self.gbuf)
        f, _, _ = self.ctx.grpo_loss_fwd_bwd(cfg, self.H, self.W, self.y, self.old, self.cs, g["adv"], g["w"], g["keep"],
                                             out=self.fbuf, dH=self.dH, dW=self.dW, workspace=self.ws)
        return g, f

    def step_dp(self, P_global):
        """The same step as one rank of a data-parallel job (counters, weights, dW and loss exchanged)."""
        from paper_2602_14338_b200 import dist as D
        g, f, _ = D.data_parallel_step(self.ctx, self.cfg, self.go, self.reward, self.cs, self.key, self.alpha, self.beta,
                                       self.H, self.W, self.y, self.old, self.gbuf, self.fbuf, self.dH, self.dW, self.ws,
                                       P_global=P_global)
        return g, f

    def step_two_calls(self):
        """The same step through the separate forward and backward calls (the backward recomputes the logits)."""
        c = self.ctx
        g = c.group_stats(self.cfg, self.go, self.reward, self.cs, key=self.key, alpha_in=self.alpha, beta_in=self.beta,
                          out=self.gbuf)
        f = c.grpo_loss_fwd(self.cfg, self.H, self.W, self.y, self.old, self.cs, g["adv"], g["w"], g["keep"], out=self.fbuf)
        c.grpo_loss_bwd(self.cfg, self.H, self.W, self.y, self.cs, g["keep"], f["lse"], f["g"], dH=self.dH, dW=self.dW,
                        workspace=self.ws, logp=f["logp"])

    def release(self):
        import torch
        for k in list(self.__dict__):
            if k not in ("base", "wl", "st", "P", "R", "T", "chunk", "cfg_over"):
                self.__dict__[k] = None
        gc.collect()
        torch.cuda.empty_cache()


def timed(fn, n, warm=1):
    """Mean milliseconds of fn over n calls after `warm` untimed ones (CUDA events on the current stream)."""
    import torch
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(n):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / n


def step_record(wl, T_kept, ms, pk, flops_per_token_factor):
    """tokens/s and the step's FLOP rate (factor * d * V FLOP per kept token) against the three peaks."""
    tf = flops_per_token_factor * T_kept * wl.d * wl.V / (ms * 1e-3) / 1e12
    return {"ms": ms, "tokens_per_s": T_kept / (ms * 1e-3), "tflops": tf, "frac_of_sustained": tf / pk["sustained"],
            "frac_of_burst": tf / pk["burst"], "frac_of_nominal_peak": tf / NOMINAL_BF16_TFLOPS}


def run_ours(args):
    import torch
    from paper_2602_14338_b200 import binding as B
    from paper_2602_14338_b200 import dist as D

    # AERO_DIST_BACKEND=gloo lets the ranks share a GPU (NCCL wants one GPU per rank): a functional check of the
    # data-parallel step where fewer GPUs than ranks are at hand, never a measurement
    rank, world, local = D.init_from_env(os.environ.get("AERO_DIST_BACKEND"))
    if world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s)")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (the library has no CPU path)")
    if local >= torch.cuda.device_count():
        if os.environ.get("AERO_DIST_BACKEND") != "gloo":
            raise SystemExit(f"bench.py: rank {rank} has no GPU of its own ({torch.cuda.device_count()} visible)")
        local = local % torch.cuda.device_count()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    pk = peaks()
    ctx = B.Context(local)
    ctx.set_tuning(gemm_sync=args.gemm_sync, gemm_pairs=args.gemm_pairs, w_hint=args.w_hint, k_zigzag=args.k_zigzag)
    if args.only_group_leg:
        print(json.dumps({"group_stage": group_stage_leg(ctx, pk, dev)}), flush=True)
        return

    t_start = time.perf_counter()
    main = Prepared(ctx, dev, args.config, rank, args.chunk_tokens, args.prompts)
    wl = main.wl
    P_global = D.total_over_ranks(main.P)
    step = (lambda: main.step_dp(P_global)) if world > 1 else main.step
    warm = max(args.warmup, 3)
    for _ in range(warm):
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
    long_step = ms_step > 1000.0

    # dominant kernel of the timed step: lmhead_kernel<MODE_FWD_P> (one launch per chunk), timed with CUDA events
    # that the library records around its launches on the context's stream, over further steps
    n_kt = 1 if long_step else 3
    ctx.enable_kernel_timing(True)
    fp_total_ms, fp_launches = 0.0, 0
    for _ in range(n_kt):
        main.step()
        ms_i, n_i = ctx.kernel_timing_ms()          # read out per step: the library keeps at most 256 pairs of events
        fp_total_ms += ms_i
        fp_launches += n_i
    ctx.enable_kernel_timing(False)
    fwdp_ms_step = fp_total_ms / n_kt
    clocks = sampler.stop()
    # the plain forward kernel (MODE_FWD, used by the separate forward call and the log-prob pass), timed over its call
    fwd_ms = timed(lambda: ctx.grpo_loss_fwd(main.cfg, main.H, main.W, main.y, main.old, main.cs, main.gbuf["adv"],
                                             main.gbuf["w"], main.gbuf["keep"], out=main.fbuf), 2 if long_step else 5)
    flops_launch = 2.0 * T_kept * wl.d * wl.V
    achieved = flops_launch / (fwdp_ms_step * 1e-3) / 1e12
    ldz = (wl.V + 63) // 64 * 64
    one_call = step_record(wl, T_kept, ms_local / args.steps, pk, 6.0)
    # the kernel is timed inside whole steps, under the power cap they run into: the sustained GEMM rate is its peak
    roofline = {"bound": "tensor", "kernel": "lmhead_kernel<MODE_FWD_P>", "achieved": achieved, "peak": pk["sustained"],
                "unit": "TFLOP/s", "frac": achieved / pk["sustained"],
                "peak_source": pk["src"] + " sustained bf16 (kernel timed inside the step)",
                "frac_of_burst": achieved / pk["burst"], "peak_burst": pk["burst"],
                "frac_of_nominal_peak": achieved / NOMINAL_BF16_TFLOPS,
                "traffic": fwdp_traffic(wl, main.chunk),
                "traffic_note": FWDP_TRAFFIC_NOTE,
                "algorithmic_bytes_per_full_launch": float(main.chunk * wl.d * 2 + wl.V * wl.d * 2 + main.chunk * ldz * 2),
                "algorithmic_bytes": float(T_kept * wl.d * 2 + wl.V * wl.d * 2 + T_kept * ldz * 2),
                "launches_per_step": fp_launches / n_kt, "ms_per_step_all_launches": fwdp_ms_step,
                "share_of_step": fwdp_ms_step / (ms_local / args.steps),
                "plain_forward_kernel": {"kernel": "lmhead_kernel<MODE_FWD>", "ms_per_launch": fwd_ms,
                                         "achieved": flops_launch / (fwd_ms * 1e-3) / 1e12,
                                         "frac": flops_launch / (fwd_ms * 1e-3) / 1e12 / pk["burst"],
                                         "peak_source": pk["src"] + " burst bf16 (kernel timed in a call of its own)",
                                         "frac_of_sustained": flops_launch / (fwd_ms * 1e-3) / 1e12 / pk["sustained"],
                                         "algorithmic_bytes": float(T_kept * wl.d * 2 + wl.V * wl.d * 2)},
                "step_executed_tflops": one_call["tflops"], "step_frac_of_sustained": one_call["frac_of_sustained"],
                "step_frac_of_burst": one_call["frac_of_burst"], "step_frac_of_nominal_peak": one_call["frac_of_nominal_peak"],
                "target": {"stage_b_frac_of_nominal_peak": TARGET_STAGE_B,
                           "met": bool(one_call["frac_of_nominal_peak"] >= TARGET_STAGE_B)}}
    # the two-call step (8 d V executed FLOPs per token), for comparison
    ms2 = timed(main.step_two_calls, 1 if long_step else 2)
    two_call = step_record(wl, T_kept, ms2, pk, 8.0)
    roofline["two_call_step"] = two_call

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warm, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
        "config": {"workload": wl.name, "P": main.P, "R": main.R, "T_input": main.T, "T_kept": T_kept, "d": wl.d, "V": wl.V,
                   "parallelism": "single GPU" if world == 1 else f"data parallel x{world}: prompts sharded, W replicated, "
                                  "all-reduce of counters, dW and loss",
                   "chunk_tokens": int(main.chunk), "step": "aero_group_stats + aero_grpo_loss_fwd_bwd (one-call step: the "
                   "forward leaves one chunk of exp(z - c_t) in bf16 for the backward)",
                   "l2": "inputs larger than L2 (H+W > 1 GB per step)", "tokens_counted": "kept tokens",
                   "input_tokens_per_s": main.T * world / (ms_step * 1e-3), "status_word": status},
        "two_call_value": two_call["tokens_per_s"],
        "two_call_note": "the same step through aero_grpo_loss_fwd + aero_grpo_loss_bwd (logits recomputed, nothing but "
                         "dz of one chunk stored)",
        "clocks": {k: clocks[k] for k in ("sm_mhz", "sm_max_mhz", "reasons")},
        "gpu_launches": int(launches),
        "roofline": roofline,
    }
    single = rank == 0 and world == 1
    if not args.no_e2e and not args.only_main:
        line["e2e"] = e2e_leg(ctx, main, args, T_kept, world, dev)
    main.release()

    if single and not args.only_main:
        subs, keep3, keep1 = {}, None, None
        for idx in [int(x) for x in args.sub_workloads.split(",") if x.strip()]:
            if idx == args.config or args.prompts > 0:
                continue
            pw = Prepared(ctx, dev, idx, rank, args.chunk_tokens)
            n = 3 if idx <= 2 else 2
            ms1 = timed(pw.step, n, warm=2)
            tk = int(pw.gbuf["counters"][1].item())
            rec = {"T_input": pw.T, "T_kept": tk, "d": pw.wl.d, "V": pw.wl.V, "steps": n,
                   "one_call": step_record(pw.wl, tk, ms1, pk, 6.0),
                   "two_call": step_record(pw.wl, tk, timed(pw.step_two_calls, 2 if idx <= 2 else 1), pk, 8.0)}
            rec["value"] = rec["one_call"]["tokens_per_s"]
            subs[pw.wl.name] = rec
            if idx == 3 and not args.no_variants_leg:
                line["k_ratio_sweep"] = k_sweep_leg(ctx, pw, pk)
            if idx == 1 and not args.no_variants_leg:
                line["variants"] = variants_leg(ctx, pw, tk, pk)
            pw.release()
        line["workloads"] = subs
        if not args.no_group_leg:
            line["group_stage"] = group_stage_leg(ctx, pk, dev)
        if not args.no_cpu_baseline:
            from paper_2602_14338_b200 import synth
            val, cores, sample, _ = time_oracle(main.base, synth.make_structure(main.base), 20.0)
            line["cpu_baseline"] = {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample}
    line["bench_wall_s"] = time.perf_counter() - t_start
    if rank == 0:
        print(json.dumps(line), flush=True)
    D.barrier()


def k_sweep_leg(ctx, pw, pk):
    """Cost of the down-sampling ratio k (Sec. 5 and the appendix give +7 / +13 / +16 % training time for k = 2, 3, 4
    on 2 x A10 with a 1.5B model): the AERO-curated batch with k = 1..4, the whole step timed per k."""
    import torch
    from paper_2602_14338_b200 import binding as B

    out, base_ms = {}, None
    for k in (1, 2, 3, 4):
        kc = B.cfg_default(**{**pw.cfg_over, "k_ratio": k})
        ms = timed(lambda: pw.step(kc), 2, warm=1)
        ck = pw.gbuf["counters"].cpu().tolist()
        base_ms = base_ms or ms
        out[str(k)] = {"kept_rollouts": ck[0], "kept_tokens": ck[1], "kept_token_fraction": ck[1] / max(ck[7], 1), "ms": ms,
                       "tokens_per_s": ck[1] / (ms * 1e-3), "time_vs_k1": ms / base_ms}
    out["paper"] = {"time_vs_k1": {"2": 1.07, "3": 1.13, "4": 1.16},
                    "context": "whole RL training step (rollout generation included) of a 1.5B model on 2 x A10; here only the "
                               "policy-objective step, whose cost follows the kept tokens"}
    return out


def variants_leg(ctx, pw, T_kept, pk):
    """The step with Eq. 2's KL term and the entropy bonus through the two calls (aero_grpo_loss_reg_fwd/_bwd) and
    through one (aero_grpo_loss_reg_fwd_bwd), the one-call step with the KL term alone (aero_grpo_loss_kl_fwd_bwd), the log-prob pass alone (aero_logprob_fwd) that produces old /
    reference log-probs, and the allocation controller on simulated prompts; on the workload passed in."""
    import copy
    import torch
    from paper_2602_14338_b200 import binding as B
    from paper_2602_14338_b200 import synth

    wl, g = pw.wl, pw.gbuf
    rcfg = copy.copy(pw.cfg)
    rcfg.kl_beta, rcfg.ent_coef = 0.04, 1e-3
    ref = (pw.old + 0.5 * pw.noise).contiguous()
    fb, lb, kb, ab = {}, {}, {}, {}

    def reg_step():
        f = ctx.grpo_loss_reg_fwd(rcfg, pw.H, pw.W, pw.y, pw.old, ref, pw.cs, g["adv"], g["w"], g["keep"], out=fb)
        ctx.grpo_loss_reg_bwd(rcfg, pw.H, pw.W, pw.y, pw.cs, g["keep"], f["lse"], f["g"], f["entropy"], g["w"], dH=pw.dH,
                              dW=pw.dW, workspace=pw.ws, logp=f["logp"])

    ms_reg = timed(reg_step, 3)
    ob = {}
    ms_reg1 = timed(lambda: ctx.grpo_loss_fwd_bwd(rcfg, pw.H, pw.W, pw.y, pw.old, pw.cs, g["adv"], g["w"], g["keep"], out=ob,
                                                  dH=pw.dH, dW=pw.dW, workspace=pw.ws, ref_logp=ref, entropy=True), 3)
    kcfg = copy.copy(pw.cfg)
    kcfg.kl_beta = 0.04
    ms_kl = timed(lambda: ctx.grpo_loss_fwd_bwd(kcfg, pw.H, pw.W, pw.y, pw.old, pw.cs, g["adv"], g["w"], g["keep"], out=kb,
                                                dH=pw.dH, dW=pw.dW, workspace=pw.ws, ref_logp=ref), 3)
    ms_lp = timed(lambda: ctx.logprob_fwd(rcfg, pw.H, pw.W, pw.y, out=lb), 3)
    # allocation controller on 2^22 simulated prompts with success rates ~ Beta(0.5, 0.5)
    Pn = 1 << 22
    thr = torch.from_numpy(synth.success_thresholds(Pn, 0.5, 0.5, seed=4301).view(np.int32)).to(pw.H.device)
    acfg = B.cfg_default(uniform_policy=B.AERO_UNIFORM_BAYES, rejection=1, k_ratio=1, seed=4302)
    l0 = ctx.launch_count()
    ctx.allocate_sim(acfg, B.alloc_cfg_default(), thr, out=ab)
    alloc_launches = ctx.launch_count() - l0
    ms_alloc = timed(lambda: ctx.allocate_sim(acfg, B.alloc_cfg_default(), thr, out=ab), 5)
    cnt = ab["counters"].cpu().tolist()
    fl = 2.0 * wl.d * wl.V
    T = pw.T
    return {"workload": wl.name,
            "allocation_sim": {"prompts": Pn, "ms": ms_alloc, "prompts_per_s": Pn / (ms_alloc * 1e-3),
                               "launches": int(alloc_launches), "mean_rollouts_generated": cnt[0] / Pn,
                               "mean_rollouts_trained": cnt[1] / Pn, "zero_accuracy_before": cnt[2] / Pn,
                               "zero_accuracy_after": cnt[3] / Pn, "iterations": cnt[5]},
            "regularised_step": {"kl_beta": 0.04, "ent_coef": 1e-3, "ms": ms_reg, "tokens_per_s": T_kept / (ms_reg * 1e-3),
                                 "executed_tflops": 4 * fl * T_kept / (ms_reg * 1e-3) / 1e12,
                                 "frac_of_sustained": 4 * fl * T_kept / (ms_reg * 1e-3) / 1e12 / pk["sustained"]},
            "regularised_step_one_call": {"kl_beta": 0.04, "ent_coef": 1e-3, "ms": ms_reg1,
                                          "tokens_per_s": T_kept / (ms_reg1 * 1e-3),
                                          "executed_tflops": 3 * fl * T_kept / (ms_reg1 * 1e-3) / 1e12,
                                          "frac_of_sustained": 3 * fl * T_kept / (ms_reg1 * 1e-3) / 1e12 / pk["sustained"],
                                          "api": "aero_grpo_loss_reg_fwd_bwd"},
            "kl_step_one_call": {"kl_beta": 0.04, "ms": ms_kl, "tokens_per_s": T_kept / (ms_kl * 1e-3),
                                 "executed_tflops": 3 * fl * T_kept / (ms_kl * 1e-3) / 1e12,
                                 "frac_of_sustained": 3 * fl * T_kept / (ms_kl * 1e-3) / 1e12 / pk["sustained"]},
            "logprob_pass": {"rows": T, "ms": ms_lp, "tokens_per_s": T / (ms_lp * 1e-3),
                             "tflops": fl * T / (ms_lp * 1e-3) / 1e12, "frac_of_burst": fl * T / (ms_lp * 1e-3) / 1e12 / pk["burst"]}}


def group_stage_leg(ctx, pk, dev):
    """Stage (a) alone on an input large enough to be bandwidth-bound (2^22 prompts of 2..16 rollouts):
    algorithmic bytes (37 per rollout + 26 per prompt) over the duration of the stage's launches."""
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
            "target": {"stage_a_frac_of_hbm": TARGET_STAGE_A, "met": bool(gbs / pk["hbm"] >= TARGET_STAGE_A)},
            "kept_rollout_frac": float(out["metrics"][2].item())}


def e2e_leg(ctx, pw, args, T_kept, world, dev):
    """Same step through the host-buffer entry point: inputs in pinned host memory, copies inside the timed region.
    With several ranks every rank runs it on its own batch and dW is all-reduced afterwards (the host-buffer call
    normalises over the rank's own batch)."""
    import torch
    from paper_2602_14338_b200 import dist as D

    st, wl, cfg = pw.st, pw.wl, pw.cfg
    P, R, T = pw.P, pw.R, pw.T
    # every rank pins its own copy of H: leave the leg out where the ranks' copies together would take more than
    # half of the host memory that is free (all ranks decide alike)
    need = float(pw.H.numel() * pw.H.element_size())
    try:
        import psutil
        free = float(psutil.virtual_memory().available)
    except Exception:
        free = float("inf")
    fits = torch.tensor([1.0 if need * world < 0.5 * free else 0.0], dtype=torch.float64, device=dev)
    if world > 1:
        torch.distributed.all_reduce(fits, op=torch.distributed.ReduceOp.MIN)
    if fits.item() == 0.0:
        return {"value": None, "unit": UNIT, "h2d_bytes_per_step": None, "d2h_bytes_per_step": None,
                "skipped": f"{world} ranks x {need / 1e9:.1f} GB of pinned H against {free / 1e9:.0f} GB of free host memory"}
    pw.ws = None                                   # the host-buffer call has a workspace of its own
    gc.collect()
    torch.cuda.empty_cache()
    pin = lambda x: x.pin_memory()
    go_h, rw_h, cs_h = pin(torch.from_numpy(st.go)), pin(torch.from_numpy(st.reward)), pin(torch.from_numpy(st.cs))
    key_h = pin(torch.from_numpy(st.key.view(np.int32)))
    al_h = pin(torch.from_numpy(st.alpha)) if st.alpha is not None else None
    be_h = pin(torch.from_numpy(st.beta)) if st.beta is not None else None
    H_h = torch.empty(pw.H.shape, dtype=pw.H.dtype, pin_memory=True)
    H_h.copy_(pw.H)
    y_h, old_h = pin(torch.from_numpy(st.y)), pin(pw.old.cpu())
    ws = torch.empty(ctx.step_workspace_bytes(P, R, T, wl.d, wl.V, pw.chunk, cfg.dtype), dtype=torch.uint8, device=dev)
    h2d = H_h.numel() * H_h.element_size() + 8 * T + 4 * (P + 1) + 16 * R + 8 + (8 * P if al_h is not None else 0)
    d2h = 4 + 64 + 32
    n = 2 if T > 2_000_000 else max(2, min(args.steps, 5))

    def host_step():
        out = ctx.grpo_step_host(cfg, go_h, rw_h, cs_h, key_h, al_h, be_h, H_h, y_h, old_h, pw.W, pw.dH, pw.dW, ws)
        if world > 1:
            D.reduce_sum_(pw.dW)
            torch.cuda.synchronize()
        return out

    host_step()
    torch.cuda.synchronize()
    D.barrier()
    t0 = time.perf_counter()
    for _ in range(n):
        loss, counters, _ = host_step()
    dt = (time.perf_counter() - t0) / n
    assert int(counters[1]) == T_kept
    units, ms_total = D.aggregate(T_kept, dt * 1e3, device=dev)
    del ws, H_h
    return {"value": units / (ms_total * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
            "ms_per_step": ms_total, "steps": n, "loss": float(loss.item()),
            "api": "aero_grpo_step_host (pinned host inputs; H copied in slices under the first chunks' kernels)"}


def spawn_ranks(args):
    """`--gpus N` without a launcher: start N ranks of this script under torch.distributed.run."""
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd))


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    elif a.gpus > 1 and "WORLD_SIZE" not in os.environ:
        spawn_ranks(a)
    else:
        run_ours(a)
