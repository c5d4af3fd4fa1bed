"""Data-parallel plumbing: one process per GPU, `torch.distributed` for the exchange.

The path shards by prompt.  Eq. 1 is per prompt, so advantages, categories, posteriors and the
keep-mask of a shard need nothing from the other ranks; token rows are independent given
(advantage, weight).  What is batch-wide are Eq. 2's normalisers (1/T_kept for the token mean of
Appendix C, 1/(P_surv n'_p |o_i|) for Eq. 2 itself) and the sums that make the loss and dW.  One
data-parallel step of a rank is therefore:

  1. aero_group_stats on the rank's own prompts
  2. all-reduce (sum) of the eight group counters                      -- 64 bytes
  3. aero_finalize_weights: local -> batch-wide denominators, on the device
  4. aero_grpo_loss_fwd_bwd on the rank's own token rows (W replicated)
  5. all-reduce (sum) of dW [V,d] fp32 and of the loss; dH stays local

The collectives are plain `all_reduce` calls of the process group (NCCL over NVLink on GPUs,
gloo on CPU): the operands are this rank's own buffers, no kernel of the library reads a peer's
memory, and nothing here uses a multicast load.

`weight_factor` states the arithmetic of step 3 on the host as well, for callers that hold the
weights in host memory (the CPU tests of this module do).
"""
from __future__ import annotations

import os

import numpy as np
import torch
import torch.distributed as dist

# indices into the group counters (AERO_CNT_* of include/aero.h)
CNT_R_KEPT, CNT_T_KEPT, CNT_P_SURV, CNT_T_PRESENT = 0, 1, 2, 7
TOKEN_MEAN, SEQ_MEAN = 0, 1
DENOM_SURVIVING, DENOM_ALL = 0, 1


def init_from_env(backend: str | None = None):
    """(rank, world, local_rank); initialises the process group when WORLD_SIZE > 1."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend or ("nccl" if torch.cuda.is_available() else "gloo"),
                                rank=rank, world_size=world)
    return rank, world, local


def barrier():
    if dist.is_initialized():
        dist.barrier()


def aggregate(units: float, elapsed_ms: float, device="cpu"):
    """Whole-job totals: sum of the units every rank processed and the slowest rank's time."""
    if not dist.is_initialized():
        return float(units), float(elapsed_ms)
    u = torch.tensor([float(units)], dtype=torch.float64, device=device)
    t = torch.tensor([float(elapsed_ms)], dtype=torch.float64, device=device)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(u.item()), float(t.item())


# ----------------------------------------------------------------------------- sharding
def shard_prompts(go, cs, world: int, rank: int):
    """Contiguous prompt range [p0, p1) of `rank`: boundaries where the running token count passes
    k/world of the total, so that ranks get about the same number of token rows.  Every prompt belongs
    to exactly one rank; a rank may get no prompt when there are fewer prompts than ranks."""
    go = np.asarray(go, dtype=np.int64)
    cs = np.asarray(cs, dtype=np.int64)
    P = len(go) - 1
    tok_before = cs[go]                      # token rows before each prompt, [P+1]
    total = int(tok_before[-1])
    bounds = [0]
    for k in range(1, world):
        p = int(np.searchsorted(tok_before, total * k / world, side="left"))
        bounds.append(min(max(p, bounds[-1]), P))
    bounds.append(P)
    return bounds[rank], bounds[rank + 1]


def shard_offsets(go, cs, p0: int, p1: int):
    """Offsets of a prompt range re-based to start at zero: (go_local, cs_local, r0, r1, t0, t1)."""
    go = np.asarray(go, dtype=np.int64)
    cs = np.asarray(cs, dtype=np.int64)
    r0, r1 = int(go[p0]), int(go[p1])
    t0, t1 = int(cs[r0]), int(cs[r1])
    return (go[p0:p1 + 1] - r0).astype(np.int32), (cs[r0:r1 + 1] - t0).astype(np.int64), r0, r1, t0, t1


# ----------------------------------------------------------------------------- exchange steps
def reduce_counters(counters_local: torch.Tensor) -> torch.Tensor:
    """Element-wise sum over ranks of the group counters ([8] int64, on whatever device they live)."""
    g = counters_local.clone()
    if dist.is_initialized():
        dist.all_reduce(g, op=dist.ReduceOp.SUM)
    return g


def reduce_sum_(t: torch.Tensor) -> torch.Tensor:
    """In-place sum over ranks (dW, the loss)."""
    if dist.is_initialized():
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return t


def total_over_ranks(n: int) -> int:
    """Sum of a host integer over ranks (the global number of prompts)."""
    if not dist.is_initialized():
        return int(n)
    t = torch.tensor([int(n)], dtype=torch.int64,
                     device="cuda" if dist.get_backend() == "nccl" else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return int(t.item())


def weight_factor(agg: int, denom: int, counters_local, counters_global, P_local: int, P_global: int) -> float:
    """local / batch-wide denominator of Eq. 2's normalisers (what aero_finalize_weights applies on the
    device): kept tokens for the token mean, surviving prompts for the sequence mean; present tokens,
    resp. all prompts, when dropped ones count too."""
    cl = [int(x) for x in counters_local]
    cg = [int(x) for x in counters_global]
    if agg == TOKEN_MEAN:
        k = CNT_T_KEPT if denom == DENOM_SURVIVING else CNT_T_PRESENT
        num, den = cl[k], cg[k]
    elif denom == DENOM_SURVIVING:
        num, den = cl[CNT_P_SURV], cg[CNT_P_SURV]
    else:
        num, den = P_local, P_global
    return num / den if den > 0 else 0.0


# ----------------------------------------------------------------------------- one step on a GPU rank
def data_parallel_step(ctx, cfg, go, reward, cs, key, alpha, beta, H, W, y, old_logp, gbuf, fbuf, dH, dW,
                       workspace, P_global: int | None = None):
    """Steps 1-5 above for this rank's shard (device tensors; `ctx` a binding.Context).  Returns the
    group outputs, the forward outputs (loss summed over ranks) and the batch-wide counters."""
    P_local = go.numel() - 1
    if P_global is None:
        P_global = total_over_ranks(P_local)
    g = ctx.group_stats(cfg, go, reward, cs, key=key, alpha_in=alpha, beta_in=beta, out=gbuf)
    counters_global = g["counters"]
    if dist.is_initialized() and dist.get_world_size() > 1:
        counters_global = reduce_counters(g["counters"])
        ctx.finalize_weights(cfg, g["w"], g["counters"], counters_global, P_local, P_global)
    f, _, _ = ctx.grpo_loss_fwd_bwd(cfg, H, W, y, old_logp, cs, g["adv"], g["w"], g["keep"], out=fbuf, dH=dH, dW=dW,
                                    workspace=workspace)
    reduce_sum_(dW)
    reduce_sum_(f["loss"])
    return g, f, counters_global
