"""GPU tests of the boundary itself: every error code for the argument error it names, the device
status word on a side stream, the bounded-wait self-test, the tuning hook's argument checks, and
the data-parallel weight finalisation (two prompt shards on one GPU against the unsharded batch)."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import aero_oracle as O
from paper_2602_14338_b200 import binding as B
from paper_2602_14338_b200 import dist as D
from paper_2602_14338_b200 import synth
from tests import aero_testlib as TL

pytestmark = pytest.mark.gpu

ERR_INVALID, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TOO_LARGE = -1, -2, -3, -4, -5


@pytest.fixture(scope="module")
def ctx():
    c = B.Context(0)
    yield c
    assert c.last_status() == 0
    c.close()


def _small_problem():
    wl = synth.scaled(synth.WORKLOADS[1], P=3, n_lo=4, n_hi=4, d=64, V=300, len_median=30.0, len_cap=64, seed=21)
    batch = TL.Batch(wl, O.Cfg())
    return wl, batch, batch.to_device()


def test_every_error_code_is_returned_for_its_argument_error(ctx):
    lib = ctx.lib
    wl, batch, dv = _small_problem()
    T, d, V, R, P = batch.T, wl.d, wl.V, batch.R, batch.P
    cfg = TL.lib_cfg(batch.ocfg, "bf16")
    z = lambda n, dt=torch.float32: torch.zeros(max(n, 1), dtype=dt, device="cuda")
    logp, lse, g, loss = z(T), z(T), z(T), z(1)
    ws = torch.empty(ctx.fwd_bwd_workspace_bytes(T, d, V, R, 128), dtype=torch.uint8, device="cuda")
    p = lambda t: t.data_ptr()

    def fwd(H=dv["H"], W=dv["W"], dd=d, cfgp=cfg, wsp=None, wsb=None, logp_=logp, ctxh=ctx.h):
        return lib.aero_grpo_loss_fwd(ctxh, C.byref(cfgp), T, dd, V, R, p(H) if H is not None else None, p(W), p(dv["y"]),
                                      p(dv["old"]), p(dv["cs"]), p(dv["adv"]), p(dv["w"]), p(dv["keep"]),
                                      p(logp_) if logp_ is not None else None, p(lse), p(g), p(loss), None, 0,
                                      p(ws) if wsp is None else wsp, ws.numel() if wsb is None else wsb)

    assert fwd() == 0
    assert fwd(H=None) == ERR_INVALID                       # null input
    assert fwd(logp_=None) == ERR_INVALID                   # null output
    assert fwd(ctxh=None) == ERR_INVALID                    # no context
    assert fwd(wsp=p(ws) + 16) == ERR_INVALID               # workspace not 256-byte aligned
    assert fwd(dd=d - 8) == ERR_UNSUPPORTED                 # d not a multiple of 64 on the tensor-core path
    bad = TL.lib_cfg(batch.ocfg, "bf16")
    bad.dtype = 7
    assert fwd(cfgp=bad) == ERR_UNSUPPORTED                 # unknown dtype
    assert fwd(wsb=1024) == ERR_WORKSPACE                   # workspace too small
    Hoff = torch.empty(T * d + 8, dtype=torch.bfloat16, device="cuda")[1:T * d + 1].view(T, d)
    assert fwd(H=Hoff) == ERR_INVALID                       # base not 16-byte aligned

    dH, dW = torch.empty_like(dv["H"]), z(V * d)

    def bwd(wsb=None, dHp=dH, T_=T):
        return lib.aero_grpo_loss_bwd(ctx.h, C.byref(cfg), T_, d, V, R, p(dv["H"]), p(dv["W"]), p(dv["y"]), p(dv["cs"]),
                                      p(dv["keep"]), p(lse), p(g), None, C.c_float(1.0), p(dHp) if dHp is not None else None,
                                      p(dW), 0, p(ws), ws.numel() if wsb is None else wsb)

    assert bwd() == 0
    assert bwd(dHp=None) == ERR_INVALID
    assert bwd(T_=-1) == ERR_INVALID
    assert bwd(T_=1 << 31) == ERR_INVALID                   # row coordinates are 32-bit
    assert bwd(wsb=4096) == ERR_WORKSPACE

    def fwd_bwd(wsb):
        return lib.aero_grpo_loss_fwd_bwd(ctx.h, C.byref(cfg), T, d, V, R, p(dv["H"]), p(dv["W"]), p(dv["y"]), p(dv["old"]),
                                          p(dv["cs"]), p(dv["adv"]), p(dv["w"]), p(dv["keep"]), p(logp), p(lse), p(g),
                                          p(loss), None, C.c_float(1.0), p(dH), p(dW), 0, p(ws), wsb)

    assert fwd_bwd(ws.numel()) == 0
    assert fwd_bwd(4096) == ERR_WORKSPACE

    # group stage
    st = batch.st
    gi = TL.group_inputs_device(st)
    out = {n: torch.zeros(max({"R": R, "P": P, "R1": R + 1, "8": 8, "4": 4}[k], 1), dtype=dt, device="cuda")
           for n, k, dt in B.Context.GROUP_OUTPUTS}
    gws = torch.empty(ctx.group_workspace_bytes(P, R), dtype=torch.uint8, device="cuda")

    def group(cfgp=cfg, alpha=None, beta=None, wsb=None, P_=P):
        ptrs = [p(out[n]) for n, _, _ in B.Context.GROUP_OUTPUTS]
        return lib.aero_group_stats(ctx.h, C.byref(cfgp), P_, R, p(gi["go"]), p(gi["reward"]), p(gi["cs"]), None, None,
                                    alpha, beta, *ptrs, p(gws), gws.numel() if wsb is None else wsb)

    assert group() == 0
    assert group(alpha=p(z(P))) == ERR_INVALID              # a prior needs both parameters
    k0 = TL.lib_cfg(batch.ocfg, "bf16")
    k0.k_ratio = 0
    assert group(cfgp=k0) == ERR_INVALID                    # k >= 1
    assert group(P_=-1) == ERR_INVALID
    assert group(wsb=16) == ERR_WORKSPACE
    # the entry point with library-owned scratch has a size limit of its own
    ptrs = [p(out[n]) for n, _, _ in B.Context.GROUP_OUTPUTS]
    rc = lib.aero_group_stats_static(ctx.h, C.byref(cfg), 65537, 65537, p(gi["go"]), p(gi["reward"]), p(gi["cs"]), None, None,
                                     None, None, *ptrs)
    assert rc == ERR_TOO_LARGE
    # a device that does not exist
    h = C.c_void_p()
    assert lib.aero_create(C.byref(h), 4096, None) == ERR_CUDA
    assert lib.aero_create(None, 0, None) == ERR_INVALID
    # tuning hook
    assert lib.aero_set_tuning(ctx.h, b"vsplit", 3) == ERR_INVALID
    assert lib.aero_set_tuning(ctx.h, b"vsplit", 8) == ERR_INVALID
    assert lib.aero_set_tuning(ctx.h, b"no_such_setting", 1) == ERR_INVALID
    assert lib.aero_set_tuning(ctx.h, None, 1) == ERR_INVALID
    assert lib.aero_set_tuning(ctx.h, b"vsplit", 2) == 0 and lib.aero_set_tuning(ctx.h, b"vsplit", 0) == 0
    assert lib.aero_set_tuning(ctx.h, b"gemm_sync", 3) == 0 and lib.aero_set_tuning(ctx.h, b"gemm_sync", -1) == 0
    for code in (ERR_INVALID, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TOO_LARGE):
        assert lib.aero_error_string(code) not in (b"ok", b"unknown error")
    torch.cuda.synchronize()
    assert ctx.last_status() == 0


def test_bounded_wait_runs_out_and_reports_it(ctx):
    """A wait on a barrier nobody arrives at (a kernel of its own, one warp) gives up after its limit, raises
    AERO_ST_TIMEOUT and ends normally; the context and the device stay usable."""
    assert ctx.last_status() == 0
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    ctx.selftest_bounded_wait(1000)                         # 1 ms
    t1.record()
    torch.cuda.synchronize()
    assert 0.9 <= t0.elapsed_time(t1) < 100.0
    assert ctx.last_status() == B.AERO_ST_TIMEOUT
    assert ctx.last_status() == 0
    wl, batch, dv = _small_problem()
    cfg = TL.lib_cfg(batch.ocfg, "bf16")
    f = ctx.grpo_loss_fwd(cfg, dv["H"], dv["W"], dv["y"], dv["old"], dv["cs"], dv["adv"], dv["w"], dv["keep"])
    ref = batch.oracle_fwd()
    assert np.abs(f["logp"][:batch.T].cpu().numpy() - ref["logp"]).max() <= 1e-2
    assert ctx.last_status() == 0
    with pytest.raises(B.AeroError):
        ctx.selftest_bounded_wait(0)


def test_status_word_on_a_side_stream():
    """The status word is read and cleared in the order of the context's own stream, also when that
    stream does not synchronise with the default stream."""
    side = torch.cuda.Stream()
    c = B.Context(0, stream=side)
    wl, batch, dv = _small_problem()
    cfg = TL.lib_cfg(batch.ocfg, "bf16")
    y_bad = dv["y"].clone()
    y_bad[5] = wl.V + 3
    keep = torch.ones_like(dv["keep"])
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        for _ in range(20):
            c.grpo_loss_fwd(cfg, dv["H"], dv["W"], dv["y"], dv["old"], dv["cs"], dv["adv"], dv["w"], keep)
            assert c.last_status() == 0
            c.grpo_loss_fwd(cfg, dv["H"], dv["W"], y_bad, dv["old"], dv["cs"], dv["adv"], dv["w"], keep)
            assert c.last_status() == B.AERO_ST_BAD_TARGET
    assert c.last_status() == 0
    c.close()


@pytest.mark.parametrize("mode", [dict(), dict(uniform_policy=O.UNIFORM_BAYES, rejection=1, agg=O.AGG_SEQ_MEAN),
                                  dict(rejection=1, denom=O.DENOM_ALL), dict(agg=O.AGG_SEQ_MEAN, denom=O.DENOM_ALL)])
def test_two_prompt_shards_on_one_gpu_equal_the_unsharded_batch(ctx, mode):
    """The data-parallel step's arithmetic with both shards run one after the other on one GPU: group stage per
    shard, counters summed, aero_finalize_weights, stage (b) per shard with loss and dW accumulated; against the
    library on the unsharded batch and against the oracle."""
    wl = synth.scaled(synth.WORKLOADS[3], P=40, n_lo=2, n_hi=9, d=128, V=1000, len_median=24.0, len_cap=60, seed=93)
    batch = TL.Batch(wl, O.Cfg(seed=wl.seed, **mode))
    st, ocfg = batch.st, batch.ocfg
    cfg = TL.lib_cfg(ocfg, "bf16")
    dv = batch.to_device()
    ref = batch.oracle_fwd()
    rdH, rdW = batch.oracle_bwd(ref)
    shards = []
    for r in range(2):
        p0, p1 = D.shard_prompts(st.go, st.cs, 2, r)
        go_l, cs_l, r0, r1, t0, t1 = D.shard_offsets(st.go, st.cs, p0, p1)
        sl = lambda a, lo, hi: None if a is None else TL.dev(a[lo:hi])
        g = ctx.group_stats(cfg, TL.dev(go_l), TL.dev(st.reward[r0:r1]), TL.dev(cs_l), key=TL.dev(st.key[r0:r1].view(np.int32)),
                            alpha_in=sl(st.alpha, p0, p1), beta_in=sl(st.beta, p0, p1))
        shards.append(dict(p=(p0, p1), r=(r0, r1), t=(t0, t1), cs=TL.dev(cs_l), g=g))
    assert shards[0]["p"][1] == shards[1]["p"][0] and 0 < shards[0]["p"][1] < wl.P
    total = shards[0]["g"]["counters"] + shards[1]["g"]["counters"]
    assert total.cpu().tolist() == batch.ref_g["counters"].tolist()
    dW = torch.zeros((wl.V, wl.d), dtype=torch.float32, device="cuda")
    dH = torch.empty_like(dv["H"])
    loss = 0.0
    w_all = []
    for s in shards:
        (p0, p1), (r0, r1), (t0, t1), g = s["p"], s["r"], s["t"], s["g"]
        ctx.finalize_weights(cfg, g["w"], g["counters"], total, p1 - p0, wl.P)
        w_all.append(g["w"][:r1 - r0].cpu().numpy())
        f, _, _ = ctx.grpo_loss_fwd_bwd(cfg, dv["H"][t0:t1], dv["W"], dv["y"][t0:t1], dv["old"][t0:t1], s["cs"], g["adv"],
                                        g["w"], g["keep"], dH=dH[t0:t1], dW=dW, accumulate_dW=True)
        loss += f["loss"].item()
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    np.testing.assert_allclose(np.concatenate(w_all), batch.ref_g["w"], rtol=2e-6, atol=0)
    assert abs(loss - ref["loss"]) <= 1e-3 * abs(ref["loss"]) + 1e-7
    rho = ref["rho"]
    edge = (np.abs(rho - 1.2) < 1e-3) | (np.abs(rho - 0.8) < 1e-3)
    assert TL.rel_l2(dH.float().cpu().numpy()[~edge], rdH[~edge]) < 1e-2
    if not edge.any():
        assert TL.rel_l2(dW.cpu().numpy(), rdW) < 1e-2
