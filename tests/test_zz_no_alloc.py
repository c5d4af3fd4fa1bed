"""The entry point that takes its scratch from the library's own device array
(aero_group_stats_static) must give what aero_group_stats gives with a caller workspace.

Collected last on purpose: the array is shared by every call in the process, so this file
also shows that the call works after everything else has run; it works equally when it is
the only test of a fresh process (the first call then does the per-device address lookup).
Two calls in a row with different batches check that what the first call left in the array
does not leak into the second."""
import numpy as np
import pytest
import torch

from oracle import aero_oracle as O
from paper_2602_14338_b200 import binding as B
from paper_2602_14338_b200 import synth
from tests import aero_testlib as TL

pytestmark = pytest.mark.gpu


def _outputs(P, R):
    z = lambda n, dt: torch.zeros(max(n, 1), dtype=dt, device="cuda")
    size = {"R": R, "P": P, "R1": R + 1, "8": 8, "4": 4}
    return {name: z(size[n], dt) for name, n, dt in B.Context.GROUP_OUTPUTS}


def _compare(a, b, P, R):
    for name, n, dt in B.Context.GROUP_OUTPUTS:
        k = {"R": R, "P": P, "R1": R + 1, "8": 8, "4": 4}[n]
        x, y = a[name][:k].cpu(), b[name][:k].cpu()
        if dt in (torch.float32,):
            # same kernels, same order of operations: the tolerance of the other group tests is ample
            np.testing.assert_allclose(x.numpy(), y.numpy(), rtol=2e-5, atol=1e-6, err_msg=name)
        else:
            assert torch.equal(x, y), name


def test_static_scratch_matches_workspace_entry_point_twice():
    ctx = B.Context(0)
    cases = [
        (synth.scaled(synth.WORKLOADS[3], P=2000, seed=501), dict(uniform_policy=O.UNIFORM_BAYES, rejection=1), False),
        (synth.scaled(synth.WORKLOADS[1], P=37, seed=502), dict(), False),      # smaller: stale scratch beyond it
        # per-prompt kept counts go through the array only under the sequence mean; absent rollouts too
        (synth.scaled(synth.WORKLOADS[3], P=900, seed=503),
         dict(uniform_policy=O.UNIFORM_BAYES, rejection=1, agg=O.AGG_SEQ_MEAN), True),
    ]
    for n_call, (wl, mode, with_keep_in) in enumerate(cases):
        st = synth.make_structure(wl)
        P, R = len(st.go) - 1, len(st.reward)
        cfg = TL.lib_cfg(O.Cfg(seed=wl.seed, **mode), "bf16")
        gi = TL.group_inputs_device(st)
        keep_in_h = (np.random.default_rng(9).random(R) < 0.85).astype(np.uint8) if with_keep_in else None
        keep_in = TL.dev(keep_in_h) if with_keep_in else None
        ref = ctx.group_stats(cfg, gi["go"], gi["reward"], gi["cs"], key=gi["key"], keep_in=keep_in,
                              alpha_in=gi["alpha"], beta_in=gi["beta"])
        out = _outputs(P, R)
        torch.cuda.synchronize()
        # free device memory as the driver reports it (it sees every allocation of the process, not only
        # torch's); the first call on a device may load the kernels' module, so the check starts with the second
        free_before = torch.cuda.mem_get_info()[0]
        held_before = torch.cuda.memory_allocated()
        ctx.group_stats_static(cfg, gi["go"], gi["reward"], gi["cs"], out, key=gi["key"], keep_in=keep_in,
                               alpha_in=gi["alpha"], beta_in=gi["beta"])
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == held_before      # the binding allocated nothing either
        if n_call > 0:
            assert torch.cuda.mem_get_info()[0] >= free_before
        _compare(out, ref, P, R)
        # and both agree with the oracle on what is exact
        oref = O.group_stats(O.Cfg(seed=wl.seed, **mode), st.go, st.reward, st.cs, key=st.key, keep_in=keep_in_h,
                             alpha_in=st.alpha, beta_in=st.beta)
        assert np.array_equal(out["keep"][:R].cpu().numpy(), oref["keep"])
        assert np.array_equal(out["counters"].cpu().numpy(), oref["counters"])
    assert ctx.last_status() == 0
    ctx.close()


def test_static_scratch_rejects_too_many_prompts():
    ctx = B.Context(0)
    P = 65536 + 1
    go = torch.arange(P + 1, dtype=torch.int32, device="cuda")
    rw = torch.zeros(P, dtype=torch.float32, device="cuda")
    cs = torch.arange(P + 1, dtype=torch.int64, device="cuda")
    out = _outputs(P, P)
    with pytest.raises(B.AeroError, match="scratch"):
        ctx.group_stats_static(B.cfg_default(), go, rw, cs, out)
    # the limit itself is accepted
    P = 65536
    out = _outputs(P, P)
    ctx.group_stats_static(B.cfg_default(), go[:P + 1].contiguous(), rw[:P].contiguous(), cs[:P + 1].contiguous(), out)
    assert int(out["counters"][0]) == 0          # single all-incorrect rollouts: every group masked
    assert ctx.last_status() == 0
    ctx.close()
