"""World-size-2 checks (gloo, CPU) of the multi-rank plumbing.

* timing plumbing: rendezvous from the environment, barrier, sum-of-units / max-of-time;
* the data-parallel step's exchange logic (paper_2602_14338_b200/dist.py): two ranks take
  disjoint prompt ranges, all-reduce the group counters, bring their weights to the batch-wide
  denominators of Eq. 2, and sum loss and dW; the result must equal the oracle on the unsharded
  batch.  There is no GPU here, so each rank's own compute is done by the oracle (tests may call
  it; the library's kernels take its place on a GPU rank) -- what is under test is the partition
  and the reductions.
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2602_14338_b200 import dist as D
    import torch.distributed as dist

    r, w, _ = D.init_from_env("gloo")
    D.barrier()
    units, ms = D.aggregate(100.0 * (r + 1), 10.0 + 5.0 * r)
    q.put((r, w, units, ms))
    D.barrier()
    dist.destroy_process_group()


def _run(target, world, *args):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=target, args=(r, world, port, q) + args) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted((q.get(timeout=300) for _ in procs), key=lambda g: g[0])
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    return got


def test_two_rank_aggregate():
    got = _run(_worker, 2)
    assert [g[0] for g in got] == [0, 1] and all(g[1] == 2 for g in got)
    assert all(g[2] == 300.0 and g[3] == 15.0 for g in got)


def test_single_process_passthrough():
    from paper_2602_14338_b200 import dist as D

    assert D.aggregate(7.0, 3.5) == (7.0, 3.5)
    assert D.total_over_ranks(5) == 5
    c = torch.arange(8, dtype=torch.int64)
    assert torch.equal(D.reduce_counters(c), c)


def test_shard_prompts_is_a_partition_balanced_by_tokens():
    from paper_2602_14338_b200 import dist as D
    from paper_2602_14338_b200 import synth

    st = synth.make_structure(synth.scaled(synth.WORKLOADS[3], P=97, seed=9))
    for world in (1, 2, 3, 8):
        ranges = [D.shard_prompts(st.go, st.cs, world, r) for r in range(world)]
        assert ranges[0][0] == 0 and ranges[-1][1] == 97
        assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
        toks = [int(st.cs[st.go[b]] - st.cs[st.go[a]]) for a, b in ranges]
        assert sum(toks) == int(st.cs[-1])
        assert max(toks) - min(toks) <= 2 * int((st.cs[st.go[1:]] - st.cs[st.go[:-1]]).max())
    # more ranks than prompts: some ranks get nothing, every prompt still has one owner
    small = synth.make_structure(synth.scaled(synth.WORKLOADS[1], P=2, seed=3))
    ranges = [D.shard_prompts(small.go, small.cs, 4, r) for r in range(4)]
    assert sum(b - a for a, b in ranges) == 2


def test_weight_factor_hand_values():
    from paper_2602_14338_b200 import dist as D

    cl = [3, 40, 2, 0, 0, 0, 0, 100]        # R_kept, T_kept, P_surv, ..., T_present
    cg = [9, 160, 5, 0, 0, 0, 0, 400]
    assert D.weight_factor(D.TOKEN_MEAN, D.DENOM_SURVIVING, cl, cg, 4, 10) == 0.25
    assert D.weight_factor(D.TOKEN_MEAN, D.DENOM_ALL, cl, cg, 4, 10) == 0.25
    assert D.weight_factor(D.SEQ_MEAN, D.DENOM_SURVIVING, cl, cg, 4, 10) == 0.4
    assert D.weight_factor(D.SEQ_MEAN, D.DENOM_ALL, cl, cg, 4, 10) == 0.4
    assert D.weight_factor(D.TOKEN_MEAN, D.DENOM_SURVIVING, [0] * 8, [0] * 8, 0, 0) == 0.0


MODES = [dict(), dict(uniform_policy=1, rejection=1, agg=1), dict(rejection=1, denom=1), dict(agg=1, denom=1)]


def _dp_worker(rank, world, port, q, mode_idx):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    torch.set_num_threads(2)
    import torch.distributed as dist
    from oracle import aero_oracle as O
    from paper_2602_14338_b200 import dist as D
    from paper_2602_14338_b200 import synth

    D.init_from_env("gloo")
    wl, st, H, W, old, rows = _dp_batch(synth)
    ocfg = O.Cfg(seed=wl.seed, **MODES[mode_idx])
    p0, p1 = D.shard_prompts(st.go, st.cs, world, rank)
    go_l, cs_l, r0, r1, t0, t1 = D.shard_offsets(st.go, st.cs, p0, p1)
    sl = lambda a, lo, hi: None if a is None else a[lo:hi]
    # 1. group stage on the rank's own prompts
    g = O.group_stats(ocfg, go_l, st.reward[r0:r1], cs_l, key=st.key[r0:r1],
                      alpha_in=sl(st.alpha, p0, p1), beta_in=sl(st.beta, p0, p1))
    # 2. + 3. batch-wide counters, then the weights' denominators
    c_loc = torch.from_numpy(g["counters"].copy())
    c_glob = D.reduce_counters(c_loc)
    P_glob = D.total_over_ranks(p1 - p0)
    w = g["w"] * D.weight_factor(ocfg.agg, ocfg.denom, c_loc.tolist(), c_glob.tolist(), p1 - p0, P_glob)
    # 4. stage (b) on the rank's own rows
    f = O.grpo_loss_fwd(ocfg, H[t0:t1], W, st.y[t0:t1], old[t0:t1], cs_l, g["adv"], w, g["keep"])
    dH, dW = O.grpo_loss_bwd(H[t0:t1], W, st.y[t0:t1], cs_l, g["keep"], f["lse"], f["g"], dw_rows=rows)
    # 5. sums over ranks
    dW_t = D.reduce_sum_(torch.from_numpy(np.ascontiguousarray(dW)))
    loss_t = D.reduce_sum_(torch.tensor([f["loss"]], dtype=torch.float64))
    q.put((rank, (p0, p1), c_glob.tolist(), P_glob, w, dH, dW_t.numpy(), float(loss_t.item())))
    D.barrier()
    dist.destroy_process_group()


def _dp_batch(synth):
    wl = synth.scaled(synth.WORKLOADS[3], P=9, n_lo=2, n_hi=7, d=32, V=200, len_median=12.0, len_cap=30, seed=88)
    st = synth.make_structure(wl)
    T = int(st.cs[-1])
    Ht, Wt = synth.make_tensors(wl, T)
    H, W = Ht.double().numpy(), Wt.double().numpy()
    old = (-5.0 + st.noise.astype(np.float64) * 6).astype(np.float64)       # some tokens clipped, most not
    rows = np.arange(wl.V)
    return wl, st, H, W, old, rows


@pytest.mark.parametrize("mode_idx", range(len(MODES)))
def test_two_prompt_shards_reduce_to_the_unsharded_batch(mode_idx):
    from oracle import aero_oracle as O
    from paper_2602_14338_b200 import synth

    got = _run(_dp_worker, 2, mode_idx)
    wl, st, H, W, old, rows = _dp_batch(synth)
    ocfg = O.Cfg(seed=wl.seed, **MODES[mode_idx])
    ref_g = O.group_stats(ocfg, st.go, st.reward, st.cs, key=st.key, alpha_in=st.alpha, beta_in=st.beta)
    ref_f = O.grpo_loss_fwd(ocfg, H, W, st.y, old, st.cs, ref_g["adv"], ref_g["w"], ref_g["keep"])
    rdH, rdW = O.grpo_loss_bwd(H, W, st.y, st.cs, ref_g["keep"], ref_f["lse"], ref_f["g"])
    assert ref_g["counters"][0] > 0 and (ref_f["ind"][ref_f["g"] == 0] == 0).any()
    (_, (a0, a1), cg0, Pg0, w0, dH0, dW0, loss0), (_, (b0, b1), cg1, Pg1, w1, dH1, dW1, loss1) = got
    assert a0 == 0 and a1 == b0 and b1 == wl.P and a1 > 0 and b1 > b0          # a real two-way split
    assert cg0 == cg1 == ref_g["counters"].tolist() and Pg0 == Pg1 == wl.P
    np.testing.assert_allclose(np.concatenate([w0, w1]), ref_g["w"], rtol=1e-12)
    np.testing.assert_allclose(np.concatenate([dH0, dH1]), rdH, rtol=1e-9, atol=1e-18)
    np.testing.assert_allclose(dW0, rdW, rtol=1e-9, atol=1e-15)
    assert np.array_equal(dW0, dW1)
    assert abs(loss0 - ref_f["loss"]) <= 1e-12 * abs(ref_f["loss"]) and loss0 == loss1
