"""The N > 1 path of bench.py on CPU: the layer does not shard, so N ranks are N independent
replicas; what the ranks share is only the timing protocol (barrier, max over ranks, aggregate =
N x per-replica work / slowest time).  Exercised here with two gloo ranks."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_take_the_slowest_time_and_sum_the_work():
    port = _free_port()
    prog = textwrap.dedent(f"""
        import os, sys, json
        sys.path.insert(0, {ROOT!r})
        import torch, torch.distributed as dist
        import bench
        from paper_2609_19242_b200 import synth
        rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
        dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=rank, world_size=world)
        # per-rank seeds give different replicas; rank 1 is the slow one
        w = synth.small(synth.WORKLOADS["tiny"], seed=rank)
        a = synth.make_inputs(w, "cpu", with_grad=False)["q_clean"]
        my_ms = 10.0 + 5.0 * rank
        dist.barrier()
        slowest = bench.max_over_ranks(my_ms, "cpu", world)
        f_fwd, f_bwd = w.flops()
        agg = bench.aggregate_tflops(f_fwd + f_bwd, slowest, world)
        sums = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(sums, a.double().sum().reshape(1))
        if rank == 0:
            print(json.dumps({{"slowest": slowest, "agg": agg, "single": bench.aggregate_tflops(f_fwd + f_bwd, 15.0, 1),
                              "distinct_inputs": bool(sums[0].item() != sums[1].item())}}))
        dist.destroy_process_group()
    """)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", prog], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    import json
    res = json.loads(outs[0][0].strip().splitlines()[-1])
    assert res["slowest"] == 15.0                       # max over ranks, not rank 0's own 10 ms
    assert abs(res["agg"] - 2 * res["single"]) < 1e-12   # two replicas' work over the slowest time
    assert res["distinct_inputs"]


def test_reference_arm_prints_nothing_on_non_zero_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_two_gloo_ranks_run_their_csbp_launches_and_reduce_the_clean_gradients():
    """Algorithms 1 and 2 with P = 2 on CPU: each rank builds the same partition, evaluates only its own
    packed blocks and clean position ranges (here with the oracle standing in for the kernels), and the
    all-reduce of the clean K/V gradient contributions -- the reduce-scatter before it is cut into shards --
    equals the unsharded gradient; the owned blocks and positions of the two ranks tile the sequence."""
    port = _free_port()
    prog = textwrap.dedent(f"""
        import os, sys, json
        sys.path.insert(0, {ROOT!r})
        import numpy as np, torch, torch.distributed as dist
        from oracle import bdlm_oracle as orc
        from paper_2609_19242_b200 import schedule
        rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
        dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=rank, world_size=world)
        L, M, H, Hkv, d = 48, 4, 2, 1, 4
        rng = np.random.default_rng(3)                      # every rank holds the same replicated inputs here
        t = {{n: rng.standard_normal((1, L, H if n[0] in "qd" else Hkv, d)) for n in
             ("q_clean", "k_clean", "v_clean", "q_noisy", "k_noisy", "v_noisy", "do_clean", "do_noisy")}}
        plan = schedule.csbp_plan(L, M, world)[rank]
        rows = np.concatenate([np.arange(b * M, (b + 1) * M) for b in plan.blocks])
        res = orc.attn_packed(None, t["k_clean"], t["v_clean"], t["q_noisy"][:, rows], t["k_noisy"][:, rows],
                              t["v_noisy"][:, rows], M, do_noisy=t["do_noisy"][:, rows], block_prefix=plan.block_prefix)
        dk, dv = res["dk_clean"], res["dv_clean"]
        for (p0, p1) in plan.clean_ranges:
            r2 = orc.attn_packed(t["q_clean"][:, p0:p1], t["k_clean"], t["v_clean"], None, t["k_noisy"][:, :M],
                                 t["v_noisy"][:, :M], M, do_clean=t["do_clean"][:, p0:p1], clean_q_pos0=p0)
            dk, dv = dk + r2["dk_clean"], dv + r2["dv_clean"]
        dk_t, dv_t = torch.from_numpy(dk.copy()), torch.from_numpy(dv.copy())
        dist.all_reduce(dk_t); dist.all_reduce(dv_t)
        owned = [None] * world
        dist.all_gather_object(owned, (plan.blocks, plan.clean_ranges))
        if rank == 0:
            full = orc.attn_backward(t["q_clean"], t["k_clean"], t["v_clean"], t["q_noisy"], t["k_noisy"], t["v_noisy"],
                                     t["do_clean"], t["do_noisy"], M)
            blocks = sorted(b for o in owned for b in o[0])
            pos = sorted(p for o in owned for (a, b) in o[1] for p in range(a, b))
            print(json.dumps({{"dk": float(np.abs(dk_t.numpy() - full[1]).max()), "dv": float(np.abs(dv_t.numpy() - full[2]).max()),
                              "blocks_ok": blocks == list(range(L // M)), "pos_ok": pos == list(range(L))}}))
        dist.destroy_process_group()
    """)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", prog], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=180) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    import json
    res = json.loads(outs[0][0].strip().splitlines()[-1])
    assert res["dk"] < 1e-11 and res["dv"] < 1e-11
    assert res["blocks_ok"] and res["pos_ok"]
