"""Host-side logic of bench.py: the reference arm's JSON contract (it runs the CPU oracle,
so it needs no GPU) and the multi-rank plumbing, exercised with two gloo ranks on CPU."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def test_reference_arm_prints_one_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--workload", "tiny_f32", "--steps", "2", "--warmup", "1"],
                         capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "Mtokens/s" and d["higher_is_better"] is True
    assert d["value"] > 0 and d["steps"] == 2 and d["warmup"] == 1
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["cpu_baseline"]["value"] == d["value"] == d["e2e"]["value"]
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0
    assert d["config"]["workload"] == "tiny_f32" and "model" not in d["config"]


def test_reference_arm_other_ranks_print_nothing():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--workload", "tiny_f32", "--steps", "1", "--warmup", "0", "--gpus", "2"],
                         capture_output=True, text=True, timeout=600, cwd=ROOT, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


def _rank_main(rank, world, port, results):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2607_22696_b200 import inputs
    wl = inputs.WORKLOADS["tiny_f32"]
    mine = bench.rank_workload(wl, rank)
    q = inputs.make_rows(mine, "q")
    slowest = bench.max_over_ranks(10.0 + 5.0 * rank, world)          # rank 1 is the slow one
    dist.barrier()
    results[rank] = (mine.seed, mine.N, float(q.double().sum()), slowest,
                     bench.aggregate_mtokens_per_s(wl, world, slowest))
    dist.destroy_process_group()


def test_two_gloo_ranks_take_different_videos_and_report_the_slowest_time():
    world, port = 2, 29517
    with mp.Manager() as manager:
        results = manager.dict()
        mp.spawn(_rank_main, args=(world, port, results), nprocs=world, join=True)
        r0, r1 = results[0], results[1]
    assert r0[0] != r1[0] and r0[1] == r1[1]            # different seeds, same shape (weak scaling)
    assert r0[2] != r1[2]                               # different data
    assert r0[3] == r1[3] == 15.0                       # max over ranks, seen by both
    assert abs(r0[4] - 2 * 256 / 15e-3 / 1e6) < 1e-12   # whole-job tokens / slowest time


def _head_shard_main(rank, world, port, results):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2607_22696_b200 import inputs, sharding
    T, H, W, heads, d, window = 3, 4, 5, 3, 32, (3, 3, 3)            # 3 heads over 2 ranks: 2 + 1
    shape = (T, H, W, heads, d)
    q, k, v = (inputs.normal(shape, 200, i, 1.0, torch.float32) for i in range(3))
    off = inputs.normal((T, H, W, heads, 27, 3), 200, 3, 1.0, torch.float32)
    lo, hi = sharding.head_range(heads, world, rank)
    mine = [sharding.shard_heads(z, world, rank) for z in (q, k, v, off)]
    h = hi - lo
    out, lse = oracle.forward(mine[0].view(-1, h, d), mine[1], mine[2], mine[3].view(-1, h, 27, 3), T, H, W, h, d, window)
    out = out.view(T, H, W, h, d).contiguous()
    # gather every rank's slice (ranks hold different head counts: pad to the largest)
    hmax = sharding.head_range(heads, world, 0)[1]
    padded = torch.zeros(T, H, W, hmax, d, dtype=out.dtype)
    padded[:, :, :, :h] = out
    bufs = [torch.zeros_like(padded) for _ in range(world)]
    dist.all_gather(bufs, padded)
    parts = []
    for r in range(world):
        rlo, rhi = sharding.head_range(heads, world, r)
        parts.append(bufs[r][:, :, :, :rhi - rlo])
    full = sharding.unshard_heads(parts)
    ref, _ = oracle.forward(q.view(-1, heads, d), k, v, off.view(-1, heads, 27, 3), T, H, W, heads, d, window)
    results[rank] = ((lo, hi), float((full - ref.view(shape)).abs().max()))
    dist.destroy_process_group()


def test_head_sharding_over_two_gloo_ranks_reproduces_the_unsharded_result():
    """Heads are independent, so the operator shards over heads with no exchange: each rank
    runs its slice (here through the CPU oracle) and the concatenation along the head axis
    equals the unsharded result exactly."""
    from paper_2607_22696_b200 import sharding
    assert [sharding.head_range(16, 8, r) for r in (0, 7)] == [(0, 2), (14, 16)]
    assert [sharding.head_range(5, 3, r) for r in range(3)] == [(0, 2), (2, 4), (4, 5)]
    world, port = 2, 29531
    with mp.Manager() as manager:
        results = manager.dict()
        mp.spawn(_head_shard_main, args=(world, port, results), nprocs=world, join=True)
        r0, r1 = results[0], results[1]
    assert r0[0] == (0, 2) and r1[0] == (2, 3)
    assert r0[1] == 0.0 and r1[1] == 0.0


def test_cpu_baseline_sample_is_an_exact_crop_of_the_workload():
    """bench.py times the oracle on a crop of the workload (some rows of some frames as queries,
    the frames their samples can reach as keys).  The crop must compute what the full problem
    computes for those queries: same outputs, same query-side gradients."""
    import importlib.util
    import dataclasses
    import oracle
    from paper_2607_22696_b200 import inputs
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    wl = dataclasses.replace(inputs.WORKLOADS["tiny_f32"], T=12, H=5, W=6, sigma=0.8, seed=77)
    sample = bench.oracle_sample(wl, 3, "cpu", frames=2)
    Tc, H, W, heads, d = sample["dims"]
    assert sample["tokens"] == 2 * 3 * W and Tc < wl.T
    out_c, lse_c = oracle.forward(sample["q"], sample["k"], sample["v"], sample["offsets"], Tc, H, W, heads, d, wl.window,
                                  qtok=sample["qtok"])
    dq_c, _, _, doff_c = oracle.backward(sample["q"], sample["k"], sample["v"], sample["offsets"], sample["dout"],
                                         Tc, H, W, heads, d, wl.window, qtok=sample["qtok"])
    # the whole problem
    q = inputs.make_rows(wl, "q", "cpu")
    k = inputs.make_rows(wl, "k", "cpu")
    v = inputs.make_rows(wl, "v", "cpu")
    dout = inputs.make_rows(wl, "dout", "cpu")
    off = inputs.make_offsets(wl, "cpu")
    P = wl.window[0] * wl.window[1] * wl.window[2]
    out_f, lse_f = oracle.forward(q.view(-1, heads, d), k, v, off.view(-1, heads, P, 3), wl.T, H, W, heads, d, wl.window)
    dq_f, _, _, doff_f = oracle.backward(q.view(-1, heads, d), k, v, off.view(-1, heads, P, 3), dout.view(-1, heads, d),
                                         wl.T, H, W, heads, d, wl.window)
    tq = wl.T // 2
    tok = torch.cat([(tq + f) * H * W + torch.arange(3 * W) for f in range(2)])
    # positions are formed in fp32 from the frame index, so a frame index shifted by the crop moves
    # the fractional parts by an ulp of the position: equal up to that, not bitwise
    for name, got, ref in (("out", out_c, out_f.view(-1, heads, d)[tok]), ("lse", lse_c, lse_f.view(-1, heads)[tok]),
                           ("dq", dq_c, dq_f.view(-1, heads, d)[tok]), ("doffsets", doff_c, doff_f.view(-1, heads, P, 3)[tok])):
        assert float((got - ref).abs().max()) <= 1e-5 * max(float(ref.abs().max()), 1.0), name
