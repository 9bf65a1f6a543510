"""Host-side logic of bench.py without a GPU: the N > 1 aggregation over independent replicas
(world size 2, gloo), the reference arm's line, and the rank rule of the reference arm."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank 1 is the slower replica: the job's time is its time, the work is the sum
    value, ms = bench.aggregate_replicas(10.0 * (rank + 1), 128, world, "cpu")
    out[rank] = (value, ms)
    dist.barrier()
    dist.destroy_process_group()


def test_replica_aggregation_world_size_2_gloo():
    ctx = mp.get_context("spawn")
    out = ctx.Manager().dict()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    for r in range(2):
        value, ms = out[r]
        assert ms == 20.0
        assert abs(value - 2 * 128 / 0.020) < 1e-6


def test_single_rank_aggregation_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    value, ms = bench.aggregate_replicas(4.0, 128, 1, "cpu")
    assert ms == 4.0 and abs(value - 32000.0) < 1e-9


def _run_bench(extra_env, *args):
    env = dict(os.environ, **extra_env)
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], env=env,
                          capture_output=True, text=True, timeout=600)


def test_reference_arm_prints_one_json_line_with_the_contract_keys():
    res = _run_bench({"RANK": "0", "WORLD_SIZE": "1"}, "--impl", "reference", "--workload", "tiny",
                     "--steps", "3", "--warmup", "1")
    assert res.returncode == 0, res.stderr
    lines = [l for l in res.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "balanced_examples_per_sec"
    assert d["unit"] == "examples/s" and d["higher_is_better"] is True
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0,
                        "d2h_bytes_per_step": 0}
    assert d["config"]["workload"] == "tiny"


def test_reference_arm_other_ranks_exit_quietly():
    res = _run_bench({"RANK": "1", "WORLD_SIZE": "2"}, "--impl", "reference", "--workload", "tiny")
    assert res.returncode == 0 and res.stdout.strip() == ""


def test_algorithmic_bytes_model():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2302_00845_b200 import synth
    wl = synth.WORKLOADS["gpt2"]
    inp = 2 * 64 * 124_000_000 * 2
    assert bench.algorithmic_bytes("gram", wl) == inp + 4 * 124_000_000
    assert bench.algorithmic_bytes("update", wl) == inp + 8 * 124_000_000
    assert inp == 31_744_000_000


class _FakeShard:
    """Stands in for a shard handle: its partial sums are a known function of the rank."""

    def __init__(self, rank):
        self.rank, self.seen = rank, []

    def begin_epoch(self):
        pass

    def step_begin(self, grads, gram):
        gram.copy_(torch.arange(gram.numel(), dtype=torch.float64) * (self.rank + 1))

    def step_finish(self, grads, gram):
        self.seen.append(gram.clone())


def _shard_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from paper_2302_00845_b200 import binding
    dist.init_process_group("gloo", rank=rank, world_size=world)
    m = 3
    fake = _FakeShard(rank)

    class OnFake(binding.ShardedCdGrab):          # the wrapper's exchange, driven without a GPU
        def __init__(self):
            self.group = None
            self._attach(fake, m, "cpu")

    sh = OnFake()
    sh.begin_epoch()
    sh.step(None)
    sh.step(None)
    out[rank] = [t.tolist() for t in fake.seen]
    dist.barrier()
    dist.destroy_process_group()


def test_sharded_wrapper_all_reduces_the_partial_sums_world_size_2_gloo():
    ctx = mp.get_context("spawn")
    out = ctx.Manager().dict()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_shard_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    want = [3.0 * i for i in range(3 * 3 + 3)]          # rank 0 gives i, rank 1 gives 2 i
    assert out[0] == [want, want] and out[1] == out[0]  # both ranks finish on the same bits


def test_traffic_figures_match_the_kernel_sources():
    """Every DRAM-traffic figure bench.py reports is tied to the kernel files it was captured with;
    a figure whose files changed reads null in the bench line, and this test says which one to
    capture again (or to re-key, when the edit left the kernel itself alone)."""
    sys.path.insert(0, ROOT)
    import bench
    stale = [k for k, v in bench.NCU_TRAFFIC.items() if v["source"] != bench.source_hash(v["files"])]
    assert not stale, f"ncu traffic figures out of date for {stale}"
