"""The N > 1 path of the benchmark on CPU: two gloo ranks on 127.0.0.1.

The sampling pass has no exchange step (every group is independent), so N GPUs run N replicas and the only
multi-rank logic is the timing contract: a step takes as long as the slowest rank (maximum over ranks), the value is the
whole job's, rank 0 alone prints, and the reference arm runs on rank 0 only."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        per_rank_ms = [10.0 + 5.0 * rank, 3.0 - rank, 7.0]          # rank 1 is slower on the first, faster on the second
        total, fwd, bwd = bench.max_over_ranks(per_rank_ms, dist, torch.device("cpu"))
        value = bench.whole_job_throughput(1e9, world, total)
        from paper_2505_11170_b200 import synthetic as syn
        mine = syn.shard(syn.llama2_1b(n_blocks=1), rank, world)
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)
        if rank == 0:
            out.put({"total": total, "fwd": fwd, "bwd": bwd, "value": value, "shards": gathered})
    finally:
        dist.destroy_process_group()


def test_two_ranks_take_the_slowest_rank_and_report_the_whole_job():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    got = out.get()
    assert got["total"] == 15.0 and got["fwd"] == 3.0 and got["bwd"] == 7.0      # element-wise maximum over ranks
    assert got["value"] == 2 * 1e9 / 15e-3                                        # both replicas count, slowest rank's time
    a, b = got["shards"]
    assert sorted(a + b) == list(range(7)) and not set(a) & set(b)               # a split of the tensors needs no exchange


class _FakeShardSampler:
    """Stands in for ShardedSetSampler on CPU: no sampling, but the same two all-reduces over world + 1 slots per tensor."""

    def __init__(self, plans, log):
        from paper_2505_11170_b200.sharding import all_reduce_slots
        self.plans, self.log, self.reduce = plans, log, all_reduce_slots
        self.n_slots = plans[0].world + 1

    def _exchange(self, step, op):
        buf = torch.zeros(len(self.plans) * self.n_slots)
        for t, p in enumerate(self.plans):
            for piece in p.pieces:
                for s in piece.slots:
                    buf[t * self.n_slots + s] = float(p.rank + 1)
        self.reduce(buf, op)
        self.log.append((op, step, buf.clone()))

    def forward(self, step):
        self._exchange(step, "max")

    def backward(self, step):
        self._exchange(step, "sum")


def _sharded_worker(rank, world, port, out):
    import bench
    from paper_2505_11170_b200 import synthetic as syn
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        specs = syn.llama2_1b(n_blocks=1)
        log = []
        timer = lambda fn, reps: [fn(k) for k in range(reps)] and (4.0 + rank)          # rank 1 is the slow one
        leg = bench.sharded_step_leg(lambda plans: _FakeShardSampler(plans, log), specs, rank, world, dist, torch.device("cpu"), timer, reps=2)
        if rank == 0:
            out.put({"leg": leg, "ops": [(op, step) for op, step, _ in log], "max_slot": float(max(b.max() for op, _, b in log if op == "max")),
                     "sum_slot": float(max(b.max() for op, _, b in log if op == "sum")), "elements": syn.total_elements(specs)})
    finally:
        dist.destroy_process_group()


def test_sharded_step_leg_covers_the_whole_set_and_reduces_over_both_ranks():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    procs = [ctx.Process(target=_sharded_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    got = out.get()
    leg = got["leg"]
    assert leg["world"] == 2 and leg["elements"] == got["elements"]               # the two shards make up every tensor
    assert leg["fwd_ms"] == 5.0 and leg["bwd_ms"] == 5.0                           # the slowest rank's time
    assert leg["all_reduce_floats_per_pass"] == 7 * 3
    assert got["ops"] == [("max", 0), ("max", 1), ("sum", 0), ("sum", 1)]
    # the cut of every tensor falls inside a group of 128 (the shard boundary is a multiple of 32, not of 128) or on one;
    # where it is inside, both ranks write the cut's slot: MAX gives the larger rank number, SUM their sum
    assert got["max_slot"] in (0.0, 2.0) and got["sum_slot"] in (0.0, 3.0)
    assert leg["end_pieces_all_ranks"] >= 0


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""                           # other ranks exit 0 without work


def test_reference_arm_line_has_the_contract_keys():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                       capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["steps"] == 1 and line["unit"] == "GB/s" and line["higher_is_better"] is True
    assert line["config"]["workload"] == "llama2_1b_linear_set_g128" and line["vs_baseline"] is None
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] == 1 and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"] == {"value": line["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
