"""The N > 1 path of the benchmark on CPU: independent replicas, one process per rank, combined by the
maximum of the ranks' times (gloo, world size 2)."""
import os
import sys

import pytest

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    slowest = bench.max_over_ranks(mine, torch.device("cpu"))
    dist.barrier()
    out[rank] = (slowest, bench.aggregate_value(1e9, 4, slowest, world))
    dist.destroy_process_group()


def test_replicas_are_combined_by_the_slowest_rank():
    world, port = 2, 29500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        assert out[0] == out[1]
        slowest, value = out[0]
    assert slowest == 15.0
    # two replicas, 4 steps of 1 GB each in 15 ms: 2 * 4 GB / 0.015 s
    assert abs(value - 2 * 4 * 1e9 / 0.015 / 1e9) < 1e-6


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, torch.device("cpu")) == 3.5
    assert bench.workload("per_tensor")[2] == 25557032 and len(bench.workload("per_tensor")[4]) == 161


def test_gpus_flag_starts_the_ranks_itself():
    """`bench.py --gpus 2` with no launcher around it starts two ranks (torch.distributed.run on 127.0.0.1) and
    reports n_gpus = 2; here through the launch-path self-test, which needs no GPU (gloo, no kernels).  Asked
    for more GPUs than the machine has, the real run exits non-zero and prints no result line."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    bench_py = os.path.join(ROOT, "bench.py")
    run = subprocess.run([sys.executable, bench_py, "--gpus", "2", "--selftest-cpu", "--steps", "3", "--warmup", "3"],
                         capture_output=True, text=True, env=env, timeout=300)
    assert run.returncode == 0, run.stderr[-2000:]
    lines = [l for l in run.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                   # rank 0 alone prints
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2 and out["ms_per_step"] == 2.0  # the slowest rank's (made-up) time
    if not torch.cuda.is_available():
        run = subprocess.run([sys.executable, bench_py, "--gpus", "2", "--steps", "3"], capture_output=True, text=True, env=env,
                             timeout=300)
        assert run.returncode != 0 and not [l for l in run.stdout.splitlines() if l.startswith("{")]
    # a launcher that started a different number of ranks than --gpus says is an error, not a line with n_gpus = 1
    env1 = dict(env, WORLD_SIZE="1", RANK="0", LOCAL_RANK="0")
    run = subprocess.run([sys.executable, bench_py, "--gpus", "2", "--selftest-cpu"], capture_output=True, text=True, env=env1, timeout=300)
    assert run.returncode != 0 and not run.stdout.strip()


# ---------------------------------------------------------------- sharded round (records all-gathered), 2 ranks
class _OracleEngine:
    """Stands in for the CUDA context on a machine without a GPU: same calls, the oracle's arithmetic."""

    def __init__(self, O, plan_job, x, xw, mem, anchors=None):
        self.O, self.plan, self.x, self.xw, self.mem, self.anchors = O, plan_job, x, xw, mem, anchors
        self.base, self.records = 0, None

    def set_sharding(self, base, R_total):
        assert R_total == self.plan.R
        self.base = base

    def compress_feedback(self, rnd, mask):
        self.records = {}
        for r in range(self.xw.shape[0]):
            if mask is None or mask[r]:
                ref = self.x if self.anchors is None else self.anchors[r]
                out = self.O.compress_worker(self.plan, rnd, self.base + r, ref, self.xw[r], self.mem[r], mode=self.O.SORT)
                assert out["rc"] == 0
                self.records[r] = out["wire"]

    def pack(self, wire_local, bits_out=None):
        for r, w in self.records.items():
            wire_local[r] = torch.from_numpy(w.view("int32"))

    def recode_gaps(self, wire_local, packed_local, mask, bits_out=None):
        local = self.O.Plan(self.xw.shape[0], self.plan.d, s=self.plan.s, sparsifier=self.plan.sparsifier,
                            quantizer=self.plan.quantizer, seed=self.plan.seed, offsets=self.plan.offsets, kseg=self.plan.kseg)
        out = self.O.recode_gaps(local, wire_local.numpy().view("uint32"), mask)
        assert out["rc"] == 0
        for r in range(self.xw.shape[0]):
            if mask is None or mask[r]:
                packed_local[r] = torch.from_numpy(out["packed"][r].view("int32"))
                if bits_out is not None:
                    bits_out[r] = int(out["bits"][r])

    def decode_gaps(self, packed, records, mask):
        out = self.O.decode_gaps(self.plan, packed.numpy().view("uint32"), mask)
        assert out["rc"] == 0
        records.copy_(torch.from_numpy(out["wire"].view("int32")))

    def unpack_accumulate(self, records, mask):
        assert self.O.unpack_accumulate(self.plan, self.x, records.numpy().view("uint32"), mask) == 0

    def broadcast(self, mask):
        import numpy as np
        for r in range(self.xw.shape[0]):
            if mask is None or mask[r]:
                self.xw[r] = self.x
                if self.anchors is not None:
                    self.anchors[r] = self.x


def _sharded_main(rank, world, port, out, gap_coded):
    sys.path.insert(0, ROOT)
    import numpy as np
    from oracle import oracle as O
    from paper_1906_02367_b200 import inputs as I, sharded
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    R, d, k = 4, 3000, 40
    plan = O.Plan(R, d, k=k, s=16, sparsifier=O.TOPK, quantizer=O.QSGD, seed=3)
    x, xw, mem = I.gaussian_round(R, d, seed=50)
    anchors = xw.copy()
    base, count = sharded.partition(R, world)[rank]
    eng = _OracleEngine(O, plan, x.copy(), xw[base:base + count].copy(), mem[base:base + count].copy(),
                        anchors[base:base + count].copy())
    wire_local = torch.zeros((count, plan.wire_words()), dtype=torch.int32)
    gap = dict(packed_local=torch.zeros((count, O.gap_words(plan)), dtype=torch.int32),
               records=torch.zeros((R, plan.wire_words()), dtype=torch.int32)) if gap_coded else {}
    job = sharded.ShardedRound(R, eng, wire_local, **gap)
    masks = [None, np.array([1, 0, 0, 1], np.uint8), np.array([0, 0, 1, 1], np.uint8)]   # the last leaves rank 0 idle
    for rnd, mask in enumerate(masks):
        eng.xw += I.gaussian_drift(R, d, 8, rnd, std=1e-2)[base:base + count]
        job.round(rnd, mask)
        if gap_coded:                     # what crossed the collective: the round's longest record, not the rows' capacity
            assert 0 < job.exchanged_words <= O.gap_words(plan)
    out[rank] = (eng.x.tobytes(), eng.xw.tobytes(), eng.mem.tobytes(), eng.anchors.tobytes())
    dist.destroy_process_group()


@pytest.mark.parametrize("gap_coded", [False, True])
def test_sharded_round_equals_the_single_process_round(gap_coded):
    import numpy as np
    sys.path.insert(0, ROOT)
    from oracle import oracle as O
    from paper_1906_02367_b200 import inputs as I
    world, port = 2, 31500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_sharded_main, args=(world, port, out, gap_coded), nprocs=world, join=True)
        got = {r: out[r] for r in range(world)}
    R, d, k = 4, 3000, 40
    plan = O.Plan(R, d, k=k, s=16, sparsifier=O.TOPK, quantizer=O.QSGD, seed=3)
    x, xw, mem = I.gaussian_round(R, d, seed=50)
    anchors = xw.copy()
    masks = [None, np.array([1, 0, 0, 1], np.uint8), np.array([0, 0, 1, 1], np.uint8)]
    for rnd, mask in enumerate(masks):
        xw += I.gaussian_drift(R, d, 8, rnd, std=1e-2)
        assert O.sync_round(plan, rnd, x, xw, mem, anchors=anchors, mask=mask)["rc"] == 0
    per = R // world
    for r in range(world):
        gx, gxw, gmem, ganch = got[r]
        assert gx == x.tobytes(), f"replica of x on rank {r}"
        assert gxw == xw[r * per:(r + 1) * per].tobytes()
        assert gmem == mem[r * per:(r + 1) * per].tobytes()
        assert ganch == anchors[r * per:(r + 1) * per].tobytes()


def test_partition_and_masks():
    sys.path.insert(0, ROOT)
    import numpy as np
    import pytest
    from paper_1906_02367_b200 import sharded
    assert sharded.partition(8, 4) == [(0, 2), (2, 2), (4, 2), (6, 2)]
    assert sharded.partition(8, 1) == [(0, 8)]
    with pytest.raises(ValueError):
        sharded.partition(8, 3)
    assert sharded.local_mask(None, 2, 2) is None
    assert sharded.local_mask([1, 0, 0, 1, 1, 1], 2, 2).tolist() == [0, 1]
    w = torch.arange(6, dtype=torch.int32).reshape(2, 3)
    assert sharded.gather_records(w, 2) is w                   # no process group: one rank holds everything
