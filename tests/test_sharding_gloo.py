"""The multi-rank path on CPU: two gloo ranks share one decision by sharding its samples.

No GPU here, so each rank's context is a stand-in with the library's three calls
(predict / get_partial_sums / decide_from_sums) computed by the oracle on the rank's own sample
range.  What is under test is the product's sharding logic: the ranges, the single all-reduce of
per-position sums, and that every rank finishes the decision a single context would make.
"""
import os
import sys

import numpy as np
import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


class OracleBackedContext:
    def __init__(self, oracle_mod, weights, lag, n_samples, sample_offset, total_samples, seed):
        self.O = oracle_mod
        self.orc = oracle_mod.CutoffOracle(weights, lag, total_samples, seed=seed)
        self.lo, self.hi, self.total = sample_offset, sample_offset + n_samples, total_samples
        self.sums = None

    def push(self, x):
        self.orc.push(x)

    def predict(self):
        if len(self.orc.history) < self.orc.window:
            return self.O.WARMUP, self.orc.N
        x = self.orc.samples(np.arange(self.lo, self.hi))
        self.sums = np.sort(x, axis=1).sum(axis=0)
        self.orc.step += 1
        return self.decide_from_sums(self.sums)

    def get_partial_sums(self):
        return self.sums

    def decide_from_sums(self, sums):
        omega = self.O.throughput(self.orc.scale() * np.asarray(sums) / self.total)
        c, degenerate = self.O.argmax_cutoff(omega)
        return (self.O.DEGENERATE if degenerate else self.O.OK), c


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from oracle import cutoff_oracle as O
    from paper_1803_04209_b200 import inputs, sharding

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = inputs.WORKLOADS["n128"]
    w = inputs.workload_weights(wl)
    trace = inputs.workload_trace(wl, 6)
    cfg = sharding.shard_config(rank, world, 96)
    ctx = OracleBackedContext(O, w, wl.lag, cfg["n_samples"], cfg["sample_offset"], cfg["total_samples"], seed=11)
    shared = sharding.ShardedDecision(ctx)
    results = []
    for x in trace:
        results.append(shared.predict())
        ctx.push(x)
    results.append(shared.predict())
    out.put((rank, cfg, results))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_make_the_single_context_decision():
    sys.path.insert(0, ROOT)
    from oracle import cutoff_oracle as O
    from paper_1803_04209_b200 import inputs, sharding

    world, port = 2, 29500 + os.getpid() % 2000
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # the ranges tile the decision
    assert [g[1]["sample_offset"] for g in got] == [0, 96]
    assert all(g[1]["total_samples"] == 192 for g in got)
    # every rank reaches the same decisions ...
    assert got[0][2] == got[1][2]
    # ... and they are the ones a single 192-sample decision makes
    wl = inputs.WORKLOADS["n128"]
    w = inputs.workload_weights(wl)
    trace = inputs.workload_trace(wl, 6)
    single = O.CutoffOracle(w, wl.lag, 192, seed=11)
    want = []
    for x in trace:
        want.append(single.predict()[:2])
        single.push(x)
    want.append(single.predict()[:2])
    assert [tuple(r) for r in got[0][2]] == [tuple(r) for r in want]
    assert any(code == O.OK for code, _ in want) and want[0][0] == O.WARMUP
    with pytest.raises(ValueError):
        sharding.shard_config(2, 2, 8)
