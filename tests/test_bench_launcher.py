"""bench.py's multi-GPU plumbing on CPU: `--gpus N` starts N ranks, the workers are partitioned over them,
the timed loop and the maximum over ranks work across processes, and exactly one JSON line comes out.  The
ranks run tests/standin_bench_rank.py (gloo, fp64 oracle as the local engine): no GPU, no product kernel."""
import json
import os
import sys

import numpy as np
import pytest

from oracle import prsgd_oracle as orc
from paper_1807_06629_b200 import sharded, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402

STANDIN = os.path.join(ROOT, "tests", "standin_bench_rank.py")


def test_partitions():
    assert [sharded.partition(64, 8, r, "strong") for r in (0, 3, 7)] == [(0, 8, 64), (24, 8, 64), (56, 8, 64)]
    assert [sharded.partition(5, 2, r, "strong") for r in (0, 1)] == [(0, 3, 5), (3, 2, 5)]
    assert [sharded.partition(64, 4, r, "weak") for r in (0, 3)] == [(0, 64, 256), (192, 64, 256)]
    with pytest.raises(ValueError):
        sharded.partition(4, 8, 0, "strong")
    with pytest.raises(ValueError):
        sharded.partition(4, 2, 0, "diagonal")


def test_a_plain_start_with_several_gpus_starts_the_ranks(monkeypatch):
    """`python bench.py --gpus 4` outside a launcher re-runs itself as 4 ranks with the same arguments."""
    seen = {}

    class Done:
        returncode = 0

    def fake(n, script_args, **kw):
        seen["n"], seen["args"] = n, list(script_args)
        return Done()
    monkeypatch.setattr(bench, "launch_ranks", fake)
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    with pytest.raises(SystemExit) as e:
        bench.main(["--gpus", "4", "--steps", "2", "--scaling", "strong"])
    assert e.value.code == 0 and seen == {"n": 4, "args": ["--gpus", "4", "--steps", "2", "--scaling", "strong"]}


def test_the_environment_a_caller_set_is_left_alone():
    with open(os.path.join(ROOT, "bench.py")) as f:
        src = f.read()
    assert "NCCL_DEBUG" not in src


@pytest.mark.parametrize("scaling", ["strong", "weak"])
def test_two_ranks_print_one_line_and_agree_with_one_process(scaling):
    steps, warmup = 2, 3
    r = bench.launch_ranks(2, ["--scaling", scaling, "--steps", str(steps), "--warmup", str(warmup)],
                           script=STANDIN, capture=True, timeout=280)
    assert r.returncode == 0, r.stderr[-3000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, r.stdout
    line = json.loads(lines[0])
    n_global = 5 if scaling == "strong" else 10
    assert line["n_gpus"] == 2 and line["scaling"] == scaling and line["steps"] == steps and line["value"] > 0
    assert line["config"]["N"] == n_global and line["local_workers"] == (3 if scaling == "strong" else 5)
    assert line["rows_identical"]                      # the run ends on an average
    # the same job in one process
    w = synth.Workload("standin", n_global, (6, 5, 4), 4, 0.05, 3, 8, 0, 16, mean_shift=0.5, gumbel=True, seed=9)
    X, Y = synth.make_pools(w)
    x0 = synth.init_params(w.dims, w.seed).astype(np.float64)
    T = (steps + warmup) * w.I
    want = orc.pr_sgd(np.tile(x0, (w.N, 1)), w.gamma, w.I, T, orc.mlp_grad_fn(w.dims, X.astype(np.float64), Y, w.B, w.seed))
    assert np.allclose(line["node_average"], want.mean(0), atol=1e-12)


def test_byte_model_follows_the_launch_rules():
    """`period_bytes` mirrors the library's launch rules: the launch counts it expects per period are the ones the
    library counts on the GPU (125 update launches per cfg4 period, ...), and the shared restart, the folding and
    the momentum options move the bytes the way the kernels do."""
    cfg4 = synth.WORKLOADS["cfg4"]
    assert bench.period_bytes(cfg4, 8496384)["head"][1] == 0       # 64 workers x 8 slices: more than one wave, not used
    h = bench.period_bytes(cfg4, 8496384, head_kernel=2)   # the class layer as one launch of its own family
    assert {k: v[1] for k, v in h.items() if v[1]} == {"forward": 65, "dx": 2, "update": 93, "update_average": 3,
                                                         "misc": 1, "head": 32}
    f = bench.period_bytes(cfg4, 8496384, head_kernel=0)
    assert {k: v[1] for k, v in f.items() if v[1]} == {"forward": 97, "dx": 2, "update": 125, "update_average": 3,
                                                         "misc": 1}            # (the class layer's segment average rides on the bias-average launch)
    assert sum(v[0] for v in f.values()) - sum(v[0] for v in h.values()) == (
        32 * 64 * (100 * 4 + 32 * 100 * 4 + 32 * (100 + 1024) * 2)      # no bias re-read, no fp32 logits, operands read once
        - 63 * 100 * 1024 * 2)                             # (its first iteration reads every worker's own copy of W_L)
    plain = 64 * 8496228                                   # parameters of all workers
    per_iter = f["update"][0] / 31.25                      # 125 launches = 31 plain iterations + the class layer's 32nd
    assert 9.0 * plain < per_iter < 10.2 * plain           # ~10 B/param, minus the bf16 copy of W_1 that is not written
    assert 9.0 * plain < h["update"][0] / 31 + h["head"][0] / 32 < 10.2 * plain
    g = bench.period_bytes(cfg4, 8496384, momentum=True)
    assert g["update"][0] > f["update"][0] + 7.5 * plain * 31 and g["update_average"][1] == 3
    c3 = synth.WORKLOADS["cfg3"].with_(I=1)
    shared, own = bench.period_bytes(c3, 4206656), bench.period_bytes(c3, 4206656, shared_restart=False)
    assert shared["forward"][0] * 5 < own["forward"][0] and shared["update_average"][0] < own["update_average"][0]
    assert own["update_average"][0] - shared["update_average"][0] == 15 * (3072 * 1024 + 1024 * 1024) * 4
    c16 = bench.period_bytes(synth.WORKLOADS["cfg3"].with_(I=16), 4206656, head_kernel=0)
    assert c16["forward"][1] == 33 and c16["dx"][1] == 16 and c16["update"][1] == 46
    c16 = bench.period_bytes(synth.WORKLOADS["cfg3"].with_(I=16), 4206656)
    assert c16["forward"][1] == 17 and c16["dx"][1] == 16 and c16["update"][1] == 30 and c16["head"][1] == 16
    c16f = bench.period_bytes(synth.WORKLOADS["cfg3"].with_(I=16), 4206656, head_forward=True)   # ... and layer 2's forward inside the head launch
    assert c16f["forward"][1] == 1 and c16f["head"][1] == 16
    assert (c16["forward"][0] + c16["head"][0]) - (c16f["forward"][0] + c16f["head"][0]) == 16 * 16 * 2 * 64 * 1024 * 2
    assert bench.period_bytes(synth.WORKLOADS["cfg3"].with_(I=16), 4206656, forward_chain=True)["forward"][1] == 16
    f32 = bench.period_bytes(synth.WORKLOADS["cfg2"], 669728)
    assert f32["forward"][1] == 24 and f32["softmax"][1] == 8 and f32["update_average"][1] == 3
