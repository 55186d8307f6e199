"""CPU-only checks of the boundary: the library loads, exports what the header
declares, and its host-side logic (layout, sizes, draw, argument checks) is right.
No kernel is launched here."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import prsgd_oracle as orc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_1807_06629_b200 import _build
    _build.build_library()
    from paper_1807_06629_b200 import binding as b
    return b


def test_library_exports_every_declared_symbol(binding):
    with open(os.path.join(ROOT, "include", "prsgd.h")) as f:
        src = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    declared = set(re.findall(r"\b(prsgd_[a-z0-9_]+)\s*\(", src))
    assert len(declared) >= 25
    for name in declared:
        assert hasattr(binding.lib, name), name
    assert declared == set(binding.EXPORTS)


def test_draw_block_matches_oracle_bit_for_bit(binding):
    rng = np.random.default_rng(0)
    for _ in range(20000):
        seed = int(rng.integers(0, 2**63)) * 2 + int(rng.integers(0, 2))
        i = int(rng.integers(0, 65536))
        t = int(rng.integers(1, 2**40))
        nb = int(rng.integers(1, 2**31))
        assert binding.prsgd_draw_block(seed, i, t, nb) == orc.draw_block(seed, i, t, nb)
    for t in range(1, 300):
        for i in range(8):
            assert binding.prsgd_draw_block(20180717, i, t, 64) == orc.draw_block(20180717, i, t, 64)


def test_layout_cfg1(binding):
    lay = binding.prsgd_layout((32, 64, 10), 16, 0, 1024)
    assert lay.m == 2762 == orc.param_count((32, 64, 10))
    assert list(lay.w_off[:2]) == [0, 2112] and list(lay.b_off[:2]) == [2048, 2752]
    assert lay.m_pad == 2784 and lay.m_pad % 32 == 0


@pytest.mark.parametrize("dims,m", [((784, 512, 512, 10), 669706), ((3072, 1024, 1024, 10), 4206602),
                                    ((1024, 2048, 2048, 1024, 100), 8496228)])
def test_layout_counts_and_alignment(binding, dims, m):
    lay = binding.prsgd_layout(dims, 32, 0, 1024)
    assert lay.m == m == orc.param_count(dims)
    L = len(dims) - 1
    prev_end = 0
    for l in range(L):
        assert lay.w_off[l] % 32 == 0 and lay.b_off[l] % 32 == 0
        assert lay.w_off[l] >= prev_end and lay.b_off[l] >= lay.w_off[l] + dims[l] * dims[l + 1]
        prev_end = lay.b_off[l] + dims[l + 1]
    assert prev_end <= lay.m_pad < prev_end + 32


def test_workspace_bytes(binding):
    pb, sb, wb = binding.prsgd_workspace_bytes(4, (32, 64, 10), 16, 0, 1024)
    assert pb == 4 * 2784 * 4 and sb == 0
    assert wb >= 2 * 4 * 16 * (64 + 10) * 4 + 2784 * 4
    pb, sb, wb = binding.prsgd_workspace_bytes(64, (1024, 2048, 2048, 1024, 100), 32, 1, 1024)
    lay = binding.prsgd_layout((1024, 2048, 2048, 1024, 100), 32, 1, 1024)
    assert pb == 64 * lay.m_pad * 4 and sb == 64 * lay.m_pad * 2


def test_bad_specs_are_refused_on_the_host(binding):
    lib = binding.lib
    lay = binding.Layout()

    def rc(dims, batch, precision, pool):
        spec = binding.make_spec(dims, batch, precision, pool, 1)
        return lib.prsgd_layout(C.byref(spec), C.byref(lay))

    assert rc((32, 64, 10), 16, 0, 1024) == 0
    assert rc((32, 64, 10), 0, 0, 1024) == -1          # batch
    assert rc((32, 64, 10), 16, 0, 1000) == -1         # pool not a multiple of batch
    assert rc((32, 0, 10), 16, 0, 1024) == -1          # zero width
    assert rc((32, 64, 10), 16, 7, 1024) == -1         # precision
    assert rc((32, 60, 10), 16, 1, 1024) == -2         # bf16 needs multiples of 64
    assert rc((64, 64, 10), 24, 1, 1008) == -2         # bf16 batch
    assert rc((64, 64, 10), 128, 1, 1024) == -2        # bf16 batch above 64: refused before any buffer is sized
    assert rc((64, 64, 10), 128, 0, 1024) == 0         # (fp32 takes it)
    assert b"multiples of 64" in lib.prsgd_last_error(None) or b"batch" in lib.prsgd_last_error(None)
    assert rc((8,) * 18, 16, 0, 1024) == -1            # more than PRSGD_MAX_LAYERS layers
    assert rc((8,) * 17, 16, 0, 1024) == 0             # exactly 16 layers
    assert rc((32, 64, 10), 257, 0, 257 * 4) == -1     # batch above 256
    assert lib.prsgd_layout(None, C.byref(lay)) == -1
    spec = binding.make_spec((32, 64, 10), 16, 0, 1024, 1)
    out = C.c_void_p()
    assert lib.prsgd_create(0, C.byref(spec), 0.1, 4, 256, None, 256, None, C.byref(out)) == -1   # N
    assert lib.prsgd_create(4, C.byref(spec), 0.0, 4, 256, None, 256, None, C.byref(out)) == -1   # gamma
    assert lib.prsgd_create(4, C.byref(spec), 0.1, -1, 256, None, 256, None, C.byref(out)) == -1  # I
    assert lib.prsgd_create(4, C.byref(spec), 0.1, 4, None, None, 256, None, C.byref(out)) == -1  # NULL store
    assert lib.prsgd_create(4, C.byref(spec), 0.1, 4, 264, None, 256, None, C.byref(out)) == -2   # alignment
    assert lib.prsgd_average_rows(None, 4, 16, 16, None) == -1
    assert lib.prsgd_average_rows(256, 0, 16, 16, None) == -1
    assert lib.prsgd_average_rows(256, 4, 16, 8, None) == -1
    assert lib.prsgd_average_rows(260, 4, 16, 16, None) == -2
    assert lib.prsgd_average_rows(256, 4, 16, 18, None) == -2
    assert lib.prsgd_local_steps(None, 1) == -1


def test_alg2_schedule_matches_oracle(binding):
    for N in (1, 2, 8):
        want = orc.alg2_schedule(N, 130)
        for s in (1, 2, 7, 8, 9, 26, 27, 28, 64, 125, 130):
            K, g = binding.prsgd_alg2_schedule(N, s)
            assert K == want[s - 1][0] and g == pytest.approx(want[s - 1][1], rel=1e-6)


def test_reference_arm_of_the_benchmark_prints_its_json_line():
    """`bench.py --impl reference` times the oracle on the host and needs no GPU."""
    import json
    import subprocess
    import sys
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "cfg1",
                          "--steps", "2", "--warmup", "3"], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == "worker-steps/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["config"]["workload"] == "cfg1"
