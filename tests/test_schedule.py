"""The tensor-core kernel's work schedule, replayed on the host for every cache length of the benchmark
configurations and of the test shapes (tests/schedule_replay.cpp compiled against csrc/mkv_schedule.h)."""
import os
import subprocess

import pytest

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(os.path.dirname(HERE), "paper_2503_00979_b200", "csrc")


@pytest.fixture(scope="module")
def replay(tmp_path_factory):
    exe = str(tmp_path_factory.mktemp("sched") / "schedule_replay")
    subprocess.run(["g++", "-O2", "-std=c++17", "-I", CSRC, os.path.join(HERE, "schedule_replay.cpp"), "-o", exe], check=True)

    def run(U, cap, hint=0, n_sm=148):
        r = subprocess.run([exe, str(U), str(cap), str(hint), str(n_sm)], capture_output=True, text=True)
        assert r.returncode == 0 and r.stdout.startswith("ok"), f"U={U} cap={cap} hint={hint} n_sm={n_sm}: {r.stdout}{r.stderr}"
        _, grid, splits, checked = r.stdout.split()
        return int(grid), int(splits), int(checked)

    return run


# (units, capacity): the benchmark configurations, whole stack and one layer (per-layer calls ask for about eight CTAs
# per unit), the capacity sweep, coarse-grained eviction (capacity C + R + T), the chunked window (units x 4 chunks)
@pytest.mark.parametrize("U,cap,hint", [
    (256, 2032, 0), (8, 2032, 8), (8192, 1056, 0), (256, 1056, 8), (2048, 4064, 0), (64, 4064, 8),
    (1024, 544, 0), (1024, 1056, 0), (1024, 2080, 0), (1024, 4128, 0), (1024, 8224, 0),
    (256, 2040, 0), (256 * 4, 4096, 0), (8 * 4, 4096, 8)])
def test_benchmark_configurations(replay, U, cap, hint):
    grid, splits, checked = replay(U, cap, hint)
    assert 1 <= grid <= 148 and splits >= 1 and checked > 0


@pytest.mark.parametrize("U", [1, 2, 3, 4, 7, 8, 16, 147, 148, 149, 300])
@pytest.mark.parametrize("cap", [1, 127, 128, 129, 166, 257, 1000, 2100])
def test_small_and_awkward_shapes(replay, U, cap):
    for hint in (0, 1, 2, 5, 8):
        replay(U, cap, hint)


def test_other_sm_counts(replay):
    # correctness must not depend on the number of SMs
    for n_sm in (1, 2, 7, 132, 160):
        replay(40, 900, 0, n_sm)
        replay(40, 900, 3, n_sm)
