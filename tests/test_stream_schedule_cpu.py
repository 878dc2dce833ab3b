"""The continuous-batching schedule (``csrc/stream_schedule.h``, the host logic behind ``aed_dec_decode_stream``) run
on the CPU against a simulated device that enforces the rules: arrival order, no slot reused before its utterance has
finished and been collected, nothing collected early or twice, lengths read back only when they are not known in
advance, and no step issued once the host's own bounds say that nothing decodes."""
import os
import subprocess

import pytest

HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.fixture(scope="module")
def exe(tmp_path_factory):
    out = tmp_path_factory.mktemp("sched") / "stream_schedule_check"
    subprocess.run(["g++", "-O1", "-std=c++17", os.path.join(HERE, "stream_schedule_check.cpp"), "-o", str(out)], check=True)
    return str(out)


def _run(exe, n, slots, early, poll, seed):
    r = subprocess.run([exe, str(n), str(slots), str(int(early)), str(poll), str(seed)], capture_output=True, text=True, timeout=60)
    assert r.returncode == 0, r.stderr
    tag, steps, row_steps, sum_true, max_forced, sum_forced = r.stdout.split()
    assert tag == "ok"
    return int(steps), int(row_steps), int(sum_true), int(max_forced), int(sum_forced)


@pytest.mark.parametrize("n,slots", [(1, 1), (7, 1), (40, 4), (40, 16), (40, 17), (200, 33), (12, 64)])
@pytest.mark.parametrize("seed", [1, 2, 3])
def test_known_lengths(exe, n, slots, seed):
    steps, row_steps, sum_true, max_forced, sum_forced = _run(exe, n, slots, False, 8, seed)
    assert row_steps == sum_true == sum_forced          # every (slot, step) pair the host counted held a decoding utterance
    assert steps >= -(-sum_forced // slots) and steps >= max_forced
    # a free slot is refilled at once: the classic bound of list scheduling (total work / machines + longest job)
    assert steps <= -(-sum_forced // slots) + max_forced
    if slots == 1:
        assert steps == sum_forced                      # one after the other
    if slots >= n:
        assert steps == max_forced                      # everything at once


@pytest.mark.parametrize("n,slots,poll", [(7, 1, 1), (40, 4, 3), (40, 16, 8), (200, 33, 5), (12, 64, 100)])
@pytest.mark.parametrize("seed", [1, 2])
def test_early_stop(exe, n, slots, poll, seed):
    steps, row_steps, sum_true, max_forced, sum_forced = _run(exe, n, slots, True, poll, seed)
    assert sum_true <= row_steps <= sum_forced          # the host's bound: between what was decoded and what was allowed
    assert steps >= -(-sum_true // slots)
    if slots >= n:
        assert steps <= max_forced
