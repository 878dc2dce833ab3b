"""The give-up path of the device code's bounded wait, run on CPU threads.

Every wait in the kernels goes through ``csrc/bounded_wait.h``.  The same source is compiled here for the host:
two threads play two warps, one arrival is withheld, and the waits must end by themselves.  A second test maps
the sticky device-side error word to the status the host reports.  Nothing is withheld on a GPU."""
import os
import subprocess

from paper_2503_05931_b200 import binding, build_ext

HERE = os.path.dirname(os.path.abspath(__file__))


def test_wait_gives_up_and_raises_the_abort_word(tmp_path):
    exe = tmp_path / "wait_host_check"
    subprocess.run(["g++", "-O1", "-std=c++17", "-pthread", os.path.join(HERE, "wait_host_check.cpp"), "-o", str(exe)],
                   check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True, timeout=60).stdout.split("\n")
    rows = {l.split()[0]: [int(v) for v in l.split()[1:]] for l in out if l.strip()}
    assert rows["complete"][:3] == [1, 1, 0]                 # both waits satisfied, abort word untouched
    r0, r1, abort_word, ms1 = rows["withheld"]
    assert (r0, r1, abort_word) == (0, 0, 1)                 # both gave up, the abort word is raised
    assert ms1 < 2000                                        # the second waiter left through the abort word, not its 5 s limit


def test_error_word_maps_to_a_status():
    build_ext.build()
    lib = binding.load_library()
    assert lib.aed_dec_status_of_error_word(0) == binding.AED_OK
    assert lib.aed_dec_status_of_error_word(1) == binding.AED_ERR_CAPACITY
    for word in (2, 3, 77):                                  # 2 is what a kernel writes when a wait ran out
        assert lib.aed_dec_status_of_error_word(word) == binding.AED_ERR_TIMEOUT
