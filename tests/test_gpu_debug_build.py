"""The bounds-checking build of the library (-DBLOAD_DEBUG): the fuzz cases, the frame-size matrix, the staged-path
cases, the per-sample frame sizes and the consumer calls run once more against it, in a child process (the library is
chosen when it is loaded), and its record of refused accesses must stay empty -- conftest.py asserts that at the end of
the child's session.  The child also compares every result with the oracle, as the ordinary run does."""
import os
import subprocess
import sys

import pytest

from paper_2310_10879_b200 import build

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_small_cases_under_the_bounds_checking_build():
    lib = build.build(debug=True)
    env = dict(os.environ, BLOAD_LIBRARY=lib)
    files = ["tests/test_gpu_fuzz.py", "tests/test_gpu_parity.py", "tests/test_gpu_var_frames.py", "tests/test_gpu_consumer.py",
             "tests/test_gpu_chunks.py"]
    select = ("fuzz or frame_sizes or staged or degenerate or toy8 or one_launch or whole_plan_unpack or block_ranges or "
              "metadata_only or blocks_of_any_size or blocks_of_any_length or few_words or not_multiples_of_4 or by_the_word_wise_walk or random_frame_sizes or multiples_of_16 or images or carry_prev or reset_state or repeat_last or "
              "chunk_plans")
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-k", select, "-p", "no:cacheprovider"] + files,
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    tail = (r.stdout or "")[-3000:] + (r.stderr or "")[-1500:]
    assert r.returncode == 0, tail
    assert " passed" in r.stdout and "error" not in r.stdout.lower().split("passed")[-1], tail


def test_the_ordinary_build_has_no_checks():
    import paper_2310_10879_b200 as B
    if os.path.basename(os.environ.get("BLOAD_LIBRARY", "")) == "libbload_debug.so":
        pytest.skip("this process runs the bounds-checking build")
    assert B.bload_debug_status() is None
