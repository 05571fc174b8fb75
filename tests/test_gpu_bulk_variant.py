"""The measurement variant of the large-frame copy path that goes through the bulk-copy engine (-DBLOAD_BULK_COPY=1:
cp.async.bulk loads completing on mbarriers, bulk stores) is built into a library of its own and must produce the same
bytes as the oracle: the frame-size matrix, the evaluation configurations at reduced size, degenerate plans and block
sub-ranges run against it in a child process, and none of its bounded mbarrier waits may have given up."""
import os
import subprocess
import sys

import pytest

from paper_2310_10879_b200 import build

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHECK = """
import sys
import pytest
rc = pytest.main(["-x", "-q", "-m", "gpu", "-p", "no:cacheprovider", "-k",
                  "frame_sizes or config_ or toy8 or degenerate or block_ranges", "tests/test_gpu_parity.py"])
import torch
import paper_2310_10879_b200 as B
plan = B.bload_plan(torch.full((40,), 50, dtype=torch.int32, device="cuda:0"), 64, 1)   # runs of 50 KB: the large-frame path
store = torch.zeros(plan.sum_t * 1024, dtype=torch.uint8, device="cuda:0")
dense = torch.empty(plan.n_blocks * 64 * 1024, dtype=torch.uint8, device="cuda:0")
B.bload_pack(plan, store, 1024, 0, plan.n_blocks, dense=dense)
B.bload_unpack(plan, dense, 1024, 0, plan.n_blocks, store)
assert B.bload_last_copy_kernel("pack") == "k7b_copy_bulk<pack>" and B.bload_last_copy_kernel("unpack") == "k7b_copy_bulk<unpack>"
timeouts = B.load().bload_bulk_copy_timeouts()
print("bulk copy timeouts:", timeouts)
sys.exit(int(rc) or (1 if timeouts else 0))
"""


def test_bulk_copy_variant_matches_the_oracle():
    lib = build.build(defines=("BLOAD_BULK_COPY=1",), out=os.path.join(ROOT, "paper_2310_10879_b200", "libbload_bulk.so"))
    r = subprocess.run([sys.executable, "-c", CHECK], cwd=ROOT, env=dict(os.environ, BLOAD_LIBRARY=lib),
                       capture_output=True, text=True, timeout=900)
    tail = (r.stdout or "")[-3000:] + (r.stderr or "")[-1500:]
    assert r.returncode == 0, tail
    assert "bulk copy timeouts: 0" in r.stdout, tail
