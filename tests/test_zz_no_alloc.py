"""The allocation-free halo exchange entry point against the regular one.

Some users of this library are only handed buffers and a stream and may not call cudaMalloc (all
device memory was given out at start-up, or an allocation's implicit synchronisation is not
acceptable where they run).  For them distdl_halo_fwd_noalloc keeps its plan tables in a fixed
1 MiB device array of the library.  This test calls it through the C ABI twice in a row, with two
different partitions so that the second call finds the first call's tables in the array, and checks
each result, bit for bit, against distdl_halo_fwd on the same inputs.  It lives in a file that
pytest collects last.
"""

import numpy as np
import pytest

import paper_2006_03108_b200 as distdl
from paper_2006_03108_b200 import inputs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

DEV = "cuda:0"

CASES = [
    ((70, 66, 72), (2, 2, 2), (4, 4, 4), (4, 4, 4)),
    ((37, 45), (3, 2), (2, 1), (1, 3)),
]


def _run_both(case, seed):
    gshape, pshape, lo, hi = case
    part = distdl.Partition(gshape, pshape, lo, hi)
    host = [inputs.uniform_pm1(part.padded_shape(w), seed + w) for w in range(part.num_workers)]
    a = [torch.from_numpy(h).to(DEV) for h in host]
    b = [torch.from_numpy(h).to(DEV) for h in host]
    distdl.halo_fwd(part, a)
    distdl.halo_fwd_noalloc(gshape, pshape, lo, hi, b)
    torch.cuda.synchronize()
    for w in range(part.num_workers):
        assert a[w].cpu().numpy().tobytes() == b[w].cpu().numpy().tobytes(), "worker %d differs" % w
        # and something did happen: the ghosts no longer hold the random input
        assert a[w].cpu().numpy().tobytes() != host[w].tobytes()


def test_halo_fwd_noalloc_matches_halo_fwd_twice_in_a_row():
    _run_both(CASES[0], 1000)
    _run_both(CASES[1], 2000)      # the array still holds the tables of the first call
    _run_both(CASES[0], 3000)


def test_halo_fwd_noalloc_rejects_plans_beyond_the_fixed_array():
    gshape, pshape = (64, 64, 64), (8, 8, 4)            # 256 workers x 26 boxes: more than 1 MiB of tables
    shards = [torch.zeros(1, device=DEV)] * 256
    with pytest.raises(distdl.DistdlError) as err:
        distdl.halo_fwd_noalloc(gshape, pshape, (1, 1, 1), (1, 1, 1), shards)
    assert err.value.status == 4 and "fixed device array" in str(err.value)
