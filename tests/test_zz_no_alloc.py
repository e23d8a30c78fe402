"""The allocation-free halo exchange entry point against the regular one.

Some users of this library are only handed buffers and a stream and may not call cudaMalloc (all
device memory was given out at start-up, or an allocation's implicit synchronisation is not
acceptable where they run).  For them distdl_halo_fwd_noalloc keeps its plan tables in a fixed
1 MiB device array of the library.  This test calls it through the C ABI twice in a row, with two
different partitions so that the second call finds the first call's tables in the array, and checks
each result, bit for bit, against distdl_halo_fwd on the same inputs and against the oracle.  Further
cases: two calls enqueued on one stream before a single synchronisation, free device memory unchanged
across calls, a plan beyond the fixed array, and a stream that is being captured (refused: the call copies
its tables from temporary host memory).  It lives in a file that pytest collects last.
"""

import numpy as np
import pytest

import oracle
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
    ref = oracle.halo_fwd_sequence(oracle.Partition(gshape, pshape, lo, hi), host)
    for w in range(part.num_workers):
        assert a[w].cpu().numpy().tobytes() == b[w].cpu().numpy().tobytes(), "worker %d differs" % w
        assert b[w].cpu().numpy().tobytes() == ref[w].tobytes(), "worker %d differs from the oracle" % w
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


def test_two_calls_on_one_stream_without_a_synchronisation_between_them():
    jobs = []
    for case, seed in ((CASES[0], 4000), (CASES[1], 5000)):
        gshape, pshape, lo, hi = case
        opart = oracle.Partition(gshape, pshape, lo, hi)
        host = [inputs.uniform_pm1(opart.padded_shape(w), seed + w) for w in range(opart.num_workers)]
        jobs.append((case, opart, host, [torch.from_numpy(h).to(DEV) for h in host]))
    torch.cuda.synchronize()
    for (gshape, pshape, lo, hi), _, _, bufs in jobs:      # the second call overwrites the tables behind the first kernel
        distdl.halo_fwd_noalloc(gshape, pshape, lo, hi, bufs)
    torch.cuda.synchronize()
    for _, opart, host, bufs in jobs:
        for got, ref in zip(bufs, oracle.halo_fwd_sequence(opart, host)):
            assert got.cpu().numpy().tobytes() == ref.tobytes()


def test_halo_fwd_noalloc_leaves_free_device_memory_unchanged():
    gshape, pshape, lo, hi = CASES[0]
    opart = oracle.Partition(gshape, pshape, lo, hi)
    bufs = [torch.zeros(opart.padded_shape(w), device=DEV) for w in range(opart.num_workers)]
    distdl.halo_fwd_noalloc(gshape, pshape, lo, hi, bufs)          # first call on the device: looks the array up
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    for _ in range(5):
        distdl.halo_fwd_noalloc(gshape, pshape, lo, hi, bufs)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0


def test_halo_fwd_noalloc_refuses_a_stream_that_is_being_captured():
    gshape, pshape, lo, hi = CASES[1]
    opart = oracle.Partition(gshape, pshape, lo, hi)
    bufs = [torch.zeros(opart.padded_shape(w), device=DEV) for w in range(opart.num_workers)]
    distdl.halo_fwd_noalloc(gshape, pshape, lo, hi, bufs)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            with pytest.raises(distdl.DistdlError) as err:
                distdl.halo_fwd_noalloc(gshape, pshape, lo, hi, bufs)
            bufs[0].add_(1.0)                                  # something to record, so that the capture ends well
    assert err.value.status == 4 and "captured" in str(err.value)
    torch.cuda.synchronize()
