"""The review rule through csd_spec_accept_static, the entry point for callers that cannot
allocate device memory (a serving loop that forbids allocator calls once it is running, or code
that owns only the buffers it was given).  Its scratch is a fixed array inside the library, so
the call takes no workspace; here it must give exactly what csd_spec_accept gives, twice in a
row (the second call finds the first call's leftovers in the shared scratch), and must refuse
problems that do not fit.  Collected last on purpose: a failure here cannot hide another test."""
import pytest
import torch

import workloads
from gpu_util import require_gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    require_gpu()
    from paper_2312_11462_b200 import binding
    return binding


def outputs(rows):
    # the caller owns every buffer, the outputs included
    return (torch.full((rows,), -7, dtype=torch.int32, device="cuda"),
            torch.full((rows,), -7, dtype=torch.int32, device="cuda"))


@pytest.mark.parametrize("rows,k,V,temperature", [(64, 4, 32000, 1.0), (16, 16, 128256, 1.0), (33, 3, 5003, 0.7),
                                                  (64, 8, 32000, 0.0)])
def test_matches_the_workspace_entry_point_twice(b, rows, k, V, temperature):
    t, d, tok = workloads.accept_case(rows, k, V, 0.5, seed=rows + k, device="cuda")
    want = b.csd_spec_accept(t, d, tok, temperature, 1.0, seed=11, step=2)
    first = b.csd_spec_accept_static(t, d, tok, temperature, 1.0, seed=11, step=2, out=outputs(rows))
    # a different problem in between leaves other data in the shared scratch
    t2, d2, tok2 = workloads.accept_case(8, 2, 4096, 2.0, seed=5, device="cuda")
    mid = b.csd_spec_accept_static(t2, d2, tok2, 1.0, out=outputs(8))
    want_mid = b.csd_spec_accept(t2, d2, tok2, 1.0)
    second = b.csd_spec_accept_static(t, d, tok, temperature, 1.0, seed=11, step=2, out=outputs(rows))
    torch.cuda.synchronize()
    for got in (first, second):
        assert torch.equal(got[0], want[0]) and torch.equal(got[1], want[1])   # integer outputs: exact
    assert torch.equal(mid[0], want_mid[0]) and torch.equal(mid[1], want_mid[1])
    # point-mass drafts (no draft logits) go through the same scratch
    a1 = b.csd_spec_accept(t, None, tok, max(temperature, 0.5), seed=3)
    a2 = b.csd_spec_accept_static(t, None, tok, max(temperature, 0.5), seed=3, out=outputs(rows))
    assert torch.equal(a1[0], a2[0]) and torch.equal(a1[1], a2[1])


def test_allocates_nothing_and_takes_empty_and_greedy_calls(b):
    t, d, tok = workloads.accept_case(32, 4, 32000, 0.5, seed=9, device="cuda")
    out = outputs(32)
    b.csd_spec_accept_static(t, d, tok, 1.0, out=out)           # the first call on a device looks the scratch up
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for step in range(3):
        b.csd_spec_accept_static(t, d, tok, 1.0, step=step, out=out)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before          # no device memory was taken
    # greedy review with draft logits present (they are ignored), against the workspace entry point
    want = b.csd_spec_accept(t, d, tok, 0.0)
    got = b.csd_spec_accept_static(t, d, tok, 0.0, out=outputs(32))
    assert torch.equal(got[0], want[0]) and torch.equal(got[1], want[1])
    # no rows: nothing to do, nothing touched
    keep = outputs(4)
    code = b.lib.csd_spec_accept_static(t.data_ptr(), None, None, tok.data_ptr(), 0, 4, 32000, 1.0, 1.0, 0, 0,
                                        keep[0].data_ptr(), keep[1].data_ptr(), None)
    torch.cuda.synchronize()
    assert code == 0 and (keep[0] == -7).all() and (keep[1] == -7).all()


def test_refuses_what_does_not_fit_and_bad_arguments(b):
    cap = b.lib.csd_spec_accept_static_capacity()
    assert cap == 2 << 20
    assert b.lib.csd_spec_accept_workspace_bytes(64, 16, 128256) <= cap      # the documented largest case fits
    rows, k, V = 256, 16, 128256
    assert b.lib.csd_spec_accept_workspace_bytes(rows, k, V) > cap
    t = torch.zeros(1, device="cuda")       # never read: the size check comes first
    out = outputs(rows)
    code = b.lib.csd_spec_accept_static(t.data_ptr(), None, None, t.data_ptr(), rows, k, V, 1.0, 1.0, 0, 0,
                                        out[0].data_ptr(), out[1].data_ptr(), None)
    assert code == 3                        # CSD_ERR_CAPACITY
    code = b.lib.csd_spec_accept_static(t.data_ptr(), None, None, t.data_ptr(), 1, 1, 8, 1.0, 0.5, 0, 0,
                                        out[0].data_ptr(), out[1].data_ptr(), None)
    assert code == 1                        # lenience below 1
