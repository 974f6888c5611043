"""The entry point that allocates nothing (egeria_sp_loss_static).

Some callers cannot get device memory when they need an evaluation -- a framework whose
caching allocator already owns the whole GPU, a latency-critical loop that must not hit
the device-wide synchronisation of an allocation, a plugin that is given a stream but no
allocator -- so they cannot provide the workspace a context needs either.  For them the
library carries a fixed scratch array in its own image.  This file checks that entry
point against the ordinary one (egeria_sp_loss_batch through a context) and against the
float64 CPU oracle, on calls in a row, because the second call finds the first call's
leftovers in the shared array.

It is named to be collected last: a run that stops at the first failure has then already
run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2201_06227_b200 import binding as eg
from paper_2201_06227_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"


def context_loss(at, ar):
    b, d = at.shape
    ctx = eg.Context([d], b, 5, 1e-3, device=DEV)
    out = ctx.egeria_sp_loss_batch([at], [ar]).cpu().numpy().astype(np.float64)[0]
    ctx.check_device_status()
    ctx.close()
    return out


def close_enough(a, ref):
    # the tolerance of the parity tests: 1e-3 relative or 1e-7 absolute
    return abs(a - ref) <= max(1e-3 * abs(ref), 1e-7)


def test_static_entry_matches_context_entry_on_consecutive_calls():
    # call 1: tensor-core path, two row groups, ragged tail; call 2: smaller b (other tile
    # layout) on a d that forces the CUDA-core path; call 3: the first shape again.
    cases = [(96, 8200, "relu", 0.2, 1), (40, 1001, "normal", 0.3, 2), (96, 8200, "relu", 0.2, 1)]
    inputs = [wl.make_pair(b, d, kind, s, seed=900 + sd, device=DEV) for b, d, kind, s, sd in cases]
    out = torch.empty(1, dtype=torch.float32, device=DEV)
    got = []
    for at, ar in inputs:                      # back to back on one stream, no sync in between
        eg.egeria_sp_loss_static(at, ar, out_loss=out)
        got.append(out.clone())
    torch.cuda.synchronize()
    got = [float(g.cpu()[0]) for g in got]
    assert eg.egeria_sp_loss_static_status() == eg.OK
    for (at, ar), g in zip(inputs, got):
        ref = context_loss(at, ar)
        assert ref > 0
        assert close_enough(g, ref), (g, ref)
        exact = oracle.sp_loss(wl.bf16_bits(at), wl.bf16_bits(ar))      # and the definition itself
        assert close_enough(g, exact), (g, exact)
    assert got[0] == got[2]                    # same input, same result, whatever ran in between


def test_static_entry_refuses_a_capturing_stream():
    """Every call copies its work split from host memory that is gone when the call returns; a
    graph would replay those copies from dead memory, so a capturing stream is turned away and
    nothing is recorded."""
    at, ar = wl.make_pair(64, 512, "normal", 0.2, seed=11, device=DEV)
    out = torch.zeros(1, dtype=torch.float32, device=DEV)
    eg.egeria_sp_loss_static(at, ar, out_loss=out)          # set-up happens here, outside any capture
    torch.cuda.synchronize()
    want = float(out.cpu()[0])
    x = torch.zeros(4, device=DEV)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        g.capture_begin()
        try:
            x.add_(1.0)
            with pytest.raises(eg.EgeriaError) as e:
                eg.egeria_sp_loss_static(at, ar, out_loss=out, stream=side)
        finally:
            g.capture_end()
    assert e.value.status == eg.ERR_INVALID_ARG
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    assert float(out.cpu()[0]) == want                      # untouched by the refused call
    got = float(eg.egeria_sp_loss_static(at, ar, out_loss=out).cpu()[0])
    assert got == want                                      # and the entry point still works


def test_static_entry_rejects_sizes_beyond_its_scratch():
    at, ar = wl.make_pair(200, 64, "normal", 0.1, seed=5, device=DEV)
    with pytest.raises(eg.EgeriaError) as e:
        eg.egeria_sp_loss_static(at, ar)
    assert e.value.status == eg.ERR_UNSUPPORTED_SHAPE
    # and stays usable afterwards
    at, ar = wl.make_pair(128, 256, "normal", 0.1, seed=6, device=DEV)
    got = float(eg.egeria_sp_loss_static(at, ar).cpu()[0])
    assert close_enough(got, context_loss(at, ar))
