"""lpdt_quantize_static: the quantizer for callers that cannot provide device scratch
(fixed-buffer training loops, plug-ins living inside someone else's memory pool).

Its range words sit in an array inside the library, shared by all calls, so the test
makes two calls in a row, the second smaller than the first and on different data, and
checks each against lpdt_quantize with an ordinary workspace: codes, scales and zero
points must be identical (integer results bit-exact, scales the same fp32 values).
Collected last on purpose: a failure here cannot hide another test's result.
"""
import numpy as np
import pytest
import torch

from paper_2111_09389_b200 import api

pytestmark = pytest.mark.gpu


def _both(x, nodes, n, mode, rounding):
    xd = torch.from_numpy(x).cuda()
    out = []
    for static in (False, True):
        q = torch.full((nodes, n), 77, dtype=torch.int8, device="cuda")
        s = torch.zeros(nodes, dtype=torch.float32, device="cuda")
        zp = torch.zeros(nodes, dtype=torch.int32, device="cuda") if mode == 1 else None
        if static:
            api.lpdt_quantize_static(xd, nodes, n, n, q, s, mode=mode, rounding=rounding, seed=99, ctr_offset=2,
                                     zero_point=zp)
        else:
            ws = torch.empty(api.lpdt_quantize_workspace_size(nodes), dtype=torch.uint8, device="cuda")
            api.lpdt_quantize(xd, nodes, n, n, q, s, ws, mode=mode, rounding=rounding, seed=99, ctr_offset=2,
                              zero_point=zp)
        torch.cuda.synchronize()
        out.append((q.cpu().numpy(), s.cpu().numpy(), None if zp is None else zp.cpu().numpy()))
    return out


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    rng = np.random.default_rng(7)
    # first call: large values on 16 nodes; second: 5 nodes of much smaller values, so a
    # stale range word from the first call would show as a wrong scale
    cases = [(16, 40000, 50.0, 0, 0), (5, 1003, 0.01, 0, 1), (3, 4096, 1.0, 1, 0)]
    for nodes, n, mag, mode, rounding in cases:
        x = (rng.standard_normal((nodes, n)) * mag).astype(np.float32)
        (q0, s0, z0), (q1, s1, z1) = _both(x, nodes, n, mode, rounding)
        assert np.array_equal(s0, s1)
        assert np.array_equal(q0, q1)
        if mode == 1:
            assert np.array_equal(z0, z1)
        assert s0.max() < 10 * mag          # scale follows this call's data only


def test_too_many_nodes_is_rejected_before_any_launch():
    nodes = 1025
    x = torch.zeros(nodes, 4, device="cuda")
    q = torch.zeros(nodes, 4, dtype=torch.int8, device="cuda")
    s = torch.zeros(nodes, device="cuda")
    with pytest.raises(api.LpdtError) as e:
        api.lpdt_quantize_static(x, nodes, 4, 4, q, s)
    assert e.value.code == 3
