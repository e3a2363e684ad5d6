"""The context-free, allocation-free router entry point gives what the ordinary one gives.

first_prefill_route_static exists for hosts that may not call cudaMalloc where they route a
batch (a framework allocator already owns the GPU's memory, a fixed memory budget, or a
latency path that cannot afford cudaMalloc's device-wide synchronisation).  It keeps its
scratch in an array built into the library, shared by every call on the device and never
cleared between calls.  The test therefore makes two calls in a row -- a long batch, then a
shorter one with different data, so the second runs over the first call's leftovers -- and
checks both against the host oracle (masks bit for bit, scores to float32 rounding) and against
first_prefill_route.  It also checks the property the entry point exists for: the device's free
memory is the same before and after a call.
This file sorts last on purpose: a run that stops at the first failure has by then run
every other test.
"""
import numpy as np
import pytest

import first_inputs as fi
import oracle
from harness import gpu_weights, to_dev, widen

pytestmark = pytest.mark.gpu


def _both(ctx, L, layer, hid, cu, rw, bias, mode):
    import torch
    from paper_2410_12513_b200 import first_prefill_route_static
    B = len(cu) - 1
    cu_t = torch.from_numpy(cu).cuda()
    hid_t = to_dev(hid, hid.dtype == np.uint16)
    rw_t = to_dev(rw, False)
    b_t = None if bias is None else torch.tensor([bias], dtype=torch.float32, device="cuda")
    m_ref = torch.full((B, L), 9, dtype=torch.uint8, device="cuda")
    s_ref = torch.full((B, L), -1.0, dtype=torch.float32, device="cuda")
    m_new, s_new = m_ref.clone(), s_ref.clone()
    ctx.prefill_route(layer, hid_t, cu_t, rw_t, b_t, 0.5, mode, m_ref, s_ref)
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    first_prefill_route_static(layer, L, hid_t, cu_t, rw_t, b_t, 0.5, mode, m_new, s_new, flags)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert ctx.device_flags() == 0 and int(flags.item()) == 0
    # against the host oracle on the same bytes
    rho, keep = oracle.route_batch(widen(hid), cu, rw, bias, 0.5, mode)
    assert np.abs(rho - 0.5).min() >= 1e-3  # (inputs chosen away from the threshold)
    assert np.array_equal(m_new[:, layer].cpu().numpy(), keep)
    assert np.abs(s_new[:, layer].cpu().numpy() - rho).max() <= 2e-6
    # and against the entry point that takes its scratch from a context
    assert np.array_equal(m_new.cpu().numpy(), m_ref.cpu().numpy())
    assert np.abs(s_new.cpu().numpy() - s_ref.cpu().numpy()).max() <= 1e-6
    return m_new[:, layer].cpu().numpy(), free0, free1


def test_static_router_matches_context_router_on_two_calls_in_a_row():
    import torch
    from paper_2410_12513_b200 import FirstContext, FirstError, first_prefill_route_static
    L, D = 3, 512
    shape = fi.ModelShape(L, D, 4, 4, 128, 1024, 64)
    ctx = FirstContext(shape, 0, 16, 2048, gpu_weights(fi.make_weights(shape, 1, False)))
    # call 1: long ragged batch, bfloat16 hidden states, the paper's mean-of-sigmoid order
    lens1 = np.array([700, 3, 1500, 64, 1, 257], np.int32)
    cu1 = np.concatenate([[0], np.cumsum(lens1)]).astype(np.int32)
    hid1 = fi.normal((int(cu1[-1]), D), 1.0, 11, "hid1", True)
    rw1 = fi.normal((D,), 0.05, 11, "rw1")
    k1, _, _ = _both(ctx, L, 1, hid1, cu1, rw1, None, 0)
    # call 2: shorter batch, float32 hidden states, pooled order, with a bias: runs over call 1's leftovers.
    # By now the array's address has been looked up, so this call must leave the device's free memory as it was.
    lens2 = np.array([5, 40, 9], np.int32)
    cu2 = np.concatenate([[0], np.cumsum(lens2)]).astype(np.int32)
    hid2 = fi.normal((int(cu2[-1]), D), 1.0, 12, "hid2", False)
    rw2 = fi.normal((D,), 0.05, 12, "rw2")
    k2, free0, free1 = _both(ctx, L, 2, hid2, cu2, rw2, 0.01, 1)
    assert free1 == free0, (free0, free1)
    assert len(k1) == 6 and len(k2) == 3
    # an empty sequence is reported through the caller's flag word and its outputs are left alone
    cu3 = torch.tensor([0, 0, 5], dtype=torch.int32, device="cuda")
    m = torch.full((2, L), 9, dtype=torch.uint8, device="cuda")
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    first_prefill_route_static(0, L, to_dev(hid2[:5], False), cu3, to_dev(rw2, False), None, 0.5, 0, m, None, flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == 16 and m[:, 0].cpu().numpy().tolist() == [9, m[1, 0].item()] and m[1, 0].item() in (0, 1)
    # without a flag word of the caller's the built-in one is used: the call succeeds, the empty sequence's
    # outputs stay as they were and the other sequence gets what the oracle gives
    m2 = torch.full((2, L), 9, dtype=torch.uint8, device="cuda")
    first_prefill_route_static(0, L, to_dev(hid2[:5], False), cu3, to_dev(rw2, False), None, 0.5, 0, m2, None, None)
    torch.cuda.synchronize()
    _, keep5 = oracle.route_batch(hid2[:5], np.array([0, 5]), rw2, None, 0.5, 0)
    assert m2[:, 0].cpu().numpy().tolist() == [9, int(keep5[0])]
    assert m[1, 0].item() == int(keep5[0])
    # sizes beyond the built-in scratch are refused before anything runs
    too_many = 1048576 + 1
    with pytest.raises(FirstError) as e:
        from paper_2410_12513_b200 import lib
        rc = lib().first_prefill_route_static(0, L, D, to_dev(hid2, False).data_ptr(), 0, cu3.data_ptr(), 2, too_many,
                                              to_dev(rw2, False).data_ptr(), None, 0.5, 0, m.data_ptr(), None, None,
                                              None)
        raise FirstError(rc, "first_prefill_route_static")
    assert e.value.status == -4
