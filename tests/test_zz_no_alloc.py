"""eesd_accept_resample_static: the acceptance step for callers that may not allocate.

Some users of the library verify a round from a place where device allocation is off limits (a
serving engine with a frozen memory plan, a plug-in that only receives its input and output
tensors).  That entry point keeps its scratch in a fixed device array inside the library.  This
file checks, through the C ABI, that it gives exactly what the ordinary entry point gives and what
the CPU oracle gives on the same logits and uniforms (integer results: bit-exact), on two calls in a row so that state left behind by the first call
cannot leak into the second, and that it refuses problems larger than its built-in scratch.
It is collected last on purpose.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import eesd_synth as synth
import oracle

pytestmark = pytest.mark.gpu


def _static(L, p, q, x, ua, ur, T):
    B, K, V = q.shape
    n = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    y = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    st = L.eesd_accept_resample_static(torch.cuda.current_stream().cuda_stream, p.data_ptr(), q.data_ptr(),
                                       x.data_ptr(), ua.data_ptr(), ur.data_ptr(), B, K, V, T,
                                       n.data_ptr(), y.data_ptr())
    return st, n, y


def test_static_scratch_entry_point_matches_the_ordinary_one_twice_in_a_row():
    import paper_2406_03853_b200 as eesd
    L = eesd.lib()
    # first call (also the per-device set-up), then a second one of a different shape
    for case, (B, K, V, T) in enumerate([(64, 16, 32000, 1.0), (8, 4, 1025, 0.7), (64, 16, 32000, 0.0)]):
        p, q, ua, ur, ud = synth.accept_case(500 + case, B, K, V, 2.0, 1.0, device="cuda")
        x = eesd.sample_rows(q.view(B * K, V), ud.view(B * K), T).view(B, K).contiguous()
        n_ref, y_ref = eesd.accept_resample(p, q, x, ua, ur, T)
        n_orc, y_orc = oracle.accept_resample_batch(p.cpu().numpy(), q.cpu().numpy(), x.cpu().numpy(), ua.cpu().numpy(),
                                                    ur.cpu().numpy(), T)
        np.testing.assert_array_equal(n_ref.cpu().numpy(), n_orc)
        np.testing.assert_array_equal(y_ref.cpu().numpy(), y_orc)
        for _ in range(2):
            st, n, y = _static(L, p, q, x, ua, ur, T)
            assert st == 0
            torch.cuda.synchronize()
            assert torch.equal(n, n_ref) and torch.equal(y, y_ref)


def test_static_scratch_entry_point_rejects_what_does_not_fit():
    import paper_2406_03853_b200 as eesd
    L = eesd.lib()
    t = torch.zeros(16, device="cuda")
    i = torch.zeros(16, dtype=torch.int32, device="cuda")
    args = (None, t.data_ptr(), t.data_ptr(), i.data_ptr(), t.data_ptr(), t.data_ptr())
    assert L.eesd_accept_resample_static(*args, 1025, 1, 8, 1.0, i.data_ptr(), i.data_ptr()) == -2   # batch too large
    assert L.eesd_accept_resample_static(*args, 400, 6, 8, 1.0, i.data_ptr(), i.data_ptr()) == -2    # 5200 rows
    assert L.eesd_accept_resample_static(*args, 0, 1, 8, 1.0, i.data_ptr(), i.data_ptr()) == -1
    assert L.eesd_accept_resample_static(None, None, None, None, None, None, 1, 1, 8, 1.0, None, None) == -1
