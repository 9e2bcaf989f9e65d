"""qlinear_decode_static: the decode call for callers that may not allocate device memory (a serving loop
whose memory was carved up front, a pool that owns the whole device, a plugin that only gets buffers).
It must give what qlinear_forward gives, on two calls in a row (its static scratch keeps the previous
call's contents).  Collected last on purpose: a failure here cannot hide the other tests' results."""
import ctypes

import numpy as np
import pytest

from oracle import qlinear_oracle as O
from workloads import configs as C

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("M,N,K,bits,group", [(1, 4096, 4096, 8, 0), (4, 2304, 2304, 4, 32), (8, 1024, 4096, 4, 0)])
def test_static_scratch_decode_matches_forward_twice(_built_library, M, N, K, bits, group):
    import torch
    import paper_2505_00232_b200 as P
    assert torch.cuda.is_available()
    layer = C.LayerSpec("t", N, K, bits, group, *((-8, 7) if bits == 4 else (-128, 127)))
    q, s = C.layer_weights(4242, layer)
    lin = P.QLinear.from_weights(q, s, bits, group, device="cuda:0")
    for call in range(2):                                   # second call: new input, scratch still holds the first
        x = C.layer_activations(4242 + call, layer, M)
        xd = torch.from_numpy(x).cuda()
        y_ref = lin.forward(xd)
        y_new = torch.full_like(y_ref, float("nan"))
        P.qlinear_decode_static(lin.desc, lin.packed, xd, out=y_new)
        torch.cuda.synchronize()
        a, b = y_new.cpu().numpy(), y_ref.cpu().numpy()
        _, A, _ = O.linear(x, q, s, group)                  # the tolerance denominator of the parity tests
        d = np.abs(a.astype(np.float64) - b.astype(np.float64))
        assert np.isfinite(a.astype(np.float32)).all()
        assert (d <= 2 * O.ELEM_TOL * A).all(), f"call {call}: worst {np.max(d / np.maximum(A, 1e-30)):.3e}"
        assert np.linalg.norm(d) <= 2 * O.REL_L2_TOL * np.linalg.norm(b.astype(np.float64))
        y64, _, _ = O.linear(x, q, s, group)
        assert O.check_against(a, y64, A)[0]                # and it meets the oracle's bar on its own


def test_static_scratch_decode_rejects_what_it_cannot_hold(_built_library):
    import torch
    import paper_2505_00232_b200 as P
    f = P.lib.qlinear_decode_static
    buf = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    x = torch.zeros((9, 64), dtype=torch.float16, device="cuda")
    y = torch.zeros((9, 16), dtype=torch.float16, device="cuda")
    d = P.Desc(16, 64, 8, 0).c()
    vp = ctypes.c_void_p
    assert f(ctypes.byref(d), vp(buf.data_ptr()), vp(x.data_ptr()), vp(y.data_ptr()), 9, 0, None) == 1   # M > 8
    assert f(ctypes.byref(d), vp(buf.data_ptr()), vp(x.data_ptr()), vp(y.data_ptr()), 0, 0, None) == 1
    assert f(ctypes.byref(d), None, vp(x.data_ptr()), vp(y.data_ptr()), 1, 0, None) == 1
    huge = P.Desc(4097 * 128, 64, 8, 0).c()                 # more row super-blocks than the static counters
    assert f(ctypes.byref(huge), vp(buf.data_ptr()), vp(x.data_ptr()), vp(y.data_ptr()), 1, 0, None) == 2
    odd = P.Desc(16, 96, 4, 32).c()                         # int4 with K % 64 != 0
    assert f(ctypes.byref(odd), vp(buf.data_ptr()), vp(x.data_ptr()), vp(y.data_ptr()), 1, 0, None) == 2
