"""Failure path on the device: a bounded wait that runs out is reported, and the device stays usable."""
import time

import numpy as np
import pytest

from workloads import configs as C

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_and_device_stays_usable(_built_library):
    import torch
    import paper_2505_00232_b200 as P
    layer = C.LayerSpec("t", 264, 512, 4, 32, -8, 7)
    q, s = C.layer_weights(7700, layer)
    lin = P.QLinear.from_weights(q, s, 4, 32, device="cuda:0")
    x1 = torch.from_numpy(C.layer_activations(7700, layer, 3)).cuda()
    x2 = torch.from_numpy(C.layer_activations(7700, layer, 200)).cuda()
    before = [lin.forward(x1).clone(), lin.forward(x2).clone()]
    assert lin.device_status() == (0, 0)
    t0 = time.time()
    lin.debug_expire_wait()                               # nothing completes this barrier: the wait gives up
    st, detail = lin.device_status()                      # synchronises
    waited = time.time() - t0
    assert st == 5 and detail == 0x9A0, (st, hex(detail))   # QL_ERR_DEVICE_TIMEOUT, the wait's code
    assert 0.2 < waited < 10.0, waited                    # bounded: about a second, not forever
    assert lin.device_status() == (0, 0)                  # reported once, then clear
    after = [lin.forward(x1), lin.forward(x2)]            # same context, same results
    for a, b in zip(before, after):
        assert torch.equal(a, b)
    assert lin.device_status() == (0, 0)
