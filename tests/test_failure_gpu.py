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
    torch.cuda.synchronize()
    # the forward calls see the code through pinned memory, without synchronising, and launch nothing
    y = torch.full((3, 264), 7.0, dtype=torch.float16, device="cuda")
    for _ in range(2):
        with pytest.raises(P.QLinearError) as err:
            lin.forward(x1, out=y)
        assert err.value.status == P.QL_ERR_DEVICE_TIMEOUT
    with pytest.raises(P.QLinearError) as err:
        P.qlinear_forward_group([lin, lin], x1)
    assert err.value.status == P.QL_ERR_DEVICE_TIMEOUT
    torch.cuda.synchronize()
    assert (y == 7.0).all()
    st, detail = lin.device_status()                      # synchronises
    waited = time.time() - t0
    assert st == 5 and detail == 0x9A0, (st, hex(detail))   # QL_ERR_DEVICE_TIMEOUT, the wait's code
    assert 0.2 < waited < 10.0, waited                    # bounded: about a second, not forever
    assert lin.device_status() == (0, 0)                  # reported once, then clear
    after = [lin.forward(x1), lin.forward(x2)]            # same context, same results
    for a, b in zip(before, after):
        assert torch.equal(a, b)
    assert lin.device_status() == (0, 0)


def test_handles_own_no_device_memory(_built_library):
    """The library's device buffers exist once per device: after the first handle, building the 28 handles of a
    4-copy layer set takes no further device memory (only the caller's packed weights do)."""
    import torch
    import paper_2505_00232_b200 as P
    first = P.QLinear.from_weights(*C.layer_weights(1, C.LayerSpec("t", 128, 256, 8, 0, -128, 127)), 8, 0, device="cuda:0")
    blobs = []
    for li, layer in enumerate(C.LLAMA31_8B):
        desc = P.Desc(layer.N, layer.K, layer.bits, layer.group)
        blobs.append((desc, torch.zeros(P.qlinear_packed_size(desc), dtype=torch.uint8, device="cuda")))
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    lins = [P.QLinear(desc, blob) for _ in range(4) for desc, blob in blobs]
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert len(lins) == 28
    assert free0 - free1 < (4 << 20), f"28 handles took {(free0 - free1) / 2**20:.1f} MiB of device memory"
    del lins, first
