"""Embedding lookup from a quantised table against the oracle's dequantised rows, bit for bit."""
import numpy as np
import pytest

from oracle import qlinear_oracle as O
from workloads import configs as C

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P(_built_library):
    import paper_2505_00232_b200 as P
    return P


@pytest.fixture(scope="module")
def torch():
    import torch
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    return torch


CASES = [
    # (N rows, K, bits, group): several row super-blocks and chunks, ragged N, a K tail for int4, every scheme
    (8, 32, 8, 0), (24, 96, 4, 32), (136, 160, 8, 0), (200, 352, 4, 32), (1000, 64, 4, 0), (520, 1056, 8, 0),
    (264, 2304, 4, 32), (40, 256, 4, 64), (16, 384, 4, 128), (4104, 4096, 4, 32),
]


@pytest.mark.parametrize("N,K,bits,group", CASES)
def test_embed_rows_equal_rounded_dequantised_rows(P, torch, N, K, bits, group):
    layer = C.LayerSpec("emb", N, K, bits, group, *((-8, 7) if bits == 4 else (-128, 127)))
    q, s = C.layer_weights(9000 + N + K, layer)
    lin = P.QLinear.from_weights(q, s, bits, group, device="cuda:0")
    rng = np.random.default_rng(N + K)
    ids = np.concatenate([[0, N - 1, N - 1, 0], rng.integers(0, N, size=61)]).astype(np.int32)
    y = lin.embed(torch.from_numpy(ids).cuda()).cpu().numpy()
    want = O.dequantize(q, s, group)[ids].astype(np.float16)            # fp64 product, one rounding to fp16
    assert y.shape == want.shape
    assert (y.view(np.uint16) == want.view(np.uint16)).all()


def test_embed_out_of_range_rows_are_zero_and_empty_call(P, torch):
    layer = C.LayerSpec("emb", 136, 160, 4, 32, -8, 7)
    q, s = C.layer_weights(9100, layer)
    lin = P.QLinear.from_weights(q, s, 4, 32, device="cuda:0")
    ids = np.array([-1, 136, 5, 2 ** 31 - 1], dtype=np.int32)
    y = lin.embed(torch.from_numpy(ids).cuda()).cpu().numpy()
    want = O.dequantize(q, s, 32)[[5]].astype(np.float16)
    assert (y[[0, 1, 3]].view(np.uint16) == 0).all()
    assert (y[2].view(np.uint16) == want[0].view(np.uint16)).all()
    empty = lin.embed(torch.empty((0,), dtype=torch.int32, device="cuda"))
    assert empty.shape == (0, 160)


def test_embed_table_is_also_an_lm_head(P, torch):
    """One blob, two uses: rows out through qlinear_embed, logits through qlinear_forward."""
    layer = C.LayerSpec("emb", 520, 256, 4, 32, -8, 7)
    q, s = C.layer_weights(9200, layer)
    x = C.layer_activations(9200, layer, 2)
    lin = P.QLinear.from_weights(q, s, 4, 32, device="cuda:0")
    ids = torch.arange(0, 520, 7, dtype=torch.int32, device="cuda")
    rows = lin.embed(ids).cpu().numpy()
    want = O.dequantize(q, s, 32)[::7].astype(np.float16)
    assert (rows.view(np.uint16) == want.view(np.uint16)).all()
    y = lin.forward(torch.from_numpy(x).cuda()).cpu().numpy()
    y64, A, _ = O.linear(x, q, s, 32)
    assert O.check_against(y, y64, A)[0]
