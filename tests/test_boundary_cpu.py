"""Host side of the C-ABI: exported symbols, packed sizes, pack/unpack round trip, error codes.
No compute call needs a GPU here."""
import ctypes
import os
import re

import numpy as np
import pytest

from workloads import configs as C

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def P(_built_library):
    import paper_2505_00232_b200 as P
    return P


def test_library_exports_every_declared_symbol(P):
    text = open(os.path.join(ROOT, "include", "qlinear.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = sorted(set(re.findall(r"\b(qlinear_[a-z0-9_]+)\s*\(", text)))
    assert declared, "no declarations found"
    raw = ctypes.CDLL(P.LIB_PATH)
    for name in declared:
        assert hasattr(raw, name), f"{name} declared in include/qlinear.h but not exported"
    assert sorted(P.EXPORTS) == declared
    assert P.lib.qlinear_version() >> 16 == 1
    assert P.status_string(0) == "ok" and "unknown" in P.status_string(99)


@pytest.mark.parametrize("layer", list(C.GEMMA2_2B) + list(C.LLAMA31_8B), ids=lambda l: f"{l.name}{l.N}x{l.K}")
def test_round_trip_config_shapes(P, layer):
    q, s = C.layer_weights(77, layer)
    d = P.Desc(layer.N, layer.K, layer.bits, layer.group)
    blob = P.qlinear_pack(d, q, s)
    assert blob.size == P.qlinear_packed_size(d)
    # packed bytes = algorithmic bytes + header (+ padding of the per-channel scale array)
    assert 0 < blob.size - layer.weight_bytes <= 512
    q2, s2 = P.qlinear_unpack(d, blob)
    assert (q2 == q).all()
    assert (s2.view(np.uint16) == s.view(np.uint16)).all()


@pytest.mark.parametrize("N,K,bits,group", [
    (8, 32, 8, 0), (8, 32, 4, 32), (8, 32, 4, 0), (24, 96, 4, 32), (136, 160, 8, 0), (200, 352, 4, 32),
    (40, 256, 4, 64), (16, 384, 4, 128), (264, 2304, 4, 32), (1000, 64, 8, 0)])
def test_round_trip_odd_shapes_and_extremes(P, N, K, bits, group):
    rng = np.random.default_rng(N * 131 + K)
    lo, hi = (-8, 7) if bits == 4 else (-128, 127)
    q = rng.integers(lo, hi + 1, size=(N, K)).astype(np.int8)
    q[0, 0], q[-1, -1], q[0, -1], q[-1, 0] = lo, hi, hi, lo
    d = P.Desc(N, K, bits, group)
    s = rng.uniform(1e-3, 1e-2, size=(N, d.n_groups)).astype(np.float16)
    blob = P.qlinear_pack(d, q, s)
    q2, s2 = P.qlinear_unpack(d, blob)
    assert (q2 == q).all() and (s2.view(np.uint16) == s.view(np.uint16)).all()
    # a different weight anywhere changes the blob (no position is dropped by the packer)
    for (n, k) in [(0, 0), (N - 1, K - 1), (N // 2, K // 3)]:
        qm = q.copy()
        qm[n, k] = lo if q[n, k] != lo else hi
        assert (P.qlinear_pack(d, qm, s) != blob).any()


def test_pack_is_deterministic_and_position_independent(P):
    layer = C.LayerSpec("t", 136, 160, 4, 32, -8, 7)
    q, s = C.layer_weights(5, layer)
    d = P.Desc(136, 160, 4, 32)
    a, b = P.qlinear_pack(d, q, s), P.qlinear_pack(d, q.copy(), s.copy())
    assert (a == b).all()
    assert a[:4].tobytes() == b"QLB1"


@pytest.mark.parametrize("N,K,bits,group", [(7, 32, 8, 0), (8, 48, 8, 0), (8, 32, 5, 0), (8, 32, 8, 32),
                                            (8, 96, 4, 64), (8, 32, 4, 16), (0, 32, 4, 32), (8, 0, 8, 0)])
def test_unsupported_descriptors(P, N, K, bits, group):
    d = P.Desc(N, K, bits, group)
    assert P.qlinear_packed_size(d) == 0
    with pytest.raises(P.QLinearError) as e:
        P.qlinear_pack(d, np.zeros((max(N, 1), max(K, 1)), np.int8), np.zeros((max(N, 1), 1), np.float16))
    assert e.value.status in (2, 1)


def test_pack_rejects_int4_out_of_range_and_bad_buffers(P):
    d = P.Desc(8, 32, 4, 32)
    q = np.zeros((8, 32), np.int8)
    s = np.ones((8, 1), np.float16)
    for bad in (8, -9, 127, -128):
        qb = q.copy()
        qb[3, 7] = bad
        with pytest.raises(P.QLinearError) as e:
            P.qlinear_pack(d, qb, s)
        assert e.value.status == 1
    dc = d.c()
    size = P.qlinear_packed_size(d)
    buf = np.zeros(size, np.uint8)
    vp = lambda a: a.ctypes.data_as(ctypes.c_void_p)
    assert P.lib.qlinear_pack(ctypes.byref(dc), None, vp(s), vp(buf), size) == 1
    assert P.lib.qlinear_pack(ctypes.byref(dc), vp(q), None, vp(buf), size) == 1
    assert P.lib.qlinear_pack(ctypes.byref(dc), vp(q), vp(s), None, size) == 1
    assert P.lib.qlinear_pack(ctypes.byref(dc), vp(q), vp(s), vp(buf), size - 1) == 1
    assert P.lib.qlinear_pack(None, vp(q), vp(s), vp(buf), size) == 1
    assert not buf.any()                                   # nothing written on error


def test_unpack_checks_header(P):
    d = P.Desc(16, 64, 8, 0)
    q = np.ones((16, 64), np.int8)
    s = np.ones((16, 1), np.float16)
    blob = P.qlinear_pack(d, q, s)
    with pytest.raises(P.QLinearError):
        P.qlinear_unpack(P.Desc(16, 64, 4, 0), blob)       # other scheme, same size class
    bad = blob.copy()
    bad[0] ^= 0xFF
    with pytest.raises(P.QLinearError):
        P.qlinear_unpack(d, bad)


def test_host_calls_that_need_no_device(P):
    assert P.lib.qlinear_destroy(None) == 0
    assert P.lib.qlinear_path_for(None, 4) == 0
    h = ctypes.c_void_p()
    d = P.Desc(16, 64, 8, 0).c()
    assert P.lib.qlinear_create(ctypes.byref(d), None, 0, ctypes.byref(h)) == 1      # null blob
    assert P.lib.qlinear_create(None, ctypes.c_void_p(256), 0, ctypes.byref(h)) == 1
    bad = P.Desc(7, 64, 8, 0).c()
    assert P.lib.qlinear_create(ctypes.byref(bad), ctypes.c_void_p(256), 0, ctypes.byref(h)) == 2
    assert P.lib.qlinear_create(ctypes.byref(d), ctypes.c_void_p(260), 0, ctypes.byref(h)) == 1  # misaligned
    assert P.lib.qlinear_forward(None, ctypes.c_void_p(16), ctypes.c_void_p(32), 1, None) == 1
    assert P.lib.qlinear_embed(None, ctypes.c_void_p(16), 1, ctypes.c_void_p(32), None) == 1
    # grouped call: null arrays, n outside 1..4 and null handles are refused before any CUDA call
    hs = (ctypes.c_void_p * 2)(None, None)
    ys = (ctypes.c_void_p * 2)(ctypes.c_void_p(32), ctypes.c_void_p(64))
    assert P.lib.qlinear_forward_group(None, 2, ctypes.c_void_p(16), ys, 1, None) == 1
    assert P.lib.qlinear_forward_group(hs, 2, ctypes.c_void_p(16), None, 1, None) == 1
    assert P.lib.qlinear_forward_group(hs, 0, ctypes.c_void_p(16), ys, 1, None) == 1
    assert P.lib.qlinear_forward_group(hs, 5, ctypes.c_void_p(16), ys, 1, None) == 1
    assert P.lib.qlinear_forward_group(hs, 2, ctypes.c_void_p(16), ys, 1, None) == 1      # null handles


def test_environment_is_read_once(P, monkeypatch):
    """Every QLINEAR_* switch is read at the first call that needs one, and never again."""
    n = P.lib.qlinear_debug_config_reads()
    assert n == 1
    monkeypatch.setenv("QLINEAR_GEMV_MAX_M", "2")
    monkeypatch.setenv("QLINEAR_GEMM_PAIR", "0")
    assert P.lib.qlinear_debug_config_reads() == 1
    h = ctypes.c_void_p()
    d = P.Desc(16, 64, 8, 0).c()
    P.lib.qlinear_create(ctypes.byref(d), ctypes.c_void_p(256), 0, ctypes.byref(h))   # fails without a device; reads nothing new
    assert P.lib.qlinear_debug_config_reads() == 1
