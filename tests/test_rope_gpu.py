"""Rotary embedding + Q/K/V layout transformation (paper Section 3.6) against the CPU oracle."""
import numpy as np
import pytest

from oracle import qlinear_oracle as O

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


def case(seed, B, S, h_q, h_kv, d_h, n_pos, theta=10000.0):
    rng = np.random.default_rng(seed)
    T = B * S
    q = (4 * rng.standard_normal((T, h_q * d_h))).astype(np.float16)
    k = (4 * rng.standard_normal((T, h_kv * d_h))).astype(np.float16)
    v = rng.standard_normal((T, h_kv * d_h)).astype(np.float16)
    pos = rng.integers(0, n_pos, size=T).astype(np.int32)
    pos[0], pos[-1] = 0, n_pos - 1
    ang = np.arange(n_pos, dtype=np.float64)[:, None] * (theta ** (-np.arange(d_h // 2) * 2.0 / d_h))[None, :]
    return q, k, v, pos, np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)


def run(P, torch, q, k, v, pos, cos, sin, B, S, h_q, h_kv, d_h):
    t = [torch.from_numpy(a).cuda() for a in (q, k, v, pos, cos, sin)]
    out = P.qlinear_rope_qkv(*t, B, S, h_q, h_kv, d_h)
    torch.cuda.synchronize()
    return [o.cpu().numpy() for o in out]


# Llama3.1-8B (32 / 8 heads of 128), Gemma2-2B (8 / 4 heads of 256), multi-head, multi-query, a batch, one token
@pytest.mark.parametrize("B,S,h_q,h_kv,d_h", [(1, 300, 32, 8, 128), (1, 129, 8, 4, 256), (2, 17, 4, 4, 64), (3, 5, 8, 1, 16),
                                              (1, 1, 32, 8, 128), (4, 1, 16, 2, 32)])
def test_parity(P, torch, B, S, h_q, h_kv, d_h):
    q, k, v, pos, cos, sin = case(B * 1000 + S + d_h, B, S, h_q, h_kv, d_h, 4096)
    qo, ko, vo = run(P, torch, q, k, v, pos, cos, sin, B, S, h_q, h_kv, d_h)
    q64, k64, v64, aq, ak = O.rope_qkv(q, k, v, pos, cos, sin, B, S, h_q, h_kv, d_h)
    assert qo.shape == q64.shape and ko.shape == k64.shape and vo.shape == v64.shape
    assert (vo.astype(np.float64) == v64).all()                          # V is only moved: bit-exact
    for got, ref, amp in ((qo, q64, aq), (ko, k64, ak)):
        d = np.abs(got.astype(np.float64) - ref)
        bound = O.rope_bound(ref, amp)
        assert (d <= bound).all(), f"worst |d| / bound = {(d / bound).max():.3e}"


def test_angle_zero_is_the_pure_layout_change(P, torch):
    B, S, h_q, h_kv, d_h = 2, 9, 12, 4, 32
    q, k, v, pos, cos, sin = case(5, B, S, h_q, h_kv, d_h, 8)
    qo, ko, vo = run(P, torch, q, k, v, pos, np.ones_like(cos), np.zeros_like(sin), B, S, h_q, h_kv, d_h)
    g = h_q // h_kv
    assert (qo == q.reshape(B, S, h_kv, g, d_h).transpose(0, 2, 1, 3, 4).reshape(B * h_kv, S * g, d_h)).all()
    assert (ko == k.reshape(B, S, h_kv, d_h).transpose(0, 2, 1, 3).reshape(B * h_kv, S, d_h)).all()
    assert (vo == v.reshape(B, S, h_kv, d_h).transpose(0, 2, 1, 3).reshape(B * h_kv, S, d_h)).all()


def test_outputs_feed_the_kv_cache_calls(P, torch):
    """The blocks this kernel writes are what the KV-cache entry points take: append K / V rows of one KV head, score the
    head's query rows against the cached keys (paper Section 3.8), against the oracle's attention scores."""
    B, S, h_q, h_kv, d_h = 1, 40, 8, 2, 128
    q, k, v, pos, cos, sin = case(6, B, S, h_q, h_kv, d_h, 64)
    pos[:] = np.arange(S)
    t = [torch.from_numpy(a).cuda() for a in (q, k, v, pos, cos, sin)]
    qo, ko, vo = P.qlinear_rope_qkv(*t, B, S, h_q, h_kv, d_h)
    q64, k64, _, _, _ = O.rope_qkv(q, k, v, pos, cos, sin, B, S, h_q, h_kv, d_h)
    for hk in range(h_kv):
        cache = P.KVCache(64, d_h, device="cuda:0")
        cache.append(ko[hk].contiguous(), vo[hk].contiguous())
        g = h_q // h_kv
        rows = qo[hk][(S - 1) * g:(S - 1) * g + g].contiguous()          # the last token's query heads of this group
        scores = cache.scores(rows)
        torch.cuda.synchronize()
        ref = q64[hk][(S - 1) * g:(S - 1) * g + g] @ k64[hk].T
        got = scores.cpu().numpy().astype(np.float64)[:, :S]
        # the cache keeps int8 keys with one scale per token: 2^-7 of the row's largest element per term
        tol = 1.5 * 2.0 ** -7 * np.abs(q64[hk][(S - 1) * g:(S - 1) * g + g]).sum(axis=1, keepdims=True) * np.abs(k64[hk]).max(axis=1)[None, :] + 1e-2
        assert (np.abs(got - ref) <= tol).all()


def test_guard_bands_and_bad_arguments(P, torch):
    B, S, h_q, h_kv, d_h = 1, 7, 4, 2, 16
    q, k, v, pos, cos, sin = case(7, B, S, h_q, h_kv, d_h, 16)
    qo, ko, vo = run(P, torch, q, k, v, pos, cos, sin, B, S, h_q, h_kv, d_h)
    assert np.isfinite(qo).all() and np.isfinite(ko).all()
    t = [torch.from_numpy(a).cuda() for a in (q, k, v, pos, cos, sin)]
    with pytest.raises(P.QLinearError):
        P.qlinear_rope_qkv(*t, B, S, 3, 2, d_h)                           # h_q not a multiple of h_kv
    with pytest.raises(P.QLinearError):
        P.qlinear_rope_qkv(*t, B, S + 1, h_q, h_kv, d_h)                  # shapes do not match
    with pytest.raises(P.QLinearError):
        P.qlinear_rope_qkv(t[0], t[1], t[2], t[3].long(), t[4], t[5], B, S, h_q, h_kv, d_h)
