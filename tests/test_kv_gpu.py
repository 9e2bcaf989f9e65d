"""The KV cache held as weights (paper Section 3.8) against the CPU oracle, through the C-ABI, on a B200: the
protocol of the paper's LLM benchmark, 1024 prefill tokens then 256 decode steps (Section 4.2), for one KV head of
a grouped-query model (4 query heads per KV head, d_h = 128)."""
import numpy as np
import pytest

from oracle import qlinear_oracle as O
from workloads import generators as gen

pytestmark = pytest.mark.gpu

CACHE, DH, GROUP = 1280, 128, 4


@pytest.fixture(scope="module")
def P(_built_library):
    import paper_2505_00232_b200 as P
    return P


@pytest.fixture(scope="module")
def torch():
    import torch
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    return torch


def tensors(seed, T):
    k = gen.normal_fp16(seed, 1, (T, DH))
    v = gen.normal_fp16(seed, 2, (T, DH))
    v[5, :] = 0                                         # a zero vector: stored as zeros with scale 1
    k[7, :] *= np.float16(40.0)                         # per-token scales really differ
    return k, v


def test_append_writes_exactly_the_oracles_integers_and_scales(P, torch):
    k, v = tensors(811, CACHE)
    cache = P.KVCache(CACHE, DH)
    kd, vd = torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda()
    cache.append(kd[:1024], vd[:1024])                  # prefill: 1024 tokens in one call
    for t in range(1024, CACHE):                        # decode: one token per step
        cache.append(kd[t:t + 1], vd[t:t + 1])
    torch.cuda.synchronize()
    assert cache.length == CACHE and cache.k.device_status() == (0, 0)
    k_q, k_s = O.kv_quantize_rows(k)
    v_q, v_s = O.kv_quantize_rows(v)
    assert (cache.k.debug_unpack().cpu().numpy() == k_q).all()           # K cache: O = positions, I = d_h
    assert (cache.v.debug_unpack().cpu().numpy() == v_q.T).all()         # V cache: O = d_h, I = positions
    _, ks_blob = P.qlinear_unpack(cache.k.desc, cache.k.packed.cpu().numpy())
    assert (ks_blob.reshape(-1).view(np.uint16) == k_s.view(np.uint16)).all()
    assert (cache.v_scale.cpu().numpy().view(np.uint16) == v_s.view(np.uint16)).all()


@pytest.mark.parametrize("R,T", [(GROUP, 1280), (GROUP, 1031), (1, 200), (GROUP * 128, 1024)],
                         ids=["decode-full-cache", "decode-partial-cache", "one-row", "prefill-512-rows"])
def test_attention_products_match_the_oracle(P, torch, R, T):
    """scores = Q K^T and out = P V through the linear kernels (R = S * h_q / h_kv query rows of one KV head),
    inside the linear layer's tolerance; positions beyond the cache length score exactly 0."""
    k, v = tensors(900 + T, T)
    qry = gen.normal_fp16(900 + T, 3, (R, DH))
    cache = P.KVCache(CACHE, DH)
    cache.append(torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda())
    sc = cache.scores(torch.from_numpy(qry).cuda())
    torch.cuda.synchronize()
    sc_np = sc.cpu().numpy()
    assert (sc_np[:, T:] == 0).all()
    # probabilities: a softmax over the live positions (computed here in fp64: masking and softmax are the caller's)
    z = sc_np[:, :T].astype(np.float64) / np.sqrt(DH)
    p = np.exp(z - z.max(axis=1, keepdims=True))
    prob = np.zeros((R, CACHE), np.float16)
    prob[:, :T] = (p / p.sum(axis=1, keepdims=True)).astype(np.float16)
    out = cache.output(torch.from_numpy(prob).cuda())
    torch.cuda.synchronize()
    sc64, A_sc, out64, A_out = O.kv_attention(qry, k, v, prob[:, :T])
    ok, rel, worst = O.check_against(sc_np[:, :T], sc64, A_sc)
    assert ok, ("scores", rel, worst)
    ok, rel, worst = O.check_against(out.cpu().numpy(), out64, A_out)
    assert ok, ("output", rel, worst)


def test_append_argument_errors(P, torch):
    cache = P.KVCache(256, 64)
    a = torch.zeros((200, 64), dtype=torch.float16, device="cuda")
    cache.append(a, a)
    with pytest.raises(P.QLinearError):
        cache.append(a, a)                              # 400 > 256 positions
    other = P.KVCache(256, 32)
    import ctypes
    vp = ctypes.c_void_p
    assert P.lib.qlinear_kv_append(cache.k._h, other.v._h, vp(a.data_ptr()), vp(a.data_ptr()), vp(cache.v_scale.data_ptr()), 0, 1, None) == 1


@pytest.mark.parametrize("n_heads", [3, 8, 11])
def test_all_heads_in_one_launch_match_the_per_head_calls(P, torch, n_heads):
    """qlinear_kv_*_heads (every KV head of a layer in one launch, value scales folded inside the decode kernel) against
    the per-head calls: the same cache bytes and scales, the same score and output bits; and the output against the
    oracle.  11 heads: more than one launch's worth."""
    T, R = 1031, GROUP
    ks, vs, qs = [], [], []
    for h in range(n_heads):
        k, v = tensors(1200 + h, T)
        ks.append(k); vs.append(v); qs.append(gen.normal_fp16(1200 + h, 3, (R, DH)))
    k_all, v_all, q_all = (torch.from_numpy(np.stack(a)).cuda() for a in (ks, vs, qs))
    heads = P.KVHeads(n_heads, CACHE, DH)
    heads.append(k_all[:, :1024].contiguous(), v_all[:, :1024].contiguous())        # prefill
    for t in range(1024, T):                                                        # decode steps, strided input
        heads.append_raw(k_all[:, t].data_ptr(), v_all[:, t].data_ptr(), T * DH, DH, 1)
    singles = [P.KVCache(CACHE, DH) for _ in range(n_heads)]
    for h, c in enumerate(singles):
        c.append(k_all[h], v_all[h])
    torch.cuda.synchronize()
    assert heads.length == T
    for h in range(n_heads):
        assert torch.equal(heads.heads[h].k.packed, singles[h].k.packed)
        assert torch.equal(heads.heads[h].v.packed, singles[h].v.packed)
        assert torch.equal(heads.heads[h].v_scale, singles[h].v_scale)
    sc = heads.scores(q_all)
    z = sc[:, :, :T].double() / np.sqrt(DH)
    prob = torch.zeros((n_heads, R, CACHE), dtype=torch.float16, device="cuda")
    prob[:, :, :T] = torch.softmax(z, dim=2).half()
    out = heads.output(prob)
    torch.cuda.synchronize()
    assert heads.heads[0].k.device_status() == (0, 0)
    for h in range(n_heads):
        assert torch.equal(sc[h], singles[h].scores(q_all[h]))
        # the product with the scales as a pass of its own (one rounding to fp16), then the plain layer
        folded = (prob[h].float() * singles[h].v_scale.float()[None, :]).half()
        assert torch.equal(out[h], singles[h].v.forward(folded))
        assert torch.equal(out[h], singles[h].output(prob[h]))
        _, _, out64, A_out = O.kv_attention(qs[h], ks[h], vs[h], prob[h, :, :T].cpu().numpy())
        ok, rel, worst = O.check_against(out[h].cpu().numpy(), out64, A_out)
        assert ok, ("output", h, rel, worst)


def test_heads_argument_errors(P, torch):
    heads = P.KVHeads(2, 256, 64)
    big = torch.zeros((2, 9, 256), dtype=torch.float16, device="cuda")
    with pytest.raises(P.QLinearError):
        heads.output(big)                               # 9 query rows: not a decode-sized product
    with pytest.raises(P.QLinearError):
        heads.append(torch.zeros((3, 1, 64), dtype=torch.float16, device="cuda"), torch.zeros((3, 1, 64), dtype=torch.float16, device="cuda"))


@pytest.mark.parametrize("d_h,cache,n_heads,R", [(128, 10240, 8, 4), (64, 20000 // 32 * 32, 8, 1), (256, 9632, 8, 8), (128, 25632, 3, 5)],
                         ids=["dh128", "dh64-one-row", "dh256-eight-rows", "three-heads-ragged"])
def test_scores_over_a_long_cache_match_the_per_head_calls(P, torch, d_h, cache, n_heads, R):
    """More than one wave of row super-blocks: the score product of all heads runs on the persistent short-K kernel
    (a CTA walks over super-blocks, the next one's bytes in flight).  Same bits as the per-head calls of the ordinary
    decode kernel; cache lengths that are not a multiple of 128; positions beyond the filled part score 0."""
    T = cache - 777
    rng = np.random.default_rng(d_h + cache)
    k = (rng.standard_normal((n_heads, T, d_h)) * rng.uniform(0.2, 3.0, size=(n_heads, T, 1))).astype(np.float16)
    q = rng.standard_normal((n_heads, R, d_h)).astype(np.float16)
    kd, qd = torch.from_numpy(k).cuda(), torch.from_numpy(q).cuda()
    heads = P.KVHeads(n_heads, cache, d_h)
    heads.append(kd, kd)
    sc = heads.scores(qd)
    torch.cuda.synchronize()
    assert heads.heads[0].k.device_status() == (0, 0)
    assert (sc[:, :, T:] == 0).all()
    for h in range(n_heads):
        if d_h <= 128:                                  # (at d_h = 256 the per-head call splits K: another order of sums)
            assert torch.equal(sc[h], heads.heads[h].scores(qd[h]))
        k_q, k_s = O.kv_quantize_rows(k[h])
        y64, A, _ = O.linear(q[h], k_q, k_s.reshape(-1, 1), 0)
        ok, rel, worst = O.check_against(sc[h, :, :T].cpu().numpy(), y64, A)
        assert ok, (h, rel, worst)


def test_small_launches_are_planned_without_clusters(P, torch):
    """A cluster launch with its cluster-wide barriers costs about a microsecond: launches of a few MB (the V-cache
    product at the protocol length) are planned without one, large layers with a long K still take clusters."""
    import ctypes

    def plan(lin, M):
        out = (ctypes.c_int32 * 8)()
        assert P.lib.qlinear_debug_plan(lin._h, M, out, 8) == 8
        return {"grid": out[1], "cl": out[2], "ks_cta": out[3], "cps": out[4]}
    v = P.KVCache(CACHE, DH).v                           # N = 128, K = 1280: 164 KB
    assert plan(v, 4)["cl"] == 1
    big = P.QLinear(P.Desc(4096, 14336, 8, 0), torch.zeros(P.qlinear_packed_size(P.Desc(4096, 14336, 8, 0)), dtype=torch.uint8, device="cuda"))
    assert plan(big, 1)["cl"] > 1
