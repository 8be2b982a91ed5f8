"""The generation step over a cache (Section 3.1, Eq. 2-3) through the C ABI against the fp64 oracle.

Tolerance: the kernel multiplies bf16 values exactly in fp32, accumulates in fp32 and takes
exponentials with ex2.approx (2 ulp), so every output element carries a few 1e-7 of the sum of
|p_j v_j|; the tests assert |got - ref| <= 1e-3 |ref| + 1e-5 (values are O(1)).  The appended cache
row must equal the new token's row bit for bit and no other cache element may change.
"""
import numpy as np
import pytest

from oracle import lookm_oracle as orc
from paper_2406_18139_b200 import synth
from tests.helpers import to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2406_18139_b200 import binding
    binding.lib()
    return binding


def _bits(shape, key, scale=1.0):
    x = synth.normal(synth.stream_key(*key), int(np.prod(shape))).reshape(shape) * scale
    return synth.f32_to_bf16_bits(x.astype(np.float32))


def close(got, ref):
    return np.abs(got - ref) <= 1e-3 * np.abs(ref) + 1e-5


def run_step(B, Hq, Hkv, n, cap, packed, seed, scale=0.0, q_scale=1.0):
    """One request: cache of n rows in a buffer with room for `cap`; returns nothing, asserts."""
    import torch
    ck_b, cv_b = _bits((Hkv, cap, 128), (seed, 1)), _bits((Hkv, cap, 128), (seed, 2))
    q_b, kn_b, vn_b = _bits((Hq, 128), (seed, 3), q_scale), _bits((Hkv, 128), (seed, 4)), _bits((Hkv, 128), (seed, 5))
    if packed:                                            # [rows, Hkv, 128]
        dk, dv = to_dev(ck_b.transpose(1, 0, 2).copy()), to_dev(cv_b.transpose(1, 0, 2).copy())
        lay = B.CacheLayout(Hq, Hkv, 128, Hkv * 128, 128, scale)
    else:                                                 # [Hkv, cap, 128]
        dk, dv = to_dev(ck_b), to_dev(cv_b)
        lay = B.CacheLayout(Hq, Hkv, 128, 128, cap * 128, scale)
    q, kn, vn = to_dev(q_b), to_dev(kn_b), to_dev(vn_b)
    out = torch.full((Hq, 128), np.nan, dtype=torch.float32, device="cuda")
    ws = B.alloc_decode_workspace(lay)
    before_k, before_v = dk.clone(), dv.clone()
    B.check(B.lookm_decode_step(q, kn, vn, dk, dv, n, lay, out, ws))
    torch.cuda.synchronize()
    f = synth.bf16_to_f32
    ref, _, _ = orc.decode_step(f(q_b), f(kn_b), f(vn_b), f(ck_b)[:, :n], f(cv_b)[:, :n],
                                scale=None if scale == 0.0 else scale)
    got = out.cpu().numpy().astype(np.float64)
    assert close(got, ref).all(), float(np.abs(got - ref).max())
    # Eq. 2: row n now holds the new token's rows; everything else is as before
    view = (lambda t: t.transpose(0, 1)) if packed else (lambda t: t)
    assert torch.equal(view(dk)[:, n], kn) and torch.equal(view(dv)[:, n], vn)
    keep = torch.ones(cap, dtype=torch.bool, device="cuda")
    keep[n] = False
    assert torch.equal(view(dk)[:, keep], view(before_k)[:, keep])
    assert torch.equal(view(dv)[:, keep], view(before_v)[:, keep])
    # a second identical step on the same state gives the same bits (fixed order of additions)
    out2 = torch.zeros_like(out)
    B.check(B.lookm_decode_step(q, kn, vn, dk, dv, n, lay, out2, ws))
    torch.cuda.synchronize()
    assert torch.equal(out, out2)


@pytest.mark.parametrize("Hq,Hkv,n,packed", [(1, 1, 0, False), (1, 1, 1, True), (4, 2, 17, False),
                                             (4, 4, 63, True), (8, 1, 64, False), (32, 8, 65, True),
                                             (6, 2, 200, False), (32, 32, 1000, False), (16, 1, 777, True)])
def test_one_step_small_caches(B, Hq, Hkv, n, packed):
    run_step(B, Hq, Hkv, n, n + 3, packed, seed=600 + n)


def test_long_cache_is_cut_into_many_splits(B):
    # 2 KV heads x 20001 rows: about 150 splits per head, combined by the last CTA to arrive
    run_step(B, 8, 2, 20000, 20001, False, seed=701)
    run_step(B, 2, 2, 5000, 5002, True, seed=702, scale=0.3)


def test_peaked_softmax_and_custom_scale(B):
    # queries 6x larger: a few rows take nearly all the weight, references move along the cache
    run_step(B, 4, 2, 3000, 3001, False, seed=703, q_scale=6.0)
    run_step(B, 4, 2, 300, 301, True, seed=704, scale=1.0)


def test_batch_of_requests_with_their_own_lengths(B):
    import torch
    n_req, Hq, Hkv = 100, 4, 2                           # more requests than one launch carries
    lens = synth.uniform_int(synth.stream_key(710), n_req, 0, 400).astype(int).tolist()
    lens[3], lens[50] = 0, 2500
    caps = [n + 1 for n in lens]
    begins = np.concatenate([[0], np.cumsum(caps)])[:-1].tolist()
    rows = sum(caps)
    ck_b, cv_b = _bits((rows, Hkv, 128), (711,)), _bits((rows, Hkv, 128), (712,))
    q_b, kn_b, vn_b = _bits((n_req, Hq, 128), (713,)), _bits((n_req, Hkv, 128), (714,)), _bits((n_req, Hkv, 128), (715,))
    dk, dv, q, kn, vn = (to_dev(t) for t in (ck_b, cv_b, q_b, kn_b, vn_b))
    lay = B.CacheLayout(Hq, Hkv, 128, Hkv * 128, 128, 0.0)
    ws = B.alloc_decode_workspace(lay, n_req)
    out = torch.full((n_req, Hq, 128), np.nan, dtype=torch.float32, device="cuda")
    B.check(B.lookm_decode_step_varlen(q, kn, vn, dk, dv, begins, lens, lay, out, ws))
    torch.cuda.synchronize()
    # two launches of at most 96 requests, each followed by one combine launch if any of its
    # requests was cut into several splits
    assert 2 <= B.lookm_last_launch_count() <= 4
    got = out.cpu().numpy().astype(np.float64)
    f = synth.bf16_to_f32
    K, V = f(ck_b), f(cv_b)
    for r in range(n_req):
        a, n = begins[r], lens[r]
        ref, ck2, _ = orc.decode_step(f(q_b[r]), f(kn_b[r]), f(vn_b[r]), K[a:a + n].transpose(1, 0, 2),
                                      V[a:a + n].transpose(1, 0, 2))
        assert close(got[r], ref).all(), r
        assert torch.equal(dk[a + n], kn[r]) and torch.equal(dv[a + n], vn[r])
    untouched = np.ones(rows, dtype=bool)
    untouched[[b + n for b, n in zip(begins, lens)]] = False
    sel = torch.from_numpy(untouched).cuda()
    assert torch.equal(dk[sel], to_dev(ck_b)[sel]) and torch.equal(dv[sel], to_dev(cv_b)[sel])


def test_compress_then_generate_three_tokens(B):
    """The path's own output as the cache.  The oracle compresses the prompt itself and its rows,
    rounded to bf16, are the cache of the oracle's three generation steps.  The GPU runs the same
    steps twice: on a copy of exactly those rows (tight tolerance: same bits in, Eq. 2-3 alone),
    and chained after its own compression into a cache with room to grow (merged rows may differ
    from the oracle's by the 2e-2 of the merge tolerance, and so may the attention output)."""
    import torch
    L, Hq, Hkv, budget, window, steps = 1500, 8, 2, 300, 32, 3
    w = synth.tiny(L, Hq, Hkv, budget, window, 2, image_spans=[(100, 700), (800, 1400)], seed=41)
    qb, kb, vb = synth.layer_tensors(w)
    f = synth.bf16_to_f32
    res = orc.compress_layer(f(qb), f(kb), f(vb), w.requests[0].mask, budget, window, 2, threads=2,
                             score_dtype=np.float32)
    ok_bits = synth.f32_to_bf16_bits(np.stack(res["out_k"]).astype(np.float32))     # [Hkv, budget, 128]
    ov_bits = synth.f32_to_bf16_bits(np.stack(res["out_v"]).astype(np.float32))
    cap = budget + steps
    clay = B.CacheLayout(Hq, Hkv, 128, 128, cap * 128, 0.0)
    dws = B.alloc_decode_workspace(clay)
    # GPU cache 1: the oracle's rows.  GPU cache 2: the GPU's own compression.
    c1k = torch.zeros(Hkv, cap, 128, dtype=torch.bfloat16, device="cuda")
    c1v = torch.zeros_like(c1k)
    c1k[:, :budget], c1v[:, :budget] = to_dev(ok_bits), to_dev(ov_bits)
    q, k, v = to_dev(qb), to_dev(kb), to_dev(vb)
    lay = B.make_layout(q, k)
    ws = B.alloc_workspace(lay, [L])
    c2k, c2v = torch.zeros_like(c1k), torch.zeros_like(c1k)
    st, out_len = B.lookm_compress_layer_opt(q, k, v, torch.from_numpy(w.requests[0].mask).cuda(), L, budget,
                                             window, 2, lay, B.make_options(out_stride_head=cap * 128),
                                             c2k, c2v, ws)
    B.check(st)
    assert out_len == budget and B.lookm_device_status(ws) == B.OK
    ref_k, ref_v = f(ok_bits), f(ov_bits)
    out1 = torch.zeros(Hq, 128, dtype=torch.float32, device="cuda")
    out2 = torch.zeros_like(out1)
    for t in range(steps):
        q_b, kn_b, vn_b = _bits((Hq, 128), (720, t, 1)), _bits((Hkv, 128), (720, t, 2)), _bits((Hkv, 128), (720, t, 3))
        dq, dkn, dvn = to_dev(q_b), to_dev(kn_b), to_dev(vn_b)
        B.check(B.lookm_decode_step(dq, dkn, dvn, c1k, c1v, budget + t, clay, out1, dws))
        B.check(B.lookm_decode_step(dq, dkn, dvn, c2k, c2v, budget + t, clay, out2, dws))
        torch.cuda.synchronize()
        ref, ref_k, ref_v = orc.decode_step(f(q_b), f(kn_b), f(vn_b), ref_k, ref_v)
        assert close(out1.cpu().numpy().astype(np.float64), ref).all(), t
        assert np.abs(out2.cpu().numpy().astype(np.float64) - ref).max() <= 2e-2, t
    assert np.array_equal(c1k.float().cpu().numpy(), ref_k) and np.array_equal(c1v.float().cpu().numpy(), ref_v)
    assert torch.equal(c2k[:, budget:], c1k[:, budget:]) and torch.equal(c2v[:, budget:], c1v[:, budget:])


@pytest.mark.parametrize("ratio", [1.0, 0.2, 0.05])
def test_7b_shape_cache_at_the_papers_three_budgets(B, ratio):
    """32 heads over a cache of 100 %, 20 % and 5 % of the 8192-token prompt (the budgets of the
    paper's speed and memory table), every head against the oracle."""
    run_step(B, 32, 32, int(ratio * 8192), int(ratio * 8192) + 8, False, seed=730 + int(100 * ratio))
