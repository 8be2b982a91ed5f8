"""Pins for the oracle's variants (selection without the text prior, eviction without merging) and
for its generation step over a cache (Section 3.1, Eq. 2-3)."""
import os

import numpy as np
import pytest

from oracle import lookm_oracle as orc
from paper_2406_18139_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(shape, key, scale=1.0):
    x = synth.normal(synth.stream_key(*key), int(np.prod(shape))).reshape(shape) * scale
    return synth.bf16_to_f32(synth.f32_to_bf16_bits(x.astype(np.float32)))


# ------------------------------------------------------------------ selection without Eq. 5 --

@pytest.mark.parametrize("L,B,M", [(40, 12, 4), (64, 20, 0), (33, 33, 5), (20, 50, 3), (16, 4, 9), (50, 1, 0)])
def test_select_without_text_prior_is_a_plain_sort_by_score(L, B, M):
    s = np.abs(synth.normal(synth.stream_key(51, L, B), L)) + 1e-3
    mask = (synth.uniform_int(synth.stream_key(52, L), L, 0, 1)).astype(np.uint8)
    kept, ev = orc.select(s, mask, B, M, text_prior=False)
    Bc = min(B, L)
    Mc = min(M, Bc)
    cand = sorted(range(L - Mc), key=lambda j: (-s[j], j))[:Bc - Mc]       # Eq. 8 on the raw scores
    want = sorted(cand) + list(range(L - Mc, L))
    assert kept.tolist() == want
    assert ev.tolist() == [j for j in range(L) if j not in set(want)]
    # the mask plays no part: any other mask gives the same lists
    k2, e2 = orc.select(s, 1 - mask, B, M, text_prior=False)
    assert np.array_equal(k2, kept) and np.array_equal(e2, ev)
    # and it equals the text-prior selection of a prompt without any text (or with text only)
    for uniform in (np.ones(L, dtype=np.uint8), np.zeros(L, dtype=np.uint8)):
        k3, _ = orc.select(s, uniform, B, M, text_prior=True)
        assert np.array_equal(k3, kept)


def test_select_without_text_prior_differs_where_the_prior_matters():
    s = np.array([5.0, 1.0, 9.0, 2.0, 7.0, 3.0, 8.0, 4.0])
    mask = np.array([1, 0, 1, 0, 1, 0, 1, 0], dtype=np.uint8)
    assert orc.select(s, mask, 4, 1, text_prior=True)[0].tolist() == [1, 3, 5, 7]    # text first
    assert orc.select(s, mask, 4, 1, text_prior=False)[0].tolist() == [2, 4, 6, 7]   # best scores
    ties = np.ones(8)
    assert orc.select(ties, mask, 4, 1, text_prior=False)[0].tolist() == [0, 1, 2, 7]  # lower position


# ------------------------------------------------------------------ eviction without merging --

def test_merge_mode_none_returns_the_kept_rows_whatever_the_lists_say():
    L, d = 30, 8
    x = _rand((L, 2, d), (53, 1))
    kept = np.array([0, 4, 9, 28, 29], dtype=np.int32)
    ev = np.array([j for j in range(L) if j not in set(kept.tolist())], dtype=np.int32)
    assign = (synth.uniform_int(synth.stream_key(54), len(ev), 0, 4)).astype(np.int32)
    sim = np.linspace(-1, 1, len(ev))
    for h in range(2):
        out = orc.merge(x, h, kept, ev, assign, sim, orc.MERGE_NONE)
        assert np.array_equal(out, x[kept, h].astype(np.float64))
        out = orc.merge(x, h, kept, ev[:0], assign[:0], sim[:0], orc.MERGE_NONE)
        assert np.array_equal(out, x[kept, h].astype(np.float64))


def test_compress_layer_evict_only_and_without_prior():
    w = synth.tiny(96, 4, 2, 24, 6, 3, image_spans=[(10, 50), (60, 85)], seed=5, head_dim=16)
    q, k, v = (synth.bf16_to_f32(t) for t in synth.layer_tensors(w))
    req = w.requests[0]
    full = orc.compress_layer(q, k, v, req.mask, 24, 6, orc.MERGE_AVERAGE)
    none = orc.compress_layer(q, k, v, req.mask, 24, 6, orc.MERGE_NONE)
    for i in range(2):
        assert np.array_equal(none["kept"][i], full["kept"][i])          # same selection
        assert np.array_equal(none["out_k"][i], k[none["kept"][i], i].astype(np.float64))
        assert np.array_equal(none["out_v"][i], v[none["kept"][i], i].astype(np.float64))
        assert len(none["assign"][i]) == 0
    plain = orc.compress_layer(q, k, v, req.mask, 24, 6, orc.MERGE_AVERAGE, text_prior=False)
    for i in range(2):
        A = plain["scores"][i]
        best = sorted(sorted(range(90), key=lambda j: (-A[j], j))[:18])
        assert plain["kept"][i].tolist() == best + list(range(90, 96))
    assert any(not np.array_equal(plain["kept"][i], full["kept"][i]) for i in range(2))


# ------------------------------------------------------------------ generation step ----------

def brute_decode(q, ck, cv, scale):
    Hq, Hkv = q.shape[0], ck.shape[0]
    G = Hq // Hkv
    out = np.zeros((Hq, q.shape[1]))
    for hq in range(Hq):
        K, V = ck[hq // G].astype(np.float64), cv[hq // G].astype(np.float64)
        s = (K @ q[hq].astype(np.float64)) * scale
        p = np.exp(s - s.max())
        out[hq] = (p / p.sum()) @ V
    return out


def test_decode_hand_case_golden():
    vals = [l for l in open(os.path.join(GOLDEN, "decode_hand_case_3.txt")) if not l.startswith("#")]
    expect = np.array([float(t) for t in vals[0].split()])
    q = np.array([[1.0, 0.0]], dtype=np.float32)
    ck = np.array([[[0.0, 5.0], [1.0, -3.0]]], dtype=np.float32)
    cv = np.array([[[1.0, 0.0], [0.0, 1.0]]], dtype=np.float32)
    out, ck2, cv2 = orc.decode_step(q, np.array([[2.0, 7.0]]), np.array([[1.0, 1.0]]), ck, cv, scale=1.0)
    assert np.allclose(out[0], expect, atol=5e-8)
    assert ck2.shape == (1, 3, 2) and ck2[0, 2].tolist() == [2.0, 7.0] and cv2[0, 2].tolist() == [1.0, 1.0]
    assert np.array_equal(ck2[:, :2], ck) and np.array_equal(cv2[:, :2], cv)
    # swapping K and V roles, or leaving the new row out, must change the result
    wrong, _, _ = orc.decode_step(q, np.array([[1.0, 1.0]]), np.array([[2.0, 7.0]]), cv, ck, scale=1.0)
    assert not np.allclose(wrong[0], expect, atol=1e-3)


def test_decode_uniform_mean_shift_invariance_and_one_hot():
    n, d, Hq, Hkv = 37, 16, 4, 2
    ck, cv = _rand((Hkv, n, d), (61, 1)), _rand((Hkv, n, d), (61, 2))
    kn, vn = _rand((Hkv, d), (61, 3)), _rand((Hkv, d), (61, 4))
    # q = 0: uniform weights -> the mean of the n + 1 value rows of the head's KV head
    out, _, cv2 = orc.decode_step(np.zeros((Hq, d), dtype=np.float32), kn, vn, ck, cv)
    for hq in range(Hq):
        assert np.allclose(out[hq], cv2[hq // 2].astype(np.float64).mean(axis=0), rtol=1e-13, atol=1e-15)
    # adding the same vector u to every key shifts every logit by q.u: the output does not move
    q = _rand((Hq, d), (61, 5))
    base, _, _ = orc.decode_step(q, kn, vn, ck, cv)
    u = np.float32(0.5) * np.ones(d, dtype=np.float32)
    moved, _, _ = orc.decode_step(q, kn + u, vn, ck + u, cv)
    assert np.allclose(moved, base, rtol=1e-9, atol=1e-12)
    # one key aligned with q and very long: the output is that row's value
    big = ck.copy()
    big[0, 11] = 64.0 * q[0]
    hot, _, _ = orc.decode_step(q, kn, vn, big, cv)
    assert np.allclose(hot[0], cv[0, 11].astype(np.float64), atol=1e-9)
    # a cache that was empty before the step: the output is the new value row
    solo, _, _ = orc.decode_step(q, kn, vn, ck[:, :0], cv[:, :0])
    assert np.allclose(solo, np.repeat(vn.astype(np.float64), 2, axis=0), rtol=1e-14)


@pytest.mark.parametrize("n,Hq,Hkv,d", [(1, 1, 1, 4), (50, 8, 2, 32), (333, 4, 4, 128)])
def test_decode_against_numpy_brute_force(n, Hq, Hkv, d):
    ck, cv = _rand((Hkv, n, d), (62, n, 1)), _rand((Hkv, n, d), (62, n, 2))
    kn, vn, q = _rand((Hkv, d), (62, n, 3)), _rand((Hkv, d), (62, n, 4)), _rand((Hq, d), (62, n, 5))
    for scale in (None, 0.21):
        out, ck2, cv2 = orc.decode_step(q, kn, vn, ck, cv, scale=scale)
        ref = brute_decode(q, ck2, cv2, (1.0 / np.sqrt(d)) if scale is None else scale)
        assert np.allclose(out, ref, rtol=1e-12, atol=1e-14)
