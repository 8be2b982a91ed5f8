"""Pins for the oracle's selection (Eq. 5-8), matching (Eq. 9) and merging (Eq. 10-12)."""
import numpy as np
import pytest

from oracle import lookm_oracle as orc
from paper_2406_18139_b200 import synth


def _rand(shape, key, scale=1.0):
    x = synth.normal(synth.stream_key(*key), int(np.prod(shape))).reshape(shape) * scale
    return synth.bf16_to_f32(synth.f32_to_bf16_bits(x.astype(np.float32)))


# ------------------------------------------------------------------ selection ---------------

def brute_select(scores, mask, B, M):
    """Literal Eq. 5 + Eq. 8: add max(A_s) to text scores, stable sort, take N, append window."""
    L = len(scores)
    B = min(B, L)
    M = min(M, B)
    boosted = np.array(scores, dtype=np.float64)
    boosted[np.asarray(mask) == 0] += boosted.max() * 4.0 + 1.0   # any boost >= max gives the same order
    cand = list(range(L - M))
    cand.sort(key=lambda j: (-boosted[j], j))
    keep = sorted(cand[:B - M]) + list(range(L - M, L))
    ev = [j for j in range(L) if j not in set(keep)]
    return np.array(keep, dtype=np.int32), np.array(ev, dtype=np.int32)


@pytest.mark.parametrize("L,B,M,n_img", [(40, 12, 4, 25), (40, 12, 4, 38), (64, 20, 0, 30),
                                         (33, 33, 5, 10), (20, 50, 3, 10), (16, 4, 9, 8)])
def test_select_against_literal_boost_and_sort(L, B, M, n_img):
    s = np.abs(synth.normal(synth.stream_key(11, L, B), L)) + 1e-3
    mask = np.zeros(L, dtype=np.uint8)
    mask[synth.uniform_int(synth.stream_key(12, L), n_img, 0, L - 1).astype(int)] = 1
    kept, ev = orc.select(s, mask, B, M)
    bk, be = brute_select(s, mask, B, M)
    assert np.array_equal(kept, bk) and np.array_equal(ev, be)
    Bc, Mc = min(B, L), min(M, min(B, L))
    assert len(kept) == Bc and len(ev) == L - Bc                      # S = N + M exactly
    assert np.array_equal(kept[Bc - Mc:], np.arange(L - Mc, L))        # window at the tail
    assert np.all(np.diff(kept) > 0) and np.all(np.diff(ev) > 0)
    assert sorted(np.concatenate([kept, ev]).tolist()) == list(range(L))
    text_cand = [j for j in range(L - Mc) if mask[j] == 0]
    if len(text_cand) <= Bc - Mc:
        assert set(text_cand) <= set(kept.tolist())                    # every text token survives
    else:
        sel = set(kept[:Bc - Mc].tolist())
        assert all(mask[j] == 0 for j in sel)                          # no image token is kept
        worst_kept = min((s[j] for j in sel), default=np.inf)
        assert all(s[j] <= worst_kept for j in text_cand if j not in sel)


def test_select_ties_prefer_lower_position_and_budget_is_monotone():
    L, M = 30, 3
    s = np.ones(L)
    s[[5, 9, 20]] = 2.0
    mask = np.ones(L, dtype=np.uint8)
    mask[[7, 8]] = 0
    kept, _ = orc.select(s, mask, 10, M)
    # 2 text, then the three 2.0 scores, then the lowest-position 1.0 scores
    assert kept.tolist() == [0, 1, 5, 7, 8, 9, 20, 27, 28, 29]
    prev = set(orc.select(s, mask, 4, M)[0].tolist())
    for B in range(5, L + 1):
        cur = set(orc.select(s, mask, B, M)[0].tolist())
        assert prev < cur and len(cur) == len(prev) + 1
        prev = cur


def test_select_text_ordered_by_score_when_text_exceeds_budget():
    s = np.array([5.0, 1.0, 9.0, 2.0, 7.0, 3.0, 8.0, 4.0])
    mask = np.array([1, 0, 1, 0, 0, 0, 1, 0], dtype=np.uint8)
    kept, ev = orc.select(s, mask, 3, 1)
    assert kept.tolist() == [4, 5, 7]          # text 7.0 and 3.0 win over text 2.0, 1.0; window = 7
    assert ev.tolist() == [0, 1, 2, 3, 6]


# ------------------------------------------------------------------ matching ----------------

def test_match_against_numpy_cosine_matrix():
    k = _rand((60, 2, 16), (21, 1))
    kept = np.array([1, 4, 9, 17, 30, 58, 59], dtype=np.int32)
    ev = np.array([j for j in range(60) if j not in set(kept.tolist())], dtype=np.int32)
    for h in range(2):
        x = k[:, h].astype(np.float64)
        xn = x / np.linalg.norm(x, axis=1, keepdims=True)
        S = xn[ev] @ xn[kept].T
        assign, sim, Sm = orc.match(k, h, kept, ev, want_matrix=True)
        assert np.allclose(Sm, S, rtol=1e-13, atol=1e-15)
        assert np.array_equal(assign, S.argmax(axis=1))
        assert np.allclose(sim, S.max(axis=1), rtol=1e-13)
        a2, s2 = orc.argmax_rows(Sm)
        assert np.array_equal(a2, assign) and np.array_equal(s2, sim)


def test_match_special_cases():
    d = 8
    k = np.zeros((7, 1, d), dtype=np.float32)
    k[0, 0, 0] = 2.0                      # kept slot 0: +e0 scaled
    k[1, 0, 1] = -0.5                     # kept slot 1: -e1 scaled
    k[2, 0, 2] = 4.0                      # kept slot 2: +e2 scaled
    k[3, 0] = [1, -7, 3, 0, 0, 0, 0, 0]   # largest |coordinate| with matching sign: -e1 -> slot 1
    k[4, 0] = 3.0 * k[2, 0]               # positive multiple of kept slot 2 -> sim 1
    k[5, 0] = k[0, 0]                     # kept slot 3 duplicates slot 0
    k[6, 0] = [5, 0, 0, 0, 0, 0, 0, 0]    # ties between slots 0 and 3 -> lower slot
    kept = np.array([0, 1, 2, 5], dtype=np.int32)
    ev = np.array([3, 4, 6], dtype=np.int32)
    assign, sim = orc.match(k, 0, kept, ev)
    assert assign.tolist() == [1, 2, 0]
    assert np.isclose(sim[0], 7 / np.sqrt(59)) and sim[1] == 1.0 and sim[2] == 1.0
    k2 = k.copy()
    k2[ev] *= np.float32(4.0)             # scale invariance of the evicted side (power of two: exact)
    a2, s2 = orc.match(k2, 0, kept, ev)
    assert np.array_equal(a2, assign) and np.allclose(s2, sim, rtol=1e-15)
    k3 = k.copy()
    k3[4, 0] = 0.0                        # zero-norm key: similarity 0 with everything, slot 0
    a3, s3 = orc.match(k3, 0, kept, ev)
    assert a3[1] == 0 and s3[1] == 0.0


def test_argmax_rows_ties_and_negative_rows():
    S = np.array([[0.1, 0.7, 0.7, -1.0], [-0.3, -0.2, -0.2, -0.9], [0.0, 0.0, 0.0, 0.0]])
    a, s = orc.argmax_rows(S)
    assert a.tolist() == [1, 1, 0] and s.tolist() == [0.7, -0.2, 0.0]


# ------------------------------------------------------------------ merging -----------------

@pytest.mark.parametrize("mode", [0, 1, 2])
def test_merge_single_kept_token_closed_forms(mode):
    L, d = 9, 6
    x = _rand((L, 1, d), (31, mode))
    kept = np.array([L - 1], dtype=np.int32)
    ev = np.arange(L - 1, dtype=np.int32)
    assign = np.zeros(L - 1, dtype=np.int32)
    sim = np.linspace(-0.5, 0.9, L - 1)
    out = orc.merge(x, 0, kept, ev, assign, sim, mode)[0]
    X = x[:, 0].astype(np.float64)
    n = L - 1
    if mode == 0:
        expect = X.mean(axis=0)                                        # mean of all L rows
    elif mode == 1:
        expect = ((1 + n / 2) * X[-1] + 0.5 * X[:-1].sum(axis=0)) / (n + 1)
    else:
        expect = (X[-1] + (sim[:, None] * X[:-1]).sum(axis=0)) / (n + 1)
    assert np.allclose(out, expect, rtol=1e-14, atol=1e-15)


def test_merge_duplicates_passthrough_and_sum_preservation():
    L, d = 40, 8
    x = _rand((L, 2, d), (32, 1))
    kept = np.array([2, 5, 11, 30, 38, 39], dtype=np.int32)
    ev = np.array([j for j in range(L) if j not in set(kept.tolist())], dtype=np.int32)
    assign = (synth.uniform_int(synth.stream_key(33), len(ev), 0, 4)).astype(np.int32)   # slot 5 gets none
    sim = np.ones(len(ev))
    X = x[:, 1].astype(np.float64)
    avg = orc.merge(x, 1, kept, ev, assign, sim, 0)
    counts = np.bincount(assign, minlength=len(kept))
    assert counts.sum() + len(kept) == L
    assert np.allclose(((counts + 1)[:, None] * avg).sum(axis=0), X.sum(axis=0), rtol=1e-13)
    assert np.array_equal(avg[5], X[39])                                # no members: untouched
    assert np.allclose(orc.merge(x, 1, kept, ev, assign, sim, 2), avg, rtol=1e-15)   # sim = 1
    # every member equal to its kept row: all three modes return the kept row
    xd = x.copy()
    xd[ev, 1] = xd[kept[assign], 1]
    for mode in (0, 1, 2):
        out = orc.merge(xd, 1, kept, ev, assign, sim, mode)
        assert np.allclose(out, xd[kept, 1].astype(np.float64), rtol=1e-14)
    # pivotal = midpoint between the kept row and the averaged result's member mean
    piv = orc.merge(x, 1, kept, ev, assign, sim, 1)
    for c in range(len(kept)):
        mem = X[ev[assign == c]]
        n = len(mem)
        assert np.allclose(piv[c], (X[kept[c]] + 0.5 * (mem + X[kept[c]]).sum(axis=0)) / (n + 1), rtol=1e-14)
    # weighted with signed weights, literal Eq. 12
    w = np.linspace(-1, 1, len(ev))
    wm = orc.merge(x, 1, kept, ev, assign, w, 2)
    for c in range(len(kept)):
        idx = np.where(assign == c)[0]
        assert np.allclose(wm[c], (X[kept[c]] + (w[idx, None] * X[ev[idx]]).sum(axis=0)) / (len(idx) + 1),
                           rtol=1e-14, atol=1e-15)


# ------------------------------------------------------------------ whole path --------------

def test_compress_layer_composition_and_edges():
    w = synth.tiny(96, 4, 2, 24, 6, 1, image_spans=[(10, 50), (60, 85)], seed=3, head_dim=16)
    q, k, v = (synth.bf16_to_f32(t) for t in synth.layer_tensors(w))
    req = w.requests[0]
    res = orc.compress_layer(q, k, v, req.mask, req.budget, req.window, req.merge_mode, threads=2)
    assert res["out_len"] == 24
    for i, h in enumerate(res["kv_heads"]):
        kept, ev = res["kept"][i], res["evicted"][i]
        assert len(kept) == 24 and len(ev) == 72
        assert np.array_equal(kept[-6:], np.arange(90, 96))
        a, s = orc.match(k, h, kept, ev)
        assert np.array_equal(a, res["assign"][i])
        assert np.allclose(res["out_v"][i], orc.merge(v, h, kept, ev, a, s, 1))
    # budget >= length: a straight copy
    res = orc.compress_layer(q, k, v, req.mask, 200, req.window, 0)
    assert res["out_len"] == 96
    assert np.array_equal(res["out_k"][1], k[:, 1].astype(np.float64))
    # window >= budget: only the last `budget` tokens are kept
    res = orc.compress_layer(q, k, v, req.mask, 10, 64, 0)
    assert np.array_equal(res["kept"][0], np.arange(86, 96))
    # packed batch = each request on its own
    cu = [0, 40, 96]
    outs = orc.compress_varlen(q, k, v, req.mask, cu, [8, 12], [2, 3], [0, 2])
    solo = orc.compress_layer(q[40:], k[40:], v[40:], req.mask[40:], 12, 3, 2)
    assert np.array_equal(outs[1]["out_k"][0], solo["out_k"][0])
