"""Pins for the oracle's cumulative attention score (Eq. 4): closed forms, invariants, brute force."""
import math
import os

import numpy as np
import pytest

from oracle import lookm_oracle as orc
from paper_2406_18139_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(shape, key, scale=1.0):
    x = synth.normal(synth.stream_key(*key), int(np.prod(shape))).reshape(shape) * scale
    return synth.bf16_to_f32(synth.f32_to_bf16_bits(x.astype(np.float32)))


def brute_scores(q, k, scale, group):
    """Materialise every causal softmax matrix and sum its columns (numpy, float64)."""
    L, Hq, d = q.shape
    Hkv = k.shape[1]
    out = np.zeros((Hkv, L))
    for hq in range(Hq):
        h = hq // group
        S = (q[:, hq].astype(np.float64) @ k[:, h].astype(np.float64).T) * scale
        S = np.where(np.tril(np.ones((L, L), dtype=bool)), S, -np.inf)
        P = np.exp(S - S.max(axis=1, keepdims=True))
        P /= P.sum(axis=1, keepdims=True)
        out[h] += P.sum(axis=0)
    return out


def test_uniform_attention_matches_harmonic_golden():
    vals = [l for l in open(os.path.join(GOLDEN, "uniform_attention_8.txt")) if not l.startswith("#")]
    expect = np.array([float(t) for t in vals[0].split()])
    q = np.zeros((8, 1, 4), dtype=np.float32)
    k = _rand((8, 1, 4), (1, 1))
    got = orc.scores(q, k)[0]
    assert np.allclose(got, expect, atol=5e-8)
    assert abs(got.sum() - 8.0) < 1e-12


@pytest.mark.parametrize("L", [1, 2, 17, 300])
def test_uniform_attention_closed_form_any_length(L):
    H = np.concatenate([[0.0], np.cumsum(1.0 / np.arange(1, L + 1))])
    q = np.zeros((L, 2, 8), dtype=np.float32)
    k = _rand((L, 1, 8), (2, L))
    got = orc.scores(q, k)[0]                       # two query heads share the KV head
    assert np.allclose(got, 2.0 * (H[L] - H[:L]), rtol=1e-13, atol=1e-13)


def test_two_token_sigmoid_closed_form():
    q = _rand((2, 1, 16), (3, 1))
    k = _rand((2, 1, 16), (3, 2))
    scale = 0.37
    s10 = float(q[1, 0].astype(np.float64) @ k[0, 0].astype(np.float64)) * scale
    s11 = float(q[1, 0].astype(np.float64) @ k[1, 0].astype(np.float64)) * scale
    sig = 1.0 / (1.0 + math.exp(-(s10 - s11)))
    got = orc.scores(q, k, scale=scale)[0]
    assert np.allclose(got, [1.0 + sig, 1.0 - sig], rtol=1e-14)


def test_hand_case_against_materialised_softmax():
    rows = {l.split()[0]: [float(t) for t in l.split()[1:]]
            for l in open(os.path.join(GOLDEN, "hand_case_8x2.txt")) if not l.startswith("#")}
    q = np.array(rows["q"], dtype=np.float32).reshape(8, 1, 2)
    k = np.array(rows["k"], dtype=np.float32).reshape(8, 1, 2)
    got = orc.scores(q, k, scale=1.0)[0]
    expect = brute_scores(q, k, 1.0, 1)[0]
    assert np.allclose(got, expect, rtol=1e-13)
    # the last key is seen by the last row only: softmax weight of logit q7.k7 = -4 in row 7
    logits7 = (q[7, 0].astype(np.float64) @ k[:, 0].astype(np.float64).T)
    assert math.isclose(got[7], math.exp(logits7[7]) / np.exp(logits7).sum(), rel_tol=1e-13)
    # swapping the operands must change the answer (guards a transposed contraction)
    assert not np.allclose(orc.scores(k, q, scale=1.0)[0], expect, rtol=1e-3)


@pytest.mark.parametrize("L,Hq,Hkv,d", [(37, 2, 2, 16), (130, 4, 2, 32), (64, 6, 2, 8)])
def test_random_against_materialised_softmax_and_invariants(L, Hq, Hkv, d):
    q = _rand((L, Hq, d), (4, L, 1), 1.5)
    k = _rand((L, Hkv, d), (4, L, 2), 1.5)
    G = Hq // Hkv
    got, lse = orc.scores(q, k, want_lse=True)
    expect = brute_scores(q, k, 1.0 / math.sqrt(d), G)
    assert np.allclose(got, expect, rtol=1e-12)
    assert np.allclose(got.sum(axis=1), G * L, rtol=1e-13)          # every row sums to one
    assert np.all(got[:, 0] >= G - 1e-12) and np.all(got[:, -1] <= G + 1e-12)
    assert np.all(got > 0)
    # log-sum-exp against scipy-free direct evaluation
    for h in range(Hkv):
        for g in range(G):
            S = (q[:, h * G + g].astype(np.float64) @ k[:, h].astype(np.float64).T) / math.sqrt(d)
            for i in (0, L // 2, L - 1):
                assert math.isclose(lse[h, g, i], math.log(np.exp(S[i, :i + 1]).sum()), rel_tol=1e-12)
    rows = np.array([0, 3, L - 1], dtype=np.int32)
    assert np.allclose(orc.lse_rows(q, k, Hq - 1, Hkv - 1, rows), lse[Hkv - 1, G - 1, rows], rtol=1e-14)


def test_scale_default_is_inverse_sqrt_head_dim_and_threads_agree():
    q = _rand((50, 4, 64), (5, 1))
    k = _rand((50, 4, 64), (5, 2))
    a = orc.scores(q, k)
    b = orc.scores(q, k, scale=0.125, threads=4)
    assert np.array_equal(a, b)
    assert not np.allclose(a, orc.scores(q, k, scale=1.0))


def test_tail_keys_only():
    q = _rand((90, 2, 16), (6, 1))
    k = _rand((90, 1, 16), (6, 2))
    full = orc.scores(q, k)
    tail = orc.scores(q, k, key_begin=70)
    assert np.all(np.isnan(tail[:, :70]))
    assert np.allclose(tail[:, 70:], full[:, 70:], rtol=1e-14)


def test_kv_head_subset():
    q = _rand((40, 4, 16), (7, 1))
    k = _rand((40, 4, 16), (7, 2))
    full = orc.scores(q, k)
    assert np.array_equal(orc.scores(q, k, kv_heads=[3, 1]), full[[3, 1]])
