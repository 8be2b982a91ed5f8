"""Per-stage parity of the CUDA path against the fp64 oracle, through the C ABI.

Each stage is fed the ORACLE's upstream result, so index outputs must be bit-exact: both sides
take the decision on the same fp32 values.  Floating-point outputs use the stated tolerances:
scores 1e-3 relative, merged K/V 2e-2 absolute (see helpers.merged_close for large magnitudes).
"""
import numpy as np
import pytest

from oracle import lookm_oracle as orc
from paper_2406_18139_b200 import synth
from tests.helpers import bf16_to_np, merged_close, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2406_18139_b200 import binding
    binding.lib()
    return binding


def _tensors(w, layer=0):
    import torch
    qb, kb, vb, mask = synth.packed_layer_tensors(w, layer)
    dev = tuple(to_dev(t) for t in (qb, kb, vb))
    host = tuple(synth.bf16_to_f32(t) for t in (qb, kb, vb))
    return dev, host, mask, torch.from_numpy(mask).cuda()


# ------------------------------------------------------------------------------ scores -------

@pytest.mark.parametrize("L,Hq,Hkv", [(1, 1, 1), (5, 2, 1), (128, 1, 1), (129, 2, 2), (300, 4, 2),
                                      (777, 8, 2), (1500, 2, 1)])
def test_scores_and_lse_match_oracle(B, L, Hq, Hkv):
    import torch
    w = synth.tiny(L, Hq, Hkv, max(1, L // 5), 2, 0, seed=L)
    (q, k, v), (qf, kf, vf), _, _ = _tensors(w)
    lay = B.make_layout(q, k)
    ws = B.alloc_workspace(lay, [L])
    scores = torch.full((Hkv, L), -1.0, dtype=torch.float32, device="cuda")
    lse = torch.full((Hq, L), -1.0, dtype=torch.float32, device="cuda")
    B.check(B.lookm_score(q, k, [0, L], lay, scores, lse, False, ws))
    assert B.lookm_device_status(ws) == B.OK
    A, lse_o = orc.scores(qf, kf, threads=4, want_lse=True)
    got = scores.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - A) <= 1e-3 * A), float((np.abs(got - A) / A).max())
    assert np.all(np.abs(got - A) <= 2e-5 * A)                 # what fp32 accumulation should give
    assert np.allclose(lse.cpu().numpy().reshape(Hkv, Hq // Hkv, L), lse_o, atol=2e-5, rtol=0)
    assert np.allclose(got.sum(axis=1), (Hq // Hkv) * L, rtol=1e-5)
    # a caller-supplied log-sum-exp skips the first sweep and must give the same scores
    scores2 = torch.zeros_like(scores)
    B.check(B.lookm_score(q, k, [0, L], lay, scores2, lse, True, ws))
    assert torch.equal(scores, scores2)
    assert B.lookm_last_launch_count() == 3                    # table writer, lse companion, sweep 2


def test_scores_custom_scale_and_strided_heads(B):
    import torch
    L, Hq, Hkv = 260, 4, 4
    w = synth.tiny(L, Hq, Hkv, 50, 4, 0, seed=9)
    (q, k, v), (qf, kf, vf), _, _ = _tensors(w)
    # interleave Q and K in one [L, 2H, 128] buffer (a fused-projection layout)
    fused = torch.stack([q, k], dim=1).reshape(L, 2 * Hq, 128).contiguous()
    fq, fk = fused[:, :Hq], fused[:, Hq:]
    lay = B.make_layout(fq, fk, softmax_scale=0.05)
    ws = B.alloc_workspace(lay, [L])
    scores = torch.zeros(Hkv, L, dtype=torch.float32, device="cuda")
    B.check(B.lookm_score(fq, fk, [0, L], lay, scores, None, False, ws))
    A = orc.scores(qf, kf, scale=0.05, threads=4)
    got = scores.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - A) <= 2e-5 * A)


def test_scores_logits_that_grow_along_the_prompt(B):
    """Logits that rise by far more than 2^60 (and past fp32's exp range) from the first keys of a
    row to its last ones: sweep 1 keeps the maximum of a row's first 32 keys as its reference and
    must notice when later keys leave it behind; rows also end at every distance from a tile edge."""
    import torch
    L, H = 700, 2
    qn = synth.normal(synth.stream_key(140), L * H * 128).reshape(L, H, 128).astype(np.float32) * 0.25
    kn = synth.normal(synth.stream_key(141), L * H * 128).reshape(L, H, 128).astype(np.float32) * 0.25
    qn[:, :, 0] = 4.0
    kn[:, 0, 0] = 8.0 * np.arange(L) / L                    # head 0: rising
    kn[:, 1, 0] = 8.0 * (1.0 - np.arange(L) / L)            # head 1: falling (reference stays the maximum)
    qb, kb = synth.f32_to_bf16_bits(qn), synth.f32_to_bf16_bits(kn)
    qf, kf = synth.bf16_to_f32(qb), synth.bf16_to_f32(kb)
    q, k = to_dev(qb), to_dev(kb)
    lay = B.make_layout(q, k, softmax_scale=4.0)
    ws = B.alloc_workspace(lay, [L])
    scores = torch.zeros(H, L, dtype=torch.float32, device="cuda")
    lse = torch.zeros(H, L, dtype=torch.float32, device="cuda")
    B.check(B.lookm_score(q, k, [0, L], lay, scores, lse, False, ws))
    assert B.lookm_device_status(ws) == B.OK
    A, lse_o = orc.scores(qf, kf, scale=4.0, want_lse=True)
    assert np.allclose(lse.cpu().numpy().reshape(H, 1, L), lse_o, rtol=1e-6, atol=2e-5)
    got = scores.cpu().numpy().astype(np.float64)
    # scores below fp32's normal range (the oracle goes down to 1e-57 here) flush to zero
    assert np.all(np.abs(got - A) <= 1e-4 * A + 1e-30)      # exponent arguments reach 130: 1e-5 relative
    assert np.allclose(got.sum(axis=1), L, rtol=1e-5)


def test_scores_packed_batch_equals_separate_requests(B):
    import torch
    lens = [200, 131, 1, 400]
    Hq, Hkv = 4, 2
    ws_list = [synth.tiny(L, Hq, Hkv, 10, 2, 0, seed=50 + i) for i, L in enumerate(lens)]
    qs, ks = [], []
    for w in ws_list:
        qb, kb, _ = synth.layer_tensors(w)
        qs.append(qb)
        ks.append(kb)
    q, k = to_dev(np.concatenate(qs)), to_dev(np.concatenate(ks))
    cu = np.concatenate([[0], np.cumsum(lens)]).tolist()
    lay = B.make_layout(q, k)
    ws = B.alloc_workspace(lay, lens)
    scores = torch.zeros(Hkv, cu[-1], dtype=torch.float32, device="cuda")
    B.check(B.lookm_score(q, k, cu, lay, scores, None, False, ws))
    assert B.lookm_device_status(ws) == B.OK
    got = scores.cpu().numpy().astype(np.float64)
    for i, L in enumerate(lens):
        A = orc.scores(synth.bf16_to_f32(qs[i]), synth.bf16_to_f32(ks[i]), threads=4)
        part = got[:, cu[i]:cu[i + 1]]
        assert np.all(np.abs(part - A) <= 2e-5 * A), i


# ------------------------------------------------------------------------------ selection ----

def _run_select(B, s32, mask, cu, budgets, windows, Hkv):
    import torch
    lens = np.diff(cu)
    Bs = [min(b, int(L)) for b, L in zip(budgets, lens)]
    Es = [int(L) - b for b, L in zip(Bs, lens)]
    lay = B.Layout(Hkv, Hkv, 128, Hkv * 128, 128, Hkv * 128, 128, 0.0)
    ws = B.alloc_workspace(lay, [int(x) for x in lens])
    kept = torch.full((max(1, Hkv * sum(Bs)),), -7, dtype=torch.int32, device="cuda")
    ev = torch.full((max(1, Hkv * sum(Es)),), -7, dtype=torch.int32, device="cuda")
    rank = torch.full((Hkv, cu[-1]), 10 ** 9, dtype=torch.int32, device="cuda")
    B.check(B.lookm_select(torch.from_numpy(s32).cuda(), torch.from_numpy(mask).cuda(), list(cu),
                           budgets, windows, Hkv, kept, ev, rank, ws))
    torch.cuda.synchronize()
    kept, ev, rank = kept.cpu().numpy(), ev.cpu().numpy(), rank.cpu().numpy()
    ko = eo = 0
    for r, L in enumerate(lens):
        a, b = int(cu[r]), int(cu[r + 1])
        for h in range(Hkv):
            k_ref, e_ref = orc.select(s32[h, a:b].astype(np.float64), mask[a:b], budgets[r], windows[r])
            k_got = kept[ko + h * Bs[r]: ko + (h + 1) * Bs[r]]
            e_got = ev[eo + h * Es[r]: eo + (h + 1) * Es[r]]
            assert np.array_equal(k_got, k_ref), (r, h)
            assert np.array_equal(e_got, e_ref), (r, h)
            rk = rank[h, a:b]
            assert np.array_equal(rk[k_ref], -1 - np.arange(Bs[r]))
            assert np.array_equal(rk[e_ref], np.arange(Es[r]))
        ko += Hkv * Bs[r]
        eo += Hkv * Es[r]


@pytest.mark.parametrize("L,budget,window,n_text", [(50, 10, 3, 5), (50, 10, 3, 30), (4096, 819, 32, 600),
                                                     (5000, 1000, 0, 0), (5000, 999, 64, 5000),
                                                     (300, 300, 10, 100), (300, 1000, 10, 100),
                                                     (300, 20, 50, 100), (9001, 1, 1, 10), (1, 1, 0, 0)])
def test_select_is_bit_exact_on_oracle_scores(B, L, budget, window, n_text):
    Hkv = 3
    s = np.abs(synth.normal(synth.stream_key(71, L, budget), Hkv * L)).reshape(Hkv, L) + 1e-4
    s32 = s.astype(np.float32)
    mask = np.ones(L, dtype=np.uint8)
    if n_text:
        mask[synth.uniform_int(synth.stream_key(72, L), n_text, 0, L - 1).astype(int)] = 0
    _run_select(B, s32, mask, [0, L], [budget], [window], Hkv)


def test_select_ties_and_duplicates_and_batches(B):
    L, Hkv = 3000, 2
    # heavy duplication: only 7 distinct score values, so every threshold is a tie
    s32 = (1.0 + (synth.uniform_int(synth.stream_key(73), Hkv * L, 0, 6).reshape(Hkv, L) % 7)).astype(np.float32)
    mask = (synth.uniform_int(synth.stream_key(74), L, 0, 9) > 1).astype(np.uint8)
    for budget, window in [(600, 32), (37, 5), (2999, 0), (1500, 1500)]:
        _run_select(B, s32, mask, [0, L], [budget], [window], Hkv)
    _run_select(B, s32, mask, [0, 700, 701, 1900, 3000], [100, 5, 1200, 300], [8, 0, 32, 400], Hkv)
    # oracle scores of a real prompt (fp32-rounded), text prior active
    w = synth.tiny(640, 2, 2, 128, 16, 0, image_spans=[(40, 300), (340, 600)], seed=4)
    qb, kb, _ = synth.layer_tensors(w)
    A = orc.scores(synth.bf16_to_f32(qb), synth.bf16_to_f32(kb), threads=4).astype(np.float32)
    _run_select(B, A, w.requests[0].mask, [0, 640], [128], [16], 2)


# ------------------------------------------------------------------------------ matching -----

def test_match_from_sim_is_bit_exact(B):
    import torch
    Hkv, lens, budgets = 2, [90, 400], [20, 130]
    cu = [0, 90, 490]
    blocks, refs = [], []
    for r, (L, b) in enumerate(zip(lens, budgets)):
        for h in range(Hkv):
            S = synth.normal(synth.stream_key(81, r, h), (L - b) * b).reshape(L - b, b).astype(np.float32)
            S[:, 3] = S[:, 7]                      # exact ties between two slots
            S[::5, :] = np.float32(0.25)           # whole rows tied: slot 0 must win
            blocks.append(S.ravel())
            refs.append(orc.argmax_rows(S.astype(np.float64)))
    sim_matrix = torch.from_numpy(np.concatenate(blocks)).cuda()
    n_ev = Hkv * sum(L - b for L, b in zip(lens, budgets))
    assign = torch.zeros(n_ev, dtype=torch.int32, device="cuda")
    sim = torch.zeros(n_ev, dtype=torch.float32, device="cuda")
    lay = B.Layout(Hkv, Hkv, 128, Hkv * 128, 128, Hkv * 128, 128, 0.0)
    ws = B.alloc_workspace(lay, lens)
    B.check(B.lookm_match_from_sim(sim_matrix, cu, budgets, Hkv, assign, sim, ws))
    torch.cuda.synchronize()
    a_ref = np.concatenate([a for a, _ in refs])
    s_ref = np.concatenate([s for _, s in refs])
    assert np.array_equal(assign.cpu().numpy(), a_ref)
    assert np.array_equal(sim.cpu().numpy().astype(np.float64), s_ref)


@pytest.mark.parametrize("L,budget,window,Hkv", [(300, 64, 8, 2), (1000, 129, 16, 3), (520, 400, 4, 1)])
def test_match_agrees_with_oracle_up_to_near_ties(B, L, budget, window, Hkv):
    import torch
    w = synth.tiny(L, Hkv, Hkv, budget, window, 0, image_spans=[(10, L // 2)], seed=L + 1)
    (q, k, v), (qf, kf, vf), mask, _ = _tensors(w)
    s = np.abs(synth.normal(synth.stream_key(91, L), Hkv * L)).reshape(Hkv, L) + 1e-3
    lists = [orc.select(s[h], mask, budget, window) for h in range(Hkv)]
    kept = torch.from_numpy(np.concatenate([a for a, _ in lists])).cuda()
    ev = torch.from_numpy(np.concatenate([b for _, b in lists])).cuda()
    E = L - budget
    assign = torch.zeros(Hkv * E, dtype=torch.int32, device="cuda")
    sim = torch.zeros(Hkv * E, dtype=torch.float32, device="cuda")
    lay = B.make_layout(None, k)
    ws = B.alloc_workspace(lay, [L])
    B.check(B.lookm_match(k, kept, ev, [0, L], [budget], lay, assign, sim, ws))
    assert B.lookm_device_status(ws) == B.OK
    a_got = assign.cpu().numpy().reshape(Hkv, E)
    s_got = sim.cpu().numpy().reshape(Hkv, E).astype(np.float64)
    for h in range(Hkv):
        a_ref, s_ref, S = orc.match(kf, h, lists[h][0], lists[h][1], want_matrix=True)
        assert np.allclose(s_got[h], s_ref, atol=2e-6, rtol=0)
        bad = np.where(a_got[h] != a_ref)[0]
        for e in bad:                                # only exact or near ties may differ
            assert S[e, a_ref[e]] - S[e, a_got[h, e]] <= 1e-4
        assert len(bad) <= E // 100


def test_match_duplicate_kept_keys_take_the_lower_slot(B):
    import torch
    L, budget = 400, 150
    w = synth.tiny(L, 1, 1, budget, 0, 0, seed=12)
    _, kb, _ = synth.layer_tensors(w)
    kb[100:140] = kb[10:50]                          # 40 kept pairs of identical keys
    kb[300:330] = kb[100:130]                        # evicted rows equal to both members of a pair
    kf = synth.bf16_to_f32(kb)
    k = to_dev(kb)
    kept_np = np.arange(0, budget, dtype=np.int32)
    ev_np = np.arange(budget, L, dtype=np.int32)
    assign = torch.zeros(L - budget, dtype=torch.int32, device="cuda")
    sim = torch.zeros(L - budget, dtype=torch.float32, device="cuda")
    lay = B.make_layout(None, k)
    ws = B.alloc_workspace(lay, [L])
    B.check(B.lookm_match(k, torch.from_numpy(kept_np).cuda(), torch.from_numpy(ev_np).cuda(), [0, L],
                          [budget], lay, assign, sim, ws))
    a_ref, s_ref = orc.match(kf, 0, kept_np, ev_np)
    a_got = assign.cpu().numpy()
    assert np.array_equal(a_got[150:180], a_ref[150:180])
    assert np.array_equal(a_got[150:180], np.arange(10, 40))
    assert np.allclose(sim.cpu().numpy()[150:180], 1.0, atol=1e-6)


@pytest.mark.parametrize("L,budget", [(384, 128), (300, 44), (200, 199), (131, 3)])
def test_match_whole_blocks_single_rows_and_strided_keys(B, L, budget):
    """The evicted rows are gathered 128 at a time: lists of exactly 128 and 256 rows, of one row, and
    of 128 rows against 3 kept keys; the keys sit in a fused [L, 3 * H, 128] buffer (strided heads)."""
    import torch
    Hkv = 2
    w = synth.tiny(L, Hkv, Hkv, budget, 0, 0, image_spans=[(5, L // 2)], seed=L + budget)
    (q, k, v), (qf, kf, vf), mask, _ = _tensors(w)
    fused = torch.stack([q, k, v], dim=1).reshape(L, 3 * Hkv, 128).contiguous()
    fk = fused[:, Hkv:2 * Hkv]
    s = np.abs(synth.normal(synth.stream_key(92, L), Hkv * L)).reshape(Hkv, L) + 1e-3
    lists = [orc.select(s[h], mask, budget, 0) for h in range(Hkv)]
    kept = torch.from_numpy(np.concatenate([a for a, _ in lists])).cuda()
    ev = torch.from_numpy(np.concatenate([b for _, b in lists])).cuda()
    E = L - budget
    assign = torch.full((Hkv * E,), -7, dtype=torch.int32, device="cuda")
    sim = torch.full((Hkv * E,), -7.0, dtype=torch.float32, device="cuda")
    lay = B.make_layout(None, fk)
    ws = B.alloc_workspace(lay, [L])
    B.check(B.lookm_match(fk, kept, ev, [0, L], [budget], lay, assign, sim, ws))
    assert B.lookm_device_status(ws) == B.OK
    a_got = assign.cpu().numpy().reshape(Hkv, E)
    s_got = sim.cpu().numpy().reshape(Hkv, E).astype(np.float64)
    for h in range(Hkv):
        a_ref, s_ref, S = orc.match(kf, h, lists[h][0], lists[h][1], want_matrix=True)
        assert np.allclose(s_got[h], s_ref, atol=2e-6, rtol=0)
        for e in np.where(a_got[h] != a_ref)[0]:
            assert S[e, a_ref[e]] - S[e, a_got[h, e]] <= 1e-4


def test_match_packed_batch_and_out_of_range_evicted_position(B):
    import torch
    Hkv = 2
    lens, budgets = [150, 400, 129], [30, 100, 1]
    w = synth.Workload("batch", 0, 77, 1, Hkv, Hkv, 128, False,
                       [synth.tiny(n, Hkv, Hkv, b, 0, 0, seed=300 + n).requests[0] for n, b in zip(lens, budgets)])
    qb, kb, vb, mask = synth.packed_layer_tensors(w, 0)
    k, kf = to_dev(kb), synth.bf16_to_f32(kb)
    cu = np.concatenate([[0], np.cumsum(lens)]).tolist()
    kept_l, ev_l = [], []
    for r, (n, b) in enumerate(zip(lens, budgets)):
        for h in range(Hkv):
            sc = np.abs(synth.normal(synth.stream_key(93, r, h), n)) + 1e-3
            a, e = orc.select(sc, mask[cu[r]:cu[r + 1]], b, 0)
            kept_l.append(a)
            ev_l.append(e)
    kept = torch.from_numpy(np.concatenate(kept_l)).cuda()
    ev = torch.from_numpy(np.concatenate(ev_l)).cuda()
    n_ev = sum(Hkv * (n - b) for n, b in zip(lens, budgets))
    assign = torch.zeros(n_ev, dtype=torch.int32, device="cuda")
    sim = torch.zeros(n_ev, dtype=torch.float32, device="cuda")
    lay = B.make_layout(None, k)
    ws = B.alloc_workspace(lay, lens)
    B.check(B.lookm_match(k, kept, ev, cu, budgets, lay, assign, sim, ws))
    assert B.lookm_device_status(ws) == B.OK
    a_got, s_got = assign.cpu().numpy(), sim.cpu().numpy().astype(np.float64)
    at = 0
    for r, (n, b) in enumerate(zip(lens, budgets)):
        for h in range(Hkv):
            E = n - b
            a_ref, s_ref, S = orc.match(kf[cu[r]:cu[r + 1]], h, kept_l[r * Hkv + h], ev_l[r * Hkv + h], want_matrix=True)
            assert np.allclose(s_got[at:at + E], s_ref, atol=2e-6, rtol=0)
            for e in np.where(a_got[at:at + E] != a_ref)[0]:
                assert S[e, a_ref[e]] - S[e, a_got[at + e]] <= 1e-4
            at += E
    # a position beyond the request is reported through the status word, never dereferenced
    ev[5] = 100000
    B.check(B.lookm_match(k, kept, ev, cu, budgets, lay, assign, sim, ws))
    assert B.lookm_device_status(ws) == B.ERR_DEVICE_BAD_INDEX
    assert B.lookm_device_status(ws) == B.OK


# ------------------------------------------------------------------------------ merging ------

@pytest.mark.parametrize("mode", [0, 1, 2])
@pytest.mark.parametrize("L,budget,Hkv", [(300, 64, 2), (2100, 300, 3)])
def test_merge_matches_oracle_on_oracle_lists(B, mode, L, budget, Hkv):
    import torch
    w = synth.tiny(L, Hkv, Hkv, budget, 8, mode, seed=L + mode)
    (q, k, v), (qf, kf, vf), mask, _ = _tensors(w)
    s = np.abs(synth.normal(synth.stream_key(95, L), Hkv * L)).reshape(Hkv, L) + 1e-3
    E = L - budget
    kept, ev, assign, sim = [], [], [], []
    for h in range(Hkv):
        a, b = orc.select(s[h], mask, budget, 8)
        # a skewed random assignment: half of the evicted rows go to 3 slots, one slot gets none
        asg = (synth.uniform_int(synth.stream_key(96, h), E, 0, budget - 2)).astype(np.int32)
        asg[::2] = asg[::2] % 3
        kept.append(a), ev.append(b), assign.append(asg)
        sim.append(np.clip(synth.normal(synth.stream_key(97, h), E) * 0.4, -1, 1).astype(np.float32))
    dev = lambda xs: torch.from_numpy(np.concatenate(xs)).cuda()
    out_k = torch.zeros(Hkv, budget, 128, dtype=torch.bfloat16, device="cuda")
    out_v = torch.zeros_like(out_k)
    lay = B.make_layout(None, k)
    ws = B.alloc_workspace(lay, [L])
    B.check(B.lookm_merge(k, v, dev(kept), dev(ev), dev(assign), dev(sim), [0, L], [budget], [mode], lay,
                          0, out_k, out_v, ws))
    assert B.lookm_device_status(ws) == B.OK
    gk, gv = bf16_to_np(out_k), bf16_to_np(out_v)
    for h in range(Hkv):
        rk = orc.merge(kf, h, kept[h], ev[h], assign[h], sim[h].astype(np.float64), mode)
        rv = orc.merge(vf, h, kept[h], ev[h], assign[h], sim[h].astype(np.float64), mode)
        assert merged_close(gk[h], rk).all() and merged_close(gv[h], rv).all()
        assert np.abs(gk[h] - rk).max() <= 2e-2 and np.abs(gv[h] - rv).max() <= 2e-2   # N(0,1) inputs
        empty = np.setdiff1d(np.arange(budget), assign[h])
        assert len(empty) > 0
        assert np.array_equal(gk[h][empty], kf[kept[h][empty], h].astype(np.float64))   # bit-exact copy


def test_merge_packed_batch_with_slots_spread_over_many_work_units(B):
    """Two requests, batch output layout, member counts from 0 to many hundreds: the kernel cuts its
    work units at fixed entry counts, so most of the large slots are summed piecewise by several
    warps; every merge mode appears once."""
    import torch
    Hkv = 3
    lens, budgets, modes = [1700, 900], [25, 60], [2, 1]
    w0 = synth.tiny(sum(lens), Hkv, Hkv, 10, 4, 0, seed=77)
    (q, k, v), (qf, kf, vf), _, _ = _tensors(w0)
    cu = [0, lens[0], sum(lens)]
    kept, ev, assign, sim, per = [], [], [], [], []
    for r, (L, bud) in enumerate(zip(lens, budgets)):
        E = L - bud
        for h in range(Hkv):
            pos = np.sort(synth.uniform_int(synth.stream_key(120, r, h), 4 * bud, 0, L - 1))
            a = np.unique(pos)[:bud].astype(np.int32)
            assert len(a) == bud
            b = np.setdiff1d(np.arange(L, dtype=np.int32), a)
            asg = synth.uniform_int(synth.stream_key(121, r, h), E, 0, bud - 1).astype(np.int32)
            asg[: (2 * E) // 3] = 3 + h                      # two thirds of the rows in one slot
            asg[asg == 1] = 2                                # slot 1 gets nobody
            sm = np.clip(synth.normal(synth.stream_key(122, r, h), E) * 0.4, -1, 1).astype(np.float32)
            kept.append(a), ev.append(b), assign.append(asg), sim.append(sm)
            per.append((r, h, a, b, asg, sm))
    dev = lambda xs: torch.from_numpy(np.concatenate(xs)).cuda()
    out_k = torch.zeros(sum(budgets), Hkv, 128, dtype=torch.bfloat16, device="cuda")
    out_v = torch.zeros_like(out_k)
    lay = B.make_layout(None, k)
    ws = B.alloc_workspace(lay, lens)
    B.check(B.lookm_merge(k, v, dev(kept), dev(ev), dev(assign), dev(sim), cu, budgets, modes, lay,
                          1, out_k, out_v, ws))
    assert B.lookm_device_status(ws) == B.OK
    gk, gv = bf16_to_np(out_k), bf16_to_np(out_v)
    out_cu = np.concatenate([[0], np.cumsum(budgets)])
    for r, h, a, b, asg, sm in per:
        kr, vr = kf[cu[r]:cu[r + 1]], vf[cu[r]:cu[r + 1]]
        rk = orc.merge(kr, h, a, b, asg, sm.astype(np.float64), modes[r])
        rv = orc.merge(vr, h, a, b, asg, sm.astype(np.float64), modes[r])
        assert merged_close(gk[out_cu[r]:out_cu[r + 1], h], rk).all()
        assert merged_close(gv[out_cu[r]:out_cu[r + 1], h], rv).all()
        assert np.array_equal(gk[out_cu[r] + 1, h], kr[a[1], h].astype(np.float64))   # no members: copied


def test_merge_long_request_with_one_huge_slot(B):
    """70,000 tokens, 300 kept, 66,000 of the evicted rows in one slot: the inversion has to count
    past 16 bits and the merge sums that slot from hundreds of work units."""
    import torch
    L, budget, mode = 70000, 300, 2
    w = synth.tiny(L, 1, 1, budget, 8, mode, seed=31)
    (q, k, v), (qf, kf, vf), mask, _ = _tensors(w)
    E = L - budget
    kept = np.sort(np.unique(synth.uniform_int(synth.stream_key(130), 4 * budget, 0, L - 1))[:budget]).astype(np.int32)
    assert len(kept) == budget
    ev = np.setdiff1d(np.arange(L, dtype=np.int32), kept)
    asg = synth.uniform_int(synth.stream_key(131), E, 0, budget - 1).astype(np.int32)
    asg[1000:67000] = 17
    sim = np.clip(synth.normal(synth.stream_key(132), E) * 0.4, -1, 1).astype(np.float32)
    dev = lambda x: torch.from_numpy(x).cuda()
    out_k = torch.zeros(1, budget, 128, dtype=torch.bfloat16, device="cuda")
    out_v = torch.zeros_like(out_k)
    lay = B.make_layout(None, k)
    ws = B.alloc_workspace(lay, [L])
    B.check(B.lookm_merge(k, v, dev(kept), dev(ev), dev(asg), dev(sim), [0, L], [budget], [mode], lay,
                          0, out_k, out_v, ws))
    assert B.lookm_device_status(ws) == B.OK
    rk = orc.merge(kf, 0, kept, ev, asg, sim.astype(np.float64), mode)
    rv = orc.merge(vf, 0, kept, ev, asg, sim.astype(np.float64), mode)
    assert merged_close(bf16_to_np(out_k)[0], rk).all() and merged_close(bf16_to_np(out_v)[0], rv).all()


def test_merge_single_kept_token_and_bad_index_status(B):
    import torch
    L = 700
    w = synth.tiny(L, 1, 1, 1, 1, 0, seed=5)
    (q, k, v), (qf, kf, vf), mask, _ = _tensors(w)
    kept = torch.tensor([L - 1], dtype=torch.int32, device="cuda")
    ev = torch.arange(L - 1, dtype=torch.int32, device="cuda")
    assign = torch.zeros(L - 1, dtype=torch.int32, device="cuda")
    sim = torch.ones(L - 1, dtype=torch.float32, device="cuda")
    out_k = torch.zeros(1, 1, 128, dtype=torch.bfloat16, device="cuda")
    out_v = torch.zeros_like(out_k)
    lay = B.make_layout(None, k)
    ws = B.alloc_workspace(lay, [L])
    B.check(B.lookm_merge(k, v, kept, ev, assign, sim, [0, L], [1], [0], lay, 0, out_k, out_v, ws))
    assert B.lookm_device_status(ws) == B.OK
    assert np.abs(bf16_to_np(out_k)[0, 0] - kf[:, 0].astype(np.float64).mean(axis=0)).max() <= 2e-3
    assert np.abs(bf16_to_np(out_v)[0, 0] - vf[:, 0].astype(np.float64).mean(axis=0)).max() <= 2e-3
    # an out-of-range assignment is reported through the status word, never dereferenced
    assign[5] = 9
    B.check(B.lookm_merge(k, v, kept, ev, assign, sim, [0, L], [1], [0], lay, 0, out_k, out_v, ws))
    assert B.lookm_device_status(ws) == B.ERR_DEVICE_BAD_INDEX
    assert B.lookm_device_status(ws) == B.OK          # reading clears it


def test_an_expired_device_wait_is_reported_and_the_context_stays_usable(B):
    """The tile kernels bound every mbarrier wait; when one runs out the CTA raises its abort flag,
    leaves, and the status word says so.  Here a one-CTA kernel waits 1 ms, through the same wait
    routine, on a barrier nobody arrives at."""
    import torch
    ws = torch.empty(4096, dtype=torch.uint8, device="cuda")
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    B.check(B.lookm_selftest_wait_expiry(1000, ws))
    t1.record()
    assert B.lookm_device_status(ws) == B.ERR_DEVICE_TIMEOUT
    assert B.lookm_device_status(ws) == B.OK              # reading clears it
    assert 0.9 <= t0.elapsed_time(t1) <= 50.0             # the limit was 1 ms; it neither returned early nor hung
    # the context still works: a real kernel of the library runs and reports no error
    L = 300
    w = synth.tiny(L, 2, 2, 60, 8, 0, seed=3)
    (q, k, v), _, mask, _ = _tensors(w)
    lay = B.make_layout(q, k)
    ws2 = B.alloc_workspace(lay, [L])
    scores = torch.zeros(2, L, dtype=torch.float32, device="cuda")
    B.check(B.lookm_score(q, k, [0, L], lay, scores, None, 0, ws2))
    assert B.lookm_device_status(ws2) == B.OK
    assert abs(float(scores.sum()) - 2 * L) <= 1e-2
