"""Parity at the full sizes of the five workloads, in the launch configuration bench.py times.

The whole layer (all heads, all requests) is compressed on the GPU; the fp64 oracle then checks
what it can compute in seconds:
  * invariants of every head (row-sum of the scores, kept count, window, text survival);
  * scores of the LAST keys of sampled heads (a key's score only needs the query rows after it,
    so the tail is cheap) and the log-sum-exp of sampled query rows anywhere in the prompt;
  * the selection, re-done by the oracle on the fp32 scores the GPU produced (bit-exact);
  * the assignment of sampled evicted tokens, up to near-ties (cosine gap <= 1e-4);
  * the merged rows of sampled heads, from the lists the GPU chose (2e-2 absolute).
Config 2 additionally runs the complete oracle on a few heads, end to end.
"""
import numpy as np
import pytest

from oracle import lookm_oracle as orc
from paper_2406_18139_b200 import synth
from tests.helpers import bf16_to_np, merged_close, to_dev
from tests.test_gpu_e2e import check_head

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2406_18139_b200 import binding
    binding.lib()
    return binding


def invariants(scores_h, kept, ev, asg, mask, L, budget, window, group):
    Bk = min(budget, L)
    M = min(window, Bk)
    assert abs(float(scores_h.astype(np.float64).sum()) - group * L) <= 1e-4 * group * L
    assert np.all(scores_h > 0)
    assert len(kept) == Bk and len(ev) == L - Bk
    assert np.all(np.diff(kept) > 0) and np.all(np.diff(ev) > 0)
    assert np.array_equal(kept[Bk - M:], np.arange(L - M, L))
    both = np.concatenate([kept, ev])
    assert len(np.unique(both)) == L and both.min() == 0 and both.max() == L - 1
    text = np.where(mask[:L - M] == 0)[0]
    if len(text) <= Bk - M:
        assert np.isin(text, kept).all()
    else:
        assert np.all(mask[kept[:Bk - M]] == 0)
    if len(asg):
        assert asg.min() >= 0 and asg.max() < Bk


def sampled_checks(B, qf, kf, vf, mask, budget, window, mode, group, scores_g, lists, gk_of, gv_of,
                   lse_g, heads, tail, n_match=48, seed=0):
    """Oracle checks of one request on the given KV heads; returns the number of near-tie cases."""
    L = len(mask)
    near = 0
    # scores of the last `tail` keys + sampled log-sum-exp rows
    tail = min(tail, L)
    A = orc.scores(qf, kf, key_begin=L - tail, kv_heads=heads, threads=len(heads))
    for i, h in enumerate(heads):
        ref = A[i, L - tail:]
        got = scores_g[h, L - tail:].astype(np.float64)
        assert np.all(np.abs(got - ref) <= 1e-3 * ref), float((np.abs(got - ref) / ref).max())
        assert np.all(np.abs(got - ref) <= 5e-5 * ref)
        rows = np.unique(synth.uniform_int(synth.stream_key(401, seed, h), 12, 0, L - 1).astype(np.int32))
        qh = h * group + (h % group)
        ref_lse = orc.lse_rows(qf, kf, qh, h, rows)
        assert np.allclose(lse_g[qh, rows], ref_lse, atol=5e-5, rtol=0)
    for h in heads:
        kept_g, ev_g, asg_g, sim_g = lists[h]
        # selection on the GPU's own fp32 scores: bit-exact
        kept_o, ev_o = orc.select(scores_g[h].astype(np.float64), mask, budget, window)
        assert np.array_equal(kept_g, kept_o) and np.array_equal(ev_g, ev_o)
        # sampled assignments
        E = len(ev_g)
        if E:
            pick = np.unique(synth.uniform_int(synth.stream_key(402, seed, h), n_match, 0, E - 1).astype(int))
            a_ref, s_ref, S = orc.match(kf, h, kept_g, ev_g[pick], want_matrix=True)
            assert np.allclose(sim_g[pick], S[np.arange(len(pick)), asg_g[pick]], atol=2e-6, rtol=0)
            for i, e in enumerate(pick):
                if asg_g[e] != a_ref[i]:
                    assert S[i, a_ref[i]] - S[i, asg_g[e]] <= 1e-4
                    near += 1
        # merged rows from the GPU's lists and weights
        rk = orc.merge(kf, h, kept_g, ev_g, asg_g, sim_g.astype(np.float64), mode)
        rv = orc.merge(vf, h, kept_g, ev_g, asg_g, sim_g.astype(np.float64), mode)
        assert merged_close(gk_of(h), rk).all() and merged_close(gv_of(h), rv).all()
    return near


def run_single(B, w, heads_full=(), heads_sampled=(), tail=768, modes=None):
    """One-prompt workloads (configs 1-4) through lookm_compress_layer."""
    import torch
    qb, kb, vb = synth.layer_tensors(w, 0)
    q, k, v = to_dev(qb), to_dev(kb), to_dev(vb)
    qf, kf, vf = (synth.bf16_to_f32(t) for t in (qb, kb, vb))
    req = w.requests[0]
    L, Hq, Hkv = req.seq_len, w.n_q_heads, w.n_kv_heads
    G = Hq // Hkv
    lay = B.make_layout(q, k)
    ws = B.alloc_workspace(lay, [L])
    mask_d = torch.from_numpy(req.mask).cuda()
    A_full = orc.scores(qf, kf, kv_heads=list(heads_full), threads=max(1, len(heads_full))) if heads_full else None
    for budget, mode in (modes or [(req.budget, req.merge_mode)]):
        Bk = min(budget, L)
        out_k = torch.zeros(Hkv, Bk, 128, dtype=torch.bfloat16, device="cuda")
        out_v = torch.zeros_like(out_k)
        st, out_len = B.lookm_compress_layer(q, k, v, mask_d, L, budget, req.window, mode, lay, out_k, out_v, ws)
        B.check(st)
        assert out_len == Bk and B.lookm_device_status(ws) == B.OK
        scores_g, lists = B.read_intermediates(ws, lay, [L], [budget])
        off = B.lookm_workspace_layout(lay, [L])
        lse_g = ws[off.lse:off.lse + 4 * Hq * L].view(torch.float32).cpu().numpy().reshape(Hq, L)
        gk, gv = bf16_to_np(out_k), bf16_to_np(out_v)
        for h in range(Hkv):
            kept, ev, asg, _ = lists[0][h]
            invariants(scores_g[h], kept, ev, asg, req.mask, L, budget, req.window, G)
        stats = {"kept_near_ties": 0, "assign_near_ties": 0}
        for i, h in enumerate(heads_full):
            kept, ev, asg, _ = lists[0][h]
            check_head(kf, vf, req.mask, h, budget, req.window, mode, A_full[i], kept, ev, asg, gk[h], gv[h], stats)
        assert stats["kept_near_ties"] <= 1
        if heads_sampled:
            sampled_checks(B, qf, kf, vf, req.mask, budget, req.window, mode, G, scores_g, lists[0],
                           lambda h: gk[h], lambda h: gv[h], lse_g, list(heads_sampled), tail)


def test_config2_8k_7b_shape_all_merge_modes(B):
    w = synth.config2()
    b = w.requests[0].budget
    run_single(B, w, heads_full=(0, 13, 31), heads_sampled=(7, 22), modes=[(b, 0), (b, 1), (b, 2)])


def test_config3_16k_13b_shape_budget_sweep(B):
    w = synth.config3()
    L = w.requests[0].seq_len
    # 10 % budget: text tokens outnumber the important slots, so only text survives the Top-N
    run_single(B, w, heads_sampled=(3, 39), tail=512,
               modes=[(int(0.1 * L), 2), (int(0.2 * L), 2), (int(0.4 * L), 2)])


def test_config4_32k_grouped_query(B):
    w = synth.config4()
    run_single(B, w, heads_sampled=(0, 7), tail=256)


def test_config5_ragged_batch(B):
    import torch
    w = synth.config5()
    qb, kb, vb, mask = synth.packed_layer_tensors(w, 0)
    q, k, v = to_dev(qb), to_dev(kb), to_dev(vb)
    lens = [r.seq_len for r in w.requests]
    budgets = [r.budget for r in w.requests]
    windows = [r.window for r in w.requests]
    modes = [r.merge_mode for r in w.requests]
    cu = w.cu_seqlens.tolist()
    Hq = Hkv = w.n_kv_heads
    lay = B.make_layout(q, k)
    ws = B.alloc_workspace(lay, lens)
    out_k = torch.zeros(sum(budgets), Hkv, 128, dtype=torch.bfloat16, device="cuda")
    out_v = torch.zeros_like(out_k)
    st, out_cu = B.lookm_compress_varlen(q, k, v, torch.from_numpy(mask).cuda(), cu, budgets, windows, modes,
                                         lay, out_k, out_v, ws)
    B.check(st)
    assert B.lookm_device_status(ws) == B.OK
    assert out_cu == np.concatenate([[0], np.cumsum(budgets)]).tolist()
    scores_g, lists = B.read_intermediates(ws, lay, lens, budgets)
    off = B.lookm_workspace_layout(lay, lens)
    T = cu[-1]
    lse_g = ws[off.lse:off.lse + 4 * Hq * T].view(torch.float32).cpu().numpy().reshape(Hq, T)
    for r, req in enumerate(w.requests):
        a, b = cu[r], cu[r + 1]
        for h in range(0, Hkv, 5):
            kept, ev, asg, _ = lists[r][h]
            invariants(scores_g[h, a:b], kept, ev, asg, req.mask, req.seq_len, req.budget, req.window, 1)
    # oracle checks on the shortest request (two heads) and two long ones (one head each)
    order = np.argsort(lens)
    for r, heads, tail in [(int(order[0]), [1, 30], 2048), (int(order[-1]), [17], 384), (int(order[8]), [5], 512)]:
        a, b = cu[r], cu[r + 1]
        qf, kf, vf = (synth.bf16_to_f32(t[a:b]) for t in (qb, kb, vb))
        gk = lambda h, r=r: bf16_to_np(out_k[out_cu[r]:out_cu[r + 1], h])
        gv = lambda h, r=r: bf16_to_np(out_v[out_cu[r]:out_cu[r + 1], h])
        sampled_checks(B, qf, kf, vf, mask[a:b], budgets[r], windows[r], modes[r], 1, scores_g[:, a:b], lists[r],
                       gk, gv, lse_g[:, a:b], heads, tail, seed=r)
