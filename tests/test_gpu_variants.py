"""The method's variants through the C ABI, against the fp64 oracle: selection without the text
prior (Eq. 8 alone), eviction without merging (Eq. 6-7 alone), very small budgets (the 95-99 %
compression of the paper's appendix), a caller-supplied row log-sum-exp (the scores of Eq. 4 come
from the prompt-encoding attention itself) and output rows written into a cache with room to grow.
"""
import numpy as np
import pytest

from oracle import lookm_oracle as orc
from paper_2406_18139_b200 import synth
from tests.helpers import bf16_to_np, to_dev
from tests.test_gpu_e2e import check_head

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2406_18139_b200 import binding
    binding.lib()
    return binding


def _setup(B, w, layer=0):
    import torch
    qb, kb, vb = synth.layer_tensors(w, layer)
    dev = tuple(to_dev(t) for t in (qb, kb, vb))
    host = tuple(synth.bf16_to_f32(t) for t in (qb, kb, vb))
    req = w.requests[0]
    lay = B.make_layout(dev[0], dev[1])
    ws = B.alloc_workspace(lay, [req.seq_len])
    return dev, host, req, lay, ws, torch.from_numpy(req.mask).cuda()


def _compress(B, dev, req, lay, ws, mask_d, budget, window, mode, options=None, cap=None):
    import torch
    q, k, v = dev
    Hkv, L = k.shape[1], req.seq_len
    Bk = min(budget, L)
    rows = cap if cap is not None else Bk
    out_k = torch.full((Hkv, rows, 128), 7.0, dtype=torch.bfloat16, device="cuda")
    out_v = torch.full_like(out_k, 7.0)
    st, out_len = B.lookm_compress_layer_opt(q, k, v, mask_d, L, budget, window, mode, lay, options,
                                             out_k, out_v, ws)
    B.check(st)
    assert out_len == Bk and B.lookm_device_status(ws) == B.OK
    return out_k, out_v, B.lookm_last_launch_count()


# ------------------------------------------------------------------ selection alone ---------

@pytest.mark.parametrize("L,budget,window", [(50, 10, 3), (4096, 819, 32), (5000, 50, 0), (300, 300, 10),
                                             (300, 20, 50), (9001, 1, 1), (1, 1, 0)])
def test_select_without_mask_is_a_plain_top_n(B, L, budget, window):
    import torch
    Hkv = 3
    s32 = (np.abs(synth.normal(synth.stream_key(171, L, budget), Hkv * L)).reshape(Hkv, L) + 1e-4).astype(np.float32)
    s32[1, ::3] = np.float32(0.5)                        # many exact ties on one head
    Bk = min(budget, L)
    lay = B.Layout(Hkv, Hkv, 128, Hkv * 128, 128, Hkv * 128, 128, 0.0)
    ws = B.alloc_workspace(lay, [L])
    kept = torch.full((Hkv * Bk,), -7, dtype=torch.int32, device="cuda")
    ev = torch.full((max(1, Hkv * (L - Bk)),), -7, dtype=torch.int32, device="cuda")
    B.check(B.lookm_select(torch.from_numpy(s32).cuda(), None, [0, L], [budget], [window], Hkv, kept, ev,
                           None, ws))
    torch.cuda.synchronize()
    kept, ev = kept.cpu().numpy().reshape(Hkv, Bk), ev.cpu().numpy()[:Hkv * (L - Bk)].reshape(Hkv, L - Bk)
    any_mask = (synth.uniform_int(synth.stream_key(172, L), L, 0, 1)).astype(np.uint8)
    for h in range(Hkv):
        k_ref, e_ref = orc.select(s32[h].astype(np.float64), any_mask, budget, window, text_prior=False)
        assert np.array_equal(kept[h], k_ref) and np.array_equal(ev[h], e_ref)


# ------------------------------------------------------------------ whole path --------------

def test_whole_path_without_text_prior(B):
    w = synth.tiny(1300, 4, 2, 260, 32, 2, image_spans=[(100, 600), (700, 1200)], seed=21)
    dev, (qf, kf, vf), req, lay, ws, mask_d = _setup(B, w)
    A = orc.scores(qf, kf, threads=4)
    stats = {"kept_near_ties": 0, "assign_near_ties": 0}
    kept_sets = {}
    for prior in (True, False):
        opt = B.make_options(no_text_prior=not prior)
        out_k, out_v, _ = _compress(B, dev, req, lay, ws, mask_d if prior else None, 260, 32, 2, opt)
        _, lists = B.read_intermediates(ws, lay, [1300], [260])
        gk, gv = bf16_to_np(out_k), bf16_to_np(out_v)
        for h in range(2):
            kept, ev, asg, _ = lists[0][h]
            check_head(kf, vf, req.mask, h, 260, 32, 2, A[h], kept, ev, asg, gk[h], gv[h], stats, text_prior=prior)
            kept_sets[(prior, h)] = kept.copy()
    assert stats["kept_near_ties"] <= 1
    # 300 text tokens exceed the 228 important slots: with the prior no image token is kept, without
    # it the best-scored tokens are, whatever their modality
    assert all(req.mask[kept_sets[(True, h)][:228]].sum() == 0 for h in range(2))
    assert all(req.mask[kept_sets[(False, h)][:228]].sum() > 0 for h in range(2))


@pytest.mark.parametrize("text_prior", [True, False])
def test_eviction_alone_copies_the_kept_rows_and_skips_matching(B, text_prior):
    w = synth.tiny(900, 4, 2, 180, 16, 3, image_spans=[(50, 400), (450, 800)], seed=22)
    dev, (qf, kf, vf), req, lay, ws, mask_d = _setup(B, w)
    A = orc.scores(qf, kf, threads=4)
    opt = B.make_options(no_text_prior=not text_prior)
    out_k, out_v, launches = _compress(B, dev, req, lay, ws, mask_d, 180, 16, B.MERGE_NONE, opt)
    assert launches == 5            # table writer, two sweeps, selection, compaction: no norms, no
    _, lists = B.read_intermediates(ws, lay, [900], [180])     # gather, no matching, no inversion
    gk, gv = bf16_to_np(out_k), bf16_to_np(out_v)
    stats = {"kept_near_ties": 0, "assign_near_ties": 0}
    for h in range(2):
        kept, ev, asg, _ = lists[0][h]
        check_head(kf, vf, req.mask, h, 180, 16, 3, A[h], kept, ev, asg, gk[h], gv[h], stats, text_prior=text_prior)
    assert stats["kept_near_ties"] == 0
    # the merging call alone, fed with lists, in the same mode and without an assignment
    import torch
    kept_all = torch.from_numpy(np.concatenate([lists[0][h][0] for h in range(2)])).cuda()
    ev_all = torch.from_numpy(np.concatenate([lists[0][h][1] for h in range(2)])).cuda()
    mk, mv = torch.zeros_like(out_k), torch.zeros_like(out_v)
    B.check(B.lookm_merge(dev[1], dev[2], kept_all, ev_all, None, None, [0, 900], [180], [B.MERGE_NONE], lay,
                          0, mk, mv, ws))
    assert B.lookm_device_status(ws) == B.OK and B.lookm_last_launch_count() == 2
    assert torch.equal(mk, out_k) and torch.equal(mv, out_v)


@pytest.mark.parametrize("ratio", [0.01, 0.02, 0.05])
def test_config1_at_very_small_budgets(B, ratio):
    """95-99 % compression (the paper's appendix table): every head of the 2048-token workload."""
    w = synth.config1()
    dev, (qf, kf, vf), req, lay, ws, mask_d = _setup(B, w)
    L = req.seq_len
    budget = int(ratio * L)                              # 20, 40, 102 rows; the window is clamped to it
    A = orc.scores(qf, kf, threads=8)
    stats = {"kept_near_ties": 0, "assign_near_ties": 0}
    for mode in (0, 2):
        out_k, out_v, _ = _compress(B, dev, req, lay, ws, mask_d, budget, req.window, mode)
        _, lists = B.read_intermediates(ws, lay, [L], [budget])
        gk, gv = bf16_to_np(out_k), bf16_to_np(out_v)
        for h in range(w.n_kv_heads):
            kept, ev, asg, _ = lists[0][h]
            assert len(kept) == budget
            check_head(kf, vf, req.mask, h, budget, req.window, mode, A[h], kept, ev, asg, gk[h], gv[h], stats)
    assert stats["kept_near_ties"] <= 1


def test_caller_supplied_log_sum_exp_skips_the_first_sweep(B):
    import torch
    w = synth.tiny(1100, 8, 2, 220, 16, 1, image_spans=[(60, 500), (560, 1000)], seed=23)
    dev, (qf, kf, vf), req, lay, ws, mask_d = _setup(B, w)
    plain_k, plain_v, n_plain = _compress(B, dev, req, lay, ws, mask_d, 220, 16, 1)
    scores_plain, _ = B.read_intermediates(ws, lay, [1100], [220])
    # the log-sum-exp as a prefill attention kernel would leave it: here the oracle's, rounded to fp32
    _, lse_o = orc.scores(qf, kf, threads=4, want_lse=True)
    lse = torch.from_numpy(lse_o.reshape(8, 1100).astype(np.float32)).cuda()
    ws.zero_()
    opt = B.make_options(lse=lse)
    out_k, out_v, n_lse = _compress(B, dev, req, lay, ws, mask_d, 220, 16, 1, opt)
    assert n_lse == n_plain                              # the companion-tensor kernel replaces sweep 1
    scores_lse, lists = B.read_intermediates(ws, lay, [1100], [220])
    A = orc.scores(qf, kf, threads=4)
    assert np.all(np.abs(scores_lse - A) <= 2e-5 * A)
    assert np.all(np.abs(scores_lse - scores_plain) <= 2e-5 * A)
    gk, gv = bf16_to_np(out_k), bf16_to_np(out_v)
    stats = {"kept_near_ties": 0, "assign_near_ties": 0}
    for h in range(2):
        kept, ev, asg, _ = lists[0][h]
        check_head(kf, vf, req.mask, h, 220, 16, 1, A[h], kept, ev, asg, gk[h], gv[h], stats)
    # the workspace's own log-sum-exp buffer was not written: sweep 1 did not run
    off = B.lookm_workspace_layout(lay, [1100])
    assert int(ws[off.lse:off.lse + 4 * 8 * 1100].view(torch.int32).abs().max()) == 0


@pytest.mark.parametrize("mode", [0, 3])
def test_output_rows_written_into_a_cache_with_room_to_grow(B, mode):
    import torch
    w = synth.tiny(800, 2, 2, 160, 8, mode, image_spans=[(40, 700)], seed=24)
    dev, _, req, lay, ws, mask_d = _setup(B, w)
    dense_k, dense_v, _ = _compress(B, dev, req, lay, ws, mask_d, 160, 8, mode)
    cap = 200
    opt = B.make_options(out_stride_head=cap * 128)
    cache_k, cache_v, _ = _compress(B, dev, req, lay, ws, mask_d, 160, 8, mode, opt, cap=cap)
    assert torch.equal(cache_k[:, :160], dense_k) and torch.equal(cache_v[:, :160], dense_v)
    assert bool((cache_k[:, 160:] == 7.0).all()) and bool((cache_v[:, 160:] == 7.0).all())   # untouched


def test_ragged_batch_mixing_eviction_alone_with_merging(B):
    import torch
    lens, budgets, windows, modes = [300, 700, 129, 513], [60, 70, 200, 100], [8, 16, 4, 0], [3, 2, 3, 0]
    Hq, Hkv = 4, 2
    reqs = [synth.tiny(L, Hq, Hkv, b, m, mo, image_spans=[(L // 10, L // 2)], seed=500 + i)
            for i, (L, b, m, mo) in enumerate(zip(lens, budgets, windows, modes))]
    parts = [synth.layer_tensors(w) for w in reqs]
    qb, kb, vb = (np.concatenate([p[i] for p in parts]) for i in range(3))
    mask = np.concatenate([w.requests[0].mask for w in reqs])
    q, k, v = to_dev(qb), to_dev(kb), to_dev(vb)
    cu = np.concatenate([[0], np.cumsum(lens)]).tolist()
    lay = B.make_layout(q, k)
    ws = B.alloc_workspace(lay, lens)
    outs = [min(b, L) for b, L in zip(budgets, lens)]
    for prior in (True, False):
        out_k = torch.zeros(sum(outs), Hkv, 128, dtype=torch.bfloat16, device="cuda")
        out_v = torch.zeros_like(out_k)
        st, out_cu = B.lookm_compress_varlen_opt(q, k, v, torch.from_numpy(mask).cuda(), cu, budgets, windows,
                                                 modes, lay, B.make_options(no_text_prior=not prior), out_k,
                                                 out_v, ws)
        B.check(st)
        assert B.lookm_device_status(ws) == B.OK
        _, lists = B.read_intermediates(ws, lay, lens, budgets)
        gk, gv = bf16_to_np(out_k), bf16_to_np(out_v)
        stats = {"kept_near_ties": 0, "assign_near_ties": 0}
        for r in range(len(lens)):
            a, b = cu[r], cu[r + 1]
            qf, kf, vf = (synth.bf16_to_f32(t[a:b]) for t in (qb, kb, vb))
            A = orc.scores(qf, kf, threads=4)
            for h in range(Hkv):
                kept_g, ev_g, asg_g, _ = lists[r][h]
                check_head(kf, vf, mask[a:b], h, budgets[r], windows[r], modes[r], A[h], kept_g, ev_g, asg_g,
                           gk[out_cu[r]:out_cu[r + 1], h], gv[out_cu[r]:out_cu[r + 1], h], stats,
                           text_prior=prior)
        assert stats["kept_near_ties"] <= 1
