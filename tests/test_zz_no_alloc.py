"""lookm_merge_noalloc, the merge step for hosts that may not allocate device memory.

A serving process that has given all device memory to its own pool, or a plug-in living inside
another program's memory budget, cannot hand the library a workspace obtained from cudaMalloc at
compression time.  For such callers the library carries a fixed scratch array in its own device
image.  This test drives that entry point through the C ABI and requires it to reproduce
lookm_merge (same kernels, so bit for bit, which is inside the 2e-2 tolerance of the other merge
tests) on two calls in a row: the second call finds the first call's leftovers in the shared
array and must not be disturbed by them.  The file name makes pytest collect it last.
"""
import numpy as np
import pytest

from oracle import lookm_oracle as orc
from paper_2406_18139_b200 import synth
from tests.helpers import bf16_to_np, merged_close, to_dev

pytestmark = pytest.mark.gpu


def _case(L, Hkv, budget, mode, seed):
    import torch
    w = synth.tiny(L, Hkv, Hkv, budget, 8, mode, seed=seed)
    qb, kb, vb = synth.layer_tensors(w)
    k, v = to_dev(kb), to_dev(vb)
    E = L - budget
    kept, ev, assign, sim = [], [], [], []
    for h in range(Hkv):
        s = np.abs(synth.normal(synth.stream_key(301, seed, h), L)) + 1e-3
        a, b = orc.select(s, w.requests[0].mask, budget, 8)
        kept.append(a), ev.append(b)
        assign.append(synth.uniform_int(synth.stream_key(302, seed, h), E, 0, budget - 1).astype(np.int32))
        sim.append(np.clip(synth.normal(synth.stream_key(303, seed, h), E) * 0.4, -1, 1).astype(np.float32))
    dev = lambda xs: torch.from_numpy(np.concatenate(xs)).cuda()
    return (k, v, dev(kept), dev(ev), dev(assign), dev(sim)), (kb, vb, kept, ev, assign, sim)


def test_noalloc_merge_equals_workspace_merge_twice_in_a_row():
    import torch
    from paper_2406_18139_b200 import binding as B
    B.lib()
    # two different problems back to back, so the second one overwrites the first one's scratch
    for L, Hkv, budget, mode, seed in [(900, 3, 150, 2, 1), (640, 2, 200, 1, 2)]:
        (k, v, kept, ev, assign, sim), host = _case(L, Hkv, budget, mode, seed)
        lay = B.make_layout(None, k)
        ws = B.alloc_workspace(lay, [L])
        ref_k = torch.zeros(Hkv, budget, 128, dtype=torch.bfloat16, device="cuda")
        ref_v = torch.zeros_like(ref_k)
        B.check(B.lookm_merge(k, v, kept, ev, assign, sim, [0, L], [budget], [mode], lay, 0, ref_k, ref_v, ws))
        assert B.lookm_device_status(ws) == B.OK
        out_k = torch.full_like(ref_k, 7.0)
        out_v = torch.full_like(ref_k, 7.0)
        B.check(B.lookm_merge_noalloc(k, v, kept, ev, assign, sim, [0, L], [budget], [mode], lay, 0,
                                      out_k, out_v))
        assert B.lookm_noalloc_status() == B.OK
        assert torch.equal(out_k, ref_k) and torch.equal(out_v, ref_v)
        # and it is the right answer, not merely the same one
        kb, vb, kept_h, ev_h, assign_h, sim_h = host
        kf, vf = synth.bf16_to_f32(kb), synth.bf16_to_f32(vb)
        gk = bf16_to_np(out_k)
        for h in range(Hkv):
            want = orc.merge(kf, h, kept_h[h], ev_h[h], assign_h[h], sim_h[h].astype(np.float64), mode)
            assert merged_close(gk[h], want).all()


def test_noalloc_merge_rejects_batches_beyond_its_scratch():
    import torch
    from paper_2406_18139_b200 import binding as B
    B.lib()
    lay = B.Layout(64, 64, 128, 64 * 128, 128, 64 * 128, 128, 0.0)
    L = 8192                                   # 64 heads x 8192 tokens needs about 21 MB > 16 MiB
    dummy = torch.zeros(64, dtype=torch.int32, device="cuda")
    st = B.lookm_merge_noalloc(dummy, dummy, dummy, dummy, dummy, dummy, [0, L], [1638], [0], lay, 0,
                               dummy, dummy)
    assert st == B.ERR_WORKSPACE_TOO_SMALL
