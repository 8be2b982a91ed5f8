"""The seeded input generator: layouts of the five workloads and bf16 exactness."""
import os

import numpy as np

from paper_2406_18139_b200 import synth


def test_layouts_have_the_stated_shapes():
    c1, c2, c3, c4 = synth.config1(), synth.config2(), synth.config3(), synth.config4()
    for w, L, n_img, text, B, M in [(c1, 2048, 3, 320, 409, 32), (c2, 8192, 12, 1280, 1638, 32),
                                    (c3, 16384, 24, 2560, 3276, 64), (c4, 32768, 52, 2816, 6553, 64)]:
        r = w.requests[0]
        assert r.seq_len == L and r.n_images == n_img and r.budget == B and r.window == M
        assert int((r.mask == 0).sum()) == text and len(r.mask) == L
        assert r.mask[0] == 0 and r.mask[-1] == 0           # prompts start and end with text
    assert synth.config3(ratio=0.1).requests[0].budget == 1638
    assert all(40 <= s <= 200 for s in c2.requests[0].segments)


def test_ragged_batch_matches_committed_table():
    w = synth.config5(seed=0)
    rows = [l.split() for l in open(os.path.join(os.path.dirname(__file__), "golden", "c5_requests.txt"))
            if not l.startswith("#")]
    assert len(rows) == len(w.requests) == 16
    for row, r in zip(rows, w.requests):
        assert [int(t) for t in row[1:]] == [r.seq_len, r.n_images, r.seq_len - 576 * r.n_images,
                                             r.budget, r.window, r.merge_mode]
        assert 2048 <= r.seq_len <= 16384 and 2 <= r.n_images <= 24
        assert 0.10 <= (r.seq_len - 576 * r.n_images) / r.seq_len <= 0.20
    assert w.cu_seqlens[-1] == w.total_tokens


def test_tensors_are_bf16_exact_clustered_and_reproducible():
    w = synth.config1()
    q, k, v = synth.layer_tensors(w)
    q2, _, _ = synth.layer_tensors(w)
    assert q.dtype == np.uint16 and np.array_equal(q, q2)
    kf = synth.bf16_to_f32(k)
    assert np.array_equal(synth.f32_to_bf16_bits(kf), k)
    r = w.requests[0]
    img0 = r.segments[0]
    a, b, far = kf[img0, 0], kf[img0 + 5, 0], kf[img0 + 100, 0]   # same patch row / another row
    cos = lambda x, y: float(x @ y / np.linalg.norm(x) / np.linalg.norm(y))
    assert cos(a, b) > 0.8 and abs(cos(a, far)) < 0.5
    assert abs(float(synth.bf16_to_f32(q).std()) - 1.0) < 0.01
    # round-to-nearest-even on a tie: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert synth.f32_to_bf16_bits(np.array([1.00390625], dtype=np.float32))[0] == 0x3F80
    assert synth.f32_to_bf16_bits(np.array([1.01171875], dtype=np.float32))[0] == 0x3F82
