"""Writes c5_requests.txt: the drawn request table of the ragged serving batch (seed 0).

Calls only the input generator; the table lets a reader see the batch without running anything
and lets a test detect a change of the generator.
Run from the repository root:  python tests/golden/make_c5_table.py
"""
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
from paper_2406_18139_b200 import synth  # noqa: E402

w = synth.config5(seed=0)
path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "c5_requests.txt")
with open(path, "w") as f:
    f.write("# ragged serving batch, seed 0: request seq_len n_images text_tokens budget window merge_mode\n")
    for i, r in enumerate(w.requests):
        f.write("%d %d %d %d %d %d %d\n" % (i, r.seq_len, r.n_images, r.seq_len - 576 * r.n_images,
                                            r.budget, r.window, r.merge_mode))
print("wrote", path)
