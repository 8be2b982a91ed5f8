"""B200-native LOOK-M prefill-time KV-cache compression (C-ABI library + thin Python binding).

Importing the package loads nothing; ``paper_2406_18139_b200.binding`` loads the CUDA library on
first use and raises if it has not been built.  ``synth`` draws the seeded synthetic prompts.
"""
