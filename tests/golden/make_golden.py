"""Writes tests/golden/tiny_ar_stream.txt: the oracle's greedy stream for the tiny fp32 config.

Calls only the workload generator and `oracle/`; never the CUDA path.
Run from the repository root:  python tests/golden/make_golden.py
"""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2311_08263_b200 import workload as wl  # noqa: E402

cfg = wl.CONFIGS["tiny"]
w = wl.make_weights(cfg)
prompt = wl.make_prompts(cfg)[0][0].numpy()
ar, _ = oracle.Oracle(cfg, w, 160).ar_generate(prompt, 64)
path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_ar_stream.txt")
with open(path, "w") as f:
    f.write("# greedy autoregressive stream (Eq. 1) of the oracle; tiny fp32 config, seed %d,\n" % cfg.seed)
    f.write("# prompt = 32 seeded ids, 64 generated tokens. Written by make_golden.py (oracle only).\n")
    f.write(" ".join(str(int(t)) for t in ar) + "\n")
print("wrote", path)
