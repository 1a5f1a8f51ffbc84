"""Writes tests/golden/stream_<config>.json for the bf16 configurations (1b, 7b, 13b): what the oracle
computes for the stated workload, so that the GPU tests can check whole streams at full model shapes
without replaying hours of CPU work.

Calls only the workload generator and `oracle/`; never the CUDA path.  Per sequence:
  1. prefill of the seeded prompt with the configuration's window size c;
  2. N_STEPS Jacobi iterations, each recorded: the window fed, accepted count and tokens, refreshed window and,
     per row, the two largest logits (ids and values) plus the logits at a fixed set of seeded vocabulary positions;
  3. the window is shrunk to one row and greedy decoding continues to gen_tokens tokens; recorded: the stream
     and the top-1/top-2 logit margin at every position (the first tokens and margins come from step 2's
     accepted rows: a window row's logits are bitwise those of the autoregressive forward of the same context).

Run from the repository root:  python tests/golden/make_streams.py 1b 7b 13b
(13b x 8 sequences takes a few hours on 8 cores; results are written after every sequence, and finished
sequences are skipped when the script is run again).
"""
import json
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2311_08263_b200 import workload as wl  # noqa: E402

N_STEPS = 8
N_POS = 8
HERE = os.path.dirname(os.path.abspath(__file__))


def top2(row):
    i1 = int(np.argmax(row))
    v1 = float(row[i1])
    tmp = row[i1]
    row[i1] = -np.inf
    i2 = int(np.argmax(row))
    v2 = float(row[i2])
    row[i1] = tmp
    return i1, v1, i2, v2


def run_sequence(cfg, w, prompt, positions):
    max_seq = len(prompt) + cfg.gen_tokens + cfg.c + 8
    o = oracle.Oracle(cfg, w, max_seq)
    o.prefill(prompt, cfg.c)
    steps, stream, margins = [], [], []
    window = None
    for _ in range(N_STEPS):
        # the window the step is fed: after a prefill the refill rule's initial guesses, later the refreshed one
        fed = window if window is not None else np.concatenate(
            [prompt[-1:], [prompt[(j - 1) % len(prompt)] for j in range(1, cfg.c)]]).astype(np.int32)
        k, acc, window, lg = o.jacobi_step(want_logits=True)
        rows = []
        for j in range(cfg.c):
            i1, v1, i2, v2 = top2(lg[j])
            rows.append({"top": [i1, i2], "top_v": [round(v1, 6), round(v2, 6)],
                         "at": [round(float(lg[j, p]), 6) for p in positions]})
            if j < k:
                margins.append(round(v1 - v2, 6))
        stream += acc.tolist()
        steps.append({"window_in": [int(t) for t in fed], "k": int(k), "accepted": acc.tolist(),
                      "window_out": [int(t) for t in window], "rows": rows})
    o.set_window(1)
    while len(stream) < cfg.gen_tokens:
        k, acc, _, lg = o.jacobi_step(want_logits=True)
        _, v1, _, v2 = top2(lg[0])
        stream.append(int(acc[0]))
        margins.append(round(v1 - v2, 6))
    o.close()
    return {"steps": steps, "stream": stream[:cfg.gen_tokens], "margins": margins[:cfg.gen_tokens]}


def main(names):
    for name in names:
        cfg = wl.CONFIGS[name]
        path = os.path.join(HERE, f"stream_{name}.json")
        out = {"config": name, "seed": cfg.seed, "c": cfg.c, "prompt_len": cfg.prompt_len, "batch": cfg.batch,
               "gen_tokens": cfg.gen_tokens, "n_steps": N_STEPS, "kv_bf16": True,
               "note": "written by tests/golden/make_streams.py from the CPU oracle alone", "sequences": []}
        if os.path.exists(path):
            old = json.load(open(path))
            if all(old.get(k) == out[k] for k in ("config", "seed", "c", "prompt_len", "batch", "gen_tokens", "n_steps")):
                out = old
        positions = [int(p) for p in wl.hash_uniform_int(cfg.seed, 11, N_POS, cfg.vocab)]
        out["positions"] = positions
        w = wl.make_weights(cfg)
        ids, lens = wl.make_prompts(cfg)
        for b in range(cfg.batch):
            if b < len(out["sequences"]):
                continue
            t0 = time.time()
            out["sequences"].append(run_sequence(cfg, w, ids[b, :int(lens[b])].numpy(), positions))
            with open(path, "w") as f:
                json.dump(out, f, separators=(",", ":"))
            print(f"{name} sequence {b}: {time.time() - t0:.0f} s", flush=True)


if __name__ == "__main__":
    main(sys.argv[1:] or ["1b", "7b", "13b"])
