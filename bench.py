#!/usr/bin/env python
"""Benchmark of the Jacobi-window decode step: accepted tokens/s and step latency.

    python bench.py --gpus N --steps K --warmup W [--workload 7b] [--impl reference]

One "step" is one fc_jacobi_step: a decoder forward over the K/V-cached prefix plus a window of c
tokens, greedy argmax, verification, K/V commit and window shift.  The default workload is the
7B Llama-shape bf16 model, prompt of 800 random ids, c = 16, batch 1, random-init weights
(synthetic: stands in for the Llama-2 checkpoints and few-shot prompts of the paper's Section 5.1).
The path does not shard: with N > 1 every rank runs an independent replica ("weak" scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2311_08263_b200 import workload as wl  # noqa: E402

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu capture
# summarised under profiles/ (None until a capture of the current kernel exists)
TRAFFIC_BYTES_PER_LAUNCH = {"7b": 415.7e6}     # profiles/gemm_umma_chain_7b_4layers.txt (same shapes per launch)

METRIC = "accepted_tokens_per_s"
UNIT = "tokens/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def step_bytes(cfg, batch, c, kv_lens):
    """Algorithmic bytes of one step: weights once, K/V read + write, embedding rows."""
    s = cfg.elem_bytes
    weights = cfg.weight_params() * s
    kv_tok = cfg.kv_bytes_per_token()
    kv_read = sum((L + c) * kv_tok for L in kv_lens)
    kv_write = batch * c * kv_tok
    return weights + kv_read + kv_write + batch * c * cfg.d_model * s


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self, timed=None):
        """timed: (first, last) sample indices of the device-timed region; sm_mhz is the median over that region
        (over all samples when it holds none), sm_mhz_all the median over warm-up + timed region + end-to-end loop."""
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.t.join(timeout=2)
        sm, sm_timed, mx, reasons = [], [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for i, r in enumerate(self.rows):
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); mx = float(r[1])
            except ValueError:
                continue
            if timed and timed[0] <= i < max(timed[1], timed[0] + 1):
                sm_timed.append(float(r[0]))
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        med_all = statistics.median(sm) if sm else None
        return {"sm_mhz": statistics.median(sm_timed) if sm_timed else med_all, "sm_mhz_all": med_all, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(sm), "samples_timed": len(sm_timed)}


def dist_setup(n_gpus):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl" if torch.cuda.is_available() else "gloo")
    return rank, world, local


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def reduce_max_sum(world, t_ms, tokens, device):
    if world == 1:
        return t_ms, tokens
    import torch.distributed as dist
    a = torch.tensor([t_ms], dtype=torch.float64, device=device)
    b = torch.tensor([tokens], dtype=torch.float64, device=device)
    dist.all_reduce(a, op=dist.ReduceOp.MAX)
    dist.all_reduce(b, op=dist.ReduceOp.SUM)
    return float(a.item()), float(b.item())


# ------------------------------------------------------------------------------------------ CPU oracle leg
def oracle_sample(cfg, weights_host, c, kv_len, reps, layers=None):
    """Times `reps` oracle Jacobi steps (c rows) at K/V length kv_len filled with seeded random K/V.

    This is the one place (besides tests and smoke) where the benchmark touches oracle/.
    Returns (seconds per step, accepted tokens per step, threads used).
    """
    import dataclasses
    import oracle
    ocfg = cfg if layers is None else dataclasses.replace(cfg, n_layers=layers)
    o = oracle.Oracle(ocfg, weights_host, kv_len + c + 8)
    kvd = cfg.n_kv_heads * cfg.head_dim
    kv = wl.hash_normal(cfg.seed, 6, kv_len * kvd).view(kv_len, kvd).numpy()
    for l in range(ocfg.n_layers):
        o.set_kv(l, kv, kv)
    # Jacobi state without a prefill: pending token + prompt-cycled guesses, then the oracle's own
    # forward and accept rule
    prompt = wl.make_prompts(cfg)[0][0].numpy()
    window = np.concatenate([prompt[-1:], prompt[:c - 1]]).astype(np.int32)
    times, acc = [], 0
    for _ in range(reps):
        t0 = time.perf_counter()
        a, _ = o.forward(window, want_logits=False)
        k, _, window2 = oracle.accept(window, a, 0, prompt)
        times.append(time.perf_counter() - t0)
        acc += k
    return sum(times) / len(times), acc / reps, oracle.threads()


def run_reference(args, cfg, rank, world):
    """--impl reference: the CPU oracle, as it stands, on this host's cores (rank 0 only)."""
    if rank != 0:
        return
    L, c = cfg.prompt_len, cfg.c
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    w = wl.make_weights(cfg, device=dev)
    wh = {k: ([t.cpu() for t in v] if isinstance(v, list) else v.cpu()) for k, v in w.items()}
    del w
    # size the per-step sample so the whole run stays within a few minutes
    t_probe, _, threads = oracle_sample(cfg, wh, c, L, 1, layers=1)
    head_frac = cfg.vocab * cfg.d_model / ((cfg.weight_params() - cfg.vocab * cfg.d_model) / cfg.n_layers + cfg.vocab * cfg.d_model)
    t_layer = t_probe * (1 - head_frac)
    t_head = t_probe * head_frac
    budget = 180.0 / max(1, args.steps + args.warmup)
    layers = int(max(1, min(cfg.n_layers, (budget - t_head) / max(t_layer, 1e-9))))
    for _ in range(args.warmup):
        oracle_sample(cfg, wh, c, L, 1, layers=layers)
    t, k, threads = oracle_sample(cfg, wh, c, L, args.steps, layers=layers)
    # a partial-depth sample is scaled to the full depth (cost is linear in layers; the head is counted once)
    t_full = (t - t_head) * cfg.n_layers / layers + t_head if layers < cfg.n_layers else t
    value = k / t_full
    sample = (f"{args.steps} oracle Jacobi steps (c={c}, kv_len={L}, seeded random K/V) over {layers} of "
              f"{cfg.n_layers} layers + LM head" + (", time scaled to full depth" if layers < cfg.n_layers else ""))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_full * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": workload_name(cfg), "batch": 1, "c": c, "kv_len": L},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def workload_name(cfg):
    return (f"{cfg.name} Llama-shape {cfg.dtype}: {cfg.n_layers} layers, d_model {cfg.d_model}, "
            f"{cfg.n_heads}q/{cfg.n_kv_heads}kv heads x {cfg.head_dim}, FFN {cfg.d_ffn}, vocab {cfg.vocab}; "
            f"prompt {cfg.prompt_len} random ids, c={cfg.c}, batch {cfg.batch}")


# ------------------------------------------------------------------------------------------ CUDA leg
def run_ours(args, cfg, rank, world, local):
    from paper_2311_08263_b200 import engine
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    c, B, P = cfg.c, cfg.batch, cfg.prompt_len
    steps, warm = args.steps, args.warmup
    e2e_steps = min(steps, 50)
    max_seq = P + (steps + warm + 2 * e2e_steps + 8) * c + 16

    t0 = time.time()
    w = wl.make_weights(cfg, device=device)
    dec = engine.Decoder(cfg, w, B, c, max_seq, device=str(device))
    ids, lens = wl.make_prompts(cfg, batch=B)
    dec.fc_prefill(ids.numpy(), lens.numpy(), c)         # first call: also loads the kernels
    torch.cuda.synchronize()
    tp = time.perf_counter()
    dec.fc_prefill(ids.numpy(), lens.numpy(), c)         # the prompt cached in blocks of 128 rows per forward
    torch.cuda.synchronize()
    prefill_ms = (time.perf_counter() - tp) * 1e3
    prefill_launches = dec.fc_last_launch_count()
    setup_s = time.time() - t0

    # ---- device-resident timing: K committed steps back to back, CUDA events, max over ranks
    # (the clock sampler runs from the warm-up to the end of the end-to-end loop; the medians are reported per region)
    sampler = ClockSampler(local)
    sampler.start()
    dec.fc_bench_steps(warm, commit=True)
    barrier(world)
    n_warm_samples = len(sampler.rows)
    torch.cuda.synchronize()
    kv0 = dec.fc_get_state()[0].copy()
    ms, tokens = dec.fc_bench_steps(steps, commit=True)
    launches = dec.fc_last_launch_count()
    torch.cuda.synchronize()
    barrier(world)
    kv1 = dec.fc_get_state()[0].copy()
    n_timed_samples = len(sampler.rows)
    ms_max, tok_sum = reduce_max_sum(world, ms, tokens, device)

    # ---- end to end: host window in, host results out, every step (wall clock)
    win = dec.fc_jacobi_step()[2]
    for _ in range(3):
        win = dec.fc_jacobi_step(win)[2]
    barrier(world)
    torch.cuda.synchronize()
    kv_e0 = dec.fc_get_state()[0].copy()
    t1 = time.perf_counter()
    e2e_tok = 0
    for _ in range(e2e_steps):
        cnt, _, win = dec.fc_jacobi_step(win)
        e2e_tok += int(cnt.sum())
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t1
    kv2 = dec.fc_get_state()[0].copy()
    clocks = sampler.stop(timed=(n_warm_samples, n_timed_samples))
    e2e_ms_max, e2e_tok_sum = reduce_max_sum(world, e2e_s * 1e3, e2e_tok, device)

    # ---- per-kernel-class device times (events around every launch of one step)
    prof = dec.fc_profile_step()
    prof = dec.fc_profile_step()
    kv_mid = [int((a + b) // 2) for a, b in zip(kv0, kv1)]
    sbytes = step_bytes(cfg, B, c, kv_mid)
    peak, peak_kind = measured_peaks()
    s = cfg.elem_bytes
    d, f = cfg.d_model, cfg.d_ffn
    qd, kvd = cfg.n_heads * cfg.head_dim, cfg.n_kv_heads * cfg.head_dim
    # dominant kernel: the chained projection launch (O, gate/up, down and the next layer's QKV in one
    # persistent kernel); algorithmic bytes = the weights it streams, once
    L = cfg.n_layers
    chain_ms, chain_n = prof.get("chain", (0.0, 0))
    if chain_n > 0:
        chain_bytes = s * (L * (d * qd + 3 * d * f) + (L - 1) * (qd + 2 * kvd) * d)
        kname = "gemm_umma_kernel<EPI_ATOMIC_ADD> (chained O + gate/up + down + next-QKV projections)"
        k_ms, k_n, k_bytes = chain_ms, chain_n, chain_bytes / chain_n
    else:
        k_ms, k_n = prof["gateup"]
        k_bytes = 2 * d * f * s
        kname = "gemm_umma_kernel<EPI_ATOMIC_ADD> (gate/up projection)"
    achieved = k_bytes * k_n / (k_ms * 1e-3) / 1e9 if k_ms > 0 else 0.0
    roofline = {"bound": "hbm", "kernel": kname,
                "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "peak_kind": f"of {peak_kind}", "traffic": TRAFFIC_BYTES_PER_LAUNCH.get(cfg.name),
                "bytes_per_launch": k_bytes, "ms_per_launch": k_ms / max(k_n, 1), "launches": k_n}
    step_ms = ms_max / steps
    step_gbs = sbytes / (step_ms * 1e-3) / 1e9
    line = {"metric": METRIC, "value": tok_sum / (ms_max * 1e-3), "unit": UNIT, "n_gpus": world, "steps": steps,
            "warmup": warm, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
            "config": {"workload": workload_name(cfg), "batch": B, "c": c, "kv_len_start": int(kv0[0]),
                       "kv_len_end": int(kv1[0]), "l2": "inputs larger than L2 (weights streamed every step)",
                       "multi_gpu": "replicas only"},
            "mean_accept": tok_sum / (steps * B * world),
            "clocks": clocks,
            "ms_x_mhz": step_ms * clocks["sm_mhz"] if clocks.get("sm_mhz") else None,
            "e2e": {"value": e2e_tok_sum / (e2e_ms_max * 1e-3), "unit": UNIT, "steps": e2e_steps,
                    "ms_per_step": e2e_ms_max / e2e_steps, "kv_len_start": int(kv_e0[0]), "kv_len_end": int(kv2[0]),
                    "h2d_bytes_per_step": B * c * 4, "d2h_bytes_per_step": B * (1 + 2 * c) * 4 + 4},
            "gpu_launches": launches,
            "prefill": {"ms": round(prefill_ms, 3), "prompt_len": P, "batch": B, "rows_per_forward": 128,
                        "forwards_per_sequence": (P - 1 + 127) // 128, "launches": prefill_launches,
                        "note": "wall clock of fc_prefill (host buffers in, synchronised), not part of the timed steps"},
            "roofline": roofline,
            "step_roofline": {"bytes_per_step": sbytes, "achieved_gbs": step_gbs, "frac_of_peak": step_gbs / peak,
                              "peak_gbs": peak, "peak_kind": peak_kind, "frac_of_8tbs": step_gbs / 8000.0},
            "kernel_ms": {k: round(v[0], 4) for k, v in prof.items()},
            "kernel_launches": {k: v[1] for k, v in prof.items()},
            "setup_s": round(setup_s, 1)}

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        wh = {k: ([t.cpu() for t in v] if isinstance(v, list) else v.cpu()) for k, v in w.items()}
        del dec
        t_probe, _, threads = oracle_sample(cfg, wh, c, P, 1, layers=1)
        layers = int(max(1, min(cfg.n_layers, 20.0 / max(t_probe, 1e-9))))
        t, k, threads = oracle_sample(cfg, wh, c, P, 1, layers=layers)
        head_frac = cfg.vocab * d / ((cfg.weight_params() - cfg.vocab * d) / cfg.n_layers + cfg.vocab * d)
        t_head = t_probe * head_frac
        t_full = (t - t_head) * cfg.n_layers / layers + t_head if layers < cfg.n_layers else t
        line["cpu_baseline"] = {"value": k / t_full, "unit": UNIT, "cores": threads, "kind": "oracle",
                                "sample": f"1 oracle Jacobi step (c={c}, kv_len={P}, seeded random K/V) over "
                                          f"{layers} of {cfg.n_layers} layers + LM head"
                                          + (", time scaled to full depth" if layers < cfg.n_layers else ""),
                                "ms_per_step": t_full * 1e3}
    if rank == 0:
        print(json.dumps(line), flush=True)


def run_sweep(args, cfg):
    """Window-step sweep (the paper's Fig. 2 experiment: forward time against window size and prompt length):
    K/V length x window rows x batch on one model shape, random weights, seeded random K/V ~ N(0,1) written
    straight into the cache, steps that do not commit so every step runs at the same length.  One JSON line per
    point: latency, algorithmic bytes and flops, fraction of the HBM roofline."""
    from paper_2311_08263_b200 import engine
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(0)
    peak, peak_kind = measured_peaks()
    w = wl.make_weights(cfg, device="cuda")
    lens = [int(x) for x in args.sweep_lens.split(",")]
    cs = [int(x) for x in args.sweep_c.split(",")]
    bs = [int(x) for x in args.sweep_batch.split(",")]
    g = torch.Generator(device="cuda")
    for L in lens:
        for B in bs:
            max_c = max(cs)
            max_seq = L + max_c + 8
            need = cfg.kv_bytes_per_token() * max_seq * B * 1.02 + 6e9
            free, _ = torch.cuda.mem_get_info()
            if need > free:
                for c in cs:
                    print(json.dumps({"sweep": cfg.name, "kv_len": L, "c": c, "batch": B, "skipped": "does not fit in device memory"}), flush=True)
                continue
            dec = engine.Decoder(cfg, w, B, max_c, max_seq)
            g.manual_seed(cfg.seed + L + B)
            kv = dec.kv.view(cfg.torch_dtype)
            for i in range(0, kv.numel(), 1 << 30):
                kv[i:i + (1 << 30)].normal_(generator=g)
            for c in cs:
                pending = wl.make_random_window(cfg, B, 1, salt=c).numpy()[:, 0]
                dec.fc_debug_set_state([L] * B, pending, c, pad_id=1)
                ms1, _ = dec.fc_bench_steps(2)
                n = int(max(3, min(50, 300.0 / max(ms1 / 2, 0.05))))
                ms, _ = dec.fc_bench_steps(n)
                step_ms = ms / n
                by = step_bytes(cfg, B, c, [L] * B)
                R = B * c
                flops = 2.0 * R * cfg.weight_params() + 4.0 * cfg.n_layers * cfg.n_heads * cfg.head_dim * B * c * (L + c / 2)
                gbs = by / (step_ms * 1e-3) / 1e9
                print(json.dumps({"sweep": cfg.name, "kv_len": L, "c": c, "batch": B, "rows": R, "ms_per_step": round(step_ms, 4),
                                  "bytes_per_step": by, "flops_per_step": flops, "achieved_gbs": round(gbs, 1),
                                  "frac_of_peak": round(gbs / peak, 4), "peak_kind": peak_kind,
                                  "frac_of_8tbs": round(gbs / 8000.0, 4),
                                  "achieved_tflops": round(flops / (step_ms * 1e-3) / 1e12, 2), "steps": n}), flush=True)
            dec.close()
            del dec, kv
            torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="7b", choices=sorted(wl.CONFIGS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layers", type=int, default=0,
                    help="profiling aid: keep only the first N layers (same kernel shapes, less device memory)")
    ap.add_argument("--sweep", action="store_true", help="window-step sweep instead of the benchmark line")
    ap.add_argument("--sweep-lens", default="512,2048,8192")
    ap.add_argument("--sweep-c", default="1,4,8,16,32,64")
    ap.add_argument("--sweep-batch", default="1,4,16,32")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    cfg = wl.CONFIGS[args.workload]
    if args.layers > 0:
        import dataclasses
        cfg = dataclasses.replace(cfg, n_layers=args.layers, name=f"{cfg.name}-first{args.layers}layers")
    if args.sweep:
        run_sweep(args, cfg)
        return
    rank, world, local = dist_setup(args.gpus)
    if args.impl == "reference":
        run_reference(args, cfg, rank, world)
    else:
        run_ours(args, cfg, rank, world, local)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
