"""Parity at the full model shapes, in the launch configuration the benchmark times.

The oracle cannot replay whole runs at these sizes in test time, so each case compares sampled outputs
the oracle can compute one by one: the logits, accepted tokens and refreshed window of Jacobi steps, and
(1.1B) a stretch of the committed stream from a real prefill.  For the 7B and 13B shapes the cache is filled
with seeded random K/V (the recipe of the window-step sweep) instead of a prefill, identically on both sides.
"""
import numpy as np
import psutil
import pytest
import torch

import oracle
from paper_2311_08263_b200 import engine, workload as wl

pytestmark = pytest.mark.gpu

LOGIT_TOL = 3e-2
MARGIN_TOL = 0.05
# K and V are bf16 on both sides.  Two implementations whose fp32 values differ at the 1e-6 level put about one K/V
# element in a thousand on different sides of a bf16 rounding boundary (measured at layer 0); each such element
# is off by a whole bf16 step (0.4-0.8 %), the next layer's K/V inherit that, and by layer 2 several per cent of
# the window's K/V elements differ by one step.  The logit difference therefore grows with depth: measured
# max-abs 4.5e-3 at 8 layers, below 3e-2 at 22 and 32 layers, 4.3e-2 at 40 layers (rms up to 8e-3 for the sequences with almost no cache).  The 40-layer case
# is held to twice the bar and to the rms; its argmax/accept parity is still exact wherever the margin allows.
LOGIT_TOL_40_LAYERS = 6e-2
LOGIT_RMS_TOL = 1.5e-2


def _host_weights(w):
    return {k: ([t.cpu() for t in v] if isinstance(v, list) else v.cpu()) for k, v in w.items()}


def _need(gpu_gb, host_gb):
    free, _ = torch.cuda.mem_get_info()
    if free < gpu_gb * 2**30:
        pytest.skip(f"needs {gpu_gb} GB of device memory")
    if psutil.virtual_memory().available < host_gb * 2**30:
        pytest.skip(f"needs {host_gb} GB of host memory for the oracle's copy of the weights")


def _check_step(cfg, lg_gpu, lg_ref, cnt, tok, win, k_ref, acc_ref, win_ref):
    err = np.abs(lg_gpu - lg_ref)
    assert err.max() < (LOGIT_TOL if cfg.n_layers <= 32 else LOGIT_TOL_40_LAYERS)
    assert np.sqrt((err ** 2).mean()) < LOGIT_RMS_TOL
    srt = np.sort(lg_ref, axis=1)
    if (srt[:, -1] - srt[:, -2]).min() > MARGIN_TOL:      # otherwise a different argmax is tolerated
        assert cnt == k_ref and tok[:cnt].tolist() == acc_ref.tolist() and win.tolist() == win_ref.tolist()
        return True
    return False


def test_1b_prefill_steps_and_stream():
    cfg = wl.CONFIGS["1b"]
    _need(8, 8)
    w = wl.make_weights(cfg, device="cuda")
    wh = _host_weights(w)
    prompt = wl.make_prompts(cfg)[0][0].numpy()
    max_seq = cfg.prompt_len + 64 + cfg.c + 8
    dec = engine.Decoder(cfg, w, 1, cfg.c, max_seq)
    o = oracle.Oracle(cfg, wh, max_seq)
    o.prefill(prompt, cfg.c)
    dec.fc_prefill(prompt, [len(prompt)], cfg.c)
    logits = dec.fc_debug_logits(True)
    for _ in range(2):
        k, acc, wnew, lg = o.jacobi_step(want_logits=True)
        cnt, tok, win = dec.fc_jacobi_step()
        if not _check_step(cfg, logits[:cfg.c].cpu().numpy(), lg, cnt[0], tok[0], win[0], k, acc, wnew):
            break
    dec.fc_debug_logits(False)
    # committed stream from a fresh prefill against the oracle's greedy stream
    n = 40
    ar, margins = oracle.Oracle(cfg, wh, max_seq).ar_generate(prompt, n)
    dec.fc_prefill(prompt, [len(prompt)], cfg.c)
    toks, lens, st = dec.fc_generate(n)
    got = toks[0, :lens[0]]
    diff = np.nonzero(got != ar)[0]
    if len(diff):
        assert margins[diff[0]] < MARGIN_TOL
    assert lens[0] == n and st.tokens == n


def _random_kv_case(cfg, lens, c, seqs_to_check):
    """Seeded random K/V of ragged lengths on both sides, then one Jacobi step compared per sequence."""
    B = len(lens)
    w = wl.make_weights(cfg, device="cuda")
    wh = _host_weights(w)
    max_seq = max(lens) + c + 8
    dec = engine.Decoder(cfg, w, B, c, max_seq)
    kvd = cfg.n_kv_heads * cfg.head_dim
    view = dec.kv_view()                       # [layer, K|V, B, kv_head, max_seq, head_dim]
    for b, L in enumerate(lens):
        for l in range(cfg.n_layers):
            kv = wl.make_random_kv(cfg, 2 * L * kvd, device="cuda", tensor_id=1000 + 64 * b + l)
            kv = kv.view(2, L, cfg.n_kv_heads, cfg.head_dim).permute(0, 2, 1, 3)
            view[l, :, b, :, :L, :] = kv
    pending = wl.make_random_window(cfg, B, 1, salt=3).numpy()[:, 0]
    window = wl.make_random_window(cfg, B, c, salt=4).numpy()
    window[:, 0] = pending
    dec.fc_debug_set_state(lens, pending, c, pad_id=0)
    logits = dec.fc_debug_logits(True)
    cnt, tok, win = dec.fc_jacobi_step(window)
    lg_all = logits[:B * c].cpu().numpy().reshape(B, c, cfg.vocab)
    prompt = np.array([0], np.int32)           # refill is the pad id on both sides
    for b in seqs_to_check:
        L = lens[b]
        o = oracle.Oracle(cfg, wh, L + c + 8)
        for l in range(cfg.n_layers):
            kv = view[l, :, b, :, :L, :].float().permute(0, 2, 1, 3).reshape(2, L, kvd).cpu().numpy()
            o.set_kv(l, kv[0], kv[1])
        am, lg = o.forward(window[b])
        k_ref, acc_ref, win_ref = oracle.accept(window[b], am, 0, prompt, refill=1, pad_id=0)
        _check_step(cfg, lg_all[b], lg, cnt[b], tok[b], win[b], k_ref, acc_ref, win_ref)
        o.close()
    return dec


def test_7b_step_at_bench_configuration():
    cfg = wl.CONFIGS["7b"]
    _need(20, 22)
    dec = _random_kv_case(cfg, [cfg.prompt_len], cfg.c, [0])
    # the step the benchmark times launches 2 * layers + 4 kernels
    assert dec.fc_last_launch_count() == 2 * cfg.n_layers + 4


def test_13b_batch8_ragged_step():
    cfg = wl.CONFIGS["13b"]
    _need(45, 40)
    lens = [1024, 700, 1000, 513, 1024, 64, 900, 1]
    _random_kv_case(cfg, lens, cfg.c, [1, 5, 7])


@pytest.mark.parametrize("hd,heads,kv_heads", [(64, 8, 8), (128, 4, 4), (64, 8, 2)])
def test_long_ragged_caches_several_chunks_per_cta(hd, heads, kv_heads):
    """Long caches in a batch: more 128-key chunks than the GPU holds CTAs, so one CTA walks over several
    consecutive chunks with running softmax statistics (ragged lengths: CTAs with fewer live chunks, with
    none, and with the window's own keys in their last chunk; with grouped queries there are two 16-row query
    tiles per kv head, each with CTAs of its own)."""
    cfg = wl.small_config(vocab=500, n_layers=2, n_heads=heads, n_kv_heads=kv_heads, head_dim=hd, d_model=512,
                          d_ffn=512, c=8, prompt_len=64, gen_tokens=8)
    lens = [6000, 4100, 129, 5000, 1, 3333, 6000, 2047, 640, 5990]
    _random_kv_case(cfg, lens, cfg.c, [0, 1, 2, 4, 7, 9])
