"""End-to-end parity of the CUDA decode path (through the C ABI) with the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2311_08263_b200 import engine, lib, workload as wl

pytestmark = pytest.mark.gpu

LOGIT_TOL = 3e-2      # max-abs logit difference allowed for bf16 configurations
MARGIN_TOL = 0.05     # streams may differ only where the oracle's top-1/top-2 margin is below this


def _setup(cfg, max_batch=1, max_c=None, max_seq=None, flags=0):
    w = wl.make_weights(cfg)
    max_c = max_c or cfg.c
    max_seq = max_seq or (cfg.prompt_len + cfg.gen_tokens + max_c + 8)
    dec = engine.Decoder(cfg, w, max_batch, max_c, max_seq, flags=flags)
    return w, dec, max_seq


# ------------------------------------------------------------------ fp32 configuration: bit-exact stream
@pytest.mark.parametrize("c", [1, 3, 8])
@pytest.mark.parametrize("refill", [0, 1])
def test_tiny_fp32_stream_and_accept_counts_exact(c, refill):
    cfg = wl.CONFIGS["tiny"]
    w, dec, max_seq = _setup(cfg, max_c=8)
    prompt = wl.make_prompts(cfg)[0][0].numpy()
    o = oracle.Oracle(cfg, w, max_seq)
    o.prefill(prompt, c, refill=refill, pad_id=3)
    want, want_counts = o.generate(cfg.gen_tokens)
    dec.fc_prefill(prompt, [len(prompt)], c, refill=refill, pad_id=3)
    toks, lens, st = dec.fc_generate(cfg.gen_tokens)
    assert lens[0] == cfg.gen_tokens
    assert toks[0].tolist() == want.tolist()
    assert st.steps == len(want_counts)
    hist = np.bincount(want_counts, minlength=65)
    assert list(st.accept_hist)[:65] == hist.tolist()
    assert dec.fc_last_launch_count() > 0


def test_tiny_fp32_stepwise_matches_oracle_every_step():
    cfg = wl.CONFIGS["tiny"]
    w, dec, max_seq = _setup(cfg)
    prompt = wl.make_prompts(cfg)[0][0].numpy()
    o = oracle.Oracle(cfg, w, max_seq)
    o.prefill(prompt, cfg.c)
    dec.fc_prefill(prompt, [len(prompt)], cfg.c)
    logits = dec.fc_debug_logits(True)
    for _ in range(12):
        k, acc, wnew, lg = o.jacobi_step(want_logits=True)
        cnt, tok, win = dec.fc_jacobi_step()
        assert cnt[0] == k and tok[0, :k].tolist() == acc.tolist() and win[0].tolist() == wnew.tolist()
        got = logits[:cfg.c].cpu().numpy()
        assert np.abs(got - lg).max() < 2e-4
    kl, ng = dec.fc_get_state()
    assert kl[0] == o.kv_len and ng[0] == o.n_gen


@pytest.mark.parametrize("c", [2, 5, 8])
def test_directed_accept_counts_through_window_in(c):
    """Prime the window with m correct continuation tokens then a wrong one: k must be m + 1."""
    cfg = wl.CONFIGS["tiny"]
    w, dec, max_seq = _setup(cfg, max_c=8)
    prompt = wl.make_prompts(cfg)[0][0].numpy()
    o = oracle.Oracle(cfg, w, max_seq)
    ar, _ = o.ar_generate(prompt, 40)
    for m in range(c):
        o.prefill(prompt, c)
        dec.fc_prefill(prompt, [len(prompt)], c)
        n = 0
        for _ in range(2):
            k, _, wo = o.jacobi_step()
            cnt, _, wg = dec.fc_jacobi_step()
            assert cnt[0] == k and wg[0].tolist() == wo.tolist()
            n += k
        win = wo.copy()
        win[1:1 + m] = ar[n:n + m]
        if 1 + m < c:
            win[1 + m] = (ar[n + m] + 1) % cfg.vocab
        k, acc, w2 = o.jacobi_step(win)
        cnt, tok, wg = dec.fc_jacobi_step(win[None])
        assert k == m + 1 and cnt[0] == k
        assert tok[0, :k].tolist() == acc.tolist() == ar[n:n + k].tolist()
        assert wg[0].tolist() == w2.tolist()


# ------------------------------------------------------------------ bf16: tolerance rule with re-synchronisation
def _compare_stream_with_resync(cfg, w, dec, prompt, c, n_tokens, max_seq):
    """Generate on the GPU; wherever the GPU stream leaves the oracle's greedy stream, the oracle's
    top-1/top-2 margin at that position must be below MARGIN_TOL; then restart both from the oracle's
    prefix and go on.  Returns the number of tolerated positions."""
    o = oracle.Oracle(cfg, w, max_seq)
    ar, margins = o.ar_generate(prompt, n_tokens)
    tolerated, pos = 0, 0
    cur = list(prompt)
    while pos < n_tokens:
        dec.fc_prefill(np.array(cur, np.int32), [len(cur)], c)
        toks, lens, _ = dec.fc_generate(n_tokens - pos)
        got = toks[0, :lens[0]]
        want = ar[pos:]
        diff = np.nonzero(got != want)[0]
        if len(diff) == 0:
            break
        i = int(diff[0])
        assert margins[pos + i] < MARGIN_TOL, (pos + i, margins[pos + i], got[i], want[i])
        tolerated += 1
        pos += i + 1
        cur = list(prompt) + ar[:pos].tolist()
    return tolerated


@pytest.mark.parametrize("flags", [lib.FC_FLAG_SIMT_GEMM, 0, lib.FC_FLAG_NO_PDL | lib.FC_FLAG_NO_CHAIN,
                                   lib.FC_FLAG_NO_FFN_SPLIT],
                         ids=["fma", "tensor", "tensor-unchained", "tensor-ffn-unsplit"])
@pytest.mark.parametrize("shape", ["gqa64", "mha128", "gqa32"])
def test_small_bf16_logits_and_stream(flags, shape):
    kw = {"gqa64": dict(n_heads=4, n_kv_heads=2, head_dim=64, d_model=256, d_ffn=512),
          "mha128": dict(n_heads=2, n_kv_heads=2, head_dim=128, d_model=256, d_ffn=640),
          "gqa32": dict(n_heads=8, n_kv_heads=2, head_dim=32, d_model=320, d_ffn=328)}[shape]
    cfg = wl.small_config(vocab=1000, n_layers=3, prompt_len=150, c=8, gen_tokens=24, **kw)
    w, dec, max_seq = _setup(cfg, flags=flags)
    prompt = wl.make_prompts(cfg)[0][0].numpy()
    o = oracle.Oracle(cfg, w, max_seq)
    o.prefill(prompt, cfg.c)
    dec.fc_prefill(prompt, [len(prompt)], cfg.c)
    logits = dec.fc_debug_logits(True)
    for _ in range(3):
        k, acc, wnew, lg = o.jacobi_step(want_logits=True)
        cnt, tok, wg = dec.fc_jacobi_step()
        got = logits[:cfg.c].cpu().numpy()
        assert np.abs(got - lg).max() < LOGIT_TOL
        srt = np.sort(lg, axis=1)
        if (srt[:, -1] - srt[:, -2]).min() > MARGIN_TOL:
            assert cnt[0] == k and tok[0, :k].tolist() == acc.tolist() and wg[0].tolist() == wnew.tolist()
        else:
            break
    dec.fc_debug_logits(False)
    _compare_stream_with_resync(cfg, w, dec, prompt, cfg.c, cfg.gen_tokens, max_seq)


@pytest.mark.parametrize("c", [1, 2, 16])
def test_bf16_window_sizes_one_and_sixteen(c):
    """c = 1 is plain autoregressive decoding through the tensor-core path (one live row in the 16-row
    accumulator); c = 16 fills it.  Four layers, so that the chained launch runs with and without a next QKV."""
    cfg = wl.small_config(vocab=800, n_layers=4, prompt_len=140, c=c, gen_tokens=12,
                          n_heads=4, n_kv_heads=4, head_dim=128, d_model=512, d_ffn=768)
    w, dec, max_seq = _setup(cfg)
    prompt = wl.make_prompts(cfg)[0][0].numpy()
    o = oracle.Oracle(cfg, w, max_seq)
    o.prefill(prompt, c)
    dec.fc_prefill(prompt, [len(prompt)], c)
    logits = dec.fc_debug_logits(True)
    for _ in range(3):
        k, acc, wnew, lg = o.jacobi_step(want_logits=True)
        cnt, tok, wg = dec.fc_jacobi_step()
        assert np.abs(logits[:c].cpu().numpy() - lg).max() < LOGIT_TOL
        srt = np.sort(lg, axis=1)
        if (srt[:, -1] - srt[:, -2]).min() > MARGIN_TOL:
            assert cnt[0] == k and tok[0, :k].tolist() == acc.tolist() and wg[0].tolist() == wnew.tolist()
        else:
            break
    dec.fc_debug_logits(False)
    _compare_stream_with_resync(cfg, w, dec, prompt, c, cfg.gen_tokens, max_seq)


def test_batch_ragged_prompts_independent_accepts():
    cfg = wl.small_config(vocab=600, n_layers=2, n_heads=4, n_kv_heads=2, head_dim=64, d_model=256, d_ffn=512,
                          prompt_len=70, c=6, gen_tokens=20)
    B = 4
    lens = [70, 33, 1, 50]
    w = wl.make_weights(cfg)
    max_seq = 70 + 20 + 6 + 8
    dec = engine.Decoder(cfg, w, B, cfg.c, max_seq)
    ids, lens_t = wl.make_prompts(cfg, batch=B, lens=lens)
    dec.fc_prefill(ids.numpy(), lens, cfg.c)
    toks, out_lens, st = dec.fc_generate(cfg.gen_tokens)
    for b in range(B):
        o = oracle.Oracle(cfg, w, max_seq)
        ar, margins = o.ar_generate(ids[b, :lens[b]].numpy(), cfg.gen_tokens)
        got = toks[b, :out_lens[b]]
        assert out_lens[b] == cfg.gen_tokens
        diff = np.nonzero(got != ar)[0]
        if len(diff):
            assert margins[diff[0]] < MARGIN_TOL
    assert st.tokens == B * cfg.gen_tokens


@pytest.mark.parametrize("B,c", [(3, 8), (4, 12), (6, 16), (10, 16), (1, 64), (3, 33)],
                         ids=["rows24", "rows48", "rows96", "rows160", "c64", "c33x3"])
@pytest.mark.parametrize("shape", ["gqa64", "gqa32", "mha64", "mha64-single-cta-tiles"])
def test_many_rows_prefill_and_steps(B, c, shape):
    """More than 16 rows per forward: the projections read their activations from the converted panel, for
    every accumulator width (32, 64, 128 rows) and for two blocks of rows; the prefill runs through the same path.
    gqa32 has k extents that are not multiples of 256, so a group of conversion units spans two rows.  In mha64 every
    weight matrix of a layer is a whole number of 256-row tiles, so beyond 64 rows the projections run as pairs of
    CTAs per tile (tcgen05 cta_group::2); the last shape runs the same model with that switched off."""
    kw = {"gqa64": dict(n_heads=4, n_kv_heads=2, head_dim=64, d_model=256, d_ffn=512),
          "gqa32": dict(n_heads=8, n_kv_heads=2, head_dim=32, d_model=320, d_ffn=328),
          "mha64": dict(n_heads=4, n_kv_heads=4, head_dim=64, d_model=256, d_ffn=512)}[shape.split("-")[0]]
    cfg = wl.small_config(vocab=700, n_layers=2, prompt_len=200, c=c, gen_tokens=12, **kw)
    lens = [200 - 17 * b for b in range(B)]
    w = wl.make_weights(cfg)
    max_seq = 200 + 12 + c + 8
    dec = engine.Decoder(cfg, w, B, c, max_seq, flags=lib.FC_FLAG_NO_CTA_PAIRS if shape.endswith("tiles") else 0)
    ids, _ = wl.make_prompts(cfg, batch=B, lens=lens)
    dec.fc_prefill(ids.numpy(), lens, c)
    logits = dec.fc_debug_logits(True)
    orcs = []
    for b in range(B):
        o = oracle.Oracle(cfg, w, max_seq)
        o.prefill(ids[b, :lens[b]].numpy(), c)
        orcs.append(o)
    in_step = True
    for _ in range(2):
        cnt, tok, wg = dec.fc_jacobi_step()
        got = logits[:B * c].cpu().numpy().reshape(B, c, cfg.vocab)
        for b in range(B):
            k, acc, wnew, lg = orcs[b].jacobi_step(want_logits=True)
            assert np.abs(got[b] - lg).max() < LOGIT_TOL
            srt = np.sort(lg, axis=1)
            if (srt[:, -1] - srt[:, -2]).min() > MARGIN_TOL:
                assert cnt[b] == k and tok[b, :k].tolist() == acc.tolist() and wg[b].tolist() == wnew.tolist()
            else:
                in_step = False
        if not in_step:
            break


def test_directed_accepts_in_a_batch_are_per_sequence():
    cfg = wl.CONFIGS["tiny"]
    B, c = 3, 6
    w = wl.make_weights(cfg)
    max_seq = 128
    dec = engine.Decoder(cfg, w, B, c, max_seq)
    ids, _ = wl.make_prompts(cfg, batch=B, lens=[32, 20, 27])
    lens = [32, 20, 27]
    dec.fc_prefill(ids.numpy(), lens, c)
    wins, ks = [], []
    for b in range(B):
        o = oracle.Oracle(cfg, w, max_seq)
        ar, _ = o.ar_generate(ids[b, :lens[b]].numpy(), 10)
        m = [0, 3, 5][b]
        win = np.zeros(c, np.int32)
        win[0] = ids[b, lens[b] - 1]
        win[1:1 + m] = ar[:m]
        if 1 + m < c:
            win[1 + m] = (ar[m] + 1) % cfg.vocab
        wins.append(win); ks.append((m + 1, ar))
    cnt, tok, _ = dec.fc_jacobi_step(np.stack(wins))
    for b in range(B):
        k, ar = ks[b]
        assert cnt[b] == k and tok[b, :k].tolist() == ar[:k].tolist()


def test_eos_and_max_tokens_truncation():
    cfg = wl.CONFIGS["tiny"]
    w, dec, max_seq = _setup(cfg)
    prompt = wl.make_prompts(cfg)[0][0].numpy()
    o = oracle.Oracle(cfg, w, max_seq)
    ar, _ = o.ar_generate(prompt, 30)
    eos = int(ar[12])
    first = int(np.where(ar == eos)[0][0])
    dec.fc_prefill(prompt, [len(prompt)], cfg.c)
    toks, lens, _ = dec.fc_generate(30, eos_id=eos)
    assert toks[0, :lens[0]].tolist() == ar[:first + 1].tolist()


def test_error_codes():
    cfg = wl.CONFIGS["tiny"]
    w, dec, max_seq = _setup(cfg, max_seq=64)
    prompt = wl.make_prompts(cfg)[0][0].numpy()
    with pytest.raises(engine.FcError) as e:
        dec.batch, dec.c = 1, 8
        dec.fc_jacobi_step()
    assert e.value.code == lib.FC_ERR_STATE
    bad = prompt.copy(); bad[3] = cfg.vocab
    with pytest.raises(engine.FcError) as e:
        dec.fc_prefill(bad, [len(bad)], 8)
    assert e.value.code == lib.FC_ERR_TOKEN_RANGE
    with pytest.raises(engine.FcError) as e:
        dec.fc_prefill(prompt, [len(prompt)], 9)
    assert e.value.code == lib.FC_ERR_CAPACITY
    dec.fc_prefill(prompt, [len(prompt)], 8)
    win = np.zeros((1, 8), np.int32); win[0, 0] = (prompt[-1] + 1) % cfg.vocab
    with pytest.raises(engine.FcError) as e:
        dec.fc_jacobi_step(win)
    assert e.value.code == lib.FC_ERR_BAD_WINDOW
    with pytest.raises(engine.FcError) as e:
        dec.fc_generate(64)           # 31 + 64 + 8 > max_seq
    assert e.value.code == lib.FC_ERR_CAPACITY
    # the failed calls left the state usable
    cnt, _, _ = dec.fc_jacobi_step()
    assert cnt[0] >= 1


# ------------------------------------------------------------------ robustness aids in place of a memory checker
def test_injected_device_timeout_is_reported_and_prefill_recovers():
    """The accept kernel raises the device error word (no wait involved): the step must return
    FC_ERR_DEVICE_TIMEOUT, further steps must be refused until fc_prefill, and after it the stream is exact again."""
    cfg = wl.CONFIGS["tiny"]
    w, dec, max_seq = _setup(cfg)
    prompt = wl.make_prompts(cfg)[0][0].numpy()
    o = oracle.Oracle(cfg, w, max_seq)
    o.prefill(prompt, cfg.c)
    want, _ = o.generate(16)
    dec.fc_prefill(prompt, [len(prompt)], cfg.c)
    dec.fc_jacobi_step()
    dec.fc_debug_inject_timeout()
    with pytest.raises(engine.FcError) as e:
        dec.fc_jacobi_step()
    assert e.value.code == lib.FC_ERR_DEVICE_TIMEOUT
    with pytest.raises(engine.FcError) as e:
        dec.fc_jacobi_step()
    assert e.value.code == lib.FC_ERR_STATE
    dec.fc_prefill(prompt, [len(prompt)], cfg.c)
    toks, lens, _ = dec.fc_generate(16)
    assert toks[0, :lens[0]].tolist() == want.tolist()
    assert dec.fc_debug_check_guards() == 0


@pytest.mark.parametrize("which", ["tiny", "bf16-batch"])
def test_canary_bands_intact_after_prefill_steps_and_generate(which):
    """Canary bands around the K/V slab, around the workspace and between its slices must hold their pattern after
    every kind of call (the stand-in for an out-of-bounds checker); damaging one on purpose from the host is seen."""
    if which == "tiny":
        cfg, B, c = wl.CONFIGS["tiny"], 1, 8
    else:
        cfg, B, c = wl.small_config(vocab=600, n_layers=2, n_heads=4, n_kv_heads=2, head_dim=64, d_model=256,
                                    d_ffn=512, prompt_len=150, c=12, gen_tokens=20), 3, 12
    w = wl.make_weights(cfg)
    max_seq = 150 + 40 + c + 8
    dec = engine.Decoder(cfg, w, B, c, max_seq)
    assert dec.fc_debug_check_guards() == 0
    lens = [min(cfg.prompt_len, 150) - 11 * b for b in range(B)]
    ids, _ = wl.make_prompts(cfg, batch=B, lens=lens)
    dec.fc_prefill(ids.numpy(), lens, c)
    assert dec.fc_debug_check_guards() == 0
    for _ in range(3):
        dec.fc_jacobi_step()
    dec.fc_generate(20)
    dec.fc_bench_steps(2, commit=False)
    dec.fc_profile_step()
    assert dec.fc_debug_check_guards() == 0
    dec._ws_alloc[10] = 0                    # damage the band in front of the workspace from the host
    assert dec.fc_debug_check_guards() == 1


# ------------------------------------------------------------------ window resize, iteration cap, continuation
@pytest.mark.parametrize("sizes", [(8, 3, 6, 1, 5), (1, 8, 2)])
def test_window_resize_between_iterations_matches_oracle(sizes):
    cfg = wl.CONFIGS["tiny"]
    w, dec, max_seq = _setup(cfg, max_c=8, max_seq=200)
    prompt = wl.make_prompts(cfg)[0][0].numpy()
    o = oracle.Oracle(cfg, w, 200)
    o.prefill(prompt, sizes[0])
    dec.fc_prefill(prompt, [len(prompt)], sizes[0])
    for i in range(20):
        k, acc, wnew = o.jacobi_step()
        cnt, tok, win = dec.fc_jacobi_step()
        assert cnt[0] == k and tok[0, :k].tolist() == acc.tolist() and win[0].tolist() == wnew.tolist()
        c_new = sizes[(i + 1) % len(sizes)]
        o.set_window(c_new)
        dec.fc_set_window(c_new)
    with pytest.raises(engine.FcError) as e:
        dec.fc_set_window(9)
    assert e.value.code == lib.FC_ERR_CAPACITY


def test_generate_with_window_argument_iteration_cap_and_continuation():
    cfg = wl.CONFIGS["tiny"]
    w, dec, max_seq = _setup(cfg, max_c=8, max_seq=200)
    prompt = wl.make_prompts(cfg)[0][0].numpy()
    o = oracle.Oracle(cfg, w, 200)
    o.prefill(prompt, 8)
    dec.fc_prefill(prompt, [len(prompt)], 8)
    # iteration cap: exactly 5 forwards, a prefix of the stream
    want, counts = o.generate(40, max_iters=5)
    toks, lens, st = dec.fc_generate(40, max_iters=5)
    assert st.steps == 5 and toks[0, :lens[0]].tolist() == want.tolist()
    # go on with another window size and a token limit, then raise the limit: the second call continues
    o.set_window(4)
    want2, _ = o.generate(24 - len(want))
    toks2, lens2, st2 = dec.fc_generate(24, c=4)
    assert toks2[0, :lens2[0]].tolist() == want2.tolist() and len(want) + lens2[0] == 24
    want3, _ = o.generate(40 - 24)
    toks3, lens3, _ = dec.fc_generate(40)
    assert toks3[0, :lens3[0]].tolist() == want3.tolist() and lens3[0] == 16
    # nothing left to do at the same limit
    toks4, lens4, st4 = dec.fc_generate(40)
    assert lens4[0] == 0 and st4.steps == 0
    assert st.ms_prefill > 0


# ------------------------------------------------------------------ answer trigger hand-off
@pytest.mark.parametrize("n_trig,c", [(0, 1), (3, 6), (5, 8)])
def test_finish_with_trigger_fp32_exact(n_trig, c):
    cfg = wl.CONFIGS["tiny"]
    w, dec, max_seq = _setup(cfg, max_c=8, max_seq=200)
    prompt = wl.make_prompts(cfg)[0][0].numpy()
    trigger = wl.hash_uniform_int(5, 9, max(n_trig, 1), cfg.vocab).numpy()[:n_trig]
    o = oracle.Oracle(cfg, w, 200)
    o.prefill(prompt, c)
    o.generate(12, max_iters=4)
    dec.fc_prefill(prompt, [len(prompt)], c)
    dec.fc_generate(12, max_iters=4)
    want = o.finish_with_trigger(trigger, 10)
    got, lens = dec.fc_finish_with_trigger(trigger, 10)
    assert got[0, :lens[0]].tolist() == want.tolist()
    with pytest.raises(engine.FcError) as e:
        dec.fc_jacobi_step()
    assert e.value.code == lib.FC_ERR_STATE
    assert dec.fc_debug_check_guards() == 0


def test_finish_with_trigger_bf16_batch_ragged_with_eos():
    """Three sequences of different lengths on the tensor-core path: each answer equals the oracle's, or leaves it
    only at a position whose margin in the oracle's greedy run over the same context is below the tolerance."""
    cfg = wl.small_config(vocab=600, n_layers=2, n_heads=4, n_kv_heads=2, head_dim=64, d_model=256, d_ffn=512,
                          prompt_len=70, c=6, gen_tokens=20)
    B, lens = 3, [70, 33, 5]
    w = wl.make_weights(cfg)
    max_seq = 70 + 8 + 6 + 4 + 16 + 8
    dec = engine.Decoder(cfg, w, B, cfg.c, max_seq)
    ids, _ = wl.make_prompts(cfg, batch=B, lens=lens)
    trigger = np.array([11, 22, 33, 44], np.int32)
    dec.fc_prefill(ids.numpy(), lens, cfg.c)
    dec.fc_generate(8)
    wins = dec.fc_jacobi_step()[2]            # the windows whose approximate tokens get handed over
    kl, ng = dec.fc_get_state()
    got, glens = dec.fc_finish_with_trigger(trigger, 12)
    for b in range(B):
        o = oracle.Oracle(cfg, w, 200)
        ar, _ = o.ar_generate(ids[b, :lens[b]].numpy(), int(ng[b]))
        assert wins[b, 0] == ar[-1]            # the GPU's exact tokens are the oracle's so far (large margins here)
        context = np.concatenate([ids[b, :lens[b]].numpy(), ar, wins[b, 1:], trigger]).astype(np.int32)
        want, margins = oracle.Oracle(cfg, w, 200).ar_generate(context, 12)
        g = got[b, :glens[b]]
        assert glens[b] == 12
        diff = np.nonzero(g != want)[0]
        if len(diff):
            assert margins[diff[0]] < MARGIN_TOL
    # EOS cut: stop each answer just after a token taken from the first answer
    eos = int(got[0, 3])
    dec.fc_prefill(ids.numpy(), lens, cfg.c)
    dec.fc_generate(8)
    dec.fc_jacobi_step()
    got2, glens2 = dec.fc_finish_with_trigger(trigger, 12, eos_id=eos)
    first = int(np.where(got[0, :12] == eos)[0][0])
    assert glens2[0] == first + 1 and got2[0, :first + 1].tolist() == got[0, :first + 1].tolist()


# ------------------------------------------------------------------ long positions on the fp32 path
def test_fp32_stream_exact_at_positions_in_the_thousands():
    """Rotary angles at positions ~3000 come from the host-built table on the FMA path too: the stream stays
    bit-exact where the device's own powf would be a few ulp off."""
    cfg = wl.CONFIGS["tiny"]
    P = 3000
    w = wl.make_weights(cfg)
    max_seq = P + 40
    dec = engine.Decoder(cfg, w, 1, 8, max_seq)
    prompt = wl.hash_uniform_int(cfg.seed, 21, P, cfg.vocab).numpy()
    o = oracle.Oracle(cfg, w, max_seq)
    o.prefill(prompt, 8)
    want, _ = o.generate(16)
    dec.fc_prefill(prompt, [P], 8)
    logits = dec.fc_debug_logits(True)
    toks, lens, _ = dec.fc_generate(16)
    assert toks[0, :lens[0]].tolist() == want.tolist()


# ------------------------------------------------------------------ run-to-run spread of the bf16 path
@pytest.mark.parametrize("flags", [0, lib.FC_FLAG_NO_FFN_SPLIT], ids=["ffn-split", "ffn-unsplit"])
def test_bf16_step_run_to_run_spread_is_bounded(flags):
    """Partial sums are added in L2 in whatever order they arrive, so two runs of the same step differ in the last
    bits.  The spread of the logits over repeated runs must stay two orders of magnitude under the parity tolerance
    (a lost update or a read of a half-added residual would be far larger), with the feed-forward block run as two
    halves and as one."""
    cfg = wl.small_config(vocab=2000, n_layers=8, n_heads=16, n_kv_heads=4, head_dim=64, d_model=1024, d_ffn=2816,
                          prompt_len=300, c=16, gen_tokens=8)
    w = wl.make_weights(cfg, device="cuda")
    prompt = wl.make_prompts(cfg)[0][0].numpy()
    dec = engine.Decoder(cfg, w, 1, cfg.c, 400, flags=flags)
    logits = dec.fc_debug_logits(True)
    dec.fc_prefill(prompt, [len(prompt)], cfg.c)
    ref = None
    spread = 0.0
    for _ in range(25):
        dec.fc_bench_steps(1, commit=False)          # the same step again: nothing is committed
        torch.cuda.synchronize()
        lg = logits[:cfg.c].clone()
        if ref is None:
            ref = lg
        spread = max(spread, float((lg - ref).abs().max()))
    assert spread < 3e-4, spread


@pytest.mark.parametrize("flags", [0, lib.FC_FLAG_NO_CTA_PAIRS], ids=["cta-pairs", "single-cta-tiles"])
def test_bf16_many_row_step_spread_and_agreement_of_the_two_tilings(flags):
    """160 rows per forward (two blocks of 128 through the activation panel; pairs of CTAs per 256-row weight tile or
    one CTA per 128-row tile): repeated runs of the same step stay within the same small spread, and the logits agree
    with the oracle's for every sequence."""
    cfg = wl.small_config(vocab=1200, n_layers=4, n_heads=8, n_kv_heads=8, head_dim=64, d_model=512, d_ffn=1536,
                          prompt_len=90, c=16, gen_tokens=4)
    B = 10
    w = wl.make_weights(cfg, device="cuda")
    lens = [90 - 7 * b for b in range(B)]
    ids, _ = wl.make_prompts(cfg, batch=B, lens=lens)
    dec = engine.Decoder(cfg, w, B, cfg.c, 120, flags=flags)
    logits = dec.fc_debug_logits(True)
    dec.fc_prefill(ids.numpy(), lens, cfg.c)
    ref = None
    spread = 0.0
    for _ in range(15):
        dec.fc_bench_steps(1, commit=False)
        torch.cuda.synchronize()
        lg = logits[:B * cfg.c].clone()
        if ref is None:
            ref = lg
        spread = max(spread, float((lg - ref).abs().max()))
    assert spread < 3e-4, spread
    got = ref.cpu().numpy().reshape(B, cfg.c, cfg.vocab)
    wc = wl.make_weights(cfg)
    for b in (0, 4, 9):
        o = oracle.Oracle(cfg, wc, 120)
        o.prefill(ids[b, :lens[b]].numpy(), cfg.c)
        _, _, _, lg = o.jacobi_step(want_logits=True)
        assert np.abs(got[b] - lg).max() < LOGIT_TOL
        o.close()


@pytest.mark.parametrize("kind", ["fp32", "bf16"])
def test_finished_sequences_are_skipped_and_the_others_unaffected(kind):
    """A batch in which sequences finish at different times (one on an EOS early in its stream, the others at
    max_tokens): finished sequences no longer take rows of the forward - the step runs over the live ones only,
    through a map from row block to sequence - and every stream still equals the oracle's autoregressive stream.
    The launch count shows the compacted steps (one extra gather launch each); a step after the end reports 0."""
    if kind == "fp32":
        cfg = wl.CONFIGS["tiny"]
        c, n_gen = 4, 24
    else:
        cfg = wl.small_config(vocab=600, n_layers=2, n_heads=4, n_kv_heads=2, head_dim=64, d_model=256, d_ffn=512,
                              prompt_len=70, c=6, gen_tokens=20)
        c, n_gen = cfg.c, cfg.gen_tokens
    B = 4
    lens = [40, 33, 7, 25] if kind == "fp32" else [70, 33, 1, 50]
    w = wl.make_weights(cfg)
    max_seq = max(lens) + n_gen + c + 8
    dec = engine.Decoder(cfg, w, B, c, max_seq)
    ids, _ = wl.make_prompts(cfg, batch=B, lens=lens)
    ars, margins = [], []
    for b in range(B):
        o = oracle.Oracle(cfg, w, max_seq)
        ar, m = o.ar_generate(ids[b, :lens[b]].numpy(), n_gen)
        ars.append(ar); margins.append(m)
        o.close()
    # an EOS that ends sequence 1 after a few tokens and occurs nowhere in the other streams
    eos = next(int(t) for t in ars[1][3:10] if all(int(t) not in ars[b].tolist() for b in (0, 2, 3)))
    want = [ar[:ar.tolist().index(eos) + 1] if eos in ar.tolist() else ar for ar in ars]
    assert len(want[1]) < n_gen and all(len(want[b]) == n_gen for b in (0, 2, 3))
    dec.fc_prefill(ids.numpy(), lens, c)
    toks, out_lens, st = dec.fc_generate(n_gen, eos_id=eos)
    for b in range(B):
        got = toks[b, :out_lens[b]]
        if kind == "fp32":
            assert got.tolist() == want[b].tolist(), b
        else:
            n = min(len(got), len(want[b]))
            diff = np.nonzero(got[:n] != want[b][:n])[0]
            if len(diff):
                assert margins[b][diff[0]] < MARGIN_TOL, (b, int(diff[0]))
            else:
                assert len(got) == len(want[b])
    # steps after sequence 1 ended carry a gather launch and fewer attention CTAs; the count of launches per step is
    # the plain step's + 1 for those steps
    per_step = (2 * cfg.n_layers + 4) if kind == "bf16" else None
    if per_step:
        assert st.steps * per_step < dec.fc_last_launch_count() <= st.steps * (per_step + 1)
    cnt, _, _ = dec.fc_jacobi_step()
    assert cnt.tolist() == [0] * B
    assert dec.fc_debug_check_guards() == 0
