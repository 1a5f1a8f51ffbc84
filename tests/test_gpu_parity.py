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
@pytest.mark.parametrize("shape", ["gqa64", "gqa32"])
def test_many_rows_prefill_and_steps(B, c, shape):
    """More than 16 rows per forward: the projections read their activations from the converted panel, for
    every accumulator width (32, 64, 128 rows) and for two blocks of rows; the prefill runs through the same path.
    gqa32 has k extents that are not multiples of 256, so a group of conversion units spans two rows."""
    kw = {"gqa64": dict(n_heads=4, n_kv_heads=2, head_dim=64, d_model=256, d_ffn=512),
          "gqa32": dict(n_heads=8, n_kv_heads=2, head_dim=32, d_model=320, d_ffn=328)}[shape]
    cfg = wl.small_config(vocab=700, n_layers=2, prompt_len=200, c=c, gen_tokens=12, **kw)
    lens = [200 - 17 * b for b in range(B)]
    w = wl.make_weights(cfg)
    max_seq = 200 + 12 + c + 8
    dec = engine.Decoder(cfg, w, B, c, max_seq)
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
