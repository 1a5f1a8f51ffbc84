"""Pins for the CPU oracle: what the paper and the mathematics fix, checked without a GPU.

Each test is chosen so that a plausible mistake in the oracle (dropped term, wrong sign or index,
transposed operand, off-by-one in the accept rule) fails at least one of them.
"""
import itertools

import numpy as np
import pytest
import torch

import oracle
from paper_2311_08263_b200 import workload as wl


def _tiny():
    cfg = wl.CONFIGS["tiny"]
    return cfg, wl.make_weights(cfg), wl.make_prompts(cfg)[0][0].numpy()


# ---------------------------------------------------------------- decoder forward vs the library
def _hf_model(cfg, w):
    from transformers import LlamaConfig, LlamaForCausalLM
    hc = LlamaConfig(hidden_size=cfg.d_model, intermediate_size=cfg.d_ffn,
                     num_hidden_layers=cfg.n_layers, num_attention_heads=cfg.n_heads,
                     num_key_value_heads=cfg.n_kv_heads, head_dim=cfg.head_dim, vocab_size=cfg.vocab,
                     rms_norm_eps=cfg.rms_eps, rope_theta=cfg.rope_theta, attention_bias=False,
                     mlp_bias=False, tie_word_embeddings=False, max_position_embeddings=1024,
                     attn_implementation="eager")
    m = LlamaForCausalLM(hc).double().eval()
    sd = {"model.embed_tokens.weight": w["tok_emb"], "model.norm.weight": w["g_final"],
          "lm_head.weight": w["lm_head"]}
    names = {"wq": "self_attn.q_proj", "wk": "self_attn.k_proj", "wv": "self_attn.v_proj",
             "wo": "self_attn.o_proj", "w_gate": "mlp.gate_proj", "w_up": "mlp.up_proj",
             "w_down": "mlp.down_proj", "g_attn": "input_layernorm", "g_ffn": "post_attention_layernorm"}
    for l in range(cfg.n_layers):
        for k, v in names.items():
            sd[f"model.layers.{l}.{v}.weight"] = w[k][l]
    res = m.load_state_dict({k: v.double() for k, v in sd.items()}, strict=False)
    assert not res.missing_keys and not res.unexpected_keys
    return m


@pytest.mark.parametrize("hq,hkv", [(4, 4), (4, 2), (4, 1)])
def test_forward_matches_huggingface_llama_fp64(hq, hkv):
    """The paper runs stock HuggingFace Llama (Section 5.1); the oracle's forward must be that
    model: same logits for a causal forward, with and without a K/V-cache split."""
    cfg = wl.small_config(dtype="f32", n_heads=hq, n_kv_heads=hkv, head_dim=32, d_model=128,
                          d_ffn=256, vocab=300, bias_beta=0.0, n_layers=3)
    w = wl.make_weights(cfg)
    toks = wl.make_prompts(cfg, lens=[29])[0][0]
    with torch.no_grad():
        ref = _hf_model(cfg, w)(toks.long()[None]).logits[0].numpy()
    o = oracle.Oracle(cfg, w, 64)
    _, lg = o.forward(toks.numpy())
    assert np.abs(lg - ref).max() < 2e-6
    # same rows through the cache: commit the first 17 tokens, then a 12-row window
    o2 = oracle.Oracle(cfg, w, 64)
    o2.prefill(toks[:18].numpy(), c=12)
    assert o2.kv_len == 17
    _, lg2 = o2.forward(toks[17:].numpy())
    assert np.abs(lg2 - ref[17:]).max() < 2e-6


def test_bias_lands_on_permuted_input_token():
    cfg = wl.small_config(dtype="f32", d_model=64, n_heads=2, n_kv_heads=2, head_dim=32, d_ffn=128,
                          vocab=50, bias_beta=0.0)
    w = wl.make_weights(cfg)
    toks = np.array([3, 9, 41], np.int32)
    _, base = oracle.Oracle(cfg, w, 16).forward(toks)
    cfg_b = wl.small_config(dtype="f32", d_model=64, n_heads=2, n_kv_heads=2, head_dim=32, d_ffn=128,
                            vocab=50, bias_beta=2.5)
    _, biased = oracle.Oracle(cfg_b, w, 16).forward(toks)
    diff = biased - base
    perm = w["bias_perm"].numpy()
    for r, t in enumerate(toks):
        expect = np.zeros(50, np.float32)
        expect[perm[t]] = 2.5
        assert np.allclose(diff[r], expect, atol=1e-6)
    assert sorted(perm.tolist()) == list(range(50))


def test_bf16_weights_are_upconverted_exactly():
    cfg = wl.small_config(dtype="bf16", d_model=64, n_heads=2, n_kv_heads=1, head_dim=32, d_ffn=128, vocab=80)
    w = wl.make_weights(cfg)
    w32 = {k: ([t.float() for t in v] if isinstance(v, list) else (v.float() if v.dtype != torch.int32 else v))
           for k, v in w.items()}
    cfg32 = wl.small_config(dtype="f32", d_model=64, n_heads=2, n_kv_heads=1, head_dim=32, d_ffn=128, vocab=80)
    toks = np.arange(10, dtype=np.int32)
    _, a = oracle.Oracle(cfg, w, 16, kv_bf16=False).forward(toks)      # weights only: K/V kept in fp32 here
    _, b = oracle.Oracle(cfg32, w32, 16).forward(toks)
    assert np.array_equal(a, b)


# ---------------------------------------------------------------- losslessness (Section 3.1 / 3.2)
@pytest.mark.parametrize("c", [1, 2, 3, 8, 16])
@pytest.mark.parametrize("refill", [0, 1])
def test_committed_stream_equals_greedy_autoregressive(c, refill):
    cfg, w, prompt = _tiny()
    o = oracle.Oracle(cfg, w, 160)
    ar, _ = o.ar_generate(prompt, 64)
    o.prefill(prompt, c, refill=refill, pad_id=7)
    toks, counts = o.generate(64)
    assert np.array_equal(toks, ar)
    assert counts.min() >= 1 and counts.max() <= c
    assert counts.sum() == 64
    if c == 1:
        assert len(counts) == 64     # window of one row is plain autoregressive decoding


def test_window_contents_never_change_the_stream():
    cfg, w, prompt = _tiny()
    o = oracle.Oracle(cfg, w, 160)
    ar, _ = o.ar_generate(prompt, 40)
    o.prefill(prompt, 8)
    rng = np.random.default_rng(0)
    out, pending = [], prompt[-1]
    while len(out) < 40:
        win = rng.integers(0, cfg.vocab, 8).astype(np.int32)
        win[0] = pending
        k, acc, wnew = o.jacobi_step(win)
        out.extend(acc.tolist())
        pending = wnew[0]
    assert out[:40] == ar.tolist()


# ---------------------------------------------------------------- accept rule: closed form given AR
def _expected_step(ar, n, window, c, prompt, refill_fn):
    """Closed form: k = 1 + longest m with window[1..m] == ar[n..n+m-1]; emitted = ar[n..n+k-1]."""
    k = 1
    while k < c and window[k] == ar[n + k - 1]:
        k += 1
    return k, ar[n:n + k]


@pytest.mark.parametrize("c", [2, 5, 8])
def test_directed_accept_counts(c):
    """Prime the window with m correct continuation tokens followed by a wrong one: the step must
    accept exactly m + 1 tokens, for every m, and the refreshed window must carry the pending
    token, the unverified outputs, and refill ids for the k-1 unseen positions."""
    cfg, w, prompt = _tiny()
    P = len(prompt)
    o = oracle.Oracle(cfg, w, 200)
    ar, _ = o.ar_generate(prompt, 80)
    for m in range(c):
        o.prefill(prompt, c)
        n = 0
        # advance a few plain steps so n_gen is not zero
        for _ in range(3):
            k, acc, wnew = o.jacobi_step()
            n += k
        win = wnew.copy()
        win[1:1 + m] = ar[n:n + m]
        if 1 + m < c:
            win[1 + m] = (ar[n + m] + 1) % cfg.vocab
        k, acc, w2, lg = o.jacobi_step(win, want_logits=True)
        assert k == m + 1
        assert np.array_equal(acc, ar[n:n + k])
        a = lg.argmax(axis=1)
        assert w2[0] == ar[n + k - 1]
        assert np.array_equal(w2[1:c - k + 1], a[k:c])
        n2 = n + k
        for j in range(c - k + 1, c):
            assert w2[j] == prompt[(n2 + j - 1) % P]
        assert o.n_gen == n2 and o.kv_len == P - 1 + n2


@pytest.mark.parametrize("V,c", [(4, 2), (4, 3), (4, 4), (8, 3)])
def test_brute_force_all_windows_tiny_vocab(V, c):
    """Enumerate every window over a tiny vocabulary and check the accepted count and tokens
    against greedy decoding done one token at a time."""
    cfg = wl.small_config(dtype="f32", n_layers=1, d_model=16, n_heads=2, n_kv_heads=1, head_dim=8,
                          d_ffn=32, vocab=V, bias_beta=0.0, seed=5 + V + c)
    w = wl.make_weights(cfg)
    # larger weights so logits are well separated
    for key in ("tok_emb", "lm_head"):
        w[key] = w[key] * 40
    prompt = np.array([1, 3 % V, 2, 0, 1], np.int32)
    o = oracle.Oracle(cfg, w, 64)
    ar, mar = o.ar_generate(prompt, c + 1)
    assert mar.min() > 1e-4
    seen_k = set()
    for guess in itertools.product(range(V), repeat=c - 1):
        o.prefill(prompt, c)
        win = np.array((prompt[-1],) + guess, np.int32)
        k, acc, w2 = o.jacobi_step(win)
        kk, emitted = _expected_step(ar, 0, win, c, prompt, None)
        assert k == kk and np.array_equal(acc, emitted)
        assert w2[0] == ar[k - 1]
        seen_k.add(k)
    assert seen_k == set(range(1, c + 1))


# ---------------------------------------------------------------- whole-stream closed forms
def test_zero_matrices_stream_is_iterated_permutation():
    cfg = wl.small_config(dtype="f32", d_model=32, n_heads=2, n_kv_heads=2, head_dim=16, d_ffn=64,
                          vocab=97, bias_beta=4.0)
    w = wl.make_weights(cfg, zero_matrices=True)
    prompt = np.array([5, 11, 60], np.int32)
    perm = w["bias_perm"].numpy()
    o = oracle.Oracle(cfg, w, 128)
    o.prefill(prompt, 6)
    toks, counts = o.generate(50)
    expect, t = [], prompt[-1]
    for _ in range(50):
        t = perm[t]
        expect.append(t)
    assert toks.tolist() == expect
    # guesses that already follow the permutation are all accepted: k = c
    o.prefill(prompt, 6)
    win = np.array([prompt[-1]] + expect[:5], np.int32)
    k, acc, _ = o.jacobi_step(win)
    assert k == 6 and acc.tolist() == expect[:6]


def test_all_equal_logits_pick_lowest_id():
    cfg = wl.small_config(dtype="f32", d_model=32, n_heads=2, n_kv_heads=2, head_dim=16, d_ffn=64,
                          vocab=33, bias_beta=0.0)
    w = wl.make_weights(cfg, zero_matrices=True)
    o = oracle.Oracle(cfg, w, 64)
    o.prefill(np.array([4, 2], np.int32), 4)
    toks, _ = o.generate(10)
    assert toks.tolist() == [0] * 10


# ---------------------------------------------------------------- stop rules
def test_max_tokens_and_eos_truncation():
    cfg, w, prompt = _tiny()
    o = oracle.Oracle(cfg, w, 160)
    ar, _ = o.ar_generate(prompt, 30)
    eos = int(ar[12])
    first = int(np.where(ar == eos)[0][0])
    o.prefill(prompt, 8)
    toks, counts = o.generate(30, eos_id=eos)
    assert toks.tolist() == ar[:first + 1].tolist()
    assert counts.sum() == first + 1
    o.prefill(prompt, 8)
    toks, counts = o.generate(5)
    assert toks.tolist() == ar[:5].tolist()


# ---------------------------------------------------------------- stored stream (drift guard)
def test_golden_tiny_stream():
    """tests/golden/tiny_ar_stream.txt is written by tests/golden/make_golden.py from the oracle
    alone; it guards the oracle and the input generator against silent drift."""
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "tiny_ar_stream.txt")
    want = [int(t) for t in open(path).read().split("\n")[-2].split()]
    cfg, w, prompt = _tiny()
    ar, _ = oracle.Oracle(cfg, w, 160).ar_generate(prompt, 64)
    assert ar.tolist() == want


# ---------------------------------------------------------------- the accept rule alone, exhaustively
@pytest.mark.parametrize("c", [1, 2, 3, 4, 5])
def test_accept_rule_exhaustive_small_vocab(c):
    """All (window, argmax) pairs over a 3-token vocabulary: properties that define the rule."""
    V, prompt = 3, np.array([2, 0, 1, 1], np.int32)
    for w in itertools.product(range(V), repeat=c):
        for a in itertools.product(range(V), repeat=c):
            for n_gen in (0, 3):
                k, acc, w2 = oracle.accept(w, a, n_gen, prompt)
                assert 1 <= k <= c
                assert all(w[j] == a[j - 1] for j in range(1, k))          # accepted guesses were right
                assert k == c or w[k] != a[k - 1]                           # and the run is maximal
                assert acc.tolist() == list(a[:k])
                assert w2[0] == a[k - 1]
                assert w2[1:c - k + 1].tolist() == list(a[k:c])
                assert w2[c - k + 1:].tolist() == [prompt[(n_gen + k + j - 1) % 4] for j in range(c - k + 1, c)]
                _, _, w3 = oracle.accept(w, a, n_gen, prompt, refill=1, pad_id=2)
                assert w3[c - k + 1:].tolist() == [2] * (k - 1)


def test_linear_matches_fp64_matmul():
    rng = np.random.default_rng(3)
    w = torch.from_numpy(rng.standard_normal((37, 72)).astype(np.float32))
    x = rng.standard_normal((5, 72)).astype(np.float32)
    y = rng.standard_normal((5, 37)).astype(np.float32)
    got = oracle.linear_add(w, x, y)
    want = y.astype(np.float64) + x.astype(np.float64) @ w.numpy().astype(np.float64).T
    assert np.abs(got - want).max() < 1e-5
    got_b = oracle.linear_add(w.to(torch.bfloat16), x, y)
    want_b = y.astype(np.float64) + x.astype(np.float64) @ w.to(torch.bfloat16).double().numpy().T
    assert np.abs(got_b - want_b).max() < 1e-5


# ---------------------------------------------------------------- bf16 storage of K/V in bf16 models
def test_bf16_rounding_matches_library():
    vals = np.concatenate([np.random.default_rng(1).standard_normal(2000).astype(np.float32) * s
                           for s in (1e-3, 1.0, 300.0)] + [np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875], np.float32)])
    want = torch.from_numpy(vals).to(torch.bfloat16).float().numpy()
    got = np.array([oracle.round_bf16(float(v)) for v in vals], np.float32)
    assert np.array_equal(got, want)


def test_bf16_model_stores_kv_in_bf16_and_stays_lossless():
    """K/V rows of a bf16 model are bf16 values; the cache-split forward still equals the one-shot forward bitwise,
    and the Jacobi stream still equals the greedy stream."""
    cfg = wl.small_config(dtype="bf16", d_model=64, n_heads=2, n_kv_heads=1, head_dim=32, d_ffn=128, vocab=80,
                          n_layers=2, bias_beta=3.0)
    w = wl.make_weights(cfg)
    toks = wl.make_prompts(cfg, lens=[20])[0][0].numpy()
    o = oracle.Oracle(cfg, w, 64)
    o.forward(toks, want_logits=False)
    k, v = o.get_kv(0, 20)
    for a in (k, v):
        assert np.array_equal(a, torch.from_numpy(a).to(torch.bfloat16).float().numpy())
    # an fp32-K/V run of the same model differs (the rounding is really applied) but only slightly
    _, lg_b = oracle.Oracle(cfg, w, 64).forward(toks)
    _, lg_f = oracle.Oracle(cfg, w, 64, kv_bf16=False).forward(toks)
    d = np.abs(lg_b - lg_f).max()
    assert 0 < d < 5e-2
    # one-shot rows == cached rows, bitwise
    o2 = oracle.Oracle(cfg, w, 64)
    o2.prefill(toks[:13], c=8)
    _, lg2 = o2.forward(toks[12:])
    assert np.array_equal(lg2, lg_b[12:])
    ar, _ = oracle.Oracle(cfg, w, 96).ar_generate(toks, 24)
    o3 = oracle.Oracle(cfg, w, 96)
    o3.prefill(toks, 6)
    st, _ = o3.generate(24)
    assert np.array_equal(st, ar)


# ---------------------------------------------------------------- iteration cap, window resize, answer trigger
def test_iteration_cap_stops_after_max_iters():
    """Upper bound on the iterations ("Iteration Stop Condition", condition 1): the stream produced within
    the cap is a prefix of the greedy stream and exactly max_iters forwards ran."""
    cfg, w, prompt = _tiny()
    o = oracle.Oracle(cfg, w, 200)
    ar, _ = o.ar_generate(prompt, 40)
    o.prefill(prompt, 8)
    toks, counts = o.generate(40, max_iters=5)
    assert len(counts) == 5 and counts.sum() == len(toks) >= 5
    assert toks.tolist() == ar[:len(toks)].tolist()
    # going on without a cap completes the same stream
    rest, _ = o.generate(40 - len(toks))
    assert np.concatenate([toks, rest]).tolist() == ar.tolist()


@pytest.mark.parametrize("sizes", [(8, 3, 12, 1, 5), (1, 16, 2)])
def test_window_resize_keeps_the_stream_lossless(sizes):
    """Changing c between iterations never changes the committed stream (it stays the greedy stream), and the
    resized window keeps the pending token and the guesses that still fit; new slots follow the refill rule."""
    cfg, w, prompt = _tiny()
    o = oracle.Oracle(cfg, w, 240)
    ar, _ = o.ar_generate(prompt, 60)
    o.prefill(prompt, sizes[0])
    got = []
    for i in range(30):
        c_old = o.c
        k, acc, wnew = o.jacobi_step()
        got += acc.tolist()
        c_new = sizes[(i + 1) % len(sizes)]
        o.set_window(c_new)
        # probe the resized window through a step that feeds it back unchanged: window_in must be accepted
        # (slot 0 is the pending token), and the kept part is the old window's head
        keep = min(c_old, c_new)
        want_w = wnew[:keep].tolist() + [int(prompt[(o.n_gen + j - 1) % len(prompt)]) for j in range(keep, c_new)]
        k2, acc2, _ = o.jacobi_step(np.array(want_w, np.int32))
        got += acc2.tolist()
        if len(got) >= 60:
            break
    assert got[:60] == ar[:len(got[:60])].tolist()


def test_window_resize_guess_positions():
    """A guess kept across a resize still refers to the same generated index: prime slot 1..m with the greedy
    continuation, shrink and grow the window, and the next step must still accept exactly those."""
    cfg, w, prompt = _tiny()
    o = oracle.Oracle(cfg, w, 200)
    ar, _ = o.ar_generate(prompt, 20)
    o.prefill(prompt, 8)
    win = np.zeros(8, np.int32)
    win[0] = prompt[-1]
    win[1:4] = ar[:3]
    win[4] = (ar[3] + 1) % cfg.vocab
    o2 = oracle.Oracle(cfg, w, 200)
    o2.prefill(prompt, 8)
    # o: plain step with the primed window -> k = 4
    k, acc, _ = o.jacobi_step(win)
    assert k == 4 and acc.tolist() == ar[:4].tolist()
    # o2: window of 3 rows holding the first two primed guesses -> k = 3 (all guesses right)
    o2.set_window(3)
    k, acc, wn = o2.jacobi_step(win[:3])
    assert k == 3 and acc.tolist() == ar[:3].tolist() and wn[0] == ar[2]


@pytest.mark.parametrize("n_trig,c", [(0, 1), (3, 6), (5, 1), (1, 8)])
def test_answer_trigger_equals_greedy_on_the_concatenated_context(n_trig, c):
    """Hand-off ("Overview of FastCoT", "Trigger Answer"): the answer decoded after prompt + exact tokens +
    approximate tokens + trigger equals plain greedy decoding (Eq. 1) of that concatenation."""
    cfg, w, prompt = _tiny()
    trigger = wl.hash_uniform_int(5, 9, max(n_trig, 1), cfg.vocab).numpy()[:n_trig]
    o = oracle.Oracle(cfg, w, 200)
    o.prefill(prompt, c)
    emitted, _ = o.generate(12, max_iters=4)
    _, _, window = o.jacobi_step()          # one more step so that the window holds real approximate tokens
    # context = prompt | all exact tokens | approximate tokens | trigger  (window[0] is the last exact token)
    o_ref = oracle.Oracle(cfg, w, 200)
    ar, _ = o_ref.ar_generate(prompt, 40)
    n_exact = o.n_gen
    context = np.concatenate([prompt, ar[:n_exact], window[1:], trigger]).astype(np.int32)
    assert window[0] == ar[n_exact - 1]
    want, _ = oracle.Oracle(cfg, w, 300).ar_generate(context, 10)
    got = o.finish_with_trigger(trigger, 10)
    assert got.tolist() == want.tolist()
    with pytest.raises(RuntimeError):
        o.jacobi_step()                      # the Jacobi state was consumed


def test_answer_trigger_empty_with_c1_is_plain_continuation_and_eos_cut():
    cfg, w, prompt = _tiny()
    ar, _ = oracle.Oracle(cfg, w, 200).ar_generate(prompt, 30)
    o = oracle.Oracle(cfg, w, 200)
    o.prefill(prompt, 1)
    o.generate(6)
    got = o.finish_with_trigger([], 20)
    assert got.tolist() == ar[6:26].tolist()
    o.prefill(prompt, 1)
    o.generate(6)
    eos = int(ar[10])
    first = 6 + int(np.where(ar[6:] == eos)[0][0])
    got = o.finish_with_trigger([], 20, eos_id=eos)
    assert got.tolist() == ar[6:first + 1].tolist()


# ---------------------------------------------------------------- layer-0 special cases with closed forms
def _f32_small(**kw):
    cfg = wl.small_config(dtype="f32", n_layers=1, vocab=300, **kw)
    return cfg, wl.make_weights(cfg)


def _normed_rows(cfg, w, tokens):
    """RMSNorm(embedding rows) * gain of layer 0, in fp64 (Llama's definition: x / sqrt(mean x^2 + eps) * g)."""
    x = w["tok_emb"].double()[torch.as_tensor(np.asarray(tokens)).long()]
    return x / torch.sqrt((x * x).mean(1, keepdim=True) + cfg.rms_eps) * w["g_attn"][0].double()


@pytest.mark.parametrize("hq,hkv", [(4, 4), (4, 2), (4, 1)])
def test_single_key_attention_returns_its_value_row(hq, hkv):
    """Empty cache, one window row: the softmax over one key is 1, so every query head's output is the value row of its
    kv head, bit for bit (head h reads kv head h // (hq / hkv))."""
    cfg, w = _f32_small(n_heads=hq, n_kv_heads=hkv, head_dim=32, d_model=hq * 32)
    o = oracle.Oracle(cfg, w, 8)
    _, _, tr = o.forward([5], want_logits=True, trace=True)
    _, v = o.get_kv(0, 1)
    hd, group = cfg.head_dim, hq // hkv
    for h in range(hq):
        kvh = h // group
        assert np.array_equal(tr["attn"][0, h * hd:(h + 1) * hd], v[0, kvh * hd:(kvh + 1) * hd])
    o.close()


def test_rope_is_the_identity_at_position_zero_and_a_rotation_of_half_split_pairs_elsewhere():
    """Position 0: q and k are the plain projections of the normalised row.  Position p: element i is paired with
    i + head_dim / 2 (not with i + 1), the pair keeps its norm and turns by p * theta^(-2i / head_dim)."""
    cfg, w = _f32_small(n_heads=2, n_kv_heads=2, head_dim=32, d_model=64)
    toks = [7, 11, 13, 17, 19]
    o = oracle.Oracle(cfg, w, 16)
    _, _, tr = o.forward(toks, want_logits=True, trace=True)
    k, _ = o.get_kv(0, len(toks))
    xn = _normed_rows(cfg, w, toks)
    q_plain = (xn @ w["wq"][0].double().T).numpy()
    k_plain = (xn @ w["wk"][0].double().T).numpy()
    assert np.abs(tr["q"][0] - q_plain[0]).max() < 2e-6 and np.abs(k[0] - k_plain[0]).max() < 2e-6
    hd, half = cfg.head_dim, cfg.head_dim // 2
    for got, plain in ((tr["q"], q_plain), (k, k_plain)):
        for p in range(1, len(toks)):
            for h in range(cfg.n_heads):
                a, b = plain[p, h * hd:h * hd + half], plain[p, h * hd + half:(h + 1) * hd]
                ga, gb = got[p, h * hd:h * hd + half].astype(np.float64), got[p, h * hd + half:(h + 1) * hd].astype(np.float64)
                assert np.abs((ga * ga + gb * gb) - (a * a + b * b)).max() < 1e-5          # norm of every pair
                ang = p * cfg.rope_theta ** (-2.0 * np.arange(half) / hd)
                turned = np.arctan2(gb, ga) - np.arctan2(b, a)
                d = (turned - ang + np.pi) % (2 * np.pi) - np.pi
                big = (a * a + b * b) > 1e-4                                               # the angle of a tiny pair is noise
                assert np.abs(d[big]).max() < 1e-4
    o.close()


@pytest.mark.parametrize("hq,hkv", [(4, 4), (4, 2)])
def test_zero_query_projection_gives_the_causal_mean_of_the_value_rows(hq, hkv):
    """W_q = 0: all scores are equal, so window row j attends uniformly to the L cached rows and window rows 0..j - the
    output is their mean value row.  Fails on an off-by-one in the causal mask, a missing normalisation or a wrong
    query-head -> kv-head map."""
    cfg, w = _f32_small(n_heads=hq, n_kv_heads=hkv, head_dim=32, d_model=hq * 32)
    w["wq"][0] = torch.zeros_like(w["wq"][0])
    L, c = 6, 5
    ids = wl.hash_uniform_int(cfg.seed, 3, L + 1, cfg.vocab).numpy()
    o = oracle.Oracle(cfg, w, L + c + 4)
    o.prefill(ids, c)                                      # caches ids[0 .. L-1]
    win = wl.hash_uniform_int(cfg.seed + 1, 4, c, cfg.vocab).numpy()
    _, _, tr = o.forward(win, want_logits=True, trace=True)
    _, v = o.get_kv(0, L + c)
    hd, group = cfg.head_dim, hq // hkv
    for j in range(c):
        want = v[:L + j + 1].astype(np.float64).mean(0)
        for h in range(hq):
            kvh = h // group
            assert np.abs(tr["attn"][j, h * hd:(h + 1) * hd] - want[kvh * hd:(kvh + 1) * hd]).max() < 2e-6
    o.close()
