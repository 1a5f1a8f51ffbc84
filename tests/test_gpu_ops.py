"""Single operations of the step through the C ABI, element by element against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2311_08263_b200 import engine, lib, workload as wl

pytestmark = pytest.mark.gpu


def _rand(seed, tid, shape, scale=1.0):
    n = int(np.prod(shape))
    return (wl.hash_normal(seed, tid, n) * scale).view(*shape)


# K spans several 64-wide k blocks plus a ragged tail; N spans several 128-row tiles plus a tail;
# R covers every accumulator width the kernel is built for and a multi-pass case (R > 256).
LINEAR_CASES = [
    (16, 256, 256), (16, 384, 1024), (8, 200, 328), (1, 128, 64), (5, 1000, 136),
    (32, 512, 512), (48, 256, 704), (100, 384, 256), (256, 256, 192), (300, 256, 128),
    (16, 4096, 4096),
]


@pytest.mark.parametrize("R,N,K", LINEAR_CASES)
def test_linear_tensor_core_bf16(R, N, K):
    w = _rand(11, 1, (N, K), 0.05).to(torch.bfloat16)
    x = _rand(11, 2, (R, K)).to(torch.bfloat16).float()        # values exactly representable in bf16
    y0 = _rand(11, 3, (R, N))
    want = oracle.linear_add(w, x.numpy(), y0.numpy())
    y = y0.cuda()
    rc = engine.fc_op_linear(x.cuda(), w.cuda(), y, use_tensor_cores=True)
    assert rc == lib.FC_OK
    got = y.cpu().numpy()
    # exact products, fp32 accumulation in a different order: error ~ K * eps * |terms|
    tol = 2e-6 * K * 0.05 * 4 + 1e-5
    assert np.abs(got - want).max() < tol
    # running it again accumulates a second time
    rc = engine.fc_op_linear(x.cuda(), w.cuda(), y, use_tensor_cores=True)
    assert rc == lib.FC_OK
    want2 = oracle.linear_add(w, x.numpy(), want)
    assert np.abs(y.cpu().numpy() - want2).max() < 2 * tol


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("R,N,K", [(8, 128, 128), (3, 77, 264), (20, 300, 512)])
def test_linear_fma(R, N, K, dtype):
    w = _rand(12, 1, (N, K), 0.05).to(dtype)
    x = _rand(12, 2, (R, K))
    y0 = _rand(12, 3, (R, N))
    want = oracle.linear_add(w, x.numpy(), y0.numpy())
    y = y0.cuda()
    assert engine.fc_op_linear(x.cuda(), w.cuda(), y, use_tensor_cores=False) == lib.FC_OK
    assert np.abs(y.cpu().numpy() - want).max() < 1e-4


def test_linear_rejects_bad_arguments():
    x = torch.zeros(4, 64, device="cuda")
    w = torch.zeros(8, 64, device="cuda", dtype=torch.bfloat16)
    y = torch.zeros(4, 8, device="cuda")
    l = lib.load()
    st = torch.cuda.current_stream().cuda_stream
    assert l.fc_op_linear(None, w.data_ptr(), y.data_ptr(), 4, 8, 64, 1, 1, st) == lib.FC_ERR_ARG
    assert l.fc_op_linear(x.data_ptr(), w.data_ptr(), y.data_ptr(), 4, 8, 60, 1, 1, st) == lib.FC_ERR_ARG
    assert l.fc_op_linear(x.data_ptr(), w.data_ptr(), y.data_ptr(), 0, 8, 64, 1, 1, st) == lib.FC_ERR_ARG
    assert l.fc_op_linear(x.data_ptr(), w.data_ptr(), y.data_ptr(), 4, 8, 32, 1, 1, st) == lib.FC_ERR_SHAPE
    assert l.fc_op_linear(x.data_ptr(), w.data_ptr(), y.data_ptr(), 4, 8, 64, 0, 1, st) == lib.FC_ERR_SHAPE


@pytest.mark.parametrize("c", [1, 2, 5, 16, 64])
@pytest.mark.parametrize("refill", [0, 1])
def test_accept_kernel_bit_exact(c, refill):
    """Integer work: accepted count, tokens, refreshed window, kv_len and n_gen must equal the oracle's
    for random windows with planted matching runs of every length, several sequences at once."""
    rng = np.random.default_rng(c * 7 + refill)
    B, V, P = 9, 50, 13
    prompt = rng.integers(0, V, (B, 16)).astype(np.int32)
    plens = rng.integers(1, P + 1, B).astype(np.int32)
    window = rng.integers(0, V, (B, c)).astype(np.int32)
    argmax = rng.integers(0, V, (B, c)).astype(np.int32)
    for b in range(B):                      # plant a correct run of length b mod c
        m = b % c
        window[b, 1:1 + m] = argmax[b, :m]
    n_gen = rng.integers(0, 40, B).astype(np.int32)
    kv_len = rng.integers(0, 100, B).astype(np.int32)
    d = lambda a: torch.from_numpy(a.copy()).cuda()
    wd, kd, nd = d(window), d(kv_len), d(n_gen)
    cnt, tok = engine.fc_op_accept(wd, d(argmax), kd, nd, d(prompt), d(plens), refill, 7)
    cnt, tok, wnew = cnt.cpu().numpy(), tok.cpu().numpy(), wd.cpu().numpy()
    for b in range(B):
        k, acc, w2 = oracle.accept(window[b], argmax[b], int(n_gen[b]), prompt[b, :plens[b]], refill, 7)
        assert cnt[b] == k
        assert tok[b, :k].tolist() == acc.tolist()
        assert wnew[b].tolist() == w2.tolist()
        assert kd[b].item() == kv_len[b] + k and nd[b].item() == n_gen[b] + k


def _oracle_attention_case(cfg, lens, c):
    """Per sequence: prefill `len` tokens on the oracle, forward a random window with tracing, and
    return the layer-0 rotated queries, the layer-0 K/V cache (committed + window rows) and the
    oracle's attention output."""
    w = wl.make_weights(cfg)
    qs, wants, ks, vs = [], [], [], []
    for b, L in enumerate(lens):
        ids = wl.hash_uniform_int(cfg.seed + b, 5, L + 1, cfg.vocab).numpy()
        o = oracle.Oracle(cfg, w, L + c + 4)
        o.prefill(ids, c)
        win = wl.hash_uniform_int(cfg.seed + 100 + b, 7, c, cfg.vocab).numpy()
        _, _, tr = o.forward(win, want_logits=True, trace=True)
        k, v = o.get_kv(0, L + c)
        qs.append(tr["q"]); wants.append(tr["attn"]); ks.append(k); vs.append(v)
    return qs, wants, ks, vs


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("hq,hkv,hd,c,lens", [
    (4, 4, 32, 8, [300, 129, 0, 517]),       # MHA, several key tiles, an empty cache, ragged lengths
    (8, 2, 64, 5, [260, 1]),                 # GQA, odd window size
    (2, 2, 128, 16, [200]),                  # head_dim 128
    (4, 1, 64, 1, [77, 130]),                # c = 1: plain autoregressive attention
])
def test_window_attention_vs_oracle(dtype, hq, hkv, hd, c, lens):
    cfg = wl.small_config(dtype="f32", n_layers=1, d_model=128, n_heads=hq, n_kv_heads=hkv, head_dim=hd,
                          d_ffn=128, vocab=300, seed=91)
    qs, wants, ks, vs = _oracle_attention_case(cfg, lens, c)
    B, max_seq = len(lens), max(lens) + c + 3
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    kc = torch.zeros(B, hkv, max_seq, hd)
    vc = torch.zeros(B, hkv, max_seq, hd)
    for b, L in enumerate(lens):
        kc[b, :, :L + c] = torch.from_numpy(ks[b]).view(L + c, hkv, hd).transpose(0, 1)
        vc[b, :, :L + c] = torch.from_numpy(vs[b]).view(L + c, hkv, hd).transpose(0, 1)
    q = torch.from_numpy(np.concatenate(qs)).to(tdt).cuda()
    out = engine.fc_op_window_attention(q, kc.to(tdt).cuda().contiguous(), vc.to(tdt).cuda().contiguous(),
                                        torch.tensor(lens, dtype=torch.int32).cuda(), c, hq, max(lens))
    want = np.concatenate(wants)
    tol = 2e-5 if dtype == "f32" else 2e-2 * max(1.0, float(np.abs(want).max()))
    assert np.abs(out.cpu().numpy() - want).max() < tol
