"""Element-wise parity of the attention kernel that the bf16 step launches (fused 1/rms + rotary embedding + K/V
write + split-KV window attention), through fc_op_fused_window_attention, against the CPU oracle's layer-0 trace.

The oracle runs a one-layer model: prefill of L tokens, then a forward over a window with tracing, which gives the
rotated queries, the attention output and the K/V cache (committed rows + the window's rows, rounded to bf16 where
stored).  The kernel gets what the step's QKV projection would hand it: the accumulators (x * gain) . W^T without
the 1/rms factor (computed here with a library matmul in fp64) and the rows' sums of squares, plus the oracle's
committed K/V rows as the cache.

Tolerances, derived from the arithmetic.  The cached rows are given exactly, so the only storage rounding that can
differ is that of the window's own K/V rows: two fp32 values that differ in the last bits can land on the two sides
of a bf16 rounding boundary (one bf16 step = 2^-8 relative).  Stored K/V must therefore agree with the oracle's to
one bf16 step, with all but a small fraction bit-identical.  For the output, a V element off by one step moves
out by at most p * 2^-8 * |v|, a K element moves a score by at most |q_i k_i| * 2^-8 / sqrt(hd); everything
else (fp32 summation order, exp, the bf16 high + low split of q and p) is ~1e-6 relative.  The bound used is
2^-8 * max|V| for the maximum and 2e-4 * max|V| for the root mean square.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2311_08263_b200 import engine, workload as wl

pytestmark = pytest.mark.gpu


def _case(hq, hkv, hd, c, lens, seed):
    cfg = wl.small_config(dtype="bf16", n_layers=1, d_model=256, n_heads=hq, n_kv_heads=hkv, head_dim=hd,
                          d_ffn=256, vocab=400, seed=seed)
    w = wl.make_weights(cfg)
    wqkv = torch.cat([w["wq"][0], w["wk"][0], w["wv"][0]]).double()
    gain = w["g_attn"][0].double()
    emb = w["tok_emb"].double()
    B, max_seq = len(lens), max(lens) + c + 5
    kvd = hkv * hd
    kc = torch.zeros(B, hkv, max_seq, hd)
    vc = torch.zeros(B, hkv, max_seq, hd)
    accs, sss, want_attn, want_k, want_v = [], [], [], [], []
    for b, L in enumerate(lens):
        ids = wl.hash_uniform_int(cfg.seed + b, 5, L + 1, cfg.vocab).numpy()
        o = oracle.Oracle(cfg, w, L + c + 4)
        o.prefill(ids, c)                                 # caches ids[0 .. L-1]
        win = wl.hash_uniform_int(cfg.seed + 100 + b, 7, c, cfg.vocab).numpy()
        _, _, tr = o.forward(win, want_logits=True, trace=True)
        k, v = o.get_kv(0, L + c)
        kc[b, :, :L] = torch.from_numpy(k[:L]).view(L, hkv, hd).transpose(0, 1)
        vc[b, :, :L] = torch.from_numpy(v[:L]).view(L, hkv, hd).transpose(0, 1)
        x = emb[torch.from_numpy(win).long()]             # [c, d] window rows entering layer 0
        accs.append(((x * gain) @ wqkv.T).float())
        sss.append((x * x).sum(1).float())
        want_attn.append(tr["attn"]); want_k.append(k[L:]); want_v.append(v[L:])
        o.close()
    return cfg, torch.cat(accs), torch.cat(sss), kc, vc, max_seq, want_attn, want_k, want_v


CASES = [
    # hq, hkv, hd, c, lens, splits per (sequence, kv head, query-tile group), query tiles per CTA (0 = the step's choice)
    (4, 4, 128, 16, [127, 128, 129, 0, 1], 0, 0),     # MHA; lengths around a tile edge, empty cache, one key
    (4, 4, 128, 16, [63, 64, 65, 191, 192], 1, 0),    # one CTA per head: every tile through the ring, ragged last tile
    (8, 2, 64, 5, [260, 1, 2047], 0, 0),              # GQA, odd window, clusters of 8 splits, sequences with empty splits
    (4, 4, 128, 1, [77, 130, 2047], 0, 0),            # c = 1: plain autoregressive attention
    (8, 2, 64, 33, [300, 6000], 0, 0),                # 94 tiles per head: long runs per CTA, 17 query tiles per kv head
    (4, 2, 128, 64, [513, 40], 0, 0),                 # c = 64: a full window tile, 8 query tiles per kv head
    (4, 2, 128, 64, [513, 40], 0, 2),                 # the same with two and with four query tiles per CTA
    (4, 2, 128, 64, [513, 40], 2, 4),
    (4, 2, 128, 100, [513, 40], 2, 0),                # c = 100: two window tiles (the second ragged), as in a prefill block
    (4, 2, 128, 100, [513, 40], 1, 2),
    (4, 4, 64, 16, [6000, 2047, 129], 4, 0),          # forced: 4 splits, running softmax statistics over ~24 tiles each
    (8, 2, 128, 16, [2047, 1], 3, 0),                 # forced odd cluster size with grouped queries (2 query tiles)
    (8, 2, 128, 16, [2047, 1], 3, 2),
    (32, 32, 128, 16, [1000], 0, 0),                  # the benchmark's attention shape: 32 heads, 4 splits of 4 tiles
    # more (sequence, kv head, query tile) units than CTA slots: two CTAs per SM on a two-stage ring, with one, two and
    # four query tiles per CTA
    (8, 8, 64, 64, [70, 1, 130, 257, 64] * 8, 0, 0),
    (8, 8, 64, 64, [70, 1, 130, 257, 64] * 8, 0, 4),
    (8, 8, 128, 64, [70, 1, 130, 257, 64] * 8, 0, 0),
    (8, 8, 128, 64, [70, 1, 130, 257, 64] * 8, 0, 4),
    (16, 8, 128, 32, [200, 5, 129] * 6, 0, 2),        # grouped queries, four tiles per kv head, two per CTA
    (16, 8, 128, 32, [200, 5, 129] * 24, 0, 0),       # enough units (more than six waves of CTAs) for the step's own choice of two
]


@pytest.mark.parametrize("hq,hkv,hd,c,lens,splits,q_tiles", CASES)
def test_fused_window_attention_vs_oracle_trace(hq, hkv, hd, c, lens, splits, q_tiles):
    cfg, acc, ss, kc, vc, max_seq, want_attn, want_k, want_v = _case(hq, hkv, hd, c, lens, seed=40 + c)
    B = len(lens)
    kcd = kc.to(torch.bfloat16).cuda().contiguous()
    vcd = vc.to(torch.bfloat16).cuda().contiguous()
    assert torch.equal(kcd.float().cpu(), kc)                   # the oracle's cached rows are bf16 values
    accd, ssd = acc.cuda().contiguous(), ss.cuda().contiguous()
    out = engine.fc_op_fused_window_attention(accd, ssd, cfg.rms_eps, cfg.d_model, cfg.rope_theta, kcd, vcd,
                                              torch.tensor(lens, dtype=torch.int32).cuda(), c, hq, max(lens), splits, q_tiles)
    out = out.cpu().numpy().reshape(B, c, hq * hd)
    assert float(accd.abs().max()) == 0.0 and float(ssd.abs().max()) == 0.0      # consumed
    for b, L in enumerate(lens):
        # the window's K/V rows as stored: within one bf16 step of the oracle's, nearly all identical
        for got_t, want in ((kcd, want_k[b]), (vcd, want_v[b])):
            got = got_t[b, :, L:L + c].float().cpu().transpose(0, 1).reshape(c, hkv * hd).numpy()
            # one step of an 8-bit significand at most; elements that are small through cancellation carry the fp32
            # summation-order difference of their 256 terms instead (absolute, ~1e-6)
            step = np.maximum(np.abs(want) * 2.0 ** -7, 1e-5)
            assert (np.abs(got - want) <= step).all(), float((np.abs(got - want) - step).max())
            assert (got != want).mean() < 0.01
        vmax = max(float(np.abs(want_v[b]).max()), float(vc[b].abs().max()))
        err = np.abs(out[b] - want_attn[b])
        assert err.max() < 2.0 ** -8 * vmax, (b, L, err.max(), vmax)
        assert np.sqrt((err ** 2).mean()) < 2e-4 * vmax, (b, L, np.sqrt((err ** 2).mean()), vmax)
    # rows beyond the window stay untouched (zero) in the cache
    for b, L in enumerate(lens):
        assert float(kcd[b, :, L + c:].float().abs().max()) == 0.0


def test_fused_window_attention_rejects_bad_arguments():
    from paper_2311_08263_b200 import lib
    l = lib.load()
    assert l.fc_op_fused_window_attention_scratch_bytes(1, 8, 4, 4, 32, 64, 10) == 0      # head_dim 32: FMA path only
    assert l.fc_op_fused_window_attention_scratch_bytes(1, 8, 4, 3, 64, 64, 10) == 0
    t = torch.zeros(64, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    n = l.fc_op_fused_window_attention_scratch_bytes(1, 8, 4, 4, 64, 64, 10)
    assert n > 0
    assert l.fc_op_fused_window_attention(None, t.data_ptr(), 1e-5, 8, 1e4, t.data_ptr(), t.data_ptr(), t.data_ptr(),
                                          t.data_ptr(), 1, 8, 4, 4, 64, 64, 10, 0, 0, t.data_ptr(), n, st) == lib.FC_ERR_ARG
    assert l.fc_op_fused_window_attention(t.data_ptr(), t.data_ptr(), 1e-5, 8, 1e4, t.data_ptr(), t.data_ptr(), t.data_ptr(),
                                          t.data_ptr(), 1, 8, 4, 4, 64, 64, 10, 0, 3, t.data_ptr(), n, st) == lib.FC_ERR_ARG
    assert l.fc_op_fused_window_attention(t.data_ptr(), t.data_ptr(), 1e-5, 8, 1e4, t.data_ptr(), t.data_ptr(),
                                          t.data_ptr(), t.data_ptr(), 1, 8, 4, 4, 64, 64, 60, 0, 0, t.data_ptr(), n,
                                          st) == lib.FC_ERR_CAPACITY
