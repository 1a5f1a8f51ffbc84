"""The allocation-free window-attention entry point against the regular one.

Some hosts of this library may not call cudaMalloc (their device memory belongs to a serving process's
arena, or they must stay out of the allocator once running).  For them the library carries a fixed
scratch array; this test calls that entry point through the C ABI twice in a row - the second time on
a different, smaller problem so that leftovers of the first call in the shared array would show - and
checks each result against fc_op_window_attention with caller-provided scratch.  This file is named so
that pytest collects it last.
"""
import numpy as np
import pytest
import torch

from paper_2311_08263_b200 import engine, lib, workload as wl

pytestmark = pytest.mark.gpu

TOL = 2e-5      # the fp32 tolerance of the attention parity test


def _case(seed, B, hq, hkv, hd, c, lens, dtype):
    max_seq = max(lens) + c + 5
    q = wl.hash_normal(seed, 1, B * c * hq * hd).view(B * c, hq * hd).to(dtype).cuda()
    k = wl.hash_normal(seed, 2, B * hkv * max_seq * hd).view(B, hkv, max_seq, hd).to(dtype).cuda()
    v = wl.hash_normal(seed, 3, B * hkv * max_seq * hd).view(B, hkv, max_seq, hd).to(dtype).cuda()
    kv_len = torch.tensor(lens, dtype=torch.int32).cuda()
    return q, k, v, kv_len, max_seq


def _noalloc(q, k, v, kv_len, c, hq, max_len):
    l = lib.load()
    B, hkv, max_seq, hd = k.shape
    out = torch.full((B * c, hq * hd), float("nan"), dtype=torch.float32, device=q.device)
    dt = lib.FC_F32 if q.dtype == torch.float32 else lib.FC_BF16
    rc = l.fc_op_window_attention_noalloc(q.data_ptr(), k.data_ptr(), v.data_ptr(), kv_len.data_ptr(),
                                          out.data_ptr(), B, c, hq, hkv, hd, max_seq, max_len, dt,
                                          torch.cuda.current_stream().cuda_stream)
    return rc, out


def test_noalloc_attention_matches_regular_entry_point_twice():
    cases = [dict(seed=5, B=3, hq=8, hkv=2, hd=64, c=8, lens=[700, 130, 0], dtype=torch.float32),
             dict(seed=6, B=1, hq=4, hkv=4, hd=128, c=16, lens=[150], dtype=torch.bfloat16)]
    for kw in cases:
        q, k, v, kv_len, _ = _case(**kw)
        c, hq, max_len = kw["c"], kw["hq"], max(kw["lens"])
        want = engine.fc_op_window_attention(q, k, v, kv_len, c, hq, max_len)
        rc, got = _noalloc(q, k, v, kv_len, c, hq, max_len)
        assert rc == lib.FC_OK
        torch.cuda.synchronize()
        assert torch.isfinite(got).all()
        assert (got - want).abs().max().item() <= TOL


def test_noalloc_attention_refuses_oversized_problems():
    l = lib.load()
    # 8 sequences x 64 rows x 32 heads at 8192 cached tokens need far more than the built-in array
    need = l.fc_op_window_attention_scratch_bytes(8, 64, 32, 32, 128, 8192, lib.FC_BF16)
    assert need > lib.FC_NOALLOC_SCRATCH_BYTES
    dummy = torch.zeros(16, device="cuda")
    rc = l.fc_op_window_attention_noalloc(dummy.data_ptr(), dummy.data_ptr(), dummy.data_ptr(), dummy.data_ptr(),
                                          dummy.data_ptr(), 8, 64, 32, 32, 128, 8192 + 64, 8192, lib.FC_BF16,
                                          torch.cuda.current_stream().cuda_stream)
    assert rc == lib.FC_ERR_CAPACITY
