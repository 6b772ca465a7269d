"""faedkv_decode_attn_static: the context-free, allocation-free decode attention.

Some callers cannot allocate device memory at the point where they need attention (they run inside
a stream capture, under a memory pool that was handed out once, or as a plugin that only receives
tensors).  For them the library carries a fixed scratch array and one extra entry point.  This file
checks, through the C ABI, that the entry point returns what faedkv_decode_attn returns -- on two
calls in a row, because the second call starts from the scratch contents the first one left -- and
that it refuses sizes that do not fit.  It is collected last on purpose.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

ATTN_MAX_ABS = 2e-3


@pytest.fixture(scope="module")
def fk():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2507_20030_b200 import binding, build
    build.build()
    binding.load()
    return binding


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_static_entry_point_matches_context_call_twice(fk, dtype):
    from paper_2507_20030_b200 import synth
    P = T = 1024
    M, B, H, HQ = 96, 2, 4, 16
    kvd = fk.BF16 if dtype == torch.bfloat16 else fk.F32
    ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=kvd,
                     prefill_mode=fk.PREFILL_SIMT)
    ctx.plan(0, fk.mask_mixed(P, M, 0, 77))
    bins = torch.from_numpy(ctx.get_bins(0)).cuda()
    K, V = synth.make_kv(123, B, H, T, 128, dtype=dtype)
    cK, cV = ctx.alloc_coef(0, B), ctx.alloc_coef(0, B)
    t_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    ctx.compress_prefill(0, K.cuda(), V.cuda(), cK, cV, t_len)
    for call in range(2):
        q = synth.make_q(123, call, B, HQ, 128, dtype=dtype).cuda()
        want = torch.empty((B, HQ, 128), dtype=dtype, device="cuda")
        ctx.decode_attn(0, q, cK, cV, t_len, want)
        got = torch.full_like(want, float("nan"))
        fk.decode_attn_static(P, H, HQ, kvd, bins, q, cK, cV, t_len, got)
        torch.cuda.synchronize()
        diff = (got.double() - want.double()).abs().max().item()
        assert np.isfinite(diff) and diff <= ATTN_MAX_ABS, (call, diff)
    ctx.close()


def test_static_entry_point_rejects_what_does_not_fit(fk):
    P, H, HQ, B, M = 1 << 20, 8, 32, 4, 64          # scores alone would need 512 MiB
    z = torch.zeros(16, device="cuda")
    bins = torch.zeros(M, dtype=torch.int32, device="cuda")
    t_len = torch.ones(B, dtype=torch.int32, device="cuda")
    q = torch.zeros((B, HQ, 128), device="cuda")
    with pytest.raises(fk.FaedkvError) as e:
        fk.decode_attn_static(P, H, HQ, fk.F32, bins, q, z, z, t_len, q)
    assert e.value.code == -3 and "static scratch" in str(e.value)
    with pytest.raises(fk.FaedkvError) as e:
        fk.decode_attn_static(64, 3, 8, fk.F32, bins[:4], q, z, z, t_len, q)
    assert e.value.code == -4
