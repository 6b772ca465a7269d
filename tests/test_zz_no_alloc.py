"""faedkv_decode_attn_static: the context-free, allocation-free decode attention.

Some callers cannot allocate device memory at the point where they need attention (they run inside
a stream capture, under a memory pool that was handed out once, or as a plugin that only receives
tensors).  For them the library carries a fixed scratch array and one extra entry point.  This file
checks, through the C ABI, that the entry point returns what the float64 oracle and what
faedkv_decode_attn return -- on two calls in a row, because the second call starts from the scratch
contents the first one left -- and that it refuses sizes that do not fit.  It is collected last on
purpose.
"""
import numpy as np
import pytest
import torch

from helpers import ATTN_MAX_ABS, oracle_decode_attn, to_np64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fk():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2507_20030_b200 import binding, build
    build.build()
    binding.load()
    return binding


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("P,M,B,H,HQ", [
    (1024, 96, 2, 4, 16),     # 4 query heads per kv head
    (200, 40, 3, 5, 5),       # P not a power of two; one query head per kv head; 5 of 32 padded columns real
    (512, 33, 1, 5, 40),      # 8 query heads per kv head; two column blocks
    (96, 20, 2, 2, 14),       # 7 query heads per kv head
])
def test_static_entry_point_matches_oracle_and_context_call_twice(fk, oracle, dtype, P, M, B, H, HQ):
    from paper_2507_20030_b200 import synth
    T = P
    kvd = fk.BF16 if dtype == torch.bfloat16 else fk.F32
    ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=kvd,
                     prefill_mode=fk.PREFILL_SIMT)
    rng = np.random.default_rng(P + M)
    mask = np.zeros(P // 2 + 1, dtype=np.uint8)
    mask[np.sort(rng.choice(P // 2 + 1, size=M, replace=False))] = 1
    mask[0] = 1
    ctx.plan(0, mask)
    host_bins = oracle.plan(P, mask)
    assert ctx.get_bins(0).tobytes() == host_bins.tobytes()
    bins = torch.from_numpy(host_bins).cuda()
    K, V = synth.make_kv(123, B, H, T, 128, dtype=dtype)
    if dtype == torch.bfloat16:
        # bf16 outputs sit on a grid of relative spacing 2^-9: with V of unit scale that rounding alone can reach
        # the absolute bar, so V is scaled by 1/8 (exact) for bf16; float32 runs unscaled
        V = (V * 0.125).to(dtype)
    cK, cV = ctx.alloc_coef(0, B), ctx.alloc_coef(0, B)
    t_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    ctx.compress_prefill(0, K.cuda(), V.cuda(), cK, cV, t_len)
    t_len[B - 1] = P // 3 + 1                      # a ragged batch: the last sequence attends to fewer positions
    torch.cuda.synchronize()
    t_np = t_len.cpu().numpy()
    for call in range(2):
        q = synth.make_q(123, call, B, HQ, 128, dtype=dtype)
        want = oracle_decode_attn(oracle, q, to_np64(cK), to_np64(cV), P, host_bins, t_np)
        ref = torch.empty((B, HQ, 128), dtype=dtype, device="cuda")
        ctx.decode_attn(0, q.cuda(), cK, cV, t_len, ref)
        got = torch.full_like(ref, float("nan"))
        fk.decode_attn_static(P, H, HQ, kvd, bins, q.cuda(), cK, cV, t_len, got)
        torch.cuda.synchronize()
        err = np.abs(to_np64(got) - want).max()
        assert np.isfinite(err) and err <= ATTN_MAX_ABS, (call, err)
        diff = (got.double() - ref.double()).abs().max().item()
        assert diff <= ATTN_MAX_ABS, (call, diff)
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
    assert e.value.code == -4                        # 8 query heads over 3 kv heads
    with pytest.raises(fk.FaedkvError) as e:
        fk.decode_attn_static(64, 9, 81, fk.F32, bins[:4], q, z, z, t_len, q)
    assert e.value.code == -4                        # 9 query heads per kv head
