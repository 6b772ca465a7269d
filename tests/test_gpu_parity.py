"""GPU parity: every call of the C ABI against the float64 oracle on the same seeded inputs.

Small cases are compared element by element; they span several tiles of every
kernel plus ragged tails (bin counts, token counts, head counts that are not
multiples of the tile sizes), both storage types, wrap-around positions, and
the degenerate masks (a single bin, all bins).
"""
import numpy as np
import pytest
import torch

from helpers import (ATTN_MAX_ABS, REL_L2_BF16, REL_L2_F32, oracle_append, oracle_compress,
                     oracle_decode_attn, oracle_reconstruct, rel_l2, to_np64)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fk():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2507_20030_b200 import binding, build
    build.build()
    binding.load()
    return binding


def _tol(dtype):
    return REL_L2_F32 if dtype == torch.float32 else REL_L2_BF16


def _kvd(fk, dtype):
    return fk.F32 if dtype == torch.float32 else fk.BF16


def _bf16_vscale(dtype):
    """bf16 outputs are rounded to a grid of relative spacing 2^-9; where an attention output approaches
    single rows of V (a window of exact tokens, a sharp softmax) that rounding alone would eat the absolute
    bar, so bf16 cases scale V by 1/4 (a power of two: exact).  float32 cases run unscaled."""
    return 0.25 if dtype == torch.bfloat16 else 1.0


def _rows_close(got, want, tol, what=""):
    """Beside the whole-tensor rel-L2 (the acceptance metric), a bound per row of 128 channels: every
    (..., row) vector must match to tol_row relative to the root-mean-square norm of its unit's non-zero rows (K has a
    few channels ten times larger than the rest, so a bound relative to each row's own norm would be
    dominated by them just like the tensor norm; the unit's typical row norm is the scale an error in ANY
    single row has to stay small against).  A wrong element in one row of a large tensor moves the
    tensor's rel-L2 by almost nothing and fails here."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    err = np.sqrt(((got - want) ** 2).sum(axis=-1))                 # [..., rows]
    sq = (want ** 2).sum(axis=-1)
    n_live = np.maximum((sq > 0).sum(axis=-1, keepdims=True), 1)     # rows past a live length are all zero: left out
    rms = np.sqrt(sq.sum(axis=-1, keepdims=True) / n_live)          # per unit, over its non-zero rows
    rms = np.where(rms > 0, rms, 1.0)
    worst = float((err / rms).max())
    assert worst <= tol, (what, worst)


# Per-row companions of the rel-L2 bars: a row's error is a sum over fewer terms than the tensor's, so its
# relative size fluctuates; 4x the tensor bar holds every row of a correct result with margin and is still
# far below the O(1) error of a wrong or missing element.
ROW_F32 = 4e-4
ROW_BF16 = 1.2e-2


def _row_tol(dtype):
    return ROW_F32 if dtype == torch.float32 else ROW_BF16


def _mask_from_bins(P, bins):
    m = np.zeros(P // 2 + 1, dtype=np.uint8)
    m[np.asarray(bins)] = 1
    return m


def _random_mask(P, M, seed):
    rng = np.random.default_rng(seed)
    bins = np.sort(rng.choice(P // 2 + 1, size=M, replace=False))
    return _mask_from_bins(P, bins)


def _make(seed, B, H, T, dtype, pos0=0):
    from paper_2507_20030_b200 import synth
    K, V = synth.make_kv(seed, B, H, T, 128, pos0=pos0, dtype=dtype, device="cpu")
    return K, V


# ----------------------------------------------------------------------------- plan
@pytest.mark.parametrize("P,M", [(64, 5), (100, 51), (2048, 256)])
def test_plan_bins_bit_exact(fk, oracle, P, M):
    ctx = fk.Context(n_layers=3, n_kv_heads=2, n_q_heads=2, n_dft=P, max_batch=1, kv_dtype=fk.F32)
    for layer in range(3):
        mask = _random_mask(P, M, 100 + layer)
        assert ctx.plan(layer, mask) == M
        got = ctx.get_bins(layer)
        want = oracle.plan(P, mask)
        assert got.dtype == np.int32 and got.tobytes() == want.tobytes()
        assert ctx.coef_bytes(layer, 1) == 1 * 2 * 2 * M * 128 * 4
    # re-planning a layer replaces its bins
    mask = _random_mask(P, M, 999)
    ctx.plan(0, mask)
    assert ctx.get_bins(0).tobytes() == oracle.plan(P, mask).tobytes()
    ctx.close()


def test_error_codes(fk):
    ctx = fk.Context(n_layers=2, n_kv_heads=2, n_q_heads=4, n_dft=64, max_batch=2, kv_dtype=fk.F32)
    dev = "cuda"
    K = torch.zeros(1, 2, 16, 128, device=dev)
    coef = torch.zeros(1, 2, 2, 4, 128, device=dev)
    t = torch.zeros(1, dtype=torch.int32, device=dev)
    with pytest.raises(fk.FaedkvError) as e:
        ctx.compress_prefill(0, K, K, coef, coef, t)
    assert e.value.code == -2                                   # not planned
    with pytest.raises(fk.FaedkvError) as e:
        ctx.plan(0, np.zeros(33, dtype=np.uint8))
    assert e.value.code == -1                                   # empty mask
    ctx.plan(0, _mask_from_bins(64, [0, 1, 2, 5]))
    with pytest.raises(fk.FaedkvError) as e:
        ctx.plan(5, _mask_from_bins(64, [0]))
    assert e.value.code == -1                                   # layer out of range
    K3 = torch.zeros(3, 2, 16, 128, device=dev)
    with pytest.raises(fk.FaedkvError) as e:
        ctx.compress_prefill(0, K3, K3, coef, coef, t)
    assert e.value.code == -3                                   # batch > max_batch
    with pytest.raises(fk.FaedkvError) as e:
        ctx._check(ctx._lib.faedkv_compress_prefill(ctx._h, 0, K.data_ptr() + 4, K.data_ptr(), 1, 16,
                                                    coef.data_ptr(), coef.data_ptr(), t.data_ptr(), None))
    assert e.value.code == -5                                   # misaligned
    with pytest.raises(fk.FaedkvError) as e:
        ctx._check(ctx._lib.faedkv_append(ctx._h, 0, None, K.data_ptr(), 1, coef.data_ptr(),
                                          coef.data_ptr(), t.data_ptr(), None))
    assert e.value.code == -1                                   # NULL tensor
    with pytest.raises(fk.FaedkvError) as e:
        ctx.reconstruct(0, coef, coef, t, 65, K, K)
    assert e.value.code == -3                                   # L > P
    assert "outside" in str(e.value)
    # the context is still usable after errors
    ctx.compress_prefill(0, K, K, coef, coef, t)
    torch.cuda.synchronize()
    assert int(t[0]) == 16 and ctx.device_status() == 0
    ctx.close()


# ----------------------------------------------------------------------------- prefill
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("P,T,M,B,H", [(64, 64, 7, 1, 1), (100, 77, 51, 2, 3), (96, 250, 33, 1, 2),
                                       (512, 512, 257, 1, 1)])
def test_prefill_simt_matches_oracle(fk, oracle, dtype, P, T, M, B, H):
    ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=H, n_dft=P, max_batch=B, kv_dtype=_kvd(fk, dtype),
                     prefill_mode=fk.PREFILL_SIMT)
    mask = _random_mask(P, M, P + T)
    ctx.plan(0, mask)
    bins = oracle.plan(P, mask)
    K, V = _make(11 + P, B, H, T, dtype)
    cK, cV = ctx.alloc_coef(0, B), ctx.alloc_coef(0, B)
    t_len = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    ctx.compress_prefill(0, K.cuda(), V.cuda(), cK, cV, t_len)
    torch.cuda.synchronize()
    assert t_len.tolist() == [T] * B
    for c, X in ((cK, K), (cV, V)):
        want = oracle_compress(oracle, X, P, bins)
        assert rel_l2(to_np64(c), want) <= REL_L2_F32
        _rows_close(to_np64(c), want, ROW_F32, "bin rows")
    ctx.close()


# ----------------------------------------------------------------------------- append
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("P,M,B,H,steps", [(64, 33, 2, 3, 70), (1000, 77, 3, 8, 12), (256, 1, 1, 5, 5)])
def test_append_matches_oracle(fk, oracle, dtype, P, M, B, H, steps):
    from paper_2507_20030_b200 import synth
    ctx = fk.Context(n_layers=2, n_kv_heads=H, n_q_heads=H, n_dft=P, max_batch=B, kv_dtype=_kvd(fk, dtype),
                     prefill_mode=fk.PREFILL_SIMT)
    mask = _random_mask(P, M, 5 * P + M)
    ctx.plan(1, mask)
    bins = oracle.plan(P, mask)
    rng = np.random.default_rng(3)
    cK = torch.from_numpy(rng.standard_normal((B, H, 2, M, 128)).astype(np.float32)).cuda()
    cV = torch.from_numpy(rng.standard_normal((B, H, 2, M, 128)).astype(np.float32)).cuda()
    refK, refV = to_np64(cK), to_np64(cV)
    t0 = np.array([0, P - 3, 5 * P + 1][:B], dtype=np.int32)       # ragged; wraps past P
    t_len = torch.from_numpy(t0.copy()).cuda()
    for s in range(steps):
        k, v = synth.make_token(77, s, B, H, 128, pos=int(t0[0]) + s, dtype=dtype)
        ctx.append(1, k.cuda(), v.cuda(), cK, cV, t_len)
        oracle_append(oracle, refK, P, bins, t0 + s, k)
        oracle_append(oracle, refV, P, bins, t0 + s, v)
    torch.cuda.synchronize()
    assert t_len.cpu().numpy().tolist() == (t0 + steps).tolist()
    assert rel_l2(to_np64(cK), refK) <= REL_L2_F32
    assert rel_l2(to_np64(cV), refV) <= REL_L2_F32
    _rows_close(to_np64(cK), refK, ROW_F32, "bin rows of K")
    _rows_close(to_np64(cV), refV, ROW_F32, "bin rows of V")
    ctx.close()


def test_appends_from_zero_equal_prefill(fk):
    """T successive appends from the zero state reproduce the batch transform (float32 rounding apart)."""
    from paper_2507_20030_b200 import synth
    P, T, M, B, H = 128, 128, 40, 1, 2
    ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=H, n_dft=P, max_batch=B, kv_dtype=fk.F32,
                     prefill_mode=fk.PREFILL_SIMT)
    ctx.plan(0, _random_mask(P, M, 1))
    K, V = synth.make_kv(5, B, H, T, 128)
    K, V = K.cuda(), V.cuda()
    cK, cV = ctx.alloc_coef(0, B), ctx.alloc_coef(0, B)
    t_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    ctx.compress_prefill(0, K, V, cK, cV, t_len)
    aK, aV = torch.zeros_like(cK), torch.zeros_like(cV)
    t2 = torch.zeros(B, dtype=torch.int32, device="cuda")
    for n in range(T):
        ctx.append(0, K[:, :, n].contiguous(), V[:, :, n].contiguous(), aK, aV, t2)
    torch.cuda.synchronize()
    assert t2.tolist() == t_len.tolist() == [T]
    assert rel_l2(to_np64(aK), to_np64(cK)) <= 1e-5
    assert rel_l2(to_np64(aV), to_np64(cV)) <= 1e-5
    ctx.close()


def test_checkpoint_restore_is_bit_exact(fk):
    """State is plain memory: append after a copy-out / copy-in equals the uninterrupted run."""
    from paper_2507_20030_b200 import synth
    P, M, B, H = 256, 48, 2, 4
    ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=H, n_dft=P, max_batch=B, kv_dtype=fk.BF16,
                     prefill_mode=fk.PREFILL_SIMT)
    ctx.plan(0, fk.mask_mixed(P, M, 0, 9))
    K, V = synth.make_kv(8, B, H, 200, 128, dtype=torch.bfloat16)
    cK, cV = ctx.alloc_coef(0, B), ctx.alloc_coef(0, B)
    t_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    ctx.compress_prefill(0, K.cuda(), V.cuda(), cK, cV, t_len)
    toks = [synth.make_token(8, s, B, H, 128, pos=200 + s, dtype=torch.bfloat16) for s in range(6)]
    for k, v in toks[:3]:
        ctx.append(0, k.cuda(), v.cuda(), cK, cV, t_len)
    saved = (cK.cpu().clone(), cV.cpu().clone(), t_len.cpu().clone())
    for k, v in toks[3:]:
        ctx.append(0, k.cuda(), v.cuda(), cK, cV, t_len)
    rK, rV, rt = saved[0].cuda(), saved[1].cuda(), saved[2].cuda()
    for k, v in toks[3:]:
        ctx.append(0, k.cuda(), v.cuda(), rK, rV, rt)
    torch.cuda.synchronize()
    assert torch.equal(rK, cK) and torch.equal(rV, cV) and torch.equal(rt, t_len)
    ctx.close()


# ----------------------------------------------------------------------------- reconstruct
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("P,M,L,B,H,tl", [(64, 33, 64, 2, 1, [64, 40]), (100, 20, 77, 1, 3, [300]),
                                          (512, 100, 512, 1, 2, [512]), (96, 1, 50, 1, 1, [96]),
                                          (2048, 256, 2048, 1, 8, [2111]),      # config-0 shape after its 64 appends
                                          (8192, 64, 5001, 2, 3, [8192, 77]),   # two-pass split 64 x 64; odd L; ragged
                                          (256, 129, 255, 1, 1, [256]),         # every bin retained
                                          # 24 column blocks of 128 x 128 points: more than the ring between the two
                                          # passes holds, so ring slots are reused; odd L
                                          (32768, 64, 20001, 1, 3, [32768]),
                                          (131072, 32, 131072, 1, 1, [100000]),  # 256 x 256 points, the largest split
                                          (64, 33, 64, 1, 2, [64])])            # the smallest grid: 8 x 4 points
def test_reconstruct_matches_oracle(fk, oracle, dtype, P, M, L, B, H, tl):
    mask = _random_mask(P, M, 9 * P + L) if M > 1 else _mask_from_bins(P, [0])
    bins = oracle.plan(P, mask)
    rng = np.random.default_rng(L)
    cK = torch.from_numpy((rng.standard_normal((B, H, 2, M, 128)) * P ** 0.5).astype(np.float32)).cuda()
    cV = torch.from_numpy((rng.standard_normal((B, H, 2, M, 128)) * P ** 0.5).astype(np.float32)).cuda()
    t_np = np.array(tl, dtype=np.int32)
    t_len = torch.from_numpy(t_np).cuda()
    wantK = oracle_reconstruct(oracle, to_np64(cK), P, bins, t_np, L)
    wantV = oracle_reconstruct(oracle, to_np64(cV), P, bins, t_np, L)
    modes = [(m, 0) for m in _decode_modes(fk, dtype, P)]
    if P & (P - 1) == 0 and P >= 64:
        modes.append((fk.DECODE_AUTO, 1))             # the FFT-shaped reconstruction's two engines, each forced:
        if P <= (1 << 17):                            # a launch per pass, and the persistent kernel
            modes.append((fk.DECODE_AUTO, 2))
    if P > 16384:
        modes = [m for m in modes if m[0] in (fk.DECODE_AUTO, fk.DECODE_FFT)]     # the dense evaluations are O(P M) per channel
    for mode, engine in modes:
        ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=H, n_dft=P, max_batch=B, kv_dtype=_kvd(fk, dtype),
                         decode_mode=mode, recon_engine=engine)
        ctx.plan(0, mask)
        Ko = torch.full((B, H, L, 128), 7.0, dtype=dtype, device="cuda")
        Vo = torch.full((B, H, L, 128), 7.0, dtype=dtype, device="cuda")
        ctx.reconstruct(0, cK, cV, t_len, L, Ko, Vo)
        torch.cuda.synchronize()
        assert rel_l2(to_np64(Ko), wantK) <= _tol(dtype), (mode, engine)
        assert rel_l2(to_np64(Vo), wantV) <= _tol(dtype), (mode, engine)
        _rows_close(to_np64(Ko), wantK, _row_tol(dtype), ("token rows of K", mode, engine))
        _rows_close(to_np64(Vo), wantV, _row_tol(dtype), ("token rows of V", mode, engine))
        for b in range(B):                                           # rows past the live length are exactly zero
            live = min(int(t_np[b]), P)
            if live < L:
                assert float(Ko[b, :, live:].abs().max()) == 0.0
        # K only
        Ko2 = torch.zeros_like(Ko)
        ctx.reconstruct(0, cK, None, t_len, L, Ko2, None)
        torch.cuda.synchronize()
        assert torch.equal(Ko2, Ko)
        assert ctx.device_status() == 0
        ctx.close()


def test_all_bins_round_trip(fk):
    """All bins retained: reconstruct(compress(x)) returns x (float32)."""
    P, B, H = 128, 1, 2
    ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=H, n_dft=P, max_batch=B, kv_dtype=fk.F32,
                     prefill_mode=fk.PREFILL_SIMT)
    ctx.plan(0, np.ones(P // 2 + 1, dtype=np.uint8))
    K, V = _make(2, B, H, P, torch.float32)
    cK, cV = ctx.alloc_coef(0, B), ctx.alloc_coef(0, B)
    t_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    ctx.compress_prefill(0, K.cuda(), V.cuda(), cK, cV, t_len)
    Ko, Vo = torch.empty_like(K, device="cuda"), torch.empty_like(V, device="cuda")
    ctx.reconstruct(0, cK, cV, t_len, P, Ko, Vo)
    torch.cuda.synchronize()
    assert rel_l2(to_np64(Ko), to_np64(K)) <= 1e-5
    assert rel_l2(to_np64(Vo), to_np64(V)) <= 1e-5
    ctx.close()


# ----------------------------------------------------------------------------- decode attention
def _decode_modes(fk, dtype, P):
    """Every evaluation of the two transforms that exists for this storage type and grid size."""
    modes = [fk.DECODE_AUTO, fk.DECODE_SIMT]
    if dtype == torch.bfloat16:
        modes.append(fk.DECODE_UMMA)
    if P & (P - 1) == 0 and P >= 64:
        modes.append(fk.DECODE_FFT)               # one kernel per column up to P = 16384
        modes.append(fk.DECODE_FFT_TWO_PASS)      # the two-pass kernels, which larger grids use
    return modes


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("P,T,M,B,H,HQ,tl,vscale", [
    (256, 256, 32, 2, 2, 8, None, 1.0),        # GQA 4, full length
    (200, 130, 37, 1, 3, 3, None, 1.0),        # MHA (1 query head per kv head), t < P, odd sizes
    (128, 128, 16, 2, 1, 8, [128, 70], 1.0),   # GQA 8, ragged lengths
    (512, 512, 64, 1, 8, 32, None, 1.0),       # 32 query heads, GQA 4
    (128, 128, 24, 1, 20, 40, None, 1.0),      # 40 query heads: two column blocks, GQA 2
    # smallest FFT-shaped grid, every bin retained, odd live length.  With all bins and few tokens the
    # softmax is sharp and the output is close to single rows of V; for bf16 tensors ONLY, V is scaled so
    # that the bf16 output grid (relative 2^-9) stays finer than the absolute tolerance.  float32 tensors
    # have no such grid and run unscaled.
    (64, 64, 33, 1, 2, 4, [33], 0.125),
    (4096, 4096, 96, 3, 2, 8, [4096, 1, 2049], 0.125),   # two-pass split 64 x 32; a one-token sequence
    # 320 columns: more than the GPU holds at once, so the column-transform path cuts the batch into two
    # runs of sequences (2 + 3) on two streams; ragged lengths
    (128, 128, 20, 5, 8, 64, [128, 9, 77, 128, 30], 0.125),
])
def test_decode_attn_matches_oracle(fk, oracle, dtype, P, T, M, B, H, HQ, tl, vscale):
    from paper_2507_20030_b200 import synth
    mask = _random_mask(P, M, 3 * P + M)
    mask[0] = 1
    M = int(mask.sum())
    bins = oracle.plan(P, mask)
    K, V = _make(21 + P, B, H, T, dtype)
    if dtype == torch.bfloat16:
        V = (V * vscale).to(dtype)            # a power of two: exact; see the note at the cases above
    q = synth.make_q(5, 0, B, HQ, 128, dtype=dtype)
    want = want2 = None
    for mode in _decode_modes(fk, dtype, P):
        ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=_kvd(fk, dtype),
                         prefill_mode=fk.PREFILL_SIMT, decode_mode=mode)
        ctx.plan(0, mask)
        cK, cV = ctx.alloc_coef(0, B), ctx.alloc_coef(0, B)
        t_len = torch.zeros(B, dtype=torch.int32, device="cuda")
        ctx.compress_prefill(0, K.cuda(), V.cuda(), cK, cV, t_len)
        if tl is not None:
            # shorter sequences: recompute their state from the first tl[b] tokens only
            for b, t in enumerate(tl):
                if t < T:
                    Kb, Vb = K[b:b + 1, :, :t].contiguous().cuda(), V[b:b + 1, :, :t].contiguous().cuda()
                    ctx.compress_prefill(0, Kb, Vb, cK[b:b + 1], cV[b:b + 1], t_len[b:b + 1])
        out = torch.full((B, HQ, 128), float("nan"), dtype=dtype, device="cuda")
        ctx.decode_attn(0, q.cuda(), cK, cV, t_len, out)
        torch.cuda.synchronize()
        t_np = t_len.cpu().numpy()
        if want is None:
            want = oracle_decode_attn(oracle, q, to_np64(cK), to_np64(cV), P, bins, t_np)
            want2 = oracle_decode_attn(oracle, q, to_np64(cK), to_np64(cV), P, bins, t_np, scale=0.05)
        err = np.abs(to_np64(out) - want).max()
        assert err <= ATTN_MAX_ABS, (mode, err)
        # explicit scale
        out2 = torch.empty_like(out)
        ctx.decode_attn(0, q.cuda(), cK, cV, t_len, out2, scale=0.05)
        torch.cuda.synchronize()
        err2 = np.abs(to_np64(out2) - want2).max()
        assert err2 <= ATTN_MAX_ABS, (mode, err2)
        assert ctx.device_status() == 0
        ctx.close()


@pytest.mark.parametrize("seed", range(12))
def test_decode_attn_random_shapes(fk, oracle, seed):
    """Seeded random shapes over every column length the one-kernel transform is instantiated for
    (P = 64 ... 16384), random retained sets, GQA factors, batch sizes and ragged live lengths (random
    coefficient planes with a decaying spectrum, so that the oracle's materialised form stays cheap):
    default mode and the two-pass kernels against the oracle."""
    from paper_2507_20030_b200 import synth
    rng = np.random.default_rng(1000 + seed)
    P = 1 << int(rng.integers(6, 15))
    GQ = int(rng.choice([1, 2, 4, 8]))
    H = int(rng.integers(1, 4))
    B = int(rng.integers(1, 4))
    M = int(rng.integers(1, min(P // 2 + 1, 96) + 1))
    HQ = H * GQ
    mask = _random_mask(P, M, seed)
    bins = oracle.plan(P, mask)
    amp = np.sqrt(P) * np.exp(-np.arange(M) / max(M / 3.0, 1.0))[None, None, None, :, None]
    cK = torch.from_numpy((rng.standard_normal((B, H, 2, M, 128)) * amp).astype(np.float32)).cuda()
    cV = torch.from_numpy((rng.standard_normal((B, H, 2, M, 128)) * amp).astype(np.float32)).cuda()
    tl = rng.integers(1, 2 * P, size=B).astype(np.int32)          # some beyond P: live length is capped
    t_len = torch.from_numpy(tl).cuda()
    q = synth.make_q(seed, 0, B, HQ, 128, dtype=torch.float32)
    want = oracle_decode_attn(oracle, q, to_np64(cK), to_np64(cV), P, bins, tl)
    for mode in (fk.DECODE_AUTO, fk.DECODE_FFT_TWO_PASS):
        ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=fk.F32, decode_mode=mode)
        ctx.plan(0, mask)
        out = torch.full((B, HQ, 128), float("nan"), dtype=torch.float32, device="cuda")
        ctx.decode_attn(0, q.cuda(), cK, cV, t_len, out)
        torch.cuda.synchronize()
        err = np.abs(to_np64(out) - want).max()
        assert err <= ATTN_MAX_ABS, (seed, P, M, B, H, GQ, mode, err)
        assert ctx.device_status() == 0
        ctx.close()


@pytest.mark.parametrize("P,M,B,H,HQ", [(32768, 48, 1, 2, 8), (131072, 32, 2, 1, 4), (16384, 64, 3, 2, 4),
                                         (8192, 64, 2, 2, 2), (4096, 32, 2, 1, 8), (65536, 32, 1, 2, 4), (262144, 32, 1, 1, 2),
                                         (524288, 32, 1, 1, 1)])       # the largest grid the FFT-shaped path takes
def test_decode_attn_fft_long_grids(fk, oracle, P, M, B, H, HQ):
    """FFT-shaped transforms at the grid sizes of the long-context workloads (few bins, so that the
    oracle's materialised reconstruction stays cheap); ragged live lengths."""
    from paper_2507_20030_b200 import synth
    dtype = torch.bfloat16
    ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=fk.BF16,
                     decode_mode=fk.DECODE_FFT)
    mask = fk.mask_mixed(P, M, 3, 17)
    ctx.plan(0, mask)
    bins = oracle.plan(P, mask)
    rng = np.random.default_rng(P + M)
    amp = np.sqrt(P) * np.exp(-np.arange(M) / (M / 3.0))[None, None, None, :, None]
    cK = torch.from_numpy((rng.standard_normal((B, H, 2, M, 128)) * amp).astype(np.float32)).cuda()
    cV = torch.from_numpy((rng.standard_normal((B, H, 2, M, 128)) * amp).astype(np.float32)).cuda()
    t_np = np.array([P, P // 3 + 1, 5][:B], dtype=np.int32)
    t_len = torch.from_numpy(t_np).cuda()
    q = synth.make_q(9, 1, B, HQ, 128, dtype=dtype)
    out = torch.empty((B, HQ, 128), dtype=dtype, device="cuda")
    ctx.decode_attn(0, q.cuda(), cK, cV, t_len, out)
    torch.cuda.synchronize()
    want = oracle_decode_attn(oracle, q, to_np64(cK), to_np64(cV), P, bins, t_np)
    err = np.abs(to_np64(out) - want).max()
    assert err <= ATTN_MAX_ABS, err
    ctx.close()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("P,M,B,H,HQ,t0", [(256, 40, 2, 2, 8, [100, 255]), (1024, 65, 1, 3, 6, [3000]),
                                           (200, 30, 2, 1, 2, [7, 199])])
def test_append_decode_attn_equals_the_two_calls(fk, oracle, dtype, P, M, B, H, HQ, t0):
    """The fused step: planes and counters bit-identical to faedkv_append, output equal to the oracle's
    attention on the updated state."""
    from paper_2507_20030_b200 import synth
    ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=_kvd(fk, dtype))
    mask = _random_mask(P, M, P + 3 * M)
    mask[0] = 1
    M = int(mask.sum())
    ctx.plan(0, mask)
    bins = oracle.plan(P, mask)
    rng = np.random.default_rng(M)
    cK = torch.from_numpy((rng.standard_normal((B, H, 2, M, 128)) * 4).astype(np.float32)).cuda()
    cV = torch.from_numpy((rng.standard_normal((B, H, 2, M, 128)) * 4).astype(np.float32)).cuda()
    sK, sV = cK.clone(), cV.clone()
    t_np = np.array(t0, dtype=np.int32)
    t_len = torch.from_numpy(t_np.copy()).cuda()
    t_sep = t_len.clone()
    out = torch.empty((B, HQ, 128), dtype=dtype, device="cuda")
    for s in range(3):
        k, v = synth.make_token(31, s, B, H, 128, pos=int(t_np[0]) + s, dtype=dtype)
        q = synth.make_q(31, s, B, HQ, 128, dtype=dtype)
        ctx.append_decode_attn(0, k.cuda(), v.cuda(), q.cuda(), cK, cV, t_len, out)
        ctx.append(0, k.cuda(), v.cuda(), sK, sV, t_sep)
        torch.cuda.synchronize()
        assert torch.equal(cK, sK) and torch.equal(cV, sV) and torch.equal(t_len, t_sep)
        want = oracle_decode_attn(oracle, q, to_np64(sK), to_np64(sV), P, bins, t_np + s + 1)
        err = np.abs(to_np64(out) - want).max()
        assert err <= ATTN_MAX_ABS, (s, err)
    ctx.close()


def test_decode_attn_dc_only_is_mean_of_v(fk):
    """Only bin 0 retained: the softmax is uniform and the output is the mean of V."""
    P, B, H, HQ = 64, 1, 2, 8
    ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=fk.F32,
                     prefill_mode=fk.PREFILL_SIMT)
    ctx.plan(0, _mask_from_bins(P, [0]))
    K, V = _make(4, B, H, P, torch.float32)
    cK, cV = ctx.alloc_coef(0, B), ctx.alloc_coef(0, B)
    t_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    ctx.compress_prefill(0, K.cuda(), V.cuda(), cK, cV, t_len)
    q = torch.randn(B, HQ, 128, generator=torch.Generator().manual_seed(1))
    out = torch.empty((B, HQ, 128), device="cuda")
    ctx.decode_attn(0, q.cuda(), cK, cV, t_len, out)
    torch.cuda.synchronize()
    want = V.double().mean(dim=2).repeat_interleave(HQ // H, dim=1).numpy()
    assert np.abs(to_np64(out) - want).max() <= 1e-5
    ctx.close()


def test_decode_attn_uneven_split_of_the_batch(fk, oracle):
    """An odd batch with more columns than the GPU holds at once: the call is cut into runs of 5 and 6
    sequences that run side by side on two streams, with different slice counts in their passes over C_V.
    Every output against the oracle (short ragged live lengths keep its materialised form cheap), the
    fused call on the same state, and the two-pass kernels, which never cut."""
    from paper_2507_20030_b200 import synth
    P, M, B, H, HQ = 16384, 512, 11, 8, 32
    dtype = torch.float32
    mask = fk.mask_mixed(P, M, 1, 23)
    bins = oracle.plan(P, mask)
    rng = np.random.default_rng(77)
    amp = np.sqrt(P) * np.exp(-np.arange(M) / (M / 3.0))[None, None, None, :, None]
    cK = torch.from_numpy((rng.standard_normal((B, H, 2, M, 128)) * amp).astype(np.float32)).cuda()
    cV = torch.from_numpy((rng.standard_normal((B, H, 2, M, 128)) * amp).astype(np.float32)).cuda()
    tl = rng.integers(1, 700, size=B).astype(np.int32)
    tl[3] = P + 5                                                 # one full-length sequence in the first run
    t_len = torch.from_numpy(tl).cuda()
    q = synth.make_q(3, 0, B, HQ, 128, dtype=dtype)
    want = oracle_decode_attn(oracle, q, to_np64(cK), to_np64(cV), P, bins, tl)
    outs = {}
    for mode in (fk.DECODE_AUTO, fk.DECODE_FFT_TWO_PASS):
        ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=fk.F32, decode_mode=mode)
        ctx.plan(0, mask)
        out = torch.full((B, HQ, 128), float("nan"), dtype=dtype, device="cuda")
        n0 = ctx.launch_count()
        for _ in range(3):                                        # repeated: a race between the runs need not show at once
            ctx.decode_attn(0, q.cuda(), cK, cV, t_len, out)
        torch.cuda.synchronize()
        if mode == fk.DECODE_AUTO:
            assert ctx.launch_count() - n0 == 3 * 5               # C_K pass, 2 column kernels, 2 passes over C_V
        err = np.abs(to_np64(out) - want).max()
        assert err <= ATTN_MAX_ABS, (mode, err)
        outs[mode] = out.clone()
        assert ctx.device_status() == 0
        ctx.close()
    assert (outs[fk.DECODE_AUTO] - outs[fk.DECODE_FFT_TWO_PASS]).abs().max().item() <= ATTN_MAX_ABS


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("GQ,P", [(3, 256), (5, 128), (6, 200), (7, 1024), (7, 96)])
def test_decode_attn_any_group_size(fk, oracle, dtype, GQ, P):
    """Query heads per kv head that do not divide 16 (7 is the grouping of the 28 / 4-head model the paper
    runs its retrieval test on): every decode mode, the fused call and the windowed step."""
    from paper_2507_20030_b200 import synth
    H, B, M, T = 3, 2, 37, P - 9
    HQ = H * GQ
    mask = _random_mask(P, M, 5 * P + GQ)
    mask[0] = 1
    bins = oracle.plan(P, mask)
    K, V = _make(400 + GQ, B, H, T, dtype)
    V = (V * (0.125 if dtype == torch.bfloat16 else 1.0)).to(dtype)   # bf16 only: output grid finer than the bar
    q = synth.make_q(6, GQ, B, HQ, 128, dtype=dtype)
    for mode in _decode_modes(fk, dtype, P):
        ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=_kvd(fk, dtype),
                         prefill_mode=fk.PREFILL_SIMT, decode_mode=mode)
        ctx.plan(0, mask)
        cK, cV = ctx.alloc_coef(0, B), ctx.alloc_coef(0, B)
        t_len = torch.zeros(B, dtype=torch.int32, device="cuda")
        ctx.compress_prefill(0, K.cuda(), V.cuda(), cK, cV, t_len)
        out = torch.full((B, HQ, 128), float("nan"), dtype=dtype, device="cuda")
        ctx.decode_attn(0, q.cuda(), cK, cV, t_len, out)
        torch.cuda.synchronize()
        want = oracle_decode_attn(oracle, q, to_np64(cK), to_np64(cV), P, bins, t_len.cpu().numpy())
        err = np.abs(to_np64(out) - want).max()
        assert err <= ATTN_MAX_ABS, (mode, err)
        # fused step on the same state
        k1, v1 = synth.make_token(400 + GQ, 0, B, H, 128, pos=T, dtype=dtype)
        v1 = (v1 * (0.125 if dtype == torch.bfloat16 else 1.0)).to(dtype)
        sK, sV, st = cK.clone(), cV.clone(), t_len.clone()
        ctx.append_decode_attn(0, k1.cuda(), v1.cuda(), q.cuda(), cK, cV, t_len, out)
        ctx.append(0, k1.cuda(), v1.cuda(), sK, sV, st)
        torch.cuda.synchronize()
        assert torch.equal(cK, sK) and torch.equal(cV, sV) and torch.equal(t_len, st)
        want = oracle_decode_attn(oracle, q, to_np64(cK), to_np64(cV), P, bins, t_len.cpu().numpy())
        err = np.abs(to_np64(out) - want).max()
        assert err <= ATTN_MAX_ABS, ("fused", mode, err)
        assert ctx.device_status() == 0
        ctx.close()


def test_windowed_step_any_group_size(fk, oracle):
    """The paper's window (S = 10, R = 50) with 7 query heads per kv head."""
    from paper_2507_20030_b200 import synth
    P, T, M, B, H, GQ, S, R = 256, 180, 33, 2, 2, 7, 10, 50
    HQ, dtype = H * GQ, torch.float32
    ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=fk.F32,
                     prefill_mode=fk.PREFILL_SIMT, n_sink=S, n_recent=R)
    mask = _random_mask(P, M, 19)
    mask[0] = 1
    ctx.plan(0, mask)
    bins = oracle.plan(P, mask)
    K, V = _make(77, B, H, T, dtype)
    units = {(b, h): oracle.WindowedUnit(P, bins, S, R) for b in range(B) for h in range(H)}
    for (b, h), u in units.items():
        u.prefill(to_np64(K[b, h]), to_np64(V[b, h]))
    cK, cV = ctx.alloc_coef(0, B), ctx.alloc_coef(0, B)
    wK, wV = ctx.alloc_window(B), ctx.alloc_window(B)
    t_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    ctx.prefill_windowed(0, K.cuda(), V.cuda(), cK, cV, wK, wV, t_len)
    out = torch.empty((B, HQ, 128), dtype=dtype, device="cuda")
    for s in range(4):
        k, v = synth.make_token(78, s, B, H, 128, pos=T + s, dtype=dtype)
        q = synth.make_q(78, s, B, HQ, 128, dtype=dtype)
        ctx.step_windowed(0, k.cuda(), v.cuda(), q.cuda(), cK, cV, wK, wV, t_len, out)
        torch.cuda.synchronize()
        got = to_np64(out)
        for (b, h), u in units.items():
            u.step(to_np64(k[b, h]), to_np64(v[b, h]))
            want = u.attention(to_np64(q[b, h * GQ:(h + 1) * GQ]))
            assert np.abs(got[b, h * GQ:(h + 1) * GQ] - want).max() <= ATTN_MAX_ABS, (s, b, h)
    assert ctx.device_status() == 0
    ctx.close()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("P", [100, 256, 32768])
def test_decode_attn_of_an_empty_sequence_is_zero(fk, oracle, dtype, P):
    """t_len = 0: Eq. 3 sums over no token; the rows of such a sequence are written as zeros (the oracle's
    reading), in every mode, and the other sequences of the batch are not disturbed."""
    from paper_2507_20030_b200 import synth
    M, B, H, HQ = 16, 3, 2, 4
    mask = fk.mask_lowpass(P, M)
    bins = oracle.plan(P, mask)
    rng = np.random.default_rng(P)
    cK = torch.from_numpy(rng.standard_normal((B, H, 2, M, 128)).astype(np.float32)).cuda()
    cV = torch.from_numpy(rng.standard_normal((B, H, 2, M, 128)).astype(np.float32)).cuda()
    tl = np.array([0, 9, 0], dtype=np.int32)
    t_len = torch.from_numpy(tl).cuda()
    q = synth.make_q(8, 0, B, HQ, 128, dtype=dtype)
    want = oracle_decode_attn(oracle, q, to_np64(cK), to_np64(cV), P, bins, tl)
    assert not want[0].any() and not want[2].any() and want[1].any()
    for mode in _decode_modes(fk, dtype, P):
        ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=_kvd(fk, dtype), decode_mode=mode)
        ctx.plan(0, mask)
        out = torch.full((B, HQ, 128), float("nan"), dtype=dtype, device="cuda")
        ctx.decode_attn(0, q.cuda(), cK, cV, t_len, out)
        torch.cuda.synchronize()
        got = to_np64(out)
        assert not got[0].any() and not got[2].any(), mode
        assert np.abs(got - want).max() <= ATTN_MAX_ABS, mode
        ctx.close()


def test_windowed_segment_on_the_next_power_of_two_grid(fk, oracle):
    """Eq. 10 transforms N - S - R tokens, which is rarely a power of two; the windowed calls want one.  The
    supported way is a grid of the next power of two: a 1024-token prompt with S = 10, R = 50 leaves a
    964-token segment on P = 1024.  Prefill, steps and the materialised cache against the oracle; the
    positions the segment has not reached are masked, so the longer grid changes nothing."""
    from paper_2507_20030_b200 import synth
    T, S, R, B, H, HQ, M = 1024, 10, 50, 1, 2, 8, 64
    seg = T - S - R
    P = 1 << (seg - 1).bit_length()
    assert P == 1024 and seg == 964
    dtype = torch.float32
    ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=fk.F32, n_sink=S, n_recent=R)
    mask = fk.mask_mixed(P, M, 0, 3)
    ctx.plan(0, mask)
    bins = oracle.plan(P, mask)
    K, V = _make(5, B, H, T, dtype)
    units = {(0, h): oracle.WindowedUnit(P, bins, S, R) for h in range(H)}
    for (b, h), u in units.items():
        u.prefill(to_np64(K[b, h]), to_np64(V[b, h]))
    cK, cV = ctx.alloc_coef(0, B), ctx.alloc_coef(0, B)
    wK, wV = ctx.alloc_window(B), ctx.alloc_window(B)
    t_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    ctx.prefill_windowed(0, K.cuda(), V.cuda(), cK, cV, wK, wV, t_len)
    out = torch.empty((B, HQ, 128), dtype=dtype, device="cuda")
    GQ = HQ // H
    for s in range(3):
        k, v = synth.make_token(6, s, B, H, 128, pos=T + s, dtype=dtype)
        q = synth.make_q(6, s, B, HQ, 128, dtype=dtype)
        ctx.step_windowed(0, k.cuda(), v.cuda(), q.cuda(), cK, cV, wK, wV, t_len, out)
        torch.cuda.synchronize()
        got = to_np64(out)
        for (b, h), u in units.items():
            u.step(to_np64(k[b, h]), to_np64(v[b, h]))
            want = u.attention(to_np64(q[b, h * GQ:(h + 1) * GQ]))
            assert np.abs(got[b, h * GQ:(h + 1) * GQ] - want).max() <= ATTN_MAX_ABS, (s, h)
    _check_materialised(fk, ctx, units, cK, cV, wK, wV, t_len, dtype)
    ctx.close()


# ----------------------------------------------------------------------------- config 0, end to end
def test_config0_end_to_end(fk, oracle):
    """1 layer, B=1, 8 kv heads, d=128, T=2048 float32, low-pass M=256; 64 appends (positions wrap onto
    slots 0..63); reconstruct L=2048; every tensor against the oracle."""
    from paper_2507_20030_b200 import synth
    P = T = 2048
    M, B, H, HQ, steps = 256, 1, 8, 32, 64
    seed = synth.config_seed(0, 0)
    ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=fk.F32)
    mask = fk.mask_lowpass(P, M)
    assert mask.tobytes() == oracle.mask_lowpass(P, M).tobytes()
    ctx.plan(0, mask)
    bins = oracle.plan(P, mask)
    assert ctx.get_bins(0).tobytes() == bins.tobytes()
    K, V = synth.make_kv(seed, B, H, T, 128, dtype=torch.float32)
    cK, cV = ctx.alloc_coef(0, B), ctx.alloc_coef(0, B)
    t_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    ctx.compress_prefill(0, K.cuda(), V.cuda(), cK, cV, t_len)
    torch.cuda.synchronize()
    refK, refV = oracle_compress(oracle, K, P, bins), oracle_compress(oracle, V, P, bins)
    assert rel_l2(to_np64(cK), refK) <= REL_L2_F32
    assert rel_l2(to_np64(cV), refV) <= REL_L2_F32
    _rows_close(to_np64(cK), refK, ROW_F32, "prefill, bin rows of K")
    _rows_close(to_np64(cV), refV, ROW_F32, "prefill, bin rows of V")
    for s in range(steps):
        k, v = synth.make_token(seed, s, B, H, 128, pos=T + s, dtype=torch.float32)
        ctx.append(0, k.cuda(), v.cuda(), cK, cV, t_len)
        oracle_append(oracle, refK, P, bins, np.array([T + s]), k)
        oracle_append(oracle, refV, P, bins, np.array([T + s]), v)
    torch.cuda.synchronize()
    assert t_len.tolist() == [T + steps]
    assert rel_l2(to_np64(cK), refK) <= REL_L2_F32
    assert rel_l2(to_np64(cV), refV) <= REL_L2_F32
    _rows_close(to_np64(cK), refK, ROW_F32, "after the appends, bin rows of K")
    _rows_close(to_np64(cV), refV, ROW_F32, "after the appends, bin rows of V")
    Ko = torch.empty((B, H, P, 128), device="cuda")
    Vo = torch.empty((B, H, P, 128), device="cuda")
    ctx.reconstruct(0, cK, cV, t_len, P, Ko, Vo)
    torch.cuda.synchronize()
    t_np = np.array([T + steps])
    for Xo, ref in ((Ko, refK), (Vo, refV)):
        want = oracle_reconstruct(oracle, ref, P, bins, t_np, P)
        assert rel_l2(to_np64(Xo), want) <= REL_L2_F32
        _rows_close(to_np64(Xo), want, ROW_F32, "token rows")
    q = synth.make_q(seed, 0, B, HQ, 128, dtype=torch.float32)
    out = torch.empty((B, HQ, 128), device="cuda")
    ctx.decode_attn(0, q.cuda(), cK, cV, t_len, out)
    torch.cuda.synchronize()
    want = oracle_decode_attn(oracle, q, refK, refV, P, bins, t_np)
    assert np.abs(to_np64(out) - want).max() <= ATTN_MAX_ABS
    ctx.close()


# ----------------------------------------------------------------------------- tensor-core prefill
@pytest.mark.parametrize("terms,tol", [(1, REL_L2_BF16), (2, REL_L2_F32)])
@pytest.mark.parametrize("P,T,M,B,H", [
    (512, 512, 128, 1, 1),      # one bin tile, 8 pipeline steps
    (512, 512, 200, 1, 2),      # two bin tiles, ragged second tile
    (1000, 700, 77, 2, 3),      # P not a power of two, T < P, ragged last token stage (700 = 10*64 + 60)
    (256, 1000, 129, 1, 2),     # T > P: positions wrap
    (2048, 2048, 256, 1, 8),    # config-0 shape in bf16
    (64, 1, 3, 1, 1),           # a single token
    (512, 300, 200, 10, 8),     # 160 tiles: more than one per SM -- a wave of whole tiles, then a wave cut along the tokens
])
def test_prefill_umma_matches_oracle(fk, oracle, terms, tol, P, T, M, B, H):
    ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=H, n_dft=P, max_batch=B, kv_dtype=fk.BF16,
                     prefill_mode=fk.PREFILL_UMMA, twiddle_terms=terms)
    mask = _random_mask(P, M, 7 * P + T)
    ctx.plan(0, mask)
    bins = oracle.plan(P, mask)
    K, V = _make(31 + P + T, B, H, T, torch.bfloat16)
    cK, cV = ctx.alloc_coef(0, B), ctx.alloc_coef(0, B)
    cK.fill_(float("nan")); cV.fill_(float("nan"))
    t_len = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    ctx.compress_prefill(0, K.cuda(), V.cuda(), cK, cV, t_len)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    assert t_len.tolist() == [T] * B
    wantK, wantV = oracle_compress(oracle, K, P, bins), oracle_compress(oracle, V, P, bins)
    errK = rel_l2(to_np64(cK), wantK)
    errV = rel_l2(to_np64(cV), wantV)
    assert errK <= tol and errV <= tol, (errK, errV)
    _rows_close(to_np64(cK), wantK, 4 * tol, "bin rows of K")
    _rows_close(to_np64(cV), wantV, 4 * tol, "bin rows of V")
    ctx.close()


def test_bounded_wait_gives_up_and_the_context_recovers(fk, oracle):
    """The give-up path of the tensor-core prefill, run for real: with the wait limit at 1 ms and one producer's
    'tile full' signal withheld at step 3, every wait of every CTA runs out; the kernel must end by itself (no
    wait is unbounded), leave a code in the status word, and the next call on the same context, hooks off,
    must be correct."""
    import time
    P = T = 1024
    M, B, H = 200, 1, 3
    ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=H, n_dft=P, max_batch=B, kv_dtype=fk.BF16,
                     prefill_mode=fk.PREFILL_UMMA)
    mask = _random_mask(P, M, 77)
    ctx.plan(0, mask)
    bins = oracle.plan(P, mask)
    K, V = _make(12, B, H, T, torch.bfloat16)
    cK, cV = ctx.alloc_coef(0, B), ctx.alloc_coef(0, B)
    t_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    ctx.compress_prefill(0, K.cuda(), V.cuda(), cK, cV, t_len)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    ctx.test_hooks(wait_limit_ns=1_000_000, withhold_step=3)
    t0 = time.perf_counter()
    ctx.compress_prefill(0, K.cuda(), V.cuda(), cK, cV, t_len)
    torch.cuda.synchronize()
    elapsed = time.perf_counter() - t0
    assert elapsed < 1.0, elapsed                     # a handful of 1 ms waits, not the default second (nor forever)
    code = ctx.device_status()
    assert code in (0x11, 0x12, 0x13, 0x14), hex(code)   # one of the kernel's time-out codes
    assert "bounded wait" in ctx._lib.faedkv_last_error(ctx._h).decode()
    # hooks off, status cleared: the context works again
    ctx.test_hooks(0, 0)
    ctx.reset_device_status()
    cK.fill_(float("nan")); cV.fill_(float("nan"))
    ctx.compress_prefill(0, K.cuda(), V.cuda(), cK, cV, t_len)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    assert rel_l2(to_np64(cK), oracle_compress(oracle, K, P, bins)) <= REL_L2_BF16
    assert rel_l2(to_np64(cV), oracle_compress(oracle, V, P, bins)) <= REL_L2_BF16
    ctx.close()


# ----------------------------------------------------------------------------- FFT-shaped prefill
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("P,T,M,B,H", [
    (512, 512, 128, 1, 1),
    (512, 300, 200, 1, 2),      # T < P: zero padding; odd split of the bins
    (256, 1000, 129, 1, 2),     # T > P: positions wrap and add; every bin retained
    (2048, 2048, 256, 1, 8),    # config-0 shape
    (64, 1, 3, 1, 1),           # a single token on the smallest grid
    (4096, 3001, 257, 2, 3),    # odd T (the last packed sample has no odd partner), several units per launch
    (8192, 8192, 96, 1, 5),     # two-pass split 64 x 64
])
def test_prefill_fft_matches_oracle(fk, oracle, dtype, P, T, M, B, H):
    """Float32-exact whatever the storage type: the FFT-shaped prefill meets the float32 bar on bf16 K/V too."""
    ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=H, n_dft=P, max_batch=B, kv_dtype=_kvd(fk, dtype),
                     prefill_mode=fk.PREFILL_FFT)
    mask = _random_mask(P, M, 11 * P + T)
    mask[0] = 1
    mask[P // 2] = 1                          # both self-conjugate bins
    ctx.plan(0, mask)
    bins = oracle.plan(P, mask)
    K, V = _make(41 + P + T, B, H, T, dtype)
    cK, cV = ctx.alloc_coef(0, B), ctx.alloc_coef(0, B)
    cK.fill_(float("nan")); cV.fill_(float("nan"))
    t_len = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    ctx.compress_prefill(0, K.cuda(), V.cuda(), cK, cV, t_len)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0 and t_len.tolist() == [T] * B
    wantK, wantV = oracle_compress(oracle, K, P, bins), oracle_compress(oracle, V, P, bins)
    errK = rel_l2(to_np64(cK), wantK)
    errV = rel_l2(to_np64(cV), wantV)
    assert errK <= REL_L2_F32 and errV <= REL_L2_F32, (errK, errV)
    _rows_close(to_np64(cK), wantK, ROW_F32, "bin rows of K")
    _rows_close(to_np64(cV), wantV, ROW_F32, "bin rows of V")
    ctx.close()


# ----------------------------------------------------------------------------- sink + recent window
def _check_materialised(fk, ctx, units, cK, cV, wK, wV, t_len, dtype):
    """Eq. 13 written out by the library against the oracle: [sink | reconstruction | waiting tokens], zeros
    behind; once with room to spare and once cut short."""
    lens = {key: u.materialise()[0].shape[0] for key, u in units.items()}
    for L in (max(lens.values()) + 3, max(1, min(lens.values()) - 2)):
        Kh, Vh = ctx.reconstruct_windowed(0, cK, cV, wK, wV, t_len, L)
        torch.cuda.synchronize()
        gK, gV = to_np64(Kh), to_np64(Vh)
        for (b, h), u in units.items():
            for got, want in ((gK[b, h], u.materialise()[0]), (gV[b, h], u.materialise()[1])):
                n = min(L, want.shape[0])
                tol = 2e-4 * max(1.0, np.abs(want).max()) + (np.abs(want[:n]) * 2.0 ** -8 if dtype == torch.bfloat16 else 0.0)
                assert np.all(np.abs(got[:n] - want[:n]) <= tol), (L, b, h, np.abs(got[:n] - want[:n]).max())
                assert not got[n:].any()
    assert ctx.device_status() == 0


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("P,T,M,B,H,HQ,S,R,steps", [
    (256, 200, 40, 2, 2, 8, 10, 50, 12),      # the paper's S = 10, R = 50; GQA 4
    (128, 64, 65, 1, 3, 3, 4, 7, 20),         # every bin retained; MHA; the ring turns over more than twice
    (512, 520, 33, 2, 1, 2, 0, 16, 5),        # no sink; the transformed segment is longer than P (wraps)
    (64, 30, 9, 1, 2, 4, 6, 0, 6),            # no ring: the new token itself is folded
    (1024, 60, 24, 2, 2, 4, 10, 50, 4),       # T = S + R: the transformed segment starts empty
])
@pytest.mark.parametrize("two_pass", [False, True])
def test_windowed_step_matches_oracle(fk, oracle, dtype, P, T, M, B, H, HQ, S, R, steps, two_pass):
    """Prefill with sink + recent window, then decode steps: attention outputs, planes, window contents
    and counters against the oracle's WindowedUnit, unit by unit; through the one-kernel column transform
    and through the two-pass transform kernels."""
    from paper_2507_20030_b200 import synth
    GQ = HQ // H
    ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=_kvd(fk, dtype),
                     prefill_mode=fk.PREFILL_SIMT, n_sink=S, n_recent=R,
                     decode_mode=fk.DECODE_FFT_TWO_PASS if two_pass else fk.DECODE_AUTO)
    mask = _random_mask(P, M, 13 * P + T)
    mask[0] = 1
    M = int(mask.sum())
    ctx.plan(0, mask)
    bins = oracle.plan(P, mask)
    assert ctx._lib.faedkv_window_bytes(ctx._h, B) == B * H * (S + R) * 128 * (4 if dtype == torch.float32 else 2)
    K, V = _make(51 + P + T, B, H, T, dtype)
    vs = _bf16_vscale(dtype)
    V = (V * vs).to(dtype)
    units = {(b, h): oracle.WindowedUnit(P, bins, S, R) for b in range(B) for h in range(H)}
    for (b, h), u in units.items():
        u.prefill(to_np64(K[b, h]), to_np64(V[b, h]))
    cK, cV = ctx.alloc_coef(0, B), ctx.alloc_coef(0, B)
    cK.fill_(float("nan")); cV.fill_(float("nan"))
    wK, wV = ctx.alloc_window(B), ctx.alloc_window(B)
    t_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    ctx.prefill_windowed(0, K.cuda(), V.cuda(), cK, cV, wK, wV, t_len)
    out = torch.empty((B, HQ, 128), dtype=dtype, device="cuda")
    for s in range(steps):
        k, v = synth.make_token(77, s, B, H, 128, pos=T + s, dtype=dtype)
        v = (v * vs).to(dtype)
        q = synth.make_q(77, s, B, HQ, 128, dtype=dtype)
        ctx.step_windowed(0, k.cuda(), v.cuda(), q.cuda(), cK, cV, wK, wV, t_len, out)
        torch.cuda.synchronize()
        got = to_np64(out)
        for (b, h), u in units.items():
            u.step(to_np64(k[b, h]), to_np64(v[b, h]))
            want = u.attention(to_np64(q[b, h * GQ:(h + 1) * GQ]))
            err = np.abs(got[b, h * GQ:(h + 1) * GQ] - want).max()
            assert err <= ATTN_MAX_ABS, (s, b, h, err)
    assert t_len.tolist() == [T + steps] * B and ctx.device_status() == 0
    gK, gV, gwK = to_np64(cK), to_np64(cV), to_np64(wK)
    for (b, h), u in units.items():
        assert rel_l2(gK[b, h], np.stack(u.CK)) <= REL_L2_F32 and rel_l2(gV[b, h], np.stack(u.CV)) <= REL_L2_F32
        _rows_close(gK[b, h], np.stack(u.CK), ROW_F32, ("bin rows of K", b, h))
        _rows_close(gV[b, h], np.stack(u.CV), ROW_F32, ("bin rows of V", b, h))
        assert np.array_equal(gwK[b, h, :S], u.sinkK)
        if R > 0:                             # ring slot of token n is (n - S) mod R
            t = T + steps
            for j, n in enumerate(range(t - R, t)):
                assert np.array_equal(gwK[b, h, S + (n - S) % R], u.recentK[j]), (b, h, n)
    _check_materialised(fk, ctx, units, cK, cV, wK, wV, t_len, dtype)
    ctx.close()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("P,Ts,M,H,HQ,S,R,D,steps", [
    (256, (200, 187), 40, 2, 8, 10, 50, 16, 40),   # the paper's window; a ragged batch folds at different steps
    (128, (64,), 65, 3, 3, 4, 7, 5, 23),           # every bin retained; MHA; several block folds
    (512, (530, 529), 33, 1, 2, 0, 16, 8, 20),     # no sink; the transformed segment is longer than P (wraps)
    (64, (31,), 9, 2, 4, 6, 0, 4, 10),             # no recent window: a block can end with the step's own token
    (64, (20, 21), 9, 1, 1, 0, 0, 2, 7),           # no window at all: nothing waits at a block boundary
    (1024, (60,), 24, 2, 4, 10, 50, 128, 140),     # T = S + R: the planes start empty; the largest block
])
@pytest.mark.parametrize("two_pass", [False, True])
def test_deferred_step_matches_oracle(fk, oracle, dtype, P, Ts, M, H, HQ, S, R, D, steps, two_pass):
    """Block-deferred fold: prefill (one call per sequence, so that the batch is ragged), then decode steps
    over the whole batch: attention outputs at every step, final planes, ring contents and counters against
    the oracle's WindowedUnit(defer=D), unit by unit."""
    from paper_2507_20030_b200 import synth
    B, GQ = len(Ts), HQ // H
    ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=_kvd(fk, dtype),
                     prefill_mode=fk.PREFILL_SIMT, n_sink=S, n_recent=R, n_defer=D,
                     decode_mode=fk.DECODE_FFT_TWO_PASS if two_pass else fk.DECODE_AUTO)
    mask = _random_mask(P, M, 17 * P + Ts[0])
    mask[0] = 1
    ctx.plan(0, mask)
    bins = oracle.plan(P, mask)
    Rc = R + D
    assert ctx._lib.faedkv_window_bytes(ctx._h, B) == B * H * (S + Rc) * 128 * (4 if dtype == torch.float32 else 2)
    cK, cV = ctx.alloc_coef(0, B), ctx.alloc_coef(0, B)
    cK.fill_(float("nan")); cV.fill_(float("nan"))
    wK, wV = ctx.alloc_window(B), ctx.alloc_window(B)
    assert wK.shape == (B, H, S + Rc, 128)
    t_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    units = {}
    for b, T in enumerate(Ts):
        K, V = _make(61 + P + T + b, 1, H, T, dtype)
        V = (V * _bf16_vscale(dtype)).to(dtype)
        for h in range(H):
            u = units[(b, h)] = oracle.WindowedUnit(P, bins, S, R, defer=D)
            u.prefill(to_np64(K[0, h]), to_np64(V[0, h]))
        ctx.prefill_windowed(0, K.cuda(), V.cuda(), cK[b:b + 1], cV[b:b + 1], wK[b:b + 1], wV[b:b + 1], t_len[b:b + 1])
    assert t_len.tolist() == list(Ts)
    out = torch.empty((B, HQ, 128), dtype=dtype, device="cuda")
    folds = 0
    for s in range(steps):
        k, v = synth.make_token(79, s, B, H, 128, pos=Ts[0] + s, dtype=dtype)
        v = (v * _bf16_vscale(dtype)).to(dtype)
        q = synth.make_q(79, s, B, HQ, 128, dtype=dtype)
        ctx.step_windowed(0, k.cuda(), v.cuda(), q.cuda(), cK, cV, wK, wV, t_len, out)
        torch.cuda.synchronize()
        got = to_np64(out)
        for (b, h), u in units.items():
            before = u.folded
            u.step(to_np64(k[b, h]), to_np64(v[b, h]))
            folds += u.folded != before
            want = u.attention(to_np64(q[b, h * GQ:(h + 1) * GQ]))
            err = np.abs(got[b, h * GQ:(h + 1) * GQ] - want).max()
            assert err <= ATTN_MAX_ABS, (s, b, h, err)
    assert folds >= B * H                      # every unit went through at least one block fold
    assert t_len.tolist() == [T + steps for T in Ts] and ctx.device_status() == 0
    gK, gV, gwK, gwV = to_np64(cK), to_np64(cV), to_np64(wK), to_np64(wV)
    for (b, h), u in units.items():
        assert rel_l2(gK[b, h], np.stack(u.CK)) <= REL_L2_F32 and rel_l2(gV[b, h], np.stack(u.CV)) <= REL_L2_F32
        _rows_close(gK[b, h], np.stack(u.CK), ROW_F32, ("bin rows of K", b, h))
        _rows_close(gV[b, h], np.stack(u.CV), ROW_F32, ("bin rows of V", b, h))
        assert np.array_equal(gwK[b, h, :S], u.sinkK)
        t = Ts[b] + steps
        first = S + u.folded
        assert u.folded == max(0, (t - S - R) // D * D) and len(u.recentK) == t - first
        for j, n in enumerate(range(first, t)):   # ring slot of token n is (n - S) mod (R + D)
            assert np.array_equal(gwK[b, h, S + (n - S) % Rc], u.recentK[j]), (b, h, n)
            assert np.array_equal(gwV[b, h, S + (n - S) % Rc], u.recentV[j]), (b, h, n)
    _check_materialised(fk, ctx, units, cK, cV, wK, wV, t_len, dtype)
    ctx.close()


@pytest.mark.parametrize("seed", range(10))
def test_windowed_random_configurations(fk, oracle, seed):
    """Seeded random window sizes, defer blocks, grids, retained sets, GQA factors and ragged batches: every
    step's attention output, the final planes and the counters against the oracle's WindowedUnit."""
    from paper_2507_20030_b200 import synth
    rng = np.random.default_rng(5000 + seed)
    P = 1 << int(rng.integers(6, 12))
    S, R = int(rng.integers(0, 9)), int(rng.integers(0, 13))
    D = int(rng.choice([1, 1, 2, 3, 7, 16]))
    GQ = int(rng.choice([1, 2, 4]))
    H = int(rng.integers(1, 4))
    HQ = H * GQ
    B = int(rng.integers(1, 4))
    M = int(rng.integers(1, min(P // 2 + 1, 40) + 1))
    steps = int(rng.integers(3, 3 * max(D, 2) + 4))
    Ts = [int(rng.integers(S + R + (1 if S + R == 0 else 0), S + R + P // 2 + 2)) for _ in range(B)]
    dtype = torch.float32 if seed % 2 == 0 else torch.bfloat16
    ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=_kvd(fk, dtype),
                     prefill_mode=fk.PREFILL_SIMT, n_sink=S, n_recent=R, n_defer=D)
    mask = _random_mask(P, M, 31 * seed + 1)
    mask[0] = 1
    ctx.plan(0, mask)
    bins = oracle.plan(P, mask)
    cK, cV = ctx.alloc_coef(0, B), ctx.alloc_coef(0, B)
    if S + R + (D if D > 1 else 0) == 0:
        ctx.close()
        pytest.skip("no window tensor in this draw")
    wK, wV = ctx.alloc_window(B), ctx.alloc_window(B)
    t_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    units = {}
    for b, T in enumerate(Ts):
        K, V = _make(900 + seed * 7 + b, 1, H, T, dtype)
        V = (V * _bf16_vscale(dtype)).to(dtype)
        for h in range(H):
            u = units[(b, h)] = oracle.WindowedUnit(P, bins, S, R, defer=D)
            u.prefill(to_np64(K[0, h]), to_np64(V[0, h]))
        ctx.prefill_windowed(0, K.cuda(), V.cuda(), cK[b:b + 1], cV[b:b + 1], wK[b:b + 1], wV[b:b + 1], t_len[b:b + 1])
    out = torch.empty((B, HQ, 128), dtype=dtype, device="cuda")
    for s_ in range(steps):
        k, v = synth.make_token(91 + seed, s_, B, H, 128, pos=Ts[0] + s_, dtype=dtype)
        v = (v * _bf16_vscale(dtype)).to(dtype)
        q = synth.make_q(91 + seed, s_, B, HQ, 128, dtype=dtype)
        ctx.step_windowed(0, k.cuda(), v.cuda(), q.cuda(), cK, cV, wK, wV, t_len, out)
        torch.cuda.synchronize()
        got = to_np64(out)
        for (b, h), u in units.items():
            u.step(to_np64(k[b, h]), to_np64(v[b, h]))
            want = u.attention(to_np64(q[b, h * GQ:(h + 1) * GQ]))
            err = np.abs(got[b, h * GQ:(h + 1) * GQ] - want).max()
            assert err <= ATTN_MAX_ABS, (seed, s_, b, h, err, (P, S, R, D, GQ, H, B, M, Ts))
    assert t_len.tolist() == [T + steps for T in Ts] and ctx.device_status() == 0
    gK, gV = to_np64(cK), to_np64(cV)
    for (b, h), u in units.items():
        assert np.abs(gK[b, h] - np.stack(u.CK)).max() <= 1e-4 * max(1.0, np.abs(np.stack(u.CK)).max())
        assert np.abs(gV[b, h] - np.stack(u.CV)).max() <= 1e-4 * max(1.0, np.abs(np.stack(u.CV)).max())
    ctx.close()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("S,R,D", [(0, 0, 4), (3, 6, 5), (10, 50, 32)])
def test_block_fold_is_bit_identical_to_single_token_updates(fk, dtype, S, R, D):
    """At every block boundary the planes of the block-deferred form equal, bit for bit, those of the
    per-step form fed the same tokens (the block fold performs the same FMAs in the same order); with no
    window at all the per-step form is faedkv_append."""
    from paper_2507_20030_b200 import synth
    P, M, B, H, HQ = 256, 48, 2, 2, 4
    T = S + R + 3 * D                              # prefill ends on a block boundary
    mask = _random_mask(P, M, 5)
    ctxs = [fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=_kvd(fk, dtype),
                       prefill_mode=fk.PREFILL_SIMT, n_sink=S, n_recent=R, n_defer=d) for d in (1, D)]
    K, V = _make(3, B, H, T, dtype)
    st = []
    for ctx in ctxs:
        ctx.plan(0, mask)
        cK, cV = ctx.alloc_coef(0, B), ctx.alloc_coef(0, B)
        wK, wV = ctx.alloc_window(B), ctx.alloc_window(B)
        t_len = torch.zeros(B, dtype=torch.int32, device="cuda")
        ctx.prefill_windowed(0, K.cuda(), V.cuda(), cK, cV, wK, wV, t_len)
        st.append((cK, cV, wK, wV, t_len))
    assert torch.equal(st[0][0], st[1][0]) and torch.equal(st[0][1], st[1][1])
    plain = None
    if S + R == 0:                                 # third arm: the plain append call
        pc = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=_kvd(fk, dtype),
                        prefill_mode=fk.PREFILL_SIMT)
        pc.plan(0, mask)
        plain = (pc, st[0][0].clone(), st[0][1].clone(), st[0][4].clone())
    out = torch.empty((B, HQ, 128), dtype=dtype, device="cuda")
    checked = 0
    for s in range(2 * D + 1):
        k, v = synth.make_token(83, s, B, H, 128, pos=T + s, dtype=dtype)
        q = synth.make_q(83, s, B, HQ, 128, dtype=dtype)
        for ctx, (cK, cV, wK, wV, t_len) in zip(ctxs, st):
            if S + R == 0 and ctx.n_defer <= 1:    # no window tensor at all: the per-step form is the fused call
                ctx.append_decode_attn(0, k.cuda(), v.cuda(), q.cuda(), cK, cV, t_len, out)
            else:
                ctx.step_windowed(0, k.cuda(), v.cuda(), q.cuda(), cK, cV, wK, wV, t_len, out)
        if plain is not None:
            plain[0].append(0, k.cuda(), v.cuda(), plain[1], plain[2], plain[3])
        torch.cuda.synchronize()
        same = torch.equal(st[0][0], st[1][0]) and torch.equal(st[0][1], st[1][1])
        if (T + s + 1 - S - R) % D == 0:
            assert same, s
            if plain is not None:
                assert torch.equal(plain[1], st[1][0]) and torch.equal(plain[2], st[1][1]), s
            checked += 1
        else:
            assert not same, s                     # between boundaries the deferred planes lag behind
    assert checked == 2
    for ctx in ctxs:
        assert ctx.device_status() == 0
        ctx.close()


@pytest.mark.parametrize("defer", [1, 4])
def test_windowed_step_replayed_as_a_cuda_graph(fk, defer):
    """The windowed step uses up to three streams of the context (window attention beside the pass over C_K,
    the second run of sequences of a call cut in two).  Captured into a CUDA graph and replayed, it must
    give bit for bit what the same steps give when launched eagerly on a copy of the state."""
    from paper_2507_20030_b200 import synth
    # 2048 points per column: 7 column CTAs fit an SM, so 5 * 256 = 1280 columns are more than the GPU holds at
    # once and the call is cut into runs of 2 + 3 sequences on two streams (checked through the launch count)
    P, M, B, H, HQ, S, R, T = 4096, 24, 5, 32, 256, 3, 6, 40
    dtype = torch.bfloat16
    ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=fk.BF16,
                     prefill_mode=fk.PREFILL_SIMT, n_sink=S, n_recent=R, n_defer=defer)
    ctx.plan(0, _random_mask(P, M, 9))
    K, V = _make(321, B, H, T, dtype)
    state = []
    for _ in range(2):
        cK, cV = ctx.alloc_coef(0, B), ctx.alloc_coef(0, B)
        wK, wV = ctx.alloc_window(B), ctx.alloc_window(B)
        t_len = torch.zeros(B, dtype=torch.int32, device="cuda")
        ctx.prefill_windowed(0, K.cuda(), V.cuda(), cK, cV, wK, wV, t_len)
        state.append((cK, cV, wK, wV, t_len, torch.empty((B, HQ, 128), dtype=dtype, device="cuda")))
    k, v = synth.make_token(7, 0, B, H, 128, pos=T, dtype=dtype)
    q = synth.make_q(7, 0, B, HQ, 128, dtype=dtype)
    k, v, q = k.cuda(), v.cuda(), q.cuda()
    steps = 2 * defer + 3
    cK, cV, wK, wV, t_len, out = state[0]
    n0 = ctx.launch_count()
    for _ in range(steps):                                        # eager
        ctx.step_windowed(0, k, v, q, cK, cV, wK, wV, t_len, out)
    torch.cuda.synchronize()
    # per step: window kernel, pass over C_K, two column kernels, two passes over C_V (+ the fold kernel when deferring)
    assert ctx.launch_count() - n0 == steps * (6 + (1 if defer > 1 else 0))
    cK, cV, wK, wV, t_len, out = state[1]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            ctx.step_windowed(0, k, v, q, cK, cV, wK, wV, t_len, out, stream=side.cuda_stream)
    torch.cuda.synchronize()
    for _ in range(steps):
        graph.replay()
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    for a, b in zip(state[0], state[1]):
        assert torch.equal(a, b)
    ctx.close()


def test_windowed_rejects_short_prefill_and_non_fft_grids(fk):
    ctx = fk.Context(n_layers=1, n_kv_heads=1, n_q_heads=1, n_dft=100, max_batch=1, kv_dtype=fk.F32, n_sink=4, n_recent=8)
    ctx.plan(0, _mask_from_bins(100, [0, 1, 2]))
    K = torch.zeros(1, 1, 11, 128, device="cuda")
    cK, w = ctx.alloc_coef(0, 1), ctx.alloc_window(1)
    t = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(fk.FaedkvError) as e:
        ctx.prefill_windowed(0, K, K, cK, cK, w, w, t)
    assert e.value.code == -3                                   # T < S + R
    K = torch.zeros(1, 1, 20, 128, device="cuda")
    ctx.prefill_windowed(0, K, K, cK, cK, w, w, t)
    x = torch.zeros(1, 1, 128, device="cuda")
    with pytest.raises(fk.FaedkvError) as e:
        ctx.step_windowed(0, x, x, x, cK, cK, w, w, t, x.clone())
    assert e.value.code == -4                                   # P = 100 has no FFT-shaped path
    ctx.close()


# ----------------------------------------------------------------------------- frequency ablation
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("P,T,C,chunks,B,H", [(1024, 1024, 22, (0, 3, 11, 21), 1, 2), (100, 100, 7, (0, 3, 6), 2, 1),
                                              (256, 200, 22, (5, 10), 1, 3)])
def test_ablate_matches_oracle(fk, oracle, dtype, P, T, C, chunks, B, H):
    """Zeroing one chunk of the two-sided spectrum of K and V (Eq. 6), inverse transform, real part:
    the removed component against the oracle's FFT definition."""
    ctx = fk.Context(n_layers=len(chunks), n_kv_heads=H, n_q_heads=H, n_dft=P, max_batch=B, kv_dtype=_kvd(fk, dtype))
    K, V = _make(61 + P, B, H, T, dtype)
    for layer, c in enumerate(chunks):
        lo, hi = fk.chunk_range(P, C, c)
        mask, gain = fk.ablation_bins(P, lo, hi)
        ctx.plan(layer, mask)
        g = torch.from_numpy(gain[ctx.get_bins(layer)]).cuda()
        wsK, wsV = ctx.alloc_coef(layer, B), ctx.alloc_coef(layer, B)
        ws_len = torch.zeros(B, dtype=torch.int32, device="cuda")
        Ko = torch.full((B, H, T, 128), float("nan"), dtype=dtype, device="cuda")
        Vo = torch.full_like(Ko, float("nan"))
        ctx.ablate(layer, K.cuda(), V.cuda(), g, wsK, wsV, ws_len, Ko, Vo)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        for X, Xo in ((K, Ko), (V, Vo)):
            x = to_np64(X)
            want = np.stack([[oracle.ablate(x[b, h], P, lo, hi) for h in range(H)] for b in range(B)])
            got = to_np64(Xo)
            if dtype == torch.float32:
                # compare what was removed: x' is close to x, so an error relative to x' would hide it
                assert rel_l2(x - got, x - want) <= REL_L2_F32, (c, rel_l2(x - got, x - want))
            else:
                assert rel_l2(got, want) <= REL_L2_BF16, (c, rel_l2(got, want))
    ctx.close()


# ----------------------------------------------------------------------------- paper-literal state forms
@pytest.mark.parametrize("P,T,M,B,H", [(64, 50, 9, 2, 2), (100, 230, 21, 1, 3)])
def test_state_forms_match_the_printed_recursions(fk, oracle, P, T, M, B, H):
    """The library's state converted to the rotating frame equals the oracle running the recursion
    R <- W_k (R + x) literally over the tokens; converted to the running mean it equals the oracle's
    exact-factor recursion; both conversions come back bit-close to the original."""
    ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=H, n_dft=P, max_batch=B, kv_dtype=fk.F32,
                     prefill_mode=fk.PREFILL_SIMT)
    mask = _random_mask(P, M, 17 * P + T)
    mask[0] = 1
    ctx.plan(0, mask)
    bins = oracle.plan(P, mask)
    M = len(bins)
    K, V = _make(71 + P, B, H, T, torch.float32)
    cK, cV = ctx.alloc_coef(0, B), ctx.alloc_coef(0, B)
    t_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    ctx.compress_prefill(0, K.cuda(), V.cuda(), cK, cV, t_len)
    rot = ctx.convert_state(0, cK, t_len, fk.STATE_SUM, fk.STATE_ROTATING, torch.empty_like(cK))
    mean = ctx.convert_state(0, cK, t_len, fk.STATE_SUM, fk.STATE_MEAN, torch.empty_like(cK))
    back1 = ctx.convert_state(0, rot.clone(), t_len, fk.STATE_ROTATING, fk.STATE_SUM)
    back2 = ctx.convert_state(0, mean.clone(), t_len, fk.STATE_MEAN, fk.STATE_SUM)
    cross = ctx.convert_state(0, rot.clone(), t_len, fk.STATE_ROTATING, fk.STATE_MEAN)
    torch.cuda.synchronize()
    x = to_np64(K)
    for b in range(B):
        for h in range(H):
            Rre, Rim = np.zeros((M, 128)), np.zeros((M, 128))
            Sre, Sim = np.zeros((M, 128)), np.zeros((M, 128))
            for n in range(T):
                oracle.rotating_frame_step(Rre, Rim, P, bins, x[b, h, n])
                oracle.running_mean_step(Sre, Sim, P, bins, n, x[b, h, n])
            assert rel_l2(to_np64(rot[b, h]), np.stack([Rre, Rim])) <= REL_L2_F32
            assert rel_l2(to_np64(mean[b, h]), np.stack([Sre, Sim])) <= REL_L2_F32
            assert rel_l2(to_np64(cross[b, h]), np.stack([Sre, Sim])) <= REL_L2_F32
    assert rel_l2(to_np64(back1), to_np64(cK)) <= 1e-6 and rel_l2(to_np64(back2), to_np64(cK)) <= 1e-6
    ctx.close()
