"""GPU parity at the full sizes of the five workload configurations, in the launch configuration the
benchmark times (default modes: tensor-core prefill with one bf16 twiddle term, FFT-shaped decode
attention).  The tensors are too large for the oracle to recompute whole, so every case runs the
complete operation on the GPU and compares SAMPLED outputs that the oracle computes one by one:
whole (sequence, kv head) units of the coefficient planes, and decode-attention outputs of single
kv heads at chosen steps.  Bin lists are compared bit for bit for every layer.

Inputs are drawn on the GPU from the seeded generators; the oracle is fed the stored values of the
sampled slices, copied back to the host.
"""
import numpy as np
import pytest
import torch

from helpers import ATTN_MAX_ABS, REL_L2_BF16, rel_l2, to_np64

pytestmark = pytest.mark.gpu

D = 128


@pytest.fixture(scope="module")
def fk():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2507_20030_b200 import binding, build
    build.build()
    binding.load()
    return binding


def _oracle_unit_state(oracle, x_prefill, P, bins, x_tokens, t0):
    """Planes of one unit: pruned DFT of x_prefill [T, d], then one append per row of x_tokens at
    positions t0, t0 + 1, ...  Returns float64 [2, M, d]."""
    re, im = oracle.compress(to_np64(x_prefill), P, bins)
    re, im = np.ascontiguousarray(re), np.ascontiguousarray(im)
    if x_tokens is not None:
        xt = to_np64(x_tokens)
        for s in range(xt.shape[0]):
            oracle.append(re, im, P, bins, t0 + s, xt[s])
    return np.stack([re, im])


def _oracle_attn_unit(oracle, q_unit, cK_unit, cV_unit, P, bins, t):
    """q_unit [GQ, d]; cK_unit, cV_unit [2, M, d] (stored float32 planes) -> [GQ, d]."""
    ck, cv = to_np64(cK_unit), to_np64(cV_unit)
    return oracle.decode_attn(to_np64(q_unit), ck[0], ck[1], cv[0], cv[1], P, bins, min(int(t), P))


def test_config1_full_prefill(fk, oracle):
    """configs[1]: 32 layers x 8 kv heads x 32768 bf16 tokens, mixed masks keeping 1/8 of the bins.
    Bins bit-exact for all 32 layers; three layers transformed at full size, two whole units of K and
    of V per layer against the oracle."""
    from paper_2507_20030_b200 import synth
    NL, H, HQ, T, M = 32, 8, 32, 32768, 4096
    P = T
    seed = synth.config_seed(1)
    ctx = fk.Context(n_layers=NL, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=1, kv_dtype=fk.BF16)
    all_bins = []
    for l in range(NL):
        mask = fk.mask_mixed(P, M, l, seed)
        assert mask.tobytes() == oracle.mask_mixed(P, M, l, seed).tobytes()
        assert ctx.plan(l, mask) == M
        bins = oracle.plan(P, mask)
        assert ctx.get_bins(l).tobytes() == bins.tobytes()
        all_bins.append(bins)
    assert len({b.tobytes() for b in all_bins}) == NL          # the masks differ per layer
    for l, heads in [(0, (0, 5)), (13, (2, 7)), (31, (3, 4))]:
        K, V = synth.make_kv(synth.config_seed(1, l), 1, H, T, D, dtype=torch.bfloat16, device="cuda")
        cK, cV = ctx.alloc_coef(l, 1), ctx.alloc_coef(l, 1)
        t_len = torch.zeros(1, dtype=torch.int32, device="cuda")
        ctx.compress_prefill(l, K, V, cK, cV, t_len)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0 and t_len.tolist() == [T]
        for h in heads:
            for x, c in ((K, cK), (V, cV)):
                want = _oracle_unit_state(oracle, x[0, h].cpu(), P, all_bins[l], None, 0)
                err = rel_l2(to_np64(c[0, h]), want)
                assert err <= REL_L2_BF16, (l, h, err)
        del K, V, cK, cV
    ctx.close()


def test_config1_fft_prefill_layer(fk, oracle):
    """configs[1], one layer through the FFT-shaped prefill: float32-exact coefficients from bf16 K/V."""
    from helpers import REL_L2_F32
    from paper_2507_20030_b200 import synth
    H, HQ, T, M, l = 8, 32, 32768, 4096, 21
    P = T
    ctx = fk.Context(n_layers=l + 1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=1, kv_dtype=fk.BF16,
                     prefill_mode=fk.PREFILL_FFT)
    mask = fk.mask_mixed(P, M, l, synth.config_seed(1))
    ctx.plan(l, mask)
    bins = oracle.plan(P, mask)
    K, V = synth.make_kv(synth.config_seed(1, l), 1, H, T, D, dtype=torch.bfloat16, device="cuda")
    cK, cV = ctx.alloc_coef(l, 1), ctx.alloc_coef(l, 1)
    t_len = torch.zeros(1, dtype=torch.int32, device="cuda")
    ctx.compress_prefill(l, K, V, cK, cV, t_len)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0 and t_len.tolist() == [T]
    for h in (1, 6):
        for x, c in ((K, cK), (V, cV)):
            want = _oracle_unit_state(oracle, x[0, h].cpu(), P, bins, None, 0)
            err = rel_l2(to_np64(c[0, h]), want)
            assert err <= REL_L2_F32, (h, err)
    ctx.close()


def _decode_case(fk, oracle, *, config, layer, B, H, HQ, T, M, mask_kind, steps, sample_units, sample_steps,
                 coef_channels=None, fused_every=2):
    """Prefill one layer at full size, run `steps` decode steps (append + attention; every
    `fused_every`-th step through the fused call, the others through the two calls), and check the
    sampled units' planes after the last step and the sampled attention outputs."""
    from paper_2507_20030_b200 import synth
    P = T
    GQ = HQ // H
    seed = synth.config_seed(config)
    ctx = fk.Context(n_layers=layer + 1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=fk.BF16)
    mask = fk.mask_lowpass(P, M) if mask_kind == "lowpass" else fk.mask_mixed(P, M, layer, seed)
    omask = oracle.mask_lowpass(P, M) if mask_kind == "lowpass" else oracle.mask_mixed(P, M, layer, seed)
    assert mask.tobytes() == omask.tobytes()
    ctx.plan(layer, mask)
    bins = oracle.plan(P, omask)
    assert ctx.get_bins(layer).tobytes() == bins.tobytes()
    lseed = synth.config_seed(config, layer)
    K, V = synth.make_kv(lseed, B, H, T, D, dtype=torch.bfloat16, device="cuda")
    # the decode tokens continue the same distributions at positions T, T+1, ...
    Kn, Vn = synth.make_kv(lseed, B, H, steps, D, pos0=T, dtype=torch.bfloat16, device="cuda", stream_tag=1)
    Q = torch.stack([synth.make_q(lseed, s, B, HQ, D, dtype=torch.bfloat16, device="cuda") for s in sample_steps])
    q_other = synth.make_q(lseed, 10 ** 6, B, HQ, D, dtype=torch.bfloat16, device="cuda")
    cK, cV = ctx.alloc_coef(layer, B), ctx.alloc_coef(layer, B)
    t_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    ctx.compress_prefill(layer, K, V, cK, cV, t_len)
    out = torch.empty((B, HQ, D), dtype=torch.bfloat16, device="cuda")
    saved = {}
    for s in range(steps):
        k_new, v_new = Kn[:, :, s].contiguous(), Vn[:, :, s].contiguous()
        q = Q[sample_steps.index(s)] if s in sample_steps else q_other
        if s % fused_every == 0:
            ctx.append_decode_attn(layer, k_new, v_new, q, cK, cV, t_len, out)
        else:
            ctx.append(layer, k_new, v_new, cK, cV, t_len)
            ctx.decode_attn(layer, q, cK, cV, t_len, out)
        if s in sample_steps:
            saved[s] = (out.clone(), {(b, h): (cK[b, h].clone(), cV[b, h].clone()) for b, h in sample_units})
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    assert t_len.tolist() == [T + steps] * B
    ch = slice(None) if coef_channels is None else coef_channels
    for b, h in sample_units:
        for x, xn, c in ((K, Kn, cK), (V, Vn, cV)):
            want = _oracle_unit_state(oracle, x[b, h][:, ch].cpu(), P, bins, xn[b, h][:, ch].cpu(), T)
            err = rel_l2(to_np64(c[b, h][:, :, ch]), want)
            assert err <= REL_L2_BF16, ("planes", b, h, err)
    for s in sample_steps:
        got, states = saved[s]
        q = Q[sample_steps.index(s)]
        for (b, h), (ck, cv) in states.items():
            want = _oracle_attn_unit(oracle, q[b, h * GQ:(h + 1) * GQ].cpu(), ck, cv, P, bins, T + s + 1)
            err = np.abs(to_np64(got[b, h * GQ:(h + 1) * GQ]) - want).max()
            assert err <= ATTN_MAX_ABS, ("attention", s, b, h, err)
    ctx.close()


def test_config2_streaming_decode(fk, oracle):
    """configs[2]: batch 16, prefill 16384 tokens at 1/8 retention, then 4096 decode steps with 32 query
    heads; one layer at full size, all steps."""
    _decode_case(fk, oracle, config=2, layer=5, B=16, H=8, HQ=32, T=16384, M=2048, mask_kind="mixed",
                 steps=4096, sample_units=[(0, 0), (11, 6)], sample_steps=[0, 2047, 4095])


def test_config3_long_context(fk, oracle):
    """configs[3]: batch 1, 131072 tokens at 1/16 retention, 256 decode steps with the fused call."""
    _decode_case(fk, oracle, config=3, layer=9, B=1, H=8, HQ=32, T=131072, M=8192, mask_kind="mixed",
                 steps=256, sample_units=[(0, 3)], sample_steps=[255], coef_channels=slice(40, 56), fused_every=1)


@pytest.mark.parametrize("T,B,r,mask_kind,layer", [
    (4096, 1, 16, "mixed", 30),
    (4096, 8, 4, "lowpass", 5),
    (4096, 8, 32, "mixed", 11),
    (4096, 32, 4, "lowpass", 0),
    (16384, 1, 8, "mixed", 3),
    (16384, 8, 32, "mixed", 7),
    (16384, 8, 16, "lowpass", 20),
    (16384, 32, 8, "lowpass", 2),
])
def test_config4_sweep_cells(fk, oracle, T, B, r, mask_kind, layer):
    """configs[4]: Llama-2-7B-shaped MHA cache (32 kv = 32 query heads); cells of the (T, batch, retention,
    mask) sweep -- every (T, batch) pair, every retention ratio and both mask kinds occur -- one layer each,
    prefill + 32 decode steps."""
    _decode_case(fk, oracle, config=4, layer=layer, B=B, H=32, HQ=32, T=T, M=T // r, mask_kind=mask_kind,
                 steps=32, sample_units=[(B - 1, 17)], sample_steps=[31])


@pytest.mark.parametrize("defer", [1, 50])
def test_config2_windowed_workflow(fk, oracle, defer):
    """configs[2] shape through the paper's own workflow (sink 10 + recent 50), per-step fold and
    block-deferred fold of 50 tokens: one layer at full size, 110 decode steps (the deferred form folds
    at steps 25 and 75), sampled units against the oracle's WindowedUnit at steps around the folds."""
    from paper_2507_20030_b200 import synth
    config, layer, B, H, HQ, T, M, S, R, steps = 2, 3, 16, 8, 32, 16384, 2048, 10, 50, 110
    sample_units, sample_steps = [(0, 1), (13, 6)], [25, 26, 109]
    P, GQ = T, HQ // H
    seed = synth.config_seed(config)
    ctx = fk.Context(n_layers=layer + 1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=fk.BF16,
                     n_sink=S, n_recent=R, n_defer=defer)
    mask = fk.mask_mixed(P, M, layer, seed)
    ctx.plan(layer, mask)
    bins = oracle.plan(P, oracle.mask_mixed(P, M, layer, seed))
    assert ctx.get_bins(layer).tobytes() == bins.tobytes()
    lseed = synth.config_seed(config, layer)
    K, V = synth.make_kv(lseed, B, H, T, D, dtype=torch.bfloat16, device="cuda")
    Kn, Vn = synth.make_kv(lseed, B, H, steps, D, pos0=T, dtype=torch.bfloat16, device="cuda", stream_tag=1)
    units = {}
    for b, h in sample_units:
        u = units[(b, h)] = oracle.WindowedUnit(P, bins, S, R, defer=defer)
        u.prefill(to_np64(K[b, h].cpu()), to_np64(V[b, h].cpu()))
    cK, cV = ctx.alloc_coef(layer, B), ctx.alloc_coef(layer, B)
    wK, wV = ctx.alloc_window(B), ctx.alloc_window(B)
    t_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    ctx.prefill_windowed(layer, K, V, cK, cV, wK, wV, t_len)
    out = torch.empty((B, HQ, D), dtype=torch.bfloat16, device="cuda")
    folds = 0
    for s in range(steps):
        k_new, v_new = Kn[:, :, s].contiguous(), Vn[:, :, s].contiguous()
        q = synth.make_q(lseed, s, B, HQ, D, dtype=torch.bfloat16, device="cuda")
        ctx.step_windowed(layer, k_new, v_new, q, cK, cV, wK, wV, t_len, out)
        for (b, h), u in units.items():
            before = u.folded
            u.step(to_np64(k_new[b, h].cpu()), to_np64(v_new[b, h].cpu()))
            folds += (u.folded - before) >= max(defer, 2)
        if s in sample_steps:
            got = to_np64(out)
            for (b, h), u in units.items():
                want = u.attention(to_np64(q[b, h * GQ:(h + 1) * GQ].cpu()))
                err = np.abs(got[b, h * GQ:(h + 1) * GQ] - want).max()
                assert err <= ATTN_MAX_ABS, ("attention", s, b, h, err)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0 and t_len.tolist() == [T + steps] * B
    assert folds == (2 * len(sample_units) if defer > 1 else 0)
    for (b, h), u in units.items():
        assert u.folded == (T + steps - S - R) // defer * defer
        for c, want in ((cK, u.CK), (cV, u.CV)):
            err = rel_l2(to_np64(c[b, h]), np.stack(want))
            assert err <= REL_L2_BF16, ("planes", b, h, err)
    ctx.close()


@pytest.mark.parametrize("config,B,H,T,M,tl_short", [
    (1, 1, 8, 32768, 4096, None),          # one persistent launch, 64 column blocks
    (2, 16, 8, 16384, 2048, 9000),         # 1024 column blocks: the ring between the passes is reused 50 times over
    (3, 1, 8, 131072, 8192, None),         # the two-kernel engine (256-point passes)
])
def test_reconstruct_full_sizes(fk, oracle, config, B, H, T, M, tl_short):
    """Reconstruction at the full sizes of configs[1], [2] and [3], in the launch configuration the benchmark
    times (bf16 rows, default engine): both tensors written whole, then single rows of sampled units compared
    with the oracle's row-wise inverse transform -- first and last rows, rows around tile and pass boundaries,
    rows around the live length of a shorter sequence, random rows."""
    from paper_2507_20030_b200 import synth
    P, layer = T, 5
    seed = synth.config_seed(config)
    ctx = fk.Context(n_layers=layer + 1, n_kv_heads=H, n_q_heads=H, n_dft=P, max_batch=B, kv_dtype=fk.BF16)
    mask = fk.mask_mixed(P, M, layer, seed)
    ctx.plan(layer, mask)
    bins = oracle.plan(P, oracle.mask_mixed(P, M, layer, seed))
    g = torch.Generator(device="cuda").manual_seed(seed + 17)
    # planes with the decaying spectrum of a real cache (large low bins), random phases
    amp = (float(np.sqrt(T)) / (1.0 + torch.arange(M, device="cuda", dtype=torch.float32) / 64.0))[None, None, None, :, None]
    cK = torch.randn((B, H, 2, M, D), generator=g, device="cuda") * amp
    cV = torch.randn((B, H, 2, M, D), generator=g, device="cuda") * amp
    tl = np.full(B, T + 3, dtype=np.int32)
    if tl_short is not None:
        tl[B // 2] = tl_short
    t_len = torch.from_numpy(tl).cuda()
    Ko = torch.full((B, H, P, D), 7.0, dtype=torch.bfloat16, device="cuda")
    Vo = torch.full_like(Ko, 7.0)
    ctx.reconstruct(layer, cK, cV, t_len, P, Ko, Vo)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    rng = np.random.default_rng(config)
    N1 = 1 << ((P // 2).bit_length() // 2)
    special = [0, 1, 2, 3, 2 * N1 - 2, 2 * N1 - 1, 2 * N1, 2 * N1 + 1, P // 2 - 1, P // 2, P // 2 + 1, P - 2, P - 1]
    units = sorted({(0, 0), (B - 1, H - 1), (B // 2, H // 2), (B // 2, 0)})
    for b, h in units:
        live = min(int(tl[b]), P)
        rows = sorted(set(special + list(rng.integers(0, P, size=40)) +
                          ([live - 2, live - 1, live, live + 1] if live < P else [])))
        rows = np.array([r for r in rows if 0 <= r < P], dtype=np.int32)
        for c, X in ((cK, Ko), (cV, Vo)):
            pl = to_np64(c[b, h])
            want = oracle.reconstruct_rows(pl[0], pl[1], P, bins, rows)
            want[rows >= live] = 0.0
            got = to_np64(X[b, h][torch.from_numpy(rows.astype(np.int64)).cuda()])
            assert not got[rows >= live].any(), (b, h)                       # rows past the live length are exactly zero
            scale = np.sqrt((want ** 2).sum(axis=1).mean())
            err = np.sqrt(((got - want) ** 2).sum(axis=1)).max() / scale     # worst row against the typical row norm
            assert err <= 4 * REL_L2_BF16, (config, b, h, err)
            assert rel_l2(got, want) <= REL_L2_BF16, (config, b, h, rel_l2(got, want))
    ctx.close()
