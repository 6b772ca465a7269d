"""Small cases of every call, run against the CHECKED build of the library (lib/libfaedkv_debug.so, selected
through FAEDKV_LIBRARY before this process starts), with canaries around every output tensor.

Not collected by pytest (tests/test_gpu_debug_build.py runs it in a process of its own, because a process
holds one build of the library).  After every call: the checked build's bounds-check word must be 0, the
canaries intact, and the result still matches the float64 oracle.
"""
import os
import sys

import numpy as np
import torch

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, HERE)
sys.path.insert(0, os.path.dirname(HERE))

import oracle                                                        # noqa: E402
from helpers import (ATTN_MAX_ABS, REL_L2_BF16, REL_L2_F32, Guarded, oracle_compress, oracle_decode_attn,   # noqa: E402
                     oracle_reconstruct, rel_l2, to_np64)
from paper_2507_20030_b200 import binding as fk, synth               # noqa: E402


def after(ctx, guards, what):
    torch.cuda.synchronize()
    w = ctx.debug_word()
    assert w == 0, f"{what}: bounds check failed, file tag {w >> 16} line {w & 0xffff}"
    assert ctx.device_status() == 0, what
    for g in guards:
        g.check(what)


def case(P, T, M, B, H, HQ, dtype, prefill_mode, decode_mode, recon_engine=0, S=0, R=0, D=0):
    kvd = fk.F32 if dtype == torch.float32 else fk.BF16
    tol = REL_L2_F32 if dtype == torch.float32 else REL_L2_BF16
    name = f"P={P} T={T} M={M} B={B} H={H} HQ={HQ} {dtype} prefill={prefill_mode} decode={decode_mode} recon={recon_engine} S={S} R={R} D={D}"
    ctx = fk.Context(n_layers=1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=kvd, prefill_mode=prefill_mode,
                     decode_mode=decode_mode, recon_engine=recon_engine, n_sink=S, n_recent=R, n_defer=D)
    rng = np.random.default_rng(P + M)
    mask = np.zeros(P // 2 + 1, dtype=np.uint8)
    mask[np.sort(rng.choice(P // 2 + 1, size=M, replace=False))] = 1
    mask[0] = 1
    ctx.plan(0, mask)
    bins = oracle.plan(P, mask)
    M = len(bins)
    K, V = synth.make_kv(7, B, H, T, 128, dtype=dtype)
    V = (V * (0.125 if dtype == torch.bfloat16 else 1.0)).to(dtype)
    gK, gV = Guarded((B, H, 2, M, 128), torch.float32, float("nan")), Guarded((B, H, 2, M, 128), torch.float32, float("nan"))
    gt = Guarded((B,), torch.int32, 0)
    cK, cV, t_len = gK.t, gV.t, gt.t
    windowed = S + R > 0 or D > 1
    if windowed:
        Rc = R + (D if D > 1 else 0)
        gwK, gwV = Guarded((B, H, S + Rc, 128), dtype, 0), Guarded((B, H, S + Rc, 128), dtype, 0)
        ctx.prefill_windowed(0, K.cuda(), V.cuda(), cK, cV, gwK.t, gwV.t, t_len)
        after(ctx, [gK, gV, gt, gwK, gwV], name + " prefill_windowed")
        units = {(b, h): oracle.WindowedUnit(P, bins, S, R, defer=max(D, 1)) if D > 1 else oracle.WindowedUnit(P, bins, S, R)
                 for b in range(B) for h in range(H)}
        for (b, h), u in units.items():
            u.prefill(to_np64(K[b, h]), to_np64(V[b, h]))
        go = Guarded((B, HQ, 128), dtype, float("nan"))
        GQ = HQ // H
        for s_ in range(max(3, D + 2)):
            k, v = synth.make_token(7, s_, B, H, 128, pos=T + s_, dtype=dtype)
            v = (v * (0.125 if dtype == torch.bfloat16 else 1.0)).to(dtype)
            q = synth.make_q(7, s_, B, HQ, 128, dtype=dtype)
            ctx.step_windowed(0, k.cuda(), v.cuda(), q.cuda(), cK, cV, gwK.t, gwV.t, t_len, go.t)
            after(ctx, [gK, gV, gt, gwK, gwV, go], name + " step_windowed")
            got = to_np64(go.t)
            for (b, h), u in units.items():
                u.step(to_np64(k[b, h]), to_np64(v[b, h]))
                want = u.attention(to_np64(q[b, h * GQ:(h + 1) * GQ]))
                assert np.abs(got[b, h * GQ:(h + 1) * GQ] - want).max() <= ATTN_MAX_ABS, name
        L = T + 8
        gKo, gVo = Guarded((B, H, L, 128), dtype, 7.0), Guarded((B, H, L, 128), dtype, 7.0)
        ctx._check(ctx._lib.faedkv_reconstruct_windowed(ctx._h, 0, cK.data_ptr(), cV.data_ptr(), gwK.t.data_ptr(), gwV.t.data_ptr(),
                                                        t_len.data_ptr(), B, L, gKo.t.data_ptr(), gVo.t.data_ptr(), None))
        after(ctx, [gKo, gVo, gK, gV], name + " reconstruct_windowed")
        ctx.close()
        return
    ctx.compress_prefill(0, K.cuda(), V.cuda(), cK, cV, t_len)
    after(ctx, [gK, gV, gt], name + " compress_prefill")
    tolp = REL_L2_BF16 if (dtype == torch.bfloat16 and prefill_mode in (fk.PREFILL_AUTO, fk.PREFILL_UMMA)) else REL_L2_F32
    assert rel_l2(to_np64(cK), oracle_compress(oracle, K, P, bins)) <= tolp, name
    assert rel_l2(to_np64(cV), oracle_compress(oracle, V, P, bins)) <= tolp, name
    k1, v1 = synth.make_token(7, 0, B, H, 128, pos=T, dtype=dtype)
    ctx.append(0, k1.cuda(), v1.cuda(), cK, cV, t_len)
    after(ctx, [gK, gV, gt], name + " append")
    assert t_len.tolist() == [T + 1] * B
    L = min(P, T + 1)
    gKo, gVo = Guarded((B, H, L, 128), dtype, 7.0), Guarded((B, H, L, 128), dtype, 7.0)
    ctx.reconstruct(0, cK, cV, t_len, L, gKo.t, gVo.t)
    after(ctx, [gKo, gVo, gK, gV], name + " reconstruct")
    t_np = t_len.cpu().numpy()
    assert rel_l2(to_np64(gKo.t), oracle_reconstruct(oracle, to_np64(cK), P, bins, t_np, L)) <= tol, name
    assert rel_l2(to_np64(gVo.t), oracle_reconstruct(oracle, to_np64(cV), P, bins, t_np, L)) <= tol, name
    q = synth.make_q(7, 0, B, HQ, 128, dtype=dtype)
    go = Guarded((B, HQ, 128), dtype, float("nan"))
    ctx.decode_attn(0, q.cuda(), cK, cV, t_len, go.t)
    after(ctx, [go, gK, gV, gt], name + " decode_attn")
    want = oracle_decode_attn(oracle, q, to_np64(cK), to_np64(cV), P, bins, t_np)
    assert np.abs(to_np64(go.t) - want).max() <= ATTN_MAX_ABS, name
    k2, v2 = synth.make_token(7, 1, B, H, 128, pos=T + 1, dtype=dtype)
    ctx.append_decode_attn(0, k2.cuda(), v2.cuda(), q.cuda(), cK, cV, t_len, go.t)
    after(ctx, [go, gK, gV, gt], name + " append_decode_attn")
    want = oracle_decode_attn(oracle, q, to_np64(cK), to_np64(cV), P, bins, t_len.cpu().numpy())
    assert np.abs(to_np64(go.t) - want).max() <= ATTN_MAX_ABS, name
    ctx.close()


def main():
    assert torch.cuda.is_available()
    lib = fk.load()
    assert lib.faedkv_debug_build() == 1, "this script must run against the checked build (FAEDKV_LIBRARY)"
    oracle.build()
    f32, bf16 = torch.float32, torch.bfloat16
    n = 0
    for dtype in (f32, bf16):
        # every evaluation of the transforms, ragged sizes
        case(100, 77, 21, 2, 3, 6, dtype, fk.PREFILL_SIMT, fk.DECODE_SIMT); n += 1
        case(256, 256, 40, 2, 2, 8, dtype, fk.PREFILL_AUTO, fk.DECODE_AUTO); n += 1
        case(256, 200, 40, 1, 2, 14, dtype, fk.PREFILL_FFT, fk.DECODE_FFT_TWO_PASS, recon_engine=1); n += 1
        case(4096, 4000, 65, 1, 3, 3, dtype, fk.PREFILL_FFT, fk.DECODE_FFT, recon_engine=2); n += 1
        case(32768, 300, 48, 1, 2, 4, dtype, fk.PREFILL_AUTO, fk.DECODE_AUTO, recon_engine=2); n += 1
        # the paper's window, per step and block-deferred
        case(256, 150, 33, 2, 2, 8, dtype, fk.PREFILL_SIMT, fk.DECODE_AUTO, S=10, R=50); n += 1
        case(512, 100, 24, 1, 2, 4, dtype, fk.PREFILL_SIMT, fk.DECODE_FFT_TWO_PASS, S=4, R=6, D=5); n += 1
    case(200, 333, 37, 1, 2, 4, bf16, fk.PREFILL_UMMA, fk.DECODE_UMMA); n += 1
    print(f"checked build: {n} cases ok")


if __name__ == "__main__":
    main()
