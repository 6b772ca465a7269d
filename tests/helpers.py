"""Glue used by the parity tests: run the float64 oracle over batched tensors and compare."""
from __future__ import annotations

import numpy as np
import torch

# Tolerances of the build's acceptance bar.
REL_L2_F32 = 1e-4     # float32 paths: coefficients, reconstructed K/V
REL_L2_BF16 = 3e-3    # bf16 storage paths
ATTN_MAX_ABS = 2e-3   # decode-attention outputs


def rel_l2(got, want) -> float:
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    den = np.sqrt((want ** 2).sum())
    return float(np.sqrt(((got - want) ** 2).sum()) / (den if den > 0 else 1.0))


def to_np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def oracle_compress(orc, K: torch.Tensor, P: int, bins: np.ndarray) -> np.ndarray:
    """K [B,H,T,d] (stored values) -> float64 planes [B,H,2,M,d]."""
    re, im = orc.compress(to_np64(K), P, bins)
    return np.stack([re, im], axis=2)


def oracle_append(orc, coef: np.ndarray, P: int, bins: np.ndarray, t_len: np.ndarray, x_new: torch.Tensor):
    """In-place on coef [B,H,2,M,d]; x_new [B,H,d]; t_len [B] are the positions used (not advanced here)."""
    x = to_np64(x_new)
    B, H = coef.shape[:2]
    for b in range(B):
        for h in range(H):
            re = np.ascontiguousarray(coef[b, h, 0])
            im = np.ascontiguousarray(coef[b, h, 1])
            orc.append(re, im, P, bins, int(t_len[b]), x[b, h])
            coef[b, h, 0], coef[b, h, 1] = re, im


def oracle_reconstruct(orc, coef: np.ndarray, P: int, bins: np.ndarray, t_len: np.ndarray, L: int) -> np.ndarray:
    """coef [B,H,2,M,d] -> [B,H,L,d]; rows >= min(t_len[b], P) are zero."""
    B, H, _, M, d = coef.shape
    out = np.zeros((B, H, L, d))
    for b in range(B):
        live = min(int(t_len[b]), P, L)
        for h in range(H):
            if live > 0:
                out[b, h, :live] = orc.reconstruct(coef[b, h, 0], coef[b, h, 1], P, bins, live)
    return out


def oracle_decode_attn(orc, q: torch.Tensor, coefK: np.ndarray, coefV: np.ndarray, P: int,
                       bins: np.ndarray, t_len: np.ndarray, scale=None) -> np.ndarray:
    """q [B,HQ,d] -> [B,HQ,d]; query head g uses kv head g // (HQ // H)."""
    qn = to_np64(q)
    B, HQ, d = qn.shape
    H = coefK.shape[1]
    G = HQ // H
    out = np.zeros((B, HQ, d))
    for b in range(B):
        L = min(int(t_len[b]), P)
        for h in range(H):
            out[b, h * G:(h + 1) * G] = orc.decode_attn(
                qn[b, h * G:(h + 1) * G], coefK[b, h, 0], coefK[b, h, 1], coefV[b, h, 0], coefV[b, h, 1],
                P, bins, L, scale)
    return out


class Guarded:
    """A device tensor with a 256-byte canary before and after it: `t` is the tensor to hand to the library,
    check() asserts that no byte outside it was written.  (The exact-zero and NaN fills of the parity tests catch
    elements a kernel failed to write; this catches writes past either end.)"""
    GUARD = 256
    PATTERN = 0xA5

    def __init__(self, shape, dtype, fill=None, device="cuda"):
        n = 1
        for s in shape:
            n *= int(s)
        nbytes = n * torch.empty((), dtype=dtype).element_size()
        self.raw = torch.full((nbytes + 2 * self.GUARD,), self.PATTERN, dtype=torch.uint8, device=device)
        self.t = self.raw[self.GUARD:self.GUARD + nbytes].view(dtype).view(*shape)
        assert self.t.data_ptr() % 16 == 0
        if fill is not None:
            self.t.fill_(fill)
        self.nbytes = nbytes

    def check(self, what=""):
        head = self.raw[:self.GUARD]
        tail = self.raw[self.GUARD + self.nbytes:]
        assert bool((head == self.PATTERN).all()), f"bytes before {what or 'the tensor'} were overwritten"
        assert bool((tail == self.PATTERN).all()), f"bytes behind {what or 'the tensor'} were overwritten"
