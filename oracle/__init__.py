"""Float64 CPU oracle of the FAEDKV / IWDFT hot path -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper over ``faedkv_oracle.c`` (plain C, compiled with gcc).  It
is imported by the tests, by the smoke check and by the benchmark's CPU-baseline
leg, and by nothing else; it shares no code with the CUDA path and does not
import it.

All arrays are float64 numpy arrays.  One "unit" is the ``[T, d]`` real matrix
of one (batch, kv head, K-or-V); its compressed state is two ``[M, d]`` planes
(real, imaginary) over the retained one-sided bins.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "faedkv_oracle.c")
_LIB_DIR = os.path.join(_HERE, "_build")
_LIB = os.path.join(_LIB_DIR, "libfaedkv_oracle.so")

_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc -O2 -fopenmp; returns the library path."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    os.makedirs(_LIB_DIR, exist_ok=True)
    tmp = _LIB + ".tmp.%d" % os.getpid()
    cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
           "-ffp-contract=off", _SRC, "-o", tmp, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


_f64p = ctypes.POINTER(ctypes.c_double)
_i32p = ctypes.POINTER(ctypes.c_int32)
_u8p = ctypes.POINTER(ctypes.c_uint8)
_int = ctypes.c_int
_i64 = ctypes.c_int64
_u64 = ctypes.c_uint64
_f64 = ctypes.c_double


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    sig = {
        "orc_weight": (_f64, [_int, _int]),
        "orc_plan": (_int, [_int, _u8p, _i32p]),
        "orc_fold_two_sided": (None, [_int, _u8p, _u8p]),
        "orc_mask_lowpass": (_int, [_int, _int, _u8p]),
        "orc_mask_mixed": (_int, [_int, _int, _int, _u64, _u8p]),
        "orc_compress": (None, [_f64p, _int, _int, _int, _i32p, _int, _i64, _f64p, _f64p]),
        "orc_compress_units": (None, [_f64p, _int, _int, _int, _int, _i32p, _int, _i64, _f64p, _f64p]),
        "orc_append": (None, [_f64p, _f64p, _int, _int, _int, _i32p, _i64, _f64p]),
        "orc_reconstruct": (None, [_f64p, _f64p, _int, _int, _int, _i32p, _int, _f64p]),
        "orc_reconstruct_rows": (None, [_f64p, _f64p, _int, _int, _int, _i32p, _i32p, _int, _f64p]),
        "orc_attention_dense": (None, [_f64p, _int, _f64p, _f64p, _int, _int, _f64, _f64p]),
        "orc_decode_attn": (None, [_f64p, _int, _f64p, _f64p, _f64p, _f64p, _int, _int, _int,
                                   _i32p, _int, _f64, _f64p]),
        "orc_rotating_frame_step": (None, [_f64p, _f64p, _int, _int, _int, _i32p, _f64p]),
        "orc_sliding_window_step": (None, [_f64p, _f64p, _int, _int, _int, _i32p, _f64p, _f64p]),
        "orc_running_mean_step": (None, [_f64p, _f64p, _int, _int, _int, _i32p, _i64, _f64p]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


def _d(a):
    assert a.dtype == np.float64 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(_f64p)


def _i(a):
    assert a.dtype == np.int32 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(_i32p)


def _u(a):
    assert a.dtype == np.uint8 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(_u8p)


def _f64arr(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def set_threads(n: int) -> None:
    """Limit the OpenMP team used by the oracle (for the 1-thread timing)."""
    _load()
    omp = ctypes.CDLL("libgomp.so.1")
    omp.omp_set_num_threads(int(n))


def weight(P: int, k: int) -> float:
    return float(_load().orc_weight(P, k))


def weights(P: int, bins: np.ndarray) -> np.ndarray:
    return np.array([weight(P, int(k)) for k in bins], dtype=np.float64)


def plan(P: int, mask: np.ndarray) -> np.ndarray:
    """One-sided keep mask (length P//2+1) -> ascending retained bin indices."""
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    assert mask.shape == (P // 2 + 1,)
    bins = np.zeros(P // 2 + 1, dtype=np.int32)
    M = _load().orc_plan(P, _u(mask), _i(bins))
    return bins[:M].copy()


def fold_two_sided(P: int, mask2: np.ndarray) -> np.ndarray:
    mask2 = np.ascontiguousarray(mask2, dtype=np.uint8)
    assert mask2.shape == (P,)
    out = np.zeros(P // 2 + 1, dtype=np.uint8)
    _load().orc_fold_two_sided(P, _u(mask2), _u(out))
    return out


def mask_lowpass(P: int, M: int) -> np.ndarray:
    out = np.zeros(P // 2 + 1, dtype=np.uint8)
    if _load().orc_mask_lowpass(P, M, _u(out)) != 0:
        raise ValueError("bad low-pass mask request")
    return out


def mask_mixed(P: int, M: int, layer: int, seed: int) -> np.ndarray:
    out = np.zeros(P // 2 + 1, dtype=np.uint8)
    if _load().orc_mask_mixed(P, M, layer, seed, _u(out)) != 0:
        raise ValueError("bad mixed mask request")
    return out


def compress(x: np.ndarray, P: int, bins: np.ndarray, pos0: int = 0):
    """Pruned DFT of x [..., T, d] along the token axis -> (Cre, Cim) [..., M, d]."""
    x = _f64arr(x)
    bins = np.ascontiguousarray(bins, dtype=np.int32)
    lead, (T, d) = x.shape[:-2], x.shape[-2:]
    U = int(np.prod(lead)) if lead else 1
    M = bins.shape[0]
    Cre = np.zeros((U, M, d), dtype=np.float64)
    Cim = np.zeros((U, M, d), dtype=np.float64)
    if U == 1:
        _load().orc_compress(_d(x), T, d, P, _i(bins), M, pos0, _d(Cre), _d(Cim))
    else:
        _load().orc_compress_units(_d(x), U, T, d, P, _i(bins), M, pos0, _d(Cre), _d(Cim))
    return Cre.reshape(*lead, M, d), Cim.reshape(*lead, M, d)


def append(Cre: np.ndarray, Cim: np.ndarray, P: int, bins: np.ndarray, t: int, xnew: np.ndarray):
    """In-place IWDFT update of one unit's [M, d] planes with the token at position t."""
    bins = np.ascontiguousarray(bins, dtype=np.int32)
    xnew = _f64arr(xnew)
    M, d = Cre.shape
    assert Cim.shape == (M, d) and xnew.shape == (d,) and bins.shape == (M,)
    _load().orc_append(_d(Cre), _d(Cim), M, d, P, _i(bins), t, _d(xnew))


def reconstruct(Cre: np.ndarray, Cim: np.ndarray, P: int, bins: np.ndarray, L: int) -> np.ndarray:
    """Pruned inverse DFT of one unit's planes -> [L, d]."""
    bins = np.ascontiguousarray(bins, dtype=np.int32)
    Cre, Cim = _f64arr(Cre), _f64arr(Cim)
    M, d = Cre.shape
    out = np.zeros((L, d), dtype=np.float64)
    _load().orc_reconstruct(_d(Cre), _d(Cim), M, d, P, _i(bins), L, _d(out))
    return out


def reconstruct_rows(Cre: np.ndarray, Cim: np.ndarray, P: int, bins: np.ndarray, rows) -> np.ndarray:
    """Pruned inverse DFT of one unit's planes at the listed positions only -> [len(rows), d]."""
    bins = np.ascontiguousarray(bins, dtype=np.int32)
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    Cre, Cim = _f64arr(Cre), _f64arr(Cim)
    M, d = Cre.shape
    out = np.zeros((rows.shape[0], d), dtype=np.float64)
    _load().orc_reconstruct_rows(_d(Cre), _d(Cim), M, d, P, _i(bins), _i(rows), int(rows.shape[0]), _d(out))
    return out


def attention_dense(q: np.ndarray, Kt: np.ndarray, Vt: np.ndarray, scale: float) -> np.ndarray:
    q, Kt, Vt = _f64arr(q), _f64arr(Kt), _f64arr(Vt)
    G, d = q.shape
    L = Kt.shape[0]
    out = np.zeros((G, d), dtype=np.float64)
    _load().orc_attention_dense(_d(q), G, _d(Kt), _d(Vt), L, d, scale, _d(out))
    return out


def decode_attn(q: np.ndarray, CKre, CKim, CVre, CVim, P: int, bins: np.ndarray, L: int,
                scale: float | None = None) -> np.ndarray:
    """q [G, d] (query heads of one kv head) against one kv head's planes -> [G, d]."""
    bins = np.ascontiguousarray(bins, dtype=np.int32)
    q = _f64arr(q)
    CKre, CKim, CVre, CVim = map(_f64arr, (CKre, CKim, CVre, CVim))
    G, d = q.shape
    M = bins.shape[0]
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    out = np.zeros((G, d), dtype=np.float64)
    _load().orc_decode_attn(_d(q), G, _d(CKre), _d(CKim), _d(CVre), _d(CVim), M, d, P,
                            _i(bins), L, scale, _d(out))
    return out


def rotating_frame_step(Rre, Rim, P, bins, xnew):
    bins = np.ascontiguousarray(bins, dtype=np.int32)
    M, d = Rre.shape
    _load().orc_rotating_frame_step(_d(Rre), _d(Rim), M, d, P, _i(bins), _d(_f64arr(xnew)))


def sliding_window_step(Sre, Sim, P, bins, x_out, x_in):
    bins = np.ascontiguousarray(bins, dtype=np.int32)
    M, d = Sre.shape
    _load().orc_sliding_window_step(_d(Sre), _d(Sim), M, d, P, _i(bins),
                                    _d(_f64arr(x_out)), _d(_f64arr(x_in)))


def running_mean_step(Sre, Sim, P, bins, t, xnew):
    bins = np.ascontiguousarray(bins, dtype=np.int32)
    M, d = Sre.shape
    _load().orc_running_mean_step(_d(Sre), _d(Sim), M, d, P, _i(bins), t, _d(_f64arr(xnew)))


# ---------------------------------------------------------------------------------------------------
# Sink and recent window (Sec. 4.2): the paper's own decode workflow for ONE (sequence, kv head) unit,
# written as a composition of the primitives above -- no new arithmetic.
class WindowedUnit:
    """State of one unit: the first S tokens (sink) and the most recent tokens in the time domain, the
    tokens between them as retained DFT coefficients of the segment that starts at token S.

    defer = 1 is the paper's step (Eq. 12): every step the token that leaves the R-token recent window is
    folded into the coefficients.  defer = D > 1 is the block form of the same update: tokens wait in the
    time domain until R + D of them are unfolded, then the D oldest are folded in one go, oldest first.
    Whenever (t - S - R) is a multiple of D the two forms hold the same state; in between the block form
    attends over up to D - 1 more exact tokens."""

    def __init__(self, P: int, bins: np.ndarray, S: int, R: int, defer: int = 1):
        self.P, self.bins, self.S, self.R = int(P), np.ascontiguousarray(bins, dtype=np.int32), int(S), int(R)
        self.D = int(defer)
        assert self.D >= 1
        self.t = 0
        self.folded = 0                              # tokens in the transformed segment
        self.sinkK = self.sinkV = None
        self.recentK, self.recentV = [], []          # unfolded tokens after the sink, oldest first
        self.CK = self.CV = None                     # (re, im) pairs of [M, d]

    def prefill(self, K: np.ndarray, V: np.ndarray) -> None:
        """Eq. 10: transform K[S : S + folded], V[S : S + folded]; keep the first S rows and the rows after
        the transformed segment as they are.  folded = T - S - R rounded down to a multiple of defer."""
        K, V = _f64arr(K), _f64arr(V)
        T, d = K.shape
        S, R = self.S, self.R
        assert T >= S + R
        self.folded = (T - S - R) // self.D * self.D
        first = S + self.folded                      # first unfolded token
        self.sinkK, self.sinkV = K[:S].copy(), V[:S].copy()
        self.recentK = [K[n].copy() for n in range(first, T)]
        self.recentV = [V[n].copy() for n in range(first, T)]
        M = self.bins.shape[0]
        if self.folded > 0:
            self.CK = [np.ascontiguousarray(a) for a in compress(K[S:first], self.P, self.bins)]
            self.CV = [np.ascontiguousarray(a) for a in compress(V[S:first], self.P, self.bins)]
        else:
            self.CK = [np.zeros((M, d)), np.zeros((M, d))]
            self.CV = [np.zeros((M, d)), np.zeros((M, d))]
        self.t = T

    def step(self, k_new: np.ndarray, v_new: np.ndarray) -> None:
        """Eq. 12: the new token enters the window; once R + defer tokens are unfolded the oldest `defer` of
        them are folded at the next positions of the transformed segment (defer = 1: the one token leaving
        the recent window; with R = 0 the new token itself)."""
        k_new, v_new = _f64arr(k_new), _f64arr(v_new)
        self.recentK.append(k_new.copy())
        self.recentV.append(v_new.copy())
        self.t += 1
        if len(self.recentK) >= self.R + self.D:
            for _ in range(self.D):
                k_old, v_old = self.recentK.pop(0), self.recentV.pop(0)
                append(self.CK[0], self.CK[1], self.P, self.bins, self.folded, k_old)
                append(self.CV[0], self.CV[1], self.P, self.bins, self.folded, v_old)
                self.folded += 1

    def materialise(self) -> tuple[np.ndarray, np.ndarray]:
        """Eq. 13: K^ = [K_sink ; K~ ; K_recent] and the same for V (Eq. 13's V row read with V~), the
        reconstruction covering the min(folded, P) positions of the transformed segment."""
        L = min(self.folded, self.P)
        parts_k, parts_v = [self.sinkK], [self.sinkV]
        if L > 0:
            parts_k.append(reconstruct(self.CK[0], self.CK[1], self.P, self.bins, L))
            parts_v.append(reconstruct(self.CV[0], self.CV[1], self.P, self.bins, L))
        if self.recentK:
            parts_k.append(np.stack(self.recentK))
            parts_v.append(np.stack(self.recentV))
        Kt = np.concatenate([p for p in parts_k if p.shape[0] > 0], axis=0)
        Vt = np.concatenate([p for p in parts_v if p.shape[0] > 0], axis=0)
        return Kt, Vt

    def attention(self, q: np.ndarray, scale: float | None = None) -> np.ndarray:
        """Eq. 13 then Eq. 3: one softmax over [sink | reconstructed segment | unfolded recent tokens]."""
        q = _f64arr(q)
        d = q.shape[1]
        if scale is None:
            scale = 1.0 / np.sqrt(d)
        Kt, Vt = self.materialise()
        return attention_dense(q, Kt, Vt, scale)


# ---------------------------------------------------------------------------------------------------
# Frequency ablation and bin selection (Sec. 3.2).  Integer logic in plain Python; the ablation itself is
# the definition written out with numpy's float64 FFT as the library step.
def chunk_range(P: int, C: int, c: int) -> tuple[int, int]:
    """Two-sided bins [lo, hi) of chunk c when the P bins are cut into C contiguous chunks of P // C bins;
    the last chunk takes the remainder."""
    assert 1 <= C <= P and 0 <= c < C
    w = P // C
    return c * w, (P if c == C - 1 else (c + 1) * w)


def ablate(x: np.ndarray, P: int, lo: int, hi: int) -> np.ndarray:
    """Eq. 6 then Eq. 5: DFT of x [T, d] (T <= P, zero-padded to the grid) along the token axis, bins
    lo <= k < hi set to zero, inverse DFT, real part, first T rows."""
    x = _f64arr(x)
    T = x.shape[0]
    assert T <= P
    X = np.fft.fft(x, n=P, axis=0)
    X[lo:hi] = 0.0
    return np.fft.ifft(X, axis=0).real[:T]


def ablation_bins(P: int, lo: int, hi: int) -> tuple[np.ndarray, np.ndarray]:
    """One-sided view of zeroing two-sided bins [lo, hi) of a REAL signal: mask[k] = 1 for every
    k in [0, P/2] whose bin k or mirror P-k is zeroed, gain[k] = the share of that bin's real component
    that disappears: 1 when both k and P-k are zeroed (or k is its own mirror), else 1/2."""
    n1 = P // 2 + 1
    mask = np.zeros(n1, dtype=np.uint8)
    gain = np.zeros(n1, dtype=np.float32)
    for k in range(n1):
        a = lo <= k < hi
        b = lo <= (P - k) % P < hi
        if a or b:
            mask[k] = 1
            gain[k] = 1.0 if (a and b) else 0.5
    return mask, gain


def mask_from_scores(P: int, C: int, delta, ratio: float) -> tuple[np.ndarray, int]:
    """Greedy selection: keep the n_keep = max(1, floor(ratio * C + 1/2)) chunks with the largest
    perplexity change delta (ties: the lower chunk index wins); a one-sided bin is kept when it or its
    mirror lies in a kept chunk."""
    delta = [float(v) for v in delta]
    assert len(delta) == C
    n_keep = max(1, int(np.floor(ratio * C + 0.5)))
    n_keep = min(n_keep, C)
    order = sorted(range(C), key=lambda c: (-delta[c], c))
    keep2 = np.zeros(P, dtype=np.uint8)
    for c in order[:n_keep]:
        lo, hi = chunk_range(P, C, c)
        keep2[lo:hi] = 1
    return fold_two_sided(P, keep2), n_keep
