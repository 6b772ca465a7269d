"""Pins of the float64 oracle against things other than itself.

Each test fixes the oracle to a closed form, a library routine that is
structurally different (numpy's FFT), an invariant the paper states, or brute
force written out independently here.  A dropped term, a wrong sign or index,
or a transposed operand in the oracle fails at least one of them.
"""
import numpy as np
import pytest

TWO_PI = 2.0 * np.pi


def _rng(seed):
    return np.random.default_rng(seed)


def _all_bins(P):
    return np.arange(P // 2 + 1, dtype=np.int32)


# ----------------------------------------------------------------- P1: numpy rfft / brute force
@pytest.mark.parametrize("P,T", [(8, 8), (16, 11), (15, 15), (21, 9), (64, 64), (100, 77), (37, 37)])
def test_compress_matches_rfft(oracle, P, T):
    """Eq. 4 restricted to retained bins == numpy.fft.rfft(x, n=P) gathered (T <= P)."""
    x = _rng(P * 1000 + T).standard_normal((T, 5))
    bins = _all_bins(P)[::2].copy() if P > 10 else _all_bins(P)
    Cre, Cim = oracle.compress(x, P, bins)
    ref = np.fft.rfft(x, n=P, axis=0)[bins]
    np.testing.assert_allclose(Cre, ref.real, atol=1e-11)
    np.testing.assert_allclose(Cim, ref.imag, atol=1e-11)


def test_compress_brute_force_tiny(oracle):
    """Direct complex-exponential sum written here, including T > P (positions wrap)."""
    P, T, d = 12, 29, 3
    x = _rng(7).standard_normal((T, d))
    bins = np.array([0, 1, 4, 6], dtype=np.int32)
    want = np.zeros((len(bins), d), dtype=np.complex128)
    for i, k in enumerate(bins):
        for n in range(T):
            want[i] += x[n] * np.exp(-1j * TWO_PI * k * n / P)
    Cre, Cim = oracle.compress(x, P, bins)
    np.testing.assert_allclose(Cre + 1j * Cim, want, atol=1e-12)


def test_compress_units_equals_single(oracle):
    P, T, d = 32, 32, 4
    x = _rng(3).standard_normal((2, 3, T, d))
    bins = np.array([0, 2, 3, 9, 16], dtype=np.int32)
    Cre, Cim = oracle.compress(x, P, bins)
    for b in range(2):
        for h in range(3):
            r1, i1 = oracle.compress(x[b, h], P, bins)
            np.testing.assert_array_equal(Cre[b, h], r1[0] if r1.ndim == 3 else r1)
            np.testing.assert_array_equal(Cim[b, h], i1[0] if i1.ndim == 3 else i1)


# ----------------------------------------------------------------- P2: constant sequence
@pytest.mark.parametrize("P,T", [(16, 16), (16, 10), (25, 40)])
def test_constant_sequence_closed_form(oracle, P, T):
    a = 1.75
    x = np.full((T, 2), a)
    bins = _all_bins(P)
    Cre, Cim = oracle.compress(x, P, bins)
    C = Cre + 1j * Cim
    for i, k in enumerate(bins):
        if k == 0:
            want = a * T
        else:
            w = np.exp(-1j * TWO_PI * k / P)
            want = a * (1 - w ** T) / (1 - w)  # geometric series
        np.testing.assert_allclose(C[i], want, atol=1e-10)
    if T == P:
        assert np.allclose(C[1:], 0, atol=1e-10) and np.allclose(C[0], a * P)


# ----------------------------------------------------------------- P3: impulse (phase sign)
def test_impulse_closed_form(oracle):
    P, n0, a = 24, 5, -2.5
    x = np.zeros((P, 1))
    x[n0] = a
    bins = _all_bins(P)
    Cre, Cim = oracle.compress(x, P, bins)
    want = a * np.exp(-1j * TWO_PI * bins * n0 / P)
    np.testing.assert_allclose(Cre[:, 0] + 1j * Cim[:, 0], want, atol=1e-12)
    np.testing.assert_allclose(np.hypot(Cre, Cim), abs(a), atol=1e-12)
    # the sign of the imaginary part distinguishes exp(-j..) from exp(+j..)
    assert Cim[1, 0] * a * np.sin(TWO_PI * n0 / P) < 0


# ----------------------------------------------------------------- P4: single cosine
@pytest.mark.parametrize("P,k0", [(32, 5), (32, 0), (32, 16), (27, 4)])
def test_single_cosine(oracle, P, k0):
    n = np.arange(P)
    x = np.cos(TWO_PI * k0 * n / P)[:, None]
    bins = _all_bins(P)
    Cre, Cim = oracle.compress(x, P, bins)
    peak = P if (k0 == 0 or (P % 2 == 0 and k0 == P // 2)) else P / 2
    want = np.zeros(len(bins))
    want[k0] = peak
    np.testing.assert_allclose(Cre[:, 0], want, atol=1e-10)
    np.testing.assert_allclose(Cim[:, 0], 0, atol=1e-10)
    # any mask containing k0 returns x
    keep = np.array(sorted({0, k0, min(k0 + 3, P // 2)}), dtype=np.int32)
    r, i = oracle.compress(x, P, keep)
    back = oracle.reconstruct(r, i, P, keep, P)
    np.testing.assert_allclose(back, x, atol=1e-12)


def test_sine_phase_and_weight(oracle):
    """x = sin(2 pi k0 n / P): C[k0] = -j P/2; reconstruct needs w_k = 2 and the minus on Im*sin."""
    P, k0 = 40, 7
    n = np.arange(P)
    x = np.sin(TWO_PI * k0 * n / P)[:, None]
    bins = np.array([k0], dtype=np.int32)
    Cre, Cim = oracle.compress(x, P, bins)
    np.testing.assert_allclose(Cre, 0, atol=1e-10)
    np.testing.assert_allclose(Cim, -P / 2, atol=1e-10)
    np.testing.assert_allclose(oracle.reconstruct(Cre, Cim, P, bins, P), x, atol=1e-12)


# ----------------------------------------------------------------- P5: appends == batch transform
@pytest.mark.parametrize("P,T,T1", [(32, 32, 0), (32, 32, 20), (24, 61, 24), (50, 37, 10)])
def test_appends_equal_batch(oracle, P, T, T1):
    d = 6
    x = _rng(P + T).standard_normal((T, d))
    bins = np.array(sorted(set(_rng(1).integers(0, P // 2 + 1, size=7).tolist())), dtype=np.int32)
    if T1 == 0:
        Cre = np.zeros((len(bins), d))
        Cim = np.zeros((len(bins), d))
    else:
        Cre, Cim = oracle.compress(x[:T1], P, bins)
        Cre, Cim = Cre.copy(), Cim.copy()
    for t in range(T1, T):
        oracle.append(Cre, Cim, P, bins, t, x[t])
    Bre, Bim = oracle.compress(x, P, bins)
    scale = np.abs(Bre).max() + np.abs(Bim).max()
    assert np.abs(Cre - Bre).max() <= 1e-12 * scale
    assert np.abs(Cim - Bim).max() <= 1e-12 * scale


def test_compress_pos0_equals_shifted(oracle):
    """A chunk transformed at offset pos0 equals that chunk's share of the whole transform."""
    P, T, d = 40, 55, 3
    x = _rng(11).standard_normal((T, d))
    bins = np.array([0, 3, 7, 20], dtype=np.int32)
    a_re, a_im = oracle.compress(x[:17], P, bins)
    b_re, b_im = oracle.compress(x[17:], P, bins, pos0=17)
    w_re, w_im = oracle.compress(x, P, bins)
    np.testing.assert_allclose(a_re + b_re, w_re, atol=1e-11)
    np.testing.assert_allclose(a_im + b_im, w_im, atol=1e-11)


# ----------------------------------------------------------------- P6: perfect reconstruction / periodic sum
@pytest.mark.parametrize("P", [16, 31, 64])
def test_all_bins_reconstruct_identity(oracle, P):
    d = 4
    for t in (P, P - 5):
        x = _rng(P + t).standard_normal((t, d))
        bins = _all_bins(P)
        Cre, Cim = oracle.compress(x, P, bins)
        back = oracle.reconstruct(Cre, Cim, P, bins, t)
        np.testing.assert_allclose(back, x, atol=1e-12)
        # rows beyond t reconstruct the zero padding
        full = oracle.reconstruct(Cre, Cim, P, bins, P)
        np.testing.assert_allclose(full[t:], 0, atol=1e-12)


def test_wraparound_periodic_sum(oracle):
    P, T, d = 20, 53, 2
    x = _rng(5).standard_normal((T, d))
    bins = _all_bins(P)
    Cre, Cim = oracle.compress(x, P, bins)
    want = np.zeros((P, d))
    for n in range(T):
        want[n % P] += x[n]
    np.testing.assert_allclose(oracle.reconstruct(Cre, Cim, P, bins, P), want, atol=1e-12)


# ----------------------------------------------------------------- P7: printed rotating-frame / sliding-window recursions
def test_rotating_frame_recursion_relation(oracle):
    """R <- W_k (R + x) (Eq. 9 without normalisation) gives R_t = W_k^t conj(C_t) for real x."""
    P, T, d = 36, 50, 3
    x = _rng(9).standard_normal((T, d))
    bins = np.array([0, 1, 5, 11, 18], dtype=np.int32)
    Rre = np.zeros((len(bins), d))
    Rim = np.zeros((len(bins), d))
    for t in range(T):
        oracle.rotating_frame_step(Rre, Rim, P, bins, x[t])
    Cre, Cim = oracle.compress(x, P, bins)
    Wt = np.exp(-1j * TWO_PI * bins * T / P)[:, None]
    want = Wt * (Cre - 1j * Cim)
    np.testing.assert_allclose(Rre + 1j * Rim, want, atol=1e-11)
    np.testing.assert_allclose(np.hypot(Rre, Rim), np.hypot(Cre, Cim), atol=1e-11)


def test_sliding_window_recursion(oracle):
    """Eq. 8 with window P tracks the last P tokens in the same newest-referenced frame."""
    P, T, d = 16, 45, 2
    x = _rng(10).standard_normal((T, d))
    bins = _all_bins(P)
    Sre = np.zeros((len(bins), d))
    Sim = np.zeros((len(bins), d))
    zero = np.zeros(d)
    for t in range(T):
        x_out = x[t - P] if t >= P else zero
        oracle.sliding_window_step(Sre, Sim, P, bins, x_out, x[t])
    # S[k] = sum over the last P tokens of x[n] W_k^(T-n)
    want = np.zeros((len(bins), d), dtype=np.complex128)
    for n in range(T - P, T):
        want += x[n][None, :] * np.exp(-1j * TWO_PI * bins * (T - n) / P)[:, None]
    np.testing.assert_allclose(Sre + 1j * Sim, want, atol=1e-11)


# ----------------------------------------------------------------- P8: running-mean normalisation with exact factors
def test_running_mean_times_t_is_sum_state(oracle):
    P, T, d = 30, 70, 3
    x = _rng(12).standard_normal((T, d))
    bins = np.array([0, 2, 7, 15], dtype=np.int32)
    Sre = np.zeros((len(bins), d))
    Sim = np.zeros((len(bins), d))
    for t in range(T):
        oracle.running_mean_step(Sre, Sim, P, bins, t, x[t])
    Cre, Cim = oracle.compress(x, P, bins)
    np.testing.assert_allclose(Sre * T, Cre, atol=1e-11)
    np.testing.assert_allclose(Sim * T, Cim, atol=1e-11)


# ----------------------------------------------------------------- P9: Parseval, projection
@pytest.mark.parametrize("P", [32, 45])
def test_parseval_and_projection(oracle, P):
    d = 3
    x = _rng(P).standard_normal((P, d))
    bins = _all_bins(P)
    Cre, Cim = oracle.compress(x, P, bins)
    w = oracle.weights(P, bins)[:, None]
    np.testing.assert_allclose((x ** 2).sum(0), (w * (Cre ** 2 + Cim ** 2)).sum(0) / P, rtol=1e-12)
    keep = bins[(bins % 3) != 1].copy()
    r, i = oracle.compress(x, P, keep)
    y = oracle.reconstruct(r, i, P, keep, P)
    r2, i2 = oracle.compress(y, P, keep)
    y2 = oracle.reconstruct(r2, i2, P, keep, P)
    np.testing.assert_allclose(y2, y, atol=1e-12)          # idempotent
    assert ((y ** 2).sum() <= (x ** 2).sum() * (1 + 1e-12))  # never gains energy
    np.testing.assert_allclose(r2, r, atol=1e-10)
    np.testing.assert_allclose(i2, i, atol=1e-10)


def test_weights(oracle):
    assert oracle.weight(16, 0) == 1.0 and oracle.weight(16, 8) == 1.0 and oracle.weight(16, 3) == 2.0
    assert oracle.weight(15, 0) == 1.0 and oracle.weight(15, 7) == 2.0


# ----------------------------------------------------------------- P10: DC-only mask
def test_dc_only(oracle):
    P, d, G = 32, 8, 4
    rng = _rng(21)
    K = rng.standard_normal((P, d))
    V = rng.standard_normal((P, d))
    q = rng.standard_normal((G, d))
    bins = np.array([0], dtype=np.int32)
    kr, ki = oracle.compress(K, P, bins)
    vr, vi = oracle.compress(V, P, bins)
    np.testing.assert_allclose(oracle.reconstruct(vr, vi, P, bins, P),
                               np.broadcast_to(V.mean(0), (P, d)), atol=1e-12)
    out = oracle.decode_attn(q, kr, ki, vr, vi, P, bins, P)
    np.testing.assert_allclose(out, np.broadcast_to(V.mean(0), (G, d)), atol=1e-12)


# ----------------------------------------------------------------- P11: all bins -> textbook attention
def _textbook_attention(q, K, V, scale):
    s = (q @ K.T) * scale
    s = s - s.max(axis=1, keepdims=True)
    p = np.exp(s)
    p /= p.sum(axis=1, keepdims=True)
    return p @ V


@pytest.mark.parametrize("P,t", [(32, 32), (33, 20)])
def test_all_bins_attention_is_textbook(oracle, P, t):
    d, G = 16, 4
    rng = _rng(P + t)
    K = rng.standard_normal((t, d))
    V = rng.standard_normal((t, d))
    q = rng.standard_normal((G, d))
    bins = _all_bins(P)
    kr, ki = oracle.compress(K, P, bins)
    vr, vi = oracle.compress(V, P, bins)
    out = oracle.decode_attn(q, kr, ki, vr, vi, P, bins, t)
    np.testing.assert_allclose(out, _textbook_attention(q, K, V, 1 / np.sqrt(d)), atol=1e-12)
    # explicit scale argument is honoured
    out2 = oracle.decode_attn(q, kr, ki, vr, vi, P, bins, t, scale=0.37)
    np.testing.assert_allclose(out2, _textbook_attention(q, K, V, 0.37), atol=1e-12)


def test_reconstruct_rows_is_the_inverse_transform_at_those_rows(oracle):
    """Row-wise reconstruction: with every bin kept it returns the input rows themselves (and x[n mod P] beyond P,
    the sum being P-periodic); with a pruned set it equals numpy's irfft of the zero-filled half spectrum."""
    P, d = 48, 5
    rng = _rng(77)
    x = rng.standard_normal((P, d))
    bins = _all_bins(P)
    cr, ci = oracle.compress(x, P, bins)
    rows = np.array([0, 1, 17, 47, 46, 5], dtype=np.int32)
    np.testing.assert_allclose(oracle.reconstruct_rows(cr, ci, P, bins, rows), x[rows], atol=1e-12)
    np.testing.assert_allclose(oracle.reconstruct_rows(cr, ci, P, bins, rows + P), x[rows], atol=1e-12)
    keep = np.array([0, 2, 3, 7, 24], dtype=np.int32)               # includes both self-conjugate bins
    kr, ki = oracle.compress(x, P, keep)
    half = np.zeros((P // 2 + 1, d), dtype=complex)
    half[keep] = kr + 1j * ki
    want = np.fft.irfft(half, n=P, axis=0)
    np.testing.assert_allclose(oracle.reconstruct_rows(kr, ki, P, keep, rows), want[rows], atol=1e-12)
    np.testing.assert_allclose(oracle.reconstruct(kr, ki, P, keep, P)[rows], want[rows], atol=1e-12)


def test_attention_over_no_token_is_zero(oracle):
    """L = 0: Eq. 3 has no token to sum over; the reading taken is the empty sum, a zero vector (never NaN),
    and one token gives that token's value row whatever the query."""
    P, d, G = 16, 8, 3
    rng = _rng(5)
    q = rng.standard_normal((G, d))
    bins = _all_bins(P)
    V = rng.standard_normal((1, d))
    kr, ki = oracle.compress(rng.standard_normal((1, d)), P, bins)
    vr, vi = oracle.compress(V, P, bins)
    out0 = oracle.decode_attn(q, kr, ki, vr, vi, P, bins, 0)
    assert out0.shape == (G, d) and not out0.any()
    out1 = oracle.decode_attn(q, kr, ki, vr, vi, P, bins, 1)
    np.testing.assert_allclose(out1, np.broadcast_to(V[0], (G, d)), atol=1e-12)


# ----------------------------------------------------------------- P12: frequency-domain attention formula
def test_frequency_domain_attention_identity(oracle):
    """softmax(q K~^T) V~ can be evaluated without materialising K~, V~:
    Qf = q C_K^T;  s[n] = scale/P sum_k w_k Re(Qf[k] e^{+j w k n});  p = softmax(s);
    Pf[k] = sum_n p[n] e^{+j w k n};  o = (1/P) sum_k w_k Re(C_V[k] Pf[k]).
    Checked against the materialised oracle."""
    P, t, d, G = 48, 40, 8, 3
    rng = _rng(33)
    K = rng.standard_normal((t, d))
    V = rng.standard_normal((t, d))
    q = rng.standard_normal((G, d))
    bins = np.array([0, 1, 2, 3, 8, 9, 17, 24], dtype=np.int32)
    kr, ki = oracle.compress(K, P, bins)
    vr, vi = oracle.compress(V, P, bins)
    want = oracle.decode_attn(q, kr, ki, vr, vi, P, bins, t)
    w = oracle.weights(P, bins)
    CK, CV = kr + 1j * ki, vr + 1j * vi
    Qf = q @ CK.T                                     # [G, M]
    n = np.arange(t)
    E = np.exp(1j * TWO_PI * np.outer(bins, n) / P)   # [M, t]
    s = ((Qf * w) @ E).real / P / np.sqrt(d)
    s -= s.max(axis=1, keepdims=True)
    p = np.exp(s)
    p /= p.sum(axis=1, keepdims=True)
    Pf = p @ E.T                                      # [G, M]
    o = ((Pf * w) @ CV).real / P
    np.testing.assert_allclose(o, want, atol=1e-13)


# ----------------------------------------------------------------- P13: update-then-prune == update retained only
def test_append_prune_commutes(oracle):
    P, d = 28, 4
    rng = _rng(14)
    x = rng.standard_normal((P, d))
    xn = rng.standard_normal(d)
    allb = _all_bins(P)
    keep_idx = np.array([0, 3, 4, 9, 14])
    keep = allb[keep_idx].copy()
    fr, fi = oracle.compress(x, P, allb)
    # prune, update only the retained bins
    ar, ai = fr[keep_idx].copy(), fi[keep_idx].copy()
    oracle.append(ar, ai, P, keep, P, xn)
    # update every bin of the pruned (zero-filled) spectrum, then prune again (Eq. 6)
    zr, zi = np.zeros_like(fr), np.zeros_like(fi)
    zr[keep_idx], zi[keep_idx] = fr[keep_idx], fi[keep_idx]
    oracle.append(zr, zi, P, allb, P, xn)
    np.testing.assert_allclose(ar, zr[keep_idx], atol=1e-13)
    np.testing.assert_allclose(ai, zi[keep_idx], atol=1e-13)


# ----------------------------------------------------------------- P14: masks and plan
def test_plan_and_fold(oracle):
    P = 10
    mask = np.array([1, 0, 1, 1, 0, 1], dtype=np.uint8)
    np.testing.assert_array_equal(oracle.plan(P, mask), [0, 2, 3, 5])
    m2 = np.zeros(P, dtype=np.uint8)
    m2[[1, 7, 5]] = 1            # 7 mirrors 3
    np.testing.assert_array_equal(oracle.fold_two_sided(P, m2), [0, 1, 0, 1, 0, 1])


def test_lowpass_mask(oracle):
    m = oracle.mask_lowpass(64, 8)
    assert m.shape == (33,) and m.sum() == 8 and m[:8].all()
    with pytest.raises(ValueError):
        oracle.mask_lowpass(64, 34)


@pytest.mark.parametrize("P,M", [(256, 32), (2048, 256), (4096, 128)])
def test_mixed_mask_properties(oracle, P, M):
    seen = set()
    for layer in range(6):
        m = oracle.mask_mixed(P, M, layer, 1234)
        bins = oracle.plan(P, m)
        assert len(bins) == M and (np.diff(bins) > 0).all()
        assert bins[0] == 0 and bins[-1] < P // 2
        n_low = ((M // 2) // 16) * 16
        np.testing.assert_array_equal(bins[:n_low], np.arange(n_low))
        chunks = bins.reshape(-1, 16)
        assert (chunks[:, 0] % 16 == 0).all() and (np.diff(chunks, axis=1) == 1).all()
        np.testing.assert_array_equal(m, oracle.mask_mixed(P, M, layer, 1234))  # reproducible
        seen.add(bins.tobytes())
    assert len(seen) == 6                                                     # differs per layer
    # a different seed gives a different selection (large grid: a chance collision is negligible)
    assert oracle.mask_mixed(4096, 256, 0, 1).tobytes() != oracle.mask_mixed(4096, 256, 0, 2).tobytes()


def test_mixed_mask_independent_restatement(oracle):
    """The shuffle restated here in Python integers (LCG mod 2^64, Fisher-Yates prefix)."""
    P, M, layer, seed = 256, 32, 3, 20030000
    g = 16
    n_low = ((M // 2) // g) * g
    cand = list(range(n_low // g, (P // 2) // g))
    s = (seed * 2654435761 + layer) % (1 << 64)
    chosen = []
    for i in range((M - n_low) // g):
        s = (s * 6364136223846793005 + 1442695040888963407) % (1 << 64)
        j = i + (s >> 33) % (len(cand) - i)
        cand[i], cand[j] = cand[j], cand[i]
        chosen.append(cand[i])
    want = sorted(list(range(n_low)) + [c * g + b for c in chosen for b in range(g)])
    got = oracle.plan(P, oracle.mask_mixed(P, M, layer, seed))
    np.testing.assert_array_equal(got, want)


# ----------------------------------------------------------------------------- structural identities
def test_shift_theorem_and_linearity(oracle):
    """Delaying the sequence by d positions multiplies bin k by e^{-j2 pi k d / P} (the `pos0` argument is
    that delay), and the transform is linear: two facts a wrong phase sign, a transposed index or a
    dropped term in the pruned DFT cannot satisfy together."""
    P, T, d = 48, 31, 5
    rng = np.random.default_rng(77)
    x, y = rng.standard_normal((T, d)), rng.standard_normal((T, d))
    mask = np.zeros(P // 2 + 1, dtype=np.uint8)
    mask[[0, 1, 4, 9, 17, 24]] = 1
    bins = oracle.plan(P, mask)
    cx = np.array(oracle.compress(x, P, bins))
    cy = np.array(oracle.compress(y, P, bins))
    cz = np.array(oracle.compress(2.5 * x - 0.75 * y, P, bins))
    assert np.abs(cz - (2.5 * cx - 0.75 * cy)).max() < 1e-11
    for delay in (1, 7, P - 3, P + 2):
        sh = np.array(oracle.compress(x, P, bins, pos0=delay))
        ph = np.exp(-2j * np.pi * bins * delay / P)[:, None]
        want = (cx[0] + 1j * cx[1]) * ph
        assert np.abs(sh[0] + 1j * sh[1] - want).max() < 1e-10, delay


def test_reconstruction_is_the_best_band_limited_fit(oracle):
    """Eq. 5 on the retained bins of Eq. 4 is the orthogonal projection of the (zero-padded) sequence onto
    those frequencies: the residual is orthogonal to every retained cosine and sine, and no other
    coefficient vector on the same bins fits better (numpy least squares on the real basis)."""
    P, d = 40, 3
    rng = np.random.default_rng(78)
    x = rng.standard_normal((P, d))
    mask = np.zeros(P // 2 + 1, dtype=np.uint8)
    mask[[0, 2, 3, 11, 20]] = 1
    bins = oracle.plan(P, mask)
    re, im = oracle.compress(x, P, bins)
    rec = oracle.reconstruct(re, im, P, bins, P)
    n = np.arange(P)[:, None]
    basis = np.concatenate([np.cos(2 * np.pi * n * bins[None, :] / P), np.sin(2 * np.pi * n * bins[None, :] / P)], axis=1)
    assert np.abs(basis.T @ (x - rec)).max() < 1e-10
    fit = basis @ np.linalg.lstsq(basis, x, rcond=None)[0]
    assert np.abs(fit - rec).max() < 1e-10


# ----------------------------------------------------------------------------- sink + recent window
def _numpy_attention(q, K, V, scale):
    s = (q @ K.T) * scale
    s -= s.max(axis=1, keepdims=True)
    p = np.exp(s)
    return (p / p.sum(axis=1, keepdims=True)) @ V


@pytest.mark.parametrize("S,R", [(3, 5), (0, 4), (6, 0), (0, 0)])
def test_windowed_all_bins_is_full_attention(oracle, S, R):
    """Every bin retained and the sequence shorter than the grid: sink + exact reconstruction + recent is
    the whole cache, so the windowed workflow equals textbook attention over all tokens (numpy),
    whatever S and R, before and after decode steps."""
    P, T, d, G, steps = 64, 30, 8, 3, 9
    rng = np.random.default_rng(S * 10 + R)
    K, V = rng.standard_normal((T + steps, d)), rng.standard_normal((T + steps, d))
    bins = oracle.plan(P, np.ones(P // 2 + 1, dtype=np.uint8))
    u = oracle.WindowedUnit(P, bins, S, R)
    u.prefill(K[:T], V[:T])
    for s in range(steps + 1):
        q = rng.standard_normal((G, d))
        got = u.attention(q, 0.3)
        want = _numpy_attention(q, K[:T + s], V[:T + s], 0.3)
        assert np.abs(got - want).max() < 1e-11, (s, np.abs(got - want).max())
        if s < steps:
            u.step(K[T + s], V[T + s])
    assert u.t == T + steps


def test_windowed_without_window_is_plain_decode(oracle):
    """S = R = 0: prefill, step and attention reduce to compress, append and decode_attn."""
    P, T, d, G = 48, 40, 6, 2
    rng = np.random.default_rng(5)
    K, V = rng.standard_normal((T + 1, d)), rng.standard_normal((T + 1, d))
    mask = np.zeros(P // 2 + 1, dtype=np.uint8)
    mask[[0, 1, 2, 5, 9, 24]] = 1
    bins = oracle.plan(P, mask)
    u = oracle.WindowedUnit(P, bins, 0, 0)
    u.prefill(K[:T], V[:T])
    u.step(K[T], V[T])
    re, im = oracle.compress(K[:T + 1], P, bins)
    assert np.abs(u.CK[0] - re).max() < 1e-11 and np.abs(u.CK[1] - im).max() < 1e-11
    q = rng.standard_normal((G, d))
    vre, vim = oracle.compress(V[:T + 1], P, bins)
    want = oracle.decode_attn(q, re, im, vre, vim, P, bins, T + 1, 0.25)
    assert np.abs(u.attention(q, 0.25) - want).max() < 1e-12


def test_windowed_folds_the_token_that_leaves_the_window(oracle):
    """After steps the transformed segment is exactly the DFT of tokens [S, t - R) at positions n - S
    (Eq. 10 and Eq. 12 agree), and the window holds the last R tokens in order."""
    P, T, d, S, R, steps = 32, 20, 4, 2, 3, 7
    rng = np.random.default_rng(11)
    K, V = rng.standard_normal((T + steps, d)), rng.standard_normal((T + steps, d))
    mask = np.zeros(P // 2 + 1, dtype=np.uint8)
    mask[[0, 3, 4, 16]] = 1
    bins = oracle.plan(P, mask)
    u = oracle.WindowedUnit(P, bins, S, R)
    u.prefill(K[:T], V[:T])
    for s in range(steps):
        u.step(K[T + s], V[T + s])
    t = T + steps
    re, im = oracle.compress(K[S:t - R], P, bins)
    assert np.abs(u.CK[0] - re).max() < 1e-11 and np.abs(u.CK[1] - im).max() < 1e-11
    assert np.array_equal(np.stack(u.recentV), V[t - R:t]) and np.array_equal(u.sinkK, K[:S])


@pytest.mark.parametrize("S,R,D", [(3, 5, 4), (0, 4, 3), (2, 0, 5), (0, 0, 2)])
def test_deferred_all_bins_is_full_attention(oracle, S, R, D):
    """Block-deferred fold, every bin retained, sequence shorter than the grid: whatever is folded and
    whatever still waits in the time domain, attention equals textbook attention over all tokens (numpy) at
    every step, across several block folds."""
    P, T, d, G, steps = 64, 27, 8, 2, 14
    rng = np.random.default_rng(100 + S * 10 + R + D)
    K, V = rng.standard_normal((T + steps, d)), rng.standard_normal((T + steps, d))
    bins = oracle.plan(P, np.ones(P // 2 + 1, dtype=np.uint8))
    u = oracle.WindowedUnit(P, bins, S, R, defer=D)
    u.prefill(K[:T], V[:T])
    folds = 0
    for s in range(steps + 1):
        q = rng.standard_normal((G, d))
        got = u.attention(q, 0.3)
        want = _numpy_attention(q, K[:T + s], V[:T + s], 0.3)
        assert np.abs(got - want).max() < 1e-11, (s, np.abs(got - want).max())
        Kh, Vh = u.materialise()                 # Eq. 13 written out: here, the cache itself
        assert np.abs(Kh - K[:T + s]).max() < 1e-11 and np.abs(Vh - V[:T + s]).max() < 1e-11
        assert u.folded % D == 0 and R <= len(u.recentK) < R + D and u.folded + len(u.recentK) + S == u.t
        if s < steps:
            before = u.folded
            u.step(K[T + s], V[T + s])
            folds += u.folded != before
    assert folds >= 2


def test_deferred_meets_the_per_step_fold_at_block_boundaries(oracle):
    """Pruned bins: whenever (t - S - R) is a multiple of D the block form holds the state of the
    per-step form (same coefficients, same window), and the coefficients are the DFT of tokens
    [S, S + folded) (Eq. 10); in between it has folded fewer tokens and holds more of them exactly."""
    P, T, d, S, R, D, steps = 32, 19, 4, 2, 3, 4, 11
    rng = np.random.default_rng(21)
    K, V = rng.standard_normal((T + steps, d)), rng.standard_normal((T + steps, d))
    mask = np.zeros(P // 2 + 1, dtype=np.uint8)
    mask[[0, 2, 7, 16]] = 1
    bins = oracle.plan(P, mask)
    a, b = oracle.WindowedUnit(P, bins, S, R), oracle.WindowedUnit(P, bins, S, R, defer=D)
    a.prefill(K[:T], V[:T])
    b.prefill(K[:T], V[:T])
    hits = 0
    for s in range(steps + 1):
        t = T + s
        assert b.folded == (t - S - R) // D * D
        re, im = oracle.compress(V[S:S + b.folded], P, bins) if b.folded else (0 * b.CV[0], 0 * b.CV[1])
        assert np.abs(b.CV[0] - re).max() < 1e-11 and np.abs(b.CV[1] - im).max() < 1e-11
        assert np.array_equal(np.stack(b.recentK), K[S + b.folded:t])
        if (t - S - R) % D == 0:
            hits += 1
            assert np.abs(a.CK[0] - b.CK[0]).max() < 1e-11 and np.abs(a.CK[1] - b.CK[1]).max() < 1e-11
            assert np.array_equal(np.stack(a.recentV), np.stack(b.recentV))
            q = rng.standard_normal((2, d))
            assert np.abs(a.attention(q) - b.attention(q)).max() < 1e-12
        else:
            assert b.folded < a.folded and len(b.recentK) > R
        if s < steps:
            a.step(K[t], V[t])
            b.step(K[t], V[t])
    assert hits >= 3


# ----------------------------------------------------------------------------- ablation and selection
def test_chunk_ranges_partition_the_grid(oracle):
    for P, C in [(64, 22), (100, 7), (2048, 22), (22, 22)]:
        edges = [oracle.chunk_range(P, C, c) for c in range(C)]
        assert edges[0][0] == 0 and edges[-1][1] == P
        assert all(edges[i][1] == edges[i + 1][0] for i in range(C - 1))
        assert all(hi - lo == P // C for lo, hi in edges[:-1]) and edges[-1][1] - edges[-1][0] >= P // C


@pytest.mark.parametrize("P,T,lo,hi", [(64, 64, 5, 9), (64, 64, 0, 3), (64, 64, 30, 35), (64, 64, 58, 64),
                                       (96, 70, 40, 56), (33, 33, 10, 20)])
def test_ablation_equals_removing_the_one_sided_components(oracle, P, T, lo, hi):
    """The FFT definition of the ablation (zero two-sided bins, inverse, real part) against a second,
    structurally different evaluation: x minus the gain-weighted reconstruction of the touched one-sided
    bins by the C oracle's loops.  Pins the mirror bookkeeping (gain 1/2 when only one of k, P-k goes)."""
    rng = np.random.default_rng(P + lo)
    x = rng.standard_normal((T, 5))
    want = oracle.ablate(x, P, lo, hi)
    mask, gain = oracle.ablation_bins(P, lo, hi)
    bins = oracle.plan(P, mask)
    re, im = oracle.compress(x, P, bins)
    g = gain[bins].astype(np.float64)[:, None]
    removed = oracle.reconstruct(re * g, im * g, P, bins, T)
    assert np.abs((x - removed) - want).max() < 1e-12
    # a range that is its own mirror image removes whole conjugate pairs: the energy drops by exactly
    # their share (Parseval), and the gains are all 1
    if T == P and lo + (hi - 1) == P:
        X = np.fft.fft(x, axis=0)
        drop = (np.abs(X[lo:hi]) ** 2).sum() / P
        assert abs(((x ** 2).sum() - (want ** 2).sum()) - drop) < 1e-9
        assert (gain[bins] == 1.0).all()
    else:
        assert (gain[bins] == 0.5).any()


def test_greedy_selection_rules(oracle):
    P, C = 220, 22
    delta = np.arange(C, dtype=np.float64)
    delta[[3, 7]] = 100.0                      # a tie at the top: chunk 3 before chunk 7
    mask, n_keep = oracle.mask_from_scores(P, C, delta, 0.125)          # 2.75 -> 3 chunks
    assert n_keep == 3
    kept2 = np.zeros(P, dtype=np.uint8)
    for c in (3, 7, 21):
        lo, hi = oracle.chunk_range(P, C, c)
        kept2[lo:hi] = 1
    assert mask.tobytes() == oracle.fold_two_sided(P, kept2).tobytes()
    assert oracle.mask_from_scores(P, C, delta, 0.001)[1] == 1          # never fewer than one chunk
    assert oracle.mask_from_scores(P, C, delta, 0.0682)[1] == 2         # 1.5004 rounds half up
    m1, _ = oracle.mask_from_scores(P, C, np.zeros(C), 0.094)           # all tied: the lowest chunks win
    lo, hi = oracle.chunk_range(P, C, 0)
    assert m1[lo:hi].all() and m1[0] == 1
