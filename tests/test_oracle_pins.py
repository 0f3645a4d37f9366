"""Pins for the CPU checker: closed forms, invariants, library routines and brute
force on tiny cases.  Each test is chosen so that a plausible slip in the checker
(a dropped term, a wrong sign or index, a swapped wall) fails it.  No GPU needed."""
import itertools
import os

import numpy as np
import pytest

import oracle

FS, C = 16000.0, 343.0
GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ step 1: RIR
def test_rir_single_image_closed_form():
    # d = 3.43 m  =>  tau = 160 samples exactly: h = delta[n-160] / d
    room, mic = [10.0, 8.0, 4.0], [2.0, 3.0, 1.5]
    src = [2.0 + 3.43, 3.0, 1.5]
    h = oracle.rir_image_method(room, [0.7] * 6, mic, src, 0, 1024)
    assert np.argmax(np.abs(h)) == 160
    assert h[160] == pytest.approx(1.0 / 3.43, rel=1e-12)
    h[160] = 0.0
    assert np.max(np.abs(h)) < 1e-12


def test_rir_zero_reflection_gives_direct_path_for_any_order():
    room, mic, src = [5.0, 4.0, 3.0], [1.0, 1.2, 1.1], [3.3, 2.9, 1.7]
    h0 = oracle.rir_image_method(room, [0.9] * 6, mic, src, 0, 2048)
    h5 = oracle.rir_image_method(room, [0.0] * 6, mic, src, 5, 2048)
    np.testing.assert_allclose(h5, h0, atol=1e-15)


@pytest.mark.parametrize("order", [0, 1, 2, 6, 10, 20])
def test_rir_image_count(order):
    room, mic, src = [5.0, 4.0, 3.0], [1.0, 1.2, 1.1], [3.3, 2.9, 1.7]
    _, n = oracle.rir_image_method(room, [0.5] * 6, mic, src, order, 64, return_count=True)
    assert n == (2 * order + 1) * (2 * order * order + 2 * order + 3) // 3


@pytest.mark.parametrize("order", [0, 1, 3])
def test_rir_cube_lattice_count_and_mirror_construction(order):
    room, mic, src = [3.1, 2.7, 2.4], [1.0, 1.3, 1.1], [2.2, 0.9, 1.6]
    beta = [0.9, 0.5, 0.8, 0.4, 0.7, 0.3]
    L = 2048
    h, n = oracle.rir_image_method(room, beta, mic, src, order, L, return_count=True, lattice="cube")
    assert n == (2 * order + 1) ** 3
    imgs = _mirror_images(room, beta, src, order, cube=True)
    assert len(imgs) == n
    f = np.array([50.0, 230.0, 700.0, 1500.0, 2900.0])
    k = np.arange(L)
    H = np.array([np.sum(h * np.exp(-2j * np.pi * fi / FS * k)) for fi in f])
    ref = np.zeros_like(H)
    scale = 0.0
    for pos, g in imgs:
        d = np.linalg.norm(np.array(pos) - np.array(mic))
        if d * FS / C + 40 < L:                          # later images fall outside the buffer
            ref += (g / d) * np.exp(-2j * np.pi * f * d / C)
        scale += g / d
    assert np.max(np.abs(H - ref)) < 2e-3 * scale
    if order:
        total = oracle.rir_image_method(room, beta, mic, src, order, L)
        assert np.max(np.abs(h - total)) > 1e-4          # the cube really holds more images


def _mirror_images(room, beta, src, order, cube=False):
    """All image sources up to `order` reflections, built by composing mirror
    reflections in the real walls (x -> -x at the wall at 0, x -> 2L - x at the wall
    at L), walls alternating along an axis.  Independent of the k = 2m - p indexing."""
    per_axis = []
    for a in range(3):
        opts = [(0, src[a], 1.0)]
        for n in range(1, order + 1):
            for first in (0, 1):
                x, g, wall = src[a], 1.0, first
                for _ in range(n):
                    x = -x if wall == 0 else 2.0 * room[a] - x
                    g *= beta[2 * a + wall]
                    wall ^= 1
                opts.append((n, x, g))
        per_axis.append(opts)
    out = []
    for (nx, x, gx), (ny, y, gy), (nz, z, gz) in itertools.product(*per_axis):
        if cube or nx + ny + nz <= order:
            out.append(((x, y, z), gx * gy * gz))
    return out


@pytest.mark.parametrize("order", [1, 3])
def test_rir_matches_mirror_construction_at_low_frequency(order):
    # Distinct beta on every wall: a swapped wall index changes the answer.
    room, mic, src = [3.1, 2.7, 2.4], [1.0, 1.3, 1.1], [2.2, 0.9, 1.6]
    beta = [0.9, 0.5, 0.8, 0.4, 0.7, 0.3]
    L = 2048
    h = oracle.rir_image_method(room, beta, mic, src, order, L)
    imgs = _mirror_images(room, beta, src, order)
    assert len(imgs) == (2 * order + 1) * (2 * order * order + 2 * order + 3) // 3
    # Below fs/4 a windowed sinc is an ideal delay to ~1e-3, so the frequency
    # response is the closed-form sum of delayed, attenuated paths.
    f = np.array([50.0, 230.0, 700.0, 1500.0, 2900.0])
    n = np.arange(L)
    H = np.array([np.sum(h * np.exp(-2j * np.pi * fi / FS * n)) for fi in f])
    ref = np.zeros_like(H)
    scale = 0.0
    for pos, g in imgs:
        d = np.linalg.norm(np.array(pos) - np.array(mic))
        ref += (g / d) * np.exp(-2j * np.pi * f * d / C)
        scale += g / d
    assert np.max(np.abs(H - ref)) < 2e-3 * scale


def test_rir_reciprocity():
    room, mic, src = [6.0, 4.5, 3.2], [1.1, 2.2, 1.4], [4.7, 0.8, 2.5]
    beta = [0.9, 0.6, 0.8, 0.7, 0.5, 0.85]
    a = oracle.rir_image_method(room, beta, mic, src, 7, 4096)
    b = oracle.rir_image_method(room, beta, src, mic, 7, 4096)
    np.testing.assert_allclose(a, b, atol=1e-13)


def test_fractional_delay_kernel_delays_a_sinusoid():
    # One image at a non-integer delay: filtering a low-frequency cosine must give
    # the same cosine delayed by tau and scaled by 1/d (sign of n - tau matters).
    d = 2.0
    tau = d * FS / C
    assert abs(tau - round(tau)) > 0.2
    h = oracle.rir_image_method([30, 30, 30], [0.0] * 6, [10, 10, 10], [10 + d, 10, 10], 0, 512)
    assert abs(np.sum(h) * d - 1.0) < 1e-3            # DC gain of the interpolator
    f = 437.0
    n = np.arange(4096)
    y = oracle.convolve_causal(np.cos(2 * np.pi * f / FS * n), h)
    ref = np.cos(2 * np.pi * f / FS * (n - tau)) / d
    assert np.max(np.abs(y[600:] - ref[600:])) < 1e-3 / d


def test_delay_kernel_window_shape():
    # One image, delay exactly n0 + 1/2 (d = 343/32000 * (2 n0 + 1), exact in binary for n0 = 100:
    # d = 2.15446875 is not, so the half-sample is checked to 1e-9 instead of assumed).
    n0 = 100
    d = C / FS * (n0 + 0.5)
    room, mic = [30.0, 30.0, 30.0], [10.0, 10.0, 10.0]
    for hw in (40, 41):
        h = oracle.rir_image_method(room, [0.0] * 6, mic, [10.0 + d, 10.0, 10.0], 0, 512,
                                    half_width=hw) * d
        tau = d * FS / C
        assert abs(tau - (n0 + 0.5)) < 1e-9
        # support: 2*hw taps for a half-sample delay, nothing beyond |n - tau| <= hw
        nz = np.nonzero(h)[0]
        assert nz[0] == n0 - hw + 1 and nz[-1] == n0 + hw
        # a Hann window closes smoothly: the outermost taps are tiny but not zero
        for edge in (n0 - hw + 1, n0 + hw):
            assert 1e-9 < abs(h[edge]) < 1e-5
        # the two taps next to the delay: sinc(1/2) = 2/pi, window ~ 1
        assert h[n0] == pytest.approx(2 / np.pi, rel=2e-3) and h[n0 + 1] == pytest.approx(2 / np.pi, rel=2e-3)
        # symmetric about the delay
        np.testing.assert_allclose(h[n0 - hw + 1: n0 + 1], h[n0 + 1: n0 + hw + 1][::-1], rtol=1e-9)
    # half width 41: |n - tau| = 20.5 is half the window, where a Hann window equals 1/2 exactly
    # and sinc(20.5) = 1/(20.5 pi) in magnitude
    assert abs(h[n0 + 21]) == pytest.approx(0.5 / (20.5 * np.pi), rel=1e-9)


def test_two_microphones_on_the_source_axis_differ_by_the_travel_time_of_their_spacing():
    # The far-field set-up of the paper's Section 4 (Fig. 4): source 5 m from a pair of
    # microphones 6.8 cm apart.  Without reflections and with the source on the array
    # axis, the second channel is the first one delayed by 0.068 fs / c = 3.172 samples
    # and weaker by the ratio of the distances.  The delay is read off the phase slope
    # of the response at low frequency, the level off its value near DC.
    room = [12.0, 6.0, 3.0]
    src = [1.0, 3.0, 1.5]
    mics = ([6.0, 3.0, 1.5], [6.068, 3.0, 1.5])
    L = 1024
    k = np.arange(L)
    w1, w2 = 2 * np.pi * 0.040, 2 * np.pi * 0.041          # (w2 - w1) tau = 1.5 < pi: no phase wrap
    tau, level = [], []
    for mic in mics:
        h = oracle.rir_image_method(room, [0.0] * 6, mic, src, 3, L)
        H1, H2 = np.sum(h * np.exp(-1j * w1 * k)), np.sum(h * np.exp(-1j * w2 * k))
        tau.append(-np.angle(H2 / H1) / (w2 - w1))
        level.append(abs(np.sum(h * np.exp(-1j * 2 * np.pi * 0.01 * k))))
    assert tau[0] == pytest.approx(5.0 * FS / C, abs=1e-3)
    assert tau[1] - tau[0] == pytest.approx(0.068 * FS / C, abs=1e-3)        # 3.172 samples
    assert 3.17 < tau[1] - tau[0] < 3.175
    assert level[0] / level[1] == pytest.approx(5.068 / 5.0, rel=1e-4)
    assert level[0] == pytest.approx(1 / 5.0, rel=1e-3)


def test_rir_taps_outside_the_buffer_are_dropped():
    room, mic, src = [5.0, 4.0, 3.0], [1.0, 1.2, 1.1], [3.3, 2.9, 1.7]
    beta = [0.8] * 6
    long = oracle.rir_image_method(room, beta, mic, src, 6, 4096)
    short = oracle.rir_image_method(room, beta, mic, src, 6, 300)
    np.testing.assert_allclose(short, long[:300], atol=1e-15)


# ------------------------------------------------------------------ step 2: reverb + mix
def test_conv_hand_case_from_fixture():
    rows = [np.array(l.split(), dtype=float)
            for l in open(os.path.join(GOLD, "conv_hand_case.txt")) if not l.startswith("#")]
    x, h, y = rows
    np.testing.assert_allclose(oracle.convolve_causal(x, h), y, atol=1e-14)


def test_conv_delta_is_identity_and_shift():
    rng = np.random.default_rng(1)
    x = rng.standard_normal(1000)
    d = np.zeros(64)
    d[0] = 1.0
    np.testing.assert_array_equal(oracle.convolve_causal(x, d), x)
    d[:] = 0
    d[17] = 1.0
    y = oracle.convolve_causal(x, d)
    np.testing.assert_array_equal(y[17:], x[:-17])
    assert not y[:17].any()


@pytest.mark.parametrize("n,l", [(1, 1), (5, 9), (1000, 37), (4099, 4096)])
def test_conv_matches_library(n, l):
    rng = np.random.default_rng(n + l)
    x, h = rng.standard_normal(n), rng.standard_normal(l)
    np.testing.assert_allclose(oracle.convolve_causal(x, h), np.convolve(x, h)[:n],
                               rtol=0, atol=1e-11)


def test_mix_hits_requested_snr_and_ignores_noise_level():
    rng = np.random.default_rng(3)
    n = 6000
    x = rng.standard_normal(n)
    rirs = [rng.standard_normal(50) * np.exp(-np.arange(50) / 10.0) for _ in range(3)]
    nz = [rng.standard_normal(n), rng.standard_normal(n)]
    out, y_s, v, g = oracle.reverb_mix(x, rirs, nz, [1.0, 0.5], 7.5)
    snr = 10 * np.log10(np.sum(y_s ** 2) / np.sum((g * v) ** 2))
    assert snr == pytest.approx(7.5, abs=1e-9)
    np.testing.assert_allclose(out, y_s + g * v)
    out2, *_ = oracle.reverb_mix(x, rirs, nz, [3.0, 1.5], 7.5)   # both weights x3
    np.testing.assert_allclose(out2, out, atol=1e-12)
    # weights really weight: v = conv(n0,h1) + 0.5 conv(n1,h2)
    np.testing.assert_allclose(v, np.convolve(nz[0], rirs[1])[:n] +
                               0.5 * np.convolve(nz[1], rirs[2])[:n], atol=1e-10)


def test_mix_without_noise_or_with_silence():
    x = np.random.default_rng(4).standard_normal(500)
    h = np.array([1.0, 0.5])
    out, y_s, v, g = oracle.reverb_mix(x, [h], [], [], 10.0)
    assert g == 0.0 and not v.any()
    np.testing.assert_array_equal(out, y_s)
    out, y_s, v, g = oracle.reverb_mix(x, [h, h], [np.zeros(500)], [1.0], 10.0)
    assert g == 0.0
    np.testing.assert_array_equal(out, y_s)


def test_looped_noise_wraps():
    bank = np.arange(100.0)
    np.testing.assert_array_equal(oracle.looped_noise(bank, 10, 4, 10),
                                  [10, 11, 12, 13, 10, 11, 12, 13, 10, 11])


# ------------------------------------------------------------------ step 3: STFT power
@pytest.mark.parametrize("n,expect", [(399, 0), (400, 1), (559, 1), (560, 2), (32000, 198),
                                      (320000, 1998), (960000, 5998), (0, 0)])
def test_frame_count_closed_form(n, expect):
    assert oracle.frame_count(n, 400, 160) == expect


@pytest.mark.parametrize("K", [512, 1024])
def test_stft_matches_library_and_parseval(K):
    rng = np.random.default_rng(K)
    x = rng.standard_normal(400 + 160 * 5 + 77)
    P = oracle.stft_power(x, 400, 160, K)
    assert P.shape == (6, K // 2 + 1)
    w = 0.5 - 0.5 * np.cos(2 * np.pi * np.arange(400) / 400)
    for t in range(6):
        fr = w * x[t * 160: t * 160 + 400]
        np.testing.assert_allclose(P[t], np.abs(np.fft.rfft(fr, K)) ** 2, rtol=1e-9, atol=1e-9)
        lhs = P[t, 0] + P[t, K // 2] + 2 * np.sum(P[t, 1:K // 2])
        assert lhs == pytest.approx(K * np.sum(fr ** 2), rel=1e-10)


def test_stft_bin_centred_cosine():
    K, k0, A = 512, 40, 0.3
    n = np.arange(400)
    # a cosine with a whole number of periods in the 400-sample window AND on a bin
    # centre: f = k0/K cycles/sample needs 400 k0 / 512 integer -> k0 = 64 q
    k0 = 64
    x = A * np.cos(2 * np.pi * k0 / K * n)
    P = oracle.stft_power(x, 400, 160, K)
    w = 0.5 - 0.5 * np.cos(2 * np.pi * n / 400)
    assert P[0, k0] == pytest.approx((A * np.sum(w) / 2) ** 2, rel=1e-9)
    assert np.argmax(P[0]) == k0


def test_stft_window_is_periodic_hann():
    # An impulse at sample n0 of the frame has |X[k]|^2 = w[n0]^2 for every k.
    x = np.zeros(400)
    x[100] = 1.0
    P = oracle.stft_power(x, 400, 160, 512)
    np.testing.assert_allclose(P[0], (0.5 - 0.5 * np.cos(2 * np.pi * 100 / 400)) ** 2, rtol=1e-9)
    x[:] = 0
    x[0] = 1.0
    assert np.max(oracle.stft_power(x, 400, 160, 512)) < 1e-25   # w[0] = 0
    x[:] = 0
    x[399] = 1.0     # periodic: w[399] = w[1] != 0 (a symmetric Hann would give 0)
    P = oracle.stft_power(x, 400, 160, 512)
    np.testing.assert_allclose(P[0], (0.5 - 0.5 * np.cos(2 * np.pi / 400)) ** 2, rtol=1e-9)


# ------------------------------------------------------------------ step 4: warp + mel + log
@pytest.mark.parametrize("alpha", [0.7, 0.8, 0.93, 1.0, 1.1, 1.3])
def test_warp_is_the_phase_of_a_first_order_allpass(alpha):
    # Eq. 1 is the phase response of (z - a)/(1 - a z), a = 1 - alpha, on |z| = 1.
    w = np.linspace(0.0, np.pi, 257)
    a = 1.0 - alpha
    z = np.exp(1j * w)
    ref = np.unwrap(np.angle((z - a) / (1.0 - a * z)))
    got = oracle.vtlp_warp(w, alpha)
    np.testing.assert_allclose(got, ref, atol=1e-12)
    assert got[0] == 0.0 and got[-1] == pytest.approx(np.pi, abs=1e-12)
    assert np.all(np.diff(got) > 0)
    if alpha < 1:
        assert np.all(got[1:-1] > w[1:-1])      # alpha < 1 moves content upward
    if alpha == 1.0:
        np.testing.assert_array_equal(got, w)


def test_mel_scale_points_from_fixture():
    # numbers, not the formula again: 700 Hz is 2595 log10(2) mel, 1000 Hz is the
    # scale's anchor (1000 mel to 0.0015 %), 6300 Hz is 2595 mel
    pts = np.loadtxt(os.path.join(GOLD, "mel_scale_points.txt"))
    assert pts.shape == (4, 2)
    np.testing.assert_allclose(oracle.hz_to_mel(pts[:, 0]), pts[:, 1], atol=1e-3)
    # 1000 mel at 1000 Hz is what the constant 2595 was chosen for
    assert abs(float(oracle.hz_to_mel(1000.0)) - 1000.0) < 0.02


def _plain_mel(n_fft, n_mel, fs):
    """Unwarped HTK-style triangles built edge by edge from bin frequencies."""
    f = np.arange(n_fft // 2 + 1) * fs / n_fft
    mel = 2595.0 * np.log10(1.0 + f / 700.0)
    top = 2595.0 * np.log10(1.0 + (fs / 2) / 700.0)
    edges = [top * i / (n_mel + 1) for i in range(n_mel + 2)]
    W = np.zeros((n_mel, f.size))
    for m in range(n_mel):
        lo, mid, hi = edges[m], edges[m + 1], edges[m + 2]
        for k, mu in enumerate(mel):
            if lo < mu <= mid:
                W[m, k] = (mu - lo) / (mid - lo)
            elif mid < mu < hi:
                W[m, k] = (hi - mu) / (hi - mid)
    return W


@pytest.mark.parametrize("K,M", [(512, 40), (512, 80), (1024, 128)])
def test_mel_alpha_one_is_the_unwarped_filterbank(K, M):
    np.testing.assert_allclose(oracle.mel_matrix(1.0, K, M), _plain_mel(K, M, FS), atol=1e-12)


@pytest.mark.parametrize("alpha", [0.8, 0.9, 1.0, 1.15, 1.2])
def test_mel_partition_of_unity(alpha):
    K, M = 512, 40
    W = oracle.mel_matrix(alpha, K, M)
    assert W.min() >= 0 and W.max() <= 1.0
    assert np.all((W > 0).sum(axis=0) <= 2)
    w = 2 * np.pi * np.arange(K // 2 + 1) / K
    mu = oracle.hz_to_mel(oracle.vtlp_warp(w, alpha) * FS / (2 * np.pi))
    e = np.linspace(0, oracle.hz_to_mel(FS / 2), M + 2)
    inside = (mu >= e[1]) & (mu <= e[M])
    np.testing.assert_allclose(W.sum(axis=0)[inside], 1.0, atol=1e-12)
    # hence energy is conserved over those bins
    P = np.random.default_rng(0).random((3, K // 2 + 1))
    P[:, ~inside] = 0
    E = np.exp(oracle.logmel(P, alpha, K, M))
    np.testing.assert_allclose(E.sum(axis=1), P.sum(axis=1), rtol=1e-10)


@pytest.mark.parametrize("alpha", [0.8, 1.0, 1.2])
def test_pure_tone_peaks_in_the_band_of_its_warped_frequency(alpha):
    K, M = 512, 40
    f_tone = 1000.0
    x = np.cos(2 * np.pi * f_tone / FS * np.arange(400 + 160))
    P = oracle.stft_power(x, 400, 160, K)
    E = np.exp(oracle.logmel(P, alpha, K, M))
    f_w = float(oracle.vtlp_warp(2 * np.pi * f_tone / FS, alpha)) * FS / (2 * np.pi)
    e = np.linspace(0, oracle.hz_to_mel(FS / 2), M + 2)
    centre_nearest = int(np.argmin(np.abs(e[1:-1] - oracle.hz_to_mel(f_w))))
    assert int(np.argmax(E[0])) == centre_nearest
    if alpha == 0.8:
        assert f_w > f_tone


def test_log_floor_and_power_law():
    P = np.zeros((2, 257))
    P[1] = 3.0
    lg = oracle.logmel(P, 0.95, 512, 40)
    assert np.all(lg[0] == np.log(1e-10))
    pw = oracle.logmel(P, 0.95, 512, 40, compression="pow15")
    np.testing.assert_allclose(pw, np.exp(lg / 15.0), rtol=1e-12)


# ------------------------------------------------------------------ waveform-domain warp
@pytest.mark.parametrize("alpha", [0.7, 0.85, 1.0, 1.2])
def test_unwarp_undoes_the_warp_of_eq1(alpha):
    w = np.linspace(0.0, np.pi, 301)
    np.testing.assert_allclose(oracle.vtlp_unwarp(oracle.vtlp_warp(w, alpha), alpha), w, atol=1e-12)
    # and it is the phase of the all-pass with the opposite coefficient
    a = -(1.0 - alpha)
    z = np.exp(1j * w)
    np.testing.assert_allclose(oracle.vtlp_unwarp(w, alpha), np.unwrap(np.angle((z - a) / (1.0 - a * z))),
                               atol=1e-12)


@pytest.mark.parametrize("n", [1, 199, 200, 801, 5000])
def test_resynthesis_without_warp_returns_the_input(n):
    x = np.random.default_rng(n).standard_normal(n)
    np.testing.assert_allclose(oracle.vtlp_resynth(x, 1.0), x, atol=1e-12)
    np.testing.assert_allclose(oracle.vtlp_resynth(x, 1.0, win=400, n_fft=512), x, atol=1e-12)


def test_resynthesis_is_linear():
    rng = np.random.default_rng(4)
    x1, x2 = rng.standard_normal(3000), rng.standard_normal(3000)
    lhs = oracle.vtlp_resynth(2.5 * x1 - 0.75 * x2, 0.87)
    rhs = 2.5 * oracle.vtlp_resynth(x1, 0.87) - 0.75 * oracle.vtlp_resynth(x2, 0.87)
    np.testing.assert_allclose(lhs, rhs, atol=1e-12)


@pytest.mark.parametrize("alpha", [0.8, 0.9, 1.1, 1.2])
def test_resynthesis_moves_a_tone_to_the_frequency_eq1_names(alpha):
    # a steady tone comes out near the warped frequency (within four bins of the 1024-point
    # transform: frames no longer add in phase, which smears the line and costs level, the
    # known weakness of warping frame by frame) and on the right side of where it started
    f0 = 1500.0
    y = oracle.vtlp_resynth(np.cos(2 * np.pi * f0 / FS * np.arange(16000)), alpha)
    S = np.abs(np.fft.rfft(y[4000:12192] * np.hanning(8192)))
    f_peak = np.argmax(S) * FS / 8192
    a = 1.0 - alpha
    z = np.exp(2j * np.pi * f0 / FS)
    f_warp = np.angle((z - a) / (1.0 - a * z)) * FS / (2 * np.pi)
    assert abs(f_peak - f_warp) <= 4 * FS / 1024
    assert (f_peak > f0 + 200) == (alpha < 1) and (f_peak < f0 - 200) == (alpha > 1)
    assert 0.2 < np.sqrt(np.mean(y[2000:14000] ** 2)) / np.sqrt(0.5) < 1.0


def test_whole_path_with_the_waveform_warp_leaves_the_filterbank_unwarped():
    from paper_1912_11040_b200 import synth
    x = synth.speech_like(np.random.default_rng(8), 6000)
    row = np.zeros(1, dtype=synth.UTT_DTYPE)[0]
    row["room"], row["mic"], row["src_pos"][0] = (50, 8, 4), (2, 3, 1.5), (2 + 42.875, 3, 1.5)
    row["n_src"], row["order"], row["alpha"], row["snr_db"] = 1, 0, 0.85, 10.0
    cfg = dict(synth._COMMON, rir_taps=4096, max_order=0, vtlp_win=800)
    out = oracle.utterance(x, np.zeros(16), row, cfg)
    xw = oracle.vtlp_resynth(x, float(np.float32(0.85)))      # the table stores the factor in fp32
    np.testing.assert_allclose(out["wave"][2000:], xw[:-2000] / 42.875, atol=1e-13)
    ref = oracle.logmel(oracle.stft_power(out["wave"], 400, 160, 512), 1.0, 512, 40, floor=cfg["log_floor"])
    np.testing.assert_allclose(out["feats"], ref, atol=1e-9)


# ------------------------------------------------------------------ whole path
def test_delta_rir_path_returns_the_input_features():
    # beta = 0 and a source 42.875 m = 343/8 m away (exact in fp32, as the table
    # stores it): tau = 2000 samples exactly, RIR = delta[n-2000]/42.875, no noise.
    from paper_1912_11040_b200 import synth
    rng = np.random.default_rng(5)
    x = synth.speech_like(rng, 8000)
    d, lag = 42.875, 2000
    row = np.zeros(1, dtype=synth.UTT_DTYPE)[0]
    row["room"] = (50, 8, 4)
    row["mic"] = (2, 3, 1.5)
    row["src_pos"][0] = (2 + d, 3, 1.5)
    row["n_src"], row["order"], row["alpha"], row["snr_db"] = 1, 4, 1.0, 10.0
    cfg = dict(synth._COMMON, rir_taps=4096, max_order=4)
    out = oracle.utterance(x, np.zeros(16), row, cfg)
    np.testing.assert_allclose(out["wave"][lag:], x[:-lag] / d, atol=1e-13)
    assert np.max(np.abs(out["wave"][:lag])) < 1e-15
    assert out["frames"] == 1 + (8000 - 400) // 160
    ref = oracle.logmel(oracle.stft_power(np.concatenate([np.zeros(lag), x[:-lag]]) / d,
                                          400, 160, 512), 1.0, 512, 40, floor=cfg["log_floor"])
    np.testing.assert_allclose(out["feats"], ref, atol=1e-9)


# ------------------------------------------------------------------ after the features
def test_mfcc_is_the_orthonormal_dct():
    import scipy.fft
    x = np.random.default_rng(21).standard_normal((7, 40))
    np.testing.assert_allclose(oracle.mfcc(x, 40), scipy.fft.dct(x, type=2, norm="ortho", axis=1),
                               atol=1e-12)
    np.testing.assert_allclose(oracle.mfcc(x, 13), scipy.fft.dct(x, type=2, norm="ortho", axis=1)[:, :13],
                               atol=1e-12)
    c = oracle.mfcc(np.full((1, 40), 2.5), 40)          # a flat spectrum has only c_0 = sqrt(M) x
    assert c[0, 0] == pytest.approx(2.5 * np.sqrt(40)) and np.max(np.abs(c[0, 1:])) < 1e-12
    assert np.sum(oracle.mfcc(x, 40) ** 2) == pytest.approx(np.sum(x ** 2))   # orthonormal


def test_mean_var_closed_forms():
    t = np.arange(101.0)
    x = np.stack([t, np.full(101, 3.0), (-1.0) ** t], axis=1)
    mu, var = oracle.mean_var(x)
    np.testing.assert_allclose(mu, [50.0, 3.0, 1 / 101], atol=1e-12)
    np.testing.assert_allclose(var, [(101 ** 2 - 1) / 12, 0.0, 1 - (1 / 101) ** 2], atol=1e-9)
    mu, var = oracle.mean_var(np.zeros((0, 5)))
    assert not mu.any() and not var.any()
