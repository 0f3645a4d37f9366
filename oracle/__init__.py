"""TEST INFRASTRUCTURE -- not part of the product.

Slow fp64 CPU definitions of the augmentation + feature path, used only by the
tests, the smoke check and the CPU-baseline timing.  The heavy loops (image
sum, direct convolution, DFT) live in aug_oracle.c; the light steps (energies,
SNR gain, mel matrix, log) are numpy written straight from their formulas.
Nothing here imports, links or shares code with the CUDA library.

Steps and where the paper fixes them:
  rir_image_method   simulator block, Sections 1 / 2.3 (method not printed there:
                     image sources, this library's reading)
  reverb_mix         simulator block, Sections 1 / 2.3 (reverberate, add noise at an SNR)
  stft_power         feature block, Section 2.3
  vtlp_warp          Eq. 1 (bilinear frequency warp), exactly as printed
  vtlp_resynth       the warp of Eq. 1 applied to the speech waveform with resynthesis
                     (Section 2.3; 50 ms window of Section 4): this library's plain
                     reading, fidelity to the authors' resynthesis PARITY UNPINNED
  mel_matrix/logmel  "mel filterbank energies", Section 2.3, with the warp of
                     Eq. 1 applied to the bin frequencies the triangles are
                     evaluated at; natural log (the paper's own power-law
                     (.)^(1/15) is `compression="pow15"`)

Parity status: every function below is pinned by closed forms, invariants and
library routines in tests/test_oracle_*.py.  What stays *unpinned* is fidelity
to the constants of the authors' own simulator and VTLP code, which the paper
defers to cited work.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

from . import build as _build

_lib = None


def _bind(lib):
    dp = ctypes.POINTER(ctypes.c_double)
    lib.orc_rir_image_method.restype = ctypes.c_int64
    lib.orc_rir_image_method.argtypes = [dp, dp, dp, dp, ctypes.c_int, ctypes.c_int, ctypes.c_double,
                                         ctypes.c_double, ctypes.c_int, ctypes.c_int, dp]
    lib.orc_convolve_causal.restype = None
    lib.orc_convolve_causal.argtypes = [dp, ctypes.c_int64, dp, ctypes.c_int64, dp]
    lib.orc_frame_count.restype = ctypes.c_int
    lib.orc_frame_count.argtypes = [ctypes.c_int64, ctypes.c_int, ctypes.c_int]
    lib.orc_stft_power.restype = None
    lib.orc_stft_power.argtypes = [dp, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                   ctypes.c_int, dp]
    return lib


def _load():
    global _lib
    if _lib is None:
        _lib = _bind(ctypes.CDLL(_build.build()))
    return _lib


def _d(a):
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


# ---------------------------------------------------------------- step 1
def rir_image_method(room, beta, mic, src, order, taps, fs=16000.0, c=343.0, half_width=40,
                     return_count=False, lattice="total"):
    """h[taps]: sum over image sources with |kx|+|ky|+|kz| <= order (lattice "total") or
    max(|kx|,|ky|,|kz|) <= order (lattice "cube") of
    (prod beta^hits / d) * Hann-windowed sinc centred at d*fs/c."""
    room, pr = _d(room)
    beta, pb = _d(beta)
    mic, pm = _d(mic)
    src, ps = _d(src)
    h = np.zeros(int(taps), dtype=np.float64)
    assert lattice in ("total", "cube")
    n = _load().orc_rir_image_method(pr, pb, pm, ps, int(order), int(lattice == "cube"), float(fs), float(c),
                                     int(half_width), int(taps),
                                     h.ctypes.data_as(ctypes.POINTER(ctypes.c_double)))
    return (h, int(n)) if return_count else h


# ---------------------------------------------------------------- step 2
def convolve_causal(x, h):
    """y[n] = sum_j h[j] x[n-j] for 0 <= n < len(x): the tail is dropped."""
    x, px = _d(x)
    h, ph = _d(h)
    y = np.zeros_like(x)
    if x.size and h.size:
        _load().orc_convolve_causal(px, x.size, ph, h.size,
                                    y.ctypes.data_as(ctypes.POINTER(ctypes.c_double)))
    return y


def looped_noise(bank, offset, length, n):
    """n samples of bank[offset : offset+length], repeated end to end."""
    idx = int(offset) + (np.arange(int(n), dtype=np.int64) % int(length))
    return np.asarray(bank, dtype=np.float64)[idx]


def snr_gain(y_s, v, snr_db):
    """Gain g on the noise so that mean(y_s^2) / mean((g v)^2) = 10^(snr_db/10);
    0 when either signal is silent."""
    n = max(len(y_s), 1)
    p_s = float(np.sum(y_s * y_s)) / n
    p_v = float(np.sum(v * v)) / n
    if p_s == 0.0 or p_v == 0.0:
        return 0.0
    return float(np.sqrt(p_s / (p_v * 10.0 ** (float(snr_db) / 10.0))))


def reverb_mix(speech, rirs, noises, weights, snr_db):
    """speech [N]; rirs: list, rirs[0] for the speech source, rirs[1+k] for noise k;
    noises: list of [N] arrays (already looped to length N); returns
    (out, y_s, v, g) with out = y_s + g v."""
    y_s = convolve_causal(speech, rirs[0])
    v = np.zeros_like(y_s)
    for k, nz in enumerate(noises):
        v += float(weights[k]) * convolve_causal(nz, rirs[1 + k])
    g = snr_gain(y_s, v, snr_db) if len(noises) else 0.0
    return y_s + g * v, y_s, v, g


# ---------------------------------------------------------------- step 3
def frame_count(n, win, hop):
    return int(_load().orc_frame_count(int(n), int(win), int(hop)))


def stft_power(wave, win, hop, n_fft):
    """P[t][k] = |sum_n hann[n] wave[t hop + n] e^{-2 pi i k n / n_fft}|^2, k = 0..n_fft/2."""
    wave, pw = _d(wave)
    T = frame_count(wave.size, win, hop)
    out = np.zeros((T, n_fft // 2 + 1), dtype=np.float64)
    if T:
        _load().orc_stft_power(pw, wave.size, int(win), int(hop), int(n_fft),
                               out.ctypes.data_as(ctypes.POINTER(ctypes.c_double)))
    return out


# ---------------------------------------------------------------- step 4
def vtlp_warp(omega, alpha):
    """Eq. 1: omega' = omega + 2 atan( (1-alpha) sin(omega) / (1 - (1-alpha) cos(omega)) )."""
    omega = np.asarray(omega, dtype=np.float64)
    a = 1.0 - float(alpha)
    return omega + 2.0 * np.arctan(a * np.sin(omega) / (1.0 - a * np.cos(omega)))


def hz_to_mel(f):
    return 2595.0 * np.log10(1.0 + np.asarray(f, dtype=np.float64) / 700.0)


def mel_matrix(alpha, n_fft, n_mel, fs=16000.0, f_lo=0.0, f_hi=None):
    """[n_mel][n_fft/2+1] triangular weights, linear in mel, peak 1, evaluated at the
    warped frequency of each DFT bin."""
    f_hi = fs / 2.0 if f_hi is None else f_hi
    k = np.arange(n_fft // 2 + 1)
    omega = 2.0 * np.pi * k / n_fft
    f_warp = vtlp_warp(omega, alpha) * fs / (2.0 * np.pi)
    mu = hz_to_mel(f_warp)
    e = np.linspace(hz_to_mel(f_lo), hz_to_mel(f_hi), n_mel + 2)
    W = np.zeros((n_mel, k.size))
    for m in range(n_mel):
        up = (mu - e[m]) / (e[m + 1] - e[m])
        down = (e[m + 2] - mu) / (e[m + 2] - e[m + 1])
        W[m] = np.maximum(0.0, np.minimum(up, down))
    return W


def logmel(power, alpha, n_fft, n_mel, fs=16000.0, f_lo=0.0, f_hi=None, floor=1e-10,
           compression="log"):
    """feat[t][m] = ln(max(sum_k W[m][k] P[t][k], floor)); `pow15` gives E^(1/15)
    (Section 2.3) with the same floor."""
    W = mel_matrix(alpha, n_fft, n_mel, fs, f_lo, f_hi)
    E = np.asarray(power, dtype=np.float64) @ W.T
    E = np.maximum(E, floor)
    if compression == "log":
        return np.log(E)
    if compression == "pow15":
        return E ** (1.0 / 15.0)
    raise ValueError(compression)


# ---------------------------------------------------------------- waveform-domain VTLP
def vtlp_unwarp(omega_out, alpha):
    """The frequency whose content Eq. 1 moves to omega_out: the map of Eq. 1 is the
    phase of a first-order all-pass with coefficient (1 - alpha); the all-pass with
    the opposite coefficient undoes it."""
    omega_out = np.asarray(omega_out, dtype=np.float64)
    a = 1.0 - float(alpha)
    return omega_out - 2.0 * np.arctan(a * np.sin(omega_out) / (1.0 + a * np.cos(omega_out)))


def vtlp_resynth(x, alpha, win=800, n_fft=1024):
    """Speech warped in the waveform domain (Section 2.3, the step before the
    simulator; 50 ms window as in Section 4).  The paper prints only the frequency
    map; this is the plain reading of "warp the spectrum and resynthesise":
      frames of `win` samples every win/4, periodic Hann, the signal zero-padded by
      win - win/4 samples in front so that every sample is covered by four frames;
      DFT of n_fft points; the new spectrum at bin k is the old one at the frequency
      Eq. 1 moves to bin k, taken by linear interpolation between the two nearest bins
      (bins 0 and n_fft/2 stay); inverse DFT, first `win` samples, Hann again,
      overlap-add, division by the summed squared windows.
    Known defect of this reading: neighbouring frames of a steady tone no longer add
    in phase, so the tone loses level.  alpha = 1 returns the input."""
    x = np.asarray(x, dtype=np.float64)
    N = x.size
    hop = win // 4
    front = win - hop
    T = -(-(N + front) // hop) if N else 0
    if T == 0:
        return x.copy()
    padded = np.zeros((T - 1) * hop + win)
    padded[front:front + N] = x
    w = 0.5 - 0.5 * np.cos(2.0 * np.pi * np.arange(win) / win)
    nb = n_fft // 2 + 1
    pos = vtlp_unwarp(2.0 * np.pi * np.arange(nb) / n_fft, alpha) * n_fft / (2.0 * np.pi)
    pos[0], pos[-1] = 0.0, float(nb - 1)
    k0 = np.minimum(np.floor(pos).astype(np.int64), nb - 2)
    fr = pos - k0
    acc = np.zeros_like(padded)
    norm = np.zeros_like(padded)
    for t in range(T):
        seg = padded[t * hop: t * hop + win] * w
        X = np.fft.rfft(seg, n_fft)
        Y = (1.0 - fr) * X[k0] + fr * X[k0 + 1]
        y = np.fft.irfft(Y, n_fft)[:win] * w
        acc[t * hop: t * hop + win] += y
        norm[t * hop: t * hop + win] += w * w
    return acc[front:front + N] / norm[front:front + N]


# ---------------------------------------------------------------- after the features
def mfcc(feats, n_cep):
    """Orthonormal DCT-II of every row: c_i = s_i sum_m x[m] cos(pi i (m + 1/2)/M),
    s_0 = sqrt(1/M), s_i = sqrt(2/M) (the MFCC baseline of Table 1 when x is log-mel)."""
    feats = np.asarray(feats, dtype=np.float64)
    M = feats.shape[-1]
    i = np.arange(int(n_cep))[:, None]
    m = np.arange(M)[None, :]
    C = np.cos(np.pi * i * (m + 0.5) / M) * np.sqrt(2.0 / M)
    C[0] *= np.sqrt(0.5)
    return feats @ C.T


def mean_var(feats):
    """Mean and population variance of each feature over the frames; zeros without frames."""
    feats = np.asarray(feats, dtype=np.float64)
    if feats.shape[0] == 0:
        return np.zeros(feats.shape[1]), np.zeros(feats.shape[1])
    mu = feats.sum(axis=0) / feats.shape[0]
    return mu, ((feats - mu) ** 2).sum(axis=0) / feats.shape[0]


# ---------------------------------------------------------------- whole path
def utterance(speech, bank, row, cfg, compression="log"):
    """One utterance through all four steps.  `row` is one record of the parameter
    table, `cfg` the configuration dictionary.  Returns a dict with rirs, y_s, v, g,
    wave, power, feats (unpadded) and frames."""
    fs = float(cfg["fs"])
    n_src = int(row["n_src"])
    rirs = [rir_image_method(row["room"], row["beta"], row["mic"], row["src_pos"][s],
                             int(row["order"]), int(cfg["rir_taps"]), fs,
                             float(cfg["sound_speed"]), int(cfg["frac_half_width"]),
                             lattice=cfg.get("image_lattice", "total"))
            for s in range(n_src)]
    n = len(speech)
    alpha_fb = float(row["alpha"])
    if int(cfg.get("vtlp_win", 0)) > 0:
        # the warp is applied to the speech waveform before the simulator; the filterbank stays unwarped
        speech = vtlp_resynth(np.asarray(speech, dtype=np.float64), alpha_fb, int(cfg["vtlp_win"]))
        alpha_fb = 1.0
    noises = [looped_noise(bank, row["noise_offset"][k], row["noise_len"][k], n)
              for k in range(n_src - 1)]
    wave, y_s, v, g = reverb_mix(np.asarray(speech, dtype=np.float64), rirs, noises,
                                 row["noise_weight"], row["snr_db"])
    power = stft_power(wave, int(cfg["win"]), int(cfg["hop"]), int(cfg["n_fft"]))
    feats = logmel(power, alpha_fb, int(cfg["n_fft"]), int(cfg["n_mel"]), fs,
                   float(cfg["f_lo"]), float(cfg["f_hi"]), float(cfg["log_floor"]), compression)
    return dict(rirs=rirs, y_s=y_s, v=v, g=g, wave=wave, power=power, feats=feats,
                frames=power.shape[0])
