"""Do the pins bite?  Each case plants one plausible mistake in a *copy* of the CPU
checker (a swapped wall, a dropped term, a wrong window, an off-by-one) and demands
that at least one pin of tests/test_oracle_pins.py fails on it.  Everything here
runs on the CPU; the real checker is restored after every case."""
import ctypes
import os
import subprocess

import numpy as np
import pytest

import oracle
import test_oracle_pins as pins

SRC = os.path.join(os.path.dirname(oracle.__file__), "aug_oracle.c")

PIN_CALLS = [
    pins.test_rir_single_image_closed_form,
    pins.test_rir_zero_reflection_gives_direct_path_for_any_order,
    lambda: pins.test_rir_image_count(6),
    lambda: pins.test_rir_matches_mirror_construction_at_low_frequency(1),
    lambda: pins.test_rir_matches_mirror_construction_at_low_frequency(3),
    pins.test_rir_reciprocity,
    lambda: pins.test_rir_cube_lattice_count_and_mirror_construction(1),
    pins.test_fractional_delay_kernel_delays_a_sinusoid,
    pins.test_delay_kernel_window_shape,
    pins.test_rir_taps_outside_the_buffer_are_dropped,
    pins.test_two_microphones_on_the_source_axis_differ_by_the_travel_time_of_their_spacing,
    pins.test_conv_hand_case_from_fixture,
    pins.test_conv_delta_is_identity_and_shift,
    lambda: pins.test_conv_matches_library(1000, 37),
    pins.test_mix_hits_requested_snr_and_ignores_noise_level,
    pins.test_mix_without_noise_or_with_silence,
    pins.test_looped_noise_wraps,
    lambda: pins.test_frame_count_closed_form(559, 1),
    lambda: pins.test_frame_count_closed_form(560, 2),
    lambda: pins.test_frame_count_closed_form(399, 0),
    lambda: pins.test_stft_matches_library_and_parseval(512),
    pins.test_stft_bin_centred_cosine,
    pins.test_stft_window_is_periodic_hann,
    lambda: pins.test_warp_is_the_phase_of_a_first_order_allpass(0.8),
    lambda: pins.test_warp_is_the_phase_of_a_first_order_allpass(1.2),
    pins.test_mel_scale_points_from_fixture,
    lambda: pins.test_mel_alpha_one_is_the_unwarped_filterbank(512, 40),
    lambda: pins.test_mel_partition_of_unity(0.9),
    lambda: pins.test_pure_tone_peaks_in_the_band_of_its_warped_frequency(0.8),
    pins.test_log_floor_and_power_law,
    lambda: pins.test_unwarp_undoes_the_warp_of_eq1(0.85),
    lambda: pins.test_resynthesis_without_warp_returns_the_input(801),
    pins.test_resynthesis_is_linear,
    lambda: pins.test_resynthesis_moves_a_tone_to_the_frequency_eq1_names(0.8),
]


def failures():
    n = 0
    for call in PIN_CALLS:
        try:
            call()
        except AssertionError:
            n += 1
    return n


def test_the_unmodified_checker_passes_every_pin():
    assert failures() == 0


C_MUTATIONS = {
    "walls swapped": ("pow(beta[2 * a], abs(m - p)) * pow(beta[2 * a + 1], abs(m))",
                      "pow(beta[2 * a + 1], abs(m - p)) * pow(beta[2 * a], abs(m))"),
    "hit count of the wall at 0": ("abs(m - p)", "abs(m)"),
    "no 1/d": ("double A = gain / d;", "double A = gain;"),
    "image mirrored the wrong way": ("(1 - 2 * p) * src[a] + 2.0 * m * room[a]",
                                     "(1 - 2 * p) * src[a] + 2.0 * (m - p) * room[a]"),
    "delay kernel window too wide": ("cos(M_PI * x / half_w)", "cos(M_PI * x / (half_w + 8))"),
    "delay sign": ("double x = (double)n - tau;", "double x = (double)n + 1.0 - tau;"),
    "L-infinity order": ("if (!cube && abs(kx) + abs(ky) + abs(kz) > order) continue;", ""),
    "cube flag ignored": ("if (!cube && abs(kx)", "if (abs(kx)"),
    "last tap dropped": ("int64_t jmax = n < L - 1 ? n : L - 1;", "int64_t jmax = n < L - 2 ? n : L - 2;"),
    "symmetric Hann": ("0.5 - 0.5 * cos(2.0 * M_PI * n / win)", "0.5 - 0.5 * cos(2.0 * M_PI * n / (win - 1))"),
    "frame count rounds up": ("return (int)(1 + (N - win) / hop);", "return (int)(1 + (N - win + hop - 1) / hop);"),
    "DFT size is the window": ("int j = (int)(((int64_t)k * n) % K);", "int j = (int)(((int64_t)k * n * K / win) % K);"),
    "amplitude spectrum": ("power[(int64_t)t * nb + k] = re * re + im * im;",
                           "power[(int64_t)t * nb + k] = sqrt(re * re + im * im);"),
}


@pytest.mark.parametrize("name", sorted(C_MUTATIONS))
def test_c_mutation_is_caught(name, tmp_path):
    old, new = C_MUTATIONS[name]
    text = open(SRC).read()
    assert text.count(old) == 1, "mutation target must be unique in the source"
    src = tmp_path / "mutant.c"
    src.write_text(text.replace(old, new))
    lib = tmp_path / "mutant.so"
    subprocess.run(["gcc", "-O1", "-fopenmp", "-fPIC", "-shared", "-std=gnu11", "-o", str(lib),
                    str(src), "-lm"], check=True)
    oracle._load()
    real = oracle._lib
    oracle._lib = oracle._bind(ctypes.CDLL(str(lib)))
    try:
        assert failures() >= 1, f"no pin noticed: {name}"
    finally:
        oracle._lib = real


def _mut_warp_sign(omega, alpha):
    omega = np.asarray(omega, dtype=np.float64)
    a = float(alpha) - 1.0                       # (alpha - 1) instead of (1 - alpha)
    return omega + 2.0 * np.arctan(a * np.sin(omega) / (1.0 - a * np.cos(omega)))


def _mut_warp_no_factor_two(omega, alpha):
    omega = np.asarray(omega, dtype=np.float64)
    a = 1.0 - float(alpha)
    return omega + np.arctan(a * np.sin(omega) / (1.0 - a * np.cos(omega)))


def _mut_mel(f):
    # break frequency 1000 Hz instead of 700 Hz (a pure rescaling of the mel axis would be
    # harmless: the edges are equally spaced in mel, so only the curvature matters)
    return 2595.0 * np.log10(1.0 + np.asarray(f, dtype=np.float64) / 1000.0)


def _mut_gain(y_s, v, snr_db):
    n = max(len(y_s), 1)
    p_s, p_v = float(np.sum(y_s * y_s)) / n, float(np.sum(v * v)) / n
    if p_s == 0.0 or p_v == 0.0:
        return 0.0
    return float(np.sqrt(p_s / (p_v * 10.0 ** (float(snr_db) / 20.0))))      # amplitude dB


def _mut_loop(bank, offset, length, n):
    idx = int(offset) + (np.arange(int(n), dtype=np.int64) % (int(length) + 1))
    return np.asarray(bank, dtype=np.float64)[idx]


def _mut_unwarp_wrong_way(omega_out, alpha):
    return oracle.vtlp_warp(omega_out, alpha)          # warps again instead of undoing


def _mut_resynth_no_norm(x, alpha, win=800, n_fft=1024):
    return 1.5 * _REAL_RESYNTH(x, alpha, win, n_fft)   # overlap-add not divided by the window sum


_REAL_RESYNTH = oracle.vtlp_resynth

PY_MUTATIONS = {
    "spectrum moved the wrong way": ("vtlp_unwarp", _mut_unwarp_wrong_way),
    "overlap-add without normalisation": ("vtlp_resynth", _mut_resynth_no_norm),
    "warp direction": ("vtlp_warp", _mut_warp_sign),
    "warp without the factor 2": ("vtlp_warp", _mut_warp_no_factor_two),
    "mel break frequency": ("hz_to_mel", _mut_mel),
    "SNR as amplitude ratio": ("snr_gain", _mut_gain),
    "noise loop one too long": ("looped_noise", _mut_loop),
}


@pytest.mark.parametrize("name", sorted(PY_MUTATIONS))
def test_python_mutation_is_caught(name, monkeypatch):
    attr, fn = PY_MUTATIONS[name]
    monkeypatch.setattr(oracle, attr, fn)
    assert failures() >= 1, f"no pin noticed: {name}"


def test_mel_scale_mutations_are_caught_by_the_numeric_pin_alone(monkeypatch):
    # the other mel tests call oracle.hz_to_mel on both sides or retype its formula;
    # the fixture of hand-worked points must notice a wrong break frequency, a wrong
    # constant and a natural logarithm by itself
    pins.test_mel_scale_points_from_fixture()
    wrong = [_mut_mel,
             lambda f: 1127.0 * np.log10(1.0 + np.asarray(f, dtype=np.float64) / 700.0),
             lambda f: 2595.0 * np.log(1.0 + np.asarray(f, dtype=np.float64) / 700.0),
             lambda f: 2595.0 * np.log10(np.asarray(f, dtype=np.float64) / 700.0 + 1e-300)]
    for fn in wrong:
        monkeypatch.setattr(oracle, "hz_to_mel", fn)
        with pytest.raises(AssertionError):
            pins.test_mel_scale_points_from_fixture()
