"""ctypes binding of libaugb200.so: the same entry points as include/aug_b200.h,
argument marshalling only.  Device buffers are torch CUDA tensors (torch is the
allocator and stream owner, nothing more); every step of the path runs in the
library's kernels.  There is no CPU fallback: a missing library raises."""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np

from .synth import S_MAX, UTT_DTYPE

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libaugb200.so")

AUG_OK, AUG_EINVAL, AUG_ECAP, AUG_ECUDA, AUG_EPARAM, AUG_ENOMEM = 0, -1, -2, -3, -4, -5
COMPRESS_LOG, COMPRESS_POW_1_15 = 0, 1
LATTICE_TOTAL, LATTICE_CUBE = 0, 1

EXPORTS = ["aug_strerror", "aug_frame_count", "aug_workspace_bytes", "aug_validate_params",
           "aug_create", "aug_destroy", "aug_last_status", "aug_rir_image_method",
           "aug_reverb_mix", "feat_stft_power", "feat_vtlp_logmel", "aug_pipeline",
           "aug_pipeline_host", "aug_enable_stage_timing", "aug_stage_times", "aug_launch_count",
           "aug_measure_fp32_peak", "feat_vtlp_logmel_noalloc", "aug_last_host_bytes", "aug_upload_noise_bank", "aug_hold_parking_slots", "aug_sample_params", "feat_mfcc", "feat_mean_var",
           "aug_bucket_by_length", "aug_vtlp_resynth"]
NOALLOC_MAX_BATCH = 256
N_STAGES = 7
STAGE_NAMES = ["rir_image", "rir_spectra", "mel_tables", "block_spectra", "convolve", "mix",
               "features"]


class AugConfig(ctypes.Structure):
    _fields_ = [("fs", ctypes.c_int32), ("win", ctypes.c_int32), ("hop", ctypes.c_int32),
                ("n_fft", ctypes.c_int32), ("n_mel", ctypes.c_int32), ("f_lo", ctypes.c_float),
                ("f_hi", ctypes.c_float), ("rir_taps", ctypes.c_int32),
                ("max_order", ctypes.c_int32), ("max_sources", ctypes.c_int32),
                ("frac_half_width", ctypes.c_int32), ("sound_speed", ctypes.c_float),
                ("log_floor", ctypes.c_float), ("pad_value", ctypes.c_float),
                ("compression", ctypes.c_int32), ("max_batch", ctypes.c_int32),
                ("max_samples", ctypes.c_int32), ("host_staging", ctypes.c_int32),
                ("image_lattice", ctypes.c_int32), ("max_bank_samples", ctypes.c_int64),
                ("vtlp_win", ctypes.c_int32), ("host_rows", ctypes.c_int32)]


class AugDist(ctypes.Structure):
    _fields_ = [("room_lo", ctypes.c_float * 3), ("room_hi", ctypes.c_float * 3),
                ("t60_lo", ctypes.c_float), ("t60_hi", ctypes.c_float), ("order", ctypes.c_int32),
                ("n_noise_lo", ctypes.c_int32), ("n_noise_hi", ctypes.c_int32),
                ("snr_lo", ctypes.c_float), ("snr_hi", ctypes.c_float),
                ("alpha_lo", ctypes.c_float), ("alpha_hi", ctypes.c_float),
                ("wall_margin", ctypes.c_float), ("min_src_mic_dist", ctypes.c_float),
                ("min_noise_len", ctypes.c_int32), ("bank_len", ctypes.c_int64)]


class AugError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {strerror(code)} ({code})")


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                               "`python -m paper_1912_11040_b200.build` (nvcc, sm_100a)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64
        L.aug_strerror.restype = ctypes.c_char_p
        L.aug_strerror.argtypes = [i32]
        L.aug_frame_count.restype = i32
        L.aug_frame_count.argtypes = [i32, i32, i32]
        L.aug_workspace_bytes.restype = i64
        L.aug_workspace_bytes.argtypes = [ctypes.POINTER(AugConfig)]
        L.aug_validate_params.restype = i32
        L.aug_validate_params.argtypes = [ctypes.POINTER(AugConfig), vp, i32, i64,
                                          ctypes.POINTER(i32)]
        L.aug_create.restype = i32
        L.aug_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(AugConfig), vp]
        L.aug_destroy.restype = i32
        L.aug_destroy.argtypes = [vp]
        L.aug_last_status.restype = i32
        L.aug_last_status.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(i32)]
        L.aug_vtlp_resynth.restype = i32
        L.aug_vtlp_resynth.argtypes = [vp, vp, i64, vp, vp, i32, vp, i64]
        L.aug_rir_image_method.restype = i32
        L.aug_rir_image_method.argtypes = [vp, vp, i32, vp]
        L.aug_reverb_mix.restype = i32
        L.aug_reverb_mix.argtypes = [vp, vp, i64, vp, vp, i64, vp, vp, i32, vp]
        L.feat_stft_power.restype = i32
        L.feat_stft_power.argtypes = [vp, vp, i64, vp, i32, vp, i32, vp]
        L.feat_vtlp_logmel.restype = i32
        L.feat_vtlp_logmel.argtypes = [vp, vp, vp, vp, i32, i32, vp]
        L.aug_pipeline.restype = i32
        L.aug_pipeline.argtypes = [vp, vp, i64, vp, vp, vp, i64, vp, i32, vp, i32, vp, vp]
        L.aug_pipeline_host.restype = i32
        L.aug_pipeline_host.argtypes = [vp, vp, i64, vp, vp, i64, vp, i32, vp, i32, vp]
        L.feat_vtlp_logmel_noalloc.restype = i32
        L.feat_vtlp_logmel_noalloc.argtypes = [ctypes.POINTER(AugConfig), vp, vp, vp, i32, i32, vp, vp]
        L.aug_enable_stage_timing.restype = i32
        L.aug_enable_stage_timing.argtypes = [vp, i32]
        L.aug_stage_times.restype = i32
        L.aug_stage_times.argtypes = [vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(i32)]
        L.aug_launch_count.restype = i64
        L.aug_launch_count.argtypes = [vp]
        L.feat_mfcc.restype = i32
        L.feat_mfcc.argtypes = [vp, vp, vp, i32, i32, i32, vp]
        L.feat_mean_var.restype = i32
        L.feat_mean_var.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp]
        L.aug_bucket_by_length.restype = i32
        L.aug_bucket_by_length.argtypes = [vp, i32, i32, vp, vp]
        L.aug_sample_params.restype = i32
        L.aug_sample_params.argtypes = [ctypes.c_uint64, ctypes.POINTER(AugDist), i32, vp, vp]
        L.aug_hold_parking_slots.restype = i32
        L.aug_hold_parking_slots.argtypes = [vp, i32]
        L.aug_upload_noise_bank.restype = i32
        L.aug_upload_noise_bank.argtypes = [vp, vp, i64]
        L.aug_last_host_bytes.restype = i32
        L.aug_last_host_bytes.argtypes = [vp, ctypes.POINTER(i64), ctypes.POINTER(i64)]
        L.aug_measure_fp32_peak.restype = i32
        L.aug_measure_fp32_peak.argtypes = [vp, ctypes.POINTER(ctypes.c_float)]
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().aug_strerror(int(code)).decode()


def aug_frame_count(n_samples: int, win: int, hop: int) -> int:
    return int(lib().aug_frame_count(int(n_samples), int(win), int(hop)))


def make_config(cfg: dict, max_batch: int, max_samples: int, *, compression: int = COMPRESS_LOG,
                host_staging: bool = False, max_bank_samples: int = 0,
                image_lattice: int = LATTICE_TOTAL) -> AugConfig:
    return AugConfig(fs=int(cfg["fs"]), win=int(cfg["win"]), hop=int(cfg["hop"]),
                     n_fft=int(cfg["n_fft"]), n_mel=int(cfg["n_mel"]), f_lo=float(cfg["f_lo"]),
                     f_hi=float(cfg["f_hi"]), rir_taps=int(cfg["rir_taps"]),
                     max_order=int(cfg["max_order"]), max_sources=int(cfg["max_sources"]),
                     frac_half_width=int(cfg["frac_half_width"]),
                     sound_speed=float(cfg["sound_speed"]), log_floor=float(cfg["log_floor"]),
                     pad_value=float(cfg["pad_value"]), compression=int(compression),
                     max_batch=int(max_batch), max_samples=int(max_samples),
                     host_staging=int(bool(host_staging)), image_lattice=int(image_lattice),
                     max_bank_samples=int(max_bank_samples), vtlp_win=int(cfg.get("vtlp_win", 0)),
                     host_rows=int(cfg.get("host_rows", 0)))


def aug_workspace_bytes(config: AugConfig) -> int:
    return int(lib().aug_workspace_bytes(ctypes.byref(config)))


def aug_validate_params(config: AugConfig, table: np.ndarray, bank_len: int):
    """Returns (status, first_bad_row)."""
    table = np.ascontiguousarray(table, dtype=UTT_DTYPE)
    bad = ctypes.c_int(-1)
    rc = lib().aug_validate_params(ctypes.byref(config), table.ctypes.data, int(table.shape[0]),
                                   int(bank_len), ctypes.byref(bad))
    return int(rc), int(bad.value)


def aug_sample_params(seed: int, dist: AugDist, lengths: np.ndarray, check: bool = True):
    """Draw one table row per utterance on the host; returns (status, table)."""
    lengths = np.ascontiguousarray(lengths, dtype=np.int32)
    table = np.zeros(lengths.shape[0], dtype=UTT_DTYPE)
    rc = int(lib().aug_sample_params(ctypes.c_uint64(int(seed)), ctypes.byref(dist),
                                     int(lengths.shape[0]), lengths.ctypes.data, table.ctypes.data))
    if check:
        _check(rc, "aug_sample_params")
    return rc, table


def aug_bucket_by_length(lengths: np.ndarray, batch: int):
    """(permutation by increasing length, longest length of each group of `batch`)."""
    lengths = np.ascontiguousarray(lengths, dtype=np.int32)
    B = int(lengths.shape[0])
    perm = np.zeros(B, dtype=np.int32)
    gmax = np.zeros(max(-(-B // int(batch)), 1), dtype=np.int32)
    _check(lib().aug_bucket_by_length(lengths.ctypes.data, B, int(batch), perm.ctypes.data,
                                      gmax.ctypes.data), "aug_bucket_by_length")
    return perm, gmax[: -(-B // int(batch))]


def aug_measure_fp32_peak(stream: Optional[int] = None) -> float:
    """fp32 FMA rate of the current device in TFLOP/s."""
    import torch
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    out = ctypes.c_float(0.0)
    _check(lib().aug_measure_fp32_peak(ctypes.c_void_p(int(stream)), ctypes.byref(out)),
           "aug_measure_fp32_peak")
    return float(out.value)


def feat_vtlp_logmel_noalloc(config: AugConfig, power_dev, counts_dev, table_dev, B: int,
                             T_max: int, feats_dev, stream: Optional[int] = None,
                             check: bool = True) -> int:
    """Step 4 for callers that may not allocate device memory: no context, the
    filterbank tables live in an array built into the library (at most
    NOALLOC_MAX_BATCH utterances per call).  Enqueues on `stream` (default: torch's
    current stream) and returns the status code; raises AugError when `check`."""
    if stream is None:
        import torch
        stream = torch.cuda.current_stream().cuda_stream
    rc = int(lib().feat_vtlp_logmel_noalloc(ctypes.byref(config), _ptr(power_dev),
                                            _ptr(counts_dev), _ptr(table_dev), int(B),
                                            int(T_max), _ptr(feats_dev),
                                            ctypes.c_void_p(int(stream))))
    if check:
        _check(rc, "feat_vtlp_logmel_noalloc")
    return rc


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _check(rc: int, what: str):
    if rc != AUG_OK:
        raise AugError(int(rc), what)


def table_to_device(table: np.ndarray, device="cuda"):
    """The parameter table as a uint8 CUDA tensor [B*160]."""
    import torch
    raw = np.ascontiguousarray(table, dtype=UTT_DTYPE).view(np.uint8).reshape(-1)
    return torch.from_numpy(raw.copy()).to(device)


class AugContext:
    """Owns one AugCtx.  Methods mirror the C entry points and raise AugError on a
    non-zero status; `check=False` returns the status instead."""

    def __init__(self, config: AugConfig, stream: Optional[int] = None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("aug_b200 needs a CUDA device (sm_100a); there is no CPU path")
        self.config = config
        self._h = ctypes.c_void_p(None)
        if stream is None:
            stream = torch.cuda.current_stream().cuda_stream
        self.stream = int(stream)
        rc = lib().aug_create(ctypes.byref(self._h), ctypes.byref(config),
                              ctypes.c_void_p(self.stream))
        _check(rc, "aug_create")

    def close(self):
        if self._h:
            lib().aug_destroy(self._h)
            self._h = ctypes.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _ret(self, rc, what, check):
        if check:
            _check(rc, what)
        return int(rc)

    def aug_last_status(self):
        utt, why = ctypes.c_int(-1), ctypes.c_int(0)
        _check(lib().aug_last_status(self._h, ctypes.byref(utt), ctypes.byref(why)),
               "aug_last_status")
        return int(utt.value), int(why.value)

    def aug_enable_stage_timing(self, on: bool):
        _check(lib().aug_enable_stage_timing(self._h, int(bool(on))), "aug_enable_stage_timing")

    def aug_stage_times(self):
        """(mean ms per stage, number of aug_pipeline calls averaged)."""
        ms = (ctypes.c_float * N_STAGES)()
        n = ctypes.c_int(0)
        _check(lib().aug_stage_times(self._h, ms, ctypes.byref(n)), "aug_stage_times")
        return [float(v) for v in ms], int(n.value)

    def aug_launch_count(self) -> int:
        return int(lib().aug_launch_count(self._h))

    def aug_last_host_bytes(self):
        """(host-to-device, device-to-host) bytes of the last aug_pipeline_host call."""
        a, b = ctypes.c_int64(0), ctypes.c_int64(0)
        _check(lib().aug_last_host_bytes(self._h, ctypes.byref(a), ctypes.byref(b)),
               "aug_last_host_bytes")
        return int(a.value), int(b.value)

    def aug_vtlp_resynth(self, speech_dev, stride, lengths_dev, table_dev, B, warped_dev, out_stride,
                         check=True):
        return self._ret(lib().aug_vtlp_resynth(self._h, _ptr(speech_dev), int(stride), _ptr(lengths_dev),
                                                _ptr(table_dev), int(B), _ptr(warped_dev),
                                                int(out_stride)), "aug_vtlp_resynth", check)

    def aug_rir_image_method(self, table_dev, B, rir_dev, check=True):
        return self._ret(lib().aug_rir_image_method(self._h, _ptr(table_dev), int(B),
                                                    _ptr(rir_dev)), "aug_rir_image_method", check)

    def aug_reverb_mix(self, speech_dev, speech_stride, lengths_dev, bank_dev, bank_len, rir_dev,
                       table_dev, B, wave_out_dev, check=True):
        return self._ret(lib().aug_reverb_mix(self._h, _ptr(speech_dev), int(speech_stride),
                                              _ptr(lengths_dev), _ptr(bank_dev), int(bank_len),
                                              _ptr(rir_dev), _ptr(table_dev), int(B),
                                              _ptr(wave_out_dev)), "aug_reverb_mix", check)

    def feat_stft_power(self, wave_dev, stride, lengths_dev, B, power_dev, T_max, counts_dev,
                        check=True):
        return self._ret(lib().feat_stft_power(self._h, _ptr(wave_dev), int(stride),
                                               _ptr(lengths_dev), int(B), _ptr(power_dev),
                                               int(T_max), _ptr(counts_dev)),
                         "feat_stft_power", check)

    def feat_vtlp_logmel(self, power_dev, counts_dev, table_dev, B, T_max, feats_dev, check=True):
        return self._ret(lib().feat_vtlp_logmel(self._h, _ptr(power_dev), _ptr(counts_dev),
                                                _ptr(table_dev), int(B), int(T_max),
                                                _ptr(feats_dev)), "feat_vtlp_logmel", check)

    def feat_mfcc(self, feats_dev, counts_dev, B, T_max, n_cep, mfcc_dev, check=True):
        return self._ret(lib().feat_mfcc(self._h, _ptr(feats_dev), _ptr(counts_dev), int(B),
                                         int(T_max), int(n_cep), _ptr(mfcc_dev)), "feat_mfcc", check)

    def feat_mean_var(self, feats_dev, counts_dev, B, T_max, D, mean_dev, var_dev, check=True):
        return self._ret(lib().feat_mean_var(self._h, _ptr(feats_dev), _ptr(counts_dev), int(B),
                                             int(T_max), int(D), _ptr(mean_dev), _ptr(var_dev)),
                         "feat_mean_var", check)

    def aug_pipeline(self, speech_dev, speech_stride, lengths_dev, lengths_host, bank_dev,
                     bank_len, table_dev, B, feats_dev, T_max, counts_dev, wave_out_dev=None,
                     check=True):
        lh = None
        if lengths_host is not None:
            lengths_host = np.ascontiguousarray(lengths_host, dtype=np.int32)
            lh = lengths_host.ctypes.data
        return self._ret(lib().aug_pipeline(self._h, _ptr(speech_dev), int(speech_stride),
                                            _ptr(lengths_dev), lh, _ptr(bank_dev), int(bank_len),
                                            _ptr(table_dev), int(B), _ptr(feats_dev), int(T_max),
                                            _ptr(counts_dev), _ptr(wave_out_dev)),
                         "aug_pipeline", check)

    def aug_hold_parking_slots(self, hold):
        _check(lib().aug_hold_parking_slots(self._h, int(bool(hold))), "aug_hold_parking_slots")

    def aug_upload_noise_bank(self, bank_host, bank_len, check=True):
        return self._ret(lib().aug_upload_noise_bank(self._h, _ptr(bank_host), int(bank_len)),
                         "aug_upload_noise_bank", check)

    def aug_pipeline_host(self, speech_host, speech_stride, lengths_host, bank_host, bank_len,
                          table_host, B, feats_host, T_max, counts_host, check=True):
        return self._ret(lib().aug_pipeline_host(self._h, _ptr(speech_host), int(speech_stride),
                                                 _ptr(lengths_host), _ptr(bank_host),
                                                 int(bank_len), _ptr(table_host), int(B),
                                                 _ptr(feats_host), int(T_max), _ptr(counts_host)),
                         "aug_pipeline_host", check)
