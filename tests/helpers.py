"""Shared by the GPU parity tests: run a workload through the CUDA library (via the
C ABI binding) and through the CPU checker, and compare."""
import numpy as np

import oracle
from paper_1912_11040_b200 import binding, synth

WAVE_REL_TOL = 1e-4      # max |wave_gpu - wave_cpu| <= 1e-4 * RMS(wave_cpu) + WAVE_ABS_FLOOR
WAVE_ABS_FLOOR = 1e-9    # for (near-)silent outputs: 2e-8 of the 0.05 input level
LOGMEL_ABS_TOL = 2e-3    # max |feat_gpu - feat_cpu|
RIR_REL_TOL = 2e-5       # relative to the largest tap


def oracle_batch(w, compression="log", utts=None):
    idx = range(w.B) if utts is None else utts
    return {b: oracle.utterance(w.speech[b, : w.lengths[b]], w.bank, w.table[b], w.cfg, compression)
            for b in idx}


class Device:
    """A workload resident on the GPU plus a context sized for it."""

    def __init__(self, w, compression=binding.COMPRESS_LOG, host_staging=False):
        import torch
        self.torch = torch
        self.w = w
        cfg = binding.make_config(w.cfg, max(w.B, 1), max(w.stride, 4), compression=compression,
                                  host_staging=host_staging, max_bank_samples=w.bank.size)
        self.cfg = cfg
        self.ctx = binding.AugContext(cfg)
        dev = "cuda"
        self.speech = torch.from_numpy(w.speech).to(dev)
        self.lengths = torch.from_numpy(w.lengths).to(dev)
        self.bank = torch.from_numpy(w.bank).to(dev)
        self.table = binding.table_to_device(w.table, dev)
        self.T_max = max(binding.aug_frame_count(int(w.lengths.max()) if w.B else 0,
                                                 cfg.win, cfg.hop), 1)
        self.S, self.L, self.M, self.nb = cfg.max_sources, cfg.rir_taps, cfg.n_mel, cfg.n_fft // 2 + 1

    def rir(self):
        t = self.torch
        out = t.full((self.w.B, self.S, self.L), float("nan"), device="cuda")
        self.ctx.aug_rir_image_method(self.table, self.w.B, out)
        t.cuda.synchronize()
        return out

    def reverb_mix(self, rir):
        t = self.torch
        out = t.full_like(self.speech, float("nan"))
        self.ctx.aug_reverb_mix(self.speech, self.w.stride, self.lengths, self.bank,
                                self.w.bank.size, rir, self.table, self.w.B, out)
        t.cuda.synchronize()
        return out

    def stft_power(self, wave, stride=None, T_max=None):
        t = self.torch
        T_max = self.T_max if T_max is None else T_max
        P = t.full((self.w.B, T_max, self.nb), float("nan"), device="cuda")
        counts = t.full((self.w.B,), -7, dtype=t.int32, device="cuda")
        self.ctx.feat_stft_power(wave, wave.shape[1] if stride is None else stride, self.lengths,
                                 self.w.B, P, T_max, counts)
        t.cuda.synchronize()
        return P, counts

    def logmel(self, P, counts):
        t = self.torch
        F = t.full((self.w.B, P.shape[1], self.M), float("nan"), device="cuda")
        self.ctx.feat_vtlp_logmel(P, counts, self.table, self.w.B, P.shape[1], F)
        t.cuda.synchronize()
        return F

    def pipeline(self, want_wave=True, T_max=None, lengths_host=True):
        t = self.torch
        T_max = self.T_max if T_max is None else T_max
        F = t.full((self.w.B, T_max, self.M), float("nan"), device="cuda")
        counts = t.full((self.w.B,), -7, dtype=t.int32, device="cuda")
        wave = t.full_like(self.speech, float("nan")) if want_wave else None
        self.ctx.aug_pipeline(self.speech, self.w.stride, self.lengths,
                              self.w.lengths if lengths_host else None, self.bank,
                              self.w.bank.size, self.table, self.w.B, F, T_max, counts, wave)
        t.cuda.synchronize()
        return F, counts, wave


def check_wave(got, ref, what=""):
    rms = float(np.sqrt(np.mean(ref ** 2))) if ref.size else 0.0
    if ref.size == 0:
        return 0.0
    err = float(np.max(np.abs(got.astype(np.float64) - ref)))
    assert err <= WAVE_REL_TOL * rms + WAVE_ABS_FLOOR, f"{what}: wave err {err:.3e} vs rms {rms:.3e}"
    return err / max(rms, 1e-300)


def check_feats(got, ref, what=""):
    if ref.size == 0:
        return 0.0
    err = float(np.max(np.abs(got.astype(np.float64) - ref)))
    assert err <= LOGMEL_ABS_TOL, f"{what}: feature err {err:.3e}"
    return err


def check_pipeline_against_oracle(dev, F, counts, wave, orc, pad_value=0.0):
    """Compare the utterances present in `orc` (dict utt -> oracle output)."""
    w = dev.w
    F = F.cpu().numpy()
    counts = counts.cpu().numpy()
    wave = None if wave is None else wave.cpu().numpy()
    worst_f = worst_w = 0.0
    for b, o in orc.items():
        T = o["frames"]
        assert counts[b] == T, f"utt {b}: frame count {counts[b]} != {T}"
        worst_f = max(worst_f, check_feats(F[b, :T], o["feats"], f"utt {b}"))
        assert np.all(F[b, T:] == pad_value), f"utt {b}: padding rows"
        if wave is not None:
            n = int(w.lengths[b])
            worst_w = max(worst_w, check_wave(wave[b, :n], o["wave"], f"utt {b}"))
    return worst_f, worst_w
