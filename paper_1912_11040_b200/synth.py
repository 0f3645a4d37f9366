"""Seeded synthetic workloads: speech-shaped audio, a noise bank and the
per-utterance parameter table.

This module only *draws inputs*.  It contains none of the arithmetic of the
augmentation / feature path (no image sum, no convolution, no DFT, no mel
filterbank): both the CUDA library and the CPU checker consume what it
returns, byte for byte, so nothing here may depend on either of them.

The five named workloads stand in for the corpora of the paper's Section 4
(LibriSpeech: 960 h over 281 241 utterances, i.e. about 12 s each; the 10 000 h
in-house set), which are not redistributable.  Shapes follow the paper's
description of the simulator in Sections 1 and 2.3: a fresh shoebox room,
reverberation time, source / noise / microphone placement, SNR and VTLP warp
factor per utterance.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, Optional

import numpy as np
from scipy.signal import lfilter

S_MAX = 4  # speech + up to three noise sources per utterance

# One row per utterance.  Field order, sizes and padding are the C struct
# AugUttParams of include/aug_b200.h (160 bytes, 8-byte aligned).
UTT_DTYPE = np.dtype(
    [
        ("room", "<f4", (3,)),          # L_x, L_y, L_z in metres
        ("beta", "<f4", (6,)),          # wall reflection: x=0, x=L_x, y=0, y=L_y, z=0, z=L_z
        ("mic", "<f4", (3,)),
        ("n_src", "<i4"),               # 1 + number of noise sources
        ("order", "<i4"),               # maximum total reflection count
        ("snr_db", "<f4"),
        ("alpha", "<f4"),               # VTLP warp factor
        ("src_pos", "<f4", (S_MAX, 3)),  # row 0 = speech source
        ("noise_offset", "<i8", (S_MAX - 1,)),
        ("noise_len", "<i4", (S_MAX - 1,)),
        ("noise_weight", "<f4", (S_MAX - 1,)),
    ],
    align=True,
)
assert UTT_DTYPE.itemsize == 160

FS = 16000


@dataclasses.dataclass
class Workload:
    """One batch of synthetic input plus the constants of its configuration."""

    name: str
    cfg: Dict[str, float]        # fs, win, hop, n_fft, n_mel, rir_taps, max_order, ...
    lengths: np.ndarray          # int32 [B]
    speech: np.ndarray           # float32 [B][stride], zero beyond lengths[b]
    bank: np.ndarray             # float32 [bank_len]
    table: np.ndarray            # UTT_DTYPE [B]

    @property
    def B(self) -> int:
        return int(self.lengths.shape[0])

    @property
    def stride(self) -> int:
        return int(self.speech.shape[1])

    @property
    def audio_seconds(self) -> float:
        return float(self.lengths.sum()) / self.cfg["fs"]


# --------------------------------------------------------------------------
# waveforms
# --------------------------------------------------------------------------

def _pink(rng: np.random.Generator, n: int) -> np.ndarray:
    """1/f-shaped noise: white noise through octave-spaced one-pole low-passes."""
    acc = np.zeros(n)
    for o in range(8):
        fc = 4000.0 / (2.0 ** o)
        a = np.exp(-2.0 * np.pi * fc / FS)
        acc += lfilter([1.0 - a], [1.0, -a], rng.standard_normal(n)) * (2.0 ** (o / 2.0))
    return acc


def _rms(x: np.ndarray) -> float:
    return float(np.sqrt(np.mean(x * x))) if x.size else 0.0


def speech_like(rng: np.random.Generator, n: int, target_rms: float = 0.05) -> np.ndarray:
    """Harmonic stack (f0 100-250 Hz, +-3 % drift at 0.5 Hz, amplitudes 1/h up to
    3.8 kHz) under a 4 Hz syllabic envelope, plus pink noise 30 dB below it."""
    if n <= 0:
        return np.zeros(0)
    t = np.arange(n) / FS
    f0 = rng.uniform(100.0, 250.0)
    psi = rng.uniform(0.0, 2.0 * np.pi)
    theta = 2.0 * np.pi * f0 * t - (0.03 * f0 / 0.5) * np.cos(2.0 * np.pi * 0.5 * t + psi)
    n_h = int(3800.0 // f0)
    ph = rng.uniform(0.0, 2.0 * np.pi, n_h)
    z = np.exp(1j * theta)
    zh = z.copy()
    acc = np.zeros(n)
    for h in range(1, n_h + 1):
        c, s = np.cos(ph[h - 1]) / h, np.sin(ph[h - 1]) / h
        acc += zh.real * c - zh.imag * s
        zh *= z
    env = 0.5 * (1.0 + np.cos(2.0 * np.pi * 4.0 * t + rng.uniform(0.0, 2.0 * np.pi)))
    voiced = acc * env
    pk = _pink(rng, n)
    r_v, r_p = _rms(voiced), _rms(pk)
    if r_p > 0:
        voiced = voiced + pk * (r_v / r_p) * 10.0 ** (-30.0 / 20.0)
    r = _rms(voiced)
    return voiced * (target_rms / r) if r > 0 else voiced


def noise_like(rng: np.random.Generator, n: int, kind: str, target_rms: float = 0.05) -> np.ndarray:
    if kind == "white":
        x = rng.standard_normal(n)
    elif kind == "pink":
        x = _pink(rng, n)
    elif kind == "babble":
        x = np.zeros(n)
        for _ in range(6):
            x += speech_like(rng, n, 1.0)
    else:
        raise ValueError(kind)
    return x * (target_rms / _rms(x))


# --------------------------------------------------------------------------
# parameter table
# --------------------------------------------------------------------------

def eyring_beta(room: np.ndarray, t60: float) -> float:
    """Wall reflection coefficient giving reverberation time t60 by Eyring's
    formula, the same on all six walls.  (Sabine's inverse exceeds full
    absorption for large rooms at short t60, so it cannot serve here.)"""
    lx, ly, lz = (float(v) for v in room)
    vol = lx * ly * lz
    surf = 2.0 * (lx * ly + ly * lz + lx * lz)
    absorb = 1.0 - np.exp(-0.161 * vol / (surf * t60))
    return float(np.sqrt(1.0 - absorb))


def _place(rng, room, others, margin=0.3, min_dist=0.5):
    for _ in range(1000):
        p = np.array([rng.uniform(margin, room[a] - margin) for a in range(3)])
        if all(np.linalg.norm(p - q) >= min_dist for q in others):
            return p
    raise RuntimeError("could not place a point in the room")


def sample_table(rng, lengths, bank_len, *, room_lo, room_hi, t60, order,
                 n_noise, snr, alpha, min_noise_len=4000, noise_align=4) -> np.ndarray:
    """Draw one table row per utterance.  Ranges are (lo, hi) pairs; a pair with
    lo == hi gives a constant.  Noise stretches start and end on multiples of
    `noise_align` samples (4 = 16 bytes, what a sampler that cares about load width
    hands out; 1 = anywhere)."""
    B = len(lengths)
    tab = np.zeros(B, dtype=UTT_DTYPE)
    for b in range(B):
        room = np.array([rng.uniform(room_lo[a], room_hi[a]) for a in range(3)])
        beta = eyring_beta(room, rng.uniform(*t60))
        mic = _place(rng, room, [])
        k = int(rng.integers(n_noise[0], n_noise[1] + 1))
        pts = [mic]
        row = tab[b]
        row["room"] = room
        row["beta"] = beta
        row["mic"] = mic
        row["n_src"] = 1 + k
        row["order"] = order
        row["snr_db"] = rng.uniform(*snr)
        row["alpha"] = rng.uniform(*alpha)
        for s in range(1 + k):
            p = _place(rng, room, pts[:1])   # only the microphone constrains a source
            row["src_pos"][s] = p
        n = int(lengths[b])
        for j in range(k):
            hi = max(min_noise_len, min(n, bank_len))
            lo = max(min_noise_len, hi // 2)
            ln = int(rng.integers(lo, hi + 1))
            ln = min(ln, bank_len)
            off = int(rng.integers(0, bank_len - ln + 1))
            if noise_align > 1:
                ln = max(noise_align, ln // noise_align * noise_align)
                off = off // noise_align * noise_align
            row["noise_len"][j] = ln
            row["noise_offset"][j] = off
            row["noise_weight"][j] = 1.0
    return tab


def redraw_noise_stretches(table: np.ndarray, lengths: np.ndarray, bank_len: int, seed: int = 0,
                           min_noise_len: int = 4000, noise_align: int = 1) -> np.ndarray:
    """A copy of `table` whose noise stretches are drawn again (same ranges as
    sample_table, own random stream) with offsets and lengths on multiples of
    `noise_align` samples; everything else is kept.  Used to time and check the same
    audio with stretches that start and end anywhere."""
    rng = np.random.default_rng(seed + 7919)
    tab = table.copy()
    for b in range(len(tab)):
        n = int(lengths[b])
        for j in range(int(tab[b]["n_src"]) - 1):
            hi = max(min_noise_len, min(n, bank_len))
            lo = max(min_noise_len, hi // 2)
            ln = min(int(rng.integers(lo, hi + 1)), bank_len)
            off = int(rng.integers(0, bank_len - ln + 1))
            if noise_align > 1:
                ln = max(noise_align, ln // noise_align * noise_align)
                off = off // noise_align * noise_align
            tab[b]["noise_len"][j] = ln
            tab[b]["noise_offset"][j] = off
    return tab


# --------------------------------------------------------------------------
# the five named workloads
# --------------------------------------------------------------------------

_COMMON = dict(fs=FS, win=400, hop=160, n_fft=512, n_mel=40, f_lo=0.0, f_hi=FS / 2.0,
               frac_half_width=40, sound_speed=343.0, log_floor=float(np.finfo(np.float32).eps),
               pad_value=0.0,
               max_sources=S_MAX)

_RECIPES = {
    # B, length range (s), rooms, T60, order, taps, noise count, kinds, SNR, alpha, mel, fft
    1: dict(B=8, dur=(2.0, 2.0), room_lo=(5, 4, 3), room_hi=(5, 4, 3), t60=(0.4, 0.4),
            order=6, taps=4096, n_noise=(1, 1), kinds=("white",), snr=(10, 10),
            alpha=(0.9, 0.9), n_mel=40, n_fft=512),
    2: dict(B=256, dur=(2.0, 20.0), room_lo=(3, 3, 3), room_hi=(10, 10, 10), t60=(0.1, 0.9),
            order=10, taps=8192, n_noise=(1, 2), kinds=("pink", "babble"), snr=(0, 30),
            alpha=(0.8, 1.2), n_mel=40, n_fft=512),
    3: dict(B=128, dur=(8.0, 8.0), room_lo=(3, 3, 2.5), room_hi=(20, 15, 5), t60=(0.3, 1.5),
            order=20, taps=24000, n_noise=(3, 3), kinds=("pink", "babble"), snr=(-5, 20),
            alpha=(0.8, 1.2), n_mel=80, n_fft=512),
    4: dict(B=4096, dur=(1.0, 6.0), room_lo=(3, 3, 3), room_hi=(10, 10, 10), t60=(0.1, 0.9),
            order=8, taps=4096, n_noise=(1, 1), kinds=("pink", "babble"), snr=(5, 25),
            alpha=(0.85, 1.15), n_mel=40, n_fft=512),
    5: dict(B=64, dur=(60.0, 60.0), room_lo=(4, 4, 4), room_hi=(12, 12, 12), t60=(0.3, 1.2),
            order=12, taps=16384, n_noise=(2, 2), kinds=("pink", "babble"), snr=(0, 20),
            alpha=(0.8, 1.2), n_mel=128, n_fft=1024),
}


def make_workload(index: int, seed: int = 0, *, batch: Optional[int] = None,
                  dur_scale: float = 1.0, bank_seconds: Optional[float] = None,
                  taps: Optional[int] = None, order: Optional[int] = None,
                  noise_align: int = 4) -> Workload:
    """Workload `index` (1..5).  `batch`, `dur_scale`, `taps`, `order` shrink a
    workload for checks the slow CPU implementation must finish; the defaults
    are the full sizes."""
    r = dict(_RECIPES[index])
    rng = np.random.default_rng(seed + index)
    B = r["B"] if batch is None else int(batch)
    lo, hi = r["dur"]
    if lo == hi:
        lengths = np.full(B, int(round(lo * dur_scale * FS)), dtype=np.int32)
    else:
        lengths = np.floor(rng.uniform(lo * dur_scale, hi * dur_scale, B) * FS).astype(np.int32)
    n_max = int(lengths.max()) if B else 0
    stride = (n_max + 3) // 4 * 4
    speech = np.zeros((B, stride), dtype=np.float32)
    for b in range(B):
        speech[b, : lengths[b]] = speech_like(rng, int(lengths[b]))

    # A finite pool of noise recordings; every (utterance, source) crops its own
    # stretch of it, shorter than the utterance so that it loops.
    if bank_seconds is None:
        bank_seconds = min(max(2.0 * hi * dur_scale, 4.0), 40.0)
    seg = int(bank_seconds * FS)
    n_seg = 8 if index == 1 else 16
    parts = [noise_like(rng, seg, r["kinds"][i % len(r["kinds"])]) for i in range(n_seg)]
    bank = np.concatenate(parts).astype(np.float32)

    ordr = r["order"] if order is None else int(order)
    table = sample_table(rng, lengths, bank.shape[0], room_lo=r["room_lo"], room_hi=r["room_hi"],
                         t60=r["t60"], order=ordr, n_noise=r["n_noise"], snr=r["snr"],
                         alpha=r["alpha"], noise_align=noise_align)
    cfg = dict(_COMMON)
    # the context is sized for what the workload holds: speech plus its largest noise count
    cfg.update(n_mel=r["n_mel"], n_fft=r["n_fft"], max_order=ordr,
               rir_taps=r["taps"] if taps is None else int(taps),
               max_sources=1 + int(r["n_noise"][1]))
    return Workload(name=f"config{index}", cfg=cfg, lengths=lengths, speech=speech,
                    bank=bank, table=table)
