"""GPU parity: every C-ABI entry point against the fp64 CPU checker, element by
element, on seeded synthetic workloads.  Tolerances (stated once in helpers.py):
frame counts and padding exact; log-mel within 2e-3 absolute; waveforms within
1e-4 of the utterance RMS; impulse responses within 2e-5 of their largest tap."""
import numpy as np
import pytest

import oracle
from paper_1912_11040_b200 import binding, synth
from helpers import (Device, RIR_REL_TOL, check_feats, check_pipeline_against_oracle, check_wave,
                     oracle_batch)

pytestmark = pytest.mark.gpu


def small(index, **kw):
    return synth.make_workload(index, seed=0, **kw)


REDUCED = {
    1: dict(),                                          # config 1 at full size
    2: dict(batch=6, dur_scale=0.15),                   # 2 partitions, 1-2 noises, ragged
    3: dict(batch=3, dur_scale=0.25),                   # 6 partitions, order 20, 3 noises, 80 mel
    4: dict(batch=12, dur_scale=0.5),                   # many short utterances
    5: dict(batch=2, dur_scale=0.06),                   # 4 partitions, 1024-point FFT, 128 mel
}


@pytest.mark.parametrize("index", [1, 2, 3, 4, 5])
def test_rir_matches_image_sum(index):
    w = small(index, **dict(REDUCED[index], batch=min(REDUCED[index].get("batch", 8), 4),
                            dur_scale=0.05))
    dev = Device(w)
    h = dev.rir().cpu().numpy()
    for b in range(w.B):
        row = w.table[b]
        for s in range(dev.S):
            if s >= row["n_src"]:
                assert not h[b, s].any()
                continue
            ref = oracle.rir_image_method(row["room"], row["beta"], row["mic"], row["src_pos"][s],
                                          int(row["order"]), dev.L)
            err = np.max(np.abs(h[b, s] - ref))
            assert err <= RIR_REL_TOL * np.max(np.abs(ref)), (index, b, s, err)


def test_rir_distinct_walls_and_cube_lattice():
    """Six different reflection coefficients (a swapped wall shows) and the cube lattice."""
    w = small(2, batch=4, dur_scale=0.05, order=5)
    rng = np.random.default_rng(3)
    w.table["beta"] = rng.uniform(0.3, 0.95, (w.B, 6)).astype(np.float32)
    for lattice, code in (("total", binding.LATTICE_TOTAL), ("cube", binding.LATTICE_CUBE)):
        cfg = binding.make_config(w.cfg, w.B, w.stride, image_lattice=code)
        ctx = binding.AugContext(cfg)
        import torch
        out = torch.full((w.B, cfg.max_sources, cfg.rir_taps), float("nan"), device="cuda")
        ctx.aug_rir_image_method(binding.table_to_device(w.table), w.B, out)
        torch.cuda.synchronize()
        h = out.cpu().numpy()
        for b in range(w.B):
            row = w.table[b]
            for s in range(int(row["n_src"])):
                ref = oracle.rir_image_method(row["room"], row["beta"], row["mic"], row["src_pos"][s],
                                              int(row["order"]), cfg.rir_taps, lattice=lattice)
                assert np.max(np.abs(h[b, s] - ref)) <= RIR_REL_TOL * np.max(np.abs(ref)), (lattice, b, s)


def test_two_microphone_array_as_paired_rows():
    """The 2-microphone far-field case of the paper's Section 4 (Fig. 4: microphones 6.8 cm
    apart): channel c of utterance u is row 2u + c of the batch, the two rows differing
    only in `mic`.  Both channels are compared with the CPU checker, impulse responses
    and the whole path, and the pair is checked to share everything but the microphone."""
    import torch
    base = small(2, batch=3, dur_scale=0.12)
    B2 = 2 * base.B
    lengths = np.repeat(base.lengths, 2)
    speech = np.repeat(base.speech, 2, axis=0)
    table = np.repeat(base.table, 2)
    for u in range(base.B):
        row = table[2 * u + 1]
        axis = int(np.argmax(row["room"]))              # shift along the longest side: stays inside
        shift = 0.068 if row["mic"][axis] + 0.068 < row["room"][axis] - 0.05 else -0.068
        row["mic"][axis] += shift
    w = synth.Workload(name="two-mic", cfg=dict(base.cfg), lengths=lengths, speech=speech,
                       bank=base.bank, table=table)
    dev = Device(w)
    assert binding.aug_validate_params(dev.cfg, w.table, w.bank.size) == (0, -1)
    for u in range(base.B):
        a, b = w.table[2 * u], w.table[2 * u + 1]
        for f in ("room", "beta", "n_src", "order", "snr_db", "alpha", "src_pos", "noise_offset",
                  "noise_len", "noise_weight"):
            assert np.array_equal(a[f], b[f]), f
        assert np.sum(np.abs(a["mic"] - b["mic"]) > 0) == 1
        assert np.array_equal(w.speech[2 * u], w.speech[2 * u + 1])
    h = dev.rir().cpu().numpy()
    F, counts, wave = dev.pipeline(want_wave=True)
    assert dev.ctx.aug_last_status() == (-1, 0)
    orc = oracle_batch(w)
    for b in range(B2):
        for s in range(int(w.table[b]["n_src"])):
            ref = orc[b]["rirs"][s]
            assert np.max(np.abs(h[b, s] - ref)) <= RIR_REL_TOL * np.max(np.abs(ref)), (b, s)
    check_pipeline_against_oracle(dev, F, counts, wave, orc)
    wv = wave.cpu().numpy()
    for u in range(base.B):
        n = int(w.lengths[2 * u])
        # two channels of one scene: same frame count, strongly correlated, not identical
        assert int(counts[2 * u]) == int(counts[2 * u + 1])
        assert np.max(np.abs(wv[2 * u, :n] - wv[2 * u + 1, :n])) > 1e-4
        assert np.max(np.abs(h[2 * u, 0] - h[2 * u + 1, 0])) > 1e-3 * np.max(np.abs(h[2 * u, 0]))


@pytest.mark.parametrize("dist", [0.05, 1.0, 60.0])
def test_rir_accumulation_scale_follows_the_direct_path(dist):
    """The response is accumulated in fixed point scaled to the direct sound: a source
    5 cm from the microphone (amplitude 20) and one 60 m away (amplitude 0.017) must
    both come out within the same relative tolerance."""
    w = small(2, batch=2, dur_scale=0.05, order=6)
    for b in range(w.B):
        row = w.table[b]
        row["room"] = (80.0, 9.0, 4.0)
        row["beta"] = (0.9, 0.8, 0.85, 0.7, 0.6, 0.75)
        row["mic"] = (5.0, 4.0, 1.5)
        row["n_src"] = 2
        row["src_pos"][0] = (5.0 + dist, 4.0, 1.5)
        row["src_pos"][1] = (5.0 + dist * 0.6, 4.0 + dist * 0.05, 1.5 + min(dist, 2.0) * 0.4)
    dev = Device(w)
    h = dev.rir().cpu().numpy()
    for b in range(w.B):
        row = w.table[b]
        for s in range(2):
            ref = oracle.rir_image_method(row["room"], row["beta"], row["mic"], row["src_pos"][s],
                                          int(row["order"]), dev.L)
            assert np.max(np.abs(ref)) > 0
            assert np.max(np.abs(h[b, s] - ref)) <= RIR_REL_TOL * np.max(np.abs(ref)), (dist, b, s)


def test_rir_closed_form_single_image():
    w = small(1, batch=1, dur_scale=0.05)
    row = w.table[0]
    row["room"], row["mic"], row["src_pos"][0] = (50, 8, 4), (2, 3, 1.5), (2 + 42.875, 3, 1.5)
    row["order"], row["n_src"] = 0, 1
    dev = Device(w)
    h = dev.rir().cpu().numpy()[0, 0]
    assert np.argmax(np.abs(h)) == 2000
    assert h[2000] == pytest.approx(1 / 42.875, rel=1e-6)
    h[2000] = 0
    assert np.max(np.abs(h)) < 1e-8


@pytest.mark.parametrize("index", [1, 2, 3, 5])
def test_reverb_mix_matches_direct_convolution(index):
    w = small(index, **REDUCED[index]) if index != 1 else small(1, batch=3)
    dev = Device(w)
    orc = oracle_batch(w)
    # feed the CPU impulse responses (rounded to fp32) so this test isolates step 2
    rir = np.zeros((w.B, dev.S, dev.L), dtype=np.float32)
    for b, o in orc.items():
        for s, h in enumerate(o["rirs"]):
            rir[b, s] = h
    import torch
    out = dev.reverb_mix(torch.from_numpy(rir).cuda()).cpu().numpy()
    for b, o in orc.items():
        n = int(w.lengths[b])
        # the reference convolves with the same fp32-rounded impulse responses
        rirs32 = [rir[b, s].astype(np.float64) for s in range(int(w.table[b]["n_src"]))]
        noises = [oracle.looped_noise(w.bank, w.table[b]["noise_offset"][k],
                                      w.table[b]["noise_len"][k], n)
                  for k in range(int(w.table[b]["n_src"]) - 1)]
        ref, *_ = oracle.reverb_mix(w.speech[b, :n].astype(np.float64), rirs32, noises,
                                    w.table[b]["noise_weight"], w.table[b]["snr_db"])
        check_wave(out[b, :n], ref, f"cfg{index} utt {b}")
        assert np.all(np.isnan(out[b, n:]))          # samples beyond the length are untouched


@pytest.mark.parametrize("index", [2, 5])
def test_reverb_mix_with_responses_of_any_effective_length(index):
    """The convolution sizes its blocks (fused route) or skips partitions (stored-spectra
    route) by the last non-zero tap of an utterance's responses.  Caller-supplied responses
    that are a single tap at 0, a single tap at the very end of the buffer, dense to the
    last tap, and all zero must all give the plain convolution."""
    import torch
    w = small(index, **dict(REDUCED[index], batch=5))
    w.table["n_src"][:] = 2
    dev = Device(w)
    L = dev.L
    rng = np.random.default_rng(11)
    rir = np.zeros((w.B, dev.S, L), dtype=np.float32)
    rir[0, 0, 0], rir[0, 1, 0] = 0.7, -0.4                       # one tap at 0: effective length 1
    rir[1, 0, L - 1], rir[1, 1, 3] = 0.5, 0.25                   # last tap of the buffer
    rir[2, :2] = rng.standard_normal((2, L)) * np.exp(-np.arange(L) / (0.2 * L)) * 0.05   # dense to the end
    rir[3, 0, : L // 3] = rng.standard_normal(L // 3) * 0.05     # speech response short, noise response long
    rir[3, 1, : L - 7] = rng.standard_normal(L - 7) * 0.05
    # utterance 4: all-zero responses
    out = dev.reverb_mix(torch.from_numpy(rir).cuda()).cpu().numpy()
    for b in range(w.B):
        n = int(w.lengths[b])
        noise = oracle.looped_noise(w.bank, w.table[b]["noise_offset"][0], w.table[b]["noise_len"][0], n)
        ref, *_ = oracle.reverb_mix(w.speech[b, :n].astype(np.float64),
                                    [rir[b, 0].astype(np.float64), rir[b, 1].astype(np.float64)], [noise],
                                    w.table[b]["noise_weight"], w.table[b]["snr_db"])
        check_wave(out[b, :n], ref, f"cfg{index} utt {b}")
    assert not out[4, : int(w.lengths[4])].any()


@pytest.mark.parametrize("index", [1, 5])
def test_stft_power_and_logmel_match(index):
    w = small(index, **REDUCED[index]) if index != 1 else small(1, batch=4)
    w.lengths[0] = 399            # shorter than a window: zero frames
    w.lengths[1] = 400            # exactly one frame
    dev = Device(w)
    P, counts = dev.stft_power(dev.speech)
    F = dev.logmel(P, counts)
    P, counts, F = P.cpu().numpy(), counts.cpu().numpy(), F.cpu().numpy()
    cfg = w.cfg
    for b in range(w.B):
        x = w.speech[b, : w.lengths[b]].astype(np.float64)
        ref = oracle.stft_power(x, cfg["win"], cfg["hop"], cfg["n_fft"])
        T = ref.shape[0]
        assert counts[b] == T == oracle.frame_count(len(x), cfg["win"], cfg["hop"])
        scale = max(ref.max(), 1e-30) if T else 1.0
        assert np.max(np.abs(P[b, :T] - ref), initial=0.0) <= 2e-6 * scale
        assert not P[b, T:].any()
        lm = oracle.logmel(P[b, :T].astype(np.float64), float(w.table[b]["alpha"]), cfg["n_fft"],
                           cfg["n_mel"], floor=cfg["log_floor"])
        check_feats(F[b, :T], lm, f"utt {b}")
        assert np.all(F[b, T:] == cfg["pad_value"])


@pytest.mark.parametrize("index", [1, 2, 3, 4, 5])
def test_pipeline_matches_oracle(index):
    w = small(index, **REDUCED[index])
    dev = Device(w)
    F, counts, wave = dev.pipeline(want_wave=True)
    worst_f, worst_w = check_pipeline_against_oracle(dev, F, counts, wave, oracle_batch(w))
    print(f"config{index} reduced: worst log-mel err {worst_f:.2e}, worst wave err/rms {worst_w:.2e}")


@pytest.mark.parametrize("index", [2, 4, 3])
def test_pipeline_with_unaligned_and_very_short_noise_stretches(index):
    """Noise stretches that start anywhere and have any length (the 128-bit load path
    needs multiples of four samples), down to loops of a few samples."""
    w = small(index, **dict(REDUCED[index], batch=4), noise_align=1)
    tab = w.table
    assert any(int(o) % 4 for o in tab["noise_offset"][:, 0]) or any(int(n) % 4 for n in tab["noise_len"][:, 0])
    tab["noise_offset"][0, 0], tab["noise_len"][0, 0] = 1001, 3        # shorter than one load
    tab["noise_offset"][1, 0], tab["noise_len"][1, 0] = 2002, 1031     # wraps many times per block
    tab["noise_offset"][2, 0], tab["noise_len"][2, 0] = 4000, 4100     # aligned start, unaligned length
    dev = Device(w)
    F, counts, wave = dev.pipeline(want_wave=True)
    assert dev.ctx.aug_last_status() == (-1, 0)
    check_pipeline_against_oracle(dev, F, counts, wave, oracle_batch(w))


def test_fused_route_sums_three_noise_sources():
    """8192 taps, rows with one, two and three noise sources: the products of all but the
    last noise wait in the parking slot and are added before the single inverse transform."""
    w = small(2, batch=3, dur_scale=0.15)
    w.cfg["max_sources"] = 4
    rng = np.random.default_rng(5)
    for b, n_src in enumerate((2, 3, 4)):
        row = w.table[b]
        row["n_src"] = n_src
        for s in range(1, n_src):
            row["src_pos"][s] = [rng.uniform(0.4, float(row["room"][a]) - 0.4) for a in range(3)]
            row["noise_len"][s - 1] = 4000 + 1236 * s
            row["noise_offset"][s - 1] = 2000 * s + 4 * b
            row["noise_weight"][s - 1] = 0.4 + 0.3 * s
    dev = Device(w)
    assert binding.aug_validate_params(dev.cfg, w.table, w.bank.size) == (0, -1)
    F, counts, wave = dev.pipeline(want_wave=True)
    assert dev.ctx.aug_last_status() == (-1, 0)
    check_pipeline_against_oracle(dev, F, counts, wave, oracle_batch(w))
    # a second call finds the slots free again and gives the same answer
    F2, counts2, wave2 = dev.pipeline(want_wave=True)
    orc = oracle_batch(w)
    check_pipeline_against_oracle(dev, F2, counts2, wave2, orc)
    # with every slot held the sources are summed in the time domain: same answer again
    dev.ctx.aug_hold_parking_slots(True)
    F3, counts3, wave3 = dev.pipeline(want_wave=True)
    check_pipeline_against_oracle(dev, F3, counts3, wave3, orc)
    dev.ctx.aug_hold_parking_slots(False)


@pytest.mark.parametrize("n_fft,win,hop", [(512, 512, 200), (512, 400, 125), (1024, 800, 200)])
def test_pipeline_with_other_window_and_hop(n_fft, win, hop):
    """Window and hop are configuration fields: a window as long as the transform with a
    stretch per tile that needs a second round of staging loads, a hop that is not a
    multiple of four samples (scalar staging), and the 50 ms window of the paper's
    Section 3 on the 1024-point transform."""
    w = small(1, batch=3, dur_scale=0.8)
    w.cfg.update(n_fft=n_fft, win=win, hop=hop)
    w.lengths[1] = win + 5 * hop + 3
    w.lengths[2] = win - 1
    dev = Device(w)
    F, counts, wave = dev.pipeline(want_wave=True)
    assert dev.ctx.aug_last_status() == (-1, 0)
    check_pipeline_against_oracle(dev, F, counts, wave, oracle_batch(w))
    assert list(counts.cpu().numpy()[1:]) == [6, 0]
    # steps 3 and 4 on their own, same settings
    P, c2 = dev.stft_power(dev.speech)
    for b in range(w.B):
        x = w.speech[b, : w.lengths[b]].astype(np.float64)
        ref = oracle.stft_power(x, win, hop, n_fft)
        assert int(c2[b]) == ref.shape[0]
        if ref.shape[0]:
            assert np.max(np.abs(P[b, : ref.shape[0]].cpu().numpy() - ref)) <= 2e-6 * ref.max()


def test_pipeline_edge_lengths_and_no_noise():
    w = small(2, batch=8, dur_scale=0.12)
    w.lengths[:6] = [0, 1, 399, 400, 559, 560]
    for b in range(6):
        w.speech[b, w.lengths[b]:] = 0
    w.table["n_src"][6] = 1        # an utterance without noise
    dev = Device(w)
    F, counts, wave = dev.pipeline(want_wave=True, lengths_host=False)
    check_pipeline_against_oracle(dev, F, counts, wave, oracle_batch(w))
    assert list(counts.cpu().numpy()[:6]) == [0, 0, 0, 1, 1, 2]
    # identical result when the host lengths are supplied, and without the waveform output
    F2, counts2, _ = dev.pipeline(want_wave=False, lengths_host=True)
    assert np.array_equal(counts.cpu().numpy(), counts2.cpu().numpy())
    assert np.max(np.abs((F - F2).cpu().numpy())) < 1e-3


@pytest.mark.parametrize("win", [800, 400])
def test_waveform_warp_matches_checker(win):
    """The warp of Eq. 1 applied to the speech waveform with resynthesis: utterances of
    awkward lengths (one sample, just under / at / over a hop and a window, several CTAs'
    worth), warp factors on both sides of 1 and 1 itself (which must return the input)."""
    import torch
    w = small(2, batch=8, dur_scale=0.12)
    w.cfg["vtlp_win"] = win
    hop = win // 4
    w.lengths[:6] = [1, hop - 1, hop, win + 1, 3 * win + 7, 0]
    w.table["alpha"][:8] = [0.8, 1.2, 0.93, 1.07, 1.0, 0.9, 0.85, 1.15]
    dev = Device(w)
    out = torch.full_like(dev.speech, float("nan"))
    dev.ctx.aug_vtlp_resynth(dev.speech, w.stride, dev.lengths, dev.table, w.B, out, w.stride)
    torch.cuda.synchronize()
    out = out.cpu().numpy()
    for b in range(w.B):
        n = int(w.lengths[b])
        ref = oracle.vtlp_resynth(w.speech[b, :n].astype(np.float64), float(w.table[b]["alpha"]), win)
        check_wave(out[b, :n], ref, f"utt {b}")
        assert np.all(np.isnan(out[b, n:]))
    b = 4                                               # alpha = 1: the input comes back
    n = int(w.lengths[b])
    assert np.max(np.abs(out[b, :n] - w.speech[b, :n])) <= 1e-5 * np.sqrt(np.mean(w.speech[b, :n] ** 2))
    # a context without the option refuses the call
    w2 = small(1, batch=1, dur_scale=0.1)
    dev2 = Device(w2)
    o2 = torch.zeros_like(dev2.speech)
    assert dev2.ctx.aug_vtlp_resynth(dev2.speech, w2.stride, dev2.lengths, dev2.table, 1, o2, w2.stride,
                                     check=False) == binding.AUG_EINVAL


def test_pipeline_with_the_waveform_warp():
    """vtlp_win > 0: speech is warped before the simulator (noise and reverberation are
    not), the filterbank stays unwarped; whole path against the checker."""
    w = small(2, **REDUCED[2])
    w.cfg["vtlp_win"] = 800
    dev = Device(w)
    F, counts, wave = dev.pipeline(want_wave=True)
    assert dev.ctx.aug_last_status() == (-1, 0)
    worst_f, worst_w = check_pipeline_against_oracle(dev, F, counts, wave, oracle_batch(w))
    print(f"waveform warp: worst log-mel err {worst_f:.2e}, worst wave err/rms {worst_w:.2e}")
    # and it differs from warping inside the filterbank
    w0 = small(2, **REDUCED[2])
    F0, _, _ = Device(w0).pipeline(want_wave=False)
    assert float((F - F0).abs().max()) > 0.05


def test_power_law_compression():
    w = small(1, batch=2)
    dev = Device(w, compression=binding.COMPRESS_POW_1_15)
    F, counts, _ = dev.pipeline(want_wave=False)
    orc = oracle_batch(w, compression="pow15")
    F = F.cpu().numpy()
    for b, o in orc.items():
        T = o["frames"]
        assert np.max(np.abs(F[b, :T] - o["feats"])) < 2e-3


def test_log_errors_above_tolerance_sit_only_in_bands_below_the_fp32_noise_floor():
    """With the clamp lowered to 1e-10 the log of a band may be off by more than the
    tolerance, but only where the band's true energy is so small that fp32 convolution
    noise (about 1e-7 of the block RMS) reaches it: silent lead-ins before the direct
    sound.  Everything above 1e-8 stays within 2e-3, which is why the default clamp
    is the fp32 epsilon."""
    w = small(3, **REDUCED[3])
    w.cfg["log_floor"] = 1e-10
    dev = Device(w)
    F, counts, _ = dev.pipeline(want_wave=False)
    F, counts = F.cpu().numpy(), counts.cpu().numpy()
    n_checked = 0
    for b, o in oracle_batch(w).items():
        T = o["frames"]
        assert counts[b] == T
        E = np.exp(o["feats"])                      # the checker's band energies (>= 1e-10)
        err = np.abs(F[b, :T] - o["feats"])
        off = err > 2e-3
        assert np.all(E[off] < 1e-8), (b, float(E[off].max()))
        n_checked += int((~off).sum())
    assert n_checked > 0


def test_host_buffer_entry_point_matches_device_one():
    import torch
    w = small(4, batch=5, dur_scale=0.3)
    dev = Device(w, host_staging=True)
    F, counts, _ = dev.pipeline(want_wave=False)
    Fh = np.full((w.B, dev.T_max, dev.M), np.nan, dtype=np.float32)
    ch = np.full(w.B, -1, dtype=np.int32)
    dev.ctx.aug_pipeline_host(w.speech, w.stride, w.lengths, w.bank, w.bank.size,
                              np.ascontiguousarray(w.table), w.B, Fh, dev.T_max, ch)
    assert np.array_equal(ch, counts.cpu().numpy())
    assert np.max(np.abs(Fh - F.cpu().numpy())) < 1e-3


def test_host_entry_point_from_pinned_memory_matches_pageable():
    """Ragged rows of a pinned batch are fetched by a kernel that reads host memory
    directly; pageable memory goes through one copy per row.  Same features either way."""
    import torch
    w = small(2, batch=12, dur_scale=0.5)
    w.lengths[3] = 0
    w.lengths[4] = 1
    dev = Device(w, host_staging=True)
    tab = np.ascontiguousarray(w.table)
    Fp = np.full((w.B, dev.T_max, dev.M), np.nan, dtype=np.float32)
    cp = np.full(w.B, -1, dtype=np.int32)
    dev.ctx.aug_pipeline_host(w.speech, w.stride, w.lengths, w.bank, w.bank.size, tab, w.B, Fp, dev.T_max, cp)
    pin = lambda a: torch.from_numpy(a).pin_memory()
    Fh, ch = torch.full((w.B, dev.T_max, dev.M), float("nan")).pin_memory(), torch.full((w.B,), -1, dtype=torch.int32).pin_memory()
    dev.ctx.aug_pipeline_host(pin(w.speech), w.stride, pin(w.lengths), pin(w.bank), w.bank.size,
                              pin(tab.view(np.uint8).reshape(-1).copy()), w.B, Fh, dev.T_max, ch)
    assert np.array_equal(ch.numpy(), cp)
    assert list(cp[3:5]) == [0, 0]
    assert np.max(np.abs(Fh.numpy() - Fp)) < 1e-3
    F, counts, _ = dev.pipeline(want_wave=False)
    assert np.array_equal(counts.cpu().numpy(), cp) and np.max(np.abs(F.cpu().numpy() - Fp)) < 1e-3


@pytest.mark.parametrize("config,batch,dur_scale", [(2, 12, 0.5), (5, 4, 0.4)])
def test_host_entry_point_valid_rows_only(config, batch, dur_scale):
    """With host_rows = VALID the host call writes the first frame_counts[b] rows of every
    utterance and leaves the rest of the caller's buffer alone, from pinned memory (a kernel
    writes short utterances, the copy engine those with 512 KB of features or more: the
    second case) and from pageable memory (one copy per utterance); the bytes it reports
    are those rows."""
    import torch
    w = small(config, batch=batch, dur_scale=dur_scale)
    w.lengths[1] = 0
    w.lengths[3] = w.lengths[3] // 2 + 1     # (second case: a full utterance followed by a long one, one copy)
    if batch > 4:
        w.lengths[4] = 1
    dev_pad = Device(w, host_staging=True)
    tab = np.ascontiguousarray(w.table)
    Fp = np.full((w.B, dev_pad.T_max, dev_pad.M), np.nan, dtype=np.float32)
    cp = np.full(w.B, -1, dtype=np.int32)
    dev_pad.ctx.aug_pipeline_host(w.speech, w.stride, w.lengths, w.bank, w.bank.size, tab, w.B, Fp,
                                  dev_pad.T_max, cp)
    w.cfg["host_rows"] = 1
    dev = Device(w, host_staging=True)
    pin = lambda a: torch.from_numpy(a).pin_memory()
    SENT = 123.25
    Fh = torch.full((w.B, dev.T_max, dev.M), SENT).pin_memory()
    ch = torch.full((w.B,), -1, dtype=torch.int32).pin_memory()
    dev.ctx.aug_pipeline_host(pin(w.speech), w.stride, pin(w.lengths), pin(w.bank), w.bank.size,
                              pin(tab.view(np.uint8).reshape(-1).copy()), w.B, Fh, dev.T_max, ch)
    Fg = np.full((w.B, dev.T_max, dev.M), SENT, dtype=np.float32)
    cg = np.full(w.B, -1, dtype=np.int32)
    dev.ctx.aug_pipeline_host(w.speech, w.stride, w.lengths, w.bank, w.bank.size, tab, w.B, Fg, dev.T_max, cg)
    for F, c in ((Fh.numpy(), ch.numpy()), (Fg, cg)):
        assert np.array_equal(c, cp)
        for b in range(w.B):
            T = int(cp[b])
            assert np.max(np.abs(F[b, :T] - Fp[b, :T]), initial=0.0) < 1e-3
            assert np.all(F[b, T:] == SENT)
    h2d, d2h = dev.ctx.aug_last_host_bytes()
    assert d2h == 4 * int(cp.sum()) * dev.M + 4 * w.B


def test_host_entry_point_with_an_uploaded_noise_bank():
    """A bank uploaded once serves later calls that pass no bank pointer; results and the
    bytes copied say so; a call with a bank of its own replaces the uploaded one."""
    w = small(2, batch=20, dur_scale=0.1)
    dev = Device(w, host_staging=True)
    args = (w.speech, w.stride, w.lengths)
    tab = np.ascontiguousarray(w.table)
    outs = []
    for use_resident in (False, True, True):
        Fh = np.full((w.B, dev.T_max, dev.M), np.nan, dtype=np.float32)
        ch = np.full(w.B, -1, dtype=np.int32)
        if use_resident and not outs[1:]:
            dev.ctx.aug_upload_noise_bank(w.bank, w.bank.size)
        dev.ctx.aug_pipeline_host(*args, None if use_resident else w.bank, w.bank.size, tab, w.B, Fh,
                                  dev.T_max, ch)
        outs.append((Fh, ch, dev.ctx.aug_last_host_bytes()[0]))
    assert np.array_equal(outs[0][1], outs[1][1]) and np.array_equal(outs[0][1], outs[2][1])
    # (the tolerance of the other host-path comparisons; nothing here needs bit equality)
    assert np.max(np.abs(outs[0][0] - outs[1][0])) < 1e-3 and np.max(np.abs(outs[0][0] - outs[2][0])) < 1e-3
    assert outs[0][2] - outs[1][2] == 4 * w.bank.size
    # without an upload of that length there is nothing to use
    assert dev.ctx.aug_pipeline_host(*args, None, w.bank.size - 4, tab, w.B, outs[0][0].copy(), dev.T_max,
                                     outs[0][1].copy(), check=False) == binding.AUG_EINVAL
    dev.ctx.aug_pipeline_host(*args, w.bank, w.bank.size, tab, w.B, outs[0][0].copy(), dev.T_max,
                              outs[0][1].copy())
    assert dev.ctx.aug_pipeline_host(*args, None, w.bank.size, tab, w.B, outs[0][0].copy(), dev.T_max,
                                     outs[0][1].copy(), check=False) == binding.AUG_EINVAL
    assert dev.ctx.aug_upload_noise_bank(w.bank, w.bank.size + 1, check=False) == binding.AUG_ECAP


def test_errors_and_status_word():
    w = small(1, batch=2, dur_scale=0.1)
    dev = Device(w)
    import torch
    F = torch.zeros((w.B, dev.T_max, dev.M), device="cuda")
    c = torch.zeros(w.B, dtype=torch.int32, device="cuda")
    args = (dev.speech, w.stride, dev.lengths, w.lengths, dev.bank, w.bank.size, dev.table)
    assert dev.ctx.aug_pipeline(*args, w.B + 1, F, dev.T_max, c, check=False) == binding.AUG_ECAP
    assert dev.ctx.aug_pipeline(*args, w.B, None, dev.T_max, c, check=False) == binding.AUG_EINVAL
    assert dev.ctx.aug_pipeline(*args, w.B, F, 1, c, check=False) == binding.AUG_ECAP
    assert dev.ctx.aug_pipeline(dev.speech, w.stride + 1, *args[2:], w.B, F, dev.T_max, c,
                                check=False) == binding.AUG_EINVAL
    # a row the kernels must reject is reported, not faulted on
    bad = w.table.copy()
    bad["n_src"][1] = 9
    tab = binding.table_to_device(bad)
    rir = torch.zeros((w.B, dev.S, dev.L), device="cuda")
    dev.ctx.aug_rir_image_method(tab, w.B, rir)
    assert dev.ctx.aug_last_status() == (1, 1)
    assert dev.ctx.aug_last_status() == (-1, 0)
    assert not rir[1].any()


def test_pipeline_runs_on_a_table_from_the_library_sampler():
    """aug_sample_params rows drive the kernels without a rejected row; results are
    finite and padded.  (Parity inputs never come from the library: those are synth's.)"""
    w = small(2, batch=16, dur_scale=0.1)
    d = binding.AugDist()
    d.room_lo[:] = (3, 3, 2.5)
    d.room_hi[:] = (10, 10, 5)
    d.t60_lo, d.t60_hi, d.order = 0.1, 0.9, int(w.cfg["max_order"])
    d.n_noise_lo, d.n_noise_hi = 0, 3
    d.snr_lo, d.snr_hi, d.alpha_lo, d.alpha_hi = 0, 30, 0.8, 1.2
    d.wall_margin, d.min_src_mic_dist, d.min_noise_len, d.bank_len = 0.3, 0.5, 4000, w.bank.size
    _, w.table = binding.aug_sample_params(123, d, w.lengths)
    w.cfg["max_sources"] = 4           # up to three noise sources per row
    dev = Device(w)
    assert binding.aug_validate_params(dev.cfg, w.table, w.bank.size) == (0, -1)
    F, counts, wave = dev.pipeline(want_wave=True)
    assert dev.ctx.aug_last_status() == (-1, 0)
    F, counts, wave = F.cpu().numpy(), counts.cpu().numpy(), wave.cpu().numpy()
    for b in range(w.B):
        T = binding.aug_frame_count(int(w.lengths[b]), 400, 160)
        assert counts[b] == T
        assert np.all(np.isfinite(F[b, :T])) and np.all(F[b, T:] == 0.0)
        assert np.all(np.isfinite(wave[b, : w.lengths[b]]))
        assert np.sqrt(np.mean(wave[b, : w.lengths[b]] ** 2)) > 1e-5


def test_mfcc_and_mean_var_match():
    import torch
    w = small(5, **REDUCED[5])              # 128 mel bands, 1024-point FFT
    w.lengths[0] = 300                      # an utterance without frames
    dev = Device(w)
    F, counts, _ = dev.pipeline(want_wave=False)
    n_cep = 20
    C = torch.full((w.B, dev.T_max, n_cep), float("nan"), device="cuda")
    dev.ctx.feat_mfcc(F, counts, w.B, dev.T_max, n_cep, C)
    mean = torch.full((w.B, dev.M), float("nan"), device="cuda")
    var = torch.full((w.B, dev.M), float("nan"), device="cuda")
    dev.ctx.feat_mean_var(F, counts, w.B, dev.T_max, dev.M, mean, var)
    torch.cuda.synchronize()
    Fh, Ch, ch = F.cpu().numpy().astype(np.float64), C.cpu().numpy(), counts.cpu().numpy()
    for b in range(w.B):
        T = int(ch[b])
        ref = oracle.mfcc(Fh[b, :T], n_cep)
        assert np.max(np.abs(Ch[b, :T] - ref), initial=0.0) <= 1e-4 * max(1.0, np.max(np.abs(ref), initial=0.0))
        assert np.all(Ch[b, T:] == w.cfg["pad_value"])
        mu, vr = oracle.mean_var(Fh[b, :T])
        np.testing.assert_allclose(mean[b].cpu().numpy(), mu, atol=1e-5 * (1 + np.max(np.abs(mu))))
        np.testing.assert_allclose(var[b].cpu().numpy(), vr, atol=1e-4 * (1 + np.max(np.abs(vr))))
    assert dev.ctx.feat_mfcc(F, counts, w.B, dev.T_max, dev.M + 1, C, check=False) == binding.AUG_EINVAL


def test_empty_batch_is_a_no_op():
    w = small(1, batch=1, dur_scale=0.1)
    dev = Device(w)
    import torch
    F = torch.full((1, dev.T_max, dev.M), 7.0, device="cuda")
    c = torch.full((1,), 7, dtype=torch.int32, device="cuda")
    assert dev.ctx.aug_pipeline(dev.speech, w.stride, dev.lengths, None, dev.bank, w.bank.size,
                                dev.table, 0, F, dev.T_max, c, check=False) == binding.AUG_OK
    torch.cuda.synchronize()
    assert float(F.min()) == 7.0 and int(c[0]) == 7


def test_pipeline_at_the_configuration_limits():
    """Largest reflection order, tap count, delay-kernel width, band count and source
    count a context accepts, on one short utterance."""
    w = small(5, batch=1, dur_scale=1.0 / 60.0, taps=24576, order=32)     # 1 s, 1024-point FFT, 128 mel
    w.cfg["frac_half_width"] = 47
    w.cfg["max_sources"] = 4
    row = w.table[0]
    rng = np.random.default_rng(9)
    row["n_src"] = 4
    row["beta"] = rng.uniform(0.6, 0.97, 6)
    for s in range(1, 4):
        row["src_pos"][s] = [rng.uniform(0.4, float(row["room"][a]) - 0.4) for a in range(3)]
    n = int(w.lengths[0])
    for k in range(3):
        row["noise_len"][k] = 5000 + 1111 * k
        row["noise_offset"][k] = 1000 * (k + 1)
        row["noise_weight"][k] = 0.5 + 0.5 * k
    dev = Device(w)
    assert binding.aug_validate_params(dev.cfg, w.table, w.bank.size) == (0, -1)
    F, counts, wave = dev.pipeline(want_wave=True)
    assert dev.ctx.aug_last_status() == (-1, 0)
    worst_f, worst_w = check_pipeline_against_oracle(dev, F, counts, wave, oracle_batch(w))
    print(f"limits: worst log-mel err {worst_f:.2e}, worst wave err/rms {worst_w:.2e}")
    # one step beyond each limit is refused when the context is created
    for field, value in [("max_order", 33), ("rir_taps", 24577), ("frac_half_width", 48), ("n_mel", 129)]:
        cfg = binding.make_config(dict(w.cfg, **{field: value}), 1, w.stride)
        with pytest.raises(binding.AugError):
            binding.AugContext(cfg)
