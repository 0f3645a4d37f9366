#!/usr/bin/env python
"""Throughput of the augmentation + feature path: audio-seconds per second.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                  [--workload 1..5]

A step is one aug_pipeline call (impulse responses, partition spectra, filterbank
tables, convolution + energies, fused mix/STFT/mel/log) over one batch of
synthetic audio.  `value` is timed with the batch already in HBM; `e2e` times
aug_pipeline_host, which copies the batch from pinned host memory, runs the path
and copies features and frame counts back.  With N > 1 every rank runs an
independent replica of the same job (the path has no exchange step); the ranks
only meet at the barriers around the timed region.

`--impl reference` times the fp64 CPU checker on bounded samples of the same
workload on the host cores.
"""
import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "audio-seconds augmented+featurised per second"
UNIT = "audio-s/s"
FP32_LANES = 128          # fp32 lanes of one multiprocessor

# DRAM bytes per audio-second (dram__bytes_read.sum + dram__bytes_write.sum of one ncu --set full
# capture per kernel on a reduced batch: profiles/ncu_config{2,3,5}_kernels.md; traffic grows in
# proportion to the audio processed).  Valid only for the kernel sources the captures were taken
# from: the hashes guard that.
NCU_TRAFFIC = {
    "bytes_per_audio_s": {
        2: {"convolve": 263.7e6 / 1039.18, "features": 150.9e6 / 1039.18, "rir_image": 45.6e6 / 1039.18},
        3: {"convolve": (79.2e6 + 30.9e6) / 128.0, "rir_image": 32.8e6 / 128.0},
        5: {"convolve": 46.3e6 / 240.0, "features": 34.1e6 / 240.0}},
    "captured_on": {2: "96 utterances", 3: "16 utterances", 5: "4 utterances"},
    # kernel -> (its source files, sha256[:16] of them when the counters were taken)
    "sources": {"convolve": (("conv.cu", "fft.cuh"), "7a79969eb6513345"),
                "features": (("feat.cu", "fft.cuh"), "6b90b8e67ab940e5"),
                "rir_image": (("rir.cu",), "9c178fa666e60507")}}


# nominal FMAs / fp32 instructions executed: convolution 480 / 736 per thread and 4096-point
# transform; fused 512-point features 6274 / 11680 per frame
FP32_INSTRUCTION_CEILING = {"convolve": 0.652, "features": 0.537}


def kernel_sources_sha(files):
    import hashlib
    h = hashlib.sha256()
    for f in files:
        h.update(open(os.path.join(ROOT, "paper_1912_11040_b200", "csrc", f), "rb").read())
    return h.hexdigest()[:16]


def workload_label(i):
    return {1: "config1: 8 x 2 s, order 6, 4096 taps, 1 white noise, 40 mel",
            2: "config2: 256 utts 2-20 s, order 10, 8192 taps, 1-2 noises, 40 mel",
            3: "config3: 128 x 8 s, order 20, 24000 taps, 3 noises, 80 mel",
            4: "config4: 4096 utts 1-6 s, order 8, 4096 taps, 1 noise, 40 mel",
            5: "config5: 64 x 60 s, order 12, 16384 taps, 2 noises, 1024-pt FFT, 128 mel"}[i]


# ------------------------------------------------------------------ algorithmic work
def conv_work(w):
    """Nominal flops and compulsory bytes of the convolution step for one batch (all its
    kernels together).  Per source one forward real FFT per block (2.5 F log2 F), 8 flops per
    bin and partition for the spectral multiply, two inverse FFTs per block (one without
    noise).  The count follows the response length the context is created for: up to 8192
    taps one partition of a 16384-point transform with 16384 - taps + 1 outputs per block
    (cut to a multiple of 4); longer ones in 4096-tap partitions of an 8192-point transform
    with 4096 outputs per block.  (The kernels do less than this when the responses end before
    their buffer does: blocks get longer, zero partitions are skipped and a long-response
    context may take the one-partition route.  The nominal count stays that of the stated
    configuration.)  Bytes: inputs read once, y_s and v written once, response spectra once."""
    taps = int(w.cfg["rir_taps"])
    if taps <= 8192:
        F, P = 16384, 1
        blk = (F - taps + 1) & ~3
    else:
        F, blk = 8192, 4096
        P = -(-taps // blk)
    fft = 2.5 * F * np.log2(F)
    spec = (F // 2) * 8.0
    flops = bytes_ = 0.0
    for b in range(w.B):
        n, S = int(w.lengths[b]), int(w.table["n_src"][b])
        nblk = -(-n // blk)
        flops += nblk * (S * fft + S * 8.0 * (F // 2) * P + (2 if S > 1 else 1) * fft)
        bytes_ += 4.0 * n * S + 4.0 * n * 2 + S * P * spec
    return {"convolve": (flops, bytes_)}


def rir_work(w):
    """Image-method kernel: ~10 flops per tap, 2 W_h + 1 taps per image; bytes = responses out."""
    taps = 2 * int(w.cfg["frac_half_width"]) + 1
    flops = bytes_ = 0.0
    for b in range(w.B):
        n = int(w.table["order"][b])
        images = (2 * n + 1) * (2 * n * n + 2 * n + 3) // 3
        S = int(w.table["n_src"][b])
        flops += 10.0 * taps * images * S
        bytes_ += 4.0 * int(w.cfg["rir_taps"]) * S
    return flops, bytes_


def feat_work(w):
    """Fused mix + STFT + mel kernel: one K-point real FFT per frame plus 4 flops per
    bin; bytes = y_s and v read once + features written once."""
    K, M = int(w.cfg["n_fft"]), int(w.cfg["n_mel"])
    flops = bytes_ = 0.0
    for b in range(w.B):
        n = int(w.lengths[b])
        T = 1 + (n - int(w.cfg["win"])) // int(w.cfg["hop"]) if n >= int(w.cfg["win"]) else 0
        flops += T * (2.5 * K * np.log2(K) + 4.0 * (K // 2 + 1))
        bytes_ += 8.0 * n + 4.0 * T * M
    return flops, bytes_


# ------------------------------------------------------------------ clocks
class ClockSampler:
    def __init__(self, index=0, period=0.002):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None
        self.period = period

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4)}
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._run, daemon=True)
            self._thr.start()

    def stop(self):
        self._stop.set()
        if self._thr is not None:
            self._thr.join()
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ------------------------------------------------------------------ CPU checker timing
def time_oracle(w, budget_s, max_seconds_per_utt=None):
    """Run the CPU checker over utterances of `w` in order until `budget_s` of wall
    time is used (at least one).  Returns (audio-s/s, description, cores)."""
    import oracle
    oracle._load()
    cores = os.cpu_count() or 1
    done_audio = 0.0
    n_utt = 0
    t0 = time.perf_counter()
    for b in range(w.B):
        n = int(w.lengths[b])
        if max_seconds_per_utt is not None:
            n = min(n, int(max_seconds_per_utt * w.cfg["fs"]))
        oracle.utterance(w.speech[b, :n], w.bank, w.table[b], w.cfg)
        done_audio += n / w.cfg["fs"]
        n_utt += 1
        if time.perf_counter() - t0 >= budget_s:
            break
    dt = time.perf_counter() - t0
    return done_audio / dt, f"first {n_utt} utterance(s), {done_audio:.1f} audio-s, {dt:.1f} s wall", cores


# ------------------------------------------------------------------ fast CPU pipeline
# A reasonable CPU implementation of the same four steps (vectorised image sum, FFT
# convolution, rfft STFT, dense mel matrix; numpy/scipy, fp64), one process per core:
# the stand-in for the paper's CPU example servers.  Context for the GPU number only;
# it shares nothing with the CUDA library or the fp64 checker.
_LATTICE = {}


def _fast_lattice(order):
    if order not in _LATTICE:
        k = np.arange(-order, order + 1)
        kx, ky, kz = np.meshgrid(k, k, k, indexing="ij")
        keep = (np.abs(kx) + np.abs(ky) + np.abs(kz)) <= order
        _LATTICE[order] = np.stack([kx[keep], ky[keep], kz[keep]], axis=1)
    return _LATTICE[order]


def _fast_rir(row, s, cfg):
    L, hw, fs, c = int(cfg["rir_taps"]), int(cfg["frac_half_width"]), float(cfg["fs"]), float(cfg["sound_speed"])
    k = _fast_lattice(int(row["order"]))
    p = k & 1
    m = (k + p) // 2
    room, src, mic = (np.asarray(row[n], dtype=np.float64) for n in ("room", "src_pos", "mic"))
    img = (1 - 2 * p) * src[s] + 2.0 * m * room
    d = np.sqrt(((img - mic) ** 2).sum(axis=1))
    beta = np.asarray(row["beta"], dtype=np.float64)
    gain = np.prod(beta[0::2] ** np.abs(m - p) * beta[1::2] ** np.abs(m), axis=1)
    tau = d * fs / c
    n0 = np.rint(tau).astype(np.int64)
    idx = n0[:, None] + np.arange(-hw, hw + 1)[None, :]
    x = idx - tau[:, None]
    val = (gain / d)[:, None] * np.sinc(x) * 0.5 * (1.0 + np.cos(np.pi * x / hw))
    ok = (idx >= 0) & (idx < L) & (np.abs(x) <= hw)
    return np.bincount(idx[ok], weights=val[ok], minlength=L)[:L]


def _fast_mel(alpha, cfg):
    K, M, fs = int(cfg["n_fft"]), int(cfg["n_mel"]), float(cfg["fs"])
    w = 2.0 * np.pi * np.arange(K // 2 + 1) / K
    a = 1.0 - float(alpha)
    fw = (w + 2.0 * np.arctan(a * np.sin(w) / (1.0 - a * np.cos(w)))) * fs / (2.0 * np.pi)
    mel = lambda f: 2595.0 * np.log10(1.0 + f / 700.0)
    e = np.linspace(mel(float(cfg["f_lo"])), mel(float(cfg["f_hi"])), M + 2)
    mu = mel(fw)[None, :]
    up = (mu - e[:-2, None]) / (e[1:-1, None] - e[:-2, None])
    dn = (e[2:, None] - mu) / (e[2:, None] - e[1:-1, None])
    return np.maximum(0.0, np.minimum(up, dn))


def fast_cpu_utterance(speech, bank, row, cfg):
    """Log-mel features [T][M] of one utterance, fp64 numpy/scipy."""
    from scipy.signal import fftconvolve
    n = len(speech)
    ys = fftconvolve(np.asarray(speech, dtype=np.float64), _fast_rir(row, 0, cfg))[:n]
    out = ys
    if int(row["n_src"]) > 1:
        v = np.zeros(n)
        for j in range(int(row["n_src"]) - 1):
            seg = np.asarray(bank[int(row["noise_offset"][j]): int(row["noise_offset"][j]) + int(row["noise_len"][j])],
                             dtype=np.float64)
            v += float(row["noise_weight"][j]) * fftconvolve(np.resize(seg, n), _fast_rir(row, 1 + j, cfg))[:n]
        es, ev = float(ys @ ys), float(v @ v)
        if es > 0 and ev > 0:
            out = ys + np.sqrt(es / (ev * 10.0 ** (float(row["snr_db"]) / 10.0))) * v
    W, H, K = int(cfg["win"]), int(cfg["hop"]), int(cfg["n_fft"])
    if n < W:
        return np.zeros((0, int(cfg["n_mel"])))
    T = 1 + (n - W) // H
    frames = np.lib.stride_tricks.as_strided(out, (T, W), (out.strides[0] * H, out.strides[0]))
    P = np.abs(np.fft.rfft(frames * (0.5 - 0.5 * np.cos(2.0 * np.pi * np.arange(W) / W)), K, axis=1)) ** 2
    return np.log(np.maximum(P @ _fast_mel(row["alpha"], cfg).T, float(cfg["log_floor"])))


def _fast_worker(job):
    speech_rows, lengths, bank, table, cfg = job
    t0 = time.perf_counter()
    for b in range(len(lengths)):
        fast_cpu_utterance(speech_rows[b][: lengths[b]], bank, table[b], cfg)
    return float(sum(lengths)) / cfg["fs"], time.perf_counter() - t0


def time_fast_cpu(w, n_utts):
    """The first n_utts utterances through fast_cpu_utterance, spread over all cores
    (spawned workers).  Returns (audio-s/s, description, workers)."""
    import multiprocessing as mp
    workers = max(1, min(os.cpu_count() or 1, n_utts))
    n_utts = min(n_utts, w.B)
    jobs = []
    for k in range(workers):
        sel = list(range(k, n_utts, workers))
        if sel:
            jobs.append(([w.speech[b, : w.lengths[b]].copy() for b in sel], [int(w.lengths[b]) for b in sel],
                         w.bank, w.table[sel].copy(), dict(w.cfg)))
    with mp.get_context("spawn").Pool(len(jobs)) as pool:
        pool.map(_fast_worker, [(j[0][:1], j[1][:1], j[2], j[3][:1], j[4]) for j in jobs])   # start-up, imports
        t0 = time.perf_counter()
        res = pool.map(_fast_worker, jobs)
        dt = time.perf_counter() - t0
    audio = sum(r[0] for r in res)
    return audio / dt, f"first {n_utts} utterance(s), {audio:.1f} audio-s, {dt:.1f} s wall, numpy/scipy fp64", len(jobs)


def run_reference(args):
    """The CPU checker as the reference arm: each step is one utterance of the
    workload (cut to 5 s) through all four steps in fp64 on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from paper_1912_11040_b200 import synth
    import oracle
    oracle._load()
    w = synth.make_workload(args.workload, seed=0, batch=min(args.steps + args.warmup, 64))
    cap = int(5.0 * w.cfg["fs"])
    audio = 0.0
    times = []
    for i in range(args.warmup + args.steps):
        b = i % w.B
        n = min(int(w.lengths[b]), cap)
        t0 = time.perf_counter()
        oracle.utterance(w.speech[b, :n], w.bank, w.table[b], w.cfg)
        dt = time.perf_counter() - t0
        if i >= args.warmup:
            times.append(dt)
            audio += n / w.cfg["fs"]
    total = float(sum(times))
    value = audio / total
    cores = os.cpu_count() or 1
    sample = (f"{args.steps} step(s) of one utterance each, cut to 5 s, of {workload_label(args.workload)}; "
              "direct fp64 convolution, image sum and DFT (OpenMP)")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / max(args.steps, 1),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic",
            "config": {"workload": workload_label(args.workload), "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


def combine_ranks(audio_seconds, ms_device, s_e2e, world, device):
    """Whole-job figures from per-rank ones: every rank is an independent replica, so
    the audio processed adds up and the job takes as long as its slowest rank."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([audio_seconds, ms_device, s_e2e], dtype=torch.float64, device=device)
    if world > 1:
        a = t.clone()
        dist.all_reduce(a[0:1], op=dist.ReduceOp.SUM)
        dist.all_reduce(a[1:3], op=dist.ReduceOp.MAX)
        t = a
    return tuple(float(v) for v in t.cpu())


# ------------------------------------------------------------------ GPU arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_1912_11040_b200 import binding, build, synth

    build.build()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # every rank runs the same kind of job on its own draw of the workload
    w = synth.make_workload(args.workload, seed=rank, batch=args.batch, noise_align=args.noise_align)
    if args.vtlp_win:
        w.cfg["vtlp_win"] = args.vtlp_win          # warp the speech waveform instead of the filterbank
    # the host entry point returns the frames of every utterance and its frame count; with
    # "padded" it also transfers the padding rows up to T_max
    w.cfg["host_rows"] = 1 if args.host_rows == "valid" else 0
    cfg = binding.make_config(w.cfg, w.B, w.stride, host_staging=True, max_bank_samples=w.bank.size)
    ctx = binding.AugContext(cfg)
    speech = torch.from_numpy(w.speech).cuda()
    lengths = torch.from_numpy(w.lengths).cuda()
    bank = torch.from_numpy(w.bank).cuda()
    table = binding.table_to_device(w.table)
    T_max = binding.aug_frame_count(int(w.lengths.max()), cfg.win, cfg.hop)
    feats = torch.empty((w.B, T_max, cfg.n_mel), device="cuda")
    counts = torch.empty(w.B, dtype=torch.int32, device="cuda")
    rc, bad = binding.aug_validate_params(cfg, w.table, w.bank.size)
    assert rc == 0, f"table row {bad} invalid"

    def step():
        ctx.aug_pipeline(speech, w.stride, lengths, w.lengths, bank, w.bank.size, table, w.B,
                         feats, T_max, counts)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    assert ctx.aug_last_status() == (-1, 0)

    # ---- device-resident timing (no stage events inside: those are taken in a pass of their own)
    sampler = ClockSampler(local_rank)
    launches0 = ctx.aug_launch_count()
    barrier()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    clocks = sampler.stop()
    ms_total = e0.elapsed_time(e1)
    launches = ctx.aug_launch_count() - launches0
    # ---- the same audio with noise stretches that start and end anywhere (the default
    # recipe hands out stretches on multiples of four samples)
    ms_unaligned = None
    if args.noise_align > 1 and not args.skip_e2e:
        table_un = binding.table_to_device(
            synth.redraw_noise_stretches(w.table, w.lengths, w.bank.size, seed=rank, noise_align=1))
        rc_un, bad_un = binding.aug_validate_params(cfg, synth.redraw_noise_stretches(
            w.table, w.lengths, w.bank.size, seed=rank, noise_align=1), w.bank.size)
        assert rc_un == 0, f"unaligned table row {bad_un} invalid"

        def step_un():
            ctx.aug_pipeline(speech, w.stride, lengths, w.lengths, bank, w.bank.size, table_un, w.B,
                             feats, T_max, counts)

        for _ in range(3):
            step_un()
        barrier()
        u0, u1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        u0.record()
        for _ in range(args.steps):
            step_un()
        u1.record()
        barrier()
        ms_unaligned = u0.elapsed_time(u1) / args.steps
        assert ctx.aug_last_status() == (-1, 0)

    # ---- per-stage times: the same steps again with an event pair around every stage
    ctx.aug_enable_stage_timing(True)
    for _ in range(min(args.steps, 100)):
        step()
    stage_ms, n_rec = ctx.aug_stage_times()
    ctx.aug_enable_stage_timing(False)

    # ---- end to end from pinned host buffers
    sp_h = torch.from_numpy(w.speech).pin_memory()
    bk_h = torch.from_numpy(w.bank).pin_memory()
    tb_h = torch.from_numpy(np.ascontiguousarray(w.table).view(np.uint8).reshape(-1).copy()).pin_memory()
    ln_h = torch.from_numpy(w.lengths).pin_memory()
    f_h = torch.empty((w.B, T_max, cfg.n_mel)).pin_memory()
    c_h = torch.empty(w.B, dtype=torch.int32).pin_memory()

    def step_e2e():
        ctx.aug_pipeline_host(sp_h, w.stride, ln_h, bk_h, w.bank.size, tb_h, w.B, f_h, T_max, c_h)

    e2e_steps = 1 if args.skip_e2e else max(3, min(args.steps, 10))
    for _ in range(0 if args.skip_e2e else 2):
        step_e2e()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        step_e2e()
    torch.cuda.synchronize()
    dt_e2e = time.perf_counter() - t0
    barrier()
    h2d, d2h = ctx.aug_last_host_bytes()     # what the library really copied (ragged rows)

    # ---- the same with the noise bank uploaded once (a noise database does not change
    # from batch to batch): only speech, lengths and the table cross the bus every step
    dt_res, h2d_res = 0.0, 0
    if not args.skip_e2e:
        ctx.aug_upload_noise_bank(bk_h, w.bank.size)

        def step_res():
            ctx.aug_pipeline_host(sp_h, w.stride, ln_h, None, w.bank.size, tb_h, w.B, f_h, T_max, c_h)

        step_res()
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            step_res()
        torch.cuda.synchronize()
        dt_res = time.perf_counter() - t0
        barrier()
        h2d_res, _ = ctx.aug_last_host_bytes()

    if world > 1:
        t_res = torch.tensor([dt_res], dtype=torch.float64, device="cuda")
        dist.all_reduce(t_res, op=dist.ReduceOp.MAX)
        dt_res = float(t_res.cpu()[0])
    audio_total, ms_total, dt_e2e = combine_ranks(w.audio_seconds, ms_total, dt_e2e, world, "cuda")
    value = audio_total * args.steps / (ms_total * 1e-3)
    e2e_value = audio_total * e2e_steps / dt_e2e

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    # ---- roofline of the dominant kernel
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    hbm_peak, hbm_src = (peaks["hbm_gbs"], "measured") if "hbm_gbs" in peaks else (6650.0, "fallback")
    fp32_measured = binding.aug_measure_fp32_peak()
    sm_count = torch.cuda.get_device_properties(local_rank).multi_processor_count
    fp32_nominal = sm_count * FP32_LANES * 2 * (clocks["sm_max_mhz"] or 1965) * 1e6 / 1e12
    idx_of = {n: i for i, n in enumerate(binding.STAGE_NAMES)}
    work = dict(conv_work(w))
    work["features"] = feat_work(w)
    work["rir_image"] = rir_work(w)
    kernels = {name: (idx_of[name], fb) for name, fb in work.items()}
    # the convolution step = its block-spectra kernel (long-response contexts) + the convolution kernels
    stage_of = {name: stage_ms[idx] for name, (idx, _) in kernels.items()}
    stage_of["convolve"] += stage_ms[idx_of["block_spectra"]]
    dom = max(kernels, key=lambda k: stage_of[k])
    per_kernel = {}
    for name, (idx, (flops, byts)) in kernels.items():
        ms = stage_of[name]
        if ms <= 0:
            continue
        t_alu, t_hbm = flops / (fp32_measured * 1e12), byts / (hbm_peak * 1e9)
        bound = "alu" if t_alu >= t_hbm else "hbm"
        per_kernel[name] = {
            "ms": ms, "bound": bound,
            "tflops": flops / (ms * 1e-3) / 1e12, "frac_fp32": flops / (ms * 1e-3) / 1e12 / fp32_measured,
            "gbs": byts / (ms * 1e-3) / 1e9, "frac_hbm": byts / (ms * 1e-3) / 1e9 / hbm_peak}
    # fp32 instructions executed per nominal FMA (ncu instruction counts in profiles/): no SIMT
    # kernel that issues one instruction per slot can exceed this share of the nominal-flop roofline
    for name, ceil in FP32_INSTRUCTION_CEILING.items():
        if name in per_kernel and not (name == "features" and int(w.cfg["n_fft"]) != 512):
            per_kernel[name]["fp32_instruction_ceiling"] = ceil
            per_kernel[name]["frac_of_instruction_ceiling"] = per_kernel[name]["frac_fp32"] / ceil
    d = per_kernel[dom]
    if d["bound"] == "alu":
        roofline = {"kernel": dom, "bound": "alu", "achieved": d["tflops"], "peak": fp32_measured,
                    "unit": "TFLOP/s", "frac": d["frac_fp32"], "traffic": None,
                    "peak_source": "fp32 FMA loop measured in this run "
                                   f"(nominal {fp32_nominal:.1f} at max clock)"}
    else:
        roofline = {"kernel": dom, "bound": "hbm", "achieved": d["gbs"], "peak": hbm_peak,
                    "unit": "GB/s", "frac": d["frac_hbm"], "traffic": None,
                    "peak_source": f"{hbm_src} copy bandwidth"}
    per_audio = NCU_TRAFFIC["bytes_per_audio_s"].get(args.workload, {})
    if (dom in per_audio and args.vtlp_win == 0
            and kernel_sources_sha(NCU_TRAFFIC["sources"][dom][0]) == NCU_TRAFFIC["sources"][dom][1]):
        roofline["traffic"] = per_audio[dom] * w.audio_seconds
        roofline["traffic_note"] = ("bytes per launch, ncu capture on %s scaled by audio-seconds; "
                                    "algorithmic bytes of this kernel: %.3e"
                                    % (NCU_TRAFFIC["captured_on"][args.workload], kernels[dom][1][1]))
    roofline["per_kernel"] = per_kernel
    roofline["stage_ms"] = dict(zip(binding.STAGE_NAMES, stage_ms))
    roofline["stage_calls_averaged"] = n_rec

    if args.cpu_budget > 0:
        cpu_val, cpu_sample, cores = time_oracle(w, args.cpu_budget)
    else:
        cpu_val, cpu_sample, cores = None, "skipped (--cpu-budget 0)", os.cpu_count() or 1
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": workload_label(args.workload), "batch": w.B, "noise_align": args.noise_align, "vtlp_win": args.vtlp_win,
                       "host_rows": args.host_rows,
                       "audio_seconds_per_step": w.audio_seconds, "parallelism": f"replicas x{world}",
                       "l2": "inputs larger than L2 (speech + noise bank "
                             f"{(speech.numel() + bank.numel()) * 4 / 1e6:.0f} MB per step)"},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "steps": e2e_steps},
            "gpu_launches": int(launches),
            "roofline": roofline,
            "cpu_baseline": {"value": cpu_val, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": cpu_sample}}
    if ms_unaligned is not None:
        line["noise_unaligned"] = {"ms_per_step": ms_unaligned,
                                   "value": w.audio_seconds * world / (ms_unaligned * 1e-3), "unit": UNIT,
                                   "note": "same audio, noise stretches at any offset and length (rank 0's "
                                           "own time); the headline uses stretches on multiples of 4 samples"}
    if dt_res > 0:
        line["e2e_resident_bank"] = {"value": audio_total * e2e_steps / dt_res, "unit": UNIT,
                                     "h2d_bytes_per_step": h2d_res, "d2h_bytes_per_step": d2h,
                                     "steps": e2e_steps,
                                     "note": "noise bank uploaded once with aug_upload_noise_bank; "
                                             "e2e above sends it with every step"}
    if args.cpu_fast_utts > 0:
        fv, fs_, fw = time_fast_cpu(w, args.cpu_fast_utts)
        line["cpu_fast"] = {"value": fv, "unit": UNIT, "cores": fw, "kind": "numpy/scipy FFT pipeline",
                            "sample": fs_}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=2, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--cpu-budget", type=float, default=15.0,
                    help="seconds of wall time given to the CPU-checker baseline")
    ap.add_argument("--cpu-fast-utts", type=int, default=64,
                    help="utterances given to the numpy/scipy CPU pipeline (0 = skip)")
    ap.add_argument("--noise-align", type=int, default=4, choices=[1, 4],
                    help="noise stretches start and end on multiples of this many samples (1 = anywhere)")
    ap.add_argument("--host-rows", choices=("valid", "padded"), default="valid",
                    help="end-to-end leg: feature rows the host call copies back (valid frames only, "
                         "or all T_max rows of every utterance with their padding)")
    ap.add_argument("--vtlp-win", type=int, default=0,
                    help="apply the warp to the speech waveform with this window (800 = 50 ms) instead of "
                         "inside the filterbank")
    ap.add_argument("--batch", type=int, default=None,
                    help="profiling runs: fewer utterances than the workload's own batch")
    ap.add_argument("--skip-e2e", action="store_true",
                    help="profiling runs: one end-to-end step instead of a timed series")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
