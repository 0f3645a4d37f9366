"""CPU-only checks of the library's host side: it loads, exports every symbol the
header declares, and its pure-host entry points behave."""
import os
import re

import numpy as np
import pytest

from paper_1912_11040_b200 import binding, build, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    build.build()


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "aug_b200.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b((?:aug|feat)_[a-z_0-9]+)\s*\(", hdr))
    assert declared == set(binding.EXPORTS)
    L = binding.lib()
    for name in declared:
        assert hasattr(L, name), name


def test_struct_layouts_match_the_header(tmp_path):
    """Compile the header with gcc and compare sizes / offsets with the Python mirrors."""
    import ctypes
    import subprocess
    src = tmp_path / "abi.c"
    src.write_text('''#include <stdio.h>
#include <stddef.h>
#include "aug_b200.h"
int main(void) {
    printf("%zu %zu %zu %zu %zu %zu %zu\\n", sizeof(AugUttParams), offsetof(AugUttParams, src_pos),
           offsetof(AugUttParams, noise_offset), offsetof(AugUttParams, noise_len),
           offsetof(AugUttParams, noise_weight), sizeof(AugConfig),
           offsetof(AugConfig, max_bank_samples));
    return 0;
}''')
    exe = tmp_path / "abi"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    got = [int(v) for v in subprocess.run([str(exe)], capture_output=True, text=True,
                                          check=True).stdout.split()]
    f = synth.UTT_DTYPE.fields
    assert got == [synth.UTT_DTYPE.itemsize, f["src_pos"][1], f["noise_offset"][1],
                   f["noise_len"][1], f["noise_weight"][1], ctypes.sizeof(binding.AugConfig),
                   binding.AugConfig.max_bank_samples.offset]


@pytest.mark.parametrize("n,expect", [(0, 0), (399, 0), (400, 1), (559, 1), (560, 2), (32000, 198)])
def test_frame_count(n, expect):
    assert binding.aug_frame_count(n, 400, 160) == expect


def test_strerror_and_workspace_size():
    assert "capacity" in binding.strerror(binding.AUG_ECAP)
    w = synth.make_workload(1, batch=2, dur_scale=0.1)
    cfg = binding.make_config(w.cfg, 2, w.stride)
    assert binding.aug_workspace_bytes(cfg) > 0
    cfg.n_fft = 300
    assert binding.aug_workspace_bytes(cfg) == binding.AUG_EINVAL
    cfg.n_fft = 512
    cfg.host_rows = 1
    assert binding.aug_workspace_bytes(cfg) > 0
    cfg.host_rows = 2
    assert binding.aug_workspace_bytes(cfg) == binding.AUG_EINVAL


def test_validate_params():
    w = synth.make_workload(2, batch=5, dur_scale=0.1)
    cfg = binding.make_config(w.cfg, 5, w.stride)
    assert binding.aug_validate_params(cfg, w.table, w.bank.size) == (0, -1)
    for field, value in [("alpha", 2.5), ("n_src", 7), ("order", 99), ("snr_db", np.nan)]:
        t = w.table.copy()
        t[field][3] = value
        assert binding.aug_validate_params(cfg, t, w.bank.size) == (binding.AUG_EPARAM, 3)
    t = w.table.copy()
    t["mic"][2] = (100, 1, 1)        # outside the room
    assert binding.aug_validate_params(cfg, t, w.bank.size) == (binding.AUG_EPARAM, 2)
    t = w.table.copy()
    t["beta"][1][4] = 1.5
    assert binding.aug_validate_params(cfg, t, w.bank.size) == (binding.AUG_EPARAM, 1)
    assert binding.aug_validate_params(cfg, w.table, 10)[0] == binding.AUG_EPARAM  # bank too short


def _dist(bank_len=200000, **kw):
    d = binding.AugDist()
    d.room_lo[:] = (3, 3, 2.5)
    d.room_hi[:] = (10, 8, 4)
    d.t60_lo, d.t60_hi, d.order = 0.2, 0.8, 6
    d.n_noise_lo, d.n_noise_hi = 0, 3
    d.snr_lo, d.snr_hi, d.alpha_lo, d.alpha_hi = 0, 20, 0.8, 1.2
    d.wall_margin, d.min_src_mic_dist, d.min_noise_len, d.bank_len = 0.3, 0.5, 4000, bank_len
    for k, v in kw.items():
        setattr(d, k, v)
    return d


def test_sample_params_rows_are_valid_deterministic_and_in_range():
    rng = np.random.default_rng(0)
    lengths = rng.integers(1000, 160000, 500).astype(np.int32)
    d = _dist()
    rc, t = binding.aug_sample_params(7, d, lengths)
    assert rc == 0
    w = synth.make_workload(2, batch=1, dur_scale=0.05)
    cfg = binding.make_config(dict(w.cfg, max_order=6, max_sources=4), 500, 160000)
    assert binding.aug_validate_params(cfg, t, d.bank_len) == (0, -1)
    assert np.all((t["room"] >= (3, 3, 2.5)) & (t["room"] <= (10, 8, 4)))
    assert np.all((t["alpha"] >= 0.8) & (t["alpha"] <= 1.2)) and np.all((t["snr_db"] >= 0) & (t["snr_db"] <= 20))
    assert set(np.unique(t["n_src"])) == {1, 2, 3, 4} and np.all(t["order"] == 6)
    # Eyring: the drawn beta corresponds to a T60 inside the requested range
    vol = t["room"].astype(np.float64).prod(axis=1)
    r = t["room"].astype(np.float64)
    surf = 2 * (r[:, 0] * r[:, 1] + r[:, 1] * r[:, 2] + r[:, 0] * r[:, 2])
    t60 = -0.161 * vol / (surf * np.log(t["beta"][:, 0].astype(np.float64) ** 2))
    assert np.all((t60 > 0.2 - 1e-4) & (t60 < 0.8 + 1e-4))
    assert np.all(t["beta"] == t["beta"][:, :1])
    # geometry: margins and minimum distance
    assert np.all(t["mic"] >= 0.3 - 1e-6) and np.all(t["mic"] <= t["room"] - 0.3 + 1e-6)
    for s in range(4):
        used = t["n_src"] > s
        dist = np.linalg.norm(t["src_pos"][used, s] - t["mic"][used], axis=1)
        assert np.all(dist >= 0.5 - 1e-5)
    # noise stretches: inside the bank, between half and the whole utterance (floored at 4000)
    for j in range(3):
        used = t["n_src"] > j + 1
        ln, n = t["noise_len"][used, j], np.maximum(lengths[used], 4000)
        assert np.all(ln <= n) and np.all(ln >= np.maximum(n // 2, 4000))
        assert np.all(t["noise_offset"][used, j] + ln <= d.bank_len)
    # counter-based: a row depends on (seed, row index) only
    _, t2 = binding.aug_sample_params(7, d, lengths[:10])
    assert t2.tobytes() == t[:10].tobytes()
    _, t3 = binding.aug_sample_params(8, d, lengths[:10])
    assert t3.tobytes() != t[:10].tobytes()
    # the draws look uniform: mean alpha near the middle of its range
    assert abs(float(t["alpha"].mean()) - 1.0) < 0.03


def test_sample_params_rejects_bad_ranges():
    lengths = np.full(4, 16000, dtype=np.int32)
    assert binding.aug_sample_params(0, _dist(alpha_hi=2.5), lengths, check=False)[0] == binding.AUG_EINVAL
    assert binding.aug_sample_params(0, _dist(n_noise_hi=4), lengths, check=False)[0] == binding.AUG_EINVAL
    assert binding.aug_sample_params(0, _dist(t60_lo=0.0), lengths, check=False)[0] == binding.AUG_EINVAL
    assert binding.aug_sample_params(0, _dist(bank_len=0), lengths, check=False)[0] == binding.AUG_EINVAL


def test_bucket_by_length():
    lengths = np.array([500, 100, 300, 100, 900, 200, 700], dtype=np.int32)
    perm, gmax = binding.aug_bucket_by_length(lengths, 3)
    assert list(perm) == [1, 3, 5, 2, 0, 6, 4]            # increasing length, ties in input order
    assert list(gmax) == [200, 700, 900]
    rng = np.random.default_rng(0)
    lengths = rng.integers(16000, 320000, 256).astype(np.int32)
    perm, gmax = binding.aug_bucket_by_length(lengths, 16)
    assert sorted(perm) == list(range(256))
    padded_sorted = int(np.sum(gmax.astype(np.int64) * 16))
    padded_plain = int(sum(lengths[i:i + 16].max() * 16 for i in range(0, 256, 16)))
    assert padded_sorted < 0.65 * padded_plain and padded_sorted >= int(lengths.sum())


def test_compute_calls_refuse_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    w = synth.make_workload(1, batch=1, dur_scale=0.1)
    with pytest.raises(RuntimeError):
        binding.AugContext(binding.make_config(w.cfg, 1, w.stride))


def test_workspace_follows_the_convolution_route():
    """Responses of up to 8192 taps are convolved without stored block spectra, longer
    ones with them: the workspace a context asks for shows which route it will take."""
    w = synth.make_workload(2, batch=2, dur_scale=0.1)
    sizes = {}
    for taps in (1, 4096, 4097, 8192, 8193, 24576):
        cfg = binding.make_config(dict(w.cfg, rir_taps=taps), 64, 160000)
        sizes[taps] = binding.aug_workspace_bytes(cfg)
        assert sizes[taps] > 0
    spectrum = 64 * cfg.max_sources * 8192 * 8              # one 16384-point spectrum per source
    assert sizes[1] - 64 * cfg.max_sources * 4 * 1 == sizes[8192] - 64 * cfg.max_sources * 4 * 8192
    blocks = -(-160000 // 4096)
    extra = sizes[8193] - sizes[8192]
    parking = 3 * 160 * 8192 * 8 + 3 * 160 * 4 + 512          # only the fused route has it (three or more sources)
    assert extra >= 64 * cfg.max_sources * blocks * 4096 * 8 - parking   # block spectra of every source
    assert extra >= spectrum // 2                              # and a third partition
    assert sizes[24576] > sizes[8193]
