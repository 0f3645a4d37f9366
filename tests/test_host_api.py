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


def test_compute_calls_refuse_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    w = synth.make_workload(1, batch=1, dur_scale=0.1)
    with pytest.raises(RuntimeError):
        binding.AugContext(binding.make_config(w.cfg, 1, w.stride))
