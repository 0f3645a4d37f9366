"""The allocation-free variant of step 4 (feat_vtlp_logmel_noalloc).

It exists for users who cannot create a context because they are not allowed to
allocate device memory (a host application owns the whole device through its own
pool, or the allocator is off limits once a real-time pipeline is running).  It
must give what feat_vtlp_logmel gives.  Two calls in a row with different tables
show that the built-in scratch array, which keeps the previous call's contents,
never leaks them into the next result.  This file is named to be collected last."""
import numpy as np
import pytest

import oracle
from paper_1912_11040_b200 import binding, synth
from helpers import Device, LOGMEL_ABS_TOL

pytestmark = pytest.mark.gpu


def _reference_and_noalloc(dev, P, counts, table_np, B):
    import torch
    tab = binding.table_to_device(table_np)
    ref = torch.full((dev.w.B, P.shape[1], dev.M), float("nan"), device="cuda")
    dev.ctx.feat_vtlp_logmel(P, counts, tab, B, P.shape[1], ref)
    got = torch.full_like(ref, float("nan"))
    binding.feat_vtlp_logmel_noalloc(dev.cfg, P, counts, tab, B, P.shape[1], got)
    torch.cuda.synchronize()
    return ref.cpu().numpy(), got.cpu().numpy()


def _check_against_cpu(w, P, counts, table_np, got, B):
    """The same power spectra through the fp64 CPU definition of the warped filterbank:
    an error common to both GPU entry points (they share kernels) would show here."""
    Ph, ch = P.cpu().numpy().astype(np.float64), counts.cpu().numpy()
    cfg = w.cfg
    for b in range(B):
        T = int(ch[b])
        ref = oracle.logmel(Ph[b, :T], float(table_np[b]["alpha"]), cfg["n_fft"], cfg["n_mel"], cfg["fs"],
                            cfg["f_lo"], cfg["f_hi"], floor=cfg["log_floor"])
        assert np.max(np.abs(got[b, :T] - ref), initial=0.0) <= LOGMEL_ABS_TOL, b
        assert np.all(got[b, T:] == cfg["pad_value"])


@pytest.mark.parametrize("index", [1, 5])
def test_noalloc_matches_context_entry_point_twice(index):
    w = synth.make_workload(index, batch=6, dur_scale=0.25 if index == 1 else 0.02)
    w.lengths[0] = 399          # an utterance without frames: all padding
    dev = Device(w)
    P, counts = dev.stft_power(dev.speech)

    # first call: the workload's own warp factors, all six utterances
    ref, got = _reference_and_noalloc(dev, P, counts, w.table, w.B)
    assert np.max(np.abs(got - ref)) <= LOGMEL_ABS_TOL
    assert np.array_equal(np.isnan(got), np.isnan(ref))
    _check_against_cpu(w, P, counts, w.table, got, w.B)

    # second call straight after: other warp factors and a smaller batch, so any
    # table entry left over from the first call would show up as a mismatch
    t2 = w.table.copy()
    t2["alpha"] = np.linspace(0.8, 1.2, w.B).astype(np.float32)[::-1]
    ref2, got2 = _reference_and_noalloc(dev, P, counts, t2, 4)
    assert np.max(np.abs(got2[:4] - ref2[:4])) <= LOGMEL_ABS_TOL
    _check_against_cpu(w, P, counts, t2, got2, 4)
    assert np.all(np.isnan(got2[4:]))                 # rows of utterances not asked for stay untouched
    assert np.max(np.abs(ref2[1:4] - ref[1:4])) > 1e-2   # the two calls really differed


def test_noalloc_rejects_what_does_not_fit():
    import torch
    w = synth.make_workload(1, batch=1, dur_scale=0.1)
    cfg = binding.make_config(w.cfg, 1, w.stride)
    x = torch.zeros(16, device="cuda")
    c = torch.zeros(4, dtype=torch.int32, device="cuda")
    too_many = binding.NOALLOC_MAX_BATCH + 1
    assert binding.feat_vtlp_logmel_noalloc(cfg, x, c, x, too_many, 1, x, check=False) == binding.AUG_ECAP
    assert "capacity" in binding.strerror(binding.AUG_ECAP)
    assert binding.feat_vtlp_logmel_noalloc(cfg, None, c, x, 1, 1, x, check=False) == binding.AUG_EINVAL
    cfg.n_fft = 2048
    assert binding.feat_vtlp_logmel_noalloc(cfg, x, c, x, 1, 1, x, check=False) == binding.AUG_EINVAL
    # the same scalar checks a context applies: band edge above Nyquist, non-finite padding
    cfg = binding.make_config(w.cfg, 1, w.stride)
    cfg.f_hi = 0.5 * cfg.fs + 100.0
    assert binding.feat_vtlp_logmel_noalloc(cfg, x, c, x, 1, 1, x, check=False) == binding.AUG_EINVAL
    cfg = binding.make_config(w.cfg, 1, w.stride)
    cfg.pad_value = float("nan")
    assert binding.feat_vtlp_logmel_noalloc(cfg, x, c, x, 1, 1, x, check=False) == binding.AUG_EINVAL
