"""Parity at the full sizes of the five named workloads, through aug_pipeline in the
launch configuration bench.py times (whole batch, host lengths supplied, no waveform
output).  The CPU checker cannot finish a full batch, so it computes a few whole
utterances per workload (features and, in a second call, the mixed waveform are
compared element by element for those); for every utterance the frame count must
equal the closed form, padding rows must hold the pad value and every feature must
be finite and above the log floor."""
import numpy as np
import pytest

from paper_1912_11040_b200 import binding, synth
from helpers import Device, check_pipeline_against_oracle, oracle_batch

pytestmark = pytest.mark.gpu

# utterances given to the CPU checker: the shortest, the longest and one in between
def _sample(w, k):
    order = np.argsort(w.lengths, kind="stable")
    picks = [int(order[0]), int(order[-1]), int(order[len(order) // 2])]
    return sorted(set(picks))[:k]


# (the last case draws noise stretches at any offset and of any length: scalar loads)
@pytest.mark.parametrize("index,n_check,noise_align",
                         [(1, 3, 4), (2, 3, 4), (3, 2, 4), (4, 3, 4), (5, 1, 4), (4, 2, 1)])
def test_full_size_workload(index, n_check, noise_align):
    w = synth.make_workload(index, seed=0, noise_align=noise_align)
    dev = Device(w)
    rc, bad = binding.aug_validate_params(dev.cfg, w.table, w.bank.size)
    assert rc == 0, bad
    F, counts, _ = dev.pipeline(want_wave=False, lengths_host=True)
    assert dev.ctx.aug_last_status() == (-1, 0)
    Fh, ch = F.cpu().numpy(), counts.cpu().numpy()

    win, hop = int(w.cfg["win"]), int(w.cfg["hop"])
    expect = np.where(w.lengths >= win, 1 + (w.lengths - win) // hop, 0)
    assert np.array_equal(ch, expect)                       # bit-exact frame counts, every utterance
    floor = np.log(w.cfg["log_floor"])
    for b in range(w.B):
        T = int(expect[b])
        assert np.all(np.isfinite(Fh[b, :T])) and np.all(Fh[b, :T] >= floor - 1e-3)
        assert np.all(Fh[b, T:] == w.cfg["pad_value"])

    picks = _sample(w, n_check)
    orc = oracle_batch(w, utts=picks)
    worst_f, _ = check_pipeline_against_oracle(dev, F, counts, None, orc)

    # the same launch with the waveform requested: compare it for the sampled utterances
    F2, counts2, wave = dev.pipeline(want_wave=True, lengths_host=True)
    _, worst_w = check_pipeline_against_oracle(dev, F2, counts2, wave, orc)
    print(f"config{index} full size ({w.B} utts, {w.audio_seconds:.0f} audio-s): utterances {picks}: "
          f"worst log-mel err {worst_f:.2e}, worst wave err/rms {worst_w:.2e}")


def test_parked_and_time_domain_noise_sums_agree_on_every_utterance():
    """Config 2 at full size with parking slots under contention (every multiprocessor's
    slots in use at once): the frequency-domain sum of several noise sources must give
    the same features, for every utterance of the batch, as the time-domain sum that a CTA
    falls back to when it finds no slot."""
    w = synth.make_workload(2, seed=0)
    dev = Device(w)
    F1, c1, _ = dev.pipeline(want_wave=False, lengths_host=True)
    dev.ctx.aug_hold_parking_slots(True)
    F2, c2, _ = dev.pipeline(want_wave=False, lengths_host=True)
    dev.ctx.aug_hold_parking_slots(False)
    assert dev.ctx.aug_last_status() == (-1, 0)
    assert np.array_equal(c1.cpu().numpy(), c2.cpu().numpy())
    assert int((w.table["n_src"] > 2).sum()) > 20                 # rows that do use the slots
    assert float((F1 - F2).abs().max()) <= 1e-3
