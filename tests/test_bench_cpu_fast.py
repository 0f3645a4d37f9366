"""The numpy/scipy pipeline bench.py times as its second CPU baseline must compute the
same features as the checker, or the comparison would be meaningless."""
import os
import sys

import numpy as np

import oracle
from paper_1912_11040_b200 import synth

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench


def test_fast_cpu_pipeline_agrees_with_the_checker():
    w = synth.make_workload(2, batch=3, dur_scale=0.1)
    for b in range(w.B):
        ref = oracle.utterance(w.speech[b, : w.lengths[b]], w.bank, w.table[b], w.cfg)
        got = bench.fast_cpu_utterance(w.speech[b, : w.lengths[b]], w.bank, w.table[b], w.cfg)
        assert got.shape == ref["feats"].shape
        assert np.max(np.abs(got - ref["feats"])) < 1e-6


def test_fast_cpu_timing_runs_on_spawned_workers():
    w = synth.make_workload(1, batch=4, dur_scale=0.25)
    rate, what, workers = bench.time_fast_cpu(w, 4)
    assert rate > 0 and workers >= 1 and "4 utterance" in what
