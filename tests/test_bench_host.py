"""Host-side accounting of bench.py (no GPU): the counts its roofline fractions are built on."""
import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench
from oracle import zipcache_oracle as zo
from workloads import get_config


def test_prefill_exponentials_count_the_unmasked_probe_entries():
    """Eq. 9: a probe row at position p attends keys 0..p; both score passes evaluate one
    exponential per such entry and query head."""
    w = get_config(1)
    P = zo.probe_positions(w.context, w.rho_recent, w.rho_random, w.seed(0))
    mask = np.arange(w.context)[None, :] <= np.asarray(P)[:, None]
    assert bench.prefill_exponentials(w, P.tolist()) == 2 * mask.sum() * w.n_q_heads * w.batch


def test_exp2_peak_is_16_results_per_clock_and_sm():
    assert bench.EXP2_PER_S_PEAK == 148 * 16 * 1.965e9


def test_prefill_bytes_cover_inputs_and_packed_outputs():
    """K twice for the score passes, K and V twice for maxima and quantiser, codes and parameters."""
    w = get_config(2)
    l, units = w.context, w.units_per_layer
    n_s = int(np.floor(w.saliency_ratio * l))
    packed = n_s * (32 * w.bits_hi + 16) + (l - n_s) * (32 * w.bits_lo + 16)
    got = bench.algorithmic_prefill_bytes(w)
    assert got >= units * (6 * l * 256 + packed)
    assert got <= units * (6 * l * 256 + packed) * 1.15   # + the probe rows of Q, a tenth of the rows
