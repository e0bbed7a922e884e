"""CUDA library against the CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest

from paper_2604_26968_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_config1_tiny_gqa_50_epochs_bit_exact():
    from lockstep import Lockstep
    w = W.config(1)
    ls = Lockstep(w, payload=True, batch_bytes=256 << 10)
    tot = dict(events=0, promoted=0, admitted=0)
    for e in range(w.epochs):
        r = ls.epoch(e)
        for k_ in tot:
            tot[k_] += r[k_]
    assert tot["events"] == 50 * 819 and tot["promoted"] > 0 and tot["admitted"] > 0
    assert ls.ora.stats()["bytes_dropped"] > 0       # the 4,096-slot ring wrapped
    ls.close()
