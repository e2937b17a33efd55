"""The latency sweep shaped like the paper's two efficiency figures (Section 3.2: decode latency
after a fixed prompt, and single-shot prefill latency, over a range of lengths) runs all three
arms -- every layer retrieval, mixed-head layers, exclusive layers -- and yields finite numbers."""
import math

import pytest

from paper_2508_12407_b200 import sweep

pytestmark = pytest.mark.gpu


def test_sweep_runs_all_arms_on_two_short_lengths():
    lengths = [256, 640]
    rows = sweep.run(lengths, decode_prompt=2048, reps=1)
    for phase in ("decode", "prefill"):
        assert list(rows[phase]) == lengths
        for n in lengths:
            assert set(rows[phase][n]) == set(sweep.ARMS)
            for arm, us in rows[phase][n].items():
                assert math.isfinite(us) and us > 0.0, (phase, n, arm, us)
    text = sweep.table(rows)
    assert text.count("\n") == 1 + 2 * len(lengths)
    # a stack with streaming layers reads fewer bytes per decoded token than full attention
    for n in lengths:
        assert rows["decode"][n]["exclusive"] < rows["decode"][n]["original"] * 1.25
