"""Algorithm 2 of the paper as a loop over the library's entry points (bench.decoding_loops), on the
reduced LlamaGen-XL shape: the bookkeeping the algorithm fixes must hold on the device's own outputs."""
import os
import sys

import pytest

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench  # noqa: E402
from vvs_synth.configs import XL_SMALL  # noqa: E402

pytestmark = pytest.mark.gpu


def test_decoding_loop_bookkeeping():
    status, res = bench.decoding_loops(XL_SMALL, 41, (("plain", 2.0), ("skipping", 0.3)), n_tokens=120, warm=False)
    assert status == 0
    plain, skipping = res["plain"], res["skipping"]
    assert plain["skipped_steps"] == 0 and plain["tokens"] >= 120
    assert skipping["skipped_steps"] > 0 and skipping["tokens"] >= 120
    for r in (plain, skipping):
        fill, tokens, prev_skip, pending = 1, 0, False, 0
        for entry in r["log"]:
            if entry[0] == "skip":
                assert not prev_skip                       # never two verification-free steps in a row (Sec. 4.1)
                gamma = entry[1]
                assert 0 <= gamma <= 5 and entry[2] >= 0.3  # Eq. 3 bound (paths of depth 5); S_bar above the threshold
                pending, tokens, prev_skip = gamma, tokens + gamma, True
            else:
                _, f, n_acc, new_len = entry
                assert f == 1 + pending                    # post verification: the unverified tokens ride along
                assert 0 <= n_acc <= 8
                fill += f + n_acc
                assert new_len == fill                     # the device's fill level after the step
                pending, tokens, prev_skip = 0, tokens + n_acc + 1, False
        assert tokens == r["tokens"] and fill == r["final_fill"]
        assert r["tokens_per_forward"] >= 1.0
    assert skipping["target_forwards"] < plain["target_forwards"]
