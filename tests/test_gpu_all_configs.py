"""Every decode step of the three larger benchmark configurations, CUDA library against the CPU
oracle, through the real decode protocol (accept + commit + next build per step, the oracle's
accept lengths driving both sides): whole runs from the warm start for the shortest and the
longest suffix length, and a stretch of consecutive steps on nearly full histories.  Accept
lengths, drafted tokens, scores and edge weights are compared after every step, the match lists
and the exported DAG of all paths every few steps, the histories at the end."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from paper_2503_05330_b200 import synth  # noqa: E402
import harness  # noqa: E402
from harness import Pair  # noqa: E402


def whole_run(wid, k, check_every, B=4, Ke=2):
    w = synth.WORKLOADS[wid]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, B=B, Ke=Ke, max_append=w.D)
    st = harness.run_step_protocol(pair, tokens, lps, [k], steps=w.steps, warm=w.k_max, check_every=check_every,
                                   check_dag=True)
    assert st["steps"] == w.steps and st["accepted"] > 0
    return pair


def near_full(wid, ks, steps, check_every, slack):
    w = synth.WORKLOADS[wid]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, B=4, Ke=2, max_append=w.D)
    start = (w.L - slack - (np.arange(w.P) * 29) % 300).astype(np.int32)        # ragged; some paths fill up on the way
    st = harness.run_step_protocol(pair, tokens, lps, ks, steps=steps, warm=0, start_lens=start,
                                   check_every=check_every, check_dag=True)
    assert st["steps"] == steps
    return pair


@pytest.mark.parametrize("k", [1, 4])
def test_config3_every_step_of_the_whole_run(k):
    whole_run(3, k, check_every=10)


def test_config3_consecutive_steps_on_nearly_full_histories():
    near_full(3, [1, 4, 2, 3], steps=120, check_every=10, slack=100)


@pytest.mark.parametrize("k", [1, 5])
def test_config4_every_step_of_the_whole_run(k):
    pair = whole_run(4, k, check_every=50)
    assert not pair.g.step_is_single_launch()       # 32 clusters of 16 do not fit the device at once: accept, then build


def test_config4_consecutive_steps_on_nearly_full_histories():
    near_full(4, [1, 5, 3], steps=60, check_every=10, slack=60)


@pytest.mark.parametrize("k", [1, 8])
def test_config5_every_step_of_the_whole_run(k):
    # prompts of this size take the probe / tile-scan / dag kernels
    pair = whole_run(5, k, check_every=25)
    assert not pair.g.step_is_single_launch()


@pytest.mark.parametrize("k", [1, 8])
def test_config5_consecutive_steps_on_nearly_full_histories(k):
    # k = 1: queries on frequent tokens match tens of thousands of positions
    near_full(5, [k], steps=110, check_every=10, slack=200)
