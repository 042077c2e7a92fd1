"""CUDA library against the CPU oracle, element by element, on the same seeded
inputs.  Integer results (tokens, positions, sums, counts) must be identical;
float weights agree within 1e-5 relative (harness.RTOL)."""
import json
import os

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2503_05330_b200 import synth  # noqa: E402
import harness  # noqa: E402
from harness import Pair, run_protocol, t32  # noqa: E402

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_worked_example_on_device():
    w = json.load(open(os.path.join(GOLDEN, "worked_example.json")))
    # logprobs whose probabilities are the example's dyadic values up to fp32 rounding
    pair = Pair(1, 3, w["capacity"], 16, 2, w["D"], B=4, Ke=4)
    a_max = max(len(p) for p in w["paths"])
    tok = np.zeros((3, a_max), np.int32); lp = np.zeros((3, a_max), np.float32)
    for i, p in enumerate(w["paths"]):
        tok[i, :len(p)] = p
        lp[i, :len(p)] = np.log(np.array(w["prob"][i]))
    pair.append(tok, lp, np.array([len(p) for p in w["paths"]], np.int32), expect_status=0)
    pair.check_history()
    t, ln = pair.build_and_compare(w["k"])
    assert t[0, :ln[0]].tolist() == w["draft"]
    assert t[2, :ln[2]].tolist() == w["other_queries"]["2"] and ln[1] == 0
    sampled = np.full((3, w["D"] + 1), 15, np.int32)
    sampled[0] = w["accept"]["sampled"]
    tau = pair.accept_and_compare(sampled, np.full(sampled.shape, -0.5, np.float32))
    assert tau[0] == w["accept"]["tau"]
    pair.check_history()


def test_fixed_point_probabilities_match_on_many_logprobs():
    P, L = 8, 4096
    rng = synth.Stream(4242)
    lp = np.concatenate([-12.0 * rng.uniform(P * L - 64), np.array([0.0, -0.0, -1e-8, -40.0, -41.0, -25.0, -21.4, -21.5]),
                         -30.0 * rng.uniform(56)]).astype(np.float32).reshape(P, L)
    tok = np.zeros((P, L), np.int32)
    pair = Pair(1, P, L, 4, 1, 2)
    pair.append(tok, lp, np.full(P, L, np.int32), expect_status=0)
    pair.check_history()


@pytest.mark.parametrize("seed", range(4))
@pytest.mark.parametrize("alpha,mode", [(1.0, 0), (0.5, 0), (0.0, 0), (1.0, 1)])
def test_dense_tiny_vocab_every_step(seed, alpha, mode):
    # tiny vocabulary: matches, merges and ties everywhere; ragged lengths
    G, N, L, V, D, k_max = 2, 4, 48, 3 + seed % 2, 4, 3
    tokens, lps = synth.small_random(G * N, L, V, 900 + seed)
    for k in range(1, k_max + 1):
        pair = Pair(G, N, L, V, k_max, D, alpha=alpha, mode=mode, B=4, Ke=3)
        start = 3 + (np.arange(G * N) * 5 + seed) % 9
        st = run_protocol(pair, tokens, lps, k, steps=40, warm=0, start_lens=start,
                          commit_in_accept=bool(seed % 2))
        assert st["steps"] > 0


def test_append_clamping_and_status_bits():
    pair = Pair(1, 4, 6, 10, 2, 2)
    tok = np.array([[1, 2, 3, 4], [1, 2, 3, 4], [1, 99, 3, 4], [1, 2, 3, 4]], np.int32)
    lp = np.full((4, 4), -0.3, np.float32)
    pair.append(tok, lp, np.array([4, 0, 4, 7], np.int32), expect_status=0x04 | 0x01)
    pair.append(tok, lp, np.array([4, 2, 0, 0], np.int32), expect_status=0x02)
    pair.append(tok, np.full((4, 4), np.nan, np.float32), np.array([0, 1, 0, 0], np.int32), expect_status=0x08)
    pair.check_history()
    pair.build_and_compare(1)
    pair.build_and_compare(2)


def test_empty_and_degenerate_states():
    # nothing appended yet, then a single token per path, then k larger than some paths
    pair = Pair(2, 3, 16, 5, 3, 3, B=2, Ke=2)
    _, ln = pair.build_and_compare(1)
    assert ln.sum() == 0
    tok = np.ones((6, 4), np.int32); lp = np.full((6, 4), -1.0, np.float32)
    pair.append(tok, lp, np.array([1, 1, 1, 0, 1, 0], np.int32), expect_status=0)
    pair.build_and_compare(1)
    pair.append(tok, lp, np.array([4, 0, 2, 4, 0, 1], np.int32), expect_status=0)
    for k in (1, 2, 3):
        pair.build_and_compare(k)
    # all paths identical and constant: every window matches
    pair = Pair(1, 4, 64, 2, 4, 8, B=3, Ke=2, alpha=0.5)
    pair.append(np.ones((4, 60), np.int32), np.full((4, 60), -0.7, np.float32), np.array([60, 33, 5, 1], np.int32),
                expect_status=0)
    for k in (1, 2, 4):
        pair.build_and_compare(k)


def test_full_paths_are_sources_only():
    N, L = 3, 32
    tokens, lps = synth.small_random(N, L, 3, 5)
    pair = Pair(1, N, L, 3, 2, 4)
    pair.append(tokens, lps, np.array([L, L - 1, 10], np.int32), expect_status=0)
    _, ln = pair.build_and_compare(1)
    assert ln[0] == 0


def test_match_workspace_overflow_is_reported_not_fatal():
    N, L = 4, 64
    pair = Pair(1, N, L, 2, 1, 2, match_capacity=100)
    pair.g.append(harness.t32(np.zeros((N, L - 1), np.int32), pair.dev),
                  harness.t32(np.full((N, L - 1), -0.5, np.float32), pair.dev),
                  harness.t32(np.full(N, L - 1, np.int32), pair.dev))
    assert pair.g.status() == 0
    pair.g.build_drafts(1)
    assert pair.g.status() == 0x20
    assert (pair.g.draft_len.cpu().numpy() == 0).all()      # every query needs more than 100 slots


@pytest.mark.parametrize("k", [1, 2, 3])
def test_config1_full_protocol(k):
    w = synth.WORKLOADS[1]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, B=8, Ke=4, max_append=w.D)
    st = run_protocol(pair, tokens, lps, k, steps=w.steps, warm=w.k_max)
    assert st["steps"] == w.steps


@pytest.mark.parametrize("k", [1, 2, 3, 4])
def test_config2_full_protocol(k):
    w = synth.WORKLOADS[2]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, B=8, Ke=4, max_append=w.D)
    st = run_protocol(pair, tokens, lps, k, steps=w.steps, warm=w.k_max, commit_in_accept=(k % 2 == 0))
    assert st["steps"] > 100


@pytest.mark.parametrize("k", [1, 4])
def test_config3_protocol(k):
    w = synth.WORKLOADS[3]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, B=8, Ke=4, max_append=w.D)
    # start from partly filled, ragged histories so the 200 steps end near capacity
    start = 1200 + (np.arange(w.P) * 37) % 500
    st = run_protocol(pair, tokens, lps, k, steps=200, warm=0, start_lens=start, check_every=10)
    assert st["steps"] == 200


@pytest.mark.parametrize("fill", [0.3, 0.97])
def test_config4_sampled_steps(fill):
    w = synth.WORKLOADS[4]
    tokens, lps = synth.make_streams(w)
    for k in (1, 3, 5):
        pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, B=4, Ke=2, max_append=w.D)
        start = (int(w.L * fill) - (np.arange(w.P) * 13) % 97).astype(np.int32)
        run_protocol(pair, tokens, lps, k, steps=3, warm=0, start_lens=start, commit_in_accept=True)
        del pair


@pytest.mark.parametrize("k", [1, 2, 8])
def test_config5_sampled_steps(k):
    # heavy fan-out: k = 1 queries on frequent tokens match tens of thousands of positions
    w = synth.WORKLOADS[5]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, B=8, Ke=4, max_append=w.D)
    start = (w.L - 40 - (np.arange(w.P) * 29) % 3000).astype(np.int32)
    sample = list(range(0, w.P, 16))
    # the oracle's brute-force scan of 2M positions per query is slow: two steps, full compare on a sample of paths
    P, L, D = pair.P, pair.L, pair.D
    pair.append(tokens[:, :int(start.max())], lps[:, :int(start.max())], start, expect_status=0)
    for step in range(2):
        lens = pair.o.lengths()
        pair.build_and_compare(k, paths=sample)
        sampled, sampled_lp = synth.sampled_window(tokens, lps, lens, D + 1)
        pair.accept_and_compare(sampled, sampled_lp)
    pair.check_history()
    torch.cuda.synchronize()


# ---- fuzzy suffix matching (tolerance 1) ---------------------------------------
@pytest.mark.parametrize("seed", range(3))
@pytest.mark.parametrize("alpha,mode", [(1.0, 0), (0.5, 0), (1.0, 1)])
def test_fuzzy_dense_tiny_vocab_every_step(seed, alpha, mode):
    G, N, L, V, D, k_max = 2, 4, 48, 3 + seed % 2, 4, 4
    tokens, lps = synth.small_random(G * N, L, V, 1900 + seed)
    for k in range(1, k_max + 1):
        pair = Pair(G, N, L, V, k_max, D, alpha=alpha, mode=mode, B=4, Ke=3, eps=1)
        start = 2 + (np.arange(G * N) * 5 + seed) % 9          # some paths shorter than k
        st = run_protocol(pair, tokens, lps, k, steps=30, warm=0, start_lens=start, commit_in_accept=bool(seed % 2))
        assert st["steps"] > 0


def test_fuzzy_hand_worked_case_on_device():
    paths = [[9, 1, 2], [1, 3, 7, 5, 5], [4, 1, 2, 7, 6, 6], [8, 8, 8]]
    pair = Pair(1, 4, 10, 16, 2, 3, B=4, Ke=4, eps=1)
    tok = np.zeros((4, 6), np.int32); lp = np.full((4, 6), -0.7, np.float32)
    for i, p in enumerate(paths):
        tok[i, :len(p)] = p
    pair.append(tok, lp, np.array([len(p) for p in paths], np.int32), expect_status=0)
    t, ln = pair.build_and_compare(2)
    assert t[0, :ln[0]].tolist() == [7, 6, 6]


@pytest.mark.parametrize("k", [2, 3])
def test_fuzzy_config1_protocol(k):
    w = synth.WORKLOADS[1]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, B=8, Ke=4, max_append=w.D, eps=1)
    st = run_protocol(pair, tokens, lps, k, steps=w.steps, warm=w.k_max)
    assert st["steps"] == w.steps


@pytest.mark.parametrize("k", [1, 2, 4])
def test_fuzzy_config2_protocol(k):
    w = synth.WORKLOADS[2]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, B=8, Ke=4, max_append=w.D, eps=1)
    start = 600 + (np.arange(w.P) * 37) % 300
    st = run_protocol(pair, tokens, lps, k, steps=60, warm=0, start_lens=start, check_every=5, commit_in_accept=True)
    assert st["steps"] == 60


@pytest.mark.parametrize("seed", range(2))
@pytest.mark.parametrize("alpha,mode,pool", [(1.0, 0, 0), (0.5, 0, 0), (1.0, 1, 0), (1.0, 2, 0), (0.5, 0, 1), (1.0, 0, 2)])
def test_fuzzy_through_the_count_and_fill_passes_dense_tiny_vocab(seed, alpha, mode, pool):
    # match_capacity below P*N*L: the build does not take the single-launch kernel, and with tolerance 1 the
    # matches are counted, given slices and written by two passes of the fuzzy scan
    G, N, L, V, D, k_max = 2, 6, 64, 3 + seed, 4, 4
    tokens, lps = synth.small_random(G * N, L, V, 9500 + seed)
    for k in range(1, k_max + 1):
        pair = Pair(G, N, L, V, k_max, D, alpha=alpha, mode=mode, pool=pool, eps=1, match_capacity=4000)
        start = 2 + (np.arange(G * N) * 5 + seed) % 11          # some paths shorter than k
        st = run_protocol(pair, tokens, lps, k, steps=20, warm=0, start_lens=start, commit_in_accept=True, check_dag=False)
        assert st["steps"] > 5


def test_fuzzy_on_a_prompt_too_large_for_the_single_launch_build():
    # 40 paths of 4096 tokens: 160 Ki tokens per prompt.  Several 1024-token tiles per path, windows that reach
    # back across tile borders, ragged ends; the wide pass takes the queries with many matches
    G, N, L, V, D = 2, 40, 4096, 60, 6
    tokens, lps = synth.small_random(G * N, L, V, 9600)
    pair = Pair(G, N, L, V, 4, D, eps=1, alpha=0.5)
    lens = (L - 8 - (np.arange(G * N) * 997) % 3000).astype(np.int32)
    lens[[0, 7, 41]] = [1024, 1025, 3]
    for c in range(0, L - 8, 2048):
        part = np.clip(lens - c, 0, 2048).astype(np.int32)
        pair.g.append(t32(tokens[:, c:c + 2048], pair.dev), t32(lps[:, c:c + 2048], pair.dev), t32(part, pair.dev))
        pair.o.append(tokens[:, c:c + 2048], lps[:, c:c + 2048], part)
    assert pair.g.status() == 0
    for k in (3, 4, 2):
        pair.build_and_compare(k, check_dag=False)
    off, _ = pair.g.matches()
    assert np.diff(off.numpy()).max() > 32


def test_fuzzy_config5():
    # the paper's experimental setting (tolerance 1) on the largest workload; the oracle's edit-distance search of
    # 2M positions per query is slow, so a handful of paths are compared
    w = synth.WORKLOADS[5]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, max_append=w.D, eps=1)
    start = (w.L - 40 - (np.arange(w.P) * 29) % 3000).astype(np.int32)
    pair.append(tokens[:, :int(start.max())], lps[:, :int(start.max())], start, expect_status=0)
    for k in (4, 8):
        pair.g.build_drafts(k)
        assert pair.g.status() == 0
        off, gpos = pair.g.matches()
        off, gpos = off.numpy(), gpos.numpy()
        gt, gl = pair.g.draft_tok.cpu().numpy(), pair.g.draft_len.cpu().numpy()
        gs = pair.g.draft_score.cpu().numpy()
        for i in (0, 37, 101, 255):
            pair.o.build_path(k, i)
            assert np.array_equal(np.sort(gpos[off[i]:off[i + 1]]), pair.o.matches(i)), (k, i)
            d, sc, _ = pair.o.draft(i)
            assert gl[i] == len(d) and np.array_equal(gt[i, :len(d)], d), (k, i)
            np.testing.assert_allclose(gs[i, :len(d)], sc, rtol=harness.RTOL, atol=0)


# ---- tree and list draft pools (ablation variants) --------------------------------
@pytest.mark.parametrize("pool", [1, 2])
@pytest.mark.parametrize("seed", range(3))
@pytest.mark.parametrize("alpha", [1.0, 0.5])
def test_pools_dense_tiny_vocab_every_step(pool, seed, alpha):
    G, N, L, V, D, k_max = 2, 4, 48, 3 + seed % 2, 4, 3
    tokens, lps = synth.small_random(G * N, L, V, 2300 + seed)
    for k in range(1, k_max + 1):
        pair = Pair(G, N, L, V, k_max, D, alpha=alpha, B=4, Ke=3, pool=pool, eps=seed % 2)
        start = 3 + (np.arange(G * N) * 5 + seed) % 9
        st = run_protocol(pair, tokens, lps, k, steps=30, warm=0, start_lens=start, commit_in_accept=bool(seed % 2))
        assert st["steps"] > 0


@pytest.mark.parametrize("pool", [1, 2])
@pytest.mark.parametrize("k", [1, 3])
def test_pools_config2_protocol(pool, k):
    # k = 1 reaches a few hundred matches per query: the block path with its prefix filter
    w = synth.WORKLOADS[2]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, max_append=w.D, pool=pool)
    start = 700 + (np.arange(w.P) * 37) % 250
    st = run_protocol(pair, tokens, lps, k, steps=60, warm=0, start_lens=start, check_every=10, commit_in_accept=True)
    assert st["steps"] == 60


@pytest.mark.parametrize("pool", [1, 2])
def test_pools_config5_heavy_fan_out(pool):
    w = synth.WORKLOADS[5]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, max_append=w.D, pool=pool)
    start = (w.L - 40 - (np.arange(w.P) * 29) % 3000).astype(np.int32)
    pair.append(tokens[:, :int(start.max())], lps[:, :int(start.max())], start, expect_status=0)
    pair.build_and_compare(1, paths=list(range(0, w.P, 16)))


# ---- limits and both match paths ------------------------------------------------------
@pytest.mark.parametrize("match_capacity", [0, 60000])
def test_maximum_k_and_draft_length_odd_capacity_both_match_paths(match_capacity):
    # k_max = 16, D = 32 (the largest supported), capacity not a multiple of 4 (scalar loads),
    # 40 paths per prompt.  match_capacity = 60000 is below P*N*L, which sends the build through
    # the probe / tile-scan / dag kernels instead of the single-launch one.
    G, N, L, V, D, k_max = 2, 40, 71, 3, 32, 16
    tokens, lps = synth.small_random(G * N, L, V, 3100)
    for k in (1, 2, 7, 16):
        pair = Pair(G, N, L, V, k_max, D, B=5, Ke=3, match_capacity=match_capacity, alpha=0.5)
        start = 20 + (np.arange(G * N) * 7) % 40
        st = run_protocol(pair, tokens, lps, k, steps=6, warm=0, start_lens=start, commit_in_accept=True)
        assert st["steps"] == 6


def test_one_path_per_prompt_never_matches():
    pair = Pair(3, 1, 32, 4, 2, 4)
    tokens, lps = synth.small_random(3, 32, 4, 77)
    pair.append(tokens[:, :20], lps[:, :20], np.full(3, 20, np.int32), expect_status=0)
    _, ln = pair.build_and_compare(1)
    assert ln.sum() == 0


def test_many_paths_per_prompt():
    # 300 paths in one prompt: the per-prompt shared tables of the kernels are sized for 1024
    G, N, L, V, D = 1, 300, 32, 6, 4
    tokens, lps = synth.small_random(N, L, V, 91)
    pair = Pair(G, N, L, V, 3, D, B=4, Ke=2)
    pair.append(tokens[:, :28], lps[:, :28], (10 + np.arange(N) % 18).astype(np.int32), expect_status=0)
    for k in (1, 2, 3):
        pair.build_and_compare(k, paths=list(range(0, N, 7)))


def test_repeated_builds_are_bit_identical():
    # sums are integers and ties have a rule, so atomics and scheduling must not show in any output
    w = synth.WORKLOADS[3]
    tokens, lps = synth.make_streams(w)
    from paper_2503_05330_b200 import binding
    s = binding.Sdms(w.G, w.N, w.L, w.V, w.k_max, w.D, B=8, Ke=4)
    dev = s.device
    n = 1500
    s.append(harness.t32(tokens[:, :n], dev), harness.t32(lps[:, :n], dev),
             harness.t32((n - (np.arange(w.P) * 11) % 200).astype(np.int32), dev))
    for k in (1, 3):
        snaps = []
        for _ in range(3):
            s.build_drafts(k)
            off, gpos = s.matches()
            off = off.numpy(); gpos = gpos.numpy()
            srt = np.concatenate([np.sort(gpos[off[i]:off[i + 1]]) for i in range(w.P)]) if len(gpos) else gpos
            dag = s.dag()
            snaps.append([s.draft_tok.cpu().numpy().copy(), s.draft_len.cpu().numpy().copy(),
                          s.draft_score.cpu().numpy().copy(), s.draft_edge_w.cpu().numpy().copy(), off, srt]
                         + [dag[key] for key in sorted(dag)])
        for other in snaps[1:]:
            for a, b in zip(snaps[0], other):
                assert np.array_equal(a, b)
    assert s.status() == 0


# ---- suffix length with back-off ------------------------------------------------------------
@pytest.mark.parametrize("eps", [0, 1])
def test_backoff_picks_the_longest_matching_suffix(eps):
    w = synth.WORKLOADS[2]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, max_append=w.D, eps=eps)
    lens = (500 + (np.arange(w.P) * 37) % 400).astype(np.int32)
    pair.append(tokens[:, :int(lens.max())], lps[:, :int(lens.max())], lens, expect_status=0)
    seen = set()
    for step in range(25):
        lens = pair.o.lengths()
        _, ln, used = pair.backoff_and_compare(w.k_max)
        seen |= set(used.tolist())
        sampled, sampled_lp = synth.sampled_window(tokens, lps, lens, w.D + 1)
        pair.accept_and_compare(sampled, sampled_lp)
    assert len(seen) >= 3                      # different paths really end up with different k
    pair.check_history()


def test_backoff_dense_tiny_vocab_and_short_paths():
    G, N, L, V, D, k_max = 2, 4, 40, 3, 4, 4
    tokens, lps = synth.small_random(G * N, L, V, 4100)
    pair = Pair(G, N, L, V, k_max, D)
    pair.append(tokens[:, :12], lps[:, :12], np.array([12, 1, 2, 3, 0, 7, 12, 5], np.int32), expect_status=0)
    for k_hi in (4, 2, 1):
        pair.backoff_and_compare(k_hi)


# ---- the whole decode step in one call -------------------------------------------------------
@pytest.mark.parametrize("seed", range(3))
@pytest.mark.parametrize("alpha,mode,pool,eps", [(1.0, 0, 0, 0), (0.5, 0, 0, 0), (1.0, 1, 0, 0), (0.5, 0, 1, 0),
                                                 (1.0, 0, 2, 0), (0.5, 0, 0, 1)])
def test_step_dense_tiny_vocab(seed, alpha, mode, pool, eps):
    G, N, L, V, D, k_max = 3, 4, 48, 3 + seed % 2, 4, 3
    tokens, lps = synth.small_random(G * N, L, V, 5200 + seed)
    pair = Pair(G, N, L, V, k_max, D, alpha=alpha, mode=mode, eps=eps, pool=pool, max_append=D - seed % 2)
    assert pair.g.step_is_single_launch()
    start = 3 + (np.arange(G * N) * 5 + seed) % 9
    st = harness.run_step_protocol(pair, tokens, lps, [1, 3, 2], steps=40, warm=0, start_lens=start)
    assert st["steps"] > 5


@pytest.mark.parametrize("wid", [1, 2])
def test_step_config_full_protocol(wid):
    w = synth.WORKLOADS[wid]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, max_append=w.D)
    assert pair.g.step_is_single_launch()
    st = harness.run_step_protocol(pair, tokens, lps, list(range(w.k_max, 0, -1)), steps=w.steps, warm=w.k_max,
                                   check_matches=False)
    assert st["steps"] > 40 and st["accepted"] > 0
    from paper_2503_05330_b200 import binding
    lens = pair.o.lengths()
    sampled, sampled_lp = synth.sampled_window(tokens, lps, lens, w.D + 1)
    n0 = binding.sdms_launch_count(pair.g.ctx)
    pair.g.step(2, harness.t32(sampled, pair.dev), harness.t32(sampled_lp, pair.dev))
    assert binding.sdms_launch_count(pair.g.ctx) == n0 + 1


def test_step_many_prompts_ragged():
    # twelve prompts of eight paths: twelve clusters resident at once, one launch per step
    w = synth.WORKLOADS[4]
    tokens, lps = synth.make_streams(w)
    G, N = 12, 8
    tokens = np.ascontiguousarray(tokens.reshape(w.G, w.N, w.L)[:G, :N].reshape(G * N, w.L))
    lps = np.ascontiguousarray(lps.reshape(w.G, w.N, w.L)[:G, :N].reshape(G * N, w.L))
    pair = Pair(G, N, w.L, w.V, w.k_max, w.D, max_append=w.D)
    assert pair.g.step_is_single_launch()
    start = (int(w.L * 0.98) - (np.arange(G * N) * 13) % 97).astype(np.int32)
    st = harness.run_step_protocol(pair, tokens, lps, [5, 1, 3], steps=12, warm=0, start_lens=start,
                                   check_matches=False)
    assert st["steps"] == 12                   # runs into full paths: those stop drafting and committing


def test_step_of_more_clusters_than_the_device_holds_takes_separate_launches():
    w = synth.WORKLOADS[4]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, max_append=w.D)
    assert not pair.g.step_is_single_launch()
    start = (int(w.L * 0.98) - (np.arange(w.P) * 13) % 97).astype(np.int32)
    st = harness.run_step_protocol(pair, tokens, lps, [5, 1, 3], steps=12, warm=0, start_lens=start,
                                   check_matches=False)
    assert st["steps"] == 12


def test_step_falls_back_to_separate_launches_for_wide_prompts():
    G, N, L, V, D, k_max = 1, 24, 64, 5, 4, 3
    tokens, lps = synth.small_random(G * N, L, V, 77)
    pair = Pair(G, N, L, V, k_max, D)
    assert not pair.g.step_is_single_launch()
    st = harness.run_step_protocol(pair, tokens, lps, [2, 1, 3], steps=20, warm=4)
    assert st["steps"] > 5


# ---- best-path search (search mode 2) --------------------------------------------------------
@pytest.mark.parametrize("seed", range(4))
@pytest.mark.parametrize("alpha,eps", [(1.0, 0), (0.5, 0), (0.0, 0), (1.0, 1)])
def test_best_path_dense_small_vocab_every_step(seed, alpha, eps):
    G, N, L, V, D, k_max = 2, 5, 56, 4 + seed, 6, 3
    tokens, lps = synth.small_random(G * N, L, V, 6100 + seed)
    for k in (1, 2):
        pair = Pair(G, N, L, V, k_max, D, alpha=alpha, mode=2, eps=eps)
        start = 4 + (np.arange(G * N) * 5 + seed) % 9
        st = run_protocol(pair, tokens, lps, k, steps=30, warm=0, start_lens=start, commit_in_accept=bool(seed % 2))
        assert st["steps"] > 5


def test_best_path_through_the_single_launch_step():
    G, N, L, V, D, k_max = 2, 6, 64, 6, 6, 3
    tokens, lps = synth.small_random(G * N, L, V, 6200)
    pair = Pair(G, N, L, V, k_max, D, alpha=1.0, mode=2)
    st = harness.run_step_protocol(pair, tokens, lps, [2, 1, 3], steps=40, warm=4)
    assert st["steps"] > 5


def best_path_fits(M, D):
    cap = 64
    while cap <= M:
        cap *= 2
    return ((2 * M * D + 1) & ~1) + D * 9 * cap <= 2 * 8192 + 8 * 1024


@pytest.mark.parametrize("table_area", [True, False])
def test_best_path_config2_heavy_queries_and_the_fallback_without_a_table_area(table_area):
    # k = 1 queries on frequent tokens find more matches than the best-path tables in shared memory hold: those
    # paths are searched over tables in the workspace's table area.  Without one (wide_table_bytes = -1) they get
    # the greedy draft and the status word says so; every other path the best path
    from oracle import Oracle
    w = synth.WORKLOADS[2]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, mode=2, max_append=w.D, wide_table_bytes=0 if table_area else -1)
    greedy = Oracle(w.G, w.N, w.L, w.V, w.D, alpha=1.0, mode=0)
    n = 1000
    lens = (n - (np.arange(w.P) * 13) % 97).astype(np.int32)
    pair.append(tokens[:, :n], lps[:, :n], lens, expect_status=0)
    greedy.append(tokens[:, :n], lps[:, :n], lens)
    fell_back = 0
    for k in (1, 2, 3, 4, 1):
        pair.o.build_all(k, nthreads=8)
        greedy.build_all(k, nthreads=8)
        pair.g.build_drafts(k)
        status = pair.g.status()
        gt, gl = pair.g.draft_tok.cpu().numpy(), pair.g.draft_len.cpu().numpy()
        gs = pair.g.draft_score.cpu().numpy()
        heavy = 0
        for i in range(w.P):
            M = len(pair.o.matches(i))
            src = pair.o if table_area or best_path_fits(M, w.D) else greedy
            heavy += not best_path_fits(M, w.D)
            d, sc, _ = src.draft(i)
            assert gl[i] == len(d) and np.array_equal(gt[i, :len(d)], d), (k, i, M)
            np.testing.assert_allclose(gs[i, :len(d)], sc, rtol=harness.RTOL, atol=0)
        assert status == (0x40 if heavy and not table_area else 0), (k, heavy, status)
        fell_back += heavy
        lens = pair.o.lengths()
        sampled, sampled_lp = synth.sampled_window(tokens, lps, lens, w.D + 1)
        tok, ln, _, _ = pair.o.drafts()
        pair.o.accept_commit(tok, ln, sampled, sampled_lp, w.D)
        greedy.accept_commit(tok, ln, sampled, sampled_lp, w.D)
        # the library commits its own drafts, which differ from the oracle's on the fallback paths:
        # feed it the oracle's instead so that both histories stay the same
        pair.g.draft_tok.copy_(torch.from_numpy(tok)); pair.g.draft_len.copy_(torch.from_numpy(ln))
        pair.g.accept(harness.t32(sampled, pair.dev), harness.t32(sampled_lp, pair.dev))
        assert pair.g.status() == 0
    pair.check_history()
    assert fell_back > 0


# ---- sliding window: runs longer than the capacity -------------------------------------------
@pytest.mark.parametrize("use_step", [False, True])
@pytest.mark.parametrize("eps", [0, 1])
def test_windowed_run_outlives_the_capacity(use_step, eps):
    G, N, L, V, D, k_max = 2, 4, 64, 5, 4, 3
    tokens, lps = synth.small_random(G * N, 4 * L, V, 9100 + eps)
    pair = Pair(G, N, L, V, k_max, D, alpha=0.5, eps=eps)
    trims = harness.run_windowed_protocol(pair, tokens, lps, [2, 1, 3], steps=90, warm=6, keep=L // 2, use_step=use_step)
    assert trims >= 2 * G * N // 2                    # every path has been trimmed, most of them twice


def test_trim_config2_then_steps_agree():
    w = synth.WORKLOADS[2]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, max_append=w.D)
    n = 1000
    lens = (n - (np.arange(w.P) * 13) % 97).astype(np.int32)
    pair.append(tokens[:, :n], lps[:, :n], lens, expect_status=0)
    keep = np.where(np.arange(w.P) % 3 == 0, w.L, 300 + 20 * np.arange(w.P)).astype(np.int32)   # some untouched
    pair.trim(keep)
    pair.check_history()
    for k in (1, 2, 4):
        pair.build_and_compare(k, check_dag=False)
    assert pair.trim(np.full(w.P, -1, np.int32)) == 0x01   # rejected, nothing changes
    pair.build_and_compare(3, check_dag=False)


# ---- zero-copy: per-step arrays in page-locked host memory -----------------------------------
def test_step_with_host_mapped_buffers():
    from paper_2503_05330_b200 import binding
    w = synth.WORKLOADS[1]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, max_append=w.D, host_io=True)
    assert not pair.g.results.is_cuda and pair.g.results.is_pinned()
    lens = pair.o.lengths()
    pair.append(tokens[:, :w.k_max], lps[:, :w.k_max], np.full(w.P, w.k_max, np.int32), expect_status=0)
    pair.build_and_compare(1, check_dag=False)
    for step in range(40):
        lens = pair.o.lengths()
        k = 1 + step % w.k_max
        sampled, sampled_lp = synth.sampled_window(tokens, lps, lens, w.D + 1)
        tok, ln, _, _ = pair.o.drafts()
        tau_o, st_o = pair.o.accept_commit(tok, ln, sampled, sampled_lp, w.D)
        pair.o.build_all(k)
        pair.g.sampled_in.copy_(torch.from_numpy(sampled))                 # host to host
        pair.g.sampled_lp_in.copy_(torch.from_numpy(sampled_lp))
        pair.g.step(k, pair.g.sampled_in, pair.g.sampled_lp_in)
        assert pair.g.status() == st_o                                      # waits for the stream
        tok, ln, _, _ = pair.o.drafts()
        assert np.array_equal(pair.g.accept_len.numpy(), tau_o)
        assert np.array_equal(pair.g.draft_len.numpy(), ln) and np.array_equal(pair.g.draft_tok.numpy(), tok)
    pair.check_history()
    # memory the device cannot see is refused before any launch
    with pytest.raises(binding.SdmsError):
        binding.sdms_host_pointer(torch.zeros(8, dtype=torch.int32))


def test_tile_scan_with_more_matches_per_tile_than_its_buffer_holds():
    # two-token alphabet, k = 1: half of a tile's 1024 positions match each of a dozen queries, far more
    # than the scanning CTA can collect; match_capacity below P*N*L selects the probe / tile-scan / dag kernels
    G, N, L, V, D = 1, 12, 1024, 2, 3
    tokens, lps = synth.small_random(G * N, L, V, 4242)
    pair = Pair(G, N, L, V, 2, D, match_capacity=120000)
    lens = (1000 - (np.arange(N) * 37) % 300).astype(np.int32)
    pair.append(tokens[:, :1000], lps[:, :1000], lens, expect_status=0)
    for k in (1, 2):
        pair.build_and_compare(k, check_dag=False)
    assert (pair.g.query_modes() == 2).all()


@pytest.mark.parametrize("match_capacity", [0, 400000])
def test_heavy_query_with_wide_fan_out_in_every_layer(match_capacity):
    # one token A at every third position: ~2700 matches per path and more than 5461 per query, so the DAG is
    # aggregated from candidates that are not staged.  A is followed by B half of the time, else by one of
    # 3000 tokens, and B by one of 3000 tokens: the first layer and the layer after B have more distinct
    # nodes than one table pass holds (the layer is redone with more residue classes), both through the
    # single-launch build and (match_capacity below P*N*L) through the probe / scan / dag kernels.
    G, N, L, V, D = 1, 8, 8192, 4000, 4
    rng = np.random.default_rng(5330)
    tokens = rng.integers(10, 3010, size=(G * N, L)).astype(np.int32)
    tokens[:, 0::3] = 1                                        # A
    after = tokens[:, 1::3]
    after[rng.random(after.shape) < 0.5] = 2                   # B
    lps = (-rng.exponential(0.5, size=tokens.shape)).astype(np.float32)
    pair = Pair(G, N, L, V, 2, D, match_capacity=match_capacity)
    lens = np.array([8101, 7900, 8002, 7603, 8176, 8050, 7999, 8182], np.int32)   # all end in A (position % 3 == 0)
    assert ((lens - 1) % 3 == 0).all()
    for c in range(0, L - 8, 2048):
        part = np.clip(lens - c, 0, 2048).astype(np.int32)
        pair.g.append(t32(tokens[:, c:c + 2048], pair.dev), t32(lps[:, c:c + 2048], pair.dev), t32(part, pair.dev))
        pair.o.append(tokens[:, c:c + 2048], lps[:, c:c + 2048], part)
    assert pair.g.status() == 0
    pair.build_and_compare(1, check_dag=False)
    off, _ = pair.g.matches()
    assert np.diff(off.numpy()).min() > 5461
    pair.build_and_compare(2, check_dag=False)


def test_heavy_query_whose_successor_claims_give_up_and_the_layer_is_redone():
    # More than 5461 matches per query again (candidates not staged; the kernel keeps a 16-bit tag of every
    # candidate's previous token).  A is followed by B half of the time, and B by one of 150 tokens chosen so that
    # they all hash to four neighbouring slots of the kernel's 1024-slot node table: claiming the successors of B
    # needs runs of more than 64 probes although the table is nearly empty, so the pass is given up after it has
    # gone over every candidate and the layer is done again with two residue classes.  The second attempt must
    # still find every successor of B.
    G, N, L, V, D = 1, 8, 8192, 1 << 20, 4
    ids = np.arange(10, V, dtype=np.uint64)
    slot = ((ids * np.uint64(2654435761)) & np.uint64(0xFFFFFFFF)) >> np.uint64(22)
    crowd = ids[(slot >= 500) & (slot < 504)][:150].astype(np.int32)
    assert len(crowd) == 150
    rng = np.random.default_rng(5331)
    tokens = rng.integers(10, 3010, size=(G * N, L)).astype(np.int32)
    tokens[:, 0::3] = 1                                        # A
    after = tokens[:, 1::3]
    is_b = rng.random(after.shape) < 0.5
    after[is_b] = 2                                            # B
    third = tokens[:, 2::3]
    nb = min(after.shape[1], third.shape[1])
    pick = crowd[rng.integers(0, len(crowd), size=third.shape)]
    third[:, :nb] = np.where(is_b[:, :nb], pick[:, :nb], third[:, :nb])
    lps = (-rng.exponential(0.5, size=tokens.shape)).astype(np.float32)
    pair = Pair(G, N, L, V, 2, D)
    lens = np.array([8101, 7900, 8002, 7603, 8176, 8050, 7999, 8182], np.int32)   # all end in A
    assert ((lens - 1) % 3 == 0).all()
    for c in range(0, L - 8, 2048):
        part = np.clip(lens - c, 0, 2048).astype(np.int32)
        pair.g.append(t32(tokens[:, c:c + 2048], pair.dev), t32(lps[:, c:c + 2048], pair.dev), t32(part, pair.dev))
        pair.o.append(tokens[:, c:c + 2048], lps[:, c:c + 2048], part)
    assert pair.g.status() == 0
    tok, ln = pair.build_and_compare(1, check_dag=False)
    off, _ = pair.g.matches()
    assert np.diff(off.numpy()).min() > 5461
    assert (ln == D).all() and (tok[:, 0] == 2).all() and np.isin(tok[:, 1], crowd).all()


def test_streaming_tile_scan_on_a_store_of_many_tiles():
    # more 1024-token tiles than the one-tile-per-CTA form launches: the scan streams its tiles through
    # shared-memory stages.  Ragged lengths: empty paths, paths that end inside their first tile, on a
    # tile boundary and one token past it, lengths that are not multiples of four.
    G, N, L, V, D = 5, 128, 8192, 300, 3
    assert G * N * (L // 1024) > 148 * 8 * 4
    tokens, lps = synth.small_random(G * N, L, V, 777)
    pair = Pair(G, N, L, V, 2, D)
    lens = (L - 8 - (np.arange(G * N) * 997) % 7000).astype(np.int32)
    lens[[0, 5, 130, 131, 200, 300, 301, 639]] = [0, 3, 1024, 1025, 4098, 2047, 1, 8184]
    for c in range(0, L - 8, 2048):                      # prefill in chunks
        part = np.clip(lens - c, 0, 2048).astype(np.int32)
        pair.g.append(t32(tokens[:, c:c + 2048], pair.dev), t32(lps[:, c:c + 2048], pair.dev), t32(part, pair.dev))
        pair.o.append(tokens[:, c:c + 2048], lps[:, c:c + 2048], part)
    assert pair.g.status() == 0
    for k in (1, 2):
        pair.build_and_compare(k, check_dag=False)
        assert (pair.g.query_modes() == 2).sum() > G * N // 2


@pytest.mark.parametrize("mode,pool", [(0, 0), (1, 0), (2, 0), (0, 1), (0, 2)])
def test_search_modes_and_pools_through_the_probe_scan_dag_kernels(mode, pool):
    # match_capacity below P*N*L: the build takes the three-kernel path, where the searches and
    # pools run inside dag_kernel instead of the single-launch kernel
    G, N, L, V, D, k_max = 2, 6, 64, 4, 5, 3
    tokens, lps = synth.small_random(G * N, L, V, 9300 + 10 * mode + pool)
    for k in (1, 2):
        pair = Pair(G, N, L, V, k_max, D, alpha=0.5, mode=mode, pool=pool, match_capacity=3000)
        start = 6 + (np.arange(G * N) * 5) % 11
        st = run_protocol(pair, tokens, lps, k, steps=25, warm=0, start_lens=start, commit_in_accept=True,
                          check_dag=False)
        assert st["steps"] > 5
        from paper_2503_05330_b200 import binding
        n0 = binding.sdms_launch_count(pair.g.ctx)
        pair.g.build_drafts(k)
        assert binding.sdms_launch_count(pair.g.ctx) == n0 + 4 + (mode == 2)   # probe, scan, dag, dag_wide (+ best paths of heavy queries)


def test_trim_on_the_three_kernel_path():
    G, N, L, V, D, k_max = 2, 6, 64, 4, 4, 3
    tokens, lps = synth.small_random(G * N, 4 * L, V, 9400)
    pair = Pair(G, N, L, V, k_max, D, match_capacity=3000)
    trims = harness.run_windowed_protocol(pair, tokens, lps, [2, 1, 3], steps=60, warm=6, keep=L // 2)
    assert trims >= G * N


@pytest.mark.parametrize("eps", [0, 1])
def test_step_with_backoff_in_one_launch(eps):
    w = synth.WORKLOADS[2]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, max_append=w.D, eps=eps)
    assert pair.g.step_is_single_launch()
    lens = (300 + (np.arange(w.P) * 37) % 400).astype(np.int32)
    pair.append(tokens[:, :int(lens.max())], lps[:, :int(lens.max())], lens, expect_status=0)
    pair.backoff_and_compare(w.k_max)
    seen = set()
    for step in range(20):
        lens = pair.o.lengths()
        sampled, sampled_lp = synth.sampled_window(tokens, lps, lens, w.D + 1)
        tok, ln, _, _ = pair.o.drafts()
        tau_o, st_o = pair.o.accept_commit(tok, ln, sampled, sampled_lp, pair.max_append)
        used = np.zeros(w.P, np.int32)                      # oracle: fixed-k builds composed per path
        for i in range(w.P):
            for k in range(w.k_max, 0, -1):
                pair.o.build_path(k, i)
                if len(pair.o.matches(i)) > 0:
                    used[i] = k
                    break
        tau_g, gt, gl, gk = pair.g.step_backoff(w.k_max, harness.t32(sampled, pair.dev), harness.t32(sampled_lp, pair.dev))
        assert pair.g.status() == st_o
        tok, ln, sc, _ = pair.o.drafts()
        assert np.array_equal(tau_g.cpu().numpy(), tau_o)
        assert np.array_equal(gk.cpu().numpy(), used)
        assert np.array_equal(gl.cpu().numpy(), ln) and np.array_equal(gt.cpu().numpy(), tok)
        np.testing.assert_allclose(pair.g.draft_score.cpu().numpy(), sc, rtol=harness.RTOL, atol=0)
        seen |= set(used.tolist())
    assert len(seen) >= 3
    pair.check_history()


# ---- optional cap on the matches per (query path, source path) --------------------------------
@pytest.mark.parametrize("seed", range(3))
@pytest.mark.parametrize("R,alpha,mode,pool,eps", [(1, 1.0, 0, 0, 0), (2, 0.5, 0, 0, 0), (3, 1.0, 1, 0, 0), (2, 1.0, 0, 1, 0),
                                                   (2, 0.5, 0, 2, 0), (2, 1.0, 0, 0, 1), (1, 1.0, 2, 0, 0)])
def test_match_cap_dense_tiny_vocab_every_step(seed, R, alpha, mode, pool, eps):
    G, N, L, V, D, k_max = 2, 4, 48, 3 + seed % 2, 4, 3
    tokens, lps = synth.small_random(G * N, L, V, 8300 + seed)
    for k in range(1, k_max + 1):
        pair = Pair(G, N, L, V, k_max, D, alpha=alpha, mode=mode, pool=pool, eps=eps, B=0 if pool else 4, Ke=3,
                    max_matches=R)
        start = 3 + (np.arange(G * N) * 5 + seed) % 9
        st = run_protocol(pair, tokens, lps, k, steps=30, warm=0, start_lens=start, commit_in_accept=bool(seed % 2))
        assert st["steps"] > 0


@pytest.mark.parametrize("R", [1, 8, 64])
def test_match_cap_config2_through_the_step(R):
    w = synth.WORKLOADS[2]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, max_append=w.D, max_matches=R)
    start = 500 + (np.arange(w.P) * 37) % 300
    st = harness.run_step_protocol(pair, tokens, lps, [1, 2, 4], steps=120, warm=0, start_lens=start, check_every=5)
    assert st["steps"] == 120


@pytest.mark.parametrize("R", [1, 8, 64])
def test_match_cap_config5_heavy_queries(R):
    # the k = 1 query with 22 938 matches keeps at most 255 * R of them
    w = synth.WORKLOADS[5]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, B=4, Ke=2, max_append=w.D, max_matches=R)
    start = (w.L - 40 - (np.arange(w.P) * 29) % 3000).astype(np.int32)
    pair.append(tokens[:, :int(start.max())], lps[:, :int(start.max())], start, expect_status=0)
    for k in (1, 2):
        pair.build_and_compare(k)
        off, _ = pair.g.matches()
        assert np.diff(off.numpy()).max() <= (w.N - 1) * R


def test_match_cap_on_the_three_kernel_path_with_more_matches_than_the_cap_in_every_path():
    G, N, L, V, D = 1, 12, 1024, 2, 3
    tokens, lps = synth.small_random(G * N, L, V, 4243)
    for R in (1, 5, 100):
        pair = Pair(G, N, L, V, 2, D, match_capacity=120000, max_matches=R, B=2, Ke=2)
        lens = (1000 - (np.arange(N) * 37) % 300).astype(np.int32)
        pair.append(tokens[:, :1000], lps[:, :1000], lens, expect_status=0)
        for k in (1, 2):
            pair.build_and_compare(k)


# ---- queries with many matches, aggregated by all SMs (probe / scan / dag / dag_wide kernels) ----
@pytest.mark.parametrize("wide_table_bytes", [0, 40 * 16 * 4096, -1])
@pytest.mark.parametrize("alpha,mode", [(1.0, 0), (0.5, 0), (1.0, 1)])
def test_wide_pass_and_its_fallbacks_agree_with_the_oracle(wide_table_bytes, alpha, mode):
    # two-token alphabet: every k = 1 query has thousands of matches and every layer two nodes; k = 3 a few
    # hundred.  Default tables hold every query; 40 * 16 * 4096 bytes hold a few and the others are aggregated
    # by their own thread block; -1 switches the pass off.
    G, N, L, V, D = 2, 12, 1024, 2, 5
    tokens, lps = synth.small_random(G * N, L, V, 4250)
    pair = Pair(G, N, L, V, 3, D, match_capacity=300000, alpha=alpha, mode=mode, wide_table_bytes=wide_table_bytes, B=2, Ke=2)
    lens = (1000 - (np.arange(G * N) * 37) % 300).astype(np.int32)
    pair.append(tokens[:, :1000], lps[:, :1000], lens, expect_status=0)
    for k in (1, 3, 2, 1):
        pair.build_and_compare(k)
        lens = pair.o.lengths()
        sampled, sampled_lp = synth.sampled_window(tokens, lps, lens, D + 1)
        pair.accept_and_compare(sampled, sampled_lp)
    pair.check_history()


def test_wide_pass_with_many_distinct_followers_and_ragged_ends():
    # vocabulary of 50 over 40 paths: k = 1 finds ~700 matches per query fanning out into all 50 tokens in every
    # layer; paths of very different lengths, so many candidates end before the last layer
    G, N, L, V, D = 3, 40, 900, 50, 16
    tokens, lps = synth.small_random(G * N, L, V, 4251)
    pair = Pair(G, N, L, V, 2, D, match_capacity=4000000, alpha=0.5)      # below P*N*L: probe / scan / dag / dag_wide
    lens = (890 - (np.arange(G * N) * 131) % 880).astype(np.int32)
    pair.append(tokens[:, :890], lps[:, :890], lens, expect_status=0)
    for k in (1, 2):
        pair.build_and_compare(k, check_dag=False)
    from paper_2503_05330_b200 import binding
    binding.sdms_profile_enable(pair.g.ctx, True)
    pair.g.build_drafts(1)
    prof = binding.sdms_profile_read(pair.g.ctx)
    assert prof["dag_wide"][1] == 1


@pytest.mark.parametrize("N,L,V,D,match_capacity", [(4, 400, 3, 32, 5000), (4, 400, 3, 10, 5000), (5, 300, 2, 3, 7000),
                                                     (24, 900, 50, 32, 400000)])
def test_wide_pass_units_split_by_layers_and_drafts_longer_than_a_batch(N, L, V, D, match_capacity):
    # few heavy queries: their chunks of 128 matches are split by layers into 2, 4 or 8 units (D = 32: eight rounds of
    # layers per thread; D = 10: three, so the last unit is short; D = 3: one, no split); many heavy queries: no split,
    # several units per CTA, and with D = 32 a thread's layers take two batches of four
    G = 1
    tokens, lps = synth.small_random(G * N, L, V, 4260 + D)
    pair = Pair(G, N, L, V, 2, D, match_capacity=match_capacity, alpha=0.5)
    n = L - 4 * (D + 1) - 4
    lens = (n - (np.arange(G * N) * 29) % (L // 3)).astype(np.int32)
    pair.append(tokens[:, :n], lps[:, :n], lens, expect_status=0)
    from paper_2503_05330_b200 import binding
    binding.sdms_profile_enable(pair.g.ctx, True)
    for k in (1, 2, 1):
        pair.build_and_compare(k, check_dag=False)
        lens = pair.o.lengths()
        sampled, sampled_lp = synth.sampled_window(tokens, lps, lens, D + 1)
        pair.accept_and_compare(sampled, sampled_lp)
    assert binding.sdms_profile_read(pair.g.ctx)["dag_wide"][1] >= 3
    pair.check_history()


# ---- several drafts per path: the B best paths of the pool ----------------------------------------
def test_beams_hand_worked_pool_on_device():
    paths = [[5, 9], [9, 1, 3, 7], [9, 2, 4, 7], [9, 2, 5, 7]]
    probs = [[.5, .5], [.5, .5, .125, .5], [.5, .25, .75, .5], [.5, .25, .5, .5]]
    pair = Pair(1, 4, 8, 10, 2, 2, mode=2, max_beams=4)
    tok = np.zeros((4, 4), np.int32); lp = np.zeros((4, 4), np.float32)
    for i, p in enumerate(paths):
        tok[i, :len(p)] = p
        lp[i, :len(p)] = np.log(np.array(probs[i]))
    pair.append(tok, lp, np.array([len(p) for p in paths], np.int32), expect_status=0)
    pair.build_and_compare(1, check_dag=False)
    t, ln, val = pair.beams_and_compare(3)
    assert [t[0, b, :ln[0, b]].tolist() for b in range(3)] == [[2, 4], [2, 5], [1, 3]]
    np.testing.assert_allclose(val[0], [1.25, 1.0, .625], rtol=1e-6)
    pair.beams_and_compare(4)


@pytest.mark.parametrize("seed", range(4))
@pytest.mark.parametrize("alpha,eps,mode", [(1.0, 0, 0), (0.5, 0, 2), (0.0, 0, 0), (1.0, 1, 2)])
def test_beams_dense_small_vocab_every_step(seed, alpha, eps, mode):
    G, N, L, V, D, k_max = 2, 5, 56, 3 + seed, 6, 3
    tokens, lps = synth.small_random(G * N, L, V, 6300 + seed)
    for k in (1, 2):
        pair = Pair(G, N, L, V, k_max, D, alpha=alpha, mode=mode, eps=eps, max_beams=8)
        lens = (4 + (np.arange(G * N) * 5 + seed) % 9).astype(np.int32)
        pair.append(tokens[:, :16], lps[:, :16], lens, expect_status=0)
        for step in range(25):
            lens = pair.o.lengths()
            if (lens >= L).all():
                break
            pair.build_and_compare(k, check_dag=False)
            for B in (1, 3, 8):
                pair.beams_and_compare(B)
            if mode == 2:                                  # the first beam is the best-path draft
                t, ln, _ = pair.g.beams(1)
                assert np.array_equal(ln[:, 0], pair.g.draft_len.cpu().numpy())
                assert np.array_equal(t[:, 0], pair.g.draft_tok.cpu().numpy())
            sampled, sampled_lp = synth.sampled_window(tokens, lps, lens, D + 1)
            pair.accept_and_compare(sampled, sampled_lp)


@pytest.mark.parametrize("wid,k", [(2, 1), (2, 3), (5, 1), (5, 3)])
def test_beams_on_benchmark_workloads(wid, k):
    # cfg2 k = 1: queries with more matches than the in-kernel best-path search takes; cfg5 k = 1: 22 938 matches
    w = synth.WORKLOADS[wid]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, max_append=w.D, max_beams=4)
    n = int(w.L * 0.97)
    lens = (n - (np.arange(w.P) * 13) % 97).astype(np.int32)
    pair.append(tokens[:, :n], lps[:, :n], lens, expect_status=0)
    sample = None if wid == 2 else list(range(0, w.P, 8))
    pair.build_and_compare(k, check_dag=False, paths=sample)
    pair.beams_and_compare(4, paths=sample)
    pair.beams_and_compare(1, paths=sample)


def test_beams_need_room_and_a_build():
    from paper_2503_05330_b200 import binding
    G, N, L, V, D = 1, 6, 64, 3, 4
    tokens, lps = synth.small_random(G * N, L, V, 6400)
    none = Pair(G, N, L, V, 2, D)                                          # max_beams = 0: the call is not available
    none.append(tokens[:, :40], lps[:, :40], np.full(N, 40, np.int32), expect_status=0)
    none.g.build_drafts(1)
    with pytest.raises(binding.SdmsError) as e:
        none.g.beams(1)
    assert e.value.code == binding.ERR_BAD_STATE
    small = Pair(G, N, L, V, 2, D, max_beams=2, wide_table_bytes=72 * 4 * 64 * 3)     # room for three small paths
    small.append(tokens[:, :40], lps[:, :40], np.full(N, 40, np.int32), expect_status=0)
    with pytest.raises(binding.SdmsError):
        small.g.beams(2)                                                   # nothing built yet
    small.g.build_drafts(2)
    with pytest.raises(binding.SdmsError):
        small.g.beams(3)                                                   # more than max_beams
    tok, ln, _ = small.g.beams(2)
    assert small.g.status() == binding.STATUS_TABLES_FULL
    small.o.build_all(2)
    served = [i for i in range(N) if ln[i, 0] > 0]
    assert 0 < len(served) < N
    for i in served:                                                       # those that found room are right
        want, _ = small.o.beams(i, 2)
        assert [tok[i, b, :ln[i, b]].tolist() for b in range(2) if ln[i, b] > 0] == want


def test_best_path_with_heavy_queries_through_build_and_step():
    # cfg2 at k = 1: many paths have more matches than the shared-memory search takes; drafts, scores and edge
    # weights of all paths against the oracle, through sdms_build_drafts and through the one-call step
    w = synth.WORKLOADS[2]
    tokens, lps = synth.make_streams(w)
    start = 850 + (np.arange(w.P) * 37) % 100
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, mode=2, max_append=w.D)
    st = run_protocol(pair, tokens, lps, 1, steps=25, warm=0, start_lens=start, commit_in_accept=True, check_dag=False)
    assert st["steps"] == 25
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, mode=2, max_append=w.D)
    st = harness.run_step_protocol(pair, tokens, lps, [1, 2], steps=25, warm=0, start_lens=start, check_every=5)
    assert st["steps"] == 25


# ---- an index that keeps tables for the shortest n-grams only ------------------------------------
@pytest.mark.parametrize("index_max_n", [1, 2])
@pytest.mark.parametrize("match_capacity", [0, 3000])
def test_short_index_dense_tiny_vocab_every_step(index_max_n, match_capacity):
    # queries longer than the longest indexed n-gram look up their last index_max_n tokens and verify (or scan for)
    # all k; both through the single-launch build and (match_capacity below P*N*L) the probe / scan / dag kernels
    G, N, L, V, D, k_max = 2, 6, 64, 4, 4, 4
    tokens, lps = synth.small_random(G * N, L, V, 9700 + index_max_n)
    for k in range(1, k_max + 1):
        pair = Pair(G, N, L, V, k_max, D, alpha=0.5, B=3, Ke=2, index_max_n=index_max_n, match_capacity=match_capacity)
        start = 3 + (np.arange(G * N) * 5) % 11
        st = run_protocol(pair, tokens, lps, k, steps=25, warm=0, start_lens=start, commit_in_accept=True)
        assert st["steps"] > 5


@pytest.mark.parametrize("wid,index_max_n", [(2, 2), (2, 1), (5, 2)])
def test_short_index_on_benchmark_workloads(wid, index_max_n):
    w = synth.WORKLOADS[wid]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, max_append=w.D, index_max_n=index_max_n)
    if wid == 2:
        start = 600 + (np.arange(w.P) * 37) % 300
        st = harness.run_step_protocol(pair, tokens, lps, [4, 1, 3, 2], steps=100, warm=0, start_lens=start, check_every=5)
        assert st["steps"] == 100
        assert (pair.g.query_modes() > 0).any()
    else:
        start = (w.L - 40 - (np.arange(w.P) * 29) % 3000).astype(np.int32)
        pair.append(tokens[:, :int(start.max())], lps[:, :int(start.max())], start, expect_status=0)
        for k in (3, 8):
            pair.build_and_compare(k, check_dag=False, paths=list(range(0, w.P, 8)))
        pair.trim(np.full(w.P, 4000, np.int32))                 # the rebuilt index has the same few tables
        pair.build_and_compare(4, check_dag=False, paths=list(range(0, w.P, 8)))


# ---- back-off of the suffix length on prompts that take the probe / scan / dag kernels ------------
@pytest.mark.parametrize("eps,L,match_capacity", [(0, 64, 3000), (1, 128, 9000)])
def test_backoff_by_rounds_dense_tiny_vocab(eps, L, match_capacity):
    # (with tolerance 1 a path that gets down to k = 1 matches every position: the list must hold N * L per path)
    G, N, V, D, k_max = 2, 6, 4, 4, 4
    tokens, lps = synth.small_random(G * N, L, V, 9800)
    pair = Pair(G, N, L, V, k_max, D, alpha=0.5, match_capacity=match_capacity, eps=eps)
    start = (2 + (np.arange(G * N) * 5) % 11).astype(np.int32)
    pair.append(tokens[:, :16], lps[:, :16], start, expect_status=0)
    seen = set()
    for step in range(20):
        lens = pair.o.lengths()
        _, _, used = pair.backoff_and_compare(k_max if step % 3 else 2)
        seen |= set(used.tolist())
        sampled, sampled_lp = synth.sampled_window(tokens, lps, lens, D + 1)
        pair.accept_and_compare(sampled, sampled_lp)
        pair.build_and_compare(1 + step % k_max, check_dag=False)      # an ordinary build in between finds a clean state
    assert len(seen) >= (3 if eps == 0 else 2)
    pair.check_history()


def test_backoff_by_rounds_with_tolerance_on_a_prompt_too_large_for_one_launch():
    # 40 paths x 4096 tokens (more than 128 Ki tokens): count / hand out / fill / dag (/ wide) once per suffix length
    G, N, L, V, D, k_max = 1, 40, 4096, 60, 6, 4
    tokens, lps = synth.small_random(G * N, L, V, 9810)
    pair = Pair(G, N, L, V, k_max, D, eps=1)
    lens = (4000 - (np.arange(G * N) * 61) % 1500).astype(np.int32)
    pair.append(tokens[:, :4000], lps[:, :4000], lens, expect_status=0)
    _, _, used = pair.backoff_and_compare(k_max)
    assert len(set(used.tolist())) >= 2 and used.min() >= 2
    sampled, sampled_lp = synth.sampled_window(tokens, lps, pair.o.lengths(), D + 1)
    pair.accept_and_compare(sampled, sampled_lp)
    pair.backoff_and_compare(3)
    pair.build_and_compare(2, check_dag=False)                          # an ordinary build afterwards finds a clean state


def test_backoff_by_rounds_config5():
    w = synth.WORKLOADS[5]
    tokens, lps = synth.make_streams(w)
    pair = Pair(w.G, w.N, w.L, w.V, w.k_max, w.D, max_append=w.D)
    start = (w.L - 40 - (np.arange(w.P) * 29) % 3000).astype(np.int32)
    pair.append(tokens[:, :int(start.max())], lps[:, :int(start.max())], start, expect_status=0)
    pair.g.build_drafts_backoff(w.k_max)
    assert pair.g.status() == 0
    used_g = pair.g.used_k.cpu().numpy()
    gt, gl = pair.g.draft_tok.cpu().numpy(), pair.g.draft_len.cpu().numpy()
    off, gpos = pair.g.matches()
    off, gpos = off.numpy(), gpos.numpy()
    for i in range(0, w.P, 8):                                          # oracle: fixed-k builds composed per path
        used = 0
        for k in range(w.k_max, 0, -1):
            pair.o.build_path(k, i)
            if len(pair.o.matches(i)) > 0:
                used = k
                break
        assert used_g[i] == used, (i, used_g[i], used)
        d, _, _ = pair.o.draft(i)
        assert gl[i] == len(d) and np.array_equal(gt[i, :len(d)], d), i
        assert np.array_equal(np.sort(gpos[off[i]:off[i + 1]]), pair.o.matches(i)), i
    assert len(set(used_g.tolist())) >= 3


def test_a_wait_that_runs_out_sets_the_status_bit_and_leaves_the_context_usable():
    # the bounded wait of the kernels, on a count that nobody raises (about half a millisecond)
    from paper_2503_05330_b200 import binding
    G, N, L, V, D = 1, 4, 48, 3, 4
    tokens, lps = synth.small_random(G * N, L, V, 77)
    pair = Pair(G, N, L, V, 2, D)
    pair.append(tokens[:, :30], lps[:, :30], np.full(N, 30, np.int32), expect_status=0)
    binding.sdms_debug_wait_timeout(pair.g.ctx)
    assert pair.g.status() == binding.STATUS_TIMEOUT
    assert pair.g.status() == 0                      # read and cleared
    pair.build_and_compare(1, check_dag=False)       # nothing else has changed
