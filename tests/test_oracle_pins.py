"""Pins of the CPU oracle against what the paper and plain mathematics fix.

Nothing here touches the CUDA library.  Each check is chosen so that a
plausible mistake in the oracle (dropped term, off-by-one position, self match,
wrong tie rule, transposed edge) fails at least one of them.
"""
import collections
import decimal
import itertools
import json
import os
import re

import numpy as np
import pytest

import oracle
from oracle import Oracle
from paper_2503_05330_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
Q30 = 1 << 30


def load_paths(o, paths, probs=None, logprobs=None):
    """Append whole paths (ragged) in one call."""
    a_max = max(len(p) for p in paths)
    tok = np.zeros((o.P, a_max), np.int32)
    cnt = np.array([len(p) for p in paths], np.int32)
    for i, p in enumerate(paths):
        tok[i, :len(p)] = p
    if probs is not None:
        pq = np.zeros((o.P, a_max), np.int32)
        for i, p in enumerate(probs):
            pq[i, :len(p)] = [int(round(x * Q30)) for x in p]
        return o.append_fixed(tok, pq, cnt)
    lp = np.zeros((o.P, a_max), np.float32)
    for i, p in enumerate(logprobs):
        lp[i, :len(p)] = p
    return o.append(tok, lp, cnt)


# ----------------------------------------------------------------------------
# fixed-point probability
# ----------------------------------------------------------------------------
def test_prob_to_fixed_against_50_digit_decimal():
    decimal.getcontext().prec = 60
    rng = synth.Stream(99)
    lps = np.concatenate([(-8.0 * rng.uniform(1500)).astype(np.float32),
                          (-1e-3 * rng.uniform(300)).astype(np.float32),
                          np.array([-20.0, -30.0, -50.0, -1e-7, -0.6931472], np.float32)])
    for lp in lps:
        exact = (decimal.Decimal(float(lp)).exp() * Q30).to_integral_value(rounding=decimal.ROUND_HALF_EVEN)
        assert oracle.prob_to_fixed(float(lp)) == int(exact), lp


def test_prob_to_fixed_special_values():
    assert oracle.prob_to_fixed(0.0) == Q30
    assert oracle.prob_to_fixed(1.5) == Q30          # a probability cannot exceed one
    assert oracle.prob_to_fixed(float("-inf")) == 0
    assert oracle.prob_to_fixed(-100.0) == 0
    assert oracle.prob_to_fixed(float("nan")) == 0
    # monotone in the logprob
    xs = np.linspace(-12, 0, 400).astype(np.float32)
    v = [oracle.prob_to_fixed(float(x)) for x in xs]
    assert all(a <= b for a, b in zip(v, v[1:]))


def test_weight_is_eq5_in_exact_cases():
    # alpha = 1: pure probability sum; alpha = 0: pure count; alpha = 1/2: dyadic mix.
    assert oracle.weight(1.0, 3 * Q30 // 4, 2) == 0.75
    assert oracle.weight(0.0, 3 * Q30 // 4, 2) == 2.0
    assert oracle.weight(0.5, 3 * Q30 // 4, 2) == 1.375
    assert oracle.weight(0.25, Q30 // 2, 3) == 0.25 * 0.5 + 0.75 * 3


# ----------------------------------------------------------------------------
# the hand-worked example
# ----------------------------------------------------------------------------
@pytest.fixture()
def worked():
    with open(os.path.join(GOLDEN, "worked_example.json")) as f:
        return json.load(f)


def make_worked(w, alpha=None, mode=0, probs=None):
    o = Oracle(1, 3, w["capacity"], 16, w["D"], alpha=w["alpha"] if alpha is None else alpha, mode=mode)
    assert load_paths(o, w["paths"], probs=probs or w["prob"]) == 0
    return o


def test_worked_example_matches_dag_and_draft(worked):
    w = worked
    o = make_worked(w)
    o.build_path(w["k"], 0)
    L = w["capacity"]
    assert o.matches(0).tolist() == [j * L + e for j, e in w["matches"]]
    for d in (1, 2, 3):
        nodes, edges = o.layer(0, d)
        assert edges == {(u, v): (int(s * Q30), c) for u, v, s, c in w["edges"][str(d)]}
        assert nodes == {v: (int(s * Q30), c) for v, s, c in w["nodes"][str(d)]}
    tok, score, edge_w = o.draft(0)
    assert tok.tolist() == w["draft"]
    assert score.tolist() == w["draft_score"]
    assert edge_w.tolist() == w["draft_edge_w"]
    assert int(score[0] * Q30) == w["draft_S_fixed"]
    # following the heaviest out-edge instead of the heaviest node would give another draft
    assert w["heaviest_out_edge_walk"] != w["draft"]
    for i, want in w["other_queries"].items():
        o.build_path(w["k"], int(i))
        assert o.draft(int(i))[0].tolist() == want


def test_worked_example_layer_argmax_mode(worked):
    o = make_worked(worked, mode=1)
    o.build_path(worked["k"], 0)
    assert o.draft(0)[0].tolist() == worked["layer_argmax_walk"]


def test_worked_example_tie_goes_to_smaller_token(worked):
    w = worked
    probs = [list(p) for p in w["prob"]]
    pj, idx, val = w["tie_variant"]["set"]
    probs[pj][idx] = val
    o = make_worked(w, probs=probs)
    o.build_path(w["k"], 0)
    nodes, _ = o.layer(0, 1)
    assert nodes[3][0] == nodes[4][0]
    assert o.draft(0)[0][0] == w["tie_variant"]["first_token"]


def test_worked_example_alpha_half(worked):
    w = worked
    o = make_worked(w, alpha=w["alpha_half_variant"]["alpha"])
    o.build_path(w["k"], 0)
    nodes, _ = o.layer(0, 1)
    assert oracle.weight(0.5, *nodes[3]) == w["alpha_half_variant"]["W_1_3"]
    assert oracle.weight(0.5, *nodes[4]) == w["alpha_half_variant"]["W_1_4"]
    assert o.draft(0)[1][0] == w["alpha_half_variant"]["W_1_3"]


def test_worked_example_accept_and_commit(worked):
    w = worked
    o = make_worked(w)
    o.build_all(w["k"])
    tok, ln, _, _ = o.drafts()
    D = w["D"]
    sampled = np.full((3, D + 1), 15, np.int32)
    sampled[0] = w["accept"]["sampled"]
    lens0 = o.lengths().copy()
    tau, st = o.accept_commit(tok, ln, sampled, np.full((3, D + 1), -0.5, np.float32), D + 1)
    assert st == 0
    assert tau[0] == w["accept"]["tau"]
    h, _ = o.history(0)
    assert h[lens0[0]:].tolist() == w["accept"]["committed"]
    # a path whose draft is rejected outright still receives the model's own token
    assert tau[2] == 0 and o.lengths()[2] == lens0[2] + 1


def test_reconverging_branches_merge_into_one_node():
    # two candidates diverge at layer 1 and meet again at layer 2 in the same
    # token: one node there, two in-edges, its score the sum over both.
    paths = [[9, 1], [1, 2, 7, 5], [1, 3, 7, 5], [8, 8]]
    probs = [[0.5, 0.5], [0.5, 0.5, 0.25, 0.5], [0.5, 0.25, 0.5, 0.5], [0.5, 0.5]]
    o = Oracle(1, 4, 8, 16, 3)
    load_paths(o, paths, probs=probs)
    o.build_path(1, 0)
    nodes, edges = o.layer(0, 2)
    assert nodes == {7: (int(0.75 * Q30), 2)}
    assert edges == {(2, 7): (Q30 // 4, 1), (3, 7): (Q30 // 2, 1)}
    nodes3, edges3 = o.layer(0, 3)
    assert edges3 == {(7, 5): (Q30, 2)}
    assert o.draft(0)[0].tolist() == [2, 7, 5]


# ----------------------------------------------------------------------------
# the match set (Eq. 3)
# ----------------------------------------------------------------------------
def regex_matches(tokens, lens, N, L, i, k):
    """Eq. 3 by overlapping regex search on byte strings (tokens < 256)."""
    q = bytes(tokens[i, lens[i] - k:lens[i]].tolist())
    g = i // N
    out = []
    for j in range(g * N, (g + 1) * N):
        if j == i:
            continue
        hay = bytes(tokens[j, :lens[j]].tolist())
        for m in re.finditer(b"(?=" + re.escape(q) + b")", hay):
            e = m.start() + k - 1
            if e <= lens[j] - 2:
                out.append(j * L + e)
    return sorted(out)


@pytest.mark.parametrize("seed", range(6))
def test_match_set_equals_regex_search(seed):
    G, N, L, V = 2, 4, 24, 3 + seed % 2
    tokens, lps = synth.small_random(G * N, L, V, seed)
    rng = synth.Stream(1000 + seed)
    lens = (3 + rng.uniform(G * N) * (L - 4)).astype(np.int32)     # ragged, none full
    o = Oracle(G, N, L, V, 4)
    o.append(tokens, lps, lens)
    for k in (1, 2, 3):
        o.build_all(k)
        for i in range(G * N):
            assert o.matches(i).tolist() == regex_matches(tokens, lens, N, L, i, k), (seed, k, i)


def test_k1_is_numpy_where():
    tokens, lps = synth.small_random(4, 40, 5, 7)
    lens = np.array([40 - 1, 33, 17, 25], np.int32)
    o = Oracle(1, 4, 40, 5, 3)
    o.append(tokens, lps, lens)
    o.build_all(1)
    for i in range(4):
        want = []
        for j in range(4):
            if j != i:
                e = np.where(tokens[j, :lens[j] - 1] == tokens[i, lens[i] - 1])[0]
                want += (j * 40 + e).tolist()
        assert o.matches(i).tolist() == want


def test_all_equal_tokens_closed_form_and_disjoint_alphabets():
    # every window of a constant path matches: len_j - k positions per other path
    L, N = 32, 3
    lens = np.array([10, 20, 31], np.int32)
    o = Oracle(1, N, L, 4, 4)
    o.append(np.full((N, L), 2, np.int32), np.full((N, L), -0.1, np.float32), lens)
    for k in (1, 2, 5):
        o.build_all(k)
        for i in range(N):
            assert len(o.matches(i)) == sum(lens[j] - k for j in range(N) if j != i)
    # paths over disjoint alphabets never match
    tok = np.stack([np.arange(L) % 3, 3 + np.arange(L) % 3, 6 + np.arange(L) % 3]).astype(np.int32)
    o = Oracle(1, N, L, 9, 4)
    o.append(tok, np.full((N, L), -0.1, np.float32), lens)
    o.build_all(1)
    assert all(len(o.matches(i)) == 0 for i in range(N))


def test_matching_never_crosses_prompts_and_needs_k_tokens():
    tok = np.tile(np.array([1, 2, 3, 1, 2, 3, 1, 2], np.int32), (4, 1))
    o = Oracle(2, 2, 16, 4, 2)
    o.append(tok, np.full(tok.shape, -0.2, np.float32), np.array([8, 8, 8, 1], np.int32))
    o.build_all(2)
    assert all(m // 16 == 1 for m in o.matches(0))       # path 0 only sees path 1
    assert all(m // 16 == 3 for m in o.matches(2))
    assert len(o.matches(3)) == 0 and o.draft(3)[0].size == 0   # one token cannot form a 2-token query


def test_full_path_builds_no_draft_but_is_still_a_source():
    tok = np.tile(np.array([1, 2, 1, 2, 1, 2, 1, 2], np.int32), (2, 1))
    o = Oracle(1, 2, 8, 4, 2)
    o.append(tok, np.full(tok.shape, -0.2, np.float32), np.array([8, 4], np.int32))
    o.build_all(1)
    assert o.draft(0)[0].size == 0              # path 0 is at capacity
    assert len(o.matches(1)) == 3               # token 2 inside the full path, last one has no follower
    assert o.draft(1)[0].tolist() == [1, 2]


# ----------------------------------------------------------------------------
# DAG aggregation (Eq. 5) - invariants and the alpha = 0 special case
# ----------------------------------------------------------------------------
def follower_slices(tokens, pqs, lens, L, D, gpos):
    j, e = divmod(int(gpos), L)
    n = min(D, lens[j] - 1 - e)
    return tokens[j, e:e + n + 1], pqs[j][e + 1:e + n + 1]


@pytest.mark.parametrize("seed", range(5))
def test_dag_invariants_and_counter(seed):
    G, N, L, V, D = 1, 5, 40, 3, 5
    tokens, lps = synth.small_random(G * N, L, V, 50 + seed)
    rng = synth.Stream(2000 + seed)
    lens = (6 + rng.uniform(N) * (L - 7)).astype(np.int32)
    for alpha in (1.0, 0.0):
        o = Oracle(G, N, L, V, D, alpha=alpha)
        o.append(tokens, lps, lens)
        pqs = [o.history(p)[1] for p in range(N)]
        k = 1 + seed % 2
        o.build_all(k)
        for i in range(N):
            m = o.matches(i)
            cands = [follower_slices(tokens, pqs, lens, L, D, g) for g in m]
            for d in range(1, D + 1):
                nodes, edges = o.layer(i, d)
                live = [(t, p) for t, p in cands if len(p) >= d]
                # counts are a Counter over follower pairs / follower tokens
                assert {key: c for key, (_, c) in edges.items()} == dict(
                    collections.Counter((int(t[d - 1]), int(t[d])) for t, _ in live))
                assert {key: c for key, (_, c) in nodes.items()} == dict(
                    collections.Counter(int(t[d]) for t, _ in live))
                # probability mass is conserved from instances to edges to nodes
                assert sum(s for s, _ in nodes.values()) == sum(int(p[d - 1]) for _, p in live)
                for v, (s, c) in nodes.items():
                    assert s == sum(es for (u2, v2), (es, _) in edges.items() if v2 == v)
                    assert c == sum(ec for (u2, v2), (_, ec) in edges.items() if v2 == v)
                # every edge starts in a node of the previous layer
                if d > 1:
                    prev_nodes, _ = o.layer(i, d - 1)
                    assert {u for u, _ in edges} <= set(prev_nodes)
                    for u, (_, c) in prev_nodes.items():
                        ended = sum(1 for t, p in cands if len(p) == d - 1 and int(t[d - 1]) == u)
                        assert sum(ec for (u2, _), (_, ec) in edges.items() if u2 == u) == c - ended
                else:
                    assert {u for u, _ in edges} <= {int(tokens[i, lens[i] - 1])}
            if alpha == 0.0:
                _, score, edge_w = o.draft(i)
                assert all(float(x).is_integer() for x in score) and all(float(x).is_integer() for x in edge_w)


def test_alpha_one_scores_agree_with_real_valued_sum():
    G, N, L, V, D = 1, 6, 64, 4, 4
    tokens, lps = synth.small_random(N, L, V, 77)
    lens = np.full(N, L - 1, np.int32)
    o = Oracle(G, N, L, V, D)
    o.append(tokens, lps, lens)
    o.build_all(1)
    for i in range(N):
        m = o.matches(i)
        for d in range(1, D + 1):
            nodes, _ = o.layer(i, d)
            real = collections.defaultdict(float)
            for g in m:
                j, e = divmod(int(g), L)
                if e + d <= lens[j] - 1:
                    real[int(tokens[j, e + d])] += float(np.exp(np.float64(lps[j, e + d])))
            for v, (s, c) in nodes.items():
                assert abs(s / Q30 - real[v]) <= c * 2.0 ** -31 + 1e-12


# ----------------------------------------------------------------------------
# greedy search against enumeration of every DAG path
# ----------------------------------------------------------------------------
def all_dag_paths(o, i, root, D):
    """Every root-to-node path of the layered DAG, by exhaustive extension."""
    layers = [o.layer(i, d) for d in range(1, D + 1)]
    paths = {()}
    frontier = [((), root)]
    for d in range(D):
        nxt = []
        for pref, u in frontier:
            for (eu, ev) in layers[d][1]:
                if eu == u:
                    nxt.append((pref + (ev,), ev))
        paths.update(p for p, _ in nxt)
        frontier = list(set(nxt))
    return paths, layers


@pytest.mark.parametrize("seed,alpha", list(itertools.product(range(5), (1.0, 0.5))))
def test_draft_is_greedy_path_of_the_dag(seed, alpha):
    G, N, L, V, D = 1, 4, 24, 3, 4
    tokens, lps = synth.small_random(N, L, V, 300 + seed)
    rng = synth.Stream(3000 + seed)
    lens = (4 + rng.uniform(N) * (L - 5)).astype(np.int32)
    o = Oracle(G, N, L, V, D, alpha=alpha)
    o.append(tokens, lps, lens)
    o.build_all(1)
    for i in range(N):
        root = int(tokens[i, lens[i] - 1])
        paths, layers = all_dag_paths(o, i, root, D)
        draft, score, edge_w = o.draft(i)
        draft = tuple(int(x) for x in draft)
        assert draft in paths                                         # a path of the DAG
        for d in range(len(draft) + 1):
            ext = sorted({p[d] for p in paths if len(p) > d and p[:d] == draft[:d]})
            if d == len(draft):
                assert d == D or not ext                              # stops at D or at a leaf
                break
            w = {v: oracle.weight(alpha, *layers[d][0][v]) for v in ext}
            best = max(w.values())
            assert draft[d] == min(v for v in ext if w[v] == best)    # argmax, ties to the smaller id
            assert score[d] == w[draft[d]]
            u = root if d == 0 else draft[d - 1]
            assert edge_w[d] == oracle.weight(alpha, *layers[d][1][(u, draft[d])])


def test_layer_argmax_mode_is_per_layer_max():
    N, L, V, D = 4, 24, 3, 4
    tokens, lps = synth.small_random(N, L, V, 411)
    o = Oracle(1, N, L, V, D, mode=1)
    o.append(tokens, lps, np.full(N, L - 2, np.int32))
    o.build_all(1)
    for i in range(N):
        draft, score, _ = o.draft(i)
        for d in range(1, D + 1):
            nodes, _ = o.layer(i, d)
            if not nodes:
                assert len(draft) == d - 1
                break
            w = {v: oracle.weight(1.0, *sc) for v, sc in nodes.items()}
            assert draft[d - 1] == min(v for v in w if w[v] == max(w.values()))


# ----------------------------------------------------------------------------
# export view, acceptance, append rules
# ----------------------------------------------------------------------------
def test_export_view_is_sorted_truncation_of_the_full_dag():
    N, L, V, D, B, Ke = 5, 48, 4, 4, 3, 2
    tokens, lps = synth.small_random(N, L, V, 512)
    o = Oracle(1, N, L, V, D, alpha=0.5)
    o.append(tokens, lps, np.full(N, L - 3, np.int32))
    o.build_all(1)
    for i in range(N):
        ex = o.export(i, B, Ke)
        for d in range(1, D + 1):
            nodes, _ = o.layer(i, d)
            order = sorted(nodes, key=lambda v: (-oracle.weight(0.5, *nodes[v]), v))
            assert ex["node_count"][d - 1] == len(nodes)
            kept = [int(x) for x in ex["node_tok"][d - 1] if x >= 0]
            assert kept == order[:B]
            if d < D:
                _, nxt = o.layer(i, d + 1)
                for b, u in enumerate(kept):
                    out = {v: sc for (uu, v), sc in nxt.items() if uu == u}
                    eorder = sorted(out, key=lambda v: (-oracle.weight(0.5, *out[v]), v))
                    assert ex["out_degree"][d - 1, b] == len(out)
                    assert [int(x) for x in ex["edge_dst"][d - 1, b] if x >= 0] == eorder[:Ke]
                    for e, v in enumerate(eorder[:Ke]):
                        assert (int(ex["edge_S"][d - 1, b, e]), int(ex["edge_cnt"][d - 1, b, e])) == out[v]


def test_accept_is_longest_common_prefix_exhaustive():
    D = 4
    cases = []
    for dl in range(D + 1):
        for draft in itertools.product((0, 1), repeat=dl):
            for samp in itertools.product((0, 1), repeat=D + 1):
                cases.append((draft, samp))
    P = len(cases)
    o = Oracle(1, P, 8, 2, D)
    dt = np.full((P, D), -1, np.int32); dlens = np.zeros(P, np.int32); sm = np.zeros((P, D + 1), np.int32)
    for p, (draft, samp) in enumerate(cases):
        dt[p, :len(draft)] = draft; dlens[p] = len(draft); sm[p] = samp
    tau = o.accept(dt, dlens, sm)
    for p, (draft, samp) in enumerate(cases):
        assert tau[p] == len(os.path.commonprefix([list(draft), list(samp[:len(draft)])]))


def test_accept_commit_appends_tau_plus_one_capped_by_max_append_and_cut_at_capacity():
    # "Draft acceptance": a path takes the accepted tokens plus the model's own next one.  Histories written
    # out by hand.  D = 4, capacity 8, four paths that all hold [7, 7, 7] except the last (7 tokens: one short
    # of the capacity) and whose whole draft [1, 2, 3, 4] is accepted (tau = 4, so tau + 1 = 5 tokens on offer).
    D, L = 4, 8
    draft = np.tile(np.array([1, 2, 3, 4], np.int32), (4, 1))
    dlen = np.array([4, 4, 2, 4], np.int32)                  # path 2 drafted two tokens only: tau = 2
    sampled = np.tile(np.array([1, 2, 3, 4, 5], np.int32), (4, 1))
    lp = np.full((4, D + 1), -0.25, np.float32)
    want = {
        # max_append: (tau, histories afterwards, status)
        5: ([4, 4, 2, 4], [[7, 7, 7, 1, 2, 3, 4, 5], [7, 7, 7, 1, 2, 3, 4, 5], [7, 7, 7, 1, 2, 3], [7] * 7 + [1]]),
        3: ([4, 4, 2, 4], [[7, 7, 7, 1, 2, 3], [7, 7, 7, 1, 2, 3], [7, 7, 7, 1, 2, 3], [7] * 7 + [1]]),
        1: ([4, 4, 2, 4], [[7, 7, 7, 1], [7, 7, 7, 1], [7, 7, 7, 1], [7] * 7 + [1]]),
    }
    for max_append, (tau_want, hist_want) in want.items():
        o = Oracle(1, 4, L, 10, D)
        load_paths(o, [[7, 7, 7], [7, 7, 7], [7, 7, 7], [7] * 7], logprobs=[[-1.0] * 3] * 3 + [[-1.0] * 7])
        tau, st = o.accept_commit(draft, dlen, sampled, lp, max_append)
        assert tau.tolist() == tau_want                       # the clamp does not change what was accepted
        assert st == 0                                        # running into the capacity here is not an error
        assert [o.history(p)[0].tolist() for p in range(4)] == hist_want, max_append
        # a full path takes nothing more and reports nothing
        tau, st = o.accept_commit(draft, dlen, sampled, lp, max_append)
        assert st == 0 and o.lengths()[3] == L and o.history(3)[0].tolist() == [7] * 7 + [1]
    # the probabilities stored with the committed tokens are those of the sampled tokens
    assert o.history(0)[1].tolist()[3:] == [oracle.prob_to_fixed(-0.25)] * 2


def test_append_rules_and_status():
    o = Oracle(1, 4, 6, 10, 2)
    tok = np.array([[1, 2, 3, 4], [1, 2, 3, 4], [1, 99, 3, 4], [1, 2, 3, 4]], np.int32)
    lp = np.full((4, 4), -0.3, np.float32)
    st = o.append(tok, lp, np.array([4, 0, 4, 7], np.int32))
    assert st == oracle.ST_BAD_TOKEN | oracle.ST_BAD_COUNT
    assert o.lengths().tolist() == [4, 0, 1, 4]          # cut before the bad token; count clamped
    st = o.append(tok, lp, np.array([4, 2, 0, 0], np.int32))
    assert st == oracle.ST_CAPACITY
    assert o.lengths().tolist() == [6, 2, 1, 4]
    assert o.history(0)[0].tolist() == [1, 2, 3, 4, 1, 2]
    lp[0, 0] = np.nan
    st = o.append(tok, lp, np.array([0, 1, 1, 1], np.int32))
    assert st == 0                                        # the NaN entry was not among the appended
    st = o.append(tok, np.full((4, 4), np.nan, np.float32), np.array([0, 1, 0, 0], np.int32))
    assert st == oracle.ST_BAD_LOGPROB and o.history(1)[1][-1] == 0


# ----------------------------------------------------------------------------
# fuzzy suffix matching (Eq. 4, tolerance 1)
# ----------------------------------------------------------------------------
def test_edit_distance_textbook_values_and_properties():
    enc = lambda w: [ord(ch) for ch in w]
    assert oracle.edit_distance(enc("kitten"), enc("sitting")) == 3
    assert oracle.edit_distance(enc("flaw"), enc("lawn")) == 2
    assert oracle.edit_distance(enc("abc"), enc("abc")) == 0
    assert oracle.edit_distance(enc("abc"), enc("")) == 3
    rng = synth.Stream(606)
    for _ in range(200):
        a = (rng.uniform(1 + int(rng.one() * 5)) * 3).astype(int).tolist()
        b = (rng.uniform(1 + int(rng.one() * 5)) * 3).astype(int).tolist()
        d = oracle.edit_distance(a, b)
        assert d == oracle.edit_distance(b, a)
        assert abs(len(a) - len(b)) <= d <= max(len(a), len(b))
        assert (d == 0) == (a == b)


def one_edit_neighbourhood(q, V):
    """Every non-empty string within one edit of q over the alphabet [0, V)."""
    out = {tuple(q)}
    for x in range(len(q)):
        out.add(tuple(q[:x] + q[x + 1:]))
        for t in range(V):
            out.add(tuple(q[:x] + [t] + q[x + 1:]))
    for x in range(len(q) + 1):
        for t in range(V):
            out.add(tuple(q[:x] + [t] + q[x:]))
    out.discard(())
    return out


@pytest.mark.parametrize("seed", range(5))
def test_fuzzy_match_set_equals_exact_search_of_the_neighbourhood(seed):
    G, N, L, V = 1, 4, 28, 3
    tokens, lps = synth.small_random(G * N, L, V, 700 + seed)
    rng = synth.Stream(7000 + seed)
    lens = (4 + rng.uniform(N) * (L - 5)).astype(np.int32)
    exact = Oracle(G, N, L, V, 3)
    fuzzy = Oracle(G, N, L, V, 3, eps=1)
    exact.append(tokens, lps, lens)
    fuzzy.append(tokens, lps, lens)
    for k in (1, 2, 3, 4):
        exact.build_all(k)
        fuzzy.build_all(k)
        for i in range(N):
            if lens[i] < k:
                assert len(fuzzy.matches(i)) == 0
                continue
            q = tokens[i, lens[i] - k:lens[i]].tolist()
            want = set()
            for var in one_edit_neighbourhood(q, V):
                pat = re.compile(b"(?=" + re.escape(bytes(var)) + b")")
                for j in range(N):
                    if j == i:
                        continue
                    for m in pat.finditer(bytes(tokens[j, :lens[j]].tolist())):
                        e = m.start() + len(var) - 1
                        if e <= lens[j] - 2:
                            want.add(j * L + e)
            got = fuzzy.matches(i).tolist()
            assert got == sorted(want), (seed, k, i)
            assert set(exact.matches(i).tolist()) <= set(got)


def test_fuzzy_candidates_with_different_last_tokens_share_a_virtual_root():
    # hand-worked: query (1,2), tolerance 1.  Path 1 = [1,3,7,5,5]: "1" (deletion) ends at 0, "1 3"
    # (substitution) at 1.  Path 2 = [4,1,2,7,6,6]: "1" ends at 1, "1 2" (exact) at 2, "1 2 7"
    # (insertion) at 3.  Five candidates whose matched windows end in 1, 3, 1, 2, 7.
    paths = [[9, 1, 2], [1, 3, 7, 5, 5], [4, 1, 2, 7, 6, 6], [8, 8, 8]]
    probs = [[0.5] * 3, [0.5, 0.5, 0.25, 0.5, 0.5], [0.5, 0.5, 0.5, 0.5, 0.25, 0.5], [0.5] * 3]
    o = Oracle(1, 4, 10, 16, 3, eps=1)
    load_paths(o, paths, probs=probs)
    o.build_path(2, 0)
    assert o.matches(0).tolist() == [10, 11, 21, 22, 23]
    # followers: [3,7,5] [7,5,5] [2,7,6] [7,6,6] [6,6]
    nodes, edges = o.layer(0, 1)
    q = lambda x: int(x * Q30)
    assert nodes == {3: (q(0.5), 1), 7: (q(0.75), 2), 2: (q(0.5), 1), 6: (q(0.25), 1)}
    assert edges == {(1, 3): (q(0.5), 1), (3, 7): (q(0.25), 1), (1, 2): (q(0.5), 1), (2, 7): (q(0.5), 1),
                     (7, 6): (q(0.25), 1)}
    nodes2, edges2 = o.layer(0, 2)
    assert nodes2 == {7: (q(0.75), 2), 5: (q(0.5), 1), 6: (q(0.75), 2)}
    tok, score, edge_w = o.draft(0)
    # layer 1: 7 (0.75) from the virtual root; layer 2: successors of 7 are 5 (0.5) and 6 (0.75);
    # layer 3: the successor of 6 is 6 (0.5 + 0.25)
    assert tok.tolist() == [7, 6, 6]
    assert score.tolist() == [0.75, 0.75, 0.75]
    assert edge_w.tolist() == [0.75, 0.25, 0.5]    # the virtual-root edge carries the whole node
    # exact matching sees only the window that ends at (2, 2)
    o0 = Oracle(1, 4, 10, 16, 3)
    load_paths(o0, paths, probs=probs)
    o0.build_path(2, 0)
    assert o0.matches(0).tolist() == [22] and o0.draft(0)[0].tolist() == [7, 6, 6]


@pytest.mark.parametrize("seed", range(3))
def test_fuzzy_draft_is_greedy_walk_from_the_virtual_root(seed):
    G, N, L, V, D = 1, 4, 24, 3, 4
    tokens, lps = synth.small_random(N, L, V, 800 + seed)
    lens = np.full(N, L - 2 - seed, np.int32)
    o = Oracle(G, N, L, V, D, eps=1)
    o.append(tokens, lps, lens)
    o.build_all(2)
    for i in range(N):
        layers = [o.layer(i, d) for d in range(1, D + 1)]
        draft, score, edge_w = o.draft(i)
        cur = None
        for d in range(D):
            nodes, edges = layers[d]
            succ = sorted(nodes) if d == 0 else sorted(v for (u, v) in edges if u == cur)
            if not succ:
                assert len(draft) == d
                break
            w = {v: oracle.weight(1.0, *nodes[v]) for v in succ}
            best = min(v for v in succ if w[v] == max(w.values()))
            assert draft[d] == best and score[d] == w[best]
            assert edge_w[d] == (w[best] if d == 0 else oracle.weight(1.0, *edges[(cur, best)]))
            cur = best


# ----------------------------------------------------------------------------
# tree and list draft pools (the paper's ablation variants)
# ----------------------------------------------------------------------------
def candidate_rows(o, tokens, lens, L, D, i):
    pqs = [o.history(p)[1] for p in range(o.P)]
    rows = []
    for g in o.matches(i):
        j, e = divmod(int(g), L)
        n = min(D, lens[j] - 1 - e)
        rows.append((int(g), [int(t) for t in tokens[j, e + 1:e + 1 + n]], [int(x) for x in pqs[j][e + 1:e + 1 + n]]))
    return rows


@pytest.mark.parametrize("seed,alpha", list(itertools.product(range(4), (1.0, 0.5))))
def test_tree_pool_is_a_greedy_walk_of_the_trie(seed, alpha):
    G, N, L, V, D = 1, 5, 40, 3, 5
    tokens, lps = synth.small_random(N, L, V, 1300 + seed)
    lens = np.full(N, L - 1 - seed, np.int32)
    o = Oracle(G, N, L, V, D, alpha=alpha, pool=1)
    o.append(tokens, lps, lens)
    o.build_all(1)
    for i in range(N):
        rows = candidate_rows(o, tokens, lens, L, D, i)
        draft, score, _ = o.draft(i)
        prefix = []
        for d in range(D + 1):
            # children of the trie node `prefix`: Counter / sums over the candidates that start with it
            live = [(t, p) for _, t, p in rows if len(t) > d and t[:d] == prefix]
            if d == len(draft):
                assert d == D or not live
                break
            w = {}
            for v in sorted({t[d] for t, _ in live}):
                w[v] = oracle.weight(alpha, sum(p[d] for t, p in live if t[d] == v), sum(1 for t, _ in live if t[d] == v))
            best = min(v for v in w if w[v] == max(w.values()))
            assert draft[d] == best and score[d] == w[best]
            prefix.append(best)


@pytest.mark.parametrize("seed,alpha", list(itertools.product(range(4), (1.0, 0.5))))
def test_list_pool_picks_the_heaviest_candidate(seed, alpha):
    G, N, L, V, D = 1, 5, 40, 3, 5
    tokens, lps = synth.small_random(N, L, V, 1400 + seed)
    lens = (L - 1 - 3 * np.arange(N)).astype(np.int32)
    o = Oracle(G, N, L, V, D, alpha=alpha, pool=2)
    o.append(tokens, lps, lens)
    o.build_all(2)
    for i in range(N):
        rows = candidate_rows(o, tokens, lens, L, D, i)
        draft, score, _ = o.draft(i)
        if not rows:
            assert len(draft) == 0
            continue
        w = [oracle.weight(alpha, sum(p), len(p)) for _, _, p in rows]
        first_best = w.index(max(w))                     # rows are in (path, position) order
        assert draft.tolist() == rows[first_best][1]
        assert score.tolist() == [oracle.weight(alpha, x, 1) for x in rows[first_best][2]]


def test_pools_agree_when_there_is_one_candidate_and_differ_on_reconvergence():
    # candidates [2,7,5] and [3,7,6] plus [2,7,6]: after "2 7" the DAG sees 6 twice (via 2 and via 3),
    # the tree only the continuations of the prefix "2 7"
    paths = [[9, 1], [1, 2, 7, 5], [1, 3, 7, 6], [1, 2, 7, 6]]
    probs = [[0.5, 0.5], [0.5, 0.5, 0.5, 0.5], [0.5, 0.25, 0.5, 0.5], [0.5, 0.5, 0.5, 0.25]]
    drafts = {}
    for pool in (0, 1, 2):
        o = Oracle(1, 4, 8, 16, 3, pool=pool)
        load_paths(o, paths, probs=probs)
        o.build_path(1, 0)
        drafts[pool] = (o.draft(0)[0].tolist(), o.draft(0)[1].tolist())
    assert drafts[0] == ([2, 7, 6], [1.0, 1.5, 0.75])     # DAG: node (3, 6) = 0.5 + 0.25
    assert drafts[1] == ([2, 7, 5], [1.0, 1.0, 0.5])      # tree: children of "2 7" are 5 (0.5) and 6 (0.25)
    assert drafts[2] == ([2, 7, 5], [0.5, 0.5, 0.5])      # list: the first candidate sums to 1.5


# ----------------------------------------------------------------------------
# best-path search (search mode 2): brute force over every path of the DAG
# ----------------------------------------------------------------------------
def py_weight(alpha, S, cnt):
    return alpha * float(S) * (1.0 / Q30) + (1.0 - alpha) * float(cnt)


def brute_force_best_path(paths, layers, alpha, D):
    """Among the paths that end at a leaf or at depth D: the largest sum of node weights, added from
    the last node towards the first; ties go to the lexicographically smallest token sequence."""
    maximal = [p for p in paths if p and (len(p) == D or not any(len(q) == len(p) + 1 and q[:len(p)] == p for q in paths))]
    best, best_total = None, None
    for p in sorted(maximal):
        total = 0.0
        for d in range(len(p) - 1, -1, -1):
            total = py_weight(alpha, *layers[d][0][p[d]]) + total
        if best is None or total > best_total:
            best, best_total = p, total
    return best, best_total


def test_best_path_differs_from_greedy_on_a_hand_worked_pool():
    # query path ends in 9.  Candidates: 9 -> 1 (.5) -> 3 (.125)   and   9 -> 2 (.25) -> 4 (.75).
    # Greedy takes 1 (.5 > .25) and is stuck with 3: total .625.  The best path is 2, 4: total 1.0.
    paths = [[5, 9], [9, 1, 3, 7], [9, 2, 4, 7]]
    probs = [[.5, .5], [.5, .5, .125, .5], [.5, .25, .75, .5]]
    for mode, expect, scores in ((0, [1, 3], [.5, .125]), (2, [2, 4], [.25, .75])):
        o = Oracle(1, 3, 8, 10, 2, alpha=1.0, mode=mode)
        assert load_paths(o, paths, probs=probs) == 0
        o.build_all(1)
        draft, score, edge_w = o.draft(0)
        assert list(draft) == expect
        assert list(score) == scores and list(edge_w) == scores


def test_best_path_tie_goes_to_the_smaller_token_and_extends_to_a_leaf():
    # two paths of equal total (.5 + .25 = .25 + .5): the one that starts with the smaller token wins;
    # a zero-weight tail is still followed to the leaf
    paths = [[5, 9], [9, 2, 4, 6], [9, 1, 3, 8]]
    probs = [[.5, .5], [.5, .5, .25, 0.0], [.5, .25, .5, 0.0]]
    o = Oracle(1, 3, 8, 10, 3, alpha=1.0, mode=2)
    assert load_paths(o, paths, probs=probs) == 0
    o.build_all(1)
    draft, score, _ = o.draft(0)
    assert list(draft) == [1, 3, 8] and list(score) == [.25, .5, 0.0]


@pytest.mark.parametrize("seed,alpha,k", list(itertools.product(range(6), (1.0, 0.5, 0.0), (1, 2))))
def test_best_path_equals_brute_force_over_all_dag_paths(seed, alpha, k):
    G, N, L, V, D = 1, 5, 28 + 12 * (seed % 2), 3 + 3 * (seed % 2), 4
    tokens, lps = synth.small_random(N, L, V, 7300 + seed)
    rng = synth.Stream(7400 + seed)
    lens = (5 + rng.uniform(N) * (L - 6)).astype(np.int32)
    o = Oracle(G, N, L, V, D, alpha=alpha, mode=2)
    g = Oracle(G, N, L, V, D, alpha=alpha, mode=0)
    o.append(tokens, lps, lens)
    g.append(tokens, lps, lens)
    o.build_all(k)
    g.build_all(k)
    for i in range(N):
        root = int(tokens[i, lens[i] - 1])
        paths, layers = all_dag_paths(o, i, root, D)
        draft, score, edge_w = o.draft(i)
        draft = tuple(int(x) for x in draft)
        if len(paths) == 1:
            assert draft == ()
            continue
        want, total = brute_force_best_path(paths, layers, alpha, D)
        assert draft == want
        for d, v in enumerate(draft):
            assert score[d] == py_weight(alpha, *layers[d][0][v])
            u = root if d == 0 else draft[d - 1]
            assert edge_w[d] == py_weight(alpha, *layers[d][1][(u, v)])
        # never worse than the greedy walk over the same DAG
        gd, gs, _ = g.draft(i)
        gtot = 0.0
        for x in reversed([float(x) for x in gs]):
            gtot = x + gtot
        assert total >= gtot


def test_best_path_and_greedy_agree_on_a_chain_and_at_depth_one():
    tokens, lps = synth.small_random(4, 24, 3, 7777)
    lens = np.array([20, 18, 22, 19], np.int32)
    for D in (1,):
        a, b = Oracle(1, 4, 24, 3, D, alpha=0.5, mode=0), Oracle(1, 4, 24, 3, D, alpha=0.5, mode=2)
        a.append(tokens, lps, lens); b.append(tokens, lps, lens)
        a.build_all(1); b.build_all(1)
        for i in range(4):
            assert list(a.draft(i)[0]) == list(b.draft(i)[0])
    # one candidate only: the pool is a chain
    paths = [[5, 9], [9, 2, 4, 6, 1]]
    probs = [[.5, .5], [.5, .5, .25, .125, .5]]
    for mode in (0, 2):
        o = Oracle(1, 2, 8, 10, 4, alpha=1.0, mode=mode)
        assert load_paths(o, paths, probs=probs) == 0
        o.build_all(1)
        assert list(o.draft(0)[0]) == [2, 4, 6, 1]


def test_best_path_really_departs_from_greedy_on_random_pools():
    differ = 0
    for seed in range(6):
        tokens, lps = synth.small_random(6, 40, 6, 7300 + seed)
        lens = np.full(6, 38, np.int32)
        a, b = Oracle(1, 6, 40, 6, 6, alpha=1.0, mode=0), Oracle(1, 6, 40, 6, 6, alpha=1.0, mode=2)
        a.append(tokens, lps, lens); b.append(tokens, lps, lens)
        a.build_all(2); b.build_all(2)
        differ += sum(list(a.draft(i)[0]) != list(b.draft(i)[0]) for i in range(6))
    assert differ >= 10


# ----------------------------------------------------------------------------
# sliding window: trimmed histories
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("seed", range(4))
def test_trim_keeps_the_newest_tokens_and_matches_follow_the_shorter_history(seed):
    G, N, L, V = 2, 4, 32, 3
    tokens, lps = synth.small_random(G * N, L, V, 8100 + seed)
    rng = synth.Stream(8200 + seed)
    lens = (8 + rng.uniform(G * N) * (L - 9)).astype(np.int32)
    keep = (2 + rng.uniform(G * N) * 30).astype(np.int32)           # some above the length: no change
    o = Oracle(G, N, L, V, 4)
    o.append(tokens, lps, lens)
    before = [o.history(p) for p in range(G * N)]
    assert o.trim(keep) == 0
    new_lens = np.minimum(lens, keep)
    assert o.lengths().tolist() == new_lens.tolist()
    shifted = np.zeros_like(tokens)
    for p in range(G * N):
        t, q = o.history(p)
        assert t.tolist() == before[p][0][lens[p] - new_lens[p]:].tolist()
        assert q.tolist() == before[p][1][lens[p] - new_lens[p]:].tolist()
        shifted[p, :new_lens[p]] = tokens[p, lens[p] - new_lens[p]:lens[p]]
    # Eq. 3 on the shorter histories, by the independent regex search
    for k in (1, 2):
        o.build_all(k)
        for i in range(G * N):
            if new_lens[i] >= k:
                assert o.matches(i).tolist() == regex_matches(shifted, new_lens, N, L, i, k), (seed, k, i)
    # a trimmed path has room again and appends where its window ends
    room = (L - new_lens).astype(np.int32)
    more = np.minimum(room, 3).astype(np.int32)
    assert o.append(tokens[:, :3], lps[:, :3], more) == 0
    assert o.lengths().tolist() == (new_lens + more).tolist()


def test_trim_rejects_negative_counts_and_keeps_the_path():
    o = Oracle(1, 2, 8, 5, 2)
    load_paths(o, [[1, 2, 3], [4, 0, 1, 2]], probs=[[.5] * 3, [.5] * 4])
    assert o.trim(np.array([-1, 2], np.int32)) == 0x01
    assert o.history(0)[0].tolist() == [1, 2, 3] and o.history(1)[0].tolist() == [1, 2]
    assert o.trim(np.array([0, 9], np.int32)) == 0
    assert o.lengths().tolist() == [0, 2]


# ----------------------------------------------------------------------------
# optional cap on the matches per (query path, source path)
# ----------------------------------------------------------------------------
def test_match_cap_hand_worked_case():
    # query path 0 ends in token 1; source path 1 holds 1 at positions 0, 2, 4, 6 (each with a follower),
    # source path 2 at position 1 only.  R = 2 keeps, per source path, the two largest end positions.
    L = 12
    paths = [[5, 1], [1, 2, 1, 3, 1, 4, 1, 6], [9, 1, 7]]
    probs = [[0.5, 0.5], [0.5, 0.5, 0.5, 0.25, 0.5, 0.5, 0.5, 0.25], [0.5, 0.5, 0.125]]
    full = Oracle(1, 3, L, 16, 2)
    load_paths(full, paths, probs=probs)
    full.build_path(1, 0)
    assert full.matches(0).tolist() == [1 * L + 0, 1 * L + 2, 1 * L + 4, 1 * L + 6, 2 * L + 1]
    capped = Oracle(1, 3, L, 16, 2, max_matches=2)
    load_paths(capped, paths, probs=probs)
    capped.build_path(1, 0)
    assert capped.matches(0).tolist() == [1 * L + 4, 1 * L + 6, 2 * L + 1]
    nodes, edges = capped.layer(0, 1)
    assert nodes == {4: (Q30 // 2, 1), 6: (Q30 // 4, 1), 7: (Q30 // 8, 1)}      # followers 2 and 3 left the pool
    assert capped.draft(0)[0].tolist() == [4, 1]
    assert full.draft(0)[0].tolist() == [2, 1]                                    # 2 (0.5) beats 4 (0.5) on the tie rule
    one = Oracle(1, 3, L, 16, 2, max_matches=1)
    load_paths(one, paths, probs=probs)
    one.build_path(1, 0)
    assert one.matches(0).tolist() == [1 * L + 6, 2 * L + 1]


@pytest.mark.parametrize("seed", range(4))
@pytest.mark.parametrize("eps", [0, 1])
def test_match_cap_keeps_the_last_R_of_every_source_path(seed, eps):
    G, N, L, V, D = 2, 4, 40, 3, 3
    tokens, lps = synth.small_random(G * N, L, V, 7300 + seed)
    lens = (L - 1 - (np.arange(G * N) * 7 + seed) % 15).astype(np.int32)
    full = Oracle(G, N, L, V, D, eps=eps)
    full.append(tokens, lps, lens)
    for R in (1, 2, 5, 1000):
        capped = Oracle(G, N, L, V, D, eps=eps, max_matches=R)
        capped.append(tokens, lps, lens)
        for k in (1, 2, 3):
            for i in range(G * N):
                full.build_path(k, i)
                capped.build_path(k, i)
                m = full.matches(i)
                want = np.concatenate([np.sort(m[m // L == j])[-R:] for j in range(G * N)]) if len(m) else m
                assert np.array_equal(capped.matches(i), want), (R, k, i)
                # the pool is built from the kept matches only: every first-layer count is a kept match
                nodes, _ = capped.layer(i, 1)
                assert sum(c for _, c in nodes.values()) == len(want)


# ----------------------------------------------------------------------------
# several drafts per path: the B best paths of the pool
# ----------------------------------------------------------------------------
def brute_force_beams(paths, layers, alpha, D, B):
    """All paths that end at a leaf or at depth D, each worth the sum of its node weights added from the
    last node towards the first; the B best by (value, larger first; token sequence as a word, smaller first)."""
    maximal = [p for p in paths if p and (len(p) == D or not any(len(q) == len(p) + 1 and q[:len(p)] == p for q in paths))]
    scored = []
    for p in maximal:
        total = 0.0
        for d in range(len(p) - 1, -1, -1):
            total = py_weight(alpha, *layers[d][0][p[d]]) + total
        scored.append((-total, p))
    scored.sort()
    return [list(p) for _, p in scored[:B]], [-t for t, _ in scored[:B]]


def test_beams_hand_worked_pool():
    # query path ends in 9.  Candidates: 9 1 3 | 9 2 4 | 9 2 5, probabilities as listed (layer 1: 1 -> .5,
    # 2 -> .25 + .25 = .5; layer 2: 3 -> .125, 4 -> .75, 5 -> .5).  Paths: [2 4] = 1.25, [2 5] = 1.0, [1 3] = .625.
    paths = [[5, 9], [9, 1, 3, 7], [9, 2, 4, 7], [9, 2, 5, 7]]
    probs = [[.5, .5], [.5, .5, .125, .5], [.5, .25, .75, .5], [.5, .25, .5, .5]]
    o = Oracle(1, 4, 8, 10, 2, alpha=1.0, mode=2)
    assert load_paths(o, paths, probs=probs) == 0
    o.build_all(1)
    toks, vals = o.beams(0, 3)
    assert toks == [[2, 4], [2, 5], [1, 3]] and vals.tolist() == [1.25, 1.0, .625]
    toks, vals = o.beams(0, 2)
    assert toks == [[2, 4], [2, 5]]
    toks, vals = o.beams(0, 8)                         # no more than there are
    assert len(toks) == 3
    assert o.beams(0, 1)[0] == [list(o.draft(0)[0])]   # the first beam is the best path
    assert o.beams(1, 4)[0] == []                      # a path without matches has no beam


def test_beams_tie_goes_to_the_smaller_word():
    # [1 3] and [2 4] are both worth .75; [1 6] too (.5 + .25): order 1 3, 1 6, 2 4
    paths = [[5, 9], [9, 1, 3], [9, 2, 4], [9, 1, 6]]
    probs = [[.5, .5], [.5, .25, .25], [.5, .5, .25], [.5, .25, .25]]
    o = Oracle(1, 4, 8, 10, 2, alpha=1.0, mode=2)
    assert load_paths(o, paths, probs=probs) == 0
    o.build_all(1)
    toks, vals = o.beams(0, 3)
    assert toks == [[1, 3], [1, 6], [2, 4]] and vals.tolist() == [.75, .75, .75]


@pytest.mark.parametrize("seed,alpha,k", list(itertools.product(range(6), (1.0, 0.5, 0.0), (1, 2))))
def test_beams_equal_brute_force_over_all_dag_paths(seed, alpha, k):
    # alpha in {1, 1/2, 0} and dyadic-free sums of 30-bit fractions: every sum here is exact in binary64
    G, N, L, V, D = 1, 5, 28 + 12 * (seed % 2), 3 + 3 * (seed % 2), 4
    tokens, lps = synth.small_random(N, L, V, 7500 + seed)
    rng = synth.Stream(7600 + seed)
    lens = (5 + rng.uniform(N) * (L - 6)).astype(np.int32)
    o = Oracle(G, N, L, V, D, alpha=alpha, mode=2)
    o.append(tokens, lps, lens)
    o.build_all(k)
    seen_many = 0
    for i in range(N):
        root = int(tokens[i, lens[i] - 1])
        paths, layers = all_dag_paths(o, i, root, D)
        for B in (1, 3, 8):
            toks, vals = o.beams(i, B)
            if len(paths) == 1:
                assert toks == []
                continue
            want, totals = brute_force_beams(paths, layers, alpha, D, B)
            assert toks == want, (i, B)
            assert vals.tolist() == totals
            assert all(len(set(map(tuple, toks))) == len(toks) for _ in (0,))      # beams are distinct paths
            seen_many += len(toks) > 1
    assert seen_many > 0
