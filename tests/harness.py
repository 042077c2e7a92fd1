"""Teacher-forced decode protocol that runs the CPU oracle and the CUDA library
side by side and compares them after every call (tests only)."""
from __future__ import annotations

import os

import numpy as np
import torch

from oracle import Oracle
from paper_2503_05330_b200 import binding, synth

RTOL = 1e-5     # float edge / node weights; tokens, positions and sums must be identical


def t32(a, dev):
    return torch.from_numpy(np.ascontiguousarray(a)).to(dev)


class Pair:
    """One oracle and one CUDA context with the same configuration."""

    def __init__(self, G, N, L, V, k_max, D, alpha=1.0, mode=0, B=0, Ke=0, max_append=None, match_capacity=0,
                 eps=0, pool=0, device="cuda:0", host_io=False, max_matches=0, wide_table_bytes=0, max_beams=0, index_max_n=0):
        self.o = Oracle(G, N, L, V, D, alpha=alpha, mode=mode, eps=eps, pool=pool, max_matches=max_matches)
        self.pool = pool
        self.g = binding.Sdms(G, N, L, V, k_max, D, device=device, alpha=alpha, search_mode=mode, B=B, Ke=Ke,
                              max_append=max_append, match_capacity=match_capacity, epsilon=eps, pool_mode=pool,
                              host_io=host_io, max_matches_per_path=max_matches, wide_table_bytes=wide_table_bytes,
                              max_beams=max_beams, index_max_n=index_max_n)
        self.dev = self.g.device
        self.P, self.L, self.D, self.N = G * N, L, D, N
        self.B, self.Ke = B, Ke
        self.max_append = D + 1 if max_append is None else max_append

    def append(self, tokens, logprobs, counts, expect_status=None):
        st_o = self.o.append(tokens, logprobs, counts)
        self.g.append(t32(tokens.astype(np.int32), self.dev), t32(logprobs.astype(np.float32), self.dev),
                      t32(counts.astype(np.int32), self.dev))
        st_g = self.g.status()
        assert st_g == st_o, (st_g, st_o)
        if expect_status is not None:
            assert st_g == expect_status
        return st_g

    def trim(self, keep):
        st_o = self.o.trim(keep)
        self.g.trim(t32(np.asarray(keep, np.int32), self.dev))
        assert self.g.status() == st_o
        return st_o

    def check_history(self):
        tok, pq, lens = self.g.history()
        ol = self.o.lengths()
        assert np.array_equal(lens, ol), (lens, ol)
        for p in range(self.P):
            ht, hp = self.o.history(p)
            assert np.array_equal(tok[p, :ol[p]], ht), p
            assert np.array_equal(pq[p, :ol[p]], hp), p

    def build_and_compare(self, k, check_matches=True, check_dag=True, paths=None):
        """Builds drafts on both sides and compares everything; returns the oracle drafts."""
        self.o.build_all(k, nthreads=min(8, os.cpu_count() or 1))
        self.g.build_drafts(k)
        assert self.g.status() == 0
        tok, ln, sc, ew = self.o.drafts()
        gt, gl = self.g.draft_tok.cpu().numpy(), self.g.draft_len.cpu().numpy()
        gs, ge = self.g.draft_score.cpu().numpy(), self.g.draft_edge_w.cpu().numpy()
        assert np.array_equal(gl, ln), (k, np.nonzero(gl != ln)[0][:8], gl, ln)
        assert np.array_equal(gt, tok), (k, np.nonzero((gt != tok).any(1))[0][:8])
        np.testing.assert_allclose(gs, sc, rtol=RTOL, atol=0)
        np.testing.assert_allclose(ge, ew, rtol=RTOL, atol=0)
        sel = range(self.P) if paths is None else paths
        if check_matches:
            off, gpos = self.g.matches()
            off, gpos = off.numpy(), gpos.numpy()
            for i in sel:
                mine = np.sort(gpos[off[i]:off[i + 1]])
                assert np.array_equal(mine, self.o.matches(i)), (k, i, len(mine), len(self.o.matches(i)))
        if check_dag and self.B > 0:
            dag = self.g.dag()
            for i in sel:
                ex = self.o.export(i, self.B, self.Ke)
                for key in ex:
                    assert np.array_equal(dag[key][i], ex[key]), (k, i, key, dag[key][i], ex[key])
        return tok, ln

    def beams_and_compare(self, B, paths=None):
        """The B best paths of the pools of the last build on both sides: tokens identical, values within RTOL."""
        tok, ln, val = self.g.beams(B)
        assert self.g.status() == 0
        for i in (range(self.P) if paths is None else paths):
            want, want_val = self.o.beams(i, B)
            got = [tok[i, b, :ln[i, b]].tolist() for b in range(B) if ln[i, b] > 0]
            assert got == want, (i, got, want)
            assert (ln[i, len(want):] == 0).all() and (tok[i, len(want):] == -1).all()
            np.testing.assert_allclose(val[i, :len(want)], want_val, rtol=RTOL, atol=0)
        return tok, ln, val

    def backoff_and_compare(self, k_hi):
        """Back-off build: per path the longest k <= k_hi with a match (oracle: fixed-k builds composed)."""
        used = np.zeros(self.P, np.int32)
        for i in range(self.P):
            for k in range(k_hi, 0, -1):
                self.o.build_path(k, i)
                if len(self.o.matches(i)) > 0:
                    used[i] = k
                    break
        self.g.build_drafts_backoff(k_hi)
        assert self.g.status() == 0
        tok, ln, sc, ew = self.o.drafts()
        assert np.array_equal(self.g.used_k.cpu().numpy(), used), (self.g.used_k.cpu().numpy(), used)
        assert np.array_equal(self.g.draft_len.cpu().numpy(), ln)
        assert np.array_equal(self.g.draft_tok.cpu().numpy(), tok)
        np.testing.assert_allclose(self.g.draft_score.cpu().numpy(), sc, rtol=RTOL, atol=0)
        np.testing.assert_allclose(self.g.draft_edge_w.cpu().numpy(), ew, rtol=RTOL, atol=0)
        off, gpos = self.g.matches()
        off, gpos = off.numpy(), gpos.numpy()
        for i in range(self.P):
            assert np.array_equal(np.sort(gpos[off[i]:off[i + 1]]), self.o.matches(i)), i
        return tok, ln, used

    def accept_and_compare(self, sampled, sampled_lp=None):
        tok, ln, _, _ = self.o.drafts()
        if sampled_lp is None:
            tau_o = self.o.accept(tok, ln, sampled)
            tau_g = self.g.accept(t32(sampled, self.dev)).cpu().numpy()
        else:
            tau_o, st_o = self.o.accept_commit(tok, ln, sampled, sampled_lp, self.max_append)
            tau_g = self.g.accept(t32(sampled, self.dev), t32(sampled_lp, self.dev)).cpu().numpy()
            assert self.g.status() == st_o
        assert np.array_equal(tau_g, tau_o), (tau_g, tau_o)
        return tau_o


def run_protocol(pair: Pair, tokens, logprobs, k, steps, warm, commit_in_accept=False, check_every=1,
                 check_matches=True, check_dag=True, start_lens=None):
    """Decode protocol: warm start, then per step build -> accept against the
    stream's own next tokens -> append what was accepted plus one token.  The
    oracle's accept lengths drive both sides.  Returns summary statistics."""
    P, L, D = pair.P, pair.L, pair.D
    lens = np.full(P, warm, np.int32) if start_lens is None else np.asarray(start_lens, np.int32)
    w = int(lens.max())
    pair.append(tokens[:, :w], logprobs[:, :w], lens, expect_status=0)
    accepted = 0
    drafted = 0
    done_steps = 0
    for step in range(steps):
        lens = pair.o.lengths()
        if (lens >= L).all():
            break
        full = step % check_every == 0
        _, ln = pair.build_and_compare(k, check_matches=check_matches and full, check_dag=check_dag and full)
        sampled, sampled_lp = synth.sampled_window(tokens, logprobs, lens, D + 1)
        if commit_in_accept:
            tau = pair.accept_and_compare(sampled, sampled_lp)
        else:
            tau = pair.accept_and_compare(sampled)
            counts = np.minimum(np.minimum(tau + 1, pair.max_append), L - lens).astype(np.int32)
            pair.append(sampled, sampled_lp, counts, expect_status=0)
        accepted += int(tau.sum())
        drafted += int(ln.sum())
        done_steps += 1
    pair.check_history()
    return dict(steps=done_steps, accepted=accepted, drafted=drafted)


def run_step_protocol(pair: Pair, tokens, logprobs, ks, steps, warm, start_lens=None, check_matches=True,
                      check_every=1, check_dag=False):
    """The same decode protocol through the one-call step: after a first build,
    every step is accept + commit + the next build (suffix length ks[step % len(ks)])
    in one call, compared with the oracle's accept_commit followed by build_all.
    Accept lengths, drafts, scores and edge weights are compared after every step; the match
    lists (and with check_dag the exported DAG) of all paths every check_every-th step."""
    P, L, D = pair.P, pair.L, pair.D
    lens = np.full(P, warm, np.int32) if start_lens is None else np.asarray(start_lens, np.int32)
    w = int(lens.max())
    pair.append(tokens[:, :w], logprobs[:, :w], lens, expect_status=0)
    pair.build_and_compare(ks[0], check_matches=check_matches, check_dag=False)
    accepted = 0
    done_steps = 0
    for step in range(steps):
        lens = pair.o.lengths()
        if (lens >= L).all():
            break
        k = ks[(step + 1) % len(ks)]
        sampled, sampled_lp = synth.sampled_window(tokens, logprobs, lens, D + 1)
        tok, ln, _, _ = pair.o.drafts()
        tau_o, st_o = pair.o.accept_commit(tok, ln, sampled, sampled_lp, pair.max_append)
        pair.o.build_all(k, nthreads=min(8, os.cpu_count() or 1))
        tau_g, gt, gl = pair.g.step(k, t32(sampled, pair.dev), t32(sampled_lp, pair.dev))
        assert pair.g.status() == st_o
        assert np.array_equal(tau_g.cpu().numpy(), tau_o), (step, tau_g, tau_o)
        tok, ln, sc, ew = pair.o.drafts()
        assert np.array_equal(gl.cpu().numpy(), ln), (step, k, gl, ln)
        assert np.array_equal(gt.cpu().numpy(), tok), (step, k)
        np.testing.assert_allclose(pair.g.draft_score.cpu().numpy(), sc, rtol=RTOL, atol=0)
        np.testing.assert_allclose(pair.g.draft_edge_w.cpu().numpy(), ew, rtol=RTOL, atol=0)
        if check_matches and step % check_every == 0:
            off, gpos = pair.g.matches()
            off, gpos = off.numpy(), gpos.numpy()
            for i in range(P):
                assert np.array_equal(np.sort(gpos[off[i]:off[i + 1]]), pair.o.matches(i)), (step, k, i)
        if check_dag and pair.B > 0 and step % check_every == 0:
            dag = pair.g.dag()
            for i in range(P):
                ex = pair.o.export(i, pair.B, pair.Ke)
                for key in ex:
                    assert np.array_equal(dag[key][i], ex[key]), (step, k, i, key)
        accepted += int(tau_o.sum())
        done_steps += 1
    pair.check_history()
    return dict(steps=done_steps, accepted=accepted)


def run_windowed_protocol(pair: Pair, tokens, logprobs, ks, steps, warm, keep, use_step=False):
    """Decode protocol that outlives the capacity: a path that comes within a draft of its capacity is
    trimmed to its newest `keep` tokens and goes on.  The streams are read round and round.  Every
    build is compared; returns how many trims happened."""
    P, L, D = pair.P, pair.L, pair.D
    T = tokens.shape[1]
    lens0 = np.full(P, warm, np.int32)
    pair.append(tokens[:, :warm], logprobs[:, :warm], lens0, expect_status=0)
    consumed = lens0.astype(np.int64)                 # tokens of the stream each path has taken so far
    trims = 0
    pair.build_and_compare(ks[0], check_dag=False)
    for step in range(steps):
        lens = pair.o.lengths()
        idx = (consumed[:, None] + np.arange(D + 1)[None, :]) % T
        sampled = np.take_along_axis(tokens, idx, 1).astype(np.int32)
        sampled_lp = np.take_along_axis(logprobs, idx, 1).astype(np.float32)
        tok, ln, _, _ = pair.o.drafts()
        k = ks[(step + 1) % len(ks)]
        if use_step:
            tau_o, st_o = pair.o.accept_commit(tok, ln, sampled, sampled_lp, pair.max_append)
            pair.o.build_all(k, nthreads=min(8, os.cpu_count() or 1))
            tau_g, gt, gl = pair.g.step(k, t32(sampled, pair.dev), t32(sampled_lp, pair.dev))
            assert pair.g.status() == st_o
            assert np.array_equal(tau_g.cpu().numpy(), tau_o)
            tok2, ln2, _, _ = pair.o.drafts()
            assert np.array_equal(gl.cpu().numpy(), ln2) and np.array_equal(gt.cpu().numpy(), tok2), step
        else:
            tau_o = pair.accept_and_compare(sampled, sampled_lp)
        consumed += pair.o.lengths() - lens
        lens = pair.o.lengths()
        near = lens > L - D - 2
        if near.any():
            pair.trim(np.where(near, keep, L).astype(np.int32))
            trims += int(near.sum())
            pair.build_and_compare(k, check_dag=False)          # drafts refer to positions: build again
        elif not use_step:
            pair.build_and_compare(k, check_dag=False)
    pair.check_history()
    return trims
