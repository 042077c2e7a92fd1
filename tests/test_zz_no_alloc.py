"""The allocation-free match entry point against the regular one.

``sdms_match_noalloc`` serves callers that cannot obtain device memory of their
own - typically a sampler plug-in inside a serving engine whose KV-cache pool
took the free HBM at start-up, where a late cudaMalloc can fail or stall the
device.  It keeps its counters in a fixed array inside the library, shared by all
calls, so the interesting failure is a second call seeing the first call's
leftovers: the test makes two calls in a row on different states and compares
each with sdms_build_drafts + sdms_get_matches on the same histories and with the
CPU oracle's match sets (Eq. 3 by brute force).  Positions are integers: the
lists must be identical after sorting each path's slice.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from oracle import Oracle  # noqa: E402
from paper_2503_05330_b200 import binding, synth  # noqa: E402


def sorted_slices(offsets, gpos):
    off = offsets.cpu().numpy()
    g = gpos.cpu().numpy()
    return off, [np.sort(g[off[i]:off[i + 1]]) for i in range(len(off) - 1)]


def test_noalloc_matches_equal_regular_matches_on_two_calls_in_a_row():
    w = synth.WORKLOADS[2]
    tokens, logprobs = synth.make_streams(w)
    dev = torch.device("cuda:0")
    s = binding.Sdms(w.G, w.N, w.L, w.V, w.k_max, w.D, device="cuda:0")
    o = Oracle(w.G, w.N, w.L, w.V, w.D)
    fills = [(np.full(w.P, 700, np.int32) - np.arange(w.P) * 11).astype(np.int32),      # ragged
             np.full(w.P, 300, np.int32)]                                              # then 300 more each
    filled = np.zeros(w.P, np.int32)
    for call, (add, k) in enumerate(zip(fills, (1, 2))):
        width = int(add.max())
        rows = np.zeros((w.P, width), np.int32); lps = np.zeros((w.P, width), np.float32)
        for p in range(w.P):
            rows[p, :add[p]] = tokens[p, filled[p]:filled[p] + add[p]]
            lps[p, :add[p]] = logprobs[p, filled[p]:filled[p] + add[p]]
        s.append(torch.from_numpy(rows).to(dev), torch.from_numpy(lps).to(dev), torch.from_numpy(add).to(dev))
        o.append(rows, lps, add)
        o.build_all(k)
        filled += add
        s.build_drafts(k)
        assert s.status() == 0
        ref_off, ref_gpos = s.matches()
        ref_off, ref = sorted_slices(ref_off, ref_gpos)
        assert ref_off[-1] > 0

        tok = torch.empty((w.P, w.L), dtype=torch.int32, device=dev)
        lens = torch.empty(w.P, dtype=torch.int32, device=dev)
        binding.sdms_debug_read_history(s.ctx, tok, None, lens)
        offsets = torch.full((w.P + 1,), -7, dtype=torch.int32, device=dev)
        gpos = torch.full((int(ref_off[-1]) + 16,), -7, dtype=torch.int32, device=dev)
        binding.sdms_match_noalloc(tok, lens, w.G, w.N, k, offsets, gpos)
        torch.cuda.synchronize()
        off, mine = sorted_slices(offsets, gpos)
        assert np.array_equal(off, ref_off), call
        for i in range(w.P):
            assert np.array_equal(mine[i], ref[i]), (call, i)
            assert np.array_equal(mine[i], o.matches(i)), (call, i)
        assert (gpos[int(off[-1]):] == -7).all()          # nothing written past the end


def test_noalloc_rejects_more_paths_than_its_fixed_scratch_holds():
    dev = torch.device("cuda:0")
    one = torch.zeros(4, dtype=torch.int32, device=dev)
    with pytest.raises(binding.SdmsError) as e:
        binding.sdms_match_noalloc(one.view(1, 4), one, binding.NOALLOC_MAX_PATHS + 1, 1, 1, one, one)
    assert e.value.code == binding.ERR_TOO_LARGE
