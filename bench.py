#!/usr/bin/env python
"""Throughput of per-step draft construction on synthetic multi-path streams.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one pass of the whole path for all paths of the workload:
sdms_build_drafts (query, match, gather, DAG, search) followed by sdms_accept
with commit (acceptance check and state update with index insertion).  The
suffix length takes every value 1..k_max equally often over the steps.  Prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2503_05330_b200 import synth  # noqa: E402

METRIC = "draft-construction paths*steps/sec at N=16 (and us/step)"
UNIT = "paths*steps/s"
L2_FLUSH_BYTES = 256 << 20
# DRAM bytes per launch of the dominant kernel from its last ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum); only quoted while the kernel sources are the ones profiled
NCU_TRAFFIC = {"kernel": "step", "bytes_per_launch": 76032,
               "sources_sha256": "82c4fa773fa1eba361a55396feeb945f28cf039ae1940f656ce90e8d14e5ec53"}


def kernel_sources_sha():
    import hashlib
    h = hashlib.sha256()
    base = os.path.join(ROOT, "paper_2503_05330_b200", "csrc")
    for name in ("dag.cu", "sdms_dev.cuh", "append_dev.cuh"):
        h.update(open(os.path.join(base, name), "rb").read())
    return h.hexdigest()


def k_of(step, k_max):
    """Suffix length of a step: every k in 1..k_max equally often, in a fixed scrambled order (so that
    evenly spaced timed steps do not always meet the same k)."""
    h = ((step + 1) * 0x9E3779B1) & 0xFFFFFFFF
    h = ((h ^ (h >> 15)) * 0x85EBCA77) & 0xFFFFFFFF
    return 1 + (h ^ (h >> 13)) % k_max


def timed_step_plan(K, S):
    """Which steps of which decode run are timed: K timed steps spread evenly over ceil(K / S) whole
    runs of S steps each (warm start .. histories full), so that a small K still sees short and long
    histories and every k alike.  The steps in between run untimed because the state has to evolve.
    Both arms of the benchmark time exactly these steps."""
    runs = -(-K // S)
    plan = []
    for r in range(runs):
        quota = K // runs + (1 if r < K % runs else 0)
        plan.append(set(int((x + 0.5) * S / quota) for x in range(quota)) if quota < S else set(range(S)))
    return plan


# ----------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on the host cores
# ----------------------------------------------------------------------------
def oracle_decode_run(w, tokens, logprobs, timed, threads=1):
    """One whole decode run on the oracle.  A step is what the CUDA arm times as one sdms_step call:
    acceptance check and commit of the drafts of decode step t, then the drafts of step t + 1.  Only the
    steps in `timed` are clocked (None: none, the run only counts its steps).
    Returns (paths*steps, seconds, timed steps, steps in the run)."""
    from oracle import Oracle
    o = Oracle(w.G, w.N, w.L, w.V, w.D)
    lens = np.full(w.P, w.k_max, np.int32)
    o.append(tokens[:, :w.k_max], logprobs[:, :w.k_max], lens)
    o.build_all(k_of(0, w.k_max), nthreads=threads)
    units, secs, done, step = 0, 0.0, 0, 0
    for step in range(w.steps):
        lens = o.lengths()
        active = int((lens < w.L).sum())
        if active == 0:
            break
        sampled, sampled_lp = synth.sampled_window(tokens, logprobs, lens, w.D + 1)
        tok, ln, _, _ = o.drafts()
        on = timed is not None and step in timed
        t0 = time.perf_counter()
        o.accept_commit(tok, ln, sampled, sampled_lp, w.D)
        o.build_all(k_of(step + 1, w.k_max), nthreads=threads)
        if on:
            secs += time.perf_counter() - t0
            units += active
            done += 1
    else:
        step = w.steps
    return units, secs, done, step


def oracle_timed_steps(w, tokens, logprobs, K, threads=1, budget_s=None):
    """Times the same K steps as Runner.timed_steps (timed_step_plan over whole runs)."""
    S = oracle_decode_run(w, tokens, logprobs, None, threads)[3]
    units, secs, done = 0, 0.0, 0
    t_all = time.perf_counter()
    for timed in timed_step_plan(K, S):
        u, t, d, _ = oracle_decode_run(w, tokens, logprobs, timed, threads)
        units += u; secs += t; done += d
        if budget_s is not None and time.perf_counter() - t_all > budget_s:
            break
    return units, secs, done, S


def oracle_run(w, tokens, logprobs, max_steps, budget_s, threads=1):
    """Decode protocol on the oracle; returns (paths*steps, seconds, steps, restarts)."""
    from oracle import Oracle
    done = 0
    units = 0
    secs = 0.0
    runs = 0
    while done < max_steps and secs < budget_s:
        o = Oracle(w.G, w.N, w.L, w.V, w.D)
        lens = np.full(w.P, w.k_max, np.int32)
        o.append(tokens[:, :w.k_max], logprobs[:, :w.k_max], lens)
        runs += 1
        step = 0
        while done < max_steps and secs < budget_s:
            lens = o.lengths()
            active = int((lens < w.L).sum())
            if active == 0 or step >= w.steps:
                break
            sampled, sampled_lp = synth.sampled_window(tokens, logprobs, lens, w.D + 1)
            t0 = time.perf_counter()
            o.build_all(k_of(step, w.k_max), nthreads=threads)
            tok, ln, _, _ = o.drafts()
            o.accept_commit(tok, ln, sampled, sampled_lp, w.D)
            secs += time.perf_counter() - t0
            units += active
            done += 1
            step += 1
    return units, secs, done, runs


def reference_main(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    tokens, logprobs = synth.make_streams(w)
    oracle_timed_steps(w, tokens, logprobs, max(args.warmup, 1))
    units, secs, steps, S = oracle_timed_steps(w, tokens, logprobs, args.steps, budget_s=150.0)
    value = units / secs
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / max(steps, 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32/int64 (f64 weights)",
        "data": "synthetic", "config": workload_config(w),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": f"the same {steps} steps the CUDA arm times: spread evenly over whole decode runs of "
                                   f"{S} steps of {w.name}, the steps in between run untimed"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def workload_config(w):
    return {"workload": w.name, "groups": w.G, "paths_per_group": w.N, "capacity": w.L, "vocab": w.V,
            "k": f"1..{w.k_max}, equally often, fixed scrambled order over the steps", "timed_steps": "spread evenly over whole decode runs", "max_draft_len": w.D,
            "l2": f"flushed between timed steps ({L2_FLUSH_BYTES >> 20} MiB write)"}


# ----------------------------------------------------------------------------
# clocks during the timed region (NVML, in-process)
# ----------------------------------------------------------------------------
class ClockSampler(threading.Thread):
    def __init__(self, index, period=0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.sm, self.reasons, self.max_sm = [], set(), None
        self._halt = threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_sm = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def run(self):
        if self.nv is None:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._halt.is_set():
            try:
                self.sm.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._halt.set()
        self.join()
        return {"sm_mhz": float(np.median(self.sm)) if self.sm else None, "sm_max_mhz": self.max_sm,
                "reasons": sorted(self.reasons), "samples": len(self.sm)}


# ----------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------
class Runner:
    """Device-resident replay of the decode protocol of one workload."""

    def __init__(self, w, seed, device, B, Ke, eps=0, pool=0, mode=0, host_io=False, backoff=False, index_max_n=0):
        import torch
        from paper_2503_05330_b200 import binding
        self.torch, self.binding, self.w, self.device = torch, binding, w, device
        self.tokens, self.logprobs = synth.make_streams(w, seed)
        self.s = binding.Sdms(w.G, w.N, w.L, w.V, w.k_max, w.D, device=device, max_append=w.D, B=B, Ke=Ke, epsilon=eps, pool_mode=pool,
                             search_mode=mode, host_io=host_io, index_max_n=index_max_n)
        dev = self.s.device
        self.warm_tok = torch.from_numpy(np.ascontiguousarray(self.tokens[:, :w.k_max])).to(dev)
        self.warm_lp = torch.from_numpy(np.ascontiguousarray(self.logprobs[:, :w.k_max])).to(dev)
        self.warm_cnt = torch.full((w.P,), w.k_max, dtype=torch.int32, device=dev)
        self.flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
        self.plan = None
        self.backoff = backoff           # every build asks for k_max and backs off to the longest k with a match

    def start_run(self, first_drafts=False):
        self.s.reset()
        self.s.append(self.warm_tok, self.warm_lp, self.warm_cnt)
        if first_drafts:                 # the drafts the first sdms_step of a run checks
            self.build(0)

    def build(self, step):
        if self.backoff:
            self.s.build_drafts_backoff(self.w.k_max)
        else:
            self.s.build_drafts(k_of(step, self.w.k_max))

    def step(self, step, sampled, lp):
        """Acceptance and commit of decode step `step`, drafts of step + 1, in one call."""
        if self.backoff:
            self.s.step_backoff(self.w.k_max, sampled, lp)
        else:
            self.s.step(k_of(step + 1, self.w.k_max), sampled, lp)

    def dry_run(self, allow_status=0):
        """Plays one run to record, per step, the sampled windows (what the model
        would return), the live path count and the algorithmic bytes."""
        torch, w, s = self.torch, self.w, self.s
        dev = s.device
        self.start_run()
        sampled_all, lp_all, active, bytes_scan, bytes_dag, bytes_io = [], [], [], [], [], []
        bytes_fused, bytes_useful, scan_queries = [], [], []
        matches = []
        accepted = []
        for step in range(w.steps):
            _, _, lens = s.history()
            live = int((lens < w.L).sum())
            if live == 0:
                break
            sm, lp = synth.sampled_window(self.tokens, self.logprobs, lens, w.D + 1)
            self.build(step)
            off, gpos = s.matches()
            gpos = gpos.numpy().astype(np.int64)
            j, e = gpos // w.L, gpos % w.L
            n_m = np.minimum(w.D, lens[j] - 1 - e)
            matches.append(len(gpos))
            bytes_scan.append(4 * int(lens.sum()))
            bytes_dag.append(int(8 * n_m.sum() + 4 * len(gpos) + w.P * (12 * w.D + 4)))
            # the fused kernel: a query answered by scanning streams the other paths of its prompt
            k = k_of(step, w.k_max)
            modes = s.query_modes()
            glen = lens.reshape(w.G, w.N).sum(1).repeat(w.N)
            probe_b = int((modes > 0).sum()) * (32 + 4 * k) + 4 * w.P
            bytes_fused.append(int(4 * (glen - lens)[modes == 2].sum()) + probe_b + bytes_dag[-1])
            bytes_useful.append(probe_b + 4 * k * len(gpos) + bytes_dag[-1])      # index model: verify each match
            scan_queries.append(int((modes == 2).sum()))
            s.accept(torch.from_numpy(sm).to(dev), torch.from_numpy(lp).to(dev))
            tau = s.accept_len.cpu().numpy()
            accepted.append(int(tau[lens < w.L].sum()))
            gained = np.minimum(np.minimum(tau + 1, w.D), w.L - lens)
            bytes_io.append(int(gained.sum()) * (8 + 8 + w.k_max * 32) + w.P * (w.D + 1) * 8)
            sampled_all.append(sm); lp_all.append(lp); active.append(live)
        assert s.status() & ~allow_status == 0
        self.plan = dict(
            sampled=torch.from_numpy(np.stack(sampled_all)).to(dev), lp=torch.from_numpy(np.stack(lp_all)).to(dev),
            step_in_host=torch.from_numpy(np.concatenate(
                [np.stack(sampled_all).reshape(len(active), -1),
                 np.stack(lp_all).view(np.int32).reshape(len(active), -1)], axis=1)).pin_memory(),
            active=active, steps=len(active),
            bytes={"scan": float(np.mean(bytes_scan)), "dag": float(np.mean(bytes_dag)),
                   "accept": float(np.mean(bytes_io)), "build_fused": float(np.mean(bytes_fused)),
                   "step": float(np.mean(bytes_fused)) + float(np.mean(bytes_io))},
            useful_bytes_build=float(np.mean(bytes_useful)), scan_queries_per_step=float(np.mean(scan_queries)),
            mean_matches_per_step=float(np.mean(matches)),
            accept_length=float(np.sum(accepted)) / float(np.sum(active)))
        return self.plan

    def timed_steps(self, K, flush=True, e2e=False, events=True):
        """Times exactly K steps (CUDA events around each step on the launch
        stream), restarting the run when it ends.  A step is one sdms_step call: acceptance check
        and commit of the drafts of decode step t, then the drafts of step t + 1.
        Returns (ms, paths*steps).  With e2e the step goes through host buffers and is also timed on
        the host clock, from the moment the model's answer is handed over in host memory to the moment
        the results have been read on the host (self.last_host_ms); events=False leaves the CUDA events out of
        that region (recording two costs the host a few microseconds that no caller pays)."""
        torch, w, s, plan = self.torch, self.w, self.s, self.plan
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
        units = 0
        done = 0
        ks = []
        host_s = 0.0
        if e2e:
            # zero-copy: the step's inputs are written into page-locked host memory that the kernel reads
            # in place, and the kernel writes drafts and accept lengths into page-locked host memory
            assert s.host_io
            h_in = plan["step_in_host"].numpy()                                # [steps][sampled | logprobs]
            step_in = s.step_in.numpy()                                        # the mapped input buffer, as the host sees it
            results = s.results.numpy()
            seen = 0
            stream = torch.cuda.current_stream()
            stream_ptr = stream.cuda_stream
        S = plan["steps"]
        for timed in timed_step_plan(K, S):
            self.start_run(first_drafts=True)
            for step in range(S):
                on = step in timed
                k_next = k_of(step + 1, w.k_max)
                if on and flush:
                    self.flush.zero_()
                if e2e:
                    if on:
                        torch.cuda.synchronize()    # the flush is over: the host clock sees this step only
                        a, b = ev[done]
                        t0 = time.perf_counter()
                        if events:
                            a.record()
                    np.copyto(step_in, h_in[step])  # host to host: the model's answer lands in the mapped buffer
                    if self.backoff:
                        self.step(step, s.sampled_in, s.sampled_lp_in)
                    else:
                        s.step_own_buffers(k_next, stream_ptr)
                    if on and events:
                        b.record()
                    stream.synchronize()            # the caller reads the result before its next step
                    if on:
                        seen += int(results[-1]) + int(results[w.P * w.D])     # an accept length and a draft length, read in place
                        host_s += time.perf_counter() - t0
                else:
                    if on:
                        a, b = ev[done]
                        a.record()
                    self.step(step, plan["sampled"][step], plan["lp"][step])
                    if on:
                        b.record()
                if on:
                    units += plan["active"][step]
                    ks.append(k_next)
                    done += 1
        assert done == K
        torch.cuda.synchronize()
        self.last_host_ms = 1e3 * host_s
        if not events:
            return 0.0, units
        per_step = [a.elapsed_time(b) for a, b in ev]
        self.last_by_k = {}
        for kk in range(1, w.k_max + 1):
            t = [per_step[x] for x in range(K) if ks[x] == kk]
            if t:
                self.last_by_k[str(kk)] = 1e3 * float(np.mean(t))
        return sum(per_step), units


def steady_state(wl, device, iters=20, peak=None, max_matches=0, ks=None, beams=0, index_max_n=0):
    """Build latency of a workload at 97 % full histories (a full path builds no draft): per k the
    median, 10th and 90th percentile of the time of sdms_build_drafts (CUDA events on the launch
    stream, L2 flushed before every call), the matches it found, the kernel's own byte count per call
    and, for prompts scanned by every query CTA, the bytes of a scan shared by the whole prompt."""
    import torch
    from paper_2503_05330_b200 import binding
    tokens, logprobs = synth.make_streams(wl)
    s = binding.Sdms(wl.G, wl.N, wl.L, wl.V, wl.k_max, wl.D, device=device, max_append=wl.D,
                     max_matches_per_path=max_matches, max_beams=beams, index_max_n=index_max_n)
    dev = s.device
    n = int(wl.L * 0.97)
    lens = (n - (np.arange(wl.P) * 13) % 97).astype(np.int32)
    s.append(torch.from_numpy(np.ascontiguousarray(tokens[:, :n])).to(dev),
             torch.from_numpy(np.ascontiguousarray(logprobs[:, :n])).to(dev), torch.from_numpy(lens).to(dev))
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    beam_out = (torch.empty((wl.P, max(beams, 1), wl.D), dtype=torch.int32, device=dev),
                torch.empty((wl.P, max(beams, 1)), dtype=torch.int32, device=dev),
                torch.empty((wl.P, max(beams, 1)), dtype=torch.float32, device=dev))
    out = {}
    for k in (ks or range(1, wl.k_max + 1)):
        for _ in range(3):
            s.build_drafts(k)
        evs = []
        for _ in range(iters):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); s.build_drafts(k); b.record()
            evs.append((a, b))
        torch.cuda.synchronize()
        t_us = 1e3 * np.array([a.elapsed_time(b) for a, b in evs])
        us = float(np.median(t_us))
        binding.sdms_profile_enable(s.ctx, True)                 # per-kernel split (events between the launches)
        for _ in range(5):
            flush.zero_()
            s.build_drafts(k)
        split = {n: 1e3 * ms / c for n, (ms, c) in binding.sdms_profile_read(s.ctx).items() if c}
        binding.sdms_profile_enable(s.ctx, False)
        off, _ = s.matches()
        m = np.diff(off.numpy())
        modes = s.query_modes()
        glen = lens.reshape(wl.G, wl.N).sum(1).repeat(wl.N)
        fused = wl.N * wl.L <= 131072
        csize = binding.sdms_build_cluster_size(s.ctx)
        if fused and csize > 1:          # a cluster of csize paths reads its prompt once for all its scan queries
            scanning = (modes == 2).reshape(-1, csize).any(1)
            scan_bytes = int(4 * glen.reshape(-1, csize)[:, 0][scanning].sum())
        elif fused:                      # every scanning query reads the other paths of its prompt
            scan_bytes = int(4 * (glen - lens)[modes == 2].sum())
        else:                            # one shared pass over the store
            scan_bytes = 4 * int(lens.sum()) if (modes == 2).any() else 0
        nbytes = scan_bytes + int((modes > 0).sum()) * (32 + 4 * k) + int(m.sum()) * (4 + 8 * wl.D) + wl.P * (12 * wl.D + 4)
        shared_scan = 4 * int(lens.reshape(wl.G, wl.N)[(modes == 2).reshape(wl.G, wl.N).any(1)].sum())   # scan model: once per prompt
        out[str(k)] = {"us": us, "p10_us": float(np.percentile(t_us, 10)), "p90_us": float(np.percentile(t_us, 90)),
                       "launches_timed": iters, "paths_per_s": wl.P / (us * 1e-6), "matches": int(m.sum()),
                       "max_matches": int(m.max()),
                       "scanned_queries": int((modes == 2).sum()), "bytes": nbytes, "gbs": nbytes / (us * 1e-6) / 1e9,
                       "frac_of_peak": None if peak is None else nbytes / (us * 1e-6) / 1e9 / peak,
                       "scan_bytes_moved": scan_bytes, "scan_bytes_shared_pass": shared_scan,
                       "kernel_us": split}
        if beams:                                            # several drafts per path from the pools of this build
            for _ in range(2):
                s.beams(beams)
            evs = []
            for _ in range(10):
                flush.zero_()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); binding.sdms_get_beams(s.ctx, beams, *beam_out); b.record()
                evs.append((a, b))
            torch.cuda.synchronize()
            out[str(k)]["get_beams_us"] = 1e3 * float(np.median([a.elapsed_time(b) for a, b in evs]))
    assert s.status() == 0
    return {"groups": wl.G, "paths_per_group": wl.N, "capacity": wl.L, "max_draft_len": wl.D, "fill": 0.97,
            "max_matches_per_path": max_matches, "index_max_n": index_max_n or wl.k_max,
            "launches_per_build": 1 if fused else 4, "build_cluster_size": binding.sdms_build_cluster_size(s.ctx), "workspace_bytes": s.workspace_bytes, "build_by_k": out}


def scan_at_scale(device, G=64, N=256, L=8192, V=151936):
    """The tile-scan kernel on a store larger than L2 (G prompts of N paths, uniform random tokens, k = 1:
    every query has more matches than an index bucket lists, so all of them are answered by the scan).
    Algorithmic bytes = the tokens of all histories, read once.  Context for the kernel that is
    bandwidth-bound by design; the benchmark workload itself never leaves L2."""
    import torch
    from paper_2503_05330_b200 import binding
    P, n = G * N, L - 8
    s = binding.Sdms(G, N, L, V, 1, 4, device=device)
    gen = torch.Generator(device=device)
    gen.manual_seed(synth.BASE_SEED)
    tok = torch.randint(0, V, (P, n), dtype=torch.int32, device=device, generator=gen)
    lp = -torch.rand((P, n), dtype=torch.float32, device=device, generator=gen)
    s.append(tok, lp, torch.full((P,), n, dtype=torch.int32, device=device))
    del tok, lp
    s.build_drafts(1)                                  # warm-up
    binding.sdms_profile_enable(s.ctx, True)
    for _ in range(5):
        s.build_drafts(1)
    torch.cuda.synchronize()
    prof = binding.sdms_profile_read(s.ctx)
    assert s.status() == 0
    ms, launches = prof["scan"]
    us = 1e3 * ms / launches
    nbytes = 4 * P * n
    out = {"groups": G, "paths_per_group": N, "capacity": L, "store_bytes": nbytes, "workspace_bytes": s.workspace_bytes,
           "scan_queries": int((s.query_modes() == 2).sum()), "us_per_launch": us, "gbs": nbytes / (us * 1e-6) / 1e9}
    del s
    torch.cuda.empty_cache()
    return out


def gather_at_scale(device, G=64, N=256, L=8192, V=16384, D=16):
    """Follower gather + DAG aggregation + search (dag_kernel) on a store larger than L2: G prompts of N
    paths, uniform random tokens over a vocabulary small enough that a k = 1 query finds a hundred-odd
    matches (N * L / V), spread at random over the prompt's histories, so that every match costs a fresh
    read of its D followers (token and probability) from HBM and no single query dominates.
    Algorithmic bytes = 8 per follower (token and probability of each of the n_m followers of every match)
    plus the match list and the outputs."""
    import torch
    from paper_2503_05330_b200 import binding
    P, n = G * N, L - 8
    s = binding.Sdms(G, N, L, V, 1, D, device=device)
    gen = torch.Generator(device=device)
    gen.manual_seed(synth.BASE_SEED + 1)
    tok = torch.randint(0, V, (P, n), dtype=torch.int32, device=device, generator=gen)
    lp = -torch.rand((P, n), dtype=torch.float32, device=device, generator=gen)
    s.append(tok, lp, torch.full((P,), n, dtype=torch.int32, device=device))
    del tok, lp
    s.build_drafts(1)                                  # warm-up
    binding.sdms_profile_enable(s.ctx, True)
    for _ in range(5):
        s.build_drafts(1)
    torch.cuda.synchronize()
    prof = binding.sdms_profile_read(s.ctx)
    assert s.status() == 0
    off, gpos = s.matches()
    gpos = gpos.numpy().astype(np.int64)
    n_m = np.minimum(D, n - 1 - gpos % L)
    m = np.diff(off.numpy())
    out = {"groups": G, "paths_per_group": N, "capacity": L, "vocab": V, "max_draft_len": D,
           "store_bytes": 8 * P * n, "workspace_bytes": s.workspace_bytes,
           "matches": int(m.sum()), "mean_matches_per_query": float(m.mean()), "max_matches_per_query": int(m.max())}
    nbytes = int(8 * n_m.sum() + 4 * len(gpos) + P * (12 * D + 4))
    for name in ("dag", "dag_wide"):
        if name in prof and prof[name][1]:
            ms, launches = prof[name]
            out[name + "_us_per_launch"] = 1e3 * ms / launches
    out["queries_by_mode"] = {str(k): int(v) for k, v in zip(*np.unique(s.query_modes(), return_counts=True))}
    us = sum(out[k] for k in out if k.endswith("_us_per_launch"))
    out.update(algorithmic_bytes=nbytes, us_per_build_gather_side=us, gbs=nbytes / (us * 1e-6) / 1e9)
    del s
    torch.cuda.empty_cache()
    return out


def rank_seed(w, rank):
    """Every rank owns its own prompts: same recipe, different seed."""
    return synth.BASE_SEED + w.index + 7919 * rank


def whole_job(times_ms, units, device):
    """Whole-job figures over all ranks: the slowest rank's time (MAX) and the
    units of all ranks (SUM).  Works with any initialised process group; without
    one it returns its inputs."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return list(times_ms), list(units)
    t = torch.tensor(times_ms, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    u = torch.tensor(units, dtype=torch.float64, device=device)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return t.tolist(), u.tolist()


def ours_main(args, w):
    import torch
    import torch.distributed as dist
    from paper_2503_05330_b200 import binding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    device = f"cuda:{local}"
    # every rank owns its own prompts (different seed): no data-path collective
    run = Runner(w, rank_seed(w, rank), device, args.dag_nodes, args.dag_edges)
    plan = run.dry_run()

    run.timed_steps(max(args.warmup, 3))
    sampler = ClockSampler(local)
    sampler.start()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    launches0 = binding.sdms_launch_count(run.s.ctx)
    t0 = time.perf_counter()
    ms, units = run.timed_steps(args.steps)
    by_k = dict(run.last_by_k)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    wall = time.perf_counter() - t0
    launches = binding.sdms_launch_count(run.s.ctx) - launches0
    clocks = sampler.stop()
    later = ClockSampler(local, period=0.2)          # the passes that follow (end to end, per kernel, other workloads, at scale)
    later.start()

    # end to end through host buffers
    hrun = Runner(w, rank_seed(w, rank), device, 0, 0, host_io=True)
    hrun.plan = plan
    hrun.timed_steps(3, e2e=True)
    _, units_e2e = hrun.timed_steps(args.steps, e2e=True, events=False)      # the headline: host clock, nothing else in the region
    host_ms_e2e = hrun.last_host_ms
    ms_e2e, _ = hrun.timed_steps(args.steps, e2e=True)                       # the same steps once more with events: the device's share
    del hrun

    # per-kernel times over a further pass of the same steps
    binding.sdms_profile_enable(run.s.ctx, True)
    run.timed_steps(args.steps)
    prof = binding.sdms_profile_read(run.s.ctx)
    binding.sdms_profile_enable(run.s.ctx, False)
    # warm-L2 figure for context (no flush between steps)
    ms_warm, units_warm = run.timed_steps(args.steps, flush=False)
    # the DAG export is an inspection call outside the step: time it once per build on a short replay
    export_us = None
    if args.dag_nodes > 0:
        run.start_run()
        evs = []
        for step in range(min(plan["steps"], 200)):
            run.s.build_drafts(k_of(step, w.k_max))
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            dag = run.s.dag_device()
            b.record()
            evs.append((a, b))
            run.s.accept(plan["sampled"][step], plan["lp"][step])
        torch.cuda.synchronize()
        export_us = 1e3 * float(np.mean([a.elapsed_time(b) for a, b in evs]))

    # the same protocol with fuzzy suffix matching (tolerance 1), the paper's experimental setting
    fuzzy = None
    if world == 1 and not args.no_fuzzy:
        frun = Runner(w, rank_seed(w, rank), device, 0, 0, eps=1)
        fplan = frun.dry_run()
        frun.timed_steps(20)
        fms, funits = frun.timed_steps(min(args.steps, 1000))
        fuzzy = {"us_per_step": 1e3 * fms / min(args.steps, 1000), "value": funits / (fms * 1e-3), "unit": UNIT,
                 "us_per_step_by_k": dict(frun.last_by_k), "mean_matches_per_step": fplan["mean_matches_per_step"]}
        del frun
    # accept length (accepted draft tokens per path and step) of the pool structures and of fuzzy
    # matching on these synthetic streams: the axes of the paper's ablation, as context only
    ablation = None
    if world == 1 and not args.no_fuzzy:
        ablation = {"dag": plan["accept_length"]}
        variant_us = {}
        if fuzzy is not None:
            ablation["dag_fuzzy"] = fplan["accept_length"]
        for name, pool, eps, mode, idx in (("tree", 1, 0, 0, 0), ("list", 2, 0, 0, 0), ("tree_fuzzy", 1, 1, 0, 0), ("list_fuzzy", 2, 1, 0, 0),
                                           ("dag_best_path", 0, 0, 2, 0), ("dag_best_path_fuzzy", 0, 1, 2, 0), ("dag_index_n2", 0, 0, 0, 2)):
            arun = Runner(w, rank_seed(w, rank), device, 0, 0, eps=eps, pool=pool, mode=mode, index_max_n=idx)
            ablation[name] = arun.dry_run(allow_status=0x40)["accept_length"]
            if eps == 0:                 # step time of the variant, measured like the headline
                arun.timed_steps(20)
                n_v = min(args.steps, 500)
                vms, _ = arun.timed_steps(n_v)
                variant_us[name] = 1e3 * vms / n_v
                arun.s.status()          # clears the best-path fallback bit
            del arun
        # suffix length with back-off: every step asks for k_max, each path uses the longest k that has a match
        brun = Runner(w, rank_seed(w, rank), device, 0, 0, backoff=True)
        bplan = brun.dry_run()
        brun.timed_steps(20)
        n_b = min(args.steps, 1000)
        bms, bunits = brun.timed_steps(n_b)
        backoff = {"us_per_step": 1e3 * bms / n_b, "value": bunits / (bms * 1e-3), "unit": UNIT,
                   "accept_length": bplan["accept_length"], "mean_matches_per_step": bplan["mean_matches_per_step"],
                   "what": "sdms_step_backoff(k_max): one launch per step, k chosen per path"}
        del brun
        # sliding window: one sdms_trim of full histories to their newer half (three launches)
        trun = Runner(w, rank_seed(w, rank), device, 0, 0)
        n_full = w.L - 1
        trun.s.reset()
        trun.s.append(torch.from_numpy(np.ascontiguousarray(trun.tokens[:, :n_full])).to(device),
                      torch.from_numpy(np.ascontiguousarray(trun.logprobs[:, :n_full])).to(device),
                      torch.full((w.P,), n_full, dtype=torch.int32, device=device))
        keep = torch.full((w.P,), w.L // 2, dtype=torch.int32, device=device)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        trun.flush.zero_()
        a.record(); trun.s.trim(keep); b.record()
        torch.cuda.synchronize()
        trim_us = 1e3 * a.elapsed_time(b)
        assert trun.s.status() == 0
        del trun
    peaks_file = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_file):
        peak, peak_src = float(json.load(open(peaks_file))["hbm_gbs"]), "measured copy bandwidth (burst)"
    else:
        peak, peak_src = 6650.0, "fallback"
    others = scale = gscale = steady2 = None
    if world == 1 and not args.no_others:
        del run.flush
        torch.cuda.empty_cache()
        steady2 = steady_state(w, device, iters=200, peak=peak)
        others = {synth.WORKLOADS[c].name: steady_state(synth.WORKLOADS[c], device, peak=peak) for c in (1, 3, 4, 5)}
        # the pool capped at the 64 / 8 most recent matches per source path (the heaviest k = 1 query keeps 255 * R at most)
        others["cfg5_n256_l8192_match_cap_64"] = steady_state(synth.WORKLOADS[5], device, peak=peak, max_matches=64, ks=(1, 2, 3))
        others["cfg5_n256_l8192_match_cap_8"] = steady_state(synth.WORKLOADS[5], device, peak=peak, max_matches=8, ks=(1, 2, 3))
        others["cfg2_n16_l1024_four_beams"] = steady_state(w, device, peak=peak, beams=4)
        # the index with tables for 1- and 2-grams only (64 bytes less per token and dropped length)
        for c in (2, 4, 5):
            others[synth.WORKLOADS[c].name + "_index_n2"] = steady_state(synth.WORKLOADS[c], device, peak=peak, index_max_n=2)
        scale = scan_at_scale(device)
        gscale = gather_at_scale(device)
    (ms, ms_e2e, host_ms_e2e), (units, units_e2e, _) = whole_job([ms, ms_e2e, host_ms_e2e], [units, units_e2e, 0.0], device)
    clocks_later = later.stop()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    per_kernel = {}
    for name, (kms, n) in prof.items():
        if n:
            us = 1e3 * kms / n
            b = plan["bytes"].get(name)
            per_kernel[name] = {"launches": n, "us_per_launch": us, "share": kms / sum(v[0] for v in prof.values()),
                                "algorithmic_bytes_per_launch": b,
                                "gbs": (b / (us * 1e-6) / 1e9) if b else None}
    dom = max((n for n in per_kernel if per_kernel[n]["gbs"] is not None), key=lambda n: per_kernel[n]["share"])
    achieved = per_kernel[dom]["gbs"]
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_source": peak_src,
                "traffic": NCU_TRAFFIC["bytes_per_launch"]
                if dom == NCU_TRAFFIC["kernel"] and kernel_sources_sha() == NCU_TRAFFIC["sources_sha256"] else None,
                "bytes_model": "what this kernel's method must read: index bucket per query, the other paths of the "
                               "prompt for each scanned query, followers of every match, outputs",
                "useful_bytes_per_launch_index_model": plan["useful_bytes_build"],
                "note": "the whole store of this workload is 128 KiB: a step is bound by launch and "
                        "dependent-access latency, not by bandwidth",
                # the figures the bandwidth clause is judged on: kernels on stores larger than L2, and the
                # build of every configuration at 97 % full histories
                "match_at_scale": None if scale is None else dict(scale, frac=scale["gbs"] / peak),
                "gather_at_scale": None if gscale is None else dict(gscale, frac=gscale["gbs"] / peak),
                "steady_state_full_history": steady2,
                "by_config": others}

    line = {
        "metric": METRIC, "value": units / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "us_per_step": 1e3 * ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int32/int64 (f64 weights)", "data": "synthetic", "config": workload_config(w),
        "e2e": {"value": units_e2e / (host_ms_e2e * 1e-3), "unit": UNIT, "us_per_step": 1e3 * host_ms_e2e / args.steps,
                "clock": "host (perf_counter): from the model's answer being handed over in host memory, through the "
                         "C-ABI call, to the results having been read on the host; the L2 flush is waited for before",
                "device_us": 1e3 * ms_e2e / args.steps,
                "device_us_from": "a second pass over the same steps with CUDA events around each call (left out of the host-clock pass)",
                "h2d_bytes_per_step": w.P * (w.D + 1) * 8 + w.P * (w.D + 1) * 4,
                "d2h_bytes_per_step": w.P * (w.D + 2) * 4,
                "how": "zero-copy: sampled tokens, logprobs and the previous drafts are read by the step kernel from "
                       "page-locked host memory, drafts and accept lengths written to it; the host reads them after "
                       "the stream has drained"},
        "gpu_launches": launches, "single_launch_step": run.s.step_is_single_launch(),
        "clocks": {**clocks, "window": "the timed steps", "later_passes": clocks_later}, "roofline": roofline, "kernels": per_kernel,
        "warm_l2_us_per_step": 1e3 * ms_warm / args.steps,
        "wall_s_timed_region": wall, "mean_matches_per_step": plan["mean_matches_per_step"],
        "scan_queries_per_step": plan["scan_queries_per_step"], "run_steps": plan["steps"], "us_per_step_by_k": by_k,
        "fuzzy_epsilon_1": fuzzy, "synthetic_accept_length": ablation,
        "variant_us_per_step": None if ablation is None else variant_us,
        "backoff_from_k_max": None if ablation is None else backoff,
        "sliding_window": None if ablation is None else {"us_per_sdms_trim_call": trim_us,
                                                          "what": "all paths full, trimmed to their newer half"},
        "dag_export": {"nodes_per_layer": args.dag_nodes, "edges_per_node": args.dag_edges,
                       "us_per_sdms_get_dag_call": export_us,
                       "note": "inspection call that re-aggregates the last build's matches; not part of a step"},
    }
    if world == 1 and not args.no_cpu_baseline:
        # the oracle as it stands: single-threaded, and with its thread fan-out over query paths on all host cores
        cores = os.cpu_count() or 1
        legs = {}
        for threads in sorted({1, cores}):
            units_c, secs_c, steps_c, runs_c = oracle_run(w, run.tokens, run.logprobs, 10 ** 9, 8.0, threads=threads)
            legs[threads] = {"value": units_c / secs_c, "us_per_step": 1e6 * secs_c / steps_c, "steps": steps_c, "runs": runs_c}
        best = max(legs, key=lambda t: legs[t]["value"])
        line["cpu_baseline"] = {"value": legs[best]["value"], "unit": UNIT, "cores": best, "kind": "oracle",
                                "us_per_step": legs[best]["us_per_step"], "host_cores": cores,
                                "by_threads": {str(t): legs[t] for t in legs},
                                "sample": f"{legs[best]['steps']} decode steps of {w.name} ({legs[best]['runs']} whole run(s) from "
                                          f"the warm start, every step timed); the faster of 1 thread and {cores} threads"}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=2)
    ap.add_argument("--dag-nodes", type=int, default=8, help="nodes per layer in the DAG export (0 = off)")
    ap.add_argument("--dag-edges", type=int, default=4)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-fuzzy", action="store_true", help="skip the extra pass with tolerance 1")
    ap.add_argument("--no-others", action="store_true", help="skip the build-only figures of the other workloads")
    ap.add_argument("--steady", type=int, default=0,
                    help="only print the build-only figures of this workload at 97 %% full histories (for profiling)")
    ap.add_argument("--gather-scale", type=int, default=0,
                    help="only run the gather / DAG kernels on this many prompts of 256 paths x 8192 tokens (for profiling)")
    ap.add_argument("--scan-scale", type=int, default=0,
                    help="only run the tile-scan kernel on this many prompts of 256 paths x 8192 tokens (for profiling)")
    args = ap.parse_args()
    if args.gather_scale:
        import torch
        torch.cuda.set_device(0)
        print(json.dumps({"gather_at_scale": gather_at_scale("cuda:0", G=args.gather_scale)}), flush=True)
        return
    if args.scan_scale:
        import torch
        torch.cuda.set_device(0)
        print(json.dumps({"scan_kernel_at_scale": scan_at_scale("cuda:0", G=args.scan_scale)}), flush=True)
        return
    if args.steady:
        import torch
        torch.cuda.set_device(0)
        wl = synth.WORKLOADS[args.steady]
        print(json.dumps({"steady_state": wl.name, **steady_state(wl, "cuda:0", iters=max(args.steps, 1))}), flush=True)
        return
    w = synth.WORKLOADS[args.workload]
    if args.impl == "reference":
        reference_main(args, w)
    else:
        ours_main(args, w)


if __name__ == "__main__":
    main()
