"""ctypes binding of ``libsdms.so``.

Module-level functions carry the names of the C entry points and only marshal
arguments (torch tensors -> device pointers, torch stream -> cudaStream_t).
``Sdms`` bundles a context with the buffers a decode loop needs.  Every step of
the path runs inside the CUDA library; nothing here computes, and there is no
CPU fallback: loading fails loudly when the library has not been built.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsdms.so")

SDMS_OK = 0
ERR_INVALID_ARG, ERR_WORKSPACE_TOO_SMALL, ERR_CUDA, ERR_BAD_STATE, ERR_TOO_LARGE = -1, -2, -3, -4, -5
NOALLOC_MAX_PATHS = 16384
STATUS_BAD_COUNT, STATUS_CAPACITY, STATUS_BAD_TOKEN = 0x01, 0x02, 0x04
STATUS_BAD_LOGPROB, STATUS_INDEX_FULL, STATUS_MATCH_OVERFLOW = 0x08, 0x10, 0x20
STATUS_SEARCH_FALLBACK, STATUS_TIMEOUT, STATUS_TABLES_FULL = 0x40, 0x80, 0x100
NUM_KERNELS = 9
KERNEL_NAMES = ("append", "probe", "scan", "dag", "accept", "build_fused", "step", "trim", "dag_wide")

EXPORTS = (
    "sdms_workspace_bytes", "sdms_create", "sdms_reset", "sdms_destroy", "sdms_append",
    "sdms_build_drafts", "sdms_build_drafts_backoff", "sdms_accept", "sdms_get_matches", "sdms_get_dag",
    "sdms_debug_read_history", "sdms_debug_read_query_modes", "sdms_get_status", "sdms_launch_count", "sdms_profile_enable",
    "sdms_profile_read", "sdms_strerror", "sdms_kernel_name", "sdms_match_noalloc", "sdms_step",
    "sdms_step_is_single_launch", "sdms_trim", "sdms_host_pointer", "sdms_step_backoff", "sdms_get_beams", "sdms_debug_wait_timeout", "sdms_build_cluster_size",
)


class SdmsConfig(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("num_groups", C.c_int32), ("paths_per_group", C.c_int32),
        ("capacity", C.c_int32), ("vocab", C.c_int32), ("k_max", C.c_int32),
        ("max_draft_len", C.c_int32), ("max_append", C.c_int32), ("dag_nodes_per_layer", C.c_int32),
        ("dag_edges_per_node", C.c_int32), ("search_mode", C.c_int32), ("alpha", C.c_float),
        ("match_capacity", C.c_int64), ("epsilon", C.c_int32), ("pool_mode", C.c_int32),
        ("max_matches_per_path", C.c_int32), ("max_beams", C.c_int32), ("wide_table_bytes", C.c_int64),
        ("index_max_n", C.c_int32), ("reserved1", C.c_int32),
    ]


def make_config(G, N, L, V, k_max, D, max_append=None, B=0, Ke=0, search_mode=0, alpha=1.0,
                match_capacity=0, epsilon=0, pool_mode=0, max_matches_per_path=0, wide_table_bytes=0, max_beams=0, index_max_n=0) -> SdmsConfig:
    return SdmsConfig(C.sizeof(SdmsConfig), G, N, L, V, k_max, D, D + 1 if max_append is None else max_append,
                      B, Ke, search_mode, alpha, match_capacity, epsilon, pool_mode, max_matches_per_path, max_beams,
                      wide_table_bytes, index_max_n, 0)


_lib = None


def lib():
    """The loaded library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                               "`python -m paper_2503_05330_b200.build` (there is no CPU fallback)")
        l = C.CDLL(LIB_PATH)
        vp, i32 = C.c_void_p, C.c_int32
        l.sdms_workspace_bytes.argtypes = [C.POINTER(SdmsConfig), C.POINTER(C.c_size_t)]
        l.sdms_create.argtypes = [C.POINTER(SdmsConfig), vp, C.c_size_t, C.POINTER(vp)]
        l.sdms_reset.argtypes = [vp, vp]
        l.sdms_destroy.argtypes = [vp]
        l.sdms_append.argtypes = [vp, vp, vp, vp, i32, vp]
        l.sdms_build_drafts.argtypes = [vp, i32, vp, vp, vp, vp, vp]
        l.sdms_build_drafts_backoff.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp]
        l.sdms_accept.argtypes = [vp, vp, vp, vp, vp, vp, vp]
        l.sdms_trim.argtypes = [vp, vp, vp]
        l.sdms_host_pointer.argtypes = [vp, C.POINTER(vp)]
        l.sdms_step.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, vp, vp]
        l.sdms_step_backoff.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        l.sdms_step_is_single_launch.argtypes = [vp, C.POINTER(C.c_int32)]
        l.sdms_build_cluster_size.argtypes = [vp, C.POINTER(C.c_int32)]
        l.sdms_get_matches.argtypes = [vp, vp, vp, C.c_size_t, vp]
        l.sdms_get_dag.argtypes = [vp] * 10
        l.sdms_get_beams.argtypes = [vp, i32, vp, vp, vp, vp]
        l.sdms_debug_read_history.argtypes = [vp] * 5
        l.sdms_debug_read_query_modes.argtypes = [vp, vp, vp]
        l.sdms_get_status.argtypes = [vp, C.POINTER(C.c_uint32), vp]
        l.sdms_debug_wait_timeout.argtypes = [vp, vp]
        l.sdms_launch_count.argtypes = [vp, C.POINTER(C.c_uint64)]
        l.sdms_profile_enable.argtypes = [vp, i32]
        l.sdms_profile_read.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(C.c_uint64)]
        l.sdms_match_noalloc.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp, C.c_size_t, vp]
        l.sdms_strerror.argtypes = [C.c_int]
        l.sdms_strerror.restype = C.c_char_p
        l.sdms_kernel_name.argtypes = [C.c_int]
        l.sdms_kernel_name.restype = C.c_char_p
        _lib = l
    return _lib


class SdmsError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {lib().sdms_strerror(code).decode()} ({code})")


def _check(code, where):
    if code != SDMS_OK:
        raise SdmsError(code, where)


_mapped = {}          # data_ptr of a page-locked host tensor -> its address on the device


def sdms_host_pointer(t) -> int:
    """Device-side address of a page-locked, mapped host tensor (raises for any other memory)."""
    out = C.c_void_p(0)
    _check(lib().sdms_host_pointer(C.c_void_p(t.data_ptr()), C.byref(out)), "sdms_host_pointer")
    return out.value


def _dp(t):
    """Pointer the kernels can use: a CUDA tensor's own, or the device-side address of a page-locked
    host tensor that the library has verified (None -> NULL)."""
    if t is None:
        return None
    assert t.is_contiguous()
    if t.is_cuda:
        return C.c_void_p(t.data_ptr())
    key = t.data_ptr()
    if key not in _mapped:
        _mapped[key] = sdms_host_pointer(t)
    return C.c_void_p(_mapped[key])


def _sp(stream):
    """cudaStream_t of a torch stream (None: the current one) or of a raw handle given as int."""
    if isinstance(stream, int):
        return C.c_void_p(stream)
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


# ---- the C entry points, one to one ------------------------------------------
def sdms_workspace_bytes(cfg: SdmsConfig) -> int:
    n = C.c_size_t(0)
    _check(lib().sdms_workspace_bytes(C.byref(cfg), C.byref(n)), "sdms_workspace_bytes")
    return n.value


def sdms_create(cfg: SdmsConfig, workspace: torch.Tensor):
    h = C.c_void_p()
    _check(lib().sdms_create(C.byref(cfg), _dp(workspace), workspace.numel() * workspace.element_size(),
                             C.byref(h)), "sdms_create")
    return h


def sdms_reset(ctx, stream=None):
    _check(lib().sdms_reset(ctx, _sp(stream)), "sdms_reset")


def sdms_destroy(ctx):
    _check(lib().sdms_destroy(ctx), "sdms_destroy")


def sdms_append(ctx, tokens, logprobs, counts, stream=None):
    assert tokens.dtype == torch.int32 and logprobs.dtype == torch.float32 and counts.dtype == torch.int32
    _check(lib().sdms_append(ctx, _dp(tokens), _dp(logprobs), _dp(counts), tokens.shape[1], _sp(stream)),
           "sdms_append")


def sdms_build_drafts(ctx, k, draft_tok, draft_len, draft_score=None, draft_edge_w=None, stream=None):
    _check(lib().sdms_build_drafts(ctx, k, _dp(draft_tok), _dp(draft_len), _dp(draft_score), _dp(draft_edge_w),
                                   _sp(stream)), "sdms_build_drafts")


def sdms_build_drafts_backoff(ctx, k_hi, draft_tok, draft_len, draft_score=None, draft_edge_w=None, used_k=None,
                              stream=None):
    _check(lib().sdms_build_drafts_backoff(ctx, k_hi, _dp(draft_tok), _dp(draft_len), _dp(draft_score),
                                           _dp(draft_edge_w), _dp(used_k), _sp(stream)), "sdms_build_drafts_backoff")


def sdms_accept(ctx, draft_tok, draft_len, sampled, sampled_logprobs, accept_len, stream=None):
    _check(lib().sdms_accept(ctx, _dp(draft_tok), _dp(draft_len), _dp(sampled), _dp(sampled_logprobs),
                             _dp(accept_len), _sp(stream)), "sdms_accept")


def sdms_trim(ctx, keep, stream=None):
    _check(lib().sdms_trim(ctx, _dp(keep), _sp(stream)), "sdms_trim")


def sdms_step(ctx, k, sampled, sampled_logprobs, accept_len, draft_tok, draft_len, draft_score, draft_edge_w,
              stream=None):
    _check(lib().sdms_step(ctx, k, _dp(sampled), _dp(sampled_logprobs), _dp(accept_len), _dp(draft_tok),
                           _dp(draft_len), _dp(draft_score), _dp(draft_edge_w), _sp(stream)), "sdms_step")


def sdms_step_backoff(ctx, k_hi, sampled, sampled_logprobs, accept_len, draft_tok, draft_len, draft_score,
                      draft_edge_w, used_k, stream=None):
    _check(lib().sdms_step_backoff(ctx, k_hi, _dp(sampled), _dp(sampled_logprobs), _dp(accept_len), _dp(draft_tok),
                                   _dp(draft_len), _dp(draft_score), _dp(draft_edge_w), _dp(used_k), _sp(stream)),
           "sdms_step_backoff")


def sdms_step_is_single_launch(ctx) -> bool:
    yes = C.c_int32(0)
    _check(lib().sdms_step_is_single_launch(ctx, C.byref(yes)), "sdms_step_is_single_launch")
    return bool(yes.value)


def sdms_build_cluster_size(ctx) -> int:
    n = C.c_int32(0)
    _check(lib().sdms_build_cluster_size(ctx, C.byref(n)), "sdms_build_cluster_size")
    return n.value


def sdms_get_matches(ctx, offsets, gpos, stream=None):
    _check(lib().sdms_get_matches(ctx, _dp(offsets), _dp(gpos), gpos.numel(), _sp(stream)), "sdms_get_matches")


def sdms_get_dag(ctx, node_tok, node_S, node_cnt, node_count, edge_dst, edge_S, edge_cnt, out_degree, stream=None):
    _check(lib().sdms_get_dag(ctx, _dp(node_tok), _dp(node_S), _dp(node_cnt), _dp(node_count), _dp(edge_dst),
                              _dp(edge_S), _dp(edge_cnt), _dp(out_degree), _sp(stream)), "sdms_get_dag")


def sdms_get_beams(ctx, num_beams, beam_tok, beam_len, beam_value, stream=None):
    _check(lib().sdms_get_beams(ctx, num_beams, _dp(beam_tok), _dp(beam_len), _dp(beam_value), _sp(stream)),
           "sdms_get_beams")


def sdms_debug_read_history(ctx, tok, pq, lens, stream=None):
    _check(lib().sdms_debug_read_history(ctx, _dp(tok), _dp(pq), _dp(lens), _sp(stream)), "sdms_debug_read_history")


def sdms_debug_read_query_modes(ctx, modes, stream=None):
    _check(lib().sdms_debug_read_query_modes(ctx, _dp(modes), _sp(stream)), "sdms_debug_read_query_modes")


def sdms_get_status(ctx, stream=None) -> int:
    f = C.c_uint32(0)
    _check(lib().sdms_get_status(ctx, C.byref(f), _sp(stream)), "sdms_get_status")
    return f.value


def sdms_debug_wait_timeout(ctx, stream=None):
    _check(lib().sdms_debug_wait_timeout(ctx, _sp(stream)), "sdms_debug_wait_timeout")


def sdms_launch_count(ctx) -> int:
    n = C.c_uint64(0)
    _check(lib().sdms_launch_count(ctx, C.byref(n)), "sdms_launch_count")
    return n.value


def sdms_profile_enable(ctx, on: bool):
    _check(lib().sdms_profile_enable(ctx, int(on)), "sdms_profile_enable")


def sdms_profile_read(ctx):
    ms = (C.c_float * NUM_KERNELS)()
    n = (C.c_uint64 * NUM_KERNELS)()
    _check(lib().sdms_profile_read(ctx, ms, n), "sdms_profile_read")
    return {KERNEL_NAMES[k]: (float(ms[k]), int(n[k])) for k in range(NUM_KERNELS)}


def sdms_match_noalloc(tok, lens, num_groups, paths_per_group, k, offsets, gpos, stream=None):
    """Eq. 3 matches straight from caller-held histories ``tok [P][L]`` / ``lens [P]``.

    For callers that cannot allocate device memory (for example a sampler plug-in
    inside a serving engine whose KV-cache pool already owns the free HBM): needs
    no context and no workspace; its only scratch is a fixed array inside the
    library.  ``offsets [P+1]`` and ``gpos`` are the caller's output tensors."""
    assert tok.dtype == torch.int32 and lens.dtype == torch.int32
    _check(lib().sdms_match_noalloc(_dp(tok), _dp(lens), num_groups, paths_per_group, tok.shape[1], k,
                                    _dp(offsets), _dp(gpos), gpos.numel(), _sp(stream)), "sdms_match_noalloc")


# ---- convenience wrapper ------------------------------------------------------
class Sdms:
    """A context plus the device buffers of one decode loop (allocation and
    marshalling only)."""

    def __init__(self, G, N, L, V, k_max, D, device="cuda:0", host_io=False, **kw):
        """host_io: the per-step buffers (`results`, `step_in`) are page-locked host memory that the
        kernels read and write in place (zero-copy) instead of device memory."""
        self.cfg = make_config(G, N, L, V, k_max, D, **kw)
        self.host_io = host_io
        self.G, self.N, self.L, self.V, self.k_max, self.D = G, N, L, V, k_max, D
        self.P = G * N
        self.B, self.Ke = self.cfg.dag_nodes_per_layer, self.cfg.dag_edges_per_node
        self.device = torch.device(device)
        nbytes = sdms_workspace_bytes(self.cfg)
        self.workspace_bytes = nbytes
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            self.ctx = sdms_create(self.cfg, self.workspace)
        P, D_ = self.P, D
        dev = self.device
        # integer results side by side, so that a caller can fetch them with one copy:
        # [draft_tok P*D | draft_len P | accept_len P]
        io = dict(dtype=torch.int32, pin_memory=True) if host_io else dict(dtype=torch.int32, device=dev)
        self.results = torch.empty(P * (D_ + 2), **io)
        self.draft_tok = self.results[:P * D_].view(P, D_)
        self.draft_len = self.results[P * D_:P * D_ + P]
        self.accept_len = self.results[P * D_ + P:]
        self.draft_score = torch.empty((P, D_), dtype=torch.float32, device=dev)
        self.draft_edge_w = torch.empty((P, D_), dtype=torch.float32, device=dev)
        # the model's answer of a step, likewise one buffer: [sampled P*(D+1) int32 | logprobs P*(D+1) float32]
        self.step_in = torch.empty(2 * P * (D_ + 1), **io)
        self.sampled_in = self.step_in[:P * (D_ + 1)].view(P, D_ + 1)
        self.sampled_lp_in = self.step_in[P * (D_ + 1):].view(torch.float32).view(P, D_ + 1)
        self._own = None

    def close(self):
        if getattr(self, "ctx", None):
            sdms_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self, stream=None):
        sdms_reset(self.ctx, stream)

    def append(self, tokens, logprobs, counts, stream=None):
        sdms_append(self.ctx, tokens, logprobs, counts, stream)

    def build_drafts(self, k, stream=None):
        sdms_build_drafts(self.ctx, k, self.draft_tok, self.draft_len, self.draft_score, self.draft_edge_w, stream)
        return self.draft_tok, self.draft_len

    def build_drafts_backoff(self, k_hi, stream=None):
        if not hasattr(self, "used_k"):
            self.used_k = torch.empty(self.P, dtype=torch.int32, device=self.device)
        sdms_build_drafts_backoff(self.ctx, k_hi, self.draft_tok, self.draft_len, self.draft_score, self.draft_edge_w,
                                  self.used_k, stream)
        return self.draft_tok, self.draft_len, self.used_k

    def accept(self, sampled, sampled_logprobs=None, stream=None):
        sdms_accept(self.ctx, self.draft_tok, self.draft_len, sampled, sampled_logprobs, self.accept_len, stream)
        return self.accept_len

    def trim(self, keep, stream=None):
        sdms_trim(self.ctx, keep, stream)

    def step(self, k, sampled, sampled_logprobs, stream=None):
        """accept + commit of the drafts held now, then the next drafts in their place."""
        sdms_step(self.ctx, k, sampled, sampled_logprobs, self.accept_len, self.draft_tok, self.draft_len,
                  self.draft_score, self.draft_edge_w, stream)
        return self.accept_len, self.draft_tok, self.draft_len

    def step_own_buffers(self, k, stream=None):
        """`step` on the context's own input buffers (`sampled_in`, `sampled_lp_in`), with the pointers marshalled
        once: for decode loops that count microseconds on the host."""
        if self._own is None:
            self._own = tuple(_dp(t) for t in (self.sampled_in, self.sampled_lp_in, self.accept_len, self.draft_tok,
                                               self.draft_len, self.draft_score, self.draft_edge_w))
        _check(lib().sdms_step(self.ctx, k, *self._own, _sp(stream)), "sdms_step")

    def step_backoff(self, k_hi, sampled, sampled_logprobs, stream=None):
        sdms_step_backoff(self.ctx, k_hi, sampled, sampled_logprobs, self.accept_len, self.draft_tok, self.draft_len,
                          self.draft_score, self.draft_edge_w, self.used_k, stream)
        return self.accept_len, self.draft_tok, self.draft_len, self.used_k

    def step_is_single_launch(self) -> bool:
        return sdms_step_is_single_launch(self.ctx)

    def status(self, stream=None) -> int:
        return sdms_get_status(self.ctx, stream)

    def matches(self, cap=None):
        """(offsets [P+1], positions) of the last build, as CPU tensors."""
        offsets = torch.empty(self.P + 1, dtype=torch.int32, device=self.device)
        probe = torch.empty(1, dtype=torch.int32, device=self.device)
        lib().sdms_get_matches(self.ctx, _dp(offsets), _dp(probe), 0, _sp(None))
        total = int(offsets[-1].item())
        gpos = torch.empty(max(total, 1), dtype=torch.int32, device=self.device)
        sdms_get_matches(self.ctx, offsets, gpos)
        return offsets.cpu(), gpos[:total].cpu()

    def dag(self):
        return {k: v.cpu().numpy() for k, v in self.dag_device().items()}

    def dag_device(self):
        P, D, B, Ke, dev = self.P, self.D, self.B, self.Ke, self.device
        r = dict(node_tok=torch.empty((P, D, B), dtype=torch.int32, device=dev),
                 node_S=torch.empty((P, D, B), dtype=torch.int64, device=dev),
                 node_cnt=torch.empty((P, D, B), dtype=torch.int32, device=dev),
                 node_count=torch.empty((P, D), dtype=torch.int32, device=dev),
                 edge_dst=torch.empty((P, D, B, Ke), dtype=torch.int32, device=dev),
                 edge_S=torch.empty((P, D, B, Ke), dtype=torch.int64, device=dev),
                 edge_cnt=torch.empty((P, D, B, Ke), dtype=torch.int32, device=dev),
                 out_degree=torch.empty((P, D, B), dtype=torch.int32, device=dev))
        sdms_get_dag(self.ctx, r["node_tok"], r["node_S"], r["node_cnt"], r["node_count"], r["edge_dst"],
                     r["edge_S"], r["edge_cnt"], r["out_degree"])
        return r

    def beams(self, num_beams):
        """(tokens [P][B][D], lengths [P][B], values [P][B]) of the last build, as numpy arrays."""
        tok = torch.empty((self.P, num_beams, self.D), dtype=torch.int32, device=self.device)
        ln = torch.empty((self.P, num_beams), dtype=torch.int32, device=self.device)
        val = torch.empty((self.P, num_beams), dtype=torch.float32, device=self.device)
        sdms_get_beams(self.ctx, num_beams, tok, ln, val)
        return tok.cpu().numpy(), ln.cpu().numpy(), val.cpu().numpy()

    def query_modes(self):
        modes = torch.empty(self.P, dtype=torch.int32, device=self.device)
        sdms_debug_read_query_modes(self.ctx, modes)
        return modes.cpu().numpy()

    def history(self):
        tok = torch.empty((self.P, self.L), dtype=torch.int32, device=self.device)
        pq = torch.empty((self.P, self.L), dtype=torch.int32, device=self.device)
        lens = torch.empty(self.P, dtype=torch.int32, device=self.device)
        sdms_debug_read_history(self.ctx, tok, pq, lens)
        return tok.cpu().numpy(), pq.cpu().numpy(), lens.cpu().numpy()
