"""Thin ctypes binding of libas_verify.so: argument marshalling only.

Every function has the name and argument order of its C counterpart in include/as_verify.h and takes
torch CUDA tensors (or numpy / lists for the host arrays).  Nothing here computes: all steps of the
verify path run in the library's kernels.  If the library has not been built the import of this
module raises; there is no fallback.
"""
from __future__ import annotations

import ctypes as C
from typing import Optional
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("AS_VERIFY_LIB") or os.path.join(_HERE, "libas_verify.so")   # override: a debug build

AS_OK, AS_ERR_INVALID_ARG, AS_ERR_UNSUPPORTED, AS_ERR_WORKSPACE, AS_ERR_CUDA, AS_ERR_DEVICE_FLAG, AS_ERR_TIMEOUT = range(7)
AS_FLAG_BAD_PAGE, AS_FLAG_BAD_TOKEN, AS_FLAG_WAIT_CAP, AS_FLAG_BAD_ACCEPT, AS_FLAG_BAD_PLAN = 1, 2, 4, 8, 16
AS_COMMIT_SCRUB = 1
AS_ATTN_AUTO, AS_ATTN_SIMT, AS_ATTN_TC = 0, 1, 2

EXPORTS = ["as_status_string", "as_last_error", "as_plan_create", "as_plan_destroy", "as_plan_workspace_bytes",
           "as_plan_bind", "as_plan_set_attn_impl", "as_plan_set_fixed_launch", "as_plan", "as_plan_device", "as_verify_attn", "as_accept", "as_accept_seeded", "as_accept_lm_head", "as_accept_lm_head_sampled", "as_accept_lm_head_scratch_bytes", "as_kv_commit",
           "as_plan_check", "as_plan_stats", "as_plan_preview", "as_plan_set_profile_events", "as_plan_launch_count", "as_plan_set_test_stall", "as_budget",
           "as_accept_greedy_static", "as_drafter_create", "as_drafter_destroy", "as_drafter_open", "as_drafter_close", "as_drafter_forget",
           "as_drafter_feed", "as_drafter_block", "as_drafter_propose"]


class LayerDesc(C.Structure):
    _fields_ = [("num_q_heads", C.c_int32), ("num_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("block_size", C.c_int32), ("window", C.c_int32), ("sm_scale", C.c_float), ("sinks", C.c_void_p)]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2608_24004_b200.build` "
                          "(there is no CPU or PyTorch fallback)")
    lib = C.CDLL(LIB_PATH)
    lib.as_status_string.restype = C.c_char_p
    lib.as_last_error.restype = C.c_char_p
    lib.as_plan_workspace_bytes.restype = C.c_size_t
    lib.as_plan_workspace_bytes.argtypes = [C.c_void_p]
    lib.as_plan_create.argtypes = [C.POINTER(C.c_void_p), C.POINTER(LayerDesc), C.c_int, C.c_int, C.c_int, C.c_int,
                                   C.c_int, C.c_int]
    lib.as_plan_destroy.argtypes = [C.c_void_p]
    lib.as_plan_bind.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t]
    lib.as_plan_set_attn_impl.argtypes = [C.c_void_p, C.c_int]
    lib.as_plan.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                            C.POINTER(C.c_int), C.c_void_p]
    lib.as_verify_attn.argtypes = [C.c_void_p, C.c_int] + [C.c_void_p] * 9
    lib.as_accept.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int] + [C.c_void_p] * 8
    lib.as_accept_seeded.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int] + [C.c_void_p] * 7
    lib.as_kv_commit.argtypes = [C.c_void_p] + [C.c_void_p] * 5 + [C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.as_plan_set_fixed_launch.argtypes = [C.c_void_p, C.c_int]
    lib.as_plan_check.argtypes = [C.c_void_p, C.POINTER(C.c_uint32), C.c_void_p]
    lib.as_plan_stats.argtypes = [C.c_void_p, C.c_int] + [C.POINTER(C.c_int)] * 4
    lib.as_plan_preview.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                                    C.c_void_p, C.POINTER(C.c_int), C.POINTER(C.c_int)]
    lib.as_plan_set_profile_events.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
    lib.as_plan_launch_count.argtypes = [C.c_void_p]
    lib.as_plan_launch_count.restype = C.c_int64
    lib.as_plan_set_test_stall.argtypes = [C.c_void_p, C.c_uint64, C.c_int]
    lib.as_accept_lm_head_scratch_bytes.restype = C.c_size_t
    lib.as_accept_lm_head_scratch_bytes.argtypes = [C.c_void_p, C.c_int, C.c_int]
    lib.as_accept_lm_head_sampled.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_int64] \
        + [C.c_void_p] * 5 + [C.c_size_t, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.as_budget.argtypes = [C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_double, C.c_double, C.c_int, C.c_void_p,
                              C.c_void_p]
    lib.as_accept_greedy_static.argtypes = [C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_int64, C.c_int,
                                            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.as_drafter_create.argtypes = [C.POINTER(C.c_void_p), C.POINTER(C.c_char_p), C.c_void_p, C.c_int]
    lib.as_drafter_destroy.argtypes = [C.c_void_p]
    lib.as_drafter_open.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.POINTER(C.c_char_p), C.POINTER(C.c_char_p), C.c_int,
                                    C.POINTER(C.c_int)]
    lib.as_drafter_close.argtypes = [C.c_void_p, C.c_int]
    lib.as_drafter_forget.argtypes = [C.c_void_p, C.c_int64, C.c_int64]
    lib.as_drafter_feed.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int]
    lib.as_drafter_block.argtypes = [C.c_void_p, C.c_int]
    lib.as_drafter_propose.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.POINTER(C.c_int), C.POINTER(C.c_int),
                                       C.POINTER(C.c_int)]
    return lib


_lib = _load()


class AsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib.as_last_error().decode()
        super().__init__(f"{where}: {_lib.as_status_string(status).decode()} ({msg})")


def _chk(status: int, where: str):
    if status != AS_OK:
        raise AsError(status, where)


def _dptr(t, dtype=None, allow_none=False):
    if t is None:
        assert allow_none
        return None
    assert isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous(), "expected a contiguous CUDA tensor"
    if dtype is not None:
        assert t.dtype == dtype, (t.dtype, dtype)
    return C.c_void_p(t.data_ptr())


def _host_i32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


class Plan:
    """Owner of one as_plan_t handle (and of the tensors that must outlive it: workspace, sinks)."""

    def __init__(self, handle, keepalive):
        self.handle = handle
        self._keep = list(keepalive)
        self.workspace = None

    def __del__(self):
        if getattr(self, "handle", None) and _lib is not None:     # at interpreter shutdown the module may be gone
            _lib.as_plan_destroy(self.handle)
            self.handle = None


def as_plan_create(kinds, max_batch, max_draft, max_blocks_per_req, num_blocks, device=0) -> Plan:
    """kinds: list of dicts(num_q_heads, num_kv_heads, head_dim, block_size, window=0, sm_scale=0.0, sinks=None)."""
    arr = (LayerDesc * len(kinds))()
    keep = []
    for i, k in enumerate(kinds):
        sinks = k.get("sinks")
        if sinks is not None:
            assert sinks.is_cuda and sinks.dtype == torch.float32 and sinks.is_contiguous()
            keep.append(sinks)
        arr[i] = LayerDesc(k["num_q_heads"], k["num_kv_heads"], k["head_dim"], k["block_size"], k.get("window", 0),
                           k.get("sm_scale", 0.0), None if sinks is None else sinks.data_ptr())
    h = C.c_void_p()
    _chk(_lib.as_plan_create(C.byref(h), arr, len(kinds), max_batch, max_draft, max_blocks_per_req, num_blocks, device),
         "as_plan_create")
    return Plan(h, keep)


def as_plan_destroy(plan: Plan):
    if plan.handle:
        _chk(_lib.as_plan_destroy(plan.handle), "as_plan_destroy")
        plan.handle = None


def as_plan_workspace_bytes(plan: Plan) -> int:
    return int(_lib.as_plan_workspace_bytes(plan.handle))


def as_plan_bind(plan: Plan, workspace: torch.Tensor):
    assert workspace.is_cuda and workspace.dtype == torch.uint8 and workspace.is_contiguous()
    _chk(_lib.as_plan_bind(plan.handle, C.c_void_p(workspace.data_ptr()), workspace.numel()), "as_plan_bind")
    plan.workspace = workspace


def as_plan_set_attn_impl(plan: Plan, impl: int):
    _chk(_lib.as_plan_set_attn_impl(plan.handle, impl), "as_plan_set_attn_impl")


def as_plan_set_fixed_launch(plan: Plan, on: bool = True):
    _chk(_lib.as_plan_set_fixed_launch(plan.handle, 1 if on else 0), "as_plan_set_fixed_launch")


def as_plan(plan: Plan, seq_lens, draft_lens, block_table: torch.Tensor, free_blocks=None, stream=None) -> int:
    """Returns the number of pages taken from free_blocks (0 when free_blocks is None)."""
    seq, dl = _host_i32(seq_lens), _host_i32(draft_lens)
    assert len(seq) == len(dl)
    free = None if free_blocks is None else _host_i32(free_blocks)
    taken = C.c_int(0)
    _chk(_lib.as_plan(plan.handle, len(seq), seq.ctypes.data_as(C.c_void_p), dl.ctypes.data_as(C.c_void_p),
                      _dptr(block_table, torch.int32), None if free is None else free.ctypes.data_as(C.c_void_p),
                      0 if free is None else len(free), C.byref(taken), _stream(stream)), "as_plan")
    return int(taken.value)


def as_accept_lm_head(plan: Plan, hidden: torch.Tensor, weight: torch.Tensor, draft_tokens, accept_len, out_tokens, stream=None):
    """Greedy acceptance from hidden states [rows, H] and the output projection's weights [V, H] (both bf16)."""
    bf, i32 = torch.bfloat16, torch.int32
    assert hidden.dim() == 2 and weight.dim() == 2 and hidden.shape[1] == weight.shape[1]
    _chk(_lib.as_accept_lm_head(plan.handle, _dptr(hidden, bf), _dptr(weight, bf), hidden.shape[1], weight.shape[0],
                                _dptr(draft_tokens, i32, True), _dptr(accept_len, i32), _dptr(out_tokens, i32),
                                _stream(stream)), "as_accept_lm_head")


def as_accept_lm_head_scratch_bytes(plan: Plan, hidden_dim: int, vocab: int) -> int:
    return int(_lib.as_accept_lm_head_scratch_bytes(plan.handle, hidden_dim, vocab))


def as_accept_lm_head_sampled(plan: Plan, hidden: torch.Tensor, weight: torch.Tensor, draft_tokens, draft_probs, temperature,
                              u, w, rng_state, scratch: torch.Tensor, accept_len, out_tokens, stream=None):
    """Rejection sampling from hidden states [rows, H] and the output projection's weights [V, H] (both bf16); scratch is a
    uint8 tensor of at least as_accept_lm_head_scratch_bytes() bytes; u / w or rng_state (uint64 {seed, step}) as in as_accept."""
    bf, i32, f32 = torch.bfloat16, torch.int32, torch.float32
    assert hidden.dim() == 2 and weight.dim() == 2 and hidden.shape[1] == weight.shape[1]
    assert draft_probs is None or (draft_probs.dim() == 2 and draft_probs.stride(1) == 1)
    _chk(_lib.as_accept_lm_head_sampled(plan.handle, _dptr(hidden, bf), _dptr(weight, bf), hidden.shape[1], weight.shape[0],
                                        _dptr(draft_tokens, i32, True), _dptr(draft_probs, f32, True),
                                        0 if draft_probs is None else draft_probs.stride(0), _dptr(temperature, f32),
                                        _dptr(u, f32, True), _dptr(w, f32, True),
                                        None if rng_state is None else C.c_void_p(rng_state.data_ptr()),
                                        C.c_void_p(scratch.data_ptr()), scratch.numel() * scratch.element_size(),
                                        _dptr(accept_len, i32), _dptr(out_tokens, i32), _stream(stream)), "as_accept_lm_head_sampled")


def as_plan_device(plan: Plan, batch: int, seq_lens: torch.Tensor, draft_lens: torch.Tensor, block_table: torch.Tensor,
                   free_blocks: Optional[torch.Tensor] = None, num_free: int = 0, stream=None) -> None:
    """The step's metadata built on the device from device-resident int32 length arrays (needs fixed launches)."""
    i32 = torch.int32
    _chk(_lib.as_plan_device(plan.handle, batch, _dptr(seq_lens, i32), _dptr(draft_lens, i32), _dptr(block_table, i32),
                             _dptr(free_blocks, i32, True), num_free, _stream(stream)), "as_plan_device")


def as_verify_attn(plan: Plan, kind: int, q, k_new, v_new, k_pool, v_pool, block_table, out, lse=None, stream=None):
    bf = torch.bfloat16
    _chk(_lib.as_verify_attn(plan.handle, kind, _dptr(q, bf), _dptr(k_new, bf), _dptr(v_new, bf), _dptr(k_pool, bf),
                             _dptr(v_pool, bf), _dptr(block_table, torch.int32), _dptr(out, bf),
                             _dptr(lse, torch.float32, True), _stream(stream)), "as_verify_attn")


def as_accept(plan: Plan, logits, vocab, draft_tokens, draft_probs, temperature, u, w, accept_len, out_tokens,
              stream=None):
    f32, i32 = torch.float32, torch.int32
    assert logits.dim() == 2 and logits.stride(1) == 1
    ld = logits.stride(0)
    if draft_probs is not None:
        assert draft_probs.stride(0) == ld, "draft_probs must share the row stride of logits"
    assert logits.is_cuda and logits.dtype == f32
    _chk(_lib.as_accept(plan.handle, C.c_void_p(logits.data_ptr()), ld, vocab, _dptr(draft_tokens, i32, True),
                        None if draft_probs is None else C.c_void_p(draft_probs.data_ptr()),
                        _dptr(temperature, f32, True), _dptr(u, f32, True), _dptr(w, f32, True),
                        _dptr(accept_len, i32), _dptr(out_tokens, i32), _stream(stream)), "as_accept")


def as_accept_seeded(plan: Plan, logits, vocab, draft_tokens, draft_probs, temperature, rng_state, accept_len,
                     out_tokens, stream=None):
    """rng_state: CUDA int64 tensor [2] = (seed, step)."""
    f32, i32 = torch.float32, torch.int32
    assert logits.dim() == 2 and logits.stride(1) == 1 and logits.is_cuda and logits.dtype == f32
    ld = logits.stride(0)
    if draft_probs is not None:
        assert draft_probs.stride(0) == ld, "draft_probs must share the row stride of logits"
    _chk(_lib.as_accept_seeded(plan.handle, C.c_void_p(logits.data_ptr()), ld, vocab, _dptr(draft_tokens, i32, True),
                               None if draft_probs is None else C.c_void_p(draft_probs.data_ptr()),
                               _dptr(temperature, f32), _dptr(rng_state, torch.int64), _dptr(accept_len, i32),
                               _dptr(out_tokens, i32), _stream(stream)), "as_accept_seeded")


def as_kv_commit(plan: Plan, accept_len, seq_lens, block_table, freed, freed_count, flags=0, k_pool=None, v_pool=None,
                 stream=None):
    i32 = torch.int32
    _chk(_lib.as_kv_commit(plan.handle, _dptr(accept_len, i32), _dptr(seq_lens, i32), _dptr(block_table, i32),
                           _dptr(freed, i32), _dptr(freed_count, i32), flags, _dptr(k_pool, torch.bfloat16, True),
                           _dptr(v_pool, torch.bfloat16, True), _stream(stream)), "as_kv_commit")


def as_plan_check(plan: Plan, stream=None, raise_on_flag=True) -> int:
    """Synchronises the stream; returns the AS_FLAG_* bits (raises AsError if any and raise_on_flag)."""
    flags = C.c_uint32(0)
    st = _lib.as_plan_check(plan.handle, C.byref(flags), _stream(stream))
    if st not in (AS_OK, AS_ERR_DEVICE_FLAG, AS_ERR_TIMEOUT) or (st != AS_OK and raise_on_flag):
        raise AsError(st, "as_plan_check")
    return int(flags.value)


def as_plan_stats(plan: Plan, kind: int = 0) -> dict:
    v = [C.c_int(0) for _ in range(4)]
    _chk(_lib.as_plan_stats(plan.handle, kind, *[C.byref(x) for x in v]), "as_plan_stats")
    return dict(num_ctas=v[0].value, num_items=v[1].value, num_merges=v[2].value, impl=v[3].value)


def as_plan_set_profile_events(plan: Plan, begin=None, end=None):
    """begin / end: torch.cuda.Event(enable_timing=True) that have been recorded at least once, or None."""
    h = lambda e: None if e is None else C.c_void_p(e.cuda_event)
    _chk(_lib.as_plan_set_profile_events(plan.handle, h(begin), h(end)), "as_plan_set_profile_events")


def as_plan_launch_count(plan: Plan) -> int:
    return int(_lib.as_plan_launch_count(plan.handle))


def as_plan_set_test_stall(plan: Plan, wait_limit_ns: int = 0, stall_after_loads: int = -1):
    """Test hook: shorter limit for the kernels' bounded waits, copy producers that stop after that many tiles."""
    _chk(_lib.as_plan_set_test_stall(plan.handle, wait_limit_ns, stall_after_loads), "as_plan_set_test_stall")


AS_STATIC_MAX_ROWS = 1024


def as_accept_greedy_static(batch, total_q, max_draft, cu_q, logits, vocab, draft_tokens, accept_len, out_tokens,
                            stream=None):
    """Greedy acceptance without a plan or workspace, for callers that must not allocate device memory
    (its scratch is a fixed array inside the library).  cu_q: int32 CUDA tensor [batch + 1]."""
    assert logits.dim() == 2 and logits.stride(1) == 1 and logits.dtype == torch.float32 and logits.is_cuda
    _chk(_lib.as_accept_greedy_static(batch, total_q, max_draft, _dptr(cu_q, torch.int32),
                                      C.c_void_p(logits.data_ptr()), logits.stride(0), vocab,
                                      _dptr(draft_tokens, torch.int32, True), _dptr(accept_len, torch.int32),
                                      _dptr(out_tokens, torch.int32), _stream(stream)), "as_accept_greedy_static")


def as_plan_preview(plan: Plan, kind: int, seq_lens, draft_lens, num_ctas: int = 0):
    """Host-only: (items int32 [n, 5] = (req, kv_head, key_begin, key_end, part_row), cta_first int32 [P+1])."""
    seq, dl = _host_i32(seq_lens), _host_i32(draft_lens)
    n, P = C.c_int(0), C.c_int(0)
    _chk(_lib.as_plan_preview(plan.handle, kind, num_ctas, len(seq), seq.ctypes.data_as(C.c_void_p),
                              dl.ctypes.data_as(C.c_void_p), None, 0, None, C.byref(n), C.byref(P)), "as_plan_preview")
    items = np.zeros((max(n.value, 1), 5), dtype=np.int32)
    cta_first = np.zeros(P.value + 1, dtype=np.int32)
    _chk(_lib.as_plan_preview(plan.handle, kind, P.value, len(seq), seq.ctypes.data_as(C.c_void_p),
                              dl.ctypes.data_as(C.c_void_p), items.ctypes.data_as(C.c_void_p), n.value,
                              cta_first.ctypes.data_as(C.c_void_p), C.byref(n), C.byref(P)), "as_plan_preview")
    return items[: n.value], cta_first


def as_budget(agree_count, num_candidates, prefix_len, alpha: float, g_min: float, max_len: int = 0):
    """Host-only: redundancy-aware draft lengths (Eq. 1-3).  Returns (draft_lens int32 [B], scores float64 [B])."""
    c, n, ln = _host_i32(agree_count), _host_i32(num_candidates), _host_i32(prefix_len)
    if not (len(c) == len(n) == len(ln)):
        raise ValueError("as_budget: arrays of different lengths")
    out = np.zeros(len(c), dtype=np.int32)
    g = np.zeros(len(c), dtype=np.float64)
    _chk(_lib.as_budget(len(c), c.ctypes.data_as(C.c_void_p), n.ctypes.data_as(C.c_void_p), ln.ctypes.data_as(C.c_void_p),
                        float(alpha), float(g_min), int(max_len), out.ctypes.data_as(C.c_void_p),
                        g.ctypes.data_as(C.c_void_p)), "as_budget")
    return out, g


class Drafter:
    """Host-only structure-isolated drafter (Sec. 4.1): thin wrapper over the as_drafter_* calls."""

    def __init__(self, token_strings):
        toks = [bytes(t) for t in token_strings]
        # (c_char_p stops at a NUL when read back, not when passed in: the library copies token_bytes[t] bytes)
        bufs = [C.create_string_buffer(t, len(t) + 1) for t in toks]
        arr = (C.c_char_p * len(toks))(*[C.cast(b, C.c_char_p) for b in bufs])
        lens = np.asarray([len(t) for t in toks], dtype=np.int32)
        self.handle = C.c_void_p()
        _chk(_lib.as_drafter_create(C.byref(self.handle), arr, lens.ctypes.data_as(C.c_void_p), len(toks)), "as_drafter_create")

    def __del__(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.as_drafter_destroy(self.handle)
            self.handle = None

    def open(self, agent: int, query: int, start_tags, end_tags) -> int:
        assert len(start_tags) == len(end_tags)
        st = (C.c_char_p * len(start_tags))(*[bytes(t) for t in start_tags])
        en = (C.c_char_p * len(end_tags))(*[bytes(t) for t in end_tags])
        req = C.c_int(-1)
        _chk(_lib.as_drafter_open(self.handle, agent, query, st, en, len(start_tags), C.byref(req)), "as_drafter_open")
        return int(req.value)

    def close(self, request: int) -> None:
        _chk(_lib.as_drafter_close(self.handle, request), "as_drafter_close")

    def forget(self, agent: int, query: int) -> None:
        _chk(_lib.as_drafter_forget(self.handle, agent, query), "as_drafter_forget")

    def feed(self, request: int, tokens) -> None:
        t = _host_i32(tokens)
        _chk(_lib.as_drafter_feed(self.handle, request, t.ctypes.data_as(C.c_void_p), len(t)), "as_drafter_feed")

    def block(self, request: int) -> int:
        return int(_lib.as_drafter_block(self.handle, request))

    def propose(self, request: int, match_len: int, max_len: int):
        """(CT as a list of token ids, n candidates, c that agree on CT): the inputs of as_budget for this request."""
        out = np.zeros(max_len, dtype=np.int32)
        ln, n, c = C.c_int(0), C.c_int(0), C.c_int(0)
        _chk(_lib.as_drafter_propose(self.handle, request, match_len, max_len, out.ctypes.data_as(C.c_void_p), C.byref(ln),
                                     C.byref(n), C.byref(c)), "as_drafter_propose")
        return [int(x) for x in out[:ln.value]], int(n.value), int(c.value)


# ------------------------------------------------------------------ convenience for tests and the benchmark

class VerifyStep:
    """Device-side state of one workload batch plus a plan: the calls a serving loop would make.
    Pure plumbing (tensor allocation and the four library calls in order)."""

    def __init__(self, batch, device="cuda", attn_impl=AS_ATTN_AUTO, max_batch=None):
        dev = torch.device(device)
        self.b = batch
        self.dev = dev
        kinds = [dict(num_q_heads=batch.num_q_heads, num_kv_heads=batch.num_kv_heads, head_dim=batch.head_dim,
                      block_size=batch.block_size, window=k.window,
                      sinks=None if k.sinks is None else k.sinks.to(dev, torch.float32).contiguous())
                 for k in batch.kinds]
        self.plan = as_plan_create(kinds, max_batch or max(batch.batch, 1), batch.k_max, batch.max_blocks,
                                   batch.num_blocks, dev.index or 0)
        if attn_impl != AS_ATTN_AUTO:
            as_plan_set_attn_impl(self.plan, attn_impl)
        self.ws = torch.empty(as_plan_workspace_bytes(self.plan), dtype=torch.uint8, device=dev)
        as_plan_bind(self.plan, self.ws)
        self.block_table = torch.as_tensor(batch.block_table, device=dev).contiguous()
        self.seq_lens = torch.as_tensor(batch.seq_lens, device=dev).contiguous()
        self.layers = [type(L)(*(getattr(L, f).to(dev) for f in ("q", "k_new", "v_new", "k_pool", "v_pool")))
                       for L in batch.layers]
        self.out = [torch.empty_like(L.q) for L in self.layers]
        self.lse = [torch.empty(L.q.shape[:2], dtype=torch.float32, device=dev) for L in self.layers]
        to = lambda a, dt: None if a is None else torch.as_tensor(a, device=dev).to(dt).contiguous()
        self.logits = None if batch.logits is None else batch.logits.to(dev)
        self.draft_tokens = to(batch.draft_tokens, torch.int32)
        if self.draft_tokens is not None and self.draft_tokens.numel() == 0:   # a step without drafts: keep a valid pointer
            self.draft_tokens = torch.zeros(1, dtype=torch.int32, device=dev)
        self.draft_probs = None if batch.draft_probs is None else batch.draft_probs.to(dev)
        self.temperature = to(batch.temperature, torch.float32)
        self.u, self.w = to(batch.u, torch.float32), to(batch.w, torch.float32)
        self.accept_len = torch.zeros(max(batch.batch, 1), dtype=torch.int32, device=dev)
        self.out_tokens = torch.zeros((max(batch.batch, 1), batch.k_max + 1), dtype=torch.int32, device=dev)
        self.freed = torch.zeros(max(batch.batch, 1) * (batch.k_max // batch.block_size + 2), dtype=torch.int32, device=dev)
        self.freed_count = torch.zeros(1, dtype=torch.int32, device=dev)
        self._args = {}

    # The tensors behind a VerifyStep never move, so each call's pointer arguments are marshalled once and
    # reused: at small batches a step is bound by these host-side calls, not by the GPU.
    def _cached(self, key, build):
        args = self._args.get(key)
        if args is None:
            args = self._args[key] = build()
        return args

    def rebind(self):
        """Call after replacing one of this object's tensors: the calls marshal their pointers afresh."""
        self._args.clear()

    def set_batch(self, batch):
        """Plans the following steps for another batch of the same shape limits (its host length arrays); the
        device tensors stay the ones this object owns."""
        self.b = batch
        self._args.pop("plan", None)

    def plan_step(self, stream=None):
        def build():
            seq, dl = _host_i32(self.b.seq_lens), _host_i32(self.b.draft_lens)
            self._plan_host = (seq, dl, C.c_int(0))                      # kept alive behind the pointers
            return (self.plan.handle, len(seq), seq.ctypes.data_as(C.c_void_p), dl.ctypes.data_as(C.c_void_p),
                    _dptr(self.block_table, torch.int32), None, 0, C.byref(self._plan_host[2]))
        _chk(_lib.as_plan(*self._cached("plan", build), _stream(stream)), "as_plan")
        return 0

    def plan_step_device(self, batch: int, draft_lens: torch.Tensor, stream=None):
        """Plans the step on the device from this object's device seq_lens and a device draft_lens tensor."""
        as_plan_device(self.plan, batch, self.seq_lens, draft_lens, self.block_table, stream=stream)

    def attn(self, kind=0, stream=None):
        def build():
            L, bf = self.layers[kind], torch.bfloat16
            return (self.plan.handle, kind, _dptr(L.q, bf), _dptr(L.k_new, bf), _dptr(L.v_new, bf), _dptr(L.k_pool, bf),
                    _dptr(L.v_pool, bf), _dptr(self.block_table, torch.int32), _dptr(self.out[kind], bf),
                    _dptr(self.lse[kind], torch.float32, True))
        _chk(_lib.as_verify_attn(*self._cached(("attn", kind), build), _stream(stream)), "as_verify_attn")

    def accept(self, stream=None):
        def build():
            f32, i32 = torch.float32, torch.int32
            lg, dp = self.logits, self.draft_probs
            assert lg.dim() == 2 and lg.stride(1) == 1 and lg.is_cuda and lg.dtype == f32
            assert dp is None or dp.stride(0) == lg.stride(0), "draft_probs must share the row stride of logits"
            return (self.plan.handle, C.c_void_p(lg.data_ptr()), lg.stride(0), self.b.vocab,
                    _dptr(self.draft_tokens, i32, True), None if dp is None else C.c_void_p(dp.data_ptr()),
                    _dptr(self.temperature, f32, True), _dptr(self.u, f32, True), _dptr(self.w, f32, True),
                    _dptr(self.accept_len, i32), _dptr(self.out_tokens, i32))
        _chk(_lib.as_accept(*self._cached("accept", build), _stream(stream)), "as_accept")

    def commit(self, flags=0, kind=0, stream=None):
        def build():
            L, i32 = self.layers[kind], torch.int32
            return (self.plan.handle, _dptr(self.accept_len, i32), _dptr(self.seq_lens, i32), _dptr(self.block_table, i32),
                    _dptr(self.freed, i32), _dptr(self.freed_count, i32), flags, _dptr(L.k_pool, torch.bfloat16, True),
                    _dptr(L.v_pool, torch.bfloat16, True))
        _chk(_lib.as_kv_commit(*self._cached(("commit", flags, kind), build), _stream(stream)), "as_kv_commit")
