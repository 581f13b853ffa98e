"""Thin ctypes binding of libpsa's C ABI (include/psa.h).

Argument marshalling only: every step of the path runs inside the library's
CUDA kernels.  torch is used for device memory and streams.  There is no CPU
fallback: if the shared library is missing or a call fails, an exception is
raised.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libpsa.so")
_lib = None

PSA_PLAN_HOST_ONLY = 1
PSA_STATIC_SCRATCH_BYTES = 32 * 1024 * 1024
PSA_DTYPE_F32, PSA_DTYPE_BF16 = 0, 1
PSA_DEVSTAT_WAIT_EXPIRED, PSA_DEVSTAT_BAD_TARGET, PSA_DEVSTAT_BAD_SEGMENT, PSA_DEVSTAT_OUT_OF_BOUNDS = 1, 2, 4, 8

EXPORTED_SYMBOLS = (
    "psa_status_string", "psa_plan", "psa_plan_upload", "psa_plan_destroy", "psa_plan_stats",
    "psa_plan_counts", "psa_plan_export", "psa_fwd", "psa_bwd", "dpo_logp", "psa_profile_events",
    "psa_bwd_static_scratch", "dpo_loss", "dpo_logp_bwd", "psa_pack_ffd", "psa_position_ids", "psa_rope",
    "psa_step_host_arena_bytes", "psa_step_host", "simpo_loss", "orpo_loss", "psa_bwd_f32",
    "psa_check_device_status", "psa_selftest_wait_expiry", "psa_logp_labels", "psa_pack_ffd_emit",
    "psa_selftest_bounds",
)


class PsaError(RuntimeError):
    def __init__(self, fn, code, text):
        super().__init__("%s failed: status %d (%s)" % (fn, code, text))
        self.code = code


def load_library():
    """Loads libpsa.so (building it first if the sources are newer and nvcc is
    present).  Raises if the library cannot be had.  With PSA_DEBUG_LIB=1 in the environment the
    debug library (libpsa_debug.so: the same code with checked global indices) is loaded instead."""
    global _lib
    if _lib is not None:
        return _lib
    from . import build as _build
    debug = os.environ.get("PSA_DEBUG_LIB", "") not in ("", "0")
    path = _build.LIB_DEBUG if debug else _LIB_PATH
    try:
        _build.build(debug=debug)
    except Exception:
        if not os.path.exists(path):
            raise
    if not os.path.exists(path):
        raise RuntimeError("%s is missing and could not be built" % path)
    lib = C.CDLL(path)
    vp, i32, i64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
    lib.psa_status_string.restype = C.c_char_p
    lib.psa_status_string.argtypes = [C.c_int]
    lib.psa_plan.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, f32, i32, vp, C.POINTER(vp)]
    lib.psa_plan_upload.argtypes = [vp, vp]
    lib.psa_plan_destroy.argtypes = [vp]
    lib.psa_plan_stats.argtypes = [vp, C.POINTER(i64), C.POINTER(i64), C.POINTER(i64), C.POINTER(i64),
                                   C.POINTER(C.c_size_t)]
    lib.psa_plan_counts.argtypes = [vp, i32, C.POINTER(i32), C.POINTER(i32)]
    lib.psa_plan_export.argtypes = [vp, i32, vp, vp]
    lib.psa_fwd.argtypes = [vp] * 8
    lib.psa_bwd.argtypes = [vp] * 13
    lib.psa_bwd_static_scratch.argtypes = [vp] * 12
    lib.psa_bwd_f32.argtypes = [vp] * 13
    lib.psa_check_device_status.argtypes = [i32]
    lib.psa_selftest_wait_expiry.argtypes = [vp, i64, vp, vp]
    lib.psa_selftest_bounds.argtypes = [vp, vp, vp]
    lib.psa_logp_labels.argtypes = [vp, vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, C.POINTER(i32)]
    lib.psa_pack_ffd_emit.argtypes = [vp, vp, vp, i32, i32, i32, vp, C.POINTER(i32), vp, vp, vp, vp, vp, vp]
    lib.psa_profile_events.argtypes = [i32, vp, vp]
    lib.dpo_loss.argtypes = [vp, vp, i32, f32, vp, vp, vp]
    lib.simpo_loss.argtypes = [vp, vp, i32, f32, f32, vp, vp, vp, vp]
    lib.orpo_loss.argtypes = [vp, vp, i32, f32, vp, vp, vp, vp]
    lib.psa_step_host.argtypes = [vp] * 11 + [C.c_size_t, vp, vp]
    lib.psa_pack_ffd.argtypes = [vp, i32, i32, vp, C.POINTER(i32)]
    lib.psa_position_ids.argtypes = [vp, vp, vp, vp, i32, vp]
    lib.psa_rope.argtypes = [vp, vp, vp, i64, i32, i32, f32, vp]
    lib.dpo_logp_bwd.argtypes = [vp, i32, i64, i64, i64, vp, vp, vp, vp, vp, i32, i32, vp, vp, vp, vp]
    lib.dpo_logp.argtypes = [vp, i32, i64, i64, i64, vp, vp, vp, vp, vp, i32, i32, vp, vp, vp]
    for name in EXPORTED_SYMBOLS:
        if name == "psa_step_host_arena_bytes":
            lib.psa_step_host_arena_bytes.restype = C.c_size_t
            lib.psa_step_host_arena_bytes.argtypes = [C.c_void_p]
        elif name != "psa_status_string":
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def _check(fn, code):
    if code != 0:
        raise PsaError(fn, code, load_library().psa_status_string(code).decode())


def _i32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _stream(stream):
    if stream is not None:
        return C.c_void_p(int(stream))
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream) if torch.cuda.is_available() else C.c_void_p(0)


def _ptr(t):
    return C.c_void_p(0) if t is None else C.c_void_p(t.data_ptr())


def _want(t, name, shape, dtype, cuda=True, placement=True):
    """Raises ValueError unless tensor `t` has exactly this shape and dtype, is contiguous and
    lives where the call needs it.  The kernels size their tensor maps and grids from the plan
    alone, so a tensor of another pack, or a buffer that is too small, would be read or written
    past its end: it has to be refused here."""
    if tuple(t.shape) != tuple(shape):
        raise ValueError("%s: shape %s, the plan needs %s" % (name, tuple(t.shape), tuple(shape)))
    if t.dtype != dtype:
        raise ValueError("%s: dtype %s, expected %s" % (name, t.dtype, dtype))
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % name)
    if placement and bool(t.is_cuda) != bool(cuda):
        raise ValueError("%s must be a %s tensor" % (name, "CUDA" if cuda else "host"))


def _want_attention(plan, bf16, f32=(), lse=None, cuda=True):
    """Checks the attention tensors of a call against the plan: `bf16` and `f32` are lists of
    (name, tensor, "q" or "kv").  Shapes and dtypes of all of them first, then where they live."""
    import torch
    T, d = plan.total_tokens, plan.head_dim
    heads = {"q": plan.n_q_heads, "kv": plan.n_kv_heads}
    for placement in (False, True):
        for name, t, kind in bf16:
            _want(t, name, (T, heads[kind], d), torch.bfloat16, cuda, placement)
        for name, t, kind in f32:
            _want(t, name, (T, heads[kind], d), torch.float32, cuda, placement)
        if lse is not None:
            _want(lse, "lse", (plan.n_q_heads, T), torch.float32, cuda, placement)


class Plan:
    """Owner of a psa_plan_t*.  One plan serves every layer of a step."""

    def __init__(self, handle, n_q_heads, n_kv_heads, head_dim):
        self._h = handle
        self.n_q_heads, self.n_kv_heads, self.head_dim = n_q_heads, n_kv_heads, head_dim
        lib = load_library()
        T, U, live, part = C.c_int64(), C.c_int64(), C.c_int64(), C.c_int64()
        ws = C.c_size_t()
        _check("psa_plan_stats", lib.psa_plan_stats(self._h, C.byref(T), C.byref(U), C.byref(live), C.byref(part),
                                                    C.byref(ws)))
        self.total_tokens, self.useful_pairs = T.value, U.value
        self.live_tiles, self.partial_tiles, self.bwd_workspace_bytes = live.value, part.value, ws.value

    def upload(self, stream=None):
        _check("psa_plan_upload", load_library().psa_plan_upload(self._h, _stream(stream)))

    def export(self, direction):
        """Tile records int32 [n_tiles, 8] and entries int32 [n_entries] of the
        forward (0) or transposed (1) map."""
        lib = load_library()
        nt, ne = C.c_int32(), C.c_int32()
        _check("psa_plan_counts", lib.psa_plan_counts(self._h, direction, C.byref(nt), C.byref(ne)))
        tiles = np.zeros((max(nt.value, 1), 8), dtype=np.int32)
        entries = np.zeros(max(ne.value, 1), dtype=np.int32)
        _check("psa_plan_export", lib.psa_plan_export(self._h, direction, tiles.ctypes.data, entries.ctypes.data))
        return tiles[:nt.value], entries[:ne.value]

    def close(self):
        if self._h:
            h, self._h = self._h, None
            load_library().psa_plan_destroy(h)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def psa_plan(cu_seqlens, prefix_len, chosen_len, rejected_len, n_q_heads, n_kv_heads, head_dim,
             softmax_scale=0.0, host_only=False, stream=None) -> Plan:
    lib = load_library()
    cu, P, Cc, R = _i32(cu_seqlens), _i32(prefix_len), _i32(chosen_len), _i32(rejected_len)
    n = len(P)
    if len(cu) != n + 1 or len(Cc) != n or len(R) != n:
        raise ValueError("cu_seqlens must have n+1 entries and the three length arrays n entries")
    out = C.c_void_p()
    flags = PSA_PLAN_HOST_ONLY if host_only else 0
    st = C.c_void_p(0) if host_only else _stream(stream)
    _check("psa_plan", lib.psa_plan(cu.ctypes.data, P.ctypes.data, Cc.ctypes.data, R.ctypes.data, n, n_q_heads,
                                    n_kv_heads, head_dim, float(softmax_scale), flags, st, C.byref(out)))
    return Plan(out, n_q_heads, n_kv_heads, head_dim)


def psa_fwd(plan: Plan, q, k, v, o=None, lse=None, status=None, stream=None):
    """q [T,Hq,d], k, v [T,Hkv,d] bf16 CUDA tensors -> (o [T,Hq,d] bf16, lse [Hq,T] fp32)."""
    import torch
    T = plan.total_tokens
    if o is None:
        o = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((plan.n_q_heads, T), dtype=torch.float32, device=q.device)
    _want_attention(plan, [("q", q, "q"), ("k", k, "kv"), ("v", v, "kv"), ("o", o, "q")], lse=lse)
    _check("psa_fwd", load_library().psa_fwd(plan._h, _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(status),
                                             _stream(stream)))
    return o, lse


def psa_bwd(plan: Plan, d_o, q, k, v, o, lse, dq=None, dk=None, dv=None, workspace=None, status=None, stream=None):
    """Returns (dq [T,Hq,d], dk, dv [T,Hkv,d]) bf16."""
    import torch
    if dq is None:
        dq = torch.empty_like(q)
    if dk is None:
        dk = torch.empty_like(k)
    if dv is None:
        dv = torch.empty_like(v)
    _want_attention(plan, [("d_o", d_o, "q"), ("q", q, "q"), ("k", k, "kv"), ("v", v, "kv"), ("o", o, "q"),
                           ("dq", dq, "q"), ("dk", dk, "kv"), ("dv", dv, "kv")], lse=lse)
    if workspace is None:
        workspace = torch.empty(max(plan.bwd_workspace_bytes, 256), dtype=torch.uint8, device=q.device)
    if not workspace.is_cuda or workspace.numel() * workspace.element_size() < plan.bwd_workspace_bytes:
        raise ValueError("workspace: a CUDA buffer of at least %d bytes is needed" % plan.bwd_workspace_bytes)
    _check("psa_bwd", load_library().psa_bwd(plan._h, _ptr(d_o), _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse),
                                             _ptr(dq), _ptr(dk), _ptr(dv), _ptr(workspace), _ptr(status),
                                             _stream(stream)))
    return dq, dk, dv


def psa_bwd_f32(plan: Plan, d_o, q, k, v, o, lse, dq=None, dk=None, dv=None, workspace=None, status=None, stream=None):
    """psa_bwd with fp32 gradient outputs: returns (dq [T,Hq,d], dk, dv [T,Hkv,d]) fp32, the
    kernels' fp32 accumulators written out without the final rounding to bf16."""
    import torch
    f32 = lambda t: torch.empty(t.shape, dtype=torch.float32, device=t.device)
    dq = f32(q) if dq is None else dq
    dk = f32(k) if dk is None else dk
    dv = f32(v) if dv is None else dv
    _want_attention(plan, [("d_o", d_o, "q"), ("q", q, "q"), ("k", k, "kv"), ("v", v, "kv"), ("o", o, "q")],
                    f32=[("dq", dq, "q"), ("dk", dk, "kv"), ("dv", dv, "kv")], lse=lse)
    if workspace is None:
        workspace = torch.empty(max(plan.bwd_workspace_bytes, 256), dtype=torch.uint8, device=q.device)
    if not workspace.is_cuda or workspace.numel() * workspace.element_size() < plan.bwd_workspace_bytes:
        raise ValueError("workspace: a CUDA buffer of at least %d bytes is needed" % plan.bwd_workspace_bytes)
    _check("psa_bwd_f32", load_library().psa_bwd_f32(plan._h, _ptr(d_o), _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse),
                                                     _ptr(dq), _ptr(dk), _ptr(dv), _ptr(workspace), _ptr(status),
                                                     _stream(stream)))
    return dq, dk, dv


def psa_check_device_status(word: int) -> int:
    """Status code for a device status word read back by the caller: 0 ok, 7 a bounded wait
    expired (outputs invalid), 6 bad labels."""
    return int(load_library().psa_check_device_status(int(word)))


def psa_selftest_wait_expiry(status, limit_clocks, waited=None, stream=None):
    """Runs the library's bounded wait on a barrier that nothing completes; after `limit_clocks`
    SM clocks the wait gives up and ORs PSA_DEVSTAT_WAIT_EXPIRED into `status` (int32 CUDA [1]).
    `waited` (int64 CUDA [1], optional) receives the clocks the wait lasted."""
    _check("psa_selftest_wait_expiry",
           load_library().psa_selftest_wait_expiry(_ptr(status), int(limit_clocks), _ptr(waited), _stream(stream)))


def psa_selftest_bounds(status, result, stream=None):
    """Runs one index inside and one outside a small tensor through the debug library's checked-index
    macro (see psa.h); `status`, `result` are int32 CUDA [1]."""
    _check("psa_selftest_bounds", load_library().psa_selftest_bounds(_ptr(status), _ptr(result), _stream(stream)))


def dpo_logp(logits, targets, segment_ids, n_segments, fork_rows=None, fork_targets=None, fork_segments=None,
             out=None, status=None, stream=None):
    """logits [n_rows, vocab] fp32 or bf16 (rows may be strided), targets / segment_ids
    int32 [n_rows], optional fork arrays int32 [n_forks] -> out fp32 [n_segments]."""
    import torch
    assert logits.is_cuda and logits.dim() == 2 and logits.stride(1) == 1
    dt = {torch.float32: PSA_DTYPE_F32, torch.bfloat16: PSA_DTYPE_BF16}[logits.dtype]
    n_rows, vocab = logits.shape
    for t in (targets, segment_ids):
        assert t.is_cuda and t.dtype == torch.int32 and t.is_contiguous() and t.numel() == n_rows
    n_forks = 0 if fork_rows is None else int(fork_rows.numel())
    if n_forks:
        for t in (fork_rows, fork_targets, fork_segments):
            assert t.is_cuda and t.dtype == torch.int32 and t.is_contiguous() and t.numel() == n_forks
    else:
        fork_rows = fork_targets = fork_segments = None
    if out is None:
        out = torch.empty(n_segments, dtype=torch.float32, device=logits.device)
    _check("dpo_logp", load_library().dpo_logp(_ptr(logits), dt, n_rows, vocab, logits.stride(0) if n_rows > 1 else vocab,
                                               _ptr(targets), _ptr(segment_ids), _ptr(fork_rows), _ptr(fork_targets),
                                               _ptr(fork_segments), n_forks, n_segments, _ptr(out), _ptr(status),
                                               _stream(stream)))
    return out


def psa_profile_events(which, start=None, stop=None, created=False):
    """Registers (or, with None, removes) a pair of torch.cuda.Event recorded right
    before and after one kernel: 0 = psa_fwd, 1 = main psa_bwd kernel, 2 = dpo_logp,
    3 = psa_bwd's delta / clear helper, 4 = psa_bwd's convert helper.  `created=True` says the
    events have been recorded before (so their CUDA events exist) and skips the dummy record."""
    if start is not None and not created:
        # torch creates the underlying cudaEvent lazily, on the first record
        start.record()
        stop.record()
    a = C.c_void_p(0) if start is None else C.c_void_p(start.cuda_event)
    b = C.c_void_p(0) if stop is None else C.c_void_p(stop.cuda_event)
    _check("psa_profile_events", load_library().psa_profile_events(which, a, b))


def psa_bwd_static_scratch(plan: Plan, d_o, q, k, v, o, lse, dq, dk, dv, status=None, stream=None):
    """psa_bwd for callers that cannot provide a workspace (for instance because all device
    memory already belongs to the framework's allocator): the scratch is a fixed 32 MiB
    array inside the library.  Nothing is allocated here either: the three gradient tensors
    must be passed in.  Plans whose scratch need exceeds PSA_STATIC_SCRATCH_BYTES raise
    PsaError (status 3).  Calls that overlap on the GPU share the array and must be serialised."""
    _want_attention(plan, [("d_o", d_o, "q"), ("q", q, "q"), ("k", k, "kv"), ("v", v, "kv"), ("o", o, "q"),
                           ("dq", dq, "q"), ("dk", dk, "kv"), ("dv", dv, "kv")], lse=lse)
    _check("psa_bwd_static_scratch",
           load_library().psa_bwd_static_scratch(plan._h, _ptr(d_o), _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse),
                                                 _ptr(dq), _ptr(dk), _ptr(dv), _ptr(status), _stream(stream)))
    return dq, dk, dv


def psa_step_host_arena_bytes(plan: Plan) -> int:
    """Bytes of device memory psa_step_host needs as its arena for this plan."""
    return int(load_library().psa_step_host_arena_bytes(plan._h))


def psa_step_host(plan: Plan, h_q, h_k, h_v, h_do, h_o, h_lse, h_dq, h_dk, h_dv, arena, status=None, stream=None):
    """Forward + backward on HOST tensors (pinned for asynchronous copies): enqueues the
    copies in, psa_fwd, psa_bwd and the copies out on `stream` and returns without
    synchronising.  `arena` is a uint8 CUDA tensor of at least psa_step_host_arena_bytes(plan)
    bytes; nothing is allocated here."""
    import torch
    _want_attention(plan, [("h_q", h_q, "q"), ("h_k", h_k, "kv"), ("h_v", h_v, "kv"), ("h_do", h_do, "q"),
                           ("h_o", h_o, "q"), ("h_dq", h_dq, "q"), ("h_dk", h_dk, "kv"), ("h_dv", h_dv, "kv")],
                    lse=h_lse, cuda=False)
    if not (arena.is_cuda and arena.dtype == torch.uint8 and arena.is_contiguous()):
        raise ValueError("arena must be a contiguous uint8 CUDA tensor")
    _check("psa_step_host",
           load_library().psa_step_host(plan._h, _ptr(h_q), _ptr(h_k), _ptr(h_v), _ptr(h_do), _ptr(h_o), _ptr(h_lse),
                                        _ptr(h_dq), _ptr(h_dk), _ptr(h_dv), _ptr(arena),
                                        C.c_size_t(arena.numel()), _ptr(status), _stream(stream)))


def dpo_loss(policy_logps, ref_logps, beta, stream=None):
    """policy_logps, ref_logps fp32 CUDA [2n] (2s chosen, 2s+1 rejected) -> (loss fp32 [1], coef fp32 [2n])
    with coef = d loss / d policy_logps; loss = mean_s -log sigmoid(beta * margin_s)."""
    import torch
    assert policy_logps.is_cuda and policy_logps.dtype == torch.float32 and policy_logps.is_contiguous()
    assert ref_logps.shape == policy_logps.shape and ref_logps.dtype == torch.float32 and ref_logps.is_contiguous()
    n = policy_logps.numel() // 2
    loss = torch.empty(1, dtype=torch.float32, device=policy_logps.device)
    coef = torch.empty(2 * n, dtype=torch.float32, device=policy_logps.device)
    _check("dpo_loss", load_library().dpo_loss(_ptr(policy_logps), _ptr(ref_logps), n, float(beta), _ptr(loss),
                                              _ptr(coef), _stream(stream)))
    return loss, coef


def simpo_loss(policy_logps, lengths, beta, gamma, status=None, stream=None):
    """policy_logps fp32 CUDA [2n], lengths int32 CUDA [2n] (scored tokens per response) ->
    (loss fp32 [1], coef fp32 [2n]); loss = mean_s -log sigmoid(beta * (lp_c/len_c - lp_r/len_r) - gamma)."""
    import torch
    assert policy_logps.is_cuda and policy_logps.dtype == torch.float32 and policy_logps.is_contiguous()
    assert lengths.is_cuda and lengths.dtype == torch.int32 and lengths.shape == policy_logps.shape
    n = policy_logps.numel() // 2
    loss = torch.empty(1, dtype=torch.float32, device=policy_logps.device)
    coef = torch.empty(2 * n, dtype=torch.float32, device=policy_logps.device)
    _check("simpo_loss", load_library().simpo_loss(_ptr(policy_logps), _ptr(lengths), n, float(beta),
                                                  float(gamma), _ptr(loss), _ptr(coef), _ptr(status),
                                                  _stream(stream)))
    return loss, coef


def orpo_loss(policy_logps, lengths, lam, status=None, stream=None):
    """policy_logps fp32 CUDA [2n], lengths int32 CUDA [2n] -> (loss fp32 [1], coef fp32 [2n]);
    loss = mean_s  -lp_c/len_c + lam * -log sigmoid(log odds ratio of the mean-token likelihoods)."""
    import torch
    assert policy_logps.is_cuda and policy_logps.dtype == torch.float32 and policy_logps.is_contiguous()
    assert lengths.is_cuda and lengths.dtype == torch.int32 and lengths.shape == policy_logps.shape
    n = policy_logps.numel() // 2
    loss = torch.empty(1, dtype=torch.float32, device=policy_logps.device)
    coef = torch.empty(2 * n, dtype=torch.float32, device=policy_logps.device)
    _check("orpo_loss", load_library().orpo_loss(_ptr(policy_logps), _ptr(lengths), n, float(lam), _ptr(loss),
                                                _ptr(coef), _ptr(status), _stream(stream)))
    return loss, coef


def dpo_logp_bwd(logits, targets, segment_ids, coef, fork_rows=None, fork_targets=None, fork_segments=None,
                 dlogits=None, status=None, stream=None):
    """Gradient of sum_g coef[g] * dpo_logp(...)[g] with respect to the logits; same dtype and
    row stride as `logits`."""
    import torch
    assert logits.is_cuda and logits.dim() == 2 and logits.stride(1) == 1
    dt = {torch.float32: PSA_DTYPE_F32, torch.bfloat16: PSA_DTYPE_BF16}[logits.dtype]
    n_rows, vocab = logits.shape
    n_forks = 0 if fork_rows is None else int(fork_rows.numel())
    if not n_forks:
        fork_rows = fork_targets = fork_segments = None
    assert coef.is_cuda and coef.dtype == torch.float32 and coef.is_contiguous()
    if dlogits is None:
        dlogits = torch.empty_strided(logits.shape, logits.stride(), dtype=logits.dtype, device=logits.device)
    assert dlogits.dtype == logits.dtype and dlogits.stride() == logits.stride()
    _check("dpo_logp_bwd", load_library().dpo_logp_bwd(
        _ptr(logits), dt, n_rows, vocab, logits.stride(0) if n_rows > 1 else vocab, _ptr(targets), _ptr(segment_ids),
        _ptr(fork_rows), _ptr(fork_targets), _ptr(fork_segments), n_forks, int(coef.numel()), _ptr(coef),
        _ptr(dlogits), _ptr(status), _stream(stream)))
    return dlogits


def psa_pack_ffd(unit_len, capacity):
    """First-fit-decreasing packing of units (P + C + R per sample) into packs of `capacity`
    tokens.  Returns (bin_of_unit int32 [n], n_bins).  Host only."""
    lens = _i32(unit_len)
    bins = np.zeros(max(len(lens), 1), dtype=np.int32)
    n_bins = C.c_int32()
    _check("psa_pack_ffd", load_library().psa_pack_ffd(lens.ctypes.data, len(lens), int(capacity), bins.ctypes.data,
                                                      C.byref(n_bins)))
    return bins[:len(lens)], n_bins.value


def psa_pack_ffd_emit(prefix_len, chosen_len, rejected_len, capacity, paired=False):
    """Packs the units with psa_pack_ffd and lays every pack out for psa_plan.  Returns
    (bin_of_unit int32 [n], packs) where packs is a list of dicts with the keys cu_seqlens,
    prefix_len, chosen_len, rejected_len (int32 arrays, ready for psa_plan) and units (the
    source unit of each sample).  paired=True gives the unshared baseline layout: two samples
    (P, C, 0), (P, R, 0) per unit.  Host only."""
    P, Cc, R = _i32(prefix_len), _i32(chosen_len), _i32(rejected_len)
    n = len(P)
    m = n * (2 if paired else 1)
    bins = np.zeros(max(n, 1), dtype=np.int32)
    off = np.zeros(n + 1, dtype=np.int32)
    unit, oP, oC, oR = (np.zeros(max(m, 1), dtype=np.int32) for _ in range(4))
    cu = np.zeros(m + n + 1, dtype=np.int32)
    n_packs = C.c_int32()
    _check("psa_pack_ffd_emit", load_library().psa_pack_ffd_emit(
        P.ctypes.data, Cc.ctypes.data, R.ctypes.data, n, int(capacity), 1 if paired else 0, bins.ctypes.data,
        C.byref(n_packs), off.ctypes.data, unit.ctypes.data, oP.ctypes.data, oC.ctypes.data, oR.ctypes.data,
        cu.ctypes.data))
    packs = []
    for b in range(n_packs.value):
        lo, hi = int(off[b]), int(off[b + 1])
        packs.append({"cu_seqlens": cu[lo + b:hi + b + 1].copy(), "prefix_len": oP[lo:hi].copy(),
                      "chosen_len": oC[lo:hi].copy(), "rejected_len": oR[lo:hi].copy(), "units": unit[lo:hi].copy()})
    return bins[:n], packs


def psa_logp_labels(token_ids, cu_seqlens, prefix_len, chosen_len, rejected_len):
    """Label layout of dpo_logp on the shared layout: returns (targets int32 [T], segment_ids
    int32 [T], fork_rows, fork_targets, fork_segments int32 [n_forks]); response ids 2s = chosen,
    2s+1 = rejected, -1 = row not scored.  Host only."""
    tok, cu = _i32(token_ids), _i32(cu_seqlens)
    P, Cc, R = _i32(prefix_len), _i32(chosen_len), _i32(rejected_len)
    n, T = len(P), int(cu[-1])
    if len(cu) != n + 1 or len(tok) < T:
        raise ValueError("cu_seqlens must have n+1 entries and token_ids at least T entries")
    targets, seg = np.zeros(max(T, 1), dtype=np.int32), np.zeros(max(T, 1), dtype=np.int32)
    fr, ft, fs = (np.zeros(max(n, 1), dtype=np.int32) for _ in range(3))
    nf = C.c_int32()
    _check("psa_logp_labels", load_library().psa_logp_labels(
        tok.ctypes.data, cu.ctypes.data, P.ctypes.data, Cc.ctypes.data, R.ctypes.data, n, targets.ctypes.data,
        seg.ctypes.data, fr.ctypes.data, ft.ctypes.data, fs.ctypes.data, C.byref(nf)))
    k = nf.value
    return targets[:T], seg[:T], fr[:k].copy(), ft[:k].copy(), fs[:k].copy()


def psa_position_ids(cu_seqlens, prefix_len, chosen_len, rejected_len):
    """Position ids int32 [T] of the shared layout: rejected tokens restart right after the prompt."""
    cu, P, Cc, R = _i32(cu_seqlens), _i32(prefix_len), _i32(chosen_len), _i32(rejected_len)
    out = np.zeros(max(int(cu[-1]), 1), dtype=np.int32)
    _check("psa_position_ids", load_library().psa_position_ids(cu.ctypes.data, P.ctypes.data, Cc.ctypes.data,
                                                              R.ctypes.data, len(P), out.ctypes.data))
    return out[:int(cu[-1])]


def psa_rope(x, position_ids, rope_theta=10000.0, out=None, stream=None):
    """Rotary embedding (rotate-half convention) of x [T, H, d] bf16 CUDA with int32 CUDA position ids [T]."""
    import torch
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous() and x.dim() == 3
    assert position_ids.is_cuda and position_ids.dtype == torch.int32 and position_ids.numel() == x.shape[0]
    if out is None:
        out = torch.empty_like(x)
    _check("psa_rope", load_library().psa_rope(_ptr(x), _ptr(out), _ptr(position_ids), x.shape[0], x.shape[1],
                                              x.shape[2], float(rope_theta), _stream(stream)))
    return out
