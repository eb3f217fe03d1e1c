"""Thin ctypes binding of libshotkv.so: argument marshalling only.

Every function has the name and argument order of its C counterpart in
`include/shotkv.h`; tensors are torch tensors whose data pointers are passed
through.  Nothing is computed here, and nothing falls back to the CPU: if the
library is missing or a call fails, a `ShotKVError` is raised.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libshotkv.so")

OK = 0
ERR_INVALID_ARG = -1
ERR_UNSUPPORTED_SHAPE = -2
ERR_BAD_OFFSETS = -3
ERR_WORKSPACE_TOO_SMALL = -4
ERR_CUDA = -5
ERR_TIMEOUT = -6
WARN_BUDGET_BELOW_ALWAYS_KEPT = 1
FLAG_TOKEN_IMPORTANCE = 1

EXPORTS = [
    "shotkv_create", "shotkv_destroy", "shotkv_last_error", "shotkv_version",
    "shotkv_budget_tokens", "shotkv_kept_capacity", "shotkv_validate", "shotkv_workspace_bytes",
    "shotkv_prefill_score", "shotkv_select_shots", "shotkv_compact_kv", "shotkv_prefill_compress",
    "shotkv_host_arena_bytes", "shotkv_prefill_compress_host",
    "shotkv_decode_workspace_bytes", "shotkv_decode_capacity", "shotkv_decode_init", "shotkv_decode_step", "shotkv_decode_step_attend",
    "shotkv_profile_enable", "shotkv_profile_read", "shotkv_launch_count", "shotkv_select_shots_static", "shotkv_plan_pieces",
    "shotkv_set_scoring_mode", "shotkv_repaired_items", "shotkv_set_pipeline_groups",
    "shotkv_set_wait_limit", "shotkv_selftest_bounded_wait", "shotkv_last_scoring_clock",
]


class ShotKVError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"shotkv error {code}: {msg}")
        self.code = code


class Dims(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("B", "L", "H", "Hkv", "d", "N", "W", "S")]


class Policy(C.Structure):
    _fields_ = [("r_p", C.c_float), ("select_mode", C.c_int32), ("r_d", C.c_float),
                ("recompress_every", C.c_int32), ("protect_recent", C.c_int32)]


class DecodeState(C.Structure):
    _fields_ = [("dims", Dims), ("policy", Policy), ("Dcap", C.c_int32), ("Mcap", C.c_int32),
                ("T", C.c_int32), ("n_dec", C.c_int32),
                ("Kd", C.c_void_p), ("Vd", C.c_void_p), ("acc", C.c_void_p), ("born", C.c_void_p),
                ("ws", C.c_void_p), ("ws_bytes", C.c_size_t)]


_lib = None


def lib() -> C.CDLL:
    """Loads libshotkv.so (once).  Raises if it has not been built: there is no fallback."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ShotKVError(ERR_CUDA, f"{LIB_PATH} not found: build it with paper_2502_01941_b200/build.py "
                                    "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH, mode=C.RTLD_GLOBAL)
    vp, i32, sz, u32 = C.c_void_p, C.c_int32, C.c_size_t, C.c_uint32
    PD, PP = C.POINTER(Dims), C.POINTER(Policy)
    sig = {
        "shotkv_create": (C.c_int, [C.POINTER(vp), C.c_int]),
        "shotkv_destroy": (None, [vp]),
        "shotkv_last_error": (C.c_char_p, [vp]),
        "shotkv_version": (C.c_char_p, []),
        "shotkv_budget_tokens": (i32, [PD, PP]),
        "shotkv_kept_capacity": (i32, [PD, PP, vp]),
        "shotkv_validate": (C.c_int, [PD, PP, vp]),
        "shotkv_workspace_bytes": (sz, [PD]),
        "shotkv_prefill_score": (C.c_int, [vp, PD, vp, vp, vp, vp, sz, vp]),
        "shotkv_select_shots": (C.c_int, [vp, PD, PP, vp, vp, vp, vp, vp, vp, i32, vp, sz, vp]),
        "shotkv_select_shots_static": (C.c_int, [vp, PD, PP, vp, vp, vp, vp, vp, vp, i32, vp]),
        "shotkv_compact_kv": (C.c_int, [vp, PD, vp, vp, vp, vp, i32, vp, vp, vp]),
        "shotkv_prefill_compress": (C.c_int, [vp, PD, PP, vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, vp, vp, u32, vp, sz, vp]),
        "shotkv_host_arena_bytes": (sz, [PD, i32]),
        "shotkv_prefill_compress_host": (C.c_int, [vp, PD, PP, vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, vp, vp, sz, vp]),
        "shotkv_decode_workspace_bytes": (sz, [PD, i32]),
        "shotkv_decode_capacity": (i32, [PP, i32]),
        "shotkv_decode_init": (C.c_int, [vp, PD, PP, i32, i32, vp, vp, vp, vp, vp, sz, C.POINTER(DecodeState)]),
        "shotkv_decode_step": (C.c_int, [vp, C.POINTER(DecodeState), vp, vp, vp, vp, vp, vp]),
        "shotkv_decode_step_attend": (C.c_int, [vp, C.POINTER(DecodeState), vp, vp, vp, vp, vp, vp, vp, vp]),
        "shotkv_plan_pieces": (i32, [PD, vp, i32, C.POINTER(i32), C.POINTER(i32), vp, i32]),
        "shotkv_profile_enable": (C.c_int, [vp, C.c_int]),
        "shotkv_profile_read": (C.c_int, [vp, C.c_int, C.POINTER(C.c_float)]),
        "shotkv_launch_count": (C.c_uint64, [vp]),
        "shotkv_set_scoring_mode": (C.c_int, [vp, C.c_int]),
        "shotkv_set_pipeline_groups": (C.c_int, [vp, C.c_int]),
        "shotkv_repaired_items": (C.c_uint64, [vp]),
        "shotkv_last_scoring_clock": (C.c_int, [vp, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]),
        "shotkv_set_wait_limit": (C.c_int, [vp, C.c_int64]),
        "shotkv_selftest_bounded_wait": (C.c_int, [vp, C.c_int64, C.POINTER(i32), vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(L, name)
        fn.restype, fn.argtypes = res, args
    _lib = L
    return L


# ------------------------------------------------------------------ marshalling helpers
def _ptr(t, *, device=None, dtype=None, name="tensor"):
    if t is None:
        return None
    if not isinstance(t, torch.Tensor):
        raise TypeError(f"{name}: expected a torch tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name}: must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name}: expected {dtype}, got {t.dtype}")
    if device == "cuda" and not t.is_cuda:
        raise ValueError(f"{name}: must be a CUDA tensor")
    if device == "cpu" and t.is_cuda:
        raise ValueError(f"{name}: must be a host tensor")
    return C.c_void_p(t.data_ptr())


def _offsets(off) -> np.ndarray:
    a = np.ascontiguousarray(off.cpu().numpy() if isinstance(off, torch.Tensor) else off, dtype=np.int32)
    return a


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def make_dims(B, L, H, Hkv, d, N, W, S) -> Dims:
    return Dims(B, L, H, Hkv, d, N, W, S)


def per_head_dims(dims: Dims) -> Dims:
    """The same tensors read as L*Hkv single-head layers: selection per KV head instead of per layer."""
    return Dims(dims.B, dims.L * dims.Hkv, dims.H // dims.Hkv, 1, dims.d, dims.N, dims.W, dims.S)


def make_policy(r_p=1.0, select_mode=0, r_d=1.0, recompress_every=1, protect_recent=0) -> Policy:
    return Policy(float(r_p), int(select_mode), float(r_d), int(recompress_every), int(protect_recent))


class Context:
    """Owns a shotkv_ctx for one CUDA device."""

    def __init__(self, device: int = 0):
        self._h = C.c_void_p()
        rc = lib().shotkv_create(C.byref(self._h), int(device))
        if rc != 0:
            self._h = C.c_void_p()
            raise ShotKVError(rc, f"shotkv_create(device={device}) failed (needs a compute-capability 10.x GPU)")
        self.device = device

    def close(self):
        if self._h:
            lib().shotkv_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def last_error(self) -> str:
        return lib().shotkv_last_error(self._h).decode()

    def check(self, rc: int) -> int:
        if rc < 0:
            raise ShotKVError(rc, self.last_error())
        return rc


def shotkv_version() -> str:
    return lib().shotkv_version().decode()


def shotkv_budget_tokens(dims: Dims, policy: Policy) -> int:
    return int(lib().shotkv_budget_tokens(C.byref(dims), C.byref(policy)))


def shotkv_kept_capacity(dims: Dims, policy: Policy, offsets) -> int:
    o = _offsets(offsets)
    return int(lib().shotkv_kept_capacity(C.byref(dims), C.byref(policy), o.ctypes.data_as(C.c_void_p)))


def shotkv_validate(dims: Dims, policy: Policy | None = None, offsets=None) -> int:
    o = _offsets(offsets) if offsets is not None else None
    return int(lib().shotkv_validate(C.byref(dims), C.byref(policy) if policy is not None else None,
                                     o.ctypes.data_as(C.c_void_p) if o is not None else None))


def shotkv_workspace_bytes(dims: Dims) -> int:
    return int(lib().shotkv_workspace_bytes(C.byref(dims)))


def shotkv_prefill_score(ctx: Context, dims: Dims, Qwin, K, token_importance, ws, stream=None) -> int:
    rc = lib().shotkv_prefill_score(ctx._h, C.byref(dims), _ptr(Qwin, device="cuda", dtype=torch.bfloat16, name="Qwin"),
                                    _ptr(K, device="cuda", dtype=torch.bfloat16, name="K"),
                                    _ptr(token_importance, device="cuda", dtype=torch.float32, name="token_importance"),
                                    _ptr(ws, device="cuda", name="ws"), ws.numel() * ws.element_size(), _stream(stream))
    return ctx.check(rc)


def shotkv_select_shots(ctx: Context, dims: Dims, policy: Policy, token_importance, offsets, shot_scores, keep,
                        kept_idx, kept_count, Mcap: int, ws, stream=None) -> int:
    o = _offsets(offsets)
    rc = lib().shotkv_select_shots(ctx._h, C.byref(dims), C.byref(policy),
                                   _ptr(token_importance, device="cuda", dtype=torch.float32, name="token_importance"),
                                   o.ctypes.data_as(C.c_void_p),
                                   _ptr(shot_scores, device="cuda", dtype=torch.float32, name="shot_scores"),
                                   _ptr(keep, device="cuda", dtype=torch.uint8, name="keep"),
                                   _ptr(kept_idx, device="cuda", dtype=torch.int32, name="kept_idx"),
                                   _ptr(kept_count, device="cuda", dtype=torch.int32, name="kept_count"),
                                   int(Mcap), _ptr(ws, device="cuda", name="ws"), ws.numel() * ws.element_size(),
                                   _stream(stream))
    return ctx.check(rc)


def shotkv_select_shots_static(ctx: Context, dims: Dims, policy: Policy, token_importance, offsets, shot_scores, keep,
                               kept_idx, kept_count, Mcap: int, stream=None) -> int:
    """shotkv_select_shots without a workspace argument: for hosts that may not allocate device
    memory when they compress (the boundary table sits in a fixed 256 KB array inside the library;
    B*(S+1) <= 65536).  Calls on one device must not overlap on the GPU."""
    o = _offsets(offsets)
    rc = lib().shotkv_select_shots_static(ctx._h, C.byref(dims), C.byref(policy),
                                          _ptr(token_importance, device="cuda", dtype=torch.float32, name="token_importance"),
                                          o.ctypes.data_as(C.c_void_p),
                                          _ptr(shot_scores, device="cuda", dtype=torch.float32, name="shot_scores"),
                                          _ptr(keep, device="cuda", dtype=torch.uint8, name="keep"),
                                          _ptr(kept_idx, device="cuda", dtype=torch.int32, name="kept_idx"),
                                          _ptr(kept_count, device="cuda", dtype=torch.int32, name="kept_count"),
                                          int(Mcap), _stream(stream))
    return ctx.check(rc)


def shotkv_compact_kv(ctx: Context, dims: Dims, K, V, kept_idx, kept_count, Mcap: int, Kc, Vc, stream=None) -> int:
    rc = lib().shotkv_compact_kv(ctx._h, C.byref(dims), _ptr(K, device="cuda", dtype=torch.bfloat16, name="K"),
                                 _ptr(V, device="cuda", dtype=torch.bfloat16, name="V"),
                                 _ptr(kept_idx, device="cuda", dtype=torch.int32, name="kept_idx"),
                                 _ptr(kept_count, device="cuda", dtype=torch.int32, name="kept_count"), int(Mcap),
                                 _ptr(Kc, device="cuda", dtype=torch.bfloat16, name="Kc"),
                                 _ptr(Vc, device="cuda", dtype=torch.bfloat16, name="Vc"), _stream(stream))
    return ctx.check(rc)


def shotkv_prefill_compress(ctx: Context, dims: Dims, policy: Policy, Qwin, K, V, offsets, shot_scores, keep,
                            kept_idx, kept_count, Mcap: int, Kc, Vc, token_importance, flags: int, ws,
                            stream=None) -> int:
    o = _offsets(offsets)
    rc = lib().shotkv_prefill_compress(
        ctx._h, C.byref(dims), C.byref(policy),
        _ptr(Qwin, device="cuda", dtype=torch.bfloat16, name="Qwin"), _ptr(K, device="cuda", dtype=torch.bfloat16, name="K"),
        _ptr(V, device="cuda", dtype=torch.bfloat16, name="V"), o.ctypes.data_as(C.c_void_p),
        _ptr(shot_scores, device="cuda", dtype=torch.float32, name="shot_scores"),
        _ptr(keep, device="cuda", dtype=torch.uint8, name="keep"),
        _ptr(kept_idx, device="cuda", dtype=torch.int32, name="kept_idx"),
        _ptr(kept_count, device="cuda", dtype=torch.int32, name="kept_count"), int(Mcap),
        _ptr(Kc, device="cuda", dtype=torch.bfloat16, name="Kc"), _ptr(Vc, device="cuda", dtype=torch.bfloat16, name="Vc"),
        _ptr(token_importance, device="cuda", dtype=torch.float32, name="token_importance"), int(flags),
        _ptr(ws, device="cuda", name="ws"), ws.numel() * ws.element_size(), _stream(stream))
    return ctx.check(rc)


def shotkv_host_arena_bytes(dims: Dims, Mcap: int) -> int:
    return int(lib().shotkv_host_arena_bytes(C.byref(dims), int(Mcap)))


def shotkv_prefill_compress_host(ctx: Context, dims: Dims, policy: Policy, Qwin_host, K_host, V_host, offsets,
                                 shot_scores_host, keep_host, kept_idx_host, kept_count_host, Mcap: int,
                                 Kc_host, Vc_host, arena, stream=None) -> int:
    o = _offsets(offsets)
    rc = lib().shotkv_prefill_compress_host(
        ctx._h, C.byref(dims), C.byref(policy),
        _ptr(Qwin_host, device="cpu", dtype=torch.bfloat16, name="Qwin_host"),
        _ptr(K_host, device="cpu", dtype=torch.bfloat16, name="K_host"),
        _ptr(V_host, device="cpu", dtype=torch.bfloat16, name="V_host"), o.ctypes.data_as(C.c_void_p),
        _ptr(shot_scores_host, device="cpu", dtype=torch.float32, name="shot_scores_host"),
        _ptr(keep_host, device="cpu", dtype=torch.uint8, name="keep_host"),
        _ptr(kept_idx_host, device="cpu", dtype=torch.int32, name="kept_idx_host"),
        _ptr(kept_count_host, device="cpu", dtype=torch.int32, name="kept_count_host"), int(Mcap),
        _ptr(Kc_host, device="cpu", dtype=torch.bfloat16, name="Kc_host"),
        _ptr(Vc_host, device="cpu", dtype=torch.bfloat16, name="Vc_host"),
        _ptr(arena, device="cuda", name="arena"), arena.numel() * arena.element_size(), _stream(stream))
    return ctx.check(rc)


def shotkv_decode_workspace_bytes(dims: Dims, Dcap: int) -> int:
    return int(lib().shotkv_decode_workspace_bytes(C.byref(dims), int(Dcap)))


def shotkv_decode_capacity(policy: Policy, steps: int) -> int:
    return int(lib().shotkv_decode_capacity(C.byref(policy), int(steps)))


def shotkv_decode_init(ctx: Context, dims: Dims, policy: Policy, Dcap: int, Mcap: int, Kd, Vd, acc, born, ws) -> DecodeState:
    st = DecodeState()
    rc = lib().shotkv_decode_init(ctx._h, C.byref(dims), C.byref(policy), int(Dcap), int(Mcap),
                                  _ptr(Kd, device="cuda", dtype=torch.bfloat16, name="Kd"),
                                  _ptr(Vd, device="cuda", dtype=torch.bfloat16, name="Vd"),
                                  _ptr(acc, device="cuda", dtype=torch.float32, name="acc"),
                                  _ptr(born, device="cuda", dtype=torch.int32, name="born"),
                                  _ptr(ws, device="cuda", name="ws"), ws.numel() * ws.element_size(), C.byref(st))
    ctx.check(rc)
    st._keepalive = (Kd, Vd, acc, born, ws)
    return st


def shotkv_decode_step(ctx: Context, state: DecodeState, q, k_new, v_new, Kc, kept_count, stream=None) -> int:
    rc = lib().shotkv_decode_step(ctx._h, C.byref(state), _ptr(q, device="cuda", dtype=torch.bfloat16, name="q"),
                                  _ptr(k_new, device="cuda", dtype=torch.bfloat16, name="k_new"),
                                  _ptr(v_new, device="cuda", dtype=torch.bfloat16, name="v_new"),
                                  _ptr(Kc, device="cuda", dtype=torch.bfloat16, name="Kc"),
                                  _ptr(kept_count, device="cuda", dtype=torch.int32, name="kept_count"), _stream(stream))
    return ctx.check(rc)


def shotkv_decode_step_attend(ctx: Context, state: DecodeState, q, k_new, v_new, Kc, Vc, kept_count, attn_out,
                              stream=None) -> int:
    rc = lib().shotkv_decode_step_attend(ctx._h, C.byref(state), _ptr(q, device="cuda", dtype=torch.bfloat16, name="q"),
                                         _ptr(k_new, device="cuda", dtype=torch.bfloat16, name="k_new"),
                                         _ptr(v_new, device="cuda", dtype=torch.bfloat16, name="v_new"),
                                         _ptr(Kc, device="cuda", dtype=torch.bfloat16, name="Kc"),
                                         _ptr(Vc, device="cuda", dtype=torch.bfloat16, name="Vc"),
                                         _ptr(kept_count, device="cuda", dtype=torch.int32, name="kept_count"),
                                         _ptr(attn_out, device="cuda", dtype=torch.float32, name="attn_out"), _stream(stream))
    return ctx.check(rc)


def shotkv_plan_pieces(dims: Dims, offsets=None, sm_count: int = 148):
    """(nchunk, chunk_keys, pieces [B][P][3]) of the scoring pass's work partition (host only)."""
    o = _offsets(offsets) if offsets is not None else None
    cap = dims.S + 80
    out = np.zeros((dims.B, cap, 3), dtype=np.int32)
    nchunk, ck = C.c_int32(), C.c_int32()
    P = int(lib().shotkv_plan_pieces(C.byref(dims), o.ctypes.data_as(C.c_void_p) if o is not None else None, int(sm_count),
                                     C.byref(nchunk), C.byref(ck), out.ctypes.data_as(C.c_void_p), cap))
    if P < 0:
        raise ShotKVError(P, "shotkv_plan_pieces rejected its arguments")
    return int(nchunk.value), int(ck.value), out[:, :P, :].copy()


SCORING_FAST, SCORING_EXACT = 0, 1


def shotkv_set_scoring_mode(ctx: Context, mode: int) -> int:
    return ctx.check(lib().shotkv_set_scoring_mode(ctx._h, int(mode)))


def shotkv_set_pipeline_groups(ctx: Context, groups: int) -> int:
    return ctx.check(lib().shotkv_set_pipeline_groups(ctx._h, int(groups)))


def shotkv_set_wait_limit(ctx: Context, cycles: int) -> int:
    return ctx.check(lib().shotkv_set_wait_limit(ctx._h, int(cycles)))


def shotkv_selftest_bounded_wait(ctx: Context, limit_cycles: int, stream=None) -> list:
    """Runs the bounded waits into their limit on a one-CTA kernel; returns the four report words.
    Synchronises the stream and leaves the context's error word raised (see the header)."""
    rep = (C.c_int32 * 4)()
    ctx.check(lib().shotkv_selftest_bounded_wait(ctx._h, int(limit_cycles), rep, _stream(stream)))
    return [int(rep[i]) for i in range(4)]


def shotkv_last_scoring_clock(ctx: Context):
    """(SM cycles, nanoseconds) of the first CTA of the latest scoring launch; synchronise first."""
    c, n = C.c_int64(), C.c_int64()
    ctx.check(lib().shotkv_last_scoring_clock(ctx._h, C.byref(c), C.byref(n)))
    return int(c.value), int(n.value)


def shotkv_repaired_items(ctx: Context) -> int:
    return int(lib().shotkv_repaired_items(ctx._h))


def shotkv_profile_enable(ctx: Context, enable: bool) -> int:
    return ctx.check(lib().shotkv_profile_enable(ctx._h, int(bool(enable))))


def shotkv_profile_read(ctx: Context, calls_back: int = 0) -> list:
    ms = (C.c_float * 4)()
    n = ctx.check(lib().shotkv_profile_read(ctx._h, int(calls_back), ms))
    return [float(ms[i]) for i in range(n)]


def shotkv_launch_count(ctx: Context) -> int:
    return int(lib().shotkv_launch_count(ctx._h))


def alloc_prefill_outputs(dims: Dims, Mcap: int, device="cuda", token_importance: bool = False) -> dict:
    """Allocates (does not compute) the output tensors and the workspace of the prefill calls."""
    B, L, S, Hkv, d, N = dims.B, dims.L, max(dims.S, 1), dims.Hkv, dims.d, dims.N
    out = dict(
        shot_scores=torch.zeros(B, L, S, dtype=torch.float32, device=device),
        keep=torch.zeros(B, L, S, dtype=torch.uint8, device=device),
        kept_idx=torch.full((B, L, Mcap), -2, dtype=torch.int32, device=device),
        kept_count=torch.zeros(B, L, dtype=torch.int32, device=device),
        Kc=torch.zeros(B, L, Hkv, Mcap, d, dtype=torch.bfloat16, device=device),
        Vc=torch.zeros(B, L, Hkv, Mcap, d, dtype=torch.bfloat16, device=device),
        ws=torch.empty(shotkv_workspace_bytes(dims), dtype=torch.uint8, device=device),
        token_importance=(torch.zeros(B, L, Hkv, N, dtype=torch.float32, device=device) if token_importance else None),
    )
    return out


__all__ = [n for n in dir() if n.startswith("shotkv_")] + [
    "Context", "Dims", "Policy", "DecodeState", "ShotKVError", "make_dims", "per_head_dims", "make_policy", "alloc_prefill_outputs",
    "OK", "ERR_INVALID_ARG", "ERR_UNSUPPORTED_SHAPE", "ERR_BAD_OFFSETS", "ERR_WORKSPACE_TOO_SMALL", "ERR_CUDA",
    "ERR_TIMEOUT", "WARN_BUDGET_BELOW_ALWAYS_KEPT", "FLAG_TOKEN_IMPORTANCE", "EXPORTS", "LIB_PATH", "lib",
    "SCORING_FAST", "SCORING_EXACT", "shotkv_set_scoring_mode", "shotkv_repaired_items", "shotkv_set_pipeline_groups",
]
