"""ctypes binding of libficoco (argument marshalling only; every step runs in the library).

PyTorch is used for device memory and streams.  Function names mirror the C ABI declared in
``include/ficoco.h``.  Importing this module never loads the library; the first call does,
and raises if ``libficoco.so`` has not been built (``python -m paper_2411_17686_b200.build``).
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple, Union

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libficoco.so")

FICOCO_FP32, FICOCO_BF16 = 0, 1
FICOCO_HAS_CLS, FICOCO_LOCAL_PENALTY, FICOCO_AVERAGE_COMPRESSION, FICOCO_BACK_TO_BACK, FICOCO_CONVERGENT = 1, 2, 4, 8, 16
KCAP = 16

INSPECT = {
    "rnorm": (0, np.float32, 1), "score_raw": (1, np.float32, 1), "score": (2, np.float32, 1),
    "src_idx": (3, np.int32, 1), "tgt_idx": (4, np.int32, 1), "corr_cnt": (5, np.int32, 1),
    "corr_tgt": (6, np.int32, KCAP), "corr_w": (7, np.float32, KCAP), "corr_c": (8, np.float32, KCAP),
    "tau": (9, np.float32, 1),
}

EXPORTS = [
    "ficoco_create", "ficoco_destroy", "ficoco_strerror", "ficoco_last_cuda_error",
    "ficoco_default_params", "ficoco_v_reduce", "ficoco_l_reduce", "ficoco_v_reduce_host",
    "ficoco_l_reduce_host", "ficoco_status", "ficoco_inspect", "ficoco_last_launch_count",
    "ficoco_profile", "ficoco_profile_read", "ficoco_vision_redundancy_noalloc",
    "ficoco_equivalent_token", "ficoco_v_reduce_relation", "ficoco_debug_waits", "ficoco_v_reduce_schedule",
    "ficoco_v_plan",
]


class ficoco_params(C.Structure):
    _fields_ = [("lambda_", C.c_double), ("beta", C.c_double), ("gamma", C.c_double),
                ("eps", C.c_double), ("penalty_coef", C.c_double), ("window", C.c_int),
                ("max_targets", C.c_int), ("flags", C.c_uint), ("reserved", C.c_int)]


class ficoco_v_args(C.Structure):
    _fields_ = [("tokens", C.c_void_p), ("seqlens", C.c_void_p), ("attn", C.c_void_p),
                ("grid_h", C.c_void_p), ("grid_w", C.c_void_p), ("pos", C.c_void_p),
                ("keep", C.c_void_p), ("out_tokens", C.c_void_p), ("kept_idx", C.c_void_p),
                ("pos_out", C.c_void_p), ("scores_out", C.c_void_p),
                ("dtype", C.c_int), ("batch", C.c_int), ("n_tokens", C.c_int), ("dim", C.c_int),
                ("heads", C.c_int), ("n_grid", C.c_int), ("n_keep", C.c_int), ("reserved", C.c_int),
                ("out_cu_seqlens", C.c_void_p)]


class ficoco_l_args(C.Structure):
    _fields_ = [("tokens", C.c_void_p), ("attn_t2v", C.c_void_p), ("keep", C.c_void_p),
                ("out_tokens", C.c_void_p), ("kept_idx", C.c_void_p), ("scores_out", C.c_void_p),
                ("dtype", C.c_int), ("batch", C.c_int), ("n_vision", C.c_int), ("n_text", C.c_int),
                ("dim", C.c_int), ("heads", C.c_int), ("n_keep", C.c_int), ("reserved", C.c_int)]


class FicocoError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"libficoco error {code}: {msg}")
        self.code = code


_lib = None


def load_library() -> C.CDLL:
    """Load libficoco.so; fails loudly when it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2411_17686_b200.build` "
            "(there is no CPU fallback)")
    lib = C.CDLL(LIB_PATH)
    lib.ficoco_create.argtypes = [C.POINTER(C.c_void_p), C.c_int, C.c_longlong, C.c_int, C.c_int, C.c_int]
    lib.ficoco_destroy.argtypes = [C.c_void_p]
    lib.ficoco_strerror.argtypes = [C.c_int]
    lib.ficoco_strerror.restype = C.c_char_p
    lib.ficoco_last_cuda_error.argtypes = [C.c_void_p]
    lib.ficoco_default_params.argtypes = [C.POINTER(ficoco_params)]
    lib.ficoco_default_params.restype = None
    lib.ficoco_equivalent_token.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_int,
                                            C.c_int, C.c_int, C.c_void_p, C.c_void_p]
    lib.ficoco_v_reduce.argtypes = [C.c_void_p, C.POINTER(ficoco_v_args), C.POINTER(ficoco_params), C.c_void_p]
    lib.ficoco_l_reduce.argtypes = [C.c_void_p, C.POINTER(ficoco_l_args), C.POINTER(ficoco_params), C.c_void_p]
    lib.ficoco_v_reduce_relation.argtypes = [C.c_void_p, C.POINTER(ficoco_v_args), C.c_void_p, C.c_int,
                                             C.POINTER(ficoco_params), C.c_void_p]
    lib.ficoco_v_reduce_host.argtypes = [C.c_void_p, C.POINTER(ficoco_v_args), C.POINTER(ficoco_params)]
    lib.ficoco_l_reduce_host.argtypes = [C.c_void_p, C.POINTER(ficoco_l_args), C.POINTER(ficoco_params)]
    lib.ficoco_status.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_int)]
    lib.ficoco_debug_waits.argtypes = [C.c_void_p, C.c_longlong, C.c_int]
    lib.ficoco_v_plan.argtypes = [C.c_void_p, C.POINTER(ficoco_v_args), C.POINTER(ficoco_params), C.c_void_p]
    lib.ficoco_v_reduce_schedule.argtypes = [C.c_void_p, C.POINTER(ficoco_v_args), C.c_int, C.c_void_p, C.c_void_p,
                                             C.POINTER(ficoco_params), C.c_void_p]
    lib.ficoco_inspect.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_size_t, C.POINTER(C.c_size_t)]
    lib.ficoco_last_launch_count.argtypes = [C.c_void_p]
    lib.ficoco_profile.argtypes = [C.c_void_p, C.c_int]
    lib.ficoco_profile_read.argtypes = [C.c_void_p, C.c_int, C.c_char_p, C.c_int, C.POINTER(C.c_double),
                                        C.POINTER(C.c_longlong)]
    lib.ficoco_vision_redundancy_noalloc.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_uint,
                                                     C.c_void_p, C.c_void_p]
    _lib = lib
    return lib


def ficoco_default_params() -> ficoco_params:
    p = ficoco_params()
    load_library().ficoco_default_params(C.byref(p))
    return p


def make_params(lam=0.35, beta=0.6, gamma=0.6, eps=0.998, penalty_coef=2.0, window=2,
                max_targets=-1, has_cls=True, local_penalty=True, average_compression=False,
                back_to_back=False, convergent=False) -> ficoco_params:
    p = ficoco_params()
    p.lambda_, p.beta, p.gamma, p.eps, p.penalty_coef = lam, beta, gamma, eps, penalty_coef
    p.window, p.max_targets = window, -1 if max_targets is None else max_targets
    p.flags = ((FICOCO_HAS_CLS if has_cls else 0) | (FICOCO_LOCAL_PENALTY if local_penalty else 0) |
               (FICOCO_AVERAGE_COMPRESSION if average_compression else 0) |
               (FICOCO_BACK_TO_BACK if back_to_back else 0) | (FICOCO_CONVERGENT if convergent else 0))
    return p


def _check(ctx, rc: int) -> None:
    if rc != 0:
        lib = load_library()
        msg = lib.ficoco_strerror(rc).decode()
        if rc == -5 and ctx is not None:
            msg += f" (cudaError {lib.ficoco_last_cuda_error(ctx)})"
        raise FicocoError(rc, msg)


def _int_array(v: Union[int, Sequence[int]]) -> Tuple[np.ndarray, int]:
    a = np.ascontiguousarray(np.atleast_1d(np.asarray(v, dtype=np.int32)))
    return a, int(a.shape[0])


def _dtype_code(t) -> int:
    import torch
    if t.dtype == torch.bfloat16:
        return FICOCO_BF16
    if t.dtype == torch.float32:
        return FICOCO_FP32
    raise TypeError(f"tokens must be bf16 or fp32, got {t.dtype}")


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


@dataclass
class VResult:
    out_tokens: "object"
    kept_idx: "object"
    pos_out: "object"
    scores: "object"
    out_rows: List[int]   # output rows per image


class Context:
    """Owns one ficoco_ctx.  Methods mirror the C entry points."""

    def __init__(self, max_tokens: int, max_dim: int, max_batch: int, max_text: int = 0, device: int = 0):
        self.lib = load_library()
        self.device = device
        h = C.c_void_p()
        _check(None, self.lib.ficoco_create(C.byref(h), device, max_tokens, max_dim, max_batch, max_text))
        self.h = h

    def close(self) -> None:
        if getattr(self, "h", None):
            self.lib.ficoco_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- device-pointer entry points -----------------------------------------------------
    def ficoco_v_reduce(self, tokens, attn, keep, grid_h, grid_w, heads: int, *, n_tokens: int = 0,
                        seqlens=None, pos=None, params: Optional[ficoco_params] = None,
                        out_tokens=None, kept_idx=None, pos_out=None, scores_out=None,
                        want_scores: bool = False, stream: Optional[int] = None,
                        relation=None, by_column: bool = False, out_cu_seqlens=None,
                        plan_only: bool = False) -> VResult:
        """tokens: cuda tensor [rows, D]; attn: cuda fp32 tensor (packed per image [H, Np]);
        keep / grid_h / grid_w: int or per-image list; seqlens: per-image rows incl. CLS or
        None with n_tokens given.  Output tensors are allocated with torch when not passed.
        relation: optional cuda fp32 tensor, the images' [Np, Np] relation blocks one after the
        other; when given the call goes to ficoco_v_reduce_relation."""
        import torch
        p = params or ficoco_default_params()
        cls = 1 if (p.flags & FICOCO_HAS_CLS) else 0
        keep_a, n_keep = _int_array(keep)
        gh_a, n_gh = _int_array(grid_h)
        gw_a, n_gw = _int_array(grid_w)
        assert n_gh == n_gw
        if seqlens is not None:
            sl, batch = _int_array(seqlens)
        else:
            sl = None
            batch = tokens.shape[0] // n_tokens if n_tokens else 0
        keeps = [int(keep_a[0 if n_keep == 1 else b]) for b in range(batch)]
        ntoks = [int(sl[b]) if sl is not None else n_tokens for b in range(batch)]
        conv = bool(p.flags & FICOCO_CONVERGENT)        # one more row per image that discards something
        out_rows = [cls + k + (1 if conv and n - cls - k > 0 else 0) for k, n in zip(keeps, ntoks)]
        dim = tokens.shape[-1]
        dev = tokens.device
        if plan_only:               # ficoco_v_plan: shapes only
            a = ficoco_v_args()
            a.seqlens = sl.ctypes.data if sl is not None else None
            a.grid_h, a.grid_w, a.keep = gh_a.ctypes.data, gw_a.ctypes.data, keep_a.ctypes.data
            a.dtype, a.batch, a.n_tokens, a.dim, a.heads = _dtype_code(tokens), batch, n_tokens, dim, heads
            a.n_grid, a.n_keep = n_gh, n_keep
            if stream is None:
                stream = torch.cuda.current_stream(dev).cuda_stream
            _check(self.h, self.lib.ficoco_v_plan(self.h, C.byref(a), C.byref(p), C.c_void_p(stream)))
            return VResult(None, None, None, None, out_rows)
        if out_tokens is None:
            out_tokens = torch.empty((sum(out_rows), dim), dtype=tokens.dtype, device=dev)
        if kept_idx is None:
            kept_idx = torch.empty((sum(out_rows),), dtype=torch.int32, device=dev)
        if pos_out is None:
            pos_out = torch.empty((max(sum(keeps), 1),), dtype=torch.int32, device=dev)
        if scores_out is None and want_scores:
            scores_out = torch.empty((attn.numel() // heads,), dtype=torch.float32, device=dev)
        a = ficoco_v_args()
        a.tokens, a.attn, a.pos = _ptr(tokens), _ptr(attn), _ptr(pos)
        a.seqlens = sl.ctypes.data if sl is not None else None
        a.grid_h, a.grid_w, a.keep = gh_a.ctypes.data, gw_a.ctypes.data, keep_a.ctypes.data
        a.out_tokens, a.kept_idx = _ptr(out_tokens), _ptr(kept_idx)
        a.pos_out, a.scores_out = _ptr(pos_out), _ptr(scores_out)
        a.dtype, a.batch, a.n_tokens, a.dim, a.heads = _dtype_code(tokens), batch, n_tokens, dim, heads
        a.n_grid, a.n_keep = n_gh, n_keep
        a.out_cu_seqlens = _ptr(out_cu_seqlens)
        if stream is None:
            stream = torch.cuda.current_stream(dev).cuda_stream
        if relation is not None:
            _check(self.h, self.lib.ficoco_v_reduce_relation(self.h, C.byref(a), _ptr(relation), int(by_column),
                                                             C.byref(p), C.c_void_p(stream)))
        else:
            _check(self.h, self.lib.ficoco_v_reduce(self.h, C.byref(a), C.byref(p), C.c_void_p(stream)))
        return VResult(out_tokens, kept_idx, pos_out, scores_out, out_rows)

    def ficoco_v_reduce_schedule(self, tokens, attns, keeps, grid_h: int, grid_w: int, heads: int, *, n_tokens: int,
                                 pos=None, params: Optional[ficoco_params] = None, out_tokens=None, kept_idx=None,
                                 pos_out=None, stream: Optional[int] = None) -> VResult:
        """A progressive schedule in one call.  attns: list of cuda fp32 tensors, one per step
        ([B, H, Np_s] over the patch tokens alive at that step); keeps: patch tokens preserved by
        each step.  Returns the last step's tokens, kept_idx (into the original rows) and pos."""
        import torch
        p = params or ficoco_default_params()
        cls = 1 if (p.flags & FICOCO_HAS_CLS) else 0
        batch = tokens.shape[0] // n_tokens
        keep_a = np.ascontiguousarray(np.asarray(keeps, dtype=np.int32))
        n_steps = int(keep_a.shape[0])
        rows = cls + int(keep_a[-1])
        dim, dev = tokens.shape[-1], tokens.device
        if out_tokens is None:
            out_tokens = torch.empty((batch * rows, dim), dtype=tokens.dtype, device=dev)
        if kept_idx is None:
            kept_idx = torch.empty((batch * rows,), dtype=torch.int32, device=dev)
        if pos_out is None:
            pos_out = torch.empty((max(batch * int(keep_a[-1]), 1),), dtype=torch.int32, device=dev)
        gh_a, gw_a = _int_array(grid_h)[0], _int_array(grid_w)[0]
        a = ficoco_v_args()
        a.tokens, a.pos = _ptr(tokens), _ptr(pos)
        a.grid_h, a.grid_w = gh_a.ctypes.data, gw_a.ctypes.data
        a.out_tokens, a.kept_idx, a.pos_out = _ptr(out_tokens), _ptr(kept_idx), _ptr(pos_out)
        a.dtype, a.batch, a.n_tokens, a.dim, a.heads = _dtype_code(tokens), batch, n_tokens, dim, heads
        a.n_grid, a.n_keep = 1, 1
        ptrs = (C.c_void_p * n_steps)(*[t.data_ptr() for t in attns])
        if stream is None:
            stream = torch.cuda.current_stream(dev).cuda_stream
        _check(self.h, self.lib.ficoco_v_reduce_schedule(self.h, C.byref(a), n_steps, keep_a.ctypes.data, ptrs,
                                                         C.byref(p), C.c_void_p(stream)))
        return VResult(out_tokens, kept_idx, pos_out, None, [rows] * batch)

    def ficoco_l_reduce(self, tokens, attn_t2v, keep, n_vision: int, n_text: int, heads: int, *,
                        params: Optional[ficoco_params] = None, out_tokens=None, kept_idx=None,
                        scores_out=None, want_scores: bool = False, stream: Optional[int] = None) -> VResult:
        """tokens: cuda tensor [B*(N+M), D]; attn_t2v: cuda fp32 [B, H, M, N]."""
        import torch
        p = params or ficoco_default_params()
        keep_a, n_keep = _int_array(keep)
        batch = tokens.shape[0] // (n_vision + n_text)
        keeps = [int(keep_a[0 if n_keep == 1 else b]) for b in range(batch)]
        conv = bool(p.flags & FICOCO_CONVERGENT)
        out_rows = [k + n_text + (1 if conv and n_vision - k > 0 else 0) for k in keeps]
        dim = tokens.shape[-1]
        dev = tokens.device
        if out_tokens is None:
            out_tokens = torch.empty((sum(out_rows), dim), dtype=tokens.dtype, device=dev)
        if kept_idx is None:
            kept_idx = torch.empty((sum(out_rows),), dtype=torch.int32, device=dev)
        if scores_out is None and want_scores:
            scores_out = torch.empty((batch * n_vision,), dtype=torch.float32, device=dev)
        a = ficoco_l_args()
        a.tokens, a.attn_t2v, a.keep = _ptr(tokens), _ptr(attn_t2v), keep_a.ctypes.data
        a.out_tokens, a.kept_idx, a.scores_out = _ptr(out_tokens), _ptr(kept_idx), _ptr(scores_out)
        a.dtype, a.batch, a.n_vision, a.n_text = _dtype_code(tokens), batch, n_vision, n_text
        a.dim, a.heads, a.n_keep = dim, heads, n_keep
        if stream is None:
            stream = torch.cuda.current_stream(dev).cuda_stream
        _check(self.h, self.lib.ficoco_l_reduce(self.h, C.byref(a), C.byref(p), C.c_void_p(stream)))
        return VResult(out_tokens, kept_idx, None, scores_out, out_rows)

    # -- host-buffer entry points (tensors live in host memory, ideally pinned) ------------
    def ficoco_v_reduce_host(self, tokens, attn, keep, grid_h, grid_w, heads: int, *, n_tokens: int = 0,
                             seqlens=None, pos=None, params: Optional[ficoco_params] = None,
                             out_tokens=None, kept_idx=None, pos_out=None, scores_out=None) -> VResult:
        import torch
        p = params or ficoco_default_params()
        cls = 1 if (p.flags & FICOCO_HAS_CLS) else 0
        keep_a, n_keep = _int_array(keep)
        gh_a, n_gh = _int_array(grid_h)
        gw_a, _ = _int_array(grid_w)
        if seqlens is not None:
            sl, batch = _int_array(seqlens)
        else:
            sl, batch = None, tokens.shape[0] // n_tokens
        keeps = [int(keep_a[0 if n_keep == 1 else b]) for b in range(batch)]
        ntoks = [int(sl[b]) if sl is not None else n_tokens for b in range(batch)]
        conv = bool(p.flags & FICOCO_CONVERGENT)
        out_rows = [cls + k + (1 if conv and n - cls - k > 0 else 0) for k, n in zip(keeps, ntoks)]
        dim = tokens.shape[-1]
        if out_tokens is None:
            out_tokens = torch.empty((sum(out_rows), dim), dtype=tokens.dtype).pin_memory()
        if kept_idx is None:
            kept_idx = torch.empty((sum(out_rows),), dtype=torch.int32).pin_memory()
        a = ficoco_v_args()
        a.tokens, a.attn, a.pos = _ptr(tokens), _ptr(attn), _ptr(pos)
        a.seqlens = sl.ctypes.data if sl is not None else None
        a.grid_h, a.grid_w, a.keep = gh_a.ctypes.data, gw_a.ctypes.data, keep_a.ctypes.data
        a.out_tokens, a.kept_idx = _ptr(out_tokens), _ptr(kept_idx)
        a.pos_out, a.scores_out = _ptr(pos_out), _ptr(scores_out)
        a.dtype, a.batch, a.n_tokens, a.dim, a.heads = _dtype_code(tokens), batch, n_tokens, dim, heads
        a.n_grid, a.n_keep = n_gh, n_keep
        _check(self.h, self.lib.ficoco_v_reduce_host(self.h, C.byref(a), C.byref(p)))
        return VResult(out_tokens, kept_idx, pos_out, scores_out, out_rows)

    def ficoco_l_reduce_host(self, tokens, attn_t2v, keep, n_vision: int, n_text: int, heads: int, *,
                             params: Optional[ficoco_params] = None, out_tokens=None, kept_idx=None,
                             scores_out=None) -> VResult:
        import torch
        p = params or ficoco_default_params()
        keep_a, n_keep = _int_array(keep)
        batch = tokens.shape[0] // (n_vision + n_text)
        keeps = [int(keep_a[0 if n_keep == 1 else b]) for b in range(batch)]
        conv = bool(p.flags & FICOCO_CONVERGENT)
        out_rows = [k + n_text + (1 if conv and n_vision - k > 0 else 0) for k in keeps]
        dim = tokens.shape[-1]
        if out_tokens is None:
            out_tokens = torch.empty((sum(out_rows), dim), dtype=tokens.dtype).pin_memory()
        if kept_idx is None:
            kept_idx = torch.empty((sum(out_rows),), dtype=torch.int32).pin_memory()
        a = ficoco_l_args()
        a.tokens, a.attn_t2v, a.keep = _ptr(tokens), _ptr(attn_t2v), keep_a.ctypes.data
        a.out_tokens, a.kept_idx, a.scores_out = _ptr(out_tokens), _ptr(kept_idx), _ptr(scores_out)
        a.dtype, a.batch, a.n_vision, a.n_text = _dtype_code(tokens), batch, n_vision, n_text
        a.dim, a.heads, a.n_keep = dim, heads, n_keep
        _check(self.h, self.lib.ficoco_l_reduce_host(self.h, C.byref(a), C.byref(p)))
        return VResult(out_tokens, kept_idx, None, scores_out, out_rows)

    # -- status / inspection ----------------------------------------------------------------
    def ficoco_status(self, stream: Optional[int] = None) -> int:
        import torch
        if stream is None:
            stream = torch.cuda.current_stream().cuda_stream
        v = C.c_int(0)
        _check(self.h, self.lib.ficoco_status(self.h, C.c_void_p(stream), C.byref(v)))
        return v.value

    def ficoco_inspect(self, what: str) -> np.ndarray:
        code, dt, width = INSPECT[what]
        n = C.c_size_t(0)
        _check(self.h, self.lib.ficoco_inspect(self.h, code, None, 0, C.byref(n)))
        buf = np.empty(n.value // 4, dtype=dt)
        if n.value:
            _check(self.h, self.lib.ficoco_inspect(self.h, code, buf.ctypes.data, n.value, None))
        return buf.reshape(-1, width) if width > 1 else buf

    def ficoco_debug_waits(self, wait_ns: int = 0, extra_arrivals: int = 0) -> None:
        _check(self.h, self.lib.ficoco_debug_waits(self.h, wait_ns, extra_arrivals))

    def ficoco_last_launch_count(self) -> int:
        return int(self.lib.ficoco_last_launch_count(self.h))

    def ficoco_profile(self, enable: bool) -> None:
        _check(self.h, self.lib.ficoco_profile(self.h, 1 if enable else 0))

    def ficoco_profile_read(self):
        """[(kernel name, total ms, launches), ...] since profiling was enabled."""
        out = []
        i = 0
        while True:
            name = C.create_string_buffer(64)
            ms, n = C.c_double(0), C.c_longlong(0)
            if self.lib.ficoco_profile_read(self.h, i, name, 64, C.byref(ms), C.byref(n)) != 0:
                break
            out.append((name.value.decode(), ms.value, n.value))
            i += 1
        return out


def ficoco_vision_redundancy_noalloc(tokens, n_tokens: int, has_cls: bool = True, v_out=None,
                                     stream: Optional[int] = None):
    """First term of Eq. 1 for a uniform batch, for callers that may not allocate device memory
    (for example a serving engine's step callback whose engine owns all of it): no context, the
    scratch is a fixed array inside the library.  ``tokens``: cuda tensor [batch * n_tokens, D];
    ``v_out``: cuda fp32 [batch * Np], which the caller should pass in (it is only created here,
    with torch, as a convenience for tests).  Limits and sharing rules: see ficoco.h."""
    import torch
    lib = load_library()
    batch = tokens.shape[0] // n_tokens
    np_ = n_tokens - (1 if has_cls else 0)
    if v_out is None:
        v_out = torch.empty((batch * np_,), dtype=torch.float32, device=tokens.device)
    if stream is None:
        stream = torch.cuda.current_stream(tokens.device).cuda_stream
    rc = lib.ficoco_vision_redundancy_noalloc(tokens.data_ptr(), _dtype_code(tokens), batch, n_tokens,
                                              tokens.shape[-1], FICOCO_HAS_CLS if has_cls else 0,
                                              v_out.data_ptr(), C.c_void_p(stream))
    _check(None, rc)
    return v_out


def ficoco_equivalent_token(keys, heads: int, head_dim: int, *, n_tokens: int = 0, seqlens=None,
                            has_cls: bool = False, a_eq=None, stream: Optional[int] = None):
    """a^Eq of the no-CLS variant.  ``keys``: cuda tensor [rows, heads * head_dim] (token-major
    key states, images packed); ``seqlens``: rows per image, or None with ``n_tokens`` given.
    Returns the cuda fp32 tensor of one value per patch token (allocated with torch when
    ``a_eq`` is not passed); use it as ``attn`` with ``heads = 1`` in ficoco_v_reduce."""
    import torch
    lib = load_library()
    cls = 1 if has_cls else 0
    if seqlens is not None:
        sl, batch = _int_array(seqlens)
        patches = int(sl.sum()) - cls * batch
        sl_ptr = sl.ctypes.data
    else:
        sl, batch = None, keys.shape[0] // n_tokens
        patches = batch * (n_tokens - cls)
        sl_ptr = None
    if a_eq is None:
        a_eq = torch.empty((patches,), dtype=torch.float32, device=keys.device)
    if stream is None:
        stream = torch.cuda.current_stream(keys.device).cuda_stream
    rc = lib.ficoco_equivalent_token(C.c_void_p(keys.data_ptr()), _dtype_code(keys), batch, n_tokens,
                                     C.c_void_p(sl_ptr), heads, head_dim, cls, C.c_void_p(a_eq.data_ptr()),
                                     C.c_void_p(stream))
    _check(None, rc)
    return a_eq


# ----------------------------------------------------------------------------------------
# numpy <-> torch helpers for the synthetic batches
# ----------------------------------------------------------------------------------------

def to_torch(arr: np.ndarray, device=None, pin: bool = False):
    """numpy fp32 / int32 / uint16(bf16 bits) -> torch tensor (bf16 for uint16)."""
    import torch
    if arr.dtype == np.uint16:
        t = torch.from_numpy(arr.view(np.int16).copy()).view(torch.bfloat16)
    else:
        t = torch.from_numpy(np.ascontiguousarray(arr).copy())
    if pin:
        t = t.pin_memory()
    if device is not None:
        t = t.to(device)
    return t


def to_numpy(t) -> np.ndarray:
    """torch tensor -> numpy (bf16 as uint16 bit patterns)."""
    import torch
    t = t.detach().cpu()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16).copy()
    return t.numpy().copy()
