"""ctypes binding of include/osscar.h.  Argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Iterable, Optional

import torch

from . import build as _build

OK = 0
E_ARG, E_SHAPE, E_NOTPD, E_WORKSPACE, E_CUDA, E_TIMEOUT, E_STATE = -1, -2, -3, -4, -5, -6, -7
BF16, FP32, FP64 = 0, 1, 2
GRAM_BEGIN, GRAM_END = 1, 2
INIT_ENERGY, INIT_MAGNITUDE, INIT_USER = 0, 1, 2
SCORE_INDEPENDENT, SCORE_PAIR_EXACT = 0, 1
ACCEPT_IMPROVING, ACCEPT_ALWAYS = 0, 1
STOP_MAX_SWAPS, STOP_NO_IMPROVEMENT, STOP_GUARD = 0, 1, 2
STOP_NAMES = {0: "max_swaps", 1: "no_improvement", 2: "guard"}
LOOP_AUTO, LOOP_PERSISTENT, LOOP_LAUNCHES = 0, 1, 2

EXPORTS = ["osscar_create", "osscar_destroy", "osscar_workspace_bytes", "osscar_set_workspace",
           "osscar_gram", "osscar_init_support", "osscar_local_search", "osscar_objective",
           "osscar_debug_get_state", "osscar_status_string", "osscar_launch_count", "osscar_trace_noalloc", "osscar_init_support_greedy", "osscar_gram_cross", "osscar_set_const_term",
           "osscar_set_wait_limit", "osscar_set_shard_reduce"]


class SearchParams(C.Structure):
    _fields_ = [("max_swaps", C.c_int32), ("score_mode", C.c_int32), ("accept_mode", C.c_int32),
                ("refresh_every", C.c_int32), ("accept_rel_tol", C.c_double), ("profile_samples", C.c_int32), ("block_pairs", C.c_int32),
                ("loop_mode", C.c_int32), ("reserved", C.c_int32), ("wait_limit_cycles", C.c_uint64)]


class SearchResult(C.Structure):
    _fields_ = [("n_swaps", C.c_int32), ("stop_reason", C.c_int32), ("n_refresh", C.c_int32), ("status", C.c_int32),
                ("obj_init", C.c_double), ("obj_final", C.c_double), ("ms_search", C.c_float),
                ("n_profiled", C.c_int32), ("ms_kernel", C.c_float * 12), ("loop_driver", C.c_int32)]


STEP_KERNELS = ["select", "pair_grams", "y_pass", "small_algebra", "staging", "h_pass", "update_hinv", "update_v",
                "update_r", "group_scores", "h_swap_rows", "h_swap_cols"]
# single-row groups run a fused five-launch step
STEP_KERNELS_G1 = ["decide", "l1_hpass_update_v", "l2_update_r_swap", "select_in", "l4_update_hinv_y"]
# block exchanges (block_pairs > 1): stages of one iteration
STEP_KERNELS_BLOCK = ["select", "gather_y", "grams_algebra_staging", "h_pass", "update_hinv", "update_v", "update_r",
                      "update_c_fix", "h_swap", "scores"]


# int reduce(void* user, void* dev_buf, int64_t count, int dtype, void* cuda_stream)
REDUCE_FN = C.CFUNCTYPE(C.c_int, C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_void_p)


class OsscarError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().osscar_status_string(status).decode() if _LIB is not None else "?"
        super().__init__(f"{where}: {msg} ({status})")


_LIB = None


def lib_path() -> str:
    return _build.LIB_PATH


def lib() -> C.CDLL:
    """Loads libosscar.so (building it with nvcc first if the sources are newer).  Raises if absent."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = _build.LIB_PATH
    if not os.path.exists(path) or (os.environ.get("OSSCAR_NO_REBUILD") is None and _build.needs_build()):
        _build.build()
    L = C.CDLL(path)
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    L.osscar_status_string.restype = C.c_char_p
    L.osscar_status_string.argtypes = [C.c_int]
    L.osscar_create.argtypes = [C.POINTER(vp), C.c_int, vp]
    L.osscar_destroy.argtypes = [vp]
    L.osscar_workspace_bytes.argtypes = [i64, i64, i32, i32, C.POINTER(C.c_size_t)]
    L.osscar_set_workspace.argtypes = [vp, vp, C.c_size_t]
    L.osscar_gram.argtypes = [vp, vp, C.c_int, i64, i64, vp, i64, C.c_int, C.c_float, vp, vp, C.POINTER(C.c_double)]
    L.osscar_init_support.argtypes = [vp, vp, vp, vp, i64, i64, i32, i32, C.c_int, vp, C.POINTER(C.c_double)]
    L.osscar_init_support_greedy.argtypes = [vp, vp, vp, vp, i64, i64, i32, i32, i32, vp, vp, C.POINTER(C.c_double), C.POINTER(i32)]
    L.osscar_gram_cross.argtypes = [vp, vp, C.c_int, vp, C.c_int, i64, i64, i64, C.c_int, C.c_float, vp, vp, C.POINTER(C.c_double)]
    L.osscar_set_const_term.argtypes = [vp, C.c_double, C.c_int]
    L.osscar_set_wait_limit.argtypes = [vp, C.c_uint64]
    L.osscar_set_shard_reduce.argtypes = [vp, REDUCE_FN, vp]
    L.osscar_local_search.argtypes = [vp, C.POINTER(SearchParams), vp, vp, vp, vp, C.POINTER(SearchResult)]
    L.osscar_objective.argtypes = [vp, vp, vp, vp, i64, i64, C.POINTER(C.c_double)]
    L.osscar_debug_get_state.argtypes = [vp, C.c_int, vp]
    L.osscar_trace_noalloc.argtypes = [vp, i64, vp, i64, i64, i64, C.c_int, vp, C.POINTER(C.c_double)]
    L.osscar_launch_count.restype = C.c_uint64
    L.osscar_launch_count.argtypes = []
    for name in EXPORTS:
        if name not in ("osscar_status_string", "osscar_launch_count"):
            getattr(L, name).restype = C.c_int
    _LIB = L
    return L


def _check(status: int, where: str):
    if status != OK:
        raise OsscarError(status, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _dev_f32(t: torch.Tensor, name: str) -> torch.Tensor:
    if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
        raise ValueError(f"{name} must be a contiguous fp32 CUDA tensor")
    return t


def osscar_trace_noalloc(A: torch.Tensor, B: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> float:
    """sum(A * B) in fp64 through the allocation-free entry point (scratch built into the library; rows <= 65536).
    For callers that may not allocate device memory; calls on one GPU must not overlap."""
    if not (A.is_cuda and B.is_cuda and A.dtype == torch.float32 and B.dtype == torch.float32 and A.dim() == 2
            and A.shape == B.shape and A.stride(1) == 1 and B.stride(1) == 1):
        raise ValueError("A and B must be fp32 CUDA matrices of one shape with unit column stride")
    dev = A.device.index
    sptr = C.c_void_p((stream or torch.cuda.current_stream(dev)).cuda_stream)
    out = C.c_double(0.0)
    _check(lib().osscar_trace_noalloc(_ptr(A), A.stride(0), _ptr(B), B.stride(0), A.shape[0], A.shape[1], dev, sptr,
                                      C.byref(out)), "osscar_trace_noalloc")
    return out.value


def launch_count() -> int:
    return int(lib().osscar_launch_count())


def osscar_workspace_bytes(d1: int, m: int, g: int, k: int) -> int:
    out = C.c_size_t(0)
    _check(lib().osscar_workspace_bytes(d1, m, g, k, C.byref(out)), "osscar_workspace_bytes")
    return out.value


@dataclass
class SearchOutput:
    support: torch.Tensor        # int32[k], sorted kept group ids (device)
    W: torch.Tensor              # d1 x m fp32, pruned rows zero (device)
    obj_trace: torch.Tensor      # float64[n_swaps + 1] (device)
    swap_trace: torch.Tensor     # int32[n_swaps, 2] (group out, group in) (device)
    n_swaps: int
    stop_reason: str
    n_refresh: int
    obj_init: float
    obj_final: float
    ms_search: float
    ms_kernel: dict              # mean device ms per kernel of a step over the profiled steps ({} if none)
    loop_driver: str = "launches"  # "persistent" (one cooperative kernel) or "launches"


class Solver:
    """One context (device + stream) and its caller-owned workspace."""

    def __init__(self, device: Optional[int] = None, stream: Optional[torch.cuda.Stream] = None):
        if not torch.cuda.is_available():
            raise OsscarError(E_CUDA, "Solver: no CUDA device; this library has no CPU path")
        self.device = torch.cuda.current_device() if device is None else int(device)
        self.stream = stream
        handle = C.c_void_p()
        sptr = C.c_void_p(stream.cuda_stream) if stream is not None else C.c_void_p(torch.cuda.current_stream(self.device).cuda_stream)
        _check(lib().osscar_create(C.byref(handle), self.device, sptr), "osscar_create")
        self._h = handle
        self._ws = None
        self._shape = None
        self._keep = []

    def close(self):
        if getattr(self, "_h", None):
            lib().osscar_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -------------------------------------------------------------- workspace
    def ensure_workspace(self, d1: int, m: int, g: int, k: int):
        need = osscar_workspace_bytes(d1, m, g, k)
        if self._ws is None or self._ws.numel() < need:
            self._ws = None
            self._ws = torch.empty(need, dtype=torch.uint8, device=f"cuda:{self.device}")
        _check(lib().osscar_set_workspace(self._h, _ptr(self._ws), self._ws.numel()), "osscar_set_workspace")
        return need

    def lend_workspace(self, nbytes: int):
        """Lends a workspace of exactly `nbytes` (staging room for the tensor-core products before a state exists)."""
        self._ws = None
        self._ws = torch.empty(int(nbytes), dtype=torch.uint8, device=f"cuda:{self.device}")
        _check(lib().osscar_set_workspace(self._h, _ptr(self._ws), self._ws.numel()), "osscar_set_workspace")

    # -------------------------------------------------------------- calls of include/osscar.h
    def gram_chunk(self, X: torch.Tensor, H: torch.Tensor, flags: int, W=None, G=None, damp: float = 0.0) -> Optional[float]:
        if X.dtype == torch.bfloat16:
            xd = BF16
        elif X.dtype == torch.float32:
            xd = FP32
        else:
            raise ValueError("X must be bf16 or fp32")
        if not (X.is_cuda and X.is_contiguous() and X.dim() == 2):
            raise ValueError("X must be a contiguous 2-D CUDA tensor")
        n, d1 = X.shape
        _dev_f32(H, "H")
        const = C.c_double(0.0)
        m = 0
        if flags & GRAM_END:
            _dev_f32(W, "W"); _dev_f32(G, "G")
            m = W.shape[1]
        _check(lib().osscar_gram(self._h, _ptr(X), xd, n, d1, _ptr(W), m, flags, damp, _ptr(H), _ptr(G), C.byref(const)), "osscar_gram")
        return const.value if flags & GRAM_END else None

    def gram(self, chunks: Iterable[torch.Tensor], W: torch.Tensor, damp: float = 0.0):
        """H, G, const from an iterable of row blocks of X (each a CUDA tensor)."""
        _dev_f32(W, "W")
        d1, m = W.shape
        H = torch.empty(d1, d1, dtype=torch.float32, device=W.device)
        G = torch.empty(d1, m, dtype=torch.float32, device=W.device)
        chunks = list(chunks) if not isinstance(chunks, (list, tuple)) else chunks
        const = None
        for i, Xc in enumerate(chunks):
            flags = (GRAM_BEGIN if i == 0 else 0) | (GRAM_END if i == len(chunks) - 1 else 0)
            const = self.gram_chunk(Xc, H, flags, W, G, damp)
        return H, G, const

    def gram_cross(self, x_chunks, y_chunks, damp: float = 0.0):
        """H = X^T X, G = X^T Y, const = ||Y||_F^2 from row blocks of the pruned model's input X and the dense
        model's output Y (CUDA tensors; X bf16 or fp32, Y bf16 or fp32)."""
        x_chunks, y_chunks = list(x_chunks), list(y_chunks)
        d1, m = x_chunks[0].shape[1], y_chunks[0].shape[1]
        dev = x_chunks[0].device
        H = torch.empty(d1, d1, dtype=torch.float32, device=dev)
        G = torch.empty(d1, m, dtype=torch.float32, device=dev)
        code = {torch.bfloat16: BF16, torch.float32: FP32}
        const = C.c_double(0.0)
        if x_chunks[0].dtype == torch.bfloat16 and y_chunks[0].dtype == torch.float32:
            need = 6 * max(c.shape[0] for c in x_chunks) * ((m + 7) // 8 * 8) + 4096
            if self._ws is None or self._ws.numel() < need:
                self._ws = torch.empty(need, dtype=torch.uint8, device=dev)
            _check(lib().osscar_set_workspace(self._h, _ptr(self._ws), self._ws.numel()), "osscar_set_workspace")
        for i, (Xc, Yc) in enumerate(zip(x_chunks, y_chunks)):
            if not (Xc.is_cuda and Yc.is_cuda and Xc.is_contiguous() and Yc.is_contiguous() and Xc.shape[0] == Yc.shape[0]):
                raise ValueError("X and Y blocks must be contiguous CUDA tensors with equal row counts")
            flags = (GRAM_BEGIN if i == 0 else 0) | (GRAM_END if i == len(x_chunks) - 1 else 0)
            _check(lib().osscar_gram_cross(self._h, _ptr(Xc), code[Xc.dtype], _ptr(Yc), code[Yc.dtype], Xc.shape[0], d1, m,
                                           flags, damp, _ptr(H), _ptr(G), C.byref(const)), "osscar_gram_cross")
        return H, G, const.value

    def set_wait_limit(self, cycles: int):
        """Budget (SM cycles) of every bounded device-side wait of this context's kernels; 0 = default."""
        _check(lib().osscar_set_wait_limit(self._h, int(cycles)), "osscar_set_wait_limit")

    def set_shard_reduce(self, fn):
        """Column shards: `fn(view, stream_ptr)` must enqueue, on the CUDA stream with that handle, an in-place sum over all
        shards of `view`, a 1-D tensor (float32 or float64) that aliases the partial sums inside this solver's
        workspace.  None removes the hook.  The workspace must be set before the calls that use the hook."""
        if fn is None:
            self._reduce_cb = None
            _check(lib().osscar_set_shard_reduce(self._h, C.cast(None, REDUCE_FN), None), "osscar_set_shard_reduce")
            return

        def trampoline(_user, buf, count, dtype, stream):
            try:
                ws = self._ws
                off = int(buf) - ws.data_ptr()
                tdt, width = (torch.float64, 8) if dtype == FP64 else (torch.float32, 4)
                if off < 0 or off + count * width > ws.numel():
                    return 1
                fn(ws[off:off + count * width].view(tdt), int(stream) if stream else 0)
                return 0
            except Exception:          # an exception must not unwind through the C caller
                import traceback
                traceback.print_exc()
                return 1

        self._reduce_cb = REDUCE_FN(trampoline)       # kept alive as long as the context may call it
        _check(lib().osscar_set_shard_reduce(self._h, self._reduce_cb, None), "osscar_set_shard_reduce")

    def set_const_term(self, value: float, enabled: bool = True):
        _check(lib().osscar_set_const_term(self._h, float(value), int(enabled)), "osscar_set_const_term")

    def init_support(self, H, G, W, g: int, k: int, mode: int = INIT_ENERGY, support: Optional[torch.Tensor] = None):
        _dev_f32(H, "H"); _dev_f32(G, "G"); _dev_f32(W, "W")
        d1, m = W.shape
        self.ensure_workspace(d1, m, g, k)
        if support is None:
            support = torch.empty(k, dtype=torch.int32, device=W.device)
        else:
            support = support.to(device=W.device, dtype=torch.int32).contiguous().clone()
        obj0 = C.c_double(0.0)
        self._keep = [H, G, W]
        self._shape = (d1, m, g, k)
        _check(lib().osscar_init_support(self._h, _ptr(H), _ptr(G), _ptr(W), d1, m, g, k, mode, _ptr(support), C.byref(obj0)),
               "osscar_init_support")
        return support, obj0.value

    def init_support_greedy(self, H, G, W, g: int, k: int, t_hat: int = 1):
        """Nested (greedy) phase of Algorithm 1 down to k groups, then the search state.  Returns
        (support int32[k] sorted, drop_trace int32[d1/g - k], obj0, iterations)."""
        _dev_f32(H, "H"); _dev_f32(G, "G"); _dev_f32(W, "W")
        d1, m = W.shape
        self.ensure_workspace(d1, m, g, k)
        support = torch.empty(k, dtype=torch.int32, device=W.device)
        drops = torch.empty(max(1, d1 // g - k), dtype=torch.int32, device=W.device)
        obj0, iters = C.c_double(0.0), C.c_int32(0)
        self._keep = [H, G, W]
        self._shape = (d1, m, g, k)
        _check(lib().osscar_init_support_greedy(self._h, _ptr(H), _ptr(G), _ptr(W), d1, m, g, k, t_hat, _ptr(support),
                                                _ptr(drops), C.byref(obj0), C.byref(iters)), "osscar_init_support_greedy")
        return support, drops[:d1 // g - k], obj0.value, iters.value

    def local_search(self, max_swaps: int, score_mode: int = SCORE_INDEPENDENT, accept_mode: int = ACCEPT_IMPROVING,
                     refresh_every: int = 0, accept_rel_tol: float = -1.0, profile_samples: int = 0,
                     block_pairs: int = 0, loop_mode: int = LOOP_AUTO, wait_limit_cycles: int = 0) -> SearchOutput:
        d1, m, g, k = self._shape
        dev = self._keep[0].device
        support = torch.empty(k, dtype=torch.int32, device=dev)
        W_out = torch.empty(d1, m, dtype=torch.float32, device=dev)
        obj_trace = torch.zeros(max_swaps + 1, dtype=torch.float64, device=dev)
        swap_trace = torch.zeros(max(1, 2 * max_swaps), dtype=torch.int32, device=dev)
        prm = SearchParams(max_swaps, score_mode, accept_mode, refresh_every, accept_rel_tol, profile_samples, block_pairs,
                           loop_mode, 0, wait_limit_cycles)
        res = SearchResult()
        _check(lib().osscar_local_search(self._h, C.byref(prm), _ptr(support), _ptr(W_out), _ptr(obj_trace), _ptr(swap_trace),
                                         C.byref(res)), "osscar_local_search")
        n = res.n_swaps
        n_obj = n // block_pairs if block_pairs > 1 else n      # one objective per iteration
        return SearchOutput(support, W_out, obj_trace[:n_obj + 1], swap_trace[:2 * n].view(n, 2), n,
                            STOP_NAMES.get(res.stop_reason, str(res.stop_reason)), res.n_refresh,
                            res.obj_init, res.obj_final, res.ms_search,
                            {n: res.ms_kernel[i] for i, n in enumerate(STEP_KERNELS_BLOCK if block_pairs > 1 else STEP_KERNELS_G1 if g == 1 else STEP_KERNELS)}
                            if res.n_profiled > 0 else {}, "persistent" if res.loop_driver == LOOP_PERSISTENT else "launches")

    def objective(self, H, W, Wt) -> float:
        _dev_f32(H, "H"); _dev_f32(W, "W"); _dev_f32(Wt, "Wt")
        d1, m = W.shape
        need = 2 * d1 * m * 4
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=W.device)
            _check(lib().osscar_set_workspace(self._h, _ptr(self._ws), self._ws.numel()), "osscar_set_workspace")
        out = C.c_double(0.0)
        _check(lib().osscar_objective(self._h, _ptr(H), _ptr(W), _ptr(Wt), d1, m, C.byref(out)), "osscar_objective")
        return out.value

    def debug_state(self, which: int) -> torch.Tensor:
        d1, m, g, k = self._shape
        nI, ng = k * g, d1 // g
        dev = self._keep[0].device
        shapes = {0: ((nI, nI), torch.float32), 1: ((nI, m), torch.float32), 2: ((d1 - nI, m), torch.float32),
                  3: ((ng - k, g, g), torch.float64), 4: ((ng,), torch.int32), 5: ((k,), torch.float64),
                  6: ((ng - k,), torch.float64)}
        shape, dt = shapes[which]
        out = torch.empty(shape, dtype=dt, device=dev)
        _check(lib().osscar_debug_get_state(self._h, which, _ptr(out)), "osscar_debug_get_state")
        return out


# ---------------------------------------------------------------------- functional forms (same names as the C ABI)
def osscar_gram(solver: Solver, chunks, W, damp: float = 0.0):
    return solver.gram(chunks, W, damp)


def osscar_init_support(solver: Solver, H, G, W, g, k, mode=INIT_ENERGY, support=None):
    return solver.init_support(H, G, W, g, k, mode, support)


def osscar_local_search(solver: Solver, max_swaps, **kw) -> SearchOutput:
    return solver.local_search(max_swaps, **kw)


def osscar_objective(solver: Solver, H, W, Wt) -> float:
    return solver.objective(H, W, Wt)
