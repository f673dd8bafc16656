"""ctypes binding of liblazyllm.so: argument marshalling only.

Every function here has the name of the C entry point it calls (include/lazyllm.h) and does
nothing but turn torch tensors into pointers and sizes.  PyTorch provides device memory and
streams; all arithmetic of the path runs in the library's kernels.  There is no fallback: if
the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblazyllm.so")

LAZY_BF16, LAZY_F32 = 0, 1
LAZY_MAX_LAYERS = 128
STATUS_NAMES = {0: "LAZY_OK", -1: "LAZY_E_BADARG", -2: "LAZY_E_BADSCHEDULE", -3: "LAZY_E_CAPACITY",
                -4: "LAZY_E_NOT_IN_AUX", -5: "LAZY_E_TIMEOUT", -6: "LAZY_E_CUDA", -7: "LAZY_E_STATE"}


class LazyError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        super().__init__(f"{fn} failed: {STATUS_NAMES.get(status, status)}")


class lazy_model_cfg(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32),
                ("head_dim", C.c_int32), ("d_ffn", C.c_int32), ("vocab", C.c_int32),
                ("rms_eps", C.c_float), ("rope_theta", C.c_float), ("dtype", C.c_int32),
                ("max_seqs", C.c_int32), ("max_prompt_tokens", C.c_int32),
                ("max_new_tokens", C.c_int32), ("n_kv_heads", C.c_int32)]


class lazy_weights(C.Structure):
    _fields_ = [("tok_embed", C.c_void_p), ("w_qkv", C.POINTER(C.c_void_p)),
                ("w_o", C.POINTER(C.c_void_p)), ("w_gate", C.POINTER(C.c_void_p)),
                ("w_up", C.POINTER(C.c_void_p)), ("w_down", C.POINTER(C.c_void_p)),
                ("g_attn", C.POINTER(C.c_void_p)), ("g_mlp", C.POINTER(C.c_void_p)),
                ("g_final", C.c_void_p), ("w_lm_head", C.c_void_p)]


class lazy_fp8_weights(C.Structure):
    _fields_ = [(n, C.POINTER(C.c_void_p)) for n in ("w_qkv", "w_o", "w_gate", "w_up", "w_down")] + \
               [(n, C.POINTER(C.c_float)) for n in ("s_qkv", "s_o", "s_gate", "s_up", "s_down")]


class lazy_schedule(C.Structure):
    _fields_ = [("n_points", C.c_int32), ("layer_entered", C.POINTER(C.c_int32)),
                ("keep_bp", C.POINTER(C.c_uint32))]


class lazy_stats(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("rows_computed", C.c_int32 * LAZY_MAX_LAYERS),
                ("kv_rows", C.c_int32 * LAZY_MAX_LAYERS), ("aux_rows", C.c_int32 * LAZY_MAX_LAYERS),
                ("revived", C.c_int32 * LAZY_MAX_LAYERS), ("kernel_launches", C.c_int64)]


LAZY_N_KERNEL_KINDS = 13
KERNEL_KINDS = ["gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down", "attention", "score", "select",
                "compact", "rmsnorm", "rope_kv", "embed", "lm_head", "other"]


class lazy_kernel_times(C.Structure):
    _fields_ = [("ms", C.c_float * LAZY_N_KERNEL_KINDS), ("launches", C.c_int32 * LAZY_N_KERNEL_KINDS),
                ("flops", C.c_double * LAZY_N_KERNEL_KINDS), ("bytes", C.c_double * LAZY_N_KERNEL_KINDS)]


# name -> (restype, argtypes); the list mirrors include/lazyllm.h
_P, _I, _F, _U, _Z = C.c_void_p, C.c_int32, C.c_float, C.c_uint32, C.c_size_t
_SIGNATURES = {
    "lazy_prefill_workspace_bytes": (_Z, [C.POINTER(lazy_model_cfg), C.POINTER(lazy_schedule)]),
    "lazy_prefill_workspace_bytes_ex": (_Z, [C.POINTER(lazy_model_cfg), C.POINTER(lazy_schedule), _I]),
    "lazy_prefill_init": (_I, [C.POINTER(lazy_model_cfg), C.POINTER(lazy_weights),
                               C.POINTER(lazy_schedule), _P, _Z, C.POINTER(_P)]),
    "lazy_prefill_run": (_I, [_P, _P, _P, C.POINTER(_I), _I, _P]),
    "lazy_decode_step": (_I, [_P, _P, _P, _P, _P]),
    "aux_cache_revive": (_I, [_P, _P, _I, _I, _P, _I, _P]),
    "lazy_get_kept": (_I, [_P, _P, _I, _I, _P, C.POINTER(_I)]),
    "lazy_get_scores": (_I, [_P, _P, _I, _I, _P, C.POINTER(_I)]),
    "lazy_set_forced_keep": (_I, [_P, _I, _I, _P, _I]),
    "lazy_set_debug_capture": (_I, [_P, _I]),
    "lazy_get_hidden": (_I, [_P, _P, _I, _P, C.POINTER(_I)]),
    "lazy_get_kv": (_I, [_P, _P, _I, _I, _P, _P, _P, C.POINTER(_I)]),
    "lazy_get_aux": (_I, [_P, _P, _I, _I, _P, _P, C.POINTER(_I)]),
    "lazy_get_revived": (_I, [_P, _P, _I, _I, _P, C.POINTER(_I)]),
    "lazy_get_stats": (_I, [_P, C.POINTER(lazy_stats)]),
    "lazy_set_kernel_timing": (_I, [_P, _I]),
    "lazy_get_kernel_times": (_I, [_P, _P, C.POINTER(lazy_kernel_times)]),
    "lazy_get_kernel_events": (_I, [_P, _P, _I, C.POINTER(_I), C.POINTER(C.c_float), C.POINTER(C.c_double),
                                    C.POINTER(C.c_double), C.POINTER(_I)]),
    "lazy_sync_status": (_I, [_P, _P]),
    "lazy_device_status": (_I, [_P]),
    "lazy_destroy": (None, [_P]),
    "lazy_strerror": (C.c_char_p, [_I]),
    "lazy_prune_op_workspace_bytes": (_Z, [_I, _I, _I, _I, _I, _I]),
    "lazy_prune_op": (_I, [_P, _I, _I, _I, _I, _I, _I, _F, _F, _U, _P, _P, _P, _P, _P, _P, _I,
                           _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _Z]),
    "lazy_k_rmsnorm": (_I, [_P, _I, _P, _P, _P, _I, _I, _F]),
    "lazy_k_gemm": (_I, [_P, _I, _I, _P, _P, _P, _P, _I, _I, _I]),
    "lazy_k_gemm_swiglu": (_I, [_P, _I, _I, _P, _P, _P, _P, _I, _I, _I]),
    "lazy_set_aux_point": (_I, [_P, _I]),
    "lazy_set_selection": (_I, [_P, _I]),
    "lazy_set_fp8_weights": (_I, [_P, C.POINTER(lazy_fp8_weights)]),
    "lazy_k_quant_rows_e4m3": (_I, [_P, _P, _P, _P, _I, _I]),
    "lazy_k_gemm_fp8": (_I, [_P, _P, _P, _P, _F, _P, _F, _P, _P, _I, _I, _I]),
    "lazy_k_gemm_scratch_bytes": (_Z, []),
    "lazy_k_gemm_ws": (_I, [_P, _I, _I, _P, _P, _P, _P, _I, _I, _I, _P, _Z]),
    "lazy_k_gemm_swiglu_ws": (_I, [_P, _I, _I, _P, _P, _P, _P, _I, _I, _I, _P, _Z]),
    "lazy_k_rope_kv": (_I, [_P, _I, _P, _P, _P, _P, _P, _I, _I, _I, _I, _F]),
    "lazy_k_attention": (_I, [_P, _I, _P, _I, _P, _P, _I, _P, _P, _I, _I, _I, _I, _I]),
    "lazy_k_score_scratch_floats": (_Z, [_I, _I, _I]),
    "lazy_k_score": (_I, [_P, _I, _P, _I, _P, _I, _P, _I, _I, _I, _I, _P, _P]),
    "lazy_k_score_static": (_I, [_P, _I, _P, _I, _P, _I, _P, _I, _I, _I, _I, _P]),
    "lazy_k_select": (_I, [_P, _P, _P, _P, _I, _P, _P]),
    "lazy_k_select_threshold": (_I, [_P, _P, _P, _I, C.c_uint32, _P, _P, _P]),
    "lazy_k_gather_rows": (_I, [_P, _P, _P, _P, _I, _I, _I]),
    "lazy_keep_count": (_I, [_I, _U, _I]),
    "lazy_status_detail": (_I, [C.POINTER(_I), C.POINTER(_I), C.POINTER(_I)]),
    "lazy_k_wait_selftest": (_I, [_P, _I, _U]),
}

_lib = None


def exported_names() -> List[str]:
    return sorted(_SIGNATURES)


def lib() -> C.CDLL:
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2407_14057_b200.build` "
                               "(there is no fallback path)")
        L = C.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def _check(fn: str, status: int) -> None:
    if status != 0:
        raise LazyError(fn, status)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def dtype_code(dt: torch.dtype) -> int:
    if dt == torch.bfloat16:
        return LAZY_BF16
    if dt == torch.float32:
        return LAZY_F32
    raise ValueError(f"unsupported dtype {dt}")


# ------------------------------------------------------------------------------- context
def _make_schedule(schedule: Sequence[Tuple[int, int]]):
    n = len(schedule)
    layers = (C.c_int32 * max(n, 1))(*[int(e) for e, _ in schedule])
    bps = (C.c_uint32 * max(n, 1))(*[int(b) for _, b in schedule])
    s = lazy_schedule(n, C.cast(layers, C.POINTER(C.c_int32)), C.cast(bps, C.POINTER(C.c_uint32)))
    return s, (layers, bps)


class LazyPrefill:
    """Owns a lazy_ctx plus the torch tensors (workspace, weights) it points into."""

    def __init__(self, shape, weights: Dict[str, object], schedule: Sequence[Tuple[int, int]],
                 dtype: torch.dtype, max_seqs: int, max_prompt_tokens: int, max_new_tokens: int = 0,
                 debug_capture: bool = False):
        L = lib()
        self.shape, self.dtype, self.schedule = shape, dtype, tuple(schedule)
        self.cfg = lazy_model_cfg(shape.n_layers, shape.d_model, shape.n_heads, shape.head_dim,
                                  shape.d_ffn, shape.vocab, shape.rms_eps, shape.rope_theta,
                                  dtype_code(dtype), max_seqs, max_prompt_tokens, max_new_tokens,
                                  getattr(shape, "n_kv_heads", 0))
        self._sched, self._sched_keep = _make_schedule(schedule)
        nbytes = L.lazy_prefill_workspace_bytes_ex(C.byref(self.cfg), C.byref(self._sched),
                                                   1 if debug_capture else 0)
        if nbytes == 0:
            raise LazyError("lazy_prefill_workspace_bytes", -1)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        self.weights = weights  # keeps the tensors alive
        n = shape.n_layers

        def arr(key):
            a = (C.c_void_p * n)(*[_ptr(lw[key]) for lw in weights["layers"]])
            return a

        self._arrs = {k: arr(k) for k in ("w_qkv", "w_o", "w_gate", "w_up", "w_down", "g_attn", "g_mlp")}
        w = lazy_weights(_ptr(weights["tok_embed"]),
                         *[C.cast(self._arrs[k], C.POINTER(C.c_void_p))
                           for k in ("w_qkv", "w_o", "w_gate", "w_up", "w_down", "g_attn", "g_mlp")],
                         _ptr(weights["g_final"]), _ptr(weights["w_lm_head"]))
        ctx = C.c_void_p()
        _check("lazy_prefill_init", L.lazy_prefill_init(C.byref(self.cfg), C.byref(w), C.byref(self._sched),
                                                        base, nbytes, C.byref(ctx)))
        self.ctx = ctx
        self._keep_alive: List[torch.Tensor] = []
        if debug_capture:
            _check("lazy_set_debug_capture", L.lazy_set_debug_capture(self.ctx, 1))

    def close(self):
        if getattr(self, "ctx", None):
            lib().lazy_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # --- calls, named after the C entry points
    def lazy_prefill_run(self, d_prompt_ids: torch.Tensor, cu_seqlens: Sequence[int],
                         d_logits: torch.Tensor) -> None:
        n_seqs = len(cu_seqlens) - 1
        cu = (C.c_int32 * (n_seqs + 1))(*[int(v) for v in cu_seqlens])
        _check("lazy_prefill_run", lib().lazy_prefill_run(self.ctx, _stream(), _ptr(d_prompt_ids), cu,
                                                          n_seqs, _ptr(d_logits)))

    def lazy_decode_step(self, d_new_ids: torch.Tensor, d_logits: torch.Tensor,
                         d_next_ids: Optional[torch.Tensor]) -> None:
        _check("lazy_decode_step", lib().lazy_decode_step(self.ctx, _stream(), _ptr(d_new_ids),
                                                          _ptr(d_logits), _ptr(d_next_ids)))

    def aux_cache_revive(self, layer: int, seq: int, d_positions: torch.Tensor) -> torch.Tensor:
        n = d_positions.numel()
        out = torch.empty((n, self.shape.d_model), dtype=self.dtype, device="cuda")
        _check("aux_cache_revive", lib().aux_cache_revive(self.ctx, _stream(), layer, seq,
                                                          _ptr(d_positions), n, _ptr(out)))
        return out

    def lazy_get_kept(self, layer_entered: int, seq: int = 0) -> torch.Tensor:
        cnt = C.c_int32()
        _check("lazy_get_kept", lib().lazy_get_kept(self.ctx, _stream(), layer_entered, seq, None, C.byref(cnt)))
        out = torch.empty(cnt.value, dtype=torch.int32, device="cuda")
        _check("lazy_get_kept", lib().lazy_get_kept(self.ctx, _stream(), layer_entered, seq, _ptr(out), C.byref(cnt)))
        return out

    def lazy_get_scores(self, layer: int, seq: int = 0) -> torch.Tensor:
        cnt = C.c_int32()
        _check("lazy_get_scores", lib().lazy_get_scores(self.ctx, _stream(), layer, seq, None, C.byref(cnt)))
        out = torch.empty(cnt.value, dtype=torch.float32, device="cuda")
        _check("lazy_get_scores", lib().lazy_get_scores(self.ctx, _stream(), layer, seq, _ptr(out), C.byref(cnt)))
        return out

    def lazy_set_forced_keep(self, layer_entered: int, seq: int, d_pos: Optional[torch.Tensor]) -> None:
        n = 0 if d_pos is None else d_pos.numel()
        if d_pos is not None:
            self._keep_alive.append(d_pos)
        _check("lazy_set_forced_keep", lib().lazy_set_forced_keep(self.ctx, layer_entered, seq, _ptr(d_pos), n))

    def lazy_set_aux_point(self, after_layer: bool) -> None:
        _check("lazy_set_aux_point", lib().lazy_set_aux_point(self.ctx, 1 if after_layer else 0))

    def lazy_set_fp8_weights(self, q: Optional[dict]) -> None:
        """q: {"layers": [{name: (codes uint8 CUDA tensor [out, in], scale)}]} for the five projection
        matrices of every layer (the output of synth.quantize_projections_e4m3 moved to the device), or None
        to return to the 16-bit weights."""
        if q is None:
            _check("lazy_set_fp8_weights", lib().lazy_set_fp8_weights(self.ctx, None))
            self._fp8 = None
            return
        names = ("w_qkv", "w_o", "w_gate", "w_up", "w_down")
        n = self.shape.n_layers
        ptrs = [(C.c_void_p * n)(*[_ptr(lq[k][0]) for lq in q["layers"]]) for k in names]
        scales = [(C.c_float * n)(*[float(lq[k][1]) for lq in q["layers"]]) for k in names]
        w = lazy_fp8_weights(*[C.cast(a, C.POINTER(C.c_void_p)) for a in ptrs],
                             *[C.cast(a, C.POINTER(C.c_float)) for a in scales])
        _check("lazy_set_fp8_weights", lib().lazy_set_fp8_weights(self.ctx, C.byref(w)))
        self._fp8 = (q, ptrs, scales)   # keeps the tensors alive (the library copies the arrays themselves)

    def lazy_set_selection(self, threshold: bool) -> None:
        _check("lazy_set_selection", lib().lazy_set_selection(self.ctx, 1 if threshold else 0))

    def lazy_get_hidden(self, layer: int) -> torch.Tensor:
        rows = C.c_int32()
        _check("lazy_get_hidden", lib().lazy_get_hidden(self.ctx, _stream(), layer, None, C.byref(rows)))
        out = torch.empty((rows.value, self.shape.d_model), dtype=self.dtype, device="cuda")
        _check("lazy_get_hidden", lib().lazy_get_hidden(self.ctx, _stream(), layer, _ptr(out), C.byref(rows)))
        return out

    def lazy_get_kv(self, layer: int, seq: int = 0):
        cnt = C.c_int32()
        _check("lazy_get_kv", lib().lazy_get_kv(self.ctx, _stream(), layer, seq, None, None, None, C.byref(cnt)))
        d = (getattr(self.shape, "n_kv_heads", 0) or self.shape.n_heads) * self.shape.head_dim
        pos = torch.empty(cnt.value, dtype=torch.int32, device="cuda")
        k = torch.empty((cnt.value, d), dtype=self.dtype, device="cuda")
        v = torch.empty((cnt.value, d), dtype=self.dtype, device="cuda")
        _check("lazy_get_kv", lib().lazy_get_kv(self.ctx, _stream(), layer, seq, _ptr(pos), _ptr(k), _ptr(v),
                                                C.byref(cnt)))
        return pos, k, v

    def lazy_get_aux(self, layer: int, seq: int = 0):
        cnt = C.c_int32()
        _check("lazy_get_aux", lib().lazy_get_aux(self.ctx, _stream(), layer, seq, None, None, C.byref(cnt)))
        pos = torch.empty(cnt.value, dtype=torch.int32, device="cuda")
        hid = torch.empty((cnt.value, self.shape.d_model), dtype=self.dtype, device="cuda")
        _check("lazy_get_aux", lib().lazy_get_aux(self.ctx, _stream(), layer, seq, _ptr(pos), _ptr(hid),
                                                  C.byref(cnt)))
        return pos, hid

    def lazy_get_revived(self, layer_entered: int, seq: int = 0) -> torch.Tensor:
        cnt = C.c_int32()
        _check("lazy_get_revived", lib().lazy_get_revived(self.ctx, _stream(), layer_entered, seq, None,
                                                          C.byref(cnt)))
        out = torch.empty(cnt.value, dtype=torch.int32, device="cuda")
        _check("lazy_get_revived", lib().lazy_get_revived(self.ctx, _stream(), layer_entered, seq, _ptr(out),
                                                          C.byref(cnt)))
        return out

    def lazy_get_stats(self) -> lazy_stats:
        s = lazy_stats()
        _check("lazy_get_stats", lib().lazy_get_stats(self.ctx, C.byref(s)))
        return s

    def lazy_set_kernel_timing(self, on, kinds: Optional[Sequence[str]] = None) -> None:
        """on: bool; kinds: optional names from KERNEL_KINDS to time only those."""
        arg = 1 if on else 0
        if on and kinds:
            arg = sum(1 << KERNEL_KINDS.index(k) for k in kinds) << 1
        _check("lazy_set_kernel_timing", lib().lazy_set_kernel_timing(self.ctx, arg))

    def lazy_get_kernel_times(self) -> Dict[str, Dict[str, float]]:
        t = lazy_kernel_times()
        _check("lazy_get_kernel_times", lib().lazy_get_kernel_times(self.ctx, _stream(), C.byref(t)))
        return {name: {"ms": t.ms[i], "launches": t.launches[i], "flops": t.flops[i], "bytes": t.bytes[i]}
                for i, name in enumerate(KERNEL_KINDS)}

    def lazy_get_kernel_events(self) -> List[Tuple[str, float, float, float]]:
        """(kind, ms, flops, bytes) of every timed launch of the latest run, in launch order."""
        cap = 4096
        kinds, ms = (C.c_int32 * cap)(), (C.c_float * cap)()
        fl, by, cnt = (C.c_double * cap)(), (C.c_double * cap)(), C.c_int32()
        _check("lazy_get_kernel_events", lib().lazy_get_kernel_events(self.ctx, _stream(), cap, kinds, ms, fl, by,
                                                                      C.byref(cnt)))
        return [(KERNEL_KINDS[kinds[i]], ms[i], fl[i], by[i]) for i in range(min(cnt.value, cap))]

    def lazy_sync_status(self) -> None:
        _check("lazy_sync_status", lib().lazy_sync_status(self.ctx, _stream()))


# ------------------------------------------------------------------------------- context-free calls
def lazy_device_status() -> None:
    _check("lazy_device_status", lib().lazy_device_status(_stream()))


def lazy_status_detail() -> Tuple[int, int, int]:
    """(where, a, b) of the latest non-OK device status this process took."""
    w, a, b = C.c_int32(), C.c_int32(), C.c_int32()
    _check("lazy_status_detail", lib().lazy_status_detail(C.byref(w), C.byref(a), C.byref(b)))
    return w.value, a.value, b.value


def lazy_k_wait_selftest(which: int, limit_us: int) -> None:
    _check("lazy_k_wait_selftest", lib().lazy_k_wait_selftest(_stream(), which, limit_us))


def lazy_keep_count(n_total: int, keep_bp: int, n_present: int) -> int:
    return int(lib().lazy_keep_count(n_total, keep_bp, n_present))


def lazy_k_rmsnorm(x: torch.Tensor, g: torch.Tensor, eps: float) -> torch.Tensor:
    y = torch.empty_like(x)
    _check("lazy_k_rmsnorm", lib().lazy_k_rmsnorm(_stream(), dtype_code(x.dtype), _ptr(x), _ptr(g), _ptr(y),
                                                  x.shape[0], x.shape[1], eps))
    return y


def lazy_k_gemm_scratch(device="cuda") -> torch.Tensor:
    """Zeroed scratch for the `scratch=` argument of lazy_k_gemm / lazy_k_gemm_swiglu."""
    return torch.zeros(lib().lazy_k_gemm_scratch_bytes(), dtype=torch.uint8, device=device)


def lazy_k_gemm(A: torch.Tensor, B: torch.Tensor, R: Optional[torch.Tensor] = None, impl: int = 0,
                out: Optional[torch.Tensor] = None, scratch: Optional[torch.Tensor] = None) -> torch.Tensor:
    M, K = A.shape
    N = B.shape[0]
    Cm = out if out is not None else torch.empty((M, N), dtype=A.dtype, device=A.device)
    if scratch is None:
        _check("lazy_k_gemm", lib().lazy_k_gemm(_stream(), dtype_code(A.dtype), impl, _ptr(A), _ptr(B), _ptr(R),
                                                _ptr(Cm), M, N, K))
    else:
        _check("lazy_k_gemm_ws", lib().lazy_k_gemm_ws(_stream(), dtype_code(A.dtype), impl, _ptr(A), _ptr(B),
                                                      _ptr(R), _ptr(Cm), M, N, K, _ptr(scratch), scratch.numel()))
    return Cm


def lazy_k_gemm_swiglu(A: torch.Tensor, Bg: torch.Tensor, Bu: torch.Tensor, impl: int = 0,
                       out: Optional[torch.Tensor] = None, scratch: Optional[torch.Tensor] = None) -> torch.Tensor:
    M, K = A.shape
    F = Bg.shape[0]
    Cm = out if out is not None else torch.empty((M, F), dtype=A.dtype, device=A.device)
    if scratch is None:
        _check("lazy_k_gemm_swiglu", lib().lazy_k_gemm_swiglu(_stream(), dtype_code(A.dtype), impl, _ptr(A),
                                                              _ptr(Bg), _ptr(Bu), _ptr(Cm), M, F, K))
    else:
        _check("lazy_k_gemm_swiglu_ws",
               lib().lazy_k_gemm_swiglu_ws(_stream(), dtype_code(A.dtype), impl, _ptr(A), _ptr(Bg), _ptr(Bu),
                                           _ptr(Cm), M, F, K, _ptr(scratch), scratch.numel()))
    return Cm


def lazy_k_quant_rows_e4m3(x: torch.Tensor):
    """(codes uint8 [M, K], scale fp32 [M]) of the per-row e4m3 quantisation of bf16 x [M, K]."""
    M, K = x.shape
    q = torch.empty((M, K), dtype=torch.uint8, device=x.device)
    sc = torch.empty(max(M, 1), dtype=torch.float32, device=x.device)
    _check("lazy_k_quant_rows_e4m3", lib().lazy_k_quant_rows_e4m3(_stream(), _ptr(x), _ptr(q), _ptr(sc), M, K))
    return q, sc[:M]


def lazy_k_gemm_fp8(A8: torch.Tensor, a_scale: torch.Tensor, B8: torch.Tensor, w_scale: float,
                    B8u: Optional[torch.Tensor] = None, w_scale_up: float = 1.0,
                    R: Optional[torch.Tensor] = None) -> torch.Tensor:
    M, K = A8.shape
    N = B8.shape[0]
    Cm = torch.empty((M, N), dtype=torch.bfloat16, device=A8.device)
    _check("lazy_k_gemm_fp8", lib().lazy_k_gemm_fp8(_stream(), _ptr(A8), _ptr(a_scale), _ptr(B8), w_scale, _ptr(B8u),
                                                    w_scale_up, _ptr(R), _ptr(Cm), M, N, K))
    return Cm


def lazy_k_rope_kv(qkv: torch.Tensor, pos: torch.Tensor, n_heads: int, head_dim: int, max_pos: int,
                   theta: float):
    """Rotates q and k inside qkv in place; returns (k_cache, v_cache)."""
    n = qkv.shape[0]
    d = n_heads * head_dim
    table = torch.empty(max_pos * head_dim, dtype=torch.float32, device=qkv.device)
    kc = torch.empty((n, d), dtype=qkv.dtype, device=qkv.device)
    vc = torch.empty((n, d), dtype=qkv.dtype, device=qkv.device)
    _check("lazy_k_rope_kv", lib().lazy_k_rope_kv(_stream(), dtype_code(qkv.dtype), _ptr(qkv), _ptr(pos),
                                                  _ptr(table), _ptr(kc), _ptr(vc), n, n_heads, head_dim,
                                                  max_pos, theta))
    return kc, vc


def lazy_k_attention(q: torch.Tensor, ldq: int, k: torch.Tensor, v: torch.Tensor, ldkv: int,
                     cu_seqlens: torch.Tensor, max_len: int, n_total: int, n_heads: int,
                     head_dim: int) -> torch.Tensor:
    o = torch.empty((n_total, n_heads * head_dim), dtype=k.dtype, device=k.device)
    _check("lazy_k_attention", lib().lazy_k_attention(_stream(), dtype_code(k.dtype), q.data_ptr(), ldq,
                                                      _ptr(k), _ptr(v), ldkv, _ptr(o), _ptr(cu_seqlens),
                                                      cu_seqlens.numel() - 1, max_len, n_total, n_heads,
                                                      head_dim))
    return o


def lazy_k_score(q: torch.Tensor, ldq: int, k: torch.Tensor, ldkv: int, cu_seqlens: torch.Tensor,
                 n_total: int, n_heads: int, head_dim: int,
                 out: Optional[Tuple[torch.Tensor, torch.Tensor]] = None) -> torch.Tensor:
    """out = (scratch, scores) buffers of an earlier call may be handed back in (timing loops)."""
    n_seqs = cu_seqlens.numel() - 1
    if out is not None:
        scratch, scores = out
    else:
        nf = lib().lazy_k_score_scratch_floats(n_seqs, n_total, n_heads)
        scratch = torch.empty(max(nf, 1), dtype=torch.float32, device=k.device)
        scores = torch.empty(n_total, dtype=torch.float32, device=k.device)
    _check("lazy_k_score", lib().lazy_k_score(_stream(), dtype_code(k.dtype), q.data_ptr(), ldq, _ptr(k), ldkv,
                                              _ptr(cu_seqlens), n_seqs, n_total, n_heads, head_dim,
                                              _ptr(scratch), _ptr(scores)))
    return scores


def lazy_k_score_static(q: torch.Tensor, ldq: int, k: torch.Tensor, ldkv: int, cu_seqlens: torch.Tensor,
                        n_total: int, n_heads: int, head_dim: int, scores: torch.Tensor) -> torch.Tensor:
    """Eq. 1 scores with the scratch held inside the library: nothing is allocated by the call, so the
    caller passes the output tensor too."""
    _check("lazy_k_score_static", lib().lazy_k_score_static(
        _stream(), dtype_code(k.dtype), q.data_ptr(), ldq, _ptr(k), ldkv, _ptr(cu_seqlens),
        cu_seqlens.numel() - 1, n_total, n_heads, head_dim, _ptr(scores)))
    return scores


def lazy_k_select(scores: torch.Tensor, cu_in: torch.Tensor, cu_keep: torch.Tensor, n_in: Optional[int] = None,
                  n_keep: Optional[int] = None, out: Optional[Tuple[torch.Tensor, torch.Tensor]] = None):
    """n_in / n_keep (totals over the batch) and out = (keep, drop) buffers may be passed by a caller that
    knows them, which keeps the call free of device reads and allocations (timing loops)."""
    n_seqs = cu_in.numel() - 1
    n_in = int(cu_in[-1].item()) if n_in is None else n_in
    n_keep = int(cu_keep[-1].item()) if n_keep is None else n_keep
    if out is not None:
        keep, drop = out
    else:
        keep = torch.empty(max(n_keep, 1), dtype=torch.int32, device=scores.device)
        drop = torch.empty(max(n_in - n_keep, 1), dtype=torch.int32, device=scores.device)
    _check("lazy_k_select", lib().lazy_k_select(_stream(), _ptr(scores), _ptr(cu_in), _ptr(cu_keep), n_seqs,
                                                _ptr(keep), _ptr(drop)))
    return keep[:n_keep], drop[:n_in - n_keep]


def lazy_k_select_threshold(scores: torch.Tensor, cu_in: torch.Tensor, prune_bp: int):
    """Returns (keep_idx, drop_idx, counts): index buffers packed per sequence from cu_in[s], counts per sequence."""
    n_seqs = cu_in.numel() - 1
    n_in = int(cu_in[-1].item())
    keep = torch.full((max(n_in, 1),), -1, dtype=torch.int32, device=scores.device)
    drop = torch.full((max(n_in, 1),), -1, dtype=torch.int32, device=scores.device)
    counts = torch.zeros(max(n_seqs, 1), dtype=torch.int32, device=scores.device)
    _check("lazy_k_select_threshold",
           lib().lazy_k_select_threshold(_stream(), _ptr(scores), _ptr(cu_in), n_seqs, prune_bp, _ptr(keep),
                                         _ptr(drop), _ptr(counts)))
    return keep, drop, counts[:n_seqs]


def lazy_k_gather_rows(src: torch.Tensor, idx: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    n = idx.numel()
    dst = out if out is not None else torch.empty((n,) + tuple(src.shape[1:]), dtype=src.dtype, device=src.device)
    row_bytes = src[0].numel() * src.element_size()
    _check("lazy_k_gather_rows", lib().lazy_k_gather_rows(_stream(), _ptr(src), _ptr(idx), _ptr(dst), n,
                                                          row_bytes, src.shape[0]))
    return dst


def lazy_prune_op(x: torch.Tensor, pos: torch.Tensor, w_qkv: torch.Tensor, w_o: torch.Tensor,
                  g_attn: torch.Tensor, n_heads: int, head_dim: int, keep_bp: int, max_pos: int,
                  rms_eps: float = 1e-6, rope_theta: float = 1e4,
                  forced_keep_idx: Optional[torch.Tensor] = None,
                  workspace: Optional[torch.Tensor] = None, outputs: Optional[dict] = None) -> dict:
    n, d = x.shape
    dt = dtype_code(x.dtype)
    if forced_keep_idx is not None:
        n_keep = forced_keep_idx.numel()
    else:
        n_keep = lazy_keep_count(n, keep_bp, n)
    n_drop = n - n_keep
    nbytes = lib().lazy_prune_op_workspace_bytes(n, d, n_heads, head_dim, dt, max_pos)
    if workspace is None:
        workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=x.device)
    base = (workspace.data_ptr() + 255) // 256 * 256
    dev = x.device
    o = outputs if outputs is not None else {
        "scores": torch.empty(n, dtype=torch.float32, device=dev),
        "keep_idx": torch.empty(n_keep, dtype=torch.int32, device=dev),
        "drop_idx": torch.empty(max(n_drop, 1), dtype=torch.int32, device=dev),
        "hidden_kept": torch.empty((n_keep, d), dtype=x.dtype, device=dev),
        "k_kept": torch.empty((n_keep, d), dtype=x.dtype, device=dev),
        "v_kept": torch.empty((n_keep, d), dtype=x.dtype, device=dev),
        "pos_kept": torch.empty(n_keep, dtype=torch.int32, device=dev),
        "aux_hidden": torch.empty((max(n_drop, 1), d), dtype=x.dtype, device=dev),
        "aux_pos": torch.empty(max(n_drop, 1), dtype=torch.int32, device=dev),
    }
    _check("lazy_prune_op", lib().lazy_prune_op(
        _stream(), dt, n, d, n_heads, head_dim, max_pos, rms_eps, rope_theta, keep_bp, _ptr(x), _ptr(pos),
        _ptr(w_qkv), _ptr(w_o), _ptr(g_attn), _ptr(forced_keep_idx),
        0 if forced_keep_idx is None else forced_keep_idx.numel(), _ptr(o["scores"]), _ptr(o["keep_idx"]),
        _ptr(o["drop_idx"]), _ptr(o["hidden_kept"]), _ptr(o["k_kept"]), _ptr(o["v_kept"]), _ptr(o["pos_kept"]),
        _ptr(o["aux_hidden"]), _ptr(o["aux_pos"]), base, nbytes))
    o["n_keep"], o["n_drop"], o["workspace"] = n_keep, n_drop, workspace
    return o
