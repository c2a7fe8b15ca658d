"""Thin ctypes binding over the C ABI of include/citrus.h.

Argument marshalling only: every step of the path runs in the CUDA library.
There is no CPU fallback; if libcitrus.so is missing or a call fails, an
exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcitrus.so")

MODE_SHARED = 0
MODE_INDIVIDUAL = 1
MODE_FP32 = 2
MODE_LAYERWISE = 4
MODE_STANDARD = 8
MODE_ACCUMULATE = 0x20000000
MODE_DEFERRED_LM = 0x40000000
MODE_POSITION_SHIFT = 0x80000000
MAX_INSTR = 4096
MAX_CANDIDATES = 49152

KERNEL_NAMES = ["attention", "score_lse", "colsum", "select", "compact", "rope"]

EXPORTS = [
    "citrus_create", "citrus_set_batch", "citrus_set_batch_lanes", "citrus_reset", "citrus_process_chunk", "citrus_process_chunk_slot",
    "citrus_process_chunk_host", "citrus_process_document_host", "citrus_process_chunk_batch", "citrus_cache_view", "citrus_step_view", "citrus_profile",
    "citrus_profile_read", "citrus_importance_static", "citrus_intersection_ratio", "citrus_set_rope_base",
    "citrus_poll_status", "citrus_set_inputs_ready", "citrus_set_attention_beside", "citrus_debug_expire_wait",
    "citrus_destroy", "citrus_strerror",
]

_lib = None


class CitrusError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {code} ({strerror(code)})")


def load() -> C.CDLL:
    """Load libcitrus.so (built by paper_2406_12018_b200.build); raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2406_12018_b200.build`; "
                           "there is no fallback path")
    lib = C.CDLL(LIB_PATH)
    vp, i = C.c_void_p, C.c_int
    lib.citrus_create.argtypes = [C.POINTER(vp), i, i, i, i, i, i, C.c_uint]
    lib.citrus_set_batch.argtypes = [vp, i]
    lib.citrus_set_batch_lanes.argtypes = [vp, i]
    lib.citrus_reset.argtypes = [vp]
    lib.citrus_process_chunk.argtypes = [vp, i, vp, vp, vp, i, vp, i, vp, vp]
    lib.citrus_process_chunk_slot.argtypes = [vp, i, i, vp, vp, vp, i, vp, i, vp, vp]
    lib.citrus_process_chunk_batch.argtypes = [vp, i, i, C.POINTER(i), C.POINTER(i), vp, vp, vp, C.POINTER(i), vp, vp, vp]
    lib.citrus_process_chunk_host.argtypes = [vp, i, i, vp, vp, vp, i, vp, i, vp, vp]
    lib.citrus_process_document_host.argtypes = [vp, i, i, vp, vp, vp, C.c_longlong, vp, i, vp, vp]
    lib.citrus_cache_view.argtypes = [vp, i, i, i, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(i)]
    lib.citrus_step_view.argtypes = [vp, i, i, i, C.POINTER(vp), C.POINTER(i), C.POINTER(vp),
                                     C.POINTER(i), C.POINTER(i), C.POINTER(i)]
    lib.citrus_intersection_ratio.argtypes = [vp, i, i, vp, vp]
    lib.citrus_set_rope_base.argtypes = [vp, C.c_double]
    lib.citrus_profile.argtypes = [vp, i]
    lib.citrus_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_longlong)]
    lib.citrus_importance_static.argtypes = [vp, i, vp, i, i, i, i, C.c_uint, vp, i, vp, vp]
    lib.citrus_poll_status.argtypes = [vp]
    lib.citrus_set_inputs_ready.argtypes = [vp, i]
    lib.citrus_set_attention_beside.argtypes = [vp, i]
    lib.citrus_debug_expire_wait.argtypes = [vp, C.c_ulonglong, vp]
    lib.citrus_destroy.argtypes = [vp]
    lib.citrus_strerror.argtypes = [i]
    lib.citrus_strerror.restype = C.c_char_p
    for name in EXPORTS:
        if name != "citrus_strerror":
            getattr(lib, name).restype = i
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load().citrus_strerror(code).decode()


def importance_static(Q_s: torch.Tensor, K: torch.Tensor, scores: torch.Tensor, stream=None,
                      status: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Eq. 1 column sums of scoring rows Q_s [n_s, H_q, D] over keys K [n, H_kv, D] into the caller's
    `scores` [H_kv, >= n] fp32, through the entry point that allocates nothing (see citrus.h).
    status: optional caller-owned int32 device word (zeroed by the caller), set to 1 if a bounded wait expires."""
    assert Q_s.is_cuda and K.is_cuda and scores.is_cuda and scores.dtype == torch.float32
    assert status is None or (status.is_cuda and status.dtype == torch.int32)
    assert Q_s.is_contiguous() and K.is_contiguous() and scores.is_contiguous() and Q_s.dtype == K.dtype
    mode = MODE_FP32 if Q_s.dtype == torch.float32 else 0
    rc = load().citrus_importance_static(Q_s.data_ptr(), Q_s.shape[0], K.data_ptr(), K.shape[0], Q_s.shape[1],
                                         K.shape[1], Q_s.shape[2], mode, scores.data_ptr(), scores.shape[1],
                                         None if status is None else status.data_ptr(), _stream_ptr(stream))
    if rc != 0:
        raise CitrusError(rc, "citrus_importance_static")
    return scores


class _DevView:
    """Zero-copy torch view of library-owned device memory."""

    def __init__(self, ptr: int, shape, typestr: str, strides=None):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": typestr, "data": (ptr, False),
                                         "version": 2, "strides": strides}


def _view(ptr, shape, typestr, itemsize, strides_elems=None):
    strides = None if strides_elems is None else tuple(s * itemsize for s in strides_elems)
    return torch.as_tensor(_DevView(ptr, shape, typestr, strides), device="cuda")


def _stream_ptr(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


class Citrus:
    """One eviction context (all layers and sequence slots of one geometry)."""

    def __init__(self, layers, q_heads, kv_heads, head_dim, budget_k, chunk_s, mode="shared", dtype="bf16",
                 lm_window=0, layerwise=False, n_seqs=1, start_size=0, accumulate=False, deferred_lm=False, position_shift=False,
                 rope_base=None):
        lib = load()
        bits = {"individual": MODE_INDIVIDUAL, "standard": MODE_STANDARD}.get(mode, MODE_SHARED)
        bits |= MODE_FP32 if dtype == "fp32" else 0
        bits |= MODE_LAYERWISE if layerwise else 0
        bits |= (int(lm_window) & 0xFFFF) << 8
        bits |= (int(start_size) & 0xF) << 24
        bits |= MODE_ACCUMULATE if accumulate else 0
        bits |= MODE_DEFERRED_LM if deferred_lm else 0
        bits |= MODE_POSITION_SHIFT if position_shift else 0
        self._h = C.c_void_p()
        rc = lib.citrus_create(C.byref(self._h), layers, q_heads, kv_heads, head_dim, budget_k, chunk_s, bits)
        if rc != 0:
            self._h = None
            raise CitrusError(rc, "citrus_create")
        self.layers, self.q_heads, self.kv_heads, self.head_dim = layers, q_heads, kv_heads, head_dim
        self.budget_k, self.chunk_s = budget_k, chunk_s
        self.individual = mode == "individual"
        # row capacity of each cache's buffers: with deferred eviction cache 0 also holds the previous chunk
        self.cap = (budget_k + (chunk_s if deferred_lm else 0), budget_k)
        self.torch_dtype = torch.float32 if dtype == "fp32" else torch.bfloat16
        if rope_base is not None:
            rc = lib.citrus_set_rope_base(self._h, float(rope_base))
            if rc != 0:
                self.close()
                raise CitrusError(rc, "citrus_set_rope_base")
        if n_seqs != 1:
            rc = lib.citrus_set_batch(self._h, n_seqs)
            if rc != 0:
                self.close()
                raise CitrusError(rc, "citrus_set_batch")

    # -- calls -------------------------------------------------------------
    def set_batch_lanes(self, n_lanes: int):
        """Side streams of the packed batch call: 0 = chosen per call, 1 = the caller's stream only, up to 8."""
        rc = load().citrus_set_batch_lanes(self._h, int(n_lanes))
        if rc != 0:
            raise CitrusError(rc, "citrus_set_batch_lanes")

    def _check(self, t: torch.Tensor, cuda: bool):
        assert t.dtype == self.torch_dtype and t.is_contiguous() and t.is_cuda == cuda

    def process_chunk(self, layer, Qc, Kc, Vc, Qi, out: Optional[torch.Tensor] = None, slot=0, stream=None):
        """Qi = None is only valid in standard mode (the chunk scores its own eviction)."""
        for t in (Qc, Kc, Vc) + (() if Qi is None else (Qi,)):
            self._check(t, True)
        if out is None:
            out = torch.empty_like(Qc)
        rc = load().citrus_process_chunk_slot(self._h, layer, slot, Qc.data_ptr(), Kc.data_ptr(), Vc.data_ptr(),
                                              Qc.shape[0], None if Qi is None else Qi.data_ptr(),
                                              0 if Qi is None else Qi.shape[0], out.data_ptr(), _stream_ptr(stream))
        if rc != 0:
            raise CitrusError(rc, "citrus_process_chunk")
        return out

    def process_chunk_batch(self, layer, slots, tok_offset, Q, K, V, instr_offset, Qi, out=None, stream=None):
        """One chunk for each active sequence, packed token-major (offsets are host lists of len(slots) + 1)."""
        for t in (Q, K, V, Qi):
            self._check(t, True)
        if out is None:
            out = torch.empty_like(Q)
        n = len(slots)
        arr = lambda xs: (C.c_int * len(xs))(*[int(x) for x in xs])
        rc = load().citrus_process_chunk_batch(self._h, layer, n, arr(slots), arr(tok_offset), Q.data_ptr(), K.data_ptr(),
                                               V.data_ptr(), arr(instr_offset), Qi.data_ptr(), out.data_ptr(),
                                               _stream_ptr(stream))
        if rc != 0:
            raise CitrusError(rc, "citrus_process_chunk_batch")
        return out

    def process_chunk_host(self, layer, Qc, Kc, Vc, Qi, out, slot=0, stream=None):
        for t in (Qc, Kc, Vc, Qi, out):
            self._check(t, False)
        rc = load().citrus_process_chunk_host(self._h, layer, slot, Qc.data_ptr(), Kc.data_ptr(), Vc.data_ptr(),
                                              Qc.shape[0], Qi.data_ptr(), Qi.shape[0], out.data_ptr(),
                                              _stream_ptr(stream))
        if rc != 0:
            raise CitrusError(rc, "citrus_process_chunk_host")
        return out

    def process_document_host(self, layer, Q, K, V, Qi, out, slot=0, stream=None):
        """A whole document from host tensors; copies and steps overlap inside the library."""
        for t in (Q, K, V, Qi, out):
            self._check(t, False)
        rc = load().citrus_process_document_host(self._h, layer, slot, Q.data_ptr(), K.data_ptr(), V.data_ptr(),
                                                 Q.shape[0], Qi.data_ptr(), Qi.shape[0], out.data_ptr(),
                                                 _stream_ptr(stream))
        if rc != 0:
            raise CitrusError(rc, "citrus_process_document_host")
        return out

    def cache_view(self, layer, which=0, slot=0) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
        """(K [H_kv, n_rows, D], V, positions [H_kv, n_rows]) views of the current cache."""
        K, V, P, n = C.c_void_p(), C.c_void_p(), C.c_void_p(), C.c_int()
        rc = load().citrus_cache_view(self._h, layer, which, slot, C.byref(K), C.byref(V), C.byref(P), C.byref(n))
        if rc != 0:
            raise CitrusError(rc, "citrus_cache_view")
        H, k, D = self.kv_heads, self.cap[which], self.head_dim
        if self.torch_dtype == torch.float32:
            Kt, Vt = (_view(p.value, (H, k, D), "<f4", 4) for p in (K, V))
        else:
            Kt, Vt = (_view(p.value, (H, k, D), "<i2", 2).view(torch.bfloat16) for p in (K, V))
        Pt = _view(P.value, (H, k), "<i4", 4)
        return Kt[:, :n.value], Vt[:, :n.value], Pt[:, :n.value]

    def intersection_ratio(self, layer, slot=0, stream=None) -> torch.Tensor:
        """[H_kv] fp32: share of the instruction cache's states that the language-modelling cache also holds."""
        out = torch.empty(self.kv_heads, dtype=torch.float32, device="cuda")
        rc = load().citrus_intersection_ratio(self._h, layer, slot, out.data_ptr(), _stream_ptr(stream))
        if rc != 0:
            raise CitrusError(rc, "citrus_intersection_ratio")
        return out

    def step_view(self, layer, which=0, slot=0):
        """(scores [H_kv, n] fp32, idx [H_kv, kept] int32, m_before) of the last call."""
        S, I = C.c_void_p(), C.c_void_p()
        stride, n, kept, m = C.c_int(), C.c_int(), C.c_int(), C.c_int()
        rc = load().citrus_step_view(self._h, layer, which, slot, C.byref(S), C.byref(stride), C.byref(I),
                                     C.byref(n), C.byref(kept), C.byref(m))
        if rc != 0:
            raise CitrusError(rc, "citrus_step_view")
        St = _view(S.value, (self.kv_heads, stride.value), "<f4", 4)[:, :n.value]
        It = _view(I.value, (self.kv_heads, self.cap[which]), "<i4", 4)[:, :kept.value]
        return St, It, m.value

    def profile(self, enable: bool):
        rc = load().citrus_profile(self._h, 1 if enable else 0)
        if rc != 0:
            raise CitrusError(rc, "citrus_profile")

    def profile_read(self):
        """{kernel name: (total ms, launches)} since the last read."""
        ms = (C.c_double * len(KERNEL_NAMES))()
        cnt = (C.c_longlong * len(KERNEL_NAMES))()
        rc = load().citrus_profile_read(self._h, ms, cnt)
        if rc != 0:
            raise CitrusError(rc, "citrus_profile_read")
        return {n: (ms[i], cnt[i]) for i, n in enumerate(KERNEL_NAMES)}

    def reset(self):
        rc = load().citrus_reset(self._h)
        if rc != 0:
            raise CitrusError(rc, "citrus_reset")

    def poll_status(self) -> int:
        return load().citrus_poll_status(self._h)

    def set_inputs_ready(self, ready: bool):
        """Promise (or withdraw the promise) that every call's inputs are complete before its first kernel can run."""
        rc = load().citrus_set_inputs_ready(self._h, 1 if ready else 0)
        if rc != 0:
            raise CitrusError(rc, "citrus_set_inputs_ready")

    def set_attention_beside(self, max_ctas: int):
        """Steps of at most max_ctas attention items run a1 on a side stream beside the scoring chain (0 = off; see citrus.h)."""
        rc = load().citrus_set_attention_beside(self._h, int(max_ctas))
        if rc != 0:
            raise CitrusError(rc, "citrus_set_attention_beside")

    def debug_expire_wait(self, limit_ns: int = 1_000_000, stream=None):
        """Test aid: let one bounded device wait run out (see citrus.h)."""
        rc = load().citrus_debug_expire_wait(self._h, limit_ns, _stream_ptr(stream))
        if rc != 0:
            raise CitrusError(rc, "citrus_debug_expire_wait")

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value is not None:
            load().citrus_destroy(self._h)
        self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
