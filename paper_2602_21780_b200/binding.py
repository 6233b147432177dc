"""ctypes binding of the xsv C-ABI library (include/xsv.h): argument
marshalling only.  Device tensors are passed as raw pointers; every step of
the path runs in the library's CUDA kernels.  Loading fails loudly when the
shared library has not been built (there is no fallback of any kind)."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libxsv.so")

XSV_OK = 0
F16, BF16 = 0, 1
ATTN_AUTO, ATTN_MMA, ATTN_TC5 = 0, 1, 2
PHASES = ("attn", "score", "select", "quant")

# every symbol include/xsv.h declares: name -> (restype, argtypes)
_vp, _i, _ll = C.c_void_p, C.c_int, C.c_longlong
SYMBOLS = {
    "xsv_cache_create": (_i, [C.POINTER(_vp), _i, _i, _i, _ll, _i]),
    "xsv_cache_set_options": (_i, [_vp, _i, _i, _i, _i, _ll]),
    "xsv_cache_set_attn_impl": (_i, [_vp, _i]),
    "xsv_step": (_i, [_vp, _i, _vp, _vp, _vp, _i, _i, _vp, _vp]),
    "xsv_step_batch": (_i, [_vp, _i, _i, _vp, _vp, _vp, _vp, _i, _vp, _vp]),
    "xsv_cache_append": (_i, [_vp, _i, _vp, _vp, _i, _i, _vp]),
    "xsv_step_host": (_i, [_vp, _i, _vp, _vp, _vp, _i, _i, _vp, _vp]),
    "xsv_cache_set_host_pipelining": (_i, [_vp, _i]),
    "xsv_cache_host_flush": (_i, [_vp, _vp]),
    "xsv_importance_scores": (_i, [_vp, _vp, _i, _i, _ll, _i, _i, _i, _vp, _vp]),
    "xsv_importance_scores_static": (_i, [_vp, _vp, _i, _i, _ll, _i, _i, _i, _vp, _vp]),
    "xsv_cache_bytes": (C.c_size_t, [_vp]),
    "xsv_cache_layer_kv_bytes": (C.c_size_t, [_vp, _i]),
    "xsv_cache_destroy": (None, [_vp]),
    "xsv_cache_len": (_ll, [_vp, _i]),
    "xsv_cache_frames": (_ll, [_vp, _i]),
    "xsv_cache_export_layer": (_i, [_vp, _i] + [_vp] * 9 + [_vp]),
    "xsv_cache_set_deferred_join": (_i, [_vp, _i]),
    "xsv_cache_join": (_i, [_vp, _vp]),
    "xsv_quantization_mse": (_i, [_vp, _i, _ll, _i, _i, _i, C.POINTER(C.c_double), _vp]),
    "xsv_cache_import_layer": (_i, [_vp, _i, _ll, _ll, _i, _i] + [_vp] * 9 + [_vp]),
    "xsv_last_scores": (_i, [_vp, _vp, _ll, C.POINTER(_ll), _vp]),
    "xsv_cache_status": (_i, [_vp, _vp]),
    "xsv_cache_status_word": (_i, [_vp, _vp]),
    "xsv_cache_set_profiling": (_i, [_vp, _i]),
    "xsv_cache_profile_read": (_i, [_vp, C.POINTER(C.c_double), C.POINTER(_ll), _i]),
    "xsv_selftest_bounded_wait": (_i, [_vp]),
    "xsv_selftest_device_table": (_i, []),
    "xsv_plan_batch_groups": (_i, [_i, C.POINTER(_i), C.POINTER(_i), _i, _i]),
    "xsv_kernel_launches": (_ll, []),
    "xsv_strerror": (C.c_char_p, [_i]),
    "xsv_last_cuda_error": (C.c_char_p, []),
}

_lib = None


def load():
    """Load libxsv.so (once) and declare the prototypes."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"xsv: {LIB_PATH} is missing -- build it with __graft_entry__.build(); "
                               "there is no fallback path")
        lib = C.CDLL(LIB_PATH)
        for name, (res, args) in SYMBOLS.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def plan_batch_groups(cache_tokens, frame_tokens, heads, multiprocessors=148):
    """Streams per attention launch that step_batch would use for streams of these cache and frame lengths
    (host arithmetic inside the library; needs no GPU)."""
    n = len(cache_tokens)
    a = (C.c_int * n)(*[int(x) for x in cache_tokens])
    f = (C.c_int * n)(*[int(x) for x in frame_tokens])
    return int(load().xsv_plan_batch_groups(n, a, f, int(heads), int(multiprocessors)))


def step_batch(caches, layer, Qs, Ks, Vs, outs, stream=None):
    """One step of several caches in one call (see xsv_step_batch): lists of CUDA tensors, one per cache."""
    n = len(caches)
    lib = load()
    arr = lambda xs: (C.c_void_p * n)(*[x.data_ptr() for x in xs])
    handles = (C.c_void_p * n)(*[c._h.value for c in caches])
    ntok = (C.c_int * n)(*[int(q.shape[1]) for q in Qs])
    _check(lib.xsv_step_batch(handles, n, layer, arr(Qs), arr(Ks), arr(Vs), ntok, _dtype_code(Qs[0]), arr(outs),
                              _stream_ptr(stream)), "xsv_step_batch")


class XsvError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        detail = f": {load().xsv_last_cuda_error().decode()}" if code == 5 else ""
        super().__init__(f"{where}: {load().xsv_strerror(code).decode()}{detail} (status {code})")


def _check(code, where):
    if code != XSV_OK:
        raise XsvError(code, where)


def _dtype_code(t):
    import torch
    if t.dtype == torch.float16:
        return F16
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"xsv: unsupported dtype {t.dtype}")


def _stream_ptr(stream):
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


class Cache:
    """xsv_cache handle.  Methods mirror the C entry points of the same name."""

    def __init__(self, layers, heads, head_dim, budget_tokens, bits):
        self._lib = load()
        self._h = C.c_void_p()
        self.layers, self.heads, self.head_dim, self.bits = layers, heads, head_dim, bits
        _check(self._lib.xsv_cache_create(C.byref(self._h), layers, heads, head_dim, int(budget_tokens), bits),
               "xsv_cache_create")

    def set_options(self, n_special=-1, pool_group=-1, quant_group=-1, max_frame_tokens=0, max_cache_tokens=-1):
        _check(self._lib.xsv_cache_set_options(self._h, n_special, pool_group, quant_group, max_frame_tokens,
                                               int(max_cache_tokens)), "xsv_cache_set_options")

    def append(self, layer, K, V, stream=None):
        """The cache update of a step without its attention (steps that do not prune)."""
        _check(self._lib.xsv_cache_append(self._h, layer, K.data_ptr(), V.data_ptr(), K.shape[1], _dtype_code(K),
                                          _stream_ptr(stream)), "xsv_cache_append")

    def set_attn_impl(self, impl):
        _check(self._lib.xsv_cache_set_attn_impl(self._h, impl), "xsv_cache_set_attn_impl")

    def step(self, layer, Q, K, V, out, stream=None):
        """Q, K, V, out: CUDA tensors [heads, n_tokens, head_dim], fp16 or bf16, contiguous."""
        for t in (Q, K, V, out):
            if not (t.is_cuda and t.is_contiguous()):
                raise ValueError("xsv.step needs contiguous CUDA tensors")
        _check(self._lib.xsv_step(self._h, layer, Q.data_ptr(), K.data_ptr(), V.data_ptr(), Q.shape[1],
                                  _dtype_code(Q), out.data_ptr(), _stream_ptr(stream)), "xsv_step")

    def step_raw(self, layer, q_ptr, k_ptr, v_ptr, n_tokens, dtype_code, out_ptr, stream_ptr):
        """Unchecked variant for hot loops: raw integer pointers."""
        return self._lib.xsv_step(self._h, layer, q_ptr, k_ptr, v_ptr, n_tokens, dtype_code, out_ptr, stream_ptr)

    def step_host(self, layer, Q, K, V, out, stream=None):
        """Same step with HOST tensors (pinned for asynchronous copies)."""
        for t in (Q, K, V, out):
            if t.is_cuda or not t.is_contiguous():
                raise ValueError("xsv.step_host needs contiguous host tensors")
        _check(self._lib.xsv_step_host(self._h, layer, Q.data_ptr(), K.data_ptr(), V.data_ptr(), Q.shape[1],
                                       _dtype_code(Q), out.data_ptr(), _stream_ptr(stream)), "xsv_step_host")

    def set_host_pipelining(self, defer_output):
        _check(self._lib.xsv_cache_set_host_pipelining(self._h, int(defer_output)), "xsv_cache_set_host_pipelining")

    def host_flush(self, stream=None):
        _check(self._lib.xsv_cache_host_flush(self._h, _stream_ptr(stream)), "xsv_cache_host_flush")

    def bytes(self):
        return int(self._lib.xsv_cache_bytes(self._h))

    def layer_kv_bytes(self, layer):
        return int(self._lib.xsv_cache_layer_kv_bytes(self._h, layer))

    def len(self, layer):
        return int(self._lib.xsv_cache_len(self._h, layer))

    def frames(self, layer):
        return int(self._lib.xsv_cache_frames(self._h, layer))

    def export_layer(self, layer, stream=None):
        """Logical state of one layer as numpy arrays (see xsv_cache_export_layer)."""
        T, H, d = self.len(layer), self.heads, self.head_dim
        G = 64
        ng = -(-T // G)
        st = dict(T=T, origin=np.zeros(T, np.int64))
        if self.bits == 16:
            st["Kraw"] = np.zeros((H, T, d), np.uint16)
            st["Vraw"] = np.zeros((H, T, d), np.uint16)
            ptrs = [None] * 6 + [st["origin"], st["Kraw"], st["Vraw"]]
        else:
            st.update(Kc=np.zeros((H, T, d), np.uint8), Ks=np.zeros((H, ng, d), np.float32),
                      Kz=np.zeros((H, ng, d), np.float32), Vc=np.zeros((H, T, d), np.uint8),
                      Vs=np.zeros((H, T), np.float32), Vz=np.zeros((H, T), np.float32))
            ptrs = [st["Kc"], st["Ks"], st["Kz"], st["Vc"], st["Vs"], st["Vz"], st["origin"], None, None]
        args = [a.ctypes.data_as(C.c_void_p) if a is not None else None for a in ptrs]
        _check(self._lib.xsv_cache_export_layer(self._h, layer, *args, _stream_ptr(stream)),
               "xsv_cache_export_layer")
        return st

    def set_deferred_join(self, on):
        _check(self._lib.xsv_cache_set_deferred_join(self._h, int(on)), "xsv_cache_set_deferred_join")

    def join(self, stream=None):
        _check(self._lib.xsv_cache_join(self._h, _stream_ptr(stream)), "xsv_cache_join")

    def import_layer(self, layer, st, frames_done, frame_tokens, dtype_code, stream=None):
        """Load a state dict as returned by export_layer (see xsv_cache_import_layer)."""
        def ptr(name):
            a = st.get(name)
            return np.ascontiguousarray(a).ctypes.data_as(C.c_void_p) if a is not None else None
        keep = {k: np.ascontiguousarray(v) for k, v in st.items() if isinstance(v, np.ndarray)}   # alive during the call
        args = [keep[k].ctypes.data_as(C.c_void_p) if k in keep else None
                for k in ("Kc", "Ks", "Kz", "Vc", "Vs", "Vz", "origin", "Kraw", "Vraw")]
        _check(self._lib.xsv_cache_import_layer(self._h, layer, int(st["T"]), int(frames_done), int(frame_tokens),
                                                int(dtype_code), *args, _stream_ptr(stream)), "xsv_cache_import_layer")

    def last_scores(self, stream=None):
        """Importance scores (Eq. 7) of the most recent pruning step; empty if it did not prune."""
        n = C.c_longlong(0)
        self._lib.xsv_last_scores(self._h, None, 0, C.byref(n), _stream_ptr(stream))   # reports the count
        if n.value == 0:
            return np.zeros(0, np.float32)
        buf = np.zeros(n.value, np.float32)
        _check(self._lib.xsv_last_scores(self._h, buf.ctypes.data_as(C.c_void_p), buf.shape[0], C.byref(n),
                                         _stream_ptr(stream)), "xsv_last_scores")
        return buf

    def status(self, stream=None):
        return int(self._lib.xsv_cache_status(self._h, _stream_ptr(stream)))

    def status_word(self, stream=None):
        return int(self._lib.xsv_cache_status_word(self._h, _stream_ptr(stream)))

    def set_profiling(self, on):
        _check(self._lib.xsv_cache_set_profiling(self._h, int(on)), "xsv_cache_set_profiling")

    def profile_read(self, reset=True):
        ms = (C.c_double * 4)()
        ln = (C.c_longlong * 4)()
        _check(self._lib.xsv_cache_profile_read(self._h, ms, ln, int(reset)), "xsv_cache_profile_read")
        return {p: (ms[i], ln[i]) for i, p in enumerate(PHASES)}

    def destroy(self):
        if self._h:
            self._lib.xsv_cache_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def importance_scores(Q, keys, n_special=5, pool_group=16, stream=None):
    """xsv_importance_scores: Q [H, F, 64], keys [H, n_keys, 64] CUDA tensors -> float32 CUDA tensor [n_keys]."""
    import torch
    scores = torch.empty(keys.shape[1], device=keys.device, dtype=torch.float32)
    _check(load().xsv_importance_scores(Q.data_ptr(), keys.data_ptr(), Q.shape[0], Q.shape[1], keys.shape[1],
                                        _dtype_code(Q), n_special, pool_group, scores.data_ptr(),
                                        _stream_ptr(stream)), "xsv_importance_scores")
    return scores


def importance_scores_static(Q, keys, scores, n_special=5, pool_group=16, stream=None):
    """xsv_importance_scores_static: as importance_scores, but the caller passes the output tensor
    (float32 CUDA, [n_keys]) and the library allocates nothing.  Returns the status code."""
    return int(load().xsv_importance_scores_static(Q.data_ptr(), keys.data_ptr(), Q.shape[0], Q.shape[1],
                                                   keys.shape[1], _dtype_code(Q), n_special, pool_group,
                                                   scores.data_ptr(), _stream_ptr(stream)))


def quantization_mse(x, bits, per_channel, stream=None):
    """xsv_quantization_mse: mean squared quantisation error of x [heads, tokens, 64] (fp16/bf16 CUDA tensor)."""
    out = C.c_double(0.0)
    _check(load().xsv_quantization_mse(x.data_ptr(), x.shape[0], x.shape[1], _dtype_code(x), int(bits),
                                       1 if per_channel else 0, C.byref(out), _stream_ptr(stream)),
           "xsv_quantization_mse")
    return out.value


def selftest_bounded_wait(stream=None):
    """xsv_selftest_bounded_wait: returns the status code (6 = the wait timed out and said so, as it should)."""
    return int(load().xsv_selftest_bounded_wait(_stream_ptr(stream)))


def kernel_launches():
    return int(load().xsv_kernel_launches())
