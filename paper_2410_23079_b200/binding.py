"""Thin ctypes binding over libbuzz.so: argument marshalling only.

PyTorch is used to own device memory and streams; every step of the path runs in the library's
kernels. There is no CPU fallback: if the shared library cannot be loaded, importing a symbol or
constructing :class:`Buzz` raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libbuzz.so")
_lib = None

BUZZ_F32, BUZZ_BF16 = 0, 1
BUZZ_FLAG_LOGN = 1
_DTYPES = {torch.float32: BUZZ_F32, torch.bfloat16: BUZZ_BF16}


class BuzzError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {error_string(code)} ({code})")


class _Shape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("layers", "max_batch", "q_heads", "kv_heads", "head_dim", "dtype",
                 "max_prompt_tokens", "flags")]


def exported_symbols() -> list[str]:
    """Every entry point include/buzz.h declares."""
    return ["buzz_workspace_bytes", "buzz_create", "buzz_destroy", "buzz_prefill", "buzz_decode_step",
            "buzz_decode_step_host", "buzz_decode_layers", "buzz_decode_layers_host", "buzz_evict", "buzz_export_state", "buzz_import_state",
            "buzz_export_prefill_scores", "buzz_prefill_static", "buzz_selftest_wait_expiry",
            "buzz_status", "buzz_launch_count", "buzz_set_decode_cluster", "buzz_set_sampling", "buzz_set_fused_evict",
            "buzz_set_policy", "buzz_error_string"]


def load_library(build_if_missing: bool = True):
    """Loads libbuzz.so (building it with nvcc first if it is absent); raises if that fails."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        if not build_if_missing:
            raise OSError(f"{_LIB_PATH} is missing; run python -m paper_2410_23079_b200.build")
        from . import build as _build
        _build.build()
    lib = ctypes.CDLL(_LIB_PATH)
    vp, ci, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    lib.buzz_workspace_bytes.restype = ci
    lib.buzz_workspace_bytes.argtypes = [ctypes.POINTER(_Shape), ci, ctypes.POINTER(sz), ctypes.POINTER(sz)]
    lib.buzz_create.restype = ci
    lib.buzz_create.argtypes = [ctypes.POINTER(vp), ci, ci, ci, ci, ci, ctypes.POINTER(_Shape), vp, sz, vp, sz]
    lib.buzz_destroy.restype = None
    lib.buzz_destroy.argtypes = [vp]
    lib.buzz_prefill.restype = ci
    lib.buzz_prefill.argtypes = [vp, ci, vp, vp, vp, vp, ci, ci, ci, vp, vp]
    lib.buzz_prefill_static.restype = ci
    lib.buzz_prefill_static.argtypes = [vp, ci, vp, vp, vp, vp, ci, ci, ci, vp, vp]
    lib.buzz_decode_step.restype = ci
    lib.buzz_decode_step.argtypes = [vp, ci, vp, vp, vp, vp, vp]
    lib.buzz_decode_step_host.restype = ci
    lib.buzz_decode_step_host.argtypes = [vp, ci, vp, vp, vp, vp, vp]
    lib.buzz_decode_layers.restype = ci
    lib.buzz_decode_layers.argtypes = [vp, ci, ctypes.POINTER(ci)] + [ctypes.POINTER(vp)] * 4 + [vp]
    lib.buzz_decode_layers_host.restype = ci
    lib.buzz_decode_layers_host.argtypes = [vp, ci, ctypes.POINTER(ci), vp, vp, vp]
    lib.buzz_evict.restype = ci
    lib.buzz_evict.argtypes = [vp, ci, vp]
    lib.buzz_export_state.restype = ci
    lib.buzz_export_state.argtypes = [vp, ci, ci, ci] + [ctypes.POINTER(ctypes.c_int32)] * 3 + [vp, vp, vp, vp]
    lib.buzz_import_state.restype = ci
    lib.buzz_import_state.argtypes = [vp, ci, ci, ci, ci, ci, ci, vp, vp, vp, vp]
    lib.buzz_export_prefill_scores.restype = ci
    lib.buzz_export_prefill_scores.argtypes = [vp, ci, ci, vp]
    lib.buzz_selftest_wait_expiry.restype = ci
    lib.buzz_selftest_wait_expiry.argtypes = [vp, ci, vp]
    lib.buzz_status.restype = ci
    lib.buzz_status.argtypes = [vp, vp]
    lib.buzz_launch_count.restype = ctypes.c_int64
    lib.buzz_launch_count.argtypes = [vp]
    lib.buzz_set_sampling.restype = ci
    lib.buzz_set_sampling.argtypes = [vp, ci, ci, ci]
    lib.buzz_set_policy.restype = ci
    lib.buzz_set_policy.argtypes = [vp, ci]
    lib.buzz_set_fused_evict.restype = ci
    lib.buzz_set_fused_evict.argtypes = [vp, ci]
    lib.buzz_set_decode_cluster.restype = ci
    lib.buzz_set_decode_cluster.argtypes = [vp, ci]
    lib.buzz_error_string.restype = ctypes.c_char_p
    lib.buzz_error_string.argtypes = [ci]
    _lib = lib
    return lib


def error_string(code: int) -> str:
    return load_library().buzz_error_string(int(code)).decode()


def _check(rc: int, where: str):
    if rc != 0:
        raise BuzzError(rc, where)


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


class Buzz:
    """One BUZZ cache object (all layers, sequences and KV heads of a model shape).

    Method names mirror the C entry points; tensors are passed by device pointer.
    """

    def __init__(self, *, sink, window, segment, hitters, budget, layers, max_batch, q_heads,
                 kv_heads, head_dim, dtype, max_prompt_tokens, logn=False, device="cuda:0"):
        self._h = None
        self._lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("libbuzz needs a CUDA device; there is no CPU fallback")
        self.device = torch.device(device)
        self.dtype = dtype
        self.budget, self.head_dim = int(budget), int(head_dim)
        self.layers, self.max_batch = int(layers), int(max_batch)
        self.q_heads, self.kv_heads = int(q_heads), int(kv_heads)
        self._shape = _Shape(layers, max_batch, q_heads, kv_heads, head_dim, _DTYPES[dtype],
                             max_prompt_tokens, BUZZ_FLAG_LOGN if logn else 0)
        sb, cb = ctypes.c_size_t(), ctypes.c_size_t()
        _check(self._lib.buzz_workspace_bytes(ctypes.byref(self._shape), budget, ctypes.byref(sb),
                                              ctypes.byref(cb)), "buzz_workspace_bytes")
        self.state_bytes, self.scratch_bytes = sb.value, cb.value
        with torch.cuda.device(self.device):
            self._state = torch.empty(sb.value, dtype=torch.uint8, device=self.device)
            self._scratch = torch.empty(cb.value, dtype=torch.uint8, device=self.device)
            h = ctypes.c_void_p()
            _check(self._lib.buzz_create(ctypes.byref(h), sink, window, segment, hitters, budget,
                                         ctypes.byref(self._shape), self._state.data_ptr(), sb.value,
                                         self._scratch.data_ptr(), cb.value), "buzz_create")
        self._h = h

    def close(self):
        if self._h is not None:
            self._lib.buzz_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- hot path --------------------------------------------------------------------------
    def prefill(self, layer, q, k, v, cu_seqlens, max_seqlen, out, stream=None):
        batch = cu_seqlens.numel() - 1
        _check(self._lib.buzz_prefill(self._h, layer, q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                      cu_seqlens.data_ptr(), batch, q.shape[0], int(max_seqlen),
                                      out.data_ptr(), _stream_ptr(stream)), "buzz_prefill")

    def prefill_static(self, layer, q, k, v, cu_seqlens, max_seqlen, out, stream=None):
        """buzz_prefill_static: prefill whose temporaries live in the library's built-in 4 MiB device
        array, for callers that must not allocate device memory. Same arguments as :meth:`prefill`;
        raises BuzzError(-6) when (q_heads + kv_heads) * tokens exceeds 1,048,576 floats."""
        batch = cu_seqlens.numel() - 1
        _check(self._lib.buzz_prefill_static(self._h, layer, q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                             cu_seqlens.data_ptr(), batch, q.shape[0], int(max_seqlen),
                                             out.data_ptr(), _stream_ptr(stream)), "buzz_prefill_static")

    def decode_step(self, layer, q, k_new, v_new, out, stream=None):
        _check(self._lib.buzz_decode_step(self._h, layer, q.data_ptr(), k_new.data_ptr(),
                                          v_new.data_ptr(), out.data_ptr(), _stream_ptr(stream)),
               "buzz_decode_step")

    def decode_step_host(self, layer, q, k_new, v_new, out, stream=None):
        _check(self._lib.buzz_decode_step_host(self._h, layer, q.data_ptr(), k_new.data_ptr(),
                                               v_new.data_ptr(), out.data_ptr(), _stream_ptr(stream)),
               "buzz_decode_step_host")

    def decode_layers(self, layers, q, k_new, v_new, out, stream=None):
        """buzz_decode_layers: one decode step of several distinct layers whose inputs (lists of device
        tensors, one per layer) are all complete; the launches overlap on the GPU."""
        n = len(layers)
        ci, vp = ctypes.c_int, ctypes.c_void_p
        arr = lambda ts: (vp * n)(*[t.data_ptr() for t in ts])
        _check(self._lib.buzz_decode_layers(self._h, n, (ci * n)(*layers), arr(q), arr(k_new), arr(v_new),
                                            arr(out), _stream_ptr(stream)), "buzz_decode_layers")

    def decode_layers_host(self, layers, in_host, out_host, stream=None):
        """buzz_decode_layers_host: `in_host` holds, per listed layer, q | k_new | v_new packed back to
        back; `out_host` receives the outputs packed in the same order."""
        n = len(layers)
        _check(self._lib.buzz_decode_layers_host(self._h, n, (ctypes.c_int * n)(*layers), in_host.data_ptr(),
                                                 out_host.data_ptr(), _stream_ptr(stream)),
               "buzz_decode_layers_host")

    def evict(self, layer=-1, stream=None):
        _check(self._lib.buzz_evict(self._h, layer, _stream_ptr(stream)), "buzz_evict")

    # -- inspection ------------------------------------------------------------------------
    def status(self, stream=None) -> int:
        return self._lib.buzz_status(self._h, _stream_ptr(stream))

    def selftest_wait_expiry(self, polls=1024, stream=None):
        """buzz_selftest_wait_expiry: lets one bounded on-device wait run out; status() then reports -4 once."""
        _check(self._lib.buzz_selftest_wait_expiry(self._h, int(polls), _stream_ptr(stream)), "buzz_selftest_wait_expiry")

    def launch_count(self) -> int:
        return self._lib.buzz_launch_count(self._h)

    def set_sampling(self, interval_new: bool, new_stride: int, old_stride: int):
        _check(self._lib.buzz_set_sampling(self._h, int(bool(interval_new)), new_stride, old_stride), "buzz_set_sampling")

    def set_policy(self, global_topk: bool):
        """buzz_set_policy: False = BUZZ's sampling module, True = global top-k of the accumulated scores."""
        _check(self._lib.buzz_set_policy(self._h, 1 if global_topk else 0), "buzz_set_policy")

    def set_fused_evict(self, on: bool):
        """buzz_set_fused_evict: decode steps run the eviction of a cache they fill in their own tail."""
        _check(self._lib.buzz_set_fused_evict(self._h, int(bool(on))), "buzz_set_fused_evict")

    def set_decode_cluster(self, cluster_size: int):
        _check(self._lib.buzz_set_decode_cluster(self._h, cluster_size), "buzz_set_decode_cluster")

    def export_state(self, layer, seq, kv_head):
        """Returns dict(n, n_old, total_len, pos, score, k, v) of one instance as host tensors."""
        n, n_old, tot = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
        pos = torch.empty(self.budget, dtype=torch.int32)
        score = torch.empty(self.budget, dtype=torch.float32)
        k = torch.empty(self.budget, self.head_dim, dtype=self.dtype)
        v = torch.empty(self.budget, self.head_dim, dtype=self.dtype)
        _check(self._lib.buzz_export_state(self._h, layer, seq, kv_head, ctypes.byref(n),
                                           ctypes.byref(n_old), ctypes.byref(tot), pos.data_ptr(),
                                           score.data_ptr(), k.data_ptr(), v.data_ptr()),
               "buzz_export_state")
        m = n.value
        return dict(n=m, n_old=n_old.value, total_len=tot.value, pos=pos[:m], score=score[:m],
                    k=k[:m], v=v[:m])

    def import_state(self, layer, seq, kv_head, n_old, total_len, pos, score, k, v):
        """Loads one instance's cache from host tensors (pos int32, score fp32, k/v of the cache dtype)."""
        pos = pos.to(torch.int32).contiguous().cpu()
        score = score.to(torch.float32).contiguous().cpu()
        k = k.to(self.dtype).contiguous().cpu()
        v = v.to(self.dtype).contiguous().cpu()
        _check(self._lib.buzz_import_state(self._h, layer, seq, kv_head, pos.numel(), int(n_old),
                                           int(total_len), pos.data_ptr(), score.data_ptr(),
                                           k.data_ptr(), v.data_ptr()), "buzz_import_state")

    def export_prefill_scores(self, kv_head, total_tokens):
        out = torch.empty(total_tokens, dtype=torch.float32)
        _check(self._lib.buzz_export_prefill_scores(self._h, kv_head, total_tokens, out.data_ptr()),
               "buzz_export_prefill_scores")
        return out
