"""ctypes binding of libearlytom.so: the same names as include/earlytom.h, argument marshalling only.

Every step of the path runs in the library's CUDA kernels; torch is used for device memory and
streams.  Importing this module fails loudly when the shared library is missing (there is no
fallback of any kind).
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

# EARLYTOM_LIB selects another build of the same library (the checked build libearlytom_debug.so)
_LIB_PATH = os.environ.get("EARLYTOM_LIB") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "lib", "libearlytom.so")

ET_F32, ET_BF16 = 0, 1
ET_MAX_MERGE_LAYERS = 8
STATUS_NAMES = ["ET_OK", "ET_ERR_INVALID_ARG", "ET_ERR_SHAPE", "ET_ERR_CAPACITY", "ET_ERR_OOM", "ET_ERR_CUDA",
                "ET_ERR_TIMEOUT", "ET_ERR_WEIGHTS"]
EXPORTS = ["et_encoder_create", "et_encode_video", "et_encode_batch", "et_encode_batch_host", "et_encode_batch_host_submit",
           "et_encode_batch_host_collect", "et_destroy",
           "et_status_string", "et_last_error", "et_kernel_launch_count", "et_profile_enable", "et_profile_read",
           "et_selftest_bounded_wait", "et_debug_build", "et_debug_status",
           "et_frame_similarity_static", "et_frame_similarity", "et_merge_plan",
           "et_merge_frames", "et_select_tokens", "et_gather_tokens", "et_linear_bf16", "et_attention", "et_attention_windowed",
           "et_attention_scores", "et_layernorm",
           # include/earlytom_llm.h
           "et_llm_create", "et_llm_prefill", "et_llm_destroy", "et_llm_last_error", "et_llm_profile_enable",
           "et_llm_profile_read", "et_rmsnorm", "et_rope", "et_swiglu", "et_attention_causal"]


class EarlyTomError(RuntimeError):
    def __init__(self, status: int, message: str = ""):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{name}: {message}" if message else name)


class et_config(C.Structure):
    _fields_ = [("image_size", C.c_int), ("patch_size", C.c_int), ("num_layers", C.c_int), ("hidden", C.c_int),
                ("heads", C.c_int), ("mlp_dim", C.c_int), ("ln_eps", C.c_float), ("gelu_tanh", C.c_int),
                ("post_layernorm", C.c_int), ("dtype", C.c_int), ("max_frames_total", C.c_int), ("max_videos", C.c_int),
                ("arch", C.c_int), ("temporal_patch", C.c_int), ("window", C.c_int), ("full_attn_mask", C.c_ulonglong),
                ("rope_theta", C.c_float)]


class et_weights(C.Structure):
    _fields_ = [("data", C.POINTER(C.c_float)), ("count", C.c_size_t)]


_U8P = C.POINTER(C.c_ubyte)
_I32P = C.POINTER(C.c_int)
_F32P = C.POINTER(C.c_float)


class et_forced_plan(C.Structure):
    _fields_ = [("n_in", C.c_int * ET_MAX_MERGE_LAYERS), ("seg_start", _U8P * ET_MAX_MERGE_LAYERS),
                ("merge_next", _U8P * ET_MAX_MERGE_LAYERS), ("n_final", C.c_int), ("keep", _U8P)]


class et_params(C.Structure):
    _fields_ = [("num_merge_layers", C.c_int), ("merge_layers", C.c_int * ET_MAX_MERGE_LAYERS),
                ("ema_alpha", C.c_double), ("tau_seg", C.c_double), ("tau_merge", C.c_double),
                ("weighted_merge", C.c_int), ("selection", C.c_int), ("retain_mode", C.c_int), ("retain", C.c_double),
                ("forced_plan", C.POINTER(et_forced_plan)), ("want_trace", C.c_int), ("sample_seed", C.c_ulonglong),
                ("window_mode", C.c_int)]


class et_trace(C.Structure):
    _fields_ = [("num_merge_layers", C.c_int), ("n_in", C.c_int * ET_MAX_MERGE_LAYERS),
                ("n_out", C.c_int * ET_MAX_MERGE_LAYERS), ("sim", _F32P * ET_MAX_MERGE_LAYERS),
                ("ema", _F32P * ET_MAX_MERGE_LAYERS), ("seg_start", _U8P * ET_MAX_MERGE_LAYERS),
                ("merge_next", _U8P * ET_MAX_MERGE_LAYERS), ("scores", _F32P), ("keep", _U8P),
                ("video_k", _I32P), ("video_w", _I32P)]


class et_result(C.Structure):
    _fields_ = [("n_videos", C.c_int), ("n_frames_in", C.c_int), ("n_frames_out", C.c_int), ("n_tokens", C.c_int),
                ("hidden", C.c_int), ("tokens_per_frame", C.c_int), ("tokens", C.c_void_p),
                ("video_frame_offsets", C.c_void_p), ("frame_offsets", C.c_void_p), ("frame_src_lo", C.c_void_p),
                ("frame_src_hi", C.c_void_p), ("frame_dynamic", C.c_void_p), ("token_pos", C.c_void_p),
                ("trace", C.POINTER(et_trace)), ("frames_per_block", C.c_int * 64)]


class et_host_buffers(C.Structure):
    _fields_ = [("tokens", C.c_void_p), ("token_pos", C.c_void_p), ("frame_offsets", C.c_void_p),
                ("frame_src_lo", C.c_void_p), ("frame_src_hi", C.c_void_p), ("frame_dynamic", C.c_void_p),
                ("video_frame_offsets", C.c_void_p), ("capacity_tokens", C.c_size_t), ("capacity_frames", C.c_size_t)]


ET_PROF_CATS = 10
PROF_NAMES = ["im2col", "gemm", "attention", "layernorm", "similarity", "plan", "merge", "scores", "select", "gather"]


class et_profile(C.Structure):
    _fields_ = [("ms", C.c_double * ET_PROF_CATS), ("work", C.c_double * ET_PROF_CATS),
                ("launches", C.c_ulonglong * ET_PROF_CATS), ("calls", C.c_int)]


class et_llm_config(C.Structure):
    _fields_ = [("vision_hidden", C.c_int), ("hidden", C.c_int), ("num_layers", C.c_int), ("heads", C.c_int),
                ("kv_heads", C.c_int), ("head_dim", C.c_int), ("mlp_dim", C.c_int), ("vocab", C.c_int),
                ("rms_eps", C.c_float), ("rope_theta", C.c_float), ("gelu_tanh", C.c_int), ("max_tokens", C.c_int),
                ("keep_kv_cache", C.c_int)]


class et_llm_weights(C.Structure):
    _fields_ = [("data", C.c_void_p), ("count", C.c_size_t), ("on_device", C.c_int)]


class et_llm_result(C.Structure):
    _fields_ = [("n_tokens", C.c_int), ("first_token", C.c_int), ("logits", C.c_void_p), ("hidden", C.c_void_p),
                ("kv_cache", C.c_void_p), ("kv_cache_rows", C.c_int)]


ET_LLM_CATS = 8
LLM_PROF_NAMES = ["embed", "norm", "gemm", "rope", "attention", "swiglu", "head"]


class et_llm_profile(C.Structure):
    _fields_ = [("ms", C.c_double * ET_LLM_CATS), ("launches", C.c_ulonglong * ET_LLM_CATS), ("calls", C.c_int)]


def load_library(path: str = _LIB_PATH) -> C.CDLL:
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with `python -m paper_2605_30010_b200.build` "
                          f"(there is no fallback path)")
    lib = C.CDLL(path)
    for name in EXPORTS:
        getattr(lib, name)      # AttributeError if a declared symbol is not exported
    vp, i, d, f = C.c_void_p, C.c_int, C.c_double, C.c_float
    lib.et_encoder_create.argtypes = [C.POINTER(et_config), C.POINTER(et_weights), C.POINTER(vp)]
    lib.et_encode_video.argtypes = [vp, vp, i, C.POINTER(et_params), vp, C.POINTER(et_result)]
    lib.et_encode_batch.argtypes = [vp, vp, _I32P, i, C.POINTER(et_params), vp, C.POINTER(et_result)]
    lib.et_encode_batch_host.argtypes = [vp, vp, _I32P, i, C.POINTER(et_params), vp, C.POINTER(et_host_buffers),
                                         C.POINTER(et_result)]
    lib.et_encode_batch_host_submit.argtypes = [vp, vp, _I32P, i, C.POINTER(et_params), vp, C.POINTER(et_host_buffers),
                                                C.POINTER(C.c_ulonglong)]
    lib.et_encode_batch_host_collect.argtypes = [vp, C.c_ulonglong, C.POINTER(et_result)]
    lib.et_destroy.argtypes = [vp]
    lib.et_destroy.restype = None
    lib.et_status_string.argtypes = [i]
    lib.et_status_string.restype = C.c_char_p
    lib.et_last_error.argtypes = [vp]
    lib.et_last_error.restype = C.c_char_p
    lib.et_kernel_launch_count.argtypes = []
    lib.et_kernel_launch_count.restype = C.c_ulonglong
    lib.et_selftest_bounded_wait.argtypes = [C.c_ulonglong, i, vp]
    lib.et_debug_build.argtypes = []
    lib.et_debug_status.argtypes = []
    lib.et_profile_enable.argtypes = [vp, i]
    lib.et_profile_read.argtypes = [vp, C.POINTER(et_profile)]
    lib.et_frame_similarity.argtypes = [vp, i, i, i, vp, vp, vp]
    lib.et_frame_similarity_static.argtypes = [vp, i, i, i, vp, vp]
    lib.et_merge_plan.argtypes = [vp, vp, i, i, d, d, d, i, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.et_merge_frames.argtypes = [vp, vp, i, i, vp, vp, vp, vp, vp, vp]
    lib.et_select_tokens.argtypes = [vp, vp, vp, vp, i, i, i, vp, vp, vp]
    lib.et_gather_tokens.argtypes = [vp, vp, i, i, i, vp, vp, f, vp, C.c_size_t, vp, vp, _I32P, vp]
    lib.et_linear_bf16.argtypes = [vp, vp, vp, vp, i, i, i, i, i, vp, i, vp, vp]
    lib.et_attention.argtypes = [vp, vp, vp, i, i, i, i, i, vp]
    lib.et_attention_windowed.argtypes = [vp, vp, vp, i, i, i, i, i, i, vp]
    lib.et_attention_scores.argtypes = [vp, vp, vp, vp, i, i, i, i, i, vp]
    lib.et_layernorm.argtypes = [vp, vp, vp, f, vp, i, i, i, vp]
    lib.et_llm_create.argtypes = [C.POINTER(et_llm_config), C.POINTER(et_llm_weights), C.POINTER(vp)]
    lib.et_llm_prefill.argtypes = [vp, _I32P, i, vp, i, _I32P, i, vp, C.POINTER(et_llm_result)]
    lib.et_llm_destroy.argtypes = [vp]
    lib.et_llm_destroy.restype = None
    lib.et_llm_last_error.argtypes = [vp]
    lib.et_llm_last_error.restype = C.c_char_p
    lib.et_llm_profile_enable.argtypes = [vp, i]
    lib.et_llm_profile_read.argtypes = [vp, C.POINTER(et_llm_profile)]
    lib.et_rmsnorm.argtypes = [vp, vp, f, vp, i, i, vp]
    lib.et_rope.argtypes = [vp, i, i, i, i, i, f, vp]
    lib.et_swiglu.argtypes = [vp, vp, i, i, vp]
    lib.et_attention_causal.argtypes = [vp, vp, i, i, i, i, i, vp, vp]
    for name in EXPORTS:
        fn = getattr(lib, name)
        if name.startswith("et_") and name not in ("et_destroy", "et_status_string", "et_last_error",
                                                  "et_kernel_launch_count", "et_llm_destroy", "et_llm_last_error"):
            fn.restype = C.c_int
    return lib


_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = load_library()
    return _lib


def _check(status: int, enc=None):
    if status != 0:
        msg = lib().et_last_error(enc).decode() if enc else ""
        raise EarlyTomError(status, msg)


def _stream_ptr(stream) -> Optional[int]:
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _ptr(t) -> C.c_void_p:
    return C.c_void_p(t.data_ptr() if t is not None else 0)


class _DevView:
    """Zero-copy view of encoder-owned device memory for torch.as_tensor."""

    def __init__(self, ptr: int, shape, typestr: str):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": typestr, "data": (int(ptr), False),
                                         "version": 3, "strides": None}


def _dev_tensor(ptr, shape, typestr):
    import torch
    n = int(np.prod(shape))
    if n == 0 or not ptr:
        dt = {"<f4": torch.float32, "<i4": torch.int32, "|u1": torch.uint8}[typestr]
        return torch.empty(tuple(shape), dtype=dt, device="cuda")
    return torch.as_tensor(_DevView(ptr, shape, typestr), device="cuda").clone()


# --------------------------------------------------------------------------------------------
# Python-side views of parameters and results
# --------------------------------------------------------------------------------------------

@dataclass
class ForcedPlan:
    seg_start: List[np.ndarray]          # per merge layer, bool/uint8 [n_in]
    merge_next: List[np.ndarray]
    keep: Optional[np.ndarray] = None    # [N, L] bool/uint8


@dataclass
class Trace:
    n_in: List[int]
    n_out: List[int]
    sim: List[np.ndarray]
    ema: List[np.ndarray]
    seg_start: List[np.ndarray]
    merge_next: List[np.ndarray]
    scores: np.ndarray
    keep: np.ndarray
    video_k: np.ndarray
    video_w: np.ndarray


@dataclass
class Result:
    n_videos: int
    n_frames_in: int
    n_frames_out: int
    n_tokens: int
    tokens: object                 # torch [n_tokens, D] float32 (cuda) or numpy for the host entry point
    video_frame_offsets: object
    frame_offsets: object
    frame_src_lo: object
    frame_src_hi: object
    frame_dynamic: object
    token_pos: object
    frames_per_block: List[int]
    trace: Optional[Trace] = None


def make_params(p, forced: Optional[ForcedPlan] = None, want_trace: bool = False):
    """p: any object with the fields of synthetic.MergePlan-like params.  Returns (et_params, keepalive)."""
    q = et_params()
    ml = list(p.merge_layers)
    q.num_merge_layers = len(ml)
    for i, l in enumerate(ml):
        q.merge_layers[i] = int(l)
    q.ema_alpha, q.tau_seg, q.tau_merge = float(p.ema_alpha), float(p.tau_seg), float(p.tau_merge)
    q.weighted_merge, q.selection, q.retain_mode = int(p.weighted_merge), int(p.selection), int(p.retain_mode)
    q.retain = float(p.retain)
    q.want_trace = 1 if want_trace else 0
    q.sample_seed = int(getattr(p, "sample_seed", 0))
    q.window_mode = int(getattr(p, "window_mode", 0))
    keep = []
    if forced is not None:
        fp = et_forced_plan()
        for i in range(len(ml)):
            s = np.ascontiguousarray(np.asarray(forced.seg_start[i]).astype(np.uint8))
            m = np.ascontiguousarray(np.asarray(forced.merge_next[i]).astype(np.uint8))
            assert s.shape == m.shape
            keep += [s, m]
            fp.n_in[i] = s.shape[0]
            fp.seg_start[i] = s.ctypes.data_as(_U8P)
            fp.merge_next[i] = m.ctypes.data_as(_U8P)
        if forced.keep is not None:
            k = np.ascontiguousarray(np.asarray(forced.keep).astype(np.uint8))
            keep.append(k)
            fp.n_final = k.shape[0]
            fp.keep = k.ctypes.data_as(_U8P)
        keep.append(fp)
        q.forced_plan = C.pointer(fp)
    return q, keep


def _np_from(ptr, n, dtype):
    if n == 0:
        return np.zeros(0, dtype=dtype)
    return np.ctypeslib.as_array(ptr, shape=(n,)).astype(dtype, copy=True)


def _read_trace(r: et_result) -> Trace:
    t = r.trace.contents
    L = r.tokens_per_frame
    nm = t.num_merge_layers
    return Trace(
        n_in=[t.n_in[i] for i in range(nm)], n_out=[t.n_out[i] for i in range(nm)],
        sim=[_np_from(t.sim[i], t.n_in[i], np.float32) for i in range(nm)],
        ema=[_np_from(t.ema[i], t.n_in[i], np.float32) for i in range(nm)],
        seg_start=[_np_from(t.seg_start[i], t.n_in[i], np.uint8).astype(bool) for i in range(nm)],
        merge_next=[_np_from(t.merge_next[i], t.n_in[i], np.uint8).astype(bool) for i in range(nm)],
        scores=_np_from(t.scores, r.n_frames_out * L, np.float32).reshape(r.n_frames_out, L),
        keep=_np_from(t.keep, r.n_frames_out * L, np.uint8).reshape(r.n_frames_out, L).astype(bool),
        video_k=_np_from(t.video_k, r.n_videos, np.int32), video_w=_np_from(t.video_w, r.n_videos, np.int32))


def _result_from_device(r: et_result, num_layers: int) -> Result:
    N, nt, D, V = r.n_frames_out, r.n_tokens, r.hidden, r.n_videos
    return Result(
        n_videos=V, n_frames_in=r.n_frames_in, n_frames_out=N, n_tokens=nt,
        tokens=_dev_tensor(r.tokens, (nt, D), "<f4"),
        video_frame_offsets=_dev_tensor(r.video_frame_offsets, (V + 1,), "<i4"),
        frame_offsets=_dev_tensor(r.frame_offsets, (N + 1,), "<i4"),
        frame_src_lo=_dev_tensor(r.frame_src_lo, (N,), "<i4"), frame_src_hi=_dev_tensor(r.frame_src_hi, (N,), "<i4"),
        frame_dynamic=_dev_tensor(r.frame_dynamic, (N,), "|u1"), token_pos=_dev_tensor(r.token_pos, (nt,), "<i4"),
        frames_per_block=[r.frames_per_block[i] for i in range(num_layers)],
        trace=_read_trace(r) if r.trace else None)


# --------------------------------------------------------------------------------------------
# The calls of the header
# --------------------------------------------------------------------------------------------

class Encoder:
    """Owns an et_encoder*.  `shape` is any object with the architecture fields of et_config."""

    def __init__(self, shape, weights: np.ndarray, dtype: int, max_frames_total: int, max_videos: int = 1):
        cfg = et_config(shape.image_size, shape.patch_size, shape.num_layers, shape.hidden, shape.heads, shape.mlp_dim,
                        float(shape.ln_eps), int(shape.gelu_tanh), int(shape.post_layernorm), int(dtype),
                        int(max_frames_total), int(max_videos), int(getattr(shape, "arch", 0)),
                        int(getattr(shape, "temporal_patch", 1)), int(getattr(shape, "window", 0)),
                        int(getattr(shape, "full_attn_mask", 0)), float(getattr(shape, "rope_theta", 0.0)))
        self.handle = et_encoder_create(cfg, weights)
        self.num_layers = shape.num_layers
        self.shape = shape

    def close(self):
        if getattr(self, "handle", None):
            et_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def encode_video(self, frames, params, forced=None, want_trace=False, stream=None) -> Result:
        return et_encode_video(self, frames, params, forced, want_trace, stream)

    def encode_batch(self, frames, video_offsets, params, forced=None, want_trace=False, stream=None) -> Result:
        return et_encode_batch(self, frames, video_offsets, params, forced, want_trace, stream)


def et_encoder_create(cfg: et_config, weights: np.ndarray) -> C.c_void_p:
    w = np.ascontiguousarray(weights, dtype=np.float32)
    wb = et_weights(w.ctypes.data_as(_F32P), w.size)
    h = C.c_void_p()
    _check(lib().et_encoder_create(C.byref(cfg), C.byref(wb), C.byref(h)))
    return h


def et_destroy(handle) -> None:
    lib().et_destroy(handle)


def et_encode_video(enc: Encoder, frames, params, forced=None, want_trace=False, stream=None) -> Result:
    assert frames.is_cuda and frames.is_contiguous() and frames.dtype.is_floating_point and frames.element_size() == 4
    q, keep = make_params(params, forced, want_trace)
    r = et_result()
    _check(lib().et_encode_video(enc.handle, _ptr(frames), int(frames.shape[0]), C.byref(q), _stream_ptr(stream),
                                 C.byref(r)), enc.handle)
    return _result_from_device(r, enc.num_layers)


def et_encode_batch(enc: Encoder, frames, video_offsets: Sequence[int], params, forced=None, want_trace=False,
                    stream=None) -> Result:
    assert frames.is_cuda and frames.is_contiguous() and frames.element_size() == 4
    offs = np.ascontiguousarray(np.asarray(video_offsets, dtype=np.int32))
    q, keep = make_params(params, forced, want_trace)
    r = et_result()
    _check(lib().et_encode_batch(enc.handle, _ptr(frames), offs.ctypes.data_as(_I32P), len(offs) - 1, C.byref(q),
                                 _stream_ptr(stream), C.byref(r)), enc.handle)
    return _result_from_device(r, enc.num_layers)


class HostBuffers:
    """Pinned host destination buffers for et_encode_batch_host."""

    def __init__(self, capacity_tokens: int, capacity_frames: int, hidden: int, max_videos: int = 1):
        import torch
        pin = dict(pin_memory=True)
        self.tokens = torch.empty((capacity_tokens, hidden), dtype=torch.float32, **pin)
        self.token_pos = torch.empty(capacity_tokens, dtype=torch.int32, **pin)
        self.frame_offsets = torch.empty(capacity_frames + 1, dtype=torch.int32, **pin)
        self.frame_src_lo = torch.empty(capacity_frames, dtype=torch.int32, **pin)
        self.frame_src_hi = torch.empty(capacity_frames, dtype=torch.int32, **pin)
        self.frame_dynamic = torch.empty(capacity_frames, dtype=torch.uint8, **pin)
        self.video_frame_offsets = torch.empty(max_videos + 1, dtype=torch.int32, **pin)
        self.c = et_host_buffers(self.tokens.data_ptr(), self.token_pos.data_ptr(), self.frame_offsets.data_ptr(),
                                 self.frame_src_lo.data_ptr(), self.frame_src_hi.data_ptr(),
                                 self.frame_dynamic.data_ptr(), self.video_frame_offsets.data_ptr(),
                                 capacity_tokens, capacity_frames)


def _host_result(enc: Encoder, r, dst: HostBuffers) -> Result:
    N, nt, V = r.n_frames_out, r.n_tokens, r.n_videos
    return Result(n_videos=V, n_frames_in=r.n_frames_in, n_frames_out=N, n_tokens=nt, tokens=dst.tokens[:nt],
                  video_frame_offsets=dst.video_frame_offsets[:V + 1], frame_offsets=dst.frame_offsets[:N + 1],
                  frame_src_lo=dst.frame_src_lo[:N], frame_src_hi=dst.frame_src_hi[:N],
                  frame_dynamic=dst.frame_dynamic[:N], token_pos=dst.token_pos[:nt],
                  frames_per_block=[r.frames_per_block[i] for i in range(enc.num_layers)])


def et_encode_batch_host(enc: Encoder, frames_host, video_offsets: Sequence[int], params, dst: HostBuffers,
                         stream=None) -> Result:
    """frames_host: CPU torch tensor (pinned for asynchronous copies) [T,3,H,W] float32."""
    assert not frames_host.is_cuda and frames_host.is_contiguous()
    offs = np.ascontiguousarray(np.asarray(video_offsets, dtype=np.int32))
    q, keep = make_params(params)
    r = et_result()
    _check(lib().et_encode_batch_host(enc.handle, _ptr(frames_host), offs.ctypes.data_as(_I32P), len(offs) - 1,
                                      C.byref(q), _stream_ptr(stream), C.byref(dst.c), C.byref(r)), enc.handle)
    return _host_result(enc, r, dst)


class HostCall:
    """A submitted host call: the ticket plus references that keep its host buffers alive until it is collected."""

    def __init__(self, ticket: int, frames_host, dst: HostBuffers):
        self.ticket, self.frames_host, self.dst = ticket, frames_host, dst


def et_encode_batch_host_submit(enc: Encoder, frames_host, video_offsets: Sequence[int], params, dst: HostBuffers,
                                stream=None) -> HostCall:
    """Enqueues upload and encode and returns at once; at most two calls in flight, collected in order."""
    assert not frames_host.is_cuda and frames_host.is_contiguous()
    offs = np.ascontiguousarray(np.asarray(video_offsets, dtype=np.int32))
    q, keep = make_params(params)
    ticket = C.c_ulonglong(0)
    _check(lib().et_encode_batch_host_submit(enc.handle, _ptr(frames_host), offs.ctypes.data_as(_I32P), len(offs) - 1,
                                             C.byref(q), _stream_ptr(stream), C.byref(dst.c), C.byref(ticket)),
           enc.handle)
    return HostCall(int(ticket.value), frames_host, dst)


def et_encode_batch_host_collect(enc: Encoder, call: HostCall) -> Result:
    r = et_result()
    _check(lib().et_encode_batch_host_collect(enc.handle, C.c_ulonglong(call.ticket), C.byref(r)), enc.handle)
    return _host_result(enc, r, call.dst)


def et_kernel_launch_count() -> int:
    return int(lib().et_kernel_launch_count())


def et_selftest_bounded_wait(limit_ns: int, arrive: bool, stream=None) -> None:
    """Raises EarlyTomError(ET_ERR_TIMEOUT) when the wait runs out (arrive = False)."""
    _check(lib().et_selftest_bounded_wait(C.c_ulonglong(int(limit_ns)), 1 if arrive else 0, _stream_ptr(stream)))


def et_debug_build() -> bool:
    return bool(lib().et_debug_build())


def et_debug_status() -> int:
    return int(lib().et_debug_status())


def et_profile_enable(enc: Encoder, on: bool) -> None:
    _check(lib().et_profile_enable(enc.handle, 1 if on else 0))


def et_profile_read(enc: Encoder) -> dict:
    """{category: {"ms", "work", "launches"}} accumulated since et_profile_enable(enc, True), plus "calls"."""
    p = et_profile()
    _check(lib().et_profile_read(enc.handle, C.byref(p)))
    out = {PROF_NAMES[i]: {"ms": p.ms[i], "work": p.work[i], "launches": int(p.launches[i])} for i in range(ET_PROF_CATS)}
    out["calls"] = p.calls
    return out


# ---- single steps (torch CUDA tensors in, torch CUDA tensors out) ---------------------------

def et_frame_similarity(x, stream=None):
    import torch
    n, L, D = x.shape
    cosb = torch.empty((max(n - 1, 1), L), dtype=torch.float32, device=x.device)
    sim = torch.zeros(max(n - 1, 1), dtype=torch.float32, device=x.device)
    _check(lib().et_frame_similarity(_ptr(x), n, L, D, _ptr(cosb), _ptr(sim), _stream_ptr(stream)))
    return sim[:n - 1], cosb[:n - 1]


def et_frame_similarity_static(x, sim_out=None, stream=None):
    """Adjacent-frame similarity without any allocation inside the library: the cosines go to the
    library's built-in scratch array.  `sim_out` (float32 cuda [n-1]) is the caller's output buffer;
    it is created here with torch only when the caller does not bring one."""
    import torch
    n, L, D = x.shape
    if sim_out is None:
        sim_out = torch.zeros(max(n - 1, 1), dtype=torch.float32, device=x.device)
    _check(lib().et_frame_similarity_static(_ptr(x), n, L, D, _ptr(sim_out), _stream_ptr(stream)))
    return sim_out[:n - 1]


def et_merge_plan(sim, video_offsets, alpha, tau_seg, tau_merge, weighted=1, stream=None):
    """sim: float32 cuda [n] (entry t = frames t, t+1).  Returns a dict of cuda tensors."""
    import torch
    n = int(sim.shape[0])
    V = int(video_offsets.shape[0]) - 1
    dev = sim.device
    o = dict(seg_start=torch.zeros(n, dtype=torch.uint8, device=dev), merge_next=torch.zeros(n, dtype=torch.uint8, device=dev),
             ema=torch.zeros(n, dtype=torch.float32, device=dev), n_out=torch.zeros(1, dtype=torch.int32, device=dev),
             src_a=torch.zeros(n, dtype=torch.int32, device=dev), src_b=torch.zeros(n, dtype=torch.int32, device=dev),
             w_a=torch.zeros(n, dtype=torch.float32, device=dev), w_b=torch.zeros(n, dtype=torch.float32, device=dev),
             new_video_offsets=torch.zeros(V + 1, dtype=torch.int32, device=dev))
    _check(lib().et_merge_plan(_ptr(sim), _ptr(video_offsets), n, V, float(alpha), float(tau_seg), float(tau_merge),
                               int(weighted), _ptr(o["seg_start"]), _ptr(o["merge_next"]), _ptr(o["ema"]),
                               _ptr(o["n_out"]), _ptr(o["src_a"]), _ptr(o["src_b"]), _ptr(o["w_a"]), _ptr(o["w_b"]),
                               _ptr(o["new_video_offsets"]), _stream_ptr(stream)))
    return o


def et_merge_frames(x, plan: dict, stream=None):
    import torch
    n = x.shape[0]
    y = torch.empty_like(x)
    _check(lib().et_merge_frames(_ptr(x), _ptr(y), n, int(x[0].numel()), _ptr(plan["n_out"]), _ptr(plan["src_a"]),
                                 _ptr(plan["src_b"]), _ptr(plan["w_a"]), _ptr(plan["w_b"]), _stream_ptr(stream)))
    return y


def et_select_tokens(scores, dynamic, k, w, window_mode=0, stream=None):
    import torch
    N, L = scores.shape
    keep = torch.zeros((N, L), dtype=torch.uint8, device=scores.device)
    count = torch.zeros(N, dtype=torch.int32, device=scores.device)
    _check(lib().et_select_tokens(_ptr(scores), _ptr(dynamic), _ptr(k), _ptr(w), N, L, int(window_mode), _ptr(keep), _ptr(count),
                                  _stream_ptr(stream)))
    return keep, count


def et_gather_tokens(x, keep, ln_g=None, ln_b=None, eps=1e-6, capacity_rows=None, stream=None):
    import torch
    N, L, D = x.shape
    cap = int(capacity_rows if capacity_rows is not None else N * L)
    tokens = torch.empty((cap, D), dtype=torch.float32, device=x.device)
    offs = torch.zeros(N + 1, dtype=torch.int32, device=x.device)
    pos = torch.zeros(cap, dtype=torch.int32, device=x.device)
    nt = C.c_int(0)
    _check(lib().et_gather_tokens(_ptr(x), _ptr(keep), N, L, D, _ptr(ln_g), _ptr(ln_b), float(eps), _ptr(tokens), cap,
                                  _ptr(offs), _ptr(pos), C.byref(nt), _stream_ptr(stream)))
    return tokens[:nt.value], offs, pos[:nt.value]


def et_linear_bf16(a, w, bias, epilogue=0, gelu_tanh=1, c=None, table=None, stream=None):
    """a [M,K] bf16, w [N,K] bf16, bias [N] f32.  Returns (c, status int)."""
    import torch
    M, K = a.shape
    N = w.shape[0]
    if c is None:
        c = torch.empty((M, N // 2 if epilogue == 4 else N), dtype=torch.bfloat16 if epilogue in (0, 1, 4) else torch.float32,
                        device=a.device)
    status = torch.zeros(1, dtype=torch.int32, device=a.device)
    _check(lib().et_linear_bf16(_ptr(a), _ptr(w), _ptr(bias), _ptr(c), M, N, K, int(epilogue), int(gelu_tanh),
                                _ptr(table), int(table.shape[0]) if table is not None else 0, _ptr(status),
                                _stream_ptr(stream)))
    return c, status


def et_attention_windowed(qkv, n, L, heads, head_dim, window_rows, stream=None):
    import torch
    dtype = ET_BF16 if qkv.dtype == torch.bfloat16 else ET_F32
    out = torch.empty((n * L, heads * head_dim), dtype=qkv.dtype, device=qkv.device)
    lse = torch.empty((n, heads, L), dtype=torch.float32, device=qkv.device)
    _check(lib().et_attention_windowed(_ptr(qkv), _ptr(out), _ptr(lse), n, L, heads, head_dim, int(window_rows), dtype,
                                       _stream_ptr(stream)))
    return out


def et_attention(qkv, n, L, heads, head_dim, stream=None):
    import torch
    dtype = ET_BF16 if qkv.dtype == torch.bfloat16 else ET_F32
    out = torch.empty((n * L, heads * head_dim), dtype=qkv.dtype, device=qkv.device)
    lse = torch.empty((n, heads, L), dtype=torch.float32, device=qkv.device)
    _check(lib().et_attention(_ptr(qkv), _ptr(out), _ptr(lse), n, L, heads, head_dim, dtype, _stream_ptr(stream)))
    return out, lse


def et_attention_scores(qkv, lse, n, L, heads, head_dim, stream=None):
    import torch
    dtype = ET_BF16 if qkv.dtype == torch.bfloat16 else ET_F32
    partial = torch.empty((n, heads, L), dtype=torch.float32, device=qkv.device)
    score = torch.empty((n, L), dtype=torch.float32, device=qkv.device)
    _check(lib().et_attention_scores(_ptr(qkv), _ptr(lse), _ptr(partial), _ptr(score), n, L, heads, head_dim, dtype,
                                     _stream_ptr(stream)))
    return score


def et_layernorm(x, g, b, eps, out_bf16=False, stream=None):
    import torch
    rows, D = x.shape
    y = torch.empty((rows, D), dtype=torch.bfloat16 if out_bf16 else torch.float32, device=x.device)
    _check(lib().et_layernorm(_ptr(x), _ptr(g), _ptr(b), float(eps), _ptr(y), rows, D, ET_BF16 if out_bf16 else ET_F32,
                              _stream_ptr(stream)))
    return y


# --------------------------------------------------------------------------------------------
# Downstream of the encoder: projector + language-model prefill (include/earlytom_llm.h)
# --------------------------------------------------------------------------------------------

@dataclass
class PrefillResult:
    n_tokens: int
    first_token: int
    logits: object        # torch fp32 [vocab] (copy)
    hidden: object        # torch fp32 [n_tokens, hidden] (copy) or None
    kv_cache: object = None   # torch bf16 [layers, n_tokens, 2*kv_heads*head_dim] (copy), on request


def et_llm_create(cfg: et_llm_config, weights) -> C.c_void_p:
    """weights: numpy fp32 blob (host) or a torch fp32 CUDA tensor (device blob)."""
    if isinstance(weights, np.ndarray):
        w = np.ascontiguousarray(weights, dtype=np.float32)
        wb = et_llm_weights(w.ctypes.data, w.size, 0)
    else:
        assert weights.is_cuda and weights.is_contiguous() and weights.element_size() == 4
        wb = et_llm_weights(weights.data_ptr(), weights.numel(), 1)
    h = C.c_void_p()
    _check(lib().et_llm_create(C.byref(cfg), C.byref(wb), C.byref(h)))
    return h


def et_llm_destroy(handle) -> None:
    lib().et_llm_destroy(handle)


class LanguageModel:
    """Owns an et_llm*.  `shape` is any object with the architecture fields of et_llm_config."""

    def __init__(self, shape, weights, max_tokens: int, keep_kv_cache: bool = False):
        cfg = et_llm_config(shape.vision_hidden, shape.hidden, shape.num_layers, shape.heads, shape.kv_heads, shape.head_dim,
                            shape.mlp_dim, shape.vocab, float(shape.rms_eps), float(shape.rope_theta), int(shape.gelu_tanh),
                            int(max_tokens), 1 if keep_kv_cache else 0)
        self.handle = et_llm_create(cfg, weights)
        self.shape = shape

    def close(self):
        if getattr(self, "handle", None):
            et_llm_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def prefill(self, prefix_ids, visual_tokens, suffix_ids, want_hidden=False, stream=None, want_kv=False) -> PrefillResult:
        return et_llm_prefill(self, prefix_ids, visual_tokens, suffix_ids, want_hidden, stream, want_kv=want_kv)


def _ids(a):
    a = np.ascontiguousarray(a if a is not None else [], dtype=np.int32)
    return a, (a.ctypes.data_as(_I32P) if a.size else None)


def et_llm_prefill(llm: LanguageModel, prefix_ids, visual_tokens, suffix_ids, want_hidden=False, stream=None,
                   copy_logits=True, want_kv=False) -> PrefillResult:
    """visual_tokens: torch fp32 CUDA [n_visual, vision_hidden] (or None)."""
    pre, pre_p = _ids(prefix_ids)
    suf, suf_p = _ids(suffix_ids)
    n_vis = 0
    if visual_tokens is not None and visual_tokens.shape[0] > 0:
        assert visual_tokens.is_cuda and visual_tokens.is_contiguous() and visual_tokens.element_size() == 4
        assert visual_tokens.shape[1] == llm.shape.vision_hidden
        n_vis = int(visual_tokens.shape[0])
    r = et_llm_result()
    st = lib().et_llm_prefill(llm.handle, pre_p, int(pre.size), _ptr(visual_tokens) if n_vis else None, n_vis, suf_p,
                              int(suf.size), _stream_ptr(stream), C.byref(r))
    if st != 0:
        raise EarlyTomError(st, lib().et_llm_last_error(llm.handle).decode())
    logits = _dev_tensor(r.logits, (llm.shape.vocab,), "<f4") if copy_logits else None
    hidden = _dev_tensor(r.hidden, (r.n_tokens, llm.shape.hidden), "<f4") if want_hidden else None
    kv = None
    if want_kv:
        if not r.kv_cache:
            raise EarlyTomError(1, "the model was created without keep_kv_cache")
        import torch
        sh = llm.shape
        full = torch.as_tensor(_DevView(r.kv_cache, (sh.num_layers, r.kv_cache_rows, 2 * sh.kv_heads * sh.head_dim * 2), "|u1"),
                               device="cuda")
        kv = full[:, :r.n_tokens].clone().view(torch.bfloat16)
    return PrefillResult(r.n_tokens, r.first_token, logits, hidden, kv)


def et_llm_profile_enable(llm: LanguageModel, on: bool) -> None:
    _check(lib().et_llm_profile_enable(llm.handle, 1 if on else 0))


def et_llm_profile_read(llm: LanguageModel) -> dict:
    p = et_llm_profile()
    _check(lib().et_llm_profile_read(llm.handle, C.byref(p)))
    return {"calls": p.calls, "ms": {n: p.ms[k] for k, n in enumerate(LLM_PROF_NAMES)},
            "launches": {n: int(p.launches[k]) for k, n in enumerate(LLM_PROF_NAMES)}}


def et_rmsnorm(x, g, eps, stream=None):
    import torch
    rows, D = x.shape
    y = torch.empty((rows, D), dtype=torch.bfloat16, device=x.device)
    _check(lib().et_rmsnorm(_ptr(x), _ptr(g), float(eps), _ptr(y), rows, D, _stream_ptr(stream)))
    return y


def et_rope(qkv, L, heads, kv_heads, head_dim, theta, stream=None):
    """In place on qkv (bf16 [rows, (heads + 2*kv_heads)*head_dim]); returns qkv."""
    _check(lib().et_rope(_ptr(qkv), int(qkv.shape[0]), int(L), heads, kv_heads, head_dim, float(theta), _stream_ptr(stream)))
    return qkv


def et_swiglu(gu, stream=None):
    import torch
    rows, M2 = gu.shape
    h = torch.empty((rows, M2 // 2), dtype=torch.bfloat16, device=gu.device)
    _check(lib().et_swiglu(_ptr(gu), _ptr(h), rows, M2 // 2, _stream_ptr(stream)))
    return h


def et_attention_causal(qkv, n_seq, L, heads, kv_heads, head_dim, stream=None):
    """Returns (out bf16 [n_seq*L, heads*head_dim], status int32[1])."""
    import torch
    out = torch.empty((n_seq * L, heads * head_dim), dtype=torch.bfloat16, device=qkv.device)
    status = torch.zeros(1, dtype=torch.int32, device=qkv.device)
    _check(lib().et_attention_causal(_ptr(qkv), _ptr(out), n_seq, L, heads, kv_heads, head_dim, _ptr(status),
                                     _stream_ptr(stream)))
    return out, status
