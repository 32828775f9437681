"""ctypes binding of libflashcache.so: argument marshalling only.

Every function here has the name and the meaning of the C entry point declared
in include/flashcache.h; tensors are passed as device pointers, the current
torch CUDA stream is passed as the stream.  All arithmetic happens in the CUDA
library.  There is no fallback: if the library has not been built this module
raises on import.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, byref, c_char_p, c_double, c_int, c_int32, c_int64, c_size_t, c_uint64, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libflashcache.so")

FC_OK = 0
FC_F32, FC_F16, FC_BF16 = 0, 1, 2
_DTYPE = {torch.float32: FC_F32, torch.float16: FC_F16, torch.bfloat16: FC_BF16}

EXPORTS = (
    "fc_create", "fc_destroy", "fc_status_string", "fc_last_device_status", "fc_launch_count", "fc_selftest_bounded_wait", "fc_measure_fp32_peak", "fc_proto_dft16_stage",
    "fc_set_group_bytes", "fc_set_chirp_band", "fc_set_internal_streams", "fc_set_l2_persist", "fc_reset_ordering", "fc_set_score_overlap", "fc_set_select_overlap", "fc_profile_begin", "fc_profile_stride", "fc_profile_end", "fc_describe_plan",
    "fc_score_workspace_bytes", "fc_select_workspace_bytes",
    "fc_score_layer", "fc_allocate_budgets", "fc_select_compact", "fc_select_compact_ex",
    "fc_select_compact_layers", "fc_layer_capacity_rows",
    "fc_power_spectrum_workspace_bytes", "fc_power_spectrum", "fc_cutoff_from_spectrum",
    "fc_decode_workspace_bytes", "fc_decode_attention",
    "fc_static_scratch_bytes", "fc_score_layer_static", "fc_static_last_device_status",
    "fc_compress_host_rows", "fc_compress_host_arena_bytes", "fc_compress_host",
)


class fc_kv_view(ctypes.Structure):
    _fields_ = [
        ("k", c_void_p), ("v", c_void_p),
        ("stride_token", c_int64), ("stride_head", c_int64),
        ("dtype", c_int32), ("num_heads", c_int32), ("head_dim", c_int32), ("batch", c_int32),
        ("cu_seqlens", POINTER(c_int32)),
    ]


class fc_select_options(ctypes.Structure):
    _fields_ = [("per_layer", c_int32), ("protect", c_void_p)]


class fc_layer_buffers(ctypes.Structure):
    _fields_ = [("k", c_void_p), ("v", c_void_p), ("scores", c_void_p), ("out_k", c_void_p), ("out_v", c_void_p),
                ("out_idx", c_void_p), ("out_capacity_rows", c_int64)]


class fc_decode_args(ctypes.Structure):
    _fields_ = [
        ("q", c_void_p), ("cache_k", c_void_p), ("cache_v", c_void_p), ("cache_rows", c_int64),
        ("offsets", c_void_p), ("tail_k", c_void_p), ("tail_v", c_void_p), ("tail_len", c_void_p),
        ("tail_capacity", c_int32), ("dtype", c_int32), ("batch", c_int32), ("num_heads", c_int32),
        ("num_q_heads", c_int32), ("head_dim", c_int32), ("max_rows", c_int64),
    ]


class fc_host_job(ctypes.Structure):
    _fields_ = [
        ("k_host", POINTER(c_void_p)), ("v_host", POINTER(c_void_p)),
        ("num_layers", c_int32), ("dtype", c_int32), ("num_heads", c_int32), ("head_dim", c_int32),
        ("batch", c_int32), ("min_keep", c_int32),
        ("cu_seqlens", POINTER(c_int32)),
        ("gamma", c_double), ("rho", c_double),
        ("arena", c_void_p), ("arena_bytes", c_size_t),
        ("out_k_host", c_void_p), ("out_v_host", c_void_p), ("out_idx_host", c_void_p),
        ("out_capacity_rows", c_int64),
        ("budgets_host", c_void_p), ("offsets_host", c_void_p), ("layer_rows_host", c_void_p),
        ("per_layer", c_int32), ("protect_host", c_void_p),
    ]


class FlashCacheError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s failed: %s (fc_status %d)" % (where, status_string(code), code))


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            "libflashcache.so is missing at %s: build it with "
            "`python -m paper_2511_16786_b200.build` (needs nvcc); there is no CPU fallback" % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    lib.fc_create.argtypes = [POINTER(c_void_p), c_int, c_int32]
    lib.fc_create.restype = c_int
    lib.fc_destroy.argtypes = [c_void_p]
    lib.fc_destroy.restype = None
    lib.fc_status_string.argtypes = [c_int]
    lib.fc_status_string.restype = c_char_p
    lib.fc_last_device_status.argtypes = [c_void_p, c_void_p]
    lib.fc_last_device_status.restype = c_int
    lib.fc_launch_count.argtypes = [c_void_p]
    lib.fc_launch_count.restype = c_uint64
    lib.fc_set_group_bytes.argtypes = [c_void_p, c_size_t]
    lib.fc_set_group_bytes.restype = c_int
    lib.fc_reset_ordering.argtypes = [c_void_p]
    lib.fc_reset_ordering.restype = c_int
    lib.fc_cutoff_from_spectrum.argtypes = [c_void_p, c_void_p, c_int32, POINTER(c_int32), c_double, c_void_p,
                                            c_void_p, c_void_p]
    lib.fc_cutoff_from_spectrum.restype = c_int
    lib.fc_proto_dft16_stage.argtypes = [c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_void_p]
    lib.fc_proto_dft16_stage.restype = c_int
    lib.fc_measure_fp32_peak.argtypes = [c_void_p, POINTER(c_double)]
    lib.fc_measure_fp32_peak.restype = c_int
    lib.fc_selftest_bounded_wait.argtypes = [c_void_p, c_void_p]
    lib.fc_selftest_bounded_wait.restype = c_int
    lib.fc_set_chirp_band.argtypes = [c_void_p, c_int32]
    lib.fc_set_chirp_band.restype = c_int
    lib.fc_set_internal_streams.argtypes = [c_void_p, c_int32]
    lib.fc_set_internal_streams.restype = c_int
    lib.fc_set_l2_persist.argtypes = [c_void_p, c_int32]
    lib.fc_set_l2_persist.restype = c_int
    lib.fc_static_last_device_status.argtypes = [c_void_p]
    lib.fc_static_last_device_status.restype = c_int
    lib.fc_set_score_overlap.argtypes = [c_void_p, c_int32]
    lib.fc_set_score_overlap.restype = c_int
    lib.fc_set_select_overlap.argtypes = [c_void_p, c_int32]
    lib.fc_set_select_overlap.restype = c_int
    lib.fc_profile_begin.argtypes = [c_void_p, c_int32, c_int32]
    lib.fc_profile_begin.restype = c_int
    lib.fc_profile_stride.argtypes = [c_void_p, c_int32]
    lib.fc_profile_stride.restype = c_int
    lib.fc_profile_end.argtypes = [c_void_p, POINTER(c_double), POINTER(c_uint64)]
    lib.fc_profile_end.restype = c_int
    lib.fc_describe_plan.argtypes = [c_void_p, c_int32, c_double, POINTER(c_int32)]
    lib.fc_describe_plan.restype = c_int
    lib.fc_score_workspace_bytes.argtypes = [c_void_p, POINTER(fc_kv_view)]
    lib.fc_score_workspace_bytes.restype = c_size_t
    lib.fc_select_workspace_bytes.argtypes = [c_void_p, POINTER(fc_kv_view)]
    lib.fc_select_workspace_bytes.restype = c_size_t
    lib.fc_score_layer.argtypes = [c_void_p, POINTER(fc_kv_view), c_double, c_void_p, c_void_p,
                                   c_void_p, c_size_t, c_void_p]
    lib.fc_score_layer.restype = c_int
    lib.fc_allocate_budgets.argtypes = [c_void_p, c_void_p, c_int32, c_int32, POINTER(c_int32),
                                        c_double, c_int32, c_void_p, c_void_p, c_void_p]
    lib.fc_allocate_budgets.restype = c_int
    lib.fc_select_compact.argtypes = [c_void_p, POINTER(fc_kv_view), c_void_p, c_void_p, c_void_p,
                                      c_void_p, c_void_p, c_void_p, c_int64, c_void_p, c_size_t, c_void_p]
    lib.fc_select_compact.restype = c_int
    lib.fc_select_compact_ex.argtypes = [c_void_p, POINTER(fc_kv_view), c_void_p, c_void_p, c_void_p,
                                         c_void_p, c_void_p, c_void_p, c_int64, POINTER(fc_select_options),
                                         c_void_p, c_size_t, c_void_p]
    lib.fc_select_compact_ex.restype = c_int
    lib.fc_select_compact_layers.argtypes = [c_void_p, POINTER(fc_kv_view), POINTER(fc_layer_buffers), c_int32,
                                             c_void_p, c_void_p, POINTER(fc_select_options), c_void_p, c_size_t,
                                             c_void_p]
    lib.fc_select_compact_layers.restype = c_int
    lib.fc_layer_capacity_rows.argtypes = [c_int32, c_int32, POINTER(c_int32), c_double, c_int32]
    lib.fc_layer_capacity_rows.restype = c_int64
    lib.fc_power_spectrum_workspace_bytes.argtypes = [c_void_p, POINTER(fc_kv_view)]
    lib.fc_power_spectrum_workspace_bytes.restype = c_size_t
    lib.fc_power_spectrum.argtypes = [c_void_p, POINTER(fc_kv_view), c_void_p, c_void_p, c_size_t, c_void_p]
    lib.fc_power_spectrum.restype = c_int
    lib.fc_decode_workspace_bytes.argtypes = [c_void_p, POINTER(fc_decode_args)]
    lib.fc_decode_workspace_bytes.restype = c_size_t
    lib.fc_decode_attention.argtypes = [c_void_p, POINTER(fc_decode_args), c_void_p, c_void_p, c_size_t, c_void_p]
    lib.fc_decode_attention.restype = c_int
    lib.fc_static_scratch_bytes.argtypes = []
    lib.fc_static_scratch_bytes.restype = c_size_t
    lib.fc_score_layer_static.argtypes = [POINTER(fc_kv_view), c_double, c_void_p, c_void_p, c_void_p]
    lib.fc_score_layer_static.restype = c_int
    lib.fc_compress_host_rows.argtypes = [c_int32, c_int32, POINTER(c_int32), c_double, c_int32]
    lib.fc_compress_host_rows.restype = c_int64
    lib.fc_compress_host_arena_bytes.argtypes = [c_void_p, POINTER(fc_host_job)]
    lib.fc_compress_host_arena_bytes.restype = c_size_t
    lib.fc_compress_host.argtypes = [c_void_p, POINTER(fc_host_job), c_void_p]
    lib.fc_compress_host.restype = c_int
    return lib


_lib = _load()


def status_string(code: int) -> str:
    return _lib.fc_status_string(int(code)).decode()


def _check(code: int, where: str):
    if code != FC_OK:
        raise FlashCacheError(code, where)


def _stream() -> c_void_p:
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def _cu_array(cu_seqlens):
    vals = [int(x) for x in cu_seqlens]
    return (c_int32 * len(vals))(*vals)


def make_view(k: torch.Tensor, v: torch.Tensor, cu_arr) -> fc_kv_view:
    """View of K, V [T, H, d] tensors (channel stride 1; V must share K's strides)."""
    if k.dim() != 3 or v.shape != k.shape or v.dtype != k.dtype:
        raise ValueError("k and v must be [T, H, d] tensors of one dtype")
    if k.stride(2) != 1 or v.stride() != k.stride():
        raise ValueError("channel stride must be 1 and v must be laid out like k")
    if k.dtype not in _DTYPE:
        raise ValueError("unsupported dtype %s" % k.dtype)
    return fc_kv_view(c_void_p(k.data_ptr()), c_void_p(v.data_ptr()), k.stride(0), k.stride(1),
                      _DTYPE[k.dtype], k.shape[1], k.shape[2], len(cu_arr) - 1,
                      ctypes.cast(cu_arr, POINTER(c_int32)))


# ----------------------------------------------------------------------------
# entry points (same names as the C ABI)
# ----------------------------------------------------------------------------
def fc_create(device: int = 0, max_seqlen: int = 65536) -> c_void_p:
    h = c_void_p()
    _check(_lib.fc_create(byref(h), int(device), int(max_seqlen)), "fc_create")
    return h


def fc_destroy(handle) -> None:
    _lib.fc_destroy(handle)


def fc_last_device_status(handle) -> int:
    return int(_lib.fc_last_device_status(handle, _stream()))


def fc_launch_count(handle) -> int:
    return int(_lib.fc_launch_count(handle))


def fc_set_group_bytes(handle, nbytes: int) -> None:
    _check(_lib.fc_set_group_bytes(handle, int(nbytes)), "fc_set_group_bytes")


def fc_cutoff_from_spectrum(handle, spectrum, cu_seqlens, share: float, omega, gamma) -> None:
    """spectrum: float64 [T, 2] from fc_power_spectrum; omega: int32 [B]; gamma: float64 [B] (device)."""
    cu = _cu_array(cu_seqlens)
    _check(_lib.fc_cutoff_from_spectrum(handle, c_void_p(spectrum.data_ptr()), len(cu) - 1,
                                        ctypes.cast(cu, POINTER(c_int32)), float(share),
                                        c_void_p(omega.data_ptr()), c_void_p(gamma.data_ptr()), _stream()),
           "fc_cutoff_from_spectrum")


def fc_proto_dft16_stage(handle, x, y, variant: int, repeat: int = 1) -> None:
    """x, y: float32 device tensors [16, ncols, 2] (complex as pairs); variant 0 FP32 pipes, 1 tensor pipe, 2 copy."""
    _check(_lib.fc_proto_dft16_stage(handle, c_void_p(x.data_ptr()), c_void_p(y.data_ptr()), int(x.shape[1]),
                                     int(variant), int(repeat), _stream()), "fc_proto_dft16_stage")


def fc_measure_fp32_peak(handle) -> float:
    """TFLOP/s the FP32 pipes sustain in a pure fused-multiply-add loop (blocks the host for a few ms)."""
    t = c_double(0.0)
    _check(_lib.fc_measure_fp32_peak(handle, byref(t)), "fc_measure_fp32_peak")
    return float(t.value)


def fc_selftest_bounded_wait(handle) -> None:
    _check(_lib.fc_selftest_bounded_wait(handle, _stream()), "fc_selftest_bounded_wait")


def fc_set_chirp_band(handle, enabled: bool) -> None:
    _check(_lib.fc_set_chirp_band(handle, 1 if enabled else 0), "fc_set_chirp_band")


def fc_set_internal_streams(handle, count: int) -> None:
    _check(_lib.fc_set_internal_streams(handle, int(count)), "fc_set_internal_streams")


def fc_set_l2_persist(handle, enabled: bool) -> None:
    _check(_lib.fc_set_l2_persist(handle, 1 if enabled else 0), "fc_set_l2_persist")


def fc_set_score_overlap(handle, enabled: bool) -> None:
    _check(_lib.fc_set_score_overlap(handle, 1 if enabled else 0), "fc_set_score_overlap")


def fc_set_select_overlap(handle, enabled: bool) -> None:
    _check(_lib.fc_set_select_overlap(handle, 1 if enabled else 0), "fc_set_select_overlap")


KERNEL_CLASSES = {"pass1": 1, "pass2": 2, "pass3": 3, "select": 4, "gather": 5, "other": 6}


def fc_profile_begin(handle, kernel_class: int, max_launches: int = 16384) -> None:
    _check(_lib.fc_profile_begin(handle, int(kernel_class), int(max_launches)), "fc_profile_begin")


def fc_profile_stride(handle, stride: int) -> None:
    _check(_lib.fc_profile_stride(handle, int(stride)), "fc_profile_stride")


def fc_profile_end(handle):
    """-> (total_ms, launches) of the kernel class given to fc_profile_begin."""
    ms, n = c_double(0.0), c_uint64(0)
    _check(_lib.fc_profile_end(handle, byref(ms), byref(n)), "fc_profile_end")
    return float(ms.value), int(n.value)


def fc_describe_plan(handle, seqlen: int, gamma: float) -> dict:
    out = (c_int32 * 4)()
    _check(_lib.fc_describe_plan(handle, int(seqlen), float(gamma), out), "fc_describe_plan")
    return dict(bluestein=bool(out[0]), band_form=out[0] == 2, nfft=int(out[1]), n1=int(out[2]), n2=int(out[3]))


def fc_score_workspace_bytes(handle, k, v, cu_seqlens) -> int:
    cu = _cu_array(cu_seqlens)
    view = make_view(k, v, cu)
    return int(_lib.fc_score_workspace_bytes(handle, byref(view)))


def fc_select_workspace_bytes(handle, k, v, cu_seqlens) -> int:
    cu = _cu_array(cu_seqlens)
    view = make_view(k, v, cu)
    return int(_lib.fc_select_workspace_bytes(handle, byref(view)))


def fc_score_layer(handle, k, v, cu_seqlens, gamma: float, scores, energy, workspace) -> None:
    """scores: float32 [H, T]; energy: float64 [B, 4]; workspace: uint8 device tensor."""
    cu = _cu_array(cu_seqlens)
    view = make_view(k, v, cu)
    _check(_lib.fc_score_layer(handle, byref(view), float(gamma), c_void_p(scores.data_ptr()),
                               c_void_p(energy.data_ptr()), c_void_p(workspace.data_ptr()),
                               workspace.numel() * workspace.element_size(), _stream()), "fc_score_layer")


def fc_static_scratch_bytes() -> int:
    return int(_lib.fc_static_scratch_bytes())


def fc_score_layer_static(k, v, cu_seqlens, gamma: float, scores, energy) -> None:
    """fc_score_layer for callers that may not allocate device memory: no handle, no
    workspace; the scratch is a fixed array inside the library (see include/flashcache.h
    for the size limits and the sharing rule).  scores: float32 [H, T]; energy: float64 [B, 4]."""
    cu = _cu_array(cu_seqlens)
    view = make_view(k, v, cu)
    _check(_lib.fc_score_layer_static(byref(view), float(gamma), c_void_p(scores.data_ptr()),
                                      c_void_p(energy.data_ptr()), _stream()), "fc_score_layer_static")


def fc_static_last_device_status() -> int:
    """Synchronises the current stream; status recorded by fc_score_layer_static calls on this device."""
    return int(_lib.fc_static_last_device_status(_stream()))


def fc_compress_host_rows(num_layers: int, cu_seqlens, rho: float, min_keep: int) -> int:
    cu = _cu_array(cu_seqlens)
    return int(_lib.fc_compress_host_rows(int(num_layers), len(cu) - 1, ctypes.cast(cu, POINTER(c_int32)),
                                          float(rho), int(min_keep)))


def fc_power_spectrum_workspace_bytes(handle, k, v, cu_seqlens) -> int:
    cu = _cu_array(cu_seqlens)
    view = make_view(k, v, cu)
    return int(_lib.fc_power_spectrum_workspace_bytes(handle, byref(view)))


def fc_power_spectrum(handle, k, v, cu_seqlens, spectrum, workspace) -> None:
    """spectrum: float64 [T, 2] on the device: (P_k[m], P_v[m]) at row cu[b] + m."""
    cu = _cu_array(cu_seqlens)
    view = make_view(k, v, cu)
    _check(_lib.fc_power_spectrum(handle, byref(view), c_void_p(spectrum.data_ptr()), c_void_p(workspace.data_ptr()),
                                  workspace.numel() * workspace.element_size(), _stream()), "fc_power_spectrum")


def make_decode_args(q, cache_k, cache_v, offsets, max_rows: int, tail_k=None, tail_v=None, tail_len=None):
    """q: [B, Hq, d]; cache_k/v: [rows, H, d]; offsets: int64 [B+1] on the device; tail_k/v: [B, cap, H, d];
    tail_len: int32 [B] on the device.  max_rows bounds kept + tail rows of any sequence."""
    B, Hq, d = (int(x) for x in q.shape)
    rows, H, _ = (int(x) for x in cache_k.shape)
    for t in (q, cache_k, cache_v):
        if not t.is_cuda or not t.is_contiguous() or t.dtype != q.dtype:
            raise ValueError("q and the cache must be contiguous device tensors of one dtype")
    a = fc_decode_args(q=q.data_ptr(), cache_k=cache_k.data_ptr(), cache_v=cache_v.data_ptr(), cache_rows=rows,
                       offsets=offsets.data_ptr(), dtype=_DTYPE[q.dtype], batch=B, num_heads=H, num_q_heads=Hq,
                       head_dim=d, max_rows=int(max_rows))
    if tail_k is not None:
        if not (tail_k.is_contiguous() and tail_v.is_contiguous() and tail_k.dtype == q.dtype):
            raise ValueError("tail_k/tail_v: contiguous [B, cap, H, d] of the cache dtype")
        a.tail_k, a.tail_v, a.tail_len = tail_k.data_ptr(), tail_v.data_ptr(), tail_len.data_ptr()
        a.tail_capacity = int(tail_k.shape[1])
    return a


def fc_decode_workspace_bytes(handle, args) -> int:
    return int(_lib.fc_decode_workspace_bytes(handle, byref(args)))


def fc_decode_attention(handle, args, out, workspace) -> None:
    """out: [B, Hq, d] device tensor of the cache dtype."""
    _check(_lib.fc_decode_attention(handle, byref(args), c_void_p(out.data_ptr()), c_void_p(workspace.data_ptr()),
                                    workspace.numel() * workspace.element_size(), _stream()), "fc_decode_attention")


def fc_reset_ordering(handle) -> None:
    _check(_lib.fc_reset_ordering(handle), "fc_reset_ordering")


def fc_allocate_budgets(handle, energy, cu_seqlens, rho: float, min_keep: int, budgets, out_offsets) -> None:
    """energy: float64 [L, B, 4]; budgets: int32 [L, B]; out_offsets: int64 [L, B+1]."""
    cu = _cu_array(cu_seqlens)
    L, B = int(energy.shape[0]), int(energy.shape[1])
    _check(_lib.fc_allocate_budgets(handle, c_void_p(energy.data_ptr()), L, B,
                                    ctypes.cast(cu, POINTER(c_int32)), float(rho), int(min_keep),
                                    c_void_p(budgets.data_ptr()), c_void_p(out_offsets.data_ptr()),
                                    _stream()), "fc_allocate_budgets")


def fc_select_compact(handle, k, v, cu_seqlens, scores, budgets, out_offsets, out_k, out_v, out_idx,
                      workspace) -> None:
    """budgets: int32 [B], out_offsets: int64 [B+1] (one layer's slices);
    out_k/out_v: [capacity, H, d]; out_idx: int32 [H, capacity]."""
    cu = _cu_array(cu_seqlens)
    view = make_view(k, v, cu)
    cap = int(out_k.shape[0])
    _check(_lib.fc_select_compact(handle, byref(view), c_void_p(scores.data_ptr()),
                                  c_void_p(budgets.data_ptr()), c_void_p(out_offsets.data_ptr()),
                                  c_void_p(out_k.data_ptr()), c_void_p(out_v.data_ptr()),
                                  c_void_p(out_idx.data_ptr()), cap, c_void_p(workspace.data_ptr()),
                                  workspace.numel() * workspace.element_size(), _stream()),
           "fc_select_compact")


def fc_select_compact_ex(handle, k, v, cu_seqlens, scores, budgets, out_offsets, out_k, out_v, out_idx,
                         workspace, per_layer: bool = False, protect=None) -> None:
    """fc_select_compact with options: per_layer (one index set per layer from the head-averaged
    score) and protect (uint8 [T] on the device, non-zero = always ranked first)."""
    cu = _cu_array(cu_seqlens)
    view = make_view(k, v, cu)
    cap = int(out_k.shape[0])
    if protect is not None and (protect.dtype != torch.uint8 or not protect.is_cuda or protect.numel() != k.shape[0]
                                or not protect.is_contiguous()):
        raise ValueError("protect: contiguous uint8 device tensor with one entry per token")
    opt = fc_select_options(per_layer=1 if per_layer else 0,
                            protect=protect.data_ptr() if protect is not None else None)
    _check(_lib.fc_select_compact_ex(handle, byref(view), c_void_p(scores.data_ptr()),
                                     c_void_p(budgets.data_ptr()), c_void_p(out_offsets.data_ptr()),
                                     c_void_p(out_k.data_ptr()), c_void_p(out_v.data_ptr()),
                                     c_void_p(out_idx.data_ptr()), cap, byref(opt), c_void_p(workspace.data_ptr()),
                                     workspace.numel() * workspace.element_size(), _stream()),
           "fc_select_compact_ex")


def fc_layer_capacity_rows(num_layers: int, cu_seqlens, rho: float, min_keep: int = 1) -> int:
    """Rows one layer's compacted cache can receive at most (sizes out_k / out_v / out_idx)."""
    cu = _cu_array(cu_seqlens)
    r = int(_lib.fc_layer_capacity_rows(int(num_layers), len(cu) - 1, ctypes.cast(cu, POINTER(c_int32)),
                                        float(rho), int(min_keep)))
    if r < 0:
        raise FlashCacheError(1, "fc_layer_capacity_rows")
    return r


def fc_select_compact_layers(handle, K_layers, V_layers, cu_seqlens, scores, budgets, out_offsets, out_k, out_v,
                             out_idx, workspace, per_layer: bool = False, protect=None) -> None:
    """All layers in one launch.  scores [L, H, T]; budgets [L, B]; out_offsets [L, B+1];
    out_k / out_v [L, capacity, H, d]; out_idx [L, H, capacity]."""
    L = len(K_layers)
    cu = _cu_array(cu_seqlens)
    view = make_view(K_layers[0], V_layers[0], cu)
    cap = int(out_k.shape[1])
    tab = (fc_layer_buffers * L)()
    for l in range(L):
        tab[l] = fc_layer_buffers(K_layers[l].data_ptr(), V_layers[l].data_ptr(), scores[l].data_ptr(),
                                  out_k[l].data_ptr(), out_v[l].data_ptr(), out_idx[l].data_ptr(), cap)
    opt = fc_select_options(per_layer=1 if per_layer else 0,
                            protect=protect.data_ptr() if protect is not None else None)
    _check(_lib.fc_select_compact_layers(handle, byref(view), tab, L, c_void_p(budgets.data_ptr()),
                                         c_void_p(out_offsets.data_ptr()), byref(opt), c_void_p(workspace.data_ptr()),
                                         workspace.numel() * workspace.element_size(), _stream()),
           "fc_select_compact_layers")


# ----------------------------------------------------------------------------
# convenience: buffers for a whole model and the three-phase pass
# ----------------------------------------------------------------------------
class Compressor:
    """Owns a handle and the device buffers of one workload shape; `compress`
    issues fc_score_layer x L, fc_allocate_budgets, fc_select_compact x L on the
    current stream.  Only allocation and call sequencing happen here."""

    def __init__(self, num_layers: int, num_heads: int, head_dim: int, cu_seqlens, dtype, rho: float,
                 gamma: float = 0.2, min_keep: int = 1, device: int = 0, group_bytes: int | None = None,
                 select_overlap: bool = True, score_overlap: bool = True, per_layer: bool = False,
                 protect=None):
        self.L, self.H, self.d = num_layers, num_heads, head_dim
        # selection options (fc_select_compact_ex): one index set per layer; uint8 [T] device mask of tokens to keep
        self.per_layer = bool(per_layer)
        self.protect = protect
        self._opt = fc_select_options(per_layer=1 if per_layer else 0,
                                      protect=protect.data_ptr() if protect is not None else None)
        self.cu = [int(x) for x in cu_seqlens]
        self.B = len(self.cu) - 1
        self.T = self.cu[-1]
        self.rho, self.gamma, self.min_keep = float(rho), float(gamma), int(min_keep)
        self.dtype = dtype
        self.device = torch.device("cuda", device)
        seqlens = [self.cu[b + 1] - self.cu[b] for b in range(self.B)]
        self.handle = fc_create(device, max(1, max(seqlens) if seqlens else 1))
        if group_bytes:
            fc_set_group_bytes(self.handle, group_bytes)
        # compress() issues select x L back to back after score x L and allocate: the documented case
        fc_set_select_overlap(self.handle, select_overlap)
        # score x L is followed by allocate (which joins the internal streams) before anything reads the scores
        fc_set_score_overlap(self.handle, score_overlap)
        dev = self.device
        self.scores = torch.empty((self.L, self.H, max(self.T, 1)), dtype=torch.float32, device=dev)
        self.energy = torch.empty((self.L, self.B, 4), dtype=torch.float64, device=dev)
        self.budgets = torch.empty((self.L, self.B), dtype=torch.int32, device=dev)
        self.offsets = torch.empty((self.L, self.B + 1), dtype=torch.int64, device=dev)
        # rows any one layer can receive (the library's own bound)
        self.capacity = max(fc_layer_capacity_rows(self.L, self.cu, self.rho, self.min_keep), 1)
        self.out_k = None
        self.out_v = None
        self.out_idx = None
        self._ws = None

    def close(self):
        if self.handle is not None:
            fc_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _workspace(self, k, v):
        need = max(fc_score_workspace_bytes(self.handle, k, v, self.cu),
                   fc_select_workspace_bytes(self.handle, k, v, self.cu))
        if need == 0:
            raise FlashCacheError(1, "fc_score_workspace_bytes")
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=self.device)
        return self._ws

    def _outputs(self, per_layer_capacity: int):
        if self.out_k is None or self.out_k.shape[1] < per_layer_capacity:
            dev = self.device
            self.out_k = torch.empty((self.L, per_layer_capacity, self.H, self.d), dtype=self.dtype, device=dev)
            self.out_v = torch.empty_like(self.out_k)
            self.out_idx = torch.empty((self.L, self.H, per_layer_capacity), dtype=torch.int32, device=dev)

    # The per-layer calls below go straight to the C entry points with arguments that are marshalled
    # once per set of tensors (views, pointers, the cu_seqlens array): the per-call Python work would
    # otherwise cost more than the selection kernels it launches.
    def _marshal(self, K_layers, V_layers):
        key = tuple(k.data_ptr() for k in K_layers) + tuple(v.data_ptr() for v in V_layers)
        if getattr(self, "_mkey", None) == key and self._m_out == (id(self.out_k), id(self._ws)):
            return self._m
        ws = self._workspace(K_layers[0], V_layers[0])
        self._outputs(self.capacity)
        cu = _cu_array(self.cu)
        views = [make_view(K_layers[l], V_layers[l], cu) for l in range(self.L)]
        P = c_void_p
        m = dict(
            cu=cu, views=views, refs=[byref(v) for v in views],
            ws=P(ws.data_ptr()), ws_bytes=ws.numel(),
            scores=[P(self.scores[l].data_ptr()) for l in range(self.L)],
            energy=[P(self.energy[l].data_ptr()) for l in range(self.L)],
            budgets=[P(self.budgets[l].data_ptr()) for l in range(self.L)],
            offsets=[P(self.offsets[l].data_ptr()) for l in range(self.L)],
            out_k=[P(self.out_k[l].data_ptr()) for l in range(self.L)],
            out_v=[P(self.out_v[l].data_ptr()) for l in range(self.L)],
            out_idx=[P(self.out_idx[l].data_ptr()) for l in range(self.L)],
            cap=int(self.out_k.shape[1]))
        tab = (fc_layer_buffers * self.L)()
        for l in range(self.L):
            tab[l] = fc_layer_buffers(K_layers[l].data_ptr(), V_layers[l].data_ptr(), self.scores[l].data_ptr(),
                                      self.out_k[l].data_ptr(), self.out_v[l].data_ptr(),
                                      self.out_idx[l].data_ptr(), m["cap"])
        m["layers"] = tab
        self._m, self._mkey, self._m_out = m, key, (id(self.out_k), id(self._ws))
        return m

    def score(self, K_layers, V_layers):
        m = self._marshal(K_layers, V_layers)
        st, h, gamma = _stream(), self.handle, c_double(self.gamma)
        call = _lib.fc_score_layer
        for l in range(self.L):
            rc = call(h, m["refs"][l], gamma, m["scores"][l], m["energy"][l], m["ws"], m["ws_bytes"], st)
            if rc != FC_OK:
                raise FlashCacheError(rc, "fc_score_layer")

    def allocate(self):
        fc_allocate_budgets(self.handle, self.energy, self.cu, self.rho, self.min_keep,
                            self.budgets, self.offsets)

    def select_compact(self, K_layers, V_layers, one_launch: bool = True):
        m = self._marshal(K_layers, V_layers)
        st, h = _stream(), self.handle
        opt = byref(self._opt)
        if one_launch:         # every layer side by side (fc_select_compact_layers)
            rc = _lib.fc_select_compact_layers(h, m["refs"][0], m["layers"], self.L, c_void_p(self.budgets.data_ptr()),
                                               c_void_p(self.offsets.data_ptr()), opt, m["ws"], m["ws_bytes"], st)
            if rc != FC_OK:
                raise FlashCacheError(rc, "fc_select_compact_layers")
            return
        call = _lib.fc_select_compact_ex
        for l in range(self.L):
            rc = call(h, m["refs"][l], m["scores"][l], m["budgets"][l], m["offsets"][l], m["out_k"][l],
                      m["out_v"][l], m["out_idx"][l], m["cap"], opt, m["ws"], m["ws_bytes"], st)
            if rc != FC_OK:
                raise FlashCacheError(rc, "fc_select_compact_ex")

    def compress(self, K_layers, V_layers):
        self.score(K_layers, V_layers)
        self.allocate()
        self.select_compact(K_layers, V_layers)

    def capture(self, K_layers, V_layers):
        """The whole `compress` sequence on these tensors as a CUDA graph (torch.cuda.CUDAGraph): one
        warm-up pass, then a capture on a side stream.  `replay()` reruns it on the tensors' current
        contents; results land in the same buffers as `compress`.  Worth it for short sequences, where
        the launches cost more than the kernels."""
        self.compress(K_layers, V_layers)
        torch.cuda.synchronize(self.device)
        self.check_device_status()
        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream(device=self.device)
        side.wait_stream(torch.cuda.current_stream(self.device))
        fc_reset_ordering(self.handle)
        try:
            # only this thread's calls belong to the capture (a collective library's watchdog thread may query events meanwhile)
            with torch.cuda.graph(graph, stream=side, capture_error_mode="thread_local"):
                self.compress(K_layers, V_layers)
        finally:
            fc_reset_ordering(self.handle)
        return graph

    def check_device_status(self):
        _check(fc_last_device_status(self.handle), "device status")


class HostResult:
    """Page-locked host buffers one fc_compress_host call fills (layout: include/flashcache.h)."""

    def __init__(self, num_layers: int, num_heads: int, head_dim: int, batch: int, rows: int, dtype):
        rows = max(int(rows), 1)
        self.out_k = torch.empty((rows, num_heads, head_dim), dtype=dtype).pin_memory()
        self.out_v = torch.empty((rows, num_heads, head_dim), dtype=dtype).pin_memory()
        self.out_idx = torch.empty((rows * num_heads,), dtype=torch.int32).pin_memory()
        self._budgets_store = torch.zeros((num_layers * max(batch, 1),), dtype=torch.int32)
        self.budgets = self._budgets_store[:num_layers * batch].view(num_layers, batch)
        self.offsets = torch.zeros((num_layers, batch + 1), dtype=torch.int64)
        self.layer_rows = torch.zeros((num_layers + 1,), dtype=torch.int64)
        self.capacity = rows
        self.num_heads = num_heads

    def layer(self, l: int):
        """(K rows, V rows, indices [H, r]) of layer l; call after the stream has been synchronised."""
        r0, r1 = int(self.layer_rows[l]), int(self.layer_rows[l + 1])
        H = self.num_heads
        return self.out_k[r0:r1], self.out_v[r0:r1], self.out_idx[H * r0:H * r1].view(H, r1 - r0)


class HostCompressor:
    """fc_compress_host for one workload shape: owns the handle and the device arena; `compress`
    takes per-layer HOST tensors [T, H, d] (page-locked for overlap) and enqueues the whole path on
    the current stream.  Two HostResult objects used in turn let the copies back of one call overlap
    the copies in of the next."""

    def __init__(self, num_layers: int, num_heads: int, head_dim: int, cu_seqlens, dtype, rho: float,
                 gamma: float = 0.2, min_keep: int = 1, device: int = 0, per_layer: bool = False, protect=None):
        self.L, self.H, self.d = int(num_layers), int(num_heads), int(head_dim)
        # selection options: one index set per layer; protect = uint8 [T] HOST tensor of tokens that must survive
        self.per_layer, self.protect = bool(per_layer), protect
        self.cu = [int(x) for x in cu_seqlens]
        self.B = len(self.cu) - 1
        self.T = self.cu[-1]
        self.rho, self.gamma, self.min_keep = float(rho), float(gamma), int(min_keep)
        self.dtype = dtype
        self.device = torch.device("cuda", device)
        seqlens = [self.cu[b + 1] - self.cu[b] for b in range(self.B)]
        self.handle = fc_create(device, max(1, max(seqlens) if seqlens else 1))
        self.rows = fc_compress_host_rows(self.L, self.cu, self.rho, self.min_keep)
        self._cu = _cu_array(self.cu)
        self._kptr = (c_void_p * self.L)()
        self._vptr = (c_void_p * self.L)()
        self._job = fc_host_job(
            k_host=ctypes.cast(self._kptr, POINTER(c_void_p)), v_host=ctypes.cast(self._vptr, POINTER(c_void_p)),
            num_layers=self.L, dtype=_DTYPE[dtype], num_heads=self.H, head_dim=self.d, batch=self.B,
            min_keep=self.min_keep, cu_seqlens=ctypes.cast(self._cu, POINTER(c_int32)),
            gamma=self.gamma, rho=self.rho, per_layer=1 if per_layer else 0,
            protect_host=protect.data_ptr() if protect is not None else None)
        if protect is not None and (protect.is_cuda or protect.dtype != torch.uint8 or protect.numel() != self.T
                                    or not protect.is_contiguous()):
            raise ValueError("protect: contiguous uint8 host tensor with one entry per token")
        need = int(_lib.fc_compress_host_arena_bytes(self.handle, byref(self._job)))
        if need == 0:
            raise FlashCacheError(2, "fc_compress_host_arena_bytes")
        self.arena = torch.empty(need, dtype=torch.uint8, device=self.device)
        self._job.arena = self.arena.data_ptr()
        self._job.arena_bytes = need

    def new_result(self) -> HostResult:
        return HostResult(self.L, self.H, self.d, self.B, self.rows, self.dtype)

    def compress(self, K_layers, V_layers, result: HostResult) -> None:
        if len(K_layers) != self.L or len(V_layers) != self.L:
            raise ValueError("one K and one V tensor per layer")
        for l in range(self.L):
            k, v = K_layers[l], V_layers[l]
            if k.is_cuda or v.is_cuda or not k.is_contiguous() or not v.is_contiguous() or k.dtype != self.dtype \
                    or v.dtype != self.dtype or tuple(k.shape) != (self.T, self.H, self.d) or k.shape != v.shape:
                raise ValueError("layer %d: expected contiguous host tensors [T, H, d] of the compressor's dtype" % l)
            self._kptr[l] = k.data_ptr()
            self._vptr[l] = v.data_ptr()
        j = self._job
        j.out_k_host, j.out_v_host, j.out_idx_host = result.out_k.data_ptr(), result.out_v.data_ptr(), result.out_idx.data_ptr()
        j.out_capacity_rows = result.capacity
        j.budgets_host, j.offsets_host = result._budgets_store.data_ptr(), result.offsets.data_ptr()
        j.layer_rows_host = result.layer_rows.data_ptr()
        _check(_lib.fc_compress_host(self.handle, byref(j), _stream()), "fc_compress_host")

    def check_device_status(self):
        _check(fc_last_device_status(self.handle), "device status")

    def close(self):
        if self.handle is not None:
            fc_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
