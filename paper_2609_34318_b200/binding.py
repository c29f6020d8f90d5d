"""ctypes binding of libhydra_attn.so: same names as the C ABI, argument marshalling only.

Every step of the path runs in the library's CUDA kernels; there is no Python or CPU fallback.
If the shared library is missing it is built with nvcc; if that fails, importing raises.
Tensors are torch CUDA tensors (used for device memory and streams only) or raw device pointers.
"""
from __future__ import annotations

import ctypes
import os
from typing import Iterable, Optional, Sequence, Tuple

import numpy as np

from . import build as _build

D_QK = 192
D_V = 128

HYDRA_OK = 0
HYDRA_ERR_INVALID_ARG = 1
HYDRA_ERR_UNSUPPORTED = 2
HYDRA_ERR_WORKSPACE_TOO_SMALL = 3
HYDRA_ERR_CUDA = 4
HYDRA_ERR_DEVICE_TIMEOUT = 5
HYDRA_ERR_NOT_SM100 = 6
HYDRA_WS_FWD, HYDRA_WS_MERGE, HYDRA_WS_BWD = 0, 1, 2


class hydra_pair_t(ctypes.Structure):
    _fields_ = [("seq", ctypes.c_int32), ("q_start", ctypes.c_int32), ("q_len", ctypes.c_int32),
                ("k_start", ctypes.c_int32), ("k_len", ctypes.c_int32), ("part_row", ctypes.c_int32),
                ("group", ctypes.c_int32), ("flags", ctypes.c_int32)]


PAIR_DTYPE = np.dtype([("seq", "<i4"), ("q_start", "<i4"), ("q_len", "<i4"), ("k_start", "<i4"),
                       ("k_len", "<i4"), ("part_row", "<i4"), ("group", "<i4"), ("flags", "<i4")])


CHUNK_DTYPE = np.dtype([("seq", "<i4"), ("start", "<i4"), ("len", "<i4"), ("row", "<i4")])


def as_chunks(chunks) -> np.ndarray:
    """A chunk table (include/hydra_attn.h, hydra_chunk_t): structured array, or an iterable of (seq, start, len, row)."""
    if isinstance(chunks, np.ndarray) and chunks.dtype == CHUNK_DTYPE:
        return np.ascontiguousarray(chunks)
    out = np.zeros(len(chunks), dtype=CHUNK_DTYPE)
    for i, c in enumerate(chunks):
        out[i] = tuple(c[n] for n in ("seq", "start", "len", "row")) if isinstance(c, dict) else tuple(c)
    return out


class HydraError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {hydra_status_string(status)} ({status})")


def _load() -> ctypes.CDLL:
    path = _build.build(force=bool(os.environ.get("HYDRA_REBUILD")))   # no-op when up to date
    lib = ctypes.CDLL(path)
    i32, i64, vp, f32 = ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p, ctypes.c_float
    sz = ctypes.c_size_t
    lib.hydra_version.restype = i32
    lib.hydra_status_string.restype = ctypes.c_char_p
    lib.hydra_status_string.argtypes = [i32]
    lib.hydra_launch_count.restype = i64
    lib.hydra_set_wait_limit_ns.argtypes = [ctypes.c_uint64]
    lib.hydra_set_wait_limit_ns.restype = None
    lib.hydra_debug_stall.argtypes = [i32, ctypes.c_uint64]
    lib.hydra_debug_stall.restype = None
    lib.hydra_shutdown.restype = None
    lib.hydra_set_plan_arena_bytes.argtypes = [ctypes.c_uint64]
    lib.hydra_set_plan_arena_bytes.restype = None
    lib.hydra_plan_build_seconds.restype = ctypes.c_double
    lib.hydra_plan_build_seconds.argtypes = [i32, vp, i32, i32, vp, i32, i32]
    lib.hydra_set_plan_prefetch.argtypes = [i32]
    lib.hydra_set_plan_prefetch.restype = None
    lib.hydra_set_fwd_short_len.argtypes = [i32]
    lib.hydra_set_fwd_short_len.restype = None
    lib.hydra_usp_factor.restype = i32
    lib.hydra_usp_factor.argtypes = [i32, i32, vp, vp]
    lib.hydra_zigzag_pairs.restype = i32
    lib.hydra_zigzag_pairs.argtypes = [vp, i32, vp, i32, vp, i32, vp, vp, vp, vp]
    for name in ("hydra_ulysses_pack", "hydra_ulysses_unpack"):
        fn = getattr(lib, name)
        fn.restype = i32
        fn.argtypes = [vp, ctypes.c_int64, i32, i32, i32, vp, vp]
    lib.hydra_bwd_bands.restype = i32
    lib.hydra_bwd_bands.argtypes = [vp, i32, i32, vp, i32, i32, ctypes.c_uint64, vp, vp, i32, vp, vp]
    lib.hydra_workspace_bytes.restype = sz
    lib.hydra_workspace_bytes.argtypes = [i32, vp, i32, i32, vp, i32]
    lib.hydra_attn_fwd.restype = i32
    lib.hydra_attn_fwd.argtypes = [vp, vp, vp, vp, i32, i32, vp, i32, i32, f32, vp, vp, vp, vp, i64,
                                   vp, sz, vp]
    lib.hydra_lse_merge.restype = i32
    lib.hydra_lse_merge.argtypes = [vp, vp, i64, vp, i32, i32, vp, i32, vp, vp, vp, sz, vp]
    f64 = ctypes.c_double
    lib.hydra_sched_targets.restype = i32
    lib.hydra_sched_targets.argtypes = [vp, i32, i32, i64, i32, f64, vp]
    lib.hydra_sched_cp.restype = i32
    lib.hydra_sched_cp.argtypes = [i64, i64, i32, i64]
    lib.hydra_sched_pack.restype = i32
    lib.hydra_sched_pack.argtypes = [vp, i32, i32, i64, i32, vp, vp, vp, vp]
    lib.hydra_lse_merge_accumulate.restype = i32
    lib.hydra_lse_merge_accumulate.argtypes = [vp, vp, i64, vp, i32, i32, vp, i32, vp, vp, vp, sz, vp]
    lib.hydra_attn_bwd.restype = i32
    lib.hydra_attn_bwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, vp, i32, i32, f32, vp, vp, vp,
                                   vp, sz, vp]
    lib.hydra_set_bwd_scratch_limit.restype = None
    lib.hydra_set_bwd_scratch_limit.argtypes = [ctypes.c_uint64]
    lib.hydra_set_bwd_band_scratch.restype = None
    lib.hydra_set_bwd_band_scratch.argtypes = [ctypes.c_uint64]
    lib.hydra_attn_bwd_accumulate.restype = i32
    lib.hydra_attn_bwd_accumulate.argtypes = lib.hydra_attn_bwd.argtypes
    lib.hydra_attn_fwd_gqa.restype = i32
    lib.hydra_attn_fwd_gqa.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp, i32, i32, f32, vp, vp, vp, vp, i64,
                                       vp, sz, vp]
    lib.hydra_workspace_bytes_gqa.restype = sz
    lib.hydra_workspace_bytes_gqa.argtypes = [i32, vp, i32, i32, i32, vp, i32]
    lib.hydra_attn_bwd_accumulate_gqa.restype = i32
    a = list(lib.hydra_attn_bwd.argtypes)
    lib.hydra_attn_bwd_accumulate_gqa.argtypes = a[:9] + [i32] + a[9:]
    lib.hydra_attn_bwd_gqa.restype = i32
    lib.hydra_attn_bwd_gqa.argtypes = a[:9] + [i32] + a[9:]
    # the same entry points with the head dimensions as arguments (d_qk, d_v after n_kv_heads)
    lib.hydra_attn_fwd_dims.restype = i32
    f = list(lib.hydra_attn_fwd_gqa.argtypes)
    lib.hydra_attn_fwd_dims.argtypes = f[:7] + [i32, i32] + f[7:]
    lib.hydra_workspace_bytes_dims.restype = sz
    lib.hydra_workspace_bytes_dims.argtypes = [i32, vp, i32, i32, i32, i32, i32, vp, i32]
    g = list(lib.hydra_attn_bwd_gqa.argtypes)
    for name in ("hydra_attn_bwd_dims", "hydra_attn_bwd_accumulate_dims"):
        getattr(lib, name).restype = i32
        getattr(lib, name).argtypes = g[:10] + [i32, i32] + g[10:]
    lib.hydra_grad_cast.restype = i32
    lib.hydra_grad_cast.argtypes = [vp, vp, i64, vp]
    # local layouts (a rank of an outer ring): chunk tables after the head dimensions
    tables = [vp, i32, i64, vp, i32, i64]
    lib.hydra_workspace_bytes_local.restype = sz
    lib.hydra_workspace_bytes_local.argtypes = [i32, vp, i32, i32, i32, i32, i32] + tables + [vp, i32]
    lib.hydra_attn_fwd_local.restype = i32
    lib.hydra_attn_fwd_local.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32] + tables + \
        [vp, i32, i32, f32, vp, vp, vp, vp, i64, vp, sz, vp]
    lib.hydra_lse_merge_local.restype = i32
    lib.hydra_lse_merge_local.argtypes = [vp, vp, i64, vp, i32, i32, vp, i32, i64, vp, i32, i32, vp, vp, vp, sz, vp]
    lib.hydra_attn_bwd_accumulate_local.restype = i32
    lib.hydra_attn_bwd_accumulate_local.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32] + tables + \
        [vp, i32, i32, f32, vp, vp, vp, vp, sz, vp]
    lib.hydra_mla_rope.restype = i32
    lib.hydra_mla_rope.argtypes = [vp, vp, i64, i32, i32, i32, i32, f32, i32, vp, vp]
    for name in ("hydra_mla_kv_assemble", "hydra_mla_kv_assemble_bwd"):
        getattr(lib, name).restype = i32
        getattr(lib, name).argtypes = [vp, vp, vp, i64, i32, i32, i32, i32, f32, vp, vp, vp]
    lib.hydra_gate_apply.restype = i32
    lib.hydra_gate_apply.argtypes = [vp, vp, i64, vp, vp]
    lib.hydra_gate_apply_bwd.restype = i32
    lib.hydra_gate_apply_bwd.argtypes = [vp, vp, vp, i64, vp, vp, vp]
    lib.hydra_poll_status.restype = i32
    lib.hydra_poll_status.argtypes = [vp, vp, vp, vp]
    lib.hydra_poll_clocks.restype = i32
    lib.hydra_poll_clocks.argtypes = [vp, vp, vp]
    lib.hydra_profile_enable.restype = None
    lib.hydra_profile_enable.argtypes = [i32]
    lib.hydra_profile_collect.restype = i32
    lib.hydra_profile_collect.argtypes = [vp, vp]
    lib.hydra_host_step_arena_bytes.restype = sz
    lib.hydra_host_step_arena_bytes.argtypes = [vp, i32, i32, vp, i32]
    lib.hydra_lse_merge_noalloc.restype = i32
    lib.hydra_lse_merge_noalloc.argtypes = [vp, vp, i64, vp, i32, i32, vp, i32, vp, vp, vp]
    lib.hydra_attn_fwd_bwd_host.restype = i32
    lib.hydra_attn_fwd_bwd_host.argtypes = [vp, vp, vp, vp, vp, i32, i32, vp, i32, i32, f32, vp, vp, vp, vp,
                                            vp, vp, sz, vp]
    return lib


_lib = _load()
LIBRARY_PATH = _build.OUT
EXPORTS = ("hydra_version", "hydra_status_string", "hydra_launch_count", "hydra_set_wait_limit_ns", "hydra_debug_stall", "hydra_set_plan_arena_bytes", "hydra_set_plan_prefetch", "hydra_set_fwd_short_len", "hydra_plan_build_seconds",
           "hydra_shutdown", "hydra_usp_factor", "hydra_zigzag_pairs", "hydra_workspace_bytes",
           "hydra_attn_fwd", "hydra_lse_merge", "hydra_attn_bwd", "hydra_poll_status",
           "hydra_profile_enable", "hydra_profile_collect", "hydra_host_step_arena_bytes",
           "hydra_attn_fwd_bwd_host", "hydra_lse_merge_noalloc", "hydra_lse_merge_accumulate",
           "hydra_sched_targets", "hydra_sched_cp", "hydra_sched_pack", "hydra_attn_bwd_accumulate",
           "hydra_grad_cast", "hydra_set_bwd_scratch_limit", "hydra_set_bwd_band_scratch", "hydra_bwd_bands", "hydra_ulysses_pack", "hydra_ulysses_unpack", "hydra_attn_fwd_gqa", "hydra_attn_bwd_accumulate_gqa", "hydra_attn_bwd_gqa", "hydra_workspace_bytes_gqa",
           "hydra_mla_rope", "hydra_mla_kv_assemble", "hydra_mla_kv_assemble_bwd", "hydra_gate_apply", "hydra_gate_apply_bwd",
           "hydra_attn_fwd_local", "hydra_lse_merge_local", "hydra_attn_bwd_accumulate_local", "hydra_workspace_bytes_local",
           "hydra_attn_fwd_dims", "hydra_attn_bwd_dims", "hydra_attn_bwd_accumulate_dims", "hydra_workspace_bytes_dims",
           "hydra_poll_clocks")
KERNEL_KINDS = ("fwd", "merge", "bwd_prep", "bwd_dkv", "bwd_dq", "grad_cast", "ulysses", "mla_ops")


# ------------------------------------------------------------------------------------------------
# marshalling helpers
# ------------------------------------------------------------------------------------------------
def _ptr(x) -> Optional[int]:
    """Device pointer of a torch tensor, or the integer / None passed through."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if not x.is_cuda or not x.is_contiguous():
        raise ValueError("tensors must be contiguous CUDA tensors")
    return x.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _cu(cu_seqlens) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int32))


def as_pairs(pairs) -> Optional[np.ndarray]:
    """Accepts None, a structured array of PAIR_DTYPE, or an iterable of dicts / tuples."""
    if pairs is None:
        return None
    if isinstance(pairs, np.ndarray) and pairs.dtype == PAIR_DTYPE:
        return np.ascontiguousarray(pairs)
    out = np.zeros(len(pairs), dtype=PAIR_DTYPE)
    for i, p in enumerate(pairs):
        if isinstance(p, dict):
            for name in ("seq", "q_start", "q_len", "k_start", "k_len", "group"):
                out[i][name] = p[name]
            out[i]["part_row"] = p.get("part_row", -1)
            out[i]["flags"] = p.get("flags", 0)
        else:
            out[i] = tuple(p)
    return out


def _pairs_arg(pairs) -> Tuple[Optional[int], int, Optional[np.ndarray]]:
    arr = as_pairs(pairs)
    if arr is None:
        return None, 0, None
    return arr.ctypes.data, len(arr), arr


def _check(status: int, where: str) -> None:
    if status != HYDRA_OK:
        raise HydraError(status, where)


# ------------------------------------------------------------------------------------------------
# the C ABI, one Python function per entry point
# ------------------------------------------------------------------------------------------------
def hydra_version() -> int:
    return int(_lib.hydra_version())


def hydra_status_string(status: int) -> str:
    return _lib.hydra_status_string(int(status)).decode()


def hydra_launch_count() -> int:
    return int(_lib.hydra_launch_count())


def hydra_set_wait_limit_ns(ns: int) -> None:
    _lib.hydra_set_wait_limit_ns(int(ns))


HYDRA_STALL_FWD, HYDRA_STALL_BWD_DKV, HYDRA_STALL_BWD_DQ = 0, 1, 2


def hydra_debug_stall(kernel: int, ns: int) -> None:
    """Test hook: the work-issuing thread of every thread block of `kernel` idles for `ns` (at most 20 ms) and
    then issues nothing, so that the bounded waits of the other roles run out (0 switches it off)."""
    _lib.hydra_debug_stall(int(kernel), int(ns))


def hydra_shutdown() -> None:
    _lib.hydra_shutdown()


def hydra_plan_build_seconds(which: int, cu_seqlens, n_heads: int, pairs=None, causal: bool = True) -> float:
    """Host-only: seconds to build the (uncached) work tables of one call of kind `which` for this problem."""
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    return float(_lib.hydra_plan_build_seconds(which, cu.ctypes.data, len(cu) - 1, n_heads, pp, npairs, int(bool(causal))))


def hydra_set_plan_prefetch(on: bool) -> None:
    """Build the merge / backward tables of a problem on the host while its forward runs (default on)."""
    _lib.hydra_set_plan_prefetch(int(bool(on)))


def hydra_set_fwd_short_len(length: int) -> None:
    """Pairs with q and kv ranges of at most `length` tokens use the short-sequence forward kernel (0: off;
    negative, the default: 2048, or 4608 with shared K / V heads or heads of 128)."""
    _lib.hydra_set_fwd_short_len(int(length))


def hydra_set_plan_arena_bytes(nbytes: int) -> None:
    """Size of the per-device arena that holds the work tables (used by the next first call on a device, or
    the first call after hydra_shutdown)."""
    _lib.hydra_set_plan_arena_bytes(int(nbytes))


def hydra_usp_factor(degree: int, heads: int) -> Tuple[int, int]:
    u, r = ctypes.c_int32(0), ctypes.c_int32(0)
    _check(_lib.hydra_usp_factor(degree, heads, ctypes.addressof(u), ctypes.addressof(r)),
           "hydra_usp_factor")
    return u.value, r.value


def hydra_zigzag_pairs(cu_seqlens, cp_r):
    """Returns (pairs structured array, part_rows, rank array, step array)."""
    cu = _cu(cu_seqlens)
    n = len(cu) - 1
    per_seq = None if isinstance(cp_r, (int, np.integer)) else np.ascontiguousarray(cp_r, dtype=np.int32)
    all_r = int(cp_r) if per_seq is None else 0
    n_pairs, part_rows = ctypes.c_int32(0), ctypes.c_int64(0)
    s = _lib.hydra_zigzag_pairs(cu.ctypes.data, n, None if per_seq is None else per_seq.ctypes.data, all_r,
                                None, 0, ctypes.addressof(n_pairs), ctypes.addressof(part_rows), None, None)
    if s not in (HYDRA_OK, HYDRA_ERR_WORKSPACE_TOO_SMALL):
        raise HydraError(s, "hydra_zigzag_pairs")
    pairs = np.zeros(n_pairs.value, dtype=PAIR_DTYPE)
    rank = np.zeros(n_pairs.value, dtype=np.int32)
    step = np.zeros(n_pairs.value, dtype=np.int32)
    if n_pairs.value:
        _check(_lib.hydra_zigzag_pairs(cu.ctypes.data, n, None if per_seq is None else per_seq.ctypes.data,
                                       all_r, pairs.ctypes.data, len(pairs), ctypes.addressof(n_pairs),
                                       ctypes.addressof(part_rows), rank.ctypes.data, step.ctypes.data),
               "hydra_zigzag_pairs")
    return pairs, int(part_rows.value), rank, step


def hydra_bwd_bands(cu_seqlens, n_heads: int, pairs, causal: bool, scratch_bytes: int):
    """Returns (clipped pairs of all bands, band index of each, number of bands); host only."""
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    n_out, n_bands = ctypes.c_int32(0), ctypes.c_int32(0)
    args = (cu.ctypes.data, len(cu) - 1, n_heads, pp, npairs, int(bool(causal)), int(scratch_bytes))
    s = _lib.hydra_bwd_bands(*args, None, None, 0, ctypes.addressof(n_out), ctypes.addressof(n_bands))
    if s not in (HYDRA_OK, HYDRA_ERR_WORKSPACE_TOO_SMALL):
        raise HydraError(s, "hydra_bwd_bands")
    out = np.zeros(n_out.value, dtype=PAIR_DTYPE)
    band = np.zeros(n_out.value, dtype=np.int32)
    if n_out.value:
        _check(_lib.hydra_bwd_bands(*args, out.ctypes.data, band.ctypes.data, len(out), ctypes.addressof(n_out),
                                    ctypes.addressof(n_bands)), "hydra_bwd_bands")
    return out, band, int(n_bands.value)


def hydra_workspace_bytes(which: int, cu_seqlens, n_heads: int, pairs=None) -> int:
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    return int(_lib.hydra_workspace_bytes(which, cu.ctypes.data, len(cu) - 1, n_heads, pp, npairs))


def hydra_attn_fwd(q, k, v, cu_seqlens, n_heads: int, pairs, causal: bool, softmax_scale: float, out, lse,
                   o_part, lse_part, part_rows: int, workspace, workspace_bytes: Optional[int] = None,
                   stream=None, check: bool = True) -> int:
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    s = _lib.hydra_attn_fwd(_ptr(q), _ptr(k), _ptr(v), cu.ctypes.data, len(cu) - 1, n_heads, pp, npairs,
                            int(bool(causal)), ctypes.c_float(float(softmax_scale)), _ptr(out), _ptr(lse),
                            _ptr(o_part), _ptr(lse_part), int(part_rows), _ptr(workspace),
                            int(workspace_bytes), _stream(stream))
    if check:
        _check(s, "hydra_attn_fwd")
    return s


def hydra_lse_merge(o_part, lse_part, part_rows: int, cu_seqlens, n_heads: int, pairs, out, lse, workspace,
                    workspace_bytes: Optional[int] = None, stream=None, check: bool = True) -> int:
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    s = _lib.hydra_lse_merge(_ptr(o_part), _ptr(lse_part), int(part_rows), cu.ctypes.data, len(cu) - 1,
                             n_heads, pp, npairs, _ptr(out), _ptr(lse), _ptr(workspace),
                             int(workspace_bytes), _stream(stream))
    if check:
        _check(s, "hydra_lse_merge")
    return s


def hydra_lse_merge_accumulate(o_part, lse_part, part_rows: int, cu_seqlens, n_heads: int, pairs, out, lse,
                               workspace, workspace_bytes: Optional[int] = None, stream=None,
                               check: bool = True) -> int:
    """Streaming merge of one ring step: folds the listed partials into the running (out, lse)."""
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    s = _lib.hydra_lse_merge_accumulate(_ptr(o_part), _ptr(lse_part), int(part_rows), cu.ctypes.data,
                                        len(cu) - 1, n_heads, pp, npairs, _ptr(out), _ptr(lse), _ptr(workspace),
                                        int(workspace_bytes), _stream(stream))
    if check:
        _check(s, "hydra_lse_merge_accumulate")
    return s


def hydra_attn_bwd(q, k, v, out, lse, dout, cu_seqlens, n_heads: int, pairs, causal: bool,
                   softmax_scale: float, dq, dk, dv, workspace, workspace_bytes: Optional[int] = None,
                   stream=None, check: bool = True) -> int:
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    s = _lib.hydra_attn_bwd(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), _ptr(dout), cu.ctypes.data,
                            len(cu) - 1, n_heads, pp, npairs, int(bool(causal)),
                            ctypes.c_float(float(softmax_scale)), _ptr(dq), _ptr(dk), _ptr(dv),
                            _ptr(workspace), int(workspace_bytes), _stream(stream))
    if check:
        _check(s, "hydra_attn_bwd")
    return s


def hydra_attn_bwd_accumulate(q, k, v, out, lse, dout, cu_seqlens, n_heads: int, pairs, causal: bool,
                              softmax_scale: float, dq_acc, dk_acc, dv_acc, workspace,
                              workspace_bytes: Optional[int] = None, stream=None, check: bool = True) -> int:
    """Backward of the listed pairs added to fp32 accumulators (one ring step at a time)."""
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    s = _lib.hydra_attn_bwd_accumulate(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), _ptr(dout),
                                       cu.ctypes.data, len(cu) - 1, n_heads, pp, npairs, int(bool(causal)),
                                       ctypes.c_float(float(softmax_scale)), _ptr(dq_acc), _ptr(dk_acc),
                                       _ptr(dv_acc), _ptr(workspace), int(workspace_bytes), _stream(stream))
    if check:
        _check(s, "hydra_attn_bwd_accumulate")
    return s


def hydra_attn_fwd_gqa(q, k, v, cu_seqlens, n_heads: int, n_kv_heads: int, pairs, causal: bool,
                       softmax_scale: float, out, lse, o_part, lse_part, part_rows: int, workspace,
                       workspace_bytes: Optional[int] = None, stream=None, check: bool = True) -> int:
    """hydra_attn_fwd with k, v of n_kv_heads heads: query head a reads KV head a // (n_heads / n_kv_heads)."""
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    s = _lib.hydra_attn_fwd_gqa(_ptr(q), _ptr(k), _ptr(v), cu.ctypes.data, len(cu) - 1, n_heads, n_kv_heads, pp,
                                npairs, int(bool(causal)), ctypes.c_float(float(softmax_scale)), _ptr(out),
                                _ptr(lse), _ptr(o_part), _ptr(lse_part), int(part_rows), _ptr(workspace),
                                int(workspace_bytes), _stream(stream))
    if check:
        _check(s, "hydra_attn_fwd_gqa")
    return s


def hydra_workspace_bytes_gqa(which: int, cu_seqlens, n_heads: int, n_kv_heads: int, pairs=None) -> int:
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    return int(_lib.hydra_workspace_bytes_gqa(which, cu.ctypes.data, len(cu) - 1, n_heads, n_kv_heads, pp, npairs))


def hydra_attn_bwd_gqa(q, k, v, out, lse, dout, cu_seqlens, n_heads: int, n_kv_heads: int, pairs, causal: bool,
                       softmax_scale: float, dq, dk, dv, workspace, workspace_bytes: Optional[int] = None,
                       stream=None, check: bool = True) -> int:
    """hydra_attn_bwd with shared KV heads: dk, dv (bf16) have n_kv_heads heads."""
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    s = _lib.hydra_attn_bwd_gqa(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), _ptr(dout), cu.ctypes.data,
                                len(cu) - 1, n_heads, n_kv_heads, pp, npairs, int(bool(causal)),
                                ctypes.c_float(float(softmax_scale)), _ptr(dq), _ptr(dk), _ptr(dv),
                                _ptr(workspace), int(workspace_bytes), _stream(stream))
    if check:
        _check(s, "hydra_attn_bwd_gqa")
    return s


def hydra_attn_bwd_accumulate_gqa(q, k, v, out, lse, dout, cu_seqlens, n_heads: int, n_kv_heads: int, pairs,
                                  causal: bool, softmax_scale: float, dq_acc, dk_acc, dv_acc, workspace,
                                  workspace_bytes: Optional[int] = None, stream=None, check: bool = True) -> int:
    """hydra_attn_bwd_accumulate with shared KV heads: dk_acc, dv_acc have n_kv_heads heads."""
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    s = _lib.hydra_attn_bwd_accumulate_gqa(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), _ptr(dout),
                                           cu.ctypes.data, len(cu) - 1, n_heads, n_kv_heads, pp, npairs,
                                           int(bool(causal)), ctypes.c_float(float(softmax_scale)), _ptr(dq_acc),
                                           _ptr(dk_acc), _ptr(dv_acc), _ptr(workspace), int(workspace_bytes),
                                           _stream(stream))
    if check:
        _check(s, "hydra_attn_bwd_accumulate_gqa")
    return s


def hydra_workspace_bytes_dims(which: int, cu_seqlens, n_heads: int, n_kv_heads: int, d_qk: int, d_v: int,
                               pairs=None) -> int:
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    return int(_lib.hydra_workspace_bytes_dims(which, cu.ctypes.data, len(cu) - 1, n_heads, n_kv_heads, int(d_qk),
                                               int(d_v), pp, npairs))


def hydra_attn_fwd_dims(q, k, v, cu_seqlens, n_heads: int, n_kv_heads: int, d_qk: int, d_v: int, pairs, causal: bool,
                        softmax_scale: float, out, lse, o_part, lse_part, part_rows: int, workspace,
                        workspace_bytes: Optional[int] = None, stream=None, check: bool = True) -> int:
    """hydra_attn_fwd_gqa with the head dimensions as arguments: (192, 128) or (128, 128)."""
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    s = _lib.hydra_attn_fwd_dims(_ptr(q), _ptr(k), _ptr(v), cu.ctypes.data, len(cu) - 1, n_heads, n_kv_heads,
                                 int(d_qk), int(d_v), pp, npairs, int(bool(causal)),
                                 ctypes.c_float(float(softmax_scale)), _ptr(out), _ptr(lse), _ptr(o_part),
                                 _ptr(lse_part), int(part_rows), _ptr(workspace), int(workspace_bytes),
                                 _stream(stream))
    if check:
        _check(s, "hydra_attn_fwd_dims")
    return s


def _bwd_dims(fn_name, q, k, v, out, lse, dout, cu_seqlens, n_heads, n_kv_heads, d_qk, d_v, pairs, causal,
              softmax_scale, dq, dk, dv, workspace, workspace_bytes, stream, check):
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    s = getattr(_lib, fn_name)(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), _ptr(dout), cu.ctypes.data,
                               len(cu) - 1, n_heads, n_kv_heads, int(d_qk), int(d_v), pp, npairs,
                               int(bool(causal)), ctypes.c_float(float(softmax_scale)), _ptr(dq), _ptr(dk),
                               _ptr(dv), _ptr(workspace), int(workspace_bytes), _stream(stream))
    if check:
        _check(s, fn_name)
    return s


def hydra_attn_bwd_dims(q, k, v, out, lse, dout, cu_seqlens, n_heads: int, n_kv_heads: int, d_qk: int, d_v: int,
                        pairs, causal: bool, softmax_scale: float, dq, dk, dv, workspace,
                        workspace_bytes: Optional[int] = None, stream=None, check: bool = True) -> int:
    """hydra_attn_bwd_gqa with the head dimensions as arguments: (192, 128) or (128, 128)."""
    return _bwd_dims("hydra_attn_bwd_dims", q, k, v, out, lse, dout, cu_seqlens, n_heads, n_kv_heads, d_qk, d_v,
                     pairs, causal, softmax_scale, dq, dk, dv, workspace, workspace_bytes, stream, check)


def hydra_attn_bwd_accumulate_dims(q, k, v, out, lse, dout, cu_seqlens, n_heads: int, n_kv_heads: int, d_qk: int,
                                   d_v: int, pairs, causal: bool, softmax_scale: float, dq_acc, dk_acc, dv_acc,
                                   workspace, workspace_bytes: Optional[int] = None, stream=None,
                                   check: bool = True) -> int:
    """hydra_attn_bwd_accumulate_gqa with the head dimensions as arguments: (192, 128) or (128, 128)."""
    return _bwd_dims("hydra_attn_bwd_accumulate_dims", q, k, v, out, lse, dout, cu_seqlens, n_heads, n_kv_heads,
                     d_qk, d_v, pairs, causal, softmax_scale, dq_acc, dk_acc, dv_acc, workspace, workspace_bytes,
                     stream, check)


def hydra_mla_rope(x, positions, n_tokens: int, n_heads: int, head_dim: int, rope_offset: int, rope_dim: int,
                   theta: float, inverse: bool, y, stream=None, check: bool = True) -> int:
    """Rotary embedding of columns [rope_offset, rope_offset + rope_dim) of every head (y may be x)."""
    s = _lib.hydra_mla_rope(_ptr(x), _ptr(positions), int(n_tokens), n_heads, head_dim, rope_offset, rope_dim,
                            ctypes.c_float(float(theta)), int(bool(inverse)), _ptr(y), _stream(stream))
    if check:
        _check(s, "hydra_mla_rope")
    return s


def hydra_mla_kv_assemble(kv_up, k_pe, positions, n_tokens: int, n_heads: int, d_nope: int, d_rope: int, d_v: int,
                          theta: float, k, v, stream=None, check: bool = True) -> int:
    """k = [key part of kv_up | rope(k_pe) shared by all heads], v = value part of kv_up."""
    s = _lib.hydra_mla_kv_assemble(_ptr(kv_up), _ptr(k_pe), _ptr(positions), int(n_tokens), n_heads, d_nope, d_rope,
                                   d_v, ctypes.c_float(float(theta)), _ptr(k), _ptr(v), _stream(stream))
    if check:
        _check(s, "hydra_mla_kv_assemble")
    return s


def hydra_mla_kv_assemble_bwd(dk, dv, positions, n_tokens: int, n_heads: int, d_nope: int, d_rope: int, d_v: int,
                              theta: float, dkv_up, dk_pe, stream=None, check: bool = True) -> int:
    s = _lib.hydra_mla_kv_assemble_bwd(_ptr(dk), _ptr(dv), _ptr(positions), int(n_tokens), n_heads, d_nope, d_rope,
                                       d_v, ctypes.c_float(float(theta)), _ptr(dkv_up), _ptr(dk_pe), _stream(stream))
    if check:
        _check(s, "hydra_mla_kv_assemble_bwd")
    return s


def hydra_gate_apply(out, gate, n_elements: int, y, stream=None, check: bool = True) -> int:
    s = _lib.hydra_gate_apply(_ptr(out), _ptr(gate), int(n_elements), _ptr(y), _stream(stream))
    if check:
        _check(s, "hydra_gate_apply")
    return s


def hydra_gate_apply_bwd(dy, out, gate, n_elements: int, d_out, d_gate, stream=None, check: bool = True) -> int:
    s = _lib.hydra_gate_apply_bwd(_ptr(dy), _ptr(out), _ptr(gate), int(n_elements), _ptr(d_out), _ptr(d_gate),
                                  _stream(stream))
    if check:
        _check(s, "hydra_gate_apply_bwd")
    return s


def _tables(q_chunks, q_rows, kv_chunks, kv_rows):
    qc, kc = as_chunks(q_chunks), as_chunks(kv_chunks)
    return (qc.ctypes.data, len(qc), int(q_rows), kc.ctypes.data, len(kc), int(kv_rows)), (qc, kc)


def hydra_workspace_bytes_local(which: int, cu_seqlens, n_heads: int, n_kv_heads: int, d_qk: int, d_v: int, q_chunks,
                                q_rows: int, kv_chunks, kv_rows: int, pairs) -> int:
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    t, _k2 = _tables(q_chunks, q_rows, kv_chunks, kv_rows)
    return int(_lib.hydra_workspace_bytes_local(which, cu.ctypes.data, len(cu) - 1, n_heads, n_kv_heads, int(d_qk),
                                                int(d_v), *t, pp, npairs))


def hydra_attn_fwd_local(q, k, v, cu_seqlens, n_heads: int, n_kv_heads: int, d_qk: int, d_v: int, q_chunks, q_rows: int,
                         kv_chunks, kv_rows: int, pairs, causal: bool, softmax_scale: float, out, lse, o_part,
                         lse_part, part_rows: int, workspace, workspace_bytes: Optional[int] = None, stream=None,
                         check: bool = True) -> int:
    """Forward of the listed pairs on LOCAL tensors (a rank of an outer ring): chunk tables say where the chunks sit."""
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    t, _k2 = _tables(q_chunks, q_rows, kv_chunks, kv_rows)
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    s = _lib.hydra_attn_fwd_local(_ptr(q), _ptr(k), _ptr(v), cu.ctypes.data, len(cu) - 1, n_heads, n_kv_heads,
                                  int(d_qk), int(d_v), *t, pp, npairs, int(bool(causal)),
                                  ctypes.c_float(float(softmax_scale)), _ptr(out), _ptr(lse), _ptr(o_part),
                                  _ptr(lse_part), int(part_rows), _ptr(workspace), int(workspace_bytes),
                                  _stream(stream))
    if check:
        _check(s, "hydra_attn_fwd_local")
    return s


def hydra_lse_merge_local(o_part, lse_part, part_rows: int, cu_seqlens, n_heads: int, q_chunks, q_rows: int, pairs,
                          accumulate: bool, out, lse, workspace, workspace_bytes: Optional[int] = None, stream=None,
                          check: bool = True) -> int:
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    qc = as_chunks(q_chunks)
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    s = _lib.hydra_lse_merge_local(_ptr(o_part), _ptr(lse_part), int(part_rows), cu.ctypes.data, len(cu) - 1, n_heads,
                                   qc.ctypes.data, len(qc), int(q_rows), pp, npairs, int(bool(accumulate)), _ptr(out),
                                   _ptr(lse), _ptr(workspace), int(workspace_bytes), _stream(stream))
    if check:
        _check(s, "hydra_lse_merge_local")
    return s


def hydra_attn_bwd_accumulate_local(q, k, v, out, lse, dout, cu_seqlens, n_heads: int, n_kv_heads: int, d_qk: int,
                                    d_v: int, q_chunks, q_rows: int, kv_chunks, kv_rows: int, pairs, causal: bool,
                                    softmax_scale: float, dq_acc, dk_acc, dv_acc, workspace,
                                    workspace_bytes: Optional[int] = None, stream=None, check: bool = True) -> int:
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    t, _k2 = _tables(q_chunks, q_rows, kv_chunks, kv_rows)
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    s = _lib.hydra_attn_bwd_accumulate_local(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), _ptr(dout),
                                             cu.ctypes.data, len(cu) - 1, n_heads, n_kv_heads, int(d_qk), int(d_v), *t,
                                             pp, npairs, int(bool(causal)), ctypes.c_float(float(softmax_scale)),
                                             _ptr(dq_acc), _ptr(dk_acc), _ptr(dv_acc), _ptr(workspace),
                                             int(workspace_bytes), _stream(stream))
    if check:
        _check(s, "hydra_attn_bwd_accumulate_local")
    return s


def hydra_set_bwd_scratch_limit(n_bytes: int) -> None:
    """Largest dS hand-off buffer the backward may ask for and use (0: always recompute)."""
    _lib.hydra_set_bwd_scratch_limit(int(n_bytes))


def hydra_ulysses_pack(x, n_tokens: int, n_heads: int, head_dim: int, cp_u: int, send, stream=None,
                       check: bool = True) -> int:
    """send[j, t, b, :] = x[t, j * (n_heads / cp_u) + b, :] (2-byte elements)."""
    s = _lib.hydra_ulysses_pack(_ptr(x), int(n_tokens), int(n_heads), int(head_dim), int(cp_u), _ptr(send),
                                _stream(stream))
    if check:
        _check(s, "hydra_ulysses_pack")
    return s


def hydra_ulysses_unpack(recv, n_tokens: int, n_heads: int, head_dim: int, cp_u: int, y, stream=None,
                         check: bool = True) -> int:
    """y[t, j * (n_heads / cp_u) + b, :] = recv[j, t, b, :] (2-byte elements)."""
    s = _lib.hydra_ulysses_unpack(_ptr(recv), int(n_tokens), int(n_heads), int(head_dim), int(cp_u), _ptr(y),
                                  _stream(stream))
    if check:
        _check(s, "hydra_ulysses_unpack")
    return s


HYDRA_BAND_AUTO = (1 << 64) - 1


def hydra_set_bwd_band_scratch(n_bytes: int) -> None:
    """Scratch for the banded backward of problems whose dS buffer is over the limit (0: off;
    HYDRA_BAND_AUTO, the default: the dS limit, for problems of at most 16 such bands)."""
    _lib.hydra_set_bwd_band_scratch(int(n_bytes))


def hydra_grad_cast(acc, grad, n_elements: Optional[int] = None, stream=None, check: bool = True) -> int:
    """grad (bf16) = acc (fp32), elementwise."""
    if n_elements is None:
        n_elements = acc.numel()
    s = _lib.hydra_grad_cast(_ptr(acc), _ptr(grad), int(n_elements), _stream(stream))
    if check:
        _check(s, "hydra_grad_cast")
    return s


def hydra_poll_status(workspace, stream=None) -> Tuple[int, int]:
    st, detail = ctypes.c_int32(0), ctypes.c_int64(-1)
    _check(_lib.hydra_poll_status(_ptr(workspace), _stream(stream), ctypes.addressof(st),
                                  ctypes.addressof(detail)), "hydra_poll_status")
    return st.value, detail.value


def hydra_poll_clocks(workspace, stream=None) -> Tuple[float, float, float]:
    """SM MHz inside the forward, key-side backward and query-side backward kernels of the last call."""
    mhz = (ctypes.c_double * 3)()
    _check(_lib.hydra_poll_clocks(_ptr(workspace), _stream(stream), ctypes.addressof(mhz)), "hydra_poll_clocks")
    return tuple(mhz)


def hydra_profile_enable(on: bool) -> None:
    _lib.hydra_profile_enable(int(bool(on)))


def hydra_profile_collect():
    """Returns ({kind: total ms}, {kind: launches}) since the last collect."""
    ms = (ctypes.c_double * len(KERNEL_KINDS))()
    n = (ctypes.c_int64 * len(KERNEL_KINDS))()
    _check(_lib.hydra_profile_collect(ctypes.addressof(ms), ctypes.addressof(n)), "hydra_profile_collect")
    return dict(zip(KERNEL_KINDS, list(ms))), dict(zip(KERNEL_KINDS, list(n)))


def hydra_host_step_arena_bytes(cu_seqlens, n_heads: int, pairs=None) -> int:
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    return int(_lib.hydra_host_step_arena_bytes(cu.ctypes.data, len(cu) - 1, n_heads, pp, npairs))


def _host_ptr(x) -> int:
    """Address of a host buffer: a CPU torch tensor (ideally pinned) or a numpy array."""
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        if not x.flags["C_CONTIGUOUS"]:
            raise ValueError("host arrays must be contiguous")
        return x.ctypes.data
    if x.is_cuda or not x.is_contiguous():
        raise ValueError("host buffers must be contiguous CPU tensors")
    return x.data_ptr()


def hydra_attn_fwd_bwd_host(q_host, k_host, v_host, dout_host, cu_seqlens, n_heads: int, pairs, causal: bool,
                            softmax_scale: float, out_host, lse_host, dq_host, dk_host, dv_host, device_arena,
                            arena_bytes: Optional[int] = None, stream=None, check: bool = True) -> int:
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    if arena_bytes is None:
        arena_bytes = device_arena.numel() * device_arena.element_size()
    s = _lib.hydra_attn_fwd_bwd_host(_host_ptr(q_host), _host_ptr(k_host), _host_ptr(v_host),
                                     _host_ptr(dout_host), cu.ctypes.data, len(cu) - 1, n_heads, pp, npairs,
                                     int(bool(causal)), ctypes.c_float(float(softmax_scale)),
                                     _host_ptr(out_host), _host_ptr(lse_host), _host_ptr(dq_host),
                                     _host_ptr(dk_host), _host_ptr(dv_host), _ptr(device_arena),
                                     int(arena_bytes), _stream(stream))
    if check:
        _check(s, "hydra_attn_fwd_bwd_host")
    return s


def hydra_lse_merge_noalloc(o_part, lse_part, part_rows: int, cu_seqlens, n_heads: int, pairs, out, lse,
                            stream=None, check: bool = True) -> int:
    """The merge for callers that must not allocate device memory (own memory pool, no-cudaMalloc
    loops): same result as hydra_lse_merge, tables kept in a fixed array inside the library, no
    workspace. Size limits apply (HYDRA_ERR_UNSUPPORTED beyond them); calls that may overlap on the
    GPU race on that array; make the first call on a device before any stream capture, and never call
    it on a stream that is capturing (refused with HYDRA_ERR_UNSUPPORTED: the tables travel from host
    arrays the next call overwrites). Host-side table building is serialised per process."""
    cu = _cu(cu_seqlens)
    pp, npairs, _keep = _pairs_arg(pairs)
    s = _lib.hydra_lse_merge_noalloc(_ptr(o_part), _ptr(lse_part), int(part_rows), cu.ctypes.data, len(cu) - 1,
                                     n_heads, pp, npairs, _ptr(out), _ptr(lse), _stream(stream))
    if check:
        _check(s, "hydra_lse_merge_noalloc")
    return s


# --------------------------------------------------------------------------------------------------
# scheduler (include/hydra_sched.h): host only
# --------------------------------------------------------------------------------------------------
class SchedTargets(ctypes.Structure):
    _fields_ = [("s_max", ctypes.c_int64), ("W", ctypes.c_double), ("C_mem", ctypes.c_int32),
                ("C_star", ctypes.c_int32), ("C_hat", ctypes.c_double), ("Lambda_star", ctypes.c_double),
                ("M_star", ctypes.c_int64)]


def hydra_sched_targets(lengths, G: int, B: int, pp: int, theta_over_c: float) -> SchedTargets:
    s = np.ascontiguousarray(lengths, dtype=np.int64)
    out = SchedTargets()
    _check(_lib.hydra_sched_targets(s.ctypes.data, len(s), int(G), int(B), int(pp), float(theta_over_c),
                                    ctypes.addressof(out)), "hydra_sched_targets")
    return out


def hydra_sched_cp(s: int, s_max: int, C: int, B: int) -> int:
    return int(_lib.hydra_sched_cp(int(s), int(s_max), int(C), int(B)))


def hydra_sched_pack(lengths, G: int, B: int, C: int, check: bool = True):
    """Returns (mb, rank0, cp, n_mb): micro-batch, first rank and group size of every document."""
    s = np.ascontiguousarray(lengths, dtype=np.int64)
    n = len(s)
    mb, rank0, cp = (np.zeros(max(n, 1), dtype=np.int32) for _ in range(3))
    n_mb = ctypes.c_int32(0)
    st = _lib.hydra_sched_pack(s.ctypes.data, n, int(G), int(B), int(C), mb.ctypes.data, rank0.ctypes.data,
                               cp.ctypes.data, ctypes.addressof(n_mb))
    if check:
        _check(st, "hydra_sched_pack")
    elif st != HYDRA_OK:
        return st
    return mb[:n], rank0[:n], cp[:n], int(n_mb.value)
