"""Thin ctypes binding of libcarnator.so: same names as the C ABI, argument marshalling only.

Every step of the path runs in the library's CUDA kernels.  PyTorch is used here for device
memory (tensors passed in, outputs and workspaces allocated) and for the current stream.
The library is loaded on first use; a missing or unloadable library raises -- there is no
fallback of any kind.
"""
from __future__ import annotations

import ctypes
import math
import os
from typing import Optional

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG_DIR, "libcarnator.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_DEVICE_TIMEOUT, ERR_DEVICE_CHECK = range(7)
IMPL_AUTO, IMPL_PORTABLE, IMPL_TCGEN05 = 0, 1, 2
MODE_TOPK, MODE_CUMMASS = 0, 1

# every symbol include/carnator.h declares
EXPORTS = [
    "carnator_build_workspace_bytes", "carnator_build_connectivity",
    "carnator_exact_workspace_bytes", "carnator_build_connectivity_exact",
    "carnator_attn_workspace_bytes", "carnator_compact_mask", "carnator_sparse_attn_compacted",
    "carnator_sparse_attn", "carnator_compacted_tiles",
    "carnator_attn_host_arena_bytes", "carnator_sparse_attn_host",
    "carnator_build_host_arena_bytes", "carnator_build_connectivity_host",
    "carnator_sparse_attn_static", "carnator_static_status",
    "carnator_regions_workspace_bytes", "carnator_build_regions", "carnator_fuse_latents",
    "carnator_region_block_flags", "carnator_sparse_attn_region",
    "carnator_seed_workspace_bytes", "carnator_seed_expansion",
    "carnator_delta_e00", "carnator_context_discrepancy", "carnator_size_discrepancy", "carnator_shape_discrepancy",
    "carnator_compatibility_gate", "carnator_clopper_pearson_upper",
    "carnator_query_status", "carnator_selftest_wait_timeout", "carnator_debug_set_builder_path", "carnator_status_string", "carnator_last_cuda_error",
    "carnator_kernel_launches", "carnator_version",
]


class Shape(ctypes.Structure):
    """Mirror of carnator_shape."""
    _fields_ = [
        ("B", ctypes.c_int32), ("H", ctypes.c_int32), ("N", ctypes.c_int32), ("D", ctypes.c_int32),
        ("n_text", ctypes.c_int32), ("T", ctypes.c_int32), ("Hg", ctypes.c_int32), ("Wg", ctypes.c_int32),
        ("block_q", ctypes.c_int32), ("block_k", ctypes.c_int32),
        ("q_stride", ctypes.c_int64 * 3), ("k_stride", ctypes.c_int64 * 3),
        ("v_stride", ctypes.c_int64 * 3), ("o_stride", ctypes.c_int64 * 3),
        ("softmax_scale", ctypes.c_float), ("attn_impl", ctypes.c_int32),
    ]

    @property
    def nqb(self) -> int:
        return -(-self.N // self.block_q)

    @property
    def nkb(self) -> int:
        return -(-self.N // self.block_k)


class BuildParams(ctypes.Structure):
    """Mirror of carnator_build_params."""
    _fields_ = [
        ("mode", ctypes.c_int32), ("keep_ratio", ctypes.c_float), ("mass", ctypes.c_float),
        ("window_frames", ctypes.c_int32), ("text_dense", ctypes.c_int32),
        ("count_includes_forced", ctypes.c_int32),
    ]


class CarnatorError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = f"{where}: {status_string(status)} (status {status})"
        detail = last_cuda_error()
        if detail:
            msg += f" [{detail}]"
        super().__init__(msg)


_lib = None


def lib() -> ctypes.CDLL:
    """Load libcarnator.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2609_32420_b200.build` "
            "(there is no fallback path)")
    L = ctypes.CDLL(LIB_PATH)
    vp, sz, i64 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int64
    ps, pp = ctypes.POINTER(Shape), ctypes.POINTER(BuildParams)
    L.carnator_build_workspace_bytes.restype = sz
    L.carnator_build_workspace_bytes.argtypes = [ps, pp]
    L.carnator_build_connectivity.restype = ctypes.c_int
    L.carnator_build_connectivity.argtypes = [vp, vp, ps, pp, vp, vp, vp, sz, vp]
    L.carnator_exact_workspace_bytes.restype = sz
    L.carnator_exact_workspace_bytes.argtypes = [ps]
    L.carnator_build_connectivity_exact.restype = ctypes.c_int
    L.carnator_build_connectivity_exact.argtypes = [vp, vp, vp, ps, pp, vp, vp, vp, sz, vp]
    L.carnator_attn_workspace_bytes.restype = sz
    L.carnator_attn_workspace_bytes.argtypes = [ps]
    L.carnator_compact_mask.restype = ctypes.c_int
    L.carnator_compact_mask.argtypes = [vp, vp, ps, vp, sz, vp]
    L.carnator_sparse_attn_compacted.restype = ctypes.c_int
    L.carnator_sparse_attn_compacted.argtypes = [vp, vp, vp, ps, vp, vp, vp, sz, vp]
    L.carnator_sparse_attn.restype = ctypes.c_int
    L.carnator_sparse_attn.argtypes = [vp, vp, vp, vp, vp, ps, vp, vp, vp, sz, vp]
    L.carnator_compacted_tiles.restype = ctypes.c_int
    L.carnator_compacted_tiles.argtypes = [ps, vp, sz, vp, ctypes.POINTER(i64)]
    L.carnator_attn_host_arena_bytes.restype = sz
    L.carnator_attn_host_arena_bytes.argtypes = [ps]
    L.carnator_sparse_attn_host.restype = ctypes.c_int
    L.carnator_sparse_attn_host.argtypes = [vp, vp, vp, vp, vp, ps, vp, vp, vp, sz, vp]
    L.carnator_build_host_arena_bytes.restype = sz
    L.carnator_build_host_arena_bytes.argtypes = [ps, pp]
    L.carnator_build_connectivity_host.restype = ctypes.c_int
    L.carnator_build_connectivity_host.argtypes = [vp, vp, ps, pp, vp, vp, sz, vp]
    L.carnator_sparse_attn_static.restype = ctypes.c_int
    L.carnator_sparse_attn_static.argtypes = [vp, vp, vp, vp, vp, ps, vp, vp, vp]
    L.carnator_static_status.restype = ctypes.c_int
    L.carnator_static_status.argtypes = [vp]
    L.carnator_regions_workspace_bytes.restype = sz
    L.carnator_regions_workspace_bytes.argtypes = [ps]
    L.carnator_build_regions.restype = ctypes.c_int
    L.carnator_build_regions.argtypes = [vp, ps, ctypes.c_int32, ctypes.c_int32, vp, vp, vp, vp, sz, vp]
    L.carnator_fuse_latents.restype = ctypes.c_int
    L.carnator_fuse_latents.argtypes = [vp, vp, vp, i64, i64, ctypes.c_int32, vp, vp]
    L.carnator_region_block_flags.restype = ctypes.c_int
    L.carnator_region_block_flags.argtypes = [vp, ps, ctypes.c_int32, ctypes.c_int32, vp, vp]
    L.carnator_sparse_attn_region.restype = ctypes.c_int
    L.carnator_sparse_attn_region.argtypes = [vp, vp, vp, vp, vp, vp, ps, vp, vp, vp, sz, vp]
    L.carnator_seed_workspace_bytes.restype = sz
    L.carnator_seed_workspace_bytes.argtypes = [ps]
    L.carnator_seed_expansion.restype = ctypes.c_int
    L.carnator_seed_expansion.argtypes = [vp, vp, vp, vp, ctypes.c_int32, ctypes.c_int32, ps, vp, vp, vp, sz, vp]
    dbl, pd = ctypes.c_double, ctypes.POINTER(ctypes.c_double)
    L.carnator_delta_e00.restype = dbl
    L.carnator_delta_e00.argtypes = [pd, pd]
    L.carnator_context_discrepancy.restype = dbl
    L.carnator_context_discrepancy.argtypes = [pd, pd, ctypes.c_int32]
    L.carnator_size_discrepancy.restype = dbl
    L.carnator_size_discrepancy.argtypes = [dbl, dbl]
    L.carnator_shape_discrepancy.restype = dbl
    L.carnator_shape_discrepancy.argtypes = [vp, ctypes.c_int32, ctypes.c_int32, vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32]
    L.carnator_compatibility_gate.restype = ctypes.c_int32
    L.carnator_compatibility_gate.argtypes = [pd, pd, vp, ctypes.c_int32]
    L.carnator_clopper_pearson_upper.restype = dbl
    L.carnator_clopper_pearson_upper.argtypes = [ctypes.c_int32, ctypes.c_int32, dbl]
    L.carnator_query_status.restype = ctypes.c_int
    L.carnator_query_status.argtypes = [vp, vp]
    L.carnator_selftest_wait_timeout.restype = ctypes.c_int
    L.carnator_selftest_wait_timeout.argtypes = [vp, ctypes.c_uint64, vp]
    L.carnator_debug_set_builder_path.restype = None
    L.carnator_debug_set_builder_path.argtypes = [ctypes.c_int32]
    L.carnator_status_string.restype = ctypes.c_char_p
    L.carnator_status_string.argtypes = [ctypes.c_int]
    L.carnator_last_cuda_error.restype = ctypes.c_char_p
    L.carnator_last_cuda_error.argtypes = []
    L.carnator_kernel_launches.restype = i64
    L.carnator_kernel_launches.argtypes = []
    L.carnator_version.restype = ctypes.c_int32
    L.carnator_version.argtypes = []
    _lib = L
    return L


def status_string(status: int) -> str:
    return lib().carnator_status_string(int(status)).decode()


def last_cuda_error() -> str:
    return lib().carnator_last_cuda_error().decode()


def kernel_launches() -> int:
    return int(lib().carnator_kernel_launches())


def version() -> int:
    return int(lib().carnator_version())


def _check(status: int, where: str):
    if status != OK:
        raise CarnatorError(status, where)


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream=None):
    import torch
    if stream is None:
        if not torch.cuda.is_available():
            return ctypes.c_void_p(None)     # argument-validation calls on a machine without a GPU
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def make_shape(B, H, N, D, n_text, T, Hg, Wg, block_q, block_k, Q=None, K=None, V=None, O=None,
               softmax_scale: float = 0.0, attn_impl: int = IMPL_AUTO) -> Shape:
    """Fill a Shape; strides are taken from the given [B,H,rows,D] tensors (contiguous [B,H,N,D] if absent)."""
    s = Shape()
    s.B, s.H, s.N, s.D = B, H, N, D
    s.n_text, s.T, s.Hg, s.Wg = n_text, T, Hg, Wg
    s.block_q, s.block_k = block_q, block_k
    default = (H * N * D, N * D, D)
    for name, t in (("q_stride", Q), ("k_stride", K), ("v_stride", V), ("o_stride", O)):
        st = default if t is None else tuple(t.stride()[:3])
        if t is not None and t.stride()[3] != 1:
            raise ValueError("head dimension must be contiguous")
        setattr(s, name, (ctypes.c_int64 * 3)(*st))
    s.softmax_scale = softmax_scale
    s.attn_impl = attn_impl
    return s


def shape_of(w, Q=None, K=None, V=None, O=None, attn_impl: int = IMPL_AUTO) -> Shape:
    """Shape of a workload record (any object with B,H,N,D,n_text,T,Hg,Wg,block)."""
    return make_shape(w.B, w.H, w.N, w.D, w.n_text, w.T, w.Hg, w.Wg, w.block, w.block, Q, K, V, O,
                      attn_impl=attn_impl)


def params_of(bp) -> BuildParams:
    p = BuildParams()
    p.mode, p.keep_ratio, p.mass = bp.mode, bp.keep_ratio, bp.mass
    p.window_frames, p.text_dense, p.count_includes_forced = bp.window_frames, bp.text_dense, bp.count_includes_forced
    return p


def _new_ws(nbytes: int, device):
    import torch
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)


# --------------------------------------------------------------------------------------------
# the calls
# --------------------------------------------------------------------------------------------
def build_workspace_bytes(shape: Shape, params: BuildParams) -> int:
    return int(lib().carnator_build_workspace_bytes(ctypes.byref(shape), ctypes.byref(params)))


def attn_workspace_bytes(shape: Shape) -> int:
    return int(lib().carnator_attn_workspace_bytes(ctypes.byref(shape)))


def build_connectivity(Q, K, shape: Shape, params: BuildParams, mask=None, pooled_scores=None, ws=None, stream=None):
    """carnator_build_connectivity.  Returns (mask uint8 [B,H,nqb,nkb], ws)."""
    import torch
    if mask is None:
        mask = torch.empty((shape.B, shape.H, shape.nqb, shape.nkb), dtype=torch.uint8, device=Q.device)
    if ws is None:
        ws = _new_ws(build_workspace_bytes(shape, params), Q.device)
    st = lib().carnator_build_connectivity(_ptr(Q), _ptr(K), ctypes.byref(shape), ctypes.byref(params), _ptr(mask),
                                           _ptr(pooled_scores), _ptr(ws), ws.numel(), _stream(stream))
    _check(st, "carnator_build_connectivity")
    return mask, ws


def exact_workspace_bytes(shape: Shape) -> int:
    return int(lib().carnator_exact_workspace_bytes(ctypes.byref(shape)))


def build_connectivity_exact(Q, K, LSE, shape: Shape, params: BuildParams, mask=None, block_mass=None, ws=None,
                             stream=None):
    """carnator_build_connectivity_exact.  Returns (mask uint8 [B,H,nqb,nkb], ws)."""
    import torch
    if mask is None:
        mask = torch.empty((shape.B, shape.H, shape.nqb, shape.nkb), dtype=torch.uint8, device=Q.device)
    if ws is None:
        ws = _new_ws(exact_workspace_bytes(shape), Q.device)
    st = lib().carnator_build_connectivity_exact(_ptr(Q), _ptr(K), _ptr(LSE), ctypes.byref(shape), ctypes.byref(params),
                                                 _ptr(mask), _ptr(block_mass), _ptr(ws), ws.numel(), _stream(stream))
    _check(st, "carnator_build_connectivity_exact")
    return mask, ws


def compact_mask(mask, recompute_rows, shape: Shape, ws=None, stream=None):
    if ws is None:
        ws = _new_ws(attn_workspace_bytes(shape), mask.device)
    st = lib().carnator_compact_mask(_ptr(mask), _ptr(recompute_rows), ctypes.byref(shape), _ptr(ws), ws.numel(),
                                     _stream(stream))
    _check(st, "carnator_compact_mask")
    return ws


def _outputs(Q, shape: Shape, O, LSE):
    import torch
    if O is None:
        O = torch.empty((shape.B, shape.H, shape.N, shape.D), dtype=torch.bfloat16, device=Q.device)
        shape.o_stride = (ctypes.c_int64 * 3)(*O.stride()[:3])
    if LSE is None:
        LSE = torch.empty((shape.B, shape.H, shape.N), dtype=torch.float32, device=Q.device)
    return O, LSE


def sparse_attn_compacted(Q, K, V, shape: Shape, ws, O=None, LSE=None, stream=None):
    O, LSE = _outputs(Q, shape, O, LSE)
    st = lib().carnator_sparse_attn_compacted(_ptr(Q), _ptr(K), _ptr(V), ctypes.byref(shape), _ptr(O), _ptr(LSE),
                                              _ptr(ws), ws.numel(), _stream(stream))
    _check(st, "carnator_sparse_attn_compacted")
    return O, LSE


def sparse_attn(Q, K, V, mask, recompute_rows, shape: Shape, O=None, LSE=None, ws=None, stream=None):
    """carnator_sparse_attn.  Returns (O bf16 [B,H,N,D], LSE fp32 [B,H,N], ws)."""
    O, LSE = _outputs(Q, shape, O, LSE)
    if ws is None:
        ws = _new_ws(attn_workspace_bytes(shape), Q.device)
    st = lib().carnator_sparse_attn(_ptr(Q), _ptr(K), _ptr(V), _ptr(mask), _ptr(recompute_rows), ctypes.byref(shape),
                                    _ptr(O), _ptr(LSE), _ptr(ws), ws.numel(), _stream(stream))
    _check(st, "carnator_sparse_attn")
    return O, LSE, ws


def compacted_tiles(shape: Shape, ws, stream=None) -> int:
    out = ctypes.c_int64(0)
    st = lib().carnator_compacted_tiles(ctypes.byref(shape), _ptr(ws), ws.numel(), _stream(stream), ctypes.byref(out))
    _check(st, "carnator_compacted_tiles")
    return int(out.value)


def query_status(ws, stream=None) -> int:
    return int(lib().carnator_query_status(_ptr(ws), _stream(stream)))


def selftest_wait_timeout(ws, limit_ns: int, stream=None) -> None:
    """carnator_selftest_wait_timeout: a bounded wait on a barrier nothing arms; query_status(ws) reports the time-out."""
    _check(lib().carnator_selftest_wait_timeout(_ptr(ws), int(limit_ns), _stream(stream)), "carnator_selftest_wait_timeout")


# byte offsets inside the 256-byte workspace header (tests of the time-out path write them)
HDR_WAIT_LIMIT_NS, HDR_DEBUG_WITHHOLD = 40, 48

BUILDER_AUTO, BUILDER_THREE_KERNELS, BUILDER_FUSED = 0, 1, 2


def debug_set_builder_path(path: int) -> None:
    """Testing aid: 0 = by size, 1 = three kernels, 2 = the fused persistent kernel where the shape allows it."""
    lib().carnator_debug_set_builder_path(int(path))


def attn_host_arena_bytes(shape: Shape) -> int:
    return int(lib().carnator_attn_host_arena_bytes(ctypes.byref(shape)))


def sparse_attn_host(Q, K, V, mask, recompute_rows, shape: Shape, O, LSE, arena, stream=None):
    """carnator_sparse_attn_host: Q..LSE are HOST tensors (pinned), arena is a device buffer."""
    st = lib().carnator_sparse_attn_host(_ptr(Q), _ptr(K), _ptr(V), _ptr(mask), _ptr(recompute_rows),
                                         ctypes.byref(shape), _ptr(O), _ptr(LSE), _ptr(arena), arena.numel(),
                                         _stream(stream))
    _check(st, "carnator_sparse_attn_host")


def build_host_arena_bytes(shape: Shape, params: BuildParams) -> int:
    return int(lib().carnator_build_host_arena_bytes(ctypes.byref(shape), ctypes.byref(params)))


def build_connectivity_host(Q, K, shape: Shape, params: BuildParams, mask, arena, stream=None):
    st = lib().carnator_build_connectivity_host(_ptr(Q), _ptr(K), ctypes.byref(shape), ctypes.byref(params),
                                                _ptr(mask), _ptr(arena), arena.numel(), _stream(stream))
    _check(st, "carnator_build_connectivity_host")


STATIC_SCRATCH_BYTES = 8 << 20


def sparse_attn_static(Q, K, V, mask, recompute_rows, shape: Shape, O, LSE, stream=None):
    """carnator_sparse_attn_static: no workspace argument -- the library's built-in scratch array is used.

    For callers that must not allocate device memory when they call (fixed memory budgets, hosts that own
    the allocator, latency-critical loops).  O and LSE must be passed in; nothing is allocated here either.
    Shapes whose workspace exceeds STATIC_SCRATCH_BYTES raise with CARNATOR_ERR_WORKSPACE.  Calls share the
    one array per device: keep them ordered on the GPU.
    """
    shape.o_stride = (ctypes.c_int64 * 3)(*O.stride()[:3])
    st = lib().carnator_sparse_attn_static(_ptr(Q), _ptr(K), _ptr(V), _ptr(mask), _ptr(recompute_rows),
                                           ctypes.byref(shape), _ptr(O), _ptr(LSE), _stream(stream))
    _check(st, "carnator_sparse_attn_static")


def static_status(stream=None) -> int:
    """carnator_static_status: the device status word of the static-scratch form on the current device (read and cleared)."""
    return int(lib().carnator_static_status(_stream(stream)))


DTYPE_F32, DTYPE_BF16 = 0, 1


def build_regions(evidence, shape: Shape, r_active: int = 2, r_context: int = 3, stream=None):
    """carnator_build_regions.  evidence uint8 [T,Hg,Wg] on the device -> (active, context, W)."""
    import torch
    active = torch.empty_like(evidence)
    context = torch.empty_like(evidence)
    W = torch.empty(evidence.shape, dtype=torch.float32, device=evidence.device)
    ws = _new_ws(int(lib().carnator_regions_workspace_bytes(ctypes.byref(shape))), evidence.device)
    st = lib().carnator_build_regions(_ptr(evidence), ctypes.byref(shape), r_active, r_context, _ptr(active), _ptr(context),
                                      _ptr(W), _ptr(ws), ws.numel(), _stream(stream))
    _check(st, "carnator_build_regions")
    return active, context, W


def fuse_latents(z_target, z_hist, W, z_out=None, stream=None):
    """carnator_fuse_latents over [channels, tokens] tensors (fp32 or bf16), W fp32 [tokens]."""
    import torch
    if z_out is None:
        z_out = torch.empty_like(z_target)
    dtype = DTYPE_F32 if z_target.dtype == torch.float32 else DTYPE_BF16
    channels, tokens = z_target.shape[0], z_target[0].numel()
    st = lib().carnator_fuse_latents(_ptr(z_target), _ptr(z_hist), _ptr(W), channels, tokens, dtype, _ptr(z_out), _stream(stream))
    _check(st, "carnator_fuse_latents")
    return z_out


def region_block_flags(region, shape: Shape, block: int, text_value: int = 1, stream=None):
    import torch
    n = shape.n_text + shape.T * shape.Hg * shape.Wg
    flags = torch.empty((-(-n // block),), dtype=torch.uint8, device=region.device)
    st = lib().carnator_region_block_flags(_ptr(region), ctypes.byref(shape), block, text_value, _ptr(flags), _stream(stream))
    _check(st, "carnator_region_block_flags")
    return flags


def sparse_attn_region(Q, K, V, mask, active_q, context_k, shape: Shape, O, LSE, ws=None, stream=None):
    """carnator_sparse_attn_region: O and LSE are updated in place; rows of inactive query blocks stay as they are."""
    if ws is None:
        ws = _new_ws(attn_workspace_bytes(shape), Q.device)
    shape.o_stride = (ctypes.c_int64 * 3)(*O.stride()[:3])
    st = lib().carnator_sparse_attn_region(_ptr(Q), _ptr(K), _ptr(V), _ptr(mask), _ptr(active_q), _ptr(context_k),
                                           ctypes.byref(shape), _ptr(O), _ptr(LSE), _ptr(ws), ws.numel(), _stream(stream))
    _check(st, "carnator_sparse_attn_region")
    return ws


def seed_workspace_bytes(shape: Shape) -> int:
    return int(lib().carnator_seed_workspace_bytes(ctypes.byref(shape)))


def seed_expansion(Q, K, LSE, seeds, n_pos: int, n_neg: int, shape: Shape, per_head=None, stream=None, ws=None,
                   return_ws: bool = False):
    """carnator_seed_expansion.  seeds: int32 device tensor [n_pos + n_neg].  Returns contrast fp32 [B,N]
    (and the workspace, whose header carries the device status, with ``return_ws``)."""
    import torch
    out = torch.empty((shape.B, shape.N), dtype=torch.float32, device=Q.device)
    if ws is None:
        ws = _new_ws(int(lib().carnator_seed_workspace_bytes(ctypes.byref(shape))), Q.device)
    st = lib().carnator_seed_expansion(_ptr(Q), _ptr(K), _ptr(LSE), _ptr(seeds), n_pos, n_neg, ctypes.byref(shape),
                                       _ptr(per_head), _ptr(out), _ptr(ws), ws.numel(), _stream(stream))
    _check(st, "carnator_seed_expansion")
    return (out, ws) if return_ws else out


# ---- host-side scalars (no GPU) ---------------------------------------------------------------------
def delta_e00(lab_a, lab_b) -> float:
    a = (ctypes.c_double * 3)(*[float(x) for x in lab_a])
    b = (ctypes.c_double * 3)(*[float(x) for x in lab_b])
    return float(lib().carnator_delta_e00(a, b))


def context_discrepancy(labs_q, labs_j) -> float:
    """labs_q, labs_j: equally long sequences of (L*, a*, b*) triples, one per shared noun."""
    n = len(labs_q)
    if n != len(labs_j):
        raise ValueError("one colour per shared noun on both sides")
    a = (ctypes.c_double * (3 * n))(*[float(x) for c in labs_q for x in c])
    b = (ctypes.c_double * (3 * n))(*[float(x) for c in labs_j for x in c])
    return float(lib().carnator_context_discrepancy(a, b, n))


def size_discrepancy(area_q: float, area_j: float) -> float:
    return float(lib().carnator_size_discrepancy(float(area_q), float(area_j)))


def shape_discrepancy(m_q, m_j, resolution: int = 32) -> float:
    """m_q, m_j: 2-D numpy uint8 indicators."""
    import numpy as np
    a = np.ascontiguousarray(m_q, dtype=np.uint8)
    b = np.ascontiguousarray(m_j, dtype=np.uint8)
    return float(lib().carnator_shape_discrepancy(a.ctypes.data, a.shape[0], a.shape[1], b.ctypes.data, b.shape[0], b.shape[1],
                                                  int(resolution)))


def compatibility_gate(d, tau, applicable=None) -> int:
    n = len(d)
    dd = (ctypes.c_double * n)(*[float(x) for x in d])
    tt = (ctypes.c_double * n)(*[float(x) for x in tau])
    ap = None
    if applicable is not None:
        ap = (ctypes.c_uint8 * n)(*[int(bool(x)) for x in applicable])
    return int(lib().carnator_compatibility_gate(dd, tt, ap, n))


def clopper_pearson_upper(unsafe: int, accepted: int, alpha: float) -> float:
    return float(lib().carnator_clopper_pearson_upper(int(unsafe), int(accepted), float(alpha)))
