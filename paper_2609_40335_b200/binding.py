"""ctypes binding of libdp_ghost.so: same names as the C ABI, argument marshalling only.

Every step runs in the CUDA kernels of the shared library; PyTorch is used for device
memory and streams.  If the library is missing or a call fails, an exception is raised --
there is no fallback implementation.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

import torch

DP_F32, DP_BF16 = 0, 1
DP_NORM_AUTO, DP_NORM_GHOST, DP_NORM_DIRECT = 0, 1, 2
DP_DEV_BAD_ID, DP_DEV_TIMEOUT, DP_DEV_BOUNDS = 1, 2, 4

_LIB_PATH = os.environ.get("DP_GHOST_LIB") or os.path.join(os.path.dirname(os.path.abspath(__file__)),
                                                       "libdp_ghost.so")
_lib = None


class DpGhostError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        super().__init__(f"{where}: status {status} ({detail})")


class _LinearDesc(C.Structure):
    _fields_ = [("A", C.c_void_p), ("lda", C.c_int64), ("d", C.c_int32),
                ("G", C.c_void_p), ("ldg", C.c_int64), ("p", C.c_int32),
                ("mode", C.c_int32), ("mode_used", C.c_int32)]


class _VectorDesc(C.Structure):
    _fields_ = [("G", C.c_void_p), ("ldg", C.c_int64), ("X", C.c_void_p), ("ldx", C.c_int64),
                ("p", C.c_int32)]


EXPORTS = ["dp_vector_norms", "dp_vector_norms_ws_bytes", "dp_clip_accumulate_vectors",
           "dp_clip_accumulate_vectors_ws_bytes", "dp_ghost_norms", "dp_ghost_norms_ws_bytes", "dp_embed_norms", "dp_embed_norms_ws_bytes",
           "dp_embed_norms_static",
           "dp_tied_cross_term", "dp_tied_cross_term_ws_bytes", "dp_clip_factors", "dp_clip_factors_sum",
           "dp_clip_accumulate", "dp_clip_accumulate_ws_bytes", "dp_clip_accumulate_grouped",
           "dp_clip_accumulate_grouped_ws_bytes", "dp_clip_accumulate_noise_grouped",
           "dp_clip_accumulate_embed_noise", "dp_clip_accumulate_embed",
           "dp_clip_accumulate_embed_ws_bytes", "dp_embed_sort", "dp_embed_sort_ws_bytes",
           "dp_clip_accumulate_embed_sorted", "dp_add_noise", "dp_add_noise_slice", "dp_noise_step_device",
           "dp_fill_noise", "dp_rdp_epsilon", "dp_sigma_for_epsilon", "dp_status_string",
           "dp_last_cuda_error", "dp_version", "dp_kernel_launches", "dp_debug_force_fma",
           "dp_debug_noise_error_scan", "dp_debug_bounds_checked", "dp_debug_bounds_probe",
           "dp_debug_tensor_map_encodes", "dp_debug_set_wait_limit",
           "dp_debug_ghost_single", "dp_set_reserved_sms"]


def lib_path() -> str:
    return _LIB_PATH


def load():
    """Load libdp_ghost.so (built by `python -m paper_2609_40335_b200.build`)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise DpGhostError(-1, "load", f"{_LIB_PATH} not found: build it first; there is no fallback")
    L = C.CDLL(_LIB_PATH)
    vp, i32, i64, f32, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_size_t
    L.dp_ghost_norms.argtypes = [C.POINTER(_LinearDesc), i32, i32, i32, i32, vp, vp, sz, vp, vp]
    L.dp_ghost_norms_ws_bytes.argtypes = [C.POINTER(_LinearDesc), i32, i32, i32, i32]
    L.dp_ghost_norms_ws_bytes.restype = sz
    L.dp_embed_norms.argtypes = [vp, vp, i64, i32, i32, i32, i32, i32, vp, vp, vp, sz, vp, vp]
    VP = C.POINTER(_VectorDesc)
    L.dp_vector_norms.argtypes = [VP, i32, i32, i32, i32, vp, vp, sz, vp]
    L.dp_vector_norms_ws_bytes.argtypes = [VP, i32, i32, i32]
    L.dp_vector_norms_ws_bytes.restype = sz
    L.dp_clip_accumulate_vectors.argtypes = [VP, i32, i32, i32, i32, vp, f32, vp, C.POINTER(vp), f32, i32,
                                             f32, f32, C.c_uint64, C.POINTER(C.c_uint32), C.c_uint32,
                                             vp, sz, vp]
    L.dp_clip_accumulate_vectors_ws_bytes.argtypes = [VP, i32, i32, i32]
    L.dp_clip_accumulate_vectors_ws_bytes.restype = sz
    L.dp_embed_norms_static.argtypes = [vp, vp, i64, i32, i32, i32, i32, i32, vp, vp, vp, vp]
    L.dp_embed_norms_ws_bytes.argtypes = [i32, i32, i32]
    L.dp_embed_norms_ws_bytes.restype = sz
    L.dp_tied_cross_term.argtypes = [vp, vp, i64, vp, i64, vp, i64, i32, i32, i32, i32, i32, vp, vp,
                                     vp, sz, vp, vp]
    L.dp_tied_cross_term_ws_bytes.argtypes = [i32, i32, i32, i32]
    L.dp_tied_cross_term_ws_bytes.restype = sz
    L.dp_clip_factors.argtypes = [vp, i32, f32, vp, vp, vp]
    L.dp_clip_factors_sum.argtypes = [vp, vp, i32, f32, vp, vp, vp]
    L.dp_clip_accumulate.argtypes = [vp, i64, vp, i64, i32, i32, i32, i32, i32, vp, f32, vp, vp, i64,
                                     f32, vp, sz, vp, vp]
    L.dp_clip_accumulate_ws_bytes.argtypes = [i32, i32, i32, i32, i32]
    L.dp_clip_accumulate_ws_bytes.restype = sz
    L.dp_clip_accumulate_grouped.argtypes = [C.POINTER(_LinearDesc), i32, i32, i32, i32, vp, f32, vp,
                                             C.POINTER(vp), C.POINTER(i64), f32, vp, sz, vp, vp]
    L.dp_clip_accumulate_grouped_ws_bytes.argtypes = [C.POINTER(_LinearDesc), i32, i32, i32, i32]
    L.dp_clip_accumulate_grouped_ws_bytes.restype = sz
    L.dp_clip_accumulate_noise_grouped.argtypes = [C.POINTER(_LinearDesc), i32, i32, i32, i32, vp, f32,
                                                   vp, C.POINTER(vp), C.POINTER(i64), f32, f32, f32,
                                                   C.c_uint64, C.POINTER(C.c_uint32), C.c_uint32,
                                                   vp, sz, vp, vp]
    L.dp_clip_accumulate_embed_noise.argtypes = [vp, vp, i64, i32, i32, i32, i32, i32, vp, f32, vp, vp,
                                                 i64, f32, f32, f32, C.c_uint64, C.c_uint32,
                                                 C.c_uint32, vp, vp, vp, sz, vp, vp]
    L.dp_clip_accumulate_embed.argtypes = [vp, vp, i64, i32, i32, i32, i32, i32, vp, f32, vp, vp, i64,
                                           f32, vp, vp, vp, sz, vp, vp]
    L.dp_clip_accumulate_embed_ws_bytes.argtypes = [i32, i32, i32, i32]
    L.dp_clip_accumulate_embed_ws_bytes.restype = sz
    L.dp_embed_sort.argtypes = [vp, i32, i32, i32, vp, vp, vp, sz, vp, vp]
    L.dp_embed_sort_ws_bytes.argtypes = [i32, i32, i32]
    L.dp_embed_sort_ws_bytes.restype = sz
    L.dp_clip_accumulate_embed_sorted.argtypes = [vp, vp, i64, i32, i32, i32, i32, i32, vp, f32, vp, vp,
                                                  i64, f32, vp, vp, vp, sz, vp, vp]
    L.dp_add_noise.argtypes = [vp, i64, f32, f32, f32, C.c_uint64, C.c_uint32, C.c_uint32, vp]
    L.dp_fill_noise.argtypes = [vp, i64, f32, f32, f32, C.c_uint64, C.c_uint32, C.c_uint32, vp]
    L.dp_add_noise_slice.argtypes = [vp, i64, i64, f32, f32, f32, C.c_uint64, C.c_uint32, C.c_uint32, vp]
    L.dp_noise_step_device.argtypes = [vp]
    L.dp_rdp_epsilon.argtypes = [C.c_double, C.c_double, i64, C.c_double, vp, vp]
    L.dp_sigma_for_epsilon.argtypes = [C.c_double, i64, C.c_double, C.c_double, C.c_double, vp]
    L.dp_status_string.argtypes = [i32]
    L.dp_status_string.restype = C.c_char_p
    L.dp_last_cuda_error.restype = i32
    L.dp_version.restype = C.c_char_p
    L.dp_kernel_launches.restype = C.c_int64
    L.dp_debug_noise_error_scan.argtypes = [f32, vp, vp]
    L.dp_debug_bounds_probe.argtypes = [i64, i64, vp, vp]
    L.dp_debug_tensor_map_encodes.restype = i64
    L.dp_debug_set_wait_limit.argtypes = [i64]
    L.dp_debug_set_wait_limit.restype = i64
    L.dp_debug_ghost_single.argtypes = [i32]
    L.dp_debug_ghost_single.restype = i32
    L.dp_debug_force_fma.argtypes = [i32]
    L.dp_debug_force_fma.restype = i32
    L.dp_set_reserved_sms.argtypes = [i32]
    L.dp_set_reserved_sms.restype = i32
    for name in EXPORTS:
        fn = getattr(L, name)
        if fn.restype is C.c_int:          # ctypes default: the dp_status functions
            fn.restype = i32
    _lib = L
    return L


def _check(st: int, where: str):
    if st != 0:
        L = load()
        msg = L.dp_status_string(st).decode()
        if st == 5:
            msg += f", cuda error {L.dp_last_cuda_error()}"
        raise DpGhostError(st, where, msg)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise DpGhostError(1, "marshal", "tensor is not on a CUDA device; there is no CPU path")
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return DP_F32
    if t.dtype == torch.bfloat16:
        return DP_BF16
    raise DpGhostError(1, "marshal", f"unsupported dtype {t.dtype}")


def _rows_ld(t: torch.Tensor) -> int:
    """Leading dimension of a (..., ld) tensor whose leading axes are densely packed."""
    if t.stride(-1) != 1:
        raise DpGhostError(1, "marshal", "innermost stride must be 1")
    ld = t.stride(-2)
    if t.dim() == 3 and t.stride(0) != t.shape[1] * ld:
        raise DpGhostError(1, "marshal", "examples must be contiguous blocks of T rows")
    return ld


def _ws(nbytes: int, ws: Optional[torch.Tensor], device) -> torch.Tensor:
    if ws is not None:
        return ws
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)


@dataclass
class Linear:
    """One linear layer d -> p: A (B,T,>=d) inputs, G (B,T,>=p) output gradients."""
    A: torch.Tensor
    G: torch.Tensor
    d: Optional[int] = None
    p: Optional[int] = None
    mode: int = DP_NORM_AUTO
    mode_used: int = -1


def _descs(layers: Sequence[Linear]):
    arr = (_LinearDesc * len(layers))()
    for k, l in enumerate(layers):
        arr[k].A = _ptr(l.A)
        arr[k].lda = _rows_ld(l.A)
        arr[k].d = l.d if l.d is not None else l.A.shape[-1]
        arr[k].G = _ptr(l.G)
        arr[k].ldg = _rows_ld(l.G)
        arr[k].p = l.p if l.p is not None else l.G.shape[-1]
        arr[k].mode = l.mode
        arr[k].mode_used = -1
    return arr


def dp_ghost_norms_ws_bytes(layers: Sequence[Linear], B: int, T: int) -> int:
    L = load()
    return int(L.dp_ghost_norms_ws_bytes(_descs(layers), len(layers), _dt(layers[0].A), B, T))


def dp_ghost_norms(layers: Sequence[Linear], B: int, T: int, sq: torch.Tensor, ws=None,
                   dev_status=None, stream=None) -> List[int]:
    """sq[i] += ||G_i^T A_i||_F^2 for every layer; returns the mode each layer ran in."""
    L = load()
    arr = _descs(layers)
    dt = _dt(layers[0].A)
    need = int(L.dp_ghost_norms_ws_bytes(arr, len(layers), dt, B, T))
    ws = _ws(need, ws, sq.device)
    st = L.dp_ghost_norms(arr, len(layers), dt, B, T, _ptr(sq), _ptr(ws), ws.numel() * ws.element_size(),
                          _ptr(dev_status), _stream(stream))
    _check(st, "dp_ghost_norms")
    used = [int(arr[k].mode_used) for k in range(len(layers))]
    for l, u in zip(layers, used):
        l.mode_used = u
    return used


def dp_embed_norms(ids: torch.Tensor, G: torch.Tensor, V: int, sq: torch.Tensor, d=None,
                   first_occ=None, ws=None, dev_status=None, stream=None):
    L = load()
    B, T = ids.shape
    d = d if d is not None else G.shape[-1]
    need = int(L.dp_embed_norms_ws_bytes(B, T, d))
    ws = _ws(need, ws, sq.device)
    st = L.dp_embed_norms(_ptr(ids), _ptr(G), _rows_ld(G), _dt(G), B, T, d, V, _ptr(sq),
                          _ptr(first_occ), _ptr(ws), ws.numel() * ws.element_size(),
                          _ptr(dev_status), _stream(stream))
    _check(st, "dp_embed_norms")


@dataclass
class Vector:
    """A bias / LayerNorm parameter: G (B,T,>=p) gradient at its output, X normalised input or None."""
    G: torch.Tensor
    X: Optional[torch.Tensor] = None
    p: Optional[int] = None


def _vdescs(params: Sequence[Vector]):
    arr = (_VectorDesc * len(params))()
    for k, v in enumerate(params):
        arr[k].G = _ptr(v.G)
        arr[k].ldg = _rows_ld(v.G)
        arr[k].X = _ptr(v.X)
        arr[k].ldx = _rows_ld(v.X) if v.X is not None else 0
        arr[k].p = v.p if v.p is not None else v.G.shape[-1]
    return arr


def dp_vector_norms_ws_bytes(params: Sequence[Vector], B: int, T: int) -> int:
    return int(load().dp_vector_norms_ws_bytes(_vdescs(params), len(params), B, T))


def dp_clip_accumulate_vectors_ws_bytes(params: Sequence[Vector], B: int, T: int) -> int:
    return int(load().dp_clip_accumulate_vectors_ws_bytes(_vdescs(params), len(params), B, T))


def dp_vector_norms(params: Sequence[Vector], B: int, T: int, sq: torch.Tensor, ws=None, stream=None):
    """sq[i] += ||sum_t G[i,t]*X[i,t]||^2 for every bias / LayerNorm parameter."""
    L = load()
    arr = _vdescs(params)
    need = int(L.dp_vector_norms_ws_bytes(arr, len(params), B, T))
    ws = _ws(need, ws, sq.device)
    st = L.dp_vector_norms(arr, len(params), _dt(params[0].G), B, T, _ptr(sq), _ptr(ws),
                           ws.numel() * ws.element_size(), _stream(stream))
    _check(st, "dp_vector_norms")


def dp_clip_accumulate_vectors(params: Sequence[Vector], B: int, T: int, sq, C_: float,
                               outs: Sequence[torch.Tensor], beta: float = 0.0, noise=None, clip=None,
                               ws=None, stream=None):
    """outs[k] = beta*outs[k] + sum_i R_i v_i; noise = (sigma, scale, seed, tensor_ids, step) adds
    the Gaussian mechanism in the same pass."""
    L = load()
    arr = _vdescs(params)
    n = len(params)
    optr = (C.c_void_p * n)(*[_ptr(o) for o in outs])
    need = int(L.dp_clip_accumulate_vectors_ws_bytes(arr, n, B, T))
    ws = _ws(need, ws, outs[0].device)
    if noise is None:
        with_noise, sigma, scale, seed, tids, step = 0, 0.0, 1.0, 0, None, 0
    else:
        sigma, scale, seed, ids_, step = noise
        with_noise, tids = 1, (C.c_uint32 * n)(*[int(t) for t in ids_])
    st = L.dp_clip_accumulate_vectors(arr, n, _dt(params[0].G), B, T, _ptr(sq), float(C_), _ptr(clip),
                                      optr, float(beta), with_noise, float(sigma), float(scale),
                                      int(seed) & (2 ** 64 - 1), tids, int(step), _ptr(ws),
                                      ws.numel() * ws.element_size(), _stream(stream))
    _check(st, "dp_clip_accumulate_vectors")


def dp_embed_norms_static(ids: torch.Tensor, G: torch.Tensor, V: int, sq: torch.Tensor, d=None,
                          first_occ=None, dev_status=None, stream=None):
    """dp_embed_norms for callers that cannot allocate: no workspace is passed or created here;
    the kernel's scratch is a fixed array inside the library (B * ceil(d/256) <= 16384, else
    status 6).  Calls that may overlap on the GPU must not be issued (they share that array)."""
    L = load()
    B, T = ids.shape
    d = d if d is not None else G.shape[-1]
    st = L.dp_embed_norms_static(_ptr(ids), _ptr(G), _rows_ld(G), _dt(G), B, T, d, V, _ptr(sq),
                                 _ptr(first_occ), _ptr(dev_status), _stream(stream))
    _check(st, "dp_embed_norms_static")


def dp_tied_cross_term(ids, G_emb, A_lm, G_lm, V: int, sq=None, cross=None, d=None, ws=None,
                       dev_status=None, stream=None):
    L = load()
    B, T = ids.shape
    d = d if d is not None else G_emb.shape[-1]
    need = int(L.dp_tied_cross_term_ws_bytes(B, T, d, V))
    dev = G_emb.device
    ws = _ws(need, ws, dev)
    st = L.dp_tied_cross_term(_ptr(ids), _ptr(G_emb), _rows_ld(G_emb), _ptr(A_lm), _rows_ld(A_lm),
                              _ptr(G_lm), _rows_ld(G_lm), _dt(G_emb), B, T, d, V, _ptr(sq),
                              _ptr(cross), _ptr(ws), ws.numel() * ws.element_size(),
                              _ptr(dev_status), _stream(stream))
    _check(st, "dp_tied_cross_term")


def dp_clip_factors(sq: torch.Tensor, C_: float, clip=None, norms=None, stream=None):
    L = load()
    _check(L.dp_clip_factors(_ptr(sq), sq.numel(), float(C_), _ptr(clip), _ptr(norms), _stream(stream)),
           "dp_clip_factors")


def dp_clip_factors_sum(sq: torch.Tensor, sq_extra: torch.Tensor, C_: float, clip=None, norms=None,
                        stream=None):
    """sq += sq_extra, then clip factors and norms from the sum (one kernel)."""
    L = load()
    _check(L.dp_clip_factors_sum(_ptr(sq), _ptr(sq_extra), sq.numel(), float(C_), _ptr(clip),
                                 _ptr(norms), _stream(stream)), "dp_clip_factors_sum")


def dp_clip_accumulate_ws_bytes(dt: int, B: int, T: int, d: int, p: int) -> int:
    return int(load().dp_clip_accumulate_ws_bytes(dt, B, T, d, p))


def dp_clip_accumulate(A, G, sq, C_: float, out, beta: float = 0.0, d=None, p=None, clip=None,
                       ws=None, dev_status=None, stream=None):
    """out (p,d) = beta*out + sum_i min(1, C/sqrt(sq[i])) * G_i^T A_i."""
    L = load()
    B, T = A.shape[0], A.shape[1]
    d = d if d is not None else A.shape[-1]
    p = p if p is not None else G.shape[-1]
    dt = _dt(A)
    need = int(L.dp_clip_accumulate_ws_bytes(dt, B, T, d, p))
    ws = _ws(need, ws, out.device)
    st = L.dp_clip_accumulate(_ptr(A), _rows_ld(A), _ptr(G), _rows_ld(G), dt, B, T, d, p, _ptr(sq),
                              float(C_), _ptr(clip), _ptr(out), out.stride(0), float(beta), _ptr(ws),
                              ws.numel() * ws.element_size(), _ptr(dev_status), _stream(stream))
    _check(st, "dp_clip_accumulate")


def dp_clip_accumulate_grouped_ws_bytes(layers: Sequence[Linear], B: int, T: int) -> int:
    return int(load().dp_clip_accumulate_grouped_ws_bytes(_descs(layers), len(layers),
                                                          _dt(layers[0].A), B, T))


def dp_clip_accumulate_grouped(layers: Sequence[Linear], B: int, T: int, sq, C_: float,
                               outs: Sequence[torch.Tensor], beta: float = 0.0, clip=None, ws=None,
                               dev_status=None, stream=None):
    """outs[k] (p_k, d_k) = beta*outs[k] + sum_i R_i G_i^T A_i for every layer, one launch."""
    L = load()
    arr = _descs(layers)
    dt = _dt(layers[0].A)
    n = len(layers)
    optr = (C.c_void_p * n)(*[_ptr(o) for o in outs])
    ldos = (C.c_int64 * n)(*[o.stride(0) for o in outs])
    need = int(L.dp_clip_accumulate_grouped_ws_bytes(arr, n, dt, B, T))
    ws = _ws(need, ws, outs[0].device)
    st = L.dp_clip_accumulate_grouped(arr, n, dt, B, T, _ptr(sq), float(C_), _ptr(clip), optr, ldos,
                                      float(beta), _ptr(ws), ws.numel() * ws.element_size(),
                                      _ptr(dev_status), _stream(stream))
    _check(st, "dp_clip_accumulate_grouped")


def dp_clip_accumulate_noise_grouped(layers: Sequence[Linear], B: int, T: int, sq, C_: float,
                                     outs: Sequence[torch.Tensor], sigma: float, scale: float,
                                     seed: int, tensor_ids: Sequence[int], step: int,
                                     beta: float = 0.0, clip=None, ws=None, dev_status=None,
                                     stream=None):
    """Clipped sums of every layer with the Gaussian noise added in the GEMM epilogue."""
    L = load()
    arr = _descs(layers)
    dt = _dt(layers[0].A)
    n = len(layers)
    optr = (C.c_void_p * n)(*[_ptr(o) for o in outs])
    ldos = (C.c_int64 * n)(*[o.stride(0) for o in outs])
    tids = (C.c_uint32 * n)(*[int(t) for t in tensor_ids])
    need = int(L.dp_clip_accumulate_grouped_ws_bytes(arr, n, dt, B, T))
    ws = _ws(need, ws, outs[0].device)
    st = L.dp_clip_accumulate_noise_grouped(arr, n, dt, B, T, _ptr(sq), float(C_), _ptr(clip), optr,
                                            ldos, float(beta), float(sigma), float(scale),
                                            int(seed) & (2 ** 64 - 1), tids, int(step), _ptr(ws),
                                            ws.numel() * ws.element_size(), _ptr(dev_status),
                                            _stream(stream))
    _check(st, "dp_clip_accumulate_noise_grouped")


def dp_clip_accumulate_embed_noise(ids, G, V: int, sq, C_: float, out, sigma: float, scale: float,
                                   seed: int, tensor_id: int, step: int, beta: float = 0.0, d=None,
                                   clip=None, perm=None, seg=None, ws=None, dev_status=None,
                                   stream=None):
    L = load()
    B, T = ids.shape
    d = d if d is not None else G.shape[-1]
    need = int(L.dp_clip_accumulate_embed_ws_bytes(B, T, d, V))
    ws = _ws(need, ws, out.device)
    st = L.dp_clip_accumulate_embed_noise(_ptr(ids), _ptr(G), _rows_ld(G), _dt(G), B, T, d, V, _ptr(sq),
                                          float(C_), _ptr(clip), _ptr(out), out.stride(0), float(beta),
                                          float(sigma), float(scale), int(seed) & (2 ** 64 - 1),
                                          int(tensor_id), int(step), _ptr(perm), _ptr(seg), _ptr(ws),
                                          ws.numel() * ws.element_size(), _ptr(dev_status),
                                          _stream(stream))
    _check(st, "dp_clip_accumulate_embed_noise")


def dp_clip_accumulate_embed(ids, G, V: int, sq, C_: float, out, beta: float = 0.0, d=None,
                             clip=None, perm=None, seg=None, ws=None, dev_status=None, stream=None):
    L = load()
    B, T = ids.shape
    d = d if d is not None else G.shape[-1]
    need = int(L.dp_clip_accumulate_embed_ws_bytes(B, T, d, V))
    ws = _ws(need, ws, out.device)
    st = L.dp_clip_accumulate_embed(_ptr(ids), _ptr(G), _rows_ld(G), _dt(G), B, T, d, V, _ptr(sq),
                                    float(C_), _ptr(clip), _ptr(out), out.stride(0), float(beta),
                                    _ptr(perm), _ptr(seg), _ptr(ws), ws.numel() * ws.element_size(),
                                    _ptr(dev_status), _stream(stream))
    _check(st, "dp_clip_accumulate_embed")


def dp_embed_sort(ids, V: int, perm, seg, ws=None, dev_status=None, stream=None):
    """Stable counting sort of the B*T token ids: perm (B*T int32), seg (V+1 int32)."""
    L = load()
    B, T = ids.shape
    ws = _ws(int(L.dp_embed_sort_ws_bytes(B, T, V)), ws, ids.device)
    st = L.dp_embed_sort(_ptr(ids), B, T, V, _ptr(perm), _ptr(seg), _ptr(ws),
                         ws.numel() * ws.element_size(), _ptr(dev_status), _stream(stream))
    _check(st, "dp_embed_sort")


def dp_clip_accumulate_embed_sorted(ids, G, V: int, sq, C_: float, out, perm, seg, beta: float = 0.0,
                                    d=None, clip=None, ws=None, dev_status=None, stream=None):
    """dp_clip_accumulate_embed with the sort (dp_embed_sort) already done."""
    L = load()
    B, T = ids.shape
    d = d if d is not None else G.shape[-1]
    ws = _ws(int(L.dp_clip_accumulate_embed_ws_bytes(B, T, d, V)), ws, out.device)
    st = L.dp_clip_accumulate_embed_sorted(_ptr(ids), _ptr(G), _rows_ld(G), _dt(G), B, T, d, V,
                                           _ptr(sq), float(C_), _ptr(clip), _ptr(out), out.stride(0),
                                           float(beta), _ptr(perm), _ptr(seg), _ptr(ws),
                                           ws.numel() * ws.element_size(), _ptr(dev_status),
                                           _stream(stream))
    _check(st, "dp_clip_accumulate_embed_sorted")


def dp_add_noise(out: torch.Tensor, sigma: float, C_: float, scale: float, seed: int,
                 tensor_id: int, step: int, n=None, stream=None):
    """out = scale * (out + sigma*C*z) in place, z from the (seed, tensor_id, step) stream."""
    L = load()
    n = out.numel() if n is None else n
    st = L.dp_add_noise(_ptr(out), n, float(sigma), float(C_), float(scale), int(seed) & (2 ** 64 - 1),
                        int(tensor_id), int(step), _stream(stream))
    _check(st, "dp_add_noise")


def dp_add_noise_slice(out: torch.Tensor, first_element: int, sigma: float, C_: float, scale: float,
                       seed: int, tensor_id: int, step: int, n=None, stream=None):
    """dp_add_noise on the slice of a tensor that starts at element `first_element` (a multiple of 4)."""
    L = load()
    n = out.numel() if n is None else n
    st = L.dp_add_noise_slice(_ptr(out), n, int(first_element), float(sigma), float(C_), float(scale),
                              int(seed) & (2 ** 64 - 1), int(tensor_id), int(step), _stream(stream))
    _check(st, "dp_add_noise_slice")


def dp_noise_step_device(counter) -> None:
    """Register (tensor of one uint32/int32 on the device) or clear (None) the device step counter."""
    _check(load().dp_noise_step_device(None if counter is None else _ptr(counter)), "dp_noise_step_device")


def dp_fill_noise(out: torch.Tensor, sigma: float, C_: float, scale: float, seed: int,
                  tensor_id: int, step: int, n=None, stream=None):
    """out = scale * sigma*C*z (write only), z from the (seed, tensor_id, step) stream."""
    L = load()
    n = out.numel() if n is None else n
    st = L.dp_fill_noise(_ptr(out), n, float(sigma), float(C_), float(scale), int(seed) & (2 ** 64 - 1),
                         int(tensor_id), int(step), _stream(stream))
    _check(st, "dp_fill_noise")


def dp_rdp_epsilon(q: float, sigma: float, steps: int, delta: float):
    """(epsilon, best order) of `steps` DP-SGD steps with sampling rate q and noise multiplier sigma."""
    eps, order = C.c_double(0.0), C.c_int32(0)
    _check(load().dp_rdp_epsilon(float(q), float(sigma), int(steps), float(delta), C.byref(eps),
                                 C.byref(order)), "dp_rdp_epsilon")
    return eps.value, order.value


def dp_sigma_for_epsilon(q: float, steps: int, target_epsilon: float, delta: float,
                         tolerance: float = 1e-6) -> float:
    """Smallest noise multiplier (to `tolerance`) that keeps epsilon within the target."""
    sigma = C.c_double(0.0)
    _check(load().dp_sigma_for_epsilon(float(q), int(steps), float(target_epsilon), float(delta),
                                       float(tolerance), C.byref(sigma)), "dp_sigma_for_epsilon")
    return sigma.value


def dp_set_reserved_sms(n: int) -> int:
    """Leave n SMs free of the library's persistent kernels (for the collectives of another
    stream); returns the previous setting."""
    return int(load().dp_set_reserved_sms(int(n)))


def dp_debug_ghost_single(on: bool) -> bool:
    return bool(load().dp_debug_ghost_single(1 if on else 0))


def dp_debug_force_fma(on: bool) -> bool:
    return bool(load().dp_debug_force_fma(1 if on else 0))


def dp_kernel_launches() -> int:
    return int(load().dp_kernel_launches())


def dp_version() -> str:
    return load().dp_version().decode()
