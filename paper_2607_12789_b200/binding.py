"""ctypes binding of libavq_attn (``include/avq_attn.h``): argument marshalling only.

Every function here hands torch device pointers and the current CUDA stream to the
C ABI; no step of the computation runs in Python or torch.  If the shared library
has not been built the first call raises - there is no CPU or torch fallback.
"""
from __future__ import annotations

import ctypes
import math
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "lib", "libavq_attn.so")

AVQ_F32, AVQ_BF16 = 0, 1
FLAG_PARENT_STAYS, FLAG_SIMT, FLAG_CORRECTING = 1, 2, 4
STATUS_NAMES = {0: "AVQ_OK", 1: "AVQ_ERR_NULL", 2: "AVQ_ERR_SHAPE", 3: "AVQ_ERR_UNSUPPORTED", 4: "AVQ_ERR_ALIGN",
                5: "AVQ_ERR_WORKSPACE", 6: "AVQ_ERR_CUDA", 7: "AVQ_ERR_DEVICE_TIMEOUT", 8: "AVQ_ERR_INDEX"}

EXPORTS = ("avq_workspace_bytes", "avq_assign", "avq_aggregate", "avq_forward", "avq_forward_host", "avq_attend",
           "avq_workspace_layout", "avq_check", "avq_status_string", "avq_version", "avq_forward_static",
           "avq_check_static", "avq_static_workspace_bytes", "avq_workspace_bytes_permuted",
           "avq_forward_permuted", "avq_codebook_update_workspace_bytes", "avq_codebook_update",
           "avq_forward_tiled")


class AvqProblem(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("H", ctypes.c_int32), ("Nq", ctypes.c_int32), ("Nk", ctypes.c_int32),
                ("d", ctypes.c_int32), ("M", ctypes.c_int32), ("C", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("scale", ctypes.c_float), ("flags", ctypes.c_uint32)]


class AvqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().avq_status_string(status).decode()
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} ({msg})")


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded shared library (loaded on first use)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2607_12789_b200.build` "
                               "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
        pp = ctypes.POINTER(AvqProblem)
        psz = ctypes.POINTER(ctypes.c_size_t)
        L.avq_workspace_bytes.restype, L.avq_workspace_bytes.argtypes = sz, [pp, i32, i32]
        L.avq_assign.restype, L.avq_assign.argtypes = i32, [pp, vp, vp, vp, vp, vp, vp]
        L.avq_aggregate.restype, L.avq_aggregate.argtypes = i32, [pp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.avq_forward.restype = i32
        L.avq_forward.argtypes = [pp, vp, vp, vp, vp, vp, i32, i32, vp, vp, vp, vp, sz, vp]
        L.avq_forward_host.restype = i32
        L.avq_forward_host.argtypes = [pp, vp, vp, vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, vp, sz, vp]
        L.avq_attend.restype = i32
        L.avq_attend.argtypes = [pp, vp, vp, vp, i32, i32, vp, vp, vp, vp, sz, vp]
        L.avq_workspace_layout.restype = i32
        L.avq_workspace_layout.argtypes = [pp, i32, i32, psz, psz, psz, psz, psz, psz]
        L.avq_check.restype, L.avq_check.argtypes = i32, [vp, vp]
        L.avq_forward_static.restype = i32
        L.avq_forward_static.argtypes = [pp, vp, vp, vp, vp, vp, i32, i32, vp, vp, vp, vp]
        L.avq_check_static.restype, L.avq_check_static.argtypes = i32, [vp]
        L.avq_static_workspace_bytes.restype, L.avq_static_workspace_bytes.argtypes = sz, []
        L.avq_workspace_bytes_permuted.restype, L.avq_workspace_bytes_permuted.argtypes = sz, [pp, i32, i32]
        L.avq_forward_permuted.restype = i32
        L.avq_forward_permuted.argtypes = [pp, vp, vp, vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, sz, vp]
        L.avq_forward_tiled.restype = i32
        L.avq_forward_tiled.argtypes = [pp, vp, vp, vp, vp, vp, i32, i32, i32, vp, vp, vp, vp, sz, vp]
        L.avq_codebook_update_workspace_bytes.restype, L.avq_codebook_update_workspace_bytes.argtypes = sz, [pp]
        L.avq_codebook_update.restype = i32
        L.avq_codebook_update.argtypes = [pp, vp, vp, vp, ctypes.c_float, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.avq_status_string.restype, L.avq_status_string.argtypes = ctypes.c_char_p, [i32]
        L.avq_version.restype, L.avq_version.argtypes = i32, []
        _lib = L
    return _lib


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return AVQ_F32
    if t.dtype == torch.bfloat16:
        return AVQ_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _ptr(t: torch.Tensor | None):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _chk(*ts: torch.Tensor) -> None:
    for t in ts:
        if not t.is_cuda or not t.is_contiguous():
            raise ValueError("tensors must be contiguous CUDA tensors")


def problem(B, H, Nq, Nk, d, M, C, dtype_code, scale, flags=0) -> AvqProblem:
    return AvqProblem(B, H, Nq, Nk, d, M, C, dtype_code, float(scale), flags)


def _problem_from(Q, K, Cp, Cc, scale, flags) -> AvqProblem:
    B, H, Nk, d = K.shape
    Nq = Q.shape[2] if Q is not None else Nk
    Hc, M, C, dc = Cc.shape
    if tuple(Cp.shape) != (H, M, d) or Hc != H or dc != d:
        raise ValueError("codebook shapes must be Cp [H,M,d], Cc [H,M,C,d]")
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    return problem(B, H, Nq, Nk, d, M, C, _dtype_code(K), scale, flags)


def workspace_bytes(prob: AvqProblem, P: int, block_q: int) -> int:
    return int(lib().avq_workspace_bytes(ctypes.byref(prob), P, block_q))


def assign(K, Cp, Cc, flags: int = 0):
    """avq_assign: returns (parent_idx, child_idx), int32 [B,H,Nk]."""
    _chk(K, Cp, Cc)
    prob = _problem_from(None, K, Cp, Cc, 1.0, flags)
    B, H, Nk, _ = K.shape
    pidx = torch.empty((B, H, Nk), dtype=torch.int32, device=K.device)
    cidx = torch.empty_like(pidx)
    st = lib().avq_assign(ctypes.byref(prob), _ptr(K), _ptr(Cp), _ptr(Cc), _ptr(pidx), _ptr(cidx), _stream())
    if st != 0:
        raise AvqError(st, "avq_assign")
    return pidx, cidx


def aggregate(V, parent_idx, child_idx, M: int, C: int, flags: int = 0):
    """avq_aggregate: returns (Vp [B,H,M,d], np [B,H,M], Vc [B,H,M,C,d], nc [B,H,M,C]), float32."""
    _chk(V, parent_idx, child_idx)
    B, H, Nk, d = V.shape
    prob = problem(B, H, Nk, Nk, d, M, C, _dtype_code(V), 1.0, flags)
    f32 = dict(dtype=torch.float32, device=V.device)
    Vp, n_p = torch.empty((B, H, M, d), **f32), torch.empty((B, H, M), **f32)
    Vc, n_c = torch.empty((B, H, M, C, d), **f32), torch.empty((B, H, M, C), **f32)
    st = lib().avq_aggregate(ctypes.byref(prob), _ptr(V), _ptr(parent_idx), _ptr(child_idx), _ptr(Vp), _ptr(n_p),
                             _ptr(Vc), _ptr(n_c), _stream())
    if st != 0:
        raise AvqError(st, "avq_aggregate")
    return Vp, n_p, Vc, n_c


class Forward:
    """Pre-sized buffers for repeated ``avq_forward`` calls on one problem shape."""

    def __init__(self, B, H, Nq, Nk, d, M, C, P, block_q, dtype=torch.bfloat16, scale=None, flags=0,
                 device="cuda", aux=False):
        self.P, self.block_q = P, block_q
        code = AVQ_F32 if dtype == torch.float32 else AVQ_BF16
        self.prob = problem(B, H, Nq, Nk, d, M, C, code, scale if scale is not None else 1.0 / math.sqrt(d), flags)
        nbytes = workspace_bytes(self.prob, P, block_q)
        if nbytes == 0:
            st = lib().avq_workspace_layout(ctypes.byref(self.prob), P, block_q, None, None, None, None, None, None)
            raise AvqError(st, "avq_workspace_bytes")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=device)
        self.nblk = (Nq + block_q - 1) // block_q
        self.topp = torch.empty((B, H, self.nblk, P), dtype=torch.int32, device=device) if aux else None
        self.importance = torch.empty((B, H, self.nblk, M), dtype=torch.float32, device=device) if aux else None
        self.dtype, self.device = dtype, device
        self.shape_y = (B, H, Nq, d)

    def __call__(self, Q, K, V, Cp, Cc, Y=None):
        _chk(Q, K, V, Cp, Cc)
        if Y is None:
            Y = torch.empty(self.shape_y, dtype=self.dtype, device=Q.device)
        st = lib().avq_forward(ctypes.byref(self.prob), _ptr(Q), _ptr(K), _ptr(V), _ptr(Cp), _ptr(Cc), self.P,
                               self.block_q, _ptr(Y), _ptr(self.topp), _ptr(self.importance),
                               _ptr(self.workspace), self.workspace.numel(), _stream())
        if st != 0:
            raise AvqError(st, "avq_forward")
        return Y

    def attend(self, Q, Cp, Cc, Y=None):
        """avq_attend: stage 3 only, over the aggregates the last full call left in the workspace."""
        _chk(Q, Cp, Cc)
        if Y is None:
            Y = torch.empty(self.shape_y, dtype=self.dtype, device=Q.device)
        st = lib().avq_attend(ctypes.byref(self.prob), _ptr(Q), _ptr(Cp), _ptr(Cc), self.P, self.block_q, _ptr(Y),
                              _ptr(self.topp), _ptr(self.importance), _ptr(self.workspace),
                              self.workspace.numel(), _stream())
        if st != 0:
            raise AvqError(st, "avq_attend")
        return Y

    def host(self, hQ, hK, hV, Cp, Cc, hY, dQ, dK, dV, dY):
        """avq_forward_host: Q, K, V, Y in (pinned) host tensors, staged through dQ..dY."""
        st = lib().avq_forward_host(ctypes.byref(self.prob), _ptr(hQ), _ptr(hK), _ptr(hV), _ptr(Cp), _ptr(Cc),
                                    self.P, self.block_q, _ptr(hY), _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(dY),
                                    _ptr(self.workspace), self.workspace.numel(), _stream())
        if st != 0:
            raise AvqError(st, "avq_forward_host")
        return hY

    def check(self) -> None:
        """avq_check: raises if a kernel recorded an expired device-side wait."""
        st = lib().avq_check(_ptr(self.workspace), _stream())
        if st != 0:
            raise AvqError(st, "avq_check")

    def intermediates(self):
        """Views of the indices and aggregates the last call left in the workspace."""
        offs = [ctypes.c_size_t() for _ in range(6)]
        st = lib().avq_workspace_layout(ctypes.byref(self.prob), self.P, self.block_q, *[ctypes.byref(o) for o in offs])
        if st != 0:
            raise AvqError(st, "avq_workspace_layout")
        p = self.prob
        BH = (p.B, p.H)

        def view(off, shape, dt):
            n = math.prod(shape) * 4
            return self.workspace[off.value:off.value + n].view(dt).view(*shape)

        return dict(parent_idx=view(offs[0], (*BH, p.Nk), torch.int32),
                    child_idx=view(offs[1], (*BH, p.Nk), torch.int32),
                    Vp=view(offs[2], (*BH, p.M, p.d), torch.float32), np=view(offs[3], (*BH, p.M), torch.float32),
                    Vc=view(offs[4], (*BH, p.M, p.C, p.d), torch.float32),
                    nc=view(offs[5], (*BH, p.M, p.C), torch.float32))


def forward(Q, K, V, Cp, Cc, P: int, block_q: int, scale=None, flags: int = 0, aux: bool = False):
    """One-shot avq_forward.  Returns Y, or (Y, topp, importance, intermediates) with ``aux``."""
    B, H, Nq, d = Q.shape
    Nk = K.shape[2]
    M, C = Cc.shape[1], Cc.shape[2]
    f = Forward(B, H, Nq, Nk, d, M, C, P, block_q, dtype=Q.dtype, scale=scale, flags=flags, device=Q.device,
                aux=aux)
    Y = f(Q, K, V, Cp, Cc)
    f.check()
    if aux:
        return Y, f.topp, f.importance, f.intermediates()
    return Y


def forward_permuted(Q, K, V, Cp, Cc, P: int, block_q: int, perm, scale=None, flags: int = 0):
    """avq_forward_permuted: query tiles follow ``perm`` (int32 [Nq]).  Returns (Y, topp, importance, status)
    where status is what avq_check reports after the call (0, or 8 if perm held an index out of range)."""
    _chk(Q, K, V, Cp, Cc, perm)
    prob = _problem_from(Q, K, Cp, Cc, scale, flags)
    B, H, Nq, d = Q.shape
    nblk = (Nq + block_q - 1) // block_q
    nbytes = int(lib().avq_workspace_bytes_permuted(ctypes.byref(prob), P, block_q))
    if nbytes == 0:
        raise AvqError(lib().avq_workspace_layout(ctypes.byref(prob), P, block_q, None, None, None, None, None, None)
                       or 3, "avq_workspace_bytes_permuted")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=Q.device)
    Y = torch.zeros_like(Q)
    topp = torch.empty((B, H, nblk, P), dtype=torch.int32, device=Q.device)
    imp = torch.empty((B, H, nblk, prob.M), dtype=torch.float32, device=Q.device)
    st = lib().avq_forward_permuted(ctypes.byref(prob), _ptr(Q), _ptr(K), _ptr(V), _ptr(Cp), _ptr(Cc), P, block_q,
                                    _ptr(perm), _ptr(Y), _ptr(topp), _ptr(imp), _ptr(ws), nbytes, _stream())
    if st != 0:
        raise AvqError(st, "avq_forward_permuted")
    return Y, topp, imp, int(lib().avq_check(_ptr(ws), _stream()))


def forward_tiled(Q, K, V, Cp, Cc, P: int, block_q: int, tile_m: int, scale=None, flags: int = 0):
    """avq_forward_tiled: selection from the tiled importance.  Returns (Y, topp, importance)."""
    _chk(Q, K, V, Cp, Cc)
    prob = _problem_from(Q, K, Cp, Cc, scale, flags | FLAG_SIMT)
    B, H, Nq, d = Q.shape
    nblk = (Nq + block_q - 1) // block_q
    nbytes = workspace_bytes(prob, P, block_q)
    if nbytes == 0:
        raise AvqError(lib().avq_workspace_layout(ctypes.byref(prob), P, block_q, None, None, None, None, None, None)
                       or 3, "avq_workspace_bytes")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=Q.device)
    Y = torch.empty_like(Q)
    topp = torch.empty((B, H, nblk, P), dtype=torch.int32, device=Q.device)
    imp = torch.empty((B, H, nblk, prob.M), dtype=torch.float32, device=Q.device)
    st = lib().avq_forward_tiled(ctypes.byref(prob), _ptr(Q), _ptr(K), _ptr(V), _ptr(Cp), _ptr(Cc), P, block_q,
                                 tile_m, _ptr(Y), _ptr(topp), _ptr(imp), _ptr(ws), nbytes, _stream())
    if st != 0:
        raise AvqError(st, "avq_forward_tiled")
    return Y, topp, imp


def codebook_update(K, Cp, Cc, Sp, Np, Sc, Nc, decay: float, flags: int = 0):
    """avq_codebook_update: EMA statistics (updated in place) and the new codebooks (Cp', Cc')."""
    _chk(K, Cp, Cc, Sp, Np, Sc, Nc)
    prob = _problem_from(None, K, Cp, Cc, 1.0, flags)
    nbytes = int(lib().avq_codebook_update_workspace_bytes(ctypes.byref(prob)))
    ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=K.device)
    Cp2, Cc2 = torch.empty_like(Cp), torch.empty_like(Cc)
    st = lib().avq_codebook_update(ctypes.byref(prob), _ptr(K), _ptr(Cp), _ptr(Cc), decay, _ptr(Sp), _ptr(Np),
                                   _ptr(Sc), _ptr(Nc), _ptr(Cp2), _ptr(Cc2), _ptr(ws), ws.numel(), _stream())
    if st != 0:
        raise AvqError(st, "avq_codebook_update")
    return Cp2, Cc2


def forward_static(Q, K, V, Cp, Cc, P: int, block_q: int, scale=None, flags: int = 0, aux: bool = False):
    """avq_forward_static: the forward pass in the library's built-in scratch array, for callers
    that cannot allocate a workspace.  Only the outputs are torch tensors here; nothing else is
    allocated on the device.  Returns Y, or (Y, topp, importance) with ``aux``."""
    _chk(Q, K, V, Cp, Cc)
    prob = _problem_from(Q, K, Cp, Cc, scale, flags)
    B, H, Nq, d = Q.shape
    nblk = (Nq + block_q - 1) // block_q
    Y = torch.empty_like(Q)
    topp = torch.empty((B, H, nblk, P), dtype=torch.int32, device=Q.device) if aux else None
    imp = torch.empty((B, H, nblk, prob.M), dtype=torch.float32, device=Q.device) if aux else None
    st = lib().avq_forward_static(ctypes.byref(prob), _ptr(Q), _ptr(K), _ptr(V), _ptr(Cp), _ptr(Cc), P, block_q,
                                  _ptr(Y), _ptr(topp), _ptr(imp), _stream())
    if st != 0:
        raise AvqError(st, "avq_forward_static")
    st = lib().avq_check_static(_stream())
    if st != 0:
        raise AvqError(st, "avq_check_static")
    return (Y, topp, imp) if aux else Y
