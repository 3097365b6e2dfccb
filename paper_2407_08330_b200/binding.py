"""ctypes binding of libhdt.so.  Argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os
import re

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIBPATH = os.path.join(_HERE, "libhdt.so")
_HEADERS = [os.path.join(_HERE, "..", "include", h) for h in ("hdt.h", "hdt_debug.h")]
_lib = None

HDT_F32, HDT_BF16 = 0, 1
HDT_MAX_STAGES = 24
_DTYPES = {torch.float32: HDT_F32, torch.bfloat16: HDT_BF16}


class HdtError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"libhdt error {code}: {msg}")
        self.code = code


class _Params(C.Structure):
    _fields_ = [("block_m", C.c_int32), ("max_stages", C.c_int32), ("block_m_upper", C.c_int32),
                ("mask_off", C.c_int32), ("deferred", C.c_int32), ("reserved", C.c_int32 * 3)]


class _StageView(C.Structure):
    _fields_ = [("n", C.c_int32), ("n_blocks", C.c_int32)] + \
               [(nm, C.c_void_p) for nm in ("tok", "par", "rng", "up", "scu", "blocks", "queue", "queue_split")] + \
               [("n_fused", C.c_int32)]


def lib():
    """Load libhdt.so; raises if it has not been built (python -m paper_2407_08330_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIBPATH):
            raise HdtError(-5, f"{_LIBPATH} is missing: build it with `python paper_2407_08330_b200/build.py` "
                               "(there is no fallback path)")
        L = C.CDLL(_LIBPATH)
        L.hdt_index_workspace_bytes.restype = C.c_size_t
        L.hdt_index_workspace_bytes.argtypes = [C.c_int32, C.c_int32, C.c_void_p]
        L.hdt_build_index.restype = C.c_int
        L.hdt_build_index.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p,
                                      C.c_void_p, C.c_size_t, C.c_void_p, C.POINTER(C.c_void_p)]
        L.hdt_index_info.restype = C.c_int
        L.hdt_index_info.argtypes = [C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
        L.hdt_index_export.restype = C.c_int
        L.hdt_index_export.argtypes = [C.c_void_p, C.c_int32, C.POINTER(_StageView)]
        L.hdt_index_destroy.restype = C.c_int
        L.hdt_index_destroy.argtypes = [C.c_void_p]
        L.hdt_attn_workspace_bytes.restype = C.c_size_t
        L.hdt_attn_workspace_bytes.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32]
        L.hdt_attn_fwd.restype = C.c_int
        L.hdt_attn_fwd.argtypes = [C.c_void_p] * 6 + [C.c_int32, C.c_int32, C.c_int32, C.c_float,
                                                      C.c_void_p, C.c_size_t, C.c_void_p]
        L.hdt_attn_bwd.restype = C.c_int
        L.hdt_attn_bwd.argtypes = [C.c_void_p] * 10 + [C.c_int32, C.c_int32, C.c_int32, C.c_float,
                                                       C.c_void_p, C.c_size_t, C.c_void_p]
        L.hdt_last_error.restype = C.c_char_p
        L.hdt_launch_count.restype = C.c_int64
        _lib = L
    return _lib


def declared_symbols():
    """Names of every function the headers under include/ declare."""
    txt = "".join(open(h).read() for h in _HEADERS)
    txt = re.sub(r"/\*.*?\*/", "", txt, flags=re.S)
    return sorted(set(re.findall(r"\b(hdt_[a-z0-9_]+)\s*\(", txt)))


def exported_symbols():
    """(declared, missing): declared functions and those libhdt.so does not export."""
    L = lib()
    names = declared_symbols()
    return names, [n for n in names if not hasattr(L, n)]


def _check(rc):
    if rc != 0:
        raise HdtError(rc, lib().hdt_last_error().decode())


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else C.c_void_p(0)


def _stream():
    # the raw handle of the current stream without building a torch.cuda.Stream object
    return C.c_void_p(torch._C._cuda_getCurrentRawStream(torch.cuda.current_device()))


def _params(block_m, max_stages, block_m_upper=0, directions=7, deferred=False):
    p = _Params()
    p.block_m, p.max_stages, p.block_m_upper = int(block_m), int(max_stages), int(block_m_upper)
    p.mask_off = (~int(directions)) & 7
    p.deferred = 1 if deferred else 0
    return p


def hdt_index_workspace_bytes(batch, total_tokens, block_m=0, max_stages=0, block_m_upper=0) -> int:
    p = _params(block_m, max_stages, block_m_upper)
    return int(lib().hdt_index_workspace_bytes(batch, total_tokens, C.cast(C.byref(p), C.c_void_p)))


class HdtIndex:
    """Owner of a built index: the opaque handle plus the device workspace it points into."""

    def __init__(self, handle, workspace, batch, total_tokens):
        self._h, self._ws = handle, workspace
        self.batch, self.total_tokens = batch, total_tokens
        self._info = None

    def _get_info(self):
        if self._info is None:
            ns, nnz, vis = C.c_int32(), C.c_int64(), C.c_int64()
            _check(lib().hdt_index_info(self._h, C.byref(ns), C.byref(nnz), C.byref(vis)))
            self._info = (ns.value, nnz.value, vis.value)
        return self._info

    @property
    def n_stages(self):
        return self._get_info()[0]

    @property
    def nnz(self):
        return self._get_info()[1]

    @property
    def visited(self):
        return self._get_info()[2]

    @property
    def handle(self):
        return self._h

    def export(self, stage):
        """Device arrays of one stage copied to host numpy arrays (parity tests, inspection)."""
        import numpy as np
        v = _StageView()
        _check(lib().hdt_index_export(self._h, stage, C.byref(v)))
        base = self._ws.data_ptr()

        def arr(ptr, count):
            off = (ptr - base) // 4
            return self._ws.view(torch.int32)[off:off + count].cpu().numpy().copy()
        B = self.batch
        return dict(n=v.n, n_blocks=v.n_blocks, tok=arr(v.tok, v.n), par=arr(v.par, v.n),
                    rng=arr(v.rng, 2 * v.n).reshape(-1, 2), up=arr(v.up, v.n), scu=arr(v.scu, B + 1),
                    blocks=arr(v.blocks, 5 * v.n_blocks).reshape(-1, 5), queue=arr(v.queue, v.n_blocks),
                    queue_split=arr(v.queue_split, v.n_blocks), n_fused=int(v.n_fused))

    def close(self):
        if self._h is not None:
            lib().hdt_index_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def hdt_build_index(level, parent, cu_seqlens, block_m=0, max_stages=0, workspace=None,
                    block_m_upper=0, directions=7, deferred=False) -> HdtIndex:
    """level int8[T], parent int32[T], cu_seqlens int32[B+1]: CUDA tensors.  directions: bits
    1 | 2 | 4 keep the child->parent, sibling<->sibling, parent->child entries (7 = full rule).
    deferred: return once the build is queued; the first call that needs the index's counts on the
    host waits for it (and raises what the build found wrong with the structure arrays)."""
    assert level.is_cuda and parent.is_cuda and cu_seqlens.is_cuda
    assert level.dtype == torch.int8 and parent.dtype == torch.int32 and cu_seqlens.dtype == torch.int32
    level, parent, cu_seqlens = level.contiguous(), parent.contiguous(), cu_seqlens.contiguous()
    T, B = level.numel(), cu_seqlens.numel() - 1
    p = _params(block_m, max_stages, block_m_upper, directions, deferred)
    need = int(lib().hdt_index_workspace_bytes(B, T, C.cast(C.byref(p), C.c_void_p)))
    if need == 0:
        raise HdtError(-1, "invalid index parameters")
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=level.device)
    h = C.c_void_p()
    _check(lib().hdt_build_index(_ptr(level), _ptr(parent), _ptr(cu_seqlens), B, T, C.cast(C.byref(p), C.c_void_p),
                                 _ptr(workspace), workspace.numel(), _stream(), C.byref(h)))
    return HdtIndex(h, workspace, B, T)


def hdt_attn_workspace_bytes(index: HdtIndex, heads, head_dim, dtype, bwd) -> int:
    return int(lib().hdt_attn_workspace_bytes(index.handle, heads, head_dim, _DTYPES[dtype], int(bwd)))


def _ws(index, heads, head_dim, dtype, bwd, device, workspace):
    if workspace is not None:      # the library checks the size itself
        return workspace, None
    need = hdt_attn_workspace_bytes(index, heads, head_dim, dtype, bwd)
    return torch.empty(max(need, 256), dtype=torch.uint8, device=device), need


def hdt_attn_fwd(index: HdtIndex, q, k, v, softmax_scale=0.0, out=None, lse=None, workspace=None):
    """q, k, v: CUDA [T, H, d] float32 or bfloat16, contiguous.  Returns (O, LSE [H, T])."""
    T, H, d = q.shape
    assert q.is_contiguous() and k.is_contiguous() and v.is_contiguous() and q.dtype == k.dtype == v.dtype
    o = torch.empty_like(q) if out is None else out
    lse = torch.empty((H, T), dtype=torch.float32, device=q.device) if lse is None else lse
    workspace, need = _ws(index, H, d, q.dtype, 0, q.device, workspace)
    _check(lib().hdt_attn_fwd(index.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), H, d,
                              _DTYPES[q.dtype], float(softmax_scale), _ptr(workspace), workspace.numel(),
                              _stream()))
    return o, lse


def hdt_attn_bwd(index: HdtIndex, q, k, v, o, lse, d_o, softmax_scale=0.0, dq=None, dk=None, dv=None,
                 workspace=None):
    """Returns (dQ, dK, dV) with the shape and dtype of q."""
    T, H, d = q.shape
    for t in (q, k, v, o, d_o):
        assert t.is_contiguous() and t.dtype == q.dtype
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(q) if dk is None else dk
    dv = torch.empty_like(q) if dv is None else dv
    workspace, need = _ws(index, H, d, q.dtype, 1, q.device, workspace)
    _check(lib().hdt_attn_bwd(index.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(d_o),
                              _ptr(dq), _ptr(dk), _ptr(dv), H, d, _DTYPES[q.dtype], float(softmax_scale),
                              _ptr(workspace), workspace.numel(), _stream()))
    return dq, dk, dv


def hdt_attn_fwd_static_max_bytes() -> int:
    lib().hdt_attn_fwd_static_max_bytes.restype = C.c_size_t
    return int(lib().hdt_attn_fwd_static_max_bytes())


def hdt_attn_fwd_static(index: HdtIndex, q, k, v, softmax_scale=0.0, out=None, lse=None):
    """Forward pass for callers that may not allocate device memory during the call: the scratch
    for the upper stages' partial results is a fixed array inside the library, so nothing is
    allocated here as long as `out` and `lse` are passed in.  Raises HdtError (-4) when the batch
    needs more scratch than hdt_attn_fwd_static_max_bytes().  Calls must not overlap on the GPU."""
    T, H, d = q.shape
    assert q.is_contiguous() and k.is_contiguous() and v.is_contiguous() and q.dtype == k.dtype == v.dtype
    o = torch.empty_like(q) if out is None else out
    lse = torch.empty((H, T), dtype=torch.float32, device=q.device) if lse is None else lse
    f = lib().hdt_attn_fwd_static
    f.restype = C.c_int
    f.argtypes = [C.c_void_p] * 6 + [C.c_int32, C.c_int32, C.c_int32, C.c_float, C.c_void_p]
    _check(f(index.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), H, d, _DTYPES[q.dtype],
             float(softmax_scale), _stream()))
    return o, lse


def hdt_hpe_workspace_bytes(index: HdtIndex, n_levels=3) -> int:
    L = lib()
    L.hdt_hpe_workspace_bytes.restype = C.c_size_t
    L.hdt_hpe_workspace_bytes.argtypes = [C.c_void_p, C.c_int32]
    return int(L.hdt_hpe_workspace_bytes(index.handle, n_levels))


def hdt_hpe(index: HdtIndex, level, parent, cu_seqlens, d_model, n_levels=3, dtype=torch.float32, x=None,
            accumulate=False, workspace=None):
    """Hierarchical positional encoding [T, d_model]; with `x` and accumulate=True it is added to x."""
    L = lib()
    L.hdt_hpe_workspace_bytes.restype = C.c_size_t
    L.hdt_hpe_workspace_bytes.argtypes = [C.c_void_p, C.c_int32]
    L.hdt_hpe.restype = C.c_int
    L.hdt_hpe.argtypes = [C.c_void_p] * 4 + [C.c_int32] * 4 + [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    T = level.numel()
    if x is None:
        x = torch.empty((T, d_model), dtype=dtype, device=level.device)
    assert x.is_contiguous() and x.shape == (T, d_model)
    need = int(L.hdt_hpe_workspace_bytes(index.handle, n_levels))
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=level.device)
    _check(L.hdt_hpe(index.handle, _ptr(level), _ptr(parent), _ptr(cu_seqlens), n_levels, d_model, _DTYPES[x.dtype],
                     int(bool(accumulate)), _ptr(x), _ptr(workspace), workspace.numel(), _stream()))
    return x


def hdt_cross_workspace_bytes(batch, total_tokens, total_q, heads, head_dim, dtype, bwd) -> int:
    L = lib()
    L.hdt_cross_workspace_bytes.restype = C.c_size_t
    L.hdt_cross_workspace_bytes.argtypes = [C.c_int32] * 7
    return int(L.hdt_cross_workspace_bytes(batch, total_tokens, total_q, heads, head_dim, _DTYPES[dtype], int(bwd)))


def _cross_common(level, cu_seqlens_k, cu_seqlens_q, q, k):
    assert level.dtype == torch.int8 and cu_seqlens_k.dtype == torch.int32 and cu_seqlens_q.dtype == torch.int32
    Tq, H, d = q.shape
    T, B = k.shape[0], cu_seqlens_k.numel() - 1
    assert cu_seqlens_q.numel() == B + 1 and level.numel() == T
    return B, T, Tq, H, d


def hdt_cross_attn_fwd(level, cu_seqlens_k, cu_seqlens_q, level_mask, q, k, v, softmax_scale=0.0, out=None, lse=None,
                       workspace=None):
    """Decoder rows q [Tq,H,d] attend to the encoder rows of k, v [T,H,d] whose level bit is set in
    level_mask.  Returns (O [Tq,H,d], LSE [H,Tq])."""
    L = lib()
    L.hdt_cross_attn_fwd.restype = C.c_int
    L.hdt_cross_attn_fwd.argtypes = [C.c_void_p] * 3 + [C.c_int32] * 4 + [C.c_void_p] * 5 + [C.c_int32] * 3 + \
                                    [C.c_float, C.c_void_p, C.c_size_t, C.c_void_p]
    B, T, Tq, H, d = _cross_common(level, cu_seqlens_k, cu_seqlens_q, q, k)
    assert q.is_contiguous() and k.is_contiguous() and v.is_contiguous()
    if out is None:
        out = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((H, Tq), dtype=torch.float32, device=q.device)
    need = hdt_cross_workspace_bytes(B, T, Tq, H, d, q.dtype, 0)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    _check(L.hdt_cross_attn_fwd(_ptr(level), _ptr(cu_seqlens_k), _ptr(cu_seqlens_q), B, T, Tq, int(level_mask), _ptr(q),
                                _ptr(k), _ptr(v), _ptr(out), _ptr(lse), H, d, _DTYPES[q.dtype], float(softmax_scale),
                                _ptr(workspace), workspace.numel(), _stream()))
    return out, lse


def hdt_cross_attn_bwd(level, cu_seqlens_k, cu_seqlens_q, level_mask, q, k, v, o, lse, do, softmax_scale=0.0, dq=None,
                       dk=None, dv=None, workspace=None):
    """Gradients (dQ [Tq,H,d], dK, dV [T,H,d]) of hdt_cross_attn_fwd."""
    L = lib()
    L.hdt_cross_attn_bwd.restype = C.c_int
    L.hdt_cross_attn_bwd.argtypes = [C.c_void_p] * 3 + [C.c_int32] * 4 + [C.c_void_p] * 9 + [C.c_int32] * 3 + \
                                    [C.c_float, C.c_void_p, C.c_size_t, C.c_void_p]
    B, T, Tq, H, d = _cross_common(level, cu_seqlens_k, cu_seqlens_q, q, k)
    assert all(x.is_contiguous() for x in (q, k, v, o, do))
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(k) if dk is None else dk
    dv = torch.empty_like(v) if dv is None else dv
    need = hdt_cross_workspace_bytes(B, T, Tq, H, d, q.dtype, 1)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    _check(L.hdt_cross_attn_bwd(_ptr(level), _ptr(cu_seqlens_k), _ptr(cu_seqlens_q), B, T, Tq, int(level_mask), _ptr(q),
                                _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(do), _ptr(dq), _ptr(dk), _ptr(dv), H, d,
                                _DTYPES[q.dtype], float(softmax_scale), _ptr(workspace), workspace.numel(), _stream()))
    return dq, dk, dv


def hdt_set_option(name: str, value: int) -> None:
    lib().hdt_set_option.restype = C.c_int
    _check(lib().hdt_set_option(C.c_char_p(name.encode()), C.c_int32(int(value))))


def hdt_device_status() -> None:
    """Wait for the current stream and raise if a kernel recorded a device-side failure."""
    lib().hdt_device_status.restype = C.c_int
    _check(lib().hdt_device_status(_stream()))


def hdt_launch_count() -> int:
    return int(lib().hdt_launch_count())
