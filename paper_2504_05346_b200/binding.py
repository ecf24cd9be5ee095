"""ctypes binding of libthanos.so: same names as the C ABI, argument marshalling only."""

from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))

F32, BF16 = 0, 1
UNSTRUCTURED, NM = 0, 1
WS_HESSIAN, WS_PREPARE, WS_PRUNE, WS_HOST_LAYER, WS_PRUNE_OUTLIERS = 0, 1, 2, 3, 4


class ThanosError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s failed: %s (status %d)" % (where, status_string(code), code))


class _Stats(ctypes.Structure):
    _fields_ = [
        ("status", ctypes.c_int32),
        ("err_index", ctypes.c_int32),
        ("n_pruned", ctypes.c_int64),
        ("r_left", ctypes.c_int64),
        ("max_s", ctypes.c_int32),
        ("n_blocks", ctypes.c_int32),
        ("n_tied", ctypes.c_int64),
        ("last_threshold_bits", ctypes.c_uint32),
        ("select_misses", ctypes.c_int32),
        ("select_rescans", ctypes.c_int32),
        ("reserved", ctypes.c_int32 * 3),
    ]


assert ctypes.sizeof(_Stats) == 64


@dataclass
class PruneStats:
    status: int
    err_index: int
    n_pruned: int
    r_left: int
    max_s: int
    n_blocks: int
    n_tied: int
    last_threshold_bits: int
    select_misses: int = 0
    select_rescans: int = 0

    @staticmethod
    def from_bytes(raw: bytes) -> "PruneStats":
        s = _Stats.from_buffer_copy(raw)
        return PruneStats(s.status, s.err_index, s.n_pruned, s.r_left, s.max_s, s.n_blocks,
                          s.n_tied, s.last_threshold_bits, s.select_misses, s.select_rescans)


_lib = None


def lib_path() -> str:
    return os.path.join(_HERE, "libthanos.so")


def load_library():
    """Load libthanos.so.  There is no fallback: a missing library is an error."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        raise FileNotFoundError(
            "%s is missing: build it with `python -m paper_2504_05346_b200.build` "
            "(there is no CPU or PyTorch fallback)" % path)
    lib = ctypes.CDLL(path)
    vp, i64, i32, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_size_t
    lib.thanos_hessian_accumulate.argtypes = [vp, i64, vp, i32, i64, i64, vp, sz, vp]
    lib.thanos_hessian_accumulate.restype = i32
    lib.thanos_hessian_accumulate_ordered.argtypes = [vp, i64, vp, i32, i64, i64, vp, sz, vp]
    lib.thanos_hessian_accumulate_ordered.restype = i32
    lib.thanos_prepare_inverse.argtypes = [vp, i64, ctypes.c_float, vp, vp, vp, sz, vp, vp]
    lib.thanos_prepare_inverse.restype = i32
    lib.thanos_prune_layer.argtypes = [vp, vp, vp, i32, i64, i64, vp, vp, i32, ctypes.c_double,
                                       i32, i32, i32, vp, sz, vp, vp]
    lib.thanos_prune_layer.restype = i32
    lib.thanos_prune_layer_outliers.argtypes = [vp, vp, vp, i32, i64, i64, vp, vp, vp, i32, i32, i32,
                                                ctypes.c_double, vp, vp, sz, vp, vp]
    lib.thanos_prune_layer_outliers.restype = i32
    lib.thanos_prune_layer_structured.argtypes = [vp, vp, vp, vp, i32, i64, i64, vp, vp, vp,
                                                  ctypes.c_double, ctypes.c_double, vp, sz, vp, vp]
    lib.thanos_prune_layer_structured.restype = i32
    lib.thanos_structured_workspace_bytes.argtypes = [i64, i64, ctypes.c_double, ctypes.c_double,
                                                      i32]
    lib.thanos_structured_workspace_bytes.restype = sz
    lib.thanos_prune_block.argtypes = [vp, vp, i64, i64, vp, vp, i32, i32, i32, i32, i64, vp, vp,
                                       sz, vp, vp]
    lib.thanos_prune_block.restype = i32
    lib.thanos_prune_layer_host.argtypes = [vp, vp, vp, vp, i32, i64, i64, i64, ctypes.c_float,
                                            i32, ctypes.c_double, i32, i32, i32, i32, vp, sz,
                                            ctypes.POINTER(_Stats), vp]
    lib.thanos_prune_layer_host.restype = i32
    lib.thanos_prune_layer_noalloc.argtypes = [vp, vp, vp, i32, i64, i64, vp, vp, i32,
                                               ctypes.c_double, i32, i32, i32, vp, vp]
    lib.thanos_prune_layer_noalloc.restype = i32
    lib.thanos_dense_product.argtypes = [vp, i64, vp, i64, vp, i64, i32, i64, i64, i64,
                                         ctypes.c_float, i32, vp, sz, vp]
    lib.thanos_dense_product.restype = i32
    lib.thanos_dense_product_workspace.argtypes = [i64, i64, i64]
    lib.thanos_dense_product_workspace.restype = sz
    lib.thanos_fp32_fma_probe.argtypes = [vp, i64, i32, i32, ctypes.POINTER(ctypes.c_double), vp]
    lib.thanos_fp32_fma_probe.restype = i32
    lib.thanos_workspace_bytes.argtypes = [i32, i64, i64, i32, i32]
    lib.thanos_workspace_bytes.restype = sz
    lib.thanos_status_string.argtypes = [i32]
    lib.thanos_status_string.restype = ctypes.c_char_p
    lib.thanos_version.argtypes = []
    lib.thanos_version.restype = i32
    lib.thanos_launch_count.argtypes = []
    lib.thanos_launch_count.restype = i64
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().thanos_status_string(int(code)).decode()


def version() -> int:
    return int(load_library().thanos_version())


def launch_count() -> int:
    return int(load_library().thanos_launch_count())


def workspace_bytes(which: int, c: int, b: int, B: int, dtype: int) -> int:
    return int(load_library().thanos_workspace_bytes(which, c, b, B, dtype))


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("unsupported dtype %s (float32 or bfloat16)" % t.dtype)


def _stream_ptr(stream) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def _check_dev(*ts):
    for t in ts:
        if not t.is_cuda or not t.is_contiguous():
            raise ValueError("expected contiguous CUDA tensors")


def _ws(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def _check(code: int, where: str):
    if code != 0:
        raise ThanosError(code, where)


def _on(t: torch.Tensor):
    """Makes the tensor's device current for the duration of a library call (kernels are
    launched on, and per-device state is looked up for, the current device)."""
    return torch.cuda.device(t.device)


def hessian_status(workspace: torch.Tensor) -> int:
    """Device status word of the last thanos_hessian_accumulate call that used `workspace`
    (synchronises): 0, or THANOS_ERR_TIMEOUT (7) if a bounded wait inside the kernel ran out."""
    return int(workspace[:4].view(torch.int32).item())


def hessian_accumulate(H: torch.Tensor, X: torch.Tensor, stream=None,
                       workspace: Optional[torch.Tensor] = None, check: bool = False,
                       ordered: bool = False) -> None:
    """H += 2 X^T X for tokens-major X [n_tok, b] (float32 or bfloat16); H float32 [b, b].
    With check=True the call's device status word is read back (this waits for the call) and a
    non-zero status raises.  ordered=True calls thanos_hessian_accumulate_ordered (fixed
    summation order: bit-reproducible results)."""
    lib = load_library()
    if not X.is_cuda or X.stride(-1) != 1:
        raise ValueError("X must be a CUDA tensor with unit inner stride")
    _check_dev(H)
    b = H.shape[0]
    n_tok = X.shape[0]
    ldx = X.stride(0) if n_tok > 1 else b
    dt = _dtype_code(X)
    if workspace is None:
        workspace = _ws(workspace_bytes(WS_HESSIAN, 0, b, 0, dt), H.device)
    with _on(H):
        fn = lib.thanos_hessian_accumulate_ordered if ordered else lib.thanos_hessian_accumulate
        _check(fn(H.data_ptr(), b, X.data_ptr(), dt, n_tok, ldx, workspace.data_ptr(),
                  workspace.numel(), _stream_ptr(stream)), "thanos_hessian_accumulate")
        if check and n_tok > 0:
            st = hessian_status(workspace)
            if st != 0:
                raise ThanosError(st, "thanos_hessian_accumulate (device)")


def prepare_inverse(H: torch.Tensor, damp_rel: float, stream=None,
                    workspace: Optional[torch.Tensor] = None, check: bool = True,
                    factor: Optional[torch.Tensor] = None,
                    xnorm: Optional[torch.Tensor] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Returns (factor U [b, b] upper-triangular with U^T U = (H + damp I)^-1, xnorm [b]);
    pass `factor` / `xnorm` to have them written into existing buffers."""
    lib = load_library()
    _check_dev(H)
    b = H.shape[0]
    if factor is None:
        factor = torch.empty((b, b), dtype=torch.float32, device=H.device)
    if xnorm is None:
        xnorm = torch.empty((b,), dtype=torch.float32, device=H.device)
    _check_dev(factor, xnorm)
    status = torch.zeros(4, dtype=torch.int32, device=H.device)
    if workspace is None:
        workspace = _ws(workspace_bytes(WS_PREPARE, 0, b, 0, F32), H.device)
    with _on(H):
        _check(lib.thanos_prepare_inverse(H.data_ptr(), b, float(damp_rel), factor.data_ptr(),
                                          xnorm.data_ptr(), workspace.data_ptr(),
                                          workspace.numel(), status.data_ptr(),
                                          _stream_ptr(stream)), "thanos_prepare_inverse")
    if check:
        st = status.cpu()
        if int(st[0]) != 0:
            raise ThanosError(int(st[0]), "thanos_prepare_inverse (column %d)" % int(st[1]))
    return factor, xnorm


def _read_stats(stats_dev: torch.Tensor) -> PruneStats:
    return PruneStats.from_bytes(bytes(stats_dev.cpu().numpy().tobytes()))


def prune_layer(W: torch.Tensor, factor: torch.Tensor, xnorm: torch.Tensor, mode: int,
                p: float = 0.0, n: int = 0, m: int = 0, B: int = 128, stream=None,
                workspace: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None,
                mask: Optional[torch.Tensor] = None, read_stats: bool = True):
    """Block sweep over one layer.  Returns (W_pruned, mask uint8, PruneStats | stats tensor)."""
    lib = load_library()
    _check_dev(W, factor, xnorm)
    c, b = W.shape
    dt = _dtype_code(W)
    if out is None:
        out = torch.empty_like(W)
    if mask is None:
        mask = torch.empty((c, b), dtype=torch.uint8, device=W.device)
    stats = torch.zeros(64, dtype=torch.uint8, device=W.device)
    if workspace is None:
        workspace = _ws(workspace_bytes(WS_PRUNE, c, b, B, dt), W.device)
    with _on(W):
        _check(lib.thanos_prune_layer(W.data_ptr(), out.data_ptr(), mask.data_ptr(), dt, c, b,
                                      factor.data_ptr(), xnorm.data_ptr(), mode, float(p), n, m, B,
                                      workspace.data_ptr(), workspace.numel(), stats.data_ptr(),
                                      _stream_ptr(stream)), "thanos_prune_layer")
    if not read_stats:
        return out, mask, stats
    st = _read_stats(stats)
    if st.status != 0:
        raise ThanosError(st.status, "thanos_prune_layer (row %d)" % st.err_index)
    return out, mask, st


def prune_block(Wc: torch.Tensor, mask: torch.Tensor, factor: torch.Tensor, xnorm: torch.Tensor,
                mode: int, n: int, m: int, B: int, j1: int, r: Optional[torch.Tensor],
                stats: torch.Tensor, stream=None, workspace: Optional[torch.Tensor] = None):
    """One block step in place on the float32 working weights Wc (and r, a 1-element int64)."""
    lib = load_library()
    _check_dev(Wc, mask, factor, xnorm)
    c, b = Wc.shape
    if workspace is None:
        workspace = _ws(workspace_bytes(WS_PRUNE, c, b, B, F32), Wc.device)
    with _on(Wc):
        _check(lib.thanos_prune_block(Wc.data_ptr(), mask.data_ptr(), c, b, factor.data_ptr(),
                                      xnorm.data_ptr(), mode, n, m, B, j1,
                                      r.data_ptr() if r is not None else None,
                                      workspace.data_ptr(), workspace.numel(), stats.data_ptr(),
                                      _stream_ptr(stream)), "thanos_prune_block")


def prune_layer_host(W_host: torch.Tensor, X_host: Optional[torch.Tensor], damp_rel: float,
                     mode: int, p: float = 0.0, n: int = 0, m: int = 0, B: int = 128,
                     arena: Optional[torch.Tensor] = None, reuse_factor: bool = False,
                     out: Optional[torch.Tensor] = None, mask: Optional[torch.Tensor] = None,
                     a: Optional[int] = None, stream=None, device="cuda"):
    """Whole path for one layer from HOST tensors (pinned or pageable); returns host tensors."""
    lib = load_library()
    if W_host.is_cuda or (X_host is not None and X_host.is_cuda):
        raise ValueError("prune_layer_host takes host tensors")
    c, b = W_host.shape
    dt = _dtype_code(W_host)
    if X_host is not None:
        if _dtype_code(X_host) != dt or not X_host.is_contiguous():
            raise ValueError("X must be contiguous and share W's dtype")
        a = X_host.shape[0]
    if a is None:
        a = 0
    if out is None:
        out = torch.empty_like(W_host)
    if mask is None:
        mask = torch.empty((c, b), dtype=torch.uint8)
    if arena is None:
        arena = _ws(workspace_bytes(WS_HOST_LAYER, c, b, B, dt), device)
    stats = _Stats()
    with _on(arena):
        code = lib.thanos_prune_layer_host(W_host.data_ptr(),
                                           X_host.data_ptr() if X_host is not None else None,
                                           out.data_ptr(), mask.data_ptr(), dt, c, b, a,
                                           float(damp_rel), mode, float(p), n, m, B,
                                           1 if reuse_factor else 0, arena.data_ptr(),
                                           arena.numel(), ctypes.byref(stats),
                                           _stream_ptr(stream))
    _check(code, "thanos_prune_layer_host")
    st = PruneStats(stats.status, stats.err_index, stats.n_pruned, stats.r_left, stats.max_s,
                    stats.n_blocks, stats.n_tied, stats.last_threshold_bits, stats.select_misses,
                    stats.select_rescans)
    if st.status != 0:
        raise ThanosError(st.status, "thanos_prune_layer_host (index %d)" % st.err_index)
    return out, mask, st


def prune_layer_noalloc(W: torch.Tensor, factor: torch.Tensor, xnorm: torch.Tensor, mode: int,
                        p: float = 0.0, n: int = 0, m: int = 0, B: int = 128, stream=None,
                        out: Optional[torch.Tensor] = None, mask: Optional[torch.Tensor] = None,
                        stats: Optional[torch.Tensor] = None):
    """thanos_prune_layer_noalloc: the sweep with the library's built-in 4 MiB scratch, for
    callers that cannot allocate a workspace.  Only the outputs are created here; pass `out`,
    `mask` and `stats` (64 bytes, uint8) and this function creates no device tensor at all.
    Calls on one device must not overlap."""
    lib = load_library()
    _check_dev(W, factor, xnorm)
    c, b = W.shape
    dt = _dtype_code(W)
    if out is None:
        out = torch.empty_like(W)
    if mask is None:
        mask = torch.empty((c, b), dtype=torch.uint8, device=W.device)
    if stats is None:
        stats = torch.zeros(64, dtype=torch.uint8, device=W.device)
    with _on(W):
        _check(lib.thanos_prune_layer_noalloc(W.data_ptr(), out.data_ptr(), mask.data_ptr(), dt, c,
                                              b, factor.data_ptr(), xnorm.data_ptr(), mode,
                                              float(p), n, m, B, stats.data_ptr(),
                                              _stream_ptr(stream)), "thanos_prune_layer_noalloc")
    st = _read_stats(stats)
    if st.status != 0:
        raise ThanosError(st.status, "thanos_prune_layer_noalloc (row %d)" % st.err_index)
    return out, mask, st


def fp32_fma_probe(out: torch.Tensor, ctas: int, iters: int, stream=None) -> float:
    """thanos_fp32_fma_probe: enqueues the FMA-chain kernel; returns its floating-point
    operation count (time it with CUDA events around this call)."""
    lib = load_library()
    _check_dev(out)
    flop = ctypes.c_double(0.0)
    with _on(out):
        _check(lib.thanos_fp32_fma_probe(out.data_ptr(), out.numel(), ctas, iters,
                                         ctypes.byref(flop), _stream_ptr(stream)),
               "thanos_fp32_fma_probe")
    return float(flop.value)


def dense_product(A: torch.Tensor, B: torch.Tensor, b_transposed: bool = False, alpha: float = 1.0,
                  out: Optional[torch.Tensor] = None, accumulate: bool = False, stream=None,
                  check: bool = True):
    """thanos_dense_product: out = (accumulate ? out : 0) + alpha * A @ (B^T if b_transposed
    else B), fp32 device matrices (rows may be strided: the last dimension is contiguous)."""
    lib = load_library()
    _check_dev(A, B)
    assert A.dtype == torch.float32 and B.dtype == torch.float32
    assert A.stride(1) == 1 and B.stride(1) == 1
    M, K = A.shape
    N = B.shape[0] if b_transposed else B.shape[1]
    assert (B.shape[1] if b_transposed else B.shape[0]) == K
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32, device=A.device)
        assert not accumulate
    assert out.stride(1) == 1
    nbytes = lib.thanos_dense_product_workspace(M, N, K)
    ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=A.device)
    with _on(A):
        _check(lib.thanos_dense_product(out.data_ptr(), out.stride(0), A.data_ptr(), A.stride(0),
                                        B.data_ptr(), B.stride(0), 1 if b_transposed else 0, M, N, K,
                                        float(alpha), 1 if accumulate else 0, ws.data_ptr(), nbytes,
                                        _stream_ptr(stream)), "thanos_dense_product")
    if check:
        st = int(ws[:4].view(torch.int32).item())
        if st != 0:
            raise ThanosError(st, "thanos_dense_product (device)")
    return out


def prune_layer_outliers(W: torch.Tensor, factor: torch.Tensor, xnorm: torch.Tensor,
                         H: torch.Tensor, n: int, m: int, alpha: float, B: int = 128, stream=None,
                         workspace: Optional[torch.Tensor] = None,
                         out: Optional[torch.Tensor] = None, mask: Optional[torch.Tensor] = None):
    """thanos_prune_layer_outliers: n:m sweep that leaves the ceil(alpha c) rows with the largest
    h_i = 1/2 W_i H W_i^T untouched.  Returns (W_pruned, mask, outlier flags uint8 [c], stats)."""
    lib = load_library()
    _check_dev(W, factor, xnorm, H)
    c, b = W.shape
    dt = _dtype_code(W)
    if out is None:
        out = torch.empty_like(W)
    if mask is None:
        mask = torch.empty((c, b), dtype=torch.uint8, device=W.device)
    flags = torch.empty((c,), dtype=torch.uint8, device=W.device)
    stats = torch.zeros(64, dtype=torch.uint8, device=W.device)
    if workspace is None:
        workspace = _ws(workspace_bytes(WS_PRUNE_OUTLIERS, c, b, B, dt), W.device)
    with _on(W):
        _check(lib.thanos_prune_layer_outliers(W.data_ptr(), out.data_ptr(), mask.data_ptr(), dt, c, b,
                                               factor.data_ptr(), xnorm.data_ptr(), H.data_ptr(), n, m,
                                               B, float(alpha), flags.data_ptr(), workspace.data_ptr(),
                                               workspace.numel(), stats.data_ptr(),
                                               _stream_ptr(stream)), "thanos_prune_layer_outliers")
    st = _read_stats(stats)
    if st.status != 0:
        raise ThanosError(st.status, "thanos_prune_layer_outliers (row %d)" % st.err_index)
    return out, mask, flags, st


def prune_layer_structured(W: torch.Tensor, factor: torch.Tensor, xnorm: torch.Tensor, p: float,
                           alpha: float = 0.0, H: Optional[torch.Tensor] = None, stream=None,
                           workspace: Optional[torch.Tensor] = None,
                           out: Optional[torch.Tensor] = None):
    """thanos_prune_layer_structured: removes the ceil(p b / (1 - alpha)) columns of smallest loss
    from all but the ceil(alpha c) outlier rows and updates the kept weights (Algorithm 2).
    Returns (W_pruned, removed columns uint8 [b], outlier rows uint8 [c], stats)."""
    lib = load_library()
    _check_dev(W, factor, xnorm)
    if alpha > 0.0:
        if H is None:
            raise ValueError("alpha > 0 needs the Hessian H")
        _check_dev(H)
    c, b = W.shape
    dt = _dtype_code(W)
    if out is None:
        out = torch.empty_like(W)
    colrm = torch.empty((b,), dtype=torch.uint8, device=W.device)
    flags = torch.empty((c,), dtype=torch.uint8, device=W.device)
    stats = torch.zeros(64, dtype=torch.uint8, device=W.device)
    if workspace is None:
        need = int(lib.thanos_structured_workspace_bytes(c, b, float(p), float(alpha), dt))
        if need == 0:
            raise ThanosError(1, "thanos_structured_workspace_bytes rejected the arguments")
        workspace = _ws(need, W.device)
    with _on(W):
        _check(lib.thanos_prune_layer_structured(W.data_ptr(), out.data_ptr(), colrm.data_ptr(),
                                                 flags.data_ptr(), dt, c, b, factor.data_ptr(),
                                                 xnorm.data_ptr(),
                                                 H.data_ptr() if H is not None else None, float(p),
                                                 float(alpha), workspace.data_ptr(), workspace.numel(),
                                                 stats.data_ptr(), _stream_ptr(stream)),
               "thanos_prune_layer_structured")
    st = _read_stats(stats)
    if st.status != 0:
        raise ThanosError(st.status, "thanos_prune_layer_structured (index %d)" % st.err_index)
    return out, colrm, flags, st
