"""ctypes binding for libfgmp.so.  Names follow include/fgmp.h; no arithmetic happens here."""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libfgmp.so")

SCORE_LP_ERROR, SCORE_HP_TO_LP = 0, 1
CLIP_NONE, CLIP_SW_BRUTE = 0, 1
OP_QUANTIZE_WEIGHTS, OP_QUANTIZE_ACTIVATIONS, OP_LINEAR, OP_CALIBRATE_TAU, OP_GLOBAL_TAU, OP_LINEAR_QUANTIZE, OP_LINEAR_FUSED, OP_LINEAR_CLASSES = 0, 1, 2, 3, 4, 5, 6, 7


class FgmpError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {status_string(code)} ({code})")
        self.code = code


class _Scales(ctypes.Structure):
    _fields_ = [("scale_fp4", ctypes.c_float), ("fp8_log2_ratio", ctypes.c_int), ("scale_fp8", ctypes.c_float)]


_lib = None


def library_path() -> str:
    return _LIB_PATH


def _load():
    """Loads the CUDA library; there is no fallback when it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2504_14152_b200.build`")
    L = ctypes.CDLL(_LIB_PATH)
    vp, i64, f32, f64, sz, ci = (ctypes.c_void_p, ctypes.c_int64, ctypes.c_float, ctypes.c_double,
                                 ctypes.c_size_t, ctypes.c_int)
    L.fgmp_weights_bytes.restype = sz
    L.fgmp_weights_bytes.argtypes = [i64, i64, i64]
    L.fgmp_acts_bytes.restype = sz
    L.fgmp_acts_bytes.argtypes = [i64, i64]
    L.fgmp_workspace_bytes.restype = sz
    L.fgmp_workspace_bytes.argtypes = [ci, i64, i64, i64]
    L.fgmp_quantize_weights.restype = ci
    L.fgmp_quantize_weights.argtypes = [vp, i64, vp, i64, i64, i64, _Scales, ci, ci, f64, f32, vp, sz, vp, vp, sz, vp]
    L.fgmp_quantize_activations.restype = ci
    L.fgmp_quantize_activations.argtypes = [vp, i64, vp, i64, i64, _Scales, ci, f32, vp, sz, vp, sz, vp]
    L.fgmp_calibrate_tau.restype = ci
    L.fgmp_calibrate_tau.argtypes = [vp, i64, vp, i64, i64, _Scales, ci, f64, vp, vp, sz, vp]
    L.fgmp_linear.restype = ci
    L.fgmp_linear.argtypes = [vp, vp, vp, ci, i64, i64, i64, i64, vp, sz, vp]
    L.fgmp_linear_classes.restype = ci
    L.fgmp_linear_classes.argtypes = [vp, vp, vp, ci, i64, i64, i64, i64, vp, sz, vp]
    L.fgmp_linear_fused.restype = ci
    L.fgmp_linear_fused.argtypes = [vp, i64, vp, _Scales, ci, f32, vp, vp, ci, i64, i64, i64, i64, vp, sz, vp, sz, vp]
    L.fgmp_linear_static.restype = ci
    L.fgmp_linear_static.argtypes = [vp, vp, vp, ci, i64, i64, i64, i64, vp, vp]
    L.fgmp_check.restype = ci
    L.fgmp_check.argtypes = [vp, vp]
    L.fgmp_linear_quantize.restype = ci
    L.fgmp_linear_quantize.argtypes = [vp, vp, i64, i64, i64, vp, _Scales, ci, ctypes.c_float, vp, sz, vp, sz, vp]
    L.fgmp_channel_mean_sq.restype = ci
    L.fgmp_channel_mean_sq.argtypes = [vp, i64, i64, i64, vp, vp]
    L.fgmp_weight_scores.restype = ci
    L.fgmp_weight_scores.argtypes = [vp, i64, vp, i64, i64, i64, _Scales, ci, ci, vp, vp, sz, vp]
    L.fgmp_global_tau.restype = ci
    L.fgmp_global_tau.argtypes = [vp, vp, ci, ctypes.c_double, vp, vp, sz, vp]
    L.fgmp_tensor_peak.restype = ci
    L.fgmp_tensor_peak.argtypes = [ci, i64, vp, sz, vp]
    L.fgmp_selftest_wait_timeout.restype = ci
    L.fgmp_selftest_wait_timeout.argtypes = [vp, sz, i64, vp]
    L.fgmp_workspace_init.restype = ci
    L.fgmp_workspace_init.argtypes = [vp, sz, vp]
    L.fgmp_unpack.restype = ci
    L.fgmp_unpack.argtypes = [vp, i64, i64, vp, vp, vp, vp, vp]
    L.fgmp_activation_scores.restype = ci
    L.fgmp_activation_scores.argtypes = [vp, i64, vp, i64, i64, _Scales, ci, vp, vp]
    L.fgmp_profile_begin.restype = ci
    L.fgmp_profile_begin.argtypes = [ctypes.c_uint]
    L.fgmp_profile_end.restype = ci
    L.fgmp_profile_end.argtypes = [ci, vp, vp]
    L.fgmp_kernel_name.restype = ctypes.c_char_p
    L.fgmp_kernel_name.argtypes = [ci]
    L.fgmp_status_string.restype = ctypes.c_char_p
    L.fgmp_status_string.argtypes = [ci]
    L.fgmp_version.restype = ci
    _lib = L
    return L


def status_string(code: int) -> str:
    return _load().fgmp_status_string(int(code)).decode()


def version() -> int:
    return _load().fgmp_version()


def _ok(code: int, what: str):
    if code != 0:
        raise FgmpError(code, what)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: torch.Tensor | None) -> int | None:
    return None if t is None else t.data_ptr()


def _alloc_aligned(nbytes: int, device) -> torch.Tensor:
    """uint8 buffer whose data pointer is 1024-byte aligned."""
    buf = torch.empty(nbytes + 1024, dtype=torch.uint8, device=device)
    off = (-buf.data_ptr()) % 1024
    return buf[off:off + nbytes]


def acts_bytes(M: int, K: int) -> int:
    return _load().fgmp_acts_bytes(M, K)


def weights_bytes(N: int, K: int, max_fp8_blocks: int) -> int:
    return _load().fgmp_weights_bytes(N, K, max_fp8_blocks)


def workspace_bytes(op: int, M: int, N: int, K: int) -> int:
    return _load().fgmp_workspace_bytes(op, M, N, K)


def workspace_init(workspace: torch.Tensor) -> torch.Tensor:
    """Clear the control area of a workspace (once, before fgmp_linear first uses it)."""
    _ok(_load().fgmp_workspace_init(workspace.data_ptr(), workspace.numel(), _stream()), "fgmp_workspace_init")
    return workspace


def alloc_workspace(op: int, M: int, N: int, K: int, device) -> torch.Tensor:
    """A cleared, 1024-byte aligned workspace for `op` on `device`."""
    return workspace_init(_alloc_aligned(workspace_bytes(op, M, N, K), device))


@dataclass
class PackedTensor:
    """An opaque packed blob on the device plus the shape it was made for."""
    blob: torch.Tensor      # uint8, 1024-byte aligned
    rows: int
    K: int
    kind: int               # 0 activations, 1 weights
    fp8_free: bool = False  # packed with an FP8 tensor scale of its own (scale_fp8 > 0): multiplied by linear_classes

    def header(self) -> dict:
        h = self.blob[:128].cpu().numpy().tobytes()
        import struct
        magic, ver, rows, K, s4, ratio, n8, tau, kind, cap, err, s8, free = struct.unpack("<IIqqfiqfIqifi", h[:68])
        return dict(magic=magic, version=ver, rows=rows, K=K, scale_fp4=s4, fp8_log2_ratio=ratio, n_fp8=n8,
                    tau_eff=tau, kind=kind, capacity=cap, error=err, scale_fp8=s8, fp8_scale_free=free)


def quantize_weights(W: torch.Tensor, fisher: torch.Tensor, *, scale_fp4: float = 0.0, ratio: int = 3, scale_fp8: float = 0.0,
                     score_mode: int = SCORE_LP_ERROR, clip_mode: int = CLIP_SW_BRUTE,
                     fp8_fraction: float = 0.1, tau: float = 0.0, max_fp8_blocks: int | None = None,
                     workspace: torch.Tensor | None = None, out: torch.Tensor | None = None) -> PackedTensor:
    """W bf16 [N, K], fisher fp32 [N, K] (both on the GPU) -> packed weights."""
    L = _load()
    assert W.is_cuda and W.dtype == torch.bfloat16 and fisher.dtype == torch.float32 and W.dim() == 2
    N, K = W.shape
    B = N * (K // 16)
    if max_fp8_blocks is None:
        max_fp8_blocks = B if fp8_fraction < 0 else min(B, int(fp8_fraction * B + 0.5) + 1)
    nbytes = L.fgmp_weights_bytes(N, K, max_fp8_blocks)
    if nbytes == 0:
        raise FgmpError(-2, "fgmp_weights_bytes")
    if out is None:
        out = _alloc_aligned(nbytes, W.device)
    ws_bytes = L.fgmp_workspace_bytes(OP_QUANTIZE_WEIGHTS, 0, N, K)
    if workspace is None:
        workspace = _alloc_aligned(ws_bytes, W.device)
    _ok(L.fgmp_quantize_weights(W.data_ptr(), W.stride(0), fisher.data_ptr(), fisher.stride(0), N, K,
                                _Scales(scale_fp4, ratio, scale_fp8), score_mode, clip_mode, float(fp8_fraction), tau,
                                out.data_ptr(), out.numel(), None, workspace.data_ptr(), workspace.numel(),
                                _stream()), "fgmp_quantize_weights")
    return PackedTensor(out, N, K, 1, scale_fp8 > 0)


def quantize_activations(X: torch.Tensor, fisher: torch.Tensor, *, scale_fp4: float, ratio: int = 3, scale_fp8: float = 0.0,
                         score_mode: int = SCORE_LP_ERROR, tau: float,
                         out: torch.Tensor | None = None) -> PackedTensor:
    """X bf16 [M, K], fisher fp32 [K] -> packed activations."""
    L = _load()
    assert X.is_cuda and X.dtype == torch.bfloat16 and fisher.dtype == torch.float32 and X.dim() == 2
    M, K = X.shape
    nbytes = L.fgmp_acts_bytes(M, K)
    if nbytes == 0:
        raise FgmpError(-2, "fgmp_acts_bytes")
    if out is None:
        out = _alloc_aligned(nbytes, X.device)
    _ok(L.fgmp_quantize_activations(X.data_ptr(), X.stride(0), fisher.data_ptr(), M, K, _Scales(scale_fp4, ratio, scale_fp8),
                                    score_mode, tau, out.data_ptr(), out.numel(), None, 0, _stream()),
        "fgmp_quantize_activations")
    return PackedTensor(out, M, K, 0, scale_fp8 > 0)


def calibrate_tau(X: torch.Tensor, fisher: torch.Tensor, *, scale_fp4: float, ratio: int = 3, scale_fp8: float = 0.0,
                  score_mode: int = SCORE_LP_ERROR, fp8_fraction: float,
                  workspace: torch.Tensor | None = None) -> torch.Tensor:
    """Returns a 1-element fp32 device tensor holding the threshold for this batch."""
    L = _load()
    M, K = X.shape
    tau = torch.empty(1, dtype=torch.float32, device=X.device)
    ws_bytes = L.fgmp_workspace_bytes(OP_CALIBRATE_TAU, M, 0, K)
    if workspace is None:
        workspace = _alloc_aligned(ws_bytes, X.device)
    _ok(L.fgmp_calibrate_tau(X.data_ptr(), X.stride(0), fisher.data_ptr(), M, K, _Scales(scale_fp4, ratio, scale_fp8),
                             score_mode, float(fp8_fraction), tau.data_ptr(), workspace.data_ptr(),
                             workspace.numel(), _stream()), "fgmp_calibrate_tau")
    return tau


def channel_mean_sq(X: torch.Tensor) -> torch.Tensor:
    """fp32 [K]: mean over the rows of X (bf16 [rows, K]) of X[r, c]^2 -- the weights of the Output Error policy."""
    L = _load()
    assert X.is_cuda and X.dtype == torch.bfloat16 and X.dim() == 2 and X.stride(1) == 1
    rows, K = X.shape
    out = torch.empty(K, dtype=torch.float32, device=X.device)
    _ok(L.fgmp_channel_mean_sq(X.data_ptr(), X.stride(0), rows, K, out.data_ptr(), _stream()), "fgmp_channel_mean_sq")
    return out


def weight_scores(W: torch.Tensor, fisher: torch.Tensor, *, scale_fp4: float = 0.0, ratio: int = 3, scale_fp8: float = 0.0,
                  score_mode: int = SCORE_LP_ERROR, clip_mode: int = CLIP_SW_BRUTE) -> torch.Tensor:
    """Block scores [N, K/16] of a weight tensor, as fgmp_quantize_weights ranks them."""
    L = _load()
    N, K = W.shape
    scores = torch.empty(N, K // 16, dtype=torch.float32, device=W.device)
    workspace = _alloc_aligned(L.fgmp_workspace_bytes(OP_QUANTIZE_WEIGHTS, 0, N, K), W.device)
    _ok(L.fgmp_weight_scores(W.data_ptr(), W.stride(0), fisher.data_ptr(), fisher.stride(0), N, K,
                             _Scales(scale_fp4, ratio, scale_fp8), score_mode, clip_mode, scores.data_ptr(),
                             workspace.data_ptr(), workspace.numel(), _stream()), "fgmp_weight_scores")
    return scores


def global_tau(score_tensors, fp8_fraction: float) -> torch.Tensor:
    """One threshold for several tensors (Eq. 10): a 1-element fp32 device tensor such that the given
    fraction of all blocks of `score_tensors` (fp32 device tensors of block scores) exceeds it."""
    L = _load()
    ts = [t.contiguous() for t in score_tensors]
    n = len(ts)
    ptrs = (ctypes.c_void_p * n)(*[t.data_ptr() for t in ts])
    counts = (ctypes.c_int64 * n)(*[t.numel() for t in ts])
    total = sum(t.numel() for t in ts)
    dev = ts[0].device
    tau = torch.empty(1, dtype=torch.float32, device=dev)
    workspace = _alloc_aligned(L.fgmp_workspace_bytes(OP_GLOBAL_TAU, total, 0, 0), dev)
    _ok(L.fgmp_global_tau(ptrs, counts, n, float(fp8_fraction), tau.data_ptr(), workspace.data_ptr(),
                          workspace.numel(), _stream()), "fgmp_global_tau")
    return tau


def activation_scores(X: torch.Tensor, fisher: torch.Tensor, *, scale_fp4: float, ratio: int = 3, scale_fp8: float = 0.0,
                      score_mode: int = SCORE_LP_ERROR) -> torch.Tensor:
    L = _load()
    M, K = X.shape
    scores = torch.empty(M, K // 16, dtype=torch.float32, device=X.device)
    _ok(L.fgmp_activation_scores(X.data_ptr(), X.stride(0), fisher.data_ptr(), M, K, _Scales(scale_fp4, ratio, scale_fp8),
                                 score_mode, scores.data_ptr(), _stream()), "fgmp_activation_scores")
    return scores


def linear(acts: PackedTensor, weights: PackedTensor, *, out_dtype=torch.float32,
           out: torch.Tensor | None = None, workspace: torch.Tensor | None = None) -> torch.Tensor:
    """Y [M, N] = acts x weights^T (FP32 accumulation).  Operands packed with an FP8 tensor scale of their
    own go through linear_classes (one accumulation per class of block pair, fp32 output)."""
    L = _load()
    assert acts.K == weights.K and acts.kind == 0 and weights.kind == 1
    if acts.fp8_free or weights.fp8_free:
        return linear_classes(acts, weights, out=out, workspace=workspace)
    M, N, K = acts.rows, weights.rows, acts.K
    if out is None:
        out = torch.empty(M, N, dtype=out_dtype, device=acts.blob.device)
    assert out.dtype in (torch.float32, torch.bfloat16)
    if workspace is None:
        workspace = alloc_workspace(OP_LINEAR, M, N, K, acts.blob.device)
    _ok(L.fgmp_linear(acts.blob.data_ptr(), weights.blob.data_ptr(), out.data_ptr(),
                      1 if out.dtype == torch.bfloat16 else 0, out.stride(0), M, N, K,
                      workspace.data_ptr(), workspace.numel(), _stream()), "fgmp_linear")
    linear.last_workspace = workspace
    return out


def linear_classes(acts: PackedTensor, weights: PackedTensor, *, out: torch.Tensor | None = None,
                   workspace: torch.Tensor | None = None) -> torch.Tensor:
    """Y fp32 [M, N] with the four classes of block pair accumulated separately, each under its own pair of
    tensor scales: the GEMM for operands whose FP8 scale is not a power of two times the NVFP4 scale."""
    L = _load()
    assert acts.K == weights.K and acts.kind == 0 and weights.kind == 1
    M, N, K = acts.rows, weights.rows, acts.K
    if out is None:
        out = torch.empty(M, N, dtype=torch.float32, device=acts.blob.device)
    assert out.dtype == torch.float32
    if workspace is None:
        workspace = alloc_workspace(OP_LINEAR_CLASSES, M, N, K, acts.blob.device)
    _ok(L.fgmp_linear_classes(acts.blob.data_ptr(), weights.blob.data_ptr(), out.data_ptr(), 0, out.stride(0), M, N, K,
                              workspace.data_ptr(), workspace.numel(), _stream()), "fgmp_linear_classes")
    linear.last_workspace = workspace
    return out


def linear_fused(X: torch.Tensor, fisher: torch.Tensor, weights: PackedTensor, *, scale_fp4: float, ratio: int = 3,
                 score_mode: int = SCORE_LP_ERROR, tau: float, out_dtype=torch.float32,
                 out: torch.Tensor | None = None, packed_out: torch.Tensor | None = None, want_packed: bool = False,
                 workspace: torch.Tensor | None = None):
    """One decode step in one call: X bf16 [M, K] is quantized (as quantize_activations would) and
    multiplied with the packed weights.  Returns Y, or (Y, PackedTensor) when the packed activations
    are asked for (want_packed / packed_out)."""
    L = _load()
    assert X.is_cuda and X.dtype == torch.bfloat16 and fisher.dtype == torch.float32 and X.dim() == 2
    assert weights.kind == 1 and X.shape[1] == weights.K
    M, K = X.shape
    N = weights.rows
    if out is None:
        out = torch.empty(M, N, dtype=out_dtype, device=X.device)
    if packed_out is None and want_packed:
        packed_out = _alloc_aligned(L.fgmp_acts_bytes(M, K), X.device)
    if workspace is None:
        workspace = alloc_workspace(OP_LINEAR_FUSED, M, N, K, X.device)
    _ok(L.fgmp_linear_fused(X.data_ptr(), X.stride(0), fisher.data_ptr(), _Scales(scale_fp4, ratio), score_mode, tau,
                            weights.blob.data_ptr(), out.data_ptr(), 1 if out.dtype == torch.bfloat16 else 0,
                            out.stride(0), M, N, K, _ptr(packed_out), 0 if packed_out is None else packed_out.numel(),
                            workspace.data_ptr(), workspace.numel(), _stream()), "fgmp_linear_fused")
    linear.last_workspace = workspace
    if packed_out is not None:
        return out, PackedTensor(packed_out, M, K, 0)
    return out


def linear_quantize(acts: PackedTensor, weights: PackedTensor, fisher_next: torch.Tensor, *, scale_fp4: float,
                    ratio: int = 3, score_mode: int = SCORE_LP_ERROR, tau: float,
                    workspace: torch.Tensor | None = None) -> PackedTensor:
    """acts x weights^T, quantized for the next layer in the GEMM's epilogue: the packed activations
    [M, N] that quantize_activations(linear(..., bf16), fisher_next, ...) would give."""
    L = _load()
    assert acts.K == weights.K and acts.kind == 0 and weights.kind == 1
    M, N, K = acts.rows, weights.rows, acts.K
    dev = acts.blob.device
    out = _alloc_aligned(L.fgmp_acts_bytes(M, N), dev)
    if workspace is None:
        workspace = alloc_workspace(OP_LINEAR_QUANTIZE, M, N, K, dev)
    _ok(L.fgmp_linear_quantize(acts.blob.data_ptr(), weights.blob.data_ptr(), M, N, K, fisher_next.data_ptr(),
                               _Scales(scale_fp4, ratio), score_mode, tau, out.data_ptr(), out.numel(),
                               workspace.data_ptr(), workspace.numel(), _stream()), "fgmp_linear_quantize")
    linear.last_workspace = workspace
    return PackedTensor(out, M, N, 0)


STATIC_SCRATCH_BYTES = 4 * 1024 * 1024


def linear_static(acts: PackedTensor, weights: PackedTensor, *, out: torch.Tensor,
                  status_out: torch.Tensor | None = None) -> torch.Tensor:
    """fgmp_linear_static: the decode-sized GEMM for callers that cannot allocate.  The scratch
    lives inside the library, so nothing is allocated here either: `out` (and `status_out`,
    int32[2], optional) must be given.  Calls must not overlap on the GPU."""
    L = _load()
    assert acts.K == weights.K and acts.kind == 0 and weights.kind == 1
    assert out.dtype in (torch.float32, torch.bfloat16)
    M, N, K = acts.rows, weights.rows, acts.K
    _ok(L.fgmp_linear_static(acts.blob.data_ptr(), weights.blob.data_ptr(), out.data_ptr(),
                             1 if out.dtype == torch.bfloat16 else 0, out.stride(0), M, N, K,
                             _ptr(status_out), _stream()), "fgmp_linear_static")
    return out


def tensor_peak(kind: int, mma_per_cta: int, workspace: torch.Tensor) -> None:
    """Launch the MMA-only loop of fgmp_tensor_peak (kind 0 bf16, 1 E4M3, 2 NVFP4); the caller times it."""
    _ok(_load().fgmp_tensor_peak(kind, mma_per_cta, workspace.data_ptr(), workspace.numel(), _stream()), "fgmp_tensor_peak")


def selftest_wait_timeout(workspace: torch.Tensor, limit_ns: int = 1_000_000) -> None:
    """Launch the one-block kernel whose bounded wait runs out (fgmp_selftest_wait_timeout)."""
    _ok(_load().fgmp_selftest_wait_timeout(workspace.data_ptr(), workspace.numel(), int(limit_ns), _stream()),
        "fgmp_selftest_wait_timeout")


def check(workspace: torch.Tensor) -> None:
    _ok(_load().fgmp_check(workspace.data_ptr(), _stream()), "fgmp_check")


def unpack(p: PackedTensor):
    """(codes4, codes8, scales, mask) canonical device arrays of a packed tensor."""
    L = _load()
    dev = p.blob.device
    KB = p.K // 16
    MW = (KB + 31) // 32
    codes4 = torch.empty(p.rows * p.K // 2, dtype=torch.uint8, device=dev)
    codes8 = torch.empty(p.rows * p.K, dtype=torch.uint8, device=dev)
    scales = torch.empty(p.rows * KB, dtype=torch.uint8, device=dev)
    mask = torch.empty(p.rows * MW, dtype=torch.int32, device=dev)
    _ok(L.fgmp_unpack(p.blob.data_ptr(), p.rows, p.K, codes4.data_ptr(), codes8.data_ptr(), scales.data_ptr(),
                      mask.data_ptr(), _stream()), "fgmp_unpack")
    return codes4, codes8, scales, mask


def kernel_names() -> list[str]:
    L = _load()
    names = []
    while True:
        name = L.fgmp_kernel_name(len(names)).decode()
        if not name:
            return names
        names.append(name)


def profile_begin(timed_kernels: list[str] | tuple[str, ...] = ()) -> None:
    """Start counting kernel launches; launches of the named kernels are also timed with
    CUDA events on their stream."""
    names = kernel_names()
    mask = 0
    for k in timed_kernels:
        mask |= 1 << names.index(k)
    _load().fgmp_profile_begin(mask)


def profile_end() -> dict:
    """{kernel name: (launches, total ms or 0.0)} since profile_begin."""
    L = _load()
    names = kernel_names()
    n = len(names)
    launches = (ctypes.c_longlong * n)()
    ms = (ctypes.c_float * n)()
    L.fgmp_profile_end(n, launches, ms)
    return {names[i]: (int(launches[i]), float(ms[i])) for i in range(n) if launches[i]}
