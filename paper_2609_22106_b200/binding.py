"""Thin ctypes binding over libprq.so (the C ABI declared in include/prq.h).

Argument marshalling only: every step of the hot path runs inside the library's CUDA
kernels.  torch is used for device memory and streams.  There is no CPU fallback: if the
library cannot be loaded or a call fails, a ``PrqError`` is raised.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# PRQ_TRACE=1 selects the developer build with clock-stamp tracing compiled in (see build.py)
LIB_PATH = os.path.join(_HERE, "libprq_trace.so" if os.environ.get("PRQ_TRACE") == "1" else "libprq.so")

OK = 0
F32, BF16 = 0, 1
ACT_IDENTITY, ACT_SCALE_PERM = 0, 1
FIELD_CODES, FIELD_SCALES, FIELD_PERM, FIELD_TOPK, FIELD_S, FIELD_INV_S, FIELD_COL_ERR = range(7)
BUF_CODES, BUF_SCALES_ROW, BUF_SCALES_SF = range(3)

EXPORTS = [
    "prq_prepare_weights", "prq_prepare_weights_opts", "prq_prepare_weights_device", "prq_prepare_weights_host", "prq_prepare_weights_host_opts", "prq_prepare_weights_search", "prq_weights_free",
    "prq_weights_clone", "prq_weights_offline_copy", "prq_fold_producer", "prq_weights_info", "prq_weights_get", "prq_act_bytes", "prq_quantize_act", "prq_linear_workspace_bytes",
    "prq_linear", "prq_linear_static_scratch", "prq_linear_fused", "prq_linear_multi", "prq_quantize_act_multi",
    "prq_linear_grouped", "prq_forward_host_scratch_bytes", "prq_forward_host",
    "prq_status_string", "prq_last_device_status", "prq_kernel_launch_count", "prq_mxf4_peak_probe",
    "prq_handover_probe", "prq_stack_gate_up", "prq_linear_gated", "prq_weights_format", "prq_act_bytes_for",
    "prq_prepare_weights_stacked",
]


class PrqError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


_lib = None


def lib():
    """Load libprq.so (built in-tree by paper_2609_22106_b200.build).  Fails loudly if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise PrqError(-1, f"libprq.so not found at {LIB_PATH}; run paper_2609_22106_b200.build.build()")
        L = ctypes.CDLL(LIB_PATH)
        vp, ci, cf, cs = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
        L.prq_prepare_weights.argtypes = [vp, ci, ci, ci, vp, cf, ci, ctypes.POINTER(vp)]
        L.prq_prepare_weights_host.argtypes = [vp, ci, ci, vp, cf, ci, vp, vp, vp, vp, vp, vp]
        L.prq_prepare_weights_opts.argtypes = [vp, ci, ci, ci, vp, cf, ci, vp, ctypes.POINTER(vp)]
        L.prq_prepare_weights_host_opts.argtypes = [vp, ci, ci, vp, cf, ci, vp, vp, vp, vp, vp, vp, vp]
        L.prq_prepare_weights_device.argtypes = [vp, ci, ci, ci, vp, cf, ci, vp, vp, ctypes.POINTER(vp)]
        L.prq_prepare_weights_search.argtypes = [vp, ci, ci, vp, ci, vp, ci, ci, ctypes.POINTER(vp),
                                                 ctypes.POINTER(cf), vp]
        L.prq_weights_clone.argtypes = [vp, ctypes.POINTER(vp)]
        L.prq_weights_offline_copy.argtypes = [vp, ctypes.POINTER(vp)]
        L.prq_fold_producer.argtypes = [vp, vp, ci, ci, vp, vp, ci, ci, vp, vp]
        L.prq_weights_free.argtypes = [vp]
        L.prq_weights_free.restype = None
        L.prq_weights_info.argtypes = [vp] + [ctypes.POINTER(ci)] * 4 + [ctypes.POINTER(cf)]
        L.prq_weights_get.argtypes = [vp, ci, ci, vp, cs]
        L.prq_act_bytes.argtypes = [ci, ci, ci, ci, ci]
        L.prq_act_bytes.restype = cs
        L.prq_quantize_act.argtypes = [vp, ci, vp, ci, ci, vp, vp, vp, vp, vp]
        L.prq_linear_workspace_bytes.argtypes = [vp, ci]
        L.prq_linear_workspace_bytes.restype = cs
        L.prq_linear.argtypes = [vp, vp, vp, ci, vp, ci, ci, vp, cs, vp]
        L.prq_linear_static_scratch.argtypes = [vp, vp, vp, ci, vp, ci, ci, vp]
        L.prq_linear_fused.argtypes = [vp, ci, vp, ci, ci, vp, ci, ci, vp]
        L.prq_quantize_act_multi.argtypes = [ci, vp, ci, vp, ci, ci, vp, vp, vp]
        L.prq_linear_multi.argtypes = [ci, vp, vp, vp, ci, vp, vp, ci, vp]
        L.prq_linear_grouped.argtypes = [vp, vp, vp, vp, ci, vp, ci, ci, vp]
        L.prq_forward_host_scratch_bytes.argtypes = [vp, ci]
        L.prq_forward_host_scratch_bytes.restype = cs
        L.prq_forward_host.argtypes = [vp, ci, vp, ci, vp, ci, vp, cs, vp]
        L.prq_status_string.argtypes = [ci]
        L.prq_status_string.restype = ctypes.c_char_p
        L.prq_last_device_status.argtypes = [vp]
        L.prq_kernel_launch_count.restype = ctypes.c_ulonglong
        L.prq_mxf4_peak_probe.argtypes = [ci, ctypes.POINTER(ci), vp]
        L.prq_handover_probe.argtypes = [ci, ci, ci, ci, vp]
        L.prq_prepare_weights_stacked.argtypes = [vp, vp, ci, ci, vp, cf, ci, vp, ctypes.POINTER(vp)]
        L.prq_weights_format.argtypes = [vp, ctypes.POINTER(ci)]
        L.prq_act_bytes_for.argtypes = [vp, ci, ci]
        L.prq_act_bytes_for.restype = cs
        L.prq_stack_gate_up.argtypes = [vp, vp, ci, ci, vp]
        L.prq_linear_gated.argtypes = [vp, vp, vp, ci, vp, vp, vp, vp, vp, vp]
        _lib = L
    return _lib


def status_string(code: int) -> str:
    if code < 0:
        return "library not loaded"
    return lib().prq_status_string(code).decode()


def _check(code: int, where: str):
    if code != OK:
        raise PrqError(code, where)


def _np_ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _stream_ptr(stream=None):
    import torch

    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def _dptr(t):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else None


class Weights:
    """Owner of a prq_weights handle."""

    def __init__(self, handle):
        self._h = handle
        ne, N, K, k = ctypes.c_int(), ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
        a = ctypes.c_float()
        _check(lib().prq_weights_info(handle, ne, N, K, k, a), "prq_weights_info")
        self.n_experts, self.N, self.K, self.k_tail, self.alpha = ne.value, N.value, K.value, k.value, a.value
        f = ctypes.c_int()
        _check(lib().prq_weights_format(handle, ctypes.byref(f)), "prq_weights_format")
        self.format = f.value

    @property
    def handle(self):
        return self._h

    def get(self, field: int, expert: int = 0) -> np.ndarray:
        Ka = self.K + self.k_tail
        shape, dt = {
            FIELD_CODES: ((self.N, Ka // 2 if self.format == FMT_MXFP4 else self.K), np.uint8),
            FIELD_SCALES: ((self.N, Ka // 32), np.uint8),
            FIELD_PERM: ((self.K,), np.int32),
            FIELD_TOPK: ((self.k_tail,), np.int32),
            FIELD_S: ((self.K,), np.float32),
            FIELD_INV_S: ((self.K,), np.float32),
            FIELD_COL_ERR: ((self.K,), np.float64),
        }[field]
        out = np.empty(shape, dt)
        _check(lib().prq_weights_get(self._h, expert, field, _np_ptr(out), out.nbytes), "prq_weights_get")
        return out

    def clone(self) -> "Weights":
        h = ctypes.c_void_p()
        _check(lib().prq_weights_clone(self._h, ctypes.byref(h)), "prq_weights_clone")
        return Weights(h)

    def offline_copy(self) -> "Weights":
        """The same prepared bytes as a plain MXFP4 layer over K + k input channels (the producer emits the tail
        channels twice; nothing is re-read)."""
        h = ctypes.c_void_p()
        _check(lib().prq_weights_offline_copy(self._h, ctypes.byref(h)), "prq_weights_offline_copy")
        return Weights(h)

    def free(self):
        if self._h:
            lib().prq_weights_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


FMT_MXFP4, FMT_MXFP8 = 0, 1


class PrepOpts(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_size_t), ("weight_scale_search", ctypes.c_int), ("gated_producer", ctypes.c_int),
                ("format", ctypes.c_int)]


def _opts(scale_search: bool, gated_producer: bool = False, fmt: int = FMT_MXFP4):
    return PrepOpts(ctypes.sizeof(PrepOpts), 1 if scale_search else 0, 1 if gated_producer else 0, fmt)


def prepare_weights(W_bf16: np.ndarray, act_amax: np.ndarray, alpha: float, k_tail: int,
                    scale_search: bool = False, gated_producer: bool = False, fmt: int = FMT_MXFP4) -> Weights:
    """W_bf16: uint16 (N, K) or (E, N, K); act_amax: float32 (K,) or (E, K).  scale_search: the E8M0-W
    variant (weight-side block-scale search).  gated_producer: W is a stacked gate / up projection in the row order
    of stack_gate_up, to be run by linear_gated."""
    W = np.ascontiguousarray(W_bf16, np.uint16)
    amax = np.ascontiguousarray(act_amax, np.float32)
    if W.ndim == 2:
        W = W[None]
        amax = amax[None]
    E, N, K = W.shape
    h = ctypes.c_void_p()
    o = _opts(scale_search, gated_producer, fmt)
    _check(lib().prq_prepare_weights_opts(_np_ptr(W), E, N, K, _np_ptr(amax), alpha, k_tail,
                                          ctypes.cast(ctypes.pointer(o), ctypes.c_void_p), ctypes.byref(h)),
           "prq_prepare_weights_opts")
    return Weights(h)


def prepare_weights_device(W, act_amax: np.ndarray, alpha: float, k_tail: int, scale_search: bool = False,
                           stream=None, gated_producer: bool = False) -> Weights:
    """W: torch CUDA tensor, bf16 (or its uint16 / int16 bit pattern), (N, K) or (E, N, K), contiguous.  The prep
    runs on the GPU; the handle equals the one prepare_weights builds from a host copy."""
    assert W.is_cuda and W.is_contiguous() and W.element_size() == 2
    amax = np.ascontiguousarray(act_amax, np.float32)
    shape = tuple(W.shape)
    if len(shape) == 2:
        shape = (1,) + shape
        amax = amax[None]
    E, N, K = shape
    h = ctypes.c_void_p()
    o = _opts(scale_search, gated_producer)
    _check(lib().prq_prepare_weights_device(W.data_ptr(), E, N, K, _np_ptr(amax), alpha, k_tail,
                                            ctypes.cast(ctypes.pointer(o), ctypes.c_void_p), _stream_ptr(stream),
                                            ctypes.byref(h)),
           "prq_prepare_weights_device")
    return Weights(h)


def prepare_weights_host(W_bf16: np.ndarray, act_amax: np.ndarray, alpha: float, k_tail: int,
                         scale_search: bool = False, fmt: int = FMT_MXFP4) -> dict:
    W = np.ascontiguousarray(W_bf16, np.uint16)
    amax = np.ascontiguousarray(act_amax, np.float32)
    N, K = W.shape
    Ka = K + k_tail
    out = dict(codes=np.empty((N, Ka // 2 if fmt == FMT_MXFP4 else K), np.uint8), scales=np.empty((N, Ka // 32), np.uint8),
               perm=np.empty(K, np.int32), s=np.empty(K, np.float32), inv_s=np.empty(K, np.float32),
               col_err=np.empty(K, np.float64))
    o = _opts(scale_search, False, fmt)
    _check(lib().prq_prepare_weights_host_opts(_np_ptr(W), N, K, _np_ptr(amax), alpha, k_tail,
                                               ctypes.cast(ctypes.pointer(o), ctypes.c_void_p), _np_ptr(out["codes"]),
                                               _np_ptr(out["scales"]), _np_ptr(out["perm"]), _np_ptr(out["s"]),
                                               _np_ptr(out["inv_s"]), _np_ptr(out["col_err"])),
           "prq_prepare_weights_host_opts")
    return out


def fold_producer(perm: np.ndarray, inv_s: np.ndarray, k_tail: int, W_up: np.ndarray, W_gate: np.ndarray = None,
                  duplicate_tail: bool = False):
    """Eq. (1): the up / gate projection weights with the down projection's 1 / s and permutation folded in.
    W_up, W_gate: uint16 (C, H).  Returns (up, gate or None) of (C or C + k_tail, H)."""
    pm = np.ascontiguousarray(perm, np.int32)
    iv = np.ascontiguousarray(inv_s, np.float32)
    Wu = np.ascontiguousarray(W_up, np.uint16)
    C, H = Wu.shape
    rows = C + (k_tail if duplicate_tail else 0)
    ou = np.empty((rows, H), np.uint16)
    Wg = og = None
    if W_gate is not None:
        Wg = np.ascontiguousarray(W_gate, np.uint16)
        og = np.empty((rows, H), np.uint16)
    _check(lib().prq_fold_producer(_np_ptr(pm), _np_ptr(iv), C, k_tail, _np_ptr(Wu), _np_ptr(Wg) if Wg is not None else None,
                                   H, 1 if duplicate_tail else 0, _np_ptr(ou), _np_ptr(og) if og is not None else None),
           "prq_fold_producer")
    return ou, og


def prepare_weights_search(W_bf16, zcal_bf16, alphas, k_tail: int):
    W = np.ascontiguousarray(W_bf16, np.uint16)
    Z = np.ascontiguousarray(zcal_bf16, np.uint16)
    al = np.ascontiguousarray(alphas, np.float32)
    N, K = W.shape
    T = Z.shape[0]
    h = ctypes.c_void_p()
    star = ctypes.c_float()
    errs = np.empty(len(al), np.float64)
    _check(lib().prq_prepare_weights_search(_np_ptr(W), N, K, _np_ptr(Z), T, _np_ptr(al), len(al), k_tail,
                                            ctypes.byref(h), ctypes.byref(star), _np_ptr(errs)),
           "prq_prepare_weights_search")
    return Weights(h), star.value, errs


def act_bytes(M: int, K: int, k_tail: int, n_groups: int, which: int) -> int:
    return int(lib().prq_act_bytes(M, K, k_tail, n_groups, which))


def quantize_act(w: Weights, x, mode: int = ACT_IDENTITY, expert_offsets=None, row_scales: bool = False,
                 out=None, stream=None):
    """x: torch bf16 CUDA tensor (M, K).  Returns (codes, scales_row or None, scales_sf) uint8 tensors."""
    import torch

    M = x.shape[0]
    ng = w.n_experts
    if out is None:
        size = (lambda which: act_bytes(M, w.K, w.k_tail, ng, which)) if w.format == FMT_MXFP4 else \
               (lambda which: int(lib().prq_act_bytes_for(w.handle, M, which)))
        codes = torch.empty(max(size(BUF_CODES), 16), dtype=torch.uint8, device=x.device)
        sf = torch.empty(max(size(BUF_SCALES_SF), 16), dtype=torch.uint8, device=x.device)
        srow = torch.empty(max(size(BUF_SCALES_ROW), 16), dtype=torch.uint8, device=x.device) if row_scales else None
    else:
        codes, srow, sf = out
    _check(lib().prq_quantize_act(w.handle, mode, _dptr(x), M, x.stride(0) if M else w.K, _dptr(expert_offsets),
                                  _dptr(codes), _dptr(srow), _dptr(sf), _stream_ptr(stream)), "prq_quantize_act")
    return codes, srow, sf


def linear_workspace_bytes(w: Weights, M: int) -> int:
    return int(lib().prq_linear_workspace_bytes(w.handle, M))


def new_workspace(w: Weights, M: int, device="cuda"):
    import torch

    return torch.zeros(max(linear_workspace_bytes(w, M), 16), dtype=torch.uint8, device=device)


def linear(w: Weights, codes, scales_sf, M: int, y_dtype: int = F32, workspace=None, out=None, stream=None):
    import torch

    if out is None:
        out = torch.empty((M, w.N), dtype=torch.float32 if y_dtype == F32 else torch.bfloat16, device=codes.device)
    if workspace is None and M > 128:   # up to 128 tokens the kernel needs no scratch: nothing to allocate or clear
        workspace = new_workspace(w, M, codes.device)
    _check(lib().prq_linear(w.handle, _dptr(codes), _dptr(scales_sf), M, _dptr(out), out.stride(0) if M else w.N,
                            y_dtype, _dptr(workspace), workspace.numel() if workspace is not None else 0,
                            _stream_ptr(stream)), "prq_linear")
    return out


def linear_static_scratch(w: Weights, codes, scales_sf, M: int, y_dtype: int = F32, out=None, stream=None):
    """prq_linear without a caller workspace: the scratch is an array inside the library (see include/prq.h
    for the size limits and the rule that overlapping calls race).  `out` must be supplied by callers that
    may not allocate; it is created here only as a convenience for tests."""
    import torch

    if out is None:
        out = torch.empty((M, w.N), dtype=torch.float32 if y_dtype == F32 else torch.bfloat16, device=codes.device)
    _check(lib().prq_linear_static_scratch(w.handle, _dptr(codes), _dptr(scales_sf), M, _dptr(out),
                                           out.stride(0) if M else w.N, y_dtype, _stream_ptr(stream)),
           "prq_linear_static_scratch")
    return out


FUSED_MAX_M = 16
MULTI_MAX = 4


def _ptr_array(ptrs):
    vals = [p.value if isinstance(p, ctypes.c_void_p) else p for p in ptrs]
    return (ctypes.c_void_p * len(vals))(*vals)


def quantize_act_multi(ws, x, mode: int = ACT_SCALE_PERM, out=None, stream=None):
    """One quantiser launch for several dense layers that read the same x.  Returns [(codes, scales_sf), ...]."""
    import torch

    M = x.shape[0]
    if out is None:
        out = []
        for w in ws:
            out.append((torch.empty(act_bytes(M, w.K, w.k_tail, 1, BUF_CODES), dtype=torch.uint8, device=x.device),
                        torch.empty(act_bytes(M, w.K, w.k_tail, 1, BUF_SCALES_SF), dtype=torch.uint8, device=x.device)))
    hs = _ptr_array([w.handle for w in ws])
    cs = _ptr_array([_dptr(c) for c, _ in out])
    ss = _ptr_array([_dptr(s) for _, s in out])
    _check(lib().prq_quantize_act_multi(len(ws), hs, mode, _dptr(x), M, x.stride(0) if M else ws[0].K, cs, ss,
                                        _stream_ptr(stream)), "prq_quantize_act_multi")
    return out


def linear_multi(ws, acts, M: int, y_dtype: int = F32, out=None, stream=None):
    """One GEMM launch (M <= 128) for several dense layers over the same tokens; acts = [(codes, scales_sf), ...]."""
    import torch

    if out is None:
        out = [torch.empty((M, w.N), dtype=torch.float32 if y_dtype == F32 else torch.bfloat16, device=acts[0][0].device)
               for w in ws]
    hs = _ptr_array([w.handle for w in ws])
    cs = _ptr_array([_dptr(c) for c, _ in acts])
    ss = _ptr_array([_dptr(s) for _, s in acts])
    ys = _ptr_array([_dptr(y) for y in out])
    ld = (ctypes.c_int * len(ws))(*[y.stride(0) if M else w.N for y, w in zip(out, ws)])
    _check(lib().prq_linear_multi(len(ws), hs, cs, ss, M, ys, ld, y_dtype, _stream_ptr(stream)), "prq_linear_multi")
    return out


def linear_fused(w: Weights, x, mode: int = ACT_IDENTITY, y_dtype: int = F32, out=None, stream=None):
    """Quantise x (M x K bf16 on the device, M <= FUSED_MAX_M) and multiply, in one launch."""
    import torch

    M = x.shape[0]
    if out is None:
        out = torch.empty((M, w.N), dtype=torch.float32 if y_dtype == F32 else torch.bfloat16, device=x.device)
    _check(lib().prq_linear_fused(w.handle, mode, _dptr(x), M, x.stride(0) if M else w.K, _dptr(out),
                                  out.stride(0) if M else w.N, y_dtype, _stream_ptr(stream)), "prq_linear_fused")
    return out


def linear_grouped(w: Weights, codes, scales_sf, expert_offsets, M_total: int, y_dtype: int = F32, out=None,
                   stream=None):
    import torch

    if out is None:
        out = torch.empty((M_total, w.N), dtype=torch.float32 if y_dtype == F32 else torch.bfloat16,
                          device=codes.device)
    _check(lib().prq_linear_grouped(w.handle, _dptr(codes), _dptr(scales_sf), _dptr(expert_offsets), M_total,
                                    _dptr(out), out.stride(0) if M_total else w.N, y_dtype, _stream_ptr(stream)),
           "prq_linear_grouped")
    return out


def forward_host_scratch_bytes(w: Weights, M: int) -> int:
    return int(lib().prq_forward_host_scratch_bytes(w.handle, M))


def forward_host(w: Weights, x_host, y_host, mode: int, scratch, y_dtype: int = F32, stream=None):
    """x_host / y_host: pinned torch CPU tensors (bf16 M x K, fp32 or bf16 M x N); scratch: CUDA uint8 tensor."""
    M = x_host.shape[0]
    _check(lib().prq_forward_host(w.handle, mode, _dptr(x_host), M, _dptr(y_host), y_dtype, _dptr(scratch),
                                  scratch.numel(), _stream_ptr(stream)), "prq_forward_host")


def last_device_status(stream=None) -> int:
    return int(lib().prq_last_device_status(_stream_ptr(stream)))


def kernel_launch_count() -> int:
    return int(lib().prq_kernel_launch_count())


MXF4_PROBE_FLOP_PER_MMA = 2 * 128 * 256 * 64


def mxf4_peak_probe(n_mma: int, stream=None) -> int:
    """Launches the tensor-pipe probe (n_mma instructions per CTA, one CTA per SM); returns the CTA count."""
    n = ctypes.c_int()
    _check(lib().prq_mxf4_peak_probe(int(n_mma), ctypes.byref(n), _stream_ptr(stream)), "prq_mxf4_peak_probe")
    return n.value


def handover_probe(n: int, grid: int, threads: int = 192, cluster: int = 1, stream=None) -> None:
    """Enqueues n empty, dependent launches shaped like the decode GEMM's (see include/prq.h); the caller times them."""
    _check(lib().prq_handover_probe(int(n), int(grid), int(threads), int(cluster), _stream_ptr(stream)),
           "prq_handover_probe")


def stack_gate_up(W_gate: np.ndarray, W_up: np.ndarray) -> np.ndarray:
    """Gate and up projection rows (C, H) uint16 interleaved in groups of 32: the stacked layer linear_gated runs."""
    Wg = np.ascontiguousarray(W_gate, np.uint16)
    Wu = np.ascontiguousarray(W_up, np.uint16)
    C, H = Wg.shape
    out = np.empty((2 * C, H), np.uint16)
    _check(lib().prq_stack_gate_up(_np_ptr(Wg), _np_ptr(Wu), C, H, _np_ptr(out)), "prq_stack_gate_up")
    return out


def linear_gated(w_gu: Weights, codes, scales_sf, M: int, w_down: Weights, row_scales: bool = False, h_check: bool = False,
                 out=None, stream=None):
    """Q(silu(gate) * up) of the stacked producer layer, written as the down projection's quantised activation.
    Returns (codes, scales_row or None, scales_sf, h or None) -- h only on request, for checks."""
    import torch

    C, k = w_down.K, w_down.k_tail
    dev = codes.device
    if out is None:
        oc = torch.empty(max(act_bytes(M, C, k, 1, BUF_CODES), 16), dtype=torch.uint8, device=dev)
        osf = torch.empty(max(act_bytes(M, C, k, 1, BUF_SCALES_SF), 16), dtype=torch.uint8, device=dev)
        orow = torch.empty(max(act_bytes(M, C, k, 1, BUF_SCALES_ROW), 16), dtype=torch.uint8, device=dev) if row_scales else None
    else:
        oc, orow, osf = out
    h = torch.empty((M, C), dtype=torch.bfloat16, device=dev) if h_check else None
    _check(lib().prq_linear_gated(w_gu.handle, _dptr(codes), _dptr(scales_sf), M, w_down.handle, _dptr(oc), _dptr(orow),
                                  _dptr(osf), _dptr(h), _stream_ptr(stream)), "prq_linear_gated")
    return oc, orow, osf, h


def prepare_weights_stacked(Ws, act_amax: np.ndarray, alpha: float, k_tail: int, scale_search: bool = False,
                            fmt: int = FMT_MXFP4) -> Weights:
    """Several layers over the same activation (list of uint16 (N_i, K) arrays) prepared as one layer; layer i's outputs
    are columns [sum N_j for j < i, + N_i) of linear()'s result.  fmt as in prepare_weights (MXFP8: k_tail 0)."""
    mats = [np.ascontiguousarray(W, np.uint16) for W in Ws]
    K = mats[0].shape[1]
    ptrs = (ctypes.c_void_p * len(mats))(*[m.ctypes.data for m in mats])
    ns = (ctypes.c_int * len(mats))(*[m.shape[0] for m in mats])
    amax = np.ascontiguousarray(act_amax, np.float32)
    h = ctypes.c_void_p()
    o = _opts(scale_search, False, fmt)
    _check(lib().prq_prepare_weights_stacked(ctypes.cast(ptrs, ctypes.c_void_p), ctypes.cast(ns, ctypes.c_void_p), len(mats), K,
                                             _np_ptr(amax), alpha, k_tail, ctypes.cast(ctypes.pointer(o), ctypes.c_void_p),
                                             ctypes.byref(h)), "prq_prepare_weights_stacked")
    return Weights(h)
