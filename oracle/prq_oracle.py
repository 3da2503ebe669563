"""ctypes front end of the PRQuant CPU oracle (``prq_oracle.c``).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this module.  It never imports the CUDA
package and the CUDA package never imports it.

Arrays: bf16 tensors travel as ``uint16`` numpy arrays, packed E2M1 codes and E8M0
scale bytes as ``uint8``.  Every function returns fresh numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "prq_oracle.c")
_LIB = os.path.join(_HERE, "libprq_oracle.so")
_lib = None

BLOCK = 32


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP for the row split of the matmul)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        )
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def num_threads() -> int:
    return int(_load().orc_num_threads())


def quantize_rows(v):
    """Q, storage half: fp32 (rows, cols) -> (packed codes (rows, cols/2), scales (rows, cols/32))."""
    v = _c(v, np.float32)
    rows, cols = v.shape
    codes = np.empty((rows, cols // 2), np.uint8)
    scales = np.empty((rows, cols // BLOCK), np.uint8)
    rc = _load().orc_quantize_rows(_p(v), ctypes.c_long(rows), ctypes.c_long(cols), _p(codes), _p(scales))
    if rc:
        raise ValueError("cols must be a multiple of 32")
    return codes, scales


def dequantize_rows(codes, scales):
    """Q, value half: -> float64 (rows, cols)."""
    codes = _c(codes, np.uint8)
    scales = _c(scales, np.uint8)
    rows, half = codes.shape
    cols = half * 2
    out = np.empty((rows, cols), np.float64)
    rc = _load().orc_dequantize_rows(_p(codes), _p(scales), ctypes.c_long(rows), ctypes.c_long(cols), _p(out))
    if rc:
        raise ValueError("cols must be a multiple of 32")
    return out


def channel_amax(z_bf16):
    z = _c(z_bf16, np.uint16)
    T, K = z.shape
    amax = np.empty(K, np.float32)
    _load().orc_channel_amax(_p(z), ctypes.c_long(T), ctypes.c_long(K), _p(amax))
    return amax


def scales_from_amax(amax, alpha: float):
    amax = _c(amax, np.float32)
    K = amax.shape[0]
    s = np.empty(K, np.float32)
    inv_s = np.empty(K, np.float32)
    _load().orc_scales_from_amax(_p(amax), ctypes.c_long(K), ctypes.c_double(alpha), _p(s), _p(inv_s))
    return s, inv_s


def quantize_rows_search(v):
    """Q with the weight-side block-scale search (E8M0-W, Ablation study): best of the floor-rule
    exponent and its two neighbours per block."""
    v = _c(v, np.float32)
    rows, cols = v.shape
    codes = np.empty((rows, cols // 2), np.uint8)
    scales = np.empty((rows, cols // BLOCK), np.uint8)
    if _load().orc_quantize_rows_search(_p(v), ctypes.c_long(rows), ctypes.c_long(cols), _p(codes), _p(scales)):
        raise ValueError("cols must be a multiple of 32")
    return codes, scales


def prepare(W_bf16, amax, alpha: float, k: int, scale_search: bool = False):
    """Algorithm 1 steps 3-7, 11 for one alpha (scale_search: the E8M0-W variant).  Returns a dict with
    s, inv_s, col_err, perm (new -> old), topk (= perm[K-k:]), wcodes, wscales, R."""
    W = _c(W_bf16, np.uint16)
    amax = _c(amax, np.float32)
    N, K = W.shape
    Ka = K + k
    s = np.empty(K, np.float32)
    inv_s = np.empty(K, np.float32)
    col_err = np.empty(K, np.float64)
    perm = np.empty(K, np.int32)
    wcodes = np.empty((N, Ka // 2), np.uint8)
    wscales = np.empty((N, Ka // BLOCK), np.uint8)
    R = np.empty((N, max(k, 1)), np.float32)
    rc = _load().orc_prepare_ex(
        _p(W), ctypes.c_long(N), ctypes.c_long(K), _p(amax), ctypes.c_double(alpha), ctypes.c_long(k),
        ctypes.c_int(1 if scale_search else 0),
        _p(s), _p(inv_s), _p(col_err), _p(perm), _p(wcodes), _p(wscales), _p(R),
    )
    if rc:
        raise ValueError("K and k must be multiples of 32 with 0 <= k <= K")
    return dict(s=s, inv_s=inv_s, col_err=col_err, perm=perm, topk=perm[K - k:].copy(), wcodes=wcodes,
                wscales=wscales, R=R[:, :k], N=N, K=K, k=k, alpha=alpha)


def quantize_act(x_bf16, perm=None, inv_s=None):
    """Eq. (1) activation side then Q by rows.  perm/inv_s None = identity (folded upstream)."""
    x = _c(x_bf16, np.uint16)
    M, K = x.shape
    codes = np.empty((M, K // 2), np.uint8)
    scales = np.empty((M, K // BLOCK), np.uint8)
    pp = _p(_c(perm, np.int32)) if perm is not None else None
    ps = _p(_c(inv_s, np.float32)) if inv_s is not None else None
    rc = _load().orc_quantize_act(_p(x), ctypes.c_long(M), ctypes.c_long(K), pp, ps, _p(codes), _p(scales))
    if rc:
        raise ValueError("K must be a multiple of 32")
    return codes, scales


def augment_act(codes, scales, k: int):
    """[Q(Zt) | Q(Zt)_tail] with the copied blocks' own scales."""
    codes = _c(codes, np.uint8)
    scales = _c(scales, np.uint8)
    M, half = codes.shape
    K = half * 2
    Ka = K + k
    ca = np.empty((M, Ka // 2), np.uint8)
    sa = np.empty((M, Ka // BLOCK), np.uint8)
    rc = _load().orc_augment_act(_p(codes), _p(scales), ctypes.c_long(M), ctypes.c_long(K), ctypes.c_long(k), _p(ca), _p(sa))
    if rc:
        raise ValueError("bad K / k")
    return ca, sa


def matmul(acodes, ascales, wcodes, wscales):
    """Eq. (3): FP64 product of the dequantised operands over K + k, ascending j."""
    acodes = _c(acodes, np.uint8)
    ascales = _c(ascales, np.uint8)
    wcodes = _c(wcodes, np.uint8)
    wscales = _c(wscales, np.uint8)
    M, half = acodes.shape
    N, half_w = wcodes.shape
    if half != half_w:
        raise ValueError("reduction lengths differ")
    Ka = half * 2
    y = np.empty((M, N), np.float64)
    rc = _load().orc_matmul(_p(acodes), _p(ascales), ctypes.c_long(M), _p(wcodes), _p(wscales),
                            ctypes.c_long(N), ctypes.c_long(Ka), _p(y))
    if rc:
        raise ValueError("K + k must be a multiple of 32")
    return y


def matmul_bf16(x_bf16, W_bf16):
    """Unquantised Y = Z W^T in FP64."""
    x = _c(x_bf16, np.uint16)
    W = _c(W_bf16, np.uint16)
    M, K = x.shape
    N, K2 = W.shape
    if K != K2:
        raise ValueError("K differs")
    y = np.empty((M, N), np.float64)
    _load().orc_matmul_bf16(_p(x), ctypes.c_long(M), _p(W), ctypes.c_long(N), ctypes.c_long(K), _p(y))
    return y


def linear(x_bf16, prep: dict, identity: bool = False):
    """The whole online path for prepared weights: quantise the activation (with the
    layer's inverse scale and permutation unless they are folded upstream), expose the
    tail, multiply.  Returns (y float64, acodes, ascales)."""
    if identity:
        ac, asc = quantize_act(x_bf16)
    else:
        ac, asc = quantize_act(x_bf16, prep["perm"], prep["inv_s"])
    ca, sa = augment_act(ac, asc, prep["k"])
    return matmul(ca, sa, prep["wcodes"], prep["wscales"]), ac, asc


def fold_producer(W_up, W_gate, perm, inv_s, k: int, dup: bool = False):
    """Eq. (1), middle line: up- and gate-projection weights with the down projection's inverse scale and
    permutation folded in (rows permuted, the up projection's rows scaled and rounded once to bf16); with dup the
    last k rows are repeated (the 'offline copy' of the Activation tail construction paragraph).
    W_up, W_gate: uint16 (C, H); returns (up, gate) of (C or C + k, H)."""
    Wu = _c(W_up, np.uint16)
    Wg = _c(W_gate, np.uint16)
    pm = _c(perm, np.int32)
    iv = _c(inv_s, np.float32)
    C, H = Wu.shape
    rows = C + (k if dup else 0)
    ou = np.empty((rows, H), np.uint16)
    og = np.empty((rows, H), np.uint16)
    rc = _load().orc_fold_producer(_p(Wu), _p(Wg), ctypes.c_long(C), ctypes.c_long(H), _p(pm), _p(iv),
                                   ctypes.c_long(k), ctypes.c_int(1 if dup else 0), _p(ou), _p(og))
    if rc != 0:
        raise ValueError("k must lie in [0, C]")
    return ou, og


def silu_mul_bf16(g, u):
    """The producer's gated activation (f of Eq. (1), middle line, for a SiLU-gated FFN): bf16(silu(g) * u) from
    FP64 gate / up sums, rounded once; returns uint16 bit patterns of the same shape."""
    g = _c(g, np.float64)
    u = _c(u, np.float64)
    h = np.empty(g.shape, np.uint16)
    _load().orc_silu_mul_bf16(_p(g), _p(u), ctypes.c_long(g.size), _p(h))
    return h


def stack_gate_up(W_gate, W_up):
    """Rows of the gate and up projections interleaved in groups of 32 (gate rows 32 b .., then up rows 32 b ..): the
    stacked producer layer whose 64-feature output groups are the two factors of one 32-channel block."""
    Wg = _c(W_gate, np.uint16)
    Wu = _c(W_up, np.uint16)
    C, H = Wg.shape
    out = np.empty((2 * C, H), np.uint16)
    o4 = out.reshape(C // BLOCK, 2, BLOCK, H)
    o4[:, 0] = Wg.reshape(C // BLOCK, BLOCK, H)
    o4[:, 1] = Wu.reshape(C // BLOCK, BLOCK, H)
    return out


# ---- second format: MXFP8 (E4M3 elements, E8M0 block scales), plain W8A8 ----

def fp8_quantize_rows(v):
    """fp32 (rows, cols) -> (E4M3 codes (rows, cols), scale bytes (rows, cols/32))."""
    v = _c(v, np.float32)
    rows, cols = v.shape
    codes = np.empty((rows, cols), np.uint8)
    scales = np.empty((rows, cols // BLOCK), np.uint8)
    if _load().orc_fp8_quantize_rows(_p(v), ctypes.c_long(rows), ctypes.c_long(cols), _p(codes), _p(scales)):
        raise ValueError("cols must be a multiple of 32")
    return codes, scales


def fp8_dequantize_rows(codes, scales):
    codes = _c(codes, np.uint8)
    scales = _c(scales, np.uint8)
    rows, cols = codes.shape
    out = np.empty((rows, cols), np.float64)
    if _load().orc_fp8_dequantize_rows(_p(codes), _p(scales), ctypes.c_long(rows), ctypes.c_long(cols), _p(out)):
        raise ValueError("cols must be a multiple of 32")
    return out


def fp8_prepare(W_bf16, amax, alpha: float):
    """Offline half of the MXFP8 layer for one alpha: scale by s = amax^alpha, quantise by rows."""
    W = _c(W_bf16, np.uint16)
    am = _c(amax, np.float32)
    N, K = W.shape
    s = np.empty(K, np.float32)
    inv_s = np.empty(K, np.float32)
    wc = np.empty((N, K), np.uint8)
    wsc = np.empty((N, K // BLOCK), np.uint8)
    if _load().orc_fp8_prepare(_p(W), ctypes.c_long(N), ctypes.c_long(K), _p(am), ctypes.c_double(alpha), _p(s), _p(inv_s),
                               _p(wc), _p(wsc)):
        raise ValueError("K must be a multiple of 32")
    return dict(alpha=alpha, s=s, inv_s=inv_s, wcodes=wc, wscales=wsc)


def fp8_quantize_act(x_bf16, inv_s=None):
    x = _c(x_bf16, np.uint16)
    M, K = x.shape
    iv = _c(inv_s, np.float32) if inv_s is not None else None
    codes = np.empty((M, K), np.uint8)
    scales = np.empty((M, K // BLOCK), np.uint8)
    if _load().orc_fp8_quantize_act(_p(x), ctypes.c_long(M), ctypes.c_long(K), _p(iv) if iv is not None else None,
                                    _p(codes), _p(scales)):
        raise ValueError("K must be a multiple of 32")
    return codes, scales


def fp8_matmul(acodes, ascales, wcodes, wscales):
    a = _c(acodes, np.uint8)
    asc = _c(ascales, np.uint8)
    w = _c(wcodes, np.uint8)
    wsc = _c(wscales, np.uint8)
    M, K = a.shape
    N = w.shape[0]
    y = np.empty((M, N), np.float64)
    if _load().orc_fp8_matmul(_p(a), _p(asc), _p(w), _p(wsc), ctypes.c_long(M), ctypes.c_long(N), ctypes.c_long(K), _p(y)):
        raise ValueError("K must be a multiple of 32")
    return y


def nrmse(y_hat, y):
    """Normalised reconstruction error ||Yhat - Y||_F / ||Y||_F (text after Eq. (3))."""
    return float(np.linalg.norm(y_hat - y) / np.linalg.norm(y))


def alpha_search(W_bf16, zcal_bf16, alphas, k: int):
    """Algorithm 1 steps 1-10: evaluate Eq. (3) on the calibration rows for every
    candidate alpha and keep the first minimiser of the normalised error.
    Pinned by a hand-worked three-candidate search (tests/golden/alpha_search_worked.txt); which alpha the
    paper's own grid would pick on its checkpoints cannot be checked here."""
    amax = channel_amax(zcal_bf16)
    y_ref = matmul_bf16(zcal_bf16, W_bf16)
    errs = []
    preps = []
    for a in alphas:
        p = prepare(W_bf16, amax, float(a), k)
        y_hat, _, _ = linear(zcal_bf16, p)
        errs.append(nrmse(y_hat, y_ref))
        preps.append(p)
    best = int(np.argmin(np.asarray(errs)))  # first minimum
    return preps[best], float(alphas[best]), errs
