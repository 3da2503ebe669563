"""Helpers shared by the GPU parity tests: expected buffer layouts and oracle references."""
import numpy as np

STAGE_K = 256
GROUP = 128


def stages(K, k):
    s1 = (K + STAGE_K - 1) // STAGE_K
    return s1, s1 + (k + STAGE_K - 1) // STAGE_K


def sf_offset(r, b):
    """Byte of (row r of a 128-row group, block b of a stage) inside the group's 1024-byte tile."""
    return (b // 4) * 512 + (r % 32) * 16 + (r // 32) * 4 + (b % 4)


def expected_sf(scales_aug, K, k, groups=None, row_group=None, row_in_group=None):
    """Tile-ordered scale buffer for augmented row-major scales (M, (K+k)/32).
    Dense: row m -> group m // 128.  Grouped: pass row_group / row_in_group per row."""
    M = scales_aug.shape[0]
    s1, S = stages(K, k)
    if row_group is None:
        row_group = np.arange(M) // GROUP
        row_in_group = np.arange(M) % GROUP
        groups = (M + GROUP - 1) // GROUP
    out = np.zeros((S, groups, 1024), np.uint8)
    nb = STAGE_K // 32
    nmain = K // 32
    for b in range(scales_aug.shape[1]):
        if b < nmain:
            st, bis = b // nb, b % nb
        else:
            st, bis = s1 + (b - nmain) // nb, (b - nmain) % nb
        off = (bis // 4) * 512 + (row_in_group % 32) * 16 + (row_in_group // 32) * 4 + (bis % 4)
        out[st, row_group, off] = scales_aug[:, b]
    return out.reshape(-1)


def unpack(codes):
    codes = np.asarray(codes, np.uint8)
    out = np.empty(codes.shape[:-1] + (codes.shape[-1] * 2,), np.uint8)
    out[..., 0::2] = codes & 0xF
    out[..., 1::2] = codes >> 4
    return out


def tolerance(y_ref):
    """Acceptance bound of the GEMM: max |y - y_ref| <= 2e-3 (||y_ref||_inf + 1)."""
    return 2e-3 * (float(np.abs(y_ref).max()) + 1.0)


def expected_sf_fp8(scales, K, groups=None):
    """Tile-ordered scale buffer of the second format (MXFP8): [128-element stage][128-row group][512 bytes], the byte of
    (row r of a group, block b of a stage) at (r % 32) * 16 + (r // 32) * 4 + b."""
    M = scales.shape[0]
    S = (K + 127) // 128
    groups = (M + GROUP - 1) // GROUP if groups is None else groups
    out = np.zeros((S, groups, 512), np.uint8)
    r = np.arange(M)
    for b in range(scales.shape[1]):
        out[b // 4, r // GROUP, ((r % GROUP) % 32) * 16 + ((r % GROUP) // 32) * 4 + b % 4] = scales[:, b]
    return out.reshape(-1)
