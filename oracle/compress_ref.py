"""CPU oracle of the offline compressor (Sec. 3.2, Eq. 6-7; Sec. 3.4).  TEST INFRASTRUCTURE ONLY.

From E dense expert matrices W_i (d_in x d_out, row-vector convention y = x W) grouped into G clusters of K = E/G
(expert slot e = g*K + i belongs to cluster g) to the layer's stored form:

    Eq. 6      W_base^g = mean of the cluster's W_i, stored as fp16
    Eq. 7      Delta W_i = W_i - W_base^g  ~  A_i B_i^T  with  A_i (d_in x r),  B_i (d_out x r):
               the truncated SVD of Delta W_i (the text after Eq. 8: "initialized with a truncated SVD", the optimal
               rank-r approximation), computed here with numpy's LAPACK SVD in fp64
    Sec. 3.4   A_i, B_i^T quantised to symmetric INT4 with one fp16 scale per 32 consecutive elements of the
               flattened factor (reduction index fastest), the storage format of the layer's descriptor
    Sec. 3.4   optional cosine gate: a residual block whose cosine similarity to the base matrix is below gamma is
               zeroed

Readings (the paper leaves them open): the residual is taken against the base AS STORED
(the fp16-rounded mean), so that the factors also absorb the rounding of the base; the singular values are split
evenly, A = U_r sqrt(S_r), B^T = sqrt(S_r) V_r^T; the gate compares <Delta W, W_base>_F / (|Delta W|_F |W_base|_F)
with gamma literally (gamma = 0 switches it off); quantiser: scale = fp16(absmax / 7) (0 for an all-zero group),
code = clamp(round_half_even(w / scale), -8, 7), even flat index in the low nibble.

Pins (tests/test_compress_oracle.py): a hand-worked 2 x 2 mean and residual; experts built as base + known rank-r
residuals are recovered to rounding; a residual with prescribed singular values gives the Eckart-Young error
sqrt(sum of the dropped sigma^2) and those sigma; the error-versus-r curve never rises; the quantiser's round trip
stays within half a scale step and reproduces a hand-written group; the gate on residuals of known cosine.
"""
from __future__ import annotations

import numpy as np


def quantize_int4_groups(w: np.ndarray):
    """w: float array whose flattened size is a multiple of 32 -> (packed uint8 [size/2], fp16 scales [size/32])."""
    flat = np.ascontiguousarray(w, dtype=np.float32).reshape(-1)
    assert flat.size % 32 == 0
    grp = flat.reshape(-1, 32)
    absmax = np.abs(grp).max(axis=1)
    scale = (absmax / np.float32(7.0)).astype(np.float16)
    sf = scale.astype(np.float32)
    codes = np.zeros_like(grp, dtype=np.int32)
    nz = sf > 0
    codes[nz] = np.clip(np.rint(grp[nz] / sf[nz, None]), -8, 7).astype(np.int32)
    nib = (codes.reshape(-1) & 0xF).astype(np.uint8)
    packed = (nib[0::2] | (nib[1::2] << 4)).astype(np.uint8)
    return packed, scale


def dequantize_int4_groups(packed: np.ndarray, scale: np.ndarray) -> np.ndarray:
    lo = (packed & 0xF).astype(np.int32)
    hi = (packed >> 4).astype(np.int32)
    codes = np.empty(packed.size * 2, np.int32)
    codes[0::2] = np.where(lo > 7, lo - 16, lo)
    codes[1::2] = np.where(hi > 7, hi - 16, hi)
    return codes.astype(np.float64) * np.repeat(scale.astype(np.float64), 32)


def shared_base(W: np.ndarray, G: int) -> np.ndarray:
    """Eq. 6: [E][d_in][d_out] -> fp16 [G][d_in][d_out], the mean over each cluster's K experts."""
    E = W.shape[0]
    K = E // G
    return W.astype(np.float64).reshape(G, K, *W.shape[1:]).mean(axis=1).astype(np.float16)


def truncated_factors(dW: np.ndarray, r: int):
    """Eq. 7 by the SVD: A (d_in x r), Bt (r x d_out), the r largest singular values, with A Bt the best rank-r
    approximation of dW in the Frobenius norm."""
    U, S, Vt = np.linalg.svd(dW.astype(np.float64), full_matrices=False)
    root = np.sqrt(S[:r])
    return U[:, :r] * root[None, :], root[:, None] * Vt[:r], S[:r]


def compress(W: np.ndarray, G: int, r: int, gamma: float = 0.0) -> dict:
    """W [E][d_in][d_out] float -> dict(B fp16 [G][d_in][d_out], Uq/Us [E][r][d_in], Vq/Vs [E][d_out][r] (packed INT4 and
    fp16 scales), A [E][d_in][r], Bt [E][r][d_out] (fp64, before quantisation), sigma [E][r], rel_err [E] (of A Bt
    against the residual), cosine [E], pruned [E])."""
    E, d_in, d_out = W.shape
    K = E // G
    B = shared_base(W, G)
    out = dict(B=B, A=np.zeros((E, d_in, r)), Bt=np.zeros((E, r, d_out)), sigma=np.zeros((E, r)), rel_err=np.zeros(E),
               cosine=np.zeros(E), pruned=np.zeros(E, np.int32),
               Uq=np.zeros((E, r * d_in // 2), np.uint8), Us=np.zeros((E, r * d_in // 32), np.float16),
               Vq=np.zeros((E, d_out * r // 2), np.uint8), Vs=np.zeros((E, d_out * r // 32), np.float16))
    for e in range(E):
        base = B[e // K].astype(np.float64)
        dW = W[e].astype(np.float64) - base
        A, Bt, S = truncated_factors(dW, r)
        nd, nb = np.linalg.norm(dW), np.linalg.norm(base)
        cos = float((dW * base).sum() / (nd * nb)) if nd > 0 and nb > 0 else 0.0
        out["cosine"][e] = cos
        out["sigma"][e] = S
        out["rel_err"][e] = np.linalg.norm(dW - A @ Bt) / nd if nd > 0 else 0.0
        if gamma > 0.0 and cos < gamma:
            out["pruned"][e] = 1           # zero block: codes and scales stay zero
            continue
        out["A"][e], out["Bt"][e] = A, Bt
        out["Uq"][e], out["Us"][e] = quantize_int4_groups(A.T)          # U layout [r][d_in]: d_in fastest
        out["Vq"][e], out["Vs"][e] = quantize_int4_groups(Bt.T)         # V layout [d_out][r]: r fastest
    return out


def reconstruct(c: dict, e: int, K: int, d_in: int, d_out: int, r: int) -> np.ndarray:
    """W~_e = W_base + deq(U_e) deq(V_e) from the stored form (Eq. 7), fp64."""
    U = dequantize_int4_groups(c["Uq"][e], c["Us"][e]).reshape(r, d_in)
    V = dequantize_int4_groups(c["Vq"][e], c["Vs"][e]).reshape(d_out, r)
    return c["B"][e // K].astype(np.float64) + U.T @ V.T
