"""Seeded synthetic inputs for the clustered-MoE layer forward.

This module only *draws and encodes data*: token activations, router
matrices, FP16 cluster bases and INT4-packed rank-r residual factors, in the
array layouts of the C boundary.  It holds none of the layer's arithmetic (no
expert FFN, no gating, no dequantisation); the CPU oracle and the CUDA
library each consume the arrays produced here and share nothing else.

Layouts (row-major, last index fastest):

    x    [T][d]          fp16    tokens
    C    [d][G]          fp32    cluster prototypes (column g is the paper's u_g, Eq. 9)
    R    [G][d][K]       fp32    in-cluster router vectors (columns are the paper's v_i, Eq. 10)
    b_c  [G], b_e [G][K] fp32    optional logit biases (only the skewed workload uses them)
    B1   [G][d][d_ff]    fp16    shared base of the up-projection   (Eq. 6)
    B2   [G][d_ff][d]    fp16    shared base of the down-projection (Eq. 6)
    U1q  [E][r][d]       int4    residual factor, reduction index fastest (Eq. 7)
    V1q  [E][d_ff][r]    int4
    U2q  [E][r][d_ff]    int4
    V2q  [E][d][r]       int4
    *s   one fp16 scale per 32 consecutive elements of the flattened factor

INT4 packing: two codes per byte, the element with the even flat index in the
low nibble, two's-complement codes in [-8, 7].

Expert slot e = g*K + j belongs to cluster g.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np

QUANT_GROUP = 32


@dataclasses.dataclass(frozen=True)
class LayerShape:
    name: str
    T: int
    d: int
    d_ff: int
    E: int
    G: int
    r: int
    k: int
    skew: bool = False

    @property
    def K(self) -> int:
        return self.E // self.G


# The five workloads: tiny, BERT-base-shaped, GPT-2-medium-shaped (compute
# bound headline), its skewed-load variant, and the decode-shaped weight
# streaming case.
CONFIGS = {
    "tiny": LayerShape("tiny", T=256, d=128, d_ff=512, E=8, G=2, r=4, k=2),
    "bert": LayerShape("bert", T=4096, d=768, d_ff=3072, E=16, G=4, r=16, k=2),
    "gpt2m": LayerShape("gpt2m", T=16384, d=1024, d_ff=4096, E=32, G=8, r=16, k=2),
    "skew": LayerShape("skew", T=16384, d=1024, d_ff=4096, E=32, G=8, r=16, k=2, skew=True),
    "decode": LayerShape("decode", T=64, d=4096, d_ff=14336, E=64, G=8, r=32, k=2),
}
CONFIG_ORDER = ["tiny", "bert", "gpt2m", "skew", "decode"]


def quantize_int4(w: np.ndarray) -> tuple[np.ndarray, np.ndarray]:
    """Symmetric INT4 encoder for one factor array.

    ``w`` is float32 with the reduction index last.  The array is flattened
    and cut into groups of 32 consecutive elements; each group gets the fp16
    scale absmax/7 (0 for an all-zero group) and codes
    clamp(round_half_even(w / scale), -8, 7).  Returns (packed uint8 of
    w.size/2 bytes, fp16 scales of w.size/32 entries).
    """
    flat = np.ascontiguousarray(w, dtype=np.float32).reshape(-1)
    if flat.size == 0:
        return np.zeros(0, np.uint8), np.zeros(0, np.float16)
    if flat.size % QUANT_GROUP:
        raise ValueError("factor size must be a multiple of 32")
    grp = flat.reshape(-1, QUANT_GROUP)
    absmax = np.max(np.abs(grp), axis=1)
    scale = (absmax / np.float32(7.0)).astype(np.float16)
    sf = scale.astype(np.float32)
    safe = np.where(sf > 0, sf, np.float32(1.0))
    q = np.rint(grp / safe[:, None])          # numpy rint rounds half to even
    q = np.where(sf[:, None] > 0, q, 0.0)
    q = np.clip(q, -8, 7).astype(np.int8).reshape(-1)
    nib = (q & 0xF).astype(np.uint8)
    packed = (nib[0::2] | (nib[1::2] << 4)).astype(np.uint8)
    return packed, scale


def zipf_shares(G: int, s: float = 1.2) -> np.ndarray:
    w = 1.0 / np.arange(1, G + 1, dtype=np.float64) ** s
    return w / w.sum()


def _calibrate_cluster_bias(x16: np.ndarray, C: np.ndarray, target: np.ndarray) -> np.ndarray:
    """Bias on the cluster logits that makes the realised top-1 cluster shares
    of *this* token batch follow ``target`` (skewed workload only).

    Deterministic fixed-point iteration: 30 rounds of
    b_g += 0.5 * sigma * (ln target_g - ln max(share_g, 1/T)), sigma = std of
    the unbiased logits (the step is scaled by sigma so that it also converges
    for small d, where the logits are narrow).
    """
    T = x16.shape[0]
    z0 = x16.astype(np.float64) @ C.astype(np.float64)
    sigma = float(z0.std())
    b = np.zeros(C.shape[1], np.float64)
    for _ in range(30):
        share = np.bincount(np.argmax(z0 + b, axis=1), minlength=C.shape[1]) / T
        b += 0.5 * sigma * (np.log(target) - np.log(np.maximum(share, 1.0 / T)))
    return b.astype(np.float32)


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round to nearest even (an encoding of the drawn data)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def make_layer(shape: LayerShape, seed: int = 0, T: int | None = None, base_scale: float = 1.0,
               factor_std: float = 0.02, base_dtype: str = "fp16") -> dict:
    """Draw one layer and one token batch.

    Draw order (float32 standard normals from numpy PCG64(seed)):
    x, C, R, B1, B2, U1, V1, U2, V2.  The second argument of the N(.,.)
    in the workload description is a standard deviation.
    Passing ``T`` overrides the number of tokens (x is drawn first, so the
    weights of a shape depend on T; use :func:`make_tokens` for extra batches
    against fixed weights).  ``base_scale`` multiplies both shared bases (0 gives a layer whose experts
    are their low-rank residuals alone) and ``factor_std`` replaces the 0.02 of the residual factors: test
    layers in which the residual terms, a few percent of the activations in the workloads, dominate.
    ``base_dtype`` "bf16" stores the two bases as bfloat16 bit patterns (uint16 arrays) instead of fp16.
    """
    T = shape.T if T is None else T
    d, d_ff, E, G, r, k = shape.d, shape.d_ff, shape.E, shape.G, shape.r, shape.k
    K = shape.K
    rng = np.random.Generator(np.random.PCG64(seed))

    def normal(size, std):
        a = rng.standard_normal(size, dtype=np.float32)
        a *= np.float32(std)
        return a

    x = normal((T, d), 1.0).astype(np.float16)
    C = normal((d, G), 0.02)
    R = normal((G, d, K), 0.02)
    B1 = normal((G, d, d_ff), base_scale / math.sqrt(d))
    B2 = normal((G, d_ff, d), base_scale / math.sqrt(d_ff))
    if base_dtype == "bf16":
        B1, B2 = to_bf16_bits(B1), to_bf16_bits(B2)
    else:
        B1, B2 = B1.astype(np.float16), B2.astype(np.float16)
    out = dict(shape=shape, T=T, seed=seed, x=x, C=C, R=R, B1=B1, B2=B2, b_c=None, b_e=None, base_dtype=base_dtype)
    for name, dims in (("U1", (E, r, d)), ("V1", (E, d_ff, r)), ("U2", (E, r, d_ff)), ("V2", (E, d, r))):
        w = normal(dims, factor_std)
        q, s = quantize_int4(w)
        out[name + "q"] = q
        out[name + "s"] = s
        del w
    if shape.skew:
        out["b_c"] = _calibrate_cluster_bias(x, C, zipf_shares(G, 1.2))
        b_e = np.zeros((G, K), np.float32)
        b_e[:, 0] = 1.0
        out["b_e"] = b_e
    return out


def make_tokens(shape: LayerShape, T: int, seed: int) -> np.ndarray:
    """An extra token batch x ~ N(0,1) in fp16, independent of the weights' stream."""
    rng = np.random.Generator(np.random.PCG64([seed, 0x70CE]))
    return rng.standard_normal((T, shape.d), dtype=np.float32).astype(np.float16)


def small_shape(name="s", T=37, d=64, d_ff=96, E=6, G=3, r=4, k=2, skew=False) -> LayerShape:
    """Helper for tests: an arbitrary small layer shape."""
    return LayerShape(name, T=T, d=d, d_ff=d_ff, E=E, G=G, r=r, k=k, skew=skew)


def make_dense_experts(E: int, G: int, d_in: int, d_out: int, seed: int = 0, spectrum=None, noise: float = 0.0,
                       base_std: float | None = None) -> np.ndarray:
    """Dense expert matrices [E][d_in][d_out] (fp32) that are correlated inside each cluster, the input of the offline
    compressor: W_e = C_g + sum_j spectrum[j] * p_j q_j^T + noise, with a cluster matrix C_g ~ N(0, base_std)
    (default 1/sqrt(d_in)), orthonormal p_j, q_j per expert (QR of seeded Gaussians) and `spectrum` the singular
    values of the expert's own part (default: 24 values decaying geometrically from 0.5).  The own parts of a cluster
    are centred (their mean over the cluster is removed) so that C_g is the cluster's mean up to the noise."""
    rng = np.random.Generator(np.random.PCG64([seed, 0xC0DE]))
    K = E // G
    spectrum = np.asarray(spectrum if spectrum is not None else 0.5 * 0.8 ** np.arange(24), np.float64)
    n = spectrum.size
    base_std = 1.0 / math.sqrt(d_in) if base_std is None else base_std
    W = np.empty((E, d_in, d_out), np.float32)
    for g in range(G):
        C = rng.standard_normal((d_in, d_out)) * base_std
        own = []
        for _ in range(K):
            P, _r = np.linalg.qr(rng.standard_normal((d_in, n)))
            Q, _r = np.linalg.qr(rng.standard_normal((d_out, n)))
            own.append((P * spectrum[None, :]) @ Q.T + noise * rng.standard_normal((d_in, d_out)))
        mean_own = sum(own) / K
        for i in range(K):
            W[g * K + i] = (C + own[i] - mean_own).astype(np.float32)
    return W
