"""CPU oracle for the routed expert SwiGLU FFN on decoded weights (numpy, fp64).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only tests, the smoke check and the
benchmark's CPU-baseline leg may import this module.  It shares nothing with
the CUDA library.

The paper names the step only as the GPU time p_n spent on all tokens routed
to expert n once its tensors are recovered (Section 3.3, scheduler notation);
it does not define the expert network.  The form used here is the standard
gated FFN of the MoE models the paper evaluates:

    g = W1 x,  u = W3 x,  h = bf16(SiLU(g) * u),  y = W2 h
    out[t] = bf16( sum_j  w[t, j] * y_{ids[t, j]}[t] )

with W1, W3 of shape [I, H], W2 of shape [H, I] (row-major, [out, in]),
SiLU(z) = z / (1 + exp(-z)), sums in fp64 and two roundings to bf16
(round-to-nearest-even): the intermediate h and the final output.
"""
import numpy as np


def bf16_to_f64(u16):
    """bf16 bit patterns -> the real numbers they denote (Section 2.2:
    (-1)^sign * 2^(exponent-127) * 1.mantissa), as float64."""
    u = np.ascontiguousarray(u16, dtype=np.uint16)
    return (u.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f64_to_bf16(x):
    """Round float64 to the nearest bf16 (ties to even), returning bit patterns.
    One rounding: the value is scaled so that one unit is the bf16 spacing at
    its magnitude (8 significant bits; fixed spacing 2^-133 below 2^-126)."""
    x = np.asarray(x, dtype=np.float64)
    with np.errstate(all="ignore"):
        return _round_bf16(x)


def _round_bf16(x):
    _, e = np.frexp(x)                       # |x| = m * 2^e, 0.5 <= m < 1
    q = np.maximum(e - 8, -133).astype(np.float64)
    unit = np.exp2(q)
    r = np.rint(x / unit) * unit             # np.rint rounds halves to even
    r = np.where(np.isfinite(x), r, x)
    r32 = r.astype(np.float32)               # exact: r has at most 8 significant bits
    big = np.abs(r) >= 2.0 ** 128            # rounds past the largest finite bf16
    r32 = np.where(big, np.sign(r).astype(np.float32) * np.float32(np.inf), r32)
    return (r32.view(np.uint32) >> 16).astype(np.uint16)


def silu(z):
    z = np.asarray(z, dtype=np.float64)
    return z / (1.0 + np.exp(-z))


def expert_ffn(tokens, topk_ids, topk_weights, w1, w3, w2):
    """tokens [T, H] bf16 patterns; topk_ids [T, k] int; topk_weights [T, k]
    float or None (= 1.0); w1[e], w3[e]: [I, H] bf16 patterns; w2[e]: [H, I].
    Returns (out bf16 patterns [T, H], y float64 [T, H] before the last rounding)."""
    x = bf16_to_f64(tokens)
    T, H = x.shape
    ids = np.asarray(topk_ids)
    k = ids.shape[1]
    wts = np.ones((T, k)) if topk_weights is None else np.asarray(topk_weights, dtype=np.float64)
    y = np.zeros((T, H), dtype=np.float64)
    cache = {}
    for t in range(T):
        for j in range(k):
            e = int(ids[t, j])
            if e not in cache:
                cache[e] = (bf16_to_f64(w1[e]), bf16_to_f64(w3[e]), bf16_to_f64(w2[e]))
            a1, a3, a2 = cache[e]
            g = a1 @ x[t]
            u = a3 @ x[t]
            h = bf16_to_f64(f64_to_bf16(silu(g) * u))
            y[t] += wts[t, j] * (a2 @ h)
    return f64_to_bf16(y), y
