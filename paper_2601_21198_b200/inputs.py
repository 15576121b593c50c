"""Seeded synthetic inputs shaped like the paper's MoE expert weights.

This module only draws numbers: it holds none of the codec's or the FFN's
arithmetic, and it is the one module that both the CUDA-side tests and the
oracle-side tests may use.  All tensors are returned as bf16 BIT PATTERNS in
numpy uint16 arrays (fp32 draws rounded to nearest-even), so that no float
conversion ever sits between a generator and a bit-exact comparison.

The paper's models (DeepSeekV2-Lite, Qwen1.5-MoE, Switch-Large-128; Section 5)
are not available; Gaussian weights with std ~0.02 give an exponent entropy of
about 2.55 bits against the 2.55-2.65 bits the paper reports (Fig. 2).
"""
import numpy as np


def _rng(seed):
    return np.random.Generator(np.random.Philox(int(seed)))


def f32_to_bf16_bits(x):
    """float32 array -> bf16 bit patterns, round-to-nearest-even (NaN kept quiet)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    b = x.view(np.uint32)
    r = ((b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        r = np.where(nan, ((b >> np.uint32(16)) | np.uint32(0x40)).astype(np.uint16), r)
    return r


def bf16_bits_to_f32(u):
    return (np.ascontiguousarray(u, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def gaussian(shape, std, seed):
    """N(0, std) weights as bf16 bit patterns."""
    n = int(np.prod(shape))
    g = _rng(seed)
    out = np.empty(n, np.uint16)
    step = 1 << 24
    for a in range(0, n, step):
        m = min(step, n - a)
        out[a:a + m] = f32_to_bf16_bits(g.standard_normal(m, dtype=np.float32) * np.float32(std))
    return out.reshape(shape)


def single_expert_matrix(seed=0):
    """One 2048x1408 expert matrix, N(0, 0.02)."""
    return gaussian((2048, 1408), 0.02, seed)


SMALL_EXPERT_TENSORS = (("gate", (1408, 2048)), ("up", (1408, 2048)), ("down", (2048, 1408)))


def small_expert_tensor(e, j, seed=1):
    """Tensor j (0 gate, 1 up, 2 down) of expert e of a DeepSeekV2-Lite /
    Qwen1.5-MoE sized layer: gate and up [1408, 2048], down [2048, 1408];
    per-expert std 0.02 * U(0.5, 1.5)."""
    std = 0.02 * float(_rng(seed + e).uniform(0.5, 1.5))
    return gaussian(SMALL_EXPERT_TENSORS[j][1], std, 10_000 + 3 * (seed + e) + j)


def small_expert_layer(n_experts=64, seed=1):
    """Yields (expert, name, array) over the whole layer."""
    for e in range(n_experts):
        for j, (name, _) in enumerate(SMALL_EXPERT_TENSORS):
            yield e, name, small_expert_tensor(e, j, seed)


def outlier_matrix(rows, cols, std, seed, frac=0.001, gain=20.0):
    """N(0, std) with a fraction `frac` of input channels (columns) scaled by
    `gain` -- the outlier-channel structure of large LLM weight matrices."""
    g = _rng(seed)
    n_out = max(1, int(round(cols * frac)))
    chans = g.choice(cols, size=n_out, replace=False)
    w = np.empty((rows, cols), np.uint16)
    step = max(1, (1 << 24) // cols)
    for a in range(0, rows, step):
        m = min(step, rows - a)
        x = g.standard_normal((m, cols), dtype=np.float32) * np.float32(std)
        x[:, chans] *= np.float32(gain)
        w[a:a + m] = f32_to_bf16_bits(x)
    return w


LARGE_EXPERT_TENSORS = ("w1", "w3", "w2")


def large_expert_tensor(e, j, seed=100, hidden=4096, inter=14336, std=0.015):
    """Tensor j (0 w1, 1 w3: [inter, hidden]; 2 w2: [hidden, inter]) of expert e:
    N(0, std) plus 0.1 % outlier channels at 20x."""
    rows, cols = (inter, hidden) if j < 2 else (hidden, inter)
    return outlier_matrix(rows, cols, std, 3 * (seed + e) + j)


def large_expert_layer(n_experts=8, seed=100, hidden=4096, inter=14336, std=0.015):
    """Yields (expert, name, array) over the whole layer."""
    for e in range(n_experts):
        for j, name in enumerate(LARGE_EXPERT_TENSORS):
            yield e, name, large_expert_tensor(e, j, seed, hidden, inter, std)


def special_patterns():
    """Every bf16 pattern that is not an ordinary normal number: +-0, all 254
    denormals, +-Inf, and a spread of quiet and signalling NaN payloads."""
    p = [0x0000, 0x8000, 0x7F80, 0xFF80]
    p += list(range(0x0001, 0x0080)) + list(range(0x8001, 0x8080))
    p += [0x7F81, 0x7FBF, 0x7FC0, 0x7FC1, 0x7FFF, 0xFF81, 0xFFBF, 0xFFC0, 0xFFFF]
    return np.array(p, dtype=np.uint16)


STRESS_FAMILIES = ("laplace", "student_t", "uniform_bits", "specials")
STRESS_CHUNKS = (1024, 16384, 262144)


def stress_tensor(index, seed=7, min_elems=1024, max_elems=4 << 20):
    """Tensor `index` of the codec stress set: size log-uniform in
    [min_elems, max_elems] (rarely a multiple of anything), family and chunk
    size cycled.  Returns (bf16 patterns 1-D, family, chunk_elems)."""
    g = _rng(seed * 1_000_003 + index)
    n = int(np.exp(g.uniform(np.log(min_elems), np.log(max_elems))))
    fam = STRESS_FAMILIES[index % 4]
    chunk = STRESS_CHUNKS[(index // 4) % 3]
    if fam == "laplace":
        x = f32_to_bf16_bits(g.laplace(0.0, 0.01, n).astype(np.float32))
    elif fam == "student_t":
        x = f32_to_bf16_bits((g.standard_t(3.0, n) * 0.01).astype(np.float32))
    elif fam == "uniform_bits":
        x = g.integers(0, 1 << 16, n, dtype=np.uint16)
    else:
        x = f32_to_bf16_bits(g.standard_normal(n, dtype=np.float32) * np.float32(0.02))
        sp = special_patterns()
        k = max(1, n // 50)
        x[g.integers(0, n, k)] = sp[g.integers(0, sp.size, k)]
    return x, fam, chunk


def tokens(T, hidden, seed):
    """T hidden states, N(0, 1), bf16 patterns [T, hidden]."""
    return gaussian((T, hidden), 1.0, 500_000 + seed)


def routing(T, n_experts=8, k=2, seed=0, zipf_s=1.2):
    """Top-k routing: expert popularity follows Zipf(zipf_s) over a seeded
    permutation of the experts; each token draws k distinct experts without
    replacement (ids in draw order).  Combine weights are the softmax over
    n_experts seeded N(0,1) logits, gathered at the chosen ids and renormalised
    to sum to one.  Returns (ids int32 [T,k], weights float32 [T,k])."""
    g = _rng(900_000 + seed)
    perm = g.permutation(n_experts)
    p = 1.0 / np.arange(1, n_experts + 1) ** zipf_s
    pop = np.empty(n_experts)
    pop[perm] = p / p.sum()
    ids = np.empty((T, k), np.int32)
    for t in range(T):
        ids[t] = g.choice(n_experts, size=k, replace=False, p=pop)
    logits = g.standard_normal((T, n_experts))
    sm = np.exp(logits - logits.max(axis=1, keepdims=True))
    sm /= sm.sum(axis=1, keepdims=True)
    w = np.take_along_axis(sm, ids.astype(np.int64), axis=1)
    w /= w.sum(axis=1, keepdims=True)
    return ids, w.astype(np.float32)
