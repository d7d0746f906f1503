"""Seeded synthetic inputs shared by the tests, the oracle checks and the benchmark.

This module holds data generation only: random draws, outlier-channel scaling
and dtype casts.  None of the quantisation method's arithmetic lives here.  The
tensors stand in for LLaMA / Mistral activations and weights: they copy the
layer shapes and the outlier-channel structure (a few channels one to two
orders of magnitude larger than the rest), not any dataset's content.

16-bit tensors are returned as ``uint16`` bit patterns so that the CPU oracle
and the GPU library read exactly the same bytes.
"""
import numpy as np


def to_bf16_bits(x):
    """float32 -> bfloat16 bit patterns, round to nearest even."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b):
    return (np.ascontiguousarray(b, np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_f16_bits(x):
    return np.ascontiguousarray(x, np.float32).astype(np.float16).view(np.uint16)


def _outlier_channels(rng, x, frac=0.01):
    """Scale round(frac * K) channels (columns), fixed by the generator state, by 10**U(1,2)."""
    K = x.shape[-1]
    n = max(1, int(round(frac * K)))
    ch = rng.choice(K, n, replace=False)
    f = 10.0 ** rng.uniform(1.0, 2.0, n)
    x[..., ch] *= f
    return x


def tiny_case(seed=0):
    """X fp32 [16,256] ~ N(0,1) with channel 7 x40; W fp32 [128,256] ~ N(0, 0.02)."""
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((16, 256))
    X[:, 7] *= 40.0
    W = 0.02 * rng.standard_normal((128, 256))
    return X.astype(np.float32), W.astype(np.float32)


def act_normal_outliers(M, K, seed=1):
    """bf16 [M,K] ~ N(0,1) with 1 % outlier channels (the activation-quantizer workload)."""
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((M, K), dtype=np.float32)
    return to_bf16_bits(_outlier_channels(rng, X))


def act_student_t(M, K, seed=2):
    """bf16 [M,K] ~ Student-t(nu=4) with 1 % outlier channels (attention/MLP input stand-in)."""
    rng = np.random.default_rng(seed)
    X = rng.standard_t(4, (M, K)).astype(np.float32)
    return to_bf16_bits(_outlier_channels(rng, X))


def act_post_silu(M, K, seed=3):
    """bf16 [M,K]: |N(0,1)| * N(0,1) products with 1 % outlier channels (gated-MLP stand-in)."""
    rng = np.random.default_rng(seed)
    X = np.abs(rng.standard_normal((M, K), dtype=np.float32)) * rng.standard_normal((M, K), dtype=np.float32)
    return to_bf16_bits(_outlier_channels(rng, X))


def weights_normal(N, K, seed=2, std=0.02):
    """bf16 [N,K] ~ N(0, std)."""
    rng = np.random.default_rng(seed + 1000)
    return to_bf16_bits(std * rng.standard_normal((N, K), dtype=np.float32))


def attention_case(heads=32, kv_heads=8, seq=4096, head_dim=128, seed=4, p_heads=None):
    """Mistral-shaped attention operands.

    Q [heads, seq, d], K [kv_heads, seq, d], V [kv_heads, seq, d] as bf16 bits;
    Q and K carry two outlier head-dim channels per KV group (same channels for
    the query heads of the group).  P [p_heads, seq, seq] fp32 rows are
    Dirichlet(0.1) draws (softmax-like: most mass on few keys, many tiny
    entries).  ``p_heads`` limits how many heads of P are generated.
    """
    rng = np.random.default_rng(seed)
    group = heads // kv_heads
    Q = rng.standard_normal((heads, seq, head_dim), dtype=np.float32)
    Kt = rng.standard_normal((kv_heads, seq, head_dim), dtype=np.float32)
    for g in range(kv_heads):
        ch = rng.choice(head_dim, 2, replace=False)
        f = (10.0 ** rng.uniform(1.0, 2.0, 2)).astype(np.float32)
        Kt[g][:, ch] *= f
        Q[g * group:(g + 1) * group][:, :, ch] *= f
    V = rng.standard_normal((kv_heads, seq, head_dim), dtype=np.float32)
    n_p = heads if p_heads is None else p_heads
    P = np.empty((n_p, seq, seq), np.float32)
    for h in range(n_p):
        g = rng.gamma(0.1, size=(seq, seq))
        g = np.maximum(g, np.finfo(np.float64).tiny)
        P[h] = (g / g.sum(-1, keepdims=True)).astype(np.float32)
    return to_bf16_bits(Q), to_bf16_bits(Kt), P, to_bf16_bits(V)
