"""Seeded synthetic inputs for the W4A4 WUSH linear layer.

This module holds input GENERATION only: no transform, no quantiser, nothing of
the method.  It is the one module the CPU oracle's tests and the CUDA path's
callers share, so that both sides read identical bytes.  Everything is drawn in
fp64 from numpy's PCG64 with fixed seeds and rounded once to bf16; arrays are
returned as bf16 BIT PATTERNS (uint16).

The five workloads stand in for linear-layer inputs of Llama-3.1-8B / 70B
(shapes) with the activation statistics the paper's setting cares about:
per-channel scale spread, a few massive outlier channels, heavy tails, and the
skewed SiLU(a)*b input of a down-projection.  No model weights, datasets or
benchmark items are involved.
"""
from dataclasses import dataclass, field
import numpy as np


@dataclass(frozen=True)
class LayerConfig:
    index: int                 # 1-based, as listed in the benchmark description
    name: str
    M: int
    K: int
    N: int
    formats: tuple             # subset of ("mxfp4", "nvfp4")
    calib_tokens: int
    x_kind: str                # "gauss_outlier" | "student_t" | "silu_gate"
    x_sigma: float             # sigma of the log-normal per-channel scale
    outlier_frac: float
    outlier_gain: float
    w_std: float
    w_row_sigma: float         # sigma of the log-normal per-row scale (0 = none)
    m_sweep: tuple = field(default=())


CONFIGS = {
    1: LayerConfig(1, "small-2048x2048-mxfp4", 128, 2048, 2048, ("mxfp4",), 512,
                   "gauss_outlier", 0.5, 0.01, 50.0, 0.02, 0.3),
    2: LayerConfig(2, "llama8b-attn-out-nvfp4", 2048, 4096, 4096, ("nvfp4",), 1024,
                   "gauss_outlier", 0.5, 0.01, 50.0, 0.02, 0.3),
    3: LayerConfig(3, "llama8b-gate-up-mxfp4", 4096, 4096, 14336, ("mxfp4",), 2048,
                   "student_t", 0.5, 0.005, 100.0, 0.02, 0.0),
    4: LayerConfig(4, "llama8b-down-both", 4096, 14336, 4096, ("mxfp4", "nvfp4"), 2048,
                   "silu_gate", 1.0, 0.0, 1.0, 0.015, 0.0),
    5: LayerConfig(5, "llama70b-mlp-msweep", 4096, 8192, 28672, ("mxfp4", "nvfp4"), 4096,
                   "gauss_outlier", 0.5, 0.01, 50.0, 0.01, 0.0,
                   m_sweep=(1, 16, 128, 1024, 4096, 16384)),
}

GROUP = {"mxfp4": 32, "nvfp4": 16, "mxfp4_ceil": 32}


def to_bf16_bits(x):
    """fp64/fp32 array -> bf16 bit patterns (uint16), round-half-even on the fp32 value."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    b = f.view(np.uint32)
    rounded = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(bits):
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def channel_scales(cfg, K=None):
    """Per-channel activation scales incl. the seeded outlier channels (seed 1000+i)."""
    K = cfg.K if K is None else K
    rng = np.random.Generator(np.random.PCG64(1000 + cfg.index))
    s = np.exp(cfg.x_sigma * rng.standard_normal(K))
    n_out = int(round(cfg.outlier_frac * K))
    if n_out > 0:
        idx = rng.choice(K, size=n_out, replace=False)
        s[idx] *= cfg.outlier_gain
    return s


def _noise(cfg, rng, rows, K, chunk=2048):
    out = np.empty((rows, K), dtype=np.float32)
    for r0 in range(0, rows, chunk):
        r1 = min(rows, r0 + chunk)
        shape = (r1 - r0, K)
        if cfg.x_kind == "gauss_outlier":
            z = rng.standard_normal(shape)
        elif cfg.x_kind == "student_t":
            z = rng.standard_t(3.0, size=shape)
        elif cfg.x_kind == "silu_gate":
            a = rng.standard_normal(shape)
            b = rng.standard_normal(shape)
            z = a / (1.0 + np.exp(-a)) * b
        else:
            raise ValueError(cfg.x_kind)
        out[r0:r1] = z
    return out


def activations(cfg, M=None, K=None, seed_base=2000):
    """X[M, K] as bf16 bits.  seed_base 2000 = inference tokens, 3000 = calibration tokens."""
    M = cfg.M if M is None else M
    K = cfg.K if K is None else K
    rng = np.random.Generator(np.random.PCG64(seed_base + cfg.index))
    z = _noise(cfg, rng, M, K)
    z *= channel_scales(cfg, K).astype(np.float32)[None, :]
    return to_bf16_bits(z)


def calibration(cfg, B=None, K=None):
    return activations(cfg, cfg.calib_tokens if B is None else B, K, seed_base=3000)


def weights(cfg, N=None, K=None, chunk=2048):
    """W[N, K] as bf16 bits (seed 4000+i)."""
    N = cfg.N if N is None else N
    K = cfg.K if K is None else K
    rng = np.random.Generator(np.random.PCG64(4000 + cfg.index))
    row = np.exp(cfg.w_row_sigma * rng.standard_normal(N)) if cfg.w_row_sigma > 0 else np.ones(N)
    out = np.empty((N, K), dtype=np.uint16)
    for r0 in range(0, N, chunk):
        r1 = min(N, r0 + chunk)
        w = cfg.w_std * rng.standard_normal((r1 - r0, K)) * row[r0:r1, None]
        out[r0:r1] = to_bf16_bits(w)
    return out


def layer_inputs(cfg, M=None, N=None, K=None, B=None):
    """All three tensors of one layer; sizes may be shrunk for quick tests."""
    return dict(X=activations(cfg, M, K), W=weights(cfg, N, K), Xc=calibration(cfg, B, K))


def correlated_layer(seed, N, K, B, rho=0.6):
    """(W bits [N, K], Xc bits [B, K]) with activations correlated ACROSS quantisation blocks: an AR(1) chain over
    the channels plus a component shared by all channels, then log-normal channel scales.  Stand-in for a layer
    whose Hessian is far from block diagonal (the case error propagation between blocks is for)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    z = rng.standard_normal((B, K))
    x = np.empty_like(z)
    x[:, 0] = z[:, 0]
    for k in range(1, K):
        x[:, k] = rho * x[:, k - 1] + np.sqrt(1.0 - rho * rho) * z[:, k]
    x += 0.5 * rng.standard_normal((B, 1))
    x *= np.exp(0.5 * rng.standard_normal(K))[None, :]
    w = 0.02 * rng.standard_normal((N, K))
    return to_bf16_bits(w), to_bf16_bits(x)
