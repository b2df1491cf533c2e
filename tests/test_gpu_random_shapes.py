"""Seeded sweeps over ragged shapes (GPU vs oracle): token counts that are no multiple of any tile
height, K tails of the 128-channel panels, both scale layouts, all three quantiser rules, random
(not WUSH-built) transforms.  Complements the fixed cases of test_gpu_parity.py."""
import numpy as np
import pytest
import torch

from oracle import formats as F
from oracle import pipeline as P
from oracle import quantizers as Q
from paper_2512_00956_b200 import wush
from parity_util import compare_quantized, dev, dev_bf16, rel_fro, untile

pytestmark = pytest.mark.gpu


def test_quantize_act_random_shapes():
    rng = np.random.default_rng(11)
    for _ in range(20):
        fmt = str(rng.choice(["mxfp4", "nvfp4", "mxfp4_ceil"]))
        g = Q.GROUP[fmt]
        K = int(rng.choice([64, 128, 256, 320, 512, 1024, 2048]))
        M = int(rng.integers(1, 1500))
        sf = int(rng.integers(0, 2))
        X_bits = F.f64_to_bf16_bits(rng.standard_normal((M, K)) * np.exp(rng.uniform(-2, 2, (1, K))))
        T_bits = F.f64_to_bf16_bits(rng.standard_normal((K // g, g, g)) / np.sqrt(g))
        v32 = P.transform_blocks(F.bf16_bits_to_f64(X_bits), F.bf16_bits_to_f64(T_bits)).astype(np.float32)
        ts = Q.nvfp4_tensor_scale(v32) if fmt == "nvfp4" else None
        ts_d = dev(np.full(4, ts, dtype=np.float32)) if ts is not None else None
        codes, scales = wush.quantize_act(dev_bf16(X_bits), dev_bf16(T_bits), fmt, ts_d, sf)
        torch.cuda.synchronize()
        sc = scales.cpu().numpy()
        if sf == wush.SF_TILED:
            sc = untile(sc, M, K // g)
        stats = compare_quantized(codes.cpu().numpy(), sc, v32, fmt, ts)
        assert stats["flipped_codes"] <= stats["guarded_elems"], (fmt, M, K, sf)


def test_quantize_weight_random_shapes():
    rng = np.random.default_rng(12)
    for _ in range(10):
        fmt = str(rng.choice(["mxfp4", "nvfp4", "mxfp4_ceil"]))
        g = Q.GROUP[fmt]
        K = int(rng.choice([64, 256, 320, 512, 1024]))
        N = int(rng.integers(1, 900))
        W_bits = F.f64_to_bf16_bits(0.02 * rng.standard_normal((N, K)))
        Tinv = (rng.standard_normal((K // g, g, g)) / np.sqrt(g)).astype(np.float32)      # any fp32 transform
        wbar = P.transform_blocks(F.bf16_bits_to_f64(W_bits), Tinv.astype(np.float64)).astype(np.float32)
        ts = Q.nvfp4_tensor_scale(wbar) if fmt == "nvfp4" else None
        codes, scales, ts_g = wush.quantize_weight(dev_bf16(W_bits), dev(Tinv), fmt, sf=wush.SF_LINEAR)
        torch.cuda.synchronize()
        if fmt == "nvfp4":
            assert abs(float(ts_g[0].item()) - float(ts)) <= 2e-7 * float(ts)
        compare_quantized(codes.cpu().numpy(), scales.cpu().numpy(), wbar, fmt, ts)


def test_calib_moments_random_shapes():
    rng = np.random.default_rng(7)
    for _ in range(20):
        g = int(rng.choice([16, 32]))
        K = int(rng.choice([64, 128, 192, 256, 320, 448, 512, 1024, 2048, 4096]))
        B = int(rng.integers(1, 3000))
        X_bits = F.f64_to_bf16_bits(rng.standard_normal((B, K)))
        X = dev_bf16(X_bits)
        mom, cnt = wush.calib_moments(X, g)
        mom2, cnt2 = wush.calib_moments(X, g, mom.clone(), cnt.clone())       # accumulates in place
        torch.cuda.synchronize()
        S = P.second_moment_sums(F.bf16_bits_to_f64(X_bits), g)
        assert int(cnt[0].item()) == B and int(cnt2[0].item()) == 2 * B
        assert rel_fro(mom.cpu().numpy(), S) <= 1e-5, (g, K, B)
        assert rel_fro(mom2.cpu().numpy(), 2 * S) <= 1e-5, (g, K, B)
