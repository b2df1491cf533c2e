"""Work distribution of the persistent two-CTA GEMM (Eq. 7, outer sum).

The clusters walk the 256 x 256 output tiles round-robin; an output element is produced by one
chain of MMAs over the whole of K whatever the number of clusters, so the result must not change
by a single bit when that number does.  The test hook `wush_debug_gemm_clusters` makes small
problems run on 1..11 clusters: every cluster then takes several tiles in a row (accumulator
hand-over, ring phases carried across tiles), with a ragged last tile column and a ragged last
tile row; the unrestricted run is checked against the fp64 oracle product.
"""
import numpy as np
import pytest
import torch

from oracle import formats as F
from oracle import pipeline as P
from oracle import quantizers as Q
from paper_2512_00956_b200 import wush
from parity_util import dev, rel_fro, tile

pytestmark = pytest.mark.gpu
G = Q.GROUP


def _operand(rng, rows, K, fmt):
    """Random E2M1 codes and scale bytes of a useful range (no quantiser involved)."""
    g = G[fmt]
    codes = rng.integers(0, 16, size=(rows, K), dtype=np.uint8)
    if fmt == "mxfp4":
        sc = rng.integers(121, 132, size=(rows, K // g), dtype=np.uint8)         # 2^-6 .. 2^4
    else:
        sc = rng.integers(0x28, 0x50, size=(rows, K // g), dtype=np.uint8)       # E4M3 0.03 .. 3.5
    return codes, sc


@pytest.mark.parametrize("fmt", ["mxfp4", "nvfp4"])
@pytest.mark.parametrize("M,N,K", [(300, 1000, 512), (520, 840, 320), (256, 2304, 256), (700, 584, 1024)])
def test_result_does_not_depend_on_the_number_of_clusters(fmt, M, N, K):
    rng = np.random.default_rng(M * 7 + N)
    xc, xs = _operand(rng, M, K, fmt)
    wc, ws = _operand(rng, N, K, fmt)
    ts = 0.0123 if fmt == "nvfp4" else None
    tsd = dev(np.full(4, ts, dtype=np.float32)) if fmt == "nvfp4" else None
    args = (dev(F.pack_e2m1(xc)), dev(tile(xs)), dev(F.pack_e2m1(wc)), dev(tile(ws)), K, fmt, tsd, tsd)
    old = wush.debug_gemm_clusters(0)
    try:
        Y0, st = wush.gemm_fp4(*args)
        Y0b, _ = wush.gemm_fp4(*args, out_dtype=torch.bfloat16)
        torch.cuda.synchronize()
        assert int(st[0].item()) == 0
        Yo = P.dequantized_product(Q.dequantize(xc, xs, fmt, ts), Q.dequantize(wc, ws, fmt, ts))
        assert rel_fro(Y0.cpu().numpy(), Yo) <= 1e-5
        for limit in (1, 2, 3, 5, 7, 11):
            wush.debug_gemm_clusters(limit)
            Y, st = wush.gemm_fp4(*args)
            Yb, _ = wush.gemm_fp4(*args, out_dtype=torch.bfloat16)
            torch.cuda.synchronize()
            assert int(st[0].item()) == 0
            assert torch.equal(Y, Y0), f"fp32 output changed with {limit} clusters"
            assert torch.equal(Yb, Y0b), f"bf16 output changed with {limit} clusters"
    finally:
        wush.debug_gemm_clusters(old)


@pytest.mark.parametrize("fmt", ["mxfp4", "nvfp4"])
@pytest.mark.parametrize("M,N,K", [(129, 8, 64), (130, 24, 192), (257, 264, 320), (513, 40, 576)])
def test_smallest_and_ragged_shapes_of_the_two_cta_path(fmt, M, N, K):
    """M just above the single-CTA limit, N of a few columns, K of one partial slab (64, 192) or of a whole
    slab plus a partial one (320, 576): against the fp64 oracle product of the same codes."""
    rng = np.random.default_rng(M + N + K)
    xc, xs = _operand(rng, M, K, fmt)
    wc, ws = _operand(rng, N, K, fmt)
    ts = 0.031 if fmt == "nvfp4" else None
    tsd = dev(np.full(4, ts, dtype=np.float32)) if fmt == "nvfp4" else None
    Y, st = wush.gemm_fp4(dev(F.pack_e2m1(xc)), dev(tile(xs)), dev(F.pack_e2m1(wc)), dev(tile(ws)), K, fmt, tsd, tsd)
    torch.cuda.synchronize()
    assert int(st[0].item()) == 0
    Yo = P.dequantized_product(Q.dequantize(xc, xs, fmt, ts), Q.dequantize(wc, ws, fmt, ts))
    assert rel_fro(Y.cpu().numpy(), Yo) <= 1e-5
