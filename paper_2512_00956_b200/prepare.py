"""Offline preparation of one linear layer (Algorithm 2, RTN case) on the GPU.

Second moments come from the library's calibration kernel (`wush_calib_moments`), the d x d
factorisations of Algorithm 1 and the inverse-transpose of Eq. 6 from `wush_build_transforms`,
the weight quantisation from `wush_quantize_weight`: nothing leaves the device.  The comparison
transforms of Sec. 5 / Table 1 (one shared Hadamard matrix, the identity, WUSH without its Hadamard
factor) come from `wush_build_transforms_kind` as well, so this module holds no arithmetic of its own.

Conventions (the paper leaves them open): damping ratio lambda = 0.01; singular values
descending and each row of U^T W'^T signed so that its largest-magnitude entry is positive
(Lemma A.1 shows this product does not depend on the square-root factor); the activation-side
transform is stored in bf16 and the weight-side one is the inverse-transpose of the STORED
values, so that (x T^T)(w Tinv^T)^T = x w^T up to fp32 rounding of Tinv.
"""
import torch

from . import wush


def fixed_transforms(kind, C, d, device):
    """The data-independent comparison transforms of Sec. 5 / Table 1, in the layout the kernels take:
    "hadamard" (the same normalised Hadamard matrix for every block, the H + Quant baseline) or
    "identity" (None + Quant).  Returns (T bf16 [C,d,d], Tinv fp32 [C,d,d]) with Tinv = T^-T of the
    stored bf16 values, exactly as for WUSH.  Both are written by the library."""
    if kind not in ("hadamard", "identity"):
        raise ValueError(kind)
    T, Tinv, info = wush.fixed_transforms(kind, C, d, device)
    if int(info.abs().max().item()) != 0:
        raise wush.WushError("wush_build_transforms_kind: singular transform")
    return T, Tinv


class QuantizedLinear:
    """Holds what the online call needs: T, packed W~ codes, TILED scale bytes, tensor scales."""

    def __init__(self, W, Xc, fmt, lam=0.01, transform="wush", method="rtn"):
        """method "rtn": the RTN case of Algorithm 2 (moments, transforms, one pass of the weight quantiser);
        "gptq": its GPTQ case (`wush_gptq_quantize_weight`; NVFP4 takes the RTN case's weight tensor scale)."""
        f, g = wush.FORMATS[fmt]
        self.fmt, self.g = fmt, g
        self.N, self.K = W.shape
        if method == "gptq":
            if transform != "wush":
                raise ValueError("the GPTQ case builds WUSH transforms")
            ts = None
            if fmt == "nvfp4":
                rtn = QuantizedLinear(W, Xc, fmt, lam)
                ts = rtn.w_tensor_scale
            self.T, self.Tinv, self.w_codes, self.w_scales, self.info = wush.gptq_quantize_weight(W, Xc, fmt, lam, ts)
            if int(self.info.abs().max().item()) != 0:
                raise wush.WushError("wush_gptq_quantize_weight: a factorisation failed (see info)")
            self.w_tensor_scale = ts
            self.x_tensor_scale = wush.act_tensor_scale(Xc, self.T, g) if fmt == "nvfp4" else None
            self._ws = None
            return
        if method != "rtn":
            raise ValueError(method)
        if transform in ("wush", "wus"):
            mom_w, cnt_w = wush.calib_moments(W, g)
            mom_x, cnt_x = wush.calib_moments(Xc, g)
            # Algorithm 1 + Eq. 6 for every block in the library's own kernel (fp64 Cholesky, Jacobi SVD)
            self.T, self.Tinv, self.info = wush.build_transforms(mom_w, int(cnt_w[0].item()), mom_x,
                                                                 int(cnt_x[0].item()), g, lam, kind=transform)
            if int(self.info.abs().max().item()) != 0:
                raise wush.WushError("wush_build_transforms: a block failed to factorise (see info)")
        else:
            self.T, self.Tinv = fixed_transforms(transform, self.K // g, g, W.device)
        self.w_codes, self.w_scales, self.w_tensor_scale = wush.quantize_weight(W, self.Tinv, fmt, sf=wush.SF_TILED)
        if fmt == "nvfp4":
            self.x_tensor_scale = wush.act_tensor_scale(Xc, self.T, g)          # static: from the calibration tokens
        else:
            self.x_tensor_scale = None
        self._ws = None

    def __call__(self, X, out=None, out_dtype=torch.float32):
        need = wush.linear_workspace_bytes(X.shape[0], self.K, self.g)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=X.device)
        Y, _ = wush.linear(X, self.T, self.w_codes, self.w_scales, self.fmt, self.x_tensor_scale,
                           self.w_tensor_scale, out_dtype=out_dtype, out=out, workspace=self._ws)
        return Y
