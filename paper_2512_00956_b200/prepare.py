"""Offline preparation of one linear layer (Algorithm 2, RTN case) on the GPU.

Second moments come from the library's calibration kernel (`wush_calib_moments`), the d x d
factorisations of Algorithm 1 and the inverse-transpose of Eq. 6 from `wush_build_transforms`,
the weight quantisation from `wush_quantize_weight`: nothing leaves the device.
`build_transforms` below is the same construction written with torch.linalg; it is kept as an
independent cross-check of the kernel and is not used by `QuantizedLinear`.

Conventions (the paper leaves them open): damping ratio lambda = 0.01; singular values
descending and each row of U^T W'^T signed so that its largest-magnitude entry is positive
(Lemma A.1 shows this product does not depend on the square-root factor); the activation-side
transform is stored in bf16 and the weight-side one is the inverse-transpose of the STORED
values, so that (x T^T)(w Tinv^T)^T = x w^T up to fp32 rounding of Tinv.
"""
import math

import torch

from . import wush


def hadamard(d, device):
    i = torch.arange(d, device=device)
    a = i[:, None] & i[None, :]
    pop = torch.zeros_like(a)
    for b in range(max(1, d.bit_length())):
        pop += (a >> b) & 1
    return torch.where(pop % 2 == 0, 1.0, -1.0).to(torch.float64) / math.sqrt(d)


def build_transforms(mom_w, n_w, mom_x, n_x, lam=0.01):
    """Unnormalised moment sums [C,d,d] (fp32) + row counts -> (T bf16 [C,d,d], Tinv fp32 [C,d,d])."""
    C, d, _ = mom_w.shape
    dev = mom_w.device
    eye = torch.eye(d, dtype=torch.float64, device=dev)
    Mw = mom_w.to(torch.float64) / float(n_w)
    Mx = mom_x.to(torch.float64) / float(n_x)
    Mw = 0.5 * (Mw + Mw.transpose(1, 2))
    Mx = 0.5 * (Mx + Mx.transpose(1, 2))
    tr_w = torch.diagonal(Mw, dim1=1, dim2=2).sum(-1)
    tr_x = torch.diagonal(Mx, dim1=1, dim2=2).sum(-1)
    Wp = torch.linalg.cholesky(Mw + (lam * tr_w / d)[:, None, None] * eye)      # W' W'^T = damped M_W
    Xp = torch.linalg.cholesky(Mx + (lam * tr_x / d)[:, None, None] * eye)
    U, S, _ = torch.linalg.svd(Wp.transpose(1, 2) @ Xp)                         # W'^T X' = U S V^T
    UtWt = U.transpose(1, 2) @ Wp.transpose(1, 2)
    pick = UtWt.abs().argmax(dim=2, keepdim=True)
    sgn = torch.sign(torch.gather(UtWt, 2, pick))
    sgn = torch.where(sgn == 0, torch.ones_like(sgn), sgn)
    UtWt = UtWt * sgn
    T = hadamard(d, dev) @ (UtWt / torch.sqrt(S)[:, :, None])                   # H S^-1/2 U^T W'^T
    T_bf16 = T.to(torch.bfloat16)
    Tinv = torch.linalg.inv(T_bf16.to(torch.float64)).transpose(1, 2)           # T_xvsh = T^-T (Eq. 6)
    return T_bf16.contiguous(), Tinv.to(torch.float32).contiguous()


def fixed_transforms(kind, C, d, device):
    """The data-independent comparison transforms of Sec. 5 / Table 1, in the layout the kernels take:
    "hadamard" (the same normalised Hadamard matrix for every block, the H + Quant baseline) or
    "identity" (None + Quant).  Returns (T bf16 [C,d,d], Tinv fp32 [C,d,d]) with Tinv = T^-T of the
    stored bf16 values, exactly as for WUSH."""
    if kind == "hadamard":
        T1 = hadamard(d, device)
    elif kind == "identity":
        T1 = torch.eye(d, dtype=torch.float64, device=device)
    else:
        raise ValueError(kind)
    T_bf16 = T1.to(torch.bfloat16)
    Tinv = torch.linalg.inv(T_bf16.to(torch.float64)).transpose(0, 1).to(torch.float32)
    return T_bf16.expand(C, d, d).contiguous(), Tinv.expand(C, d, d).contiguous()


class QuantizedLinear:
    """Holds what the online call needs: T, packed W~ codes, TILED scale bytes, tensor scales."""

    def __init__(self, W, Xc, fmt, lam=0.01, transform="wush"):
        f, g = wush.FORMATS[fmt]
        self.fmt, self.g = fmt, g
        self.N, self.K = W.shape
        if transform == "wush":
            mom_w, cnt_w = wush.calib_moments(W, g)
            mom_x, cnt_x = wush.calib_moments(Xc, g)
            # Algorithm 1 + Eq. 6 for every block in the library's own kernel (fp64 Cholesky, Jacobi SVD)
            self.T, self.Tinv, self.info = wush.build_transforms(mom_w, int(cnt_w[0].item()), mom_x,
                                                                 int(cnt_x[0].item()), g, lam)
            if int(self.info.abs().max().item()) != 0:
                raise wush.WushError("wush_build_transforms: a block failed to factorise (see info)")
        else:
            self.T, self.Tinv = fixed_transforms(transform, self.K // g, g, W.device)
        self.w_codes, self.w_scales, self.w_tensor_scale = wush.quantize_weight(W, self.Tinv, fmt, sf=wush.SF_TILED)
        if fmt == "nvfp4":
            v = wush.transform_act_f32(Xc, self.T, g)                            # static activation tensor scale
            self.x_tensor_scale = (v.abs().max().to(torch.float32) / 2688.0).reshape(1).repeat(4).contiguous()
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
