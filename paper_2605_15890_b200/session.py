"""Convenience holder of a plan and its device buffers (torch tensors).

Pure plumbing around the C entry points: allocation of the message / scale /
status buffers with torch and lifetime of the plan handle. No arithmetic.
"""
import numpy as np
import torch

from . import binding as B


class Session:
    def __init__(self, n, k, d, row_ptr, col_idx, a, w, p, bits, bucket=512, seed=0, flags=0,
                 device="cuda:0"):
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.n, self.k, self.d, self.bucket = n, k, d, bucket
        self.bits = np.ascontiguousarray(bits, np.uint8)
        self.plan = B.agc_plan_create(n, k, d, row_ptr, col_idx, a, w, p, bits, bucket, seed, flags)
        self.codes = torch.empty(B.agc_codes_bytes(self.plan) // 4, dtype=torch.int32, device=self.device)
        self.scales = torch.empty(B.agc_scales_bytes(self.plan) // 4, dtype=torch.float32,
                                  device=self.device)
        self.status = torch.zeros(1, dtype=torch.int32, device=self.device)
        self.uses_tma = B.agc_plan_uses_tma(self.plan)
        self.first_block = 0

    def set_first_block(self, first_block):
        """Place this plan's coordinates at pack block `first_block` of a longer vector."""
        B.agc_plan_set_first_block(self.plan, first_block)
        self.first_block = first_block

    def close(self):
        if self.plan is not None:
            B.agc_plan_destroy(self.plan)
            self.plan = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def encode(self, G, rnd, stream=None):
        """G: (k, ld) float32 CUDA tensor with ld >= d."""
        assert G.dtype == torch.float32 and G.is_cuda and G.dim() == 2 and G.stride(1) == 1
        B.agc_encode_quantize(self.plan, G, G.stride(0), rnd, self.codes, self.scales, self.status, stream)

    def decode(self, masks, lr=None, ghat=None, beta=None, stream=None):
        """masks: (R, n) uint8 CUDA tensor."""
        assert masks.dtype == torch.uint8 and masks.is_cuda and masks.is_contiguous()
        R = masks.shape[0] if masks.dim() == 2 else 1
        B.agc_decode(self.plan, self.codes, self.scales, masks, R, lr, ghat, beta, self.status, stream)

    def residuals(self, masks, g_ref, stream=None):
        """||g_hat^(r) - g_ref||^2 of every realisation: float64 CUDA tensor [R]; no g_hat is stored."""
        assert masks.dtype == torch.uint8 and masks.is_cuda and masks.is_contiguous()
        assert g_ref.dtype == torch.float32 and g_ref.is_cuda and g_ref.is_contiguous() and g_ref.numel() == self.d
        R = masks.shape[0] if masks.dim() == 2 else 1
        out = torch.empty(R, dtype=torch.float64, device=masks.device)
        B.agc_decode_residuals(self.plan, self.codes, self.scales, masks, R, g_ref, out, stream)
        return out

    def worker_words(self, i):
        lo = B.agc_worker_offset(self.plan, i) // 4
        hi = B.agc_worker_offset(self.plan, i + 1) // 4
        return lo, hi

    def codes_host(self):
        return self.codes.cpu().numpy().view(np.uint32)

    def scales_host(self):
        nb = (self.d + self.bucket - 1) // self.bucket if self.bucket else 1
        return self.scales.cpu().numpy().reshape(self.n, nb)
