"""LSTM layer under a row pattern on its hidden units, driven through the C ABI.

This module only owns buffers and the order of the calls: every product and every cell update runs in
the library's kernels (`ard_lstm_gate_gemm`, `ard_lstm_gates`, `ard_lstm_gates_bwd`,
`ard_lstm_gate_gemm_bwd`, `ard_bwd_weight`).  One pattern serves all time steps of a sequence (Sec. 7).

Layout: XH [T+1][B][I+H] bf16 holds [x_t, h_{t-1}] side by side, so the cell kernel writes h_t straight into
the operand of step t+1 (full width, zeros at dropped units); C [T+1][B][H] fp32 holds the cell state compact
over kept units; G [T][B][4H] fp32 the saved gate activations; Z [B][4H] fp32 the pre-activations of a step.
"""
from __future__ import annotations

import torch

from . import ard


class LstmLayer:
    def __init__(self, ctx, pat, T, B, I, H, W_nm):
        """W_nm: bf16 [4H][I+H] neuron-major weight (gate blocks i|f|g|o along the rows)."""
        self.ctx, self.pat, self.T, self.B, self.I, self.H = ctx, pat, T, B, I, H
        self.KH = I + H
        self.W = W_nm
        bf, f32 = torch.bfloat16, torch.float32
        self.XH = torch.zeros((T + 1, B, self.KH), dtype=bf, device="cuda")
        self.C = torch.zeros((T + 1, B, H), dtype=f32, device="cuda")
        self.G = torch.zeros((T, B, 4 * H), dtype=f32, device="cuda")
        self.Z = torch.zeros((B, 4 * H), dtype=f32, device="cuda")
        self.DZ = torch.zeros((T, B, 4 * H), dtype=bf, device="cuda")
        self.D = torch.zeros((T, B, self.KH), dtype=f32, device="cuda")   # [dx_t | total dh_{t-1}]
        self.dc = torch.zeros((B, H), dtype=f32, device="cuda")
        self.dW = torch.zeros((4 * H, self.KH), dtype=f32, device="cuda")

    def load_inputs(self, X):
        """X: bf16 [T][B][I]."""
        self.XH[:self.T, :, :self.I] = X

    def forward(self, alpha):
        ard.ard_lstm_forward(self.ctx, self.pat, self.T, self.B, self.I, self.H, alpha, self.XH, self.W, self.KH,
                             None, self.C, self.G, self.Z)
        return self.XH[1:, :, self.I:]

    def backward(self, alpha, dH):
        """dH: fp32 [T][B][H], gradient with respect to every h_t.  Returns (dX [T][B][I] fp32 view, dW)."""
        ctx, pat, T, B, H, KH, I = self.ctx, self.pat, self.T, self.B, self.H, self.KH, self.I
        self.D.zero_()
        self.D[1:, :, I:] = dH[:-1]            # upstream gradient of h_{t-1}; the data GEMM of step t adds to it
        self.dc.zero_()
        dh_last = dH[T - 1].contiguous()
        ard.ard_lstm_backward(ctx, pat, T, B, I, H, alpha, self.XH, self.W, KH, self.C, self.G, dh_last, self.D,
                              self.dc, self.DZ, self.dW)
        return self.D[:, :, :I], self.dW
