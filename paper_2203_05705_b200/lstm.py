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


class LstmStack:
    """Stack of LSTM layers with dropout on the layer OUTPUTS only (ard.h, "stacked LSTM"): every layer is computed
    in full, its row pattern masks what it hands up, and the consumer contracts over kept units only.

    Buffers and call order only.  Per layer l: `out_pats[l]` is the row pattern over its H units (sampled by the
    caller once per iteration), a dense pattern over (I+H -> H) serves the layer's own kernels and, for l > 0, a
    dense pattern over (I -> 4H) the products of its input half.  Yc[l] [T*B][H] bf16 holds the kept units of
    h_1..h_T side by side (unscaled); the rescale alpha_l rides on the consumer's products.
    """

    def __init__(self, ctx, T, B, dims, weights):
        """dims = [I0, H0, H1, ...]; weights[l]: bf16 [4 H_l][I_l + H_l] neuron-major, gate blocks i|f|g|o."""
        self.ctx, self.T, self.B, self.dims = ctx, T, B, list(dims)
        self.L = len(dims) - 1
        bf, f32 = torch.bfloat16, torch.float32
        self.layers, self.out_pats, self.gate_pats, self.Yc, self.dYc, self.Wk, self.dWk = [], [], [], [], [], [], []
        for l in range(self.L):
            I, H = dims[l], dims[l + 1]
            pat = ard.ard_pattern_create(ctx, ard.ARD_ROW, I + H, H, 0)           # stays dense
            self.layers.append(LstmLayer(ctx, pat, T, B, I, H, weights[l]))
            self.out_pats.append(ard.ard_pattern_create(ctx, ard.ARD_ROW, H, H, 0))
            self.gate_pats.append(ard.ard_pattern_create(ctx, ard.ARD_ROW, I, 4 * H, 0) if l > 0 else None)
            self.Yc.append(torch.zeros((T * B, H), dtype=bf, device="cuda"))
            self.dYc.append(torch.zeros((T * B, H), dtype=bf, device="cuda"))
            self.Wk.append(torch.zeros((4 * H, I), dtype=bf, device="cuda") if l > 0 else None)
            self.dWk.append(torch.zeros((4 * H, I), dtype=f32, device="cuda") if l > 0 else None)
        self.dh_last = [torch.zeros((B, dims[l + 1]), dtype=f32, device="cuda") for l in range(self.L)]

    def close(self):
        for p in self.out_pats + [q for q in self.gate_pats if q is not None] + [ly.pat for ly in self.layers]:
            ard.ard_pattern_destroy(p)

    def forward(self, X, alphas):
        """X: bf16 [T][B][I0].  Returns Yc of the top layer ([T*B][H], first n_keep columns valid, unscaled)."""
        ctx, T, B = self.ctx, self.T, self.B
        for l, ly in enumerate(self.layers):
            I, H, KH = ly.I, ly.H, ly.KH
            if l == 0:
                ly.load_inputs(X)
                ard.ard_lstm_forward(ctx, ly.pat, T, B, I, H, 1.0, ly.XH, ly.W, KH, None, ly.C, ly.G, ly.Z)
            else:
                # input half over the kept outputs of the layer below: both operands compact
                ard.ard_compact_weight_cols(ctx, self.gate_pats[l], self.out_pats[l - 1], ard.ARD_BF16, I, 4 * H, ly.W, KH,
                                            self.Wk[l], I)
                ard.ard_layer_fwd(ctx, self.gate_pats[l], self.out_pats[l - 1], ard.ARD_BF16, T * B, I, 4 * H, alphas[l - 1],
                                  self.Yc[l - 1], I, self.Wk[l], I, None, ly.G, 4 * H,
                                  ard.ARD_OUT_COMPACT | ard.ARD_FLAG_OUT_F32)
                ard.ard_lstm_forward_from_gates(ctx, ly.pat, T, B, I, H, 1.0, ly.XH, ly.W, KH, None, ly.C, ly.G)
            h1 = ly.XH.data_ptr() + (B * KH + I) * 2                    # h_1: the h half of XH[1]
            ard.ard_compact_cols(ctx, self.out_pats[l], ard.ARD_BF16, T * B, H, h1, KH, self.Yc[l], H)
        return self.Yc[-1]

    def backward(self, dYc_top, alphas):
        """dYc_top: bf16 [T*B][H_top], gradient with respect to the kept units of the top layer's masked output
        (first n_keep columns).  Returns (dX [T][B][I0] fp32 view, [dW_l fp32 [4H][I+H]])."""
        ctx, T, B = self.ctx, self.T, self.B
        dYc = dYc_top
        for l in reversed(range(self.L)):
            ly = self.layers[l]
            I, H, KH = ly.I, ly.H, ly.KH
            # upstream gradient of h_t, full width with the rescale: h half of D[t+1] for t < T-1, dH_last for t = T-1
            ly.D.zero_()
            ly.dc.zero_()
            dh_last = self.dh_last[l]
            if T > 1:
                ard.ard_expand_cols(ctx, self.out_pats[l], ard.ARD_BF16, (T - 1) * B, H, alphas[l], dYc, H,
                                    ly.D.data_ptr() + (B * KH + I) * 4, KH)
            ard.ard_expand_cols(ctx, self.out_pats[l], ard.ARD_BF16, B, H, alphas[l], dYc.data_ptr() + (T - 1) * B * H * 2, H,
                                dh_last, H)
            if l == 0:
                ard.ard_lstm_backward(ctx, ly.pat, T, B, I, H, 1.0, ly.XH, ly.W, KH, ly.C, ly.G, dh_last, ly.D, ly.dc, ly.DZ,
                                      ly.dW)
            else:
                ard.ard_lstm_backward_recurrent(ctx, ly.pat, T, B, I, H, 1.0, ly.XH, ly.W, KH, ly.C, ly.G, dh_last, ly.D,
                                                ly.dc, ly.DZ, ly.dW)
                gp, ip = self.gate_pats[l], self.out_pats[l - 1]
                # gradient with respect to the masked output y of the layer below (its rescale is applied when it is
                # expanded into that layer's upstream gradient); the weight gradient carries the rescale of G
                ard.ard_layer_bwd_data(ctx, gp, ip, ard.ARD_BF16, T * B, I, 4 * H, 1.0, ly.DZ, 4 * H, 1, self.Wk[l], I,
                                       None, 0, self.dYc[l - 1], I)
                ard.ard_layer_bwd_weight(ctx, gp, ip, ard.ARD_BF16, ard.ARD_F32, T * B, I, 4 * H, alphas[l - 1], self.Yc[l - 1], I,
                                         ly.DZ, 4 * H, 1, self.dWk[l], I, 0)
                ard.ard_expand_weight_grad_cols(ctx, gp, ip, ard.ARD_F32, I, 4 * H, self.dWk[l], I, ly.dW, KH, 1)
                dYc = self.dYc[l - 1]
        return self.layers[0].D[:, :, :self.dims[0]], [ly.dW for ly in self.layers]
