"""Residual stack of K selective-SSM layers (Section 3.2; Algorithms 1 and 4 on one device):
y_k = y_{k-1} + SSM_k(Norm(y_{k-1})).  This module only sequences calls of the C-ABI library - every
tensor operation (RMSNorm, the layer forward, the residual add, the adjoint gradients, the RMSNorm VJP)
runs in the library's kernels; torch supplies device buffers.

Two gradient modes:
  "paper"   - Proposition 3 as printed: every layer receives the top gradient dL/dy_K itself and treats its
              input Norm(y_{k-1}) as a constant, so all layers are independent given the stored activations.
  "chained" - backpropagation through the whole stack: G_K = dL/dy_K, and going down
              G_{k-1} = G_k + RMSNormVJP(y_{k-1}, dx_k) with layer k driven by G_k.
"""
from __future__ import annotations

import torch

from . import binding as B


class Stack:
    def __init__(self, thetas, batch, seqlen, d_model, d_state=16, dtype=torch.float32, device="cuda:0", tbar=None,
                 eps=1e-6, paper_streams=1):
        self.thetas = thetas
        self.K = len(thetas)
        self.eps = eps
        io = B.AS_F32 if dtype == torch.float32 else B.AS_BF16
        self.shape = B.make_shape(batch, seqlen, d_model, d_state, io)
        self.tbar = seqlen if tbar is None else tbar
        _, gbytes = B.as_workspace_bytes(self.shape, self.tbar)
        self.ws = B.alloc_workspace(gbytes, device)
        self.ys = None       # y_0 .. y_K
        self.yhat = torch.empty(batch, seqlen, d_model, dtype=dtype, device=device)
        self.ytilde = torch.empty_like(self.yhat)
        # "paper" mode only: the layers are independent, so they may run on several streams at once (the layer
        # dimension of Section 4.2); every extra stream owns a workspace and a normalised-input buffer
        self.extra = [(torch.cuda.Stream(device=device), B.alloc_workspace(gbytes, device), torch.empty_like(self.yhat))
                      for _ in range(max(0, paper_streams - 1))]

    def forward(self, y0: torch.Tensor):
        """Runs the stack, keeping y_0..y_K (the per-layer inputs are re-normalised in the backward)."""
        self.ys = [y0]
        for th in self.thetas:
            B.as_rmsnorm_fwd(self.shape, self.ys[-1], self.yhat, self.eps)
            B.as_ssm_forward(self.shape, th, self.yhat, self.ytilde, self.ws)
            yk = torch.empty_like(y0)
            B.as_residual_add(self.shape, self.ys[-1], self.ytilde, yk)
            self.ys.append(yk)
        return self.ys[-1]

    def adjoint_grad(self, g: torch.Tensor, mode: str = "chained", record=None):
        """Per-layer parameter gradients from the top gradient g = dL/dy_K.  Returns (list of grads, G_0 or None).
        `record`, if a dict, receives {k: (layer input, upstream gradient)} copies for the layers it has keys for."""
        assert self.ys is not None, "call forward() first"
        dev = g.device
        grads = [None] * self.K
        if mode == "paper" and self.extra and record is None:
            return self._paper_grad_concurrent(g), None
        G = g.clone() if mode == "chained" else g
        for k in range(self.K - 1, -1, -1):
            B.as_rmsnorm_fwd(self.shape, self.ys[k], self.yhat, self.eps)
            if record is not None and k in record:
                record[k] = (self.yhat.clone(), G.clone())
            gk = B.alloc_grads(self.shape, dev, with_dx=(mode == "chained"))
            B.as_adjoint_grad(self.shape, self.thetas[k], self.yhat, G, self.tbar, gk, self.ws)
            if mode == "chained":
                B.as_rmsnorm_bwd_add(self.shape, self.ys[k], gk["dx"], G, self.eps)
                gk["dx"] = None
            grads[k] = gk
        return grads, (G if mode == "chained" else None)

    def _paper_grad_concurrent(self, g: torch.Tensor):
        """Proposition 3 with the layers spread round-robin over the stack's streams."""
        main = torch.cuda.current_stream()
        lanes = [(main, self.ws, self.yhat)] + self.extra
        for st, _, _ in self.extra:
            st.wait_stream(main)
        grads = [None] * self.K
        for k in range(self.K - 1, -1, -1):
            st, ws, yhat = lanes[k % len(lanes)]
            gk = B.alloc_grads(self.shape, g.device, with_dx=False)   # allocated on the main stream, which joins below
            with torch.cuda.stream(st):
                B.as_rmsnorm_fwd(self.shape, self.ys[k], yhat, self.eps)
                B.as_adjoint_grad(self.shape, self.thetas[k], yhat, g, self.tbar, gk, ws)
            grads[k] = gk
        for st, _, _ in self.extra:
            main.wait_stream(st)
        return grads
