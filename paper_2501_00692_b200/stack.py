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
                 eps=1e-6):
        self.thetas = [dict(t) for t in thetas]   # own dicts: a packed copy of the weights is added below
        self.K = len(thetas)
        self.eps = eps
        self.device = device
        io = B.AS_F32 if dtype == torch.float32 else B.AS_BF16
        self.shape = B.make_shape(batch, seqlen, d_model, d_state, io)
        self.tbar = seqlen if tbar is None else tbar
        _, gbytes = B.as_workspace_bytes(self.shape, self.tbar)
        self.ws = B.alloc_workspace(gbytes, device)
        self.ys = None       # y_0 .. y_K
        self.yhat = torch.empty(batch, seqlen, d_model, dtype=dtype, device=device)
        self.ytilde = torch.empty_like(self.yhat)
        # the bf16 tensor-core contractions read [W_delta; W_B; W_C] as one matrix: packed once here, per layer
        if io == B.AS_BF16 and d_model % 32 == 0:
            for th in self.thetas:
                if th.get("Wcat") is None:
                    th["Wcat"] = torch.empty(B.as_wcat_bytes(self.shape), dtype=torch.uint8, device=device)
                    B.as_pack_weights(self.shape, 1, th, th["Wcat"])
        self._stacked = None   # parameters with a leading [K] dimension, built on first use of the batched call
        self._ws_layers = None

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

    def adjoint_grad(self, g: torch.Tensor, mode: str = "chained", record=None, batched=True):
        """Per-layer parameter gradients from the top gradient g = dL/dy_K.  Returns (list of grads, G_0 or None).
        `record`, if a dict, receives {k: (layer input, upstream gradient)} copies for the layers it has keys for.
        In "paper" mode the layers are independent and go to the library as one call (`batched=False`: layer by layer)."""
        assert self.ys is not None, "call forward() first"
        dev = g.device
        if mode == "paper" and batched:
            return self._paper_grad_batched(g, record), None
        grads = [None] * self.K
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

    def _paper_grad_batched(self, g: torch.Tensor, record=None):
        """Proposition 3: all K layers in one as_adjoint_grad_layers call (stacked parameters, stacked layer inputs,
        the one upstream gradient shared)."""
        K, sh = self.K, self.shape
        if self._stacked is None:
            keys = ["W_delta", "b_delta", "W_B", "W_C", "A_log"] + (["Wcat"] if self.thetas[0].get("Wcat") is not None else [])
            self._stacked = {k: torch.stack([th[k] for th in self.thetas]).contiguous() for k in keys}
            self._ws_layers = B.alloc_workspace(B.as_workspace_bytes_layers(sh, K, self.tbar), self.device)
            self._xall = torch.empty(K, sh.batch, sh.seqlen, sh.d_model, dtype=self.yhat.dtype, device=self.device)
        for k in range(K):
            B.as_rmsnorm_fwd(sh, self.ys[k], self._xall[k], self.eps)
            if record is not None and k in record:
                record[k] = (self._xall[k].clone(), g.clone())
        gl = B.alloc_grads_layers(sh, K, g.device)
        B.as_adjoint_grad_layers(sh, K, self._stacked, self._xall, g, self.tbar, gl, self._ws_layers)
        self.ws_last = self._ws_layers
        return [{k: (v[i] if v is not None else None) for k, v in gl.items()} for i in range(K)]
