"""One more independent pin of the oracle's derivative formulas: reverse-mode autodiff (torch, fp64, CPU) of the
plainly written forward recurrence must equal the oracle's hand-written backpropagation."""
import numpy as np
import torch

from oracle import ssm_oracle as O


def test_bptt_equals_autograd():
    rng = np.random.default_rng(21)
    P, N, T = 5, 4, 12
    th = dict(W_delta=rng.normal(size=(P, P)) / np.sqrt(P), b_delta=rng.uniform(-1, 1, P),
              W_B=rng.normal(size=(N, P)) / np.sqrt(P), W_C=rng.normal(size=(N, P)) / np.sqrt(P),
              A_log=rng.uniform(0, np.log(16), (P, N)))
    x = rng.normal(size=(T, P)); g = rng.normal(size=(T, P))
    tt = {k: torch.tensor(v, dtype=torch.float64, requires_grad=True) for k, v in th.items()}
    xt = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    A = -torch.exp(tt["A_log"])
    h = torch.zeros(P, N, dtype=torch.float64)
    loss = 0.0
    for t in range(T):
        delta = torch.nn.functional.softplus(tt["W_delta"] @ xt[t] + tt["b_delta"])
        Bt = tt["W_B"] @ xt[t]; Ct = tt["W_C"] @ xt[t]
        h = torch.exp(delta[:, None] * A) * h + (delta * xt[t])[:, None] * Bt[None, :]
        loss = loss + (torch.tensor(g[t]) * (h @ Ct)).sum()
    loss.backward()
    ref = O.bptt_grad(th, x, g)
    for name, key in (("W_delta", "dW_delta"), ("b_delta", "db_delta"), ("W_B", "dW_B"), ("W_C", "dW_C"), ("A_log", "dA_log")):
        assert np.abs(tt[name].grad.numpy() - ref[key]).max() < 1e-11, name
    assert np.abs(xt.grad.numpy() - ref["dx"]).max() < 1e-11
    assert np.abs(O.adjoint_grad(th, x, g, T)["dx"] - xt.grad.numpy()).max() < 1e-11
