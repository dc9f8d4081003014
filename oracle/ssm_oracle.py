"""fp64 CPU oracle for adjoint-method gradients of a diagonal selective SSM layer.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what the
CUDA library must compute.  Only the tests, the smoke check and the CPU-baseline
leg of the benchmark may import it; the product path never does.  It shares no
code with the CUDA sources.

Model (Section 3.1 "State-space models", the five steps of SSM(.), specialised to
a diagonal selective SSM as in Section 4.5 "Parallel computing"; per sequence):

    u_t   = W_delta x_t + b_delta,   Delta_t = softplus(u_t)              [P]
    B_t   = W_B x_t,                 C_t     = W_C x_t                    [N]
    A     = -exp(A_log)                                                   [P,N]
    abar_t[p,n] = exp(Delta_t[p] A[p,n]),  bbar_t[p,n] = Delta_t[p] B_t[n] x_t[p]
    h_t   = abar_t * h_{t-1} + bbar_t,     h_0 = 0                         [P,N]
    y_t[p] = sum_n C_t[n] h_t[p,n]

This is the paper's h^t = A^t h^{t-1} + B^t x^t, y^t = C^t h^t with state dimension
P*N, A^t = diag(abar_t), and the nets A(.), B(.), C(.) being single linear maps
(softplus on Delta only).

Gradients (Proposition 2, Eq. 7 "truncated adjoint sharding", Algorithms 2-4), with
g_t = dl^t/dy^t given:

    (v lambda^{t,i})[p,n] = g_t[p] C_t[n] prod_{j=i+1..t} abar_j[p,n]
    token t reaches source tokens i in [max(1, t+1-Tbar), t]   (Eq. 7, Alg. 2/3 index ranges)
    the C-net term is summed over every t (first line of Eq. 7), never windowed.

All arrays are float64 numpy.  Time indices in code are 0-based: token t of the
paper is index t-1; H[t] below holds h_t with H[0] = h_0 = 0.

Pins (tests/test_oracle_pins.py): adjoint == hand BPTT; truncated == full for
Tbar >= T; central finite differences; VJP counts incl. the printed 64 % figure;
impulse window edges; windowed-BPTT brute force; Tbar = 1 closed form; LTI
geometric closed forms; explicit O(T^2) forward sum; the C-VJP identity of
Appendix A.3; linearity / permutation invariants; stack modes vs finite differences;
scalar structure: masked T x T product form of the forward, finite differences of the tied rate.
Unpinned by anything printed in the paper: absolute gradient values on the named
workloads (the paper prints none), the RMSNorm epsilon, the error metric.
"""
from __future__ import annotations

import numpy as np

RMS_EPS = 1e-6


# --------------------------------------------------------------------------- nets
def softplus(u):
    return np.maximum(u, 0.0) + np.log1p(np.exp(-np.abs(u)))


def sigmoid(u):
    return np.where(u >= 0, 1.0 / (1.0 + np.exp(-np.abs(u))), np.exp(-np.abs(u)) / (1.0 + np.exp(-np.abs(u))))


def nets(theta, x):
    """Steps 1-3 of SSM(.): the input-dependent Delta_t, B_t, C_t (and the constant A)."""
    u = x @ theta["W_delta"].T + theta["b_delta"]
    delta = softplus(u)
    Bm = x @ theta["W_B"].T
    Cm = x @ theta["W_C"].T
    A = -np.exp(theta["A_log"])
    return u, delta, Bm, Cm, A


# --------------------------------------------------------------------------- scans
def scan_forward(delta, xs, Bm, Cm, A):
    """Steps 4-5 of SSM(.) for the channels present in `delta`/`xs`/`A`.

    delta, xs: [T,Pc]; Bm, Cm: [T,N]; A: [Pc,N].  Returns y [T,Pc], H [T+1,Pc,N], abar [T,Pc,N].
    """
    T, Pc = delta.shape
    N = A.shape[1]
    H = np.zeros((T + 1, Pc, N))
    abar = np.empty((T, Pc, N))
    y = np.empty((T, Pc))
    for t in range(T):
        abar[t] = np.exp(delta[t][:, None] * A)
        bbar = (delta[t] * xs[t])[:, None] * Bm[t][None, :]
        H[t + 1] = abar[t] * H[t] + bbar
        y[t] = H[t + 1] @ Cm[t]
    return y, H, abar


def mu_direct(abar, g, Cm, tbar):
    """Summed adjoint cotangent mu_i = sum over the tokens t whose window contains i of
    g_t (x) lambda^{t,i}, by the definition: for every t walk back over its window
    multiplying by abar one step at a time (Alg. 2's running products, applied to v*C)."""
    T, Pc, N = abar.shape
    mu = np.zeros((T, Pc, N))
    for t in range(T):
        lam = g[t][:, None] * Cm[t][None, :]
        for i in range(t, max(0, t - tbar + 1) - 1, -1):
            mu[i] += lam
            lam = lam * abar[i]
    return mu


def mu_block(abar, g, Cm, tbar):
    """Same mu as `mu_direct` in O(T): cut time into blocks of length Tbar; for i in block
    [s,e): mu_i = R_i + D_i * Q_{i+Tbar-1}, with R the reverse recurrence restarted at the
    block end, D_i = prod_{j=i+1..e-1} abar_j, and Q_m = sum_{t=e..m} gC_t prod_{j=e..t} abar_j
    a forward prefix inside the next block.  No subtraction, all factors <= 1."""
    T, Pc, N = abar.shape
    mu = np.zeros((T, Pc, N))
    gC = lambda t: g[t][:, None] * Cm[t][None, :]
    L = min(tbar, T)
    for s in range(0, T, L):
        e = min(s + L, T)
        e2 = min(e + L, T)
        Q = np.zeros((L + 1, Pc, N))  # Q[k] = prefix over tokens e..e+k-1 ; Q[0] = 0
        pref = np.ones((Pc, N))
        for k, t in enumerate(range(e, e2)):
            pref = pref * abar[t]
            Q[k + 1] = Q[k] + gC(t) * pref
        for k in range(e2 - e + 1, L + 1):
            Q[k] = Q[e2 - e]
        R = np.zeros((Pc, N))
        D = np.ones((Pc, N))
        for i in range(e - 1, s - 1, -1):
            if i < e - 1:
                R = R * abar[i + 1]
                D = D * abar[i + 1]
            R = R + gC(i)
            nxt = i + tbar - 1 - (e - 1)  # number of next-block tokens inside window(i)
            mu[i] = R + D * Q[max(0, min(nxt, L))]
    return mu


def token_cotangents(mu, H, abar, g, delta, xs, u, Bm, A):
    """Algorithm 3 for every source token i at once: from mu_i, h_{i-1}, h_i form the three
    cotangents (v lambda (x) h^{i-1} for the A-net, v lambda for the B-net, g (x) h^t for the
    C-net) and pull them back to Delta_i, B_i, C_i, x_i (direct path) and A_log."""
    dabar = mu * H[:-1]                                   # cotangent of abar_i
    dC = np.einsum("tp,tpn->tn", g, H[1:])                # not windowed
    s = np.einsum("tpn,tn->tp", mu, Bm)
    ddelta = np.einsum("tpn,pn->tp", dabar * abar, A) + xs * s
    dB = np.einsum("tpn,tp->tn", mu, delta * xs)
    du = ddelta * sigmoid(u)
    dA_log = np.einsum("tpn,tp->pn", dabar * abar, delta) * A
    dx_dir = delta * s
    return {"du": du, "dB": dB, "dC": dC, "dx_dir": dx_dir, "dA_log": dA_log, "ddelta": ddelta}


# --------------------------------------------------------------------------- one layer, one sequence
def ssm_forward(theta, x):
    """SSM(X) = Y for one sequence x [T,P]."""
    u, delta, Bm, Cm, A = nets(theta, x)
    y, _, _ = scan_forward(delta, x, Bm, Cm, A)
    return y


def _assemble(theta, x, du, dB, dC, dx_dir, dA_log):
    """The net-VJPs of Alg. 3 (linear nets): weight gradients and the input gradient."""
    return {
        "dW_delta": du.T @ x,
        "db_delta": du.sum(axis=0),
        "dW_B": dB.T @ x,
        "dW_C": dC.T @ x,
        "dA_log": dA_log,
        "dx": dx_dir + du @ theta["W_delta"] + dB @ theta["W_B"] + dC @ theta["W_C"],
        "du": du, "dB": dB, "dC": dC, "dx_dir": dx_dir,
    }


def adjoint_grad(theta, x, g, tbar, tier="direct", channel_block=None):
    """Adjoint-method gradient (Prop. 2; Eq. 7 when tbar < T) for one sequence.

    tier "direct" forms mu by the defining double sum, "block" by the O(T) block form.
    `channel_block` only bounds memory: channels are independent in the scan, and the two
    sums over channels (dB_i, dC_i) are added block by block.
    """
    T, P = x.shape
    if tbar < 1:
        raise ValueError("tbar must be >= 1")
    u, delta, Bm, Cm, A = nets(theta, x)
    N = A.shape[1]
    cb = P if channel_block is None else channel_block
    du = np.empty((T, P)); dx_dir = np.empty((T, P)); y = np.empty((T, P))
    dB = np.zeros((T, N)); dC = np.zeros((T, N)); dA_log = np.empty((P, N))
    for p0 in range(0, P, cb):
        sl = slice(p0, min(P, p0 + cb))
        yb, H, abar = scan_forward(delta[:, sl], x[:, sl], Bm, Cm, A[sl])
        mu = (mu_direct if tier == "direct" else mu_block)(abar, g[:, sl], Cm, tbar)
        tok = token_cotangents(mu, H, abar, g[:, sl], delta[:, sl], x[:, sl], u[:, sl], Bm, A[sl])
        du[:, sl] = tok["du"]; dx_dir[:, sl] = tok["dx_dir"]; y[:, sl] = yb
        dB += tok["dB"]; dC += tok["dC"]; dA_log[sl] = tok["dA_log"]
    out = _assemble(theta, x, du, dB, dC, dx_dir, dA_log)
    out["y"] = y
    return out


def adjoint_grad_literal(theta, x, g, tbar):
    """Algorithm 4 as printed, one sequence: for every token t call Alg. 3 (which calls Alg. 2),
    and add each individual (t,i) vector-Jacobian product straight into the gradient.  No summed
    cotangent is ever formed.  O(T*Tbar*P*(N+P)); tiny shapes only."""
    T, P = x.shape
    u, delta, Bm, Cm, A = nets(theta, x)
    N = A.shape[1]
    _, H, abar = scan_forward(delta, x, Bm, Cm, A)
    sig = sigmoid(u)
    W_delta, W_B, W_C = theta["W_delta"], theta["W_B"], theta["W_C"]
    out = {k: np.zeros_like(theta[k]) for k in ("W_delta", "b_delta", "W_B", "W_C", "A_log")}
    dx = np.zeros((T, P))
    for t in range(T):
        i_lo = max(0, t + 1 - tbar)
        # Alg. 2: zeta = (A^t ... A^{i_lo+1}, ..., A^t, I); lambda^{t,i} = C^t zeta
        zeta = [None] * (t - i_lo + 1)
        run = np.ones((P, N))
        for k, i in enumerate(range(t, i_lo - 1, -1)):
            zeta[t - i] = run.copy()          # product of abar_j for j = i+1..t
            run = run * abar[i]
        # Alg. 3: C-net VJP at token t
        cotC = g[t] @ H[t + 1]                                # [N]
        out["W_C"] += np.outer(cotC, x[t])
        dx[t] += W_C.T @ cotC
        for i in range(i_lo, t + 1):
            vlam = g[t][:, None] * Cm[t][None, :] * zeta[t - i]   # [P,N]
            cotA = vlam * H[i]                                # v lambda (x) h^{i-1}  (diagonal A)
            cotB = vlam                                       # cotangent of bbar_i = B^i x^i
            ddelta = (cotA * abar[i] * A).sum(axis=1) + (cotB * Bm[i][None, :]).sum(axis=1) * x[i]
            out["A_log"] += cotA * abar[i] * delta[i][:, None] * A
            dBi = (cotB * (delta[i] * x[i])[:, None]).sum(axis=0)
            dx[i] += delta[i] * (cotB * Bm[i][None, :]).sum(axis=1)
            dui = ddelta * sig[i]
            out["W_delta"] += np.outer(dui, x[i])
            out["b_delta"] += dui
            out["W_B"] += np.outer(dBi, x[i])
            dx[i] += W_delta.T @ dui + W_B.T @ dBi
    return {"dW_delta": out["W_delta"], "db_delta": out["b_delta"], "dW_B": out["W_B"],
            "dW_C": out["W_C"], "dA_log": out["A_log"], "dx": dx}


def bptt_grad(theta, x, g):
    """Backpropagation through time by hand (the nested expansion the adjoint method replaces,
    Section 3.3): one reverse sweep carrying dL/dh_t."""
    T, P = x.shape
    u, delta, Bm, Cm, A = nets(theta, x)
    N = A.shape[1]
    _, H, abar = scan_forward(delta, x, Bm, Cm, A)
    dh = np.zeros((P, N))
    du = np.zeros((T, P)); dB = np.zeros((T, N)); dC = np.zeros((T, N)); dx_dir = np.zeros((T, P))
    dA_log = np.zeros((P, N))
    sig = sigmoid(u)
    for t in range(T - 1, -1, -1):
        dh = dh + np.outer(g[t], Cm[t])                 # y_t = C_t h_t
        dC[t] = g[t] @ H[t + 1]
        d_abar = dh * H[t]                              # h_t = abar_t h_{t-1} + bbar_t
        d_bbar = dh
        d_e = d_abar * abar[t]                          # abar = exp(e), e = delta * A
        d_delta = (d_e * A).sum(axis=1)
        dA_log += d_e * delta[t][:, None] * A           # dA/dA_log = A
        d_delta += (d_bbar * Bm[t][None, :]).sum(axis=1) * x[t]      # bbar = delta B x
        dB[t] = (d_bbar * (delta[t] * x[t])[:, None]).sum(axis=0)
        dx_dir[t] = (d_bbar * Bm[t][None, :]).sum(axis=1) * delta[t]
        du[t] = d_delta * sig[t]
        dh = abar[t] * dh
    return _assemble(theta, x, du, dB, dC, dx_dir, dA_log)


def windowed_bptt_bruteforce(theta, x, g, tbar):
    """Truncation stated independently: for each t, backpropagate l^t alone through the state
    transitions t, t-1, ..., t-Tbar+1 and stop, treating h_{t-Tbar} as a constant of the forward
    pass ("only perform the VJPs back to the last Tbar states").  Sum over t."""
    T, P = x.shape
    u, delta, Bm, Cm, A = nets(theta, x)
    N = A.shape[1]
    _, H, abar = scan_forward(delta, x, Bm, Cm, A)
    du = np.zeros((T, P)); dB = np.zeros((T, N)); dC = np.zeros((T, N)); dx_dir = np.zeros((T, P))
    dA_log = np.zeros((P, N))
    sig = sigmoid(u)
    for t in range(T):
        dh = np.outer(g[t], Cm[t])
        dC[t] += g[t] @ H[t + 1]
        for i in range(t, max(-1, t - tbar), -1):
            d_e = dh * H[i] * abar[i]
            d_delta = (d_e * A).sum(axis=1) + (dh * Bm[i][None, :]).sum(axis=1) * x[i]
            dA_log += d_e * delta[i][:, None] * A
            dB[i] += (dh * (delta[i] * x[i])[:, None]).sum(axis=0)
            dx_dir[i] += (dh * Bm[i][None, :]).sum(axis=1) * delta[i]
            du[i] += d_delta * sig[i]
            dh = abar[i] * dh
    return _assemble(theta, x, du, dB, dC, dx_dir, dA_log)


# --------------------------------------------------------------------------- batches
PARAM_GRADS = ("dW_delta", "db_delta", "dW_B", "dW_C", "dA_log")


# ---------------------------------------------------------------------------------------------
# scalar structure (the "Scalar SSM" row of Table 1, Section 4.5): one decay rate per channel,
# A[p, n] = a[p] for every state n, so that A^t is a scalar multiple of the identity on each
# channel's N states.  It is the diagonal layer with the N entries of a row of A_log tied together:
# the forward is unchanged, and the gradient of a tied parameter is the sum of the gradients of
# the entries it is tied to (chain rule).
# ---------------------------------------------------------------------------------------------
def untie_scalar_A(theta, N):
    """theta with A_log [P] -> the equivalent diagonal theta with A_log [P,N] (rows constant)."""
    th = dict(theta)
    a = np.asarray(theta["A_log"], dtype=np.float64)
    assert a.ndim == 1
    th["A_log"] = np.repeat(a[:, None], N, axis=1)
    return th


def scalar_adjoint_grad(theta, x, g, tbar, N, **kw):
    """Adjoint-method gradient of the scalar-structure layer for one sequence: dA_log is [P]."""
    out = adjoint_grad(untie_scalar_A(theta, N), x, g, tbar, **kw)
    out["dA_log"] = out["dA_log"].sum(axis=1)
    return out


def scalar_forward_quadratic(theta, x, N):
    """Forward of the scalar-structure layer written as one masked T x T product per channel (no recurrence):
        y_t[p] = sum_{j<=t} exp(a_p * sum_{i=j+1..t} Delta_i[p]) * (C_t . B_j) * Delta_j[p] x_j[p]
    Used only to pin the recurrent forward; O(T^2 P)."""
    a = -np.exp(np.asarray(theta["A_log"], dtype=np.float64))          # [P]
    _, delta, Bm, Cm, _ = nets(untie_scalar_A(theta, N), x)
    T, P = x.shape
    G = Cm @ Bm.T                                                      # [T,T]  C_t . B_j
    cum = np.cumsum(delta, axis=0)                                     # [T,P]
    y = np.zeros((T, P))
    for p in range(P):
        L = np.exp(a[p] * (cum[:, None, p] - cum[None, :, p]))         # exp(a * sum_{i=j+1..t} Delta_i)
        L = np.tril(L)
        y[:, p] = (L * G) @ (delta[:, p] * x[:, p])
    return y


def batched(fn, theta, x, g, *args, **kw):
    """Apply a one-sequence gradient routine to x, g [B,T,P]: parameter gradients are summed
    over the batch (Table 1's "bs"), per-token outputs are stacked."""
    outs = [fn(theta, x[b], g[b], *args, **kw) for b in range(x.shape[0])]
    res = {}
    for k in outs[0]:
        if k in PARAM_GRADS:
            res[k] = sum(o[k] for o in outs)
        else:
            res[k] = np.stack([o[k] for o in outs])
    return res


# --------------------------------------------------------------------------- residual stack
def rmsnorm(y, eps=RMS_EPS):
    """Gain-free RMSNorm over the model dimension (the "Norm" of Section 3.2)."""
    return y / np.sqrt(np.mean(y * y, axis=-1, keepdims=True) + eps)


def rmsnorm_vjp(y, d, eps=RMS_EPS):
    r = np.sqrt(np.mean(y * y, axis=-1, keepdims=True) + eps)
    yh = y / r
    return (d - yh * np.mean(d * yh, axis=-1, keepdims=True)) / r


def stack_forward(thetas, y0, store=None):
    """Section 3.2 / Alg. 1 lines 5-7 on one sequence: y_k = y_{k-1} + SSM_k(Norm(y_{k-1})).

    `store`, if given, models the storage format of the activations: it is applied to every tensor
    the stack keeps or hands from one layer to the next (the normalised input, the layer output,
    the residual sum).  The default keeps everything in float64.  It changes no formula."""
    keep = (lambda a: a) if store is None else store
    ys = [y0]
    yhats = []
    for th in thetas:
        yhats.append(keep(rmsnorm(ys[-1])))
        ys.append(keep(ys[-1] + keep(ssm_forward(th, yhats[-1]))))
    return ys, yhats


def stack_grad(thetas, y0, g, tbar, mode="chained", tier="direct", store=None):
    """Gradients of every layer of the residual stack from one upstream g = dL/dy_K.

    mode "paper": Proposition 3 as printed - every layer receives g itself and its input
    Norm(y_{k-1}) is a constant.  mode "chained": true backpropagation through the stack,
    G_K = g, G_{k-1} = G_k + RMSNormVJP(y_{k-1}, dx_k), layer k driven by G_k.
    `store` as in `stack_forward`; in the backward it is applied to the input gradient dx_k a layer
    hands down and to the running upstream gradient G_k."""
    keep = (lambda a: a) if store is None else store
    ys, yhats = stack_forward(thetas, y0, store)
    K = len(thetas)
    grads = [None] * K
    G = g
    for k in range(K - 1, -1, -1):
        grads[k] = adjoint_grad(thetas[k], yhats[k], G if mode == "chained" else g, tbar, tier=tier)
        if mode == "chained":
            G = keep(G + rmsnorm_vjp(ys[k], keep(grads[k]["dx"])))
    return grads, (G if mode == "chained" else None)


# --------------------------------------------------------------------------- bookkeeping
def vjp_count(T, tbar=None):
    """Number of A-net (equally B-net) VJPs per layer: token t performs one per source token in
    its window (Section 4.3): t of them in the full form, min(t, Tbar) when truncated."""
    tbar = T if tbar is None else tbar
    return sum(min(t, tbar) for t in range(1, T + 1))
