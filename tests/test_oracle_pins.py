"""Pins of the fp64 oracle against what the paper and the mathematics fix (CPU only)."""
import os

import numpy as np
import pytest

from oracle import ssm_oracle as O

GRADS = O.PARAM_GRADS + ("dx",)


def make_theta(rng, P, N, b_lo=-4.0, b_hi=-2.0):
    return dict(W_delta=rng.normal(size=(P, P)) / np.sqrt(P), b_delta=rng.uniform(b_lo, b_hi, P),
                W_B=rng.normal(size=(N, P)) / np.sqrt(P), W_C=rng.normal(size=(N, P)) / np.sqrt(P),
                A_log=rng.uniform(0, np.log(16), (P, N)))


def maxdiff(a, b, keys=GRADS):
    return max(np.abs(a[k] - b[k]).max() / (np.abs(b[k]).max() + 1e-300) for k in keys)


@pytest.fixture
def tiny():
    rng = np.random.default_rng(7)
    P, N, T = 6, 4, 16
    th = make_theta(rng, P, N, -1.0, 1.0)   # larger Delta: every term is exercised
    return th, rng.normal(size=(T, P)), rng.normal(size=(T, P))


def loss(theta, x, g):
    return float(np.sum(g * O.ssm_forward(theta, x)))


# P9: the recurrence equals the explicit O(T^2) sum y_t = sum_{s<=t} C_t prod_{j=s+1..t} abar_j bbar_s
def test_forward_equals_explicit_sum(tiny):
    th, x, _ = tiny
    T, P = x.shape
    A = -np.exp(th["A_log"])
    u = x @ th["W_delta"].T + th["b_delta"]
    delta = np.log1p(np.exp(u))
    y = np.zeros((T, P))
    for t in range(T):
        Ct = th["W_C"] @ x[t]
        for s in range(t + 1):
            decay = np.exp(A * delta[s + 1:t + 1].sum(axis=0)[:, None])
            bbar = (delta[s] * x[s])[:, None] * (th["W_B"] @ x[s])[None, :]
            y[t] += (decay * bbar) @ Ct
    assert np.abs(y - O.ssm_forward(th, x)).max() < 1e-12


# P1: adjoint gradients equal backprop gradients (abstract; Prop. 2)
def test_adjoint_equals_bptt(tiny):
    th, x, g = tiny
    b = O.bptt_grad(th, x, g)
    for fn in (lambda: O.adjoint_grad(th, x, g, x.shape[0]),
               lambda: O.adjoint_grad(th, x, g, x.shape[0], tier="block"),
               lambda: O.adjoint_grad_literal(th, x, g, x.shape[0])):
        assert maxdiff(fn(), b) < 1e-12


# P2: truncated == full once the window covers the sequence (Eq. 7: second sums are empty)
def test_truncated_equals_full_when_window_covers(tiny):
    th, x, g = tiny
    T = x.shape[0]
    full = O.adjoint_grad(th, x, g, T)
    for tb in (T, T + 5, 10 * T):
        for tier in ("direct", "block"):
            assert maxdiff(O.adjoint_grad(th, x, g, tb, tier=tier), full) < 1e-13
    assert maxdiff(O.adjoint_grad(th, x, g, T // 2), full) > 1e-6   # a shorter window is not full


# P3: central finite differences of L = sum <g_t, y_t> for every parameter entry and x
def test_finite_differences(tiny):
    th, x, g = tiny
    a = O.bptt_grad(th, x, g)
    eps = 1e-6
    for name, key in (("W_delta", "dW_delta"), ("b_delta", "db_delta"), ("W_B", "dW_B"),
                      ("W_C", "dW_C"), ("A_log", "dA_log")):
        fd = np.zeros_like(th[name])
        it = np.nditer(th[name], flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            tp = {k: v.copy() for k, v in th.items()}
            tm = {k: v.copy() for k, v in th.items()}
            tp[name][idx] += eps
            tm[name][idx] -= eps
            fd[idx] = (loss(tp, x, g) - loss(tm, x, g)) / (2 * eps)
        assert np.abs(fd - a[key]).max() / np.abs(a[key]).max() < 1e-7, name
    fd = np.zeros_like(x)
    for idx in np.ndindex(*x.shape):
        xp = x.copy(); xm = x.copy()
        xp[idx] += eps; xm[idx] -= eps
        fd[idx] = (loss(th, xp, g) - loss(th, xm, g)) / (2 * eps)
    assert np.abs(fd - a["dx"]).max() / np.abs(a["dx"]).max() < 1e-7


# P4: VJP counts (Section 4.3) incl. the printed 64 % reduction
def test_vjp_counts_golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "vjp_counts.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    for T, tb, cnt in rows:
        T, tb, cnt = int(T), int(tb), int(cnt)
        assert O.vjp_count(T, tb or None) == cnt
    assert O.vjp_count(10000) == (1 + 10000) * 10000 // 2
    red = 1 - O.vjp_count(10000, 2000) / O.vjp_count(10000)
    assert round(100 * red) == 64
    for T, tb in ((12, 5), (40, 40), (9, 1)):
        assert O.vjp_count(T, tb) == tb * T - tb * (tb - 1) // 2


# P5: impulse upstream gradient: window edges are exact (Eq. 7; Alg. 2/3 index ranges)
@pytest.mark.parametrize("tier", ["direct", "block", "literal"])
def test_impulse_window_edges(tiny, tier):
    th, x, _ = tiny
    T, P = x.shape
    tp, pp = 11, 2
    g = np.zeros((T, P)); g[tp, pp] = 1.0
    for tb in (1, 3, 4, 12, 13):
        if tier == "literal":
            # the literal routine exposes only final gradients: compare with the windowed brute force
            a = O.adjoint_grad_literal(th, x, g, tb)
            assert maxdiff(a, O.windowed_bptt_bruteforce(th, x, g, tb)) < 1e-12
            continue
        a = O.adjoint_grad(th, x, g, tb, tier=tier)
        lo = max(0, tp - tb + 1)
        for name in ("du", "dB", "dx_dir"):
            nz = np.abs(a[name]).max(axis=1) > 0
            want = np.zeros(T, bool); want[lo:tp + 1] = True
            assert (nz == want).all(), (name, tb)
        nzC = np.abs(a["dC"]).max(axis=1) > 0
        assert nzC.sum() == 1 and nzC[tp]
        # only channel pp is driven
        assert np.abs(np.delete(a["du"], pp, axis=1)).max() == 0


# P6: truncated adjoint == windowed-BPTT brute force (meaning of truncation, Section 4.3)
def test_truncated_equals_windowed_bptt(tiny):
    th, x, g = tiny
    for tb in (1, 2, 3, 5, 7, 11, 16):
        w = O.windowed_bptt_bruteforce(th, x, g, tb)
        for tier in ("direct", "block"):
            assert maxdiff(O.adjoint_grad(th, x, g, tb, tier=tier), w) < 1e-12
        assert maxdiff(O.adjoint_grad_literal(th, x, g, tb), w) < 1e-12


# P7: Tbar = 1 closed form: mu_i = g_i (x) C_i
def test_tbar_one_closed_form(tiny):
    th, x, g = tiny
    u, delta, Bm, Cm, A = O.nets(th, x)
    _, H, abar = O.scan_forward(delta, x, Bm, Cm, A)
    for fn in (O.mu_direct, O.mu_block):
        mu = fn(abar, g, Cm, 1)
        assert np.abs(mu - g[:, :, None] * Cm[:, None, :]).max() == 0
    a = O.adjoint_grad(th, x, g, 1)
    dB = np.einsum("tp,tn,tp->tn", g, Cm, delta * x)
    assert np.abs(a["dB"] - dB).max() < 1e-14


# P8: LTI special case (W_delta = 0, constant x): geometric closed forms for h_t and mu_i
def test_lti_closed_form():
    rng = np.random.default_rng(3)
    P, N, T = 3, 4, 40
    th = make_theta(rng, P, N)
    th["W_delta"][:] = 0
    x = np.tile(rng.normal(size=(1, P)), (T, 1))
    g = np.tile(rng.normal(size=(1, P)), (T, 1))
    u, delta, Bm, Cm, A = O.nets(th, x)
    _, H, abar = O.scan_forward(delta, x, Bm, Cm, A)
    a = abar[0]
    bbar = (delta[0] * x[0])[:, None] * Bm[0][None, :]
    for t in (1, 2, 17, T):
        assert np.abs(H[t] - bbar * (1 - a ** t) / (1 - a)).max() < 1e-13
    gC = g[0][:, None] * Cm[0][None, :]
    for tb in (1, 5, 13, T, 3 * T):
        for fn in (O.mu_direct, O.mu_block):
            mu = fn(abar, g, Cm, tb)
            for i in (0, 7, T - 6, T - 1):
                k = min(tb, T - i)
                assert np.abs(mu[i] - gC * (1 - a ** k) / (1 - a)).max() < 1e-13


# P10: the C-net VJP identity of Appendix A.3: (dl/dy) C_theta h = sum((dl/dy (x) h) o dC/dtheta)
def test_c_vjp_identity(tiny):
    th, x, g = tiny
    T, P = x.shape
    N = th["W_C"].shape[0]
    u, delta, Bm, Cm, A = O.nets(th, x)
    _, H, _ = O.scan_forward(delta, x, Bm, Cm, A)
    dWC = np.zeros_like(th["W_C"])
    for t in range(T):
        outer = g[t][:, None] * H[t + 1]                    # dl/dy (x) h : [P, N] (per-channel state)
        for n in range(N):
            for q in range(P):
                # C_t[n] = sum_q W_C[n,q] x_t[q]  =>  d y_t[p] / d W_C[n,q] = h_t[p,n] x_t[q]
                dWC[n, q] += outer[:, n].sum() * x[t, q]
    assert np.abs(dWC - O.adjoint_grad(th, x, g, T)["dW_C"]).max() < 1e-12


# P11: linearity in g; g = 0; channel permutation equivariance
def test_linearity_and_permutation(tiny):
    th, x, g = tiny
    T, P = x.shape
    rng = np.random.default_rng(11)
    g2 = rng.normal(size=g.shape)
    a1 = O.adjoint_grad(th, x, g, 5); a2 = O.adjoint_grad(th, x, g2, 5)
    a12 = O.adjoint_grad(th, x, 2 * g - 3 * g2, 5)
    for k in GRADS:
        assert np.abs(a12[k] - (2 * a1[k] - 3 * a2[k])).max() < 1e-12
    z = O.adjoint_grad(th, x, 0 * g, 5)
    assert all(np.abs(z[k]).max() == 0 for k in GRADS)
    perm = rng.permutation(P)
    thp = dict(W_delta=th["W_delta"][perm][:, perm], b_delta=th["b_delta"][perm],
               W_B=th["W_B"][:, perm], W_C=th["W_C"][:, perm], A_log=th["A_log"][perm])
    ap = O.adjoint_grad(thp, x[:, perm], g[:, perm], 5)
    assert np.abs(ap["dW_delta"] - a1["dW_delta"][perm][:, perm]).max() < 1e-12
    assert np.abs(ap["dA_log"] - a1["dA_log"][perm]).max() < 1e-12
    assert np.abs(ap["dx"] - a1["dx"][:, perm]).max() < 1e-12
    assert np.abs(ap["dW_B"] - a1["dW_B"][:, perm]).max() < 1e-12


# P13: block form == direct sum on shapes with several blocks and a ragged last block
def test_block_equals_direct_ragged():
    rng = np.random.default_rng(5)
    P, N, T = 5, 16, 61
    th = make_theta(rng, P, N, -6.0, -3.0)
    x = rng.normal(size=(T, P)); g = rng.normal(size=(T, P))
    for tb in (1, 2, 7, 8, 9, 16, 30, 31, 60, 61, 62, 100):
        d = O.adjoint_grad(th, x, g, tb)
        b = O.adjoint_grad(th, x, g, tb, tier="block")
        assert maxdiff(b, d, GRADS + ("du", "dB", "dC")) < 1e-12, tb
    cb = O.adjoint_grad(th, x, g, 9, tier="block", channel_block=2)
    assert maxdiff(cb, O.adjoint_grad(th, x, g, 9), GRADS + ("du", "dB", "dC", "y")) < 1e-12


def test_batched_sums_parameter_grads(tiny):
    th, x, g = tiny
    xb = np.stack([x, x[::-1].copy()]); gb = np.stack([g, 2 * g])
    r = O.batched(O.adjoint_grad, th, xb, gb, 4)
    r0 = O.adjoint_grad(th, xb[0], gb[0], 4); r1 = O.adjoint_grad(th, xb[1], gb[1], 4)
    assert np.abs(r["dW_B"] - (r0["dW_B"] + r1["dW_B"])).max() < 1e-13
    assert np.abs(r["dx"][1] - r1["dx"]).max() == 0


def test_tbar_below_one_is_an_error(tiny):
    th, x, g = tiny
    with pytest.raises(ValueError):
        O.adjoint_grad(th, x, g, 0)


# ------------------------------------------------------------------ stack (Section 3.2, Prop. 3)
def stack_loss(thetas, y0, g):
    ys, _ = O.stack_forward(thetas, y0)
    return float(np.sum(g * ys[-1]))


def test_rmsnorm_vjp_fd():
    rng = np.random.default_rng(2)
    y = rng.normal(size=(3, 7)); d = rng.normal(size=(3, 7))
    v = O.rmsnorm_vjp(y, d)
    eps = 1e-6
    fd = np.zeros_like(y)
    for idx in np.ndindex(*y.shape):
        yp = y.copy(); ym = y.copy(); yp[idx] += eps; ym[idx] -= eps
        fd[idx] = np.sum(d * (O.rmsnorm(yp) - O.rmsnorm(ym))) / (2 * eps)
    assert np.abs(fd - v).max() < 1e-8
    assert abs(np.mean(O.rmsnorm(y) ** 2, axis=-1) - 1).max() < 1e-5


def test_stack_chained_equals_fd_and_paper_mode_is_detached():
    rng = np.random.default_rng(9)
    P, N, T, K = 4, 3, 9, 3
    thetas = [make_theta(rng, P, N, -1.0, 1.0) for _ in range(K)]
    y0 = rng.normal(size=(T, P)); g = rng.normal(size=(T, P))
    grads, G0 = O.stack_grad(thetas, y0, g, T, mode="chained")
    eps = 1e-6
    for k in range(K):
        for name, key in (("W_delta", "dW_delta"), ("A_log", "dA_log"), ("W_C", "dW_C"), ("b_delta", "db_delta"),
                          ("W_B", "dW_B")):
            fd = np.zeros_like(thetas[k][name])
            for idx in np.ndindex(*fd.shape):
                tp = [{a: b.copy() for a, b in th.items()} for th in thetas]
                tm = [{a: b.copy() for a, b in th.items()} for th in thetas]
                tp[k][name][idx] += eps; tm[k][name][idx] -= eps
                fd[idx] = (stack_loss(tp, y0, g) - stack_loss(tm, y0, g)) / (2 * eps)
            assert np.abs(fd - grads[k][key]).max() / np.abs(fd).max() < 1e-6, (k, name)
    fd0 = np.zeros_like(y0)
    for idx in np.ndindex(*y0.shape):
        yp = y0.copy(); ym = y0.copy(); yp[idx] += eps; ym[idx] -= eps
        fd0[idx] = (stack_loss(thetas, yp, g) - stack_loss(thetas, ym, g)) / (2 * eps)
    assert np.abs(fd0 - G0).max() / np.abs(fd0).max() < 1e-6
    # paper mode (Prop. 3 as printed): each layer alone, input detached, driven by g itself;
    # equals finite differences of sum <g, SSM_k(const input)> and equals chained only for k = K
    pg, _ = O.stack_grad(thetas, y0, g, T, mode="paper")
    ys, yhats = O.stack_forward(thetas, y0)
    for k in range(K):
        ref = O.bptt_grad(thetas[k], yhats[k], g)
        assert maxdiff(pg[k], ref, O.PARAM_GRADS) < 1e-12
    assert maxdiff(pg[K - 1], grads[K - 1], O.PARAM_GRADS) < 1e-12
    assert maxdiff(pg[0], grads[0], O.PARAM_GRADS) > 1e-4


# ---- scalar structure (Table 1 "Scalar SSM": one decay rate per channel) -----------------------------------------
def _scalar_theta(tiny):
    th, x, g = tiny
    ths = dict(th)
    ths["A_log"] = th["A_log"][:, 0].copy()          # [P]
    return ths, x, g, th["A_log"].shape[1]


def test_scalar_forward_equals_masked_product_form(tiny):
    # with A^t a multiple of the identity the recurrence collapses to y = (L o (C B^T)) (Delta x) per channel
    ths, x, _, N = _scalar_theta(tiny)
    y_rec = O.ssm_forward(O.untie_scalar_A(ths, N), x)
    y_quad = O.scalar_forward_quadratic(ths, x, N)
    assert np.abs(y_rec - y_quad).max() / np.abs(y_rec).max() < 1e-12


def test_scalar_rate_gradient_by_finite_differences(tiny):
    ths, x, g, N = _scalar_theta(tiny)
    for tbar in (x.shape[0], 5):
        a = O.scalar_adjoint_grad(ths, x, g, tbar, N)
        assert a["dA_log"].shape == ths["A_log"].shape
        if tbar < x.shape[0]:
            continue          # the truncated form is not the gradient of a scalar loss: only its shape is checked here
        eps = 1e-6
        fd = np.zeros_like(ths["A_log"])
        for p in range(fd.size):
            tp = {k: v.copy() for k, v in ths.items()}; tm = {k: v.copy() for k, v in ths.items()}
            tp["A_log"][p] += eps; tm["A_log"][p] -= eps
            lp = float(np.sum(g * O.scalar_forward_quadratic(tp, x, N)))
            lm = float(np.sum(g * O.scalar_forward_quadratic(tm, x, N)))
            fd[p] = (lp - lm) / (2 * eps)
        assert np.abs(fd - a["dA_log"]).max() / np.abs(a["dA_log"]).max() < 1e-7


def test_scalar_truncated_rate_gradient_is_windowed_bptt(tiny):
    # truncated form with tied rates against the brute-force per-token windowed backpropagation, tied the same way
    ths, x, g, N = _scalar_theta(tiny)
    a = O.scalar_adjoint_grad(ths, x, g, 5, N)
    b = O.windowed_bptt_bruteforce(O.untie_scalar_A(ths, N), x, g, 5)
    assert np.abs(a["dA_log"] - b["dA_log"].sum(axis=1)).max() / np.abs(a["dA_log"]).max() < 1e-10
    for k in ("dW_delta", "dW_B", "dW_C", "db_delta", "dx"):
        assert np.abs(a[k] - b[k]).max() / np.abs(b[k]).max() < 1e-10, k


# the stack's storage hook changes no formula: identity == default, and a rounding hook is applied to every stored tensor
def test_stack_store_hook():
    rng = np.random.default_rng(31)
    P, N, T, K = 5, 3, 9, 3
    ths = [make_theta(rng, P, N, -1.0, 1.0) for _ in range(K)]
    y0, g = rng.normal(size=(T, P)), rng.normal(size=(T, P))
    a, Ga = O.stack_grad(ths, y0, g, 4, mode="chained")
    b, Gb = O.stack_grad(ths, y0, g, 4, mode="chained", store=lambda v: v)
    assert np.array_equal(Ga, Gb) and all(np.array_equal(a[k]["dW_B"], b[k]["dW_B"]) for k in range(K))
    q = lambda v: np.round(v * 64) / 64
    ys, yhats = O.stack_forward(ths, y0, store=q)
    assert all(np.array_equal(q(v), v) for v in ys[1:] + yhats)
    assert np.abs(ys[-1] - O.stack_forward(ths, y0)[0][-1]).max() > 0
    _, Gq = O.stack_grad(ths, y0, g, 4, mode="chained", store=q)
    assert np.array_equal(q(Gq), Gq)


# the multi-process harness of the GPU tests composes the oracle's own functions: same result as adjoint_grad
def test_parallel_harness_equals_adjoint_grad():
    import oracle_parallel as OP
    rng = np.random.default_rng(41)
    P, N, T = 10, 4, 37
    th = make_theta(rng, P, N, -1.0, 1.0)
    x, g = rng.normal(size=(2, T, P)), rng.normal(size=(2, T, P))
    for tier, tbar in (("block", 9), ("direct", 5), ("block", T)):
        ref = O.batched(O.adjoint_grad, th, x, g, tbar, tier=tier)
        got = OP.batched_adjoint_grad(th, x, g, tbar, tier=tier, channel_block=3, want=("absq",))
        for k in GRADS + ("y",):
            assert np.abs(got[k] - ref[k]).max() <= 1e-13 * (np.abs(ref[k]).max() + 1e-300), (tier, k)
        assert got["absq"].shape == (P, N) and (got["absq"] >= 0).all()


def test_parallel_stack_harness_equals_stack_grad():
    import oracle_parallel as OP
    from gpu_util import bf16_round
    rng = np.random.default_rng(5)
    P, N, T, K = 12, 16, 40, 3
    ths = [make_theta(rng, P, N) for _ in range(K)]
    y0, g = rng.normal(size=(T, P)), rng.normal(size=(T, P))
    for mode in ("chained", "paper"):
        for store in (None, bf16_round):
            a, Ga = O.stack_grad(ths, y0, g, 7, mode=mode, tier="block", store=store)
            b, Gb = OP.stack_grad(ths, y0, g, 7, mode, store, channel_block=5)
            for k in range(K):
                for name in O.PARAM_GRADS:
                    assert np.abs(a[k][name] - b["grads"][k][name]).max() <= 1e-12 * np.abs(a[k][name]).max()
            if mode == "chained":
                assert np.abs(Ga - Gb).max() <= 1e-12 * np.abs(Ga).max()
            assert np.abs(b["yK"] - O.stack_forward(ths, y0, store)[0][-1]).max() <= 1e-12
