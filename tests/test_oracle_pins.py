"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests compares the oracle with itself or with the CUDA path: each
expected value is a closed form, a brute-force definition, a textbook routine or
a number the paper prints.  Section / equation references are to the paper.
"""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rel(a, b):
    return np.linalg.norm(np.asarray(a) - np.asarray(b)) / np.linalg.norm(np.asarray(b))


def draw(T, D, seed, gate_mean=2.0, unit=True, Dv=None):
    rng = np.random.default_rng(seed)
    Dv = D if Dv is None else Dv
    q = rng.standard_normal((T, D))
    k = rng.standard_normal((T, D))
    if unit:
        q /= np.linalg.norm(q, axis=1, keepdims=True)
        k /= np.linalg.norm(k, axis=1, keepdims=True)
    v = rng.standard_normal((T, Dv))
    gate = 1.0 / (1.0 + np.exp(-rng.normal(gate_mean, 1.0, T)))
    lam = np.log1p(np.exp(rng.standard_normal(T))) + 1e-2
    return q, k, v, gate, lam


def as_bthd(*arrs):
    """[T, D] / [T] single-head arrays -> ABI layout with B = heads = 1."""
    out = []
    for a in arrs:
        out.append(a[None, :, None, :] if a.ndim == 2 else a[None, :, None])
    return out


def cheb_T(n, x):
    """Chebyshev polynomial of the first kind for x >= 1."""
    return np.cosh(n * np.arccosh(x))


# --------------------------------------------------------------------------- exact target
def test_exact_branch_is_the_weighted_ridge_argmin():
    """Eq. (3) with eta_{t,i} = prod_{j>i} gamma_j (Section 4.1, gating): the exact output
    U_t (H_t + lam_t I)^{-1} q_t equals S_t q_t with S_t the argmin, found here by stacked
    least squares, with no use of H or U."""
    T, D, Dv = 12, 5, 4
    q, k, v, gate, lam = draw(T, D, 11, unit=False, Dv=Dv)
    res = oracle.fwd(*as_bthd(q, k, v, gate, lam), n_iter=3, exact=True)
    for t in range(T):
        eta = np.array([np.prod(gate[i + 1:t + 1]) for i in range(t + 1)])
        # rows: sqrt(eta_i) k_i^T  -> sqrt(eta_i) v_i^T ; sqrt(lam) I -> 0
        Aa = np.vstack([np.sqrt(eta)[:, None] * k[:t + 1], np.sqrt(lam[t]) * np.eye(D)])
        Bb = np.vstack([np.sqrt(eta)[:, None] * v[:t + 1], np.zeros((D, Dv))])
        St = np.linalg.lstsq(Aa, Bb, rcond=None)[0].T      # S (Dv x D) minimises the objective
        assert rel(res["out_exact"][0, t, 0], St @ q[t]) < 1e-11


def test_exact_branch_matches_recursive_least_squares_for_unit_gates():
    """Eq. (KF) with eta == 1 is textbook recursive least squares with Phi_0 = I / lam."""
    T, D = 20, 6
    q, k, v, gate, lam = draw(T, D, 5, unit=False)
    gate[:] = 1.0
    lam[:] = 0.37
    res = oracle.fwd(*as_bthd(q, k, v, gate, lam), n_iter=2, exact=True)
    S = np.zeros((D, D))
    Phi = np.eye(D) / 0.37
    for t in range(T):
        kt, vt = k[t], v[t]
        denom = 1.0 + kt @ Phi @ kt
        S = S - np.outer(S @ kt - vt, kt @ Phi) / denom
        Phi = Phi - np.outer(Phi @ kt, kt @ Phi) / denom     # Woodbury / Sherman-Morrison
        assert rel(res["out_exact"][0, t, 0], S @ q[t]) < 1e-10


def test_cholesky_solve_against_lapack():
    rng = np.random.default_rng(3)
    M = rng.standard_normal((9, 9))
    A = M @ M.T + 0.1 * np.eye(9)
    b = rng.standard_normal(9)
    assert rel(oracle.cholesky_solve(A, b), np.linalg.solve(A, b)) < 1e-12
    with pytest.raises(np.linalg.LinAlgError):
        oracle.cholesky_solve(-np.eye(3), np.ones(3))


# --------------------------------------------------------------------------- Algorithm 1
def test_omega_schedule_lemma3_and_lemma4():
    """Lemma 3: 2 = w_0 >= w_1 >= ... >= w_r >= w* > 1 and 4 - rho^2 w_i in [2, 4].
    Lemma 4: w_i - w* <= R^i (w_0 - w*)."""
    for L, mu in [(1.02, 0.02), (3.0, 1.0), (1.0 + 1e-4, 1e-4), (2.0, 1.999)]:
        r = 40
        w = oracle.omega_schedule(L, mu, r)
        rho = (L - mu) / (L + mu)
        # w* = 2 (1 - sqrt(1 - rho^2)) / rho^2, written without the cancellation at small rho
        wstar = 2 / (1 + np.sqrt(1 - rho ** 2))
        if rho > 0.1:
            assert abs(wstar - 2 * (1 - np.sqrt(1 - rho ** 2)) / rho ** 2) < 1e-12
        kappa = L / mu
        R = (kappa - 1) / (kappa + 1) * (np.sqrt(kappa) - 1) / (np.sqrt(kappa) + 1)
        assert w[0] == 2.0
        assert np.all(np.diff(w) <= 1e-15)
        assert np.all(w >= wstar - 1e-12) and wstar > 1
        assert np.all(4 - rho ** 2 * w >= 2 - 1e-12) and np.all(4 - rho ** 2 * w <= 4)
        i = np.arange(r + 1)
        assert np.all(w - wstar <= R ** i * (w[0] - wstar) + 1e-13)
        # fixed point of the weight schedule
        assert abs(4 / (4 - rho ** 2 * wstar) - wstar) < 1e-12


def _golden_rows():
    rows = []
    with open(os.path.join(GOLDEN, "remark_kappa51.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, p, val, tol = line.split()
            rows.append((name, int(p), float(val), float(tol)))
    return rows


def test_printed_contraction_numbers_for_kappa_51():
    """Remark after Lemma 4: printed R^i and R_a^i for kappa = 51 bound what the oracle does.
    (a) the printed R^i (inflated by its printing tolerance) bounds (w_i - w*)/(w_0 - w*);
    (b) twice the printed R_a^n (inflated likewise) bounds the relative error of xi_{n-1}
        on a spectrum that fills [mu, L], and the bound is nearly attained."""
    L, mu = 1.02, 0.02
    rows = _golden_rows()
    w = oracle.omega_schedule(L, mu, 30)
    rho = (L - mu) / (L + mu)
    wstar = 2 * (1 - np.sqrt(1 - rho ** 2)) / rho ** 2
    kappa = L / mu
    R = (kappa - 1) / (kappa + 1) * (np.sqrt(kappa) - 1) / (np.sqrt(kappa) + 1)
    Ra = (np.sqrt(kappa) - 1) / (np.sqrt(kappa) + 1)
    # the oracle's own schedule contracts at least as fast as the printed R
    D = 64
    eig = np.linspace(mu, L, D)
    rng = np.random.default_rng(0)
    Qm = np.linalg.qr(rng.standard_normal((D, D)))[0]
    A = (Qm * eig) @ Qm.T
    xstar_coeff = np.ones(D)                      # equal weight on every eigen-direction of x*
    xstar = Qm @ xstar_coeff
    qv = A @ xstar
    for name, p, val, tol in rows:
        if name == "R":
            assert abs(R ** p - val) <= tol * val + 1e-12
            assert (w[p] - wstar) <= val * (1 + tol) * (w[0] - wstar)
        else:
            assert abs(Ra ** p - val) <= tol * val + 1e-12
            xi = oracle.chebyshev(A, qv, L, mu, p - 1)     # p-1 iterations <-> polynomial degree p
            err = np.linalg.norm(xi - xstar) / np.linalg.norm(xstar)
            assert err <= 2 * val * (1 + tol)
            worst = np.max(np.abs(Qm.T @ (xi - xstar)))    # error on the worst eigen-direction
            assert worst >= 0.5 * val * (1 - tol)          # edge eigenvalue mu attains 1/T_p ~ 2 R_a^p


@pytest.mark.parametrize("r", [0, 1, 2, 5, 10, 30])
def test_chebyshev_iterate_equals_closed_polynomial_form(r):
    """xi_r = (I - P_{r+1}(A)) A^{-1} q with P_n(z) = T_n((L+mu-2z)/(L-mu)) / T_n((L+mu)/(L-mu)),
    the classical characterisation of the Chebyshev Iteration (xi_r = p_r(A) q, Appendix proof of
    Lemma 2).  Evaluated through an eigendecomposition, independent of any recurrence for xi."""
    D = 16
    rng = np.random.default_rng(7 + r)
    M = rng.standard_normal((D, D))
    Hm = M @ M.T / D
    lam = 0.3
    A = Hm + lam * np.eye(D)
    f = np.linalg.norm(Hm, "fro")
    L, mu = f + lam, lam
    q = rng.standard_normal(D)
    xi = oracle.chebyshev(A, q, L, mu, r)
    ev, V = np.linalg.eigh(A)
    n = r + 1
    sigma = (L + mu) / (L - mu)
    arg = (L + mu - 2 * ev) / (L - mu)             # in [-1, 1] for ev in [mu, L]
    Tn = np.cos(n * np.arccos(np.clip(arg, -1, 1)))
    Pn = Tn / cheb_T(n, sigma)
    expect = V @ ((1 - Pn) / ev * (V.T @ q))
    assert rel(xi, expect) < 1e-11


def test_chebyshev_handedness_against_hand_computed_first_steps():
    """r = 1 by hand from Algorithm 1: xi_1 = xi_0 - (2 w_1/(L+mu)) (A xi_0 - q) + (w_1 - 1) xi_0.
    Catches a swapped sign or a dropped momentum term on a 2x2 example with printed numbers."""
    A = np.array([[2.0, 0.5], [0.5, 1.0]])
    q = np.array([1.0, -1.0])
    L, mu = 3.0, 0.5
    rho = (L - mu) / (L + mu)
    w1 = 4 / (4 - 2 * rho ** 2)
    xi0 = 2 * q / (L + mu)
    xi1 = xi0 - 2 * w1 / (L + mu) * (A @ xi0 - q) + (w1 - 1) * xi0
    assert rel(oracle.chebyshev(A, q, L, mu, 0), xi0) < 1e-15
    assert rel(oracle.chebyshev(A, q, L, mu, 1), xi1) < 1e-15
    # numbers: rho = 5/7, w1 = 4/(4 - 50/49) = 196/146
    assert abs(w1 - 196 / 146) < 1e-15
    assert rel(xi0, [4 / 7, -4 / 7]) < 1e-15


def test_chebyshev_converges_to_cholesky_within_the_sharp_bound():
    """||xi_r - x*|| <= ||x*|| / T_{r+1}((L+mu)/(L-mu)) whenever spec(A) is inside [mu, L], which
    L = ||H||_F + lam, mu = lam guarantees (Section 4.1, eq. (4)).  Checked per token of a gated
    sequence through the oracle's x and its exact branch; convergence is monotone in the bound."""
    T, D = 48, 8
    q, k, v, gate, lam = draw(T, D, 21)
    args = as_bthd(q, k, v, gate, lam)
    prev_bound_violation = 0.0
    worst_ratio = 0.0
    errs = []
    for r in [0, 1, 2, 4, 8, 16, 32, 64]:
        res = oracle.fwd(*args, n_iter=r, exact=True, want_x=True)
        fro = res["fro"][0, :, 0]
        e_tot = 0.0
        for t in range(T):
            # x* through numpy from the definition of H_t
            eta = np.array([np.prod(gate[i + 1:t + 1]) for i in range(t + 1)])
            Ht = (k[:t + 1].T * eta) @ k[:t + 1]
            assert abs(np.linalg.norm(Ht, "fro") - fro[t]) < 1e-12
            xs = np.linalg.solve(Ht + lam[t] * np.eye(D), q[t])
            L, mu = fro[t] + lam[t], lam[t]
            bound = 1.0 / cheb_T(r + 1, (L + mu) / (L - mu))
            err = np.linalg.norm(res["x"][0, t, 0] - xs) / np.linalg.norm(xs)
            assert err <= bound * (1 + 1e-9) + 1e-13
            worst_ratio = max(worst_ratio, err / bound)
            e_tot += err
        errs.append(e_tot / T)
    assert worst_ratio > 0.99          # attained at the first token (spectrum = {mu, L})
    assert all(b < a for a, b in zip(errs, errs[1:]))
    assert errs[-1] < 1e-6


@pytest.mark.parametrize("r", [0, 1, 2, 3, 8])
def test_first_token_closed_form(r):
    """Unit k_1 and zero initial state: H_1 = k k^T, ||H_1||_F = 1, L = 1 + lam, mu = lam,
    spec(A_1) = {mu, L}.  Sherman-Morrison gives the exact output v (k.q)/(1+lam); the Chebyshev
    iterate multiplies the component along k by 1 - (-1)^{r+1}/T_{r+1}(1 + 2 lam)."""
    D = 7
    rng = np.random.default_rng(2)
    q = rng.standard_normal((1, D))
    k = rng.standard_normal((1, D))
    k /= np.linalg.norm(k)
    v = rng.standard_normal((1, D))
    lam = np.array([0.23])
    gate = np.array([0.6])     # multiplies the zero state: no effect
    res = oracle.fwd(*as_bthd(q, k, v, gate, lam), n_iter=r, exact=True)
    kq = float(k[0] @ q[0])
    exact = v[0] * kq / (1 + lam[0])
    n = r + 1
    ch = exact * (1 - (-1) ** n / cheb_T(n, 1 + 2 * lam[0]))
    assert abs(res["fro"][0, 0, 0] - 1.0) < 1e-14
    assert rel(res["out_exact"][0, 0, 0], exact) < 1e-13
    assert rel(res["out"][0, 0, 0], ch) < 1e-12


def test_large_lambda_limit():
    """lam_t * o_t -> U_t q_t as lam_t grows (already true for r = 0: xi_0 = 2q/(L+mu) -> q/lam);
    the deviation is O(||H||/lam)."""
    T, D = 16, 6
    q, k, v, gate, _ = draw(T, D, 9)
    devs = []
    for lam_val in [1e2, 1e4, 1e6]:
        lam = np.full(T, lam_val)
        for r in (0, 3):
            res = oracle.fwd(*as_bthd(q, k, v, gate, lam), n_iter=r)
            U = np.zeros((D, D))
            worst = 0.0
            for t in range(T):
                U = gate[t] * U + np.outer(v[t], k[t])
                worst = max(worst, rel(lam_val * res["out"][0, t, 0], U @ q[t]))
            devs.append((lam_val, r, worst))
            assert worst < 5.0 / lam_val
    assert devs[-1][2] < 1e-5


def test_scaled_identity_state_is_solved_at_once():
    """L = mu (H = 0): rho = 0, every omega_i = 1 and xi_i = q / lam for all i (remark in the proof
    of Lemma 3).  All-zero keys keep H = 0, and U = 0 gives zero output."""
    D = 5
    A = 0.7 * np.eye(D)
    q = np.arange(1.0, D + 1)
    for r in (0, 1, 4):
        assert rel(oracle.chebyshev(A, q, 0.7, 0.7, r), q / 0.7) < 1e-15
    w = oracle.omega_schedule(0.7, 0.7, 5)
    assert w[0] == 2.0 and np.all(w[1:] == 1.0)


# --------------------------------------------------------------------------- recurrence structure
def test_state_closed_form_and_gate_order():
    """H_T = sum_j (prod_{i>j} gamma_i) k_j k_j^T and the same for U (unrolled eq. (CH)); gamma_1
    multiplies the initial state only.  With a non-zero state_in the decay of the initial state
    by prod gamma is visible, which fixes the decay-then-write order."""
    T, D, Dv = 10, 4, 3
    q, k, v, gate, lam = draw(T, D, 4, Dv=Dv)
    rng = np.random.default_rng(1)
    M = rng.standard_normal((D, D))
    H0 = M @ M.T
    U0 = rng.standard_normal((Dv, D))
    s_in = np.concatenate([H0.ravel(), U0.ravel()])[None, None]
    res = oracle.fwd(*as_bthd(q, k, v, gate, lam), n_iter=1, state_in=s_in)
    w = np.array([np.prod(gate[j + 1:]) for j in range(T)])
    Hexp = np.prod(gate) * H0 + (k.T * w) @ k
    Uexp = np.prod(gate) * U0 + (v.T * w) @ k
    st = res["state"][0, 0]
    assert rel(st[:D * D].reshape(D, D), Hexp) < 1e-13
    assert rel(st[D * D:].reshape(Dv, D), Uexp) < 1e-13
    # token t uses the state that already contains token t
    f0 = np.linalg.norm(gate[0] * H0 + np.outer(k[0], k[0]), "fro")
    assert abs(res["fro"][0, 0, 0] - f0) < 1e-12


def test_chunkwise_frobenius_identity():
    """Section 4.2.1: ||H_c||_F^2 = zeta_c^2 ||H_0||_F^2 + 2 zeta_c sum_j M_{j,c} k_j^T H_0 k_j
    + column-sum(((G o G) M) o M), with M_{j,c} = zeta_c / zeta_j for j <= c and 0 otherwise.
    The three-term formula, typed here from the paper, must reproduce the oracle's direct norm."""
    C, D = 16, 6
    q, k, v, gate, lam = draw(2 * C, D, 8)
    args = as_bthd(q, k, v, gate, lam)
    res_first = oracle.fwd(*[a[:, :C] for a in args], n_iter=0)
    res_all = oracle.fwd(*args, n_iter=0)
    H0 = res_first["state"][0, 0][:D * D].reshape(D, D)       # state entering the second chunk
    K = k[C:]
    zeta = np.cumprod(gate[C:])
    Mjc = np.triu(zeta[None, :] / zeta[:, None])              # [j, c], zero for j > c
    G = K @ K.T
    t1 = zeta ** 2 * np.sum(H0 * H0)
    quad = np.einsum("jd,de,je->j", K, H0, K)
    t2 = 2 * zeta * np.sum(quad[:, None] * Mjc, axis=0)
    t3 = np.sum(((G * G) @ Mjc) * Mjc, axis=0)
    assert rel(np.sqrt(t1 + t2 + t3), res_all["fro"][0, C:, 0]) < 1e-13


@pytest.mark.parametrize("C", [4, 8, 16])
def test_chunkwise_row_form_reproduces_the_tokenwise_recurrence(C):
    """Section 4.2.1: with the chunk-initial state stored, H_{[t]+c} xi = zeta_c H_0 xi +
    sum_{j<=c} (zeta_c/zeta_j) k_j k_j^T xi; the same unrolling gives U_{[t]+c} xi.  Running
    Algorithm 1 on whole chunks with these products gives the token-wise result for every C."""
    T, D, r = 32, 5, 6
    q, k, v, gate, lam = draw(T, D, 12)
    res = oracle.fwd(*as_bthd(q, k, v, gate, lam), n_iter=r)
    H0 = np.zeros((D, D))
    U0 = np.zeros((D, D))
    out = np.zeros((T, D))
    for n in range(T // C):
        s = slice(n * C, (n + 1) * C)
        Q, K, V, g, lm = q[s], k[s], v[s], gate[s], lam[s]
        zeta = np.cumprod(g)
        Gam = np.tril(zeta[:, None] / zeta[None, :])          # [c, j]
        f = res["fro"][0, s, 0]
        L, mu = f + lm, lm
        rho = (L - mu) / (L + mu)
        om = np.full(C, 2.0)
        Xp = np.zeros((C, D))
        X = 2 * Q / (L + mu)[:, None]
        for _ in range(r):
            om = 4 / (4 - rho ** 2 * om)
            Y = zeta[:, None] * (X @ H0) + (Gam * (X @ K.T)) @ K + lm[:, None] * X
            Xn = X - (2 * om / (L + mu))[:, None] * (Y - Q) + (om - 1)[:, None] * (X - Xp)
            Xp, X = X, Xn
        out[s] = zeta[:, None] * (X @ U0.T) + (Gam * (X @ K.T)) @ V
        w = Gam[-1]
        H0 = zeta[-1] * H0 + (K.T * w) @ K
        U0 = zeta[-1] * U0 + (V.T * w) @ K
    assert rel(out, res["out"][0, :, 0]) < 1e-12


def test_decode_step_continues_the_forward_recurrence():
    """Eq. (CH) is one recurrence: T tokens forward, then one decode step per token, equals
    T + n tokens forward; a prefill split with state_in equals the whole prefill."""
    T, n, D = 24, 5, 6
    q, k, v, gate, lam = draw(T + n, D, 30)
    args = as_bthd(q, k, v, gate, lam)
    whole = oracle.fwd(*args, n_iter=4, exact=True)
    head = oracle.fwd(*[a[:, :T] for a in args], n_iter=4)
    state = head["state"]
    for t in range(T, T + n):
        step = oracle.decode(state, *[a[:, t] for a in args], n_iter=4, exact=True)
        state = step["state"]
        assert rel(step["out"][0, 0], whole["out"][0, t, 0]) < 1e-13
        assert rel(step["out_exact"][0, 0], whole["out_exact"][0, t, 0]) < 1e-12
    assert rel(state, whole["state"]) < 1e-14
    tail = oracle.fwd(*[a[:, T:] for a in args], n_iter=4, state_in=head["state"])
    assert rel(tail["out"], whole["out"][:, T:]) < 1e-13


def test_heads_and_batches_are_independent_and_layout_is_bthd():
    """A [B,T,heads,d] call equals per-(b,h) single-head calls (pins the memory layout)."""
    B, T, Hh, D = 2, 9, 3, 4
    rng = np.random.default_rng(0)
    q = rng.standard_normal((B, T, Hh, D))
    k = rng.standard_normal((B, T, Hh, D))
    v = rng.standard_normal((B, T, Hh, D))
    gate = rng.uniform(0.5, 1.0, (B, T, Hh))
    lam = rng.uniform(0.1, 1.0, (B, T, Hh))
    full = oracle.fwd(q, k, v, gate, lam, n_iter=3)
    for b in range(B):
        for h in range(Hh):
            one = oracle.fwd(q[b:b + 1, :, h:h + 1], k[b:b + 1, :, h:h + 1], v[b:b + 1, :, h:h + 1],
                             gate[b:b + 1, :, h:h + 1], lam[b:b + 1, :, h:h + 1], n_iter=3)
            assert np.array_equal(one["out"][0, :, 0], full["out"][b, :, h])
            assert np.array_equal(one["state"][0, 0], full["state"][b, h])


def test_adaptive_regularisation_gives_kappa_bound():
    """Section 4.1, eq. (4): lam_t = a ||H_t||_F gives L/mu = (a+1)/a (51 for a = 0.02); the
    adaptive mode equals the absolute mode fed with a * fro."""
    T, D, a = 12, 5, 0.02
    q, k, v, gate, _ = draw(T, D, 14)
    a_arr = np.full(T, a)
    ad = oracle.fwd(*as_bthd(q, k, v, gate, a_arr), n_iter=5, lam_mode=1)
    fro = ad["fro"][0, :, 0]
    ab = oracle.fwd(*as_bthd(q, k, v, gate, a * fro), n_iter=5)
    assert rel(ad["out"], ab["out"]) < 1e-14
    assert np.allclose((fro + a * fro) / (a * fro), 51.0)


# --------------------------------------------------------------------------- backward solve for dq
def test_fixed_iteration_solve_is_linear_and_self_adjoint():
    """Section 4.2.2 ("Backward Pass", implicit differentiation), Lemma 2: with r fixed the Chebyshev map q -> x is x = p_r(A) q,
    a polynomial in the symmetric matrix A = H_t + lambda_t I whose coefficients depend on (L, mu, r) only.
    Hence it is linear in the right-hand side and self-adjoint, so dL/dq = CH(A, dL/dx, r): the same solve
    with another right-hand side.  Checked on the oracle's per-token solves: <CH(u), w> = <u, CH(w)> and
    CH(a u + b w) = a CH(u) + b CH(w), token by token, with H_t built by the recurrence."""
    T, D, r = 24, 16, 7
    _, k, v, gate, lam = draw(T, D, seed=31)
    rng = np.random.default_rng(32)
    u, w = rng.standard_normal((T, D)), rng.standard_normal((T, D))

    def solve(rhs):
        return oracle.fwd(*as_bthd(rhs, k, v, gate, lam), n_iter=r, want_x=True)["x"][0, :, 0]

    xu, xw, xc = solve(u), solve(w), solve(0.3 * u - 1.7 * w)
    lhs = np.einsum("td,td->t", xu, w)
    rhs = np.einsum("td,td->t", u, xw)
    assert np.allclose(lhs, rhs, rtol=1e-10, atol=1e-12)
    assert rel(xc, 0.3 * xu - 1.7 * xw) < 1e-12


def test_solve_gradient_matches_finite_differences():
    """The same statement as a gradient check: for the loss sum_t <g_t, x_t(q)>, dL/dq_t = CH(A_t, g_t, r);
    compared with central differences of the oracle's forward solve (the map is linear, so they agree to
    rounding)."""
    T, D, r = 6, 8, 5
    q, k, v, gate, lam = draw(T, D, seed=41)
    g = np.random.default_rng(42).standard_normal((T, D))

    def solve(rhs):
        return oracle.fwd(*as_bthd(rhs, k, v, gate, lam), n_iter=r, want_x=True)["x"][0, :, 0]

    dq = solve(g)
    eps = 1e-3
    for (t, i) in [(0, 0), (2, 5), (5, 7)]:
        e = np.zeros_like(q)
        e[t, i] = eps
        fd = (np.sum(g * solve(q + e)) - np.sum(g * solve(q - e))) / (2 * eps)
        assert abs(fd - dq[t, i]) <= 1e-8 * max(1.0, abs(dq[t, i]))


# --------------------------------------------------------------------------- beta-augmented write
def test_beta_write_equals_rescaled_keys_and_values():
    """Remark "canonical beta_t-augmented variant" (Section 4.1): H_t = gamma_t H_{t-1} + beta_t k k^T and
    U_t = gamma_t U_{t-1} + beta_t v k^T.  Writing beta_t k k^T = (sqrt(beta_t) k)(sqrt(beta_t) k)^T and
    beta_t v k^T = (sqrt(beta_t) v)(sqrt(beta_t) k)^T reduces it to the beta == 1 recurrence (pinned above) on
    rescaled keys and values; queries are untouched, so outputs, norms and states must agree."""
    T, D, r = 40, 12, 6
    q, k, v, gate, lam = draw(T, D, seed=51)
    beta = 1.0 / (1.0 + np.exp(-np.random.default_rng(52).standard_normal(T)))
    a = oracle.fwd(*as_bthd(q, k, v, gate, lam), n_iter=r, beta=beta[None, :, None], exact=True)
    sb = np.sqrt(beta)[:, None]
    b = oracle.fwd(*as_bthd(q, sb * k, sb * v, gate, lam), n_iter=r, exact=True)
    for name in ("out", "out_exact", "fro", "state"):
        assert rel(a[name], b[name]) < 1e-12, name
    # and it is not a no-op
    c = oracle.fwd(*as_bthd(q, k, v, gate, lam), n_iter=r)
    assert rel(a["out"], c["out"]) > 1e-2


def test_beta_zero_tokens_write_nothing():
    """A token with beta_t = 0 only decays the state: the next state is gamma_t times the previous one."""
    T, D = 5, 6
    q, k, v, gate, lam = draw(T, D, seed=53)
    beta = np.array([1.0, 1.0, 0.0, 0.0, 1.0])
    res = [oracle.fwd(*as_bthd(q[:n], k[:n], v[:n], gate[:n], lam[:n]), n_iter=2, beta=beta[None, :n, None])["state"]
           for n in (2, 4)]
    assert rel(res[1], gate[2] * gate[3] * res[0]) < 1e-13


# --------------------------------------------------------------------------- alpha-connection
def test_alpha_connection_is_a_convex_combination_of_two_reads():
    """Section 4.3 ("Architectural Consideration"): the read uses alpha_t x_t + (1 - alpha_t) q_t.  By linearity of the read,
    y_t(alpha) = alpha_t U_t x_t + (1 - alpha_t) U_t q_t, where U_t x_t is the alpha == 1 output (pinned above) and
    U_t q_t is gated linear attention, written out here by brute force from the definition of U_t."""
    T, D, r = 30, 10, 5
    q, k, v, gate, lam = draw(T, D, seed=61)
    alpha = 1.0 / (1.0 + np.exp(-np.random.default_rng(62).standard_normal(T)))
    y1 = oracle.fwd(*as_bthd(q, k, v, gate, lam), n_iter=r)["out"][0, :, 0]
    ya = oracle.fwd(*as_bthd(q, k, v, gate, lam), n_iter=r, alpha=alpha[None, :, None])["out"][0, :, 0]
    lin = np.zeros_like(y1)
    for t in range(T):
        for i in range(t + 1):
            lin[t] += np.prod(gate[i + 1:t + 1]) * v[i] * (k[i] @ q[t])
    assert rel(ya, alpha[:, None] * y1 + (1 - alpha[:, None]) * lin) < 1e-12
