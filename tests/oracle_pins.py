"""Pin checks for the fp64 oracle, written as functions of the oracle module so that the same
checks can be run against deliberately broken copies (see test_oracle_mutations.py).

No expected value below is produced by the function it checks: they come from closed forms,
50-digit scalar hand arithmetic stored under tests/golden/, a library SVD, or invariants the
paper states (Lemma 1, Lemma 2)."""
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
NS_A, NS_B, NS_C = 3.4445, -4.7750, 2.0315   # printed under Eq. newton_schulz


def _rows(name):
    out = []
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            out.append([float(t) for t in line.split()])
    return out


def quintic(x, a=NS_A, b=NS_B, c=NS_C):
    return a * x + b * x ** 3 + c * x ** 5


def ns_svd_route(M, T=5, a=NS_A, b=NS_B, c=NS_C, eps=0.0):
    """Closed form of Eq. newton_schulz: the iteration maps each singular value through p, T times,
    and leaves the singular vectors alone.  Uses the library SVD, not the matrix iteration."""
    M = np.asarray(M, dtype=np.float64)
    nrm = np.sqrt((M * M).sum())
    if nrm == 0.0:
        return np.zeros_like(M)
    U, S, Vt = np.linalg.svd(M, full_matrices=False)
    s = S / (nrm + eps)
    for _ in range(T):
        s = quintic(s, a, b, c)
    return (U * s) @ Vt


def muon_reference_step(W, G, M_prev, lr, mu, lam, gamma, T=5):
    """Eq. muon_momentum / muon_ns / muon_update written separately from the oracle, with the
    orthogonalisation taken through the SVD closed form."""
    M = mu * M_prev + G
    O = ns_svd_route(M, T)
    return W - lr * (gamma * O + lam * W), M, O


# ---------------------------------------------------------------------------------------------

def check_scalar_orbits(orc):
    """P4: on diagonal input the iteration is the scalar quintic; stored 50-digit orbits."""
    for row in _rows("ns_scalar_orbits.txt"):
        x0, orbit = row[0], row[1:]
        # a 2x2 diagonal with entries (x0, 0) has Frobenius norm x0; rescale so that X_0 = diag(x0, y0)
        y0 = np.sqrt(max(0.0, 1.0 - x0 * x0)) if x0 < 1 else 0.0
        M = np.diag([x0, y0]) * 7.0            # any positive scale: X_0 = M/||M||_F = diag(x0, y0)
        for T in range(1, 6):
            X = orc.newton_schulz(M, T=T, eps=0.0)
            assert abs(X[0, 0] - orbit[T - 1]) < 1e-12, (x0, T, X[0, 0], orbit[T - 1])
            assert abs(X[0, 1]) < 1e-15 and abs(X[1, 0]) < 1e-15


def check_quintic_band(orc):
    """P4: p(1) = a+b+c = 0.7010; after 5 iterations singular values that start in [0.003, 1]
    lie in [0.68183, 1.20237] (they do not converge to 1)."""
    rng = np.random.default_rng(5)
    for (m, n) in [(6, 9), (16, 16), (24, 8)]:
        M = rng.standard_normal((m, n))
        O = orc.newton_schulz(M, T=5, eps=0.0)
        s0 = np.linalg.svd(M, compute_uv=False) / np.linalg.norm(M)
        s5 = np.linalg.svd(O, compute_uv=False)
        assert s0.min() > 0.003
        assert s5.min() >= 0.68183 - 1e-9 and s5.max() <= 1.20237 + 1e-9, (s5.min(), s5.max())
    X = orc.newton_schulz(np.array([[1.0]]), T=1, eps=0.0)
    assert abs(X[0, 0] - 0.7010) < 1e-13


def check_hand_2x2(orc):
    """P6: two full steps on diagonal 2x2 matrices against stored scalar hand arithmetic."""
    hp = orc.Hyper(lr=0.1, momentum=0.5, accel_beta=0.9, accel_alpha=-5.0, weight_decay=0.1,
                   ns_steps=5, norm_eps=0.0)
    W = np.diag([1.0, -1.0])
    st = orc.OracleState(2, 2)
    Gs = [np.diag([3.0, 4.0]), np.diag([4.0, 3.0])]
    for row, G in zip(_rows("hand_2x2.txt"), Gs):
        _, A11, A22, Gt11, Gt22, M11, M22, nrm, O11, O22, W11, W22 = row
        W, O = orc.mona_step(W, G, st, hp)
        np.testing.assert_allclose(np.diag(st.A), [A11, A22], rtol=0, atol=1e-13)
        np.testing.assert_allclose(np.diag(st.M), [M11, M22], rtol=0, atol=1e-13)
        np.testing.assert_allclose(np.linalg.norm(st.M), nrm, rtol=0, atol=1e-12)
        np.testing.assert_allclose(np.diag(O), [O11, O22], rtol=0, atol=1e-12)
        np.testing.assert_allclose(np.diag(W), [W11, W22], rtol=0, atol=1e-12)
        np.testing.assert_allclose(st.G_prev, G, rtol=0, atol=0)
        assert abs(W[0, 1]) < 1e-15 and abs(W[1, 0]) < 1e-15


def check_hand_3x2(orc):
    """P7: tall, non-diagonal case against the SVD closed form stored in the fixture; also shows
    that O differs entry-wise from U V^T (the singular values land in a band)."""
    rows = _rows("hand_3x2.txt")
    nrm = rows[0][0]
    s5 = np.array(rows[2])
    UVt, NS, W1 = np.array(rows[3:6]), np.array(rows[6:9]), np.array(rows[9:12])
    M = np.array([[1., 2.], [3., 4.], [5., 6.]])
    assert abs(np.sqrt(91.0) - nrm) < 1e-12                       # 1+4+9+16+25+36 = 91
    O = orc.newton_schulz(M, T=5, eps=0.0)
    np.testing.assert_allclose(O, NS, rtol=0, atol=2e-12)
    np.testing.assert_allclose(np.sort(np.linalg.svd(O, compute_uv=False)), np.sort(s5), atol=2e-12)
    assert np.abs(O - UVt).max() > 0.05
    # same singular vectors as U V^T: U V^T O^T must be symmetric positive definite
    P = UVt.T @ O
    np.testing.assert_allclose(P, P.T, atol=1e-11)
    assert np.linalg.eigvalsh(0.5 * (P + P.T)).min() > 0.6
    hp = orc.Hyper(lr=0.1, momentum=0.5, accel_beta=0.9, accel_alpha=-5.0, weight_decay=0.1,
                   ns_steps=5, norm_eps=0.0)
    st = orc.OracleState(3, 2)
    Wn, _ = orc.mona_step(0.1 * np.ones((3, 2)), M, st, hp)
    np.testing.assert_allclose(Wn, W1, rtol=0, atol=2e-12)
    # the update scale depends on max(m, n) only
    assert abs(orc.update_scale(3, 2) - 0.2 * np.sqrt(3.0)) < 1e-15
    assert abs(orc.update_scale(2, 3) - 0.2 * np.sqrt(3.0)) < 1e-15
    assert abs(orc.update_scale(5, 7, 1, 0.37) - 0.37) < 1e-15


def check_constant_gradient(orc):
    """P1: G_k = g for all k.  Closed forms: A_k = (1-beta_a) beta_a^(k-1) g,
    M_k = c_k g with c_k = mu c_{k-1} + 1 + alpha (1-beta_a) beta_a^(k-1) > 0, hence O_k = NS(g)
    at every step and the W trajectory is Muon's: W_{k+1} = (1 - eta lambda) W_k - eta gamma NS(g)."""
    rng = np.random.default_rng(11)
    m, n = 5, 8
    g = rng.standard_normal((m, n))
    W = rng.standard_normal((m, n)) * 0.02
    hp = orc.Hyper(lr=1e-2, momentum=0.95, accel_beta=0.99, accel_alpha=-50.0, weight_decay=0.1,
                   ns_steps=5, norm_eps=0.0)
    st = orc.OracleState(m, n)
    c_expected = [0.5, 0.98, 1.44095, 1.883753, 2.309267345]       # from the recurrence, by hand
    O_g = ns_svd_route(g, 5)
    gamma = 0.2 * np.sqrt(8.0)
    W_ref = W.copy()
    c = 0.0
    for k in range(1, 41):
        W, O = orc.mona_step(W, g, st, hp)
        coef_a = (1 - 0.99) * 0.99 ** (k - 1)
        c = 0.95 * c + 1.0 + (-50.0) * coef_a
        if k <= 5:
            assert abs(c - c_expected[k - 1]) < 1e-12
        np.testing.assert_allclose(st.A, coef_a * g, rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(st.M, c * g, rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(O, O_g, rtol=0, atol=1e-11)
        W_ref = (1 - 1e-2 * 0.1) * W_ref - 1e-2 * gamma * O_g
        np.testing.assert_allclose(W, W_ref, rtol=0, atol=1e-11)
    # the acceleration term decays geometrically to zero
    assert np.linalg.norm(st.A) < 0.01 * 0.99 ** 39 * np.linalg.norm(g) * (1 + 1e-9)


def check_alpha_zero_is_muon(orc):
    """P2: with alpha = 0 the M, O, W sequences are Muon's (Eq. muon_momentum..muon_update),
    while A still evolves as the EMA of differences."""
    rng = np.random.default_rng(3)
    m, n = 7, 4
    W = rng.standard_normal((m, n)) * 0.02
    Wr, Mr = W.copy(), np.zeros((m, n))
    hp = orc.Hyper(lr=2e-2, momentum=0.9, accel_beta=0.95, accel_alpha=0.0, weight_decay=0.05,
                   ns_steps=5, norm_eps=0.0)
    st = orc.OracleState(m, n)
    gamma = 0.2 * np.sqrt(7.0)
    A_ref, G_prev = np.zeros((m, n)), np.zeros((m, n))
    for k in range(6):
        G = rng.standard_normal((m, n))
        W, O = orc.mona_step(W, G, st, hp)
        Wr, Mr, Or = muon_reference_step(Wr, G, Mr, 2e-2, 0.9, 0.05, gamma, 5)
        A_ref = 0.95 * A_ref + 0.05 * (G - G_prev)
        G_prev = G
        np.testing.assert_allclose(st.M, Mr, rtol=0, atol=1e-13)
        np.testing.assert_allclose(O, Or, rtol=0, atol=1e-10)
        np.testing.assert_allclose(W, Wr, rtol=0, atol=1e-11)
        np.testing.assert_allclose(st.A, A_ref, rtol=0, atol=1e-13)
    assert np.linalg.norm(st.A) > 0.01


def check_general_step_unrolled(orc):
    """Random gradients, alpha != 0: A_k, G~_k and M_k against their unrolled sums
    A_k = (1-beta_a) sum_j beta_a^(k-j) (G_j - G_{j-1}),  M_k = sum_j mu^(k-j) (G_j + alpha A_j),
    and O, W against the SVD closed form of the orthogonalisation."""
    rng = np.random.default_rng(17)
    m, n = 4, 6
    beta, alpha, mu, lr, lam = 0.9, -3.0, 0.8, 0.05, 0.2
    hp = orc.Hyper(lr=lr, momentum=mu, accel_beta=beta, accel_alpha=alpha, weight_decay=lam,
                   ns_steps=4, norm_eps=0.0)
    st = orc.OracleState(m, n)
    W = rng.standard_normal((m, n))
    Gs = [np.zeros((m, n))]
    As = [np.zeros((m, n))]
    for k in range(1, 6):
        G = rng.standard_normal((m, n)) + 0.3
        Gs.append(G)
        A_k = sum((1 - beta) * beta ** (k - j) * (Gs[j] - Gs[j - 1]) for j in range(1, k + 1))
        As.append(A_k)
        M_k = sum(mu ** (k - j) * (Gs[j] + alpha * As[j]) for j in range(1, k + 1))
        O_k = ns_svd_route(M_k, 4)
        W_exp = W - lr * (0.2 * np.sqrt(6.0) * O_k + lam * W)
        W, O = orc.mona_step(W, G, st, hp)
        np.testing.assert_allclose(st.A, A_k, rtol=0, atol=1e-13)
        np.testing.assert_allclose(st.M, M_k, rtol=0, atol=1e-12)
        np.testing.assert_allclose(O, O_k, rtol=0, atol=1e-10)
        np.testing.assert_allclose(W, W_exp, rtol=0, atol=1e-11)
        np.testing.assert_allclose(st.G_prev, G, rtol=0, atol=0)


def check_svd_route_and_brute_force(orc):
    """P3 + P9: matrix iteration against the SVD closed form on tiny random shapes, including
    rank-deficient and zero input, wide, tall and square."""
    rng = np.random.default_rng(23)
    shapes = [(2, 2), (2, 5), (5, 2), (3, 3), (6, 9), (9, 6), (1, 4), (4, 1)]
    for (m, n) in shapes:
        for T in (1, 3, 5):
            M = rng.standard_normal((m, n)) * 10 ** rng.uniform(-3, 2)
            np.testing.assert_allclose(orc.newton_schulz(M, T=T, eps=0.0), ns_svd_route(M, T),
                                       rtol=0, atol=5e-11)
    u, v = rng.standard_normal((6, 1)), rng.standard_normal((1, 9))
    M = u @ v + 0.5 * (rng.standard_normal((6, 1)) @ rng.standard_normal((1, 9)))    # rank 2
    np.testing.assert_allclose(orc.newton_schulz(M, eps=0.0), ns_svd_route(M), atol=5e-11)
    Z = orc.newton_schulz(np.zeros((3, 4)))                     # default eps: 0/eps = 0
    assert np.all(Z == 0.0)
    # eps enters as X_0 = M/(||M||_F + eps)
    M = rng.standard_normal((3, 5))
    np.testing.assert_allclose(orc.newton_schulz(M, T=2, eps=0.5), ns_svd_route(M, 2, eps=0.5), atol=1e-11)
    # custom coefficients reach the right places: with (a,b,c) = (2,0,0), X_T = 2^T X_0, etc.
    X0 = M / np.linalg.norm(M)
    np.testing.assert_allclose(orc.newton_schulz(M, T=3, a=2.0, b=0.0, c=0.0, eps=0.0), 8.0 * X0, atol=1e-13)
    np.testing.assert_allclose(orc.newton_schulz(M, T=1, a=0.0, b=1.0, c=0.0, eps=0.0), X0 @ X0.T @ X0, atol=1e-13)
    np.testing.assert_allclose(orc.newton_schulz(M, T=1, a=0.0, b=0.0, c=1.0, eps=0.0),
                               X0 @ X0.T @ X0 @ X0.T @ X0, atol=1e-13)


def check_symmetries(orc):
    """P5 + P8: NS(M^T)^T = NS(M); NS(cM) = NS(M) for c > 0; NS(-M) = -NS(M);
    NS(Q M R) = Q NS(M) R for orthogonal Q, R; O keeps M's row and column space."""
    rng = np.random.default_rng(29)
    M = rng.standard_normal((5, 8))
    O = orc.newton_schulz(M, eps=0.0)
    np.testing.assert_allclose(orc.newton_schulz(M.T, eps=0.0).T, O, atol=1e-12)
    np.testing.assert_allclose(orc.newton_schulz(37.5 * M, eps=0.0), O, atol=1e-12)
    np.testing.assert_allclose(orc.newton_schulz(-M, eps=0.0), -O, atol=1e-12)
    Q, _ = np.linalg.qr(rng.standard_normal((5, 5)))
    R, _ = np.linalg.qr(rng.standard_normal((8, 8)))
    np.testing.assert_allclose(orc.newton_schulz(Q @ M @ R, eps=0.0), Q @ O @ R, atol=1e-11)
    B = rng.standard_normal((6, 2)) @ rng.standard_normal((2, 7))       # rank 2
    Ob = orc.newton_schulz(B, eps=0.0)
    U, S, Vt = np.linalg.svd(B)
    assert np.abs(U[:, 2:].T @ Ob).max() < 1e-9 and np.abs(Ob @ Vt[2:].T).max() < 1e-9


def check_lemma_bounds(orc):
    """P8: Lemma 1 and Lemma 2 with G = max_k ||G_k||_F."""
    rng = np.random.default_rng(31)
    m, n = 6, 5
    hp = orc.Hyper(accel_beta=0.9, accel_alpha=-5.0, momentum=0.9)
    st = orc.OracleState(m, n)
    W = np.zeros((m, n))
    Gs = [rng.standard_normal((m, n)) * (1 + (k % 3)) * (-1) ** k for k in range(60)]
    Gmax = max(np.linalg.norm(G) for G in Gs)
    for G in Gs:
        A_new, Gt = orc.acceleration(G, st.G_prev, st.A, 0.9, -5.0)
        assert np.linalg.norm(Gt) <= Gmax * (1 + 2 * 5.0) + 1e-12
        W, _ = orc.mona_step(W, G, st, hp)
        assert np.linalg.norm(st.A) <= 2 * Gmax + 1e-12
        assert np.linalg.norm(st.M) <= Gmax * (1 + 2 * 5.0) / (1 - 0.9) + 1e-9


def check_first_step(orc):
    """Zero initial state: D_1 = G_1, A_1 = (1-beta_a) G_1, G~_1 = (1 + alpha (1-beta_a)) G_1 = M_1."""
    G = np.arange(1.0, 13.0).reshape(3, 4)
    st = orc.OracleState(3, 4)
    hp = orc.Hyper(accel_beta=0.98, accel_alpha=-25.0, momentum=0.95)
    orc.mona_step(np.zeros((3, 4)), G, st, hp)
    np.testing.assert_allclose(st.A, 0.02 * G, rtol=1e-13)
    np.testing.assert_allclose(st.M, 0.5 * G, rtol=1e-13)


def check_bf16_rounding(orc):
    """MONA-Lite storage: round_bf16 against values fixed by the format (8 significant bits, ties to
    even) and against an independent library conversion (torch's float32 -> bfloat16)."""
    import torch
    exact = [(1.0, 1.0), (1.0 + 2.0 ** -8, 1.0),                       # tie -> even (1.0)
             (1.0078125 + 2.0 ** -8, 1.015625),                        # tie -> even (1.015625)
             (1.0 + 2.0 ** -8 + 2.0 ** -20, 1.0078125),                # just above the tie
             (0.3, 0.30078125), (0.03, 0.030029296875), (-0.3, -0.30078125), (3.0, 3.0), (0.0, 0.0),
             (1e-3, 0.00099945068359375)]
    for x, want in exact:
        got = float(orc.round_bf16(np.array([x]))[0])
        assert got == want, (x, got, want)
    rng = np.random.default_rng(11)
    x = (rng.standard_normal(20000) * np.exp(rng.uniform(-20, 20, 20000))).astype(np.float32)
    lib = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(orc.round_bf16(x), lib)


def check_lite_hand_2x2(orc):
    """MONA-Lite: two steps on diagonal 2x2 matrices against exact rational arithmetic with bfloat16
    storage of A_k and G_{k-1} (tests/golden/hand_lite_2x2.txt)."""
    hp = orc.Hyper(lr=0.1, momentum=0.5, accel_beta=0.9, accel_alpha=-5.0, weight_decay=0.1, ns_steps=5, norm_eps=0.0,
                   state_dtype="bf16")
    st = orc.OracleState(2, 2)
    W = np.diag([1.0, -1.0])
    Gs = [np.diag([0.3, 3.0]), np.diag([0.3, 4.0])]
    for row, G in zip(_rows("hand_lite_2x2.txt"), Gs):
        # what the step sees before it stores: recompute G~ from the stored A
        W, _ = orc.mona_step(W, G, st, hp)
        A, Gt, M, Gp = row[1:3], row[3:5], row[5:7], row[7:9]
        assert np.allclose(np.diag(st.A), A, rtol=0, atol=1e-15), (np.diag(st.A), A)
        assert np.allclose(np.diag(st.M), M, rtol=0, atol=1e-15), (np.diag(st.M), M)
        assert np.allclose(np.diag(st.G_prev), Gp, rtol=0, atol=1e-15), (np.diag(st.G_prev), Gp)
        assert st.A[0, 1] == 0 and st.M[1, 0] == 0
    # full-precision storage is untouched by the switch: the fp32-state run differs from the Lite run
    st32 = orc.OracleState(2, 2)
    hp32 = orc.Hyper(lr=0.1, momentum=0.5, accel_beta=0.9, accel_alpha=-5.0, weight_decay=0.1, ns_steps=5, norm_eps=0.0)
    orc.mona_step(np.diag([1.0, -1.0]), Gs[0], st32, hp32)
    assert abs(st32.A[0, 0] - 0.03) < 1e-17 and st32.G_prev[0, 0] == 0.3


def check_lite_exactly_representable(orc):
    """MONA-Lite: when every stored quantity is exactly representable in bfloat16 the Lite trajectory
    equals the full-precision one (beta_a = 0.5, dyadic gradients)."""
    g = np.array([[0.5, -0.25], [1.0, 2.0], [0.125, 4.0]])
    kw = dict(lr=0.1, momentum=0.5, accel_beta=0.5, accel_alpha=-1.0, weight_decay=0.0, ns_steps=2)
    a, b = orc.OracleState(3, 2), orc.OracleState(3, 2)
    Wa = Wb = np.ones((3, 2))
    for k in range(3):
        Wa, _ = orc.mona_step(Wa, g * (k + 1), a, orc.Hyper(**kw))
        Wb, _ = orc.mona_step(Wb, g * (k + 1), b, orc.Hyper(state_dtype="bf16", **kw))
    assert np.array_equal(a.A, b.A) and np.array_equal(a.M, b.M) and np.array_equal(a.G_prev, b.G_prev) and np.array_equal(Wa, Wb)


def check_muon_step(orc):
    """Plain Muon (Eq. muon_momentum / muon_ns / muon_update): three steps against the separately written
    reference above, whose orthogonalisation goes through the SVD closed form; A and G_prev stay untouched."""
    rng = np.random.default_rng(3)
    hp = orc.Hyper(lr=0.02, momentum=0.9, weight_decay=0.05, norm_eps=0.0)
    for (m, n) in [(4, 7), (6, 3)]:
        W = rng.standard_normal((m, n)) * 0.1
        Wr, Mr = W.copy(), np.zeros((m, n))
        st = orc.OracleState(m, n)
        for _ in range(3):
            G = rng.standard_normal((m, n))
            W, O = orc.muon_step(W, G, st, hp)
            Wr, Mr, Or = muon_reference_step(Wr, G, Mr, hp.lr, hp.momentum, hp.weight_decay, 0.2 * np.sqrt(max(m, n)))
            assert np.allclose(st.M, Mr, rtol=0, atol=1e-13) and np.allclose(O, Or, rtol=0, atol=1e-10)
            assert np.allclose(W, Wr, rtol=0, atol=1e-12)
        assert not st.A.any() and not st.G_prev.any()


ALL_CHECKS = [check_muon_step, check_bf16_rounding, check_lite_hand_2x2, check_lite_exactly_representable, check_scalar_orbits, check_quintic_band, check_hand_2x2, check_hand_3x2,
              check_constant_gradient, check_alpha_zero_is_muon, check_general_step_unrolled,
              check_svd_route_and_brute_force, check_symmetries, check_lemma_bounds, check_first_step]
