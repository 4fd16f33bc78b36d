"""Derives the hand-checkable expected values stored beside this file.

Nothing here touches the CUDA library or the oracle.  The 2x2 case is diagonal, so every matrix
product collapses to scalar arithmetic, redone below with 50-digit decimals exactly as a person
would on paper.  The 3x2 case goes through a library SVD: in exact arithmetic the quintic
iteration of Eq. newton_schulz acts on the singular values only,
    NS_T(M) = U diag(p^T(sigma_i / ||M||_F)) V^T,   p(x) = a x + b x^3 + c x^5,
which is a closed form, not the matrix iteration the oracle runs.

The MONA-Lite case repeats the diagonal 2x2 steps with A_k and G_{k-1} rounded to bfloat16 when stored.
The rounding is done here on exact rationals from the definition of the format (8 significant bits,
nearest, ties to even), not on bit patterns.

Usage:  python tests/golden/derive_hand_values.py   (rewrites the .txt files)
"""
from decimal import Decimal as D, getcontext
from fractions import Fraction as F
import os

import numpy as np

getcontext().prec = 50
HERE = os.path.dirname(os.path.abspath(__file__))
a, b, c = D("3.4445"), D("-4.7750"), D("2.0315")


def p(x):
    return a * x + b * x ** 3 + c * x ** 5


def orbit(x, T=5):
    out = []
    for _ in range(T):
        x = p(x)
        out.append(x)
    return out


def fmt(x):
    return f"{x:.15f}"


def write_orbits():
    lines = ["# Scalar orbits of p(x) = a x + b x^3 + c x^5 with (a, b, c) = (3.4445, -4.7750, 2.0315),",
             "# the coefficients printed under Eq. newton_schulz.  For a diagonal matrix the iteration of",
             "# Eq. newton_schulz is this scalar map applied to each diagonal entry.",
             "# columns: x0  p(x0)  p^2(x0)  p^3(x0)  p^4(x0)  p^5(x0)"]
    for x0 in ("0.6", "0.8", "1", "0.05", "0.003"):
        lines.append(" ".join([x0] + [fmt(v) for v in orbit(D(x0))]))
    open(os.path.join(HERE, "ns_scalar_orbits.txt"), "w").write("\n".join(lines) + "\n")


def write_2x2():
    # Algorithm 1 on W_0 = diag(1, -1), G_1 = diag(3, 4), G_2 = diag(4, 3);
    # beta_a = 0.9, alpha = -5, mu = 0.5, eta = 0.1, lambda = 0.1, T = 5, gamma = 0.2 sqrt(2), eps = 0.
    beta, alpha, mu, eta, lam = D("0.9"), D("-5"), D("0.5"), D("0.1"), D("0.1")
    gamma = D("0.2") * D(2).sqrt()
    W = [D(1), D(-1)]
    Gs = [[D(3), D(4)], [D(4), D(3)]]
    A = [D(0), D(0)]; M = [D(0), D(0)]; Gp = [D(0), D(0)]
    lines = ["# Hand-computed two steps of Algorithm 1 on 2x2 diagonal matrices (all off-diagonals are 0).",
             "# W_0 = diag(1,-1), G_1 = diag(3,4), G_2 = diag(4,3); beta_a=0.9 alpha=-5 mu=0.5 eta=0.1",
             "# lambda=0.1 T=5 gamma=0.2*sqrt(2) eps=0.  Lines 4-10 of Algorithm 1 with Eq. newton_schulz",
             "# reduced to the scalar quintic on each diagonal entry.",
             "# columns: step  A11 A22  Gt11 Gt22  M11 M22  normF  O11 O22  W11 W22"]
    for k, G in enumerate(Gs, 1):
        Dk = [G[i] - Gp[i] for i in range(2)]
        A = [beta * A[i] + (1 - beta) * Dk[i] for i in range(2)]
        Gt = [G[i] + alpha * A[i] for i in range(2)]
        M = [mu * M[i] + Gt[i] for i in range(2)]
        nrm = (M[0] ** 2 + M[1] ** 2).sqrt()
        O = [orbit(M[i] / nrm)[-1] for i in range(2)]
        W = [W[i] - eta * (gamma * O[i] + lam * W[i]) for i in range(2)]
        Gp = G
        lines.append(" ".join([str(k)] + [fmt(v) for v in (A + Gt + M + [nrm] + O + W)]))
    open(os.path.join(HERE, "hand_2x2.txt"), "w").write("\n".join(lines) + "\n")


def write_3x2():
    # M = [[1,2],[3,4],[5,6]] through the SVD closed form (library routine: numpy.linalg.svd).
    M = np.array([[1., 2.], [3., 4.], [5., 6.]])
    U, S, Vt = np.linalg.svd(M, full_matrices=False)
    nrm = np.sqrt((M * M).sum())
    sig = S / nrm
    pf = lambda x: float(a) * x + float(b) * x ** 3 + float(c) * x ** 5
    s5 = sig.copy()
    for _ in range(5):
        s5 = pf(s5)
    NS = (U * s5) @ Vt
    UVt = U @ Vt
    # one full step: W_0 = 0.1 * ones, G_1 = M, same hyper-parameters as the 2x2 case, gamma = 0.2 sqrt(3).
    # Step 1 from zero state: A_1 = (1-beta_a) G_1, G~_1 = (1 + alpha (1-beta_a)) G_1 = 0.5 G_1 = M_1,
    # and NS is invariant to positive scaling, so O_1 = NS_5(M).
    eta, lam, gamma = 0.1, 0.1, 0.2 * np.sqrt(3.0)
    W1 = 0.1 * np.ones((3, 2)) - eta * (gamma * NS + lam * 0.1 * np.ones((3, 2)))
    lines = ["# 3x2 case M = [[1,2],[3,4],[5,6]] via the SVD closed form of Eq. newton_schulz",
             "# (NS_T(M) = U diag(p^T(sigma/||M||_F)) V^T).  Rows: normF; sigma/normF (2);",
             "# p^5 of those (2); U V^T (3 rows); NS_5(M) (3 rows); W_1 of a full step of Algorithm 1 with",
             "# W_0 = 0.1*ones, G_1 = M, beta_a=0.9 alpha=-5 mu=0.5 eta=0.1 lambda=0.1 gamma=0.2*sqrt(3) (3 rows)."]
    lines.append(f"{nrm:.13f}")
    lines.append(" ".join(f"{v:.13f}" for v in sig))
    lines.append(" ".join(f"{v:.13f}" for v in s5))
    for blk in (UVt, NS, W1):
        for r in blk:
            lines.append(" ".join(f"{v:.13f}" for v in r))
    open(os.path.join(HERE, "hand_3x2.txt"), "w").write("\n".join(lines) + "\n")


def bf16(x: F) -> F:
    """Nearest number with 8 significant binary digits, ties to the even last digit (exact rationals)."""
    if x == 0:
        return x
    sign = -1 if x < 0 else 1
    x = abs(x)
    e = 0
    while F(2) ** (e + 1) <= x:
        e += 1
    while F(2) ** e > x:
        e -= 1
    unit = F(2) ** (e - 7)              # spacing of 8-bit significands in [2^e, 2^(e+1))
    q = x / unit
    lo = q.numerator // q.denominator
    rem = q - lo
    if rem > F(1, 2) or (rem == F(1, 2) and lo % 2 == 1):
        lo += 1
    return sign * lo * unit


def write_lite_2x2():
    # Lines 4-7 and 10 of Algorithm 1 on diagonal 2x2 matrices with bfloat16 storage of A_k and G_{k-1}:
    # G_1 = diag(0.3, 3), G_2 = diag(0.3, 4); beta_a = 0.9, alpha = -5, mu = 0.5.
    beta, alpha, mu = F(9, 10), F(-5), F(1, 2)
    Gs = [[F(3, 10), F(3)], [F(3, 10), F(4)]]
    A = [F(0), F(0)]; M = [F(0), F(0)]; Gp = [F(0), F(0)]
    lines = ["# MONA-Lite (G_{k-1} and A_k stored in bfloat16: nearest, ties to even; exact rational arithmetic otherwise).",
             "# Two steps of lines 4-7 and 10 of Algorithm 1 on diagonal 2x2 matrices: G_1 = diag(0.3, 3), G_2 = diag(0.3, 4);",
             "# beta_a=0.9 alpha=-5 mu=0.5.  A is rounded when stored and the stored value enters G~; G_prev is the rounded G.",
             "# e.g. bf16(0.3) = 0.30078125, bf16(0.03) = 0.030029296875.",
             "# columns: step  A11 A22  Gt11 Gt22  M11 M22  Gprev11 Gprev22"]
    for k, G in enumerate(Gs, 1):
        Dk = [G[i] - Gp[i] for i in range(2)]
        A = [bf16(beta * A[i] + (1 - beta) * Dk[i]) for i in range(2)]
        Gt = [G[i] + alpha * A[i] for i in range(2)]
        M = [mu * M[i] + Gt[i] for i in range(2)]
        Gp = [bf16(G[i]) for i in range(2)]
        lines.append(" ".join([str(k)] + [f"{float(v):.16f}" for v in (A + Gt + M + Gp)]))
    open(os.path.join(HERE, "hand_lite_2x2.txt"), "w").write("\n".join(lines) + "\n")


if __name__ == "__main__":
    write_orbits(); write_2x2(); write_3x2(); write_lite_2x2()
