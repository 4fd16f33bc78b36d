"""Plain fp64 CPU oracle for the MONA matrix-optimizer step.

TEST INFRASTRUCTURE ONLY.  This module is the slow, obviously-correct statement of what the
optimizer step computes.  It is imported by the tests, by the smoke check and by the benchmark's
CPU-baseline leg, never by the product path, and it shares no code with the CUDA library.

Everything is float64 numpy.  Each function follows the paper step by step, in the paper's
notation, with no blocking, fusion or reordering:

  * Algorithm 1 (MONA Optimizer)            -> OracleState, mona_step
  * Eq. alto_diff / alto_accel / alto_grad  -> acceleration(): D_k, A_k, G~_k
  * Eq. muon_momentum                       -> momentum(): M_k = mu M_{k-1} + G~_k
  * Eq. newton_schulz                       -> newton_schulz(): X_0 = M/||M||_F, quintic iteration
  * gamma = 0.2 sqrt(max(m, n))             -> update_scale()
  * Eq. muon_update                         -> apply_update(): W <- W - eta (gamma O + lambda W)
  * plain Muon, the baseline (Eq. muon_momentum, muon_ns, muon_update)        -> muon_step()
  * MONA-Lite (section "Efficient Deployment with Reduced Overhead"): G_{k-1} and A_k kept in
    bfloat16, equations unchanged          -> round_bf16(), Hyper.state_dtype = "bf16"

Readings taken where the paper is silent (all are arguments, none is hidden):
  * First step: G_0 = 0 (Algorithm 1, line 1), so D_1 = G_1.
  * Momentum is the literal heavy-ball form of Eq. muon_momentum: no (1 - mu) factor, no look-ahead.
  * X_0 = M / (||M||_F + eps); the paper has no eps, so eps is an argument (default 1e-7) and
    M = 0 gives O = 0.
  * The iteration is applied to the m x n matrix as written, never transposed.
  * gamma uses max(m, n) of the individual matrix.
  * Weight decay sits inside the eta bracket and uses W_k (the value before the update).
  * MONA-Lite: the paper only says the two buffers are stored in bfloat16.  Taken here as: A_k is
    formed in full precision, rounded once (nearest, ties to even) when it is stored, and the stored
    value is the one G~_k uses, so that the state alone determines the next step; G_{k-1} is the
    rounded G_k.  M_k and everything downstream stay in full precision.

Every function here is pinned by tests that do not call it to produce their expected value
(closed forms, scalar hand arithmetic, a library SVD, invariants); nothing is "parity unpinned".
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

# Coefficients printed under Eq. newton_schulz.
NS_A = 3.4445
NS_B = -4.7750
NS_C = 2.0315


@dataclass
class Hyper:
    """REQUIRE line of Algorithm 1: eta, mu, (beta_a, alpha), lambda, T, gamma (rule or value)."""
    lr: float = 1e-3             # eta
    momentum: float = 0.95       # mu
    accel_beta: float = 0.99     # beta_a
    accel_alpha: float = -50.0   # alpha
    weight_decay: float = 0.1    # lambda
    ns_steps: int = 5            # T
    ns_a: float = NS_A
    ns_b: float = NS_B
    ns_c: float = NS_C
    norm_eps: float = 1e-7
    scale_mode: int = 0          # 0: gamma = scale_value * sqrt(max(m, n)); 1: gamma = scale_value
    scale_value: float = 0.2
    state_dtype: str = "fp32"    # "bf16": MONA-Lite, G_{k-1} and A_k stored in bfloat16


class OracleState:
    """Algorithm 1, line 1: M_0 = 0, A_0 = 0, G_0 = 0 for one m x n matrix."""

    def __init__(self, m: int, n: int):
        self.M = np.zeros((m, n), dtype=np.float64)
        self.A = np.zeros((m, n), dtype=np.float64)
        self.G_prev = np.zeros((m, n), dtype=np.float64)

    def copy(self) -> "OracleState":
        s = OracleState(*self.M.shape)
        s.M, s.A, s.G_prev = self.M.copy(), self.A.copy(), self.G_prev.copy()
        return s


def round_bf16(x):
    """Value of x after storage in bfloat16 (1 sign, 8 exponent, 7 fraction bits): the nearest
    representable number, ties to the even fraction.  Done on the bit pattern of the float32 value,
    of which a bfloat16 is the upper half."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = u + 0x7FFF + ((u >> 16) & 1)
    return ((u >> 16) << 16).astype(np.uint32).view(np.float32).astype(np.float64)


def keep(x):
    """Full-precision storage."""
    return x


def acceleration(G, G_prev, A_prev, beta_a, alpha, store=keep):
    """Eq. alto_diff, alto_accel, alto_grad (Algorithm 1, lines 4-6).  `store` is the storage format
    of A_k (identity, or round_bf16 for MONA-Lite)."""
    D = G - G_prev
    A = store(beta_a * A_prev + (1.0 - beta_a) * D)
    G_tilde = G + alpha * A
    return A, G_tilde


def momentum(M_prev, G_tilde, mu):
    """Eq. muon_momentum with G~ in place of G (Algorithm 1, line 7)."""
    return mu * M_prev + G_tilde


def newton_schulz(M, T=5, a=NS_A, b=NS_B, c=NS_C, eps=1e-7):
    """Eq. newton_schulz: X_0 = M / ||M||_F, then T times
    X <- a X + b X X^T X + c X X^T X X^T X, products taken left to right as printed."""
    M = np.asarray(M, dtype=np.float64)
    X = M / (np.linalg.norm(M, "fro") + eps)
    for _ in range(T):
        Xt = X.T
        X = a * X + b * (X @ Xt @ X) + c * (X @ Xt @ X @ Xt @ X)
    return X


def update_scale(m, n, scale_mode=0, scale_value=0.2):
    """gamma = 0.2 sqrt(max(m, n)) (the RMS-matching rule), or a fixed value when overridden."""
    if scale_mode == 0:
        return scale_value * float(np.sqrt(max(m, n)))
    return float(scale_value)


def apply_update(W, O, lr, gamma, weight_decay):
    """Eq. muon_update (Algorithm 1, line 9): W_{k+1} = W_k - eta (gamma O_k + lambda W_k)."""
    return W - lr * (gamma * O + weight_decay * W)


def mona_step(W, G, state: OracleState, hp: Hyper):
    """One pass of the loop body of Algorithm 1 for one matrix.

    W, G are m x n arrays (any float dtype; widened to float64).  `state` is updated in place.
    Returns (W_next, O) as float64 arrays."""
    W = np.asarray(W, dtype=np.float64)
    G = np.asarray(G, dtype=np.float64)
    store = round_bf16 if hp.state_dtype == "bf16" else keep
    A, G_tilde = acceleration(G, state.G_prev, state.A, hp.accel_beta, hp.accel_alpha, store)
    M = momentum(state.M, G_tilde, hp.momentum)
    O = newton_schulz(M, hp.ns_steps, hp.ns_a, hp.ns_b, hp.ns_c, hp.norm_eps)
    gamma = update_scale(W.shape[0], W.shape[1], hp.scale_mode, hp.scale_value)
    W_next = apply_update(W, O, hp.lr, gamma, hp.weight_decay)
    state.A = A
    state.M = M
    state.G_prev = store(G.copy())   # Algorithm 1, line 10
    return W_next, O


def muon_step(W, G, state: OracleState, hp: Hyper):
    """One step of plain Muon for one matrix, the baseline the paper compares with:
    Eq. muon_momentum M_k = mu M_{k-1} + G_k, Eq. muon_ns O_k = NewtonSchulz(M_k, T), Eq. muon_update.
    Only state.M is used and updated."""
    W = np.asarray(W, dtype=np.float64)
    G = np.asarray(G, dtype=np.float64)
    M = momentum(state.M, G, hp.momentum)
    O = newton_schulz(M, hp.ns_steps, hp.ns_a, hp.ns_b, hp.ns_c, hp.norm_eps)
    gamma = update_scale(W.shape[0], W.shape[1], hp.scale_mode, hp.scale_value)
    W_next = apply_update(W, O, hp.lr, gamma, hp.weight_decay)
    state.M = M
    return W_next, O
