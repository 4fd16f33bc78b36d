"""Plants plausible mistakes in copies of the oracle (on the CPU) and requires the pin checks to
catch every one of them: a dropped term, a wrong sign, a stale operand, a misplaced factor."""
import inspect
import sys
import types

import pytest

import oracle.mona_oracle as orc
from tests import oracle_pins

MUTATIONS = {
    "diff_sign": ("D = G - G_prev", "D = G_prev - G"),
    "ema_missing_one_minus_beta": ("(1.0 - beta_a) * D", "D"),
    "ema_swapped_weights": ("beta_a * A_prev + (1.0 - beta_a) * D", "(1.0 - beta_a) * A_prev + beta_a * D"),
    "accel_sign": ("G_tilde = G + alpha * A", "G_tilde = G - alpha * A"),
    "accel_stale_A": ("G_tilde = G + alpha * A", "G_tilde = G + alpha * A_prev"),
    "momentum_dampened": ("return mu * M_prev + G_tilde", "return mu * M_prev + (1.0 - mu) * G_tilde"),
    "momentum_ignores_accel": ("M = momentum(state.M, G_tilde, hp.momentum)", "M = momentum(state.M, G, hp.momentum)"),
    "accel_after_orthogonalisation": ("    gamma = update_scale(", "    O = O + hp.accel_alpha * A\n    gamma = update_scale("),
    "ns_drop_quintic_term": (" + c * (X @ Xt @ X @ Xt @ X)", ""),
    "ns_swap_b_c": ("b * (X @ Xt @ X) + c *", "c * (X @ Xt @ X) + b *"),
    "ns_one_iteration_short": ("for _ in range(T):", "for _ in range(T - 1):"),
    "ns_no_normalisation": ('X = M / (np.linalg.norm(M, "fro") + eps)', "X = M / (1.0 + eps)"),
    "ns_spectral_norm": ('np.linalg.norm(M, "fro")', "np.linalg.norm(M, 2)"),
    "ns_gram_on_wrong_side": ("b * (X @ Xt @ X)", "b * (X @ X @ Xt)"),
    "scale_uses_min": ("np.sqrt(max(m, n))", "np.sqrt(min(m, n))"),
    "decay_outside_lr": ("W - lr * (gamma * O + weight_decay * W)", "W - lr * gamma * O - weight_decay * W"),
    "update_sign": ("W - lr * (gamma * O + weight_decay * W)", "W + lr * (gamma * O + weight_decay * W)"),
    "decay_sign": ("gamma * O + weight_decay * W", "gamma * O - weight_decay * W"),
    "prev_grad_not_stored": ("state.G_prev = store(G.copy())", "pass"),
    "lite_accel_uses_unrounded_A": ("    A = store(beta_a * A_prev + (1.0 - beta_a) * D)\n    G_tilde = G + alpha * A\n    return A, G_tilde",
                                    "    A = beta_a * A_prev + (1.0 - beta_a) * D\n    G_tilde = G + alpha * A\n    return store(A), G_tilde"),
    "lite_prev_grad_not_rounded": ("state.G_prev = store(G.copy())", "state.G_prev = G.copy()"),
    "lite_momentum_rounded_too": ("    state.M = M\n", "    state.M = store(M)\n"),
    "lite_round_truncates": ("u = u + 0x7FFF + ((u >> 16) & 1)", "u = u + 0"),
    "muon_step_forgets_momentum": ("    state.M = M\n    return W_next, O\n", "    return W_next, O\n"),
    "muon_step_adds_acceleration": ("    M = momentum(state.M, G, hp.momentum)\n    O = newton_schulz(M, hp.ns_steps", "    M = momentum(state.M, G + hp.accel_alpha * (1.0 - hp.accel_beta) * G, hp.momentum)\n    O = newton_schulz(M, hp.ns_steps"),
    "lite_round_half_up": ("u = u + 0x7FFF + ((u >> 16) & 1)", "u = u + 0x8000"),
    "state_M_not_stored": ("state.M = M\n", "pass\n"),
    "coefficient_a": ("NS_A = 3.4445", "NS_A = 3.4454"),
    "coefficient_c": ("NS_C = 2.0315", "NS_C = 2.0351"),
}


def _mutant(old, new):
    src = inspect.getsource(orc)
    assert src.count(old) >= 1, f"mutation target not found: {old!r}"
    mod = types.ModuleType("oracle_mutant")
    sys.modules["oracle_mutant"] = mod        # dataclasses looks the defining module up by name
    exec(compile(src.replace(old, new), "oracle_mutant", "exec"), mod.__dict__)
    return mod


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(name):
    mod = _mutant(*MUTATIONS[name])
    caught = []
    for check in oracle_pins.ALL_CHECKS:
        try:
            check(mod)
        except Exception as exc:          # assertion, shape error, ...: all count as "caught"
            caught.append(check.__name__)
    assert caught, f"no pin check notices the planted mistake {name!r}"
