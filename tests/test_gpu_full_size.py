"""Parity at benchmark scale, in the launch configuration bench.py times: one layer of the ~7B MoE set
(64 + 64 wide 768x2048 experts, 64 tall 2048x768 experts, four 2048x2048 attention matrices, one 1536x2048
shared expert; 322 M parameters), default chunk budget (chunks of 93 + 35 wide experts), two chunks in flight.
The oracle follows a sample of the matrices (first, last, one inside each chunk) through every step; the
library processes all of them."""
import pytest

import paper_2605_26842_b200 as pkg
from paper_2605_26842_b200 import synth
from tests.parity_util import TOL_O_BF16, TOL_O_MAX_BF16, TOL_STATE, TOL_STATE_MAX, TOL_W, run_case

pytestmark = pytest.mark.gpu


def test_one_layer_of_the_7b_set_sampled():
    wl = synth.workload(3, layers=1)
    shapes = [(s.batch, s.rows, s.cols) for s in wl.specs]
    assert shapes[:3] == [(64, 768, 2048), (64, 768, 2048), (64, 2048, 768)]
    # w1: first matrix and one in the middle of the first chunk; w3: index 28 is the last matrix of the first
    # 93-matrix chunk, 29 the first of the second, 63 the last; w2 (tall): first and last; every attention
    # matrix's bucket through one of them; the shared expert
    sample = {0: [0, 37], 1: [28, 29, 63], 2: [0, 63], 3: [0], 6: [0], 7: [0]}
    hp = pkg.default_hparams(accel_beta=wl.accel_beta, accel_alpha=wl.accel_alpha)
    errs = run_case(shapes, steps=2, hp=hp, rho=wl.rho, sigma=wl.sigma, seed=wl.seed, sample=sample)
    assert errs["M"] <= TOL_STATE and errs["A"] <= TOL_STATE and errs["Gprev"] <= TOL_STATE, errs
    assert errs["O"] <= TOL_O_BF16 and errs["dW"] <= TOL_W, errs
    # buckets: 128 wide experts (2 chunks), 64 tall experts, 4 attention matrices, 1 shared expert: 5 chunks,
    # each one prologue + one Newton-Schulz launch (all 15 GEMMs) + one update
    assert errs["launches"] == 5 * 3, errs["launches"]


def test_one_layer_of_the_7b_set_ten_steps():
    """The "parameters after 10 steps" clause at benchmark scale: the same one-layer set, ten steps, a sample of
    matrices from every bucket followed by the oracle throughout and compared after step 10."""
    wl = synth.workload(3, layers=1)
    shapes = [(s.batch, s.rows, s.cols) for s in wl.specs]
    sample = {0: [37], 1: [28, 29], 2: [63], 3: [0], 7: [0]}
    hp = pkg.default_hparams(accel_beta=wl.accel_beta, accel_alpha=wl.accel_alpha)
    errs = run_case(shapes, steps=10, hp=hp, rho=wl.rho, sigma=wl.sigma, seed=wl.seed + 1, sample=sample, heavy_tail=True, check_at={10})
    assert errs["M"] <= TOL_STATE and errs["A"] <= TOL_STATE and errs["Gprev"] <= TOL_STATE, errs
    assert errs["M_max"] <= TOL_STATE_MAX and errs["A_max"] <= TOL_STATE_MAX, errs
    assert errs["O"] <= TOL_O_BF16 and errs["O_max"] <= TOL_O_MAX_BF16 and errs["dW"] <= TOL_W, errs


def test_shard_stress_shapes_with_bf16_gradients():
    """The shapes of the large-MoE shard configuration (1024x4096 experts wide and tall, 4096x4096 attention),
    bfloat16 gradients, its beta_a = 0.975 / alpha = -20: two steps, every matrix followed by the oracle."""
    import torch
    hp = pkg.default_hparams(accel_beta=0.975, accel_alpha=-20.0)
    errs = run_case([(2, 1024, 4096), (1, 4096, 1024), (1, 4096, 4096)], steps=2, hp=hp, grad_dtype=torch.bfloat16, seed=1238)
    assert errs["M"] <= TOL_STATE and errs["A"] <= TOL_STATE and errs["Gprev"] <= TOL_STATE, errs
    assert errs["O"] <= TOL_O_BF16 and errs["dW"] <= TOL_W, errs
