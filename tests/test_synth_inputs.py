"""The synthetic gradient process has the statistics the benchmark recipe states: zero mean, variance sigma^2,
lag-1 autocorrelation rho, for both noise families (normal; Student-t with 4 degrees of freedom scaled to unit
variance).  Runs on the CPU: the generator is plain torch and device-agnostic."""
import math

import pytest
import torch

from paper_2605_26842_b200 import synth


@pytest.mark.parametrize("dist,rho,dtype", [("normal", 0.9, torch.float32), ("student_t4", 0.8, torch.float32),
                                            ("normal", 0.9, torch.bfloat16)])
def test_gradient_process_moments(dist, rho, dtype):
    sigma = 1e-3
    wl = synth.Workload("stat", [synth.MatrixSpec("w", 512, 1024, 2)], steps=4, rho=rho, sigma=sigma, dist=dist,
                        grad_dtype=dtype, seed=77)
    gp = synth.GradientProcess(wl, "cpu")
    n = wl.n_params
    prev = None
    for k in range(4):
        g = gp.next()[0].float().flatten().double()
        mean, var = g.mean().item(), g.var().item()
        # standard errors: mean sigma / sqrt(n); variance sigma^2 sqrt((kurtosis - 1) / n).  Student-t(4) has no finite
        # fourth moment, so its sample variance converges slowly: a wider band there
        assert abs(mean) <= 6 * sigma / math.sqrt(n), (k, mean)
        band = 0.02 if dist == "normal" else 0.15
        if dtype == torch.bfloat16:
            band += 0.01        # rounding to 8 significant bits adds ~2^-18 relative variance, and a little bias
        assert abs(var / sigma ** 2 - 1.0) <= band, (k, var)
        if prev is not None:
            corr = ((g - g.mean()) * (prev - prev.mean())).mean().item() / math.sqrt(var * prev.var().item())
            assert abs(corr - rho) <= (0.01 if dist == "normal" else 0.05), (k, corr)
        prev = g


def test_student_t_noise_is_heavy_tailed():
    wl = synth.Workload("stat", [synth.MatrixSpec("w", 1024, 1024)], steps=1, dist="student_t4", seed=5)
    gp = synth.GradientProcess(wl, "cpu")
    g = gp.next()[0].flatten().double() / wl.sigma
    # P(|t_4| / sqrt(2) > 5) = P(|t_4| > 7.07) ~ 2.1e-3; a unit normal would give 5.7e-7
    frac = (g.abs() > 5).double().mean().item()
    assert 1e-3 < frac < 4e-3, frac


def test_initial_weights_and_config_shapes():
    wl = synth.workload(3, layers=1)
    assert [(s.batch, s.rows, s.cols) for s in wl.specs[:3]] == [(64, 768, 2048), (64, 768, 2048), (64, 2048, 768)]
    assert wl.accel_alpha == pytest.approx(-25.0)
    small = synth.Workload("w", [synth.MatrixSpec("w", 256, 512, 4)], steps=1)
    w = synth.init_params(small, "cpu")[0]
    assert abs(w.mean().item()) < 3e-4 and abs(w.std().item() / 0.02 - 1.0) < 0.01
