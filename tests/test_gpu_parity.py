"""CUDA library against the fp64 oracle, element by element on the same seeded inputs (through the C ABI)."""
import pytest
import torch

import paper_2605_26842_b200 as pkg
from tests.parity_util import (LITE_MAX_FLIPPED, TOL_A_LITE, TOL_M_LITE, TOL_O_BF16, TOL_O_FP32, TOL_O_MAX_BF16,
                               TOL_O_MAX_FP32, TOL_STATE, TOL_STATE_MAX, TOL_W, run_case)

pytestmark = pytest.mark.gpu


def check(errs, tol_o):
    assert errs["M"] <= TOL_STATE and errs["A"] <= TOL_STATE and errs["Gprev"] <= TOL_STATE, errs
    assert errs["O"] <= tol_o, errs
    assert errs["dW"] <= max(TOL_W, tol_o), errs
    # no single element far off (an unwritten or misplaced patch would pass the Frobenius gates)
    assert errs["M_max"] <= TOL_STATE_MAX and errs["A_max"] <= TOL_STATE_MAX and errs["Gprev_max"] <= TOL_STATE_MAX, errs
    assert errs["O_max"] <= (TOL_O_MAX_FP32 if tol_o == TOL_O_FP32 else TOL_O_MAX_BF16), errs


def test_config0_fp32_validation():
    """256x512, 5 steps, fp32 validation Newton-Schulz: O within 1e-4, state within 1e-6."""
    hp = pkg.default_hparams(ns_precision=1)
    errs = run_case([(1, 256, 512)], steps=5, hp=hp, seed=1234)
    check(errs, TOL_O_FP32)


def test_config0_bf16_tensor_cores():
    """256x512, 5 steps, bf16 operands / fp32 accumulate on tcgen05: O within 2e-2."""
    errs = run_case([(1, 256, 512)], steps=5, seed=1234)
    check(errs, TOL_O_BF16)


@pytest.mark.parametrize("shape", [(1, 128, 256), (1, 256, 128), (3, 192, 320), (2, 320, 192), (1, 64, 128),
                                   (2, 512, 1024), (2, 1024, 512), (1, 768, 2048), (1, 2048, 768), (1, 1024, 1024),
                                   (1, 72, 200), (1, 1000, 136), (1, 2816, 1024), (1, 1024, 2816)])
def test_tensor_core_shapes(shape):
    """Wide, tall, square, ragged (not multiples of the 128x256 tile) and stacked shapes on the tcgen05 path."""
    errs = run_case([shape], steps=2, seed=hash(shape) % 1000)
    check(errs, TOL_O_BF16)


@pytest.mark.parametrize("shape", [(1, 128, 256), (2, 320, 192), (1, 40, 72), (1, 33, 17), (1, 32, 1024), (1, 5, 3),
                                   (1, 512, 1024)])
def test_fp32_shapes(shape):
    """fp32 validation mode incl. shapes that never go to the tensor cores (odd sizes, min(m,n) < 64)."""
    hp = pkg.default_hparams(ns_precision=1)
    errs = run_case([shape], steps=3, hp=hp, seed=7)
    check(errs, TOL_O_FP32)


def test_small_and_odd_shapes_in_default_mode():
    """Router-like 32x1024 (shorter side < 64), 33x17 (sides not a multiple of 8) and 8x24 take the fp32 FMA
    path in the default precision mode too: everything still runs on the GPU, to the fp32 tolerance."""
    errs = run_case([(1, 32, 1024), (1, 33, 17), (1, 8, 24)], steps=2, seed=5)
    check(errs, TOL_O_FP32)


def test_mixed_set_ten_steps():
    """A small MoE-like set (stacked experts, attention, router), 10 steps: parameters within 3e-2."""
    shapes = [(4, 256, 512), (4, 512, 256), (1, 512, 512), (1, 32, 512)]
    errs = run_case(shapes, steps=10, seed=42)
    check(errs, TOL_O_BF16)


def test_update_fused_into_the_last_gemm_matches_too():
    """fuse_update = 1: the last X' = B' X applies Eq. muon_update in its epilogue (fp32 O_k from the accumulator)."""
    shapes = [(3, 256, 512), (2, 512, 256), (1, 320, 192)]
    errs = run_case(shapes, steps=3, seed=43, options=pkg.default_options(fuse_update=1))
    check(errs, TOL_O_BF16)
    assert errs["launches"] == 3 * 2        # per chunk: prologue, Newton-Schulz (update inside)


@pytest.mark.parametrize("delay", [1, 2, 7])
def test_work_order_delay_does_not_change_results(delay):
    """ns_delay only moves work items in the kernel's hand-out order: results are bit-identical to the default."""
    dev = torch.device("cuda", 0)
    gen = torch.Generator().manual_seed(19)
    shapes = [(9, 256, 384), (3, 512, 256)]
    W0 = [torch.randn(s, generator=gen) * 0.02 for s in shapes]
    G = [[torch.randn(s, generator=gen) * 1e-3 for s in shapes] for _ in range(2)]
    hp = pkg.default_hparams()

    def run(opts):
        p = [w.clone().to(dev) for w in W0]
        opt = pkg.MonaOptimizer(p, options=opts)
        for k in range(2):
            opt.step(hp, p, [g.to(dev) for g in G[k]])
        torch.cuda.synchronize()
        assert opt.poll_status()[0] == 0
        out = [t.clone() for t in p]
        opt.close()
        return out
    a, b = run(pkg.default_options()), run(pkg.default_options(ns_delay=delay))
    for x, y in zip(a, b):
        assert torch.equal(x, y)


def test_zero_gradient_from_zero_state():
    """M = 0 (zero gradient, zero state): X_0 = 0 / (0 + eps) = 0, so O_k is exactly 0, only weight decay acts,
    W <- (1 - eta lambda) W, and nothing is reported (the norm is finite).  Both Newton-Schulz paths."""
    dev = torch.device("cuda", 0)
    gen = torch.Generator().manual_seed(2)
    shapes = [(2, 256, 384), (1, 384, 256), (1, 32, 256), (1, 33, 17)]
    for precision in (0, 1):
        hp = pkg.default_hparams(ns_precision=precision)
        p = [(torch.randn(s, generator=gen) * 0.02).to(dev) for s in shapes]
        w0 = [t.clone() for t in p]
        g = [torch.zeros(s, device=dev) for s in shapes]
        o = [torch.full(s, 7.0, device=dev) for s in shapes]
        opt = pkg.MonaOptimizer(p)
        opt.step_ex(hp, p, g, o, 7)
        st, bad = opt.poll_status()
        assert st == 0 and bad == -1
        for i in range(len(shapes)):
            assert torch.count_nonzero(o[i]).item() == 0
            for view in opt.state_views(i):
                assert torch.count_nonzero(view).item() == 0
            expect = w0[i].double() * (1.0 - hp.lr * hp.weight_decay)
            assert (p[i].double() - expect).abs().max().item() <= 1e-7 * w0[i].abs().max().item()
        opt.close()


def test_alpha_zero_is_muon():
    """alpha = 0: Algorithm 1 with the acceleration weight switched off must take Muon's steps (M, O, W against the
    oracle's separately written Muon), although A and G_prev still evolve."""
    hp = pkg.default_hparams(accel_alpha=0.0)
    errs = run_case([(2, 256, 384), (1, 384, 128), (1, 40, 72)], steps=4, hp=hp, seed=29, muon=True, compare_aux=False)
    assert errs["M"] <= TOL_STATE and errs["M_max"] <= TOL_STATE_MAX, errs
    assert errs["O"] <= TOL_O_BF16 and errs["O_max"] <= TOL_O_MAX_BF16 and errs["dW"] <= TOL_W, errs


def test_bf16_gradients_and_padding():
    errs = run_case([(3, 128, 384)], steps=3, grad_dtype=torch.bfloat16, pad=64, seed=9)
    check(errs, TOL_O_BF16)


def test_heavy_tailed_gradients():
    hp = pkg.default_hparams(accel_beta=0.98, accel_alpha=-25.0)
    errs = run_case([(2, 384, 512)], steps=4, hp=hp, rho=0.8, heavy_tail=True, seed=11)
    check(errs, TOL_O_BF16)


@pytest.mark.parametrize("T", [0, 1, 2, 4])
def test_ns_step_counts(T):
    hp = pkg.default_hparams(ns_steps=T)
    errs = run_case([(1, 128, 256)], steps=2, hp=hp, seed=3)
    check(errs, TOL_O_BF16)


def test_more_iterations_than_one_launch_holds():
    """T = 7: the Newton-Schulz kernel takes five iterations per launch, so this is two launches per chunk (5 + 2),
    the second continuing on the first one's iterate."""
    hp = pkg.default_hparams(ns_steps=7)
    errs = run_case([(2, 256, 384), (1, 384, 256)], steps=2, hp=hp, seed=8)
    check(errs, TOL_O_BF16)
    assert errs["launches"] == 2 * 4        # per chunk: prologue, two Newton-Schulz launches, update


def test_many_small_matrices_span_several_chunks():
    """600 stacked 64x128 matrices: more than one chunk holds (512), one tile per GEMM and matrix, so the kernel's work
    order and its per-matrix completion counters carry the whole load; a sample is followed by the oracle."""
    errs = run_case([(600, 64, 128)], steps=2, seed=12, sample={0: [0, 1, 255, 511, 512, 599]})
    check(errs, TOL_O_BF16)


def test_a_layer_of_paper_shaped_experts_in_both_orientations():
    """128 + 128 experts of 256 x 768 and 768 x 256 (the expert shape of the paper's smallest model): every product of such
    a matrix is one or three tiles of 4 or 12 k-slices, so the launch is thousands of short items bound by their
    epilogues; sampled matrices are followed by the oracle."""
    errs = run_case([(128, 256, 768), (128, 768, 256)], steps=2, seed=31, sample={0: [0, 63, 127], 1: [0, 64, 127]})
    check(errs, TOL_O_BF16)


def test_fixed_scale_and_other_hyperparameters():
    hp = pkg.default_hparams(scale_mode=1, scale_value=0.37, lr=5e-3, momentum=0.8, weight_decay=0.0,
                             accel_beta=0.9, accel_alpha=-5.0)
    errs = run_case([(1, 256, 256)], steps=3, hp=hp, seed=13)
    check(errs, TOL_O_BF16)


@pytest.mark.parametrize("shapes,grad_dtype,steps", [([(1, 256, 512)], torch.float32, 5), ([(2, 512, 256), (1, 32, 1024)], torch.float32, 10),
                                                     ([(3, 128, 384)], torch.bfloat16, 4), ([(1, 33, 17)], torch.float32, 3)])
def test_mona_lite_state_storage(shapes, grad_dtype, steps):
    """MONA-Lite: A_k and G_{k-1} stored in bfloat16.  G_prev must equal the oracle's bit for bit (with
    bfloat16 gradients it is the gradient itself); A may sit one bfloat16 step away on a small fraction of
    the elements (the value that is rounded is formed in fp32 here and in fp64 in the oracle), never more."""
    errs = run_case(shapes, steps=steps, grad_dtype=grad_dtype, seed=21, lite=True)
    assert errs["Gprev_exact"], errs
    # a disagreement is made of roundings that went the other way: at most one fresh bfloat16 step per step taken
    # (measured at the scale of the EMA's operands), on a small fraction of the elements
    assert errs["A_worst_steps"] <= steps + 1 and errs["A_flipped"] <= LITE_MAX_FLIPPED, errs
    assert errs["A"] <= TOL_A_LITE and errs["M"] <= TOL_M_LITE, errs
    assert errs["O"] <= TOL_O_BF16 and errs["dW"] <= TOL_W, errs


@pytest.mark.parametrize("shape", [(3, 256, 768), (3, 768, 256), (1, 1024, 1536), (1, 1536, 1024), (1, 1024, 3072),
                                   (1, 3072, 1024)])
def test_paper_expert_shapes(shape):
    """Expert matrices of the paper's three models (FFN width x hidden and its transpose)."""
    errs = run_case([shape], steps=2, seed=31)
    check(errs, TOL_O_BF16)


@pytest.mark.parametrize("shapes,grad_dtype,steps", [([(1, 256, 512)], torch.float32, 5), ([(2, 512, 256), (1, 32, 1024), (1, 33, 17)], torch.float32, 10),
                                                     ([(3, 128, 384)], torch.bfloat16, 4)])
def test_single_buffer_state_format(shapes, grad_dtype, steps):
    """state_dtype = MONA_STATE_COMBINED: one fp32 buffer Z_k = beta_a A_k - (1 - beta_a) G_k instead of A_k and
    G_{k-1}.  Same step as Algorithm 1: M, O and W against the oracle as usual, Z against the same combination
    of the oracle's A_k and G_k, all to the fp32 state tolerance."""
    errs = run_case(shapes, steps=steps, grad_dtype=grad_dtype, seed=23, combined=True)
    assert errs["M"] <= TOL_STATE and errs["A"] <= TOL_STATE, errs
    assert errs["O"] <= TOL_O_BF16 and errs["dW"] <= TOL_W, errs


def test_plain_muon_path():
    """algorithm = 1: Eq. muon_momentum without the acceleration term; A and G_prev are neither read nor written
    (they stay at their initial zero, so their error against the oracle's untouched zero state is exactly 0)."""
    hp = pkg.default_hparams(algorithm=1)
    errs = run_case([(2, 256, 384), (1, 384, 128), (1, 40, 72)], steps=4, hp=hp, seed=17, muon=True)
    assert errs["A"] == 0.0 and errs["Gprev"] == 0.0, errs
    check(errs, TOL_O_BF16)


def test_nonfinite_gradient_is_reported():
    dev = torch.device("cuda", 0)
    p = [torch.zeros(2, 128, 128, device=dev), torch.zeros(1, 64, 64, device=dev)]
    g = [torch.full((2, 128, 128), 1e-3, device=dev), torch.full((1, 64, 64), 1e-3, device=dev)]
    g[0][1, 5, 7] = float("nan")
    opt = pkg.MonaOptimizer(p)
    opt.step(pkg.default_hparams(), p, g)
    st, bad = opt.poll_status()
    assert pkg.STATUS_NAMES[st] == "MONA_ERR_NONFINITE" and bad == 1
    st, bad = opt.poll_status()          # the word is cleared by the first poll
    assert st == 0 and bad == -1
    opt.close()


def test_argument_errors_on_device():
    dev = torch.device("cuda", 0)
    p = [torch.zeros(1, 64, 64, device=dev)]
    g = [torch.zeros(1, 64, 64, device=dev)]
    opt = pkg.MonaOptimizer(p)
    hp = pkg.default_hparams()
    with pytest.raises(pkg.MonaError) as e:
        opt.step(hp, p, [None])
    assert e.value.status == 1
    mis = torch.zeros(64 * 64 + 1, device=dev)[1:].view(1, 64, 64)
    with pytest.raises(pkg.MonaError) as e:
        opt.step(hp, p, [mis])
    assert e.value.status == 3
    with pytest.raises(pkg.MonaError) as e:
        opt.step(pkg.default_hparams(ns_precision=5), p, g)
    assert e.value.status == 1
    opt.close()


def test_deterministic_and_resumable():
    """Same inputs give bit-identical state and parameters; 4 steps equal 2 + checkpoint/restore + 2."""
    dev = torch.device("cuda", 0)
    gen = torch.Generator().manual_seed(5)
    shapes = [(3, 256, 384), (1, 384, 256)]
    W0 = [torch.randn(s, generator=gen) * 0.02 for s in shapes]
    G = [[torch.randn(s, generator=gen) * 1e-3 for s in shapes] for _ in range(4)]
    hp = pkg.default_hparams()

    def run(split):
        p = [w.clone().to(dev) for w in W0]
        opt = pkg.MonaOptimizer(p)
        for k in range(4):
            if split and k == 2:
                saved = opt.state.clone()
                opt.close()
                opt = pkg.MonaOptimizer(p)
                opt.state.copy_(saved)
            opt.step(hp, p, [g.to(dev) for g in G[k]])
        torch.cuda.synchronize()
        out = [t.clone() for t in p] + [opt.state.clone()]
        opt.close()
        return out

    a, b, c = run(False), run(False), run(True)
    for x, y, z in zip(a, b, c):
        assert torch.equal(x, y) and torch.equal(x, z)


def test_step_host_matches_step_and_returns_parameters():
    """mona_step_host (pinned host gradients in, parameters out, transfers pipelined with the chunks) gives
    bit-identical parameters and state to mona_step on the same inputs, and the host copy equals the device's.
    A small chunk budget makes descriptors straddle chunks and both workspace slots take part."""
    dev = torch.device("cuda", 0)
    gen = torch.Generator().manual_seed(77)
    shapes = [(5, 256, 384), (5, 256, 384), (3, 384, 256), (1, 32, 256)]
    W0 = [torch.randn(s, generator=gen) * 0.02 for s in shapes]
    G = [[torch.randn(s, generator=gen) * 1e-3 for s in shapes] for _ in range(3)]
    hp = pkg.default_hparams()
    pkg.set_chunk_budget(2 << 20)            # 3 matrices of 256x384 per chunk
    try:
        def run(host):
            p = [w.clone().to(dev) for w in W0]
            opt = pkg.MonaOptimizer(p)
            g_dev = [torch.zeros_like(w, device=dev) for w in W0]
            g_host = [torch.empty(s, pin_memory=True) for s in shapes]
            p_host = [torch.zeros(s, pin_memory=True) for s in shapes]
            for k in range(3):
                if host:
                    for h_, g in zip(g_host, G[k]):
                        h_.copy_(g)
                    opt.step_host(hp, p, g_dev, g_host, p_host)
                    torch.cuda.synchronize()
                    for ph, pd in zip(p_host, p):
                        assert torch.equal(ph, pd.cpu())
                else:
                    opt.step(hp, p, [g.to(dev) for g in G[k]])
            torch.cuda.synchronize()
            assert opt.poll_status()[0] == 0
            out = [t.clone() for t in p] + [opt.state.clone()]
            opt.close()
            return out
        a, b = run(False), run(True)
        for x, y in zip(a, b):
            assert torch.equal(x, y)
    finally:
        pkg.set_chunk_budget(768 << 20)


def test_chunk_overlap_does_not_change_results():
    """Two chunks in flight on two streams (default) and everything on the caller's stream give bit-identical
    parameters and state."""
    dev = torch.device("cuda", 0)
    gen = torch.Generator().manual_seed(9)
    shapes = [(7, 256, 384), (2, 384, 256), (1, 512, 512)]
    W0 = [torch.randn(s, generator=gen) * 0.02 for s in shapes]
    G = [[torch.randn(s, generator=gen) * 1e-3 for s in shapes] for _ in range(3)]
    hp = pkg.default_hparams()
    pkg.set_chunk_budget(2 << 20)
    try:
        def run(overlap):
            pkg.set_chunk_overlap(overlap)
            p = [w.clone().to(dev) for w in W0]
            opt = pkg.MonaOptimizer(p)
            for k in range(3):
                opt.step(hp, p, [g.to(dev) for g in G[k]])
            torch.cuda.synchronize()
            out = [t.clone() for t in p] + [opt.state.clone()]
            opt.close()
            return out
        a, b = run(True), run(False)
        for x, y in zip(a, b):
            assert torch.equal(x, y)
    finally:
        pkg.set_chunk_overlap(True)
        pkg.set_chunk_budget(768 << 20)


def test_a_wait_that_cannot_end_times_out_and_the_handle_survives():
    """Failure detection without a fault: a launch whose stages expect bytes that never come must give up after its
    bounded wait, report MONA_ERR_TIMEOUT through the status word, release tensor memory and leave the context
    usable - the next step on the same handle is correct."""
    import time
    dev = torch.device("cuda", 0)
    gen = torch.Generator().manual_seed(3)
    p = [(torch.randn(1, 256, 512, generator=gen) * 0.02).to(dev)]
    g = [(torch.randn(1, 256, 512, generator=gen) * 1e-3).to(dev)]
    opt = pkg.MonaOptimizer(p)
    t0 = time.time()
    opt.selftest_timeout()
    st, bad = opt.poll_status()
    assert pkg.STATUS_NAMES[st] == "MONA_ERR_TIMEOUT", (st, bad)
    assert time.time() - t0 < 20.0
    assert opt.poll_status()[0] == 0                 # latched once, then cleared
    opt.close()
    # same device, fresh handle and a full parity case: nothing was left behind
    errs = run_case([(1, 256, 512)], steps=2, seed=5)
    check(errs, TOL_O_BF16)
