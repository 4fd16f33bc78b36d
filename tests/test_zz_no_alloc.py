"""The allocation-free prologue entry point, through the C ABI: against the fp64 oracle's acceleration and
momentum steps, and against the handle-based prologue, on two calls in a row.

Collected last on purpose (file name): a run that stops at the first failure has then already run
every other test.  It must pass alone in a fresh process and after the rest of the suite, so it makes
no assumption about what the library's built-in scratch array holds when it starts.

Why the entry point exists: some users of the library cannot allocate device memory at call time
(their framework's allocator owns the whole GPU, or they run where cudaMalloc's device-wide stall is
not allowed), so the small reduction scratch lives inside the library instead of in a workspace."""
import numpy as np
import pytest
import torch

import oracle.mona_oracle as orc
import paper_2605_26842_b200 as pkg

pytestmark = pytest.mark.gpu

TOL_STATE = 1e-6


def rel(a, b):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    n = np.linalg.norm(b)
    return np.linalg.norm(a - b) / n if n > 0 else np.linalg.norm(a - b)


# shapes: a benchmark expert; ragged; tiny with an element count that is not a multiple of 4 (scalar path), in fp32 and
# with bfloat16 gradients; bfloat16 gradients on the vector path; just above 4 Mi elements (slab length grows past 16 Ki);
# exactly the 16 Mi-element limit
@pytest.mark.parametrize("shape,dtype", [((768, 2048), torch.float32), ((1000, 136), torch.float32),
                                         ((33, 17), torch.float32), ((33, 17), torch.bfloat16),
                                         ((512, 1024), torch.bfloat16), ((2056, 2048), torch.float32),
                                         ((4096, 4096), torch.float32)])
def test_noalloc_prologue_matches_oracle_and_handle_prologue_twice_in_a_row(shape, dtype):
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    gen = torch.Generator().manual_seed(321)
    hp = pkg.default_hparams(accel_beta=0.98, accel_alpha=-25.0)
    W = torch.zeros((1,) + shape, device=dev)
    opt = pkg.MonaOptimizer([W], grad_dtype=dtype)
    M = torch.zeros(shape, device=dev)
    A = torch.zeros(shape, device=dev)
    Gp = torch.zeros(shape, device=dev)
    inv = torch.full((1,), -1.0, device=dev)
    xhat = torch.zeros(shape, dtype=torch.bfloat16, device=dev)
    M_ref, A_ref, G_ref = (np.zeros(shape) for _ in range(3))
    for call in range(2):                      # two calls in a row: the second starts from the first's state
        g = (torch.randn(shape, generator=gen) * 1e-3).to(dtype)
        g_dev = g.to(dev)
        opt.step_ex(hp, [W], [g_dev.view((1,) + shape)], None, 1)      # existing entry point, prologue phase only
        pkg.prologue_noalloc(g_dev, M, A, Gp, inv, hp, xhat)
        torch.cuda.synchronize()
        # the paper's equations in fp64 on the same bits (Algorithm 1, lines 4-7 and 10)
        G = g.double().numpy()
        A_ref, G_tilde = orc.acceleration(G, G_ref, A_ref, hp.accel_beta, hp.accel_alpha)
        M_ref = orc.momentum(M_ref, G_tilde, hp.momentum)
        G_ref = G
        for name, got, ref in (("M", M, M_ref), ("A", A, A_ref), ("G_prev", Gp, G_ref)):
            assert rel(got.cpu().numpy(), ref) <= TOL_STATE, (call, name)
        nrm = float(np.linalg.norm(M_ref))
        assert abs(inv.item() * (nrm + hp.norm_eps) - 1.0) <= 1e-6, (call, inv.item(), nrm)
        assert torch.equal(xhat, M.to(torch.bfloat16))
        # and the handle-based prologue on the same inputs
        Mr, Ar, Gr = (t[0] for t in opt.state_views(0))
        for got, ref in ((M, Mr), (A, Ar), (Gp, Gr)):
            assert rel(got.cpu().numpy(), ref.cpu().numpy()) <= TOL_STATE, call
    st, bad = opt.poll_status()
    assert st == 0
    opt.close()


def test_noalloc_prologue_reports_a_nonfinite_norm_through_its_result():
    """There is no status word on this path: a nan gradient must leave a nan (or zero) reciprocal norm, and the next
    call on clean inputs must be unaffected by what the scratch array kept."""
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    hp = pkg.default_hparams()
    shape = (64, 96)
    M, A, Gp = (torch.zeros(shape, device=dev) for _ in range(3))
    inv = torch.full((1,), 3.0, device=dev)
    g = torch.full(shape, 1e-3, device=dev)
    g[5, 7] = float("nan")
    pkg.prologue_noalloc(g, M, A, Gp, inv, hp)
    torch.cuda.synchronize()
    assert not (np.isfinite(inv.item()) and inv.item() > 0.0)
    M, A, Gp = (torch.zeros(shape, device=dev) for _ in range(3))
    g = torch.full(shape, 1e-3, device=dev)
    pkg.prologue_noalloc(g, M, A, Gp, inv, hp)
    torch.cuda.synchronize()
    # G~ = (1 + alpha (1 - beta_a)) g = g / 2 with the default alpha = -1 / (2 (1 - beta_a))
    expect = 1.0 / (0.5e-3 * np.sqrt(shape[0] * shape[1]) + hp.norm_eps)
    assert abs(inv.item() / expect - 1.0) <= 1e-5


def test_noalloc_prologue_refuses_oversized_and_bad_arguments():
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    hp = pkg.default_hparams()
    small = torch.zeros(8, 8, device=dev)
    inv = torch.zeros(1, device=dev)

    class Shaped:            # a stand-in that reports a huge shape without owning that much memory
        def __init__(self, t, shape):
            self.t, self.shape, self.dtype = t, shape, t.dtype

        def data_ptr(self):
            return self.t.data_ptr()

    with pytest.raises(pkg.MonaError) as e:
        pkg.prologue_noalloc(Shaped(small, (8192, 4096)), small, small, small, inv, hp)
    assert e.value.status == 2 and "16777216" in str(e.value)
    with pytest.raises(pkg.MonaError) as e:
        pkg.prologue_noalloc(Shaped(small, (4097, 4096)), small, small, small, inv, hp)     # one row over the limit
    assert e.value.status == 2
    with pytest.raises(pkg.MonaError) as e:
        pkg.prologue_noalloc(Shaped(small, (0, 4)), small, small, small, inv, hp)
    assert e.value.status == 1
    mis = torch.zeros(65, device=dev)[1:].view(8, 8)
    with pytest.raises(pkg.MonaError) as e:
        pkg.prologue_noalloc(mis, small, small, small, inv, hp)
    assert e.value.status == 3
    with pytest.raises(pkg.MonaError) as e:
        pkg.prologue_noalloc(small, small, small, small, inv, pkg.default_hparams(algorithm=1))
    assert e.value.status == 1
