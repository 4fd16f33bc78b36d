"""The allocation-free prologue entry point against the handle-based prologue, through the C ABI.

Collected last on purpose (file name): a run that stops at the first failure has then already run
every other test.  It must pass alone in a fresh process and after the rest of the suite, so it makes
no assumption about what the library's built-in scratch array holds when it starts.

Why the entry point exists: some users of the library cannot allocate device memory at call time
(their framework's allocator owns the whole GPU, or they run where cudaMalloc's device-wide stall is
not allowed), so the small reduction scratch lives inside the library instead of in a workspace."""
import pytest
import torch

import paper_2605_26842_b200 as pkg

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape,dtype", [((768, 2048), torch.float32), ((1000, 136), torch.float32),
                                         ((33, 17), torch.float32), ((512, 1024), torch.bfloat16)])
def test_noalloc_prologue_matches_handle_prologue_twice_in_a_row(shape, dtype):
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
    for call in range(2):                      # two calls in a row: the second starts from the first's state
        g = (torch.randn(shape, generator=gen) * 1e-3).to(dtype).to(dev)
        opt.step_ex(hp, [W], [g.view((1,) + shape)], None, 1)          # existing entry point, prologue phase only
        pkg.prologue_noalloc(g, M, A, Gp, inv, hp, xhat)
        torch.cuda.synchronize()
        Mr, Ar, Gr = (t[0] for t in opt.state_views(0))
        # same kernel arithmetic on the same inputs: elementwise state agrees to the state tolerance (1e-6)
        for got, ref in ((M, Mr), (A, Ar), (Gp, Gr)):
            err = (got.double() - ref.double()).norm() / ref.double().norm()
            assert err <= 1e-6, (call, err.item())
        nrm = Mr.double().norm().item()
        assert abs(inv.item() * (nrm + hp.norm_eps) - 1.0) <= 1e-6, (call, inv.item(), nrm)
        assert torch.equal(xhat, M.to(torch.bfloat16))
    st, bad = opt.poll_status()
    assert st == 0
    opt.close()


def test_noalloc_prologue_refuses_oversized_and_bad_arguments():
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    hp = pkg.default_hparams()
    small = torch.zeros(8, 8, device=dev)
    inv = torch.zeros(1, device=dev)
    fake = torch.empty(0, device=dev)

    class Shaped:            # a stand-in that reports a huge shape without owning that much memory
        def __init__(self, t, shape):
            self.t, self.shape, self.dtype = t, shape, t.dtype

        def data_ptr(self):
            return self.t.data_ptr()

    with pytest.raises(pkg.MonaError) as e:
        pkg.prologue_noalloc(Shaped(small, (8192, 4096)), small, small, small, inv, hp)
    assert e.value.status == 2 and "16777216" in str(e.value)
    with pytest.raises(pkg.MonaError) as e:
        pkg.prologue_noalloc(Shaped(small, (0, 4)), small, small, small, inv, hp)
    assert e.value.status == 1
    mis = torch.zeros(65, device=dev)[1:].view(8, 8)
    with pytest.raises(pkg.MonaError) as e:
        pkg.prologue_noalloc(mis, small, small, small, inv, hp)
    assert e.value.status == 3
