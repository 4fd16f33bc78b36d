"""Shared driver of the GPU parity tests: runs the CUDA library and the fp64 oracle on the same seeded
inputs and returns relative errors.  The oracle and the library never see each other's outputs."""
import math

import numpy as np
import torch

import oracle.mona_oracle as orc
import paper_2605_26842_b200 as pkg

# Tolerances (relative Frobenius error against the fp64 oracle):
TOL_STATE = 1e-6        # fp32 elementwise state M, A, G_prev
TOL_O_BF16 = 2e-2       # orthogonalised update, bf16 tensor-core Newton-Schulz
TOL_O_FP32 = 1e-4       # orthogonalised update, fp32 validation mode
TOL_W = 3e-2            # parameter displacement W_k - W_0 after up to 10 steps


def rel(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    d = np.linalg.norm(a - b)
    n = np.linalg.norm(b)
    return d / n if n > 0 else d


def oracle_hyper(hp) -> orc.Hyper:
    return orc.Hyper(lr=hp.lr, momentum=hp.momentum, accel_beta=hp.accel_beta, accel_alpha=hp.accel_alpha,
                     weight_decay=hp.weight_decay, ns_steps=hp.ns_steps, ns_a=hp.ns_a, ns_b=hp.ns_b, ns_c=hp.ns_c,
                     norm_eps=hp.norm_eps, scale_mode=hp.scale_mode, scale_value=hp.scale_value)


def ar1_grads(shapes, steps, rho, sigma, seed, dtype=torch.float32, heavy_tail=False):
    """List (per step) of lists (per shape) of CPU tensors following the AR(1) gradient process."""
    gen = torch.Generator().manual_seed(seed)
    out, prev = [], None
    for k in range(steps):
        cur = []
        for i, s in enumerate(shapes):
            z = torch.randn(s, generator=gen)
            if heavy_tail:
                chi = sum(torch.randn(s, generator=gen) ** 2 for _ in range(4)) / 4.0
                z = z / chi.sqrt() / math.sqrt(2.0)
            g = sigma * z if k == 0 else rho * prev[i] + math.sqrt(1 - rho * rho) * sigma * z
            cur.append(g)
        prev = cur
        out.append([g.to(dtype) for g in cur])
    return out


def run_case(shapes, steps=3, hp=None, grad_dtype=torch.float32, rho=0.9, sigma=1e-3, seed=0, heavy_tail=False,
             pad=0, sample=None):
    """shapes: list of (batch, rows, cols).  `pad` adds that many elements between stacked matrices
    (batch_stride > rows*cols).  `sample`: dict spec index -> list of batch indices the oracle follows
    (default: all).  Returns dict of max relative errors over steps and sampled matrices."""
    dev = torch.device("cuda", 0)
    hp = hp or pkg.default_hparams()
    ohp = oracle_hyper(hp)
    gen = torch.Generator().manual_seed(seed + 1000)
    W0 = [torch.randn(s, generator=gen) * 0.02 for s in shapes]
    grads_seq = ar1_grads(shapes, steps, rho, sigma, seed, grad_dtype, heavy_tail)

    def device_buffer(t, dtype):
        b, r, c = t.shape
        stride = r * c + pad
        buf = torch.zeros(b * stride, dtype=dtype, device=dev)
        view = torch.as_strided(buf, (b, r, c), (stride, c, 1))
        view.copy_(t.to(dtype))
        return buf, view

    pbufs, pviews = zip(*[device_buffer(w, torch.float32) for w in W0])
    gbufs, gviews = zip(*[device_buffer(g, grad_dtype) for g in grads_seq[0]])
    obufs, oviews = zip(*[device_buffer(torch.zeros_like(w), torch.float32) for w in W0])

    descs = [pkg.MatrixDesc(s[1], s[2], s[0], s[1] * s[2] + pad, 1 if grad_dtype == torch.bfloat16 else 0, 0) for s in shapes]
    opt = pkg.MonaOptimizer.__new__(pkg.MonaOptimizer)
    _init_from_descs(opt, descs, dev)

    sample = sample or {i: list(range(s[0])) for i, s in enumerate(shapes)}
    states = {(i, b): orc.OracleState(shapes[i][1], shapes[i][2]) for i in sample for b in sample[i]}
    Wref = {(i, b): W0[i][b].double().numpy() for i in sample for b in sample[i]}
    errs = {"M": 0.0, "A": 0.0, "Gprev": 0.0, "O": 0.0, "W": 0.0, "dW": 0.0}
    for k in range(steps):
        for gv, g in zip(gviews, grads_seq[k]):
            gv.copy_(g)
        opt.step_ex(hp, pbufs, gbufs, obufs, 7)
        st, bad = opt.poll_status()
        assert st == 0, (pkg.STATUS_NAMES[st], bad)
        for i in sample:
            Mv, Av, Gv = opt.state_views(i)
            for b in sample[i]:
                Wn, O = orc.mona_step(Wref[(i, b)], grads_seq[k][i][b].double().numpy(), states[(i, b)], ohp)
                Wref[(i, b)] = Wn
                s = states[(i, b)]
                errs["M"] = max(errs["M"], rel(Mv[b].cpu().numpy(), s.M))
                errs["A"] = max(errs["A"], rel(Av[b].cpu().numpy(), s.A))
                errs["Gprev"] = max(errs["Gprev"], rel(Gv[b].cpu().numpy(), s.G_prev))
                errs["O"] = max(errs["O"], rel(oviews[i][b].cpu().numpy(), O))
                got = pviews[i][b].double().cpu().numpy()
                w0 = W0[i][b].double().numpy()
                errs["W"] = max(errs["W"], rel(got, Wn))
                errs["dW"] = max(errs["dW"], rel(got - w0, Wn - w0))
    errs["launches"] = opt.last_launch_count()
    opt.close()
    return errs


def _init_from_descs(opt, descs, dev):
    """MonaOptimizer built from explicit descriptors (lets tests choose batch_stride and grad dtype)."""
    import ctypes as C
    from paper_2605_26842_b200 import binding
    L = pkg.lib()
    opt.descs = list(descs)
    opt.device = dev.index
    sb, wb = pkg.query_sizes(opt.descs)
    opt.state = torch.empty(sb, dtype=torch.uint8, device=dev)
    opt.workspace = torch.empty(wb, dtype=torch.uint8, device=dev)
    opt._h = C.c_void_p()
    st = L.mona_create(C.byref(opt._h), binding._desc_array(opt.descs), len(opt.descs), opt.state.data_ptr(), sb,
                       opt.workspace.data_ptr(), wb, opt.device)
    if st:
        msg = L.mona_last_error(opt._h).decode() if opt._h else ""
        raise pkg.MonaError(st, msg)
