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
# Element-wise companions of the Frobenius gates: max_i |x_i - ref_i| / (rms(ref) + |ref_i|).  A Frobenius norm can hide a small
# patch that is plainly wrong (an unwritten corner of a tile is ~3e-4 of a matrix's energy); the largest single
# deviation cannot.  The numbers are this build's, not the paper's: rounding noise of relative size r spread over
# n elements peaks near r * sqrt(2 ln n) ~ 5.5 r for the matrices tested, heavy-tailed inputs reach a little further,
# so the gates sit at 8x (O) and 10x (state) the Frobenius tolerances; an element that was never written, or written
# from the wrong place, is off by ~1 rms or more (0.5 on this scale) and fails them by a wide margin.
TOL_STATE_MAX = 1e-5
TOL_O_MAX_BF16 = 8 * TOL_O_BF16
TOL_O_MAX_FP32 = 8 * TOL_O_FP32
# MONA-Lite (A_k, G_{k-1} stored in bfloat16).  G_prev is a rounding of the fp32 input and must agree
# bit for bit.  A_k is rounded from a value the GPU forms in fp32 and the oracle in fp64: the two differ
# by ~6e-8 relative, the rounding interval is 2^-8 relative, so about 3e-5 of the elements round the other
# way per step and stay one step apart for ~1/(1-beta_a) steps.  After k <= 10 steps a fraction ~3e-4 of the
# elements is off by one bfloat16 step (<= 2^-7 relative): sqrt(3e-4) * 2^-8 ~ 7e-5 relative Frobenius error
# of A, and alpha * (that error) / |M| ~ 4e-5 of M (measured with fp32 gradients: ~5e-6 and ~3e-6).  With
# bfloat16 gradients D_k is a difference of 8-bit significands and the EMA lands near rounding ties far more
# often (measured 1.0e-4 and 6e-5), so the gates leave a factor of a few over the estimate.
TOL_A_LITE = 5e-4
TOL_M_LITE = 3e-4
LITE_MAX_FLIPPED = 1e-2  # largest fraction of elements of A allowed to sit one bfloat16 step from the oracle's


def rel(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    d = np.linalg.norm(a - b)
    n = np.linalg.norm(b)
    return d / n if n > 0 else d


def maxrel(a, b):
    """Largest element-wise deviation, each element's error measured against rms(reference) + |its own reference value|:
    in units of the matrix's typical magnitude for ordinary elements, and relative for the outliers of heavy-tailed
    inputs (an element 40 rms large carries 40x the rounding error of a typical one)."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    if not a.size:
        return 0.0
    r = float(np.sqrt(np.mean(b * b)))
    if r == 0.0:
        return float(np.max(np.abs(a - b)))
    return float(np.max(np.abs(a - b) / (r + np.abs(b))))


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
             pad=0, sample=None, lite=False, muon=False, combined=False, compare_aux=True, options=None, check_at=None):
    """shapes: list of (batch, rows, cols).  `pad` adds that many elements between stacked matrices
    (batch_stride > rows*cols).  `sample`: dict spec index -> list of batch indices the oracle follows
    (default: all).  `muon`: the oracle runs plain Muon; with `compare_aux=False` only M, O and W are compared
    (the library may then run MONA with alpha = 0, whose A and G_prev still evolve).  `options`: mona_options for
    the handle.  `check_at`: steps (1-based) after which the comparison is made (default: every step).
    Returns dict of max relative errors over the compared steps and sampled matrices."""
    dev = torch.device("cuda", 0)
    hp = hp or pkg.default_hparams()
    ohp = oracle_hyper(hp)
    if lite:
        ohp.state_dtype = "bf16"
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

    descs = [pkg.MatrixDesc(s[1], s[2], s[0], s[1] * s[2] + pad, 1 if grad_dtype == torch.bfloat16 else 0, 2 if combined else (1 if lite else 0)) for s in shapes]
    opt = pkg.MonaOptimizer.__new__(pkg.MonaOptimizer)
    _init_from_descs(opt, descs, dev, options)

    sample = sample or {i: list(range(s[0])) for i, s in enumerate(shapes)}
    states = {(i, b): orc.OracleState(shapes[i][1], shapes[i][2]) for i in sample for b in sample[i]}
    Wref = {(i, b): W0[i][b].double().numpy() for i in sample for b in sample[i]}
    A_before = {}
    errs = {"M": 0.0, "A": 0.0, "Gprev": 0.0, "O": 0.0, "W": 0.0, "dW": 0.0, "A_flipped": 0.0, "A_worst_steps": 0.0, "Gprev_exact": True,
            "M_max": 0.0, "A_max": 0.0, "Gprev_max": 0.0, "O_max": 0.0}
    for k in range(steps):
        for gv, g in zip(gviews, grads_seq[k]):
            gv.copy_(g)
        opt.step_ex(hp, pbufs, gbufs, obufs, 7)
        st, bad = opt.poll_status()
        assert st == 0, (pkg.STATUS_NAMES[st], bad)
        compare = check_at is None or (k + 1) in check_at
        for i in sample:
            Mv, Av, Gv = opt.state_views(i)
            for b in sample[i]:
                A_before[(i, b)] = states[(i, b)].A.copy()
                step_fn = orc.muon_step if muon else orc.mona_step
                Wn, O = step_fn(Wref[(i, b)], grads_seq[k][i][b].double().numpy(), states[(i, b)], ohp)
                Wref[(i, b)] = Wn
                s = states[(i, b)]
                if not compare:
                    continue
                if combined:
                    # the library keeps Z_k = beta_a A_k - (1 - beta_a) G_k; the same combination of the oracle's state
                    z_ref = ohp.accel_beta * s.A - (1.0 - ohp.accel_beta) * s.G_prev
                    errs["M"] = max(errs["M"], rel(Mv[b].cpu().numpy(), s.M))
                    errs["A"] = max(errs["A"], rel(Av[b].double().cpu().numpy(), z_ref))
                    errs["M_max"] = max(errs["M_max"], maxrel(Mv[b].cpu().numpy(), s.M))
                    errs["A_max"] = max(errs["A_max"], maxrel(Av[b].double().cpu().numpy(), z_ref))
                    assert Gv is None
                    errs["O"] = max(errs["O"], rel(oviews[i][b].cpu().numpy(), O))
                    errs["O_max"] = max(errs["O_max"], maxrel(oviews[i][b].cpu().numpy(), O))
                    got = pviews[i][b].double().cpu().numpy()
                    w0 = W0[i][b].double().numpy()
                    errs["W"] = max(errs["W"], rel(got, Wn))
                    errs["dW"] = max(errs["dW"], rel(got - w0, Wn - w0))
                    continue
                a_gpu, g_gpu = Av[b].double().cpu().numpy(), Gv[b].double().cpu().numpy()
                errs["M"] = max(errs["M"], rel(Mv[b].cpu().numpy(), s.M))
                errs["M_max"] = max(errs["M_max"], maxrel(Mv[b].cpu().numpy(), s.M))
                if not compare_aux:      # the oracle runs another algorithm on the auxiliary state (e.g. Muon against alpha = 0)
                    errs["O"] = max(errs["O"], rel(oviews[i][b].cpu().numpy(), O))
                    errs["O_max"] = max(errs["O_max"], maxrel(oviews[i][b].cpu().numpy(), O))
                    got = pviews[i][b].double().cpu().numpy()
                    w0 = W0[i][b].double().numpy()
                    errs["W"] = max(errs["W"], rel(got, Wn))
                    errs["dW"] = max(errs["dW"], rel(got - w0, Wn - w0))
                    continue
                errs["A"] = max(errs["A"], rel(a_gpu, s.A))
                errs["Gprev"] = max(errs["Gprev"], rel(g_gpu, s.G_prev))
                errs["A_max"] = max(errs["A_max"], maxrel(a_gpu, s.A))
                errs["Gprev_max"] = max(errs["Gprev_max"], maxrel(g_gpu, s.G_prev))
                if lite:
                    errs["Gprev_exact"] = errs["Gprev_exact"] and bool(np.array_equal(g_gpu, s.G_prev))
                    diff = np.abs(a_gpu - s.A)
                    errs["A_flipped"] = max(errs["A_flipped"], float((diff > 0).mean()))
                    # size of the disagreement in bfloat16 steps (spacing <= 2^-7 |x|) at the scale of the larger of
                    # A_k and beta_a A_{k-1}: where the two terms of the EMA cancel, one step of the carried-over
                    # A_{k-1} is several steps of the small result
                    step = np.maximum(np.maximum(np.abs(s.A), ohp.accel_beta * np.abs(A_before[(i, b)])), 1e-30) * 2.0 ** -7
                    errs["A_worst_steps"] = max(errs["A_worst_steps"], float((diff / step).max()))
                errs["O"] = max(errs["O"], rel(oviews[i][b].cpu().numpy(), O))
                errs["O_max"] = max(errs["O_max"], maxrel(oviews[i][b].cpu().numpy(), O))
                got = pviews[i][b].double().cpu().numpy()
                w0 = W0[i][b].double().numpy()
                errs["W"] = max(errs["W"], rel(got, Wn))
                errs["dW"] = max(errs["dW"], rel(got - w0, Wn - w0))
    errs["launches"] = opt.last_launch_count()
    opt.close()
    return errs


def _init_from_descs(opt, descs, dev, options=None):
    """MonaOptimizer built from explicit descriptors (lets tests choose batch_stride and grad dtype)."""
    import ctypes as C
    from paper_2605_26842_b200 import binding
    L = pkg.lib()
    opt.descs = list(descs)
    opt.device = dev.index
    opt.options = options if options is not None else pkg.default_options()
    sb, wb = pkg.query_sizes(opt.descs, opt.options)
    opt.state = torch.empty(sb, dtype=torch.uint8, device=dev)
    opt.workspace = torch.empty(wb, dtype=torch.uint8, device=dev)
    opt._h = C.c_void_p()
    st = L.mona_create_opt(C.byref(opt._h), binding._desc_array(opt.descs), len(opt.descs), C.byref(opt.options),
                           opt.state.data_ptr(), sb, opt.workspace.data_ptr(), wb, opt.device)
    if st:
        msg = L.mona_last_error(opt._h).decode() if opt._h else ""
        raise pkg.MonaError(st, msg)
