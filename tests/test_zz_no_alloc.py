"""cada_server_update_noalloc against the regular path.

The entry point under test serves callers that cannot allocate device memory (for example a
plug-in running inside an application whose memory pool owns the GPU): it applies the server
update of Eqs. 2a-2c to buffers the caller already has, with its scratch built into the
library.  A one-worker CADA run is the yardstick: with M = 1 the aggregate of Eq. 2a is exactly
the worker's stored gradient, so feeding that gradient and the pre-step state to the new entry
point must reproduce what cada_step did to theta, h, vhat and the squared step norm.  Two
iterations in a row are compared, because the built-in scratch carries over between calls.
This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest

from paper_2012_15469_b200 import binding as B
from paper_2012_15469_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 1e-5      # the parity tolerance used throughout the GPU tests


def _rel(a, b):
    return float(np.max(np.abs(a.astype(np.float64) - b.astype(np.float64))) / max(float(np.max(np.abs(b))), 1e-30))


def test_noalloc_server_update_matches_cada_step_twice():
    import torch
    from paper_2012_15469_b200 import build as build_mod
    build_mod.build()
    assert torch.cuda.is_available()
    w = synth.workload("C3").scaled(M=1, n_samples=200, batch=16, lam=1e-3)      # p = 7850: several blocks and a ragged tail
    Xs, ys, _ = synth.make_host_data(w)
    t0 = synth.random_theta(w, 0.05)
    run = B.Cada(model=w.model, rule=B.CADA_RULE_CADA2, X=[torch.from_numpy(Xs[0]).cuda()], y=[torch.from_numpy(ys[0]).cuda()],
                 theta0=torch.from_numpy(t0).cuda(), batch=w.batch, alpha=w.alpha, beta1=w.beta1, beta2=w.beta2, eps=w.eps,
                 c=0.0, d_max=w.d_max, D=w.D, lam=w.lam, n_features=w.n_features, n_classes=w.n_classes,
                 has_bias=w.has_bias, seed=w.sample_seed)
    stream = torch.cuda.current_stream()
    theta = torch.from_numpy(t0).cuda()
    h = torch.zeros(w.p, device="cuda")
    vhat = torch.zeros(w.p, device="cuda")
    sq = torch.zeros(1, dtype=torch.float64, device="cuda")
    for it in range(2):
        run.step(1)
        nabla = torch.from_numpy(run.read(B.CADA_BUF_G)[0]).cuda()               # M = 1: the aggregate is this slot
        rc = B.cada_server_update_noalloc(theta.data_ptr(), h.data_ptr(), vhat.data_ptr(), nabla.data_ptr(), w.p,
                                          w.alpha, w.beta1, w.beta2, w.eps, sq.data_ptr(), stream.cuda_stream)
        assert rc == B.CADA_OK
        torch.cuda.synchronize()
        assert _rel(theta.cpu().numpy(), run.read(B.CADA_BUF_THETA)) <= TOL, it
        assert _rel(h.cpu().numpy(), run.read(B.CADA_BUF_H)) <= TOL, it
        assert _rel(vhat.cpu().numpy(), run.read(B.CADA_BUF_VHAT)) <= TOL, it
        want = run.stats().last_step_sqnorm
        assert abs(sq.item() - want) <= TOL * want, (it, sq.item(), want)
    run.close()


@pytest.mark.parametrize("p", [1, 1023, 1025, B.CADA_NOALLOC_MAX_P])
def test_noalloc_server_update_matches_the_oracle(p):
    """Directly against the CPU oracle's statement of Eqs. 2a-2c, from one vector element up to the largest length the
    built-in scratch serves, again on two calls in a row (state and scratch carry over)."""
    import torch
    from oracle import cada_oracle as O
    rng = np.random.default_rng(p)
    theta = rng.standard_normal(p).astype(np.float32)
    h = (0.1 * rng.standard_normal(p)).astype(np.float32)
    vhat = (0.01 * rng.random(p)).astype(np.float32)
    alpha, beta1, beta2, eps = (np.float32(v).item() for v in (0.01, 0.9, 0.99, 1e-8))
    d_theta, d_h, d_vhat = (torch.from_numpy(a).cuda() for a in (theta, h, vhat))
    sq = torch.zeros(1, dtype=torch.float64, device="cuda")
    o_theta, o_h, o_vhat = (a.astype(np.float64) for a in (theta, h, vhat))
    for it in range(2):
        nabla = rng.standard_normal(p).astype(np.float32)
        d_nabla = torch.from_numpy(nabla).cuda()
        rc = B.cada_server_update_noalloc(d_theta.data_ptr(), d_h.data_ptr(), d_vhat.data_ptr(), d_nabla.data_ptr(), p,
                                          alpha, beta1, beta2, eps, sq.data_ptr(), torch.cuda.current_stream().cuda_stream)
        assert rc == B.CADA_OK
        torch.cuda.synchronize()
        new_theta, o_h, o_vhat = O.server_update(o_theta, o_h, o_vhat, nabla.astype(np.float64), alpha, beta1, beta2, eps)
        want_sq = float(np.sum((new_theta - o_theta) ** 2))
        o_theta = new_theta
        assert _rel(d_theta.cpu().numpy(), o_theta) <= TOL and _rel(d_h.cpu().numpy(), o_h) <= TOL, (p, it)
        assert _rel(d_vhat.cpu().numpy(), o_vhat) <= TOL, (p, it)
        assert abs(sq.item() - want_sq) <= TOL * want_sq, (p, it, sq.item(), want_sq)
        # next call starts from the library's fp32 state, as the lock-step protocol does
        o_theta, o_h, o_vhat = (t.cpu().numpy().astype(np.float64) for t in (d_theta, d_h, d_vhat))


def test_noalloc_rejects_what_it_cannot_serve():
    import torch
    buf = torch.zeros(8, device="cuda")
    sq = torch.zeros(1, dtype=torch.float64, device="cuda")
    args = (buf.data_ptr(), buf.data_ptr(), buf.data_ptr(), buf.data_ptr())
    assert B.cada_server_update_noalloc(*args, B.CADA_NOALLOC_MAX_P + 1, 0.01, 0.9, 0.99, 1e-8, sq.data_ptr(), 0) == B.CADA_ERR_UNSUPPORTED
    assert B.cada_server_update_noalloc(*args, 0, 0.01, 0.9, 0.99, 1e-8, sq.data_ptr(), 0) == B.CADA_ERR_INVALID_ARG
    assert B.cada_server_update_noalloc(0, *args[1:], 8, 0.01, 0.9, 0.99, 1e-8, sq.data_ptr(), 0) == B.CADA_ERR_INVALID_ARG
    assert B.cada_server_update_noalloc(*args, 8, 0.01, 1.0, 0.99, 1e-8, sq.data_ptr(), 0) == B.CADA_ERR_INVALID_ARG
