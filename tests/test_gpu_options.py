"""GPU parity of the options beyond Algorithm 1's basic form: the recursive aggregate of Eq. 3, the diminishing
step size of Theorem 2 and per-worker minibatch sizes (the supplement's fixed batch ratio over workers of different
size).  Same lock-step protocol and tolerances as the main parity tests."""
import numpy as np
import pytest

from paper_2012_15469_b200 import synth
from paper_2012_15469_b200 import binding as B
from oracle import cada_oracle as O
import parity_harness as PH

pytestmark = pytest.mark.gpu

RULES = [O.RULE_CADA1, O.RULE_CADA2]


@pytest.fixture(scope="module", autouse=True)
def _lib():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2012_15469_b200 import build as build_mod
    build_mod.build()
    B.load_library()


def case(w, rule, iters, *, Xs=None, ys=None, theta0=None, resync=True, tol=1e-5, check_grads=True, server=0, c=None,
         **opt):
    if Xs is None:
        Xs, ys, t0 = synth.make_host_data(w)
        theta0 = t0 if theta0 is None else theta0
    gpu = PH.make_gpu(w, rule, Xs, ys, theta0, server=server, c=c, **opt)
    orc = PH.make_oracle(w, rule, Xs, ys, theta0, server=server, c=c, **opt)
    rep = PH.lockstep(gpu, orc, iters, rule=rule, resync=resync, tol=tol, check_grads=check_grads)
    gpu.close()
    return rep


# ---- Eq. 3 ----------------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("rule", RULES)
def test_recursive_aggregate_small_logistic(rule):
    w = synth.workload("C2")
    rep = case(w, rule, 150, aggregate=B.CADA_AGG_RECURSIVE)
    assert rep.skips > 0 and rep.uploads > rep.forced
    print("Eq. 3, C2", rule, rep)


def test_recursive_aggregate_free_running():
    """No re-synchronisation: the fp32 running sum of Eq. 3 carries its rounding forward, so the bound is the looser
    one of the free-running tests."""
    w = synth.workload("C2")
    print("Eq. 3 drift", case(w, O.RULE_CADA2, 300, aggregate=B.CADA_AGG_RECURSIVE, resync=False, tol=2e-4))


def test_recursive_aggregate_softmax_long_rows_and_lag():
    print("Eq. 3, C3", case(synth.workload("C3"), O.RULE_CADA2, 60, aggregate=B.CADA_AGG_RECURSIVE))
    w = synth.workload("C5").scaled(n_features=1024, batch=50, M=4, n_samples=96, D=6, lam=1e-4)
    t0 = synth.random_theta(w, 0.02)
    print("Eq. 3, long rows", case(w, O.RULE_CADA1, 20, theta0=t0, aggregate=B.CADA_AGG_RECURSIVE))
    w = synth.workload("C2").scaled(alpha=0.1, D=20)
    rep = case(w, O.RULE_LAG, 120, server=B.CADA_SERVER_SGD, c=3000.0, aggregate=B.CADA_AGG_RECURSIVE)
    assert rep.skips > 0
    print("Eq. 3, LAG + SGD", rep)


def test_recursive_aggregate_equals_slot_sum_on_device():
    """Two library runs on the same data, one per aggregate: same decisions and iterates within fp32 rounding."""
    w = synth.workload("C1")
    Xs, ys, t0 = synth.make_host_data(w)
    a = PH.make_gpu(w, O.RULE_CADA2, Xs, ys, t0)
    b = PH.make_gpu(w, O.RULE_CADA2, Xs, ys, t0, aggregate=B.CADA_AGG_RECURSIVE)
    a.step(100); b.step(100)
    sa, sb = a.stats(), b.stats()
    assert sa.uploads_total > 0 and abs(sa.uploads_total - sb.uploads_total) <= 0.02 * sa.uploads_total
    assert PH.rel_inf(b.read(B.CADA_BUF_THETA), a.read(B.CADA_BUF_THETA).astype(np.float64)) <= 1e-3
    G = b.read(B.CADA_BUF_G).astype(np.float64)
    assert PH.rel_inf(b.read(B.CADA_BUF_NABLA), G.mean(axis=0)) <= 1e-4      # Eq. 3 still tracks the slot mean
    a.close(); b.close()


# ---- Theorem 2 -------------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("rule", RULES)
def test_diminishing_step_small_logistic(rule):
    w = synth.workload("C2")
    rep = case(w, rule, 120, alpha=0.5, alpha_K0=25.0)           # runs in the one-launch kernel
    assert rep.skips > 0
    print("Theorem 2, C2", rule, rep)


def test_diminishing_step_three_kernel_path_and_sgd_server():
    print("Theorem 2, C3", case(synth.workload("C3"), O.RULE_CADA2, 60, alpha=0.3, alpha_K0=10.0))
    w = synth.workload("C2").scaled(D=20)
    print("Theorem 2, LAG + SGD", case(w, O.RULE_LAG, 60, server=B.CADA_SERVER_SGD, alpha=2.0, alpha_K0=8.0))


def test_diminishing_step_first_steps_have_the_closed_form_size():
    """AMSGrad server from h = vhat = 0 with b1=.9, b2=.99: step 0 moves every coordinate with |g| >> sqrt(eps) by
    alpha_0 = alpha / K0, so ||theta^1 - theta^0||^2 is about p (alpha/K0)^2."""
    w = synth.workload("C2")
    Xs, ys, t0 = synth.make_host_data(w)
    gpu = PH.make_gpu(w, O.RULE_CADA2, Xs, ys, t0, alpha=0.8, alpha_K0=4.0)
    gpu.step(1)
    s = gpu.stats().last_step_sqnorm
    assert abs(s - w.p * 0.2 ** 2) <= 0.02 * w.p * 0.2 ** 2
    gpu.close()


# ---- per-worker batch sizes -----------------------------------------------------------------------------------------

def test_batch_ratio_over_unequal_workers_small_logistic():
    """The covtype-shaped setting of the supplement: workers of different size, one batch ratio."""
    w = synth.workload("C2").scaled(M=6, n_samples=4000)
    Xs, ys, t0 = synth.make_host_data(w)
    sizes = [4000, 2500, 1000, 700, 333, 40]
    Xs = [x[:n].copy() for x, n in zip(Xs, sizes)]
    ys = [y[:n].copy() for y, n in zip(ys, sizes)]
    bm = [max(1, round(0.025 * n)) for n in sizes]              # 100, 62, 25, 18, 8, 1
    assert max(bm) == w.batch and min(bm) == 1
    for rule in RULES:
        print("batch ratio, one-launch kernel", rule, case(w, rule, 80, Xs=Xs, ys=ys, theta0=t0, batch_m=bm))
    # same data through the three-kernel path (the recursive aggregate rules the one-launch kernel out)
    print("batch ratio, generic kernel", case(w, O.RULE_CADA2, 40, Xs=Xs, ys=ys, theta0=t0, batch_m=bm,
                                              aggregate=B.CADA_AGG_RECURSIVE))


@pytest.mark.parametrize("C", [10, 20])
def test_per_worker_batch_softmax(C):
    """C = 10 runs the 8-row softmax kernel, C = 20 the generic one; sizes below, inside and at the row-block edges."""
    w = synth.workload("C3").scaled(n_features=50, n_classes=C, batch=21, M=5, n_samples=150, D=6, lam=1e-3)
    Xs, ys, _ = synth.make_host_data(w)
    t0 = synth.random_theta(w, 0.2)
    print("per-worker batch, softmax", C, case(w, O.RULE_CADA2, 20, Xs=Xs, ys=ys, theta0=t0, batch_m=[21, 8, 9, 1, 16]))


def test_per_worker_batch_long_rows():
    w = synth.workload("C5").scaled(n_features=2048, batch=37, M=6, n_samples=96, D=6, lam=1e-4)
    Xs, ys, _ = synth.make_host_data(w)
    t0 = synth.random_theta(w, 0.02)
    for rule in RULES:
        print("per-worker batch, long rows", rule,
              case(w, rule, 14, Xs=Xs, ys=ys, theta0=t0, batch_m=[37, 4, 5, 1, 36, 20]))
    # many workers of very different size: the units (4 rows) are dealt to the 148 CTAs by their true count, so a CTA's run
    # crosses several workers and large workers span several CTAs
    w = synth.workload("C5").scaled(n_features=1024, batch=64, M=200, n_samples=80, D=6, lam=1e-4)
    Xs, ys, _ = synth.make_host_data(w)
    t0 = synth.random_theta(w, 0.02)
    bm = [1 + (7 * m * m) % 64 for m in range(w.M)]
    print("per-worker batch, 200 workers", case(w, O.RULE_CADA2, 10, Xs=Xs, ys=ys, theta0=t0, batch_m=bm))


def test_per_worker_batch_validation():
    w = synth.workload("C1")
    Xs, ys, t0 = synth.make_host_data(w)
    for bad in ([0] * w.M, [w.batch + 1] * w.M):
        with pytest.raises(B.CadaError) as e:
            PH.make_gpu(w, O.RULE_CADA2, Xs, ys, t0, batch_m=bad)
        assert e.value.code == B.CADA_ERR_INVALID_ARG
    w4 = synth.workload("C4").scaled(M=2, n_samples=200)
    X4, y4, t4 = synth.make_host_data(w4)
    with pytest.raises(B.CadaError) as e:
        PH.make_gpu(w4, O.RULE_CADA2, X4, y4, t4, batch_m=[5, 5])
    assert e.value.code == B.CADA_ERR_UNSUPPORTED
    with pytest.raises(B.CadaError):
        PH.make_gpu(w, O.RULE_CADA2, Xs, ys, t0, aggregate=7)
    with pytest.raises(B.CadaError):
        PH.make_gpu(w, O.RULE_CADA2, Xs, ys, t0, alpha_K0=-1.0)


# ---- workers split over several handles (one per GPU in a real run) ---------------------------------------------------

def _sharded_lockstep(w, rule, G, iters, *, aggregate=0, server=0, c=None, **kw):
    """G handles on one GPU, handle r holding the workers m = r (mod G); a device-side add stands in for the all-reduce
    of the p-vectors.  Their union must follow the oracle's one-server run like a single handle does."""
    import torch
    Xs, ys, t0 = synth.make_host_data(w)
    parts = [list(range(r, w.M, G)) for r in range(G)]
    gpus = []
    for r, ms in enumerate(parts):
        wl = w.scaled(M=len(ms))
        gpus.append(PH.make_gpu(wl, rule, [Xs[m] for m in ms], [ys[m] for m in ms], t0, aggregate=aggregate, server=server, c=c,
                                M_total=w.M, m_first=r, m_stride=G))
    orc = PH.make_oracle(w, rule, Xs, ys, t0, aggregate=aggregate, server=server, c=c)
    sums = [torch.zeros(w.p, device="cuda") for _ in range(G)]
    uploads = 0
    for k in range(iters):
        out = orc.propose()
        for g, s_ in zip(gpus, sums):
            g.step_local(s_)
        total = torch.stack(sums).sum(dim=0)
        for g in gpus:
            g.step_apply(total)
        up = np.zeros(w.M, dtype=bool)
        for r, ms in enumerate(parts):
            bits = gpus[r].read(B.CADA_BUF_LAST_MASK)
            up[ms] = (bits & 1).astype(bool)
            assert np.array_equal(((bits >> 1) & 1).astype(bool), out["forced"][ms])
        for m in np.nonzero(up != out["upload"])[0]:
            margin = abs(out["lhs"][m] - out["rhs"]) / max(out["lhs"][m], out["rhs"], 1e-300)
            assert margin <= 1e-4, (k, m, margin)
        orc.commit(up)
        uploads += int(up.sum())
        thetas = [g.read(B.CADA_BUF_THETA) for g in gpus]
        for t in thetas[1:]:
            assert np.array_equal(t, thetas[0])                 # replicas of the server state stay identical
        for buf, ref in ((B.CADA_BUF_THETA, orc.theta), (B.CADA_BUF_H, orc.h), (B.CADA_BUF_VHAT, orc.vhat)):
            assert PH.rel_inf(gpus[0].read(buf), ref) <= 1e-5, (k, buf)
        # re-synchronise the oracle with the handles' fp32 state
        orc.theta = thetas[0].astype(np.float64)
        orc.h = gpus[0].read(B.CADA_BUF_H).astype(np.float64)
        orc.vhat = gpus[0].read(B.CADA_BUF_VHAT).astype(np.float64)
        orc.ring = gpus[0].read(B.CADA_BUF_RING).astype(np.float64)
        for r, ms in enumerate(parts):
            orc.G[ms] = gpus[r].read(B.CADA_BUF_G)
            if rule == O.RULE_CADA2:
                orc.theta_hat[ms] = gpus[r].read(B.CADA_BUF_THETA_HAT)
            elif rule == O.RULE_CADA1:
                orc.delta_stored[ms] = gpus[r].read(B.CADA_BUF_DELTA_STORED)
        if rule == O.RULE_CADA1:
            orc.theta_tilde = gpus[0].read(B.CADA_BUF_THETA_TILDE).astype(np.float64)
        if aggregate:
            orc.nabla_rec = gpus[0].read(B.CADA_BUF_NABLA).astype(np.float64)
    stats = [g.stats() for g in gpus]
    assert sum(s_.uploads_total for s_ in stats) == orc.uploads_total == uploads
    assert sum(s_.uploads_forced for s_ in stats) == orc.uploads_forced
    assert all(s_.k == iters and s_.status_flags == 0 for s_ in stats)
    for g in gpus:
        g.close()
    return uploads


@pytest.mark.parametrize("rule", RULES)
@pytest.mark.parametrize("name,kw,G", [("C2", dict(D=8), 2), ("C3", dict(M=6, n_samples=300, D=8), 3),
                                       ("C5", dict(n_features=1024, batch=40, M=5, n_samples=96, D=6, lam=1e-4), 2)])
def test_workers_split_over_handles(rule, name, kw, G):
    """Algorithm 1's workers are independent until the server's sum (Eq. 2a): G handles, each holding every G-th worker
    and sampling that worker's rows of the one-server run, with the sum of their p-vectors handed to every handle, follow
    the oracle's single-server trajectory within the usual tolerances, with exactly its upload counts."""
    w = synth.workload(name).scaled(**kw)
    n = _sharded_lockstep(w, rule, G, 40)
    assert 0 < n < 40 * w.M


def test_workers_split_recursive_aggregate_and_sgd_server():
    w = synth.workload("C2").scaled(D=10, alpha=0.1)
    assert _sharded_lockstep(w, O.RULE_CADA2, 4, 40, aggregate=B.CADA_AGG_RECURSIVE) > 0
    assert _sharded_lockstep(w, O.RULE_LAG, 2, 40, server=B.CADA_SERVER_SGD, c=3000.0) > 0


def test_split_network_matches_one_handle():
    """The network workload split over two handles against ONE handle holding all workers: same decisions, iterates equal
    to fp32 rounding (the sum is taken in a different order)."""
    import torch
    w = synth.workload("C4").scaled(M=4, n_samples=300, D=6)
    Xs, ys, t0 = synth.make_host_data(w)
    one = PH.make_gpu(w, O.RULE_CADA2, Xs, ys, t0)
    parts = [[0, 2], [1, 3]]
    two = [PH.make_gpu(w.scaled(M=2), O.RULE_CADA2, [Xs[m] for m in ms], [ys[m] for m in ms], t0, M_total=4, m_first=r, m_stride=2)
           for r, ms in enumerate(parts)]
    sums = [torch.zeros(w.p, device="cuda") for _ in two]
    for k in range(25):
        one.step(1)
        for g, s_ in zip(two, sums):
            g.step_local(s_)
        total = sums[0] + sums[1]
        for g in two:
            g.step_apply(total)
        mask = np.zeros(4, dtype=np.uint8)
        for r, ms in enumerate(parts):
            mask[ms] = two[r].read(B.CADA_BUF_LAST_MASK)
        assert np.array_equal(mask, one.read(B.CADA_BUF_LAST_MASK)), k
        assert PH.rel_inf(two[0].read(B.CADA_BUF_THETA), one.read(B.CADA_BUF_THETA).astype(np.float64)) <= 1e-5, k
        for g in two:                                              # keep the two runs on one trajectory
            for buf in (B.CADA_BUF_THETA, B.CADA_BUF_H, B.CADA_BUF_VHAT, B.CADA_BUF_RING):
                g.write(buf, one.read(buf))
    assert sum(g.stats().uploads_total for g in two) == one.stats().uploads_total
    one.close()
    for g in two:
        g.close()


def test_split_handle_rejects_whole_steps_and_misuse():
    import torch
    w = synth.workload("C2").scaled(M=2, n_samples=200)
    Xs, ys, t0 = synth.make_host_data(w)
    g = PH.make_gpu(w, O.RULE_CADA2, Xs, ys, t0, M_total=4, m_first=0, m_stride=2)
    assert g.stats().path == B.CADA_PATH_THREE_KERNELS              # the one-launch paths are not used by a split handle
    s_ = torch.zeros(w.p, device="cuda")
    for call in (lambda: g.step(1), lambda: g.step_apply(s_)):
        with pytest.raises(B.CadaError) as e:
            call()
        assert e.value.code == B.CADA_ERR_INVALID_ARG
    g.step_local(s_)
    with pytest.raises(B.CadaError):
        g.step_local(s_)
    g.step_apply(s_)
    assert g.stats().k == 1
    g.close()
