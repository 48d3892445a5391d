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
