"""GPU parity: libcada through its C ABI against the CPU oracle on identical seeded inputs."""
import math

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


_DATA = {}


def data(w):
    key = (w.name, w.M, w.n_samples, w.n_features)
    if key not in _DATA:
        _DATA[key] = synth.make_host_data(w)
    return _DATA[key]


def run_case(w, rule, iters, *, c=None, resync=True, check_grads=False, tol=1e-5, theta0=None, tau0=None, **kw):
    Xs, ys, t0 = data(w)
    if theta0 is not None:
        t0 = theta0
    gpu = PH.make_gpu(w, rule, Xs, ys, t0, c=c, tau0=tau0)
    orc = PH.make_oracle(w, rule, Xs, ys, t0, c=c, tau0=tau0)
    rep = PH.lockstep(gpu, orc, iters, rule=rule, resync=resync, check_grads=check_grads, tol=tol, **kw)
    gpu.close()
    return rep


@pytest.mark.parametrize("rule", RULES)
def test_c1_full_run(rule):
    w = synth.workload("C1")
    rep = run_case(w, rule, w.iters, check_grads=True)
    assert rep.skips > 0 and rep.uploads > rep.forced        # both branches of the rule were taken
    print("C1", rule, rep)


@pytest.mark.parametrize("rule", RULES)
@pytest.mark.parametrize("c", [0.0, 0.3, 0.6, 1.2])
def test_c2_c_grid(rule, c):
    w = synth.workload("C2")
    rep = run_case(w, rule, 150, c=c)
    if c == 0.0:
        assert rep.skips == 0
    print("C2", rule, c, rep)


@pytest.mark.parametrize("rule", RULES)
def test_c2_free_running_drift(rule):
    """Without re-synchronisation the two trajectories may drift; the bound is looser."""
    w = synth.workload("C2")
    rep = run_case(w, rule, 300, resync=False, tol=2e-4)
    print("C2 drift", rule, rep)


@pytest.mark.parametrize("rule", RULES)
def test_c3_softmax(rule):
    w = synth.workload("C3")
    rep = run_case(w, rule, 120, check_grads=True)
    print("C3", rule, rep)


@pytest.mark.parametrize("rule", RULES)
def test_infinite_c_uploads_every_D(rule):
    w = synth.workload("C1").scaled(D=7)
    rep = run_case(w, rule, 30, c=math.inf)
    assert rep.uploads == w.M * math.ceil(30 / 7) and rep.forced == rep.uploads


def test_ragged_shapes_and_nonzero_start():
    """Odd feature count, batch not a multiple of the row chunk, unequal worker sizes, theta0 != 0."""
    w = synth.workload("C2").scaled(n_features=37, M=3, batch=19, n_samples=211, has_bias=1, lam=1e-3, D=5)
    Xs, ys, _ = synth.make_host_data(w)
    Xs[1], ys[1] = Xs[1][:57].copy(), ys[1][:57].copy()
    _DATA[(w.name, w.M, w.n_samples, w.n_features)] = (Xs, ys, None)
    t0 = synth.random_theta(w, 0.3)
    for rule in RULES:
        rep = run_case(w, rule, 40, theta0=t0, check_grads=True, tau0=[1, 3, 5])
        print("ragged", rule, rep)


@pytest.mark.parametrize("M", [9, 16, 24, 40, 70])
def test_small_logistic_worker_counts(M):
    """The one-launch path over its layouts: one cluster with 1, 2 or 4 workers per CTA (odd and full cluster
    sizes), and, beyond 64 workers, the grid-wide form with one CTA per worker."""
    w = synth.workload("C2").scaled(M=M, n_samples=300, batch=23, D=6)
    Xs, ys, t0 = data(w)
    probe = PH.make_gpu(w, O.RULE_CADA2, Xs, ys, t0)
    assert probe.stats().path == (B.CADA_PATH_ONE_LAUNCH_CLUSTER if M <= 64 else B.CADA_PATH_ONE_LAUNCH_GRID)
    probe.close()
    for rule in RULES:
        rep = run_case(w, rule, 30, check_grads=True)
        assert rep.skips > 0 and rep.forced > 0
        print("workers", M, rule, rep)


def test_two_live_handles_of_different_shape_share_a_kernel():
    """Launch limits (dynamic shared memory) belong to the kernel, not to a handle: creating a second, smaller handle
    must not take the first one's away.  Long rows of two lengths on the streaming kernel, stepped alternately."""
    big = synth.workload("C5").scaled(n_features=4096, batch=16, M=3, n_samples=64, D=5)
    small = synth.workload("C5").scaled(n_features=256, batch=16, M=3, n_samples=64, D=5)
    Xb, yb, tb = synth.make_host_data(big)
    Xs, ys, ts = synth.make_host_data(small)
    a = PH.make_gpu(big, O.RULE_CADA2, Xb, yb, tb)
    b = PH.make_gpu(small, O.RULE_CADA2, Xs, ys, ts)          # created later, needs less
    oa = PH.make_oracle(big, O.RULE_CADA2, Xb, yb, tb)
    ob = PH.make_oracle(small, O.RULE_CADA2, Xs, ys, ts)
    for _ in range(3):
        PH.lockstep(a, oa, 2, rule=O.RULE_CADA2)
        PH.lockstep(b, ob, 2, rule=O.RULE_CADA2)
    a.close(); b.close()


def test_single_worker_single_row():
    w = synth.workload("C1").scaled(M=1, batch=1, n_samples=9)
    for rule in RULES:
        run_case(w, rule, 25, check_grads=True)


def test_explicit_indices_and_history():
    import torch
    w = synth.workload("C1").scaled(M=4, batch=6, n_samples=50)
    Xs, ys, t0 = synth.make_host_data(w)
    rng = np.random.default_rng(3)
    K = 12
    idx = rng.integers(0, 50, size=(K, w.M, w.batch)).astype(np.int32)
    gpu = PH.make_gpu(w, O.RULE_CADA2, Xs, ys, t0, history=K)
    orc = PH.make_oracle(w, O.RULE_CADA2, Xs, ys, t0)
    gpu.set_indices(torch.from_numpy(idx).cuda())
    rep = PH.lockstep(gpu, orc, K, rule=O.RULE_CADA2, idx_fn=lambda k: idx[k], check_grads=True)
    hist_mask = gpu.read(B.CADA_BUF_HIST_MASK)
    hist_rhs = gpu.read(B.CADA_BUF_HIST_RHS)
    assert hist_mask.shape == (K, w.M) and int((hist_mask & 1).sum()) == rep.uploads
    assert hist_rhs[0] == 0.0 and np.all(hist_rhs[1:] > 0)
    # after the explicit block is consumed the hashed stream resumes at the current k
    PH.lockstep(gpu, orc, 3, rule=O.RULE_CADA2)
    gpu.close()


def test_bad_index_is_flagged_not_faulted():
    import torch
    w = synth.workload("C1").scaled(M=2, batch=4, n_samples=20)
    Xs, ys, t0 = synth.make_host_data(w)
    gpu = PH.make_gpu(w, O.RULE_CADA2, Xs, ys, t0)
    idx = torch.tensor([[[0, 1, 2, 99], [3, -5, 1, 0]]], dtype=torch.int32).cuda()
    gpu.set_indices(idx)
    gpu.step(1)
    assert gpu.stats().status_flags & B.CADA_FLAG_BAD_INDEX
    gpu.close()


def test_multi_iteration_call_equals_single_steps_bitwise():
    w = synth.workload("C2").scaled(M=5, n_samples=500)
    Xs, ys, t0 = synth.make_host_data(w)
    a = PH.make_gpu(w, O.RULE_CADA1, Xs, ys, t0)
    b = PH.make_gpu(w, O.RULE_CADA1, Xs, ys, t0)
    a.step(40)
    for _ in range(40):
        b.step(1)
    for buf in (B.CADA_BUF_THETA, B.CADA_BUF_H, B.CADA_BUF_VHAT, B.CADA_BUF_G, B.CADA_BUF_DELTA_STORED, B.CADA_BUF_TAU):
        assert np.array_equal(a.read(buf), b.read(buf))
    assert a.stats().uploads_total == b.stats().uploads_total
    a.close(); b.close()


@pytest.mark.parametrize("M,rule", [(20, O.RULE_CADA2), (20, O.RULE_CADA1), (40, O.RULE_CADA2), (13, O.RULE_CADA1)])
def test_one_launch_many_iterations_equals_single_launches_bitwise(M, rule):
    """Inside one launch the CTAs of the cluster run ahead of one another by up to an iteration (one barrier per
    iteration, two slot buffers); launched one iteration at a time they cannot.  3,000 iterations both ways must leave
    the same bits everywhere, for 1, 2 and 4 workers per CTA."""
    w = synth.workload("C2").scaled(M=M, n_samples=400, batch=37, D=9)
    Xs, ys, t0 = data(w)
    a = PH.make_gpu(w, rule, Xs, ys, t0)
    b = PH.make_gpu(w, rule, Xs, ys, t0)
    assert a.stats().path == B.CADA_PATH_ONE_LAUNCH_CLUSTER
    K = 3000
    a.step(K)
    for _ in range(K):
        b.step(1)
    second = B.CADA_BUF_DELTA_STORED if rule == O.RULE_CADA1 else B.CADA_BUF_THETA_HAT
    for buf in (B.CADA_BUF_THETA, B.CADA_BUF_H, B.CADA_BUF_VHAT, B.CADA_BUF_G, second, B.CADA_BUF_TAU, B.CADA_BUF_RING,
                B.CADA_BUF_UPLOADS_PER_WORKER, B.CADA_BUF_GRAD_FRESH, B.CADA_BUF_LAST_MASK):
        assert np.array_equal(a.read(buf), b.read(buf)), buf
    sa, sb = a.stats(), b.stats()
    assert (sa.k, sa.uploads_total, sa.uploads_forced, sa.near_ties) == (sb.k, sb.uploads_total, sb.uploads_forced, sb.near_ties)
    assert sa.status_flags == 0 and 0 < sa.uploads_total < K * M
    a.close(); b.close()


def test_checkpoint_restore_is_bitwise():
    w = synth.workload("C2").scaled(M=4, n_samples=300)
    Xs, ys, t0 = synth.make_host_data(w)
    rule = O.RULE_CADA2
    a = PH.make_gpu(w, rule, Xs, ys, t0)
    a.step(30)
    bufs = [B.CADA_BUF_THETA, B.CADA_BUF_H, B.CADA_BUF_VHAT, B.CADA_BUF_G, B.CADA_BUF_THETA_HAT, B.CADA_BUF_TAU,
            B.CADA_BUF_RING, B.CADA_BUF_K]
    saved = {b_: a.read(b_) for b_ in bufs}
    a.step(30)
    b = PH.make_gpu(w, rule, Xs, ys, t0)
    for b_, v in saved.items():
        b.write(b_, v)
    b.step(30)
    for b_ in bufs:
        assert np.array_equal(a.read(b_), b.read(b_)), b_
    a.close(); b.close()


def _host_counted_workloads():
    """Small shapes served by the two kernels that take the iteration number from the host's count."""
    soft = synth.workload("C3").scaled(n_features=61, n_classes=7, batch=12, M=3, n_samples=90, D=5)
    long_rows = synth.workload("C5").scaled(n_features=512, batch=16, M=3, n_samples=64, D=5)
    net = synth.workload("C4").scaled(n_features=120, n_hidden=24, n_classes=5, batch=12, M=3, n_samples=90, D=5)
    many = synth.workload("C3").scaled(n_features=40, n_classes=20, batch=10, M=3, n_samples=80, D=5)     # generic gradient + trigger kernel
    return [(soft, B.CADA_PATH_SOFTMAX_CLUSTER), (long_rows, B.CADA_PATH_THREE_KERNELS), (net, B.CADA_PATH_MLP_CLUSTER),
            (many, B.CADA_PATH_THREE_KERNELS)]


@pytest.mark.parametrize("which", [0, 1, 2, 3])
def test_checkpoint_restore_with_host_counted_iterations(which):
    """The softmax cluster kernel and the long-row kernel fetch their rows from the host's iteration count: a restored
    run (state and k written back through cada_write) must continue bit for bit, also across a multi-iteration call.
    Inside a multi-iteration call the update kernel leaves the newest window term as block partials for the next
    iteration's deciding kernel to add up, in single-iteration calls it adds them itself: one 17-iteration call and 17
    one-iteration calls must agree in every bit, the window included."""
    w, path = _host_counted_workloads()[which]
    Xs, ys, t0 = synth.make_host_data(w)
    rule = O.RULE_CADA2
    a = PH.make_gpu(w, rule, Xs, ys, t0)
    assert a.stats().path == path
    a.step(13)
    bufs = [B.CADA_BUF_THETA, B.CADA_BUF_H, B.CADA_BUF_VHAT, B.CADA_BUF_G, B.CADA_BUF_THETA_HAT, B.CADA_BUF_TAU,
            B.CADA_BUF_RING, B.CADA_BUF_K]
    saved = {b_: a.read(b_) for b_ in bufs}
    a.step(17)
    b = PH.make_gpu(w, rule, Xs, ys, t0)
    b.step(4)                                   # a different history first: the restore must override its count as well
    for b_, v in saved.items():
        b.write(b_, v)
    for _ in range(17):
        b.step(1)
    for b_ in bufs:
        assert np.array_equal(a.read(b_), b.read(b_)), b_
    assert int(a.read(B.CADA_BUF_K)[0]) == 30
    a.close(); b.close()


@pytest.mark.parametrize("which", [0, 1, 2])
def test_explicit_indices_history_and_host_steps_with_host_counted_iterations(which):
    import torch
    w, _ = _host_counted_workloads()[which]
    Xs, ys, t0 = synth.make_host_data(w)
    rule = O.RULE_CADA1
    rng = np.random.default_rng(11 + which)
    K = 9
    idx = rng.integers(0, w.n_samples, size=(K, w.M, w.batch)).astype(np.int32)
    kw = MLP_KW if w.model == synth.MODEL_MLP2 else {}
    gpu = PH.make_gpu(w, rule, Xs, ys, t0, history=K)
    orc = PH.make_oracle(w, rule, Xs, ys, t0)
    PH.lockstep(gpu, orc, 3, rule=rule, check_grads=True, **kw)                # hashed stream, k = 0..2
    gpu.set_indices(torch.from_numpy(idx).cuda())
    rep = PH.lockstep(gpu, orc, K, rule=rule, idx_fn=lambda k: idx[k - 3], check_grads=True, **kw)
    assert int((gpu.read(B.CADA_BUF_HIST_MASK) & 1).sum()) >= rep.uploads - w.M * 3
    PH.lockstep(gpu, orc, 4, rule=rule, **kw)                                   # back on the hashed stream at k = 12
    gpu.close()
    # cada_step_host on the rows the hashed stream would pick follows the resident run
    a = PH.make_gpu(w, rule, Xs, ys, t0)
    b = PH.make_gpu(w, rule, Xs, ys, t0, host_step=True)
    ydt = torch.float32 if w.model == synth.MODEL_LOGISTIC else torch.int32
    xdt = torch.bfloat16 if w.x_bf16 else torch.float32
    hx = torch.zeros((w.M, w.batch, w.ldx), dtype=xdt).pin_memory()
    hy = torch.empty((w.M, w.batch), dtype=ydt).pin_memory()
    th = torch.empty(w.p, dtype=torch.float32).pin_memory()
    mk = torch.empty(w.M, dtype=torch.uint8).pin_memory()
    for k in range(8):
        rows = O.sample_indices(w.sample_seed, k, w.M, w.batch, [x.shape[0] for x in Xs])
        for m in range(w.M):
            hx[m, :, :Xs[m].shape[1]] = torch.from_numpy(Xs[m][rows[m]]).to(xdt)
            hy[m] = torch.from_numpy(ys[m][rows[m]])
        a.step(1)
        b.step_host(hx, hy, th, mk)
        assert PH.rel_inf(th.numpy(), a.read(B.CADA_BUF_THETA).astype(np.float64)) <= 1e-5
        assert np.array_equal(a.read(B.CADA_BUF_LAST_MASK), mk.numpy())
    a.close(); b.close()


def test_host_minibatch_step_matches_resident_step():
    """cada_step_host on the rows the hashed stream would pick gives the same iterate."""
    import torch
    w = synth.workload("C2").scaled(M=4, n_samples=300)
    Xs, ys, t0 = synth.make_host_data(w)
    rule = O.RULE_CADA2
    a = PH.make_gpu(w, rule, Xs, ys, t0)
    b = PH.make_gpu(w, rule, Xs, ys, t0, host_step=True)
    hx = torch.empty((w.M, w.batch, w.ldx), dtype=torch.float32).pin_memory()
    hy = torch.empty((w.M, w.batch), dtype=torch.float32).pin_memory()
    th = torch.empty(w.p, dtype=torch.float32).pin_memory()
    mk = torch.empty(w.M, dtype=torch.uint8).pin_memory()
    for k in range(20):
        idx = O.sample_indices(w.sample_seed, k, w.M, w.batch, [x.shape[0] for x in Xs])
        for m in range(w.M):
            hx[m] = torch.from_numpy(Xs[m][idx[m]])
            hy[m] = torch.from_numpy(ys[m][idx[m]])
        a.step(1)
        b.step_host(hx, hy, th, mk)
        # the resident run may take the one-launch kernel, whose sums are ordered differently
        assert PH.rel_inf(th.numpy(), a.read(B.CADA_BUF_THETA).astype(np.float64)) <= 1e-5
        assert np.array_equal(a.read(B.CADA_BUF_LAST_MASK), mk.numpy())
    a.close(); b.close()


@pytest.mark.parametrize("name,kw", [("C2", dict(M=4, n_samples=300)), ("C3", dict(M=3, n_samples=200, batch=16)),
                                     ("C5", dict(n_features=512, batch=16, M=3, n_samples=64, D=5)),
                                     ("C4", dict(M=3, n_samples=200, D=5))])
def test_streamed_minibatches_match_single_host_steps(name, kw):
    """cada_step_host_n (copies of step i+1 overlapped with step i, results copied back per step, one synchronisation)
    against n calls of cada_step_host on the same host minibatches: same bits in theta and in the masks of every step."""
    import torch
    w = synth.workload(name).scaled(**kw)
    Xs, ys, t0 = synth.make_host_data(w)
    rule = O.RULE_CADA2
    a = PH.make_gpu(w, rule, Xs, ys, t0, host_step=True)
    b = PH.make_gpu(w, rule, Xs, ys, t0, host_step=True)
    n = 11
    xdt = torch.bfloat16 if w.x_bf16 else torch.float32
    ydt = torch.float32 if w.model == synth.MODEL_LOGISTIC else torch.int32
    hx = torch.zeros((n, w.M, w.batch, w.ldx), dtype=xdt).pin_memory()
    hy = torch.zeros((n, w.M, w.batch), dtype=ydt).pin_memory()
    rng = np.random.default_rng(5)
    for k in range(n):
        for m in range(w.M):
            rows = rng.integers(0, Xs[m].shape[0], size=w.batch)
            hx[k, m, :, :Xs[m].shape[1]] = torch.from_numpy(Xs[m][rows]).to(xdt)
            hy[k, m] = torch.from_numpy(ys[m][rows])
    th_a = torch.empty(w.p, dtype=torch.float32).pin_memory(); mk_a = torch.empty(w.M, dtype=torch.uint8).pin_memory()
    th_b = torch.empty((n, w.p), dtype=torch.float32).pin_memory(); mk_b = torch.empty((n, w.M), dtype=torch.uint8).pin_memory()
    b.step_host_n(4, hx, hy, th_b, mk_b)                       # two calls: the halves are handed over between calls as well
    b.step_host_n(n - 4, hx[4:], hy[4:], th_b[4:], mk_b[4:])
    for k in range(n):
        a.step_host(hx[k], hy[k], th_a, mk_a)
        assert np.array_equal(th_a.numpy(), th_b[k].numpy()), k
        assert np.array_equal(mk_a.numpy(), mk_b[k].numpy()), k
    assert a.stats().uploads_total == b.stats().uploads_total and b.stats().k == n
    a.close(); b.close()


@pytest.mark.parametrize("name,kw,rule", [
    ("C2", dict(M=5, n_samples=300), O.RULE_CADA1),                       # row pitch = staged pitch: one bulk copy per worker and step
    ("C1", dict(M=6, n_samples=200), O.RULE_CADA2),                       # the same with one worker per CTA and short rows
    ("C2", dict(M=5, n_samples=300, ldx=80), O.RULE_CADA2),               # wide caller pitch: one bulk copy per row
    ("C2", dict(M=3, n_samples=200, batch=30), O.RULE_CADA2),             # batch not a multiple of 4: labels in 4-byte pieces
    ("C2", dict(M=9, n_samples=200, batch=30, ldx=64), O.RULE_CADA1)])
def test_streamed_minibatches_fetched_by_the_kernel_match_the_staged_copies(name, kw, rule):
    """Small logistic problems on the one-cluster path: with every buffer page-locked, cada_step_host_n runs its n iterations in
    ONE launch whose producer warps fetch each step's rows from the caller's host memory; with pageable buffers it stages each
    step through the copy engine.  Same arithmetic either way: theta and the masks of every step agree bitwise, and the
    launch counts show that the two calls took the two routes."""
    import torch
    w = synth.workload(name).scaled(**kw)
    Xs, ys, t0 = synth.make_host_data(w)
    a = PH.make_gpu(w, rule, Xs, ys, t0, host_step=True)
    b = PH.make_gpu(w, rule, Xs, ys, t0, host_step=True)
    assert a.stats().path == B.CADA_PATH_ONE_LAUNCH_CLUSTER
    n = 45                                                      # the streamed kernel hands the masks over 16 steps at a time
    hx = torch.zeros((n, w.M, w.batch, w.ldx), dtype=torch.float32)
    hy = torch.zeros((n, w.M, w.batch), dtype=torch.float32)
    rng = np.random.default_rng(11)
    for k in range(n):
        for m in range(w.M):
            rows = rng.integers(0, Xs[m].shape[0], size=w.batch)
            hx[k, m, :, :Xs[m].shape[1]] = torch.from_numpy(Xs[m][rows])
            hy[k, m] = torch.from_numpy(ys[m][rows])
    th_a = torch.empty((n, w.p), dtype=torch.float32); mk_a = torch.empty((n, w.M), dtype=torch.uint8)
    th_b = torch.full((n, w.p), np.nan, dtype=torch.float32).pin_memory(); mk_b = torch.full((n, w.M), 255, dtype=torch.uint8).pin_memory()
    l0a, l0b = a.stats().kernel_launches, b.stats().kernel_launches
    a.step_host_n(n, hx, hy, th_a, mk_a)                        # pageable: staged copies, a launch per step
    hxp, hyp = hx.pin_memory(), hy.pin_memory()
    b.step_host_n(9, hxp, hyp, th_b, mk_b)                      # page-locked: one launch per call
    b.step_host_n(n - 9, hxp[9:], hyp[9:], th_b[9:], mk_b[9:])
    assert np.array_equal(th_a.numpy(), th_b.numpy())
    assert np.array_equal(mk_a.numpy(), mk_b.numpy())
    sa, sb = a.stats(), b.stats()
    assert sa.k == n and sb.k == n and sa.uploads_total == sb.uploads_total
    assert sb.kernel_launches - l0b == 2 and sa.kernel_launches - l0a >= n
    for which in (B.CADA_BUF_THETA, B.CADA_BUF_VHAT, B.CADA_BUF_G, B.CADA_BUF_RING, B.CADA_BUF_TAU,
                  B.CADA_BUF_DELTA_STORED if rule == O.RULE_CADA1 else B.CADA_BUF_THETA_HAT):
        assert np.array_equal(a.read(which), b.read(which)), which
    b.step(3); a.step(3)                                        # the resident stream carries on from the same state
    assert np.array_equal(a.read(B.CADA_BUF_THETA), b.read(B.CADA_BUF_THETA))
    a.close(); b.close()


def test_nonfinite_input_raises_flag():
    w = synth.workload("C1").scaled(M=2, batch=4, n_samples=20)
    Xs, ys, t0 = synth.make_host_data(w)
    Xs[0][:, 3] = np.nan
    gpu = PH.make_gpu(w, O.RULE_CADA2, Xs, ys, t0)
    gpu.step(2)
    st = gpu.stats()
    assert st.status_flags & B.CADA_FLAG_NONFINITE and st.rc == B.CADA_ERR_NONFINITE and st.k == 2
    with pytest.raises(B.CadaError) as e:                  # the problem surfaces at the next step as well
        gpu.step(1)
    assert e.value.code == B.CADA_ERR_NONFINITE
    gpu.close()


def test_bounded_wait_that_runs_out_is_reported_not_hung():
    """The grid-wide one-launch kernel (more than 64 workers) synchronises its CTAs through flags in global memory that
    each CTA polls a bounded number of times.  With the bound set to a single poll the first CTA to reach the barrier
    finds flags that nobody has set yet, gives up, raises CADA_FLAG_TIMEOUT and returns; the rest follow through the same
    bound.  The launch ends, the context stays usable, and the handle reports CADA_ERR_TIMEOUT from then on."""
    w = synth.workload("C2").scaled(M=70, n_samples=300, batch=23, D=6)
    Xs, ys, t0 = data(w)
    gpu = PH.make_gpu(w, O.RULE_CADA2, Xs, ys, t0)
    assert gpu.stats().path == B.CADA_PATH_ONE_LAUNCH_GRID
    gpu.step(5)                                             # the default bound is never reached
    assert gpu.stats().rc == B.CADA_OK
    gpu.set_wait_limit(0)
    gpu.step(50)
    st = gpu.stats()                                        # synchronises: the launch has ended
    assert st.status_flags & B.CADA_FLAG_TIMEOUT and st.rc == B.CADA_ERR_TIMEOUT
    with pytest.raises(B.CadaError) as e:
        gpu.step(1)
    assert e.value.code == B.CADA_ERR_TIMEOUT
    gpu.close()
    # the device and the library are unaffected: a fresh handle on the same data runs and matches the oracle
    rep = run_case(w, O.RULE_CADA2, 10)
    assert rep.iters == 10


# ------------------------------------------------------------------------------------------
# long-row logistic shapes (the streaming gradient kernel)
# ------------------------------------------------------------------------------------------

@pytest.mark.parametrize("F,has_bias,batch,M", [(4096, 0, 64, 5), (4096, 1, 37, 3), (2048, 0, 50, 4), (1000, 1, 33, 3),
                                                 (512, 0, 7, 2), (256, 1, 4, 1), (3072, 0, 130, 150)])
def test_long_row_logistic_shapes(F, has_bias, batch, M):
    """Rows of 1-16 KB; batches that are not multiples of the 4-row pipeline stage; more workers than
    SMs' worth of units and fewer; bias column on and off."""
    w = synth.workload("C5").scaled(n_features=F, has_bias=has_bias, batch=batch, M=M, n_samples=96, D=6, lam=1e-4)
    Xs, ys, _ = synth.make_host_data(w)
    _DATA[(w.name, w.M, w.n_samples, w.n_features)] = (Xs, ys, None)
    t0 = synth.random_theta(w, 0.02)
    for rule in RULES:
        rep = run_case(w, rule, 14, theta0=t0, check_grads=True)
        print("long rows", F, has_bias, batch, M, rule, rep)


# ------------------------------------------------------------------------------------------
# 2-layer ReLU network with bf16 operands (C4)
# ------------------------------------------------------------------------------------------

# The network rounds the operands of its products to bf16, and a rounding is an integer decision taken from a
# floating-point sum (fp32 in the library, fp64 in the oracle).  The lock-step protocol hands the library's unrounded
# a1, dz2 and dz1 to the oracle, which takes over a differing rounding where the two unrounded values agree to 1e-5 of
# the operand's largest entry (the same tie rule as for upload decisions and for the sign of z1); the unrounded operands
# themselves must agree to 1e-5 everywhere.  With equal rounded operands on both sides what is left is fp32 against fp64
# accumulation, so the network is held to the tolerances of the fp32 models.  Its innovation d_m = g_m - g'_m is the
# difference of two separately evaluated gradients and is therefore judged against |g_m|; the left-hand side's allowance
# carries the matching cancellation factor (parity_harness.lockstep).
MLP_KW = dict(round_ties=True, innovation_noise_floor=True)


@pytest.mark.parametrize("rule", [O.RULE_CADA2, O.RULE_CADA1])
def test_c4_mlp_full_shape(rule):
    w = synth.workload("C4")
    rep = run_case(w, rule, 60, check_grads=True, **MLP_KW)
    print("C4", rule, rep)


def test_mlp_ragged_shapes():
    """Hidden width, class count, batch and feature count that are not multiples of any tile (plain-FMA kernels)."""
    w = synth.workload("C4").scaled(n_features=100, n_hidden=37, n_classes=7, batch=150, M=3, n_samples=220, D=6)
    Xs, ys, t0 = synth.make_host_data(w)
    _DATA[(w.name, w.M, w.n_samples, w.n_features)] = (Xs, ys, t0)
    for rule in RULES:
        rep = run_case(w, rule, 25, check_grads=True, **MLP_KW)
        print("mlp ragged", rule, rep)


@pytest.mark.parametrize("F,H,C,batch,M,D", [(200, 40, 7, 100, 3, 6), (776, 200, 10, 128, 10, 4), (88, 248, 16, 33, 2, 5),
                                             (896, 64, 3, 128, 4, 7)])
def test_mlp_cluster_kernel_shapes(F, H, C, batch, M, D):
    """The one-launch network path with the features split over the cluster (feature counts that are not a multiple of 16,
    or above 784): a ragged last feature slice, a single slice, the
    widest supported hidden layer and class count, eight slices, batches that leave ragged row groups and row blocks,
    and a short maximum staleness so that the ring of first-layer operand images wraps, forced uploads occur and the
    CADA1 snapshot is retaken several times inside the run."""
    w = synth.workload("C4").scaled(n_features=F, n_hidden=H, n_classes=C, batch=batch, M=M, n_samples=260, D=D, lam=1e-3)
    Xs, ys, t0 = synth.make_host_data(w)
    _DATA[(w.name, w.M, w.n_samples, w.n_features)] = (Xs, ys, t0)
    probe = PH.make_gpu(w, O.RULE_CADA2, Xs, ys, t0)
    assert probe.stats().path == B.CADA_PATH_MLP_CLUSTER
    probe.close()
    for rule in RULES:
        rep = run_case(w, rule, 3 * D + 4, check_grads=True, tau0=[1 + (m % D) for m in range(M)], **MLP_KW)
        assert rep.forced > 0
        print("mlp cluster", F, H, C, batch, rule, rep)


@pytest.mark.parametrize("F,H,C,batch,M,D", [(128, 36, 16, 16, 2, 5), (400, 248, 3, 37, 3, 6), (256, 64, 7, 128, 2, 4),
                                             (640, 100, 10, 60, 3, 7), (784, 200, 10, 112, 2, 3), (784, 200, 10, 128, 10, 4),
                                             (96, 248, 16, 33, 2, 5), (16, 4, 3, 1, 2, 3)])
def test_mlp_hidden_split_kernel_shapes(F, H, C, batch, M, D):
    """The one-launch network path with the hidden layer split over the cluster: one to seven 112-feature chunks with a
    ragged last one, all chunks resident or two / three of them passing through the stages a second time, one, two, four,
    seven and eight hidden slices with a ragged last slice, one and two class tiles, batches of 1 to 128 rows (ragged row
    groups, ragged row ownership, the full accumulator height), and a short maximum staleness so that the ring of
    operand images wraps, forced uploads occur and the CADA1 snapshot is retaken several times inside the run."""
    w = synth.workload("C4").scaled(n_features=F, n_hidden=H, n_classes=C, batch=batch, M=M, n_samples=260, D=D, lam=1e-3)
    Xs, ys, t0 = synth.make_host_data(w)
    _DATA[(w.name, w.M, w.n_samples, w.n_features)] = (Xs, ys, t0)
    probe = PH.make_gpu(w, O.RULE_CADA2, Xs, ys, t0)
    assert probe.stats().path == B.CADA_PATH_MLP_HIDDEN_SPLIT
    probe.close()
    for rule in RULES:
        rep = run_case(w, rule, 3 * D + 4, check_grads=True, tau0=[1 + (m % D) for m in range(M)], **MLP_KW)
        assert rep.forced > 0
        print("mlp hidden split", F, H, C, batch, rule, rep)


def test_mlp_per_product_tensor_core_kernels():
    """More than eight 112-feature slices: the cluster kernel declines and the per-product tcgen05 kernels (one launch per
    product, first-layer weights re-rounded every iteration, trigger kernel) serve the shape."""
    w = synth.workload("C4").scaled(n_features=1000, n_hidden=64, n_classes=5, batch=64, M=2, n_samples=200, D=5)
    Xs, ys, t0 = synth.make_host_data(w)
    _DATA[(w.name, w.M, w.n_samples, w.n_features)] = (Xs, ys, t0)
    probe = PH.make_gpu(w, O.RULE_CADA2, Xs, ys, t0)
    st = probe.stats()
    probe.step(1)
    assert st.path == B.CADA_PATH_THREE_KERNELS and probe.stats().kernel_launches - st.kernel_launches == 6
    probe.close()
    for rule in RULES:
        rep = run_case(w, rule, 14, check_grads=True, **MLP_KW)
        print("mlp per-product kernels", rule, rep)


def test_mlp_cluster_checkpoint_restore_is_bitwise():
    """The ring of operand images is derived state: a run restored through cada_write (iterates, staleness, k) rebuilds
    it and continues bit for bit, under both rules."""
    w = synth.workload("C4").scaled(M=4, n_samples=300, D=5)
    Xs, ys, t0 = synth.make_host_data(w)
    for rule, second in ((O.RULE_CADA2, B.CADA_BUF_THETA_HAT), (O.RULE_CADA1, B.CADA_BUF_DELTA_STORED)):
        a = PH.make_gpu(w, rule, Xs, ys, t0)
        assert a.stats().path == B.CADA_PATH_MLP_HIDDEN_SPLIT
        a.step(13)
        bufs = [B.CADA_BUF_THETA, B.CADA_BUF_H, B.CADA_BUF_VHAT, B.CADA_BUF_G, second, B.CADA_BUF_TAU, B.CADA_BUF_RING, B.CADA_BUF_K]
        if rule == O.RULE_CADA1:
            bufs.append(B.CADA_BUF_THETA_TILDE)
        saved = {b_: a.read(b_) for b_ in bufs}
        a.step(9)
        b = PH.make_gpu(w, rule, Xs, ys, t0)
        b.step(3)
        for b_, v in saved.items():
            b.write(b_, v)
        for _ in range(9):
            b.step(1)
        for b_ in bufs:
            assert np.array_equal(a.read(b_), b.read(b_)), (rule, b_)
        assert a.stats().uploads_total > 0 and a.stats().status_flags == 0
        a.close(); b.close()


@pytest.mark.parametrize("C,F,batch,has_bias,M", [(3, 37, 19, 0, 3), (16, 130, 8, 1, 3), (20, 50, 21, 1, 3), (3, 9, 3, 1, 2),
                                                  (7, 61, 33, 1, 5), (11, 40, 5, 0, 40), (13, 29, 64, 1, 20),
                                                  (10, 203, 300, 1, 3)])
def test_softmax_ragged_shapes(C, F, batch, has_bias, M):
    """Class counts below, at and above the specialised kernels' limit (16; above it the generic kernel runs), every
    column-group width of the cluster kernel, feature counts that leave ragged slices (down to a slice holding only
    the bias column), batches that are not multiples of 4 or 8 rows, a batch too large for the cluster kernel (300:
    the 8-row kernel runs), few and many workers, with and without the bias row."""
    w = synth.workload("C3").scaled(n_features=F, n_classes=C, batch=batch, has_bias=has_bias, M=M, n_samples=150, D=6,
                                    lam=1e-3)
    Xs, ys, _ = synth.make_host_data(w)
    _DATA[(w.name, w.M, w.n_samples, w.n_features)] = (Xs, ys, None)
    t0 = synth.random_theta(w, 0.2)
    probe = PH.make_gpu(w, O.RULE_CADA2, Xs, ys, t0)
    assert probe.stats().path == (B.CADA_PATH_SOFTMAX_CLUSTER if C <= 16 and batch <= 256 else B.CADA_PATH_THREE_KERNELS)
    probe.close()
    for rule in RULES:
        rep = run_case(w, rule, 20, theta0=t0, check_grads=True)
        print("softmax ragged", C, F, batch, rule, rep)


# ------------------------------------------------------------------------------------------
# stochastic LAG (Eq. 4) with the SGD server, the paper's comparator
# ------------------------------------------------------------------------------------------

def _lag_case(w, iters, c=None, **kw):
    Xs, ys, t0 = data(w)
    gpu = PH.make_gpu(w, O.RULE_LAG, Xs, ys, t0, server=B.CADA_SERVER_SGD, c=c)
    orc = PH.make_oracle(w, O.RULE_LAG, Xs, ys, t0, server=1, c=c)
    rep = PH.lockstep(gpu, orc, iters, rule=O.RULE_LAG, check_grads=True, **kw)
    gpu.close()
    return rep


def test_lag_sgd_logistic_small_and_long_rows():
    # at the paper's scale of c the rule (almost) never skips: the left-hand side is dominated by sampling variance,
    # which is the paper's point about stochastic LAG (Section 2.1); a very large c exercises the skip branch
    rep = _lag_case(synth.workload("C2").scaled(alpha=0.1, D=20), 60)
    print("LAG C2 c=0.6", rep)
    rep = _lag_case(synth.workload("C2").scaled(alpha=0.1, D=20), 120, c=3000.0)
    assert rep.skips > 0 and rep.uploads > rep.forced
    print("LAG C2 c=3000", rep)
    w = synth.workload("C5").scaled(n_features=1024, batch=50, M=4, n_samples=96, D=8, alpha=0.05)
    print("LAG long rows", _lag_case(w, 20))


def test_lag_sgd_softmax_and_mlp():
    print("LAG C3", _lag_case(synth.workload("C3").scaled(alpha=0.1, D=20, M=4), 40))
    w = synth.workload("C4").scaled(alpha=0.05, D=10, M=3)
    print("LAG C4", _lag_case(w, 20, **MLP_KW))


def test_lag_with_the_adam_server():
    """Eq. 4 as a third trigger on top of Eqs. 2a-2c (the rule and the server are independent switches)."""
    w = synth.workload("C2").scaled(D=20, M=6)
    Xs, ys, t0 = data(w)
    gpu = PH.make_gpu(w, O.RULE_LAG, Xs, ys, t0)
    orc = PH.make_oracle(w, O.RULE_LAG, Xs, ys, t0)
    rep = PH.lockstep(gpu, orc, 80, rule=O.RULE_LAG, check_grads=True)
    print("LAG + AMSGrad", rep)
    gpu.close()


# ------------------------------------------------------------------------------------------
# full-data evaluation (loss of Eq. 1 and accuracy)
# ------------------------------------------------------------------------------------------

@pytest.mark.parametrize("name,kw", [("C1", dict(M=4, n_samples=777)), ("C3", dict(M=3, n_samples=500)),
                                     ("C4", dict(M=2, n_samples=300))])
def test_evaluation_pass(name, kw):
    w = synth.workload(name).scaled(**kw)
    Xs, ys, t0 = synth.make_host_data(w)
    Xs[0], ys[0] = Xs[0][: w.n_samples // 3].copy(), ys[0][: w.n_samples // 3].copy()      # unequal workers
    rule = O.RULE_CADA2
    gpu = PH.make_gpu(w, rule, Xs, ys, t0)
    orc = PH.make_oracle(w, rule, Xs, ys, t0)
    for stage in range(2):
        loss, acc = gpu.eval()
        want_loss, want_acc = orc.evaluate()
        n_rows = sum(x.shape[0] for x in Xs)
        assert abs(loss - want_loss) <= 2e-5 * abs(want_loss), (stage, loss, want_loss)
        assert abs(acc - want_acc) <= 2.0 / n_rows, (stage, acc, want_acc)
        gpu.step(15)
        PH.sync_oracle_to_gpu(orc, gpu, rule)
    gpu.close()


def test_communication_saving_on_c2():
    """The paper's headline behaviour on the covtype-shaped workload: for a comparable full-data loss after the
    same number of iterations, CADA2 uploads far fewer gradients than distributed AMSGrad (c = 0), while the
    stochastic LAG rule at the same c skips (almost) nothing."""
    w = synth.workload("C2")
    Xs, ys, t0 = data(w)
    out = {}
    for name, rule, c in (("adam", O.RULE_CADA2, 0.0), ("cada2", O.RULE_CADA2, 0.6), ("lag", O.RULE_LAG, 0.6)):
        gpu = PH.make_gpu(w, rule, Xs, ys, t0, c=c)
        gpu.step(w.iters)
        loss, acc = gpu.eval()
        out[name] = (gpu.stats().uploads_total, loss, acc)
        gpu.close()
    print("uploads / loss / accuracy:", out)
    assert out["adam"][0] == w.M * w.iters
    assert out["cada2"][0] < 0.5 * out["adam"][0]
    assert out["cada2"][1] < 1.05 * out["adam"][1] + 1e-3
    assert out["lag"][0] > 0.9 * out["adam"][0]
