"""Pins for the CPU oracle: each test checks it against something the paper or the mathematics
fixes independently of the oracle's own formulas (library routines, finite differences,
hand-worked values, limiting cases, invariants)."""
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import cada_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _load(name):
    with open(os.path.join(GOLD, name)) as f:
        return json.load(f)


def _toy(kind, seed=0, n=40, F=6, C=4, H=5):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((n, F)).astype(np.float32)
    if kind == O.MODEL_LOGISTIC:
        y = np.where(rng.random(n) < 0.5, 1.0, -1.0).astype(np.float32)
    else:
        y = rng.integers(0, C, size=n).astype(np.int32)
    return X, y


# ------------------------------------------------------------------------------------------
# sampler and bf16 rounding
# ------------------------------------------------------------------------------------------

def test_splitmix64_published_vectors():
    v = _load("splitmix64_vectors.json")
    got0 = O.splitmix64(0, np.arange(5))
    assert [int(x) for x in got0] == [int(s, 16) for s in v["seed0"]]
    got1 = O.splitmix64(1234567, np.arange(5))
    assert [int(x) for x in got1] == [int(s) for s in v["seed1234567"]]


def test_sampler_is_counter_based_and_in_range():
    M, B = 3, 17
    ns = [5, 1000, 29000]
    a = O.sample_indices(42, 7, M, B, ns)
    assert a.shape == (M, B)
    for m in range(M):
        assert a[m].min() >= 0 and a[m].max() < ns[m]
        # element (k, m, j) is output number (k*M+m)*B+j of the stream, reduced mod N_m
        for j in (0, 5, 16):
            n = (7 * M + m) * B + j
            assert a[m, j] == int(O.splitmix64(42, np.array([n]))[0]) % ns[m]
    # different iterations give different draws; same (seed,k) reproduces
    assert not np.array_equal(a, O.sample_indices(42, 8, M, B, ns))
    assert np.array_equal(a, O.sample_indices(42, 7, M, B, ns))


def test_sampler_roughly_uniform():
    idx = O.sample_indices(3, 0, 1, 200000, [10])[0]
    counts = np.bincount(idx, minlength=10)
    assert np.all(np.abs(counts - 20000) < 5 * math.sqrt(20000 * 0.9))


def test_round_bf16_matches_torch():
    rng = np.random.default_rng(1)
    a = np.concatenate([rng.standard_normal(4096) * 10.0 ** rng.integers(-6, 6, 4096),
                        # exact midpoints between neighbouring bf16 values (ties to even)
                        np.array([1.00390625, 1.01171875, -1.00390625, 3.0078125, 0.0, -0.0])]).astype(np.float32)
    want = torch.from_numpy(a).to(torch.bfloat16).to(torch.float64).numpy()
    got = O.round_bf16(a)
    assert np.array_equal(got, want)


# ------------------------------------------------------------------------------------------
# losses against torch's library routines; gradients against autograd and finite differences
# ------------------------------------------------------------------------------------------

def _torch_loss(kind, X, y, theta, F, C, H, has_bias, lam):
    X = torch.from_numpy(X.astype(np.float64))
    if kind == O.MODEL_LOGISTIC:
        z = X @ theta[:F] + (theta[F] if has_bias else 0.0)
        t = torch.from_numpy((y.astype(np.float64) + 1) / 2)
        data = torch.nn.functional.binary_cross_entropy_with_logits(z, t)
    elif kind == O.MODEL_SOFTMAX:
        z = X @ theta[:F * C].reshape(F, C)
        if has_bias:
            z = z + theta[F * C:]
        data = torch.nn.functional.cross_entropy(z, torch.from_numpy(y.astype(np.int64)))
    else:
        o = 0
        W1 = theta[o:o + F * H].reshape(F, H); o += F * H
        b1 = theta[o:o + H]; o += H
        W2 = theta[o:o + H * C].reshape(H, C); o += H * C
        b2 = theta[o:o + C]
        z = torch.relu(X @ W1 + b1) @ W2 + b2
        data = torch.nn.functional.cross_entropy(z, torch.from_numpy(y.astype(np.int64)))
    return data + 0.5 * lam * (theta @ theta)


@pytest.mark.parametrize("kind,has_bias", [(O.MODEL_LOGISTIC, 0), (O.MODEL_LOGISTIC, 1),
                                           (O.MODEL_SOFTMAX, 0), (O.MODEL_SOFTMAX, 1), (O.MODEL_MLP2, 1)])
def test_loss_and_grad_against_torch(kind, has_bias):
    F, C, H, lam = 6, 4, 5, 0.05
    X, y = _toy(kind, seed=3, F=F, C=C, H=H)
    model = O.Model(kind, F, C, H, has_bias, lam)
    rng = np.random.default_rng(5)
    theta = rng.standard_normal(model.p)
    th = torch.tensor(theta, dtype=torch.float64, requires_grad=True)
    L = _torch_loss(kind, X, y, th, F, C, H, has_bias, lam)
    L.backward()
    assert abs(model.loss(X, y, theta) - L.item()) < 1e-12 * max(1.0, abs(L.item()))
    g = model.grad(X, y, theta)
    assert np.allclose(g, th.grad.numpy(), rtol=1e-11, atol=1e-13)


@pytest.mark.parametrize("kind", [O.MODEL_LOGISTIC, O.MODEL_SOFTMAX, O.MODEL_MLP2, O.MODEL_LSQ])
def test_grad_finite_differences(kind):
    F, C, H = 4, 3, 3
    rng = np.random.default_rng(9)
    X = rng.standard_normal((4, F)).astype(np.float32)
    if kind == O.MODEL_LOGISTIC:
        y = np.array([1, -1, -1, 1], dtype=np.float32)
    elif kind == O.MODEL_LSQ:
        y = rng.standard_normal(4).astype(np.float32)
    else:
        y = np.array([0, 2, 1, 2], dtype=np.int32)
    model = O.Model(kind, F, C, H, has_bias=0 if kind == O.MODEL_LSQ else 1, lam=0.01)
    theta = rng.standard_normal(model.p) * 0.7
    g = model.grad(X, y, theta)
    eps = 1e-6
    for i in range(model.p):
        e = np.zeros(model.p); e[i] = eps
        fd = (model.loss(X, y, theta + e) - model.loss(X, y, theta - e)) / (2 * eps)
        assert abs(fd - g[i]) <= 1e-6 * max(1.0, abs(g[i])), (i, fd, g[i])


def test_logistic_saturation_is_stable():
    model = O.Model(O.MODEL_LOGISTIC, 1)
    X = np.array([[1000.0], [-1000.0]], dtype=np.float32)
    y = np.array([1.0, 1.0], dtype=np.float32)
    g = model.grad(X, y, np.array([1.0]))
    # sigma(1000)-1 = 0, sigma(-1000)-1 = -1  ->  mean of (0*1000, -1*-1000) = 500
    assert np.isfinite(g).all() and abs(g[0] - 500.0) < 1e-9
    assert abs(model.loss(X, y, np.array([1.0])) - 500.0) < 1e-9


def test_mlp_bf16_mode_is_a_small_perturbation_and_exact_on_representable_operands():
    F, C, H = 8, 3, 4
    X, y = _toy(O.MODEL_MLP2, seed=11, n=16, F=F, C=C, H=H)
    X = O.round_bf16(X).astype(np.float32)
    exact = O.Model(O.MODEL_MLP2, F, C, H, 1, 0.0, bf16=False)
    quant = O.Model(O.MODEL_MLP2, F, C, H, 1, 0.0, bf16=True)
    theta = np.random.default_rng(2).standard_normal(exact.p) * 0.5
    g0, g1 = exact.grad(X, y, theta), quant.grad(X, y, theta)
    rel = np.linalg.norm(g1 - g0) / np.linalg.norm(g0)
    assert 0 < rel < 2e-2                    # operand rounding is 2^-9 relative per factor
    # forward pass with operands that are already representable is untouched by the rounding
    theta_q = O.round_bf16(theta)
    theta_q[F * H:F * H + H] = 0.0           # b1 = 0, so a1 = relu(x.W1)
    Xs = np.zeros_like(X); Xs[:, 0] = 1.0    # a1 = relu(W1[0]) exactly representable
    assert abs(exact.loss(Xs, y, theta_q) - quant.loss(Xs, y, theta_q)) < 1e-15


def _hand_mlp():
    from fractions import Fraction
    v = _load("mlp_bf16_hand.json")
    num = lambda seq: np.array([float(Fraction(t)) for t in seq])
    X = num(v["x"]).astype(np.float32)[None, :]
    theta = num(v["theta"])
    assert np.array_equal(theta.astype(np.float32).astype(np.float64), theta)        # the inputs are fp32 values
    model = O.Model(O.MODEL_MLP2, v["n_features"], v["n_classes"], v["n_hidden"], 1, 0.0, bf16=True)
    return v, model, X, np.array([v["label"]], dtype=np.int32), theta, num(v["gradient"])


def test_mlp_bf16_rounding_placement_hand_worked():
    """Fixes WHERE the bf16 roundings of the network's products sit: the hand-worked gradient in the golden file has
    every rounded operand off the bf16 grid, so that each rounding, and the absence of one on the biases and bias
    gradients, moves a stored value."""
    v, model, X, y, theta, want = _hand_mlp()
    got = model.grad(X, y, theta)
    assert np.max(np.abs(got - want)) < 1e-15, (got, want)


def test_mlp_bf16_pin_is_sensitive_to_every_rounding(monkeypatch):
    """Plants each possible mistake in the oracle: with the n-th rounding of the gradient evaluation left out (or with
    the biases / bias gradients rounded as well) the hand-worked values are missed by far more than the pin's tolerance."""
    v, model, X, y, theta, want = _hand_mlp()
    n_roundings = len(v["roundings"])
    calls = []
    real_q = O.Model._q
    monkeypatch.setattr(O.Model, "_q", lambda self, a: (calls.append(1), real_q(self, a))[1])
    model.grad(X, y, theta)
    assert len(calls) == n_roundings                     # the list in the golden file names every rounding once
    for skip in range(n_roundings):
        count = [0]

        def q_skipping(self, a, skip=skip, count=count):
            count[0] += 1
            return np.asarray(a, dtype=np.float64) if count[0] - 1 == skip else real_q(self, a)

        monkeypatch.setattr(O.Model, "_q", q_skipping)
        got = model.grad(X, y, theta)
        assert np.max(np.abs(got - want)) > 1e-4, (v["roundings"][skip], "is not pinned")
    monkeypatch.setattr(O.Model, "_q", real_q)
    # rounding what the contract leaves in full precision is caught too: biases (forward), bias gradients (backward)
    F, H, C = v["n_features"], v["n_hidden"], v["n_classes"]
    th_b = theta.copy()
    th_b[F * H:F * H + H] = O.round_bf16(theta[F * H:F * H + H])
    assert np.max(np.abs(model.grad(X, y, th_b) - want)) > 1e-4
    got = model.grad(X, y, theta)
    for sl in (slice(F * H, F * H + H), slice(F * H + H + H * C, None)):
        assert np.max(np.abs(O.round_bf16(got[sl]) - want[sl])) > 1e-4


# ------------------------------------------------------------------------------------------
# server update (Eqs. 2a-2c)
# ------------------------------------------------------------------------------------------

def test_server_update_hand_worked():
    v = _load("server_update_hand.json")
    theta, h, vhat = np.array([v["theta0"]]), np.zeros(1), np.zeros(1)
    steps = [-1.0, -0.5, -0.525 / math.sqrt(0.3475)]
    for k, nab in enumerate(v["nabla"]):
        new_theta, h, vhat = O.server_update(theta, h, vhat, np.array([nab]), v["alpha"], v["beta1"], v["beta2"], v["eps"])
        assert abs(h[0] - v["h"][k]) < 1e-15
        assert abs(vhat[0] - v["vhat"][k]) < 1e-15
        assert abs((new_theta - theta)[0] - steps[k]) < 1e-15
        theta = new_theta


def test_server_update_equals_torch_amsgrad_when_v_is_monotone():
    """If every coordinate's squared gradient never decreases, v never decreases, vhat = v and
    Eq. 2b coincides with textbook AMSGrad; torch's bias corrections are undone through the
    step size and its epsilon is set to zero (Eq. 2c has it inside the root)."""
    rng = np.random.default_rng(4)
    p, K, alpha, b1, b2 = 7, 12, 0.03, 0.9, 0.99
    base = rng.standard_normal(p)
    base[np.abs(base) < 0.1] = 0.5
    grads = [base * (1.0 + 0.3 * k) * (1 if k % 3 else -1) for k in range(K)]
    th = torch.zeros(p, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([th], lr=alpha, betas=(b1, b2), eps=0.0, amsgrad=True)
    theta, h, vhat = np.zeros(p), np.zeros(p), np.zeros(p)
    for k, g in enumerate(grads):
        t = k + 1
        for grp in opt.param_groups:
            grp["lr"] = alpha * (1 - b1 ** t) / math.sqrt(1 - b2 ** t)
        th.grad = torch.from_numpy(g.copy())
        opt.step()
        theta, h, vhat = O.server_update(theta, h, vhat, g, alpha, b1, b2, 0.0)
        assert np.allclose(theta, th.detach().numpy(), rtol=1e-12, atol=1e-14)


def test_first_step_closed_form():
    """With h0 = vhat0 = 0 the first step is -alpha(1-b1)g/sqrt(eps+(1-b2)g^2): -alpha*sign(g)
    for b1=.9, b2=.99 and |g| >> sqrt(eps), so the first window entry is about alpha^2 p."""
    g = np.array([3.0, -0.5, 2.0, -7.0])
    theta, h, vhat = O.server_update(np.zeros(4), np.zeros(4), np.zeros(4), g, 0.01, 0.9, 0.99, 1e-8)
    assert np.allclose(theta, -0.01 * np.sign(g), rtol=1e-6)


# ------------------------------------------------------------------------------------------
# the rule: hand-worked trajectory with a skip, rule uploads and a forced upload
# ------------------------------------------------------------------------------------------

@pytest.mark.parametrize("rule,key", [(O.RULE_CADA2, "lhs_cada2"), (O.RULE_CADA1, "lhs_cada1")])
def test_hand_worked_lsq_trajectory(rule, key):
    v = _load("cada_lsq_hand.json")
    X = [np.array([[1.0]], dtype=np.float32), np.array([[2.0]], dtype=np.float32)]
    y = [np.array([0.0], dtype=np.float32), np.array([2.0], dtype=np.float32)]
    orc = O.CadaOracle(O.Model(O.MODEL_LSQ, 1), rule, X, y, np.array([v["theta0"]]), batch=1,
                       alpha=v["alpha"], beta1=v["beta1"], beta2=v["beta2"], eps=v["eps"], c=v["c"],
                       d_max=v["d_max"], D=v["D"])
    for k in range(5):
        out = orc.step()
        assert out["rhs"] == v["rhs"][k], k
        assert list(out["lhs"]) == v[key][k], k
        assert [int(u) for u in out["upload"]] == v["upload"][k], k
        assert [int(u) for u in out["forced"]] == v["forced"][k], k
        assert orc.theta[0] == v["theta"][k] and orc.h[0] == v["h"][k] and orc.vhat[0] == v["vhat"][k], k
        assert list(orc.G[:, 0]) == v["G_after"][k], k
        assert list(orc.tau) == v["tau_after"][k], k
    assert (orc.uploads_total, orc.uploads_forced, orc.uploads_rule) == (
        v["uploads_total"], v["uploads_forced"], v["uploads_rule"])


# ------------------------------------------------------------------------------------------
# limiting cases and invariants on a small logistic problem
# ------------------------------------------------------------------------------------------

def _problem(M=4, n=200, F=5, seed=0):
    rng = np.random.default_rng(seed)
    ts = rng.standard_normal(F)
    X, y = [], []
    for m in range(M):
        x = (rng.standard_normal((n, F)) + 0.3 * m).astype(np.float32)
        X.append(x)
        y.append(np.where(x @ ts + 0.5 * rng.standard_normal(n) > 0, 1.0, -1.0).astype(np.float32))
    return X, y


def _make(rule, c, X, y, *, D=10, d_max=4, K=None, alpha=0.05, kind=O.MODEL_LOGISTIC, seed=77, **kw):
    F = X[0].shape[1]
    model = O.Model(kind, F, has_bias=1, lam=1e-3, **kw)
    return O.CadaOracle(model, rule, X, y, np.zeros(model.p), batch=8, alpha=alpha, beta1=0.9, beta2=0.99,
                        eps=1e-8, c=c, d_max=d_max, D=D, seed=seed)


def _independent_amsgrad(X, y, K, *, seed, B, alpha, lam, b1=0.9, b2=0.99, eps=1e-8):
    """Distributed AMSGrad in the paper's form (Section 1 / Eq. 2 with fresh gradients): every
    worker's gradient comes from torch autograd on torch's own loss, averaged, then Eqs. 2a-2c
    retyped with torch ops.  Shares only the index stream with the oracle."""
    M, F = len(X), X[0].shape[1]
    th = torch.zeros(F + 1, dtype=torch.float64)
    h = torch.zeros_like(th); vh = torch.zeros_like(th)
    for k in range(K):
        idx = O.sample_indices(seed, k, M, B, [x.shape[0] for x in X])
        tot = torch.zeros_like(th)
        for m in range(M):
            t = th.clone().requires_grad_(True)
            xb = torch.from_numpy(X[m][idx[m]].astype(np.float64))
            tb = torch.from_numpy((y[m][idx[m]].astype(np.float64) + 1) / 2)
            L = torch.nn.functional.binary_cross_entropy_with_logits(xb @ t[:F] + t[F], tb) + 0.5 * lam * (t @ t)
            L.backward()
            tot += t.grad
        nab = tot / M
        h = b1 * h + (1 - b1) * nab
        vh = torch.maximum(b2 * vh + (1 - b2) * nab * nab, vh)
        th = th - alpha * h / torch.sqrt(eps + vh)
    return th.numpy()


@pytest.mark.parametrize("rule", [O.RULE_CADA1, O.RULE_CADA2])
def test_c_zero_is_distributed_amsgrad(rule):
    X, y = _problem()
    K = 25
    orc = _make(rule, 0.0, X, y)
    for _ in range(K):
        out = orc.step()
        assert out["upload"].all()
    assert orc.uploads_total == len(X) * K
    ref = _independent_amsgrad(X, y, K, seed=77, B=8, alpha=0.05, lam=1e-3)
    assert np.allclose(orc.theta, ref, rtol=1e-10, atol=1e-12)


def test_single_worker_c_zero_is_single_node_amsgrad():
    X, y = _problem(M=1)
    orc = _make(O.RULE_CADA2, 0.0, X, y)
    for _ in range(15):
        orc.step()
    ref = _independent_amsgrad(X, y, 15, seed=77, B=8, alpha=0.05, lam=1e-3)
    assert np.allclose(orc.theta, ref, rtol=1e-10, atol=1e-12)


@pytest.mark.parametrize("rule", [O.RULE_CADA1, O.RULE_CADA2])
def test_c_infinite_uploads_only_every_D(rule):
    X, y = _problem()
    D, K = 7, 30
    orc = _make(rule, math.inf, X, y, D=D)
    for k in range(K):
        G_before = orc.G.copy()
        out = orc.step()
        if k % D == 0:
            assert out["upload"].all() and out["forced"].all()
        else:
            assert not out["upload"].any()
            assert np.array_equal(orc.G, G_before)
    assert orc.uploads_total == len(X) * math.ceil(K / D)
    assert orc.uploads_rule == 0


def test_rules_coincide_when_the_rule_cannot_matter():
    X, y = _problem()
    for c in (0.0, math.inf):
        a, b = _make(O.RULE_CADA1, c, X, y), _make(O.RULE_CADA2, c, X, y)
        for _ in range(25):
            a.step(); b.step()
        assert np.array_equal(a.theta, b.theta) and np.array_equal(a.vhat, b.vhat)


@pytest.mark.parametrize("rule", [O.RULE_CADA1, O.RULE_CADA2])
def test_invariants(rule):
    X, y = _problem(M=5)
    D, d_max, alpha = 6, 4, 0.05
    orc = _make(rule, 2.0, X, y, D=D, d_max=d_max, alpha=alpha)
    b1, b2 = 0.9, 0.99
    b3 = b1 * b1 / b2
    bound = alpha ** 2 * orc.p / ((1 - b2) * (1 - b3))          # Lemma 4
    last_upload = np.full(5, -1)
    skipped = 0
    for k in range(60):
        vh_before = orc.vhat.copy()
        out = orc.step()
        skipped += int((~out["upload"]).sum())
        last_upload[out["upload"]] = k
        assert np.all(k - last_upload < D)                        # at least one upload in any D iterations
        assert np.all((orc.tau >= 1) & (orc.tau <= D))
        assert np.all(orc.vhat >= vh_before)                      # vhat = max(v, vhat)
        assert np.all(orc.ring <= bound * (1 + 1e-12))
        assert np.allclose(orc.last_nabla, orc.nabla_rec, rtol=1e-12, atol=1e-15)   # recursive form of the aggregate
        assert orc.uploads_forced + orc.uploads_rule == orc.uploads_total
        # window holds the last d_max squared step norms
    assert skipped > 0 and orc.uploads_rule > 0                   # the case exercises both branches


def test_window_is_last_dmax_step_norms():
    X, y = _problem()
    orc = _make(O.RULE_CADA2, 0.5, X, y, d_max=3)
    steps = []
    for k in range(8):
        rhs_expected = (0.5 / 3) * sum(steps[-3:])
        th = orc.theta.copy()
        out = orc.step()
        assert abs(out["rhs"] - rhs_expected) <= 1e-15 * max(1.0, rhs_expected)
        steps.append(float(np.sum((orc.theta - th) ** 2)))


def test_upload_count_monotone_in_c():
    X, y = _problem(M=6, n=400)
    for rule in (O.RULE_CADA1, O.RULE_CADA2):
        counts = []
        for c in (0.0, 0.3, 0.6, 1.2, 5.0, math.inf):
            orc = _make(rule, c, X, y, D=20, d_max=5)
            for _ in range(80):
                orc.step()
            counts.append(orc.uploads_total)
        assert counts[0] == 6 * 80 and counts[-1] == 6 * 4
        assert all(a >= b for a, b in zip(counts, counts[1:])), counts


def test_lag_rule_compares_against_stored_gradient():
    """Eq. 4: the stochastic-LAG left-hand side is the squared distance between the fresh
    gradient and the copy the server holds (different iterate AND different sample)."""
    X, y = _problem()
    orc = _make(O.RULE_LAG, 0.6, X, y)
    orc.step()
    G = orc.G.copy()
    out = orc.propose()
    for m in range(len(X)):
        assert abs(out["lhs"][m] - float(np.sum((out["g"][m] - G[m]) ** 2))) < 1e-15


def test_rounding_hint_is_used_only_inside_the_tie_band():
    """The tie protocol for bf16 roundings: another implementation's rounding is taken over only where its unrounded
    operand agrees with the oracle's to 1e-5 of the operand's largest entry (so that the rounding boundary lies that
    close to the oracle's own value); a hint that differs by more is ignored, and so is every hint in fp64 mode."""
    model = O.Model(O.MODEL_MLP2, 2, 2, 1, 1, 0.0, bf16=True)
    mid = 1.0 + 2.0 ** -8                          # boundary between the bf16 neighbours 1 and 1 + 2^-7
    a = np.array([mid - 3e-7, 3.0, 1.003])
    assert np.array_equal(model._q_tie(a, None), [1.0, 3.0, 1.0])
    model.round_ties = 0
    near = np.array([mid + 3e-7, 3.0, 1.003])      # first entry: 6e-7 apart, rounds up on the other side
    assert np.array_equal(model._q_tie(a, near), [1.0 + 2.0 ** -7, 3.0, 1.0]) and model.round_ties == 1
    far = np.array([mid + 1e-3, 3.0, 1.0045])      # apart by far more than 3e-5: the oracle keeps its own roundings
    assert np.array_equal(model._q_tie(a, far), [1.0, 3.0, 1.0]) and model.round_ties == 1
    exact = O.Model(O.MODEL_MLP2, 2, 2, 1, 1, 0.0, bf16=False)
    assert np.array_equal(exact._q_tie(a, near), a) and exact.round_ties == 0
    # through the gradient: hints equal to the oracle's own operands change nothing
    X = np.array([[0.5, 1.5], [1.25, -0.75]], dtype=np.float32)
    y = np.array([0, 1], dtype=np.int32)
    theta = np.random.default_rng(4).standard_normal(model.p) * 0.7
    base = model.grad(X, y, theta)
    own = {k: v.copy() for k, v in model.last_operands.items()}
    assert np.array_equal(model.grad(X, y, theta, operand_hint=own), base) and model.round_ties == 1


def test_relu_hint_is_used_only_inside_the_tie_band():
    """The derivative mask of the hidden layer follows the oracle's own sign of z1 except where |z1| is below
    the tie threshold, where a supplied decision is adopted (and counted)."""
    F, C, H = 3, 2, 2
    model = O.Model(O.MODEL_MLP2, F, C, H, 1, 0.0)
    X = np.array([[1.0, 0.0, 0.0], [0.0, 1.0, 0.0]], dtype=np.float32)
    y = np.array([0, 1], dtype=np.int32)
    W1 = np.array([[0.5, 2e-6], [-0.7, -3e-6], [0.1, 0.2]])        # z1 = rows 0/1 of W1: one clear and one tiny entry each
    theta = np.concatenate([W1.ravel(), np.zeros(H), np.array([0.3, -0.2, 0.4, 0.1]), np.zeros(C)])
    base = model.grad(X, y, theta)
    same = model.grad(X, y, theta, relu_hint=np.array([[True, True], [False, False]]))     # agrees with the signs
    assert np.array_equal(base, same)
    model.relu_ties = 0
    flipped_clear = model.grad(X, y, theta, relu_hint=np.array([[False, True], [True, False]]))   # clear entries: ignored
    assert np.array_equal(base, flipped_clear) and model.relu_ties == 0
    flipped_tiny = model.grad(X, y, theta, relu_hint=np.array([[True, False], [False, True]]))    # tiny entries: adopted
    assert model.relu_ties == 2 and not np.array_equal(base, flipped_tiny)
    # adopting "inactive" for unit 1 of row 0 removes that row's contribution to W1[:, 1]
    assert flipped_tiny[0 * H + 1] == 0.0 and base[0 * H + 1] != 0.0


def test_hand_worked_lag_with_sgd_server():
    v = _load("lag_sgd_hand.json")
    X = [np.array([[1.0], [1.0]], dtype=np.float32)]
    y = [np.array([0.0, 1.0], dtype=np.float32)]
    orc = O.CadaOracle(O.Model(O.MODEL_LSQ, 1), O.RULE_LAG, X, y, np.array([v["theta0"]]), batch=1, alpha=v["alpha"],
                       beta1=0.9, beta2=0.99, eps=1e-8, c=v["c"], d_max=v["d_max"], D=v["D"], server="sgd")
    for k, row in enumerate(v["rows"]):
        out = orc.step(np.array([[row]]))
        # at k = 0 the server holds 0, so LHS = g^2 = 1; afterwards the stored gradient of the last upload
        assert out["lhs"][0] == v["lhs"][k] and out["rhs"] == v["rhs"][k], k
        assert int(out["upload"][0]) == v["upload"][k] and int(out["forced"][0]) == v["forced"][k], k
        assert orc.G[0, 0] == v["G_after"][k] and orc.theta[0] == v["theta"][k], k
    assert np.all(orc.h == 0) and np.all(orc.vhat == 0)          # the SGD server keeps no moments


def test_evaluate_against_torch():
    """Full-data objective of Eq. 1 (mean over workers of each worker's mean loss, regulariser included) and pooled
    accuracy, against torch's loss routine and arg-max."""
    X, y = [], []
    rng = np.random.default_rng(21)
    F, C = 5, 3
    for n in (30, 50):                                   # unequal workers: Eq. 1 weighs workers, not rows
        X.append(rng.standard_normal((n, F)).astype(np.float32))
        y.append(rng.integers(0, C, size=n).astype(np.int32))
    model = O.Model(O.MODEL_SOFTMAX, F, C, 0, 1, 0.02)
    theta = rng.standard_normal(model.p)
    orc = O.CadaOracle(model, O.RULE_CADA2, X, y, theta, batch=4, alpha=0.01, beta1=0.9, beta2=0.99, eps=1e-8, c=0.5, d_max=3, D=5)
    loss, acc = orc.evaluate()
    th = torch.tensor(theta)
    want, ok = 0.0, 0
    for xm, ym in zip(X, y):
        z = torch.from_numpy(xm.astype(np.float64)) @ th[:F * C].reshape(F, C) + th[F * C:]
        want += torch.nn.functional.cross_entropy(z, torch.from_numpy(ym.astype(np.int64))).item() / 2
        ok += int((z.argmax(dim=1).numpy() == ym).sum())
    want += 0.5 * 0.02 * float(th @ th)
    assert abs(loss - want) < 1e-12 and acc == ok / 80


# ------------------------------------------------------------------------------------------
# recursive aggregate (Eq. 3), diminishing step size (Theorem 2), per-worker batch sizes
# ------------------------------------------------------------------------------------------

@pytest.mark.parametrize("rule,key", [(O.RULE_CADA2, "lhs_cada2"), (O.RULE_CADA1, "lhs_cada1")])
def test_recursive_aggregate_reproduces_the_hand_worked_trajectory(rule, key):
    """Eq. 3 refines nabla^{k-1} by the uploaded innovations; in exact (here dyadic) arithmetic it is the slot sum of
    Eq. 2a, so the hand-worked values must come out unchanged."""
    v = _load("cada_lsq_hand.json")
    X = [np.array([[1.0]], dtype=np.float32), np.array([[2.0]], dtype=np.float32)]
    y = [np.array([0.0], dtype=np.float32), np.array([2.0], dtype=np.float32)]
    orc = O.CadaOracle(O.Model(O.MODEL_LSQ, 1), rule, X, y, np.array([v["theta0"]]), batch=1,
                       alpha=v["alpha"], beta1=v["beta1"], beta2=v["beta2"], eps=v["eps"], c=v["c"],
                       d_max=v["d_max"], D=v["D"], aggregate="recursive")
    for k in range(5):
        out = orc.step()
        assert list(out["lhs"]) == v[key][k] and [int(u) for u in out["upload"]] == v["upload"][k], k
        assert orc.theta[0] == v["theta"][k] and orc.h[0] == v["h"][k] and orc.vhat[0] == v["vhat"][k], k
        assert orc.last_nabla[0] == sum(v["G_after"][k]) / 2, k


@pytest.mark.parametrize("rule", [O.RULE_CADA1, O.RULE_CADA2, O.RULE_LAG])
def test_recursive_aggregate_follows_the_slot_sum(rule):
    X, y = _problem()
    a = _make(rule, 0.6, X, y)
    F = X[0].shape[1]
    model = O.Model(O.MODEL_LOGISTIC, F, has_bias=1, lam=1e-3)
    b = O.CadaOracle(model, rule, X, y, np.zeros(model.p), batch=8, alpha=0.05, beta1=0.9, beta2=0.99, eps=1e-8,
                     c=0.6, d_max=4, D=10, seed=77, aggregate="recursive")
    skipped = 0
    for k in range(120):
        oa, ob = a.step(), b.step()
        assert np.array_equal(oa["upload"], ob["upload"]), k
        skipped += int(np.sum(~oa["upload"]))
        assert np.max(np.abs(a.theta - b.theta)) <= 1e-12 * max(1.0, np.max(np.abs(a.theta))), k
    assert skipped > 0 or rule == O.RULE_LAG      # stale slots were exercised (Eq. 4 hardly ever skips at this c)


def test_diminishing_step_closed_form_on_a_quadratic():
    """Theorem 2's alpha_k = 2 / (mu (k + K0)).  One worker, one row x = a, l = (a theta - b)^2 / 2, so mu = a^2 and
    theta^{k+1} - theta* = (1 - 2/(k + K0)) (theta^k - theta*).  With K0 = 3 the factors telescope:
    prod_{k<K} (k+1)/(k+3) = 2 / ((K+1)(K+2))."""
    a_, b_ = 2.0, 3.0
    X, y = [np.array([[a_]], dtype=np.float32)], [np.array([b_], dtype=np.float32)]
    orc = O.CadaOracle(O.Model(O.MODEL_LSQ, 1), O.RULE_CADA2, X, y, np.array([5.0]), batch=1, alpha=2.0 / a_ ** 2,
                       beta1=0.9, beta2=0.99, eps=1e-8, c=0.0, d_max=2, D=5, server="sgd", alpha_K0=3.0)
    star, e0 = b_ / a_, 5.0 - b_ / a_
    for K in range(1, 30):
        orc.step()
        assert abs((orc.theta[0] - star) - e0 * 2.0 / ((K + 1) * (K + 2))) <= 1e-13 * abs(e0), K


def test_diminishing_step_scales_the_amsgrad_step():
    """Eq. 2c with alpha replaced by alpha_k: from h = vhat = 0, at every k, the step is alpha/(k+K0) times the
    direction, so two runs that differ only in K0 take first steps in the ratio of their alpha_0."""
    X, y = _problem(M=2)
    steps = []
    for K0 in (2.0, 8.0):
        model = O.Model(O.MODEL_LOGISTIC, X[0].shape[1], has_bias=1, lam=1e-3)
        orc = O.CadaOracle(model, O.RULE_CADA2, X, y, np.zeros(model.p), batch=8, alpha=0.4, beta1=0.9, beta2=0.99,
                           eps=1e-8, c=0.5, d_max=4, D=10, seed=3, alpha_K0=K0)
        orc.step()
        steps.append(orc.theta.copy())
    assert np.allclose(steps[0] * 2.0, steps[1] * 8.0, rtol=1e-13, atol=0)
    g = np.array([1.5, -2.0])
    t1, _, _ = O.server_update(np.zeros(2), np.zeros(2), np.zeros(2), g, 0.4 / 8.0, 0.9, 0.99, 1e-8)
    assert np.allclose(t1, -(0.4 / 8.0) * 0.1 * g / np.sqrt(1e-8 + 0.01 * g * g), rtol=1e-14)


def test_per_worker_batch_sizes_against_autograd():
    """Batch ratio of the supplement: worker m averages over its own number of rows.  One SGD-server step with c = 0
    (every worker uploads) must equal theta - alpha * mean_m grad_m, each grad_m from torch autograd over the first
    batch_m[m] rows of the worker's index stream."""
    X, y = _problem(M=3, n=50)
    F = X[0].shape[1]
    model = O.Model(O.MODEL_LOGISTIC, F, has_bias=1, lam=1e-2)
    rng = np.random.default_rng(5)
    theta0 = rng.standard_normal(model.p)
    bm = [8, 3, 1]
    orc = O.CadaOracle(model, O.RULE_CADA2, X, y, theta0, batch=8, alpha=0.1, beta1=0.9, beta2=0.99, eps=1e-8,
                       c=0.0, d_max=4, D=10, seed=11, server="sgd", batch_m=bm)
    idx = O.sample_indices(11, 0, 3, 8, [50, 50, 50])
    grads = []
    for m in range(3):
        t = torch.tensor(theta0, dtype=torch.float64, requires_grad=True)
        rows = idx[m][: bm[m]]
        xb = torch.tensor(X[m][rows], dtype=torch.float64)
        yb = torch.tensor(y[m][rows], dtype=torch.float64)
        z = xb @ t[:F] + t[F]
        loss = torch.nn.functional.softplus(-yb * z).mean() + 0.5 * 1e-2 * (t @ t)
        loss.backward()
        grads.append(t.grad.numpy())
    orc.step()
    assert np.allclose(orc.theta, theta0 - 0.1 * np.mean(grads, axis=0), rtol=1e-12, atol=1e-14)
    assert np.allclose(orc.G, np.array(grads), rtol=1e-12, atol=1e-14)
