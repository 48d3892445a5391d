"""Lock-step comparison of libcada (through its C ABI) with the CPU oracle on identical inputs.

Protocol per iteration:
  1. the oracle evaluates both gradients of every worker and its own decisions (``propose``);
  2. the library runs one iteration; its decisions and left-hand sides are read back;
  3. forced uploads (tau >= D) are integer logic and must agree; a rule decision may differ only
     when the oracle's margin |LHS - RHS| / max(LHS, RHS) is within ``band`` (1e-4), in which case
     the oracle adopts the library's decision and the hit is counted;
  4. the oracle commits; theta, h and vhat must agree to ``tol`` (1e-5) in the max-norm relative
     sense  max|gpu - oracle| / max|oracle|;
  5. optionally the oracle's state is then overwritten by the library's (``resync``) so that the
     next comparison measures that step's error alone rather than accumulated drift.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional

import numpy as np

from oracle import cada_oracle as O
from paper_2012_15469_b200 import binding as B
from paper_2012_15469_b200 import synth


@dataclasses.dataclass
class Report:
    iters: int = 0
    band_hits: int = 0
    max_rel_theta: float = 0.0
    max_rel_h: float = 0.0
    max_rel_vhat: float = 0.0
    max_rel_lhs: float = 0.0
    max_rel_rhs: float = 0.0
    uploads: int = 0
    skips: int = 0
    forced: int = 0
    relu_ties: int = 0          # MLP: hidden-unit sign decisions the oracle took over from the library (inside its tie band)
    max_relu_ties_per_iter: int = 0
    round_ties: int = 0         # MLP: bf16 rounding decisions taken over from the library (unrounded operands within the tie band)
    max_operand_dev: float = 0.0    # MLP: largest max-norm-relative distance between the two sides' unrounded operands
    max_grad_err: float = 0.0   # with check_grads: worst max-norm-relative error of a worker gradient ...
    max_innov_err: float = 0.0  # ... and of an innovation (against |g| with innovation_noise_floor, else against |d|)
    max_lhs_excess: float = 0.0     # worst left-hand-side deviation divided by its cancellation factor
    max_adopted_margin: float = 0.0  # largest margin |LHS - RHS| / max at which a differing decision was adopted
    max_rel_step: float = 0.0   # worst relative deviation of the squared step norm pushed into the window


def rel_inf(a: np.ndarray, b: np.ndarray) -> float:
    """max|a-b| / max|b| (0 when both vanish)."""
    den = float(np.max(np.abs(b))) if b.size else 0.0
    num = float(np.max(np.abs(a.astype(np.float64) - b))) if b.size else 0.0
    if den == 0.0:
        return 0.0 if num == 0.0 else float("inf")
    return num / den


def make_oracle(w: synth.Workload, rule: int, Xs, ys, theta0, *, c=None, tau0=None, seed=None, server=0,
                aggregate=0, alpha_K0=0.0, batch_m=None, alpha=None) -> O.CadaOracle:
    model = O.Model(w.model, w.n_features, w.n_classes, w.n_hidden, w.has_bias, w.lam, bf16=w.x_bf16)
    return O.CadaOracle(model, rule, Xs, ys, theta0, batch=w.batch,
                        alpha=np.float32(w.alpha if alpha is None else alpha).item(),
                        beta1=np.float32(w.beta1).item(), beta2=np.float32(w.beta2).item(),
                        eps=np.float32(w.eps).item(), c=np.float32(w.c if c is None else c).item(),
                        d_max=w.d_max, D=w.D, seed=w.sample_seed if seed is None else seed, tau0=tau0,
                        server="sgd" if server else "amsgrad", aggregate="recursive" if aggregate else "slots",
                        alpha_K0=np.float32(alpha_K0).item(), batch_m=batch_m)


def make_gpu(w: synth.Workload, rule: int, Xs, ys, theta0, *, c=None, tau0=None, seed=None, history=0,
             host_step=False, device="cuda", server=0, aggregate=0, alpha_K0=0.0, batch_m=None, alpha=None,
             M_total=0, m_first=0, m_stride=0) -> B.Cada:
    import torch

    if w.x_bf16:
        Xd = [torch.from_numpy(x).to(device).to(torch.bfloat16).contiguous() for x in Xs]
    else:
        Xd = [torch.from_numpy(x).to(device) for x in Xs]
    yd = [torch.from_numpy(y).to(device) for y in ys]
    t0 = torch.from_numpy(np.asarray(theta0, dtype=np.float32)).to(device)
    return B.Cada(model=w.model, rule=rule, X=Xd, y=yd, theta0=t0, batch=w.batch,
                  alpha=w.alpha if alpha is None else alpha, beta1=w.beta1,
                  beta2=w.beta2, eps=w.eps, c=w.c if c is None else c, d_max=w.d_max, D=w.D, lam=w.lam,
                  n_features=w.n_features, n_classes=w.n_classes, n_hidden=w.n_hidden, has_bias=w.has_bias,
                  seed=w.sample_seed if seed is None else seed, tau0=tau0, history_capacity=history,
                  host_step=host_step, server=server, aggregate=aggregate, alpha_K0=alpha_K0, batch_m=batch_m,
                  M_total=M_total, m_first=m_first, m_stride=m_stride)


def sync_oracle_to_gpu(orc: O.CadaOracle, gpu: B.Cada, rule: int) -> None:
    orc.theta = gpu.read(B.CADA_BUF_THETA).astype(np.float64)
    orc.h = gpu.read(B.CADA_BUF_H).astype(np.float64)
    orc.vhat = gpu.read(B.CADA_BUF_VHAT).astype(np.float64)
    orc.G = gpu.read(B.CADA_BUF_G).astype(np.float64)
    orc.ring = gpu.read(B.CADA_BUF_RING).astype(np.float64)
    if orc.aggregate == "recursive":
        orc.nabla_rec = gpu.read(B.CADA_BUF_NABLA).astype(np.float64)
    if rule == O.RULE_CADA2:
        orc.theta_hat = gpu.read(B.CADA_BUF_THETA_HAT).astype(np.float64)
    elif rule == O.RULE_CADA1:
        orc.delta_stored = gpu.read(B.CADA_BUF_DELTA_STORED).astype(np.float64)
        orc.theta_tilde = gpu.read(B.CADA_BUF_THETA_TILDE).astype(np.float64)


def lockstep(gpu: B.Cada, orc: O.CadaOracle, iters: int, *, rule: int, tol: float = 1e-5, band: float = 1e-4,
             resync: bool = True, idx_fn=None, check_grads: bool = False, grad_tol: float = 2e-5,
             innovation_noise_floor: bool = False, lhs_tol: float = 1e-4, rhs_tol: Optional[float] = None,
             relu_ties_per_iter: int = 50, round_ties: bool = False, operand_tol: float = 1e-5,
             step_tol: Optional[float] = None) -> Report:
    """``innovation_noise_floor``: judge the innovation d_m against the scale of g_m (quantised models, where both
    gradients carry rounding noise proportional to |g| and their difference can be much smaller than either).

    ``lhs_tol`` bounds the relative deviation of the library's left-hand sides (Eqs. 6/8) from the oracle's at every
    iteration (1e-4, the width of the decision band: a larger deviation could move a decision that lies outside it),
    times the cancellation factor of the difference the norm is taken of: the library squares a difference
    e = a - b of two fp32 vectors, so the relative error of ||e||^2 grows like (||a|| + ||b||) / ||e||.  For CADA1 that
    is (d_m, stored innovation), for the stochastic-LAG rule (g_m, server copy); CADA2's d_m is formed without
    cancellation for the logistic and softmax models (factor 1), while the network's d_m is the difference of two
    separately evaluated gradients.  ``rhs_tol`` bounds the deviation of the right-hand side (default: 1e-9 with
    re-synchronisation, where both sides sum the same window in fp64, else ``20 * tol``).  ``relu_ties_per_iter`` caps
    the hidden-unit sign decisions the MLP oracle may take over from the library in one iteration.  ``round_ties``
    (MLP): hand the library's unrounded a1, dz2 and dz1 to the oracle, which adopts a differing bf16 rounding where the
    unrounded values agree within its tie band; the unrounded operands must agree to ``operand_tol`` everywhere."""
    rep = Report()
    if not resync:
        lhs_tol = max(lhs_tol, 20 * tol)            # free-running: the two trajectories drift apart
    if rhs_tol is None:
        rhs_tol = 1e-9 if resync else 20 * tol
    if step_tol is None:            # the step is a difference of fp32 iterates: its relative accuracy is that of theta times |theta| / |step|
        step_tol = 1e-3 if resync else 4e-3
    for it in range(iters):
        idx = idx_fn(orc.k) if idx_fn is not None else None
        gpu.step(1)
        hint, operands = None, None
        if orc.model.kind == O.MODEL_MLP2:      # decisions z1 > 0 of the library, adopted by the oracle inside its tie band only
            z1 = gpu.read(B.CADA_BUF_MLP_Z1)
            hint = z1 > 0
            if round_ties:
                operands = {"a1": np.maximum(z1, 0.0), "dz2": gpu.read(B.CADA_BUF_MLP_DZ2), "dz1": gpu.read(B.CADA_BUF_MLP_DZ1)}
        ties_before, rties_before = orc.model.relu_ties, orc.model.round_ties
        out = orc.propose(idx, relu_hint=hint, operand_hint=operands)
        rep.round_ties += orc.model.round_ties - rties_before
        for key, dev in out["operand_dev"].items():
            assert dev <= operand_tol, f"iteration {orc.k}: unrounded operand {key} differs by {dev:.3e}; so far {rep}"
            rep.max_operand_dev = max(rep.max_operand_dev, dev)
        ties = orc.model.relu_ties - ties_before
        rep.relu_ties += ties
        rep.max_relu_ties_per_iter = max(rep.max_relu_ties_per_iter, ties)
        assert ties <= relu_ties_per_iter, f"iteration {orc.k}: {ties} hidden-unit sign decisions taken over from the library"
        bits = gpu.read(B.CADA_BUF_LAST_MASK)
        up_gpu = (bits & 1).astype(bool)
        forced_gpu = ((bits >> 1) & 1).astype(bool)
        lhs_gpu = gpu.read(B.CADA_BUF_LAST_LHS)
        rhs_gpu = gpu.stats().last_rhs
        assert np.array_equal(forced_gpu, out["forced"]), f"iteration {orc.k}: forced-upload sets differ"
        decision = out["upload"].copy()
        for m in np.nonzero(up_gpu != out["upload"])[0]:
            lhs, rhs = out["lhs"][m], out["rhs"]
            margin = abs(lhs - rhs) / max(lhs, rhs, 1e-300)
            assert margin <= band, (f"iteration {orc.k}, worker {m}: decisions differ outside the band: "
                                    f"oracle LHS={lhs:.9e} RHS={rhs:.9e} margin={margin:.3e} gpu LHS={lhs_gpu[m]:.9e}")
            decision[m] = up_gpu[m]
            rep.band_hits += 1
            rep.max_adopted_margin = max(rep.max_adopted_margin, margin)
        if check_grads:
            g = gpu.read(B.CADA_BUF_GRAD_FRESH)
            d = gpu.read(B.CADA_BUF_INNOV_FRESH)
            for m in range(orc.M):
                ge = rel_inf(g[m], out["g"][m])
                assert ge <= grad_tol, f"iteration {orc.k}, worker {m}: gradient off by {ge:.3e}; so far {rep}"
                rep.max_grad_err = max(rep.max_grad_err, ge)
                if innovation_noise_floor:
                    err = float(np.max(np.abs(d[m] - out["d"][m]))) / float(np.max(np.abs(out["g"][m])))
                    assert err <= 2 * grad_tol, f"iteration {orc.k}, worker {m}: innovation off by {err:.3e} of |g|; so far {rep}"
                    rep.max_innov_err = max(rep.max_innov_err, err)
                elif np.max(np.abs(out["d"][m])) > 0:
                    err = rel_inf(d[m], out["d"][m])
                    assert err <= 10 * grad_tol, f"iteration {orc.k}, worker {m}: innovation off by {err:.3e}; so far {rep}"
                    rep.max_innov_err = max(rep.max_innov_err, err)
        big = np.maximum(out["lhs"], 1e-300)
        ok = out["lhs"] > 1e-30
        if ok.any():
            # cancellation factor of the difference whose norm the left-hand side is (see the docstring)
            norm = lambda a: np.sqrt(np.sum(np.square(a), axis=1))
            pair = np.zeros(orc.M)
            if rule == O.RULE_CADA1:
                pair = norm(out["d"]) + norm(orc.delta_stored)
            elif rule == O.RULE_LAG:
                pair = norm(out["g"]) + norm(orc.G)
            if innovation_noise_floor and rule != O.RULE_LAG:
                pair = pair + 2.0 * norm(out["g"])
            kappa = np.maximum(1.0, pair / np.sqrt(big))
            dev = np.where(ok, np.abs(lhs_gpu - out["lhs"]) / big, 0.0)
            excess = dev / kappa
            worst = int(np.argmax(excess))
            assert excess[worst] <= lhs_tol, (
                f"iteration {orc.k}, worker {worst}: left-hand side off by {dev[worst]:.3e} with cancellation factor "
                f"{kappa[worst]:.3g} (oracle {out['lhs'][worst]:.9e}, library {lhs_gpu[worst]:.9e}); so far {rep}")
            rep.max_rel_lhs = max(rep.max_rel_lhs, float(np.max(dev)))
            rep.max_lhs_excess = max(rep.max_lhs_excess, float(excess[worst]))
        if np.isfinite(out["rhs"]) and out["rhs"] > 0:
            dev_r = abs(rhs_gpu - out["rhs"]) / out["rhs"]
            assert dev_r <= rhs_tol, f"iteration {orc.k}: right-hand side off by {dev_r:.3e}; so far {rep}"
            rep.max_rel_rhs = max(rep.max_rel_rhs, dev_r)
        orc.commit(decision)
        rt = rel_inf(gpu.read(B.CADA_BUF_THETA), orc.theta)
        rh = rel_inf(gpu.read(B.CADA_BUF_H), orc.h)
        rv = rel_inf(gpu.read(B.CADA_BUF_VHAT), orc.vhat)
        assert rt <= tol and rh <= tol and rv <= tol, (f"iteration {orc.k - 1}: rel err theta={rt:.3e} h={rh:.3e} vhat={rv:.3e} > {tol}; "
                                                     f"so far {rep}")
        rep.max_rel_theta, rep.max_rel_h, rep.max_rel_vhat = max(rep.max_rel_theta, rt), max(rep.max_rel_h, rh), max(rep.max_rel_vhat, rv)
        assert np.array_equal(gpu.read(B.CADA_BUF_TAU), orc.tau.astype(np.int32)), f"iteration {orc.k - 1}: staleness differs"
        # the newest window term ||theta^{k+1} - theta^k||^2 (compared before any re-synchronisation overwrites the oracle's)
        slot = (orc.k - 1) % orc.d_max
        step_o, step_g = float(orc.ring[slot]), float(gpu.read(B.CADA_BUF_RING)[slot])
        if step_o > 0:
            rs = abs(step_g - step_o) / step_o
            assert rs <= step_tol, f"iteration {orc.k - 1}: squared step norm off by {rs:.3e} (oracle {step_o:.9e}, library {step_g:.9e}); so far {rep}"
            rep.max_rel_step = max(rep.max_rel_step, rs)
        # the records an upload refreshes (compared before any re-synchronisation can hide a stale copy)
        rg = rel_inf(gpu.read(B.CADA_BUF_G), orc.G)
        assert rg <= 20 * tol, f"iteration {orc.k - 1}: stored gradients differ, rel err {rg:.3e}"
        if rule == O.RULE_CADA2:
            rr = rel_inf(gpu.read(B.CADA_BUF_THETA_HAT), orc.theta_hat)
        elif rule == O.RULE_LAG:
            rr = 0.0
        else:
            rr = max(rel_inf(gpu.read(B.CADA_BUF_DELTA_STORED), orc.delta_stored),
                     rel_inf(gpu.read(B.CADA_BUF_THETA_TILDE), orc.theta_tilde))
        assert rr <= 20 * tol, f"iteration {orc.k - 1}: upload records differ, rel err {rr:.3e}"
        if orc.aggregate == "recursive":
            rn = rel_inf(gpu.read(B.CADA_BUF_NABLA), orc.nabla_rec)
            assert rn <= 20 * tol, f"iteration {orc.k - 1}: recursive aggregate differs, rel err {rn:.3e}"
        rep.uploads += int(decision.sum()); rep.skips += int((~decision).sum()); rep.forced += int(out["forced"].sum())
        rep.iters += 1
        if resync:
            sync_oracle_to_gpu(orc, gpu, rule)
    st = gpu.stats()
    assert st.k == orc.k
    assert st.uploads_total == orc.uploads_total and st.uploads_forced == orc.uploads_forced and st.uploads_rule == orc.uploads_rule
    assert np.array_equal(gpu.read(B.CADA_BUF_UPLOADS_PER_WORKER), orc.uploads_per_worker)
    assert st.status_flags == 0
    return rep
