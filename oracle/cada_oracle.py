"""TEST INFRASTRUCTURE ONLY -- slow, plain, double-precision statement of one CADA iteration.

This file restates, step by step and in the paper's notation, what "CADA: Communication-
Adaptive Distributed Adam" (arXiv 2012.15469) computes: Algorithm 1 with the CADA1 rule
(Eq. 6) or the CADA2 rule (Eq. 8), the forced upload at staleness D, the stale-gradient
aggregation (Eq. 2a) and the AMSGrad-style server update (Eqs. 2a-2c).  It exists so that
the CUDA library can be checked against it.  It shares no code with that library and must
never be imported by it: only tests, the smoke check and the benchmark's CPU-baseline leg
may use it.

Arithmetic is float64 throughout (inputs are the same fp32 bytes the GPU sees, widened).
numpy's matmul is the only library primitive used; there is no blocking, fusion or
reordering beyond what the equations state.

Pins (all in tests/test_oracle_*.py, none of which re-use this file's formulas):
  * losses against torch's library cross-entropy routines; gradients against central finite
    differences of those losses and against torch autograd;
  * the server update against hand-worked values of Eqs. 2a-2c (tests/golden/) and, where
    the recursion coincides with textbook AMSGrad, against torch.optim.Adam(amsgrad=True);
  * the upload rule against a hand-worked least-squares trajectory (tests/golden/) that
    contains a skip, a rule-triggered upload and a forced upload;
  * c = 0 (every worker uploads: distributed AMSGrad), c = +inf (uploads only every D),
    M = 1, the slot-sum / recursive-innovation equivalence, Lemma 4's step bound, and the
    monotonicity of v-hat;
  * the minibatch sampler against published SplitMix64 output vectors;
  * bfloat16 rounding against torch's conversion; the placement of the network's operand roundings
    against a hand-worked gradient whose operands all lie off the bfloat16 grid (tests/golden/).
Functions with no independent pin: none ("parity unpinned" would be stated here).
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence

import numpy as np

MODEL_LOGISTIC = 0
MODEL_SOFTMAX = 1
MODEL_MLP2 = 2
MODEL_LSQ = 100          # oracle-only least-squares loss used by the hand-worked pin

RULE_CADA1 = 1
RULE_CADA2 = 2
RULE_LAG = 3             # stochastic LAG rule, Eq. 4 (one gradient per worker-iteration)

_U64 = np.uint64


# ----------------------------------------------------------------------------------------------
# Minibatch sampler.  The paper only says "a randomly selected ... minibatch" (Section 1) with
# samples independent across iterations (Assumption 2).  Reading: B indices drawn uniformly
# with replacement from worker m's rows by the SplitMix64 generator (Steele, Lea, Flood,
# OOPSLA 2014) used as a counter-based generator:
#     out(n) = mix(seed + (n + 1) * 0x9E3779B97F4A7C15),  n = (k * M + m) * B + j
#     idx    = out(n) mod N_m
# ----------------------------------------------------------------------------------------------

def splitmix64(seed: int, n: np.ndarray) -> np.ndarray:
    """n-th output (n = 0, 1, ...) of SplitMix64 started from ``seed``; vectorised over n."""
    with np.errstate(over="ignore"):
        n = np.asarray(n, dtype=np.uint64)
        z = _U64(seed & 0xFFFFFFFFFFFFFFFF) + (n + _U64(1)) * _U64(0x9E3779B97F4A7C15)
        z = (z ^ (z >> _U64(30))) * _U64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> _U64(27))) * _U64(0x94D049BB133111EB)
        return z ^ (z >> _U64(31))


def sample_indices(seed: int, k: int, M: int, B: int, n_samples: Sequence[int]) -> np.ndarray:
    """Row indices xi_m^k for every worker: int64 array [M, B]."""
    out = np.empty((M, B), dtype=np.int64)
    j = np.arange(B, dtype=np.uint64)
    for m in range(M):
        n = _U64((k * M + m) * B) + j
        out[m] = (splitmix64(seed, n) % _U64(int(n_samples[m]))).astype(np.int64)
    return out


# ----------------------------------------------------------------------------------------------
# bfloat16 rounding (round to nearest, ties to even) of float64/float32 values -> float64.
# Only the MLP workload uses it: operands of each dense product are rounded, sums are not.
# ----------------------------------------------------------------------------------------------

def round_bf16(a: np.ndarray) -> np.ndarray:
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> _U64(16)) & _U64(1)
    r = ((u + _U64(0x7FFF) + lsb) & _U64(0xFFFF0000)).astype(np.uint32)
    return r.view(np.float32).astype(np.float64).reshape(np.shape(a))


# ----------------------------------------------------------------------------------------------
# Losses and their minibatch gradients (supplement, "Simulation details": logistic loss for
# the binary case, cross-entropy for the multi-class case, both with an l2 regulariser).
# Reading of the regulariser: (lam/2)*||theta||^2 over ALL of theta (bias included), inside
# every worker's loss, so each worker gradient carries + lam*theta.
# theta layouts:  logistic  [w (F) | b (1 if has_bias)]
#                 softmax   [W (F x C, row-major) | b (C if has_bias)]
#                 mlp2      [W1 (F x H) | b1 (H) | W2 (H x C) | b2 (C)]
#                 lsq       [w (F)]           loss = 1/(2B) * sum (x_i.w - y_i)^2
# ----------------------------------------------------------------------------------------------

def _sigmoid(z):
    e = np.exp(-np.abs(z))
    return np.where(z >= 0, 1.0 / (1.0 + e), e / (1.0 + e))


def _log1pexp(z):
    return np.maximum(z, 0.0) + np.log1p(np.exp(-np.abs(z)))


def _softmax_rows(z):
    z = z - z.max(axis=1, keepdims=True)
    e = np.exp(z)
    return e / e.sum(axis=1, keepdims=True)


def _logsumexp_rows(z):
    mx = z.max(axis=1)
    return mx + np.log(np.exp(z - mx[:, None]).sum(axis=1))


RELU_TIE = 1e-5          # |z1| below which the sign of a hidden pre-activation counts as undecided (see Model.grad)
ROUND_TIE = 1e-5         # max-norm-relative agreement of two unrounded operands below which a differing bf16 rounding is a tie


class Model:
    """Shape record + loss/gradient of one of the supported models."""
    relu_ties = 0
    round_ties = 0

    def __init__(self, kind: int, n_features: int, n_classes: int = 1, n_hidden: int = 0,
                 has_bias: int = 0, lam: float = 0.0, bf16: bool = False):
        self.kind, self.F, self.C, self.H = kind, n_features, n_classes, n_hidden
        self.has_bias, self.lam, self.bf16 = int(has_bias), float(lam), bool(bf16)
        if kind in (MODEL_LOGISTIC,):
            self.p = self.F + self.has_bias
        elif kind == MODEL_SOFTMAX:
            self.p = self.F * self.C + self.has_bias * self.C
        elif kind == MODEL_MLP2:
            self.p = self.F * self.H + self.H + self.H * self.C + self.C
        elif kind == MODEL_LSQ:
            self.p = self.F
        else:
            raise ValueError("unknown model")

    # -- minibatch loss (mean over rows, plus regulariser) -------------------------------------
    def loss(self, Xb: np.ndarray, yb: np.ndarray, theta: np.ndarray) -> float:
        Xb = np.asarray(Xb, dtype=np.float64)[:, : self.F]
        theta = np.asarray(theta, dtype=np.float64)
        reg = 0.5 * self.lam * float(theta @ theta)
        if self.kind == MODEL_LOGISTIC:
            z = Xb @ theta[: self.F] + (theta[self.F] if self.has_bias else 0.0)
            y = np.asarray(yb, dtype=np.float64)
            return float(np.mean(_log1pexp(-y * z))) + reg        # log(1 + exp(-y z)), y = +-1
        if self.kind == MODEL_SOFTMAX:
            W = theta[: self.F * self.C].reshape(self.F, self.C)
            z = Xb @ W
            if self.has_bias:
                z = z + theta[self.F * self.C:]
            y = np.asarray(yb, dtype=np.int64)
            return float(np.mean(_logsumexp_rows(z) - z[np.arange(len(y)), y])) + reg
        if self.kind == MODEL_MLP2:
            z2 = self._mlp_forward(Xb, theta)[0]
            y = np.asarray(yb, dtype=np.int64)
            return float(np.mean(_logsumexp_rows(z2) - z2[np.arange(len(y)), y])) + reg
        # least squares
        r = Xb @ theta - np.asarray(yb, dtype=np.float64)
        return 0.5 * float(np.mean(r * r)) + reg

    def _q(self, a):
        return round_bf16(a) if self.bf16 else a

    def _q_tie(self, a, other):
        """Rounding of an operand of a dense product with the tie protocol of the parity tests.  A bfloat16 rounding
        is an integer decision taken from a floating-point sum: an implementation that forms the sum in another
        precision decides differently whenever the sum lies closer to a rounding boundary than the two sums lie to each
        other.  ``other`` is that implementation's UNROUNDED operand.  Where the two roundings differ although the
        unrounded values agree within ROUND_TIE of the operand's largest magnitude (the boundary then lies between them,
        i.e. within that distance of this oracle's own value), the other rounding is adopted and counted in
        ``round_ties``; everywhere else, and always when ``other`` is None, the oracle's own rounding stands."""
        q = self._q(a)
        if other is None or not self.bf16:
            return q
        other = np.asarray(other, dtype=np.float64)
        q_other = round_bf16(other)
        scale = float(np.max(np.abs(a))) if a.size else 0.0
        tie = (q != q_other) & (np.abs(a - other) <= ROUND_TIE * scale)
        self.round_ties += int(np.sum(tie))
        return np.where(tie, q_other, q)

    def _mlp_split(self, theta):
        F, H, C = self.F, self.H, self.C
        o = 0
        W1 = theta[o:o + F * H].reshape(F, H); o += F * H
        b1 = theta[o:o + H]; o += H
        W2 = theta[o:o + H * C].reshape(H, C); o += H * C
        b2 = theta[o:o + C]
        return W1, b1, W2, b2

    def _mlp_forward(self, Xb, theta, a1_other=None):
        """Returns (z2, z1, a1, rounded a1); ``a1_other``: another implementation's unrounded a1 (see _q_tie)."""
        W1, b1, W2, b2 = self._mlp_split(theta)
        z1 = self._q(Xb) @ self._q(W1) + b1            # operands rounded, sum and bias not
        a1 = np.maximum(z1, 0.0)
        a1q = self._q_tie(a1, a1_other)
        z2 = a1q @ self._q(W2) + b2
        return z2, z1, a1, a1q

    # -- predictions (sign of the logit / arg-max class) ------------------------------------------
    def predict(self, Xb: np.ndarray, theta: np.ndarray) -> np.ndarray:
        Xb = np.asarray(Xb, dtype=np.float64)[:, : self.F]
        theta = np.asarray(theta, dtype=np.float64)
        if self.kind == MODEL_LOGISTIC:
            z = Xb @ theta[: self.F] + (theta[self.F] if self.has_bias else 0.0)
            return np.where(z >= 0.0, 1.0, -1.0)
        if self.kind == MODEL_SOFTMAX:
            z = Xb @ theta[: self.F * self.C].reshape(self.F, self.C)
            if self.has_bias:
                z = z + theta[self.F * self.C:]
            return np.argmax(z, axis=1)
        z2 = self._mlp_forward(Xb, theta)[0]
        return np.argmax(z2, axis=1)

    # -- minibatch gradient --------------------------------------------------------------------
    def grad(self, Xb: np.ndarray, yb: np.ndarray, theta: np.ndarray, relu_hint: Optional[np.ndarray] = None,
             operand_hint: Optional[dict] = None) -> np.ndarray:
        """``relu_hint`` (MLP only, bool [B, H]): another implementation's decisions z1 > 0.  relu'(z1) is an
        integer decision taken from a floating-point sum; where |z1| <= RELU_TIE the two sides cannot be expected
        to agree, so the hinted decision is adopted there (and counted in ``relu_ties``).  Elsewhere it is ignored.
        ``operand_hint`` (MLP with bf16 operands only): that implementation's unrounded "a1" [B, H], "dz2" [B, C] and
        "dz1" [B, H]; their roundings are adopted under the tie rule of ``_q_tie`` and nowhere else.  The unrounded
        operands this call formed are left in ``self.last_operands`` for comparison."""
        Xb = np.asarray(Xb, dtype=np.float64)[:, : self.F]
        theta = np.asarray(theta, dtype=np.float64)
        B = Xb.shape[0]
        g = np.empty(self.p, dtype=np.float64)
        if self.kind == MODEL_LOGISTIC:
            z = Xb @ theta[: self.F] + (theta[self.F] if self.has_bias else 0.0)
            t = (np.asarray(yb, dtype=np.float64) + 1.0) / 2.0          # {0,1} target
            r = _sigmoid(z) - t
            g[: self.F] = Xb.T @ r / B
            if self.has_bias:
                g[self.F] = r.mean()
        elif self.kind == MODEL_SOFTMAX:
            FC = self.F * self.C
            W = theta[:FC].reshape(self.F, self.C)
            z = Xb @ W
            if self.has_bias:
                z = z + theta[FC:]
            R = _softmax_rows(z)
            R[np.arange(B), np.asarray(yb, dtype=np.int64)] -= 1.0
            g[:FC] = (Xb.T @ R / B).ravel()
            if self.has_bias:
                g[FC:] = R.mean(axis=0)
        elif self.kind == MODEL_MLP2:
            F, H, C = self.F, self.H, self.C
            W1, b1, W2, b2 = self._mlp_split(theta)
            oh = operand_hint or {}
            z2, z1, a1, a1q = self._mlp_forward(Xb, theta, oh.get("a1"))
            dz2 = _softmax_rows(z2)
            dz2[np.arange(B), np.asarray(yb, dtype=np.int64)] -= 1.0
            dz2 /= B
            dz2q = self._q_tie(dz2, oh.get("dz2"))
            dW2 = a1q.T @ dz2q
            db2 = dz2.sum(axis=0)
            da1 = dz2q @ self._q(W2).T
            active = z1 > 0.0                                         # relu'(0) = 0
            if relu_hint is not None:
                tie = np.abs(z1) <= RELU_TIE
                self.relu_ties += int(np.sum(tie & (relu_hint != active)))
                active = np.where(tie, relu_hint, active)
            dz1 = np.where(active, da1, 0.0)
            dW1 = self._q(Xb).T @ self._q_tie(dz1, oh.get("dz1"))
            db1 = dz1.sum(axis=0)
            self.last_operands = {"a1": a1, "dz2": dz2, "dz1": dz1}
            g[:] = np.concatenate([dW1.ravel(), db1, dW2.ravel(), db2])
        else:
            r = Xb @ theta - np.asarray(yb, dtype=np.float64)
            g[:] = Xb.T @ r / B
        return g + self.lam * theta


# ----------------------------------------------------------------------------------------------
# Server update, Eqs. 2a-2c
# ----------------------------------------------------------------------------------------------

def server_update(theta, h, vhat, nabla, alpha, beta1, beta2, eps):
    """One application of Eqs. 2a-2c to the aggregated (possibly stale) gradient ``nabla``.

    h' = beta1 h + (1-beta1) nabla;  v' = beta2 vhat + (1-beta2) nabla^2 (v-hat on the right, as
    printed in Eq. 2b and used again in the proofs of Lemmas 3-4);  vhat' = max(v', vhat);
    theta' = theta - alpha (eps I + Vhat')^(-1/2) h'.  Returns (theta', h', vhat').
    """
    h_new = beta1 * h + (1.0 - beta1) * nabla
    v_new = beta2 * vhat + (1.0 - beta2) * nabla * nabla
    vhat_new = np.maximum(v_new, vhat)
    theta_new = theta - alpha * h_new / np.sqrt(eps + vhat_new)
    return theta_new, h_new, vhat_new


# ----------------------------------------------------------------------------------------------
# The CADA iteration
# ----------------------------------------------------------------------------------------------

class CadaOracle:
    """State and one-iteration step of Algorithm 1.

    ``propose()`` evaluates both gradients of every worker and the rule (the worker side of
    Algorithm 1); ``commit(upload)`` applies a set of upload decisions and runs the server
    update.  ``step()`` = commit(propose().upload).  The split lets a parity test override a
    decision whose margin lies inside the agreed tie band.

    Readings of points the paper leaves open (each is a constructor argument or noted here):
      * tau_m^0 defaults to D, so every worker uploads at k = 0 through "tau >= D".
      * skip iff LHS <= RHS (Eqs. 6, 8 are non-strict); upload = not(LHS <= RHS) or tau >= D.
      * RHS = (c/d_max) * sum of the last d_max squared step norms; terms before k = 0 are 0
        (theta^{-D} = ... = theta^0, supplement "Supporting Lemmas"); c = +inf gives RHS = +inf.
      * the newest window term at iteration k is ||theta^k - theta^{k-1}||^2.
      * CADA1: the snapshot is refreshed when k mod D == 0, before the gradients of that
        iteration; the stored innovation of the last upload is used as it is.
      * v^{k+1} = beta2 * vhat^k + (1-beta2) * grad^2 (Eq. 2b uses v-hat, not v);
        theta^{k+1} = theta^k - alpha * h^{k+1} / sqrt(eps + vhat^{k+1}) (Eq. 2c), no bias
        correction, h^0 = vhat^0 = 0.
    """

    def __init__(self, model: Model, rule: int, X: List[np.ndarray], y: List[np.ndarray],
                 theta0: np.ndarray, *, batch: int, alpha: float, beta1: float, beta2: float,
                 eps: float, c: float, d_max: int, D: int, seed: int = 0,
                 tau0: Optional[Sequence[int]] = None, server: str = "amsgrad", aggregate: str = "slots",
                 alpha_K0: float = 0.0, batch_m: Optional[Sequence[int]] = None):
        self.model, self.rule = model, int(rule)
        self.X, self.y = X, y
        self.M = len(X)
        self.n_samples = [int(x.shape[0]) for x in X]
        self.B = int(batch)
        self.alpha, self.beta1, self.beta2, self.eps = float(alpha), float(beta1), float(beta2), float(eps)
        self.c, self.d_max, self.D, self.seed = float(c), int(d_max), int(D), int(seed)
        self.server = server          # "amsgrad": Eqs. 2a-2c; "sgd": theta <- theta - alpha * nabla (Section 2.1, the LAG comparator)
        # "slots": nabla^k = (1/M) sum_m G_m, the definition in Eq. 2a; "recursive": Eq. 3, the server keeps only
        # nabla^{k-1} and adds the uploaded innovations delta_m^k / M
        assert aggregate in ("slots", "recursive")
        self.aggregate = aggregate
        # Theorem 2: alpha_k = alpha / (k + K0) (the theorem's 2/mu is `alpha`); K0 = 0 keeps alpha constant
        self.alpha_K0 = float(alpha_K0)
        # batch ratio of the supplement ("Simulation details"): worker m averages over its first batch_m[m] <= batch
        # sampled rows; the index stream keeps the stride `batch`
        self.batch_m = [self.B] * len(X) if batch_m is None else [int(b) for b in batch_m]
        assert all(1 <= b <= self.B for b in self.batch_m)
        p, M = model.p, self.M
        self.p = p
        self.theta = np.asarray(theta0, dtype=np.float64).copy()
        assert self.theta.shape == (p,)
        self.h = np.zeros(p)
        self.vhat = np.zeros(p)
        self.G = np.zeros((M, p))                        # server's copy of each worker's last upload
        self.theta_hat = np.tile(self.theta, (M, 1))     # CADA2: iterate of worker m's last upload
        self.theta_tilde = self.theta.copy()             # CADA1: snapshot
        self.delta_stored = np.zeros((M, p))             # CADA1: innovation stored at last upload
        self.tau = np.full(M, self.D, dtype=np.int64) if tau0 is None else np.asarray(tau0, dtype=np.int64).copy()
        self.ring = np.zeros(self.d_max)                 # squared step norms, slot k mod d_max
        self.k = 0
        self.nabla_rec = np.zeros(p)                     # recursive-innovation form of the aggregate
        self.uploads_total = 0
        self.uploads_forced = 0
        self.uploads_rule = 0
        self.uploads_per_worker = np.zeros(M, dtype=np.int64)
        self._pending = None

    # -- worker side ---------------------------------------------------------------------------
    def rhs(self) -> float:
        """Right-hand side of Eqs. 6 / 8."""
        if math.isinf(self.c):
            return math.inf
        return (self.c / self.d_max) * float(np.sum(self.ring))

    def propose(self, idx: Optional[np.ndarray] = None, relu_hint: Optional[np.ndarray] = None,
                operand_hint: Optional[dict] = None) -> dict:
        """``relu_hint``: bool [M, 2, B, H] (MLP only), decisions z1 > 0 at (theta^k, old iterate); ``operand_hint``: dict
        of arrays [M, 2, B, .] keyed "a1", "dz2", "dz1"; see Model.grad.  With an operand hint the result also carries
        ``operand_dev``: per key, the largest max-norm-relative distance between the hinted and the oracle's own
        unrounded operand over all (worker, iterate) pairs."""
        if idx is None:
            idx = sample_indices(self.seed, self.k, self.M, self.B, self.n_samples)
        idx = np.asarray(idx)
        if self.rule == RULE_CADA1 and self.k % self.D == 0:      # Algorithm 1: snapshot step
            self.theta_tilde = self.theta.copy()
        rhs = self.rhs()
        M, p = self.M, self.p
        g = np.empty((M, p))
        d = np.zeros((M, p))
        lhs = np.empty(M)
        operand_dev = {}
        for m in range(M):
            rows = idx[m][: self.batch_m[m]]
            Xb = self.X[m][rows]
            yb = self.y[m][rows]
            h0 = None if relu_hint is None else relu_hint[m][0][: self.batch_m[m]]
            h1 = None if relu_hint is None else relu_hint[m][1][: self.batch_m[m]]
            kw0 = {} if h0 is None else {"relu_hint": h0}
            kw1 = {} if h1 is None else {"relu_hint": h1}
            if operand_hint is not None:
                nb = self.batch_m[m]
                kw0["operand_hint"] = {key: v[m][0][:nb] for key, v in operand_hint.items()}
                kw1["operand_hint"] = {key: v[m][1][:nb] for key, v in operand_hint.items()}
            g[m] = self.model.grad(Xb, yb, self.theta, **kw0)
            self._note_operands(operand_dev, kw0)
            if self.rule == RULE_CADA1:
                d[m] = g[m] - self.model.grad(Xb, yb, self.theta_tilde, **kw1)      # tilde-delta_m^k
                self._note_operands(operand_dev, kw1)
                e = d[m] - self.delta_stored[m]
            elif self.rule == RULE_CADA2:
                d[m] = g[m] - self.model.grad(Xb, yb, self.theta_hat[m], **kw1)     # same sample, old iterate
                self._note_operands(operand_dev, kw1)
                e = d[m]
            else:                                                           # stochastic LAG, Eq. 4
                e = g[m] - self.G[m]
            lhs[m] = float(e @ e)
        forced = self.tau >= self.D
        violated = ~(lhs <= rhs)
        upload = violated | forced
        self._pending = (g, d)
        return {"idx": idx, "lhs": lhs, "rhs": rhs, "forced": forced, "violated": violated,
                "upload": upload, "g": g, "d": d, "operand_dev": operand_dev}

    def _note_operands(self, dev: dict, kw: dict) -> None:
        """Test bookkeeping only: distance between hinted operands and the ones the last gradient call formed."""
        for key, other in (kw.get("operand_hint") or {}).items():
            own = self.model.last_operands[key]
            scale = float(np.max(np.abs(own)))
            err = float(np.max(np.abs(own - other))) / scale if scale > 0 else 0.0
            dev[key] = max(dev.get(key, 0.0), err)

    # -- server side ---------------------------------------------------------------------------
    def commit(self, upload: np.ndarray) -> None:
        g, d = self._pending
        self._pending = None
        upload = np.asarray(upload, dtype=bool)
        forced = self.tau >= self.D
        for m in range(self.M):
            if upload[m]:
                self.nabla_rec += (g[m] - self.G[m]) / self.M      # delta_m^k / M (recursive form)
                self.G[m] = g[m]
                self.theta_hat[m] = self.theta
                self.delta_stored[m] = d[m]
                self.tau[m] = 1
                self.uploads_total += 1
                self.uploads_per_worker[m] += 1
                if forced[m]:
                    self.uploads_forced += 1
                else:
                    self.uploads_rule += 1
            else:
                self.tau[m] += 1
        if self.aggregate == "recursive":
            nabla = self.nabla_rec.copy()                           # Eq. 3
        else:
            nabla = self.G.sum(axis=0) / self.M                     # Eq. 2a
        self.last_nabla = nabla
        alpha_k = self.alpha / (self.k + self.alpha_K0) if self.alpha_K0 > 0 else self.alpha    # Theorem 2
        if self.server == "sgd":
            theta_new = self.theta - alpha_k * nabla                                      # Section 2.1
        else:
            theta_new, self.h, self.vhat = server_update(self.theta, self.h, self.vhat, nabla, alpha_k,
                                                         self.beta1, self.beta2, self.eps)   # Eqs. 2a-2c
        step = theta_new - self.theta
        self.ring[self.k % self.d_max] = float(step @ step)
        self.theta = theta_new
        self.k += 1

    def evaluate(self):
        """Objective of Eq. 1 at the current iterate over all rows, L = (1/M) sum_m L_m(theta) (each L_m carries the
        regulariser), and the fraction of all rows that are classified correctly (the curves of Section 4)."""
        loss, correct, rows = 0.0, 0, 0
        for m in range(self.M):
            loss += self.model.loss(self.X[m], self.y[m], self.theta)
            correct += int(np.sum(self.model.predict(self.X[m], self.theta) == self.y[m]))
            rows += self.n_samples[m]
        return loss / self.M, correct / rows

    def step(self, idx: Optional[np.ndarray] = None) -> dict:
        out = self.propose(idx)
        self.commit(out["upload"])
        return out
