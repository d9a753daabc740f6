"""CPU oracle for the BASE batched MoE decode layer. TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 NumPy statement of what the layer computes, written from the
paper's definitions. Only the tests, the smoke check and the benchmark's CPU
baseline may import it; the CUDA path shares no code with it and never calls it.

Notation follows the paper: N routed experts (``E`` in array shapes), router
top-K, expert budget M, batch of T decode tokens, hidden z_t, normalised input
z-bar, router weights w_{t,u}, predictor (a_u, b_u), predicted removal cost
c_{t,u} = w_{t,u}^2 * exp(a_u . z-bar_t + b_u), batch score D-hat_u, active set A,
executed routes R'_t.

All inputs are float arrays that already hold the storage-precision values
(bf16-representable weights and hidden states, fp32 biases); arithmetic is fp64.

Every function below is pinned by tests that do not re-use it (brute force,
identities, closed forms, exhaustive search, library cross-checks). What cannot
be pinned: the paper prints no numeric input -> output example for the layer, so
agreement with the paper's own experiments is "parity unpinned".
"""

from __future__ import annotations

import numpy as np

GATE_RULE_PAPER = 0       # Sec. 3.5: denominator from the token's ORIGINAL top-K
GATE_RULE_RENORM = 1      # OEA-style: renormalise over the executed experts
GATE_RULE_ONE = 2         # every executed expert enters with weight 1 (always-on shared experts, Sec. 3.1)
FILL_BACKFILL = 0         # Sec. 3.5: next-preferred experts inside the active set
FILL_DROP = 1             # fill-rule ablation: unavailable routes are simply removed
ROUTER_NORM_TOPK = 0      # router weights renormalised over the token's top-K
ROUTER_NORM_ALL = 1       # plain softmax over all experts, no renormalisation after the top-K
# what a routed pair contributes to its expert's batch score (App. Selection-Rule Ablation)
SCORE_PREDICTED = 0       # w^2 exp(a . z-bar + b): the method (Eq. log_energy_predictor)
SCORE_WEIGHT_SQ = 1       # squared router-weight sum
SCORE_WEIGHT = 2          # router-weight sum
SCORE_STATIC = 3          # static energy w^2 mu_u, with mu_u = exp(b_u)
SCORE_TOP1_UNION = 4      # 1 per token whose first choice the expert is (positive exactly on the top-1 union)


# ----------------------------------------------------------------------------- router (Sec. 3.1)

def router_logits(z, router_w, router_bias):
    """l[t,e] = z_t . W_r[e] + bias[e], rounded to fp32 (the precision logits are exchanged in)."""
    l = np.asarray(z, np.float64) @ np.asarray(router_w, np.float64).T + np.asarray(router_bias, np.float64)
    return l.astype(np.float32)


def rank_desc(values):
    """Indices sorted by value descending; equal values keep the lower index first; NaN last."""
    v = np.asarray(values, np.float64)
    v = np.where(np.isnan(v), -np.inf, v)
    return np.argsort(-v, kind="stable")


def route_topk(logits, K, router_norm=ROUTER_NORM_TOPK):
    """Token-choice top-K routing (Sec. 3.1).

    ROUTER_NORM_TOPK: softmax scores renormalised over R_t (sum_u w_{t,u} = 1), the reading used for the
    Qwen3 and Mixtral shapes. ROUTER_NORM_ALL: plain softmax probabilities over all experts, not
    renormalised after the top-K (the convention of the paper's other two models, Sec. 4.1); then
    sum_u w_{t,u} < 1. Only the denominator S changes.

    Returns order [T,E] (full ranking by logit), R [T,K], q [T,E] = exp(l - max_e l),
    S [T] = the denominator, w [T,K] = q[R_t] / S_t.
    """
    l = np.asarray(logits, np.float64)
    T, E = l.shape
    order = np.stack([rank_desc(l[t]) for t in range(T)])
    R = order[:, :K]
    q = np.exp(l - l.max(axis=1, keepdims=True))
    if router_norm == ROUTER_NORM_ALL:
        S = q.sum(axis=1)
    else:
        S = np.take_along_axis(q, R, axis=1).sum(axis=1)
    w = np.take_along_axis(q, R, axis=1) / S[:, None]
    return order, R, q, S, w


# ----------------------------------------------------------------------------- predictor (Sec. 3.4, Eq. log_energy_predictor)

def normalise(z):
    """z-bar = z / ||z||_2 per token (zero rows stay zero)."""
    z = np.asarray(z, np.float64)
    n = np.sqrt((z * z).sum(axis=1, keepdims=True))
    return z / np.maximum(n, 1e-30)


def predict_costs(z, R, w, pred_A, pred_b, score_rule=SCORE_PREDICTED):
    """c[t,u] = w_{t,u}^2 * exp(a_u . z-bar_t + b_u) for u in R_t, 0 elsewhere. Shape [T,E].

    ``score_rule`` swaps the contribution for one of the ablation scores of App. Selection-Rule Ablation."""
    zbar = normalise(z)
    A = np.asarray(pred_A, np.float64)
    b = np.asarray(pred_b, np.float64)
    T, K = R.shape
    costs = np.zeros((T, A.shape[0]), np.float64)
    for t in range(T):
        for k in range(K):
            u = int(R[t, k])
            if u < 0:
                continue
            if score_rule == SCORE_PREDICTED:
                s_hat = float(A[u] @ zbar[t]) + b[u]
                costs[t, u] = w[t, k] ** 2 * np.exp(s_hat)
            elif score_rule == SCORE_WEIGHT_SQ:
                costs[t, u] = w[t, k] ** 2
            elif score_rule == SCORE_WEIGHT:
                costs[t, u] = w[t, k]
            elif score_rule == SCORE_STATIC:
                costs[t, u] = w[t, k] ** 2 * np.exp(b[u])
            elif score_rule == SCORE_TOP1_UNION:
                costs[t, u] = 1.0 if k == 0 else 0.0
            else:
                raise ValueError(score_rule)
    return costs


def aggregate(costs):
    """D-hat_u = sum over the batch of c[t,u]."""
    return np.asarray(costs, np.float64).sum(axis=0)


def select_top(scores, M):
    """Active set: the min(M, N) experts with the largest score (ties: lower id). Returns (ids, mask)."""
    scores = np.asarray(scores, np.float64)
    M = min(int(M), scores.shape[0])
    ids = rank_desc(scores)[:M]
    mask = np.zeros(scores.shape[0], np.uint8)
    mask[ids] = 1
    return ids.astype(np.int32), mask


# ----------------------------------------------------------------------------- restricted routing (Sec. 3.5)

def restrict_routes(order, R, q, S, mask, K, gate_rule=GATE_RULE_PAPER, fill=FILL_BACKFILL):
    """Executed routes R'_t and gates.

    Backfill: the token's K highest-ranked experts inside the active set. Gate of an executed expert
    is its own router score q over the ORIGINAL top-K denominator S_t (paper rule), or over the sum
    of the executed scores (renorm rule), or simply 1 (the rule for always-on shared experts). Empty slots: id -1, gate 0. Returns (ids [T,K], gates [T,K]).
    """
    T = order.shape[0]
    ids = np.full((T, K), -1, np.int32)
    gates = np.zeros((T, K), np.float64)
    for t in range(T):
        if fill == FILL_BACKFILL:
            kept = [int(u) for u in order[t] if mask[u]][:K]
        else:
            kept = [int(u) for u in R[t] if mask[u]]
        for k, u in enumerate(kept):
            ids[t, k] = u
            gates[t, k] = q[t, u]
        if gate_rule == GATE_RULE_ONE:
            gates[t] = (ids[t] >= 0).astype(np.float64)
            continue
        den = S[t] if gate_rule == GATE_RULE_PAPER else gates[t].sum()
        if den > 0:
            gates[t] /= den
    return ids, gates


# ----------------------------------------------------------------------------- experts (SwiGLU)

def silu(x):
    return x / (1.0 + np.exp(-x))


def expert_ffn(x, w_gate, w_up, w_down):
    """E_u(x) = W_down ( silu(W_gate x) * (W_up x) ) for rows x [n,d]; w_gate,w_up [I,d]; w_down [d,I]."""
    x = np.asarray(x, np.float64)
    g = x @ np.asarray(w_gate, np.float64).T
    u = x @ np.asarray(w_up, np.float64).T
    return (silu(g) * u) @ np.asarray(w_down, np.float64).T


def execute(z, ids, gates, expert_weights):
    """y_t = sum_k gates[t,k] * E_{ids[t,k]}(z_t). ``expert_weights(u)`` -> (w_gate, w_up, w_down)."""
    z = np.asarray(z, np.float64)
    y = np.zeros_like(z)
    dispatched = sorted({int(u) for u in ids.ravel() if u >= 0})
    for u in dispatched:
        tt, kk = np.nonzero(ids == u)
        out = expert_ffn(z[tt], *expert_weights(u))
        y[tt] += gates[tt, kk][:, None] * out
    return y, dispatched


# ----------------------------------------------------------------------------- the layer

def moe_decode_layer(z, logits, pred_A, pred_b, expert_weights, K, M,
                     gate_rule=GATE_RULE_PAPER, fill=FILL_BACKFILL, forced_mask=None, score_rule=SCORE_PREDICTED,
                     router_norm=ROUTER_NORM_TOPK):
    """One BASE decode step of one MoE layer, in the paper's order:
    route -> predict costs -> aggregate -> top-M -> restrict routes -> execute.

    ``forced_mask`` replaces the predicted selection (used to compare near-ties).
    Returns a dict with every intermediate.
    """
    order, R, q, S, w = route_topk(logits, K, router_norm)
    costs = predict_costs(z, R, w, pred_A, pred_b, score_rule)
    scores = aggregate(costs)
    sel, mask = select_top(scores, M)
    if forced_mask is not None:
        mask = np.asarray(forced_mask, np.uint8)
    Kx = min(K, int(mask.sum()))
    ids, gates = restrict_routes(order, R, q, S, mask, K, gate_rule, fill)
    y, dispatched = execute(z, ids, gates, expert_weights)
    return dict(order=order, R=R, w=w, S=S, q=q, costs=costs, scores=scores, selected=sel, mask=mask,
                exec_ids=ids, exec_gates=gates, y=y, dispatched=dispatched, n_dispatched=len(dispatched),
                max_exec=Kx)


def stack_next_hidden(x, y):
    """Wiring of consecutive layers in the stack workload: x' = rmsnorm(x + y) without gain."""
    h = np.asarray(x, np.float64) + np.asarray(y, np.float64)
    return h / np.sqrt(np.mean(h * h, axis=1, keepdims=True))


# ----------------------------------------------------------------------------- independent reference objects
# These are written separately from the functions above and are what the pins compare against.

def dense_topk_moe(z, logits, expert_weights, K):
    """Plain top-K MoE: y_t = sum_{u in R_t} w_{t,u} E_u(z_t), w = softmax over the K largest logits."""
    z = np.asarray(z, np.float64)
    l = np.asarray(logits, np.float64)
    y = np.zeros_like(z)
    for t in range(z.shape[0]):
        top = sorted(range(l.shape[1]), key=lambda e: (-l[t, e], e))[:K]
        p = np.exp(l[t, top] - l[t, top].max())
        p /= p.sum()
        for u, wu in zip(top, p):
            y[t] += wu * expert_ffn(z[t:t + 1], *expert_weights(u))[0]
    return y


def layer_drop(z, logits, expert_weights, K, omitted):
    """Dense top-K MoE with the contributions of the experts in ``omitted`` deleted: no backfill, no
    renormalisation. This is the object Eq. error_decomposition speaks about."""
    z = np.asarray(z, np.float64)
    l = np.asarray(logits, np.float64)
    y = np.zeros_like(z)
    for t in range(z.shape[0]):
        top = sorted(range(l.shape[1]), key=lambda e: (-l[t, e], e))[:K]
        p = np.exp(l[t, top] - l[t, top].max())
        p /= p.sum()
        for u, wu in zip(top, p):
            if u in omitted:
                continue
            y[t] += wu * expert_ffn(z[t:t + 1], *expert_weights(u))[0]
    return y


def contributions(z, R, w, expert_weights):
    """a[t,k,:] = w_{t,u} E_u(z_t) for u = R[t,k] (Sec. 3.2)."""
    z = np.asarray(z, np.float64)
    T, K = R.shape
    a = np.zeros((T, K, z.shape[1]))
    for t in range(T):
        for k in range(K):
            a[t, k] = w[t, k] * expert_ffn(z[t:t + 1], *expert_weights(int(R[t, k])))[0]
    return a


def true_removal_cost(a, R, E):
    """D_u = sum_{t: u in R_t} ||a_{t,u}||^2 (Eq. individual_expert_damage; equals D*_u)."""
    D = np.zeros(E)
    en = (a * a).sum(axis=2)
    for t in range(R.shape[0]):
        for k in range(R.shape[1]):
            D[int(R[t, k])] += en[t, k]
    return D


def exact_error(a, R, mask):
    """(E(A), individual damage, cross terms) of Eq. error_decomposition for active mask A."""
    total = indiv = cross = 0.0
    for t in range(R.shape[0]):
        U = [k for k in range(R.shape[1]) if not mask[int(R[t, k])]]
        if not U:
            continue
        total += float(np.sum(a[t, U].sum(axis=0) ** 2))
        indiv += float(sum(a[t, k] @ a[t, k] for k in U))
        cross += 2.0 * float(sum(a[t, U[i]] @ a[t, U[j]] for i in range(len(U)) for j in range(i + 1, len(U))))
    return total, indiv, cross


def cross_term_stats(a_t):
    """(rho_t, c-bar_t, |U_t|_eff) for the omitted contributions a_t [n,d] of one token (App. cross-term)."""
    m = np.sqrt((a_t * a_t).sum(axis=1))
    rho = float(np.sum(a_t.sum(axis=0) ** 2) / np.sum(m * m))
    n = a_t.shape[0]
    num = den = 0.0
    for i in range(n):
        for j in range(n):
            if i != j:
                cos = float(a_t[i] @ a_t[j]) / (m[i] * m[j])
                num += m[i] * m[j] * cos
                den += m[i] * m[j]
    cbar = num / den if den > 0 else 0.0
    eff = float(m.sum() ** 2 / np.sum(m * m))
    return rho, cbar, eff


def energy_retained(mask, D_star, M):
    """ER = sum_{u in A} D*_u / sum_{u in A*} D*_u with A* the top-M of D* (Eq. energy_retained)."""
    best = np.sort(np.asarray(D_star))[::-1][:M].sum()
    return float(np.asarray(D_star)[np.asarray(mask, bool)].sum() / best)


# ----------------------------------------------------------------------------- calibration (App. Calibration Details)

def ridge_fit(X, y, lam):
    """Centred closed-form ridge: a = (G_c + lam I)^-1 q_c, b = y-bar - a . x-bar."""
    X = np.asarray(X, np.float64)
    y = np.asarray(y, np.float64)
    xm = X.mean(axis=0)
    ym = y.mean()
    Xc = X - xm
    G = Xc.T @ Xc
    qc = Xc.T @ (y - ym)
    a = np.linalg.solve(G + lam * np.eye(X.shape[1]), qc)
    return a, float(ym - a @ xm)


def lambda_grid(n=25, lo=1e-4, hi=1e2):
    """The ridge penalties tried per expert: n values logarithmically spaced from lo to hi (App. Calibration Details)."""
    return lo * (hi / lo) ** (np.arange(n, dtype=np.float64) / (n - 1))


def ridge_log_evidence(X, y, lambdas):
    """Log marginal likelihood of each ridge penalty, up to a constant that does not depend on it.

    Model behind the centred ridge of App. Calibration Details: y = X a + b 1 + noise, noise ~ N(0, s2 I),
    a ~ N(0, (s2 / lam) I), flat prior on the intercept b, noise variance s2 at its maximising value. With
    G_c = X_c^T X_c, q_c = X_c^T y_c (centred statistics, n pairs, d features) and the eigenvalues theta_i and
    eigenvectors v_i of G_c -- the one eigendecomposition that serves every penalty --

        r(lam) = y_c.y_c - sum_i (v_i.q_c)^2 / (theta_i + lam)      (= y_c.y_c - q_c^T (G_c + lam I)^-1 q_c)
        L(lam) = -(n - 1)/2 * log r(lam) - 1/2 * sum_i log(1 + theta_i / lam).

    The paper names the criterion but prints no formula; this is this implementation's reading. r is
    floored at 1e-12 * y_c.y_c + 1e-300 (an exact fit must not produce log 0). Returns L [len(lambdas)].
    """
    X = np.asarray(X, np.float64)
    y = np.asarray(y, np.float64)
    n = X.shape[0]
    Xc = X - X.mean(axis=0)
    yc = y - y.mean()
    theta, V = np.linalg.eigh(Xc.T @ Xc)
    theta = np.maximum(theta, 0.0)
    proj = (V.T @ (Xc.T @ yc)) ** 2
    yy = float(yc @ yc)
    out = np.empty(len(lambdas))
    for i, lam in enumerate(np.asarray(lambdas, np.float64)):
        r = max(yy - float((proj / (theta + lam)).sum()), 1e-12 * yy + 1e-300)
        out[i] = -0.5 * (n - 1) * np.log(r) - 0.5 * float(np.log1p(theta / lam).sum())
    return out


def select_lambda(X, y, lambdas, default_index=None):
    """Index of the penalty with the largest evidence (the first one on a tie). An expert with fewer than two
    pairs has no centred statistics to judge by and takes default_index (the middle of the grid if None)."""
    if default_index is None:
        default_index = len(lambdas) // 2
    if np.asarray(X).shape[0] < 2:
        return default_index
    return int(np.argmax(ridge_log_evidence(X, y, lambdas)))


def fit_predictor(z_calib, logits_calib, expert_weights, K, E, lam=1e-2, eps=1e-12):
    """Fit (a_u, b_u) per expert on routed calibration pairs.

    lam: a fixed ridge penalty, or an array of candidates from which every expert takes the one of largest
    evidence (select_lambda).

    Target s = log(||E_u(z)||^2 + eps) (Sec. 3.4), features z-bar. The intercept is shifted by
    log(mean energy / mean exp(s-hat)) so that the mean predicted energy equals the mean true
    energy on the expert's calibration pairs (the retransformation correction the appendix
    mentions without a formula; this ratio-of-means form is this implementation's reading). Experts with no routed pair get a = 0, b = log(mean energy of all).
    Returns A [E,d] fp64, b [E] fp64, and the per-pair energies for inspection.
    """
    z = np.asarray(z_calib, np.float64)
    _, R, _, _, _ = route_topk(logits_calib, K)
    zbar = normalise(z)
    d = z.shape[1]
    A = np.zeros((E, d))
    b = np.zeros(E)
    all_energy = []
    fitted = np.zeros(E, bool)
    for u in range(E):
        tt = np.nonzero((R == u).any(axis=1))[0]
        if tt.size == 0:
            continue
        out = expert_ffn(z[tt], *expert_weights(u))
        energy = (out * out).sum(axis=1)
        all_energy.append(energy)
        s = np.log(energy + eps)
        lam_u = lam if np.isscalar(lam) else float(np.asarray(lam)[select_lambda(zbar[tt], s, lam)])
        a_u, b_u = ridge_fit(zbar[tt], s, lam_u)
        s_hat = zbar[tt] @ a_u + b_u
        b_u += float(np.log(np.mean(energy) / np.mean(np.exp(s_hat))))
        A[u], b[u], fitted[u] = a_u, b_u, True
    if all_energy and not fitted.all():
        b[~fitted] = np.log(np.mean(np.concatenate(all_energy)))
    return A, b
