"""Binary64 closed forms from the paper, used to pin the sampler.

TEST INFRASTRUCTURE ONLY.  Nothing here draws random numbers: each function
returns probabilities, estimator values or variances exactly as the paper's
equations give them, so that the outcome frequencies of the binary32 sampler
can be compared with them.
"""
from __future__ import annotations

import itertools

import numpy as np


# ---------------------------------------------------------------- 1:2 -------
def mvue12(a1: float, a2: float):
    """Sec. 4.1, last equation: (p_1, v_1, v_2) of the optimal 1:2 estimator."""
    m1, m2 = abs(a1), abs(a2)
    s = m1 + m2
    p1 = m1 / s
    return p1, np.sign(a1) * s, np.sign(a2) * s


def var12_of_v1(a1: float, a2: float, v1: float) -> float:
    """Sec. 4.1: block variance of an unbiased 1:2 estimator as a function of v_1
    (positive a_1, a_2; v_1 > a_1)."""
    return v1 * a1 - a1 ** 2 + a2 ** 2 * v1 / (v1 - a1) - a2 ** 2


def var12_opt(a1: float, a2: float) -> float:
    """Sec. 4.1: variance of the optimal 1:2 estimator, 2 |a_1| |a_2|."""
    return 2.0 * abs(a1) * abs(a2)


# ---------------------------------------------------------------- 1:M -------
def var1m_opt(a) -> float:
    """Sec. 4.1's argument for a block of M with one survivor: theta_i = a_i / p_i w.p. p_i, sum p_i = 1; the
    variance sum a_i^2 / p_i - a_i^2 is least at p_i = |a_i| / S, where it is S^2 - sum a_i^2."""
    m = np.abs(np.asarray(a, dtype=np.float64))
    return float(m.sum() ** 2 - np.sum(m ** 2))


def var1m_of_p(a, p) -> float:
    """Variance of the keep-one unbiased estimator with survival probabilities p (p_i > 0 wherever a_i != 0)."""
    m = np.abs(np.asarray(a, dtype=np.float64))
    p = np.asarray(p, dtype=np.float64)
    nz = m > 0
    return float(np.sum(m[nz] ** 2 / p[nz] - m[nz] ** 2))


# ---------------------------------------------------------------- 2:4 -------
def block_variance(a, p) -> float:
    """Sec. 4.2: Var_B = sum_i a_i^2 / p_i - a_i^2 for theta_i = a_i / p_i w.p. p_i."""
    a = np.abs(np.asarray(a, dtype=np.float64))
    p = np.asarray(p, dtype=np.float64)
    nz = a > 0
    return float(np.sum(a[nz] ** 2 / p[nz] - a[nz] ** 2))


def marginals24(a):
    """Sec. 4.2: the optimal survival probabilities p_i of a block of four.

    Either p_i = 2 a_i / sum_j a_j for all i, or, when one element would need
    p > 1, that element gets p = 1 and the others a_k / sum_{j != i} a_j.
    """
    m = np.abs(np.asarray(a, dtype=np.float64))
    total = m.sum()
    top = int(np.argmax(m))
    rest = total - m[top]
    if m[top] >= rest:
        p = m / rest if rest > 0 else np.zeros(4)
        p[top] = 1.0
        return p
    return 2.0 * m / total


def var24_uncapped(a) -> float:
    """App. A.3: sum_{i<j} a_i a_j - (1/2) sum_i a_i^2 when no p_i is capped."""
    m = np.abs(np.asarray(a, dtype=np.float64))
    cross = sum(m[i] * m[j] for i, j in itertools.combinations(range(4), 2))
    return float(cross - 0.5 * np.sum(m ** 2))


def pair_table24(s):
    """App. A.2: p_ij for magnitudes sorted ascending, s = [a_1, a_2, a_3, a_4].

    Returns a dict keyed by the 1-based sorted indices (i, j), i < j.
    """
    a1, a2, a3, a4 = (float(x) for x in s)
    tot = a1 + a2 + a3 + a4
    if a4 >= a1 + a2 + a3:                                    # case 3
        r = a1 + a2 + a3
        return {(1, 2): 0.0, (1, 3): 0.0, (2, 3): 0.0,
                (1, 4): a1 / r, (2, 4): a2 / r, (3, 4): a3 / r}
    if a4 <= 2 * a1 + a3:                                     # case 1
        return {(1, 2): 0.0,
                (1, 3): (2 * a1 + a3 - a4) / (2 * tot),
                (1, 4): (2 * a1 - a3 + a4) / (2 * tot),
                (2, 3): (2 * a2 + a3 - a4) / (2 * tot),
                (2, 4): (2 * a2 - a3 + a4) / (2 * tot),
                (3, 4): (-a1 - a2 + a3 + a4) / tot}
    return {(1, 2): 0.0, (1, 3): 0.0,                         # case 2
            (1, 4): 2 * a1 / tot,
            (2, 3): (a1 + a2 + a3 - a4) / tot,
            (2, 4): (-a1 + a2 - a3 + a4) / tot,
            (3, 4): (-a1 - a2 + a3 + a4) / tot}


def outcome_law24(a):
    """Law of the six position pairs of the ORIGINAL block under App. A.2, with
    ties broken by position (stable sort).  Returns {(i, j): prob}, 0-based, i < j."""
    m = np.abs(np.asarray(a, dtype=np.float64))
    order = sorted(range(4), key=lambda i: (m[i], i))
    table = pair_table24([m[i] for i in order])
    law = {pr: 0.0 for pr in itertools.combinations(range(4), 2)}
    for (i, j), p in table.items():
        u, v = order[i - 1], order[j - 1]
        law[(min(u, v), max(u, v))] += p
    return law


def systematic_law24(a):
    """Law of the six position pairs when the pair is drawn by systematic sampling from the
    optimal marginals of Sec. 4.2: element k owns an interval of length H p_k (in block
    order), t is uniform on [0, H) and the owners of t and t + H survive.  Computed as the
    measure of {t : t in I_i, t + H in I_j}, i.e. |I_i  intersect  (I_j - H)| / H, in
    binary64 from marginals24, with no reference to how the sampler walks its thresholds.
    Needs at least two non-zeros.  Returns {(i, j): prob}, 0-based, i < j."""
    m = np.abs(np.asarray(a, dtype=np.float64))
    p = marginals24(m)
    edges = np.concatenate([[0.0], np.cumsum(p)])          # in units of H: total length 2
    law = {pr: 0.0 for pr in itertools.combinations(range(4), 2)}
    for i, j in law:
        lo = max(edges[i], edges[j] - 1.0)
        hi = min(edges[i + 1], edges[j + 1] - 1.0)
        law[(i, j)] = max(0.0, hi - lo)
    return law


# ------------------------------------------------- approx-MVUE 2:4 (Sec. 4.4) ---
def approx24_ordered_law(a):
    """Sec. 4.4: P[i drawn first, j drawn second] = (a_i / sum) (a_j / (sum - a_i)), as a 4x4
    matrix (zero diagonal).  Needs at least two non-zeros."""
    m = np.abs(np.asarray(a, dtype=np.float64))
    total = m.sum()
    law = np.zeros((4, 4))
    for i in range(4):
        for j in range(4):
            if i != j and m[i] > 0 and m[j] > 0:
                law[i, j] = m[i] / total * m[j] / (total - m[i])
    return law


def approx24_inclusion(a):
    """Sec. 4.4, the numbered equation: p_i = |a_i|/sum + sum_{k != i} (|a_k|/sum)(|a_i| / sum_{j != k} |a_j|)."""
    m = np.abs(np.asarray(a, dtype=np.float64))
    total = m.sum()
    p = np.zeros(4)
    for i in range(4):
        p[i] = m[i] / total + sum(m[k] / total * m[i] / (total - m[k]) for k in range(4) if k != i and m[k] > 0)
    return p


def approx24_variance(a) -> float:
    """Block variance of approx-MVUE: Sec. 4.2's variance equation at the inclusion probabilities of Sec. 4.4."""
    return block_variance(a, approx24_inclusion(a))


def opt24_variance(a) -> float:
    """Block variance of the optimal 2:4 estimator: the same equation at the optimal marginals."""
    return block_variance(a, marginals24(a))


# ------------------------------------------- 1:2 comparison estimators -------
def estimator12(name: str, a1: float, a2: float):
    """Table 2's 1:2 pruners as a list of (probability, [theta_1, theta_2])."""
    m1, m2 = abs(a1), abs(a2)
    if name == "mvue":
        p, v1, v2 = mvue12(a1, a2)
        return [(p, [v1, 0.0]), (1 - p, [0.0, v2])]
    if name == "greedy":
        return [(1.0, [0.0, a2] if m1 <= m2 else [a1, 0.0])]
    if name == "biased":
        p = m1 / (m1 + m2)
        return [(p, [a1, 0.0]), (1 - p, [0.0, a2])]
    if name == "uniform":
        return [(0.5, [a1, 0.0]), (0.5, [0.0, a2])]
    if name == "unbiased":
        return [(0.5, [2 * a1, 0.0]), (0.5, [0.0, 2 * a2])]
    raise KeyError(name)


def mean_and_variance(outcomes):
    """E[theta] and sum_i Var[theta_i] of a finite law given as (prob, vector) pairs."""
    probs = np.array([p for p, _ in outcomes])
    vecs = np.array([v for _, v in outcomes], dtype=np.float64)
    mean = (probs[:, None] * vecs).sum(0)
    var = (probs[:, None] * (vecs - mean) ** 2).sum()
    return mean, float(var)


# ------------------------------------------- sequential draws without replacement -------
def sequential_inclusion(a, n_draws: int):
    """Inclusion probabilities of n_draws sequential draws without replacement, each proportional to magnitude among
    the elements still there (Sec. 4.4's procedure, any block size), by brute force over every ordered sequence in
    binary64.  Needs at least n_draws non-zeros."""
    m = np.abs(np.asarray(a, dtype=np.float64))
    p = np.zeros(len(m))
    for seq in itertools.permutations(range(len(m)), n_draws):
        prob, left = 1.0, m.sum()
        for k in seq:
            prob *= m[k] / left
            left -= m[k]
        for k in seq:
            p[k] += prob
    return p


def sequential_set_law(a, n_draws: int):
    """{frozenset of drawn positions: probability} for the same procedure."""
    m = np.abs(np.asarray(a, dtype=np.float64))
    law = {}
    for seq in itertools.permutations(range(len(m)), n_draws):
        prob, left = 1.0, m.sum()
        for k in seq:
            prob *= m[k] / left
            left -= m[k]
        key = frozenset(seq)
        law[key] = law.get(key, 0.0) + prob
    return law
