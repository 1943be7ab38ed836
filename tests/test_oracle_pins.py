"""Pins for the fp64 CPU oracle: what the paper and the mathematics fix.

Nothing here touches a GPU or the CUDA library.
"""
import math

import numpy as np
import pytest

import oracle
from paper_2605_03110_b200 import workloads as wl
from label_model import cascade_from_labels, full_from_labels

TAU = 0.3
THR = 1.0 - TAU * TAU


def rows_at_angles(deg, norms, d=2, embed=None):
    X = np.zeros((len(deg), d))
    for i, (a, n) in enumerate(zip(deg, norms)):
        X[i, 0] = n * math.cos(math.radians(a))
        X[i, 1] = n * math.sin(math.radians(a))
    if embed is not None:                     # rotate the plane into d dims
        Q, _ = np.linalg.qr(np.random.default_rng(embed).standard_normal((d, d)))
        X = X @ Q
    return X


def acos(deg):
    return abs(math.cos(math.radians(deg)))


# ---------------------------------------------------------------- worked example A
# Six planar tokens at 0,20,40,60,90,180 degrees with arbitrary positive norms.
# |cos| of angle differences is textbook trigonometry; Definition 1 then fixes
# gamma and R by hand.  Discriminates "all earlier tokens" from "earlier
# representatives only" (token 2) and |.| from signed (token 5).
EX_A_DEG = [0, 20, 40, 60, 90, 180]
EX_A_NORM = [1, 2, 0.5, 3, 1, 7]


@pytest.mark.parametrize("d,embed", [(2, None), (16, 7)])
def test_example_a_full(d, embed):
    X = rows_at_angles(EX_A_DEG, EX_A_NORM, d, embed)
    rep, gamma = oracle.select_full(X, TAU)
    expect = [0.0, acos(20), acos(20), acos(20), acos(30), 1.0]
    assert np.allclose(gamma, expect, atol=1e-12)
    assert rep.tolist() == [0, 4]


@pytest.mark.parametrize("causal", [False, True])
def test_example_a_cascade_chain(causal):
    X = rows_at_angles(EX_A_DEG, EX_A_NORM)
    s1 = oracle.cascade_step(X, TAU, [0, 4], causal=causal)
    assert s1.rem.tolist() == []
    assert s1.add.tolist() == [2, 3]
    assert s1.rep.tolist() == [0, 2, 3, 4]
    # cross maxima: t1 vs {0,4}; t2; t3; t5 (non-causal sees both reps)
    assert math.isclose(s1.gamma_cross[1], acos(20), abs_tol=1e-12)
    assert math.isclose(s1.gamma_cross[2], max(acos(40), acos(50)) if not causal else acos(40), abs_tol=1e-12)
    assert math.isclose(s1.gamma_cross[3], max(acos(60), acos(30)) if not causal else acos(60), abs_tol=1e-12)
    assert math.isclose(s1.gamma_cross[5], 1.0, abs_tol=1e-12)
    s2 = oracle.cascade_step(X, TAU, s1.rep, causal=causal)
    assert s2.rem.tolist() == [3]            # token 3 vs token 2: cos 20 deg
    assert s2.add.tolist() == []
    assert s2.rep.tolist() == [0, 2, 4]
    # token 4 (90 deg) is compared with ALL earlier inherited reps, token 3 (60 deg) included
    assert np.allclose(s2.gamma_rep, [0.0, acos(40), acos(20), acos(30)], atol=1e-12)
    s3 = oracle.cascade_step(X, TAU, s2.rep, causal=causal)
    assert s3.rep.tolist() == [0, 2, 4] and s3.add.size == 0 and s3.rem.size == 0


# ---------------------------------------------------------------- worked example B
# Discriminates Algorithm 1's unmasked cross check from the causal variant.
def test_example_b_literal_vs_causal():
    X0 = rows_at_angles([0, 10, 90], [1, 1, 1])
    rep0, _ = oracle.select_full(X0, TAU)
    assert rep0.tolist() == [0, 2]
    X1 = rows_at_angles([0, 85, 90], [2, 1, 3])
    rep_full, _ = oracle.select_full(X1, TAU)
    assert rep_full.tolist() == [0, 1]
    lit = oracle.cascade_step(X1, TAU, rep0, causal=False)
    assert lit.rep.tolist() == [0, 2] and lit.add.size == 0 and lit.rem.size == 0
    assert math.isclose(lit.gamma_cross[1], acos(5), abs_tol=1e-12)
    cau = oracle.cascade_step(X1, TAU, rep0, causal=True)
    assert cau.rep.tolist() == [0, 1, 2] and cau.add.tolist() == [1]
    assert math.isclose(cau.gamma_cross[1], acos(85), abs_tol=1e-12)
    nxt = oracle.cascade_step(X1, TAU, cau.rep, causal=True)
    assert nxt.rep.tolist() == [0, 1] and nxt.rem.tolist() == [2]


# ---------------------------------------------------------------- closed forms
def test_duplicates_always_redundant():
    rng = np.random.default_rng(1)
    X = rng.standard_normal((40, 24))
    X[17] = -3.5 * X[4]
    X[30] = 0.25 * X[9]
    rep, gamma = oracle.select_full(X, TAU)
    assert abs(gamma[17] - 1.0) < 1e-12 and abs(gamma[30] - 1.0) < 1e-12
    assert 17 not in rep and 30 not in rep
    assert 0 in rep                               # first token always representative


def test_orthogonal_rows_all_representative():
    d = 32
    Q, _ = np.linalg.qr(np.random.default_rng(2).standard_normal((d, d)))
    X = Q[:20] * np.linspace(0.1, 9.0, 20)[:, None]
    rep, gamma = oracle.select_full(X, TAU)
    assert rep.tolist() == list(range(20))
    assert np.all(gamma < 1e-12)
    c = oracle.cascade_step(X, TAU, rep)
    assert c.rep.tolist() == list(range(20)) and c.add.size == 0 and c.rem.size == 0
    # from a subset: every missing token is decorrelated from the reps -> all added
    c2 = oracle.cascade_step(X, TAU, [0, 5, 6])
    assert c2.rep.tolist() == list(range(20)) and c2.add.size == 17


def test_chord_identity_threshold_angle():
    # |cos theta| >= 1 - tau^2  <=>  chord ||xhat_s - xhat_t|| <= sqrt(2) tau
    crit = math.degrees(math.acos(THR))           # 24.49...
    assert abs(crit - 24.4946) < 1e-3
    for theta in np.arange(1.0, 89.0, 0.37):
        X = rows_at_angles([0, theta], [1.7, 0.4])
        rep, gamma = oracle.select_full(X, TAU)
        chord = 2.0 * math.sin(math.radians(theta) / 2.0)
        redundant = chord <= math.sqrt(2.0) * TAU
        assert (1 not in rep) == redundant
        assert math.isclose(gamma[1], 1.0 - chord * chord / 2.0, abs_tol=1e-12)


def test_strict_inequality_at_threshold():
    # tau^2 = 0.75 -> thr = 0.25 exactly; xhat_0 = (1,0,0,0), xhat_1 = (.25,.25,.5,.75*...)
    # construct a pair whose cosine is exactly 0.25 in fp64: x1 = (1,1,1,...) with d=16
    d = 16
    X = np.zeros((2, d))
    X[0, 0] = 1.0
    X[1, :] = 1.0                                  # cos = 1/sqrt(16) = 0.25 exactly
    tau = math.sqrt(0.75)
    thr = 1.0 - tau * tau
    _, gamma = oracle.select_full(X, tau)
    assert gamma[1] == 0.25
    rep, _ = oracle.select_full(X, tau)
    # gamma == thr (up to the rounding of tau*tau) must not be "below": use the computed thr
    assert (1 in rep) == (0.25 < thr)
    rep_lo, _ = oracle.select_full(X, math.sqrt(0.75 + 1e-9))
    rep_hi, _ = oracle.select_full(X, math.sqrt(0.75 - 1e-9))
    assert 1 not in rep_lo and 1 in rep_hi


def test_zero_norm_row():
    X = np.random.default_rng(3).standard_normal((6, 8))
    X[2] = 0.0
    Xhat, norm = oracle.normalize(X)
    assert norm[2] == 0.0 and np.all(Xhat[2] == 0.0)
    assert np.allclose(np.linalg.norm(Xhat[[0, 1, 3, 4, 5]], axis=1), 1.0)
    rep, gamma = oracle.select_full(X, TAU)
    assert gamma[2] == 0.0 and 2 in rep


# ---------------------------------------------------------------- independent statement
def numpy_full(X, tau):
    Xh = X / np.linalg.norm(X, axis=1, keepdims=True)
    G = np.abs(Xh @ Xh.T)
    g = np.max(np.tril(G, -1), axis=1)
    return np.nonzero(g < 1 - tau * tau)[0], g


def brute_cascade(X, tau, R, causal=False):
    """Pure-Python statement of Algorithm 1 on tiny inputs."""
    thr = 1 - tau * tau
    Xh = [row / np.linalg.norm(row) for row in X]
    R = list(R)
    valid = []
    for i, s in enumerate(R):
        g = max([abs(float(Xh[s] @ Xh[R[j]])) for j in range(i)], default=0.0)
        if g < thr:
            valid.append(s)
    new = []
    for t in range(len(X)):
        if t in R:
            continue
        g = max([abs(float(Xh[t] @ Xh[s])) for s in valid if (not causal or s < t)], default=0.0)
        if g < thr:
            new.append(t)
    return sorted(valid + new), new, [s for s in R if s not in valid]


@pytest.mark.parametrize("T,d,seed", [(1, 4, 0), (2, 3, 1), (37, 5, 2), (200, 64, 3), (512, 96, 4)])
def test_full_matches_numpy_tril(T, d, seed):
    rng = np.random.default_rng(seed)
    base = rng.standard_normal((max(1, T // 6), d))
    X = base[rng.integers(0, base.shape[0], T)] + 0.15 * rng.standard_normal((T, d))
    rep, gamma = oracle.select_full(X, TAU)
    rep_np, g_np = numpy_full(X, TAU)
    assert np.allclose(gamma, g_np, atol=1e-12)
    assert rep.tolist() == rep_np.tolist()
    some = list(range(0, T, 7))
    assert np.allclose(oracle.full_rows(X, some), g_np[some], atol=1e-12)


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("causal", [False, True])
def test_cascade_matches_brute_force(seed, causal):
    rng = np.random.default_rng(100 + seed)
    T, d = 28, 6
    base = rng.standard_normal((5, d))
    X0 = base[rng.integers(0, 5, T)] + 0.2 * rng.standard_normal((T, d))
    X1 = X0 + 0.25 * rng.standard_normal((T, d))
    R0, _ = oracle.select_full(X0, TAU)
    # also try an arbitrary inherited set, not only one produced by the method
    for R in (R0.tolist(), sorted(rng.choice(T, 9, replace=False).tolist()), [], list(range(T))):
        got = oracle.cascade_step(X1, TAU, R, causal=causal)
        rep, new, rem = brute_cascade(X1, TAU, R, causal)
        assert got.rep.tolist() == rep and got.add.tolist() == new and got.rem.tolist() == rem


def test_cascade_empty_and_complete_inherited_sets():
    X = np.random.default_rng(5).standard_normal((12, 40))
    e = oracle.cascade_step(X, TAU, [])
    assert e.rep.tolist() == list(range(12)) and e.add.size == 12 and e.rem.size == 0
    full, gamma = oracle.select_full(X, TAU)
    c = oracle.cascade_step(X, TAU, list(range(12)))       # r = T: step 2 is the full T x T check
    assert np.allclose(c.gamma_rep, gamma, atol=1e-14)
    assert c.rep.tolist() == full.tolist() and c.add.size == 0


# ---------------------------------------------------------------- counts and helpers
def test_op_count_closed_forms(golden):
    for T, d, r in [(512, 768, 146), (2048, 4096, 447), (8192, 4096, 1), (16, 8, 16), (16, 8, 0)]:
        assert oracle.op_count(False, T, d) == T * T * d
        assert oracle.op_count(True, T, d, r) == T * r * d == r * r * d + (T - r) * r * d
    for kind, *f in golden("table7_and_cost_model.txt"):
        if kind == "indep":
            _, L, T, printed = f
            L, T = int(L), int(T)
            units = L * oracle.op_count(False, T, 1)          # d divided out
            assert units == L * T * T
            assert abs(units / 1e6 - float(printed)) < 0.006
    # cost-model products the paper prints (GFLOP)
    oc = oracle.op_count
    vals = {
        "28*512^2*4096": 28 * oc(False, 512, 4096),
        "512*4096*(512+27*240)": oc(False, 512, 4096) + 27 * oc(True, 512, 4096, 240),
        "28*2048^2*4096": 28 * oc(False, 2048, 4096),
        "2048*4096*(2048+27*240)": oc(False, 2048, 4096) + 27 * oc(True, 2048, 4096, 240),
        "2048^2*4096": oc(False, 2048, 4096),
        "8192^2*4096": oc(False, 8192, 4096),
        "8192*450*4096": oc(True, 8192, 4096, 450),
    }
    for kind, *f in golden("table7_and_cost_model.txt"):
        if kind == "cost":
            expr, printed = f
            digits = len(printed.split(".")[1]) if "." in printed else 0
            assert abs(vals[expr] / 1e9 - float(printed)) <= 0.6 * 10 ** (-digits), expr


def test_jaccard_reproduces_table1(golden):
    for model, rl, rl1, jac, inter in golden("table1_jaccard.txt"):
        rl, rl1, inter = int(rl), int(rl1), int(inter)
        a = np.arange(rl, dtype=np.int32)                       # overlap = last `inter` of a
        b = np.concatenate([np.arange(rl - inter, rl), np.arange(1000, 1000 + rl1 - inter)]).astype(np.int32)
        j = oracle.jaccard(a, b)
        assert j == pytest.approx(inter / (rl + rl1 - inter), abs=1e-15)
        assert abs(j - float(jac)) < 6e-4, (model, rl, rl1)
    assert oracle.jaccard([], []) == 1.0
    assert oracle.jaccard([1, 2], []) == 0.0


def test_turnover_reproduces_table6(golden):
    rows = golden("table6_gptj_cascade.txt")
    prev = int(rows[0][1])
    for layer, r, adds, rems, turn in rows[1:]:
        r, adds, rems = int(r), int(adds), int(rems)
        assert r == prev + adds - rems                           # accounting identity
        eta = oracle.turnover(adds, rems, prev)
        assert abs(100 * eta - float(turn)) < 0.51, layer
        prev = r
    assert abs(100 * oracle.turnover(131, 0, 69) - 189.9) < 0.06  # Table 3
    assert abs(100 * oracle.turnover(38, 55, 164) - 56.7) < 0.06
    assert math.isnan(oracle.turnover(1, 0, 0))


# ---------------------------------------------------------------- invariants on the workloads
SMALL = wl.scaled(wl.CONFIGS[3], T=384, d=256, L=6, P=40, rho=0.05, phi=0.01, u=0.03)


def chain(cfg, causal=False):
    Xs, labels = wl.generate_all(cfg, seed=0)
    out = []
    R = None
    for l, X in enumerate(Xs):
        X64 = wl.as_f64(X[0])
        full, gamma = oracle.select_full(X64, cfg.tau)
        if l == 0:
            R, step = full, None
        else:
            step = oracle.cascade_step(X64, cfg.tau, R, causal=causal)
            R_prev, R = R, step.rep
        out.append(dict(X=X64, labels=labels[l][0], full=full, gamma=gamma, step=step,
                        R=R, R_prev=None if l == 0 else R_prev))
    return out


@pytest.mark.parametrize("causal", [False, True])
def test_invariants_and_label_prediction(causal):
    cfg = SMALL
    thr = 1 - cfg.tau ** 2
    n_missed = 0
    R_lab = None
    for l, st in enumerate(chain(cfg, causal)):
        X, lab = st["X"], st["labels"]
        Xh = X / np.linalg.norm(X, axis=1, keepdims=True)
        G = np.abs(Xh @ Xh.T)
        # label-level prediction (no Gram involved)
        assert st["full"].tolist() == full_from_labels(lab).tolist()
        if l == 0:
            R_lab = full_from_labels(lab)
            assert st["R"].tolist() == R_lab.tolist()
        else:
            R_lab, add_lab, rem_lab = cascade_from_labels(lab, R_lab, causal)
            s = st["step"]
            assert s.rep.tolist() == R_lab.tolist()
            assert s.add.tolist() == add_lab.tolist() and s.rem.tolist() == rem_lab.tolist()
            Rp = st["R_prev"]
            valid = np.setdiff1d(Rp, s.rem)
            # structure
            assert s.rep[0] == 0 and np.all(np.diff(s.rep) > 0)
            assert set(s.rem) <= set(Rp) and not (set(s.add) & set(Rp))
            assert s.rep.size == Rp.size + s.add.size - s.rem.size
            assert set(s.rep) == set(valid) | set(s.add)
            # separation: (valid, valid) pairs; (new, valid) pairs (earlier ones when causal)
            Gv = G[np.ix_(valid, valid)]
            assert np.all(Gv[np.tril_indices(valid.size, -1)] < thr)
            for t in s.add:
                cols = valid[valid < t] if causal else valid
                assert np.all(G[t, cols] < thr)
            # the margin the workload promises: nothing near the threshold
            assert np.all(np.abs(s.gamma_rep - thr) > 0.02)
            nonrep = np.setdiff1d(np.arange(X.shape[0]), Rp)
            assert np.all(np.abs(s.gamma_cross[nonrep] - thr) > 0.02)
            missed = np.setdiff1d(st["full"], s.rep)
            n_missed += missed.size
            if causal:                                           # Proposition 3
                assert missed.size == 0
        # full selection: reps pairwise separated
        Gr = G[np.ix_(st["full"], st["full"])]
        assert np.all(Gr[np.tril_indices(st["full"].size, -1)] < thr)
    # without the causal restriction the superset property of Proposition 3 does not hold: on this
    # workload a later inherited representative shadows earlier tokens of its cluster
    assert (n_missed == 0) if causal else (n_missed > 0)


def test_unchanged_layer_keeps_inherited_set():
    cfg = wl.scaled(wl.CONFIGS[1], T=300, d=128, L=1, P=30)
    Xs, labels = wl.generate_all(cfg)
    X = wl.as_f64(Xs[0][0])
    R, gamma = oracle.select_full(X, cfg.tau)
    s = oracle.cascade_step(X, cfg.tau, R)
    # removals are impossible on the same layer; additions are exactly the
    # non-reps with no representative witness (none on a prototype workload)
    assert s.rem.size == 0 and set(R) <= set(s.rep)
    Xh = X / np.linalg.norm(X, axis=1, keepdims=True)
    G = np.abs(Xh @ Xh.T)
    nonrep = np.setdiff1d(np.arange(cfg.T), R)
    witness = (G[np.ix_(nonrep, R)] >= 1 - cfg.tau ** 2).any(axis=1)
    assert s.add.tolist() == nonrep[~witness].tolist()
    assert s.add.size == 0 and s.rep.tolist() == R.tolist()
    assert np.allclose(s.gamma_rep, gamma[R], atol=1.0)         # sanity only
    # with the full set inherited gamma_rep is a sub-maximum of gamma
    assert np.all(s.gamma_rep <= gamma[R] + 1e-15)


def test_forced_valid_and_row_sampling():
    st = chain(SMALL)[2]
    X, Rp = st["X"], st["R_prev"]
    ref = st["step"]
    fv = np.ones(Rp.size, dtype=np.uint8)
    fv[np.isin(Rp, ref.rem)] = 0
    again = oracle.cascade_step(X, SMALL.tau, Rp, force_valid=fv)
    assert again.rep.tolist() == ref.rep.tolist()
    nonrep = np.setdiff1d(np.arange(X.shape[0]), Rp)[::5]
    part = oracle.cascade_step(X, SMALL.tau, Rp, only_rows=nonrep)
    assert np.allclose(part.gamma_cross[nonrep], ref.gamma_cross[nonrep], atol=0)
    assert part.add.tolist() == [t for t in ref.add.tolist() if t in set(nonrep.tolist())]


# ---------------------------------------------------------------- nearest representative (Section 2.3)
def test_nearest_on_example_a_and_brute_force():
    X = rows_at_angles(EX_A_DEG, EX_A_NORM)
    near, g = oracle.nearest(X, [0, 4])                 # reps at 0 and 90 degrees
    assert near.tolist() == [0, 0, 0, 4, 4, 0]          # 20,40 -> 0; 60 -> 90 (cos 30 > cos 60); 180 -> 0
    assert np.allclose(g, [1.0, acos(20), acos(40), acos(30), 1.0, 1.0], atol=1e-12)
    rng = np.random.default_rng(9)
    Y = rng.standard_normal((60, 7))
    R = sorted(rng.choice(60, 11, replace=False).tolist())
    near, g = oracle.nearest(Y, R)
    Yh = Y / np.linalg.norm(Y, axis=1, keepdims=True)
    G = np.abs(Yh @ Yh[R].T)
    for t in range(60):
        if t in R:
            assert near[t] == t and abs(g[t] - 1.0) < 1e-12
        else:
            assert near[t] == R[int(np.argmax(G[t]))] and abs(g[t] - G[t].max()) < 1e-12
    assert oracle.nearest(Y, [])[0].tolist() == [-1] * 60


def test_nearest_ties_go_to_the_lowest_index_and_labels_agree():
    X = np.zeros((4, 3))
    X[0] = [1, 0, 0]; X[1] = [1, 0, 0]; X[2] = [0, 1, 0]; X[3] = [2, 0, 0]
    near, _ = oracle.nearest(X, [0, 1, 2])
    assert near[3] == 0                                  # exact tie between reps 0 and 1
    st = chain(SMALL)[3]
    near, g = oracle.nearest(st["X"], st["R"])
    lab = st["labels"]
    nonrep = np.setdiff1d(np.arange(lab.size), st["R"])
    # a redundant token's nearest representative carries its prototype label
    assert np.all(lab[near[nonrep]] == lab[nonrep]) and np.all(g[nonrep] > 0.9)


def test_tau_update_rule_by_hand_and_by_fractions():
    """Section 8.1, reading: tau' = clip(tau + gain * (target - rho)).  Pinned by values worked
    by hand in binary-exact numbers, by exact rational arithmetic, and by its properties: a
    stable set (turnover below target) tightens the threshold (tau grows), an evolving one
    loosens it, gain 0 or an undefined turnover leave tau alone, the bounds hold."""
    from fractions import Fraction
    f = oracle.tau_update
    # binary-exact operands: every intermediate is exact, so the result is too
    assert f(0.25, 0.125, 0.25, 0.5, 0.0625, 0.75) == 0.3125        # 0.25 + 0.5 * 0.125
    assert f(0.25, 0.5, 0.25, 0.5, 0.0625, 0.75) == 0.125           # 0.25 - 0.5 * 0.25
    assert f(0.25, 4.0, 0.25, 0.5, 0.0625, 0.75) == 0.0625          # clipped below
    assert f(0.5, 0.0, 1.0, 1.0, 0.0625, 0.75) == 0.75              # clipped above
    assert f(0.3, 0.05, 0.1, 0.0, 0.1, 0.6) == 0.3                  # gain 0
    assert f(0.3, float("nan"), 0.1, 0.5, 0.1, 0.6) == 0.3          # empty inherited set
    assert f(0.05, float("nan"), 0.1, 0.5, 0.1, 0.6) == 0.1         # ... still clipped
    rng = np.random.default_rng(3)
    for _ in range(200):
        tau, rho, target, gain = rng.uniform(0.05, 0.9), rng.uniform(0, 1.5), rng.uniform(0, 0.5), \
            rng.uniform(0, 2)
        got = f(tau, rho, target, gain, 0.05, 0.9)
        exact = Fraction(tau) + Fraction(gain) * (Fraction(target) - Fraction(rho))
        exact = min(Fraction(0.9), max(Fraction(0.05), exact))
        assert abs(Fraction(got) - exact) <= Fraction(1, 2 ** 50)    # three roundings of fp64
        assert 0.05 <= got <= 0.9
        if 0.05 < got < 0.9:
            assert (got > tau) == (rho < target) or got == tau
    # the turnover it is fed is Eq. 6
    assert oracle.turnover(3, 1, 8) == 0.5 and np.isnan(oracle.turnover(2, 0, 0))
