"""Pins for the FP64 oracle: each test checks it against something other than itself (direct least-squares
solves, direct inverses, brute force, closed forms), on problems small enough to enumerate."""
import itertools
import os

import numpy as np
import pytest

import obc_synth
import oracle

DAMP = obc_synth.DAMP_REL


def _problem(d_row, d_col, n, seed, kind="correlated"):
    W, X = obc_synth.make_small(d_row, d_col, n, seed, kind)
    H = oracle.hessian(X, plain_loops=True)
    lam = DAMP * np.trace(H) / d_col
    Hd = H + lam * np.eye(d_col)
    Hinv, info = oracle.inverse(H, DAMP)
    assert info == 0
    # ||v X_aug||^2 = ||v X||^2 + (lam/2)||v||^2 = (1/2) v^T Hd v : the dampened objective as plain least squares
    X_aug = np.concatenate([X.astype(np.float64), np.sqrt(lam / 2.0) * np.eye(d_col)], axis=1)
    return W.astype(np.float64), X.astype(np.float64), Hd, Hinv, X_aug


def _masked_lstsq(w0, X_aug, F):
    """argmin_v ||w0 X_aug - v X_aug[F]||^2 solved directly (Eq. 2 restricted to the support F)."""
    v = np.zeros_like(w0)
    if len(F):
        sol, *_ = np.linalg.lstsq(X_aug[F].T, X_aug.T @ w0, rcond=None)
        v[F] = sol
    return v


def test_hessian_is_twice_gram():
    W, X = obc_synth.make_small(2, 7, 33, 5)
    ref = 2.0 * np.einsum("in,jn->ij", X.astype(np.longdouble), X.astype(np.longdouble)).astype(np.float64)
    assert np.allclose(oracle.hessian(X, plain_loops=True), ref, rtol=1e-14, atol=0)
    assert np.allclose(oracle.hessian(X), ref, rtol=1e-13, atol=0)
    assert np.array_equal(oracle.hessian(X, True), oracle.hessian(X, True).T)


def test_inverse_matches_direct_inverse_and_flags_singular():
    _, _, Hd, Hinv, _ = _problem(1, 12, 80, 3)
    assert np.allclose(Hinv, np.linalg.inv(Hd), rtol=1e-9, atol=1e-14)
    assert np.array_equal(Hinv, Hinv.T)
    # duplicate input channel, no dampening: not positive definite -> reported, not returned
    Xs = np.random.default_rng(0).normal(size=(4, 10)).astype(np.float32)
    Xs[3] = Xs[1]
    _, info = oracle.inverse(oracle.hessian(Xs, True), 0.0)
    assert info == 4


@pytest.mark.parametrize("kind,seed", [("correlated", 0), ("relu", 1), ("correlated", 2)])
def test_pin_a_b_weights_are_masked_lstsq_and_lemma1(kind, seed):
    """(a) after every step the remaining weights are the masked least-squares optimum;
    (b) the eliminated inverse restricted to the remaining set is inv(H[M,M])  (Lemma 1)."""
    d = 10
    W, X, Hd, Hinv, X_aug = _problem(3, d, 64, seed, kind)
    for r in range(W.shape[0]):
        active = list(range(d))
        for t in range(d):
            res = oracle.eliminate_one_row(Hinv, W[r], steps=t + 1)
            assert res["status"] == 0
            active = [j for j in range(d) if j not in set(res["order"][:t + 1].tolist())]
            want = _masked_lstsq(W[r], X_aug, active)
            assert np.allclose(res["w"], want, rtol=1e-8, atol=1e-11)
            assert np.all(res["w"][res["order"][:t + 1]] == 0.0)
            if active:
                direct = np.linalg.inv(Hd[np.ix_(active, active)])
                assert np.allclose(res["Hi"][np.ix_(active, active)], direct, rtol=1e-8, atol=1e-13)
            dead = res["order"][:t + 1]
            assert np.all(res["Hi"][dead, :] == 0.0) and np.all(res["Hi"][:, dead] == 0.0)
            assert np.array_equal(res["w_trace"][t + 1], res["w"])


def test_pin_c_first_pick_is_brute_force():
    """Eq. 3: the first pick minimises the true loss increase over all single removals, and that increase
    is half the recorded score (the Hessian carries the factor 2)."""
    d = 9
    W, X, Hd, Hinv, X_aug = _problem(6, d, 50, 7)
    res = oracle.run_rows(Hinv, W, steps=1)
    for r in range(W.shape[0]):
        inc = []
        for j in range(d):
            F = [i for i in range(d) if i != j]
            v = _masked_lstsq(W[r], X_aug, F)
            inc.append(np.sum(((W[r] - v) @ X_aug) ** 2))
        assert int(np.argmin(inc)) == res["order"][r, 0]
        assert np.isclose(0.5 * res["loss"][r, 0], min(inc), rtol=1e-9)
        assert np.isclose(res["loss"][r, 0], W[r, res["order"][r, 0]] ** 2 / Hinv[res["order"][r, 0]] [res["order"][r, 0]])
        srt = np.sort(inc)
        assert np.isclose(res["margin"][r, 0], (srt[1] - srt[0]) / srt[1], rtol=1e-6)


def _grid_for(W, bits=3, symmetric=False):
    return oracle.minmax_grid(W, bits, symmetric)


@pytest.mark.parametrize("mode", ["prune", "quant"])
def test_pin_d_loss_trace_telescopes(mode):
    """half the sum of the recorded losses equals the layer error of the final weights."""
    d = 12
    W, X, Hd, Hinv, X_aug = _problem(4, d, 70, 11)
    kw = {}
    if mode == "quant":
        sc, ze, mq = _grid_for(W)
        kw = dict(mode="quant", scale=sc, zero=ze, maxq=mq)
    for T in (1, 5, d):
        res = oracle.run_rows(Hinv, W, steps=T, **kw)
        for r in range(W.shape[0]):
            dw = res["w"][r] - W[r]
            direct = np.sum((dw @ X_aug) ** 2)
            assert np.isclose(0.5 * res["loss"][r].sum(), direct, rtol=1e-8, atol=1e-14)
            assert np.isclose(direct, 0.5 * dw @ Hd @ dw, rtol=1e-9)


def test_pin_e_pruning_is_obq_with_zero_quantiser():
    d = 14
    W, X, Hd, Hinv, _ = _problem(5, d, 90, 13)
    a = oracle.run_rows(Hinv, W, want_trace=True)
    b = oracle.run_rows(Hinv, W, mode="quant", scale=np.ones(5), zero=np.zeros(5), maxq=0, want_trace=True)
    assert np.array_equal(a["order"], b["order"])
    assert np.array_equal(a["loss"], b["loss"])
    assert np.array_equal(a["w_trace"], b["w_trace"])
    assert np.all(b["codes"] == 0)


def test_pin_f_obq_invariants():
    """outputs on the grid, codes in range, and at every step the unquantised weights are the
    equality-constrained least-squares optimum given the already fixed ones (Eq. 6-7)."""
    d = 11
    W, X, Hd, Hinv, _ = _problem(4, d, 60, 17)
    sc, ze, mq = _grid_for(W, bits=3)
    res = oracle.run_rows(Hinv, W, mode="quant", scale=sc, zero=ze, maxq=mq, want_trace=True)
    assert np.all(res["codes"] >= 0) and np.all(res["codes"] <= mq)
    for r in range(4):
        assert np.allclose(res["w"][r], sc[r] * (res["codes"][r] - ze[r]), rtol=0, atol=1e-15)
        assert sorted(res["order"][r].tolist()) == list(range(d))
        for t in range(1, d):
            Q = res["order"][r, :t]
            F = np.array([j for j in range(d) if j not in set(Q.tolist())])
            wt = res["w_trace"][r, t]
            fixed = sc[r] * (res["codes"][r, Q] - ze[r])
            assert np.array_equal(wt[Q], fixed)
            want = W[r, F] - np.linalg.solve(Hd[np.ix_(F, F)], Hd[np.ix_(F, Q)] @ (fixed - W[r, Q]))
            assert np.allclose(wt[F], want, rtol=1e-8, atol=1e-12)


def test_pin_g_diagonal_hessian_special_case():
    """orthogonal input channels: nothing is compensated, prune order is ascending w_j^2 H_jj, OBQ is
    plain round-to-nearest."""
    d = 9
    W, X = obc_synth.make_small(3, d, 40, 19, "orthogonal")
    H = oracle.hessian(X, True)
    assert np.abs(H - np.diag(np.diag(H))).max() < 1e-6 * np.abs(H).max()
    H = np.diag(np.diag(H))
    Hinv, _ = oracle.inverse(H, 0.0)
    res = oracle.run_rows(Hinv, W, want_trace=True)
    W64 = W.astype(np.float64)
    for r in range(3):
        assert np.array_equal(res["order"][r], np.argsort(W64[r] ** 2 * np.diag(H), kind="stable"))
        for t in range(d + 1):
            keep = np.ones(d, bool); keep[res["order"][r, :t]] = False
            assert np.allclose(res["w_trace"][r, t], np.where(keep, W64[r], 0.0), rtol=0, atol=1e-15)
    sc, ze, mq = _grid_for(W, bits=4)
    q = oracle.run_rows(Hinv, W, mode="quant", scale=sc, zero=ze, maxq=mq)
    rtn = np.clip(np.rint(W64 / sc[:, None]) + ze[:, None], 0, mq)
    assert np.array_equal(q["codes"], rtn.astype(np.int32))


def test_pin_h_hand_worked_sizes():
    lines = open(os.path.join(os.path.dirname(__file__), "golden", "two_by_two.txt")).read().splitlines()
    g = {l.split()[0]: np.array(l.split()[1:], dtype=np.float64) for l in lines if l and not l.startswith("#")}
    H = g["H"].reshape(2, 2)
    Hinv, info = oracle.inverse(H, 0.0)
    res = oracle.eliminate_one_row(Hinv, g["w"], steps=1)
    assert res["order"][0] == int(g["order"][0])
    assert np.allclose(res["w"], g["w_after_first"], rtol=1e-14)
    assert np.isclose(res["Hi"][1, 1], g["hinv_after_first_11"][0], rtol=1e-14)
    full = oracle.eliminate_one_row(Hinv, g["w"])
    assert full["order"].tolist() == g["order"].astype(int).tolist()
    assert np.allclose(full["loss"], g["loss"], rtol=1e-14)
    # d_col = 1: Hinv = 1/h, loss = w^2 h, the weight ends at 0
    one = oracle.eliminate_one_row(np.array([[0.25]]), np.array([3.0]))
    assert one["order"].tolist() == [0] and np.isclose(one["loss"][0], 36.0) and one["w"][0] == 0.0
    assert one["margin"][0] == 1.0


def test_ties_go_to_lowest_index_and_teacher_forcing_reports_gap():
    Hinv = np.diag([1.0, 1.0, 2.0, 1.0])
    w = np.array([0.5, 0.0, 0.0, 0.5])
    res = oracle.eliminate_one_row(Hinv, w)
    assert res["order"].tolist() == [1, 2, 0, 3]
    assert res["margin"][0] == 0.0           # exact tie between the two zero weights
    forced = oracle.eliminate_one_row(Hinv, w, forced=np.array([2, 1, 3, 0], np.int32))
    assert forced["order"].tolist() == [2, 1, 3, 0]
    assert forced["best"].tolist() == [1, 1, 0, 0]
    assert np.all(forced["forced_gap"] == 0.0)   # every forced pick ties with the oracle's own
    bad = oracle.eliminate_one_row(Hinv, w, forced=np.array([0, 1, 2, 3], np.int32))
    assert bad["forced_gap"][0] == 1.0 and bad["best"][0] == 1


def _alg2_bruteforce(L, k):
    """simulate 'prune the globally smallest next loss' with a linear scan each time"""
    rows, d = L.shape
    cnt = np.zeros(rows, int)
    for _ in range(k):
        nxt = [L[i, cnt[i]] if cnt[i] < d else np.inf for i in range(rows)]
        cnt[int(np.argmin(nxt))] += 1          # argmin returns the lowest row among ties
    return cnt


def _prefixmax_select(L, k):
    """k smallest under the lexicographic key (prefix-max of the row's losses, row, step)"""
    rows, d = L.shape
    key = np.maximum.accumulate(L, axis=1)
    trip = sorted((key[i, t], i, t) for i in range(rows) for t in range(d))[:k]
    cnt = np.zeros(rows, int)
    for _, i, _ in trip:
        cnt[i] += 1
    return cnt


@pytest.mark.parametrize("seed", range(6))
def test_pin_i_global_step(seed):
    rng = np.random.default_rng(seed)
    rows, d = 7, 9
    L = rng.exponential(size=(rows, d))
    if seed % 2:                                   # plant ties and non-monotone rows
        L = np.round(L * 3) / 3
    P = np.stack([rng.permutation(d) for _ in range(rows)]).astype(np.int32)
    for k in (0, 1, 5, 17, 40, rows * d - 1, rows * d):
        cnt, mask = oracle.global_mask(L, P, k)
        assert cnt.sum() == k and (mask == 0).sum() == k
        assert np.array_equal(cnt, _alg2_bruteforce(L, k))
        assert np.array_equal(cnt, _prefixmax_select(L, k))
        for i in range(rows):
            assert sorted(np.nonzero(mask[i] == 0)[0].tolist()) == sorted(P[i, :cnt[i]].tolist())
    Lm = np.sort(rng.exponential(size=(rows, d)), axis=1)      # monotone rows: plain k-smallest
    k = 23
    cnt, _ = oracle.global_mask(Lm, P, k)
    thr = np.sort(Lm.ravel())[k - 1]
    assert np.array_equal(cnt, (Lm <= thr).sum(axis=1))
    with pytest.raises(ValueError):
        oracle.global_mask(L, P, rows * d + 1)


def test_pin_j_compound_subproblem():
    """the elimination path restricted to the survivors equals the directly formed sub-problem."""
    d = 13
    W, X, Hd, Hinv, X_aug = _problem(3, d, 70, 23)
    for r, cnt in enumerate((0, 4, 9)):
        seq = oracle.eliminate_one_row(Hinv, W[r], steps=cnt)
        pruned = seq["order"][:cnt]
        F, wF, HiF = oracle.group_obs_state(Hinv, W[r], pruned)
        assert np.allclose(HiF, np.linalg.inv(Hd[np.ix_(F, F)]), rtol=1e-8, atol=1e-13)
        assert np.allclose(seq["Hi"][np.ix_(F, F)], HiF, rtol=1e-8, atol=1e-13)
        assert np.allclose(seq["w"][F], wF, rtol=1e-8, atol=1e-12)
        assert np.allclose(wF, _masked_lstsq(W[r], X_aug, list(F))[F], rtol=1e-8, atol=1e-12)
        comp = oracle.compound_row(Hinv, W[r], pruned, bits=4, symmetric=True)
        assert np.all(comp["w"][pruned] == 0.0) and np.all(comp["codes"][pruned] == -1)
        assert np.allclose(comp["w"][F], comp["scale"] * (comp["codes"][F] - comp["zero"]), atol=1e-15)
        # same thing through the sequential path with the survivors' mask
        act = np.zeros(d, np.uint8); act[F] = 1
        seq_q = oracle.eliminate_one_row(seq["Hi"], seq["w"], steps=len(F), mode="quant", scale=comp["scale"],
                                         zero=comp["zero"], maxq=comp["maxq"], active0=act)
        assert np.array_equal(seq_q["order"][:len(F)], comp["order"])
        assert np.array_equal(seq_q["codes"][F], comp["codes"][F])


def test_minmax_grid_hand_cases():
    W = np.array([[-1.0, 0.5, 2.0, 0.0], [0.25, 0.5, 1.0, 0.75], [0.0, 0.0, 0.0, 0.0], [-3.0, -1.0, -2.0, -0.5]])
    sc, ze, mq = oracle.minmax_grid(W, 2, False)
    assert mq == 3
    assert np.allclose(sc, [1.0, 1.0 / 3.0, 1.0, 1.0]) and np.array_equal(ze, [1.0, 0.0, 0.0, 3.0])
    sc, ze, mq = oracle.minmax_grid(W, 4, True)
    assert mq == 14 and np.all(ze == 7.0) and np.allclose(sc, [2.0 / 7, 1.0 / 7, 1.0, 3.0 / 7])
    mask = np.array([[1, 1, 0, 1]] * 4, np.uint8)
    sc, _, _ = oracle.minmax_grid(W, 2, False, mask)
    assert np.isclose(sc[0], 0.5)                      # the 2.0 entry is masked out: range [-1, 0.5]


def test_outlier_rule_takes_largest_error_first():
    Hinv = np.diag([1.0, 1.0, 1.0])
    w = np.array([0.1, 5.0, 9.0])       # grid {0,1,2,3}: entries 1 and 2 lie outside, errors 2 and 6
    plain = oracle.eliminate_one_row(Hinv, w, mode="quant", scale=1.0, zero=0.0, maxq=3)
    assert plain["order"].tolist() == [0, 1, 2]
    out = oracle.eliminate_one_row(Hinv, w, mode="quant", scale=1.0, zero=0.0, maxq=3, flags=oracle.FLAG_OUTLIERS)
    assert out["order"].tolist() == [2, 1, 0]
    assert out["codes"].tolist() == [0, 3, 3]


def test_pin_k_deterministic_and_config1_fast():
    W, X, spec = obc_synth.make_layer("C1")
    H = oracle.hessian(X)
    Hinv, info = oracle.inverse(H, DAMP)
    assert info == 0
    a = oracle.run_rows(Hinv, W, want_trace=True)
    b = oracle.run_rows(Hinv, W, want_trace=True)
    for key in ("order", "loss", "w", "w_trace"):
        assert np.array_equal(a[key], b[key])
    assert np.all(a["status"] == 0)
    k = obc_synth.pruned_count(spec.d_row, spec.d_col, 0.5)
    cnt, mask = oracle.global_mask(a["loss"], a["order"], k)
    What = oracle.weights_from_trace(a["w_trace"], cnt)
    assert (mask == 0).sum() == k == 1024 and np.all(What[mask == 0] == 0.0)
    # the trace-reload weights are the masked least-squares optimum of their own mask
    lam = DAMP * np.trace(H) / spec.d_col
    X_aug = np.concatenate([X.astype(np.float64), np.sqrt(lam / 2) * np.eye(spec.d_col)], axis=1)
    for r in (0, 13, 31):
        F = np.nonzero(mask[r])[0]
        assert np.allclose(What[r], _masked_lstsq(W[r].astype(np.float64), X_aug, list(F)), rtol=1e-6, atol=1e-10)


@pytest.mark.parametrize("nm", [(2, 4), (4, 8), (1, 4)])
def test_pin_nm_pattern(nm):
    """N:M pruning (Section 3, "N:M Sparsity"): (1) every block of M consecutive weights ends with exactly N
    non-zeros; (2) every pick is the brute-force minimiser of the true loss increase over the weights still
    allowed (blocks that have not yet lost M - N), checked by solving each candidate's masked least-squares problem
    directly; (3) the final weights are the masked least-squares optimum for the final support; (4) with a
    diagonal Hessian each block simply loses its M - N smallest w_j^2 H_jj."""
    n_keep, m = nm
    d = 16
    W, X, Hd, Hinv, X_aug = _problem(3, d, 80, 31 + m)
    res = oracle.run_rows(Hinv, W, nm=nm, want_trace=True)
    steps = d // m * (m - n_keep)
    assert res["order"].shape[1] == steps and np.all(res["status"] == 0)
    for r in range(W.shape[0]):
        pruned = []
        for t in range(steps):
            cnt = np.bincount(np.array(pruned, dtype=np.int64) // m, minlength=d // m)
            allowed = [j for j in range(d) if j not in pruned and cnt[j // m] < m - n_keep]
            base = np.sum(((W[r] - res["w_trace"][r, t]) @ X_aug) ** 2)
            inc = {}
            for j in allowed:
                F = [i for i in range(d) if i not in pruned and i != j]
                v = _masked_lstsq(W[r], X_aug, F)
                inc[j] = np.sum(((W[r] - v) @ X_aug) ** 2) - base
            best = min(inc, key=lambda j: (inc[j], j))
            assert best == res["order"][r, t]
            assert np.isclose(0.5 * res["loss"][r, t], inc[best], rtol=1e-6, atol=1e-12)
            pruned.append(int(res["order"][r, t]))
        nz = (res["w"][r] != 0.0).reshape(d // m, m).sum(axis=1)
        assert np.all(nz == n_keep)
        keep = [j for j in range(d) if j not in pruned]
        assert np.allclose(res["w"][r], _masked_lstsq(W[r], X_aug, keep), rtol=1e-8, atol=1e-11)
    Wo, Xo = obc_synth.make_small(2, d, 40, 77, "orthogonal")
    Ho = np.diag(np.diag(oracle.hessian(Xo, True)))
    Hio, _ = oracle.inverse(Ho, 0.0)
    ro = oracle.run_rows(Hio, Wo, nm=nm)
    score = Wo.astype(np.float64) ** 2 * np.diag(Ho)
    for r in range(2):
        want = set()
        for b in range(d // m):
            idx = np.argsort(score[r, b * m:(b + 1) * m], kind="stable")[:m - n_keep] + b * m
            want |= set(idx.tolist())
        assert set(ro["order"][r].tolist()) == want
        assert np.array_equal(ro["order"][r], np.array(sorted(want, key=lambda j: (score[r, j], j))))


@pytest.mark.parametrize("c", [2, 4, 8])
def test_pin_block_pruning(c):
    """Block pruning (Section 3, "Block-Sparsity", Eq. 5): (1) every pick is the brute-force minimiser over the remaining
    blocks of the true loss increase, which is half the recorded block score; (2) after every block step the
    remaining weights are the masked least-squares optimum and the reduced inverse is inv(H[M,M]); (3) with c = 1 the
    procedure is Algorithm 1; (4) with a diagonal Hessian the block score is sum w_j^2 H_jj over the block."""
    d = 12 if c < 8 else 24
    W, X, Hd, Hinv, X_aug = _problem(3, d, 70, 41 + c)
    nblk = d // c
    for r in range(W.shape[0]):
        removed = []
        for t in range(nblk):
            res = oracle.run_rows_blocks(Hinv, W[r], c, steps=t + 1, return_hi=True)
            assert res["status"][0] == 0
            keep_before = [j for j in range(d) if j not in removed]
            base = np.sum(((W[r] - _masked_lstsq(W[r], X_aug, keep_before)) @ X_aug) ** 2)
            inc = {}
            for q in range(nblk):
                blk = list(range(q * c, q * c + c))
                if blk[0] in removed:
                    continue
                F = [j for j in keep_before if j not in blk]
                inc[q] = np.sum(((W[r] - _masked_lstsq(W[r], X_aug, F)) @ X_aug) ** 2) - base
            best = min(inc, key=lambda q: (inc[q], q))
            picked = res["order"][0, t * c:(t + 1) * c]
            assert picked.tolist() == list(range(best * c, best * c + c))
            assert np.isclose(0.5 * res["loss"][0, t * c], inc[best], rtol=1e-6, atol=1e-12)
            assert np.all(res["loss"][0, t * c + 1:(t + 1) * c] == 0.0)
            removed += picked.tolist()
            keep = [j for j in range(d) if j not in removed]
            assert np.allclose(res["w"][0], _masked_lstsq(W[r], X_aug, keep), rtol=1e-8, atol=1e-11)
            assert np.all(res["w"][0][removed] == 0.0)
            if keep:
                assert np.allclose(res["Hi"][0][np.ix_(keep, keep)], np.linalg.inv(Hd[np.ix_(keep, keep)]), rtol=1e-8, atol=1e-13)
    one = oracle.run_rows_blocks(Hinv, W, 1)
    ref = oracle.run_rows(Hinv, W)
    assert np.array_equal(one["order"], ref["order"]) and np.allclose(one["loss"], ref["loss"], rtol=1e-12)
    assert np.allclose(one["w"], ref["w"], atol=1e-14)
    Wo, Xo = obc_synth.make_small(2, d, 40, 5, "orthogonal")
    Ho = np.diag(np.diag(oracle.hessian(Xo, True)))
    Hio, _ = oracle.inverse(Ho, 0.0)
    ro = oracle.run_rows_blocks(Hio, Wo, c)
    score = (Wo.astype(np.float64) ** 2 * np.diag(Ho)).reshape(2, nblk, c).sum(axis=2)
    for r in range(2):
        assert np.array_equal(ro["order"][r, ::c] // c, np.argsort(score[r], kind="stable"))
        assert np.allclose(ro["loss"][r, ::c], np.sort(score[r]), rtol=1e-12)


def test_golden_c1_trace_is_reproduced():
    """the stored C1 trace (written by tests/golden/make_c1_trace.py from the oracle alone) is reproduced: guards
    the oracle's arithmetic against unintended changes"""
    import importlib.util
    here = os.path.join(os.path.dirname(__file__), "golden")
    spec = importlib.util.spec_from_file_location("make_c1_trace", os.path.join(here, "make_c1_trace.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    order, loss, codes, qorder = mod.compute()
    want = {}
    for line in open(os.path.join(here, "c1_trace_rows.txt")):
        if line.startswith("#"):
            continue
        name, r, *vals = line.split()
        want[(name, int(r))] = vals
    for r in range(3):
        assert [int(v) for v in want[("order", r)]] == order[r].tolist()
        assert [int(v) for v in want[("codes", r)]] == codes[r].tolist()
        assert [int(v) for v in want[("qorder", r)]] == qorder[r].tolist()
        assert np.allclose([float(v) for v in want[("loss", r)]], loss[r], rtol=1e-12, atol=0)


def test_pin_refit_is_the_regularised_least_squares_optimum():
    """the dense refit (appendix "Sequential Quantization with OBQ") is the minimiser of ||Y - W X||^2 + (lambda/2)||W||^2:
    zero gradient, equality with a least-squares solve of the augmented system, and recovery of the generating
    weights when Y = W0 X exactly and there is no dampening"""
    rng = np.random.default_rng(3)
    d, R, n = 11, 4, 90
    W0, X = obc_synth.make_small(R, d, n, 61)
    X = X.astype(np.float64)
    Y = W0.astype(np.float64) @ X + 0.1 * rng.normal(size=(R, n))
    W = oracle.refit(X, Y, DAMP)
    lam = DAMP * np.trace(2.0 * X @ X.T) / d
    grad = -2.0 * (Y - W @ X) @ X.T + lam * W
    assert np.abs(grad).max() <= 1e-9 * np.abs(2.0 * Y @ X.T).max()
    X_aug = np.concatenate([X, np.sqrt(lam / 2.0) * np.eye(d)], axis=1)
    Y_aug = np.concatenate([Y, np.zeros((R, d))], axis=1)
    sol, *_ = np.linalg.lstsq(X_aug.T, Y_aug.T, rcond=None)
    assert np.allclose(W, sol.T, rtol=1e-9, atol=1e-12)
    assert np.allclose(oracle.refit(X, W0.astype(np.float64) @ X, 0.0), W0, rtol=1e-8, atol=1e-10)
