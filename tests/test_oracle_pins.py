"""Pins for the CPU oracle: everything here checks oracle/ against something
other than itself -- values the paper prints, closed forms, invariants,
special cases that reduce to a library routine, and brute force on tiny
inputs.  No GPU, no CUDA library."""

import itertools
import math

import numpy as np
import pytest

from oracle import brace_oracle as O


def _mat(*rows):
    return np.array(rows, dtype=np.float32)


# ---------------------------------------------------------------- printed values
def test_worked_example_share_reduce_and_share_only(golden):
    """Section 2.2 worked example: hop-1 reduced value, ownership, final sum."""
    g = golden("rar_worked_example.txt")
    U = _mat(g["g1"], g["g2"], g["g3"])
    tr = O.ring_round(U, rule=O.RULE_SUM, granule=1)
    # hop 1: the receiver named in the paper holds the named sub-vector reduced to -2
    seg, val = tr.rs_states[0][g["hop1_receiver"]]
    assert seg == g["hop1_subvector"]
    assert val.tolist() == [g["hop1_reduced"]]
    # that value is what Client 1 forwards to Client 2 at hop 2: Client 2 then
    # holds sub-vector 3 fully reduced = -10 + 7 + 8 = 5
    seg2, val2 = tr.rs_states[1][1]
    assert seg2 == 2 and val2.tolist() == [5]
    # ownership after n-1 hops
    seg_o, val_o = tr.owned[g["owner_client"]]
    assert seg_o == g["owner_subvector"]
    assert val_o.tolist() == [g["owner_value"]]
    # every client ends with the sum
    for c in range(3):
        assert tr.outputs[c].tolist() == g["final"]


def test_attacked_example(golden):
    """Section 3, first paragraph: altered Client 1 shifts the plain RAR result."""
    g = golden("rar_attacked_example.txt")
    U = _mat(g["g1"], g["g2"], g["g3"])
    tr = O.ring_round(U, rule=O.RULE_SUM, granule=1)
    for c in range(3):
        assert tr.outputs[c].tolist() == g["final"]


def test_comm_cost_closed_forms(golden):
    """Table 1: bits sent per client by the simulated schedule equal the closed forms."""
    rows = golden("comm_cost_table1.txt")["rows"]
    rng = np.random.default_rng(1)
    for n, d, m, sc, rar, brace in rows:
        assert O.cost_sc(m, n, d) == sc
        num, den = O.cost_rar(m, n, d)
        assert num % den == 0 and num // den == rar
        num, den = O.cost_brace(m, n, d)
        assert num % den == 0 and num // den == brace
        U = rng.standard_normal((n, d)).astype(np.float32)
        tb = O.ring_round(U, rule=O.RULE_SIGN_CONSENSUS, lam=0, granule=1, keep_states=False)
        assert O.sent_bits(tb, m, O.RULE_SIGN_CONSENSUS).tolist() == [brace] * n
        ts = O.ring_round(U, rule=O.RULE_SUM, granule=1, keep_states=False)
        assert O.sent_bits(ts, m, O.RULE_SUM).tolist() == [rar] * n


def test_derived_sign_example():
    """Signs of the Section 2.2 gradients sum to [3, 1, 1]; lambda = 2 (the value
    Section 3 uses for its three-client illustration) keeps only the unanimous one."""
    U = _mat([5, 2, -10], [8, -4, 7], [9, 3, 8])
    assert O.sign_sum_direct(U).tolist() == [3, 1, 1]
    assert O.gar_direct(U, 2).tolist() == [1, -1, -1]
    tr = O.ring_round(U, lam=2, granule=1)
    for c in range(3):
        assert tr.outputs[c].tolist() == [1, -1, -1]
    # the attacked gradient of Section 3 has the same signs: BRACE is unmoved
    Ua = _mat([5, 2, -200], [8, -4, 7], [9, 3, 8])
    assert O.gar_direct(Ua, 2).tolist() == [1, -1, -1]


# ---------------------------------------------------------------- sign / lambda / bits
def test_sgn_special_values():
    x = np.array([0.0, -0.0, 1e-45, -1e-45, np.inf, -np.inf, np.nan, 3.4e38, -3.4e38, 2.0, -7.5],
                 dtype=np.float32)
    assert O.sgn(x).tolist() == [0, 0, 1, -1, 1, -1, 0, 1, -1, 1, -1]
    assert O.sgn(x, zero_sign=1).tolist() == [1, 1, 1, -1, 1, -1, 0, 1, -1, 1, -1]
    assert O.sgn(x, zero_sign=-1).tolist() == [-1, -1, 1, -1, 1, -1, 0, 1, -1, 1, -1]


@pytest.mark.parametrize("n", [2, 3, 7])
def test_lambda_int_matches_real_comparison(n):
    for lam in [-n - 3.5, -n - 1, -n - 0.5, -n, -1.5, -1, -0.25, 0, 0.5, 1, 1.999, 2, n - 0.5, n, n + 4.2]:
        li = O.lambda_int(lam, n)
        assert -n - 1 <= li <= n
        for s in range(-n, n + 1):
            assert (s > li) == (s > lam), (n, lam, s)
    with pytest.raises(ValueError):
        O.lambda_int(float("nan"), n)
    with pytest.raises(ValueError):
        O.lambda_int(float("inf"), n)


def test_pack_bits_layout():
    assert O.pack_bits(np.array([1, -1, -1, 1])).tolist() == [0b1001]
    v = -np.ones(70, dtype=np.int8)
    v[0] = v[31] = v[32] = v[69] = 1
    w = O.pack_bits(v)
    assert w.tolist() == [(1 << 31) | 1, 1, 1 << 5]
    assert O.pack_bits(v, words=5).tolist() == [(1 << 31) | 1, 1, 1 << 5, 0, 0]
    rng = np.random.default_rng(5)
    for d in [1, 31, 32, 33, 64, 100, 257]:
        v = rng.choice([-1, 1], size=d).astype(np.int8)
        assert np.array_equal(O.pack_bits(v), O.pack_bits_fast(v))
        assert np.array_equal(O.pack_bits(v, words=12), O.pack_bits_fast(v, words=12))


# ---------------------------------------------------------------- partition
@pytest.mark.parametrize("n,d,G", [(3, 3, 1), (4, 10, 1), (5, 3, 1), (8, 100000, 128), (20, 1663370, 128),
                                   (100, 25557032, 128), (5, 8, 2), (5, 8, 128), (7, 1000, 32), (16, 124439808, 128)])
def test_partition_properties(n, d, G):
    b = O.partition(n, d, G)
    assert len(b) == n
    assert b[0][0] == 0 and b[-1][1] == d
    for j in range(n):
        assert b[j][0] <= b[j][1]
        if j:
            assert b[j][0] == b[j - 1][1]
        assert b[j][0] % G == 0 or b[j][0] == d
    sizes = [e - s for s, e in b]
    assert sum(sizes) == d
    if G == 1:
        assert max(sizes) - min(sizes) <= 1
        if d % n == 0:
            assert sizes == [d // n] * n
    else:
        # "roughly equal": sizes differ by at most one granule (plus the ragged tail)
        assert max(sizes) - min(sizes) <= 2 * G


def test_partition_printed_example_is_singletons():
    assert O.partition(3, 3, 1) == [(0, 1), (1, 2), (2, 3)]


# ---------------------------------------------------------------- closed form / invariants
@pytest.mark.parametrize("n,d,G", [(2, 5, 1), (3, 17, 2), (5, 64, 32), (8, 1000, 128), (13, 777, 1), (20, 5000, 128)])
def test_output_domain_identical_clients_and_direct(n, d, G):
    rng = np.random.default_rng(n * 1000 + d)
    U = rng.standard_normal((n, d)).astype(np.float32)
    U[rng.random((n, d)) < 0.2] = 0.0
    for lam in [-2, 0, 1, 2.5]:
        tr = O.ring_round(U, lam=lam, granule=G)
        out = tr.outputs
        assert set(np.unique(out).tolist()) <= {-1, 1}          # Appendix A: 2*I - 1, never 0
        for c in range(1, n):
            assert np.array_equal(out[c], out[0])                # Section 3 Phase IV
        assert np.array_equal(out[0], O.gar_direct(U, lam))      # procedure == definition
        S = O.sign_sum_direct(U)
        assert np.array_equal(out[0], 2 * (S > math.floor(lam)).astype(np.int8) - 1)
        # owned partials are the full sign sums of their sub-vectors
        for c in range(n):
            j, part = tr.owned[c]
            assert j == (c + 1) % n
            b, e = tr.bounds[j]
            assert np.array_equal(part, S[b:e])


def test_threshold_special_cases():
    rng = np.random.default_rng(3)
    n, d = 6, 50
    U = rng.standard_normal((n, d)).astype(np.float32)
    assert (O.gar_direct(U, n) == -1).all() and (O.ring_round(U, lam=n).outputs == -1).all()
    assert (O.gar_direct(U, n + 10) == -1).all()
    assert (O.gar_direct(U, -n - 1) == 1).all() and (O.ring_round(U, lam=-n - 1).outputs == 1).all()
    assert (O.gar_direct(U, -n - 0.5) == 1).all()
    Z = np.zeros((n, d), dtype=np.float32)
    assert (O.gar_direct(Z, 0) == -1).all()        # S = 0 <= 0
    assert (O.gar_direct(Z, -1) == 1).all()        # S = 0 > -1
    assert (O.gar_direct(Z, 0, zero_sign=1) == 1).all()   # zeros vote +1: S = n > 0
    assert (O.gar_direct(Z, n - 1, zero_sign=1) == 1).all()
    assert (O.gar_direct(Z, -n, zero_sign=-1) == -1).all()  # S = -n, tie -> -1
    # n identical clients: S = n * sign(g)
    g = rng.standard_normal(d).astype(np.float32)
    I = np.tile(g, (n, 1))
    for lam in [0, n - 1]:
        assert np.array_equal(O.gar_direct(I, lam), np.where(g > 0, 1, -1))
    assert (O.gar_direct(I, -n) == np.where(g < 0, -1, 1)).all()   # tie at S = -n gives -1


def test_invariance_permutation_granule_rotation():
    rng = np.random.default_rng(11)
    n, d = 7, 300
    U = rng.standard_normal((n, d)).astype(np.float32)
    U[rng.random((n, d)) < 0.1] = 0
    base = O.ring_round(U, lam=1, granule=1).outputs[0]
    for G in [2, 3, 32, 128, 1000]:
        assert np.array_equal(O.ring_round(U, lam=1, granule=G).outputs[0], base)
    for _ in range(5):
        perm = rng.permutation(n)
        assert np.array_equal(O.ring_round(U[perm], lam=1, granule=32).outputs[0], base)
    for r in range(1, n):
        assert np.array_equal(O.ring_round(np.roll(U, r, axis=0), lam=1, granule=32).outputs[0], base)


@pytest.mark.parametrize("n,f,lam", [(10, 2, 0), (10, 3, 1), (100, 20, 5), (9, 4, 0), (20, 4, 1)])
def test_robustness_property(n, f, lam):
    """If the n-f honest clients agree on a sign and their margin over the f
    Byzantine votes clears lambda, the Byzantine values cannot change the output."""
    rng = np.random.default_rng(n + f)
    d = 40
    honest_pos = np.abs(rng.standard_normal((n - f, d))).astype(np.float32) + 0.1
    for byz in [rng.standard_normal((f, d)) * 1e6, -np.ones((f, d)) * 1e30, np.zeros((f, d)), np.ones((f, d))]:
        U = np.vstack([byz.astype(np.float32), honest_pos])
        if (n - f) - f > lam:
            assert (O.ring_round(U, lam=lam, granule=4, keep_states=False).outputs == 1).all()
        U = np.vstack([byz.astype(np.float32), -honest_pos])
        if -(n - f) + f <= lam:
            assert (O.ring_round(U, lam=lam, granule=4, keep_states=False).outputs == -1).all()


# ---------------------------------------------------------------- plain RAR (degenerate rule)
@pytest.mark.parametrize("n,d,G", [(2, 9, 1), (4, 1000, 128), (7, 333, 1), (20, 4096, 128)])
def test_sum_rule_is_the_sum(n, d, G):
    rng = np.random.default_rng(n + d)
    U = (rng.standard_normal((n, d)) * 3).astype(np.float32)
    tr = O.ring_round(U, rule=O.RULE_SUM, granule=G)
    for c in range(1, n):
        assert np.array_equal(tr.outputs[c], tr.outputs[0])
    # library routine: numpy's float64 sum; float32 ring-order error stays inside
    # the textbook bound (n-1) * 2^-24 * sum|x|
    ref = np.sum(U.astype(np.float64), axis=0)
    assert np.allclose(O.sum_direct_f64(U), ref, rtol=0, atol=1e-12)
    bound = (n - 1) * 2.0 ** -24 * np.sum(np.abs(U.astype(np.float64)), axis=0)
    assert (np.abs(tr.outputs[0].astype(np.float64) - ref) <= bound + 1e-30).all()
    # exact order: sub-vector j is reduced starting at client j going downstream
    for j, (b, e) in enumerate(tr.bounds):
        acc = U[j, b:e].copy()
        for i in range(1, n):
            acc = np.float32(1) * (acc + U[(j + i) % n, b:e])
        assert np.array_equal(tr.outputs[0][b:e], acc)
    # mean = sum / n
    trm = O.ring_round(U, rule=O.RULE_SUM, granule=G, mean=True)
    assert np.allclose(trm.outputs[0], ref / n, rtol=1e-5, atol=1e-6)
    assert np.array_equal(trm.outputs[0], tr.outputs[0] / np.float32(n))


def test_sum_rule_integer_inputs_exact():
    rng = np.random.default_rng(0)
    U = rng.integers(-1000, 1000, size=(9, 200)).astype(np.float32)
    tr = O.ring_round(U, rule=O.RULE_SUM, granule=8)
    assert np.array_equal(tr.outputs[3], U.astype(np.int64).sum(0).astype(np.float32))


# ---------------------------------------------------------------- brute force on tiny inputs
def _expected_from_digits(digits_per_client, lam):
    pos = sum(1 for t in digits_per_client if t == 2)
    neg = sum(1 for t in digits_per_client if t == 0)
    return 1 if (pos - neg) > lam else -1


@pytest.mark.parametrize("n", [2, 3, 4, 5])
def test_brute_force_all_sign_patterns(n):
    """Every one of the 3^n (negative, zero, positive) patterns visits every
    coordinate, for d = 1..8 (d < n and n not dividing d included), every
    integer lambda in [-n-1, n] with G = 1, and G in {2, 128} for three lambdas.
    Expected values come from counting the pattern's digits, not from floats."""
    patterns = list(itertools.product([0, 1, 2], repeat=n))
    P = len(patterns)
    mags = np.array([0.5, 3.0, 1e-30, 7e20], dtype=np.float32)
    for d in range(1, 9):
        for m in range(P):
            U = np.zeros((n, d), dtype=np.float32)
            pats = [patterns[(m + k) % P] for k in range(d)]
            for k, pat in enumerate(pats):
                for i, t in enumerate(pat):
                    U[i, k] = (t - 1) * mags[(i + k) % 4]
            settings = [(lam, 1) for lam in range(-n - 1, n + 1)]
            settings += [(lam, G) for G in (2, 128) for lam in (-1, 0, 1)]
            if m % 9:                       # full lambda sweep on a ninth of the matrices
                settings = [(0, 1), (1, 2), (-1, 128)]
            for lam, G in settings:
                exp = [_expected_from_digits(p, lam) for p in pats]
                tr = O.ring_round(U, lam=lam, granule=G, keep_states=False)
                assert tr.outputs[0].tolist() == exp, (n, d, m, lam, G)
                assert (tr.outputs == tr.outputs[0]).all()
                assert O.gar_direct(U, lam).tolist() == exp


def test_brute_force_per_hop_partials():
    """After share-reduce hop s, client r holds sub-vector (r-1-s) mod n reduced
    over clients r-s-1 .. r (s+2 consecutive clients ending at r): checked by
    summing digits with plain Python integers."""
    rng = np.random.default_rng(4)
    for n, d, G in [(3, 5, 1), (4, 8, 2), (5, 7, 1), (5, 40, 8)]:
        digits = rng.integers(0, 3, size=(n, d))
        U = ((digits - 1) * 2.5).astype(np.float32)
        tr = O.ring_round(U, lam=0, granule=G)
        assert len(tr.rs_states) == n - 1
        for s in range(n - 1):
            for r in range(n):
                j, part = tr.rs_states[s][r]
                assert j == (r - 1 - s) % n
                b, e = tr.bounds[j]
                exp = [sum(int(digits[(r - i) % n, k]) - 1 for i in range(s + 2)) for k in range(b, e)]
                assert part.tolist() == exp


# ---------------------------------------------------------------- attack injection
def test_inject_scale_own_and_gaussian_closed_forms():
    H = _mat([1, -2, 0.5], [3, 4, 5], [6, 7, 8])
    out = O.inject_attack(O.ATTACK_SCALE_OWN, H, [0], scale=-10.0)
    assert out.tolist() == [[-10, 20, -5], [3, 4, 5], [6, 7, 8]]
    z = _mat([0.5, -1.0, 2.0])
    out = O.inject_attack(O.ATTACK_GAUSSIAN, H, [1], sigma=200.0, noise=z)
    assert out.tolist() == [[1, -2, 0.5], [100, -200, 400], [6, 7, 8]]
    # product rounds once, exactly like a float32 multiply
    rng = np.random.default_rng(2)
    h = rng.standard_normal((2, 1000)).astype(np.float32)
    out = O.inject_attack(O.ATTACK_SCALE_OWN, h, [1], scale=0.3)
    assert np.array_equal(out[1], np.float32(0.3) * h[1])
    assert np.array_equal(out[0], h[0])


def test_inject_mean_and_mean_shift_against_numpy():
    H = _mat([9, 9, 9], [1, 2, 3], [3, 4, 5])
    out = O.inject_attack(O.ATTACK_SCALED_MEAN, H, [0], scale=-5.0)
    assert out[0].tolist() == [-10, -15, -20]           # -5 * mean([1,3]), ...
    out = O.inject_attack(O.ATTACK_MEAN_SHIFT, H, [0], kappa=3.0)
    assert out[0].tolist() == [-1, 0, 1]                # mean 2,3,4; population std 1
    rng = np.random.default_rng(8)
    n, f, d = 12, 3, 500
    Hh = (rng.standard_normal((n, d)) * 0.01).astype(np.float32)
    byz = [0, 5, 7]
    good = [i for i in range(n) if i not in byz]
    mean = np.mean(Hh[good].astype(np.float64), axis=0)
    std = np.std(Hh[good].astype(np.float64), axis=0)   # ddof = 0
    out = O.inject_attack(O.ATTACK_SCALED_MEAN, Hh, byz, scale=-5.0)
    for i in byz:
        assert np.allclose(out[i], -5 * mean, rtol=1e-6, atol=0)
    out = O.inject_attack(O.ATTACK_MEAN_SHIFT, Hh, byz, kappa=3.0)
    for i in byz:
        assert np.allclose(out[i], mean - 3 * std, rtol=1e-6, atol=0)
    for i in good:
        assert np.array_equal(out[i], Hh[i])
    # identical honest rows: std is exactly zero
    same = np.tile(Hh[1], (n, 1))
    out = O.inject_attack(O.ATTACK_MEAN_SHIFT, same, [0], kappa=3.0)
    assert np.array_equal(out[0], Hh[1])


def test_inject_sparse_noise():
    H = _mat([1, 1, 1, 1], [2, 2, 2, 2])
    z = _mat([5, 6, 7, 8])
    u = _mat([0.05, 0.1, 0.5, 0.0999])
    out = O.inject_attack(O.ATTACK_SPARSE_NOISE, H, [1], sigma=2.0, prob=0.1, noise=z, uniform=u)
    assert out.tolist() == [[1, 1, 1, 1], [10, 0, 0, 16]]
    rng = np.random.default_rng(6)
    d = 200000
    Hh = rng.standard_normal((2, d)).astype(np.float32)
    out = O.inject_attack(O.ATTACK_SPARSE_NOISE, Hh, [0], sigma=1.0, prob=0.1,
                          noise=rng.standard_normal((1, d)).astype(np.float32),
                          uniform=rng.random((1, d)).astype(np.float32))
    frac = np.count_nonzero(out[0]) / d
    assert abs(frac - 0.1) < 0.005


def test_inject_under_brace_sign_flip_equivalence():
    """A Byzantine client sending -10x its honest update is, after Phase I, a
    plain sign flip (Byzantine clients quantize like everyone else)."""
    rng = np.random.default_rng(10)
    H = rng.standard_normal((8, 256)).astype(np.float32)
    a = O.inject_attack(O.ATTACK_SCALE_OWN, H, [0], scale=-10.0)
    b = H.copy()
    b[0] = -H[0]
    assert np.array_equal(O.gar_direct(a, 0), O.gar_direct(b, 0))


# ---------------------------------------------------------------- the other sign rules of Section 5.2
@pytest.mark.parametrize("n", [2, 3, 4, 5])
def test_majority_sign_and_abs_consensus_brute_force(n):
    """All 3^n patterns; expected values from counting digits with Python integers:
    majority sign = +1 iff positives outnumber negatives (tie -> -1);
    abs consensus = +1 iff |positives - negatives| > lambda."""
    patterns = list(itertools.product([0, 1, 2], repeat=n))
    d = len(patterns)
    U = np.zeros((n, d), dtype=np.float32)
    for k, pat in enumerate(patterns):
        for i, t in enumerate(pat):
            U[i, k] = (t - 1) * (0.25 + i)
    margin = [sum(1 for t in p if t == 2) - sum(1 for t in p if t == 0) for p in patterns]
    for G in (1, 4, 128):
        tr = O.ring_round(U, rule=O.RULE_MAJORITY_SIGN, lam=3.0, granule=G, keep_states=False)   # lambda is ignored
        assert tr.outputs[0].tolist() == [1 if m > 0 else -1 for m in margin]
        assert (tr.outputs == tr.outputs[0]).all()
        for lam in range(-2, n + 1):
            tr = O.ring_round(U, rule=O.RULE_ABS_CONSENSUS, lam=lam, granule=G, keep_states=False)
            assert tr.outputs[0].tolist() == [1 if abs(m) > lam else -1 for m in margin]
            assert (tr.outputs == tr.outputs[0]).all()
            assert np.array_equal(O.gar_direct(U, lam, rule=O.RULE_ABS_CONSENSUS), tr.outputs[0])
    assert np.array_equal(O.gar_direct(U, 0, rule=O.RULE_MAJORITY_SIGN), O.gar_direct(U, 0))   # == Eq. (1), lambda 0


def test_abs_consensus_is_symmetric_and_is_the_union_of_both_directions():
    rng = np.random.default_rng(21)
    n, d = 11, 4000
    U = rng.standard_normal((n, d)).astype(np.float32)
    U[rng.random((n, d)) < 0.2] = 0
    for lam in (0, 2, 4.5, 10):
        a = O.gar_direct(U, lam, rule=O.RULE_ABS_CONSENSUS)
        assert np.array_equal(a, O.gar_direct(-U, lam, rule=O.RULE_ABS_CONSENSUS))
        both = np.maximum(O.gar_direct(U, lam), O.gar_direct(-U, lam))
        assert np.array_equal(a, both)
    assert (O.gar_direct(U, -1, rule=O.RULE_ABS_CONSENSUS) == 1).all()
    assert (O.gar_direct(U, n, rule=O.RULE_ABS_CONSENSUS) == -1).all()
    # sent bits equal BRACE's (Section 5.2: same communication cost)
    V = rng.standard_normal((4, 8)).astype(np.float32)
    for rule in (O.RULE_MAJORITY_SIGN, O.RULE_ABS_CONSENSUS):
        tr = O.ring_round(V, rule=rule, lam=1, granule=1, keep_states=False)
        assert O.sent_bits(tr, 8, rule).tolist() == [54] * 4      # Table 1 row n=4, d=8, m=8


# ---------------------------------------------------------------- the model update after a round
def test_apply_update_closed_forms(golden):
    g = golden("rar_worked_example.txt")
    U = _mat(g["g1"], g["g2"], g["g3"])
    tr = O.ring_round(U, rule=O.RULE_SUM, granule=1)
    w0 = np.zeros((3, 3), dtype=np.float32)
    # Section 2.2: w - (eta / n) * sum; with eta = n = 3 and w = 0 every client lands on -sum
    w1 = O.apply_update(w0, tr.outputs, 3.0, O.RULE_SUM)
    assert w1.tolist() == [[-22, -1, -5]] * 3
    trm = O.ring_round(U, rule=O.RULE_SUM, granule=1, mean=True)
    assert np.allclose(O.apply_update(w0, trm.outputs, 3.0, O.RULE_SUM, mean=True), np.array([[-22, -1, -5]] * 3),
                       rtol=1e-6)
    # Appendix A: BRACE moves every coordinate by exactly eta, against the aggregate's sign, no 1/n
    rng = np.random.default_rng(12)
    n, d, eta = 6, 500, 0.125
    V = rng.standard_normal((n, d)).astype(np.float32)
    w = rng.standard_normal((n, d)).astype(np.float32)
    tb = O.ring_round(V, lam=1, granule=16, keep_states=False)
    w2 = O.apply_update(w, tb.outputs, eta, O.RULE_SIGN_CONSENSUS)
    assert np.array_equal(np.abs(w2 - w.astype(np.float64)), np.full((n, d), eta))
    assert np.array_equal(np.sign(w.astype(np.float64) - w2), tb.outputs.astype(np.float64))
    # identical starting points stay identical across clients (all clients hold the same aggregate)
    same = np.tile(w[0], (n, 1))
    w3 = O.apply_update(same, tb.outputs, eta, O.RULE_SIGN_CONSENSUS)
    assert (w3 == w3[0]).all()


# ---------------------------------------------------------------- coordinate-wise median / trimmed mean (Section 5.1)
def test_coordinate_median_and_trimmed_mean_against_library_routines():
    from scipy import stats
    rng = np.random.default_rng(33)
    for n in (3, 4, 8, 9, 20, 100):
        U = rng.standard_normal((n, 300)).astype(np.float32)
        U[rng.random((n, 300)) < 0.1] = 0.0
        med = O.coordinate_median(U)
        assert np.allclose(med, np.median(U.astype(np.float64), axis=0), rtol=1e-7, atol=0)
        for trim in sorted({0, 1, n // 5, (n - 1) // 2}):
            if 2 * trim >= n:
                continue
            tm = O.coordinate_trimmed_mean(U, trim)
            # scipy cuts int(proportion * n) values from each end of the sorted column
            ref = stats.trim_mean(U.astype(np.float64), (trim + 0.5) / n, axis=0) if trim else U.astype(np.float64).mean(0)
            assert np.allclose(tm, ref, rtol=1e-6, atol=1e-9), (n, trim)
        if n % 2:
            assert np.array_equal(O.coordinate_trimmed_mean(U, (n - 1) // 2), med)   # all but the middle trimmed
    # hand-checked columns
    U = _mat([5, 1, 9, -2], [3, 7, 9, 4], [4, 100, 9, 0], [-6, 2, 9, 8])
    assert O.coordinate_median(U).tolist() == [3.5, 4.5, 9.0, 2.0]
    assert O.coordinate_trimmed_mean(U, 1).tolist() == [3.5, 4.5, 9.0, 2.0]
    assert O.coordinate_trimmed_mean(U, 0).tolist() == [1.5, 27.5, 9.0, 2.5]
    assert O.coordinate_median(U[:3]).tolist() == [4.0, 7.0, 9.0, 0.0]
    # order of the clients does not matter; one outlier cannot move the median past its neighbours
    perm = rng.permutation(4)
    assert np.array_equal(O.coordinate_median(U[perm]), O.coordinate_median(U))
    V = U.copy()
    V[2, 1] = 1e30
    assert O.coordinate_median(V).tolist() == O.coordinate_median(U).tolist()
    with pytest.raises(ValueError):
        O.coordinate_trimmed_mean(U, 2)


# ---------------------------------------------------------------- random draws of the attacks
def _kat_rows():
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")
    rows, numer = [], None
    with open(path) as fh:
        for line in fh:
            line = line.strip()
            if line.startswith("# uniform_numerators:"):
                numer = [int(v) for v in line.split(":")[1].split()]
            if not line or line.startswith("#"):
                continue
            rows.append([int(v, 16) for v in line.split()])
    return rows, numer


def test_philox_known_answer_vectors():
    """The published known-answer vectors of Philox4x32-10."""
    rows, _ = _kat_rows()
    assert len(rows) == 3
    for r in rows:
        got = O.philox4x32_10([np.array([c], dtype=np.uint32) for c in r[0:4]], r[4:6])
        assert [int(g[0]) for g in got] == r[6:10]
    # vectorised over counters: same answers in one call
    ctr = [np.array([r[i] for r in rows], dtype=np.uint32) for i in range(4)]
    key = [np.array([r[4 + i] for r in rows], dtype=np.uint32) for i in range(2)]
    got = O.philox4x32_10(ctr, key)
    for t, r in enumerate(rows):
        assert [int(g[t]) for g in got] == r[6:10]


def test_draw_layout_counter_and_key_fields():
    """Where seed, round, client, stream and coordinate go: block q = k div 4 -> counter
    (q lo, q hi, client, round * 256 + stream), key (seed lo, seed hi); word k mod 4.
    Philox itself is pinned by the known-answer vectors, so the field layout is checked
    through it; the all-zero case is the first published vector."""
    rows, numer = _kat_rows()
    assert O.draw_words(0, 0, 0, O.STREAM_UNIFORM, 4).tolist() == rows[0][6:10]
    u = O.draw_uniform(0, 0, 0, 4)
    assert [int(round(float(x) * 2 ** 24)) for x in u] == numer
    seed, rnd, client, stream, d = 0x299F31D0A4093822, 0x037073, 0x13198A2E, 0x44, 27
    w = O.draw_words(seed, rnd, client, stream, d)
    assert w.dtype == np.uint32 and w.shape == (d,)
    for k in (0, 1, 5, 11, 24, 26):
        q = k // 4
        ref = O.philox4x32_10([np.array([v], dtype=np.uint32) for v in (q, 0, client, rnd * 256 + stream)],
                              [seed & 0xFFFFFFFF, seed >> 32])
        assert int(w[k]) == int(ref[k % 4][0])
    # the third published vector has exactly this key, client word and round/stream word
    assert rnd * 256 + stream == rows[2][3] and client == rows[2][2]
    assert [seed & 0xFFFFFFFF, seed >> 32] == rows[2][4:6]
    # every field matters, and a prefix does not depend on d
    base = O.draw_words(5, 1, 2, 0, 64)
    for other in (O.draw_words(6, 1, 2, 0, 64), O.draw_words(5 + (1 << 32), 1, 2, 0, 64), O.draw_words(5, 2, 2, 0, 64),
                  O.draw_words(5, 1, 3, 0, 64), O.draw_words(5, 1, 2, 1, 64)):
        assert (other != base).mean() > 0.9
    assert np.array_equal(O.draw_words(5, 1, 2, 0, 13), base[:13])
    assert np.array_equal(O.draw_words(5, 1, 2, 0, 21, start=40), base[40:61])         # a window of the same row
    assert np.array_equal(O.draw_normal(5, 1, 2, 9, start=8), O.draw_normal(5, 1, 2, 17)[8:])
    assert np.array_equal(O.draw_uniform(5, 1, 2, 9, start=8), O.draw_uniform(5, 1, 2, 17)[8:])
    big = (1 << 34) + 8                                                                # block index needs its high word
    hi = O.draw_words(5, 1, 2, 0, 4, start=big)
    ref = O.philox4x32_10([np.array([v], dtype=np.uint32) for v in ((big // 4) & 0xFFFFFFFF, (big // 4) >> 32, 2, 256)], [5, 0])
    assert [int(x) for x in hi] == [int(r[0]) for r in ref]
    for bad in ((-1, 0, 0, 0), (1 << 64, 0, 0, 0), (0, 1 << 24, 0, 0), (0, 0, 0, 256)):
        with pytest.raises(ValueError):
            O.draw_words(bad[0], bad[1], bad[2], bad[3], 4)


def test_uniform_and_normal_draws_have_their_distributions():
    """Uniforms are multiples of 2^-24 in [0, 1); normals pass a Kolmogorov-Smirnov test against
    scipy's normal distribution; different clients / rounds are uncorrelated."""
    from scipy import stats
    d = 400_001
    u = O.draw_uniform(2501017392, 3, 7, d)
    assert u.dtype == np.float32 and u.min() >= 0.0 and u.max() < 1.0
    assert np.array_equal(u.astype(np.float64) * 2 ** 24, np.rint(u.astype(np.float64) * 2 ** 24))
    assert stats.kstest(u.astype(np.float64), "uniform").pvalue > 1e-3
    z = O.draw_normal(2501017392, 3, 7, d)
    assert z.dtype == np.float32 and np.isfinite(z).all()
    assert stats.kstest(z.astype(np.float64), "norm").pvalue > 1e-3
    assert abs(float(z.mean())) < 0.01 and abs(float(z.var()) - 1.0) < 0.01
    assert abs(np.corrcoef(z[0::2][: d // 2], z[1::2][: d // 2])[0, 1]) < 0.01       # the two outputs of a pair
    z2 = O.draw_normal(2501017392, 3, 8, d)
    z3 = O.draw_normal(2501017392, 4, 7, d)
    assert abs(np.corrcoef(z, z2)[0, 1]) < 0.01 and abs(np.corrcoef(z, z3)[0, 1]) < 0.01
    assert abs(np.corrcoef(z, u)[0, 1]) < 0.01


def test_normal_draws_invert_to_their_words():
    """Box-Muller run backwards: from a pair (z0, z1), exp(-(z0^2 + z1^2) / 2) is u1 and the angle
    atan2(z1, z0) / (2 pi) is u2 -- both must be the 24-bit fractions of the pair's two words.
    A swapped cos / sin, a wrong radius or the wrong words fail this."""
    seed, rnd, client, d = 99, 5, 11, 20_000
    z = O.draw_normal(seed, rnd, client, d).astype(np.float64).reshape(-1, 2)
    w = O.draw_words(seed, rnd, client, O.STREAM_NORMAL, d).reshape(-1, 2)
    u1 = ((w[:, 0] >> 8).astype(np.float64) + 1.0) / 2 ** 24
    u2 = (w[:, 1] >> 8).astype(np.float64) / 2 ** 24
    r2 = (z * z).sum(1)
    assert np.allclose(np.exp(-0.5 * r2), u1, rtol=2e-6, atol=0)
    ang = np.mod(np.arctan2(z[:, 1], z[:, 0]) / (2 * np.pi), 1.0)
    err = np.abs(ang - u2)
    err = np.minimum(err, 1.0 - err)
    ok = r2 > 1e-6                                     # a zero radius has no angle
    assert err[ok].max() < 1e-6
    # odd d: the last coordinate is the first output of its pair
    assert np.array_equal(O.draw_normal(seed, rnd, client, 7), O.draw_normal(seed, rnd, client, 8)[:7])


def test_cospi_sinpi_exact_at_quarter_turns():
    x = np.array([0.0, 0.25, 0.5, 0.75, 1.0, 1.25, 1.5, 1.75, 1.0 / 3.0])
    c, s = O._cospi_sinpi(x)
    h = math.sqrt(0.5)
    assert np.allclose(c[:8], [1, h, 0, -h, -1, -h, 0, h], rtol=1e-15, atol=0)
    assert np.allclose(s[:8], [0, h, 1, h, 0, -h, -1, -h], rtol=1e-15, atol=0)
    assert c[2] == 0.0 and c[6] == 0.0 and s[0] == 0.0 and s[4] == 0.0       # exact zeros, not 6e-17
    assert abs(c[8] - 0.5) < 1e-15


def test_attack_draws_shapes_and_rows():
    noise, unif = O.attack_draws(O.ATTACK_SPARSE_NOISE, 7, 2, [5, 1], 33)
    assert noise.shape == (2, 33) and unif.shape == (2, 33)
    assert np.array_equal(noise[1], O.draw_normal(7, 2, 1, 33)) and np.array_equal(unif[0], O.draw_uniform(7, 2, 5, 33))
    noise, unif = O.attack_draws(O.ATTACK_GAUSSIAN, 7, 2, [0], 8)
    assert unif is None and noise.shape == (1, 8)
    assert O.attack_draws(O.ATTACK_MEAN_SHIFT, 7, 2, [0], 8) == (None, None)
