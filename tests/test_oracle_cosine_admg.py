"""Pins of the oracle's cosine similarity (Section 3.2, summand of C_l) and of ADMG (Algorithm 1)."""
import itertools
import math
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "admg_sets.txt")


# ------------------------------------------------------------------ cosine: closed forms
def test_cosine_of_a_vector_with_itself_is_one():
    x = np.linspace(-3, 5, 257).astype(np.float32)
    assert oracle.cosine(x, x) == pytest.approx(1.0, abs=1e-15)


def test_cosine_scale_invariance_and_sign():
    rng = np.random.default_rng(0)
    x = rng.standard_normal(300).astype(np.float32)
    y = rng.standard_normal(300).astype(np.float32)
    c = oracle.cosine(x, y)
    assert oracle.cosine(4 * x, y) == pytest.approx(c, abs=1e-12)
    assert oracle.cosine(x, 0.25 * y) == pytest.approx(c, abs=1e-12)
    assert oracle.cosine(x, 8 * x) == pytest.approx(1.0, abs=1e-15)
    assert oracle.cosine(x, -x) == pytest.approx(-1.0, abs=1e-15)
    assert oracle.cosine(y, x) == pytest.approx(c, abs=1e-15)  # symmetric
    assert -1.0 <= c <= 1.0


def test_cosine_orthogonal_is_zero_and_known_angles():
    e1 = np.array([1, 0, 0, 0], np.float32)
    e2 = np.array([0, 2, 0, 0], np.float32)
    assert oracle.cosine(e1, e2) == 0.0
    # 3-4-5 triangle: cos between (3,4) and (3,0) is 3/5
    assert oracle.cosine(np.array([3, 4], np.float32), np.array([3, 0], np.float32)) == pytest.approx(0.6, abs=1e-15)
    # 45 degrees
    assert oracle.cosine(np.array([1, 1], np.float32), np.array([1, 0], np.float32)) == pytest.approx(
        1 / math.sqrt(2), abs=1e-15)


@pytest.mark.parametrize("r", [0.0, 0.125, 0.5, 1.0, 4.0])
def test_cosine_residual_with_orthogonal_update(r):
    # y = x + o with o orthogonal to x and ||o|| = r ||x||  =>  cos = 1/sqrt(1+r^2)
    x = np.zeros(64, np.float32)
    o = np.zeros(64, np.float32)
    x[:32] = 2.0
    o[32:] = 2.0 * r
    assert oracle.cosine(x, x + o) == pytest.approx(1 / math.sqrt(1 + r * r), abs=1e-12)


def test_cosine_matches_numpy_float64():
    rng = np.random.default_rng(1)
    for n in (1, 7, 256, 4099):
        x = rng.standard_normal(n).astype(np.float32)
        y = (x + 0.3 * rng.standard_normal(n)).astype(np.float32)
        ref = float(np.dot(x.astype(np.float64), y.astype(np.float64)) /
                    (np.linalg.norm(x.astype(np.float64)) * np.linalg.norm(y.astype(np.float64))))
        assert oracle.cosine(x, y) == pytest.approx(ref, abs=1e-12)


def test_cosine_zero_rows_do_not_divide_by_zero():
    z = np.zeros(16, np.float32)
    assert oracle.cosine(z, z) == 0.0
    assert np.isfinite(oracle.cosine(z, np.ones(16, np.float32)))


# ------------------------------------------------------------------ ADMG: hand-derived sets
def _parse_set(s):
    s = s.strip()
    return set() if s == "-" else {int(t) for t in s.split(",")}


def _golden_rows():
    rows = []
    with open(GOLDEN) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            head, hot, ra, rm = [p.strip() for p in line.split("|")]
            L, m, n = (int(t) for t in head.split())
            rows.append((L, m, n, _parse_set(hot), _parse_set(ra), _parse_set(rm)))
    return rows


@pytest.mark.parametrize("L,m,n,hot,want_attn,want_mlp", _golden_rows())
def test_admg_hand_derived_sets(L, m, n, hot, want_attn, want_mlp):
    alpha = 0.985
    C = np.full(L, 0.9, np.float32)
    for l in hot:
        C[l - 1] = 0.99
    ra, rm = oracle.admg(C, alpha, m, n)
    assert {i + 1 for i in np.flatnonzero(ra)} == want_attn
    assert {i + 1 for i in np.flatnonzero(rm)} == want_mlp


def test_admg_counts_for_table2_hyperparameters():
    # Table 2: (alpha, m, n) = (0.985, 3, 2) for the Llama-2-13B models, (0.985, 4, 3) for CodeLlama-13B; L = 40
    C = np.zeros(40, np.float32)
    _, rm = oracle.admg(C, 0.985, 3, 2)
    assert rm.sum() == 12
    _, rm = oracle.admg(C, 0.985, 4, 3)
    assert rm.sum() == 9


def test_admg_threshold_is_inclusive():
    alpha = np.float32(0.985)
    C = np.array([alpha, np.nextafter(alpha, np.float32(0)), np.nextafter(alpha, np.float32(2)), 0.0], np.float32)
    ra, rm = oracle.admg(C, float(alpha), 0, 0, oracle.USE_CS)
    assert ra.tolist() == [1, 0, 1, 0]
    assert rm.sum() == 0


# ------------------------------------------------------------------ ADMG: brute force over all masks, L = 2
def _predicate_holds(mask_attn, mask_mlp, C, alpha, m, n, flags):
    """Does the pair of sets satisfy Algorithm 1's set definitions, checked member by member?"""
    L = len(C)
    n_eff = n if flags & oracle.USE_RULE2 else 0
    for l in range(1, L + 1):
        in_mlp = bool(flags & oracle.USE_RULE1) and m >= 1 and any(l == j * m for j in range(1, L + 1)) and l <= L - n_eff
        in_cs = bool(flags & oracle.USE_CS) and np.float32(C[l - 1]) >= np.float32(alpha) and l <= L - n_eff
        if bool(mask_mlp[l - 1]) != in_mlp:
            return False
        if bool(mask_attn[l - 1]) != (in_cs or in_mlp):
            return False
    return True


@pytest.mark.parametrize("flags", [oracle.USE_CS, oracle.USE_CS | oracle.USE_RULE2,
                                   oracle.USE_RULE1 | oracle.USE_RULE2, oracle.ADMG_ALL])
def test_admg_brute_force_two_layers(flags):
    alpha = 0.5
    grid = [0.0, 0.5, 0.9]
    for c1, c2 in itertools.product(grid, grid):
        C = np.array([c1, c2], np.float32)
        for m in (1, 2):
            for n in (0, 1, 2):
                got_a, got_m = oracle.admg(C, alpha, m, n, flags)
                sat = [(a, b) for a in itertools.product((0, 1), repeat=2) for b in itertools.product((0, 1), repeat=2)
                       if _predicate_holds(a, b, C, alpha, m, n, flags)]
                assert len(sat) == 1, (C, m, n, sat)
                assert sat[0] == (tuple(got_a.tolist()), tuple(got_m.tolist())), (C, m, n, flags)


def test_admg_structural_invariants():
    rng = np.random.default_rng(3)
    for _ in range(200):
        L = int(rng.integers(1, 48))
        C = rng.uniform(0.5, 1.0, L).astype(np.float32)
        m = int(rng.integers(0, 6))
        n = int(rng.integers(0, 6))
        for flags in range(8):
            ra, rm = oracle.admg(C, 0.9, m, n, flags)
            assert np.all(ra >= rm)  # remove_MLP is a subset of remove_ATTN
            if flags & oracle.USE_RULE2 and n > 0:
                assert ra[max(0, L - n):].sum() == 0 and rm[max(0, L - n):].sum() == 0  # last n layers are kept
            if not flags & oracle.USE_RULE1:
                assert rm.sum() == 0
            if not flags & (oracle.USE_RULE1 | oracle.USE_CS):
                assert ra.sum() == 0


def test_admg_table5_subsets_nest():
    # Table 5: CS only; CS + rule 2; rules 1 & 2; all three
    C = np.array([0.99, 0.5, 0.99, 0.5, 0.99, 0.99], np.float32)
    cs, _ = oracle.admg(C, 0.985, 3, 2, oracle.USE_CS)
    cs2, _ = oracle.admg(C, 0.985, 3, 2, oracle.USE_CS | oracle.USE_RULE2)
    r12a, r12m = oracle.admg(C, 0.985, 3, 2, oracle.USE_RULE1 | oracle.USE_RULE2)
    alla, allm = oracle.admg(C, 0.985, 3, 2, oracle.ADMG_ALL)
    assert cs.tolist() == [1, 0, 1, 0, 1, 1]
    assert cs2.tolist() == [1, 0, 1, 0, 0, 0]
    assert r12a.tolist() == [0, 0, 1, 0, 0, 0] and r12m.tolist() == [0, 0, 1, 0, 0, 0]
    assert alla.tolist() == [1, 0, 1, 0, 0, 0] and allm.tolist() == [0, 0, 1, 0, 0, 0]
    assert np.all(alla == (cs2 | r12a))
