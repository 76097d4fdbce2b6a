"""The archive of kernel variants (MAP-Elites grid, transition ring buffer, gradient estimates;
paper Sections 3.2 and 3.3): the plain Python reference against values worked out by hand from the
paper's formulas, then the C++ implementation in the kf library against the reference on seeded
random histories.  No GPU involved."""
import math

import numpy as np
import pytest

from oracle import archive_ref as ref
from paper_2603_12440_b200 import archive as kfa


# ------------------------------------------------------------------------------- reference vs the paper
def test_fitness_function_values():
    # Section 3.2, "Fitness Function": correctness first, then speed-up normalised by the target (default 2x)
    assert ref.fitness(False, False, 5.0) == 0.0
    assert ref.fitness(True, False, 5.0) == 0.1
    assert ref.fitness(True, True, 0.0) == 0.5
    assert ref.fitness(True, True, 1.0) == 0.75
    assert ref.fitness(True, True, 2.0) == 1.0
    assert ref.fitness(True, True, 7.0) == 1.0                     # capped
    assert ref.fitness(True, True, 1.5, target=3.0) == 0.75


def test_insertion_keeps_the_best_per_cell_and_classifies_outcomes():
    a = ref.Archive(capacity=8)
    assert a.insert((1, 2, 3), 0.6, 10) == ref.IMPROVEMENT         # empty cell
    assert a.insert((1, 2, 3), 0.6, 11) == ref.NEUTRAL             # not better: discarded
    assert a.cells[(1, 2, 3)] == (0.6, 10)
    assert a.insert((1, 2, 3), 0.7, 12) == ref.IMPROVEMENT
    assert a.cells[(1, 2, 3)] == (0.7, 12)
    # with a parent: improvement = archive update (even below the parent's fitness), else by the sign of delta f
    assert a.insert((0, 0, 0), 0.55, 13, parent=(1, 2, 3), parent_fit=0.7, iteration=1) == ref.IMPROVEMENT   # new cell
    assert a.insert((1, 2, 3), 0.65, 14, parent=(1, 2, 3), parent_fit=0.7, iteration=2) == ref.REGRESSION
    assert a.insert((1, 2, 3), 0.7, 15, parent=(0, 0, 0), parent_fit=0.55, iteration=3) == ref.NEUTRAL
    assert [t[3] for t in a.ring] == [ref.IMPROVEMENT, ref.REGRESSION, ref.NEUTRAL]
    assert [round(t[2], 12) for t in a.ring] == [-0.15, -0.05, 0.15]


def _two_transitions():
    a = ref.Archive(capacity=8, half_life=10.0)
    a.insert((1, 1, 1), 0.6, 1)
    a.insert((2, 1, 1), 0.8, 2, parent=(1, 1, 1), parent_fit=0.6, iteration=20)     # +0.2, new cell: improvement
    a.insert((0, 1, 2), 0.5, 3, parent=(1, 1, 1), parent_fit=0.6, iteration=10)     # -0.1, new cell: improvement
    a.insert((0, 1, 2), 0.4, 4, parent=(1, 1, 1), parent_fit=0.6, iteration=20)     # -0.2, no update: regression
    return a


def test_fitness_gradient_eq1_by_hand():
    a = _two_transitions()
    # from (1,1,1) at now = 20: weights 1, 2^-1, 1
    #   d0: (+0.2 * +1 * 1  +  -0.1 * -1 * 0.5  +  -0.2 * -1 * 1) / 3 = 0.45 / 3
    #   d1: no movement
    #   d2: (0 + -0.1 * +1 * 0.5 + -0.2 * +1 * 1) / 3 = -0.25 / 3
    g = a.grad_fitness((1, 1, 1), now=20)
    assert g == pytest.approx([0.15, 0.0, -0.25 / 3], abs=1e-15)
    assert a.grad_fitness((3, 3, 3), now=20) == [0.0, 0.0, 0.0]    # no transitions from there


def test_improvement_rate_gradient_eq2_by_hand():
    a = _two_transitions()
    # d0: up {t1: improvement} -> 1; down {t2: improvement, t3: regression} -> 1/2;  R0 = 1/2
    # d2: up {t2, t3} -> 1/2; down {} -> 0;  R2 = 1/2
    assert a.grad_rate((1, 1, 1)) == pytest.approx([0.5, 0.0, 0.5], abs=1e-15)


def test_exploration_gradient_eq3_by_hand():
    a = ref.Archive(capacity=4, low_quality=0.5)
    for i in range(4):
        for j in range(4):
            for k in range(4):
                if (i, j, k) != (3, 1, 1):
                    a.insert((i, j, k), 0.9, 0)
    # one empty cell at L1 distance 2 along d0:  (0.9 - 0) / 2 * (2, 0, 0) / 2, |E| = 1
    assert a.grad_explore((1, 1, 1)) == pytest.approx([0.45, 0.0, 0.0], abs=1e-15)
    # a low-quality cell (below half the best) joins E with its own fitness; a mediocre one does not
    a.cells[(1, 1, 3)] = (0.4, 0)
    a.cells[(1, 3, 1)] = (0.5, 0)
    e = a.grad_explore((1, 1, 1))
    assert e == pytest.approx([0.45 / 2, 0.0, (0.9 - 0.4) / 2 * 2 / 2 / 2], abs=1e-15)
    # mirror symmetry of the grid: the lone elite in one corner is pushed along (+,+,+), in the other along (-,-,-)
    lone = ref.Archive(capacity=1)
    lone.insert((0, 0, 0), 1.0, 0)
    far = ref.Archive(capacity=1)
    far.insert((3, 3, 3), 1.0, 0)
    g0, g3 = lone.grad_explore((0, 0, 0)), far.grad_explore((3, 3, 3))
    assert g0[0] > 0 and g0[1] == pytest.approx(g0[0], rel=1e-14) and g0[2] == pytest.approx(g0[0], rel=1e-14)
    assert g3 == pytest.approx([-v for v in g0], abs=1e-15)


def test_combined_gradient_weights_and_sampling():
    a = _two_transitions()
    g, gf, gr, ge = a.gradient((1, 1, 1), now=20)
    assert g == pytest.approx([0.4 * gf[d] + 0.4 * gr[d] + 0.2 * ge[d] for d in range(3)], abs=1e-15)
    w = a.sampling_weights(now=20)
    assert set(w) == set(a.cells) and sum(w.values()) == pytest.approx(1.0, abs=1e-15)
    norm = {c: math.sqrt(sum(v * v for v in a.gradient(c, 20)[0])) for c in a.cells}
    c1, c2 = (1, 1, 1), (2, 1, 1)
    assert w[c1] / w[c2] == pytest.approx(math.exp(norm[c1] - norm[c2]), rel=1e-13)


def test_ring_buffer_drops_the_oldest():
    a = ref.Archive(capacity=3)
    a.insert((0, 0, 0), 0.5, 0)
    for it in range(5):
        a.insert((1, 0, 0), 0.5 + 0.01 * it, it, parent=(0, 0, 0), parent_fit=0.5, iteration=it)
    assert [t[4] for t in a.ring] == [2, 3, 4]


# ------------------------------------------------------------------------------- C++ against the reference
@pytest.fixture(scope="module")
def lib_ok():
    from paper_2603_12440_b200 import binding
    binding.lib()
    return True


def test_cpp_fitness_matches(lib_ok):
    for comp, corr, s, t in [(0, 0, 3.0, 2.0), (1, 0, 3.0, 2.0), (1, 1, 0.0, 2.0), (1, 1, 1.3, 2.0), (1, 1, 9.0, 2.0), (1, 1, 1.0, 3.0)]:
        assert kfa.fitness(comp, corr, s, t) == ref.fitness(bool(comp), bool(corr), s, t)


@pytest.mark.parametrize("seed,capacity,steps", [(1, 16, 60), (2, 64, 400), (3, 500, 400)])
def test_cpp_archive_matches_reference_on_random_histories(lib_ok, seed, capacity, steps):
    r = np.random.Generator(np.random.PCG64(seed))
    a = kfa.Archive(capacity=capacity, half_life=25.0, low_quality=0.6)
    b = ref.Archive(capacity=capacity, half_life=25.0, low_quality=0.6)
    for it in range(steps):
        occupied = sorted(b.cells)
        child = tuple(int(v) for v in r.integers(0, 4, 3))
        fit = float(np.round(r.uniform(0.0, 1.0), 3))
        if occupied and r.uniform() < 0.85:
            parent = occupied[int(r.integers(0, len(occupied)))]
            if r.uniform() < 0.5:                                   # most children stay near their parent
                child = tuple(int(np.clip(parent[d] + r.integers(-1, 2), 0, 3)) for d in range(3))
            pf = b.cells[parent][0]
            assert a.insert(child, fit, it, parent, pf, it) == b.insert(child, fit, it, parent, pf, it)
        else:
            assert a.insert(child, fit, it) == b.insert(child, fit, it)
    assert a.transitions() == len(b.ring) == min(capacity, a.transitions())
    for i in range(4):
        for j in range(4):
            for k in range(4):
                got = a.cell((i, j, k))
                assert got == b.cells.get((i, j, k))
                g, gf, gr, ge = a.gradient((i, j, k), steps)
                rg, rf, rr, re_ = b.gradient((i, j, k), steps)
                for x, y in ((g, rg), (gf, rf), (gr, rr), (ge, re_)):
                    assert x == pytest.approx(y, rel=1e-12, abs=1e-15)
    wa, wb = a.sampling_weights(steps), b.sampling_weights(steps)
    assert set(wa) == set(wb)
    for c in wb:
        assert wa[c] == pytest.approx(wb[c], rel=1e-12)
    a.close()


def test_cpp_rejects_bad_arguments(lib_ok):
    with pytest.raises(ValueError):
        kfa.Archive(capacity=0)
    with pytest.raises(ValueError):
        kfa.Archive(capacity=4, half_life=0.0)
    a = kfa.Archive(capacity=4)
    with pytest.raises(ValueError):
        a.insert((0, 4, 0), 0.5)
    with pytest.raises(ValueError):
        a.insert((0, 0, 0), 0.5, parent=(-1, 0, 0))
    assert a.cell((0, 0, 0)) is None and a.transitions() == 0      # nothing changed
    assert a.sampling_weights(0) == {}
