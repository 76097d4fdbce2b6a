"""Plain Python reference of the search-side bookkeeping the paper describes around its kernels:
the MAP-Elites grid over (d_mem, d_algo, d_sync), the fitness function, the ring buffer of
parent -> child transitions and the three gradient estimates.  TEST INFRASTRUCTURE ONLY: the
product implementation is the C++ in the kf library; nothing outside tests/ may import this file.

What follows the paper, by passage:
  * grid, insertion rule                     Section 3.2, "MAP-Elites Algorithm": a child replaces the incumbent of
                                             its cell if it improves on it, or if the cell is empty
  * descriptors d in {0,1,2,3}^3, 64 cells   Section 3.2, "Kernel-Specific Behavioral Descriptors"
  * fitness f(k)                             Section 3.2, "Fitness Function"
  * transition record and outcomes           Section 3.3, "Transition Tracking and gradient estimation"
  * gradient estimates                       Section 3.3, Eq. 1 (fitness), Eq. 2 (improvement rate), Eq. 3 (exploration),
                                             combined with weights (0.4, 0.4, 0.2)
  * selection weights exp(|gradient|)        Section 3.3, "Gradient-to-Prompt Translation" (cells with strong
                                             gradient magnitudes are sampled more often)

Where the paper is silent this file takes the readings listed in the design notes: time decay
w(t) = 2^(-(now - iteration_t) / half_life); the set E of Eq. 3 = empty cells (fitness 0) plus occupied
cells whose fitness is below `low_quality` times the best fitness in the archive, the cell itself
excluded; Eq. 3's proportionality constant = 1 / |E|; conditional probabilities over an empty set = 0.
Everything is float64 and written as the formulas read, one loop per sum.
"""
import math

BINS = 4
DIMS = 3
ALPHA, BETA, GAMMA = 0.4, 0.4, 0.2
IMPROVEMENT, NEUTRAL, REGRESSION = 1, 0, -1


def fitness(compiled: bool, correct: bool, speedup: float, target: float = 2.0) -> float:
    if not compiled:
        return 0.0
    if not correct:
        return 0.1
    return 0.5 + 0.5 * min(1.0, speedup / target)


def sign(v):
    return (v > 0) - (v < 0)


class Archive:
    def __init__(self, capacity: int, half_life: float = 50.0, low_quality: float = 0.5):
        self.cells = {}                 # coords -> (fitness, ident)
        self.ring = []                  # at most `capacity` transitions, oldest first
        self.capacity = capacity
        self.half_life = half_life
        self.low_quality = low_quality

    # ---- archive -----------------------------------------------------------------------------
    def insert(self, coords, fit, ident, parent=None, parent_fit=0.0, iteration=0):
        """Offer a child; returns its outcome.  With a parent the transition is recorded."""
        coords = tuple(coords)
        old = self.cells.get(coords)
        became_elite = old is None or fit > old[0]
        if became_elite:
            self.cells[coords] = (fit, ident)
        if parent is None:
            return IMPROVEMENT if became_elite else NEUTRAL
        df = fit - parent_fit
        outcome = IMPROVEMENT if became_elite else (REGRESSION if df < 0 else NEUTRAL)
        self.ring.append((tuple(parent), coords, df, outcome, iteration))
        if len(self.ring) > self.capacity:
            self.ring.pop(0)
        return outcome

    # ---- gradients ---------------------------------------------------------------------------
    def grad_fitness(self, b, now):
        T = [t for t in self.ring if t[0] == tuple(b)]
        g = [0.0] * DIMS
        if not T:
            return g
        for d in range(DIMS):
            acc = 0.0
            for (bp, bc, df, _, it) in T:
                acc += df * sign(bc[d] - bp[d]) * 2.0 ** (-(now - it) / self.half_life)
            g[d] = acc / len(T)
        return g

    def grad_rate(self, b):
        T = [t for t in self.ring if t[0] == tuple(b)]
        g = [0.0] * DIMS
        for d in range(DIMS):
            up = [t for t in T if t[1][d] - t[0][d] > 0]
            dn = [t for t in T if t[1][d] - t[0][d] < 0]
            p_up = sum(1 for t in up if t[3] == IMPROVEMENT) / len(up) if up else 0.0
            p_dn = sum(1 for t in dn if t[3] == IMPROVEMENT) / len(dn) if dn else 0.0
            g[d] = p_up - p_dn
        return g

    def grad_explore(self, b):
        b = tuple(b)
        fmax = max((f for f, _ in self.cells.values()), default=0.0)
        E = []
        for i in range(BINS):
            for j in range(BINS):
                for k in range(BINS):
                    c = (i, j, k)
                    if c == b:
                        continue
                    if c not in self.cells:
                        E.append((c, 0.0))
                    elif self.cells[c][0] < self.low_quality * fmax:
                        E.append((c, self.cells[c][0]))
        g = [0.0] * DIMS
        if not E:
            return g
        for (c, fc) in E:
            dist = sum(abs(c[d] - b[d]) for d in range(DIMS))
            for d in range(DIMS):
                g[d] += (fmax - fc) / dist * (c[d] - b[d]) / dist
        return [v / len(E) for v in g]

    def gradient(self, b, now):
        gf, gr, ge = self.grad_fitness(b, now), self.grad_rate(b), self.grad_explore(b)
        return [ALPHA * gf[d] + BETA * gr[d] + GAMMA * ge[d] for d in range(DIMS)], gf, gr, ge

    def sampling_weights(self, now):
        """Occupied cells -> probability, proportional to exp(|combined gradient|_2)."""
        w = {}
        for c in self.cells:
            g = self.gradient(c, now)[0]
            w[c] = math.exp(math.sqrt(sum(v * v for v in g)))
        s = sum(w.values())
        return {c: v / s for c, v in w.items()}
