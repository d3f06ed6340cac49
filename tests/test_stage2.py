"""Stage 2 (Algorithm 2): the library's allocators against the oracle and against brute force."""
import numpy as np
import pytest

from oracle import lexi_stage2 as ref
from paper_2509_02753_b200 import binding as B


def _table(seed, L, k_max, monotone=True):
    r = np.random.default_rng(seed)
    D = r.uniform(0.1, 2.0, size=(L, k_max))
    if monotone:                       # loss falls as k grows and is 0 at k_max (Algorithm 1 at k_base)
        D = np.sort(D, axis=1)[:, ::-1].copy()
        D[:, -1] = 0.0
    return D


# ---- pins of the oracle itself
def test_oracle_brute_force_on_a_hand_case():
    D = np.array([[5.0, 1.0, 0.0], [4.0, 3.9, 0.0], [0.3, 0.2, 0.0]])
    # budget 5 over 3 layers, k in 1..3; all six feasible vectors by hand:
    # (3,1,1)=0+4+0.3=4.3 (1,3,1)=5+0+0.3=5.3 (1,1,3)=9 (2,2,1)=1+3.9+0.3=5.2 (2,1,2)=1+4+0.2=5.2 (1,2,2)=5+3.9+0.2=9.1
    k, v = ref.brute_force(D, 1, 5)
    assert k == [3, 1, 1] and v == pytest.approx(4.3)


def test_oracle_evolutionary_stays_feasible_and_reaches_the_optimum_on_small_cases():
    for seed in range(4):
        D = _table(seed, 5, 4)
        rnd = np.random.default_rng(100 + seed).integers(0, 2 ** 32, size=200000, dtype=np.uint64)
        k, v = ref.evolutionary(D, 1, 11, rnd, n_pop=16, g_max=400)
        assert sum(k) == 11 and all(1 <= x <= 4 for x in k)
        assert v == pytest.approx(ref.phi(D, k))
        kb, vb = ref.brute_force(D, 1, 11)
        assert v == pytest.approx(vb)          # small search space: the search finds the minimum


def test_oracle_evolutionary_three_generations_traced_by_hand():
    """Algorithm 2 step by step on a case small enough to work out on paper.  L = 3, k in 1..3, budget
    6, two initial members, tournament of 2, eta = 0.5, D_j(k) = [[9,4,0],[5,1,0],[3,2,0]].  Every
    number the search consumes is written below with what it decides; the expected members were
    derived by hand from Algorithm 2 and the conventions in the oracle's header, not by running it.

    initial member 0: 0 -> layer 0 (2,1,1); 0 -> layer 0 (3,1,1); open layers now {1,2}: 1 -> layer 2: (3,1,2), phi 0+5+2 = 7
    initial member 1: 2 -> (1,1,2); 2 -> (1,1,3); open {0,1}: 5 % 2 = 1 -> layer 1: (1,2,3), phi 9+1+0 = 10
    generation 1: tournament 1 draws members 1 (phi 10) then 0 (phi 7): 0 wins; tournament 2 draws 1, 3 % 2 = 1:
        member 1.  coins 2,1,4 -> even,odd,even -> genes from p2,p1,p2: (1,1,3).  2147483647 / 2^32 < 0.5: mutate,
        a = 2 % 3 = 2, b = 1 % 2 = 1 (below a: stays 1): (1,0,4).  projection: clip -> (1,1,3), one unit short; the
        gain of a unit is 9-4 = 5 in layer 0, 5-1 = 4 in layer 1, layer 2 is full: (2,1,3), phi 4+5+0 = 9
    generation 2: draws 5 % 3 = 2, 8 % 3 = 2 -> member 2; draws 3 % 3 = 0 (phi 7), 4 % 3 = 1 (phi 10) -> member 0.
        coins 1,0,1 -> p1,p2,p1 = (2,1,3).  2147483648 / 2^32 = 0.5 is not < 0.5: no mutation.  feasible already.
    generation 3: draws 2 then 3 (both phi 9): the first drawn keeps a tie -> 2; draws 3 then 2 -> 3.  coins 0,0,0
        -> (2,1,3).  0 < 0.5: mutate, a = 0, b = 0 -> steps over a -> 1: (3,0,3).  clip -> (3,1,3), one unit over;
        giving one up costs 4-0 = 4 in layer 0 and 2-0 = 2 in layer 2: (3,1,2), phi 7.
    result: members 0 and 4 tie at phi 7; the earlier one is returned."""
    D = np.array([[9.0, 4.0, 0.0], [5.0, 1.0, 0.0], [3.0, 2.0, 0.0]])
    rnd = [0, 0, 1, 2, 2, 5,
           1, 0, 1, 3, 2, 1, 4, 2147483647, 2, 1,
           5, 8, 3, 4, 1, 0, 1, 2147483648,
           2, 3, 3, 2, 0, 0, 0, 0, 0, 0]
    trace = []
    k, v = ref.evolutionary(D, 1, 6, rnd, n_pop=2, g_max=3, eta_mut=0.5, tournament=2, trace=trace)
    assert trace[0] == {"init": [[3, 1, 2], [1, 2, 3]]}
    assert trace[1] == {"parents": (0, 1), "crossed": [1, 1, 3], "mutated": [1, 0, 4], "projected": [2, 1, 3]}
    assert trace[2] == {"parents": (2, 0), "crossed": [2, 1, 3], "mutated": [2, 1, 3], "projected": [2, 1, 3]}
    assert trace[3] == {"parents": (2, 3), "crossed": [2, 1, 3], "mutated": [3, 0, 3], "projected": [3, 1, 2]}
    assert k == [3, 1, 2] and v == 7.0
    # the stream is consumed exactly: one number fewer is an error, not a silent reuse
    with pytest.raises(IndexError):
        ref.evolutionary(D, 1, 6, rnd[:-1], n_pop=2, g_max=3, eta_mut=0.5, tournament=2)


def test_oracle_evolutionary_without_mutation_a_lone_member_reproduces_itself():
    """eta = 0 and a population of one: both parents are that member, crossover of equal parents
    changes nothing, nothing mutates, the child is feasible already - every generation's child is
    the initial member (Algorithm 2: offspring inherit each layer from one of the two parents)."""
    D = _table(3, 6, 4)
    rnd = np.random.default_rng(9).integers(0, 2 ** 32, size=5000, dtype=np.uint64)
    trace = []
    k, _ = ref.evolutionary(D, 1, 13, rnd, n_pop=1, g_max=40, eta_mut=0.0, tournament=3, trace=trace)
    first = trace[0]["init"][0]
    assert sum(first) == 13 and k == first
    for g in trace[1:]:
        assert g["crossed"] == first and g["mutated"] == first and g["projected"] == first


def test_oracle_evolutionary_operators_behave_as_algorithm_2_states_them():
    """Over 1500 generations on a random stream: (a) crossover takes each gene from one parent, and
    where the parents differ about half come from each (alpha_j ~ Bernoulli(0.5)); (b) a mutation is
    one +1 and one -1 (sum of Delta_j = 0) and fires in about eta of the generations; (c) every member
    is feasible after projection; (d) a larger tournament picks fitter parents (selection sees phi)."""
    D = _table(11, 8, 5)
    L, k_max, k_min, budget, eta = 8, 5, 1, 22, 0.3
    rnd = np.random.default_rng(21).integers(0, 2 ** 32, size=400000, dtype=np.uint64)

    def run(tournament):
        trace = []
        ref.evolutionary(D, k_min, budget, rnd, n_pop=12, g_max=1500, eta_mut=eta, tournament=tournament, trace=trace)
        pop = [list(m) for m in trace[0]["init"]]
        fit = [ref.phi(D, m) for m in pop]
        from_p1 = from_p2 = fired = 0
        rank_sum = 0.0
        for g in trace[1:]:
            p1, p2 = pop[g["parents"][0]], pop[g["parents"][1]]
            for j in range(L):
                assert g["crossed"][j] in (p1[j], p2[j])
                if p1[j] != p2[j]:
                    from_p1 += g["crossed"][j] == p1[j]
                    from_p2 += g["crossed"][j] == p2[j]
            delta = sorted(m - c for m, c in zip(g["mutated"], g["crossed"]))
            assert delta in ([0] * L, [-1] + [0] * (L - 2) + [1])
            fired += delta != [0] * L
            assert sum(g["projected"]) == budget and all(k_min <= v <= k_max for v in g["projected"])
            rank_sum += sum(sum(f < fit[i] for f in fit) / len(pop) for i in g["parents"]) / 2
            pop.append(list(g["projected"]))
            fit.append(ref.phi(D, pop[-1]))
        return from_p1, from_p2, fired, rank_sum / 1500

    a, b, fired, rank1 = run(1)
    assert a + b > 300 and abs(a / (a + b) - 0.5) < 0.06
    assert abs(fired / 1500 - eta) < 0.05
    _, _, _, rank4 = run(4)
    assert rank1 > 0.3            # tournament of one: parents are plain draws
    assert rank4 < 0.6 * rank1    # tournament of four: markedly fitter parents


def test_oracle_projection_moves_the_fewest_units_and_is_optimal_on_convex_tables():
    """Proj of Algorithm 2: the result is feasible, differs from the clipped vector by exactly
    |sum - budget| single units all in one direction (no nearer feasible point exists), and for
    tables with diminishing returns it is the cheapest of those nearest points (brute force)."""
    import itertools
    r = np.random.default_rng(4)
    for case in range(40):
        L, k_max, k_min = 4, 4, 1
        steps = np.sort(r.uniform(0.0, 1.0, size=(L, k_max - 1)), axis=1)[:, ::-1]   # decreasing gains: convex D
        D = np.concatenate([np.cumsum(steps[:, ::-1], axis=1)[:, ::-1], np.zeros((L, 1))], axis=1)
        k_in = r.integers(-1, 7, size=L).tolist()
        budget = int(r.integers(L * k_min, L * k_max + 1))
        out = ref._project(D, k_in, k_min, k_max, budget)
        clipped = [min(max(v, k_min), k_max) for v in k_in]
        assert sum(out) == budget and all(k_min <= v <= k_max for v in out)
        diff = [o - c for o, c in zip(out, clipped)]
        need = budget - sum(clipped)
        assert sum(abs(x) for x in diff) == abs(need)
        assert all(x * need >= 0 for x in diff)
        best = min(ref.phi(D, kk) for kk in itertools.product(range(k_min, k_max + 1), repeat=L)
                   if sum(kk) == budget and all((a_ - c_) * need >= 0 for a_, c_ in zip(kk, clipped))
                   and sum(abs(a_ - c_) for a_, c_ in zip(kk, clipped)) == abs(need))
        assert ref.phi(D, out) == pytest.approx(best, abs=1e-12)


# ---- the library against the oracle
@pytest.mark.parametrize("L,k_max,k_min,budget", [(1, 4, 1, 3), (4, 3, 1, 7), (6, 4, 2, 17), (7, 3, 1, 7), (5, 2, 1, 10)])
def test_exact_allocator_equals_brute_force(L, k_max, k_min, budget):
    for seed in range(3):
        D = _table(seed * 7 + L, L, k_max, monotone=(seed != 1))
        k, v = B.moe_lexi_allocate_exact(D, k_min, budget)
        kb, vb = ref.brute_force(D, k_min, budget)
        assert sum(k) == budget and all(k_min <= x <= k_max for x in k)
        assert v == pytest.approx(vb, abs=1e-12)
        assert v == pytest.approx(ref.phi(D, k), abs=1e-12)


def test_exact_allocator_at_model_scale():
    """Mixtral-shaped: 32 layers, k in {1,2}, budget 48 -> the 16 least sensitive layers drop to k=1."""
    r = np.random.default_rng(5)
    D = np.zeros((32, 2))
    D[:, 0] = r.uniform(0.5, 3.0, size=32)
    k, v = B.moe_lexi_allocate_exact(D, 1, 48)
    assert sum(k) == 48
    dropped = sorted(np.argsort(D[:, 0])[:16].tolist())
    assert sorted(j for j in range(32) if k[j] == 1) == dropped
    assert v == pytest.approx(np.sort(D[:, 0])[:16].sum())


@pytest.mark.parametrize("L,k_max,k_min,budget,g_max", [(4, 3, 1, 7, 50), (16, 8, 2, 80, 300), (26, 6, 2, 104, 200)])
def test_evolutionary_allocator_follows_the_oracle_step_for_step(L, k_max, k_min, budget, g_max):
    D = _table(L, L, k_max)
    rnd = np.random.default_rng(L).integers(0, 2 ** 32, size=400000, dtype=np.uint64).astype(np.uint32)
    for eta, tour in ((0.3, 3), (1.0, 1), (0.0, 4)):
        k, v = B.moe_lexi_allocate_evolutionary(D, k_min, budget, rnd, n_pop=24, g_max=g_max, eta_mut=eta,
                                                tournament=tour)
        ko, vo = ref.evolutionary(D, k_min, budget, rnd, n_pop=24, g_max=g_max, eta_mut=eta, tournament=tour)
        assert k == ko                     # integer result: identical
        assert v == pytest.approx(vo, abs=1e-12)
        ke, ve = B.moe_lexi_allocate_exact(D, k_min, budget)
        assert v >= ve - 1e-12             # never below the true optimum


def test_bad_problems_are_refused():
    D = _table(1, 4, 3)
    with pytest.raises(B.MoEError):
        B.moe_lexi_allocate_exact(D, 1, 13)            # budget above L * k_max
    with pytest.raises(B.MoEError):
        B.moe_lexi_allocate_exact(D, 1, 3)             # budget below L * k_min
    with pytest.raises(B.MoEError):
        B.moe_lexi_allocate_evolutionary(D, 1, 7, np.zeros(10, dtype=np.uint32), g_max=100)   # stream too short
