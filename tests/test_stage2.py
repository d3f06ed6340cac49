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
