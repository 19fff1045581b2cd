"""Plain restatement of the cost model of Section 3.2 (TEST INFRASTRUCTURE, not the product).

Lemma 3.1 (Eq. 3) and the two conditions of Theorem 3.2, written out term by term in float64.
The first condition is pinned by the worked numbers of Table 1 / Section 4.2
(tests/golden/table1_model_insertion.txt); the second, for which the paper prints no numbers, by the
step of the theorem's proof it comes from: it is the sign of the last two terms of the difference of
two Lemma 3.1 totals (tests/test_cost_model.py).
"""


def total_time(T, L, beta, N):
    """T = sum_{i=1}^{n-1} (N / L_i) T_i + beta (N / L_{n-1}) T_n   (Lemma 3.1, Eq. 3)."""
    n = len(T)
    assert len(L) == n - 1 and n >= 2
    acc = 0.0
    for i in range(n - 1):
        acc += N / L[i] * T[i]
    return acc + beta * (N / L[n - 2]) * T[n - 1]


def insertion_sides(T_new, T_i, L_new, L_i, L_i_new):
    """(T_new / T_i,  L_new (1 / L_i - 1 / L_{i-new})): inserting the model pays off iff left < right (Theorem 3.2)."""
    return T_new / T_i, L_new * (1.0 / L_i - 1.0 / L_i_new)


def insertion_sides_drafter(T_new, T_next, L_new, L_i, beta):
    """(T_new / T_{i+1},  beta (L_new / L_i - 1)): the second condition of Theorem 3.2, read from its proof.

    The statement's subscripts are garbled; the proof's three-model case fixes them: with M_new between M_1 and
    the drafter M_2, the last two terms of (time with M_new) - (time without) are
    N / L_new T_new + beta N (1 / L_new - 1 / L_i) T_{i+1}, negative iff left < right.  L_new is the acceptance
    length of the pair (M_new, M_{i+1}) -- the same L_new as in the first condition -- L_i that of (M_i, M_{i+1})
    before the insertion, beta the drafter's scaling factor of Lemma 3.1."""
    return T_new / T_next, beta * (L_new / L_i - 1.0)
