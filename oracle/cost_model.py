"""Plain restatement of the cost model of Section 3.2 (TEST INFRASTRUCTURE, not the product).

Lemma 3.1 (Eq. 3) and the first condition of Theorem 3.2, written out term by term in float64.
Pinned by the worked numbers of Table 1 / Section 4.2 (tests/golden/table1_model_insertion.txt).
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
