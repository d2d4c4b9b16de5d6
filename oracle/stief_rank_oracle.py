"""CPU oracle for the sequential budgeted rank selector (the paper's Sec. 3.4 "Rank selection", Eq. 15-17, and
Algorithm 2 with the cost of Eq. 23).

TEST INFRASTRUCTURE ONLY: imported by the tests (and nothing in the product).  Exact rational arithmetic
(`fractions.Fraction`), one layer at a time in the algorithm's order; shares no code with the library.

What the paper fixes: the budget starts at B_1 = L * rho; before layer l (1-based) the per-layer budget is the mean of
what is left over the layers still to choose; among the candidate pairs whose cost c = (r_K + r_V) / (2 d_h) does not
exceed it, the pair of least error is taken; its cost is subtracted; the next layer's surface is evaluated on what the
chosen prefix produces (so a surface may depend on the earlier choices: it is asked for only then).

Readings where the paper is silent or at odds with itself:
* Eq. 15 prints the divisor L - (l + 1), Algorithm 2 prints L - l + 1.  The text calls tau "the current average
  remaining budget", and only L - l + 1 is the number of layers still to choose (the other is zero one layer before the
  end), so Algorithm 2's divisor is used.
* Ties in the error: the cheaper pair; at equal cost the smaller key rank (the paper reports values as the harder side).
* No feasible pair (rho below the cheapest candidate's cost): an error naming the layer, not a silent fallback.
* rho is taken as the exact value of the float that is passed.
"""
from __future__ import annotations

from fractions import Fraction


class Infeasible(Exception):
    def __init__(self, layer):
        super().__init__(f"no candidate pair fits the budget at layer {layer}")
        self.layer = layer


def cost(r_k: int, r_v: int, d_h: int = 128) -> Fraction:
    """Normalised cache cost of a rank pair (Eq. 23; the same ratio as Eq. 3)."""
    return Fraction(r_k + r_v, 2 * d_h)


def select_ranks(L: int, cand_k, cand_v, rho: float, surface, d_h: int = 128):
    """Algorithm 2.  ``surface(l, chosen)`` returns the error table of layer l (0-based) as a nested sequence
    [len(cand_k)][len(cand_v)], given the list ``chosen`` of the (r_K, r_V) already selected for layers 0 .. l-1.
    Returns (ranks, spent): the L selected pairs and the total cost as a Fraction."""
    B = L * Fraction(rho)                                   # B_1 = L rho
    chosen = []
    for l in range(L):
        tau = B / (L - l)                                   # layers l .. L-1 are still to choose (Algorithm 2's divisor)
        delta = surface(l, list(chosen))
        best = None
        for i, rk in enumerate(cand_k):
            for j, rv in enumerate(cand_v):
                c = cost(rk, rv, d_h)
                if c > tau:
                    continue
                key = (delta[i][j], c, rk)
                if best is None or key < best[0]:
                    best = (key, rk, rv, c)
        if best is None:
            raise Infeasible(l)
        chosen.append((best[1], best[2]))
        B -= best[3]                                        # Eq. 17
    return chosen, L * Fraction(rho) - B
