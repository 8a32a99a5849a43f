"""Index arithmetic used by the tests to address one chosen mapping (test-side only)."""
from __future__ import annotations


def divisor_lists(p):
    return [list(p.divs[d][:p.ndiv[d]]) for d in range(4)]


def tiling_index(p, tile_dims):
    """Index t of the tiling with tile extents (i_G, k_G, l_G, j_G)."""
    divs = divisor_lists(p)
    t = 0
    for d in range(4):
        t = t * p.ndiv[d] + divs[d].index(tile_dims[d])
    return t


def row_index(p, phi, pi, beta):
    """Row r of (fusion mode, loop order, buffering levels of A,B,C,D,E)."""
    orders = list(p.order_id[:p.n_orders])
    phis = list(p.phi_id[:p.n_phi])
    oi = orders.index(pi)
    bA, bB, bC, bD, bE = [b - 3 for b in beta]
    if phi == 0:
        assert phis[0] == 0
        return oi * 3125 + bA * 625 + bB * 125 + bC * 25 + bD * 5 + bE
    assert bC == 0
    base = p.n_orders * 3125 if phis[0] == 0 else 0
    unfused = [f for f in phis if f != 0]
    base += unfused.index(phi) * p.n_orders * 625
    return base + oi * 625 + bA * 125 + bB * 25 + bD * 5 + bE


def candidate_index(p, tile_dims, phi, pi, beta, sm=(0, 0)):
    return (tiling_index(p, tile_dims) * p.R + row_index(p, phi, pi, beta)) * 9 + sm[0] * 3 + sm[1]


def exponent_vector(value, bounds):
    """Exponents of the eight (distinct prime) loop bounds in `value`."""
    q = []
    for b in bounds:
        e = 0
        while value % b == 0:
            value //= b
            e += 1
        q.append(e)
    assert value == 1
    return q
