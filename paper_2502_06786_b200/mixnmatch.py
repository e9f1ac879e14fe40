"""Layer-wise Mix'n'Match (Section 3.2, "Mix'n'Match"; Appendix, four strategies): which of the nested precisions
each layer is served at.  Host-side bookkeeping only: every layer keeps its int8 codes (or its packed planes), and a
strategy is a list of r per layer that the caller passes to matq_slice_pack / matq_gemv layer by layer.

The paper names the strategies and their shape but not how an odd count is split between the two ends; here the
extra layer goes to the START of the stack.
"""
from __future__ import annotations

STRATEGIES = ("pyramid", "reverse_pyramid", "increasing", "decreasing")


def _ends_in(outer: int, n_outer: int, mid: int, n_mid: int, centre: int, n_centre: int) -> list[int]:
    """outer precision at both ends, centre precision in the middle, mid precision between them."""
    o_front, o_back = (n_outer + 1) // 2, n_outer // 2
    m_front, m_back = (n_mid + 1) // 2, n_mid // 2
    return [outer] * o_front + [mid] * m_front + [centre] * n_centre + [mid] * m_back + [outer] * o_back


def assign(n8: int, n4: int, n2: int, strategy: str = "pyramid") -> list[int]:
    """Precision r of every layer, first layer first, for n8 + n4 + n2 layers.

    pyramid          int2 at the start and the end, int8 in the centre, int4 in between (the paper's best)
    reverse_pyramid  int8 at the start and the end, int2 in the centre, int4 in between
    increasing       int2 layers first, then int4, then int8
    decreasing       int8 layers first, then int4, then int2
    """
    if min(n8, n4, n2) < 0:
        raise ValueError("layer counts must be non-negative")
    if strategy == "pyramid":
        return _ends_in(2, n2, 4, n4, 8, n8)
    if strategy == "reverse_pyramid":
        return _ends_in(8, n8, 4, n4, 2, n2)
    if strategy == "increasing":
        return [2] * n2 + [4] * n4 + [8] * n8
    if strategy == "decreasing":
        return [8] * n8 + [4] * n4 + [2] * n2
    raise ValueError(f"unknown strategy {strategy!r}; one of {STRATEGIES}")


def effective_bits(rs, overflow_fraction: float = 0.0) -> float:
    """Average bits per weight of equally sized layers served at precisions rs; an extra-precision layer costs one
    more bit per overflow element (Errata: 2.05 bits at 5 % overflow), counted for the r < 8 layers."""
    rs = list(rs)
    if not rs:
        raise ValueError("no layers")
    return sum(r + (overflow_fraction if r < 8 else 0.0) for r in rs) / len(rs)


def counts_for_budget(n_layers: int, max_bits: float) -> list[tuple[int, int, int]]:
    """Every (n8, n4, n2) with n8 + n4 + n2 = n_layers whose effective bits do not exceed max_bits, most bits first."""
    out = []
    for n8 in range(n_layers + 1):
        for n4 in range(n_layers - n8 + 1):
            n2 = n_layers - n8 - n4
            bits = (8 * n8 + 4 * n4 + 2 * n2) / n_layers
            if bits <= max_bits + 1e-12:
                out.append((bits, n8, n4, n2))
    out.sort(key=lambda t: (-t[0], -t[1]))
    return [(n8, n4, n2) for _, n8, n4, n2 in out]
