"""Integer cost accounting of a TLinFormer block -- TEST INFRASTRUCTURE ONLY.

The paper counts one unit per (query, key, feature) triple.  This file lists
the attention calls of one block, layer by layer as Appendix A enumerates them,
and adds up query*key pairs; the closed forms of Eq. (cache miss, full form) and
Eq. (cache hit) are then identities a test can check against this enumeration.
Notation: N total length, W_oh history summary window, W_og generation window,
H_depth the number of intermediate self-attention layers, D the model width.
"""
from __future__ import annotations


def miss_layers(N: int, W_oh: int, W_og: int, H_depth: int):
    """[(name, queries, keys)] for a cache-miss pass, in the appendix's order."""
    hist = N - W_og
    layers = [("ctx_first_focused", W_oh, hist)]
    layers += [(f"ctx_self_{i}", W_oh, W_oh) for i in range(H_depth)]
    layers += [("ctx_restore", hist, W_oh)]
    layers += [("gen_cross_history", W_og, hist)]
    layers += [(f"gen_cross_ctx_{i}", W_og, W_oh) for i in range(H_depth + 1)]
    # the paper charges the in-window causal attention as a full W_og x W_og square
    layers += [(f"gen_causal_{i}", W_og, W_og) for i in range(H_depth + 2)]
    return layers


def hit_layers(N: int, W_oh: int, W_og: int, H_depth: int):
    """[(name, queries, keys)] for a cache-hit step; only the newest token queries the history/context."""
    hist = N - W_og
    layers = [("gen_cross_history", 1, hist)]
    layers += [(f"gen_cross_ctx_{i}", 1, W_oh) for i in range(H_depth + 1)]
    layers += [(f"gen_causal_{i}", W_og, W_og) for i in range(H_depth + 2)]
    return layers


def pairs(layers) -> int:
    return sum(qn * kn for _, qn, kn in layers)


def miss_closed_form(N: int, W_oh: int, W_og: int, H_depth: int, D: int) -> int:
    """Eq. (total cost, cache miss, full form)."""
    return D * (N * (2 * W_oh + W_og) + H_depth * (W_oh ** 2 + W_og ** 2 + W_og * W_oh) + W_og ** 2 - W_og * W_oh)


def hit_closed_form(N: int, W_oh: int, W_og: int, H_depth: int, D: int) -> int:
    """Eq. (total cost, cache hit)."""
    return D * N - D * W_og + (H_depth + 1) * D * W_oh + (H_depth + 2) * D * W_og ** 2


def allowed_pairs(N: int, W: int, causal_window: int) -> int:
    """Exact number of (query, key) pairs one forward call evaluates: history unmasked + triangle."""
    return W * N if not causal_window else W * (N - W) + W * (W + 1) // 2
