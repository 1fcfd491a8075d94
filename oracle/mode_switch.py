"""Oracle for the decode profitability rule (test infrastructure only).

Section 3.3 and Appendix D of the paper: a routed layer saves, per skipped
row, that layer's read of the row's resident KV; over L_r routed layers with a
fraction s of decisions skipping, a step holding V resident tokens removes
s * L_r * b * V bytes, i.e. s * L_r * b * V / BW of time, against a fixed
per-step cost tau.  Routing pays above

    V* = tau * BW / (s * L_r * b).

Served thresholds (Appendix D, "The served thresholds and the rule"): exit at
V*, enter at 1.25 V*; the printed thresholds are these rounded to the nearest
10k tokens.  Between the two the state is kept (hysteresis): routing turns on
when V reaches `enter`, off for newly starting requests when V falls to
`exit`.  Plain Python floats, written from the definition; pinned by the
values the paper prints (tests/golden/breakeven_tokens.txt).
"""
from __future__ import annotations

import math


def breakeven_tokens(tau_s: float, bandwidth_bytes_per_s: float, skip_fraction: float, routed_layers: int,
                     kv_bytes_per_token_layer: float) -> float:
    return tau_s * bandwidth_bytes_per_s / (skip_fraction * routed_layers * kv_bytes_per_token_layer)


def thresholds(v_star: float, round_to: float = 10_000.0):
    """(exit, enter) = (V*, 1.25 V*), each rounded half up to a multiple of round_to (0: no rounding)."""
    def rnd(x):
        return x if round_to <= 0 else math.floor(x / round_to + 0.5) * round_to
    return rnd(v_star), rnd(1.25 * v_star)


def next_state(routed: bool, resident_tokens: float, exit_tokens: float, enter_tokens: float) -> bool:
    if resident_tokens >= enter_tokens:
        return True
    if resident_tokens <= exit_tokens:
        return False
    return routed
