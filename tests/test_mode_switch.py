"""The decode profitability rule: the oracle against the values the paper
prints, and the library's host functions against the oracle."""
import os
import random

import pytest

from oracle import mode_switch as ref
from paper_2609_37062_b200 import build as da_build

da_build.build()
from paper_2609_37062_b200 import binding as da  # noqa: E402

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "breakeven_tokens.txt")
TAU, LR, B = 2.67e-3, 16, 4096.0


def rows():
    with open(GOLDEN) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                bw, s, vk, dec, ex, en = line.split()
                yield float(bw) * 1e9, float(s), float(vk), int(dec), float(ex), float(en)


def test_oracle_reproduces_every_printed_value():
    n = 0
    for bw, s, vk, dec, ex, en in rows():
        v = ref.breakeven_tokens(TAU, bw, s, LR, B)
        assert round(v / 1e3, dec) == vk, (bw, s, v)
        if ex:
            assert ref.thresholds(v) == (ex * 1e3, en * 1e3), (bw, s, ref.thresholds(v))
        n += 1
    assert n == 10


def test_hysteresis_keeps_its_state_inside_the_band():
    ex, en = 160e3, 200e3
    state = False
    trace = []
    for v in (100e3, 170e3, 199e3, 200e3, 180e3, 161e3, 160e3, 170e3, 250e3, 190e3):
        state = ref.next_state(state, v, ex, en)
        trace.append(state)
    assert trace == [False, False, False, True, True, True, False, False, True, True]


def test_library_matches_the_oracle():
    for bw, s, *_ in rows():
        assert da.decode_attn_breakeven_tokens(TAU, bw, s, LR, B) == ref.breakeven_tokens(TAU, bw, s, LR, B)
    rng = random.Random(7)
    for _ in range(500):
        tau, bw = rng.uniform(1e-4, 1e-2), rng.uniform(1e11, 1e13)
        s, lr, b = rng.uniform(0.01, 1.0), rng.randint(1, 64), rng.choice([512.0, 4096.0, 16384.0])
        v = ref.breakeven_tokens(tau, bw, s, lr, b)
        assert da.decode_attn_breakeven_tokens(tau, bw, s, lr, b) == v
        for rt in (0.0, 1000.0, 10000.0):
            assert da.decode_attn_switch_thresholds(v, rt) == ref.thresholds(v, rt)
        ex, en = ref.thresholds(v)
        state_a = state_b = False
        for _ in range(20):
            x = rng.uniform(0.5 * ex, 1.5 * en)
            state_a = ref.next_state(state_a, x, ex, en)
            state_b = da.decode_attn_switch_next(state_b, x, ex, en)
            assert state_a == state_b


def test_library_rejects_nonsense():
    for args in [(-1.0, 1e12, 0.5, 16, 4096.0), (1e-3, 0.0, 0.5, 16, 4096.0), (1e-3, 1e12, 0.0, 16, 4096.0),
                 (1e-3, 1e12, 1.5, 16, 4096.0), (1e-3, 1e12, 0.5, 0, 4096.0), (1e-3, 1e12, 0.5, 16, 0.0)]:
        with pytest.raises(da.DecodeAttnError) as e:
            da.decode_attn_breakeven_tokens(*args)
        assert e.value.status == da.DA_ERR_INVALID_ARG
