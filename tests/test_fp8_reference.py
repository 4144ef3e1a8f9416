"""Pins of the test-side FP8 row quantiser (parity_harness.fp8_round_rows), which feeds the oracle the values the FP8
storage mode keeps.  It is checked against the format's definition written out by brute force: all 256 byte codes of
e4m3 decoded from their bit fields, nearest code with ties to the even mantissa, and the smallest power-of-two scale
found by search."""
import math

import numpy as np
import torch

from parity_harness import fp8_round_rows


def _e4m3_grid():
    """Every finite non-negative value of the format from its bit fields: exponent bias 7, 3 mantissa bits, subnormals
    at exponent field 0, and the code 1111.111 not a number."""
    vals = []
    for code in range(128):
        ex, man = code >> 3, code & 7
        if ex == 15 and man == 7:
            continue
        vals.append((man / 8.0) * 2.0 ** -6 if ex == 0 else (1 + man / 8.0) * 2.0 ** (ex - 7))
    return vals


def _brute_row(row):
    grid = _e4m3_grid()
    amax = max(abs(float(x)) for x in row)
    if amax == 0:
        return [0.0] * len(row)
    e = -200
    while amax / 2.0 ** e > 448.0:
        e += 1
    e = max(-120, min(120, e))
    out = []
    for x in row:
        y = abs(float(x)) / 2.0 ** e
        best, bi = None, -1
        for i, g in enumerate(grid):
            dist = abs(g - y)
            if best is None or dist < best or (dist == best and i % 2 == 0):   # equal distance: the even mantissa
                best, bi = dist, i
        out.append(math.copysign(grid[bi] * 2.0 ** e, float(x)))
    return out


def test_grid_has_the_formats_landmarks():
    g = _e4m3_grid()
    assert len(g) == 127 and max(g) == 448.0 and g[1] == 2.0 ** -9 and g[8] == 2.0 ** -6 and g == sorted(g)


def test_hand_worked_rows():
    # largest element 448: scale 1.  449: scale 2, 224.5 lies between 224 and 240 and goes to 224, so 448 comes back.
    # 0.3: scale 2^-10, 307.2 lies between 288 and 320 and goes to 320, so 0.3125.
    r = fp8_round_rows(torch.tensor([[448.0, 1.0, 17.0, -19.0]], dtype=torch.float64))[0].tolist()
    assert r == [448.0, 1.0, 16.0, -20.0]          # 17 and 19 are ties between 16|18 and 18|20: even mantissas 16, 20
    r = fp8_round_rows(torch.tensor([[449.0, 3.0]], dtype=torch.float64))[0].tolist()
    assert r == [448.0, 3.0 + 0.0]                 # 1.5 * 2 after scale 2
    r = fp8_round_rows(torch.tensor([[0.3, 0.0]], dtype=torch.float64))[0].tolist()
    assert r == [0.3125, 0.0]
    assert fp8_round_rows(torch.zeros(2, 8)).abs().max().item() == 0.0


def test_matches_brute_force_on_bf16_rows():
    g = torch.Generator().manual_seed(5)
    x = torch.randn(40, 16, generator=g) * torch.logspace(-6, 5, 40).unsqueeze(1)
    x[3, 5] = 0.0; x[7] *= 1e-3; x[9, 0] = 1000.0 * x[9].abs().max()      # a zero, a tiny row, an outlier (subnormals)
    x = x.to(torch.bfloat16)
    got = fp8_round_rows(x)
    for i in range(x.shape[0]):
        assert got[i].tolist() == _brute_row(x[i].double().tolist()), i


def test_properties_every_stored_value_is_a_bf16_and_rounding_is_idempotent():
    g = torch.Generator().manual_seed(6)
    x = (torch.randn(200, 128, generator=g) * 3.0).to(torch.bfloat16)
    r = fp8_round_rows(x)
    assert torch.equal(r, r.to(torch.bfloat16).double())
    assert torch.equal(fp8_round_rows(r), r)
    big = x.double().abs() >= x.double().abs().amax(-1, keepdim=True) * 2.0 ** -8      # elements in the normal range
    rel = ((r - x.double()).abs() / x.double().abs().clamp_min(1e-30))[big]
    assert rel.max().item() <= 2.0 ** -4 + 1e-12
