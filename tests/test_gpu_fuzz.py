"""Seeded random shapes (rows, hidden size and vocabulary all ragged with respect to the tile
sizes), both storage types, both schedules, every output against the oracle."""
import numpy as np
import pytest

from paper_2510_17891_b200 import synth
from tests.test_gpu_parity_small import run_and_compare

pytestmark = pytest.mark.gpu


def _cases(n=24, seed=20251017):
    r = np.random.default_rng(seed)
    out = []
    for i in range(n):
        P, G = int(r.integers(1, 5)), int(r.integers(1, 9))
        T = int(r.integers(1, 700))
        H = 8 * int(r.integers(1, 90))
        V = 8 * int(r.integers(1, 400))
        while P * G * T * H * V > 3e9:          # keep the fp64 oracle in the seconds range
            T = max(1, T // 2)
        out.append(dict(P=P, G=G, T=T, H=H, V=V, dtype="bf16" if i % 4 else "f32",
                        len_lo=float(r.choice([0.0, 0.3, 1.0])), degenerate_frac=float(r.choice([0.0, 0.5])),
                        real_plan_reward=bool(i % 2), bnd_of_T=bool(i % 3 == 0),
                        alpha=float(r.choice([0.0, 0.1, 1.0])), eps=float(r.choice([0.1, 0.2])),
                        fused=bool(r.integers(0, 2)), use_hint=bool(r.integers(0, 2))))
    return out


@pytest.fixture(scope="module")
def trl():
    import paper_2510_17891_b200 as t
    t.load_library()
    return t


@pytest.mark.parametrize("case", _cases(), ids=lambda c: f"P{c['P']}G{c['G']}T{c['T']}H{c['H']}V{c['V']}{c['dtype']}{'F' if c['fused'] else ''}")
def test_random_shape(trl, case):
    c = dict(case)
    alpha, eps, fused, use_hint = c.pop("alpha"), c.pop("eps"), c.pop("fused"), c.pop("use_hint")
    w = synth.scaled(synth.CONFIGS[2], name="fuzz_" + "_".join(str(v) for v in case.values()), sigma_old=0.12, **c)
    run_and_compare(trl, w, alpha=alpha, eps=eps, fused=fused, use_hint=use_hint)
