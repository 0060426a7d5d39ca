"""The work partition of the streaming GEMM (host arithmetic, no GPU): every (16-row tile,
512-wide k chunk) unit is multiplied exactly once, split tiles pair up between neighbouring CTAs,
and the units per CTA differ by at most one."""
import pytest

from paper_2506_03700_b200 import binding

SHAPES = [  # (N, K, mode) -- the GEMMs of the 8B / 1B / 13B shapes and some ragged ones
    (6144, 4096, 0), (4096, 4096, 0), (28672, 4096, 1), (4096, 14336, 0), (128256, 4096, 0),
    (3072, 2048, 0), (16384, 2048, 1), (2048, 8192, 0), (15360, 5120, 0), (27648, 5120, 1),
    (5120, 13824, 0), (1408, 256, 1), (256, 704, 0), (1000, 192, 0), (48, 64, 0), (2368, 57344, 0),
]


def units_of(N, K, mode, grid, cta, split=True):
    p = binding.debug_gemm_plan(N, K, mode, grid, cta, split)
    nch = (K + 511) // 512
    units = []
    if not p["split"]:
        for t in range(p["t0"], p["t1"]):
            units += [(t, k) for k in range(nch)]
        return p, units
    assert 1 <= p["n"] <= 8
    for kc in range(nch):
        for s in range(p["n"]):
            if s == 0:
                if kc < p["s0_pub_k1"]:
                    units.append((p["tb"], kc))
                elif kc >= p["s0_own_k0"]:
                    units.append((p["ta"], kc))
            elif s == p["n"] - 1 and kc >= p["sl_k1"]:
                pass
            else:
                units.append((p["ta"] + s, kc))
    return p, units


@pytest.mark.parametrize("N,K,mode", SHAPES)
@pytest.mark.parametrize("grid", [1, 7, 132, 148, 160])
def test_every_unit_once(N, K, mode, grid):
    tiles = (N // 2) // 16 if mode == 1 else (N + 15) // 16
    nch = (K + 511) // 512
    seen = {}
    counts = []
    plans = []
    for cta in range(grid):
        p, units = units_of(N, K, mode, grid, cta)
        plans.append(p)
        counts.append(len(units))
        for u in units:
            seen[u] = seen.get(u, 0) + 1
    assert len(seen) == tiles * nch and all(v == 1 for v in seen.values())
    if plans[0]["split"]:
        assert max(counts) - min(counts) <= 1
        for cta, p in enumerate(plans):
            # a tail part (chunks from s0_own_k0 > 0 of tile ta) is completed by the head part of the CTA before
            if p["s0_own_k0"] > 0:
                q = plans[cta - 1]
                head_k1 = q["s0_pub_k1"] if q["s0_pub_k1"] > 0 else q["sl_k1"]
                head_tile = q["tb"] if q["s0_pub_k1"] > 0 else q["ta"] + q["n"] - 1
                assert cta > 0 and head_tile == p["ta"] and head_k1 == p["s0_own_k0"]


def test_whole_tiles_when_not_asked_to_split():
    for cta in range(148):
        p, _ = units_of(28672, 4096, 1, 148, cta, split=False)
        assert p["split"] == 0


def test_8b_gate_up_is_split_evenly():
    counts = [len(units_of(28672, 4096, 1, 148, c)[1]) for c in range(148)]
    assert set(counts) == {48, 49} and sum(counts) == 896 * 8


def test_bad_arguments():
    with pytest.raises(binding.AdaError):
        binding.debug_gemm_plan(4096, 100, 0, 148, 0)
    with pytest.raises(binding.AdaError):
        binding.debug_gemm_plan(4096, 4096, 0, 148, 148)
