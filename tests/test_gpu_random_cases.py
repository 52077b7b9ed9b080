"""Seeded random sweep: shapes, partitions, recipes, scale modes, flags and value mixes drawn at random,
every case compared with the oracle element by element.  Complements the hand-picked cases: it walks
combinations nobody thought of (odd leading dimensions, tiny tensors with three formats, special values
in ragged tiles, supplied group amax with every partition)."""
import numpy as np
import pytest

from paper_2512_22804_b200 import binding as mb
from paper_2512_22804_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu

TWO = (mb.MOR_FMT_E4M3, mb.MOR_FMT_BF16)
THREE = (mb.MOR_FMT_E4M3, mb.MOR_FMT_E5M2, mb.MOR_FMT_BF16)
PARTITIONS = [(0, 0), (1, 128), (128, 128), (64, 64), (1, 0), (128, 1)]


def draw_case(rng):
    rows, cols = int(rng.integers(1, 420)), int(rng.integers(1, 700))
    kind = rng.integers(0, 4)
    if kind == 0:
        bits = wl.weight_like(rows, cols, seed=int(rng.integers(1 << 30)))
    elif kind == 1:
        bits = wl.activation_like(rows, cols, n_outlier_cols=min(3, cols), seed=int(rng.integers(1 << 30)))
    elif kind == 2:
        bits = wl.gradient_like(rows, cols, seed=int(rng.integers(1 << 30)))
    else:                                       # values on the FP8 grids, many exact ties in Eq. 3
        bits = wl.to_bf16_bits(np.ldexp(rng.integers(-15, 16, size=(rows, cols)).astype(np.float64), rng.integers(-12, 3, size=(rows, cols))))
    n_special = int(rng.integers(0, 4))
    special = [0x0000, 0x8000, 0x0001, 0x807F, 0x7F7F, 0xFF7F, 0x0080, 0x3F80]
    if rng.random() < 0.25:
        special += [0x7F80, 0xFF80, 0x7FC0, 0xFFFF]                        # inf and NaN now and then
    for _ in range(n_special):
        bits[int(rng.integers(rows)), int(rng.integers(cols))] = special[int(rng.integers(len(special)))]
    block = PARTITIONS[int(rng.integers(len(PARTITIONS)))]
    if block == (1, 0):
        formats, crit = TWO, mb.MOR_CRIT_TENSOR_MEAN_REL
    elif block == (0, 0):
        formats, crit = TWO, int(rng.integers(0, 3))
    else:
        formats = THREE if rng.random() < 0.5 else TWO
        crit = mb.MOR_CRIT_BLOCK_VS_E5M2 if formats is THREE else int(rng.integers(0, 3))
    recipe = mb.Recipe(block, formats, crit, float(rng.choice([0.045, 0.05, 0.02, 0.3])), int(rng.integers(0, 3)), int(rng.integers(0, 4)))
    ld = (cols + 7) // 8 * 8 + 8 * int(rng.integers(0, 3))
    return bits, recipe, ld, bool(rng.random() < 0.3)


@pytest.mark.parametrize("seed", range(60))
def test_random_case(seed):
    rng = np.random.default_rng(1000 + seed)
    bits, recipe, ld, supplied = draw_case(rng)
    stats = tuple(recipe.block) != (1, 0) and seed % 2 == 0
    rep = parity.run_and_compare(bits, recipe, pad_to=ld, block_stats=stats, group_amax_supplied=supplied)
    assert rep.n_exempt <= max(1, rep.n_blocks // 500)
