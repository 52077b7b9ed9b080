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


def draw_batch(rng):
    """Several mid-sized tensors for one batched call: one or two partitions (so that launches hold several
    tensors and every thread block walks through many tiles), random recipes, BF16 copy and fake-quantised
    output asked for on some tensors only."""
    n = int(rng.integers(2, 8))
    parts = [PARTITIONS[int(rng.integers(len(PARTITIONS)))] for _ in range(2)]
    hosts, recipes, fallback, fake = [], [], [], []
    for _ in range(n):
        rows, cols = int(rng.integers(300, 2600)), int(rng.integers(300, 2600)) // 8 * 8
        seed = int(rng.integers(1 << 30))
        gen = int(rng.integers(0, 3))
        bits = (wl.weight_like(rows, cols, seed=seed) if gen == 0 else wl.gradient_like(rows, cols, seed=seed) if gen == 1
                else wl.activation_like(rows, cols, n_outlier_cols=3, seed=seed))
        if rng.random() < 0.3:
            bits[int(rng.integers(rows)), int(rng.integers(cols))] = [0x7F80, 0x7FC0, 0x0001][int(rng.integers(3))]
        block = parts[int(rng.integers(2))]
        if block in ((1, 0), (0, 0)):
            formats, crit = TWO, mb.MOR_CRIT_TENSOR_MEAN_REL
        else:
            formats = THREE if rng.random() < 0.4 else TWO
            crit = mb.MOR_CRIT_BLOCK_VS_E5M2 if formats is THREE else int(rng.integers(0, 3))
        recipes.append(mb.Recipe(block, formats, crit, 0.045, int(rng.integers(0, 3)), int(rng.integers(0, 4))))
        hosts.append(bits)
        fallback.append(bool(rng.random() < 0.3) and block != (128, 1) and crit != mb.MOR_CRIT_TENSOR_MEAN_REL)
        fake.append(bool(rng.random() < 0.3) and block != (128, 1))
    return hosts, recipes, fallback, fake, (1, 0) in parts


@pytest.mark.parametrize("seed", range(8))
def test_random_batch(seed):
    import torch

    from oracle import mor_oracle as orc

    hosts, recipes, fallback, fake, has_channel = draw_batch(np.random.default_rng(90000 + seed))
    stats = bool(seed % 2) and not has_channel
    plan = mb.BatchPlan([parity.to_device(h) for h in hosts], recipes, block_stats=stats, fallback=fallback, fake_quant=fake)
    plan.run()
    plan.run()
    torch.cuda.synchronize()
    for host, r, out, fb, fq in zip(hosts, recipes, plan.outs, fallback, fake):
        ob = parity.oracle_block(r.block, host.shape[1])
        ref = orc.run(host, ob, list(r.formats), r.criterion, r.threshold, r.scale_mode, r.flags, n_threads=8)
        rep = parity.compare(host, r, out, ref, check_block_stats=stats)
        assert rep.n_exempt <= max(2, rep.n_blocks // 500)
        if fq and not parity.exempt_blocks(ref, r).any():
            want = orc.fake_quant(host, ref, ob, list(r.formats), r.criterion, r.threshold, r.scale_mode, r.flags)
            np.testing.assert_array_equal(out.fake_quant.view(torch.int16).cpu().numpy().view(np.uint16), want)
        if fb:
            sel = out.sel.cpu().numpy()
            mask = np.kron(sel == mb.MOR_FMT_BF16, np.ones(ob, dtype=bool))[:host.shape[0], :host.shape[1]]
            np.testing.assert_array_equal(out.bf16_fallback.view(torch.int16).cpu().numpy().view(np.uint16), np.where(mask, host, 0))


@pytest.mark.parametrize("seed", range(24))
def test_random_pair_rows_and_columns(seed):
    """The same tensor with 1x128 and with 128x1 blocks in one call (one read of each tile), one to three
    pairs per call, random shape, recipe, scale mode and flags; both results against the oracle."""
    import torch

    from oracle import mor_oracle as orc

    rng = np.random.default_rng(70000 + seed)
    bits, _, _, supplied = draw_case(rng)
    if seed % 6 == 0:
        bits = wl.gradient_like(int(rng.integers(600, 2400)), int(rng.integers(600, 2400)), seed=seed)
    formats = THREE if rng.random() < 0.5 else TWO
    crit = mb.MOR_CRIT_BLOCK_VS_E5M2 if formats is THREE else int(rng.integers(0, 3))
    mode, flags = int(rng.integers(0, 3)), int(rng.integers(0, 4))
    recipes = [mb.Recipe((1, 128), formats, crit, 0.045, mode, flags), mb.Recipe((128, 1), formats, crit, 0.045, mode, flags)]
    rows, cols = bits.shape
    host = np.full((rows, (cols + 7) // 8 * 8 + 8 * int(rng.integers(0, 2))), 0x7FC1, dtype=np.uint16)
    host[:, :cols] = bits
    x = parity.to_device(host)[:, :cols]
    n_pairs = int(rng.integers(1, 4))
    ga = torch.tensor([orc.tensor_amax(bits)] * (2 * n_pairs), dtype=torch.float32, device="cuda") if supplied else None
    stats = bool(seed % 2)
    plan = mb.BatchPlan([x, x] * n_pairs, recipes * n_pairs, block_stats=stats, group_amax=ga)
    plan.run()
    plan.run()
    torch.cuda.synchronize()
    bits = np.ascontiguousarray(bits)
    refs = [orc.run(bits, parity.oracle_block(r.block, cols), list(r.formats), r.criterion, r.threshold, r.scale_mode, r.flags)
            for r in recipes]
    for k, out in enumerate(plan.outs):
        rep = parity.compare(bits, recipes[k & 1], out, refs[k & 1], check_block_stats=stats)
        assert rep.n_exempt <= max(2, rep.n_blocks // 500)
