"""Host-side check of the Jacobi block schedule (recursive halving) that the eigen-solver kernels use.

The formulas below restate `step_plan` / `find_holder` of csrc/atomo_eig.cu; the properties are what the kernels
rely on: at every step each block is in exactly one pair, every pair of blocks meets exactly once per sweep, a
CTA keeps its first block for a whole level, and the inverse map sends a block to the CTA that pairs it next."""
import pytest


def step_level(nb, local):
    lg, base = nb.bit_length() - 1, 0
    while local - base >= (1 << (lg - 1)):
        base += 1 << (lg - 1)
        lg -= 1
    return lg, local - base


def step_plan(nb, local, slot):
    lg, t = step_level(nb, local)
    m = 1 << (lg - 1)
    grp, k = slot >> (lg - 1), slot & (m - 1)
    return (grp << lg) + k, (grp << lg) + m + ((k + t) & (m - 1)), t == 0, t == m - 1


def find_holder(nb, local, blk):
    lg, t = step_level(nb, local)
    m = 1 << (lg - 1)
    grp, pos = blk >> lg, blk & ((1 << lg) - 1)
    role = int(pos >= m)
    return grp * m + (((pos - m - t) & (m - 1)) if role else pos), role


@pytest.mark.parametrize("nb", [2, 4, 8, 16, 32, 64, 256, 1024])
def test_every_pair_once_per_sweep(nb):
    met = set()
    resident = {}
    for local in range(nb - 1):
        seen = set()
        for slot in range(nb // 2):
            bi, bj, first, last = step_plan(nb, local, slot)
            assert bi != bj and bi not in seen and bj not in seen
            seen |= {bi, bj}
            met.add((min(bi, bj), max(bi, bj)))
            assert find_holder(nb, local, bi) == (slot, 0) and find_holder(nb, local, bj) == (slot, 1)
            if not first:
                assert resident[slot] == bi              # the first block stays for the whole level
            resident[slot] = bi
        assert len(seen) == nb
    assert len(met) == nb * (nb - 1) // 2
