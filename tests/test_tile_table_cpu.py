"""The partition of a ragged tensor list into tiles (host logic of the CUDA library, no GPU):
every element in exactly one tile, in order; power-of-two tile sizes; the last, incomplete
round over the blocks cut into at most one piece per block; and the room the size query
reserves for the tables is never exceeded."""
import numpy as np
import pytest


@pytest.fixture(scope="module")
def B():
    from paper_1810_05486_b200 import binding
    return binding


def descs_of(B, tensors):
    return B.make_descs([dict(theta=0x10000, comp=0x20000 if cb else None, numel=n, theta_bits=tb, comp_bits=cb,
                              exp_theta=-10) for n, tb, cb in tensors])


def check_partition(table, tensors):
    """Every tensor's elements [0, numel) covered once, in order, tensors in order."""
    pos = [0] * len(tensors)
    last_tensor = 0
    for t, first, count in table:
        assert t >= last_tensor
        last_tensor = t
        assert first == pos[t] and count > 0
        pos[t] += count
    assert pos == [n for n, _, _ in tensors]


def whole_tile_size(tb, cb, which, chunk8):
    if which == 1:
        return 32768 if (tb == 8 and cb <= 8) else 16384
    return chunk8 if tb == 8 else 8192


@pytest.mark.parametrize("seed", range(40))
def test_random_lists_are_partitioned_exactly_on_any_number_of_blocks(B, seed):
    rng = np.random.default_rng(seed)
    n_tensors = int(rng.integers(1, 30))
    scale = int(rng.choice([2_000, 100_000, 3_000_000]))
    tensors = [(int(rng.integers(1, scale)), int(rng.choice([8, 16])), int(rng.choice([0, 8, 16])))
               for _ in range(n_tensors)]
    if seed % 5 == 0:                      # long enough for the large tiles and the second table
        tensors.append((40_000_000, 8, 8))
    descs = descs_of(B, tensors)
    reserve = 1024
    for sms in (0, 1, 2, 7, 108, 132, 148, 160, 1024, 5000):
        for which in (0, 1):
            table = B.kahan_sgd_tile_table(descs, sms, which)
            if which == 1 and not table:
                continue
            check_partition(table, tensors)
            sizes = {c for _, _, c in table}
            whole = B.kahan_sgd_tile_table(descs, 0, which)
            assert len(table) <= len(whole) + reserve            # what the size query reserves
            # a full tile is a power of two; a shorter one ends its tensor
            for t, first, count in table:
                assert count & (count - 1) == 0 or first + count == tensors[t][0]
            if sms == 0:
                continue
            # all rounds but the last hold whole tiles; the last has at most one piece per block
            full_rounds = len(whole) // sms
            assert table[:full_rounds * sms] == whole[:full_rounds * sms]
            assert len(table) - full_rounds * sms <= max(min(sms, reserve), len(whole) - full_rounds * sms)
            for t, first, count in table[full_rounds * sms:]:
                assert count >= 512 or first + count == tensors[t][0]


def test_the_cases_the_rule_is_stated_for(B):
    # 19 tiles left over on 148 blocks: 4 pieces each would be 76, 8 would be 152: 4 pieces of 2048
    descs = descs_of(B, [(8192 * (2 * 148 + 19), 16, 16)])
    table = B.kahan_sgd_tile_table(descs, 148)
    assert len(table) == 2 * 148 + 19 * 4
    assert {c for _, _, c in table[:2 * 148]} == {8192} and {c for _, _, c in table[2 * 148:]} == {2048}
    # one tile on its own: 16 pieces of 512 elements (a piece has at least 512)
    assert [c for _, _, c in B.kahan_sgd_tile_table(descs_of(B, [(8192, 16, 16)]), 148)] == [512] * 16
    # a tile count that is a multiple of the block count, and more than half a round left over: nothing is cut
    for tiles in (148, 296, 148 + 75, 148 + 147):
        table = B.kahan_sgd_tile_table(descs_of(B, [(8192 * tiles, 16, 16)]), 148)
        assert len(table) == tiles and {c for _, _, c in table} == {8192}
    # no device given: whole tiles
    assert len(B.kahan_sgd_tile_table(descs_of(B, [(8192 * 5, 16, 16)]), 0)) == 5
    # a short list has no table for steps on 8-bit gradients; invalid arguments are refused
    assert B.kahan_sgd_tile_table(descs_of(B, [(8192 * 5, 16, 16)]), 148, which=1) == []
    with pytest.raises(B.KahanSgdError):
        B.kahan_sgd_tile_table(descs_of(B, [(8192, 16, 16)]), -1)
    with pytest.raises(B.KahanSgdError):
        B.kahan_sgd_tile_table(descs_of(B, [(0, 16, 16)]), 148)
