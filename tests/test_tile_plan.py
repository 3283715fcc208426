"""Host logic of the CTA-pair GEMM's work split (runs without a GPU): whatever T, N and the number of resident pairs,
the tiles of all pairs cover every 256-row block x 16-column unit exactly once, widths are multiples of 16 within
[16, 256] that differ by at most 16, and no pair gets more than one tile above the average."""
import itertools

import pytest

import paper_2512_14481_b200 as P


def all_tiles(T, N, pairs):
    return [P.sasq_static_w8a8_linear_tiles(T, N, pairs, p) for p in range(pairs)]


@pytest.mark.parametrize("T,N", [(129, 8), (256, 4096), (257, 1024), (300, 776), (2048, 4096), (2048, 11008),
                                 (4096, 5120), (4096, 13824), (8192, 4096), (8192, 11008), (16384, 4096),
                                 (1000, 264), (513, 24)])
@pytest.mark.parametrize("pairs", [74, 66, 1, 7])
def test_tiles_cover_the_output_exactly_once(T, N, pairs):
    per_pair = all_tiles(T, N, pairs)
    row_blocks, units = (T + 255) // 256, (N + 15) // 16
    seen = set()
    widths = set()
    for tiles in per_pair:
        for row0, col0, width in tiles:
            assert row0 % 256 == 0 and col0 % 16 == 0 and width % 16 == 0 and 16 <= width <= 256
            widths.add(width)
            for u in range(col0 // 16, (col0 + width) // 16):
                key = (row0 // 256, u)
                assert key not in seen
                seen.add(key)
    assert len(seen) == row_blocks * units
    assert max(widths) - min(widths) <= 16
    counts = [len(t) for t in per_pair]
    assert max(counts) - min(counts) <= 1


def test_llama_shapes_fill_the_waves():
    # columns a pair has to compute vs the ideal share: within 9 % for the benchmark's shapes on 74 pairs (2048 x 4096
    # has 8 row blocks x 18 tiles = 144 tiles for 148 slots, two tiles of up to 240 columns per pair)
    for T, N in [(2048, 4096), (2048, 11008), (8192, 4096), (8192, 11008)]:
        per_pair = all_tiles(T, N, 74)
        most = max(sum(w for _, _, w in tiles) for tiles in per_pair)
        ideal = ((T + 255) // 256) * N / 74
        assert most <= 1.09 * ideal, (T, N, most, ideal)


def test_invalid_arguments():
    lib = P.load_library()
    assert lib.sasq_static_w8a8_linear_tiles(0, 8, 4, 0, None, 0) == -1
    assert lib.sasq_static_w8a8_linear_tiles(256, 8, 4, 4, None, 0) == -1
    assert lib.sasq_static_w8a8_linear_tiles(256, 8, 0, 0, None, 0) == -1


# ---------------------------------------------------------------------------
# how sasq_static_w8a8_linear_multi cuts a list of problems into launches (host logic, no device)
# ---------------------------------------------------------------------------
LLAMA7B = [(4096, 4096)] * 4 + [(4096, 11008)] * 2 + [(11008, 4096)]          # (K, N) of the seven linears


def launches(shapes, pairs=74):
    return P.sasq_static_w8a8_linear_multi_launches(shapes, pairs)


def test_multi_prefill_problems_share_launches_within_the_code_budget():
    layer = lambda T: [(T, N, K) for K, N in LLAMA7B]
    assert launches(layer(2048)) == 1            # 73 MB of int8 codes: one launch
    assert launches(layer(129)) == 1
    assert launches(layer(4096)) == 2            # 146 MB: cut where the running sum passes 80 MiB
    assert launches(layer(16384)) == 7           # every problem's codes alone exceed the budget
    assert launches([(300, 128, 64)] * 8) == 1 and launches([(300, 128, 64)] * 9) == 2     # 8 problems per launch
    assert launches([(256 * 600, 128, 16)] * 2) == 2                                      # 1024 row blocks per launch
    assert launches([]) == 0 and launches([(0, 128, 64)] * 3) == 0


def test_multi_small_t_problems_share_a_launch_only_if_they_fill_the_chip():
    layer = lambda T: [(T, N, K) for K, N in LLAMA7B]
    for T in (1, 16, 128):
        assert launches(layer(T)) == 1                       # 200+ tiles for 74 pairs
        assert launches(layer(T)[:3]) == 1                   # q/k/v: too few tiles for the CTA pairs, but their 96
                                                             # 128-channel tiles fit the device: one small-T launch
        assert launches([(T, 1032, 512), (T, 520, 2048), (T + 1, 2048, 256)]) == 2     # another T: a launch of its own
        assert launches(layer(T)[4:6]) == 1                  # gate/up: 106 tiles
        assert launches(layer(T)[:1]) == 1
    # a small-T problem whose 128-channel tiles outnumber the SMs needs a quantizer launch of its own
    assert launches([(16, 19200, 80)]) == 2
    # the same list on a (hypothetical) device with fewer resident pairs fills the pairs and goes to them
    assert launches(layer(16)[:3], pairs=32) == 1


def test_multi_launches_invalid_arguments():
    import pytest
    with pytest.raises(ValueError):
        launches([(16, 0, 64)])
    with pytest.raises(ValueError):
        launches([(16, 128, 64)], pairs=0)
