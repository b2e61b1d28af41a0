"""Host logic of pvf_score's work split (no GPU): every row tile is covered, no more blocks than SMs, the kernel
choice follows the row count."""
import pytest

from paper_2601_12247_b200 import binding

SHAPES = [(126464, 4096), (152064, 3584), (4096, 256), (100, 64), (16, 8), (70000, 512)]


@pytest.mark.parametrize("V,D", SHAPES)
@pytest.mark.parametrize("n_sm", [148, 132, 2, 1])
def test_plan_covers_the_work(V, D, n_sm):
    rows = list(range(1, 70)) + [96, 127, 128, 129, 160, 191, 192, 193, 224, 288, 448, 449, 255, 256, 257, 300, 511, 512, 513, 1000, 1024, 4096, 8192, 8193,
                                 13704, 16384, 32768, 103042]
    for M in rows:
        p = binding.score_plan_for_shape(V, D, n_sm, M)
        paired = p["kernel"] in (2, 3)                                            # blocks work in pairs
        granule = 32 if paired else 16
        if p["kernel"] == 3:                                                      # swapped: one row tile of up to 512 rows
            assert p["row_tiles"] == 1 and p["waves"] == 1 and p["tiles_per_wave"] == 1
        else:
            tile_rows = 256 if p["kernel"] == 2 else 128
            assert p["row_tiles"] == -(-M // tile_rows)
        assert p["tiles_per_wave"] * p["waves"] >= p["row_tiles"]                 # every row tile gets a wave
        assert (p["waves"] - 1) * p["tiles_per_wave"] < p["row_tiles"]            # and no wave is empty
        assert 1 <= p["splits"] <= -(-V // granule)                               # no range without a granule
        per_tile = 2 if paired else 1
        workers = p["tiles_per_wave"] * p["splits"]
        if p["last_wave_tiles"]:                                                  # a partial last wave, split over more pairs
            assert p["kernel"] == 2 and 0 < p["last_wave_tiles"] < p["tiles_per_wave"]
            assert (p["waves"] - 1) * p["tiles_per_wave"] + p["last_wave_tiles"] == p["row_tiles"]
            assert p["splits"] <= p["last_wave_splits"] <= -(-V // granule)
            assert p["last_wave_tiles"] * p["last_wave_splits"] <= n_sm // 2
            workers = max(workers, p["last_wave_tiles"] * p["last_wave_splits"])
        else:
            assert p["waves"] * p["tiles_per_wave"] == p["row_tiles"] or p["kernel"] != 2
        assert p["ctas"] == workers * per_tile and 1 <= p["ctas"] <= max(n_sm, per_tile)
        swap_window = 32 < M <= 64 or 128 < M <= 192 or 256 < M <= 448
        if M <= 32:
            assert p["kernel"] == 0 and p["row_tiles"] == 1 and p["waves"] == 1
        elif n_sm < 2:
            assert p["kernel"] == 1
        elif swap_window:
            assert p["kernel"] == 3
        elif M <= 128:
            assert p["kernel"] == 1
        else:
            assert p["kernel"] == 2
        if p["kernel"] == 2:
            assert p["ctas"] % 2 == 0 and M > 192 and not swap_window
            # the hidden states of a wave stay L2-resident beside the weight stream
            assert p["tiles_per_wave"] == 1 or p["tiles_per_wave"] * 256 * D * 2 <= 40 << 20
        if p["kernel"] == 3:
            assert p["ctas"] % 2 == 0 and swap_window


def test_llada_shape_choices_on_148_sms():
    plan = lambda M: binding.score_plan_for_shape(126464, 4096, 148, M)
    assert plan(32) == dict(ctas=148, splits=148, waves=1, kernel=0, row_tiles=1, tiles_per_wave=1, last_wave_tiles=0,
                            last_wave_splits=0)
    assert plan(256)["kernel"] == 2 and plan(256)["splits"] == 74 and plan(256)["waves"] == 1
    assert plan(48) == dict(ctas=148, splits=74, waves=1, kernel=3, row_tiles=1, tiles_per_wave=1, last_wave_tiles=0,
                            last_wave_splits=0)
    assert plan(160)["kernel"] == 3 and plan(96)["kernel"] == 1 and plan(200)["kernel"] == 2
    assert plan(300)["kernel"] == 3 and plan(448)["kernel"] == 3 and plan(449)["kernel"] == 2
    assert plan(1024)["kernel"] == 2 and plan(1024)["ctas"] == 144
    # config 3's draft pass: 128 tiles of 256 rows = seven waves of 18 tiles x 4 pairs and a last wave of 2 tiles x 37
    assert plan(32768) == dict(ctas=148, splits=4, waves=8, kernel=2, row_tiles=128, tiles_per_wave=18, last_wave_tiles=2,
                               last_wave_splits=37)
    p = plan(103042)
    assert p["kernel"] == 2 and p["tiles_per_wave"] == 18 and p["waves"] == 23 and p["last_wave_tiles"] == 7


def test_invalid_arguments():
    with pytest.raises(binding.PvfError):
        binding.score_plan_for_shape(0, 4096, 148, 32)
    with pytest.raises(binding.PvfError):
        binding.score_plan_for_shape(126464, 4096, 148, 0)
