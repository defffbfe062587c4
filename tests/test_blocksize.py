"""Block-size selection (Section 5.1): the walk over candidate sizes with an injected timer (CPU), and one real run
on the GPU."""
import pytest

from paper_2108_11033_b200 import blocksize as bs


def fake_timer(table):
    return lambda layer: table[(layer["bh"], layer["bw"])]


def test_walk_stops_at_the_first_size_that_no_longer_pays():
    sizes = [(1, 4), (2, 8), (4, 16), (8, 32), (16, 64)]
    table = {(1, 4): 10.0, (2, 8): 5.0, (4, 16): 3.0, (8, 32): 2.95, (16, 64): 1.0}
    size, ms, trace = bs.find_opt_blk((64, 128), 4.0, sizes, time_layer=fake_timer(table), threshold=1.05)
    assert size == (4, 16) and ms == 3.0
    assert [t[0] for t in trace] == sizes[:4]          # (16, 64) is never timed: the walk ended at (8, 32)


def test_walk_degenerate_cases():
    one = [(4, 16)]
    assert bs.find_opt_blk((64, 128), 4.0, one, time_layer=fake_timer({(4, 16): 2.0}))[0] == (4, 16)   # first size always accepted
    assert bs.find_opt_blk((64, 128), 4.0, [], time_layer=fake_timer({}))[0] is None
    table = {(2, 8): 4.0, (4, 16): 2.0, (8, 32): 1.0}
    size, ms, trace = bs.find_opt_blk((64, 128), 4.0, list(table), time_layer=fake_timer(table), threshold=1.5)
    assert size == (8, 32) and len(trace) == 3        # every step pays: the largest size wins
    slower = {(2, 8): 1.0, (4, 16): 2.0}
    assert bs.find_opt_blk((64, 128), 4.0, list(slower), time_layer=fake_timer(slower))[0] == (2, 8)


def test_synthesized_layer_has_the_asked_rate_and_structure():
    from oracle import bcr_oracle as orc
    layer = bs.synthesize(256, 512, 8.0, (8, 32))
    assert layer["W"].shape == (256, 512) and layer["mask"].shape == (256, 512)
    _, ok = orc.extract_blocks(layer["mask"], 8, 32)
    assert ok
    assert 6.0 < layer["mask"].size / layer["mask"].sum() < 10.5


@pytest.mark.gpu
def test_find_opt_blk_on_the_gpu():
    sizes = [(1, 4), (2, 8), (4, 16), (8, 32), (16, 64)]
    size, ms, trace = bs.find_opt_blk((1024, 1024), 10.0, sizes, N=64, threshold=1.05, reps=5)
    assert size in sizes and ms > 0 and 1 <= len(trace) <= len(sizes)
    assert all(t[1] > 0 for t in trace)
