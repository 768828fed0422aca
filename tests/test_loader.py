"""The host loader thread (no GPU needed): its batches are bit-exact the dataset entries the oracle's order names,
over several epochs, shuffled and not; the ring blocks and releases as documented."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_1412_2302_b200 import alexnet as A


def dataset(n, seed=3):
    rng = np.random.default_rng(seed)
    img = rng.integers(0, 256, size=(n, 256, 256, 3), dtype=np.uint8)
    lab = rng.integers(0, 1000, size=(n,), dtype=np.int32)
    return img, lab


def test_loader_order_is_a_permutation_per_epoch():
    for shuffle in (False, True):
        order = np.concatenate(O.loader_order(23, 4, 77, shuffle, 15))      # 20 samples per epoch, 3 epochs
        for e in range(3):
            ep = order[20 * e:20 * (e + 1)]
            assert sorted(ep.tolist()) == list(range(20))                   # the incomplete last batch is dropped
            if not shuffle:
                assert ep.tolist() == list(range(20))
    s = np.concatenate(O.loader_order(23, 4, 77, True, 10))
    assert s[:20].tolist() != list(range(20)) and s[:20].tolist() != s[20:40].tolist()     # shuffled, and anew per epoch
    assert np.concatenate(O.loader_order(23, 4, 78, True, 5)).tolist() != s[:20].tolist()  # depends on the seed
    # Fisher-Yates with a good hash is uniform: all 24 orders of 4 items turn up about equally over many seeds
    counts = {}
    for seed in range(2400):
        counts[tuple(O.loader_order(4, 4, seed, True, 1)[0].tolist())] = counts.get(tuple(O.loader_order(4, 4, seed, True, 1)[0].tolist()), 0) + 1
    assert len(counts) == 24 and min(counts.values()) > 60 and max(counts.values()) < 150


@pytest.mark.parametrize("shuffle", [False, True])
def test_loader_batches_match_oracle_order(shuffle):
    img, lab = dataset(11)
    ld = A.Loader(img, lab, batch=3, depth=3, seed=1234, shuffle=shuffle)
    want = O.loader_order(11, 3, 1234, shuffle, 8)                          # 9 samples per epoch: almost three epochs
    for b in range(8):
        bi, bl, idx = ld.next()
        assert idx == b
        assert np.array_equal(bi, img[want[b]]) and np.array_equal(bl, lab[want[b]])
        ld.release()
    ld.close()


def test_loader_ring_blocks_and_releases():
    img, lab = dataset(8)
    ld = A.Loader(img, lab, batch=2, depth=2, seed=5, shuffle=False)
    a = ld.next()
    b = ld.next()
    assert (a[2], b[2]) == (0, 1)
    with pytest.raises(A.AlexNetError) as e:          # both slots held
        ld.next(timeout_ms=50)
    assert e.value.code == A.ERR_STATE
    first = a[0].copy()
    ld.release()
    c = ld.next()
    assert c[2] == 2 and np.array_equal(c[0], img[4:6])
    assert np.array_equal(b[0], img[2:4])             # the held slot was not overwritten
    assert np.array_equal(first, img[0:2])
    ld.release(); ld.release()
    with pytest.raises(A.AlexNetError):
        ld.release()                                   # nothing held
    ld.close()
    with pytest.raises(A.AlexNetError):
        A.Loader(img, lab, batch=16, depth=2)          # fewer images than one batch
