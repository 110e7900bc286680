"""The process pool of oracle instances (block ranges) against one oracle on the whole vector."""
import numpy as np
import pytest

from oracle import Oracle
from oracle_pool import OraclePool, split_blocks, blockwise_check


def test_split_blocks_tiles_the_block_list():
    for sizes, parts in [([5], 4), ([1, 1, 1], 3), ([100, 1, 1, 1, 1], 3), ([7] * 50, 16),
                         ([51_000_000] + [1000] * 289, 16)]:
        r = split_blocks(sizes, parts)
        assert r[0][0] == 0 and r[-1][1] == len(sizes) and len(r) <= parts
        assert all(a[1] == b[0] for a, b in zip(r, r[1:])) and all(b1 > b0 for b0, b1 in r)


@pytest.mark.parametrize("nproc", [2, 3])
def test_pool_equals_single_oracle_bit_for_bit(nproc):
    rng = np.random.default_rng(3)
    sizes = [33, 5, 700, 64, 1, 4097, 10]
    off = np.concatenate([[0], np.cumsum(sizes)])
    M, steps = 3, 4
    ref = Oracle(off, M, 0.9, 0.1)
    pool = OraclePool(off, M, 0.9, 0.1, nproc=nproc)
    try:
        assert pool.W == ref.W and len(pool.ranges) == nproc
        x0 = rng.standard_normal(off[-1]).astype(np.float32)
        ref.x[:] = x0
        pool.state[:] = x0
        pool.set_x_from_state()
        ref.set_weight_decay(0.01); pool.set_weight_decay(0.01)
        for t in range(steps):
            if t == 2:
                ref.set_eta(0.05); pool.set_eta(0.05)
            for i in range(M):
                g = rng.standard_normal(off[-1]).astype(np.float32)
                ref.worker_step(i, g)
                pool.grad[:] = g
                pool.hint[:] = ref.words(i)
                ad, first, scales = pool.worker_step(i)
                assert len(ad) == 0 and first == -1 and np.array_equal(scales, ref.scales(i))
            ref.server_step()
            pool.hint[:] = ref.words(-1)
            ad, first, scales = pool.server_step()
            assert len(ad) == 0 and first == -1 and np.array_equal(scales, ref.scales(-1))
        assert pool.t == ref.t == steps
        for kind, i, vec in [("x", -1, ref.x), ("e", -1, ref.residual(-1)), ("m", 1, ref.momentum(1)),
                             ("e", 2, ref.residual(2)), ("mt", -1, ref.decay_momentum)]:
            pool.state[:] = vec
            assert pool.compare(kind, i) == ([], 0)
        # a wrong bit outside the tie zone and a wrong state element are both reported, with
        # their position in the whole vector
        pool.state[:] = ref.x
        pool.state[40] += 1.0
        bad, mism = pool.compare("x")
        assert mism == 1 and [b for b, _, _ in bad] == [2]
        for i in range(M):
            g = rng.standard_normal(off[-1]).astype(np.float32)
            ref.worker_step(i, g)
            pool.grad[:] = g
            h = ref.words(i).copy()
            if i == 1:
                j = int(np.argmax(np.abs(ref.last_p[off[5]:off[6]]))) + int(off[5])   # far from zero
                word = int(pool.woffsets[5]) + (j - int(off[5])) // 32
                h[word] ^= np.uint32(1 << ((j - int(off[5])) % 32))
            pool.hint[:] = h
            ad, first, _ = pool.worker_step(i)
            assert len(ad) == 0 and first == (word if i == 1 else -1)
    finally:
        pool.close()


def test_blockwise_check_counts_values_that_differ():
    ref = np.array([1.0, -2.0, 0.0, 4.0], dtype=np.float32)
    got = ref.copy(); got[2] = -0.0                      # the two zeros are the same number
    assert blockwise_check(got, ref, np.array([0, 2, 4])) == ([], 0)
    got[3] = np.nextafter(np.float32(4.0), np.float32(5.0))   # one ulp off: within 1e-5, but counted
    assert blockwise_check(got, ref, np.array([0, 2, 4])) == ([], 1)
