"""Pins of the oracle's paged block movement (gather / scatter / copy): brute force with explicit
index arithmetic on flat arrays, and the inverse / untouched-words properties."""
import numpy as np
import pytest

import oracle

LAYOUTS = {
    # name: (strides(block, head, token), words per block)
    "head_major": lambda Hkv, bs, D: ((Hkv * bs * D, bs * D, D), Hkv * bs * D),
    "token_major": lambda Hkv, bs, D: ((bs * Hkv * D, D, Hkv * D), bs * Hkv * D),
    "padded_rows": lambda Hkv, bs, D: ((Hkv * bs * (D + 8) + 16, bs * (D + 8), D + 8), Hkv * bs * (D + 8) + 16),
}


def make_pool(layout, NB, Hkv, bs, D, seed):
    strides, words = LAYOUTS[layout](Hkv, bs, D)
    rng = np.random.default_rng(seed)
    k = rng.integers(0, 65536, NB * words, dtype=np.uint16)
    v = rng.integers(0, 65536, NB * words, dtype=np.uint16)
    return k, v, strides


def brute_gather(cache, ids, strides, Hkv, bs, D):
    """Word by word, from the addressing rule: element (n, h, s, i) lives at n*bstr + h*hstr + s*tstr + i."""
    bstr, hstr, tstr = strides
    out = np.zeros(len(ids) * Hkv * bs * D, np.uint16)
    for j, n in enumerate(ids):
        for h in range(Hkv):
            for s in range(bs):
                for i in range(D):
                    out[((j * Hkv + h) * bs + s) * D + i] = cache[n * bstr + h * hstr + s * tstr + i]
    return out.reshape(len(ids), Hkv, bs, D)


@pytest.mark.parametrize("layout", sorted(LAYOUTS))
def test_gather_matches_word_by_word_addressing(layout):
    NB, Hkv, bs, D = 7, 2, 4, 8
    k, v, strides = make_pool(layout, NB, Hkv, bs, D, 1)
    ids = [5, 0, 6, 2]
    kp, vp = oracle.gather_blocks(k, v, ids, num_kv_heads=Hkv, block_size=bs, head_dim=D, strides=strides)
    assert np.array_equal(kp, brute_gather(k, ids, strides, Hkv, bs, D))
    assert np.array_equal(vp, brute_gather(v, ids, strides, Hkv, bs, D))


@pytest.mark.parametrize("layout", sorted(LAYOUTS))
def test_scatter_writes_listed_blocks_only_and_inverts_gather(layout):
    NB, Hkv, bs, D = 9, 2, 4, 8
    k, v, strides = make_pool(layout, NB, Hkv, bs, D, 2)
    kw = dict(num_kv_heads=Hkv, block_size=bs, head_dim=D, strides=strides)
    rng = np.random.default_rng(3)
    ids = [8, 1, 4]
    kp = rng.integers(0, 65536, (3, Hkv, bs, D), dtype=np.uint16)
    vp = rng.integers(0, 65536, (3, Hkv, bs, D), dtype=np.uint16)
    k2, v2 = k.copy(), v.copy()
    oracle.scatter_blocks(kp, vp, ids, k2, v2, **kw)
    # what was scattered reads back, word for word, through the brute-force addressing
    assert np.array_equal(brute_gather(k2, ids, strides, Hkv, bs, D), kp)
    assert np.array_equal(brute_gather(v2, ids, strides, Hkv, bs, D), vp)
    # every word outside the listed blocks' addressed elements is untouched (padding words included)
    touched = np.zeros(k.size, bool)
    bstr, hstr, tstr = strides
    for n in ids:
        for h in range(Hkv):
            for s in range(bs):
                a = n * bstr + h * hstr + s * tstr
                touched[a:a + D] = True
    assert np.array_equal(k2[~touched], k[~touched]) and np.array_equal(v2[~touched], v[~touched])
    # gather then scatter to the same ids is the identity
    k3, v3 = k.copy(), v.copy()
    oracle.scatter_blocks(*oracle.gather_blocks(k, v, ids, **kw), ids, k3, v3, **kw)
    assert np.array_equal(k3, k) and np.array_equal(v3, v)


def test_copy_is_gather_then_scatter_and_a_migration_round_trip_preserves_sequences():
    NB, Hkv, bs, D = 12, 2, 4, 8
    k, v, strides = make_pool("head_major", NB, Hkv, bs, D, 4)
    kw = dict(num_kv_heads=Hkv, block_size=bs, head_dim=D, strides=strides)
    src, dst = [3, 7, 0], [10, 2, 5]
    k2, v2 = k.copy(), v.copy()
    oracle.copy_blocks(k2, v2, src, dst, **kw)
    k3, v3 = k.copy(), v.copy()
    oracle.scatter_blocks(*oracle.gather_blocks(k, v, src, **kw), dst, k3, v3, **kw)
    assert np.array_equal(k2, k3) and np.array_equal(v2, v3)
    for s, d in zip(src, dst):
        assert np.array_equal(brute_gather(k2, [d], strides, Hkv, bs, D), brute_gather(k, [s], strides, Hkv, bs, D))
    # migration: pack on the sender, unpack into another pool with another layout, contents equal
    kr, vr, rstrides = make_pool("token_major", 6, Hkv, bs, D, 5)
    oracle.scatter_blocks(*oracle.gather_blocks(k, v, src, **kw), [4, 1, 3], kr, vr, num_kv_heads=Hkv,
                          block_size=bs, head_dim=D, strides=rstrides)
    assert np.array_equal(brute_gather(kr, [4, 1, 3], rstrides, Hkv, bs, D), brute_gather(k, src, strides, Hkv, bs, D))


def test_ids_outside_the_pool_are_skipped():
    NB, Hkv, bs, D = 4, 1, 2, 8
    k, v, strides = make_pool("head_major", NB, Hkv, bs, D, 6)
    kw = dict(num_kv_heads=Hkv, block_size=bs, head_dim=D, strides=strides)
    kp, vp = oracle.gather_blocks(k, v, [1, -1, 4, 3], **kw)
    assert not kp[1].any() and not kp[2].any()
    assert np.array_equal(kp[[0, 3]], brute_gather(k, [1, 3], strides, Hkv, bs, D))
    k2, v2 = k.copy(), v.copy()
    oracle.scatter_blocks(kp, vp, [1, -1, 4, 3], k2, v2, **kw)
    assert np.array_equal(k2, k)
    oracle.copy_blocks(k2, v2, [0, 9], [2, 1], **kw)
    assert np.array_equal(brute_gather(k2, [2], strides, Hkv, bs, D), brute_gather(k, [0], strides, Hkv, bs, D))
    assert np.array_equal(brute_gather(k2, [1], strides, Hkv, bs, D), brute_gather(k, [1], strides, Hkv, bs, D))
