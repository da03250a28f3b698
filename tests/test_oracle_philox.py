"""Pins for the oracle's counter-based RNG and the draws built on it."""
import os

import numpy as np

import oracle


def test_philox_known_answers(golden_dir):
    rows = [l.split() for l in open(os.path.join(golden_dir, "philox4x32_10_kat.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        out = oracle.philox4x32_10(v[0:4], v[4:6])
        assert [int(x) for x in out] == v[6:10]


def test_philox_is_a_bijection_on_small_sample():
    # distinct counters under one key give distinct blocks (Philox is a keyed permutation)
    seen = set()
    for c in range(2000):
        seen.add(tuple(int(x) for x in oracle.philox4x32_10([c, 0, 0, 0], [7, 9])))
    assert len(seen) == 2000


def test_action_word_keying():
    # word t&3 of the block with counter (env, t>>2, 0, 0), key = (seed lo, seed hi)
    seed = 0x1234_5678_9ABC_DEF0
    for env, t in [(0, 0), (5, 1), (5, 2), (5, 3), (5, 4), (77, 1003), (2**32 - 1, 2**34 + 6)]:
        blk = oracle.philox4x32_10([env, (t >> 2) & 0xFFFFFFFF, 0, 0], [seed & 0xFFFFFFFF, seed >> 32])
        assert oracle.action_word(seed, env, t) == int(blk[t & 3])
    # four consecutive steps share one block; the next four use the next counter
    words = [oracle.action_word(0, 3, t) for t in range(8)]
    assert words[:4] == [int(x) for x in oracle.philox4x32_10([3, 0, 0, 0], [0, 0])]
    assert words[4:] == [int(x) for x in oracle.philox4x32_10([3, 1, 0, 0], [0, 0])]


def test_uniform_endpoints_and_exactness():
    assert oracle.uniform01(0) == 0.0
    assert oracle.uniform01(0xFF) == 0.0                      # low 8 bits are dropped
    assert oracle.uniform01(0x100) == np.float32(2.0 ** -24)
    assert oracle.uniform01(0xFFFFFFFF) == np.float32(1.0 - 2.0 ** -24)
    assert oracle.uniform01(0x80000000) == 0.5


def test_random_action_mapping():
    C, A, S = oracle.CARTPOLE, oracle.ACROBOT, oracle.SYNTH
    for kind in (C, S):
        assert oracle.random_action(kind, 0x7FFFFFFF) == 0
        assert oracle.random_action(kind, 0x80000000) == 1
    # floor(3w / 2^32): thirds of the 32-bit range
    assert oracle.random_action(A, 0) == 0
    assert oracle.random_action(A, 0x55555555) == 0
    assert oracle.random_action(A, 0x55555556) == 1
    assert oracle.random_action(A, 0xAAAAAAAA) == 1
    assert oracle.random_action(A, 0xAAAAAAAB) == 2
    assert oracle.random_action(A, 0xFFFFFFFF) == 2


def test_draw_state_keying_and_range():
    seed = 42
    for kind, S, lo, width in [(oracle.CARTPOLE, 4, -0.05, 0.1), (oracle.ACROBOT, 4, -0.1, 0.2), (oracle.SYNTH, 64, -1.0, 2.0)]:
        for env, r in [(0, 0), (9, 3), (123456, 17)]:
            st = oracle.draw_state(kind, S, seed, env, r)
            assert st.shape == (S,)
            for j in range(S // 4):
                blk = oracle.philox4x32_10([env, r, 1, j], [seed, 0])
                for i in range(4):
                    u = (int(blk[i]) >> 8) / 2.0 ** 24          # exact in double
                    exact = lo + width * u                       # double reference of the range map
                    assert abs(float(st[4 * j + i]) - exact) <= 1.2e-7 * max(width, 1.0)
            assert np.all(st >= np.float32(lo)) and np.all(st < np.float32(lo + width) + 1e-7)
    # draws differ between reset indices and between envs
    a = oracle.draw_state(oracle.CARTPOLE, 4, 0, 1, 0)
    assert not np.array_equal(a, oracle.draw_state(oracle.CARTPOLE, 4, 0, 1, 1))
    assert not np.array_equal(a, oracle.draw_state(oracle.CARTPOLE, 4, 0, 2, 0))


def test_range_map_is_single_rounding():
    # fma(u, width, lo): the largest u must stay strictly below lo+width for CartPole and SYNTH
    top = 1.0 - 2.0 ** -24
    assert np.float32(np.float64(np.float32(0.1)) * top + np.float64(np.float32(-0.05))) < np.float32(0.05) + 1e-9


def test_action_stream_statistics():
    w = np.array([oracle.action_word(0, e, t) for e in range(64) for t in range(256)], dtype=np.uint64)
    bits = (w >> np.uint64(31)).astype(np.float64)
    n = bits.size
    assert abs(bits.mean() - 0.5) < 4 * 0.5 / np.sqrt(n)
    tern = ((w * np.uint64(3)) >> np.uint64(32)).astype(int)
    counts = np.bincount(tern, minlength=3)
    assert np.all(np.abs(counts / n - 1 / 3) < 4 * np.sqrt(2 / 9 / n))


def test_bit_sliced_action_stream():
    seed = 77
    for env, t in [(0, 0), (3, 1), (3, 31), (3, 32), (3, 127), (3, 128), (9, 1000), (5, (1 << 34) + 77)]:
        tb = (t >> 2) & 0xFFFFFFFF
        blk = oracle.philox4x32_10([env, tb >> 5, 2, 0], [seed, 0])
        b = t & 127
        assert oracle.action_bit(seed, env, t) == (int(blk[b >> 5]) >> (b & 31)) & 1
    bits = np.array([oracle.action_bit(1, e, t) for e in range(16) for t in range(1024)])
    assert abs(bits.mean() - 0.5) < 4 * 0.5 / np.sqrt(bits.size)
    # a rollout in this mode takes exactly these actions, and differs from the word stream
    a = oracle.OracleSim(oracle.CARTPOLE, 8, seed=1, action_stream=1).rollout(300)
    want = np.array([[oracle.action_bit(1, e, t) for e in range(8)] for t in range(300)], dtype=np.int8)
    assert np.array_equal(a["act"], want)
    b = oracle.OracleSim(oracle.CARTPOLE, 8, seed=1).rollout(300)
    assert not np.array_equal(a["act"], b["act"])
