"""Pins of the entropy-coding oracle (oracle/rans_oracle.cpp) against what the paper and the
mathematics fix: the rANS recurrences of App. A evaluated with unbounded Python integers, the
discrete logistic of Sec. 3 in float64, exact round trips, the code length against the ideal
-log2 p, and the block/stream partition against numpy slicing."""
import math

import numpy as np
import pytest

import iodf_synth as S
import oracle as O

M = 1 << 16
WIN = 2048


@pytest.fixture(scope="module")
def codec():
    return S.logistic_codec()


def _cf(codec, ls, r):
    k = int(np.clip(r, -WIN, WIN)) + WIN
    c = O.rans_cum(codec, ls, k)
    return c, O.rans_cum(codec, ls, k + 1) - c


def test_cumulative_counts_are_a_distribution(codec):
    for ls in range(64):
        cum = np.array([O.rans_cum(codec, ls, k) for k in range(2 * WIN + 2)], dtype=np.int64)
        assert cum[0] == 0 and cum[-1] == M
        assert np.all(np.diff(cum) >= 1)                       # every symbol can be coded


def test_frequencies_follow_the_discrete_logistic(codec):
    """Sec. 3: p(r) = sigma((r + 1/2)/s) - sigma((r - 1/2)/s). The table form deviates by the extra
    count per symbol, the rounding of G (1/2), the 1/64 grid of the sigmoid's argument (slope <= 1/4)
    and the rounding of the reciprocal scale (relative 1/(2 R), times max x sigma'(x) = 0.224)."""
    top = M - (2 * WIN + 1)
    rmin = float(codec["R"].min())
    tol = top * (1.0 / (4 * 64) + 0.224 * 0.5 / rmin) + 0.5 + 1e-6
    sig = lambda x: 1.0 / (1.0 + math.exp(-x)) if x > -700 else 0.0
    rng = np.random.default_rng(1)
    for _ in range(3000):
        ls = int(rng.integers(0, 64))
        s = float(codec["scales"][ls])
        r = int(rng.integers(-WIN + 1, WIN))
        k = r + WIN
        want = k + top * sig((r - 0.5) / s)                    # lower edge of symbol k
        assert abs(O.rans_cum(codec, ls, k) - want) <= tol
    # a sharp prior puts nearly all mass on r = 0, a flat one spreads it
    assert _cf(codec, 0, 0)[1] > 0.7 * M
    assert _cf(codec, 63, 0)[1] < 0.005 * M           # (one step of the 1/64 grid, 240 counts, lands here)


def test_streaming_state_equals_the_unbounded_recurrence_of_appendix_a(codec):
    """App. A: X_t = floor(X_{t-1} / F) M + C + (X_{t-1} mod F), decoded by s: C_s <= X_t mod M < C_s + F_s,
    X_{t-1} = floor(X_t / M) F + (X_t mod M) - C. While the state stays below 2^32 the streaming
    coder moves no word out and its final state is that recurrence started at X_0 = 2^16."""
    rng = np.random.default_rng(2)
    for trial in range(50):
        n = int(rng.integers(1, 24))
        ls = np.zeros(n, np.int32)                             # s = 0.25: r = 0 has p ~ 0.76
        mu = rng.integers(-1000, 1000, n).astype(np.int32)
        z = mu + (rng.random(n) < 0.1).astype(np.int32)        # mostly r = 0, some r = 1
        X = 1 << 16
        for i in range(n - 1, -1, -1):                         # the coder pushes last to first
            C, F = _cf(codec, 0, int(z[i] - mu[i]))
            X = (X // F) * M + C + (X % F)
        words = O.rans_encode_stream(codec, z, mu, ls)
        if X < (1 << 32):
            assert len(words) == 2 and int(words[0]) | (int(words[1]) << 16) == X
        # the decode equations take X back through the same symbols
        for i in range(n):
            slot = X % M
            r = next(r for r in (0, 1) if _cf(codec, 0, r)[0] <= slot < sum(_cf(codec, 0, r)))
            assert r == int(z[i] - mu[i])
            C, F = _cf(codec, 0, r)
            X = (X // M) * F + slot - C
        assert X == 1 << 16


def _draw(codec, rng, n, escapes=0.0):
    mu = rng.integers(-300, 300, n).astype(np.int32)
    ls = rng.integers(0, 64, n).astype(np.int32)
    r = np.round(rng.logistic(0.0, codec["scales"][ls])).astype(np.int64)
    far = rng.random(n) < escapes
    r[far] = rng.integers(-2**31 + 400, 2**31 - 400, int(far.sum()))
    z = np.clip(mu + r, -2**31, 2**31 - 1).astype(np.int32)
    return z, mu, ls


@pytest.mark.parametrize("n,escapes", [(0, 0.0), (1, 0.0), (257, 0.0), (1000, 0.05), (300, 1.0)])
def test_stream_round_trip(codec, n, escapes):
    rng = np.random.default_rng(10 + n)
    z, mu, ls = _draw(codec, rng, n, escapes)
    words = O.rans_encode_stream(codec, z, mu, ls)
    assert len(words) <= 3 * n + 2
    np.testing.assert_array_equal(O.rans_decode_stream(codec, words, mu, ls), z)


def test_edges_of_the_window_and_of_int32(codec):
    mu = np.array([0, 0, 0, 0, 5, -5, 2**31 - 1, -2**31], np.int32)
    z = np.array([2047, 2048, -2047, -2048, 2**31 - 1, -2**31, -2**31, 2**31 - 1], np.int32)
    ls = np.array([63, 63, 0, 0, 17, 17, 40, 40], np.int32)
    words = O.rans_encode_stream(codec, z, mu, ls)
    np.testing.assert_array_equal(O.rans_decode_stream(codec, words, mu, ls), z)
    # a truncated or altered stream is rejected or decodes to something else, never silently equal
    with pytest.raises(RuntimeError):
        O.rans_decode_stream(codec, words[:-1], mu, ls)


def test_code_length_is_close_to_the_ideal(codec):
    """Sum of -log2(F/M) over the symbols (32 bits more per escape), plus the 32-bit final state;
    16-bit renormalisation of a 32-bit state loses well under 0.1 %."""
    rng = np.random.default_rng(3)
    z, mu, ls = _draw(codec, rng, 20000, 0.01)
    ideal = 0.0
    for i in range(len(z)):
        r = int(z[i]) - int(mu[i])
        ideal += -math.log2(_cf(codec, int(ls[i]), r)[1] / M) + (32 if abs(r) >= WIN else 0)
    bits = 16 * len(O.rans_encode_stream(codec, z, mu, ls))
    assert ideal - 16 <= bits <= ideal * 1.001 + 48


def test_batch_partition_into_blocks_and_streams(codec):
    """Blocks in z order then the final block; stream j of a block holds elements j, j + ns, ...;
    a level without a prior head and the final block use mu = 0 and the fixed scale index."""
    model = S.make_model(0xC0DE, 3, 16, 16, [True, True, False], 1, 8)
    model["levels"][1]["prior"] = None                        # a split level with a fixed prior
    d = 3 * 16 * 16
    blocks = O.rans_blocks(model)
    assert blocks == [(0, 6 * 64, 0), (6 * 64, 12 * 16, -1), (6 * 64 + 12 * 16, 48 * 4, -1)]
    d_fact = 6 * 64
    rng = np.random.default_rng(4)
    B = 3
    z = rng.integers(-600, 600, (B, d)).astype(np.int32)
    prior = np.stack([rng.integers(-100, 100, (B, d_fact)), rng.integers(0, 64, (B, d_fact))], axis=1).astype(np.int32)
    small = dict(codec, elems_per_stream=100)
    words, counts = O.rans_encode(small, model, z, prior)
    s = 0
    for (zo, n, po) in blocks:
        ns = -(-n // 100)
        for j in range(ns):
            idx = np.arange(j, n, ns)
            mu = prior[:, 0, po + idx] if po >= 0 else np.zeros((B, len(idx)), np.int32)
            ls = prior[:, 1, po + idx] if po >= 0 else np.full((B, len(idx)), codec["final_ls"], np.int32)
            for b in range(B):
                w = O.rans_encode_stream(small, z[b, zo + idx], mu[b], ls[b])
                assert counts[b, s] == len(w)
                np.testing.assert_array_equal(words[b, s, :len(w)], w)
            s += 1
    assert s == words.shape[1]
    # block-wise decode, deepest block first, fills z back
    out = np.full_like(z, 12345)
    for q in range(len(blocks) - 1, -1, -1):
        O.rans_decode_block(small, model, words, counts, prior, q, out)
    np.testing.assert_array_equal(out, z)
