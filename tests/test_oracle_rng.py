"""Pins for the oracle's Philox4x32-10 and its counter layout (CPU only)."""
import os

import numpy as np
import pytest

import oracle


def _triton_philox(seed, c0, c1, c2, c3):
    """Philox4x32-10 as implemented by Triton's language library, run on the CPU
    by its interpreter: an implementation written by other people from the same
    published definition."""
    os.environ["TRITON_INTERPRET"] = "1"
    torch = pytest.importorskip("torch")
    triton = pytest.importorskip("triton")
    tl = pytest.importorskip("triton.language")

    @triton.jit
    def kern(out, seed, c0p, c1p, c2p, c3p, n: tl.constexpr):
        i = tl.arange(0, n)
        a, b, c, d = tl.philox(seed, tl.load(c0p + i), tl.load(c1p + i), tl.load(c2p + i),
                               tl.load(c3p + i))
        tl.store(out + i, a)
        tl.store(out + n + i, b)
        tl.store(out + 2 * n + i, c)
        tl.store(out + 3 * n + i, d)

    n = len(c0)
    out = torch.zeros(4 * n, dtype=torch.int32)
    args = [torch.from_numpy(np.asarray(c, dtype=np.uint32).view(np.int32).copy()) for c in (c0, c1, c2, c3)]
    kern[(1,)](out, seed, *args, n)
    return out.numpy().view(np.uint32).reshape(4, n).T


def test_philox_matches_independent_implementation():
    rng = np.random.default_rng(123)
    n = 1024
    for seed in (0, 1, 0xDEADBEEF, 0x0123456789ABCDEF, 2 ** 63 - 1):
        ctr = rng.integers(0, 2 ** 32, size=(n, 4), dtype=np.uint64).astype(np.uint32)
        ctr[0] = 0
        ctr[1] = 0xFFFFFFFF
        ctr[2] = (1, 0, 0, 0)
        ctr[3] = (0, 0, 0, 1)
        # no skip here: if the independent implementation cannot run, the generator is unpinned and the run
        # must not pass as if it had been checked
        ref = _triton_philox(seed, ctr[:, 0], ctr[:, 1], ctr[:, 2], ctr[:, 3])
        key = [seed & 0xFFFFFFFF, seed >> 32]
        for i in range(n):
            assert (oracle.philox(ctr[i], key) == ref[i]).all(), (seed, i)


def test_word_layout():
    # word(seed, gen, row, col, stream) = output word col%4 of
    # counter (col/4, row, gen low, stream + 16*gen high), key = (seed low, seed high)
    rng = np.random.default_rng(5)
    for _ in range(200):
        seed = int(rng.integers(0, 2 ** 63)) * 2 + int(rng.integers(0, 2))
        gen = int(rng.integers(0, 2 ** 40))
        row = int(rng.integers(0, 2 ** 32))
        col = int(rng.integers(0, 2 ** 20))
        stream = int(rng.integers(0, 4))
        out = oracle.philox([col >> 2, row, gen & 0xFFFFFFFF, stream | ((gen >> 32) << 4)],
                            [seed & 0xFFFFFFFF, seed >> 32])
        assert oracle.word(seed, gen, row, col, stream) == int(out[col & 3])


def test_streams_rows_generations_are_distinct():
    base = oracle.word(7, 3, 11, 5, oracle.STREAM_MUT)
    others = {oracle.word(8, 3, 11, 5, oracle.STREAM_MUT), oracle.word(7, 4, 11, 5, oracle.STREAM_MUT),
              oracle.word(7, 3, 12, 5, oracle.STREAM_MUT), oracle.word(7, 3, 11, 6, oracle.STREAM_MUT),
              oracle.word(7, 3, 11, 5, oracle.STREAM_SEL_A), oracle.word(7 + 2 ** 32, 3, 11, 5, oracle.STREAM_MUT),
              oracle.word(7, 3 + 2 ** 32, 11, 5, oracle.STREAM_MUT)}
    assert base not in others and len(others) == 7


def test_word_statistics():
    ws = np.array([oracle.word(99, 1, r, c, oracle.STREAM_MUT) for r in range(64) for c in range(256)],
                  dtype=np.uint64)
    n = ws.size
    # mean of a uniform 32-bit word, 5 sigma
    assert abs(ws.mean() / 2 ** 32 - 0.5) < 5 * (1 / 12) ** 0.5 / n ** 0.5
    for bit in (0, 1, 15, 16, 31):
        ones = int(((ws >> np.uint64(bit)) & np.uint64(1)).sum())
        assert abs(ones - n / 2) < 5 * (n / 4) ** 0.5
