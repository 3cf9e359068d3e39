"""Pins for the oracle's bit stream writer and reader: a hand-worked golden stream, exact
round trips over every layout parameter, and the accounting identities of the layout."""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "stream_8sym.txt")


def _read_golden():
    out = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        key, *vals = line.split()
        out[key] = [int(v, 0) for v in vals]
    return out


def test_golden_stream_by_hand():
    g = _read_golden()
    q = np.array(g["symbols"], dtype=np.uint8).reshape(4, 2)
    for splits, key in ((1, "chunk_len"), (2, "chunk_len_split2")):
        s = oracle.encode(q, np.array(g["lengths"]), 2, chunk_pixels=1, pixel_splits=splits, tile_pixels=2)
        assert s.words.tolist() == g["words"]
        assert s.chunk_len.tolist() == g[key]
        assert s.tile_off.tolist() == g["tile_off"]
        assert s.total_bits == 256
        assert np.array_equal(oracle.decode_symbols(s, np.array(g["lengths"]), 2), q)


@pytest.mark.parametrize("bits,k,per_channel,pixels,cp,splits,tp", [
    (1, 3, False, 17, 1, 1, 4), (2, 8, True, 64, 4, 1, 16), (4, 16, False, 130, 1, 2, 128),
    (5, 7, True, 257, 2, 1, 128), (8, 4, False, 300, 8, 1, 128), (8, 5, True, 33, 1, 1, 128),
    (3, 64, False, 129, 4, 1, 128), (4, 2, False, 1, 1, 2, 128), (6, 32, True, 200, 1, 4, 128),
])
def test_round_trip_and_accounting(bits, k, per_channel, pixels, cp, splits, tp):
    rng = np.random.default_rng(bits * 1000 + pixels)
    nsym = 1 << bits
    # skewed symbols so that code lengths differ
    q = np.minimum(rng.geometric(0.4, size=(pixels, k)) - 1, nsym - 1).astype(np.uint8)
    hist = oracle.histogram(q, bits, per_channel)
    ln = oracle.huffman_lengths(hist, 12)
    s = oracle.encode(q, ln, bits, chunk_pixels=cp, pixel_splits=splits, tile_pixels=tp)
    assert np.array_equal(oracle.decode_symbols(s, ln, bits), q)
    # accounting: tile payload = sum of code lengths of its pixels; tiles padded to 128 bits
    n_tiles = -(-pixels // tp)
    assert len(s.tile_off) == n_tiles + 1 and s.tile_off[0] == 0
    lens = np.stack([ln[j if per_channel else 0][q[:, j]] for j in range(k)], axis=1).astype(np.int64)
    per_pixel = lens.sum(axis=1)
    for t in range(n_tiles):
        payload = int(per_pixel[t * tp:(t + 1) * tp].sum())
        assert s.tile_off[t] % 128 == 0
        assert int(s.tile_off[t + 1] - s.tile_off[t]) == -(-payload // 128) * 128
    assert s.total_bits == int(s.tile_off[-1]) == 32 * len(s.words)
    # every chunk's length is the sum of the code lengths of its symbols (pixel-major order)
    cs = cp * k // splits
    flat = lens.reshape(-1)
    assert len(s.chunk_len) == -(-flat.shape[0] // cs)
    for c in range(len(s.chunk_len)):
        assert int(s.chunk_len[c]) == int(flat[c * cs:(c + 1) * cs].sum())
    # chunk starts: consecutive inside a tile, restarting at every tile
    starts = s.chunk_starts()
    cpt = tp * k // cs
    for c in range(len(s.chunk_len)):
        t = c // cpt
        assert int(starts[c]) == int(s.tile_off[t]) + int(flat[t * tp * k:c * cs].sum())


def test_wrong_chunk_length_is_corrupt():
    rng = np.random.default_rng(5)
    q = rng.integers(0, 4, size=(40, 8)).astype(np.uint8)
    ln = np.array([[1, 2, 3, 3]], dtype=np.uint8)
    s = oracle.encode(q, ln, 2, chunk_pixels=1, pixel_splits=2, tile_pixels=16)
    s.chunk_len = s.chunk_len.copy()
    s.chunk_len[5] += 1
    with pytest.raises(ValueError):
        oracle.decode_symbols(s, ln, 2)


def test_chunk_longer_than_16_bits_is_rejected():
    q = np.full((128, 64), 3, dtype=np.uint8)
    ln = np.array([[1, 2, 3, 12]], dtype=np.uint8)
    with pytest.raises(ValueError):
        oracle.encode(q, ln, 2, chunk_pixels=128, tile_pixels=128)      # 128 * 64 * 12 bits in one chunk


def test_corrupt_stream_is_reported_not_crashed():
    q = np.zeros((8, 4), dtype=np.uint8)
    ln = np.array([[1, 2, 3, 3]], dtype=np.uint8)
    s = oracle.encode(q, ln, 2, chunk_pixels=1, tile_pixels=8)
    s.words = s.words[:0]
    with pytest.raises(ValueError):
        oracle.decode_symbols(s, ln, 2)
