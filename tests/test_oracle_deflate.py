"""Pins for the oracle of the deflation step (Module 7 / Module 8, Section III-E; RFC 1951).

The encoder is pinned by an independent decoder (zlib inflates every stream back to the input) and
by streams and sizes counted by hand from the format (tests/golden/deflate_examples.txt); the decoder
by an independent encoder (zlib's own fixed-Huffman and stored streams)."""
import os
import zlib

import numpy as np
import pytest

from oracle import deflate_oracle as D

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "deflate_examples.txt")


def sparse_floats(rng, n_bytes, sparsity, dtype=np.float32):
    w = rng.standard_normal((n_bytes + 3) // 4 * 2).astype(np.float32)
    w[rng.random(w.size) < sparsity] = 0
    if dtype != np.float32:
        w = (w.view(np.uint32) >> 16).astype(np.uint16)
    return w.view(np.uint8)[:n_bytes].copy()


def inputs():
    rng = np.random.default_rng(7)
    for n in [0, 1, 2, 3, 4, 5, 258, 259, 260, 261, 262, 511, 512, 513, 1024, 16383, 16384, 16385, 40000, 70001]:
        yield f"zeros{n}", np.zeros(n, np.uint8)
        yield f"random{n}", rng.integers(0, 256, n, dtype=np.uint8)
        yield f"sparse_f32_{n}", sparse_floats(rng, n, 0.75)
        yield f"sparse_bf16_{n}", sparse_floats(rng, n, 0.6, np.uint16)
        yield f"runs{n}", np.repeat(rng.integers(0, 256, n // 5 + 1, dtype=np.uint8), rng.integers(1, 12, n // 5 + 1))[:n].copy()
    yield "ff_run", np.full(3000, 255, np.uint8)
    half = np.zeros(2 * D.CHUNK + 100, np.uint8)
    half[D.CHUNK:] = rng.integers(0, 256, D.CHUNK + 100, dtype=np.uint8)     # a fixed chunk, then stored chunks
    yield "fixed_then_stored", half


@pytest.mark.parametrize("name,data", list(inputs()), ids=[n for n, _ in inputs()])
def test_zlib_inflates_what_the_oracle_deflates(name, data):
    stream, chunk_offset, sub_bits = D.deflate(data)
    assert zlib.decompress(stream.tobytes(), wbits=-15) == data.tobytes()
    # the index: chunks in order, the last offset is the size, worst case respected
    n_chunks = max(1, -(-data.size // D.CHUNK))
    assert chunk_offset.size == n_chunks + 1 and chunk_offset[0] == 0 and chunk_offset[-1] == stream.size
    assert np.all(np.diff(chunk_offset.astype(np.int64)) > 0)
    assert stream.size <= data.size + 5 * n_chunks
    # every chunk decodes on its own from its byte offset (what makes chunk-parallel inflation possible):
    # a decoder started there reads that chunk's block first
    for c in range(n_chunks):
        d = zlib.decompressobj(wbits=-15)
        part = d.decompress(stream[int(chunk_offset[c]):].tobytes())
        assert part == data[c * D.CHUNK:].tobytes()
    assert sub_bits.size == n_chunks * D.SUBS_PER_CHUNK
    assert np.all(np.diff(sub_bits.reshape(n_chunks, -1).astype(np.int64), axis=1) >= 0)


def test_sub_block_offsets_start_tokens():
    """Decoding from a sub-block's bit offset yields that sub-block: re-align the bits behind a fresh
    fixed-block header and let zlib decode them."""
    rng = np.random.default_rng(3)
    data = sparse_floats(rng, 3 * D.CHUNK + 777, 0.8)
    stream, chunk_offset, sub_bits = D.deflate(data)
    bits = np.unpackbits(stream, bitorder="little")
    for c, s in [(0, 0), (0, 1), (0, 30), (1, 7), (2, 16), (3, 0), (3, 1)]:
        base = 8 * int(chunk_offset[c])
        start, end = (base + int(sub_bits[c * D.SUBS_PER_CHUNK + s + k]) for k in (0, 1))
        lo = c * D.CHUNK + s * D.SUB
        want = data[lo: min(lo + D.SUB, data.size)].tobytes()
        hdr = np.array([1, 1, 0], np.uint8)                       # BFINAL 1, BTYPE 01 (value 1, low bit first)
        eob = np.zeros(7, np.uint8)                               # symbol 256
        z = np.packbits(np.concatenate([hdr, bits[start:end], eob]), bitorder="little").tobytes()
        assert zlib.decompress(z, wbits=-15) == want


def test_oracle_inflates_zlib_streams():
    rng = np.random.default_rng(11)
    for n in [0, 1, 100, 5000, 70000]:
        a = np.repeat(rng.integers(0, 256, n // 3 + 1, dtype=np.uint8), 3)[:n].copy()
        a[::17] = 7
        c = zlib.compressobj(9, zlib.DEFLATED, -15, 9, zlib.Z_FIXED)        # fixed codes, matches at any distance
        z = c.compress(a.tobytes()) + c.flush()
        got = D.inflate(np.frombuffer(z, np.uint8), n)
        assert got is not None and got.tobytes() == a.tobytes()
        c = zlib.compressobj(0, zlib.DEFLATED, -15)                         # stored blocks
        z = c.compress(a.tobytes()) + c.flush()
        got = D.inflate(np.frombuffer(z, np.uint8), n)
        assert got is not None and got.tobytes() == a.tobytes()


def test_oracle_inflate_rejects_damage():
    data = np.zeros(5000, np.uint8)
    stream, _, _ = D.deflate(data)
    assert D.inflate(stream[:-1], 5000) is None                  # truncated
    assert D.inflate(stream, 4999) is None                       # output does not fit
    skewed = (np.random.default_rng(0).integers(0, 256, 20000, dtype=np.uint8) // 3).tobytes()
    dyn = zlib.compress(skewed, 9)[2:-4]                         # zlib picks dynamic codes here
    assert (dyn[0] >> 1) & 3 == 2 and D.inflate(np.frombuffer(dyn, np.uint8), 20000) is None


def test_hand_counted_streams_and_sizes():
    made = {"zeros16384": np.zeros(16384, np.uint8), "zeros32768": np.zeros(32768, np.uint8),
            "alt_low1000": np.tile(np.array([1, 2], np.uint8), 500),
            "alt_high1000": np.tile(np.array([200, 201], np.uint8), 500)}
    seen = 0
    for line in open(GOLDEN):
        p = line.split()
        if not p or p[0].startswith("#"):
            continue
        if p[0] == "stream":
            data = np.frombuffer(bytes.fromhex("" if p[1] == "-" else p[1]), np.uint8)
            stream, _, _ = D.deflate(data)
            assert stream.tobytes().hex() == p[2]
            assert zlib.decompress(bytes.fromhex(p[2]), wbits=-15) == data.tobytes()   # the hand count itself
        else:
            stream, _, _ = D.deflate(made[p[1]])
            assert stream.size == int(p[2]), p[1]
        seen += 1
    assert seen == 6


def test_sparser_is_smaller_and_dense_does_not_grow():
    """Section III-E: zeroed weights repeat, so sparse models deflate; dense ones gain nothing."""
    rng = np.random.default_rng(5)
    sizes = [D.deflate(sparse_floats(rng, 200000, s))[0].size for s in (0.0, 0.5, 0.75, 0.9, 0.98)]
    assert sizes == sorted(sizes, reverse=True)
    assert sizes[0] <= 200000 + 5 * 13 and sizes[-1] < 0.1 * 200000
