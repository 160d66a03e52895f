"""Pins for the oracle's chunk codec (storage-mediated path, Section 4.4).

The checksum is held against zlib and the published Adler-32 example; the byte layout against
streams typed by hand from the format's description (not produced by any code of this
repository); the reader against the writer's inverse property and against corruption."""
import zlib

import numpy as np
import pytest

import oracle

# Worked example: list 0 = {(1, 0x3C00), (258, 0xBC01), (70000, 0x0001)}, list 1 empty,
# list 2 = {(7, 0x8000), (9, 0x7FC0)}; 8 entries per chunk -> one chunk per non-empty list.
LP = np.array([0, 3, 3, 5], np.uint64)
OFF = np.array([1, 258, 70000, 7, 9], np.uint32)
VAL = np.array([0x3C00, 0xBC01, 0x0001, 0x8000, 0x7FC0], np.uint16)


def _header(fmt, lst, first, count, payload):
    head = b"".join(int(w).to_bytes(4, "little") for w in [0x43455444, fmt, lst, first, count, len(payload)])
    return head + zlib.adler32(head + payload).to_bytes(4, "little") + bytes(4)


def _hand_stream_plain():
    # indices as little-endian int32, then values as little-endian BF16 patterns, zero fill to 16
    p0 = bytes.fromhex("01000000" "02010000" "70110100" "003c" "01bc" "0100") + bytes(14)
    p1 = bytes.fromhex("07000000" "09000000" "0080" "c07f") + bytes(4)
    assert len(p0) == 32 and len(p1) == 16
    return _header(0, 0, 0, 3, p0) + p0 + _header(0, 2, 0, 2, p1) + p1


def _hand_stream_planes():
    # six planes of 16 bytes: index bytes 0..3, value bytes 0..1
    def plane(*b):
        return bytes(b) + bytes(16 - len(b))
    p0 = (plane(0x01, 0x02, 0x70) + plane(0x00, 0x01, 0x11) + plane(0x00, 0x00, 0x01) + plane() +
          plane(0x00, 0x01, 0x01) + plane(0x3C, 0xBC, 0x00))
    p1 = (plane(0x07, 0x09) + plane() + plane() + plane() + plane(0x00, 0xC0) + plane(0x80, 0x7F))
    return _header(1, 0, 0, 3, p0) + p0 + _header(1, 2, 0, 2, p1) + p1


def _hand_stream_delta_planes():
    # as the byte planes, but the index planes hold 1, 258 - 1 = 257 = 0x101, 70000 - 258 = 69742 = 0x1106E
    def plane(*b):
        return bytes(b) + bytes(16 - len(b))
    p0 = (plane(0x01, 0x01, 0x6E) + plane(0x00, 0x01, 0x10) + plane(0x00, 0x00, 0x01) + plane() +
          plane(0x00, 0x01, 0x01) + plane(0x3C, 0xBC, 0x00))
    p1 = (plane(0x07, 0x02) + plane() + plane() + plane() + plane(0x00, 0xC0) + plane(0x80, 0x7F))
    return _header(2, 0, 0, 3, p0) + p0 + _header(2, 2, 0, 2, p1) + p1


def test_adler32_matches_zlib_and_the_published_example():
    assert oracle.adler32(b"Wikipedia") == 0x11E60398
    assert oracle.adler32(b"") == 1
    rng = np.random.default_rng(5)
    for n in (1, 2, 15, 16, 5551, 5552, 5553, 70000, 400000):
        data = rng.integers(0, 256, n, dtype=np.uint8).tobytes()
        assert oracle.adler32(data) == zlib.adler32(data)
    assert oracle.adler32(b"\xff" * 300000) == zlib.adler32(b"\xff" * 300000)


@pytest.mark.parametrize("fmt,hand", [(0, _hand_stream_plain), (1, _hand_stream_planes),
                                      (2, _hand_stream_delta_planes)])
def test_worked_example_matches_the_hand_typed_stream(fmt, hand):
    stream, directory = oracle.pack_chunks(LP, OFF, VAL, 8, fmt)
    expect = hand()
    assert stream.tobytes() == expect
    sizes = [64, 48] if fmt == 0 else [128, 128]      # header + payload of the two chunks
    assert directory.tolist() == [[0, 0, 0], [sizes[0], 2, 0], [sizes[0] + sizes[1], 0xFFFFFFFF, 0]]
    off, val, rejected, written = oracle.unpack_chunks(np.frombuffer(expect, np.uint8), directory, LP)
    assert rejected == 0 and written == 5
    assert np.array_equal(off, OFF) and np.array_equal(val, VAL)


def _random_lists(rng, n_lists, max_len):
    lens = rng.integers(0, max_len + 1, n_lists)
    lens[rng.integers(0, n_lists)] = 0
    lp = np.concatenate([[0], np.cumsum(lens)]).astype(np.uint64)
    off = np.concatenate([np.sort(rng.choice(1 << 26, int(n), replace=False)) for n in lens] +
                         [np.zeros(0, np.int64)]).astype(np.uint32)
    val = rng.integers(0, 1 << 16, off.size).astype(np.uint16)
    return lp, off, val


@pytest.mark.parametrize("fmt", [0, 1, 2])
@pytest.mark.parametrize("chunk_entries", [8, 16, 64, 4096])
def test_round_trip_and_structure(fmt, chunk_entries):
    rng = np.random.default_rng(100 + chunk_entries + fmt)
    lp, off, val = _random_lists(rng, 23, 300)
    stream, d = oracle.pack_chunks(lp, off, val, chunk_entries, fmt)
    n_chunks = d.shape[0] - 1
    lens = np.diff(lp).astype(np.int64)
    assert n_chunks == int(np.sum((lens + chunk_entries - 1) // chunk_entries))
    assert int(d[-1, 0]) == stream.size and np.all(d[:, 0] % 16 == 0)
    covered = np.zeros(int(lp[-1]), np.int32)
    for c in range(n_chunks):
        h = np.frombuffer(stream[int(d[c, 0]):int(d[c, 0]) + 32].tobytes(), "<u4")
        assert h[0] == 0x43455444 and h[1] == fmt and h[2] == d[c, 1] and h[3] == d[c, 2] and h[7] == 0
        count = int(h[4])
        assert 0 < count <= chunk_entries and int(h[3]) % chunk_entries == 0
        assert int(h[5]) == (-(-6 * count // 16) * 16 if fmt == 0 else 6 * (-(-count // 16) * 16))
        assert int(d[c + 1, 0] - d[c, 0]) == 32 + int(h[5])
        chunk = stream[int(d[c, 0]):int(d[c + 1, 0])].tobytes()
        assert int(h[6]) == zlib.adler32(chunk[:24] + chunk[32:])
        a = int(lp[int(h[2])]) + int(h[3])
        covered[a:a + count] += 1
    assert np.all(covered == 1)
    off2, val2, rejected, written = oracle.unpack_chunks(stream, d, lp)
    assert rejected == 0 and written == int(lp[-1])
    assert np.array_equal(off2, off) and np.array_equal(val2, val)


def test_all_formats_carry_the_same_entries():
    rng = np.random.default_rng(9)
    lp, off, val = _random_lists(rng, 7, 1000)
    off[-1] = 0xFFFFFFF0                                  # indices above 2^31 keep their bits
    a = oracle.unpack_chunks(*oracle.pack_chunks(lp, off, val, 64, 0), lp)
    for fmt in (1, 2):
        b = oracle.unpack_chunks(*oracle.pack_chunks(lp, off, val, 64, fmt), lp)
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    assert np.array_equal(a[0], off) and np.array_equal(a[1], val)


@pytest.mark.parametrize("fmt", [0, 1, 2])
def test_every_corrupted_payload_byte_and_header_field_is_rejected(fmt):
    stream, d = oracle.pack_chunks(LP, OFF, VAL, 8, fmt)
    first_chunk = slice(int(LP[0]), int(LP[1]))
    for pos in range(32, int(d[1, 0])):            # payload of chunk 0, padding included
        bad = stream.copy()
        bad[pos] ^= 0x40
        off, val, rejected, written = oracle.unpack_chunks(bad, d, LP)
        assert rejected == 1 and written == 2, pos
        assert not off[first_chunk].any() and np.array_equal(off[3:], OFF[3:])
    for pos in range(0, 28):                       # every checked header byte
        bad = stream.copy()
        bad[pos] ^= 0x01
        assert oracle.unpack_chunks(bad, d, LP)[2] == 1, pos
    bad_dir = d.copy()
    bad_dir[0, 2] = 8                              # directory and header disagree
    assert oracle.unpack_chunks(stream, bad_dir, LP)[2] == 1
    for row, value in ((1, int(d[1, 0]) + 8), (2, stream.size + 16), (1, 16)):
        bad_dir = d.copy()                         # chunk off its boundary / past the end / too short
        bad_dir[row, 0] = value
        assert oracle.unpack_chunks(stream, bad_dir, LP)[2] >= 1


def test_empty_delta_has_no_chunks():
    lp = np.zeros(5, np.uint64)
    stream, d = oracle.pack_chunks(lp, np.zeros(0, np.uint32), np.zeros(0, np.uint16), 64, 0)
    assert stream.size == 0 and d.tolist() == [[0, 0xFFFFFFFF, 0]]
    with pytest.raises(ValueError):
        oracle.pack_chunks(lp, np.zeros(0, np.uint32), np.zeros(0, np.uint16), 12, 0)


def test_byte_planes_and_gaps_compress_better_than_the_plain_layout():
    pa = pytest.importorskip("pyarrow")
    rng = np.random.default_rng(3)
    mask = rng.random(4_000_000) < 0.015            # the paper's change density
    off = np.nonzero(mask)[0].astype(np.uint32)
    w = (rng.standard_normal(off.size) * 0.02).astype(np.float32)
    val = oracle.bf16_rne(w)
    lp = np.array([0, off.size], np.uint64)
    size = {}
    for fmt in (0, 1, 2):
        stream, _ = oracle.pack_chunks(lp, off, val, 65536, fmt)
        size[fmt] = len(pa.compress(stream.tobytes(), codec="zstd", asbytes=True))
    assert size[1] < 0.7 * size[0]
    assert size[2] < 0.92 * size[1]                       # gaps instead of indices: smaller again
