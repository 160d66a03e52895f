// CPU oracle for the chunk codec of the storage-mediated path.
//
// THIS IS TEST INFRASTRUCTURE, NOT PRODUCT CODE (see dte_oracle.cpp): a plain sequential
// writer and reader of the chunk stream, byte by byte, sharing nothing with the CUDA library.
//
// What the paper fixes (Section 4.4 and the evaluation's data-volume paragraph): nothing but
// the changed elements is written out, in chunks, four bytes of index and two bytes of BF16
// value per element, and a manifest says where each chunk lies, how long it is and what it must
// hash to.  The paper prints no byte layout, so the layout below is this build's reading of it:
//
//   stream  = chunks back to back, each starting on a 16-byte boundary
//   chunk   = 32-byte header + payload, covering at most C consecutive entries of ONE list
//             (lists in order, entries of a list in ascending order; an empty list has no chunk)
//   header  = eight little-endian uint32:
//             magic 0x43455444 ("DTEC"), format, list, first_entry (rank of the chunk's first
//             entry within its list), count, payload_bytes, checksum, 0
//   payload, format 0 (plain):  count x int32 index, then count x BF16 value, then zero bytes
//             up to a multiple of 16
//   payload, format 1 (byte planes): six planes of P = count rounded up to a multiple of 16
//             bytes each - byte 0, 1, 2, 3 of every index, then byte 0, 1 of every value - each
//             zero-padded to P.  Same information, transposed so that a byte-oriented
//             compressor sees the slowly varying high bytes together.
//   payload, format 2 (delta byte planes): as format 1, but the index planes hold the gaps
//             g_0 = index_0, g_i = index_i - index_{i-1} (entries of a list ascend, so gaps are
//             small and their upper planes are almost all zero); the reader restores the indices
//             by a running sum modulo 2^32.
//   checksum = Adler-32 (RFC 1950) of the first 24 header bytes followed by the payload
//             bytes, padding included (so a damaged count or list is caught as well)
//   directory entry per chunk = {byte offset in the stream, list, first_entry}; one more entry
//             at the end holds the stream's total size.
//
// Parity pins ("not gpu" tests): Adler-32 against zlib and the published "Wikipedia" vector;
// both formats against bytes typed by hand from the description above; unpack(pack(x)) == x;
// every single-byte corruption of a payload is rejected.

#include <cstdint>
#include <cstring>
#include <vector>

namespace {

constexpr uint32_t kMagic = 0x43455444u;
constexpr uint32_t kHeaderBytes = 32;

inline uint64_t round16(uint64_t x) { return (x + 15) / 16 * 16; }

constexpr uint32_t kFormats = 3;

inline uint64_t payload_bytes(uint64_t count, uint32_t format) {
    return format == 0 ? round16(6 * count) : 6 * round16(count);
}

inline void put_u32(uint8_t* p, uint32_t x) {
    p[0] = (uint8_t)(x & 0xFF);
    p[1] = (uint8_t)((x >> 8) & 0xFF);
    p[2] = (uint8_t)((x >> 16) & 0xFF);
    p[3] = (uint8_t)((x >> 24) & 0xFF);
}

inline uint32_t get_u32(const uint8_t* p) {
    return (uint32_t)p[0] | ((uint32_t)p[1] << 8) | ((uint32_t)p[2] << 16) | ((uint32_t)p[3] << 24);
}

// RFC 1950, section 8.2: s1 = 1 + sum of bytes, s2 = sum of the running s1, both mod 65521.
uint32_t adler32(const uint8_t* p, uint64_t n, uint32_t start = 1) {
    uint32_t s1 = start & 0xFFFFu, s2 = start >> 16;
    for (uint64_t i = 0; i < n; ++i) {
        s1 = (s1 + p[i]) % 65521u;
        s2 = (s2 + s1) % 65521u;
    }
    return (s2 << 16) | s1;
}

// Checksum of a chunk: the running Adler-32 over header bytes [0, 24), continued over the payload.
uint32_t chunk_checksum(const uint8_t* header, uint64_t pb) {
    return adler32(header + kHeaderBytes, pb, adler32(header, 24));
}

void write_payload(uint8_t* pay, const uint32_t* idx, const uint16_t* val, uint64_t count,
                   uint32_t format) {
    std::memset(pay, 0, payload_bytes(count, format));
    if (format == 0) {
        for (uint64_t i = 0; i < count; ++i) put_u32(pay + 4 * i, idx[i]);
        for (uint64_t i = 0; i < count; ++i) {
            pay[4 * count + 2 * i] = (uint8_t)(val[i] & 0xFF);
            pay[4 * count + 2 * i + 1] = (uint8_t)(val[i] >> 8);
        }
    } else {
        const uint64_t P = round16(count);
        for (uint64_t i = 0; i < count; ++i) {
            uint32_t x = idx[i];
            if (format == 2 && i > 0) x = idx[i] - idx[i - 1];   // the gap to the previous entry of the chunk
            for (int b = 0; b < 4; ++b) pay[b * P + i] = (uint8_t)((x >> (8 * b)) & 0xFF);
            pay[4 * P + i] = (uint8_t)(val[i] & 0xFF);
            pay[5 * P + i] = (uint8_t)(val[i] >> 8);
        }
    }
}

}  // namespace

extern "C" {

uint32_t oracle_adler32(const uint8_t* p, uint64_t n) { return adler32(p, n); }

// Serialises the lists.  Call with out == NULL to size: *n_chunks and the return value (stream
// bytes) are always exact.  dir: (n_chunks + 1) x 3 uint64 = {byte offset, list, first_entry};
// the last row is {total bytes, 0xFFFFFFFF, 0}.  Returns UINT64_MAX for a bad argument.
uint64_t oracle_pack_chunks(uint64_t n_lists, const uint64_t* list_ptr, const uint32_t* offsets,
                            const uint16_t* values, uint32_t chunk_entries, uint32_t format,
                            uint8_t* out, uint64_t* dir, uint64_t* n_chunks) {
    if (chunk_entries == 0 || chunk_entries % 8 != 0 || format >= kFormats) return UINT64_MAX;
    uint64_t bytes = 0, chunks = 0;
    for (uint64_t l = 0; l < n_lists; ++l) {
        const uint64_t n = list_ptr[l + 1] - list_ptr[l];
        for (uint64_t first = 0; first < n; first += chunk_entries) {
            const uint64_t count = n - first < chunk_entries ? n - first : chunk_entries;
            const uint64_t pb = payload_bytes(count, format);
            if (out) {
                uint8_t* h = out + bytes;
                uint8_t* pay = h + kHeaderBytes;
                write_payload(pay, offsets + list_ptr[l] + first, values + list_ptr[l] + first,
                              count, format);
                put_u32(h + 0, kMagic);
                put_u32(h + 4, format);
                put_u32(h + 8, (uint32_t)l);
                put_u32(h + 12, (uint32_t)first);
                put_u32(h + 16, (uint32_t)count);
                put_u32(h + 20, (uint32_t)pb);
                put_u32(h + 28, 0);
                put_u32(h + 24, chunk_checksum(h, pb));
            }
            if (dir) {
                dir[3 * chunks + 0] = bytes;
                dir[3 * chunks + 1] = l;
                dir[3 * chunks + 2] = first;
            }
            bytes += kHeaderBytes + pb;
            chunks += 1;
        }
    }
    if (dir) {
        dir[3 * chunks + 0] = bytes;
        dir[3 * chunks + 1] = 0xFFFFFFFFull;
        dir[3 * chunks + 2] = 0;
    }
    *n_chunks = chunks;
    return bytes;
}

// Reads a stream back into lists laid out by `list_ptr` (from the manifest).  A chunk is
// rejected, and none of its entries written, when the directory places it outside the stream
// or off a 16-byte boundary, when its header is inconsistent (magic, format, list or range
// outside the lists, payload size, chunk extent in the directory) or when the
// chunk's checksum differs from the header's.  Returns the number of rejected chunks;
// *entries_written counts the accepted entries.
uint64_t oracle_unpack_chunks(const uint8_t* stream, uint64_t stream_bytes, const uint64_t* dir,
                              uint64_t n_chunks, uint64_t n_lists, const uint64_t* list_ptr,
                              uint32_t* offsets, uint16_t* values, uint64_t* entries_written) {
    uint64_t rejected = 0, written = 0;
    for (uint64_t c = 0; c < n_chunks; ++c) {
        const uint64_t begin = dir[3 * c], end = dir[3 * (c + 1)];
        // the directory must place the chunk inside the stream, on a 16-byte boundary
        if (begin % 16 != 0 || end < begin || end - begin < kHeaderBytes || end > stream_bytes) {
            rejected += 1;
            continue;
        }
        const uint8_t* h = stream + begin;
        const uint64_t extent = end - begin;
        const uint32_t magic = get_u32(h), format = get_u32(h + 4), list = get_u32(h + 8);
        const uint32_t first = get_u32(h + 12), count = get_u32(h + 16), pb = get_u32(h + 20);
        const uint32_t sum = get_u32(h + 24);
        bool ok = magic == kMagic && format < kFormats && list < n_lists &&
                  count > 0;
        ok = ok && list == dir[3 * c + 1] && first == dir[3 * c + 2];
        ok = ok && (uint64_t)first + count <= list_ptr[list + 1] - list_ptr[list];
        ok = ok && pb == payload_bytes(count, format) && extent == kHeaderBytes + (uint64_t)pb;
        const uint8_t* pay = h + kHeaderBytes;
        ok = ok && chunk_checksum(h, pb) == sum;
        if (!ok) {
            rejected += 1;
            continue;
        }
        uint32_t* o = offsets + list_ptr[list] + first;
        uint16_t* v = values + list_ptr[list] + first;
        if (format == 0) {
            for (uint32_t i = 0; i < count; ++i) {
                o[i] = get_u32(pay + 4 * (uint64_t)i);
                v[i] = (uint16_t)(pay[4 * (uint64_t)count + 2 * i] |
                                  (pay[4 * (uint64_t)count + 2 * i + 1] << 8));
            }
        } else {
            const uint64_t P = round16(count);
            uint32_t running = 0;
            for (uint32_t i = 0; i < count; ++i) {
                const uint32_t x = (uint32_t)pay[i] | ((uint32_t)pay[P + i] << 8) |
                                   ((uint32_t)pay[2 * P + i] << 16) | ((uint32_t)pay[3 * P + i] << 24);
                running = format == 2 ? running + x : x;       // gaps add up to the index
                o[i] = running;
                v[i] = (uint16_t)(pay[4 * P + i] | (pay[5 * P + i] << 8));
            }
        }
        written += count;
    }
    *entries_written = written;
    return rejected;
}

}  // extern "C"
