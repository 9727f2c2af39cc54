/* CPU oracle for the deflation of inactive variants (TEST INFRASTRUCTURE, not a product path).
 *
 * Only the test-suite, the smoke check and the benchmark's CPU-baseline leg use this file.  It is
 * a plain, sequential, byte-at-a-time restatement and shares nothing with the CUDA library.
 *
 * What it restates.  Phase 3, Module 7 (Model Deflater) packs the pruned variants with the
 * lossless DEFLATE format (RFC 1951); Module 8 inflates one of them again.  The zeroed weights
 * that survive the rebuild repeat, which is what makes the variants compressible (Section III-E).
 *
 *   orc_deflate  writes an RFC 1951 stream for a byte buffer.  The format leaves the choice of
 *                matches and block types to the encoder; the choices made here are the reading
 *                this build fixes (stated below), so that an encoder is a function of its input.
 *   orc_inflate  a sequential RFC 1951 decoder for stored and fixed-Huffman blocks with matches
 *                at any distance (it is not tied to the choices of orc_deflate).
 *
 * Encoder choices (the reading):
 *   - The input is cut into chunks of 16384 bytes.  A chunk becomes one block: fixed Huffman
 *     codes (BTYPE 01) unless that is longer than a stored block (BTYPE 00) of the same bytes.
 *     Every block but the last is followed by an empty stored block (3 header bits, padding to a
 *     byte boundary, LEN = 0, NLEN = 0xFFFF), so every chunk starts on a byte boundary.  The last
 *     block has BFINAL set.  An empty input is one (final) chunk of no bytes.
 *   - A chunk is cut into sub-blocks of 512 bytes.  Inside a sub-block, every maximal run of L
 *     equal bytes is coded as one literal followed by its L-1 repeats: first as many matches of
 *     (length 258, distance 1) as fit, then one match (length rem, distance 1) when rem >= 3 repeats
 *     remain, else rem literals.  Nothing refers back across the start of a sub-block.
 *   - Beside the stream: the byte offset of every chunk and, per sub-block, the bit offset (from
 *     its chunk's first byte) at which its first token starts (stored chunk: where its bytes start).
 *
 * Pins (CPU tests): zlib inflates every stream orc_deflate writes back to the input; orc_inflate
 * decodes streams written by zlib's own fixed-Huffman encoder; hand-counted sizes of all-zero and
 * incompressible inputs.  The paper prints no compressed sizes for synthetic data: against the
 * paper itself, parity is unpinned.
 */
#include <stdint.h>
#include <stddef.h>
#include <string.h>

#define CHUNK 16384u
#define SUB 512u
#define SUBS_PER_CHUNK (CHUNK / SUB)

/* RFC 1951, section 3.2.5: base length and extra bits of length codes 257..285 */
static const unsigned len_base[29] = {3, 4, 5, 6, 7, 8, 9, 10, 11, 13, 15, 17, 19, 23, 27, 31,
                                      35, 43, 51, 59, 67, 83, 99, 115, 131, 163, 195, 227, 258};
static const unsigned len_extra[29] = {0, 0, 0, 0, 0, 0, 0, 0, 1, 1, 1, 1, 2, 2, 2, 2,
                                       3, 3, 3, 3, 4, 4, 4, 4, 5, 5, 5, 5, 0};
/* base distance and extra bits of distance codes 0..29 */
static const unsigned dist_base[30] = {1, 2, 3, 4, 5, 7, 9, 13, 17, 25, 33, 49, 65, 97, 129, 193, 257, 385,
                                       513, 769, 1025, 1537, 2049, 3073, 4097, 6145, 8193, 12289, 16385, 24577};
static const unsigned dist_extra[30] = {0, 0, 0, 0, 1, 1, 2, 2, 3, 3, 4, 4, 5, 5, 6, 6, 7, 7,
                                        8, 8, 9, 9, 10, 10, 11, 11, 12, 12, 13, 13};

/* ---- bit writer: bits fill each byte from its least significant bit (section 3.1.1) ---- */
typedef struct {
    uint8_t* out; /* NULL: only count */
    uint64_t bit; /* next bit position */
} bitw;

static void put_bit(bitw* w, unsigned b) {
    if (w->out) {
        if ((w->bit & 7) == 0) w->out[w->bit >> 3] = 0;
        w->out[w->bit >> 3] |= (uint8_t)((b & 1u) << (w->bit & 7));
    }
    w->bit++;
}
/* data elements other than Huffman codes: least significant bit first */
static void put_bits_lsb(bitw* w, unsigned v, unsigned n) {
    for (unsigned i = 0; i < n; ++i) put_bit(w, (v >> i) & 1u);
}
/* Huffman codes: most significant bit first */
static void put_code(bitw* w, unsigned code, unsigned n) {
    for (unsigned i = n; i-- > 0;) put_bit(w, (code >> i) & 1u);
}
static void pad_to_byte(bitw* w) {
    while (w->bit & 7) put_bit(w, 0);
}

/* fixed Huffman code of a literal/length symbol 0..287 (section 3.2.6) */
static void put_litlen_symbol(bitw* w, unsigned s) {
    if (s <= 143) put_code(w, 0x30 + s, 8);
    else if (s <= 255) put_code(w, 0x190 + (s - 144), 9);
    else if (s <= 279) put_code(w, s - 256, 7);
    else put_code(w, 0xC0 + (s - 280), 8);
}

static void put_match(bitw* w, unsigned length, unsigned distance) {
    unsigned c = 28;
    while (len_base[c] > length) --c; /* the last code whose base does not exceed the length (258 has its own) */
    put_litlen_symbol(w, 257 + c);
    put_bits_lsb(w, length - len_base[c], len_extra[c]);
    unsigned d = 29;
    while (dist_base[d] > distance) --d;
    put_code(w, d, 5);
    put_bits_lsb(w, distance - dist_base[d], dist_extra[d]);
}

/* tokens of one sub-block */
static void put_sub_block(bitw* w, const uint8_t* p, size_t n) {
    size_t i = 0;
    while (i < n) {
        size_t j = i + 1;
        while (j < n && p[j] == p[i]) ++j;
        size_t repeats = j - i - 1;
        put_litlen_symbol(w, p[i]);
        while (repeats >= 258) {
            put_match(w, 258, 1);
            repeats -= 258;
        }
        if (repeats >= 3) put_match(w, (unsigned)repeats, 1);
        else
            for (size_t r = 0; r < repeats; ++r) put_litlen_symbol(w, p[i]);
        i = j;
    }
}

/* One chunk as a fixed-Huffman block (plus the empty stored block when it is not the last one).
 * sub_bits (nullable) receives the start of every sub-block.  Returns the bytes used. */
static size_t fixed_chunk(const uint8_t* p, size_t n, int last, uint8_t* out, uint32_t* sub_bits) {
    bitw w = {out, 0};
    put_bit(&w, last ? 1 : 0);
    put_bits_lsb(&w, 1, 2);
    for (unsigned s = 0; s < SUBS_PER_CHUNK; ++s) {
        size_t lo = (size_t)s * SUB < n ? (size_t)s * SUB : n;
        size_t hi = lo + SUB < n ? lo + SUB : n;
        if (sub_bits) sub_bits[s] = (uint32_t)w.bit;
        put_sub_block(&w, p + lo, hi - lo);
    }
    put_litlen_symbol(&w, 256);
    if (!last) {
        put_bit(&w, 0);
        put_bits_lsb(&w, 0, 2);
        pad_to_byte(&w);
        put_bits_lsb(&w, 0x0000, 16);
        put_bits_lsb(&w, 0xFFFF, 16);
    } else {
        pad_to_byte(&w);
    }
    return (size_t)(w.bit >> 3);
}

size_t orc_deflate_n_chunks(size_t n) { return n == 0 ? 1 : (n + CHUNK - 1) / CHUNK; }

/* worst case: every chunk stored */
size_t orc_deflate_bound(size_t n) { return n + 5 * orc_deflate_n_chunks(n); }

/* src[n] -> stream (capacity orc_deflate_bound(n)); chunk_offset[n_chunks + 1]; sub_bits[32 * n_chunks].
 * Returns the stream size in bytes. */
size_t orc_deflate(const uint8_t* src, size_t n, uint8_t* stream, uint64_t* chunk_offset, uint32_t* sub_bits) {
    const size_t n_chunks = orc_deflate_n_chunks(n);
    size_t pos = 0;
    for (size_t c = 0; c < n_chunks; ++c) {
        const uint8_t* p = src + c * CHUNK;
        const size_t len = n - c * CHUNK < CHUNK ? n - c * CHUNK : CHUNK;
        const int last = c + 1 == n_chunks;
        chunk_offset[c] = pos;
        const size_t fixed_bytes = fixed_chunk(p, len, last, NULL, NULL);
        const size_t stored_bytes = 5 + len;
        if (fixed_bytes <= stored_bytes) {
            pos += fixed_chunk(p, len, last, stream + pos, sub_bits + c * SUBS_PER_CHUNK);
        } else {
            bitw w = {stream + pos, 0};
            put_bit(&w, last ? 1 : 0);
            put_bits_lsb(&w, 0, 2);
            pad_to_byte(&w);
            put_bits_lsb(&w, (unsigned)len, 16);
            put_bits_lsb(&w, (unsigned)len ^ 0xFFFFu, 16);
            memcpy(stream + pos + 5, p, len);
            for (unsigned s = 0; s < SUBS_PER_CHUNK; ++s) {
                size_t lo = (size_t)s * SUB < len ? (size_t)s * SUB : len;
                sub_bits[c * SUBS_PER_CHUNK + s] = (uint32_t)(8 * (5 + lo));
            }
            pos += stored_bytes;
        }
    }
    chunk_offset[n_chunks] = pos;
    return pos;
}

/* ---- sequential decoder ---- */
typedef struct {
    const uint8_t* in;
    size_t n_in;
    uint64_t bit;
    int overrun;
} bitr;

static unsigned get_bit(bitr* r) {
    if ((r->bit >> 3) >= r->n_in) {
        r->overrun = 1;
        return 0;
    }
    unsigned b = (r->in[r->bit >> 3] >> (r->bit & 7)) & 1u;
    r->bit++;
    return b;
}
static unsigned get_bits_lsb(bitr* r, unsigned n) {
    unsigned v = 0;
    for (unsigned i = 0; i < n; ++i) v |= get_bit(r) << i;
    return v;
}

/* read one fixed-Huffman literal/length symbol: extend the code bit by bit until it is one of the
 * four ranges of section 3.2.6 */
static int get_litlen_symbol(bitr* r) {
    unsigned code = 0;
    for (unsigned n = 1; n <= 9; ++n) {
        code = (code << 1) | get_bit(r);
        if (n == 7 && code <= 0x17) return 256 + (int)code;
        if (n == 8 && code >= 0x30 && code <= 0xBF) return (int)(code - 0x30);
        if (n == 8 && code >= 0xC0 && code <= 0xC7) return 280 + (int)(code - 0xC0);
        if (n == 9 && code >= 0x190) return 144 + (int)(code - 0x190);
    }
    return -1;
}

/* Returns the bytes written, or -1 on a malformed / unsupported stream or too small a buffer. */
long long orc_inflate(const uint8_t* stream, size_t n_stream, uint8_t* dst, size_t cap) {
    bitr r = {stream, n_stream, 0, 0};
    size_t out = 0;
    for (;;) {
        const unsigned final = get_bit(&r);
        const unsigned type = get_bits_lsb(&r, 2);
        if (r.overrun) return -1;
        if (type == 0) {
            while (r.bit & 7) get_bit(&r);
            const unsigned len = get_bits_lsb(&r, 16), nlen = get_bits_lsb(&r, 16);
            if (r.overrun || (len ^ 0xFFFFu) != nlen) return -1;
            if ((r.bit >> 3) + len > n_stream || out + len > cap) return -1;
            memcpy(dst + out, stream + (r.bit >> 3), len);
            out += len;
            r.bit += 8ull * len;
        } else if (type == 1) {
            for (;;) {
                const int s = get_litlen_symbol(&r);
                if (s < 0 || r.overrun) return -1;
                if (s == 256) break;
                if (s < 256) {
                    if (out >= cap) return -1;
                    dst[out++] = (uint8_t)s;
                    continue;
                }
                if (s > 285) return -1;
                const unsigned length = len_base[s - 257] + get_bits_lsb(&r, len_extra[s - 257]);
                unsigned d = 0;
                for (int i = 0; i < 5; ++i) d = (d << 1) | get_bit(&r);
                if (d > 29) return -1;
                const unsigned distance = dist_base[d] + get_bits_lsb(&r, dist_extra[d]);
                if (r.overrun || distance > out || out + length > cap) return -1;
                for (unsigned i = 0; i < length; ++i, ++out) dst[out] = dst[out - distance];
            }
        } else {
            return -1; /* dynamic Huffman blocks are not produced by orc_deflate */
        }
        if (final) break;
    }
    return (long long)out;
}
