// Deflation of inactive variants - Phase 3, Module 7 (Model Deflater) and the inflation of
// Module 8 (Section III-E): a rebuilt variant still holds the zeroed weights of its surviving
// channels, and those repeat, so the variant is packed as a DEFLATE stream (RFC 1951) while it is
// not in use and unpacked when it is switched in.
//
// The stream is plain RFC 1951 (any inflater reads it); the encoder's free choices are made so
// that both directions run in parallel:
//   chunk      16384 input bytes = one block (fixed Huffman codes, or stored when that is shorter),
//              followed - unless it is the last - by an empty stored block, which puts the next
//              chunk on a byte boundary;
//   sub-block  512 input bytes: runs of equal bytes are coded as a literal plus matches at
//              distance 1 and never reach back across the start of a sub-block.
// One warp takes a chunk, one lane a sub-block.  Beside the stream the encoder writes the byte
// offset of every chunk and the bit offset of every sub-block, which is all the decoder needs to
// start 32 lanes per chunk at once.
//
//   k_deflate_encode  per chunk: count the bits of every sub-block, scan, then write the bits into the
//                     chunk's (zeroed) slot of the workspace;
//   k_deflate_scan    exclusive scan of the chunk sizes -> chunk offsets;
//   k_deflate_pack    moves every slot to its byte offset in the stream;
//   k_inflate         per group of chunks: stored chunks copied and the others zeroed by the whole block, then a
//                     thread per sub-block (taken in order of size) decodes it and stores the non-zero bytes.
#include "dnns_internal.cuh"

namespace dnns {

namespace {

constexpr uint32_t kChunk = DNNS_DEFLATE_CHUNK;
constexpr uint32_t kSub = DNNS_DEFLATE_SUB;
constexpr uint32_t kSubs = kChunk / kSub;           // 32: one lane each
constexpr uint32_t kSlotBytes = kChunk + 32;        // image of one chunk: at most 5 + 16384 bytes, padded
constexpr int kWarpsPerBlock = 4;
constexpr unsigned kFull = 0xffffffffu;

static_assert(kSubs == 32, "one lane per sub-block");

// ---- token costs and codes (RFC 1951, sections 3.2.5 and 3.2.6) ----
__device__ __forceinline__ uint32_t literal_bits(uint32_t v) { return v < 144 ? 8u : 9u; }

// A match of `len` (3..258) at distance 1: Huffman code of the length symbol (most significant bit
// first, hence reversed here), its extra bits, then the 5-bit distance code 0.  Returns the bit
// string (first bit = bit 0) and its length.
__device__ __forceinline__ uint32_t match_code(uint32_t len, uint32_t& n_bits) {
    const uint32_t x = len - 3;
    uint32_t sym, e = 0, extra = 0;
    if (len == 258) {
        sym = 285;
    } else if (x < 8) {
        sym = 257 + x;
    } else {
        e = (31 - __clz(x)) - 2;               // lengths come in groups of four codes per power of two
        sym = 257 + 4 * (e + 1) + ((x >> e) & 3u);
        extra = x & ((1u << e) - 1u);
    }
    uint32_t code, nb;
    if (sym <= 279) code = sym - 256, nb = 7;
    else code = 0xC0 + (sym - 280), nb = 8;
    n_bits = nb + e + 5;
    return (__brev(code) >> (32 - nb)) | (extra << nb);
}

__device__ __forceinline__ uint32_t literal_code(uint32_t v, uint32_t& n_bits) {
    if (v < 144) {
        n_bits = 8;
        return __brev(0x30 + v) >> 24;
    }
    n_bits = 9;
    return __brev(0x190 + (v - 144)) >> 23;
}

struct CountSink {
    uint32_t bits = 0;
    __device__ __forceinline__ void literal(uint32_t v, uint32_t times) { bits += times * literal_bits(v); }
    __device__ __forceinline__ void match(uint32_t len) {
        uint32_t n;
        match_code(len, n);
        bits += n;
    }
};

// Appends bit strings at a bit position of a zeroed image of the block.  Neighbouring lanes
// share the words at their borders, so words are merged with atomicOr (no value comes back).
struct WriteSink {
    uint32_t* words;
    uint32_t widx, fill;
    uint64_t acc = 0;
    __device__ __forceinline__ WriteSink(uint32_t* w, uint32_t bit_pos) : words(w), widx(bit_pos >> 5), fill(bit_pos & 31) {}
    __device__ __forceinline__ void put(uint32_t v, uint32_t n) {
        acc |= (uint64_t)v << fill;
        fill += n;
        if (fill >= 32) {
            atomicOr(&words[widx++], (uint32_t)acc);
            acc >>= 32;
            fill -= 32;
        }
    }
    __device__ __forceinline__ void literal(uint32_t v, uint32_t times) {
        uint32_t n;
        const uint32_t c = literal_code(v, n);
        for (uint32_t t = 0; t < times; ++t) put(c, n);
    }
    __device__ __forceinline__ void match(uint32_t len) {
        uint32_t n;
        const uint32_t c = match_code(len, n);
        put(c, n);
    }
    __device__ __forceinline__ void finish() {
        if (fill) atomicOr(&words[widx], (uint32_t)acc);
    }
};

// A run of `len` equal bytes: one literal, then its repeats as matches of 258, one shorter match
// when at least 3 repeats remain, else literals.
template <typename Sink>
__device__ __forceinline__ void emit_run(Sink& s, uint32_t v, uint32_t len) {
    uint32_t rep = len - 1;
    s.literal(v, 1);
    while (rep >= 258) {
        s.match(258);
        rep -= 258;
    }
    if (rep >= 3) s.match(rep);
    else if (rep) s.literal(v, rep);
}

// Bit i of the result: byte i of w differs from the byte before it (byte 0 from the top byte of `before`).
__device__ __forceinline__ uint32_t run_starts(uint32_t w, uint32_t before) {
    const uint32_t diff = w ^ __funnelshift_l(before, w, 8);  // every byte against its predecessor
    const uint32_t nz = (((diff & 0x7F7F7F7Fu) + 0x7F7F7F7Fu) | diff) & 0x80808080u;  // top bit of every non-zero byte
    return (((nz >> 7) * 0x00204081u) >> 21) & 0xFu;  // the four flags side by side
}

// Walk the n (<= 512) bytes of a sub-block at p (16-byte aligned) and hand its runs to the sink.  Sixteen
// bytes at a time: the positions where a run starts are found with word operations, and only those are
// visited (a lane steps from run to run, not from byte to byte).  Four vectors are always in flight.
template <typename Sink>
__device__ __forceinline__ void parse_sub_block(Sink& s, const uint8_t* p, uint32_t n) {
    uint32_t run_val = 0, run_start = 0;  // the open run: its byte and where it began
    bool open = false;
    const uint32_t n_vec = n / 16;
    const uint4* pv = reinterpret_cast<const uint4*>(p);
    const uint4 zero4 = make_uint4(0, 0, 0, 0);
    uint4 q0 = n_vec > 0 ? __ldg(pv) : zero4, q1 = n_vec > 1 ? __ldg(pv + 1) : zero4;
    uint4 q2 = n_vec > 2 ? __ldg(pv + 2) : zero4, q3 = n_vec > 3 ? __ldg(pv + 3) : zero4;
    uint32_t last = 0;  // the word before the current vector
    for (uint32_t v = 0; v < n_vec; ++v) {
        const uint4 q = q0;
        q0 = q1, q1 = q2, q2 = q3;
        if (v + 4 < n_vec) q3 = __ldg(pv + v + 4);
        uint32_t heads = run_starts(q.x, last) | (run_starts(q.y, q.x) << 4) | (run_starts(q.z, q.y) << 8) |
                         (run_starts(q.w, q.z) << 12);
        if (v == 0) heads |= 1u;  // the first byte of the sub-block always starts a run
        last = q.w;
        while (heads) {
            const uint32_t j = __ffs(heads) - 1;
            heads &= heads - 1;
            const uint32_t pos = v * 16 + j;
            if (open) emit_run(s, run_val, pos - run_start);
            const uint32_t word = j < 8 ? (j < 4 ? q.x : q.y) : (j < 12 ? q.z : q.w);
            run_val = (word >> (8 * (j & 3))) & 0xFFu;
            run_start = pos;
            open = true;
        }
    }
    for (uint32_t i = n_vec * 16; i < n; ++i) {  // only the very end of the data
        const uint32_t b = p[i];
        if (!open || b != run_val) {
            if (open) emit_run(s, run_val, i - run_start);
            run_val = b, run_start = i, open = true;
        }
    }
    if (open) emit_run(s, run_val, n - run_start);
}

// Bytes [4k, 4k+4) of a chunk of n bytes at p (4-byte aligned) as a word; bytes past the end read as 0.
__device__ __forceinline__ uint32_t chunk_word(const uint8_t* p, uint32_t n, uint32_t k) {
    if (4 * k + 4 <= n) return __ldg(reinterpret_cast<const uint32_t*>(p) + k);
    uint32_t w = 0;
    for (uint32_t j = 4 * k; j < n; ++j) w |= (uint32_t)p[j] << (8 * (j & 3));
    return w;
}

__global__ void __launch_bounds__(kWarpsPerBlock * 32) k_deflate_encode(const uint8_t* __restrict__ src, uint64_t n_bytes,
                                                                         uint32_t n_chunks, uint8_t* slots,
                                                                         uint32_t* sizes, uint32_t* sub_bits) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (uint32_t c = blockIdx.x * kWarpsPerBlock + warp; c < n_chunks; c += gridDim.x * kWarpsPerBlock) {
        const uint64_t c0 = (uint64_t)c * kChunk;
        const uint32_t n = (uint32_t)min((uint64_t)kChunk, n_bytes - c0);  // an empty input has one chunk of 0 bytes
        const bool last = c + 1 == n_chunks;
        const uint32_t lo = min(n, lane * kSub), n_lane = min(n - lo, kSub);
        const uint8_t* p = src + c0 + lo;

        CountSink cnt;
        parse_sub_block(cnt, p, n_lane);
        uint32_t incl = cnt.bits;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t y = __shfl_up_sync(kFull, incl, d);
            if (lane >= d) incl += y;
        }
        const uint32_t tokens = __shfl_sync(kFull, incl, 31);
        const uint32_t start = 3 + incl - cnt.bits;       // after the 3 header bits
        const uint32_t block_bits = 3 + tokens + 7;       // header, tokens, end-of-block symbol
        const uint32_t fixed_bytes = last ? (block_bits + 7) / 8 : (block_bits + 3 + 7) / 8 + 4;
        const uint32_t stored_bytes = 5 + n;
        const bool fixed = fixed_bytes <= stored_bytes;
        const uint32_t bytes = fixed ? fixed_bytes : stored_bytes;
        const uint32_t words = (bytes + 3) / 4;
        uint32_t* img = reinterpret_cast<uint32_t*>(slots + (size_t)c * kSlotBytes);  // the chunk's slot

        if (fixed) {
            for (uint32_t i = lane; i < words + 1; i += 32) img[i] = 0;
            __syncwarp();  // orders the zeroes before the other lanes' ORs
            WriteSink wr(img, start);
            if (lane == 0) atomicOr(&img[0], (last ? 1u : 0u) | 2u);  // BFINAL, BTYPE = 01 (low bit first)
            parse_sub_block(wr, p, n_lane);
            wr.finish();
            // the end-of-block symbol and the empty stored block's header are zero bits: already there
            if (!last && lane == 0) {
                const uint32_t at = bytes - 2;            // NLEN = 0xFFFF closes the empty stored block
                atomicOr(&img[at >> 2], 0xFFu << (8 * (at & 3)));
                atomicOr(&img[(at + 1) >> 2], 0xFFu << (8 * ((at + 1) & 3)));
            }
            sub_bits[(size_t)c * kSubs + lane] = start;
        } else {
            // stored: BFINAL / BTYPE 00 / padding in one byte, LEN, NLEN, then the chunk's bytes, which
            // sit 5 bytes into the image: image word j holds chunk bytes [4j - 5, 4j - 1)
            const uint8_t* q = src + c0;
            const uint32_t len = n & 0xFFFFu, nlen = ~n & 0xFFFFu;
            for (uint32_t j = lane; j < words + 1; j += 32) {
                uint32_t w;
                if (j == 0) w = (last ? 1u : 0u) | (len << 8) | (nlen << 24);
                else if (j == 1) w = (nlen >> 8) | (chunk_word(q, n, 0) << 8);
                else w = __funnelshift_r(chunk_word(q, n, j - 2), chunk_word(q, n, j - 1), 24);
                img[j] = w;
            }
            sub_bits[(size_t)c * kSubs + lane] = 8 * (5 + lo);
        }
        if (lane == 0) sizes[c] = bytes;
    }
}

__global__ void __launch_bounds__(1024) k_deflate_scan(const uint32_t* __restrict__ sizes, uint32_t n_chunks,
                                                       uint64_t* chunk_offset) {
    __shared__ uint64_t scratch[33];
    uint64_t carry = 0;
    for (uint32_t base = 0; base < n_chunks; base += 1024) {
        const uint32_t i = base + threadIdx.x;
        const uint64_t x = i < n_chunks ? sizes[i] : 0;
        uint64_t total;
        const uint64_t ex = block_exclusive_scan<uint64_t>(x, scratch, &total);
        if (i < n_chunks) chunk_offset[i] = carry + ex;
        carry += total;
        __syncthreads();
    }
    if (threadIdx.x == 0) chunk_offset[n_chunks] = carry;
}

// Word j of a byte string that starts `shift` bytes into aligned word array w.
__device__ __forceinline__ uint32_t unaligned_word(const uint32_t* w, uint32_t j, uint32_t shift) {
    return shift ? __funnelshift_r(w[j], w[j + 1], 8 * shift) : w[j];
}

__global__ void __launch_bounds__(kWarpsPerBlock * 32) k_deflate_pack(const uint8_t* __restrict__ slots,
                                                                       const uint32_t* __restrict__ sizes,
                                                                       const uint64_t* __restrict__ chunk_offset,
                                                                       uint32_t n_chunks, uint8_t* stream) {
    const int lane = threadIdx.x & 31;
    for (uint32_t c = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5); c < n_chunks; c += gridDim.x * kWarpsPerBlock) {
        const uint32_t* slot = reinterpret_cast<const uint32_t*>(slots + (size_t)c * kSlotBytes);
        const uint8_t* slot_b = reinterpret_cast<const uint8_t*>(slot);
        const uint32_t n = sizes[c];
        uint8_t* d = stream + chunk_offset[c];
        // bytes up to the first aligned destination word, then whole words, then the rest
        const uint32_t head = min(n, (uint32_t)((4 - (reinterpret_cast<uintptr_t>(d) & 3)) & 3));
        if ((uint32_t)lane < head) d[lane] = slot_b[lane];
        const uint32_t n_words = (n - head) / 4;
        uint32_t* dw = reinterpret_cast<uint32_t*>(d + head);
        for (uint32_t j = lane; j < n_words; j += 32) dw[j] = unaligned_word(slot, j, head);  // the slot has a spare word
        const uint32_t done = head + 4 * n_words;
        if (done + lane < n) d[done + lane] = slot_b[done + lane];
    }
}

// ---- the decoder
// What the next 9 stream bits (as a code, first bit on top) say, for all 512 values: bits the code takes, whether
// it is a literal (its value) or a length (base, number of extra bits), or something this decoder rejects.
//   bits 0..8   literal value, or length base - 3 (0..255)
//   bits 9..12  code bits (7, 8, 9)
//   bits 13..15 extra bits of a length
//   bit 16      length (a match follows); bit 17: rejected (end of block before the data is there, unassigned symbol)
__device__ __forceinline__ uint32_t token_entry(uint32_t code9) {
    uint32_t sym, used;
    if ((code9 >> 2) <= 0x17) sym = 256 + (code9 >> 2), used = 7;
    else if ((code9 >> 1) <= 0xBF) sym = (code9 >> 1) - 0x30, used = 8;
    else if ((code9 >> 1) <= 0xC7) sym = 280 + (code9 >> 1) - 0xC0, used = 8;
    else sym = 144 + code9 - 0x190, used = 9;
    if (sym < 256) return sym | (used << 9);
    const uint32_t idx = sym - 257;
    if (sym == 256 || idx > 28) return (used << 9) | (1u << 17);
    uint32_t base, e = 0;
    if (idx < 8) base = idx;
    else if (idx == 28) base = 255;
    else e = (idx >> 2) - 1, base = (4 + (idx & 3)) << e;
    return base | (used << 9) | (e << 13) | (1u << 16);
}

// A block takes groups of kGroup chunks, one sub-block per thread.  First all its threads prepare the group's
// destination together: a stored chunk is copied, a chunk of fixed Huffman codes is zeroed (whole lines).  The
// sub-blocks differ a lot in tokens - a dense one has 512 literals, a masked one a handful of matches - and the
// index says how many bits each one has, so the threads take them in order of size: the lanes of a warp then walk
// about equally many tokens, in one loop that is the same for literals and matches (read 32 bits at the lane's bit
// position, look the code up, advance).  Only non-zero bytes are stored: a match on a zero (nearly every match,
// the masked weights) just moves the output position on.
constexpr uint32_t kGroup = 4;
constexpr int kInflateThreads = kGroup * kSubs;

__global__ void __launch_bounds__(kInflateThreads) k_inflate(const uint32_t* __restrict__ stream_w, uint64_t stream_bytes,
                                                             const uint64_t* __restrict__ chunk_offset,
                                                             const uint32_t* __restrict__ sub_bits, uint64_t n_bytes,
                                                             uint32_t n_chunks, uint8_t* dst, uint32_t* status) {
    __shared__ uint32_t s_token[512];
    __shared__ uint64_t s_off[kGroup + 1];
    __shared__ uint32_t s_type[kGroup];  // 0 stored, 1 fixed Huffman, 3 nothing to decode (rejected)
    __shared__ uint32_t s_key[kInflateThreads];
    __shared__ uint16_t s_take[kInflateThreads];
    for (uint32_t r = threadIdx.x; r < 512; r += kInflateThreads) s_token[r] = token_entry(r);
    const uint64_t n_words = (stream_bytes + 3) / 4;
    auto word = [&](uint64_t i) -> uint32_t { return i < n_words ? __ldg(stream_w + i) : 0u; };
    auto fail = [&]() { atomicCAS(status, 0u, (uint32_t)DNNS_ERR_UNSUPPORTED); };
    const uint32_t n_groups = (n_chunks + kGroup - 1) / kGroup;
    for (uint32_t g = blockIdx.x; g < n_groups; g += gridDim.x) {
        const uint32_t c_first = g * kGroup, c_count = min(kGroup, n_chunks - c_first);
        __syncthreads();  // the previous group is done with the shared state
        if (threadIdx.x <= c_count) {
            const uint64_t off = chunk_offset[c_first + threadIdx.x];  // (the array has one entry past the last chunk)
            s_off[threadIdx.x] = off;
            if (threadIdx.x < c_count) {
                uint32_t type = 3;
                if (off < stream_bytes) type = ((word(off >> 2) >> (8 * (off & 3))) >> 1) & 3u;
                if (type >= 2) {
                    fail();
                    type = 3;
                }
                s_type[threadIdx.x] = type;
            }
        }
        __syncthreads();
        // ---- all threads: copy the stored chunks, zero the others
        for (uint32_t k = 0; k < c_count; ++k) {
            const uint64_t c0 = (uint64_t)(c_first + k) * kChunk;
            const uint32_t n = (uint32_t)min((uint64_t)kChunk, n_bytes - c0);
            uint8_t* chunk = dst + c0;
            if (s_type[k] == 0) {
                // the chunk's bytes start 5 bytes into its block
                const uint64_t a = s_off[k] + 5;
                const uint32_t shift = (uint32_t)(a & 3);
                const uint64_t w0 = a >> 2;
                for (uint32_t j = threadIdx.x; j < n / 4; j += kInflateThreads)
                    reinterpret_cast<uint32_t*>(chunk)[j] = shift ? __funnelshift_r(word(w0 + j), word(w0 + j + 1), 8 * shift) : word(w0 + j);
                for (uint32_t j = (n & ~3u) + threadIdx.x; j < n; j += kInflateThreads) {
                    const uint64_t b = a + j;
                    chunk[j] = (uint8_t)(word(b >> 2) >> (8 * (b & 3)));
                }
            } else if (s_type[k] == 1) {
                const uint32_t n_vec = n / 16;
                for (uint32_t j = threadIdx.x; j < n_vec; j += kInflateThreads) reinterpret_cast<uint4*>(chunk)[j] = make_uint4(0, 0, 0, 0);
                for (uint32_t j = n_vec * 16 + threadIdx.x; j < n; j += kInflateThreads) chunk[j] = 0;
            }
        }
        // ---- the sub-blocks in order of their size in the stream (0 where there is nothing to decode)
        {
            const uint32_t k = threadIdx.x / kSubs, sb = threadIdx.x % kSubs;
            uint32_t size = 0;
            if (k < c_count && s_type[k] == 1) {
                const uint32_t* bits = sub_bits + (size_t)(c_first + k) * kSubs;
                const uint64_t end = sb + 1 < kSubs ? bits[sb + 1] : (s_off[k + 1] - s_off[k]) * 8;
                const uint32_t start = bits[sb];
                size = end > start ? (uint32_t)min(end - start, (uint64_t)0xFFFFFFu) : 1u;
            }
            s_key[threadIdx.x] = (size << 8) | threadIdx.x;  // no two alike
        }
        __syncthreads();  // also orders the zeroes before the bytes
        {
            const uint32_t mine = s_key[threadIdx.x];
            uint32_t rank = 0;
            for (uint32_t j = 0; j < (uint32_t)kInflateThreads; ++j) rank += s_key[j] < mine;
            s_take[rank] = (uint16_t)threadIdx.x;
        }
        __syncthreads();
        const uint32_t which = s_take[threadIdx.x], k = which / kSubs, lane_sb = which % kSubs;
        bool busy = false;
        const uint32_t* wp = stream_w;   // stream words from the one with the chunk's first byte
        uint64_t w_left = 0;             // words from wp to the end of the stream
        uint8_t* out = nullptr;
        uint32_t n_lane = 0, pos = 0, acc = 0, prev = 0;
        // the bits ahead: at least 33 of them in buf at every token, the stream word after them already on its way
        uint64_t buf = 0;
        uint32_t have = 0, nxt = 0, wi = 0;
        auto stream_word = [&](uint32_t i) -> uint32_t { return i < w_left ? __ldg(wp + i) : 0u; };
        if (k < c_count && s_type[k] == 1) {
            const uint64_t c0 = (uint64_t)(c_first + k) * kChunk;
            const uint32_t n = (uint32_t)min((uint64_t)kChunk, n_bytes - c0);
            const uint32_t lo = min(n, lane_sb * kSub);
            n_lane = min(n - lo, kSub);
            const uint64_t off = s_off[k];
            out = dst + c0 + lo;
            wp = stream_w + (off >> 2);
            w_left = n_words - (off >> 2);
            const uint32_t bit = 8 * (uint32_t)(off & 3) + sub_bits[(size_t)(c_first + k) * kSubs + lane_sb];
            wi = bit >> 5;
            buf = (((uint64_t)stream_word(wi + 1) << 32) | stream_word(wi)) >> (bit & 31);
            have = 64 - (bit & 31);
            nxt = stream_word(wi + 2);
            wi += 3;
            busy = n_lane != 0;
        }
        while (__any_sync(kFull, busy)) {
            if (busy) {
                const uint32_t x = (uint32_t)buf;  // the next 32 stream bits
                const uint32_t t = s_token[__brev(x) >> 23];
                uint32_t used = (t >> 9) & 15u;
                if (t & (3u << 16)) {
                    // a length: extra bits, then the 5-bit distance code, which must say distance 1
                    const uint32_t e = (t >> 13) & 7u, rest = x >> used;
                    const uint32_t len = 3u + (t & 511u) + (rest & ((1u << e) - 1u));
                    used += e + 5;
                    if ((t >> 17) || ((rest >> e) & 31u) != 0 || pos == 0 || pos + len > n_lane) {
                        busy = false;
                        fail();
                    } else if (prev == 0) {
                        // zeros are there already; a word in the making is complete (the run covers its rest)
                        if (pos & 3) *reinterpret_cast<uint32_t*>(out + (pos & ~3u)) = acc, acc = 0;
                        pos += len;
                    } else {
                        for (uint32_t q = 0; q < len; ++q) {
                            acc |= prev << (8 * (pos & 3));
                            if ((++pos & 3) == 0) *reinterpret_cast<uint32_t*>(out + pos - 4) = acc, acc = 0;
                        }
                    }
                } else {
                    prev = t & 255u;
                    acc |= prev << (8 * (pos & 3));
                    if ((++pos & 3) == 0) {
                        if (acc) *reinterpret_cast<uint32_t*>(out + pos - 4) = acc;
                        acc = 0;
                    }
                }
                buf >>= used, have -= used;
                if (have <= 32) {
                    buf |= (uint64_t)nxt << have;
                    have += 32;
                    nxt = stream_word(wi++);
                }
                if (busy && pos >= n_lane) {
                    // the data may end inside a word
                    for (uint32_t j = 0; j < (pos & 3); ++j) out[(pos & ~3u) + j] = (uint8_t)(acc >> (8 * j));
                    busy = false;
                }
            }
        }
    }
}

int launch_deflate(const void* src, uint64_t n_bytes, uint32_t n_chunks, void* stream_out, uint64_t* chunk_offset,
                   uint32_t* sub_bits, void* ws, int n_sm, cudaStream_t st) {
    uint8_t* slots = static_cast<uint8_t*>(ws);
    uint32_t* sizes = reinterpret_cast<uint32_t*>(slots + (size_t)n_chunks * kSlotBytes);
    const uint32_t blocks = (n_chunks + kWarpsPerBlock - 1) / kWarpsPerBlock;
    const uint32_t grid = min(blocks, (uint32_t)n_sm * 16u * 8u);
    k_deflate_encode<<<grid, kWarpsPerBlock * 32, 0, st>>>(static_cast<const uint8_t*>(src), n_bytes, n_chunks, slots,
                                                              sizes, sub_bits);
    k_deflate_scan<<<1, 1024, 0, st>>>(sizes, n_chunks, chunk_offset);
    k_deflate_pack<<<grid, kWarpsPerBlock * 32, 0, st>>>(slots, sizes, chunk_offset, n_chunks,
                                                         static_cast<uint8_t*>(stream_out));
    return cudaGetLastError() == cudaSuccess ? 3 : -1;
}

size_t deflate_workspace_bytes(uint32_t n_chunks) { return (size_t)n_chunks * kSlotBytes + (((size_t)n_chunks * 4 + 255) & ~(size_t)255); }

int launch_inflate(const void* stream_in, uint64_t stream_bytes, const uint64_t* chunk_offset, const uint32_t* sub_bits,
                   uint64_t n_bytes, uint32_t n_chunks, void* dst, uint32_t* status, cudaStream_t st) {
    const uint32_t blocks = (n_chunks + kGroup - 1) / kGroup;
    k_inflate<<<blocks, kInflateThreads, 0, st>>>(static_cast<const uint32_t*>(stream_in), stream_bytes, chunk_offset,
                                                      sub_bits, n_bytes, n_chunks, static_cast<uint8_t*>(dst), status);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace

}  // namespace dnns

extern "C" {

size_t dnns_deflate_chunks(size_t n_bytes) { return n_bytes == 0 ? 1 : (n_bytes + DNNS_DEFLATE_CHUNK - 1) / DNNS_DEFLATE_CHUNK; }

size_t dnns_deflate_bound(size_t n_bytes) { return n_bytes + 5 * dnns_deflate_chunks(n_bytes); }

size_t dnns_deflate_workspace_bytes(size_t n_bytes) {
    return dnns::deflate_workspace_bytes((uint32_t)dnns_deflate_chunks(n_bytes));
}

static bool deflate_size_ok(size_t n_bytes) { return n_bytes <= ((size_t)1 << 40); }
static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

dnns_status dnns_deflate(const void* src_dev, size_t n_bytes, void* stream_dev, size_t stream_capacity,
                         uint64_t* chunk_offset_dev, uint32_t* sub_bits_dev, void* ws_dev, size_t ws_bytes, void* stream) {
    if (!stream_dev || !chunk_offset_dev || !sub_bits_dev || !ws_dev || (n_bytes && !src_dev)) return DNNS_ERR_INVALID_ARG;
    if (!aligned16(src_dev) || !aligned16(stream_dev) || !aligned16(ws_dev)) return DNNS_ERR_INVALID_ARG;
    if (!deflate_size_ok(n_bytes)) return DNNS_ERR_UNSUPPORTED;
    if (stream_capacity < ((dnns_deflate_bound(n_bytes) + 3) & ~(size_t)3) || ws_bytes < dnns_deflate_workspace_bytes(n_bytes))
        return DNNS_ERR_WORKSPACE;
    int dev = 0, n_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return DNNS_ERR_CUDA;
    const int n = dnns::launch_deflate(src_dev, n_bytes, (uint32_t)dnns_deflate_chunks(n_bytes), stream_dev, chunk_offset_dev,
                                       sub_bits_dev, ws_dev, n_sm, static_cast<cudaStream_t>(stream));
    return n < 0 ? DNNS_ERR_CUDA : DNNS_OK;
}

dnns_status dnns_inflate(const void* stream_dev, size_t stream_bytes, const uint64_t* chunk_offset_dev,
                         const uint32_t* sub_bits_dev, size_t n_bytes, void* dst_dev, uint32_t* status_dev, void* stream) {
    if (!stream_dev || !chunk_offset_dev || !sub_bits_dev || !status_dev || (n_bytes && !dst_dev)) return DNNS_ERR_INVALID_ARG;
    if (!aligned16(stream_dev) || !aligned16(dst_dev) || stream_bytes == 0) return DNNS_ERR_INVALID_ARG;
    if (!deflate_size_ok(n_bytes)) return DNNS_ERR_UNSUPPORTED;
    const int n = dnns::launch_inflate(stream_dev, stream_bytes, chunk_offset_dev, sub_bits_dev, n_bytes,
                                       (uint32_t)dnns_deflate_chunks(n_bytes), dst_dev, status_dev,
                                       static_cast<cudaStream_t>(stream));
    return n < 0 ? DNNS_ERR_CUDA : DNNS_OK;
}

}  // extern "C"
