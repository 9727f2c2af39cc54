// Steps 2 and 3.
//
//   mask       (Section III-C: the insignificant weights are set to zero, the sparse model keeps
//              its size) - a weight survives when its magnitude key is above tau, or equals tau
//              and at least n_tie equal keys precede it in its segment.  The per-tile tie tables
//              written by the threshold step tell every tile, without looking at any other
//              tile, whether its ties are all masked, all kept, or split (one tile per segment
//              at most, which then ranks its ties with a block scan).
//   structures (Module 2, Sparsity Analyser) in two kernels: the sweep over the weights packs one
//              "non-zero" bit per element into the workspace (32 times less data than the
//              weights, still in L2 when it is read back); k_flags turns those bits into the
//              all-zero 2-D kernels and from those into the filters (rows) and input columns that
//              still hold something.
//
// The sweep kernel runs either step alone or both at once (the non-zero bits are then taken from
// the masked values while they are still in registers).
#include "dnns_internal.cuh"

namespace dnns {

namespace {

constexpr unsigned kFull = 0xffffffffu;
DNNS_BOUNDS_COUNTER  // (checked build: index violations counted in this file)

// OR the per-lane bit groups (P bits each, lane order = element order) of 32/P neighbouring
// lanes into one word; every lane of the group gets the word.
template <int P>
__device__ __forceinline__ uint32_t gather_word(uint32_t bits, int lane) {
    constexpr int G = 32 / P;
    uint32_t v = bits << (P * (lane & (G - 1)));
#pragma unroll
    for (int d = 1; d < G; d <<= 1) v |= __shfl_xor_sync(kFull, v, d);
    return v;
}

// Any bit set in [lo, hi) of a packed bit array.
__device__ __forceinline__ bool any_bits(const uint32_t* bits, uint32_t lo, uint32_t hi) {
    uint32_t acc = 0;
    while (lo < hi) {
        const uint32_t off = lo & 31, n = min(32u - off, hi - lo);
        const uint32_t m = (n == 32 ? 0xffffffffu : ((1u << n) - 1u)) << off;
        acc |= bits[lo >> 5] & m;
        lo += n;
    }
    return acc != 0;
}

// The kernel-map word of 32 consecutive 3x3 kernels from their 288 element bits (9 words): the
// position of every 9-bit field is a compile-time constant, so a field costs a funnel shift, a
// mask and a compare.
__device__ __forceinline__ uint32_t kernel_word_3x3(const uint32_t* p) {
    uint32_t w[10];
#pragma unroll
    for (int i = 0; i < 9; ++i) w[i] = __ldg(p + i);
    w[9] = 0;
    uint32_t word = 0;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        const int idx = (9 * j) >> 5, off = (9 * j) & 31;
        const uint32_t field = __funnelshift_r(w[idx], w[idx + 1], off) & 0x1FFu;
        word |= field ? (1u << j) : 0u;
    }
    return word;
}

// OR `bits` into a global flag word unless they are already there.  The plain read may be stale,
// which only costs a redundant atomic; flags saturate early, so almost every update ends at the read.
__device__ __forceinline__ void or_if_missing(uint32_t* word, uint32_t bits) {
    if ((__ldcg(word) & bits) != bits) atomicOr(word, bits);
}

// From the packed element bits to kernel map, filter flags and input-column flags.
//
// Tensors whose filters are a power-of-two number of kernel-map words (I = 32, 64, 128, ...) are cut
// into units of kFlagRows filters x up to 32 map words per filter; one warp per unit.  In every
// step the 32 lanes build 32 consecutive words of the unit (a copy of the element bits for 1x1
// kernels, else one test per 2-D kernel) and store them plainly, as the unit owns them.  A lane
// always meets the same input-column word, so the column OR stays in a register until the end of
// the unit and costs one shuffle reduction and at most one atomic per word; filter flags cost at
// most one atomic per step.  This keeps the number of atomics on the few flag words small even
// though every unit of a tensor runs at the same time.
// Other shapes take units of 32 kernels, one per lane, each kernel setting its own two flags.
__global__ void __launch_bounds__(256) k_flags(Tables tb, const uint32_t* __restrict__ ebits_all, uint32_t* nz_map,
                                               uint32_t* out_nz, uint32_t* in_nz) {
    const int lane = threadIdx.x & 31;
    const uint32_t n_warps = gridDim.x * (blockDim.x >> 5), warp = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const uint32_t per = (tb.n_flag_units + n_warps - 1) / n_warps;
    const uint32_t lo = min(tb.n_flag_units, warp * per), hi = min(tb.n_flag_units, lo + per);
    if (lo >= hi) return;
    uint32_t t = tb.flag_unit_tensor[lo];  // the tensor holding unit lo
    uint32_t unit = lo;
    while (unit < hi) {
        const uint32_t t_begin = tb.flag_prefix[t], t_end = tb.flag_prefix[t + 1];
        if (unit >= t_end) {
            ++t;
            continue;
        }
        const TensorDesc& d = tb.tensors[t];
        const uint32_t KK = d.KK, I = d.I, O = d.O, n_kernels = O * I;
        const uint32_t* ebits = ebits_all + d.off_mask;
        const uint32_t n_ewords = (d.numel + 31) / 32, n_mwords = (n_kernels + 31) / 32;  // extents (checked build)
        (void)n_ewords, (void)n_mwords;
        uint32_t* g_in = in_nz + d.off_innz;
        uint32_t* g_out = out_nz + d.off_outnz;
        uint32_t* g_map = nz_map ? nz_map + d.off_nzmap : nullptr;
        const uint32_t wpr = (I % 32 == 0 && ((I / 32) & (I / 32 - 1)) == 0) ? I / 32 : 0;  // map words per filter
        const uint32_t run_end = min(hi, t_end);
        if (wpr) {
            const uint32_t n_chunks = (wpr + 31) / 32, cw = min(wpr, 32u);  // column chunks per filter block, words in each
            const int cw_shift = __ffs(cw) - 1;
            for (; unit < run_end; ++unit) {
                const uint32_t local = unit - t_begin, rb = local / n_chunks, cc = local - rb * n_chunks;
                const uint32_t row0 = rb * kFlagRows, iw = cc * 32 + (lane & (cw - 1));
                uint32_t acc = 0, rows = 0;  // column OR of this lane's words; filters of the unit that hold something
                constexpr int kMaxSteps = kFlagRows;  // cw <= 32 words per filter and chunk
                const uint32_t n_steps = (kFlagRows * cw + 31) / 32;
                // first all the words of the unit (their loads are independent and overlap) ...
                uint32_t words[kMaxSteps];
#pragma unroll
                for (int step = 0; step < kMaxSteps; ++step) {
                    words[step] = 0;
                    const uint32_t k = step * 32 + lane;
                    const uint32_t o = row0 + (k >> cw_shift);
                    if ((uint32_t)step < n_steps && k < kFlagRows * cw && o < O) {
                        const uint32_t gw = o * wpr + iw;  // this lane's word of the kernel map
                        uint32_t word = 0;
                        if (KK == 1) {
                            word = __ldg(ebits + DNNS_IDX(gw, n_ewords));
                        } else if (KK == 9) {
                            word = kernel_word_3x3(ebits + (DNNS_IDX(gw * 9 + 8, n_ewords) == gw * 9 + 8 ? (size_t)gw * 9 : (size_t)0));
                        } else {
                            const uint32_t q0 = gw * 32;
                            for (uint32_t j = 0; j < 32; ++j)
                                word |= (uint32_t)any_bits(ebits, (q0 + j) * KK, (q0 + j + 1) * KK) << j;
                        }
                        if (g_map) g_map[DNNS_IDX(gw, n_mwords)] = word;
                        words[step] = word;
                    }
                    acc |= words[step];
                }
                // ... then one vote per step: one bit per group of cw lanes = per filter of the step
                // (the trip count is the same in every lane)
                const uint32_t group_mask = cw == 32 ? 0xffffffffu : ((1u << cw) - 1u);
#pragma unroll
                for (int step = 0; step < kMaxSteps; ++step) {
                    if ((uint32_t)step >= n_steps) break;
                    const uint32_t nzl = __ballot_sync(kFull, words[step] != 0);
                    for (uint32_t g = 0; g < min(32u >> cw_shift, kFlagRows); ++g)
                        if ((nzl >> (g << cw_shift)) & group_mask) rows |= 1u << (((step * 32) >> cw_shift) + g);
                }
                // kFlagRows divides 32, so the filters of a unit share one flag word
                if (lane == 0 && rows) or_if_missing(&g_out[DNNS_IDX(row0 >> 5, (O + 31) / 32)], rows << (row0 & 31));
                for (uint32_t sft = cw; sft < 32; sft <<= 1) acc |= __shfl_xor_sync(kFull, acc, sft);
                if ((uint32_t)lane < cw && acc) or_if_missing(&g_in[DNNS_IDX(iw, (I + 31) / 32)], acc);
            }
        } else {
            // one kernel per lane, every kernel sets its own two flags
            for (; unit < run_end; ++unit) {
                const uint32_t q = (unit - t_begin) * 32 + lane;
                const bool bit = q < n_kernels && any_bits(ebits, q * KK, (q + 1) * KK);
                const uint32_t word = __ballot_sync(kFull, bit);
                if (lane == 0 && g_map) g_map[DNNS_IDX(unit - t_begin, n_mwords)] = word;
                if (bit) {
                    const uint32_t o = q / I, i = q - o * I;
                    or_if_missing(&g_in[DNNS_IDX(i >> 5, (I + 31) / 32)], 1u << (i & 31));
                    or_if_missing(&g_out[DNNS_IDX(o >> 5, (O + 31) / 32)], 1u << (o & 31));
                }
            }
        }
    }
}

// Each block owns a contiguous range of tiles.  Inside a tensor the loop is software-pipelined:
// the 16-byte loads of the next tile (and its two tie-table words) are issued before the current
// tile is processed, so a block always has a tile in flight while it masks and stores the
// previous one.  Whole tiles whose ties do not split take a lean path; the last
// (ragged) tile of a tensor and the one tile per segment that ranks its ties take the general one.
template <int DT, bool DO_MASK, bool DO_STRUCT>
__global__ void __launch_bounds__(kTileThreads, 4) k_sweep(Tables tb, ThresholdWs ws, const dnns_threshold* __restrict__ thr,
                                                           int variant, const char* src_arena, char* dst_arena,
                                                           uint32_t* mask_bits, uint32_t* clear_a, uint32_t n_clear_a,
                                                           uint32_t* clear_b, uint32_t n_clear_b) {
    constexpr int P = Elem<DT>::kPerVec;
    if (DO_STRUCT) {
        // the flag words that k_flags (the next kernel in the stream) ORs into start at zero
        for (uint32_t i = blockIdx.x * kTileThreads + threadIdx.x; i < n_clear_a; i += gridDim.x * kTileThreads) clear_a[i] = 0;
        for (uint32_t i = blockIdx.x * kTileThreads + threadIdx.x; i < n_clear_b; i += gridDim.x * kTileThreads) clear_b[i] = 0;
    }
    constexpr int G = 32 / P;  // lanes per bit word
    constexpr uint32_t kTileElems = kTileBytes / Elem<DT>::kBytes;
    constexpr uint32_t kKeyMask = DT == DNNS_F32 ? 0x7FFFFFFFu : 0x7FFF7FFFu;
    __shared__ uint32_t scratch[33];
    const int lane = threadIdx.x & 31;
    const bool word_lane = (lane & (G - 1)) == 0;

    const uint32_t per = (tb.n_tiles + gridDim.x - 1) / gridDim.x;
    const uint32_t lo = min(tb.n_tiles, blockIdx.x * per), hi = min(tb.n_tiles, lo + per);
    uint32_t tile = lo;
    while (tile < hi) {
        // ---- per-tensor context: constant over the run of tiles [tile, span_end)
        const TensorDesc& d = tb.tensors[tb.tile_tensor[tile]];
        const uint32_t span_end = min(hi, d.tile0 + d.n_tiles);
        const uint32_t numel = d.numel, tile0 = d.tile0;
        const char* src = src_arena ? src_arena + d.arena_off : static_cast<const char*>(d.src);
        char* dst = nullptr;
        // keep iff key >= thr_eff, except where the ties split; use_tables: thr_eff depends on the tile
        uint32_t tau = 0, thr_uniform = 0;
        uint64_t n_tie = 0;
        bool use_tables = false;
        if (DO_MASK) {
            dst = dst_arena ? dst_arena + d.arena_off : static_cast<char*>(const_cast<void*>(d.src));
            if (d.seg >= 0) {
                const dnns_threshold r = thr[(size_t)variant * tb.n_segs + d.seg];
                tau = r.tau_bits;
                n_tie = r.n_tie;
                if (r.n_below + r.n_tie == 0) thr_uniform = 0;                 // k = 0: keep everything
                else if (r.n_tie >= r.n_equal) thr_uniform = tau + 1;          // every key equal to tau is masked
                else use_tables = true;
            } else if (dst == src && !DO_STRUCT && !mask_bits) {
                tile = span_end;  // untouched tensor, in place, nothing else to produce
                continue;
            }
        }
        const uint32_t* tie_before = ws.tie_prefix + (size_t)variant * tb.n_tiles;
        const uint32_t* tie_here = ws.tile_ties + (size_t)variant * tb.n_tiles;
        uint32_t* mask_words = mask_bits ? mask_bits + d.off_mask : nullptr;
        uint32_t* nz_words = DO_STRUCT ? tb.ebits + d.off_mask : nullptr;  // same packing as the mask bits

        uint4 nxt[kVecPerThread];
        uint32_t nxt_before = 0, nxt_here = 0;
        auto issue = [&](uint32_t t) {
            const uint32_t e0 = (t - tile0) * kTileElems;
            if (e0 + kTileElems <= numel) {
                const uint4* p = reinterpret_cast<const uint4*>(src + (size_t)e0 * Elem<DT>::kBytes) + threadIdx.x;
#pragma unroll
                for (int u = 0; u < kVecPerThread; ++u) nxt[u] = DO_MASK ? p[u * kTileThreads] : __ldg(p + u * kTileThreads);
            } else {
#pragma unroll
                for (int u = 0; u < kVecPerThread; ++u)
                    load_vec<DT, !DO_MASK>(src, e0 + (u * kTileThreads + threadIdx.x) * P, numel, nxt[u]);
            }
            if (DO_MASK && use_tables) {
                nxt_before = tie_before[t];
                nxt_here = tie_here[t];
            }
        };
        issue(tile);
        for (; tile < span_end; ++tile) {
            uint4 v[kVecPerThread];
#pragma unroll
            for (int u = 0; u < kVecPerThread; ++u) v[u] = nxt[u];
            const uint32_t before = nxt_before, here = nxt_here;
            if (tile + 1 < span_end) issue(tile + 1);

            const uint32_t e0 = (tile - tile0) * kTileElems;
            const uint32_t n_e = min(kTileElems, numel - e0);
            // the one tile per segment where the ties split ranks them: those below `quota` are masked
            uint32_t thr_eff = thr_uniform, quota = 0;
            bool split = false;
            if (DO_MASK && use_tables) {
                if (before >= n_tie) thr_eff = tau;
                else if ((uint64_t)before + here <= n_tie) thr_eff = tau + 1;
                else {
                    thr_eff = tau + 1;
                    split = true;
                    quota = (uint32_t)(n_tie - before);
                }
            }

            if (n_e == kTileElems && !split) {
                // ---- lean path: a whole tile, one threshold for all its keys
                uint4* out = DO_MASK ? reinterpret_cast<uint4*>(dst + (size_t)e0 * Elem<DT>::kBytes) + threadIdx.x : nullptr;
                // survivors of a non-zero threshold are non-zero: their keep bits are their non-zero bits
                const bool zeros_survive = !DO_MASK || thr_eff == 0;
#pragma unroll
                for (int u = 0; u < kVecPerThread; ++u) {
                    const uint32_t vi = u * kTileThreads + threadIdx.x;
                    uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                    uint32_t keep = 0, nz = 0;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t m = w[j] & kKeyMask;
                        if (DT == DNNS_F32) {
                            const bool k = m >= thr_eff;
                            if (DO_MASK) {
                                w[j] = k ? w[j] : 0u;
                                keep |= k ? (1u << j) : 0u;
                            }
                            if (zeros_survive) nz |= m != 0 ? (1u << j) : 0u;
                        } else {
                            const uint32_t m0 = m & 0xFFFFu, m1 = m >> 16;
                            const bool k0 = m0 >= thr_eff, k1 = m1 >= thr_eff;
                            if (DO_MASK) {
                                w[j] &= (k0 ? 0x0000FFFFu : 0u) | (k1 ? 0xFFFF0000u : 0u);
                                keep |= (k0 ? (1u << (2 * j)) : 0u) | (k1 ? (2u << (2 * j)) : 0u);
                            }
                            if (zeros_survive) nz |= (m0 != 0 ? (1u << (2 * j)) : 0u) | (m1 != 0 ? (2u << (2 * j)) : 0u);
                        }
                    }
                    if (DO_MASK) {
                        out[u * kTileThreads] = make_uint4(w[0], w[1], w[2], w[3]);
                        if (zeros_survive) nz &= keep;
                    }
                    uint32_t keep_word = 0;
                    if (DO_MASK && (mask_words || (DO_STRUCT && !zeros_survive))) keep_word = gather_word<P>(keep, lane);
                    if (DO_MASK && mask_words && word_lane) mask_words[e0 / 32 + vi / G] = keep_word;
                    if (DO_STRUCT) {
                        const uint32_t nz_word = zeros_survive ? gather_word<P>(nz, lane) : keep_word;
                        if (word_lane) nz_words[e0 / 32 + vi / G] = nz_word;
                    }
                }
            } else {
                // ---- general path: ragged last tile of a tensor, or the tile whose ties split
                uint32_t tie_carry = 0;
#pragma unroll
                for (int u = 0; u < kVecPerThread; ++u) {
                    const uint32_t vi = u * kTileThreads + threadIdx.x;  // vector index inside the tile
                    const uint32_t e = e0 + vi * P;
                    const int n = e >= numel ? 0 : (int)min((uint32_t)P, numel - e);  // valid elements
                    uint32_t key[P];
                    vec_keys<DT>(v[u], key);
                    uint32_t keep = 0, nz = 0;
                    if (DO_MASK) {
                        uint32_t tie_rank = 0;
                        if (split) {
                            uint32_t c = 0;
#pragma unroll
                            for (int j = 0; j < P; ++j) c += (j < n && key[j] == tau);
                            uint32_t total;
                            tie_rank = tie_carry + block_exclusive_scan<uint32_t>(c, scratch, &total);
                            tie_carry += total;
                        }
#pragma unroll
                        for (int j = 0; j < P; ++j) {
                            bool k = key[j] >= thr_eff;
                            if (split && key[j] == tau) k = tie_rank++ >= quota;
                            k = k && j < n;
                            keep |= (uint32_t)k << j;
                            nz |= (uint32_t)(k && key[j] != 0) << j;
                        }
                        uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                        if (DT == DNNS_F32) {
#pragma unroll
                            for (int j = 0; j < 4; ++j) w[j] = (keep >> j) & 1u ? w[j] : 0u;
                        } else {
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const uint32_t m = ((keep >> (2 * j)) & 1u ? 0x0000FFFFu : 0u) |
                                                   ((keep >> (2 * j + 1)) & 1u ? 0xFFFF0000u : 0u);
                                w[j] &= m;
                            }
                        }
                        store_vec<DT>(dst, e, numel, make_uint4(w[0], w[1], w[2], w[3]));
                        if (mask_words) {
                            const uint32_t word = gather_word<P>(keep, lane);
                            if (word_lane && (vi / G) * 32 < n_e) mask_words[e0 / 32 + vi / G] = word;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < P; ++j) nz |= (uint32_t)(j < n && key[j] != 0) << j;
                    }
                    if (DO_STRUCT) {
                        const uint32_t word = gather_word<P>(nz, lane);
                        if (word_lane && (vi / G) * 32 < n_e) nz_words[e0 / 32 + vi / G] = word;
                    }
                }
            }
        }
    }
}


// The fused sweep for up to kMultiMax variants of one portfolio at once: every tile of the dense weights is
// read once and masked against each variant's threshold in turn, so a variant costs one write of the
// model plus 1/G of a read instead of a read and a write.  Same tile walk and the same two paths as
// k_sweep<mask, structures>; the per-variant state (threshold, tie tables, destinations) is an array.
// STORE = false: the masked weights are not written at all (the rebuild then masks the dense weights on its
// way, dnns_compact_masked); what remains are each variant's mask bits and element bits.
template <int DT, int G, bool STORE>
__global__ void __launch_bounds__(kTileThreads, (G == 1 || DT == DNNS_BF16) ? 4 : 3) k_sweep_multi(Tables tb, ThresholdWs ws, const dnns_threshold* __restrict__ thr,
                                                                 MultiSweepArgs ma, uint32_t n_clear_a, uint32_t n_clear_b) {
    constexpr int P = Elem<DT>::kPerVec;
    constexpr int GL = 32 / P;  // lanes per bit word
    constexpr uint32_t kTileElems = kTileBytes / Elem<DT>::kBytes;
    constexpr uint32_t kKeyMask = DT == DNNS_F32 ? 0x7FFFFFFFu : 0x7FFF7FFFu;
    __shared__ uint32_t scratch[33];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        for (uint32_t i = blockIdx.x * kTileThreads + threadIdx.x; i < n_clear_a; i += gridDim.x * kTileThreads) ma.clear_a[g][i] = 0;
        for (uint32_t i = blockIdx.x * kTileThreads + threadIdx.x; i < n_clear_b; i += gridDim.x * kTileThreads) ma.clear_b[g][i] = 0;
    }
    const int lane = threadIdx.x & 31;
    const bool word_lane = (lane & (GL - 1)) == 0;
    const uint32_t per = (tb.n_tiles + gridDim.x - 1) / gridDim.x;
    const uint32_t lo = min(tb.n_tiles, blockIdx.x * per), hi = min(tb.n_tiles, lo + per);
    uint32_t tile = lo;
    while (tile < hi) {
        const TensorDesc& d = tb.tensors[tb.tile_tensor[tile]];
        const uint32_t span_end = min(hi, d.tile0 + d.n_tiles);
        const uint32_t numel = d.numel, tile0 = d.tile0;
        const char* src = static_cast<const char*>(d.src);
        const uint64_t arena_off = d.arena_off;
        const uint32_t off_mask = d.off_mask;
        uint32_t tau[G], thr_uniform[G], n_tie[G];  // n_tie saturated to 32 bits: tile counts never reach it otherwise
        bool use_tables[G];
        bool any_tables = false;
#pragma unroll
        for (int g = 0; g < G; ++g) {
            tau[g] = thr_uniform[g] = n_tie[g] = 0;
            use_tables[g] = false;
            if (d.seg >= 0) {
                const dnns_threshold r = thr[(size_t)ma.variant[g] * tb.n_segs + d.seg];
                tau[g] = r.tau_bits;
                n_tie[g] = (uint32_t)min(r.n_tie, (uint64_t)0xFFFFFFFFu);
                if (r.n_below + r.n_tie == 0) thr_uniform[g] = 0;
                else if (r.n_tie >= r.n_equal) thr_uniform[g] = tau[g] + 1;
                else use_tables[g] = true;
                any_tables |= use_tables[g];
            }
        }
        uint4 nxt[kVecPerThread];
        uint32_t nxt_before[G], nxt_here[G];
#pragma unroll
        for (int g = 0; g < G; ++g) nxt_before[g] = nxt_here[g] = 0;
        auto issue = [&](uint32_t t) {
            const uint32_t e0 = (t - tile0) * kTileElems;
            if (e0 + kTileElems <= numel) {
                const uint4* p = reinterpret_cast<const uint4*>(src + (size_t)e0 * Elem<DT>::kBytes) + threadIdx.x;
#pragma unroll
                for (int u = 0; u < kVecPerThread; ++u) nxt[u] = __ldg(p + u * kTileThreads);
            } else {
#pragma unroll
                for (int u = 0; u < kVecPerThread; ++u)
                    load_vec<DT>(src, e0 + (u * kTileThreads + threadIdx.x) * P, numel, nxt[u]);
            }
            if (any_tables) {
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    if (use_tables[g]) {
                        nxt_before[g] = ws.tie_prefix[(size_t)ma.variant[g] * tb.n_tiles + t];
                        nxt_here[g] = ws.tile_ties[(size_t)ma.variant[g] * tb.n_tiles + t];
                    }
                }
            }
        };
        issue(tile);
        for (; tile < span_end; ++tile) {
            uint4 v[kVecPerThread];
#pragma unroll
            for (int u = 0; u < kVecPerThread; ++u) v[u] = nxt[u];
            uint32_t thr_eff[G], quota[G];
            bool any_split = false;
#pragma unroll
            for (int g = 0; g < G; ++g) {
                thr_eff[g] = thr_uniform[g];
                quota[g] = 0xFFFFFFFFu;  // no split
                if (use_tables[g]) {
                    const uint32_t before = nxt_before[g], here = nxt_here[g];
                    if (before >= n_tie[g]) thr_eff[g] = tau[g];
                    else {
                        thr_eff[g] = tau[g] + 1;
                        if ((uint64_t)before + here > n_tie[g]) {
                            quota[g] = n_tie[g] - before;  // this tile ranks its ties: those below quota are masked
                            any_split = true;
                        }
                    }
                }
            }
            if (tile + 1 < span_end) issue(tile + 1);

            const uint32_t e0 = (tile - tile0) * kTileElems;
            const uint32_t n_e = min(kTileElems, numel - e0);
            if (n_e == kTileElems && !any_split) {
                // ---- lean path: a whole tile, one threshold per variant
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    uint4* out = STORE ? reinterpret_cast<uint4*>(ma.dst[g] + arena_off + (size_t)e0 * Elem<DT>::kBytes) + threadIdx.x : nullptr;
                    uint32_t* mask_words = ma.mask_bits[g] ? ma.mask_bits[g] + off_mask : nullptr;
                    uint32_t* nz_words = ma.ebits[g] + off_mask;
                    const uint32_t te = thr_eff[g];
                    const uint32_t te2 = te * 0x00010001u;  // the threshold in both halves of a word (16-bit keys)
                    const bool zeros_survive = te == 0;
#pragma unroll
                    for (int u = 0; u < kVecPerThread; ++u) {
                        const uint32_t vi = u * kTileThreads + threadIdx.x;
                        uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                        uint32_t keep = 0, nz = 0;
                        if (DT == DNNS_F32) {
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const uint32_t m = w[j] & kKeyMask;
                                const bool k = m >= te;
                                w[j] = k ? w[j] : 0u;
                                keep |= k ? (1u << j) : 0u;
                                if (zeros_survive) nz |= m != 0 ? (1u << j) : 0u;
                            }
                        } else {
                            // Both 15-bit keys of a word at once: with bit 15 of each half set (the sign bits are
                            // not part of the key), subtracting the threshold leaves that bit standing exactly
                            // where key >= threshold, and no borrow crosses into the other half (te <= 0x8000).
                            // ge has the low key's flag at bit 0 and the high key's at bit 16; the eight flags of
                            // the vector are packed with three shifted adds and one fold.
                            uint32_t ge[4];
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                ge[j] = (((w[j] | 0x80008000u) - te2) >> 15) & 0x00010001u;
                                w[j] &= ge[j] * 0xFFFFu;
                            }
                            const uint32_t sk = ge[0] + (ge[1] << 2) + (ge[2] << 4) + (ge[3] << 6);
                            keep = (sk | (sk >> 15)) & 0xFFu;
                            if (zeros_survive) {  // te == 0: everything is kept, the non-zero flags are key >= 1
                                const uint32_t orig[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                                uint32_t sn = 0;
#pragma unroll
                                for (int j = 0; j < 4; ++j)
                                    sn += ((((orig[j] | 0x80008000u) - 0x00010001u) >> 15) & 0x00010001u) << (2 * j);
                                nz = (sn | (sn >> 15)) & 0xFFu;
                            }
                        }
                        if (STORE) out[u * kTileThreads] = make_uint4(w[0], w[1], w[2], w[3]);
                        // survivors of a non-zero threshold are non-zero: their keep bits are their non-zero bits
                        const uint32_t keep_word = (mask_words || !zeros_survive) ? gather_word<P>(keep, lane) : 0u;
                        const uint32_t nz_word = zeros_survive ? gather_word<P>(nz, lane) : keep_word;
                        if (word_lane) {
                            if (mask_words) mask_words[e0 / 32 + vi / GL] = keep_word;
                            nz_words[e0 / 32 + vi / GL] = nz_word;
                        }
                    }
                }
            } else {
                // ---- general path: ragged last tile of a tensor, or a tile that ranks the ties of some variant
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    char* dst = STORE ? ma.dst[g] + arena_off : nullptr;
                    uint32_t* mask_words = ma.mask_bits[g] ? ma.mask_bits[g] + off_mask : nullptr;
                    uint32_t* nz_words = ma.ebits[g] + off_mask;
                    const uint32_t te = thr_eff[g], tg = tau[g], qg = quota[g];
                    const bool split = qg != 0xFFFFFFFFu;
                    uint32_t tie_carry = 0;
#pragma unroll
                    for (int u = 0; u < kVecPerThread; ++u) {
                        const uint32_t vi = u * kTileThreads + threadIdx.x;
                        const uint32_t e = e0 + vi * P;
                        const int n = e >= numel ? 0 : (int)min((uint32_t)P, numel - e);
                        uint32_t key[P];
                        vec_keys<DT>(v[u], key);
                        uint32_t tie_rank = 0;
                        if (split) {
                            uint32_t c = 0;
#pragma unroll
                            for (int j = 0; j < P; ++j) c += (j < n && key[j] == tg);
                            uint32_t total;
                            tie_rank = tie_carry + block_exclusive_scan<uint32_t>(c, scratch, &total);
                            tie_carry += total;
                        }
                        uint32_t keep = 0, nz = 0;
#pragma unroll
                        for (int j = 0; j < P; ++j) {
                            bool k = key[j] >= te;
                            if (split && key[j] == tg) k = tie_rank++ >= qg;
                            k = k && j < n;
                            keep |= (uint32_t)k << j;
                            nz |= (uint32_t)(k && key[j] != 0) << j;
                        }
                        uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                        if (DT == DNNS_F32) {
#pragma unroll
                            for (int j = 0; j < 4; ++j) w[j] = (keep >> j) & 1u ? w[j] : 0u;
                        } else {
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                w[j] &= ((keep >> (2 * j)) & 1u ? 0x0000FFFFu : 0u) | ((keep >> (2 * j + 1)) & 1u ? 0xFFFF0000u : 0u);
                        }
                        if (STORE) store_vec<DT>(dst, e, numel, make_uint4(w[0], w[1], w[2], w[3]));
                        const uint32_t keep_word = gather_word<P>(keep, lane), nz_word = gather_word<P>(nz, lane);
                        if (word_lane && (vi / GL) * 32 < n_e) {
                            if (mask_words) mask_words[e0 / 32 + vi / GL] = keep_word;
                            nz_words[e0 / 32 + vi / GL] = nz_word;
                        }
                    }
                }
            }
        }
    }
}

template <int DT>
void launch_dt(bool do_mask, bool do_struct, dim3 grid, cudaStream_t st, const Tables& tb, const ThresholdWs& ws,
               const dnns_threshold* thr, int variant, const char* src_arena, char* dst_arena, uint32_t* mask_bits,
               uint32_t* out_nz, uint32_t n_out, uint32_t* in_nz, uint32_t n_in) {
    ScopedKernel timed(do_mask && do_struct ? "k_sweep<mask+structures>" : (do_mask ? "k_sweep<mask>" : "k_sweep<structures>"), st);
    if (do_mask && do_struct)
        k_sweep<DT, true, true><<<grid, kTileThreads, 0, st>>>(tb, ws, thr, variant, src_arena, dst_arena, mask_bits,
                                                               out_nz, n_out, in_nz, n_in);
    else if (do_mask)
        k_sweep<DT, true, false><<<grid, kTileThreads, 0, st>>>(tb, ws, thr, variant, src_arena, dst_arena, mask_bits,
                                                                nullptr, 0, nullptr, 0);
    else
        k_sweep<DT, false, true><<<grid, kTileThreads, 0, st>>>(tb, ws, thr, variant, src_arena, dst_arena, mask_bits,
                                                                out_nz, n_out, in_nz, n_in);
}

}  // namespace

int launch_tile_sweep(const Tables& tb, const ThresholdWs& ws, bool do_mask, bool do_struct,
                      const dnns_threshold* thr_dev, int variant, const void* src_arena, void* dst_arena,
                      uint32_t* mask_bits, uint32_t* nz_map, uint32_t* out_nz, uint32_t* in_nz, uint32_t n_out_words,
                      uint32_t n_in_words, int n_sm, cudaStream_t st) {
    const dim3 grid(min((uint32_t)n_sm * 4u, tb.n_tiles));
    if (tb.dtype == DNNS_F32)
        launch_dt<DNNS_F32>(do_mask, do_struct, grid, st, tb, ws, thr_dev, variant, (const char*)src_arena,
                            (char*)dst_arena, mask_bits, out_nz, n_out_words, in_nz, n_in_words);
    else
        launch_dt<DNNS_BF16>(do_mask, do_struct, grid, st, tb, ws, thr_dev, variant, (const char*)src_arena,
                             (char*)dst_arena, mask_bits, out_nz, n_out_words, in_nz, n_in_words);
    if (do_struct) {
        const uint32_t blocks = min((uint32_t)n_sm * 64u, (tb.n_flag_units + 7) / 8);  // one unit per warp if possible
        ScopedKernel timed("k_flags", st);
        k_flags<<<max(blocks, 1u), 256, 0, st>>>(tb, tb.ebits, nz_map, out_nz, in_nz);
    }
    return cudaGetLastError() == cudaSuccess ? (do_struct ? 2 : 1) : -1;
}


int launch_multi_sweep(const Tables& tb, const ThresholdWs& ws, const dnns_threshold* thr_dev, const MultiSweepArgs& ma,
                       int n_variants, uint32_t* const* nz_map, uint32_t n_out_words, uint32_t n_in_words, int n_sm,
                       cudaStream_t st) {
    const dim3 grid(min((uint32_t)n_sm * ((n_variants == 1 || tb.dtype == DNNS_BF16) ? 4u : 3u), tb.n_tiles));  // resident blocks per SM
    const bool store = ma.dst[0] != nullptr;
    {
        ScopedKernel timed(store ? "k_sweep_multi" : "k_sweep_bits", st);
#define DNNS_LAUNCH_MULTI(DT, G)                                                                                   \
    do {                                                                                                           \
        if (store) k_sweep_multi<DT, G, true><<<grid, kTileThreads, 0, st>>>(tb, ws, thr_dev, ma, n_out_words, n_in_words); \
        else k_sweep_multi<DT, G, false><<<grid, kTileThreads, 0, st>>>(tb, ws, thr_dev, ma, n_out_words, n_in_words);     \
    } while (0)
        if (tb.dtype == DNNS_F32) {
            if (n_variants == 1) DNNS_LAUNCH_MULTI(DNNS_F32, 1);
            else if (n_variants == 2) DNNS_LAUNCH_MULTI(DNNS_F32, 2);
            else if (n_variants == 3) DNNS_LAUNCH_MULTI(DNNS_F32, 3);
            else DNNS_LAUNCH_MULTI(DNNS_F32, 4);
        } else {
            if (n_variants == 1) DNNS_LAUNCH_MULTI(DNNS_BF16, 1);
            else if (n_variants == 2) DNNS_LAUNCH_MULTI(DNNS_BF16, 2);
            else if (n_variants == 3) DNNS_LAUNCH_MULTI(DNNS_BF16, 3);
            else DNNS_LAUNCH_MULTI(DNNS_BF16, 4);
        }
#undef DNNS_LAUNCH_MULTI
    }
    const uint32_t blocks = min((uint32_t)n_sm * 64u, (tb.n_flag_units + 7) / 8);
    for (int g = 0; g < n_variants; ++g) {
        ScopedKernel timed("k_flags", st);
        k_flags<<<max(blocks, 1u), 256, 0, st>>>(tb, ma.ebits[g], nz_map ? nz_map[g] : nullptr, ma.clear_a[g], ma.clear_b[g]);
    }
    return cudaGetLastError() == cudaSuccess ? 1 + n_variants : -1;
}

#ifdef DNNS_BOUNDS_CHECK
unsigned int bounds_violations_sweep(bool reset) {
    unsigned int n = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&n, g_bounds_violations, sizeof(n)) != cudaSuccess) return 0xFFFFFFFFu;
    if (reset) cudaMemcpyToSymbol(g_bounds_violations, &zero, sizeof(zero));
    return n;
}
#endif

}  // namespace dnns
