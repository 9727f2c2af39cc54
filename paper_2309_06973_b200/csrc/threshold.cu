// Step 1: exact k-th-magnitude threshold (the ranking of Phase 1, Section III-C) as a radix
// select over magnitude keys, for all prune counts of a portfolio at once.
//
//   pass 1  one sweep over the weights: histogram of the top 15 key bits per segment, kept in
//           128 KB of shared memory per block and merged into global memory on segment change;
//   select1 per segment: prefix sums of the histogram locate, for every k, the first-digit
//           bucket of the k-th key.  A 15-bit key (bf16) is finished here;
//   pass 2  (31-bit keys) second sweep: keys whose first digit was selected by some variant are
//           counted by their low 16 bits in a per-(segment, digit) global histogram;
//   select2 locates the low digit: tau, n_below, n_equal, n_tie;
//   ties    a sweep that counts, per 16 KB tile, the keys equal to tau_v - only run when some
//           variant must mask part of the weights equal to tau (n_tie < n_equal); followed by
//           an exclusive scan per (variant, segment).  The mask kernel then needs no ordering
//           between tiles to mask exactly k weights.  The scan kernel also finds, for such a
//           variant, the position (tensor, element) of the first weight equal to tau that stays:
//           every equal weight before it is masked, every one from it on is kept.
#include "dnns_internal.cuh"

namespace dnns {

namespace {

constexpr int kHistThreads = 1024;

// Bit `i` of a 32768-bit bitmap in shared memory, i = the 15 bits of x starting at bit SHIFT.
template <int SHIFT>
__device__ __forceinline__ uint32_t bitmap_test(const uint32_t* bm, uint32_t x) {
    return (bm[(x >> (SHIFT + 5)) & 0x3FFu] >> ((x >> SHIFT) & 31u)) & 1u;
}

// Walk the block's contiguous share of the tile list.  For every run of tiles of one prunable
// tensor: on_span(d) (block-uniform, may synchronise; false skips the run), then
// on_tile(tile, n_e, v) per tile (n_e valid elements; vectors past the end hold zeros), with the
// next tile's loads already in flight.
template <int DT, typename SpanFn, typename TileFn>
__device__ __forceinline__ void walk_prunable_tiles(const Tables& tb, SpanFn on_span, TileFn on_tile) {
    constexpr int P = Elem<DT>::kPerVec;
    constexpr uint32_t kTileElems = kTileBytes / Elem<DT>::kBytes;
    const uint32_t per = (tb.n_tiles + gridDim.x - 1) / gridDim.x;
    const uint32_t lo = min(tb.n_tiles, blockIdx.x * per), hi = min(tb.n_tiles, lo + per);
    uint32_t tile = lo;
    while (tile < hi) {
        const TensorDesc& d = tb.tensors[tb.tile_tensor[tile]];
        const uint32_t span_end = min(hi, d.tile0 + d.n_tiles);
        if (d.seg < 0 || !on_span(d)) {
            tile = span_end;
            continue;
        }
        const uint32_t numel = d.numel, tile0 = d.tile0;
        const char* src = static_cast<const char*>(d.src);
        uint4 nxt[kVecPerThread];
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
        };
        issue(tile);
        for (; tile < span_end; ++tile) {
            uint4 v[kVecPerThread];
#pragma unroll
            for (int u = 0; u < kVecPerThread; ++u) v[u] = nxt[u];
            if (tile + 1 < span_end) issue(tile + 1);
            on_tile(tile, min(kTileElems, numel - (tile - tile0) * kTileElems), v);
        }
    }
}

// The keys of a tile that pass a bitmap filter: f(key, element offset in the tile) is called by the thread holding the key.
// SHIFT32 / the two 16-bit halves select which 15 bits of a stored word index the bitmap.
template <int DT, int SHIFT32, typename F>
__device__ __forceinline__ void for_filtered_keys(const uint4 (&v)[kVecPerThread], uint32_t n_e, const uint32_t* bm, F f) {
    constexpr int P = Elem<DT>::kPerVec;
    constexpr uint32_t kTileElems = kTileBytes / Elem<DT>::kBytes;
#pragma unroll
    for (int u = 0; u < kVecPerThread; ++u) {
        const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
        uint32_t hits = 0;
        if (DT == DNNS_F32) {
#pragma unroll
            for (int j = 0; j < 4; ++j) hits |= bitmap_test<SHIFT32>(bm, w[j]) << j;
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                hits |= (bitmap_test<0>(bm, w[j]) << (2 * j)) | (bitmap_test<16>(bm, w[j]) << (2 * j + 1));
        }
        if (n_e != kTileElems) {  // ragged tile: drop the slots past the end of the tensor
            const uint32_t first = (u * kTileThreads + threadIdx.x) * P;
            hits &= first >= n_e ? 0u : (n_e - first >= (uint32_t)P ? 0xFFu : ((1u << (n_e - first)) - 1u));
        }
        while (hits) {
            const int j = __ffs(hits) - 1;
            hits &= hits - 1;
            uint32_t x = DT == DNNS_F32 ? j : j >> 1;
            x = x == 0 ? w[0] : (x == 1 ? w[1] : (x == 2 ? w[2] : w[3]));
            f(DT == DNNS_F32 ? (x & 0x7FFFFFFFu) : ((x >> (16 * (j & 1))) & 0x7FFFu), (uint32_t)((u * kTileThreads + threadIdx.x) * P + j));
        }
    }
}

// ---------------------------------------------------------------- select 1
// One block per segment (or the last block of the first sweep, segment after segment).
// Prune counts handed over as a kernel argument (no copy to stage, nothing to capture but the launch).
constexpr int kInlineCounts = 64;
struct InlineCounts {
    uint64_t k[kInlineCounts];
};

// What select 1 keeps in shared memory.
struct Select1Shared {
    uint64_t scratch[33];
    uint64_t k[kMaxVariants];
    uint32_t digit[kMaxVariants];
};

// The selection for one segment, by all 1024 threads of a block (the block of k_select1, or the block of the first
// sweep that finished last).
template <int DT>
__device__ __forceinline__ void select1_segment(const Tables& tb, const ThresholdWs& ws, uint32_t seg, int n_k,
                                                dnns_threshold* __restrict__ thr, const InlineCounts& counts,
                                                bool counts_inline, Select1Shared& sm) {
    uint64_t* const scratch = sm.scratch;
    uint64_t* const s_k = sm.k;
    uint32_t* const s_digit = sm.digit;
    const uint32_t S = tb.n_segs;
    if ((int)threadIdx.x < n_k) {
        const size_t idx = (size_t)threadIdx.x * S + seg;
        s_k[threadIdx.x] = counts_inline ? counts.k[idx] : ws.k_dev[idx];  // one round trip for all k
        s_digit[threadIdx.x] = 0xFFFFFFFFu;  // stays so if no bin reaches rank k (weights rewritten under the sweep): nothing selected
    }
    // A warp owns 1024 consecutive bins = 256 vectors of four; a lane loads vectors lane, lane + 32, .. of them, so
    // that every load of the warp is one contiguous 512 bytes (a thread reading its own 32 consecutive bins would
    // touch 32 lines per load, and one SM keeps only so many requests in flight).  Bin order inside the warp: group
    // j (32 vectors), lane, element.  (A segment holds fewer than 2^32 keys: 32-bit sums.)
    const uint32_t* h = ws.hist1 + (size_t)seg * kHistBins;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint4* hv = reinterpret_cast<const uint4*>(h) + warp * 256;
    uint32_t c[32], gs[8], before[8];  // the lane's bins; the sum of its vector in group j; keys of the warp before that vector
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint4 v = __ldcg(hv + j * 32 + lane);  // (written by other blocks' atomics)
        c[4 * j] = v.x, c[4 * j + 1] = v.y, c[4 * j + 2] = v.z, c[4 * j + 3] = v.w;
        gs[j] = v.x + v.y + v.z + v.w;
    }
    uint32_t warp_sum = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        uint32_t incl = gs[j];
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t y = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += y;
        }
        before[j] = warp_sum + incl - gs[j];
        warp_sum += __shfl_sync(0xffffffffu, incl, 31);
    }
    uint64_t total;
    const uint64_t warp_base = __shfl_sync(0xffffffffu, block_exclusive_scan<uint64_t>(lane == 0 ? warp_sum : 0u, scratch, &total), 0);
    uint32_t* bm = ws.bitmap + (size_t)seg * kBitmapWords;
    bm[threadIdx.x] = 0;  // 1024 words
    for (int v = 0; v < n_k; ++v) {
        const uint64_t k = s_k[v];  // published by the barriers of the scan above
        SelectState* st = &ws.sel[(size_t)v * S + seg];
        if (k == 0) {
            if (threadIdx.x == 0) {
                *st = SelectState{0, 0, 0xFFFFFFFFu, 0, 0, 0};
                s_digit[v] = 0xFFFFFFFFu;
            }
            continue;
        }
        // the vector of this thread whose keys reach rank k, then the first of its four bins that does (one thread)
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint64_t start = warp_base + before[j];
            if (start < k && k <= start + gs[j]) {
                uint64_t cum = start;
                int b = 0;
                uint32_t cnt = 0;
                bool found = false;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    if (!found) {
                        if (cum + c[4 * j + q] >= k) {
                            b = q;
                            cnt = c[4 * j + q];
                            found = true;
                        } else {
                            cum += c[4 * j + q];
                        }
                    }
                }
                const uint32_t digit = (uint32_t)warp * 1024u + (uint32_t)(j * 32 + lane) * 4u + (uint32_t)b;
                *st = SelectState{k, cum, digit, 0, cnt, 0};
                s_digit[v] = digit;
            }
        }
    }
    __syncthreads();
    if ((int)threadIdx.x < n_k) {
        // variants that selected the same first digit share one second-pass histogram: its slot is
        // the rank of the digit among the distinct selected digits of the segment
        const uint32_t dg = s_digit[threadIdx.x];
        if (dg != 0xFFFFFFFFu) {
            uint32_t slot = 0;
            for (int u = 0; u < n_k; ++u) {
                const uint32_t du = s_digit[u];
                bool first = du != 0xFFFFFFFFu && du < dg;  // count each smaller digit once
                for (int t = 0; t < u && first; ++t)
                    if (s_digit[t] == du) first = false;
                slot += first;
            }
            ws.sel[(size_t)threadIdx.x * S + seg].slot = slot;
            atomicOr(&bm[dg >> 5], 1u << (dg & 31));
        }
    }
    if (DT == DNNS_BF16) {
        // a 15-bit key is fully resolved by the first digit
        __syncthreads();
        if ((int)threadIdx.x < n_k) {
            const int v = threadIdx.x;
            const SelectState st = ws.sel[(size_t)v * S + seg];
            dnns_threshold r{0, 0, 0, 0, 0};
            uint32_t need = 0;
            if (st.k) {
                r.tau_bits = st.digit;
                r.n_below = st.below;
                r.n_tie = st.k - st.below;
                r.n_equal = st.count;
                need = r.n_tie < r.n_equal;
            }
            thr[(size_t)v * S + seg] = r;
            ws.need[(size_t)v * S + seg] = need;
            if (need) {
                atomicOr(ws.any_need, 1u);
                atomicOr(&ws.tie_bitmap[(size_t)seg * kBitmapWords + (r.tau_bits >> 5)], 1u << (r.tau_bits & 31));
            }
        }
    }
}

template <int DT>
__global__ void __launch_bounds__(1024) k_select1(Tables tb, ThresholdWs ws, int n_k, dnns_threshold* __restrict__ thr,
                                                  InlineCounts counts, bool counts_inline) {
    __shared__ Select1Shared sm;
    select1_segment<DT>(tb, ws, blockIdx.x, n_k, thr, counts, counts_inline, sm);
}

// ---------------------------------------------------------------- pass 1
// Count one stored word's key(s) by first digit; digit 0 (exact zeros, mostly) in a register.
template <int DT>
__device__ __forceinline__ void count_word(uint32_t w, uint32_t* sh, uint32_t& zeros) {
    const uint32_t hi = (w >> 14) & 0x1FFFCu;  // 4 * (bits 16..30)
    if (hi == 0) ++zeros;
    else atomicAdd(reinterpret_cast<uint32_t*>(reinterpret_cast<char*>(sh) + hi), 1u);
    if (DT == DNNS_BF16) {
        const uint32_t lo = (w << 2) & 0x1FFFCu;  // 4 * (bits 0..14)
        if (lo == 0) ++zeros;
        else atomicAdd(reinterpret_cast<uint32_t*>(reinterpret_cast<char*>(sh) + lo), 1u);
    }
}

template <int DT>
__global__ void __launch_bounds__(kHistThreads, 1) k_hist1(Tables tb, ThresholdWs ws, int n_k, dnns_threshold* __restrict__ thr,
                                                           InlineCounts counts, bool counts_inline, bool then_select) {
    uint32_t* const hist1 = ws.hist1;
    constexpr uint32_t P = Elem<DT>::kPerVec;
    constexpr int U = 4;
    extern __shared__ uint32_t sh[];  // kHistBins counters
    for (uint32_t b = threadIdx.x; b < kHistBins; b += kHistThreads) sh[b] = 0;
    __syncthreads();

    const uint32_t per = (tb.n_tiles + gridDim.x - 1) / gridDim.x;
    const uint32_t lo = min(tb.n_tiles, blockIdx.x * per), hi = min(tb.n_tiles, lo + per);
    int cur_seg = -1;
    uint32_t zeros = 0;

    auto flush = [&](int seg) {
        // merge this block's counters into the segment's global histogram and clear them
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) zeros += __shfl_xor_sync(0xffffffffu, zeros, d);
        if ((threadIdx.x & 31) == 0 && zeros) atomicAdd(&sh[0], zeros);
        zeros = 0;
        __syncthreads();
        if (seg >= 0) {
            uint32_t* g = hist1 + (size_t)seg * kHistBins;
            for (uint32_t b = threadIdx.x; b < kHistBins; b += kHistThreads) {
                const uint32_t c = sh[b];
                if (c) {
                    atomicAdd(&g[b], c);
                    sh[b] = 0;
                }
            }
        }
        __syncthreads();
    };

    uint32_t tile = lo;
    while (tile < hi) {
        const TensorDesc& d = tb.tensors[tb.tile_tensor[tile]];
        const uint32_t span_end = min(hi, d.tile0 + d.n_tiles);
        if (d.seg >= 0) {
            if (d.seg != cur_seg) {
                flush(cur_seg);
                cur_seg = d.seg;
            }
            // elements [e0, e1) of this tensor: whole vectors in batches of U per thread with the
            // next batch in flight, then the remaining vectors, then the last few elements
            const uint32_t e0 = (tile - d.tile0) * tb.tile_elems;
            const uint32_t e1 = min(d.numel, (span_end - d.tile0) * tb.tile_elems);
            const uint32_t n_vec = (e1 - e0) / P;
            const uint4* p = reinterpret_cast<const uint4*>(static_cast<const char*>(d.src) + (size_t)e0 * Elem<DT>::kBytes);
            const uint32_t n_batch = n_vec / (U * kHistThreads);
            if (n_batch) {
                uint4 nxt[U];
                const uint4* q = p + threadIdx.x;
#pragma unroll
                for (int u = 0; u < U; ++u) nxt[u] = __ldg(q + u * kHistThreads);
                for (uint32_t b = 0; b < n_batch; ++b) {
                    uint4 cur[U];
#pragma unroll
                    for (int u = 0; u < U; ++u) cur[u] = nxt[u];
                    if (b + 1 < n_batch) {
                        q += U * kHistThreads;
#pragma unroll
                        for (int u = 0; u < U; ++u) nxt[u] = __ldg(q + u * kHistThreads);
                    }
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        count_word<DT>(cur[u].x, sh, zeros);
                        count_word<DT>(cur[u].y, sh, zeros);
                        count_word<DT>(cur[u].z, sh, zeros);
                        count_word<DT>(cur[u].w, sh, zeros);
                    }
                }
            }
            for (uint32_t i = n_batch * U * kHistThreads + threadIdx.x; i < n_vec; i += kHistThreads) {
                const uint4 c = __ldg(p + i);
                count_word<DT>(c.x, sh, zeros);
                count_word<DT>(c.y, sh, zeros);
                count_word<DT>(c.z, sh, zeros);
                count_word<DT>(c.w, sh, zeros);
            }
            const uint32_t e = e0 + n_vec * P + threadIdx.x;
            if (e < e1) {
                uint32_t key;
                if (DT == DNNS_F32) key = static_cast<const uint32_t*>(d.src)[e] & 0x7FFFFFFFu;
                else key = static_cast<const uint16_t*>(d.src)[e] & 0x7FFFu;
                const uint32_t dg = digit_of<DT>(key);
                if (dg == 0) ++zeros;
                else atomicAdd(&sh[dg], 1u);
            }
        }
        tile = span_end;
    }
    flush(cur_seg);
    if (then_select) {
        // few segments: the block that finishes last selects the first digits at once - it is resident, while a
        // kernel of its own would have to wait for a free SM beside whatever else is running
        __shared__ Select1Shared sm;
        __shared__ uint32_t s_last;
        __threadfence();  // this thread's additions to the global histograms, before the ticket
        __syncthreads();
        if (threadIdx.x == 0) s_last = atomicAdd(ws.hist_done, 1u) == gridDim.x - 1;
        __syncthreads();
        if (s_last) {
            __threadfence();
            for (uint32_t seg = 0; seg < tb.n_segs; ++seg) {
                select1_segment<DT>(tb, ws, seg, n_k, thr, counts, counts_inline, sm);
                __syncthreads();
            }
        }
    }
}

// ---------------------------------------------------------------- pass 2 (31-bit keys)
// Load a segment's bitmap into shared memory together with, per word, the number of set bits in
// earlier words, so that rank(digit) - the digit's histogram slot - is one popcount away.
__device__ __forceinline__ void load_bitmap_with_ranks(const uint32_t* g_bm, uint32_t* s_bm, uint32_t* s_rank,
                                                       uint32_t* scratch) {
    constexpr int W = kBitmapWords / kTileThreads;  // words per thread
    uint32_t w[W], c = 0;
#pragma unroll
    for (int i = 0; i < W; ++i) {
        w[i] = g_bm[threadIdx.x * W + i];
        c += __popc(w[i]);
    }
    uint32_t total;
    uint32_t ex = block_exclusive_scan<uint32_t>(c, scratch, &total);
#pragma unroll
    for (int i = 0; i < W; ++i) {
        s_bm[threadIdx.x * W + i] = w[i];
        s_rank[threadIdx.x * W + i] = ex;
        ex += __popc(w[i]);
    }
    __syncthreads();
}

constexpr uint32_t kTieStage = 1024;  // listed keys a block of the second sweep holds before it writes them out

__global__ void __launch_bounds__(kTileThreads, 4) k_hist2(Tables tb, ThresholdWs ws, int n_k) {
    __shared__ uint32_t s_bm[kBitmapWords], s_rank[kBitmapWords];
    __shared__ uint32_t scratch[33];
    __shared__ unsigned long long s_ent[kTieStage];
    __shared__ uint32_t s_n, s_base;
    const bool listing = ws.tie_list != nullptr;
    uint32_t tiles_done = 0;
    int cur_seg = -1;
    uint32_t* h2 = nullptr;
    uint32_t zeros = 0;  // exact zeros among the selected keys: counted in a register, added once
    if (threadIdx.x == 0) s_n = 0;
    auto flush_zeros = [&]() {
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) zeros += __shfl_xor_sync(0xffffffffu, zeros, d);
        if ((threadIdx.x & 31) == 0 && zeros) atomicAdd(&h2[0], zeros);  // digit 0 has rank 0, low digit 0
        zeros = 0;
    };
    // the staged entries go to the list: one reservation for the block (block-uniform; s_n is settled)
    auto flush_list = [&]() {
        const uint32_t n = min(s_n, kTieStage);
        if (threadIdx.x == 0) s_base = atomicAdd(ws.tie_list_n, n);
        __syncthreads();
        for (uint32_t i = threadIdx.x; i < n; i += kTileThreads)
            if (s_base + i < ws.tie_list_cap) ws.tie_list[s_base + i] = s_ent[i];
        __syncthreads();
        if (threadIdx.x == 0) s_n = 0;
        __syncthreads();
    };
    walk_prunable_tiles<DNNS_F32>(
        tb,
        [&](const TensorDesc& d) {
            if (d.seg != cur_seg) {
                if (cur_seg >= 0) flush_zeros();
                cur_seg = d.seg;
                load_bitmap_with_ranks(ws.bitmap + (size_t)cur_seg * kBitmapWords, s_bm, s_rank, scratch);
                h2 = ws.hist2 + (size_t)cur_seg * n_k * kLowBins;
            }
            return true;
        },
        [&](uint32_t tile, uint32_t n_e, const uint4(&v)[kVecPerThread]) {
            // which of the thread's 16 keys have a selected first digit (bit 4 * u + j), and how many of those are not zero
            uint32_t hits = 0;
#pragma unroll
            for (int u = 0; u < kVecPerThread; ++u) {
                const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                uint32_t h = 0;
#pragma unroll
                for (int q = 0; q < 4; ++q) h |= bitmap_test<16>(s_bm, w[q]) << q;
                if (n_e != kTileBytes / 4) {  // ragged tile: drop the slots past the end of the tensor
                    const uint32_t first = (u * kTileThreads + threadIdx.x) * 4;
                    h &= first >= n_e ? 0u : (n_e - first >= 4u ? 0xFu : ((1u << (n_e - first)) - 1u));
                }
                hits |= h << (4 * u);
            }
            auto key_of = [&](int b) {
                const int u = b >> 2, q = b & 3;
                const uint4 x = u == 0 ? v[0] : (u == 1 ? v[1] : (u == 2 ? v[2] : v[3]));
                return (q == 0 ? x.x : (q == 1 ? x.y : (q == 2 ? x.z : x.w))) & 0x7FFFFFFFu;
            };
            uint32_t mine = __popc(hits);  // non-zero selected keys of this thread: they are listed
            if (s_bm[0] & 1u) {  // digit 0 is selected (a tau below 2^16): exact zeros are counted, not listed
                mine = 0;
                for (uint32_t m = hits; m; m &= m - 1) {
                    const uint32_t key = key_of(__ffs(m) - 1);
                    if (key == 0) ++zeros, hits &= ~(1u << (__ffs(m) - 1));
                    else ++mine;
                }
            }
            // the warp reserves its places in the block's stage with one addition
            uint32_t at = 0;
            if (listing) {
                const int lane = threadIdx.x & 31;
                uint32_t incl = mine;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, d);
                    if (lane >= d) incl += y;
                }
                const uint32_t total = __shfl_sync(0xffffffffu, incl, 31);
                uint32_t base = 0;
                if (total) {
                    if (lane == 31) base = atomicAdd(&s_n, total);
                    base = __shfl_sync(0xffffffffu, base, 31);
                }
                at = base + incl - mine;
            }
            for (uint32_t m = hits; m; m &= m - 1) {
                const int b = __ffs(m) - 1;
                const uint32_t key = key_of(b);
                const uint32_t dg = key >> 16;
                const uint32_t slot = s_rank[dg >> 5] + __popc(s_bm[dg >> 5] & ((1u << (dg & 31)) - 1u));
                atomicAdd(&h2[(size_t)slot * kLowBins + (key & 0xFFFFu)], 1u);
                if (listing) {
                    const uint32_t off = ((b >> 2) * kTileThreads + threadIdx.x) * 4 + (b & 3);
                    const unsigned long long e = (unsigned long long)(tile * (kTileBytes / 4) + off) | ((unsigned long long)(key & 0xFFFFu) << 32) |
                                                 ((unsigned long long)slot << 48) | ((unsigned long long)cur_seg << 56);
                    if (at < kTieStage) {
                        s_ent[at] = e;
                    } else {  // the stage is full (a tile dense with selected keys): straight to the list
                        const uint32_t g = atomicAdd(ws.tie_list_n, 1u);
                        if (g < ws.tie_list_cap) ws.tie_list[g] = e;
                    }
                    ++at;
                }
            }
            // every fourth tile the block looks whether the stage is half full (every thread looks at the counter after
            // its warp's reservation, the last warp to reserve sees them all)
            if (listing && (++tiles_done & 3) == 0 && __syncthreads_or(s_n >= kTieStage / 2)) flush_list();
        });
    if (cur_seg >= 0) flush_zeros();
    if (listing) {
        __syncthreads();
        if (s_n) flush_list();
    }
}

// ---------------------------------------------------------------- select 2 (31-bit keys)
// One block per (variant, segment).
__global__ void __launch_bounds__(1024) k_select2(Tables tb, ThresholdWs ws, int n_k, dnns_threshold* __restrict__ thr) {
    __shared__ uint64_t scratch[33];
    const uint32_t S = tb.n_segs;
    const uint32_t v = blockIdx.x / S, seg = blockIdx.x % S;
    const size_t idx = (size_t)v * S + seg;
    const SelectState st = ws.sel[idx];
    if (st.k == 0) {
        if (threadIdx.x == 0) {
            thr[idx] = dnns_threshold{0, 0, 0, 0, 0};
            ws.need[idx] = 0;
        }
        return;
    }
    // A warp owns 2048 consecutive bins = 512 vectors of four; a lane loads vectors lane, lane + 32, .. of them: every
    // load of the warp is one contiguous 512 bytes.  Bin order inside the warp: group j (32 vectors), lane, element.
    const uint32_t* h = ws.hist2 + ((size_t)seg * n_k + st.slot) * kLowBins;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint4* hv = reinterpret_cast<const uint4*>(h) + warp * 512;
    uint32_t part[16], before[16];  // the sum of the lane's vector in group j; keys of the warp before that vector
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const uint4 q = hv[j * 32 + lane];
        part[j] = q.x + q.y + q.z + q.w;
    }
    uint32_t warp_sum = 0;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        uint32_t incl = part[j];
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t y = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += y;
        }
        before[j] = warp_sum + incl - part[j];
        warp_sum += __shfl_sync(0xffffffffu, incl, 31);
    }
    uint64_t total;
    const uint64_t warp_base =
        st.below + __shfl_sync(0xffffffffu, block_exclusive_scan<uint64_t>(lane == 0 ? warp_sum : 0u, scratch, &total), 0);
    int jj = -1;
    uint64_t cum = 0;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const uint64_t start = warp_base + before[j];
        if (start < st.k && st.k <= start + part[j]) jj = j, cum = start;
    }
    if (jj >= 0) {
        // this thread's vector jj holds the k-th key: one more load for its four bins
        const uint32_t vec = (uint32_t)warp * 512u + (uint32_t)(jj * 32 + lane);
        const uint4 q = reinterpret_cast<const uint4*>(h)[vec];
        const uint32_t c4[4] = {q.x, q.y, q.z, q.w};
        bool found = false;
        uint32_t b = 0, cnt = 0;
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            if (!found) {
                if (cum + c4[t] >= st.k) b = (uint32_t)t, cnt = c4[t], found = true;
                else cum += c4[t];
            }
        }
        dnns_threshold r;
        r.tau_bits = (st.digit << 16) | (vec * 4u + b);
        r.pad = 0;
        r.n_below = cum;
        r.n_tie = st.k - cum;
        r.n_equal = cnt;
        thr[idx] = r;
        const uint32_t need = r.n_tie < r.n_equal;
        ws.need[idx] = need;
        if (need) {
            const uint32_t low = r.tau_bits & 0x7FFFu;  // the tie sweep filters keys by these 15 bits
            atomicOr(ws.any_need, 1u);
            atomicOr(&ws.tie_bitmap[(size_t)seg * kBitmapWords + (low >> 5)], 1u << (low & 31));
        }
    }
}

// ---------------------------------------------------------------- tie counts per tile
// Keys are filtered by the low 15 bits of the thresholds that need tie tables (a 15-bit key is its
// own filter), then compared exactly.  Counts go straight to the per-tile table in global memory;
// exact zeros, the one value that can fill whole tiles, are counted per warp first.
template <int DT>
__global__ void __launch_bounds__(kTileThreads, 4) k_ties(Tables tb, ThresholdWs ws, int n_k,
                                                          const dnns_threshold* __restrict__ thr) {
    if (*ws.any_need == 0 || (ws.ties_if && *ws.ties_if == 0)) return;
    // 31-bit keys: a bitmap of the low 15 bits of the thresholds filters the keys, survivors are compared with
    // every threshold.  15-bit keys: a key is its own index into a byte table that names the first variant
    // whose threshold it equals (0: none) - one lookup per key and one counter update per hit, because keys
    // equal to a threshold are common there (thousands per threshold).
    __shared__ uint32_t s_bm[DT == DNNS_F32 ? kBitmapWords : 1];
    __shared__ uint8_t s_slot[DT == DNNS_BF16 ? kHistBins : 4];
    __shared__ uint32_t s_tau[kMaxVariants], s_need[kMaxVariants];
    __shared__ uint32_t s_cnt[kTileThreads / 32][kMaxVariants];  // per warp: ties of the current tile, per variant
    __shared__ uint32_t s_any, s_zero_tau;
    const uint32_t S = tb.n_segs;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < (kTileThreads / 32) * kMaxVariants; i += kTileThreads) (&s_cnt[0][0])[i] = 0;
    int cur_seg = -1;
    walk_prunable_tiles<DT>(
        tb,
        [&](const TensorDesc& d) {
            if (d.seg != cur_seg) {
                __syncthreads();
                cur_seg = d.seg;
                if (threadIdx.x == 0) s_any = s_zero_tau = 0;
                if (DT == DNNS_BF16)
                    for (uint32_t i = threadIdx.x; i < kHistBins / 4; i += kTileThreads) reinterpret_cast<uint32_t*>(s_slot)[i] = 0;
                __syncthreads();
                if (DT == DNNS_F32)
                    for (uint32_t w = threadIdx.x; w < kBitmapWords; w += kTileThreads)
                        s_bm[w] = ws.tie_bitmap[(size_t)cur_seg * kBitmapWords + w];
                if ((int)threadIdx.x < n_k) {
                    const size_t idx = (size_t)threadIdx.x * S + cur_seg;
                    const uint32_t need = ws.need[idx], tau = thr[idx].tau_bits;
                    s_tau[threadIdx.x] = tau;
                    s_need[threadIdx.x] = need;
                    if (need) s_any = 1;
                    if (need && tau == 0) s_zero_tau = 1;
                }
                __syncthreads();
                if (DT == DNNS_BF16 && threadIdx.x == 0) {
                    // the first variant (in index order) that needs tie counts for a key owns the key's counter;
                    // variants with the same threshold copy it when the tile's counts are sent
                    for (int vv = n_k - 1; vv >= 0; --vv)
                        if (s_need[vv] && s_tau[vv] != 0) s_slot[s_tau[vv]] = (uint8_t)(vv + 1);
                }
                __syncthreads();
            }
            return s_any != 0;  // no variant of this segment splits its ties: nothing to count
        },
        [&](uint32_t tile, uint32_t n_e, const uint4(&v)[kVecPerThread]) {
            uint32_t zeros = 0;
            if (DT == DNNS_F32) {
                for_filtered_keys<DT, 0>(v, n_e, s_bm, [&](uint32_t key, uint32_t) {
                    if (key == 0) {
                        ++zeros;
                        return;
                    }
                    for (int vv = 0; vv < n_k; ++vv)
                        if (s_need[vv] && s_tau[vv] == key) atomicAdd(&s_cnt[warp][vv], 1u);
                });
            } else {
                constexpr uint32_t kTileElems = kTileBytes / Elem<DT>::kBytes;
#pragma unroll
                for (int u = 0; u < kVecPerThread; ++u) {
                    const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                    const uint32_t first = (u * kTileThreads + threadIdx.x) * 8;
                    // elements past a ragged end were loaded as zeros: they must not count as zero keys
                    const uint32_t valid = n_e == kTileElems ? 8u : (first >= n_e ? 0u : min(8u, n_e - first));
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const uint32_t key = (w[j >> 1] >> (16 * (j & 1))) & 0x7FFFu;
                        if ((uint32_t)j >= valid) continue;
                        if (key == 0) {
                            ++zeros;
                            continue;
                        }
                        const uint32_t slot = s_slot[key];
                        if (slot) atomicAdd(&s_cnt[warp][slot - 1], 1u);
                    }
                }
            }
            // a warp sends its counts of the tile to the table in one atomic per variant: keys equal to
            // tau are common in 15-bit keys, and thousands of single atomics on one word would queue up
            __syncwarp();
            for (int vv = lane; vv < n_k; vv += 32) {
                uint32_t c = s_cnt[warp][vv];
                if (DT == DNNS_BF16 && s_need[vv] && s_tau[vv] != 0) c = s_cnt[warp][s_slot[s_tau[vv]] - 1];  // the owner's count
                if (c) atomicAdd(&ws.tile_ties[(size_t)vv * tb.n_tiles + tile], c);
            }
            __syncwarp();
            for (int vv = lane; vv < n_k; vv += 32) s_cnt[warp][vv] = 0;
            __syncwarp();
            if (s_zero_tau) {
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) zeros += __shfl_xor_sync(0xffffffffu, zeros, d);
                if ((threadIdx.x & 31) == 0 && zeros)
                    for (int vv = 0; vv < n_k; ++vv)
                        if (s_need[vv] && s_tau[vv] == 0) atomicAdd(&ws.tile_ties[(size_t)vv * tb.n_tiles + tile], zeros);
            }
        });
}

// Exclusive scan of the tile counts over the tiles of a segment, one block per (variant, segment); every thread
// owns a contiguous run of tiles: one pass of independent loads, one block scan.  The mask kernel then needs no
// ordering between tiles.
//
// The same block then finds where the variant's ties split.  Weights equal to tau are masked in index order until
// n_tie of them are gone; the first one that stays is the tie of rank n_tie.  Its tile follows from the scanned
// counts (the last tile whose exclusive prefix is <= n_tie), its place in the tile from one ranking of that tile's
// ties (a 16 KB tile is one 16-byte vector per thread).
template <int DT>
__global__ void __launch_bounds__(1024) k_tie_scan(Tables tb, ThresholdWs ws, const dnns_threshold* __restrict__ thr) {
    constexpr int P = Elem<DT>::kPerVec;
    constexpr uint32_t kTileElems = kTileBytes / Elem<DT>::kBytes;
    static_assert(kTileBytes / 16 == 1024, "one vector of the tile per thread");
    __shared__ uint32_t scratch[33];
    const uint32_t S = tb.n_segs;
    const uint32_t v = blockIdx.x / S, seg = blockIdx.x % S;
    const size_t idx = (size_t)v * S + seg;
    if (ws.ties_if && *ws.ties_if == 0) return;  // the lists gave the split
    if (*ws.any_need == 0 || !ws.need[idx]) {
        if (threadIdx.x == 0) ws.split[idx] = TieSplit{0xFFFFFFFFu, 0u};  // no weight equal to tau stays
        return;
    }
    const SegDesc sd = tb.segs[seg];
    const uint32_t* cnt = ws.tile_ties + (size_t)v * tb.n_tiles;
    uint32_t* pre = ws.tie_prefix + (size_t)v * tb.n_tiles;
    // a warp owns a contiguous run of tiles and reads them 32 at a time (coalesced); two passes: the warps' sums, then
    // the prefixes in order
    const dnns_threshold r = thr[idx];
    const uint32_t n_tie = (uint32_t)r.n_tie;  // below n_equal, which fits 32 bits
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t n = sd.tile_end - sd.tile_begin, per_warp = (n + 31) / 32;
    const uint32_t w0 = min(sd.tile_end, sd.tile_begin + warp * per_warp), w1 = min(sd.tile_end, w0 + per_warp);
    constexpr int kScanBatch = 4;
    uint32_t warp_sum = 0;
    for (uint32_t base = w0; base < w1; base += 32 * kScanBatch) {
        uint32_t c[kScanBatch];
#pragma unroll
        for (int i = 0; i < kScanBatch; ++i) c[i] = base + i * 32 + lane < w1 ? cnt[base + i * 32 + lane] : 0u;
#pragma unroll
        for (int i = 0; i < kScanBatch; ++i) warp_sum += c[i];
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) warp_sum += __shfl_xor_sync(0xffffffffu, warp_sum, d);
    uint32_t total;
    uint32_t before = __shfl_sync(0xffffffffu, block_exclusive_scan<uint32_t>(lane == 0 ? warp_sum : 0u, scratch, &total), 0);
    // the tile that holds the tie of rank n_tie is found by exactly one thread (the defaults stand only if the counts
    // do not add up to the record, i.e. the weights were rewritten under the sweeps: a valid tile, a rank nobody has)
    __shared__ uint32_t s_tile, s_want;
    if (threadIdx.x == 0) s_tile = sd.tile_begin, s_want = 0xFFFFFFFFu;
    __syncthreads();
    for (uint32_t base = w0; base < w1; base += 32) {
        const uint32_t t = base + lane;
        const uint32_t c = t < w1 ? cnt[t] : 0u;
        uint32_t incl = c;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t y = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += y;
        }
        const uint32_t ex = before + incl - c;
        if (t < w1) {
            pre[t] = ex;
            if (ex <= n_tie && n_tie < ex + c) s_tile = t, s_want = n_tie - ex;
        }
        before += __shfl_sync(0xffffffffu, incl, 31);
    }
    __syncthreads();
    const uint32_t tile = s_tile, want = s_want;  // rank, inside the tile, of the tie that stays
    const uint32_t t = tb.tile_tensor[tile];
    const TensorDesc& d = tb.tensors[t];
    const uint32_t e = (tile - d.tile0) * kTileElems + threadIdx.x * P;
    uint4 vec;
    const int nv = load_vec<DT>(d.src, e, d.numel, vec);
    uint32_t key[P];
    vec_keys<DT>(vec, key);
    uint32_t c = 0;
#pragma unroll
    for (int j = 0; j < P; ++j) c += (j < nv && key[j] == r.tau_bits);
    uint32_t rank = block_exclusive_scan<uint32_t>(c, scratch, &total);
    if (rank <= want && want < rank + c) {
#pragma unroll
        for (int j = 0; j < P; ++j) {
            if (j < nv && key[j] == r.tau_bits) {
                if (rank == want) ws.split[idx] = TieSplit{t, e + j};
                ++rank;
            }
        }
    }
}

// ---------------------------------------------------------------- the tie split from the lists (31-bit keys)
// One pass over the list of the second sweep: the entries whose segment, histogram slot and low key bits are those of a
// variant's tau are the weights equal to tau; their positions go to the variant's short list.
__global__ void __launch_bounds__(256) k_tie_find(Tables tb, ThresholdWs ws, int n_k, const dnns_threshold* __restrict__ thr) {
    __shared__ uint32_t s_code[kTieListMaxPairs];  // segment << 24 | slot << 16 | low 16 bits of tau; 0xFFFFFFFF: not wanted
    if (*ws.any_need == 0) return;
    const uint32_t S = tb.n_segs, n_pairs = (uint32_t)n_k * S;
    for (uint32_t i = threadIdx.x; i < n_pairs; i += blockDim.x) {
        const uint32_t seg = i % S;
        const dnns_threshold r = thr[i];
        s_code[i] = ws.need[i] && r.tau_bits != 0 ? (seg << 24) | (ws.sel[i].slot << 16) | (r.tau_bits & 0xFFFFu) : 0xFFFFFFFFu;
    }
    __syncthreads();
    const uint32_t n = min(*ws.tie_list_n, ws.tie_list_cap);
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        const unsigned long long e = ws.tie_list[i];
        const uint32_t code = (uint32_t)(e >> 32);
        for (uint32_t q = 0; q < n_pairs; ++q) {
            if (s_code[q] == code) {
                const uint32_t at = atomicAdd(&ws.tie_match_n[q], 1u);
                if (at < kTieMatchCap) ws.tie_match[(size_t)q * kTieMatchCap + at] = (uint32_t)e;
            }
        }
    }
}

// Per (variant, segment): the weights equal to tau are masked in index order, so the first one that stays is the one
// with n_tie of them before it.  Where the lists cannot say (they ran over, tau is zero - zeros are not listed -, or
// there are more equal weights than a short list holds), a flag sends the call to the tie sweep.
template <int DT>
__global__ void __launch_bounds__(256) k_tie_pick(Tables tb, ThresholdWs ws, const dnns_threshold* __restrict__ thr) {
    constexpr uint32_t kTileElems = kTileBytes / Elem<DT>::kBytes;
    __shared__ uint32_t s_pos[kTieMatchCap];
    const uint32_t idx = blockIdx.x;
    if (*ws.any_need == 0 || !ws.need[idx]) {
        if (threadIdx.x == 0) ws.split[idx] = TieSplit{0xFFFFFFFFu, 0u};  // no weight equal to tau stays
        return;
    }
    const dnns_threshold r = thr[idx];
    const uint32_t m = ws.tie_match_n[idx];
    if (*ws.tie_list_n > ws.tie_list_cap || r.tau_bits == 0 || (uint64_t)m != r.n_equal || m > kTieMatchCap) {
        if (threadIdx.x == 0) atomicOr(ws.tie_fallback, 1u);
        return;
    }
    for (uint32_t i = threadIdx.x; i < m; i += blockDim.x) s_pos[i] = ws.tie_match[(size_t)idx * kTieMatchCap + i];
    __syncthreads();
    const uint32_t n_tie = (uint32_t)r.n_tie;
    for (uint32_t i = threadIdx.x; i < m; i += blockDim.x) {
        const uint32_t mine = s_pos[i];
        uint32_t before = 0;
        for (uint32_t q = 0; q < m; ++q) before += s_pos[q] < mine;
        if (before == n_tie) {
            const uint32_t tile = mine / kTileElems, t = tb.tile_tensor[tile];
            ws.split[idx] = TieSplit{t, (tile - tb.tensors[t].tile0) * kTileElems + mine % kTileElems};
        }
    }
}

}  // namespace

cudaError_t init_kernel_attributes() {
    cudaError_t e = cudaFuncSetAttribute(k_hist1<DNNS_F32>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)(kHistBins * 4));
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(k_hist1<DNNS_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kHistBins * 4));
}

int launch_threshold(const Tables& tb, const ThresholdWs& ws, int n_k, const uint64_t* k_host, dnns_threshold* thr_dev,
                     int n_sm, cudaStream_t st) {
    const uint32_t S = tb.n_segs;
    // few counts travel as a kernel argument, many through the workspace
    InlineCounts counts{};
    const bool counts_inline = (size_t)n_k * S <= kInlineCounts;
    if (counts_inline) {
        for (size_t i = 0; i < (size_t)n_k * S; ++i) counts.k[i] = k_host[i];
    } else if (cudaMemcpyAsync(ws.k_dev, k_host, 8ull * n_k * S, cudaMemcpyHostToDevice, st) != cudaSuccess) {
        return -1;
    }
    const int hist_grid = (int)min((uint32_t)n_sm, tb.n_tiles);
    // few segments: the first sweep's last block selects the first digits itself (one launch less in the chain)
    const bool fused = ws.hist_done != nullptr && S <= kFusedSelectSegs;
    const int sweep_grid = (int)min((uint32_t)n_sm * 4u, tb.n_tiles);
    int launches = 0;
    if (tb.dtype == DNNS_F32) {
        { ScopedKernel t("k_hist1", st); k_hist1<DNNS_F32><<<hist_grid, kHistThreads, kHistBins * 4, st>>>(tb, ws, n_k, thr_dev, counts, counts_inline, fused); }
        if (!fused) { ScopedKernel t("k_select1", st); k_select1<DNNS_F32><<<S, 1024, 0, st>>>(tb, ws, n_k, thr_dev, counts, counts_inline); }
        { ScopedKernel t("k_hist2", st); k_hist2<<<sweep_grid, kTileThreads, 0, st>>>(tb, ws, n_k); }
        { ScopedKernel t("k_select2", st); k_select2<<<S * n_k, 1024, 0, st>>>(tb, ws, n_k, thr_dev); }
        launches = fused ? 3 : 4;
        if (ws.tie_list) {
            // the place where the weights equal to tau split, from the lists of the second sweep; the tie sweep and its
            // scan stand by behind a flag (huge blocks of equal weights, tau = 0)
            const int find_grid = (int)min((uint32_t)n_sm * 4u, (ws.tie_list_cap + 255u) / 256u);
            { ScopedKernel t("k_tie_find", st); k_tie_find<<<find_grid, 256, 0, st>>>(tb, ws, n_k, thr_dev); }
            { ScopedKernel t("k_tie_pick", st); k_tie_pick<DNNS_F32><<<S * n_k, 256, 0, st>>>(tb, ws, thr_dev); }
            launches += 2;
        }
        ThresholdWs tw = ws;
        tw.ties_if = ws.tie_list ? ws.tie_fallback : nullptr;
        { ScopedKernel t("k_ties", st); k_ties<DNNS_F32><<<sweep_grid, kTileThreads, 0, st>>>(tb, tw, n_k, thr_dev); }
        { ScopedKernel t("k_tie_scan", st); k_tie_scan<DNNS_F32><<<S * n_k, 1024, 0, st>>>(tb, tw, thr_dev); }
        launches += 2;
    } else {
        { ScopedKernel t("k_hist1", st); k_hist1<DNNS_BF16><<<hist_grid, kHistThreads, kHistBins * 4, st>>>(tb, ws, n_k, thr_dev, counts, counts_inline, fused); }
        if (!fused) { ScopedKernel t("k_select1", st); k_select1<DNNS_BF16><<<S, 1024, 0, st>>>(tb, ws, n_k, thr_dev, counts, counts_inline); }
        { ScopedKernel t("k_ties", st); k_ties<DNNS_BF16><<<sweep_grid, kTileThreads, 0, st>>>(tb, ws, n_k, thr_dev); }
        { ScopedKernel t("k_tie_scan", st); k_tie_scan<DNNS_BF16><<<S * n_k, 1024, 0, st>>>(tb, ws, thr_dev); }
        launches = fused ? 3 : 4;
    }
    return cudaGetLastError() == cudaSuccess ? launches : -1;
}

// The per-tile tables of the weights equal to tau on their own (the sweeps that mask tile by tile read them; a
// threshold call that found the tie split in its lists leaves them out).
int launch_tie_tables(const Tables& tb, const ThresholdWs& ws, int n_k, const dnns_threshold* thr_dev, int n_sm,
                      cudaStream_t st) {
    const uint32_t S = tb.n_segs;
    const int sweep_grid = (int)min((uint32_t)n_sm * 4u, tb.n_tiles);
    if (cudaMemsetAsync(ws.tile_ties, 0, 4ull * n_k * tb.n_tiles, st) != cudaSuccess) return -1;
    ThresholdWs tw = ws;
    tw.ties_if = nullptr;
    if (tb.dtype == DNNS_F32) {
        { ScopedKernel t("k_ties", st); k_ties<DNNS_F32><<<sweep_grid, kTileThreads, 0, st>>>(tb, tw, n_k, thr_dev); }
        { ScopedKernel t("k_tie_scan", st); k_tie_scan<DNNS_F32><<<S * n_k, 1024, 0, st>>>(tb, tw, thr_dev); }
    } else {
        { ScopedKernel t("k_ties", st); k_ties<DNNS_BF16><<<sweep_grid, kTileThreads, 0, st>>>(tb, tw, n_k, thr_dev); }
        { ScopedKernel t("k_tie_scan", st); k_tie_scan<DNNS_BF16><<<S * n_k, 1024, 0, st>>>(tb, tw, thr_dev); }
    }
    return cudaGetLastError() == cudaSuccess ? 2 : -1;
}

}  // namespace dnns
