// Steps 2 and 3 as one tile kernel.
//
//   mask       (Section III-C: the insignificant weights are set to zero, the sparse model keeps
//              its size) - a weight survives when its magnitude key is above tau, or equals tau
//              and at least n_tie equal keys precede it in its segment.  The per-tile tie tables
//              written by the threshold step tell every tile, without looking at any other
//              tile, whether its ties are all masked, all kept, or split (one tile per segment
//              at most, which then ranks its ties with a block scan).
//   structures (Module 2, Sparsity Analyser) - the non-zero bits of the tile's elements go to
//              shared memory; from them the all-zero 2-D kernels, and from those the filters
//              (rows) and input columns that still hold something, are OR-ed into the packed
//              global flag arrays (test first, atomic only when a bit is still missing).
//
// The same kernel runs either step alone or both in one sweep (the structures are then derived
// from the masked values while they are still in registers).
#include "dnns_internal.cuh"

namespace dnns {

namespace {

constexpr unsigned kFull = 0xffffffffu;

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

// Any bit set in [lo, hi) of a shared-memory bit array.
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

// From the element bits of one tile (elements [e0, e0+n_e) of tensor d) to kernel map, filter
// flags and input-column flags.  Kernel q = (o, i) covers elements [q*KK, (q+1)*KK); a kernel cut
// by the tile edge is OR-ed by both tiles.  kbits_buf receives the kernel bits of the tile, kernel
// q at bit q - (q0 & ~31); for 1x1 kernels the element bits are used as they are.
// Global flag words are read first and only updated (atomicOr) when a bit is still missing: a
// stale read costs a redundant atomic at worst, and flags saturate early in a sweep.
// There is no barrier at the end: the caller alternates between two sets of bit buffers.
__device__ __forceinline__ void tile_structures(const TensorDesc& d, uint32_t e0, uint32_t n_e, const uint32_t* ebits,
                                                uint32_t* kbits_buf, uint32_t* nz_map, uint32_t* out_nz,
                                                uint32_t* in_nz) {
    const uint32_t KK = d.KK, I = d.I;
    const uint32_t q0 = e0 / KK, q1 = (e0 + n_e - 1) / KK;
    const uint32_t qa = q0 & ~31u;
    const uint32_t n_words = ((q1 - qa) >> 5) + 1;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t* kbits = ebits;  // KK == 1: kernels are elements and the tile starts on a word
    if (KK != 1) {
        for (uint32_t w = warp; w < n_words; w += kTileThreads / 32) {
            const uint32_t q = qa + 32 * w + lane;
            bool bit = false;
            if (q >= q0 && q <= q1) {
                const uint32_t lo = max(q * KK, e0) - e0, hi = min((q + 1) * KK, e0 + n_e) - e0;
                bit = any_bits(ebits, lo, hi);
            }
            const uint32_t word = __ballot_sync(kFull, bit);
            if (lane == 0) kbits_buf[w] = word;
        }
        __syncthreads();
        kbits = kbits_buf;
    }
    uint32_t* g_in = in_nz + d.off_innz;
    uint32_t* g_out = out_nz + d.off_outnz;
    uint32_t* g_map = nz_map ? nz_map + d.off_nzmap : nullptr;
    const bool row_words = (I % 32 == 0);  // 32 consecutive kernels never cross a filter boundary
    for (uint32_t w = threadIdx.x; w < n_words; w += kTileThreads) {
        uint32_t bits = kbits[w];
        if (!bits) continue;
        const uint32_t qb = qa + 32 * w;
        if (g_map) {
            // only the first and last word can hold kernels shared with a neighbouring tile
            if (KK == 1 || (w != 0 && w != n_words - 1)) g_map[qb >> 5] = bits;
            else atomicOr(&g_map[qb >> 5], bits);
        }
        if (row_words) {
            const uint32_t o = qb / I, iw = (qb - o * I) >> 5, ob = 1u << (o & 31);
            uint32_t* pi = &g_in[iw];
            uint32_t* po = &g_out[o >> 5];
            const uint32_t gi = __ldcg(pi), go = __ldcg(po);  // both reads in flight together
            if ((gi & bits) != bits) atomicOr(pi, bits);
            if (!(go & ob)) atomicOr(po, ob);
        } else {
            while (bits) {
                const uint32_t q = qb + __ffs(bits) - 1;
                bits &= bits - 1;
                const uint32_t o = q / I, i = q - o * I;
                uint32_t* pi = &g_in[i >> 5];
                uint32_t* po = &g_out[o >> 5];
                const uint32_t gi = __ldcg(pi), go = __ldcg(po);
                if (!((gi >> (i & 31)) & 1u)) atomicOr(pi, 1u << (i & 31));
                if (!((go >> (o & 31)) & 1u)) atomicOr(po, 1u << (o & 31));
            }
        }
    }
}

// Each block owns a contiguous range of tiles.  Inside a tensor the loop is software-pipelined:
// the 16-byte loads of the next tile (and its two tie-table words) are issued before the current
// tile is processed, so a block always has a tile in flight while it masks, stores and updates
// the flags of the previous one.  Whole tiles whose ties do not split take a lean path; the last
// (ragged) tile of a tensor and the one tile per segment that ranks its ties take the general one.
template <int DT, bool DO_MASK, bool DO_STRUCT>
__global__ void __launch_bounds__(kTileThreads, 4) k_sweep(Tables tb, ThresholdWs ws, const dnns_threshold* __restrict__ thr,
                                                           int variant, const char* src_arena, char* dst_arena,
                                                           uint32_t* mask_bits, uint32_t* nz_map, uint32_t* out_nz,
                                                           uint32_t* in_nz) {
    constexpr int P = Elem<DT>::kPerVec;
    constexpr int G = 32 / P;  // lanes per bit word
    constexpr uint32_t kTileElems = kTileBytes / Elem<DT>::kBytes;
    constexpr uint32_t kKeyMask = DT == DNNS_F32 ? 0x7FFFFFFFu : 0x7FFF7FFFu;
    __shared__ uint32_t s_ebits[2][kTileElems / 32];
    __shared__ uint32_t s_kbits[2][DO_STRUCT ? kTileElems / 32 + 1 : 1];
    __shared__ uint32_t scratch[33];
    const int lane = threadIdx.x & 31;
    const bool word_lane = (lane & (G - 1)) == 0;
    int buf = 0;

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
            uint32_t* ebits = s_ebits[buf];

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
                        if (word_lane) ebits[vi / G] = nz_word;
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
                        if (word_lane) ebits[vi / G] = word;
                    }
                }
            }
            if (DO_STRUCT) {
                __syncthreads();
                tile_structures(d, e0, n_e, ebits, s_kbits[buf], nz_map, out_nz, in_nz);
                buf ^= 1;
            }
        }
    }
}

template <int DT>
void launch_dt(bool do_mask, bool do_struct, dim3 grid, cudaStream_t st, const Tables& tb, const ThresholdWs& ws,
               const dnns_threshold* thr, int variant, const char* src_arena, char* dst_arena, uint32_t* mask_bits,
               uint32_t* nz_map, uint32_t* out_nz, uint32_t* in_nz) {
    if (do_mask && do_struct)
        k_sweep<DT, true, true><<<grid, kTileThreads, 0, st>>>(tb, ws, thr, variant, src_arena, dst_arena, mask_bits,
                                                               nz_map, out_nz, in_nz);
    else if (do_mask)
        k_sweep<DT, true, false><<<grid, kTileThreads, 0, st>>>(tb, ws, thr, variant, src_arena, dst_arena, mask_bits,
                                                                nz_map, out_nz, in_nz);
    else
        k_sweep<DT, false, true><<<grid, kTileThreads, 0, st>>>(tb, ws, thr, variant, src_arena, dst_arena, mask_bits,
                                                                nz_map, out_nz, in_nz);
}

}  // namespace

int launch_tile_sweep(const Tables& tb, const ThresholdWs& ws, bool do_mask, bool do_struct,
                      const dnns_threshold* thr_dev, int variant, const void* src_arena, void* dst_arena,
                      uint32_t* mask_bits, uint32_t* nz_map, uint32_t* out_nz, uint32_t* in_nz, int n_sm,
                      cudaStream_t st) {
    const dim3 grid(min((uint32_t)n_sm * 4u, tb.n_tiles));
    if (tb.dtype == DNNS_F32)
        launch_dt<DNNS_F32>(do_mask, do_struct, grid, st, tb, ws, thr_dev, variant, (const char*)src_arena,
                            (char*)dst_arena, mask_bits, nz_map, out_nz, in_nz);
    else
        launch_dt<DNNS_BF16>(do_mask, do_struct, grid, st, tb, ws, thr_dev, variant, (const char*)src_arena,
                             (char*)dst_arena, mask_bits, nz_map, out_nz, in_nz);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace dnns
