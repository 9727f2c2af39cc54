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

// OR `bits` into a global flag word unless they are already there.  The plain read may be stale,
// which only costs a redundant atomic; flags saturate early in a sweep, so almost every update
// ends at the read.
__device__ __forceinline__ void or_if_missing(uint32_t* word, uint32_t bits) {
    if ((__ldcg(word) & bits) != bits) atomicOr(word, bits);
}

// From the element bits of one tile (elements [e0, e0+n_e) of tensor d) to kernel map, filter
// flags and input-column flags.  Kernel q = (o, i) covers elements [q*KK, (q+1)*KK); a kernel cut
// by the tile edge is OR-ed by both tiles.  s_kbits receives the kernel bits of the tile, kernel
// q at bit q - (q0 & ~31); for 1x1 kernels the element bits are used as they are.
// Ends with a barrier, after which ebits and s_kbits may be overwritten.
__device__ void tile_structures(const TensorDesc& d, uint32_t e0, uint32_t n_e, const uint32_t* ebits,
                                uint32_t* s_kbits, uint32_t* nz_map, uint32_t* out_nz, uint32_t* in_nz) {
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
            if (lane == 0) s_kbits[w] = word;
        }
        __syncthreads();
        kbits = s_kbits;
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
            const uint32_t o = qb / I, iw = (qb - o * I) >> 5;
            or_if_missing(&g_in[iw], bits);
            or_if_missing(&g_out[o >> 5], 1u << (o & 31));
        } else {
            while (bits) {
                const uint32_t q = qb + __ffs(bits) - 1;
                bits &= bits - 1;
                const uint32_t o = q / I, i = q - o * I;
                or_if_missing(&g_in[i >> 5], 1u << (i & 31));
                or_if_missing(&g_out[o >> 5], 1u << (o & 31));
            }
        }
    }
    __syncthreads();
}

template <int DT, bool DO_MASK, bool DO_STRUCT>
__global__ void __launch_bounds__(kTileThreads) k_sweep(Tables tb, ThresholdWs ws, const dnns_threshold* __restrict__ thr,
                                                        int variant, const char* src_arena, char* dst_arena,
                                                        uint32_t* mask_bits, uint32_t* nz_map, uint32_t* out_nz,
                                                        uint32_t* in_nz) {
    constexpr int P = Elem<DT>::kPerVec;
    constexpr int G = 32 / P;  // lanes per bit word
    __shared__ uint32_t s_ebits[kTileBytes / Elem<DT>::kBytes / 32];
    __shared__ uint32_t s_kbits[DO_STRUCT ? kTileBytes / Elem<DT>::kBytes / 32 + 1 : 1];
    __shared__ uint32_t scratch[33];
    const int lane = threadIdx.x & 31;

    for (uint32_t tile = blockIdx.x; tile < tb.n_tiles; tile += gridDim.x) {
        const TensorDesc& d = tb.tensors[tb.tile_tensor[tile]];
        const uint32_t e0 = (tile - d.tile0) * tb.tile_elems;
        const uint32_t n_e = min(tb.tile_elems, d.numel - e0);
        const char* src = src_arena ? src_arena + d.arena_off : static_cast<const char*>(d.src);
        char* dst = nullptr;

        // How this tile treats its keys: keep iff key >= thr_eff, except in the one tile per
        // segment where the ties split (split = true: ties ranked below `quota` are masked).
        uint32_t thr_eff = 0, tau = 0, quota = 0;
        bool split = false;
        if (DO_MASK) {
            dst = dst_arena ? dst_arena + d.arena_off : static_cast<char*>(const_cast<void*>(d.src));
            if (d.seg >= 0) {
                const dnns_threshold r = thr[(size_t)variant * tb.n_segs + d.seg];
                tau = r.tau_bits;
                if (r.n_below + r.n_tie == 0) {
                    thr_eff = 0;  // k = 0
                } else if (r.n_tie >= r.n_equal) {
                    thr_eff = tau + 1;  // every key equal to tau is masked
                } else {
                    const uint64_t before = ws.tie_prefix[(size_t)variant * tb.n_tiles + tile];
                    const uint64_t here = ws.tile_ties[(size_t)variant * tb.n_tiles + tile];
                    if (before >= r.n_tie) thr_eff = tau;
                    else if (before + here <= r.n_tie) thr_eff = tau + 1;
                    else {
                        thr_eff = tau + 1;
                        split = true;
                        quota = (uint32_t)(r.n_tie - before);
                    }
                }
            } else if (dst == src && !DO_STRUCT && !mask_bits) {
                continue;  // untouched tensor, in place, nothing else to produce
            }
        }

        uint4 v[kVecPerThread];
        int n[kVecPerThread];
#pragma unroll
        for (int u = 0; u < kVecPerThread; ++u)
            n[u] = load_vec<DT, !DO_MASK>(src, e0 + (u * kTileThreads + threadIdx.x) * P, d.numel, v[u]);

        uint32_t tie_carry = 0;
#pragma unroll
        for (int u = 0; u < kVecPerThread; ++u) {
            const uint32_t vi = u * kTileThreads + threadIdx.x;  // vector index inside the tile
            uint32_t key[P];
            vec_keys<DT>(v[u], key);
            uint32_t keep = 0, nz = 0;
            if (DO_MASK) {
                uint32_t tie_rank = 0;
                if (split) {
                    uint32_t c = 0;
#pragma unroll
                    for (int j = 0; j < P; ++j) c += (j < n[u] && key[j] == tau);
                    uint32_t total;
                    tie_rank = tie_carry + block_exclusive_scan<uint32_t>(c, scratch, &total);
                    tie_carry += total;
                }
#pragma unroll
                for (int j = 0; j < P; ++j) {
                    bool k = key[j] >= thr_eff;
                    if (split && key[j] == tau) k = tie_rank++ >= quota;
                    k = k && j < n[u];
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
                store_vec<DT>(dst, e0 + vi * P, d.numel, make_uint4(w[0], w[1], w[2], w[3]));
                if (mask_bits) {
                    const uint32_t word = gather_word<P>(keep, lane);
                    if ((lane & (G - 1)) == 0 && (vi / G) * 32 < n_e) mask_bits[d.off_mask + e0 / 32 + vi / G] = word;
                }
            } else {
#pragma unroll
                for (int j = 0; j < P; ++j) nz |= (uint32_t)(j < n[u] && key[j] != 0) << j;
            }
            if (DO_STRUCT) {
                const uint32_t word = gather_word<P>(nz, lane);
                if ((lane & (G - 1)) == 0) s_ebits[vi / G] = word;
            }
        }
        if (DO_STRUCT) {
            __syncthreads();
            tile_structures(d, e0, n_e, s_ebits, s_kbits, nz_map, out_nz, in_nz);
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
    const dim3 grid(min((uint32_t)n_sm * 8u, tb.n_tiles));
    if (tb.dtype == DNNS_F32)
        launch_dt<DNNS_F32>(do_mask, do_struct, grid, st, tb, ws, thr_dev, variant, (const char*)src_arena,
                            (char*)dst_arena, mask_bits, nz_map, out_nz, in_nz);
    else
        launch_dt<DNNS_BF16>(do_mask, do_struct, grid, st, tb, ws, thr_dev, variant, (const char*)src_arena,
                             (char*)dst_arena, mask_bits, nz_map, out_nz, in_nz);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace dnns
