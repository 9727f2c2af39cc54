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
//           between tiles to mask exactly k weights.
#include "dnns_internal.cuh"

namespace dnns {

namespace {

constexpr int kHistThreads = 1024;

// Visit the vectors of elements [e0, e1) of one tensor with all threads of the block; e0 is a
// multiple of the vector width.  f(vector, n_valid) is called once per vector.
template <int DT, int THREADS, typename F>
__device__ __forceinline__ void for_each_vec(const void* base, uint32_t e0, uint32_t e1, uint32_t numel, F f) {
    constexpr uint32_t P = Elem<DT>::kPerVec;
    constexpr int U = 4;
    const uint32_t v0 = e0 / P, v1 = (e1 + P - 1) / P;
    uint32_t i = v0 + threadIdx.x;
    for (; i + (U - 1) * THREADS < v1; i += U * THREADS) {
        uint4 v[U];
        int n[U];
#pragma unroll
        for (int u = 0; u < U; ++u) n[u] = load_vec<DT>(base, (i + u * THREADS) * P, numel, v[u]);
#pragma unroll
        for (int u = 0; u < U; ++u) f(v[u], n[u]);
    }
    for (; i < v1; i += THREADS) {
        uint4 v;
        const int n = load_vec<DT>(base, i * P, numel, v);
        f(v, n);
    }
}

// ---------------------------------------------------------------- pass 1
template <int DT>
__global__ void __launch_bounds__(kHistThreads, 1) k_hist1(Tables tb, uint32_t* __restrict__ hist1) {
    extern __shared__ uint32_t sh[];  // kHistBins counters
    for (uint32_t b = threadIdx.x; b < kHistBins; b += kHistThreads) sh[b] = 0;
    __syncthreads();

    const uint32_t per = (tb.n_tiles + gridDim.x - 1) / gridDim.x;
    const uint32_t lo = min(tb.n_tiles, blockIdx.x * per), hi = min(tb.n_tiles, lo + per);
    int cur_seg = -1;
    uint32_t zeros = 0;  // keys with first digit 0 (exact zeros, mostly): counted in a register

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
            const uint32_t e0 = (tile - d.tile0) * tb.tile_elems;
            const uint32_t e1 = min(d.numel, (span_end - d.tile0) * tb.tile_elems);
            for_each_vec<DT, kHistThreads>(d.src, e0, e1, d.numel, [&](const uint4& v, int n) {
                uint32_t key[Elem<DT>::kPerVec];
                vec_keys<DT>(v, key);
#pragma unroll
                for (int j = 0; j < Elem<DT>::kPerVec; ++j) {
                    const uint32_t dg = digit_of<DT>(key[j]);
                    if (j < n) {
                        if (dg == 0) ++zeros;
                        else atomicAdd(&sh[dg], 1u);
                    }
                }
            });
        }
        tile = span_end;
    }
    flush(cur_seg);
}

// ---------------------------------------------------------------- select 1
// One block per segment.  Thread t owns bins [32t, 32t+32).
template <int DT>
__global__ void __launch_bounds__(1024) k_select1(Tables tb, ThresholdWs ws, int n_k, dnns_threshold* __restrict__ thr) {
    __shared__ uint64_t scratch[33];
    __shared__ uint32_t s_digit[kMaxVariants];
    const uint32_t seg = blockIdx.x, S = tb.n_segs;
    const uint32_t* h = ws.hist1 + (size_t)seg * kHistBins;
    uint32_t c[32];
    uint64_t sum = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint4 v = reinterpret_cast<const uint4*>(h)[threadIdx.x * 8 + j];
        c[4 * j] = v.x, c[4 * j + 1] = v.y, c[4 * j + 2] = v.z, c[4 * j + 3] = v.w;
        sum += (uint64_t)v.x + v.y + v.z + v.w;
    }
    uint64_t total;
    const uint64_t excl = block_exclusive_scan<uint64_t>(sum, scratch, &total);
    uint32_t* bm = ws.bitmap + (size_t)seg * kBitmapWords;
    bm[threadIdx.x] = 0;  // 1024 words
    for (int v = 0; v < n_k; ++v) {
        const uint64_t k = ws.k_dev[(size_t)v * S + seg];
        SelectState* st = &ws.sel[(size_t)v * S + seg];
        if (k == 0) {
            if (threadIdx.x == 0) {
                *st = SelectState{0, 0, 0xFFFFFFFFu, 0, 0, 0};
                s_digit[v] = 0xFFFFFFFFu;
            }
            continue;
        }
        if (excl < k && k <= excl + sum) {
            // b = the first of this thread's bins whose inclusive prefix reaches k
            uint64_t cum = excl;
            int b = 0;
            uint32_t cnt = 0;
            bool found = false;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                if (!found) {
                    if (cum + c[j] >= k) {
                        b = j;
                        cnt = c[j];
                        found = true;
                    } else {
                        cum += c[j];
                    }
                }
            }
            const uint32_t digit = threadIdx.x * 32 + b;
            *st = SelectState{k, cum, digit, 0, cnt, 0};
            s_digit[v] = digit;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        // variants that selected the same first digit share one second-pass histogram
        int n_slots = 0;
        for (int v = 0; v < n_k; ++v) {
            const uint32_t dg = s_digit[v];
            if (dg == 0xFFFFFFFFu) continue;
            int slot = -1;
            for (int u = 0; u < v; ++u)
                if (s_digit[u] == dg) {
                    slot = (int)ws.sel[(size_t)u * S + seg].slot;
                    break;
                }
            if (slot < 0) {
                slot = n_slots++;
                bm[dg >> 5] |= 1u << (dg & 31);
            }
            ws.sel[(size_t)v * S + seg].slot = (uint32_t)slot;
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
            if (need) atomicOr(ws.any_need, 1u);
        }
    }
}

// ---------------------------------------------------------------- pass 2 (31-bit keys)
__global__ void __launch_bounds__(kTileThreads) k_hist2(Tables tb, ThresholdWs ws, int n_k) {
    __shared__ uint32_t s_bm[kBitmapWords];
    __shared__ uint32_t s_digit[kMaxVariants], s_slot[kMaxVariants];
    const uint32_t S = tb.n_segs;
    int cur_seg = -1;
    for (uint32_t tile = blockIdx.x; tile < tb.n_tiles; tile += gridDim.x) {
        const TensorDesc& d = tb.tensors[tb.tile_tensor[tile]];
        if (d.seg < 0) continue;
        if (d.seg != cur_seg) {
            __syncthreads();
            cur_seg = d.seg;
            for (uint32_t w = threadIdx.x; w < kBitmapWords; w += kTileThreads)
                s_bm[w] = ws.bitmap[(size_t)cur_seg * kBitmapWords + w];
            if ((int)threadIdx.x < n_k) {
                const SelectState st = ws.sel[(size_t)threadIdx.x * S + cur_seg];
                s_digit[threadIdx.x] = st.digit;
                s_slot[threadIdx.x] = st.slot;
            }
            __syncthreads();
        }
        uint32_t* h2 = ws.hist2 + (size_t)cur_seg * n_k * kLowBins;
        const uint32_t e0 = (tile - d.tile0) * tb.tile_elems;
        uint4 v[kVecPerThread];
        int n[kVecPerThread];
#pragma unroll
        for (int u = 0; u < kVecPerThread; ++u)
            n[u] = load_vec<DNNS_F32>(d.src, e0 + (u * kTileThreads + threadIdx.x) * 4, d.numel, v[u]);
#pragma unroll
        for (int u = 0; u < kVecPerThread; ++u) {
            uint32_t key[4];
            vec_keys<DNNS_F32>(v[u], key);
            bool hit[4];
            bool any = false;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t dg = key[j] >> 16;
                hit[j] = j < n[u] && ((s_bm[dg >> 5] >> (dg & 31)) & 1u);
                any |= hit[j];
            }
            if (!__any_sync(0xffffffffu, any)) continue;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const unsigned act = __ballot_sync(0xffffffffu, hit[j]);
                if (!hit[j]) continue;
                const unsigned peers = __match_any_sync(act, key[j]);
                if ((threadIdx.x & 31) == (unsigned)(__ffs(peers) - 1)) {
                    const uint32_t dg = key[j] >> 16;
                    uint32_t slot = 0;
                    for (int vv = 0; vv < n_k; ++vv)
                        if (s_digit[vv] == dg) {
                            slot = s_slot[vv];
                            break;
                        }
                    atomicAdd(&h2[(size_t)slot * kLowBins + (key[j] & 0xFFFFu)], (uint32_t)__popc(peers));
                }
            }
        }
    }
}

// ---------------------------------------------------------------- select 2 (31-bit keys)
// One block per (variant, segment).  Thread t owns low digits [64t, 64t+64).
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
    const uint32_t* h = ws.hist2 + ((size_t)seg * n_k + st.slot) * kLowBins;
    uint64_t sum = 0;
    for (int j = 0; j < 16; ++j) {
        const uint4 q = reinterpret_cast<const uint4*>(h)[threadIdx.x * 16 + j];
        sum += (uint64_t)q.x + q.y + q.z + q.w;
    }
    uint64_t total;
    const uint64_t excl = st.below + block_exclusive_scan<uint64_t>(sum, scratch, &total);
    if (excl < st.k && st.k <= excl + sum) {
        uint64_t cum = excl;
        uint32_t b = 0, cnt = 0;
        for (int j = 0; j < 64; ++j) {
            const uint32_t cj = h[threadIdx.x * 64 + j];
            if (cum + cj >= st.k) {
                b = j;
                cnt = cj;
                break;
            }
            cum += cj;
        }
        dnns_threshold r;
        r.tau_bits = (st.digit << 16) | (threadIdx.x * 64 + b);
        r.pad = 0;
        r.n_below = cum;
        r.n_tie = st.k - cum;
        r.n_equal = cnt;
        thr[idx] = r;
        const uint32_t need = r.n_tie < r.n_equal;
        ws.need[idx] = need;
        if (need) atomicOr(ws.any_need, 1u);
    }
}

// ---------------------------------------------------------------- tie counts per tile
template <int DT>
__global__ void __launch_bounds__(kTileThreads) k_ties(Tables tb, ThresholdWs ws, int n_k,
                                                       const dnns_threshold* __restrict__ thr) {
    if (*ws.any_need == 0) return;
    __shared__ uint32_t s_bm[kBitmapWords];
    __shared__ uint32_t s_tau[kMaxVariants], s_need[kMaxVariants], s_cnt[kMaxVariants];
    __shared__ uint32_t s_any;
    const uint32_t S = tb.n_segs;
    int cur_seg = -1;
    for (uint32_t tile = blockIdx.x; tile < tb.n_tiles; tile += gridDim.x) {
        const TensorDesc& d = tb.tensors[tb.tile_tensor[tile]];
        if (d.seg < 0) continue;
        if (d.seg != cur_seg) {
            __syncthreads();
            cur_seg = d.seg;
            if (threadIdx.x == 0) s_any = 0;
            __syncthreads();
            for (uint32_t w = threadIdx.x; w < kBitmapWords; w += kTileThreads)
                s_bm[w] = ws.bitmap[(size_t)cur_seg * kBitmapWords + w];
            if ((int)threadIdx.x < n_k) {
                const size_t idx = (size_t)threadIdx.x * S + cur_seg;
                s_tau[threadIdx.x] = thr[idx].tau_bits;
                s_need[threadIdx.x] = ws.need[idx];
                s_cnt[threadIdx.x] = 0;
                if (ws.need[idx]) s_any = 1;
            }
            __syncthreads();
        }
        if (!s_any) continue;
        const uint32_t e0 = (tile - d.tile0) * tb.tile_elems;
        uint4 v[kVecPerThread];
        int n[kVecPerThread];
#pragma unroll
        for (int u = 0; u < kVecPerThread; ++u)
            n[u] = load_vec<DT>(d.src, e0 + (u * kTileThreads + threadIdx.x) * Elem<DT>::kPerVec, d.numel, v[u]);
#pragma unroll
        for (int u = 0; u < kVecPerThread; ++u) {
            uint32_t key[Elem<DT>::kPerVec];
            vec_keys<DT>(v[u], key);
#pragma unroll
            for (int j = 0; j < Elem<DT>::kPerVec; ++j) {
                const uint32_t dg = digit_of<DT>(key[j]);
                if (j < n[u] && ((s_bm[dg >> 5] >> (dg & 31)) & 1u)) {
                    for (int vv = 0; vv < n_k; ++vv)
                        if (s_need[vv] && s_tau[vv] == key[j]) atomicAdd(&s_cnt[vv], 1u);
                }
            }
        }
        __syncthreads();
        if ((int)threadIdx.x < n_k) {
            ws.tile_ties[(size_t)threadIdx.x * tb.n_tiles + tile] = s_cnt[threadIdx.x];
            s_cnt[threadIdx.x] = 0;
        }
        __syncthreads();
    }
}

// Exclusive scan of the tile counts over the tiles of a segment, one block per (variant, segment).
__global__ void __launch_bounds__(1024) k_tie_scan(Tables tb, ThresholdWs ws) {
    if (*ws.any_need == 0) return;
    __shared__ uint32_t scratch[33];
    const uint32_t S = tb.n_segs;
    const uint32_t v = blockIdx.x / S, seg = blockIdx.x % S;
    if (!ws.need[(size_t)v * S + seg]) return;
    const SegDesc sd = tb.segs[seg];
    const uint32_t* cnt = ws.tile_ties + (size_t)v * tb.n_tiles;
    uint32_t* pre = ws.tie_prefix + (size_t)v * tb.n_tiles;
    uint32_t carry = 0;
    for (uint32_t base = sd.tile_begin; base < sd.tile_end; base += 1024) {
        const uint32_t t = base + threadIdx.x;
        const uint32_t x = t < sd.tile_end ? cnt[t] : 0;
        uint32_t total;
        const uint32_t ex = block_exclusive_scan<uint32_t>(x, scratch, &total);
        if (t < sd.tile_end) pre[t] = carry + ex;
        carry += total;
    }
}

}  // namespace

cudaError_t init_kernel_attributes() {
    cudaError_t e = cudaFuncSetAttribute(k_hist1<DNNS_F32>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)(kHistBins * 4));
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(k_hist1<DNNS_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kHistBins * 4));
}

int launch_threshold(const Tables& tb, const ThresholdWs& ws, int n_k, int /*n_k_stride*/, dnns_threshold* thr_dev,
                     int n_sm, cudaStream_t st) {
    const uint32_t S = tb.n_segs;
    const int hist_grid = (int)min((uint32_t)n_sm, tb.n_tiles);
    const int sweep_grid = (int)min((uint32_t)n_sm * 8u, tb.n_tiles);
    int launches = 0;
    if (tb.dtype == DNNS_F32) {
        k_hist1<DNNS_F32><<<hist_grid, kHistThreads, kHistBins * 4, st>>>(tb, ws.hist1);
        k_select1<DNNS_F32><<<S, 1024, 0, st>>>(tb, ws, n_k, thr_dev);
        k_hist2<<<sweep_grid, kTileThreads, 0, st>>>(tb, ws, n_k);
        k_select2<<<S * n_k, 1024, 0, st>>>(tb, ws, n_k, thr_dev);
        k_ties<DNNS_F32><<<sweep_grid, kTileThreads, 0, st>>>(tb, ws, n_k, thr_dev);
        launches = 5;
    } else {
        k_hist1<DNNS_BF16><<<hist_grid, kHistThreads, kHistBins * 4, st>>>(tb, ws.hist1);
        k_select1<DNNS_BF16><<<S, 1024, 0, st>>>(tb, ws, n_k, thr_dev);
        k_ties<DNNS_BF16><<<sweep_grid, kTileThreads, 0, st>>>(tb, ws, n_k, thr_dev);
        launches = 3;
    }
    k_tie_scan<<<S * n_k, 1024, 0, st>>>(tb, ws);
    ++launches;
    return cudaGetLastError() == cudaSuccess ? launches : -1;
}

}  // namespace dnns
