// Zero structures of a whole portfolio from ONE sweep over the dense weights (Module 2, the Sparsity
// Analyser, for every variant at once).  The sweep does not depend on the thresholds and is enqueued by the
// threshold call, beside its ranking kernels; the flag kernel runs once the thresholds are known.
//
// Step 2 keeps a weight of variant v when its magnitude key lies above tau_v, or equals tau_v and the
// weight comes at or after the place where v stops masking such weights.  A filter (row) of a tensor
// therefore still holds something for variant v exactly when its LARGEST key does - and so does an
// input column.  The sweep records, per filter and per input column of every tensor, the largest key;
// a small kernel then compares those maxima with every variant's threshold and writes the variant's
// filter flags and input-column flags.  Only where a maximum equals tau in the one tensor in which the
// variant's equal weights split does it look at the weights again (that row or column alone).
//
//   k_extrema        the sweep: 16 KB tiles, contiguous tile ranges per block, next tile in flight.
//                    Row maxima: warp reduction, one atomic per warp and row.  Column maxima: where the
//                    row length divides the tile, a thread meets the same columns in every tile and
//                    keeps them in registers; otherwise per-vector maxima go to a table in shared
//                    memory.  The table is merged into global memory when the block changes tensor.
//   k_extrema_rows   the same maxima for tensors with long rows of whole 16-byte vectors, row by row (below).
//   k_extrema_flags  per (variant, flag word): 32 comparisons, one ballot, one store.
#include "dnns_internal.cuh"

namespace dnns {

namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr uint32_t kColTab = 8192;  // input columns of a tensor that fit the shared-memory table

template <int DT>
__global__ void __launch_bounds__(kTileThreads, 3) k_extrema(Tables tb, uint32_t* __restrict__ rowmax, uint32_t* __restrict__ colmax) {
    constexpr int P = Elem<DT>::kPerVec;
    constexpr uint32_t kTileElems = kTileBytes / Elem<DT>::kBytes;
    constexpr uint32_t kKeyMask = DT == DNNS_F32 ? 0x7FFFFFFFu : 0x7FFF7FFFu;
    __shared__ uint32_t s_col[kColTab];
    const int lane = threadIdx.x & 31;
    for (uint32_t i = threadIdx.x; i < kColTab; i += kTileThreads) s_col[i] = 0;
    __syncthreads();

    // contiguous tile ranges of about equal cost (tiles of tensors whose column maxima stay in registers are cheaper)
    const uint32_t lo = tb.extrema_bounds[blockIdx.x], hi = tb.extrema_bounds[blockIdx.x + 1];
    uint32_t tile = lo;
    while (tile < hi) {
        // ---- per-tensor context: constant over the run of tiles [tile, span_end)
        const TensorDesc& d = tb.tensors[tb.tile_tensor[tile]];
        const uint32_t span_end = min(hi, d.tile0 + d.n_tiles);
        if (d.by_rows) {  // the row-walking sweep's
            tile = span_end;
            continue;
        }
        const uint32_t numel = d.numel, tile0 = d.tile0, KK = d.KK, I = d.I, L = I * KK;
        const char* src = static_cast<const char*>(d.src);
        uint32_t* g_row = rowmax + d.off_row;
        uint32_t* g_col = colmax + d.off_col;
        const bool tab = I <= kColTab;                                      // column maxima through the shared table
        const bool fixed_cols = kTileElems % L == 0 && L % P == 0 && tab;  // a thread meets the same columns in every tile
        const bool warp_in_row = L % (32u * P) == 0;                       // the 32 vectors a warp holds never straddle rows
        const uint64_t inv_L = ~0ull / L + 1;  // e / L = umul64hi(e, inv_L) for e, L < 2^32 (L a power of two: wraps to the exact quotient)
        const bool lean = L % P == 0 && L >= 32u * P;  // whole tiles of such tensors take the short path below
        const uint32_t step_row = (kTileThreads * P) / L, step_pos = (kTileThreads * P) - step_row * L;
        auto col_max = [&](uint32_t col, uint32_t m) {
            if (tab) atomicMax(&s_col[col], m);
            else atomicMax(&g_col[col], m);
        };
        uint32_t acc[kVecPerThread][4];  // fixed_cols: running maxima of this thread's words (both halves for 2-byte keys)
#pragma unroll
        for (int u = 0; u < kVecPerThread; ++u)
#pragma unroll
            for (int w = 0; w < 4; ++w) acc[u][w] = 0;

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
            const uint32_t e0 = (tile - tile0) * kTileElems;
            if (lean && e0 + kTileElems <= numel) {
                // ---- a whole tile of a tensor whose rows are multiples of a vector and at least a warp's span long:
                // every vector lies in one row, a warp's 32 vectors in at most two neighbouring rows
                uint32_t r0 = (uint32_t)__umul64hi((uint64_t)(e0 + threadIdx.x * P), inv_L), pos0 = e0 + threadIdx.x * P - r0 * L;
#pragma unroll
                for (int u = 0; u < kVecPerThread; ++u) {
                    uint32_t key[P];
                    vec_keys<DT>(v[u], key);
                    uint32_t m = key[0];
#pragma unroll
                    for (int j = 1; j < P; ++j) m = max(m, key[j]);
                    const uint32_t ra = __shfl_sync(kFull, r0, 0);
                    const uint32_t ma = __reduce_max_sync(kFull, r0 == ra ? m : 0u), mb = __reduce_max_sync(kFull, r0 == ra ? 0u : m);
                    if (lane == 0) {
                        if (ma) atomicMax(&g_row[ra], ma);
                        if (mb) atomicMax(&g_row[ra + 1], mb);
                    }
                    if (fixed_cols) {
                        const uint32_t w[4] = {v[u].x & kKeyMask, v[u].y & kKeyMask, v[u].z & kKeyMask, v[u].w & kKeyMask};
#pragma unroll
                        for (int k = 0; k < 4; ++k) acc[u][k] = DT == DNNS_F32 ? max(acc[u][k], w[k]) : __vmaxu2(acc[u][k], w[k]);
                    } else if (KK == 9) {
                        const uint32_t col = pos0 / 9u, first = 9u - (pos0 - col * 9u);  // elements of the vector in column `col`
                        uint32_t ca = 0, cb = 0;
#pragma unroll
                        for (int j = 0; j < P; ++j) {
                            ca = max(ca, (uint32_t)j < first ? key[j] : 0u);
                            cb = max(cb, (uint32_t)j < first ? 0u : key[j]);
                        }
                        if (ca) col_max(col, ca);
                        if (cb) col_max(col + 1, cb);
                    } else {
                        uint32_t col = KK == 1 ? pos0 : pos0 / KK, rem = pos0 - col * KK, cur = 0;
#pragma unroll
                        for (int j = 0; j < P; ++j) {
                            if (rem == KK) {
                                if (cur) col_max(col, cur);
                                ++col, rem = 0, cur = 0;
                            }
                            cur = max(cur, key[j]);
                            ++rem;
                        }
                        if (cur) col_max(col, cur);
                    }
                    // the thread's next vector lies kTileThreads * P elements further on
                    r0 += step_row;
                    pos0 += step_pos;
                    if (pos0 >= L) pos0 -= L, ++r0;
                }
                continue;
            }
#pragma unroll
            for (int u = 0; u < kVecPerThread; ++u) {
                const uint32_t e = e0 + (u * kTileThreads + threadIdx.x) * P;
                const int n = e >= numel ? 0 : (int)min((uint32_t)P, numel - e);  // valid elements
                const uint32_t r0 = L == 1 ? e : (uint32_t)__umul64hi((uint64_t)e, inv_L), pos0 = e - r0 * L;  // e / L, e % L
                const bool whole = n > 0 && pos0 + (uint32_t)n <= L;  // the vector lies in one row
                uint32_t key[P];
                vec_keys<DT>(v[u], key);
                uint32_t m = 0;
#pragma unroll
                for (int j = 0; j < P; ++j) m = max(m, j < n ? key[j] : 0u);
                // ---- row maxima: one atomic per row that the warp's 32 vectors touch
                if (warp_in_row) {  // the 32 vectors of the warp lie in one row (a ragged end holds zeros)
                    const uint32_t mm = __reduce_max_sync(kFull, m);
                    if (lane == 0 && mm) atomicMax(&g_row[r0], mm);
                } else {
                    const bool has = whole && m != 0;
                    unsigned todo = __ballot_sync(kFull, has);
                    while (todo) {
                        const int leader = __ffs(todo) - 1;
                        const uint32_t rr = __shfl_sync(kFull, r0, leader);
                        const bool mine = has && r0 == rr;
                        const unsigned grp = __ballot_sync(kFull, mine);
                        if (mine) {
                            const uint32_t mm = __reduce_max_sync(grp, m);
                            if (lane == leader) atomicMax(&g_row[rr], mm);
                        }
                        todo &= ~grp;
                    }
                }
                // ---- column maxima
                if (fixed_cols) {
                    // (a ragged vector holds zeros past the end of the tensor: harmless)
                    const uint32_t w[4] = {v[u].x & kKeyMask, v[u].y & kKeyMask, v[u].z & kKeyMask, v[u].w & kKeyMask};
#pragma unroll
                    for (int k = 0; k < 4; ++k) acc[u][k] = DT == DNNS_F32 ? max(acc[u][k], w[k]) : __vmaxu2(acc[u][k], w[k]);
                } else if (whole && n == P && KK == 9) {
                    // 3x3 kernels: the P <= 9 elements of the vector belong to one column or to two neighbours
                    const uint32_t col = pos0 / 9u, first = 9u - (pos0 - col * 9u);  // elements of the vector in column `col`
                    uint32_t ma = 0, mb = 0;
#pragma unroll
                    for (int j = 0; j < P; ++j) {
                        ma = max(ma, (uint32_t)j < first ? key[j] : 0u);
                        mb = max(mb, (uint32_t)j < first ? 0u : key[j]);
                    }
                    if (ma) col_max(col, ma);
                    if (mb) col_max(col + 1, mb);
                } else if (n > 0) {
                    if (whole) {
                        // runs of elements of one column: one table update per run
                        uint32_t col = KK == 1 ? pos0 : pos0 / KK, rem = pos0 - col * KK, cur = 0;
#pragma unroll
                        for (int j = 0; j < P; ++j) {
                            if (j < n) {
                                if (rem == KK) {
                                    if (cur) col_max(col, cur);
                                    ++col, rem = 0, cur = 0;
                                }
                                cur = max(cur, key[j]);
                                ++rem;
                            }
                        }
                        if (cur) col_max(col, cur);
                    } else {
                        // the vector crosses into the next row: element by element, rows included
#pragma unroll
                        for (int j = 0; j < P; ++j) {  // (unrolled: the keys stay in registers)
                            if (j < n && key[j]) {
                                const uint32_t ee = e + j, r = ee / L, pos = ee - r * L;
                                atomicMax(&g_row[r], key[j]);
                                col_max(pos / KK, key[j]);
                            }
                        }
                    }
                }
            }
        }
        // ---- the block leaves the tensor: registers to table, table to global memory
        if (fixed_cols) {
#pragma unroll
            for (int u = 0; u < kVecPerThread; ++u) {
                const uint32_t pos0 = ((u * kTileThreads + threadIdx.x) * P) % L;  // L divides the tile and is a multiple of P
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (DT == DNNS_F32) {
                        if (acc[u][k]) atomicMax(&s_col[(pos0 + k) / KK], acc[u][k]);
                    } else {
                        const uint32_t a = acc[u][k] & 0xFFFFu, b = acc[u][k] >> 16;
                        if (a) atomicMax(&s_col[(pos0 + 2 * k) / KK], a);
                        if (b) atomicMax(&s_col[(pos0 + 2 * k + 1) / KK], b);
                    }
                }
            }
        }
        if (tab) {
            __syncthreads();
            for (uint32_t i = threadIdx.x; i < I; i += kTileThreads) {
                const uint32_t m = s_col[i];
                if (m) {
                    atomicMax(&g_col[i], m);
                    s_col[i] = 0;
                }
            }
            __syncthreads();
        }
    }
}

// The same maxima for tensors with long rows of whole 16-byte vectors, row by row: a block takes a unit (a block of
// rows by a chunk of at most 128 vectors of every row), a warp takes every eighth row of it, a lane the vectors
// lane, lane + 32, .. of the chunk.  A lane thus meets the same columns in every row and keeps their maxima in
// registers - no index arithmetic per key - and a row's maximum is one warp reduction and one atomic per row and
// chunk.  At the end of the unit the warps' column maxima meet in shared memory and go out, one atomic per
// element column.
template <int DT>
__global__ void __launch_bounds__(kTileThreads, 3) k_extrema_rows(Tables tb, uint32_t* __restrict__ rowmax, uint32_t* __restrict__ colmax) {
    constexpr int P = Elem<DT>::kPerVec;
    constexpr int kV = kExtremaChunkVecs / 32;  // vectors of a row per lane
    constexpr uint32_t kKeyMask = DT == DNNS_F32 ? 0x7FFFFFFFu : 0x7FFF7FFFu;
    constexpr int kWarps = kTileThreads / 32;
    __shared__ uint32_t s_col[kExtremaChunkVecs * P];  // largest key per element column of the chunk
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (uint32_t unit = blockIdx.x; unit < tb.n_extrema_units; unit += gridDim.x) {
        const ExtremaUnit un = tb.extrema_units[unit];
        const TensorDesc& d = tb.tensors[un.tensor];
        const uint32_t KK = d.KK, L = (uint32_t)d.I * KK;
        const size_t row_bytes = (size_t)L * Elem<DT>::kBytes;
        const char* chunk = static_cast<const char*>(d.src) + (size_t)un.vec0 * 16;
        for (uint32_t i = threadIdx.x; i < kExtremaChunkVecs * P; i += kTileThreads) s_col[i] = 0;
        __syncthreads();
        uint32_t acc[kV][4];
#pragma unroll
        for (int k = 0; k < kV; ++k)
#pragma unroll
            for (int w = 0; w < 4; ++w) acc[k][w] = 0;
        uint4 nxt[kV];
        auto issue = [&](uint32_t r) {
            const uint4* p = reinterpret_cast<const uint4*>(chunk + (size_t)r * row_bytes);
#pragma unroll
            for (int k = 0; k < kV; ++k)
                nxt[k] = (uint32_t)(lane + 32 * k) < un.n_vec ? __ldg(p + lane + 32 * k) : make_uint4(0, 0, 0, 0);
        };
        const uint32_t r_end = un.row0 + un.n_rows;
        uint32_t r = un.row0 + warp;
        if (r < r_end) issue(r);
        for (; r < r_end; r += kWarps) {
            uint4 v[kV];
#pragma unroll
            for (int k = 0; k < kV; ++k) v[k] = nxt[k];
            if (r + kWarps < r_end) issue(r + kWarps);
            uint32_t m = 0;
#pragma unroll
            for (int k = 0; k < kV; ++k) {
                const uint32_t w[4] = {v[k].x & kKeyMask, v[k].y & kKeyMask, v[k].z & kKeyMask, v[k].w & kKeyMask};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    acc[k][q] = DT == DNNS_F32 ? max(acc[k][q], w[q]) : __vmaxu2(acc[k][q], w[q]);
                    m = DT == DNNS_F32 ? max(m, w[q]) : __vmaxu2(m, w[q]);
                }
            }
            if (DT == DNNS_BF16) m = max(m & 0xFFFFu, m >> 16);
            m = __reduce_max_sync(kFull, m);
            if (lane == 0 && m) atomicMax(&rowmax[d.off_row + r], m);
        }
        // the warps' column maxima meet in shared memory
#pragma unroll
        for (int k = 0; k < kV; ++k) {
            const uint32_t vi = lane + 32 * k;
            if (vi >= un.n_vec) continue;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (DT == DNNS_F32) {
                    if (acc[k][q]) atomicMax(&s_col[vi * P + q], acc[k][q]);
                } else {
                    const uint32_t a = acc[k][q] & 0xFFFFu, b = acc[k][q] >> 16;
                    if (a) atomicMax(&s_col[vi * P + 2 * q], a);
                    if (b) atomicMax(&s_col[vi * P + 2 * q + 1], b);
                }
            }
        }
        __syncthreads();
        // element columns to input columns (KK elements each)
        const uint32_t e0 = un.vec0 * P, n_e = un.n_vec * P;
        for (uint32_t i = threadIdx.x; i < n_e; i += kTileThreads) {
            const uint32_t m = s_col[i];
            if (m) atomicMax(&colmax[d.off_col + (KK == 1 ? e0 + i : (e0 + i) / KK)], m);
        }
        __syncthreads();
    }
}

// Per-variant arguments of the flag kernel.
struct ExtremaFlagArgs {
    int32_t variant[kPortfolioMax];
    uint32_t* out_nz[kPortfolioMax];
    uint32_t* in_nz[kPortfolioMax];
};

template <int DT>
__device__ __forceinline__ uint32_t key_at(const void* src, uint32_t idx) {
    if (DT == DNNS_F32) return __ldg(static_cast<const uint32_t*>(src) + idx) & 0x7FFFFFFFu;
    return __ldg(static_cast<const uint16_t*>(src) + idx) & 0x7FFFu;
}

// One block per (tensor, variant), one warp per flag word: bit = the filter / input column still holds a non-zero
// weight after step 2 of that variant.
template <int DT>
__global__ void __launch_bounds__(256) k_extrema_flags(Tables tb, const uint32_t* __restrict__ rowmax,
                                                       const uint32_t* __restrict__ colmax,
                                                       const dnns_threshold* __restrict__ thr,
                                                       const TieSplit* __restrict__ split, ExtremaFlagArgs fa) {
    const TensorDesc& d = tb.tensors[blockIdx.x];
    const int vslot = blockIdx.y, variant = fa.variant[vslot];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const uint32_t O = d.O, I = d.I, KK = d.KK, L = I * KK;
    // what step 2 does to this tensor: 0 nothing, 1 keep iff key >= thr_eff, 2 the weights equal to tau split inside it
    uint32_t mode = 0, tau = 0, thr_eff = 0, split_elem = 0;
    if (d.seg >= 0) {
        const size_t idx = (size_t)variant * tb.n_segs + d.seg;
        const dnns_threshold r = thr[idx];
        const TieSplit sp = split[idx];
        tau = r.tau_bits;
        if (r.n_below + r.n_tie != 0) {
            if (blockIdx.x == sp.tensor) mode = 2, split_elem = sp.elem;
            else mode = 1, thr_eff = blockIdx.x < sp.tensor ? tau + 1u : tau;
        }
    }
    const uint32_t out_words = (O + 31) / 32, in_words = (I + 31) / 32;
    for (uint32_t w = warp; w < out_words + in_words; w += n_warps) {
        const bool is_row = w < out_words;
        const uint32_t j = (is_row ? w : w - out_words) * 32 + lane, extent = is_row ? O : I;
        uint32_t m = 0;
        if (j < extent) m = is_row ? rowmax[d.off_row + j] : colmax[d.off_col + j];
        bool nz = m != 0 && (mode == 0 || (mode == 1 ? m >= thr_eff : m > tau));
        // the largest key equals tau in the tensor where such weights split: some of them stay, some do not
        unsigned open = __ballot_sync(kFull, j < extent && mode == 2 && tau != 0 && m == tau);
        while (open) {
            const int who = __ffs(open) - 1;
            open &= open - 1;
            const uint32_t jj = (is_row ? w : w - out_words) * 32 + who;
            bool found = false;
            if (is_row) {
                // filter jj: its weights equal to tau stay from element split_elem of the tensor on
                const uint32_t begin = jj * L, end = begin + L;
                if (begin >= split_elem) found = true;
                else if (end > split_elem)
                    for (uint32_t e = split_elem + lane; e < end && !found; e += 32) found = key_at<DT>(d.src, e) == tau;
            } else {
                // input column jj: the KK elements of every filter's 2-D kernel on that column
                for (uint32_t q = lane; q < O * KK && !found; q += 32) {
                    const uint32_t o = q / KK, e = o * L + jj * KK + (q - o * KK);
                    found = e >= split_elem && key_at<DT>(d.src, e) == tau;
                }
            }
            found = __any_sync(kFull, found);
            if (lane == who) nz = found;
        }
        const uint32_t word = __ballot_sync(kFull, nz);
        if (lane == 0) {
            if (is_row) fa.out_nz[vslot][d.off_outnz + w] = word;
            else fa.in_nz[vslot][d.off_innz + (w - out_words)] = word;
        }
    }
}

}  // namespace

int launch_extrema(const Tables& tb, uint32_t* rowmax, uint32_t* colmax, int n_sm, cudaStream_t st) {
    const dim3 grid(min((uint32_t)n_sm * 3u, tb.n_tiles));  // three resident blocks per SM
    int launches = 1;
    if (tb.n_extrema_units) {
        // tensors with long rows of whole vectors, row by row (most of a CNN's weights); the rest tile by tile
        const dim3 grid_rows(min((uint32_t)n_sm * 3u, tb.n_extrema_units));
        ScopedKernel timed("k_extrema_rows", st);
        if (tb.dtype == DNNS_F32) k_extrema_rows<DNNS_F32><<<grid_rows, kTileThreads, 0, st>>>(tb, rowmax, colmax);
        else k_extrema_rows<DNNS_BF16><<<grid_rows, kTileThreads, 0, st>>>(tb, rowmax, colmax);
        ++launches;
    }
    ScopedKernel timed("k_extrema_sweep", st);
    if (tb.dtype == DNNS_F32) k_extrema<DNNS_F32><<<grid, kTileThreads, 0, st>>>(tb, rowmax, colmax);
    else k_extrema<DNNS_BF16><<<grid, kTileThreads, 0, st>>>(tb, rowmax, colmax);
    return cudaGetLastError() == cudaSuccess ? launches : -1;
}

int launch_extrema_flags(const Tables& tb, const uint32_t* rowmax, const uint32_t* colmax, const dnns_threshold* thr,
                         const TieSplit* split, int first_variant, int n_variants, uint32_t* const* out_nz,
                         uint32_t* const* in_nz, cudaStream_t st) {
    ExtremaFlagArgs fa{};
    for (int v = 0; v < n_variants; ++v) fa.variant[v] = first_variant + v, fa.out_nz[v] = out_nz[v], fa.in_nz[v] = in_nz[v];
    ScopedKernel timed("k_extrema_flags", st);
    const dim3 grid(tb.n_tensors, n_variants);
    if (tb.dtype == DNNS_F32) k_extrema_flags<DNNS_F32><<<grid, 256, 0, st>>>(tb, rowmax, colmax, thr, split, fa);
    else k_extrema_flags<DNNS_BF16><<<grid, 256, 0, st>>>(tb, rowmax, colmax, thr, split, fa);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace dnns
