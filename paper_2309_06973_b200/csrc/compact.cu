// Step 5: the rebuild - Module 4, the Model Pruner (Algorithm 2): every layer is re-created with
// |C'_in| x |C'_out| channels and its surviving out-channels, biases and in-channels are moved
// over, all layers in one batch.  Here that is one gather over every tensor, BatchNorm vector
// and bias of the model:
//   layout kernel  sizes each rebuilt item from the keep counts, places it at a 256-byte aligned
//                  offset of the destination arena and cuts it into 16 KB gather units;
//   gather kernel  walks the units: destination element (a, c, r) of an item reads source element
//                  (keep_out[a], keep_in[c], r).  Stores are 16-byte vectors in destination
//                  order; rows that lose no input channel are copied with 16-byte loads too.
#include "dnns_internal.cuh"

namespace dnns {

namespace {

constexpr int kThreads = 256;
constexpr uint32_t kUnitBytes = 16384;

// Checked build (-DDNNS_BOUNDS_CHECK, a second library used by the tests only): every index that depends on
// data - keep lists, source elements, mask bits - is compared with its extent first; a violation is counted
// and the access goes to element 0 instead, so nothing faults.  The normal build compiles the checks away.
#ifdef DNNS_BOUNDS_CHECK
__device__ unsigned int g_bounds_violations = 0;
#define DNNS_IDX(i, n) ((uint32_t)(i) < (uint32_t)(n) ? (uint32_t)(i) : (atomicAdd(&g_bounds_violations, 1u), 0u))
#else
#define DNNS_IDX(i, n) (i)
#endif

__global__ void __launch_bounds__(1024) k_compact_layout(Tables tb, CompactWs ws, const int32_t* __restrict__ keep_count,
                                                         uint64_t dst_bytes, uint64_t* dst_offsets,
                                                         int32_t* dst_shapes) {
    __shared__ uint64_t scratch[33];
    uint64_t carry_bytes = 0, carry_units = 0;
    for (uint32_t base = 0; base < tb.n_items; base += 1024) {
        const uint32_t i = base + threadIdx.x;
        uint64_t bytes = 0, units = 0;
        if (i < tb.n_items) {
            const ItemDesc& it = tb.items[i];
            const int64_t On = keep_count[it.out_group];
            const int64_t Cn = it.in_group >= 0 ? keep_count[it.in_group] : it.Cin;
            const uint64_t raw = (uint64_t)(On * Cn * it.blk) * it.elem_bytes;
            bytes = (raw + 255) & ~(uint64_t)255;
            units = (raw + kUnitBytes - 1) / kUnitBytes;
            ws.item_dims[2 * i] = (int32_t)On;
            ws.item_dims[2 * i + 1] = (int32_t)Cn;
            if (it.tensor >= 0) {
                dst_shapes[2 * it.tensor] = (int32_t)On;
                dst_shapes[2 * it.tensor + 1] = (int32_t)(Cn * tb.tensors[it.tensor].S);
            }
        }
        uint64_t tot_b, tot_u;
        const uint64_t ex_b = block_exclusive_scan<uint64_t>(bytes, scratch, &tot_b);
        const uint64_t ex_u = block_exclusive_scan<uint64_t>(units, scratch, &tot_u);
        if (i < tb.n_items) {
            ws.item_off[i] = carry_bytes + ex_b;
            dst_offsets[i] = carry_bytes + ex_b;
            ws.unit_prefix[i] = (uint32_t)(carry_units + ex_u);
        }
        carry_bytes += tot_b;
        carry_units += tot_u;
    }
    if (threadIdx.x == 0) {
        if (carry_bytes > dst_bytes) {
            atomicCAS(tb.status, 0u, (uint32_t)DNNS_ERR_WORKSPACE);
            carry_units = 0;  // nothing is copied
        }
        ws.unit_prefix[tb.n_items] = (uint32_t)carry_units;
    }
}

template <int BYTES>
__device__ __forceinline__ uint32_t load_elem(const void* base, uint32_t idx) {
    if (BYTES == 4) return __ldg(static_cast<const uint32_t*>(base) + idx);
    return __ldg(static_cast<const uint16_t*>(base) + idx);
}

// Masking on the fly (the rebuild reading the dense model): what steps 2 decided for one tensor and variant.
struct MaskCtx {
    uint32_t tau;          // threshold key of the tensor's ranking segment
    uint32_t mode;         // 0: nothing is masked; 1: every key equal to tau is masked; 2: the mask bits decide those
    const uint32_t* bits;  // the tensor's packed mask bits (1 = kept), consulted for key == tau in mode 2 only
    uint32_t numel;        // elements of the tensor (extent of the bits; read by the checked build)
};

// The element as step 2 leaves it: itself when its key lies above tau (or equals it and its mask bit is set), else +0.
template <int BYTES>
__device__ __forceinline__ uint32_t masked_elem(uint32_t x, const MaskCtx& m, uint32_t src_idx) {
    const uint32_t key = x & (BYTES == 4 ? 0x7FFFFFFFu : 0x7FFFu);
    bool keep = key > m.tau;
    if (key == m.tau && m.mode == 2) {
        const uint32_t i = DNNS_IDX(src_idx, m.numel);
        keep = (__ldg(m.bits + (i >> 5)) >> (i & 31)) & 1u;
    }
    return (keep || m.mode == 0) ? x : 0u;
}

// The same for the VE elements of a 16-byte vector whose first element has source index src_idx.
template <int BYTES>
__device__ __forceinline__ uint4 masked_vec(uint4 v, const MaskCtx& m, uint32_t src_idx) {
    if (m.mode == 0) return v;
    uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        if (BYTES == 4) {
            w[j] = masked_elem<4>(w[j], m, src_idx + j);
        } else {
            w[j] = masked_elem<2>(w[j] & 0xFFFFu, m, src_idx + 2 * j) | (masked_elem<2>(w[j] >> 16, m, src_idx + 2 * j + 1) << 16);
        }
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// Gather a run of consecutive units of one item whose elements are BYTES wide, starting at
// destination element f0.  A unit is 4 x 16-byte destination vectors per thread.
template <int BYTES, bool MASKED>
__device__ __forceinline__ void gather_run(const ItemDesc& it, const char* src, char* dst, const int32_t* ko,
                                           const int32_t* ki, uint32_t On, uint32_t Cn, uint32_t f0, uint32_t n_units,
                                           const MaskCtx& mk) {
    constexpr uint32_t VE = 16 / BYTES;  // elements per 16-byte vector
    constexpr int U = kUnitBytes / 16 / kThreads;
    constexpr uint32_t kUnitElems = kUnitBytes / BYTES;
    constexpr uint32_t kNone = 0xFFFFFFFFu;
    const uint32_t blk = it.blk, Cin = it.Cin;
    const uint32_t Ln = Cn * blk, L = Cin * blk;  // new and old row length
    const uint32_t total = On * Ln;
    const uint32_t src_numel = (uint32_t)it.O * L;  // elements of the source item
    (void)src_numel;
    // A thread's destination vectors are kStride elements apart, unit after unit, so its position
    // (row a, offset rem in the row) is advanced with one add and one compare instead of a division.
    constexpr uint32_t kStride = kThreads * VE;
    const uint32_t step_a = kStride / Ln, step_rem = kStride - step_a * Ln;
    uint32_t pos_f = f0 + threadIdx.x * VE;
    uint32_t pos_a = pos_f / Ln, pos_rem = pos_f - pos_a * Ln;
    auto advance = [&]() {
        pos_f += kStride;
        pos_a += step_a;
        pos_rem += step_rem;
        if (pos_rem >= Ln) {
            pos_rem -= Ln;
            ++pos_a;
        }
    };
    if ((Cn == Cin) && (L % VE == 0) && ((reinterpret_cast<uintptr_t>(src) & 15) == 0)) {
        // Rows lose no input channel: every destination vector is one aligned source vector of row
        // ko[a].  The loads of the next unit are issued before the current unit is stored.
        uint4 nxt[U];
        bool nxt_ok[U];
        uint32_t nxt_src[MASKED ? U : 1];  // source index of the vector's first element (for the mask bits)
        auto issue = [&]() {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                nxt_ok[u] = pos_f < total;
                if (nxt_ok[u]) {
                    const uint32_t s0 = (uint32_t)ko[DNNS_IDX(pos_a, On)] * L + pos_rem;
                    nxt[u] = __ldg(reinterpret_cast<const uint4*>(src + (size_t)DNNS_IDX(s0, src_numel - (VE - 1)) * BYTES));
                    if (MASKED) nxt_src[u] = s0;
                }
                advance();
            }
        };
        issue();
        for (uint32_t n = 0; n < n_units; ++n) {
            uint4 cur[U];
            bool ok[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                ok[u] = nxt_ok[u];
                cur[u] = (MASKED && ok[u]) ? masked_vec<BYTES>(nxt[u], mk, nxt_src[u]) : nxt[u];
            }
            const uint32_t fu = f0 + n * kUnitElems;
            if (n + 1 < n_units) issue();
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (ok[u]) *reinterpret_cast<uint4*>(dst + (size_t)(fu + (u * kThreads + threadIdx.x) * VE) * BYTES) = cur[u];
        }
        return;
    }
    // General case: element (a, c, r) of the new row-major layout reads (ko[a], ki[c], r).  Per
    // pass: all source positions, then all 16 element loads of the thread, then the stores.
    constexpr int UG = BYTES == 4 ? U : U / 2;
#pragma unroll 1
    for (uint32_t pass = 0; pass < n_units * (U / UG); ++pass) {
        const uint32_t fp = f0 + pass * UG * kThreads * VE;
        uint32_t idx[UG][VE];
#pragma unroll
        for (int u = 0; u < UG; ++u) {
            const uint32_t f = fp + (u * kThreads + threadIdx.x) * VE;
#pragma unroll
            for (uint32_t e = 0; e < VE; ++e) idx[u][e] = kNone;
            uint32_t a = pos_a;
            const uint32_t rem = pos_rem;
            advance();
            if (f >= total) continue;
            if (rem + VE <= Ln && blk == 1) {
                // 1x1 kernels, vector inside one filter: one kept-channel lookup per element
                const uint32_t row = (uint32_t)ko[DNNS_IDX(a, On)] * Cin;
#pragma unroll
                for (uint32_t e = 0; e < VE; ++e) idx[u][e] = row + (ki ? (uint32_t)ki[DNNS_IDX(rem + e, Cn)] : rem + e);
                continue;
            }
            if (rem + VE <= Ln && blk >= VE) {
                // vector inside one filter and at most two input channels: two lookups
                const uint32_t c0 = blk == 9 ? rem / 9u : rem / blk, r0 = rem - c0 * blk, n0 = blk - r0;
                const uint32_t row = (uint32_t)ko[DNNS_IDX(a, On)] * Cin;
                const uint32_t base0 = (row + (ki ? (uint32_t)ki[DNNS_IDX(c0, Cn)] : c0)) * blk + r0;
                uint32_t base1 = 0;
                if (n0 < VE) base1 = (row + (ki ? (uint32_t)ki[DNNS_IDX(c0 + 1, Cn)] : c0 + 1)) * blk - n0;
#pragma unroll
                for (uint32_t e = 0; e < VE; ++e) idx[u][e] = (e < n0 ? base0 : base1) + e;
                continue;
            }
            if (Ln >= VE) {
                // vectors that cross into the next filter or reach the end of the item: one formula per element
                // (element e sits at offset rem + e of row a, or past its end in row a + 1), no walk
                const uint32_t row0 = (uint32_t)ko[DNNS_IDX(a, On)] * Cin;
                const uint32_t row1 = a + 1 < On ? (uint32_t)ko[a + 1] * Cin : 0u;
#pragma unroll
                for (uint32_t e = 0; e < VE; ++e) {
                    uint32_t re = rem + e;
                    const bool wrap = re >= Ln;
                    re = wrap ? re - Ln : re;
                    const uint32_t c = blk == 1 ? re : (blk == 9 ? re / 9u : re / blk), r = re - c * blk;
                    const uint32_t col = ki ? (uint32_t)ki[DNNS_IDX(c, Cn)] : c;
                    if (f + e < total) idx[u][e] = ((wrap ? row1 : row0) + col) * blk + r;
                }
                continue;
            }
            // rows shorter than a vector: walk element by element
            uint32_t c = blk == 1 ? rem : (blk == 9 ? rem / 9u : rem / blk), r = rem - c * blk;
            uint32_t row = (uint32_t)ko[DNNS_IDX(a, On)] * Cin, col = ki ? (uint32_t)ki[DNNS_IDX(c, Cn)] : c;
            const uint32_t nv = min(VE, total - f);
#pragma unroll
            for (uint32_t e = 0; e < VE; ++e) {
                if (e < nv) {
                    idx[u][e] = (row + col) * blk + r;
                    if (++r == blk) {
                        r = 0;
                        if (++c == Cn) {
                            c = 0;
                            ++a;
                            if (a < On) row = (uint32_t)ko[a] * Cin;
                        }
                        if (a < On) col = ki ? (uint32_t)ki[c] : c;
                    }
                }
            }
        }
        uint32_t w[UG][4];
#pragma unroll
        for (int u = 0; u < UG; ++u) {
#pragma unroll
            for (int j = 0; j < 4; ++j) w[u][j] = 0;
#pragma unroll
            for (uint32_t e = 0; e < VE; ++e) {
                uint32_t x = idx[u][e] != kNone ? load_elem<BYTES>(src, DNNS_IDX(idx[u][e], src_numel)) : 0u;
                if (MASKED && idx[u][e] != kNone) x = masked_elem<BYTES>(x, mk, idx[u][e]);  // no source element: no mask bit to look at
                if (BYTES == 4) w[u][e] = x;
                else w[u][e >> 1] |= x << (16 * (e & 1));
            }
        }
#pragma unroll
        for (int u = 0; u < UG; ++u) {
            const uint32_t f = fp + (u * kThreads + threadIdx.x) * VE;
            if (f >= total) continue;
            if (f + VE <= total) {
                *reinterpret_cast<uint4*>(dst + (size_t)f * BYTES) = make_uint4(w[u][0], w[u][1], w[u][2], w[u][3]);
            } else {
#pragma unroll
                for (uint32_t e = 0; e < VE; ++e) {
                    if (e < total - f) {
                        if (BYTES == 4) reinterpret_cast<uint32_t*>(dst)[f + e] = w[u][e];
                        else reinterpret_cast<uint16_t*>(dst)[f + e] = (uint16_t)(w[u][e >> 1] >> (16 * (e & 1)));
                    }
                }
            }
        }
    }
}

// Blocks take chunks of consecutive gather units and walk the items that own them.
//
// INLINE_LAYOUT (models of up to kInlineItems items): every block derives the destination layout
// itself, in shared memory, from the keep counts - a few hundred items, one scan - instead of waiting
// for a separate one-block kernel; block 0 also writes the offsets and shapes the caller asked for.
constexpr uint32_t kInlineItems = 1024;

// MASKED: the source is the dense model and step 2 is applied to every element on its way (thr, variant, mask_bits).
template <int WBYTES, bool INLINE_LAYOUT, bool MASKED>  // WBYTES: element width of the weight tensors (BatchNorm, bias: 4 bytes)
__global__ void __launch_bounds__(kThreads, 4) k_compact_gather(Tables tb, CompactWs ws, const char* src_arena,
                                                                const int32_t* __restrict__ keep_idx, char* dst_arena,
                                                                const int32_t* __restrict__ keep_count, uint64_t dst_bytes,
                                                                uint64_t* dst_offsets, int32_t* dst_shapes,
                                                                const dnns_threshold* __restrict__ thr, int variant,
                                                                const uint32_t* __restrict__ mask_bits) {
    __shared__ uint32_t s_unit_prefix[INLINE_LAYOUT ? kInlineItems + 1 : 1];
    __shared__ uint64_t s_item_off[INLINE_LAYOUT ? kInlineItems : 1];
    __shared__ int32_t s_item_dims[INLINE_LAYOUT ? 2 * kInlineItems : 1];
    __shared__ uint64_t scratch[33];
    if (INLINE_LAYOUT) {
        constexpr uint32_t kPer = kInlineItems / kThreads;  // consecutive items per thread
        uint64_t bytes[kPer], units[kPer], sum_b = 0, sum_u = 0;
#pragma unroll
        for (uint32_t k = 0; k < kPer; ++k) {
            const uint32_t i = threadIdx.x * kPer + k;
            bytes[k] = units[k] = 0;
            if (i < tb.n_items) {
                const ItemDesc& it = tb.items[i];
                const int64_t On = keep_count[it.out_group];
                const int64_t Cn = it.in_group >= 0 ? keep_count[it.in_group] : it.Cin;
                const uint64_t raw = (uint64_t)(On * Cn * it.blk) * it.elem_bytes;
                bytes[k] = (raw + 255) & ~(uint64_t)255;
                units[k] = (raw + kUnitBytes - 1) / kUnitBytes;
                s_item_dims[2 * i] = (int32_t)On;
                s_item_dims[2 * i + 1] = (int32_t)Cn;
                if (blockIdx.x == 0 && it.tensor >= 0) {
                    dst_shapes[2 * it.tensor] = (int32_t)On;
                    dst_shapes[2 * it.tensor + 1] = (int32_t)(Cn * tb.tensors[it.tensor].S);
                }
            }
            sum_b += bytes[k];
            sum_u += units[k];
        }
        uint64_t tot_b, tot_u;
        uint64_t ex_b = block_exclusive_scan<uint64_t>(sum_b, scratch, &tot_b);
        uint64_t ex_u = block_exclusive_scan<uint64_t>(sum_u, scratch, &tot_u);
        const bool fits = tot_b <= dst_bytes;
#pragma unroll
        for (uint32_t k = 0; k < kPer; ++k) {
            const uint32_t i = threadIdx.x * kPer + k;
            if (i < tb.n_items) {
                s_item_off[i] = ex_b;
                s_unit_prefix[i] = (uint32_t)ex_u;
                if (blockIdx.x == 0) dst_offsets[i] = ex_b;
            }
            ex_b += bytes[k];
            ex_u += units[k];
        }
        if (threadIdx.x == 0) {
            s_unit_prefix[tb.n_items] = fits ? (uint32_t)tot_u : 0u;  // too small an arena: nothing is copied
            if (!fits && blockIdx.x == 0) atomicCAS(tb.status, 0u, (uint32_t)DNNS_ERR_WORKSPACE);
        }
        __syncthreads();
    }
    const uint32_t* unit_prefix = INLINE_LAYOUT ? s_unit_prefix : ws.unit_prefix;
    const uint64_t* item_off = INLINE_LAYOUT ? s_item_off : ws.item_off;
    const int32_t* item_dims = INLINE_LAYOUT ? s_item_dims : ws.item_dims;
    const uint32_t total_units = unit_prefix[tb.n_items];
    // Units are dealt to the blocks in chunks, round robin: items differ a lot in cost per unit (plain
    // row copies against element gathers), and interleaving evens that out without any shared counter.
    constexpr uint32_t kChunkUnits = 2;
    for (uint32_t u_lo = blockIdx.x * kChunkUnits; u_lo < total_units; u_lo += gridDim.x * kChunkUnits) {
        const uint32_t u_hi = min(total_units, u_lo + kChunkUnits);
        // the item holding the first unit: last i with unit_prefix[i] <= u_lo
        uint32_t item = 0, hi = tb.n_items;
        while (hi - item > 1) {
            const uint32_t mid = (item + hi) >> 1;
            if (unit_prefix[mid] <= u_lo) item = mid;
            else hi = mid;
        }
        uint32_t unit = u_lo;
        while (unit < u_hi) {
            const uint32_t item_begin = unit_prefix[item], item_end = unit_prefix[item + 1];
            if (unit >= item_end) {  // items that shrank to nothing own no units
                ++item;
                continue;
            }
            const ItemDesc& it = tb.items[item];
            const uint32_t On = item_dims[2 * item], Cn = item_dims[2 * item + 1];
            const char* src;
            MaskCtx mk{0u, 0u, nullptr, 0u};
            if (it.tensor >= 0) {
                const TensorDesc& d = tb.tensors[it.tensor];
                src = src_arena ? src_arena + d.arena_off : static_cast<const char*>(d.src);
                if (MASKED && d.seg >= 0) {
                    const dnns_threshold r = thr[(size_t)variant * tb.n_segs + d.seg];
                    mk.tau = r.tau_bits;
                    mk.mode = r.n_below + r.n_tie == 0 ? 0u : (r.n_tie >= r.n_equal ? 1u : 2u);
                    mk.bits = mask_bits + d.off_mask;
                    mk.numel = d.numel;
                }
            } else {
                src = static_cast<const char*>(it.src);
            }
            char* dst = dst_arena + item_off[item];
            const int32_t* ko = keep_idx + tb.groups[it.out_group].off_idx;
            const int32_t* ki = it.in_group >= 0 ? keep_idx + tb.groups[it.in_group].off_idx : nullptr;
            const uint32_t run_end = min(u_hi, item_end);
            const uint32_t f0 = (unit - item_begin) * (kUnitBytes / it.elem_bytes);
            if (WBYTES == 4 || it.elem_bytes == 4) gather_run<4, MASKED>(it, src, dst, ko, ki, On, Cn, f0, run_end - unit, mk);
            else gather_run<2, MASKED>(it, src, dst, ko, ki, On, Cn, f0, run_end - unit, mk);
            unit = run_end;
        }
    }
}

}  // namespace

int launch_compact(const Tables& tb, const CompactWs& ws, const void* src_arena, const int32_t* keep_idx,
                   const int32_t* keep_count, void* dst_arena, uint64_t dst_bytes, uint64_t* dst_offsets,
                   int32_t* dst_shapes, int n_sm, cudaStream_t st, const dnns_threshold* thr, int variant,
                   const uint32_t* mask_bits) {
    const char* src = (const char*)src_arena;
    char* dst = (char*)dst_arena;
    const int grid = n_sm * 4;
    const bool masked = thr != nullptr;
    int launches = 1;
#define DNNS_GATHER(W, INL, M)                                                                                        \
    k_compact_gather<W, INL, M><<<grid, kThreads, 0, st>>>(tb, ws, src, keep_idx, dst, keep_count, dst_bytes, dst_offsets, \
                                                           dst_shapes, thr, variant, mask_bits)
#define DNNS_GATHER_DT(INL)                                  \
    do {                                                     \
        if (tb.dtype == DNNS_F32) {                          \
            if (masked) DNNS_GATHER(4, INL, true);           \
            else DNNS_GATHER(4, INL, false);                 \
        } else {                                             \
            if (masked) DNNS_GATHER(2, INL, true);           \
            else DNNS_GATHER(2, INL, false);                 \
        }                                                    \
    } while (0)
    if (tb.n_items <= kInlineItems) {
        ScopedKernel timed(masked ? "k_compact_gather<masked>" : "k_compact_gather", st);
        DNNS_GATHER_DT(true);
    } else {
        {
            ScopedKernel timed_layout("k_compact_layout", st);
            k_compact_layout<<<1, 1024, 0, st>>>(tb, ws, keep_count, dst_bytes, dst_offsets, dst_shapes);
        }
        ScopedKernel timed(masked ? "k_compact_gather<masked>" : "k_compact_gather", st);
        DNNS_GATHER_DT(false);
        launches = 2;
    }
#undef DNNS_GATHER_DT
#undef DNNS_GATHER
    return cudaGetLastError() == cudaSuccess ? launches : -1;
}

}  // namespace dnns

#ifdef DNNS_BOUNDS_CHECK
// Checked build only: violations counted so far on the current device (and the counter reset).
extern "C" unsigned int dnns_check_bounds_violations() {
    unsigned int n = 0, zero = 0;
    if (cudaDeviceSynchronize() != cudaSuccess || cudaMemcpyFromSymbol(&n, dnns::g_bounds_violations, sizeof(n)) != cudaSuccess)
        return 0xFFFFFFFFu;
    cudaMemcpyToSymbol(dnns::g_bounds_violations, &zero, sizeof(zero));
    return n;
}
#endif
