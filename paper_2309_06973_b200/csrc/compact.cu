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

// Gather one unit of an item whose elements are BYTES wide.
template <int BYTES>
__device__ __forceinline__ void gather_unit(const ItemDesc& it, const char* src, char* dst, const int32_t* ko,
                                            const int32_t* ki, uint32_t On, uint32_t Cn, uint32_t f0) {
    constexpr uint32_t VE = 16 / BYTES;  // elements per 16-byte vector
    const uint32_t blk = it.blk, Cin = it.Cin;
    const uint32_t Ln = Cn * blk, L = Cin * blk;  // new and old row length
    const uint32_t total = On * Ln;
    const uint32_t f1 = min(total, f0 + kUnitBytes / BYTES);
    const bool rows_intact = (Cn == Cin) && (L % VE == 0) && ((reinterpret_cast<uintptr_t>(src) & 15) == 0);
    for (uint32_t f = f0 + threadIdx.x * VE; f < f1; f += kThreads * VE) {
        uint32_t a = f / Ln, rem = f - a * Ln;
        if (rows_intact && f + VE <= total) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(src + ((size_t)ko[a] * L + rem) * BYTES));
            *reinterpret_cast<uint4*>(dst + (size_t)f * BYTES) = v;
            continue;
        }
        uint32_t c = rem / blk, r = rem - c * blk;
        uint32_t row = (uint32_t)ko[a] * Cin, col = ki ? (uint32_t)ki[c] : c;
        uint32_t w[4] = {0, 0, 0, 0};
        const uint32_t nv = min(VE, total - f);
        for (uint32_t e = 0; e < nv; ++e) {
            const uint32_t x = load_elem<BYTES>(src, (row + col) * blk + r);
            if (BYTES == 4) w[e] = x;
            else w[e >> 1] |= x << (16 * (e & 1));
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
        if (nv == VE) {
            *reinterpret_cast<uint4*>(dst + (size_t)f * BYTES) = make_uint4(w[0], w[1], w[2], w[3]);
        } else {
            for (uint32_t e = 0; e < nv; ++e) {
                if (BYTES == 4) reinterpret_cast<uint32_t*>(dst)[f + e] = w[e];
                else reinterpret_cast<uint16_t*>(dst)[f + e] = (uint16_t)(w[e >> 1] >> (16 * (e & 1)));
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads) k_compact_gather(Tables tb, CompactWs ws, const char* src_arena,
                                                             const int32_t* __restrict__ keep_idx, char* dst_arena) {
    const uint32_t total_units = ws.unit_prefix[tb.n_items];
    for (uint32_t unit = blockIdx.x; unit < total_units; unit += gridDim.x) {
        // the item holding this unit: last i with unit_prefix[i] <= unit
        uint32_t lo = 0, hi = tb.n_items;
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (ws.unit_prefix[mid] <= unit) lo = mid;
            else hi = mid;
        }
        const ItemDesc& it = tb.items[lo];
        const uint32_t On = ws.item_dims[2 * lo], Cn = ws.item_dims[2 * lo + 1];
        const char* src;
        if (it.tensor >= 0) {
            const TensorDesc& d = tb.tensors[it.tensor];
            src = src_arena ? src_arena + d.arena_off : static_cast<const char*>(d.src);
        } else {
            src = static_cast<const char*>(it.src);
        }
        char* dst = dst_arena + ws.item_off[lo];
        const int32_t* ko = keep_idx + tb.groups[it.out_group].off_idx;
        const int32_t* ki = it.in_group >= 0 ? keep_idx + tb.groups[it.in_group].off_idx : nullptr;
        const uint32_t f0 = (unit - ws.unit_prefix[lo]) * (kUnitBytes / it.elem_bytes);
        if (it.elem_bytes == 4) gather_unit<4>(it, src, dst, ko, ki, On, Cn, f0);
        else gather_unit<2>(it, src, dst, ko, ki, On, Cn, f0);
    }
}

}  // namespace

int launch_compact(const Tables& tb, const CompactWs& ws, const void* src_arena, const int32_t* keep_idx,
                   const int32_t* keep_count, void* dst_arena, uint64_t dst_bytes, uint64_t* dst_offsets,
                   int32_t* dst_shapes, int n_sm, cudaStream_t st) {
    k_compact_layout<<<1, 1024, 0, st>>>(tb, ws, keep_count, dst_bytes, dst_offsets, dst_shapes);
    k_compact_gather<<<n_sm * 8, kThreads, 0, st>>>(tb, ws, (const char*)src_arena, keep_idx, (char*)dst_arena);
    return cudaGetLastError() == cudaSuccess ? 2 : -1;
}

}  // namespace dnns
