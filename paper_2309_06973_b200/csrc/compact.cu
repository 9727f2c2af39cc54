// Step 5: the rebuild - Module 4, the Model Pruner (Algorithm 2): every layer is re-created with
// |C'_in| x |C'_out| channels and its surviving out-channels, biases and in-channels are moved
// over, all layers in one batch.  Here that is one gather over every tensor, BatchNorm vector
// and bias of the model:
//   layout kernel  sizes each rebuilt item from the keep counts, places it at a 256-byte aligned
//                  offset of the destination arena and cuts it into units of work (run once per set of keep
//                  counts, right after the channels were planned);
//   gather kernel  destination element (a, c, r) of an item reads source element
//                  (keep_out[a], keep_in[c], r).
//
// Weight tensors whose filters (rows) are a multiple of 16 bytes long take the staged path: a
// producer warp brings the kept rows of a unit - whole rows, or a range of input channels of one
// long row - into shared memory with bulk copies (cp.async.bulk, completion on an mbarrier), a ring
// of kStages buffers deep; eight consumer warps read the surviving elements out of the buffer, one
// destination element per lane (a pair for 2-byte elements), so that the buffer is read without
// bank conflicts and the stores of a warp are one contiguous run.  Every global access of that path
// is contiguous; the only indexed reads are the kept-channel list (cached) and shared memory.
// BatchNorm vectors and biases are copied by single warps; tensors with other row lengths take the
// element path (gather_run): 16 KB destination units, source positions computed per element.
#include "dnns_internal.cuh"

#pragma nv_diag_suppress 186  // "pointless comparison of unsigned integer with zero": thresholds that are 0 in one instantiation

namespace dnns {

namespace {

constexpr int kThreads = 256;
constexpr uint32_t kUnitBytes = 16384;

DNNS_BOUNDS_COUNTER  // (checked build: index violations counted in this file)

template <int BYTES>
__device__ __forceinline__ uint32_t load_elem(const void* base, uint32_t idx) {
    if (BYTES == 4) return __ldg(static_cast<const uint32_t*>(base) + idx);
    return __ldg(static_cast<const uint16_t*>(base) + idx);
}

// Masking on the fly (the rebuild reading the dense model): what step 2 decides for one tensor and variant.
// A weight stays when its key lies above tau, or equals tau and the weight comes at or after the place where the
// variant stops masking such weights (threshold step: TieSplit).  Away from that place one comparison settles it.
struct MaskCtx {
    uint32_t tau;         // threshold key of the tensor's ranking segment
    uint32_t mode;        // 0: nothing is masked; 1: keep iff key >= thr_eff; 2: the split lies in this tensor
    uint32_t thr_eff;     // mode 1: tau + 1 where the weights equal to tau are masked, tau where they stay
    uint32_t split_elem;  // mode 2: weights equal to tau stay from this element of the tensor on
};

// The element as step 2 leaves it (src_idx: its index in the source tensor), else +0.
template <int BYTES>
__device__ __forceinline__ uint32_t masked_elem(uint32_t x, const MaskCtx& m, uint32_t src_idx) {
    const uint32_t key = x & (BYTES == 4 ? 0x7FFFFFFFu : 0x7FFFu);
    bool keep;
    if (m.mode == 2) keep = key > m.tau || (key == m.tau && src_idx >= m.split_elem);
    else keep = key >= m.thr_eff;
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
__device__ __noinline__ void gather_run(const ItemDesc& it, const char* src, char* dst, const int32_t* ko,
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

// ---------------------------------------------------------------------------------------------
// The staged path
// ---------------------------------------------------------------------------------------------
constexpr int kStages = 3;                 // ring of stage buffers per block (three blocks per SM)
constexpr uint32_t kStageBytes = 18432;    // two 3x3 filters of 256 channels, one of 512 (fp32)
constexpr int kConsumers = kThreads;       // threads 0..255 consume, the warp after them produces
constexpr int kGatherThreads = kConsumers + 32;
constexpr int kProducerWarp = kConsumers / 32;
constexpr uint32_t kMaxRowsPerUnit = 256;  // rows of one unit (eight rounds of a row per lane of the producer)
constexpr uint32_t kRowMapMax = 4608;      // destination row lengths (elements) that get a row map
constexpr uint32_t kMaxChunkTab = 127;     // chunks per row whose places in the keep list are tabulated per item
constexpr uint32_t kWaitLimitNs = 500u * 1000u * 1000u;  // a wait that lasts this long is given up (status TIMEOUT)

enum : uint32_t { kUnitStop = 0, kUnitCopy = 1, kUnitGather = 2 };

// What the producer tells the consumers about the unit it put into a stage buffer.
struct UnitDesc {
    char* dst;           // destination of the unit's first row, first kept channel of the chunk
    const int32_t* ki;   // kept input channels, from the first one inside this chunk on
    const int32_t* ko;   // kept filters, from the unit's first row on
    uint32_t kind;
    uint32_t n_r;        // rows
    uint32_t Wd, Ws;     // elements per row at the destination / in the stage buffer
    uint32_t Ln;         // elements of a whole destination row
    uint32_t c_lo;       // first input channel in the stage buffer
    uint32_t blk, magic; // elements per (row, channel); floor(2^32 / blk) + 1
    uint32_t L;          // elements of a whole source row
    uint32_t n_ki;       // kept input channels inside this chunk (extent of ki; read by the checked build)
    const int32_t* ki_all;  // the item's whole list of kept input channels
    uint32_t map_seq;    // non-zero: the unit's item has a row map; it changes from one such item to the next
    uint32_t map_base;   // destination column of the unit's first column in a whole row
    MaskCtx mk;
};
template <int BYTES>
struct ElemWord;
template <>
struct ElemWord<4> {
    typedef uint32_t type;
};
template <>
struct ElemWord<2> {
    typedef uint16_t type;
};

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"  // may sleep up to the hint (ns) before it answers
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_addr(bar)), "r"(parity), "r"(20000u)
        : "memory");
    return done != 0;
}
__device__ __forceinline__ uint64_t global_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Wait for a phase of an mbarrier, but not for ever: false when the wait was given up (or another
// thread of the block gave up before).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_ns();
    for (uint32_t spin = 1;; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spin & 63u) == 0 && (*abort_flag || global_ns() - t0 > kWaitLimitNs)) return false;
    }
}
// Bulk copy global -> shared, completion counted in bytes on an mbarrier.  Addresses and size are multiples of 16.
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_addr(smem_dst)),
                 "l"(gmem_src), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}

// First p in [0, n) with list[p] >= c (n when none): where a range of source channels starts in the keep list.
__device__ __forceinline__ uint32_t lower_bound_idx(const int32_t* list, uint32_t n, uint32_t c) {
    uint32_t lo = 0, hi = n;
    while (lo < hi) {
        const uint32_t mid = (lo + hi) >> 1;
        if ((uint32_t)__ldg(list + mid) < c) lo = mid + 1;
        else hi = mid;
    }
    return lo;
}

// The unit shape of a staged item: blocks of rows by pieces of rows when input channels are dropped, else longer
// pieces (whole rows where they fit), which need fewer copies.
struct Geometry {
    uint32_t ru, ch, nch;
};
__device__ __forceinline__ Geometry geometry_of(const ItemDesc& it, uint32_t Cn) {
    if (Cn == (uint32_t)it.Cin) return Geometry{(uint32_t)it.ru_c, (uint32_t)it.ch_c, (uint32_t)it.nch_c};
    return Geometry{(uint32_t)it.ru, (uint32_t)it.ch, (uint32_t)it.nch};
}

// ---- the layout of one variant
// From the keep counts: rows and channels every item keeps, its 256-byte aligned place in the destination arena,
// its units of work, and where each block of the gather starts.  One block per variant; the tables stay in the
// workspace until the keep counts change (dnns_propagate_keep* runs this right after planning the channels).
constexpr uint32_t kLayoutTab = 4096;  // items whose prefix sums the layout kernel also keeps in shared memory
__global__ void __launch_bounds__(1024) k_rebuild_layout(Tables tb, LayoutBatch lb, uint32_t n_blocks) {
    __shared__ uint64_t scratch[33];
    __shared__ uint32_t s_cost_pre[kLayoutTab], s_unit_pre[kLayoutTab];  // searched below: thousands of probes, none to global memory
    const bool in_smem = tb.n_items <= kLayoutTab;
    const int32_t* __restrict__ keep_count = lb.keep_count[blockIdx.x];
    const RebuildSlot slot = lb.slot[blockIdx.x];
    uint64_t carry_bytes = 0, carry_uc = 0;  // carry_uc: cost << 32 | units (each stays below 2^32)
    for (uint32_t base = 0; base < tb.n_items; base += 1024) {
        const uint32_t i = base + threadIdx.x;
        uint64_t bytes = 0, uc = 0;
        RebuildItem r{0, 0, 0, 0, 0, 0, 0, 0};
        if (i < tb.n_items) {
            const ItemDesc& it = tb.items[i];
            r.On = (uint32_t)keep_count[it.out_group];
            r.Cn = it.in_group >= 0 ? (uint32_t)keep_count[it.in_group] : (uint32_t)it.Cin;
            const uint64_t raw = (uint64_t)r.On * r.Cn * (uint32_t)it.blk * (uint32_t)it.elem_bytes;
            bytes = (raw + 255) & ~(uint64_t)255;
            if (it.kind == kItemStaged) {
                if (r.On && r.Cn) {
                    const Geometry g = geometry_of(it, r.Cn);
                    const uint32_t rows = min(g.ru, r.On), chn = min(g.ch, (uint32_t)it.Cin);
                    const uint32_t src = rows * chn * (uint32_t)it.blk * (uint32_t)it.elem_bytes;  // at most a stage buffer
                    const uint32_t dst = (uint32_t)((uint64_t)src * r.Cn / (uint32_t)it.Cin);
                    r.s_units = ((r.On + g.ru - 1) / g.ru) * g.nch;
                    r.s_cost = (src + dst + 63) >> 6;
                    uc = (uint64_t)(r.s_units * r.s_cost) << 32;
                }
            } else if (it.kind == kItemElement) {
                uc = (raw + kUnitBytes - 1) / kUnitBytes;
            }
        }
        uint64_t tot_b, tot_uc;
        const uint64_t ex_b = block_exclusive_scan<uint64_t>(bytes, scratch, &tot_b);
        const uint64_t ex_uc = block_exclusive_scan<uint64_t>(uc, scratch, &tot_uc);
        if (i < tb.n_items) {
            r.off256 = (uint32_t)((carry_bytes + ex_b) >> 8);
            r.cost_pre = (uint32_t)((carry_uc + ex_uc) >> 32);
            r.unit_pre = (uint32_t)(carry_uc + ex_uc);
            slot.items[i] = r;
            if (in_smem) s_cost_pre[i] = r.cost_pre, s_unit_pre[i] = r.unit_pre;
        }
        carry_bytes += tot_b;
        carry_uc += tot_uc;
    }
    const uint32_t total_cost = (uint32_t)(carry_uc >> 32), total_units = (uint32_t)carry_uc;
    if (threadIdx.x == 0) {
        RebuildHeader h{};
        h.total_bytes = carry_bytes;
        h.total_cost = total_cost;
        h.total_units = total_units;
        *slot.header = h;
    }
    __syncthreads();  // the item table is read back below (same block: visible after the barrier)
    // where every range of the cost axis starts: the last item whose earlier cost is <= the range's start
    for (uint32_t r = threadIdx.x; r < rebuild_ranges(n_blocks); r += 1024) {
        const uint32_t lo = rebuild_range_lo(r, n_blocks, total_cost);
        uint32_t item = 0, top = tb.n_items;
        while (top - item > 1) {
            const uint32_t mid = (item + top) >> 1;
            if ((in_smem ? s_cost_pre[mid] : slot.items[mid].cost_pre) <= lo) item = mid;
            else top = mid;
        }
        slot.range_item[r] = item;
    }
    // the item of every 16 KB unit of the element path
    for (uint32_t u = threadIdx.x; u < total_units; u += 1024) {
        uint32_t item = 0, top = tb.n_items;
        while (top - item > 1) {
            const uint32_t mid = (item + top) >> 1;
            if ((in_smem ? s_unit_pre[mid] : slot.items[mid].unit_pre) <= u) item = mid;
            else top = mid;
        }
        slot.unit_item[u] = item;
    }
}

// ---- consumers
// The unit in a stage buffer is a matrix of n_r rows by Ws source elements (row r at r * Ws); its destination is
// n_r rows of Wd elements, row r at dst + r * Ln.

// Step 2 on the words of a 16-byte vector when every key equal to tau is treated alike: keep iff key >= thr_eff.
template <int BYTES>
__device__ __forceinline__ uint4 threshold_vec(uint4 v, uint32_t thr_eff) {
    uint32_t w[4] = {v.x, v.y, v.z, v.w};
    if (BYTES == 4) {
#pragma unroll
        for (int j = 0; j < 4; ++j) w[j] = (w[j] & 0x7FFFFFFFu) >= thr_eff ? w[j] : 0u;
    } else {
        // both 15-bit keys of a word at once: with bit 15 of each half set, subtracting the threshold leaves that
        // bit standing exactly where key >= threshold, and no borrow crosses into the other half (thr_eff <= 0x8000)
        const uint32_t te2 = thr_eff * 0x00010001u;
#pragma unroll
        for (int j = 0; j < 4; ++j) w[j] &= ((((w[j] | 0x80008000u) - te2) >> 15) & 0x00010001u) * 0xFFFFu;
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// A unit whose rows lose no channel and land on 16-byte boundaries: 16-byte vectors straight across.
template <int BYTES, bool MASKED>
__device__ __forceinline__ void consume_copy(const UnitDesc& desc, const unsigned char* stage, int ctid) {
    constexpr uint32_t VE = 16 / BYTES;
    // (fields read once into registers: the stores below could alias the descriptor as far as the compiler knows)
    char* const dst = desc.dst;
    const uint32_t vpr = desc.Ws / VE, n_vec = desc.n_r * vpr;  // vectors per row, in the unit
    const uint4* s = reinterpret_cast<const uint4*>(stage);
    const uint32_t row_pitch = desc.Ln * BYTES;  // a unit spans less than 2^32 destination bytes
    const uint32_t mode = MASKED ? desc.mk.mode : 0u, thr_eff = desc.mk.thr_eff;
    if (MASKED && mode == 2) {
        // around the place where the weights equal to tau split: element by element, by source position
        const MaskCtx mk = desc.mk;
        const int32_t* ko = desc.ko;
        const uint32_t L = desc.L, first = desc.c_lo * desc.blk;
        for (uint32_t v = ctid; v < n_vec; v += kConsumers) {
            const uint32_t row = v / vpr, col = v - row * vpr;
            const uint4 x = masked_vec<BYTES>(s[v], mk, (uint32_t)__ldg(ko + row) * L + first + col * VE);
            *reinterpret_cast<uint4*>(dst + (size_t)row * row_pitch + (size_t)col * 16) = x;
        }
        return;
    }
    const bool mask = mode == 1;
    if (row_pitch == vpr * 16) {  // whole rows: the destination is one run as well
        uint4* g = reinterpret_cast<uint4*>(dst);
#pragma unroll 4
        for (uint32_t v = ctid; v < n_vec; v += kConsumers) g[v] = mask ? threshold_vec<BYTES>(s[v], thr_eff) : s[v];
        return;
    }
    const uint32_t step_row = kConsumers / vpr, step_col = kConsumers - step_row * vpr;
    const uint32_t step_off = step_row * row_pitch + step_col * 16, wrap_off = row_pitch - vpr * 16;
    uint32_t row = (uint32_t)ctid / vpr, col = (uint32_t)ctid - row * vpr;
    uint32_t off = row * row_pitch + col * 16;
#pragma unroll 2
    for (uint32_t v = ctid; v < n_vec; v += kConsumers) {
        *reinterpret_cast<uint4*>(dst + off) = mask ? threshold_vec<BYTES>(s[v], thr_eff) : s[v];
        col += step_col;
        off += step_off;
        if (col >= vpr) {
            col -= vpr;
            off += wrap_off;
        }
    }
}

// A unit that loses input channels.  A thread owns destination columns (column j of the unit: input channel
// p = j / blk of the kept list, element j % blk of its 2-D kernel) and walks down the rows, so that the source
// offset of a column is found once per unit and the loop is a shared-memory load, the mask and a store; the
// lanes of a warp hold neighbouring columns, which keeps the shared-memory reads free of bank conflicts and a
// warp's stores contiguous.  The source offsets come from the item's row map in shared memory (rowmap, when the
// descriptor names one) or from the kept-channel list.  Narrow units put several rows side by side; in wide ones
// a thread walks down several columns at once.  CAREFUL: the unit holds the place where the weights equal to
// tau split (one row of one tensor per variant), and those weights compare their source position.
template <int BYTES, bool MASKED, bool CAREFUL>
__device__ __forceinline__ void consume_gather(const UnitDesc& desc, const unsigned char* stage, const uint16_t* rowmap, int ctid) {
    typedef typename ElemWord<BYTES>::type T;
    constexpr int kColBatch = 4;
    // (fields read once into registers: the stores below could alias the descriptor as far as the compiler knows)
    const uint32_t Wd = desc.Wd, Ws = desc.Ws, n_r = desc.n_r, blk = desc.blk, Ln = desc.Ln;
    const uint32_t map_seq = desc.map_seq, map_base = desc.map_base, first = desc.c_lo * blk, c_lo = desc.c_lo;
    const uint32_t magic = desc.magic, n_ki = desc.n_ki, L = desc.L;
    const int32_t* const ki = desc.ki;
    const int32_t* const ko = desc.ko;
    const uint32_t mode = MASKED ? desc.mk.mode : 0u, tau = desc.mk.tau, split_elem = desc.mk.split_elem;
    (void)n_ki;
    constexpr uint32_t key_mask = BYTES == 4 ? 0x7FFFFFFFu : 0x7FFFu;
    // keep iff key >= thr_eff (0: everything stays)
    const uint32_t thr_eff = mode == 0 ? 0u : (mode == 1 ? desc.mk.thr_eff : tau + 1u);
    const T* sbase = reinterpret_cast<const T*>(stage);
    T* dbase = reinterpret_cast<T*>(desc.dst);
    // position of destination column `col` in a row of the stage buffer
    auto source_offset = [&](uint32_t col) -> uint32_t {
        uint32_t soff;
        if (map_seq) {
            soff = (uint32_t)rowmap[map_base + col] - first;
        } else {
            const uint32_t p = blk == 1 ? col : (blk == 9 ? col / 9u : __umulhi(col, magic));
            soff = ((uint32_t)__ldg(ki + DNNS_IDX(p, n_ki)) - c_lo) * blk + (col - p * blk);
        }
#ifdef DNNS_BOUNDS_CHECK
        if (soff >= Ws) {
            atomicAdd(&g_bounds_violations, 1u);
            soff = 0;
        }
#endif
        return soff;
    };
    auto masked = [&](uint32_t x, uint32_t row, uint32_t soff) -> uint32_t {
        if (!MASKED) return x;
        const uint32_t key = x & key_mask;
        bool keep = key >= thr_eff;
        if (CAREFUL && key == tau) keep = (uint32_t)__ldg(ko + row) * L + first + soff >= split_elem;
        return keep ? x : 0u;
    };
    if (Wd > kConsumers / 2) {
        for (uint32_t cb = ctid; cb < Wd; cb += kConsumers * kColBatch) {
            uint32_t soff[kColBatch];
            bool ok[kColBatch];
#pragma unroll
            for (int c = 0; c < kColBatch; ++c) {
                ok[c] = cb + c * kConsumers < Wd;
                soff[c] = ok[c] ? source_offset(cb + c * kConsumers) : 0u;
            }
            const T* sp = sbase;
            T* dp = dbase + cb;
#pragma unroll 2
            for (uint32_t row = 0; row < n_r; ++row) {
                uint32_t x[kColBatch];
#pragma unroll
                for (int c = 0; c < kColBatch; ++c) x[c] = sp[soff[c]];
#pragma unroll
                for (int c = 0; c < kColBatch; ++c)
                    if (ok[c]) dp[c * kConsumers] = (T)masked(x[c], row, soff[c]);
                sp += Ws;
                dp += Ln;
            }
        }
        return;
    }
    // columns side by side: the next power of two at or above Wd
    const uint32_t cp = Wd <= 1 ? 1u : 1u << (32 - __clz(Wd - 1));
    const uint32_t row_par = kConsumers / cp, rp = (uint32_t)ctid / cp, col = (uint32_t)ctid - rp * cp;
    if (col >= Wd) return;
    const uint32_t soff = source_offset(col);
    const T* sp = sbase + soff + rp * Ws;
    T* dp = dbase + col + (size_t)rp * Ln;
    const uint32_t s_step = row_par * Ws;
    const uint32_t d_step = row_par * Ln;
#pragma unroll 4
    for (uint32_t row = rp; row < n_r; row += row_par) {
        *dp = (T)masked(*sp, row, soff);
        sp += s_step;
        dp += d_step;
    }
}

// ---- the kernel
//
// Work is dealt out statically from the variant's prepared layout: the staged units of all items lie on one
// axis of cost (bytes read and written, a constant per unit of an item), cut into gridDim.x equal ranges, a
// block owning the units that start in its range; vector items go to single warps, the 16 KB units of the
// element path to blocks, round robin in pairs.
//
// MASKED: the source is the dense model and step 2 is applied to every element on its way (thr, variant, split).
template <int WBYTES, bool MASKED>  // WBYTES: element width of the weight tensors (BatchNorm, bias: 4 bytes)
__global__ void __launch_bounds__(kGatherThreads, 3) k_compact_gather(Tables tb, GatherBatch gb,
                                                                      const dnns_threshold* __restrict__ thr,
                                                                      const TieSplit* __restrict__ split) {
    extern __shared__ uint4 s_stage_mem[];  // kStages buffers of kStageBytes
    __shared__ __align__(8) uint64_t s_full[kStages], s_empty[kStages];
    __shared__ UnitDesc s_desc[kStages];
    __shared__ uint32_t s_abort;
    __shared__ uint32_t s_chunk_start[kMaxChunkTab + 1];  // the producer's: first kept channel at or above every chunk start
    // The consumers' row map of the item they are working on: position in a source row of every element of a
    // destination row (ki[j / blk] * blk + j % blk), built once per item and block.
    __shared__ uint16_t s_rowmap[kRowMapMax];
    unsigned char* const stage_mem = reinterpret_cast<unsigned char*>(s_stage_mem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&s_full[s], 1);                // the producer's arrive; the bytes of its copies
            mbar_init(&s_empty[s], kConsumers / 32);  // one arrive per consumer warp
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // a job whose arena is too small for its variant copies nothing
    auto job_fits = [&](int j) { return gb.job[j].lay.header->total_bytes <= gb.job[j].dst_bytes; };
    volatile uint32_t* abort_flag = &s_abort;
    auto give_up = [&]() {
        *abort_flag = 1;
        atomicCAS(tb.status, 0u, (uint32_t)DNNS_ERR_TIMEOUT);
    };
    auto mask_ctx = [&](const ItemDesc& it, int variant) {
        MaskCtx mk{0u, 0u, 0u, 0u};
        if (MASKED && it.tensor >= 0 && it.seg >= 0) {
            const size_t idx = (size_t)variant * tb.n_segs + it.seg;
            const dnns_threshold r = thr[idx];
            const TieSplit sp = split[idx];
            mk.tau = r.tau_bits;
            if (r.n_below + r.n_tie == 0) {
                mk.mode = 0;
            } else if ((uint32_t)it.tensor == sp.tensor) {
                mk.mode = 2, mk.split_elem = sp.elem;
            } else {  // tensors before the split have their weights equal to tau masked, tensors after it keep them
                mk.mode = 1, mk.thr_eff = (uint32_t)it.tensor < sp.tensor ? r.tau_bits + 1u : r.tau_bits;
            }
        }
        return mk;
    };

    if (warp == kProducerWarp) {
        // ================= producer: takes ranges of the cost axes of the jobs, walks their units, fills the ring =====
        const uint32_t per_job = rebuild_ranges(gridDim.x), n_ranges = per_job * (uint32_t)gb.n;
        RebuildHeader* const counters = gb.job[0].lay.header;
        auto next_range = [&]() {  // the counter's value k stands for range gridDim.x + k
            uint32_t r = 0;
            if (lane == 0) r = atomicAdd(&counters->next_range, 1u);
            return gridDim.x + __shfl_sync(0xffffffffu, r, 0);
        };
        uint32_t issued = 0, map_seq = 0;
        bool alive = true;
        int cur_job = -1;
        uint32_t total_cost = 0;
        uint32_t range = blockIdx.x, range_after = next_range();
        for (; alive && range < n_ranges; range = range_after, range_after = range < n_ranges ? next_range() : n_ranges) {
            const int jb = (int)(range / per_job);
            const uint32_t rj = range - (uint32_t)jb * per_job;
            if (jb != cur_job) {
                cur_job = jb;
                total_cost = job_fits(jb) ? gb.job[jb].lay.header->total_cost : 0u;
            }
            const GatherJob& job = gb.job[jb];
            const RebuildItem* __restrict__ ritems = job.lay.items;
            const int32_t* __restrict__ keep_idx = job.keep_idx;
            const uint32_t lo = rebuild_range_lo(rj, gridDim.x, total_cost), hi = rebuild_range_lo(rj + 1, gridDim.x, total_cost);
            if (lo >= hi) continue;
            for (uint32_t item = job.lay.range_item[rj]; alive && item < tb.n_items; ++item) {
                const RebuildItem z = ritems[item];
                if (z.cost_pre >= hi) break;
                if (z.s_units == 0) continue;
                const uint32_t pre = z.cost_pre;
                const uint32_t j_lo = lo > pre ? (lo - pre + z.s_cost - 1) / z.s_cost : 0u;
                const uint32_t j_hi = min(z.s_units, (hi - pre + z.s_cost - 1) / z.s_cost);
                if (j_lo >= j_hi) continue;
                const ItemDesc it = tb.items[item];
                const char* src = job.src_arena ? job.src_arena + it.arena_off : static_cast<const char*>(it.src);
                char* dst = job.dst_arena + ((uint64_t)z.off256 << 8);
                const int32_t* ko = keep_idx + it.ko_off;
                const int32_t* ki = keep_idx + it.ki_off;
                const uint32_t blk = it.blk, Cin = it.Cin, L = Cin * blk, Ln = z.Cn * blk;
                const MaskCtx mk = mask_ctx(it, job.variant);
                const Geometry g = geometry_of(it, z.Cn);
                const uint32_t nch = g.nch, ru = g.ru, ch = g.ch;
                const bool identity = z.Cn == Cin;  // no input channel is dropped: kept channel p is channel p
                const bool use_map = !identity && Ln <= kRowMapMax && L <= 65536u;
                if (use_map) ++map_seq;
                // where every chunk of channels starts in the keep list (the same for all rows of the item)
                const bool bounds_tab = nch > 1 && !identity && nch <= kMaxChunkTab;
                if (bounds_tab) {
                    __syncwarp();
                    for (uint32_t c = lane; c <= nch; c += 32) s_chunk_start[c] = c == nch ? z.Cn : lower_bound_idx(ki, z.Cn, c * ch);
                    __syncwarp();
                }
                uint32_t rg = j_lo / nch, cc = j_lo - rg * nch;
                int32_t rows[kMaxRowsPerUnit / 32];  // this lane's source rows of the current row group (-2: none)
                for (uint32_t j = j_lo; alive && j < j_hi; ++j) {
                    const uint32_t a0 = rg * ru, n_r = min(ru, z.On - a0);
                    if (cc == 0 || j == j_lo) {
#pragma unroll
                        for (uint32_t k = 0; k < kMaxRowsPerUnit / 32; ++k) {
                            const uint32_t r = k * 32 + lane;
                            rows[k] = r < n_r ? __ldg(ko + DNNS_IDX(a0 + r, z.On)) : -2;
                        }
                    }
                    const uint32_t c_lo = cc * ch, c_hi = min(Cin, c_lo + ch);
                    uint32_t p_lo = 0, p_hi = z.Cn;
                    if (identity) {
                        p_lo = c_lo, p_hi = c_hi;
                    } else if (bounds_tab) {
                        p_lo = s_chunk_start[cc], p_hi = s_chunk_start[cc + 1];
                    } else if (nch > 1) {
                        p_lo = lower_bound_idx(ki, z.Cn, c_lo);
                        p_hi = c_hi == Cin ? z.Cn : lower_bound_idx(ki, z.Cn, c_hi);
                    }
                    if (++cc == nch) cc = 0, ++rg;
                    if (p_hi == p_lo) continue;  // every channel of this chunk is dropped: nothing to bring in
                    const uint32_t Ws = (c_hi - c_lo) * blk, Wd = (p_hi - p_lo) * blk;
                    const uint32_t row_bytes = Ws * WBYTES;
                    char* const unit_dst = dst + ((size_t)a0 * Ln + (size_t)p_lo * blk) * WBYTES;
                    // rows that lose nothing and start on 16-byte boundaries are copied as they are
                    const bool image = Wd == Ws && (reinterpret_cast<uintptr_t>(unit_dst) & 15) == 0 &&
                                       (n_r == 1 || ((size_t)Ln * WBYTES & 15) == 0);
                    // the tensor where the weights equal to tau split: rows wholly before the split mask them, rows wholly
                    // after it keep them, and only a unit with a row across the split looks at positions
                    MaskCtx unit_mk = mk;
                    if (MASKED && mk.mode == 2) {
                        const uint32_t first_row = (uint32_t)__shfl_sync(0xffffffffu, rows[0], 0);
                        uint32_t last_row = 0;
#pragma unroll
                        for (uint32_t k = 0; k < kMaxRowsPerUnit / 32; ++k)
                            if ((n_r - 1) / 32 == k) last_row = (uint32_t)__shfl_sync(0xffffffffu, rows[k], (n_r - 1) & 31);
                        if ((uint64_t)(last_row + 1) * L <= mk.split_elem) unit_mk.mode = 1, unit_mk.thr_eff = mk.tau + 1u;
                        else if ((uint64_t)first_row * L >= mk.split_elem) unit_mk.mode = 1, unit_mk.thr_eff = mk.tau;
                    }
                    const uint32_t s = issued % kStages, use = issued / kStages;
                    if (!mbar_wait(&s_empty[s], (use & 1u) ^ 1u, abort_flag)) {
                        give_up();
                        alive = false;
                        break;
                    }
                    if (lane == 0) {
                        UnitDesc& d = s_desc[s];
                        d.dst = unit_dst;
                        d.ki = ki + p_lo;
                        d.ko = ko + a0;
                        d.n_r = n_r;
                        d.Wd = Wd, d.Ws = Ws, d.Ln = Ln, d.c_lo = c_lo, d.blk = blk, d.magic = it.magic, d.L = L;
                        d.n_ki = p_hi - p_lo;
                        d.ki_all = ki;
                        d.map_seq = use_map ? map_seq : 0u;
                        d.map_base = p_lo * blk;
                        d.mk = unit_mk;
                        d.kind = image ? kUnitCopy : kUnitGather;
                        mbar_arrive_expect_tx(&s_full[s], n_r * row_bytes);
                    }
                    __syncwarp();
                    // one bulk copy per run of consecutive source rows (whole rows only), 32 rows per round
                    unsigned char* const stage = stage_mem + (size_t)s * kStageBytes;
                    const char* const src_col = src + (size_t)c_lo * blk * WBYTES;
#pragma unroll
                    for (uint32_t k = 0; k < kMaxRowsPerUnit / 32; ++k) {
                        if (k * 32 < n_r) {
                            const uint32_t r = k * 32 + lane;
                            const int32_t row = rows[k];
                            const bool valid = row >= 0;
                            const int32_t prev = __shfl_up_sync(0xffffffffu, row, 1);
                            const bool head = valid && (lane == 0 || row != prev + 1 || nch > 1);
                            const uint32_t heads = __ballot_sync(0xffffffffu, head);
                            const uint32_t n_valid = __popc(__ballot_sync(0xffffffffu, valid));
                            if (head) {
                                const uint32_t later = lane == 31 ? 0u : (heads >> (lane + 1));
                                const uint32_t len = later ? (uint32_t)__ffs(later) : n_valid - lane;
                                bulk_load(stage + (size_t)r * row_bytes, src_col + (size_t)DNNS_IDX(row, it.O) * L * WBYTES,
                                          len * row_bytes, &s_full[s]);
                            }
                        }
                    }
                    ++issued;
                }
            }
        }
        if (lane == 0 && atomicAdd(&counters->done_blocks, 1u) == gridDim.x - 1) {
            // every block has taken its last range: the counters are ready for the next launch on this layout
            counters->next_range = 0;
            counters->done_blocks = 0;
        }
        if (alive) {  // tell the consumers that this was all
            const uint32_t s = issued % kStages, use = issued / kStages;
            if (mbar_wait(&s_empty[s], (use & 1u) ^ 1u, abort_flag)) {
                if (lane == 0) {
                    s_desc[s].kind = kUnitStop;
                    mbar_arrive(&s_full[s]);
                }
            } else {
                give_up();
                alive = false;
            }
        }
        if (!alive) {
            // given up: the copies still in flight must land before the block's shared memory is released
            const uint32_t first = issued > (uint32_t)kStages ? issued - kStages : 0u;
            for (uint32_t u = first; u < issued; ++u) {
                const uint64_t t0 = global_ns();
                while (!mbar_try_wait(&s_full[u % kStages], (u / kStages) & 1u) && global_ns() - t0 < kWaitLimitNs) {
                }
            }
        }
        return;
    }

    // ================= consumers =================
    for (int jb = 0; jb < gb.n; ++jb) {
        const GatherJob& job = gb.job[jb];
        const RebuildItem* __restrict__ ritems = job.lay.items;
        const int32_t* __restrict__ keep_idx = job.keep_idx;
        if (!job_fits(jb)) {
            if (blockIdx.x == 0 && threadIdx.x == 0) atomicCAS(tb.status, 0u, (uint32_t)DNNS_ERR_WORKSPACE);
            continue;
        }
        // what the caller asked for beside the arena: the offset of every item, the new shape of every tensor
        for (uint32_t i = blockIdx.x * kConsumers + threadIdx.x; i < tb.n_items; i += gridDim.x * kConsumers) {
            const RebuildItem z = ritems[i];
            job.dst_offsets[i] = (uint64_t)z.off256 << 8;
            const ItemDesc& it = tb.items[i];
            if (it.tensor >= 0) {
                job.dst_shapes[2 * it.tensor] = (int32_t)z.On;
                job.dst_shapes[2 * it.tensor + 1] = (int32_t)(z.Cn * (uint32_t)it.S);
            }
        }
        // vector items (BatchNorm vectors, biases): v'[a] = v[keep[a]], a warp per piece of kVecPiece rows; all index
        // loads of a piece are issued before the first value is fetched
        {
            const uint32_t n_warps = gridDim.x * (kConsumers / 32), gwarp = blockIdx.x + gridDim.x * warp;  // neighbours in different blocks
            for (uint32_t r = gwarp; r < tb.n_vec_items; r += n_warps) {
                const uint32_t i = tb.vec_items[2 * r], a0 = tb.vec_items[2 * r + 1] * kVecPiece;
                const ItemDesc& it = tb.items[i];
                const RebuildItem z = ritems[i];
                if (a0 >= z.On) continue;
                const uint32_t* src = static_cast<const uint32_t*>(it.src);
                uint32_t* dst = reinterpret_cast<uint32_t*>(job.dst_arena + ((uint64_t)z.off256 << 8));
                const int32_t* ko = keep_idx + it.ko_off;
                constexpr int kPer = kVecPiece / 32;
                int32_t row[kPer];
                uint32_t val[kPer];
#pragma unroll
                for (int k = 0; k < kPer; ++k) {
                    const uint32_t a = a0 + k * 32 + lane;
                    row[k] = a < z.On ? __ldg(ko + a) : -1;
                }
#pragma unroll
                for (int k = 0; k < kPer; ++k) val[k] = row[k] >= 0 ? __ldg(src + DNNS_IDX(row[k], it.O)) : 0u;
#pragma unroll
                for (int k = 0; k < kPer; ++k)
                    if (row[k] >= 0) dst[a0 + k * 32 + lane] = val[k];
            }
        }
        // the element path (rows that are not multiples of 16 bytes): 16 KB destination units, a block per pair
        {
            const uint32_t total_units = job.lay.header->total_units;
            constexpr uint32_t kChunkUnits = 2;
            for (uint32_t u_lo = blockIdx.x * kChunkUnits; u_lo < total_units; u_lo += gridDim.x * kChunkUnits) {
                const uint32_t u_hi = min(total_units, u_lo + kChunkUnits);
                uint32_t unit = u_lo;
                while (unit < u_hi) {
                    const uint32_t item = job.lay.unit_item[unit];
                    const RebuildItem z = ritems[item];
                    const ItemDesc& it = tb.items[item];
                    const uint32_t item_begin = z.unit_pre;
                    const uint32_t item_end = item_begin + (uint32_t)(((uint64_t)z.On * z.Cn * (uint32_t)it.blk * (uint32_t)it.elem_bytes + kUnitBytes - 1) / kUnitBytes);
                    const char* src = (it.tensor >= 0 && job.src_arena) ? job.src_arena + it.arena_off : static_cast<const char*>(it.src);
                    const MaskCtx mk = mask_ctx(it, job.variant);
                    char* dst = job.dst_arena + ((uint64_t)z.off256 << 8);
                    const int32_t* ko = keep_idx + it.ko_off;
                    const int32_t* ki = it.in_group >= 0 ? keep_idx + it.ki_off : nullptr;
                    const uint32_t run_end = min(u_hi, item_end);
                    const uint32_t f0 = (unit - item_begin) * (kUnitBytes / it.elem_bytes);
                    if (WBYTES == 4 || it.elem_bytes == 4) gather_run<4, MASKED>(it, src, dst, ko, ki, z.On, z.Cn, f0, run_end - unit, mk);
                    else gather_run<2, MASKED>(it, src, dst, ko, ki, z.On, z.Cn, f0, run_end - unit, mk);
                    unit = run_end;
                }
            }
        }
    }
    // then the ring
    uint32_t cur_map = 0;
    for (uint32_t taken = 0;; ++taken) {
        const uint32_t s = taken % kStages, use = taken / kStages;
        if (!mbar_wait(&s_full[s], use & 1u, abort_flag)) {
            give_up();
            break;
        }
        const UnitDesc& d = s_desc[s];
        const uint32_t kind = d.kind;
        if (kind == kUnitStop) break;
        const unsigned char* stage = stage_mem + (size_t)s * kStageBytes;
        if (kind == kUnitGather && d.map_seq != 0 && d.map_seq != cur_map) {
            // a new item: all consumers are done with the old map once they meet here, then build the new one
            asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory");
            const uint32_t blk = d.blk, Ln = d.Ln, magic = d.magic;
            const int32_t* __restrict__ ki_all = d.ki_all;
            for (uint32_t j = threadIdx.x; j < Ln; j += kConsumers) {
                const uint32_t p = blk == 1 ? j : (blk == 9 ? j / 9u : __umulhi(j, magic));
                s_rowmap[j] = (uint16_t)((uint32_t)__ldg(ki_all + DNNS_IDX(p, Ln / blk)) * blk + (j - p * blk));
            }
            cur_map = d.map_seq;
            asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory");
        }
        if (kind == kUnitCopy) consume_copy<WBYTES, MASKED>(d, stage, threadIdx.x);
        else if (MASKED && d.mk.mode == 2) consume_gather<WBYTES, MASKED, true>(d, stage, s_rowmap, threadIdx.x);
        else consume_gather<WBYTES, MASKED, false>(d, stage, s_rowmap, threadIdx.x);
        __syncwarp();
        if (lane == 0) mbar_arrive(&s_empty[s]);
    }
}

}  // namespace

cudaError_t init_compact_attributes() {
    cudaError_t e = cudaSuccess;
#define DNNS_SET(W, M)                                                                                          \
    if (e == cudaSuccess)                                                                                       \
        e = cudaFuncSetAttribute(k_compact_gather<W, M>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kStages * kStageBytes));
    DNNS_SET(4, true) DNNS_SET(4, false) DNNS_SET(2, true) DNNS_SET(2, false)
#undef DNNS_SET
    return e;
}

int gather_grid(int n_sm) { return n_sm * 3 < 1024 ? n_sm * 3 : 1024; }  // three resident blocks per SM

int launch_rebuild_layout(const Tables& tb, const LayoutBatch& lb, int n_layouts, int n_sm, cudaStream_t st) {
    ScopedKernel timed("k_rebuild_layout", st);
    k_rebuild_layout<<<n_layouts, 1024, 0, st>>>(tb, lb, (uint32_t)gather_grid(n_sm));
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_compact(const Tables& tb, const GatherBatch& gb, int n_sm, cudaStream_t st, const dnns_threshold* thr,
                   const TieSplit* split) {
    const int grid = gather_grid(n_sm);
    const size_t smem = (size_t)kStages * kStageBytes;
    const bool masked = thr != nullptr;
    ScopedKernel timed(masked ? "k_compact_gather<masked>" : "k_compact_gather", st);
#define DNNS_GATHER(W, M) k_compact_gather<W, M><<<grid, kGatherThreads, smem, st>>>(tb, gb, thr, split)
    if (tb.dtype == DNNS_F32) {
        if (masked) DNNS_GATHER(4, true);
        else DNNS_GATHER(4, false);
    } else {
        if (masked) DNNS_GATHER(2, true);
        else DNNS_GATHER(2, false);
    }
#undef DNNS_GATHER
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace dnns

#ifdef DNNS_BOUNDS_CHECK
// Checked build only: violations counted so far on the current device (and the counter reset).
extern "C" unsigned int dnns_check_bounds_violations() {
    unsigned int n = 0, zero = 0;
    if (cudaDeviceSynchronize() != cudaSuccess || cudaMemcpyFromSymbol(&n, dnns::g_bounds_violations, sizeof(n)) != cudaSuccess)
        return 0xFFFFFFFFu;
    cudaMemcpyToSymbol(dnns::g_bounds_violations, &zero, sizeof(zero));
    return n + dnns::bounds_violations_sweep(true) + dnns::bounds_violations_propagate(true);
}
#endif
