// Internal declarations shared by the kernels of libdnns: device-side descriptor tables, the
// workspace map and the launch wrappers.  Nothing here is part of the public ABI.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "dnns.h"

namespace dnns {

// A tile is 16 KB of one tensor: the unit of work of every sweep and the granularity of the
// tie tables.  Tiles never straddle tensors; the last tile of a tensor may be ragged.
constexpr uint32_t kTileBytes = 16384;
constexpr int kTileThreads = 256;
constexpr int kVecPerThread = kTileBytes / 16 / kTileThreads;  // 4 x 16-byte vectors per thread

constexpr uint32_t kHistBins = 32768;    // first radix digit: the top 15 bits of a key
constexpr uint32_t kLowBins = 65536;     // second digit of a 31-bit key
constexpr uint32_t kBitmapWords = kHistBins / 32;
constexpr int kMaxVariants = 64;
constexpr uint32_t kFlagRows = 8;         // filters per unit of the flag kernel (divides 32)

struct TensorDesc {
    const void* src;        // the model's tensor
    const float* bias;      // nullable
    uint64_t arena_off;     // byte offset in a masked arena
    uint32_t numel;
    int32_t O, I, KK, S;    // KK = KH*KW, S = in_spatial
    int32_t out_group, in_group;
    int32_t seg;            // ranking segment, -1 when not prunable
    int32_t bn;             // BatchNorm that follows it, -1 when none
    uint32_t tile0, n_tiles;
    uint32_t off_mask, off_nzmap, off_outnz, off_innz;  // word offsets into the packed bit arrays
    uint32_t off_row, off_col;  // element offsets of the tensor's filters / input columns in the per-row / per-column tables
    uint32_t by_rows, pad;      // the sweep for the largest keys walks this tensor row by row (long rows of whole vectors)
};

struct GroupDesc {
    int32_t C;
    uint32_t flags;
    uint32_t off_bits;      // word offset of the keep bits
    uint32_t off_idx;       // element offset of the keep index list
    int32_t prod_begin, prod_end;  // range in prod_list (tensor ids writing this group)
    int32_t cons_begin, cons_end;  // range in cons_list (tensor ids reading this group)
};

struct BnDesc {
    const float *gamma, *beta, *mean, *var;
    int32_t C, tensor;
    int32_t bias_item;  // gather item of the tensor's bias, -1 when it has none
    float eps;
};

// What the keep propagation needs of one producer / consumer of a group, next to the lists of
// tensor ids, so that a flag word is two dependent loads away instead of four.
struct ProducerDesc {
    const float *beta, *gamma, *mean, *bias;  // BatchNorm after the producer (beta null: none) and its bias (nullable)
    uint32_t off_outnz;
    uint32_t pad;
};
struct ConsumerDesc {
    uint32_t off_innz;
    int32_t S;
};

struct SegDesc {
    uint32_t tile_begin, tile_end;  // tiles [begin, end) cover the segment (tiles of other tensors in between count 0)
    uint64_t size;
};

// One gather job of the rebuild: a weight tensor, a BatchNorm vector or a bias.
enum : int32_t { kItemElement = 0, kItemStaged = 1, kItemVector = 2 };
struct ItemDesc {
    const void* src;        // the vector, or the model's own weight tensor
    uint64_t arena_off;     // weight tensors: byte offset in a masked arena
    int32_t tensor;         // tensor index for weight items, -1 otherwise
    int32_t O, Cin, blk;    // rows, input channels, elements per (row, input channel)
    int32_t out_group, in_group;  // in_group -1: columns are kept as they are
    int32_t elem_bytes;
    uint32_t ko_off, ki_off;      // element offsets of the two groups' keep index lists
    int32_t seg;                  // ranking segment of a weight tensor, -1 when not prunable (or no tensor)
    uint32_t off_mask, numel;     // weight tensors: word offset of the packed mask bits, elements
    int32_t S;                    // weight tensors: columns per input channel (shapes are reported in columns)
    // How the rebuild handles the item:
    //   kItemStaged   rows brought into shared memory by bulk copies (weight tensors whose rows are multiples of 16 bytes)
    //   kItemVector   one value per row (BatchNorm vectors, biases): a warp copies v'[a] = v[keep[a]]
    //   kItemElement  source position computed per destination element, 16 KB destination units, a block per unit
    int32_t kind;
    int32_t ru;      // staged: rows per unit
    int32_t ch;      // input channels per chunk of a row (a multiple of 8 when a row is cut, else Cin)
    int32_t nch;     // chunks per row
    int32_t ru_c, ch_c, nch_c;  // the same for a variant that drops none of the item's input channels: longer pieces
    uint32_t magic;  // floor(2^32 / blk) + 1 for blk > 1: j / blk = umulhi(j, magic) for the j that occur
    int32_t vec_rank;  // vector items: index among the vector items
};

// What the keep counts of one variant make of an item (written by the layout kernel, read by the gather).
struct RebuildItem {
    uint32_t On, Cn;     // rows and input channels that stay
    uint32_t off256;     // offset in the destination arena, in units of 256 bytes
    uint32_t s_units;    // staged units
    uint32_t s_cost;     // bytes a staged unit reads and writes, in 64-byte granules
    uint32_t cost_pre;   // cost of the staged units of all earlier items
    uint32_t unit_pre;   // 16 KB destination units (element path) of all earlier items
    uint32_t pad;
};
struct RebuildHeader {
    uint64_t total_bytes;  // destination bytes the variant needs
    uint32_t total_cost, total_units;
    uint32_t next_range;   // ranges handed out beyond every block's first one (the first job's header counts for a launch)
    uint32_t done_blocks;  // blocks of the running gather that took their last range; the last one clears both counters
    uint32_t pad[10];
};
// The cost axis of the staged units of a variant is cut into kRangesPerBlock equal ranges per block of the gather.
// A launch rebuilds one or several variants; their ranges form one sequence, of which every block takes the one
// with its own index first and then whatever a counter hands out as blocks come free - units differ in cost per
// byte, and the small ranges even that out.
constexpr uint32_t kRangesPerBlock = 6;
__host__ __device__ inline uint32_t rebuild_ranges(uint32_t n_blocks) { return n_blocks * kRangesPerBlock; }
__host__ __device__ inline uint32_t rebuild_range_lo(uint32_t r, uint32_t n_blocks, uint32_t total_cost) {
    return (uint32_t)((uint64_t)total_cost * r / rebuild_ranges(n_blocks));
}
// One prepared layout in the workspace.
struct RebuildSlot {
    RebuildHeader* header;
    RebuildItem* items;        // [n_items]
    uint32_t* range_item;      // [rebuild_ranges(n_blocks)] the item in which each range of the cost axis starts
    uint32_t* unit_item;       // [max_units] the item of every unit of the element path
};
constexpr uint32_t kVecPiece = 256;  // rows of a vector item that one warp of the gather copies
// One variant of a gather launch.
struct GatherJob {
    RebuildSlot lay;
    const char* src_arena;   // masked arena to read, NULL: the model's own tensors
    const int32_t* keep_idx;
    char* dst_arena;
    uint64_t dst_bytes;
    uint64_t* dst_offsets;
    int32_t* dst_shapes;
    int32_t variant;         // masking rebuild: variant of the threshold call
    int32_t pad;
};
struct GatherBatch {
    int32_t n, pad;
    GatherJob job[DNNS_PORTFOLIO_MAX];
};
constexpr int kLayoutBatch = 8;  // layouts one launch of the layout kernel prepares
struct LayoutBatch {
    const int32_t* keep_count[kLayoutBatch];
    RebuildSlot slot[kLayoutBatch];
};

// Per (variant, segment) state of the radix select between its two passes.
struct SelectState {
    uint64_t k;
    uint64_t below;   // keys whose first digit is below `digit`
    uint32_t digit;   // first digit of the k-th key
    uint32_t slot;    // which second-pass histogram of the segment serves this digit
    uint32_t count;   // keys in that first-digit bucket
    uint32_t pad;
};

// A piece of work of the row-walking sweep for the largest keys: a block of rows (filters) of one tensor by a chunk of
// at most kExtremaChunkVecs 16-byte vectors of every row.
constexpr uint32_t kExtremaChunkVecs = 128;   // four vectors per lane of a warp
constexpr uint32_t kExtremaMinVecs = 96;      // rows shorter than this stay with the tile-walking sweep
constexpr uint32_t kExtremaUnitBytes = 256 * 1024;
struct ExtremaUnit {
    uint32_t tensor, row0, n_rows;
    uint32_t vec0, n_vec;  // the chunk: vectors [vec0, vec0 + n_vec) of a row
    uint32_t pad[3];
};
// Whether the row-walking sweep takes a tensor of O rows of L elements, and how it cuts it.
__host__ __device__ inline bool extrema_by_rows(uint64_t O, uint64_t L, uint32_t elem_bytes, uint32_t* n_chunks, uint32_t* rows_per_unit) {
    const uint64_t row_bytes = L * elem_bytes;
    if (row_bytes % 16 != 0 || row_bytes / 16 < kExtremaMinVecs || row_bytes >= (1ull << 31)) return false;
    const uint32_t nv = (uint32_t)(row_bytes / 16);
    const uint32_t chunks = (nv + kExtremaChunkVecs - 1) / kExtremaChunkVecs;
    const uint32_t chunk_bytes = (nv < kExtremaChunkVecs ? nv : kExtremaChunkVecs) * 16;
    uint32_t rows = kExtremaUnitBytes / chunk_bytes;
    rows = rows < 8 ? 8 : rows;
    if (rows > O) rows = (uint32_t)O;
    *n_chunks = chunks, *rows_per_unit = rows;
    return true;
}

struct Tables {
    const TensorDesc* tensors;
    const GroupDesc* groups;
    const BnDesc* bns;
    const SegDesc* segs;
    const ItemDesc* items;
    const uint32_t* tile_tensor;
    const int32_t* prod_list;
    const int32_t* cons_list;
    const ProducerDesc* producers;  // parallel to prod_list
    const ConsumerDesc* consumers;  // parallel to cons_list
    const uint32_t* flag_prefix;  // [n_tensors + 1] units of the flag kernel before each tensor
    const uint32_t* flag_unit_tensor;  // [n_flag_units] the tensor a unit belongs to
    uint32_t* ebits;        // packed "element is non-zero" bits of the latest sweep (same packing as the mask bits)
    uint32_t* status;       // device status word (a dnns_status, 0 = ok)
    uint32_t* shift_zero;   // per producer and channel (packed like the filter flags): a zero filter emits a structurally zero constant
    const uint32_t* extrema_bounds;  // [extrema_blocks + 1] tile ranges of the blocks of the extrema sweep (about equal cost)
    const ExtremaUnit* extrema_units;  // [n_extrema_units] work of the row-walking extrema sweep
    uint32_t n_extrema_units, pad_units;
    const uint32_t* vec_items;  // [n_vec_items][2] pieces of the vector items (BatchNorm vectors, biases) of the rebuild: item, piece
    uint32_t n_tensors, n_groups, n_bn, n_segs, n_items, n_tiles, n_flag_units, n_vec_items, extrema_blocks;
    uint32_t tile_elems;    // 4096 (fp32) or 8192 (bf16)
    int32_t dtype;
};

// Where a variant stops masking the weights equal to tau, in the ranking order of its segment (tensors in descriptor
// order, row-major inside): the first such weight that stays.  tensor = 0xFFFFFFFF: none of them stays.
struct TieSplit {
    uint32_t tensor, elem;
};

struct ThresholdWs {
    uint64_t* k_dev;        // [n_k][S]
    uint32_t* hist1;        // [S][kHistBins]
    uint32_t* hist2;        // [S][n_k][kLowBins] (fp32 only)
    uint32_t* bitmap;       // [S][kBitmapWords]: first digits that some variant selected
    uint32_t* tie_bitmap;   // [S][kBitmapWords]: low 15 bits of the thresholds that need tie tables
    SelectState* sel;       // [n_k][S]
    uint32_t* need;         // [n_k][S]: the variant masks only part of the weights equal to tau
    uint32_t* any_need;     // [1]
    uint32_t* tile_ties;    // [max_variants][n_tiles]: weights equal to tau_v in the tile
    uint32_t* tie_prefix;   // [max_variants][n_tiles]: those in earlier tiles of the segment
    TieSplit* split;        // [n_k][S]
    uint32_t* hist_done;    // [1] blocks of the first sweep that are done (NULL: the digit selection is a launch of its own)
    // 31-bit keys: the second sweep lists the keys it counts with their positions, so that the place where the weights
    // equal to tau split is found without another sweep (tie_list NULL: no lists, the tie sweep always runs)
    unsigned long long* tie_list;  // entries: position | low 16 key bits << 32 | histogram slot << 48 | segment << 56
    uint32_t tie_list_cap;
    uint32_t* tie_list_n;     // [1] entries appended (may exceed the capacity: then the list is not used)
    uint32_t* tie_match;      // [n_k][S][kTieMatchCap] positions of the weights equal to tau
    uint32_t* tie_match_n;    // [n_k][S]
    uint32_t* tie_fallback;   // [1] set when the lists cannot answer: the tie sweep and its scan run after all
    const uint32_t* ties_if;  // non-null: the tie sweep and its scan return at once while this word is zero
};
constexpr uint32_t kTieMatchCap = 1024;   // weights equal to tau per (variant, segment) that the lists handle
constexpr uint32_t kTieListMaxSegs = 255, kTieListMaxPairs = 1024;  // segment and slot fit a byte; (variant, segment) pairs in shared memory
constexpr uint32_t kFusedSelectSegs = 4;  // up to this many segments the first sweep's last block selects the digits

constexpr int kMultiMax = DNNS_MULTI_MAX;  // variants one multi-variant sweep can produce
constexpr int kPortfolioMax = DNNS_PORTFOLIO_MAX;  // variants one portfolio-wide call (zero structures, keep sets) can take

// Per-variant arguments of the multi-variant sweep (unused slots repeat slot 0).
struct MultiSweepArgs {
    int32_t variant[kMultiMax];
    char* dst[kMultiMax];            // masked arenas
    uint32_t* mask_bits[kMultiMax];  // nullable
    uint32_t* ebits[kMultiMax];      // packed element bits in the workspace, one buffer per slot
    uint32_t* clear_a[kMultiMax];    // filter flags (out_nz) ...
    uint32_t* clear_b[kMultiMax];    // ... and input-column flags (in_nz): cleared by the sweep, OR-ed by k_flags
};

constexpr int kMaxCascadePasses = 64;

// Scratch of the fixed-point keep propagation.
struct CascadeWs {
    uint32_t* rem[2];        // removal words of all groups (packed like the keep bits), previous / next pass
    uint32_t* lost;          // dead channels that somebody still reads, as judged by the last pass
    uint32_t* live;          // filter flags, then (at live_in_offset words) input-column flags of the current pass
    uint32_t live_in_offset;
    uint32_t* changed;       // [kMaxCascadePasses + 1] pass p removed something
};

// ---- optional per-kernel timing (dnns_plan_profile): while a plan's profile is on, every kernel launch
// of its calls is bracketed by a pair of CUDA events on the launching stream.
struct KernelTimer;
struct ScopedKernel {
    KernelTimer* t;
    cudaStream_t st;
    int rec;
    ScopedKernel(const char* name, cudaStream_t stream);  // records the start event when a profile is on
    ~ScopedKernel();                                       // records the stop event
};

// ---- launch wrappers (each returns the number of kernels it launched, or -1 on a CUDA error) ----
int launch_threshold(const Tables& tb, const ThresholdWs& ws, int n_k, const uint64_t* k_host, dnns_threshold* thr_dev,
                     int n_sm, cudaStream_t st);
int launch_tie_tables(const Tables& tb, const ThresholdWs& ws, int n_k, const dnns_threshold* thr_dev, int n_sm,
                      cudaStream_t st);  // per-tile counts of the weights equal to tau and their prefix sums, on their own
int launch_tile_sweep(const Tables& tb, const ThresholdWs& ws, bool do_mask, bool do_struct,
                      const dnns_threshold* thr_dev, int variant, const void* src_arena, void* dst_arena,
                      uint32_t* mask_bits, uint32_t* nz_map, uint32_t* out_nz, uint32_t* in_nz, uint32_t n_out_words,
                      uint32_t n_in_words, int n_sm, cudaStream_t st);
int launch_multi_sweep(const Tables& tb, const ThresholdWs& ws, const dnns_threshold* thr_dev, const MultiSweepArgs& ma,
                       int n_variants, uint32_t* const* nz_map, uint32_t n_out_words, uint32_t n_in_words, int n_sm,
                       cudaStream_t st);
int launch_propagate(const Tables& tb, const uint32_t* out_nz, const uint32_t* in_nz, uint32_t policy,
                     int32_t min_keep, uint32_t* keep_bits, int32_t* keep_idx, int32_t* keep_count, uint64_t* stats,
                     cudaStream_t st);
int launch_propagate_multi(const Tables& tb, int n_variants, const uint32_t* const* out_nz, const uint32_t* const* in_nz,
                           uint32_t policy, int32_t min_keep, uint32_t* const* keep_bits, int32_t* const* keep_idx,
                           int32_t* const* keep_count, uint64_t* stats, cudaStream_t st);
int launch_propagate_cascade(const Tables& tb, const CascadeWs& cw, const uint32_t* nz_map, uint32_t policy,
                             int32_t min_keep, int32_t max_passes, uint32_t* keep_bits, int32_t* keep_idx,
                             int32_t* keep_count, uint64_t* stats, uint32_t n_keep_words, uint32_t n_live_words, int n_sm,
                             cudaStream_t st);
int launch_rebuild_layout(const Tables& tb, const LayoutBatch& lb, int n_layouts, int n_sm, cudaStream_t st);
int launch_compact(const Tables& tb, const GatherBatch& gb, int n_sm, cudaStream_t st, const dnns_threshold* thr = nullptr,
                   const TieSplit* split = nullptr);
int gather_grid(int n_sm);  // blocks of the gather kernel (the layout is cut for this many)
int launch_extrema(const Tables& tb, uint32_t* rowmax, uint32_t* colmax, int n_sm, cudaStream_t st);  // (one or two launches)
int launch_extrema_flags(const Tables& tb, const uint32_t* rowmax, const uint32_t* colmax, const dnns_threshold* thr,
                         const TieSplit* split, int first_variant, int n_variants, uint32_t* const* out_nz,
                         uint32_t* const* in_nz, cudaStream_t st);
// One 16 KB tile of a rebuilt tensor that the conv+BN fusion scales (listed by its first kernel, read by its second).
struct FoldJob {
    char* w;             // the rebuilt tensor
    const float* scale;  // per-filter factors
    uint32_t Ln, total;  // elements per filter, elements of the tensor
    uint32_t e0, pad;    // first element of the tile
};
int launch_fold(const Tables& tb, void* arena, const uint64_t* offsets, const int32_t* shapes, uint32_t* job_count,
                FoldJob* jobs, int n_sm, cudaStream_t st);
cudaError_t init_kernel_attributes();
cudaError_t init_compact_attributes();
constexpr uint32_t kGatherStageBytes = 18432;  // one stage buffer of the staged rebuild
constexpr uint32_t kGatherPieceBytes = 2304;   // longest piece of a row in a unit (64 channels of a 3x3 fp32 filter)

// ---- checked build (-DDNNS_BOUNDS_CHECK, a second library used by the tests only): indices into keep lists, source
// elements, bit arrays and flag words are compared with their extent first; a violation is counted (one counter per
// source file, summed by dnns_check_bounds_violations) and the access goes to element 0 instead, so nothing faults.
// The normal build compiles the checks away.
#ifdef DNNS_BOUNDS_CHECK
#define DNNS_BOUNDS_COUNTER __device__ unsigned int g_bounds_violations = 0;
#define DNNS_IDX(i, n) ((uint32_t)(i) < (uint32_t)(n) ? (uint32_t)(i) : (atomicAdd(&g_bounds_violations, 1u), 0u))
unsigned int bounds_violations_sweep(bool reset);      // counters of the other source files (compact.cu holds its own)
unsigned int bounds_violations_propagate(bool reset);
#else
#define DNNS_BOUNDS_COUNTER
#define DNNS_IDX(i, n) (i)
#endif

// ---- small device helpers ----
template <int DT>
struct Elem;
template <>
struct Elem<DNNS_F32> {
    static constexpr int kPerVec = 4;
    static constexpr int kBytes = 4;
};
template <>
struct Elem<DNNS_BF16> {
    static constexpr int kPerVec = 8;
    static constexpr int kBytes = 2;
};

// Magnitude keys of the elements of one 16-byte vector, in element order.
template <int DT>
__device__ __forceinline__ void vec_keys(const uint4& v, uint32_t (&key)[Elem<DT>::kPerVec]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    if (DT == DNNS_F32) {
#pragma unroll
        for (int j = 0; j < 4; ++j) key[j] = w[j] & 0x7FFFFFFFu;
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            key[2 * j] = w[j] & 0x7FFFu;
            key[2 * j + 1] = (w[j] >> 16) & 0x7FFFu;
        }
    }
}

// First radix digit (top 15 bits) of a key.
template <int DT>
__device__ __forceinline__ uint32_t digit_of(uint32_t key) {
    return DT == DNNS_F32 ? key >> 16 : key;
}

// Load the vector holding elements [e, e + kPerVec) of a tensor of `numel` elements; elements
// past the end read as zero.  Returns how many elements are valid.
template <int DT, bool READ_ONLY = true>
__device__ __forceinline__ int load_vec(const void* base, uint32_t e, uint32_t numel, uint4& v) {
    constexpr int P = Elem<DT>::kPerVec;
    if (e + P <= numel) {
        const uint4* p = reinterpret_cast<const uint4*>(static_cast<const char*>(base) + (size_t)e * Elem<DT>::kBytes);
        v = READ_ONLY ? __ldg(p) : *p;   // READ_ONLY = false when the kernel may overwrite the tensor in place
        return P;
    }
    v = make_uint4(0, 0, 0, 0);
    if (e >= numel) return 0;
    const int n = (int)(numel - e);
    uint32_t w[4] = {0, 0, 0, 0};
    if (DT == DNNS_F32) {
        const uint32_t* p = static_cast<const uint32_t*>(base) + e;
        for (int j = 0; j < n; ++j) w[j] = p[j];
    } else {
        const uint16_t* p = static_cast<const uint16_t*>(base) + e;
        for (int j = 0; j < n; ++j) w[j >> 1] |= (uint32_t)p[j] << (16 * (j & 1));
    }
    v = make_uint4(w[0], w[1], w[2], w[3]);
    return n;
}

template <int DT>
__device__ __forceinline__ void store_vec(void* base, uint32_t e, uint32_t numel, const uint4& v) {
    constexpr int P = Elem<DT>::kPerVec;
    if (e + P <= numel) {
        *reinterpret_cast<uint4*>(static_cast<char*>(base) + (size_t)e * Elem<DT>::kBytes) = v;
        return;
    }
    if (e >= numel) return;
    const int n = (int)(numel - e);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    if (DT == DNNS_F32) {
        uint32_t* p = static_cast<uint32_t*>(base) + e;
        for (int j = 0; j < n; ++j) p[j] = w[j];
    } else {
        uint16_t* p = static_cast<uint16_t*>(base) + e;
        for (int j = 0; j < n; ++j) p[j] = (uint16_t)(w[j >> 1] >> (16 * (j & 1)));
    }
}

// Exclusive prefix sum over the threads of a block (blockDim.x a multiple of 32, at most 1024).
// `scratch` holds 33 words of shared memory.  Returns the exclusive prefix; *total gets the sum.
template <typename T>
__device__ __forceinline__ T block_exclusive_scan(T x, T* scratch, T* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
    T incl = x;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        T y = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += y;
    }
    __syncthreads();
    if (lane == 31) scratch[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        T w = lane < nwarp ? scratch[lane] : T(0);
        T wi = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            T y = __shfl_up_sync(0xffffffffu, wi, d);
            if (lane >= d) wi += y;
        }
        scratch[lane] = wi - w;
        if (lane == 31) scratch[32] = wi;
    }
    __syncthreads();
    *total = scratch[32];
    return scratch[warp] + incl - x;
}

}  // namespace dnns
