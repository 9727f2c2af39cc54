// Host side of libdnns: model validation, table construction, workspace map and the C entry
// points.  Every entry point checks its arguments on the host, enqueues kernels and returns.
#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include <string>

#include <nvtx3/nvToolsExt.h>

#include "dnns_internal.cuh"

using namespace dnns;

namespace dnns {

struct KernelTimer {
    struct Rec {
        const char* name;
        cudaEvent_t start, stop;
    };
    bool on = false;
    std::vector<Rec> recs;
    void clear() {
        for (Rec& r : recs) {
            cudaEventDestroy(r.start);
            cudaEventDestroy(r.stop);
        }
        recs.clear();
    }
};

static thread_local KernelTimer* g_timer = nullptr;  // the profile of the plan whose call is running on this thread

ScopedKernel::ScopedKernel(const char* name, cudaStream_t stream) : t(g_timer), st(stream), rec(-1) {
    if (!t || !t->on) return;
    KernelTimer::Rec r{name, nullptr, nullptr};
    if (cudaEventCreate(&r.start) != cudaSuccess) return;
    if (cudaEventCreate(&r.stop) != cudaSuccess) {
        cudaEventDestroy(r.start);
        return;
    }
    t->recs.push_back(r);
    rec = (int)t->recs.size() - 1;
    cudaEventRecord(r.start, st);
}

ScopedKernel::~ScopedKernel() {
    if (rec >= 0) cudaEventRecord(t->recs[rec].stop, st);
}

}  // namespace dnns

namespace {

constexpr uint64_t kAlign = 256;
inline uint64_t align_up(uint64_t x, uint64_t a = kAlign) { return (x + a - 1) / a * a; }

// Byte offsets of every section of the workspace.
struct WsMap {
    uint64_t tensors, groups, bns, segs, items, tile_tensor, prod_list, cons_list, producers, consumers, flag_prefix, flag_unit_tensor, status;
    uint64_t tables_end;  // everything before this is uploaded once at plan creation
    uint64_t k_dev, bitmap, sel, tie_prefix, tie_split, layouts, ebits, rowmax, colmax;
    uint64_t vec_items, extrema_bounds, extrema_units;
    uint64_t casc_rem0, casc_rem1, casc_lost, casc_live, casc_changed;
    uint64_t shift_zero;             // bit words of the keep propagation's statistics
    uint64_t fold_count, fold_jobs;  // the conv+BN fusion's list of tiles that hold rebuilt weights
    uint64_t clear_begin;  // [clear_begin, hist2 + used part) is zeroed by every threshold call
    uint64_t any_need, hist_done, tie_list_n, tie_fallback, tie_match_n, need, tie_bitmap, tile_ties, hist1, hist2;
    uint64_t tie_list, tie_match;  // (outside the cleared region)
    uint64_t total;
};

struct Counts {
    uint32_t T = 0, G = 0, B = 0, S = 0, items = 0, tiles = 0, n_bias = 0;
    uint64_t mask_words = 0, keep_words = 0, out_words = 0, in_words = 0, flag_units = 0;
    uint64_t sum_O = 0, sum_I = 0;           // filters / input columns of all tensors
    uint64_t tie_list_entries = 0;           // entries of the second ranking sweep's list (0: the plan keeps none)
    uint32_t extrema_units = 0;              // units of the row-walking sweep for the largest keys
    uint32_t n_vec = 0, element_units = 0;   // vector items of the rebuild; 16 KB units its element path can need at most
    int dtype = 0, elem_bytes = 4;
};

// Units of the flag kernel a tensor is cut into: kFlagRows filters x 32 kernel-map words when a filter is a
// power-of-two number of map words, else 32 kernels.
uint64_t flag_units_of(const dnns_tensor& t) {
    const uint64_t n_kernels = (uint64_t)t.O * t.I, wpr = t.I / 32;
    if (t.I % 32 == 0 && (wpr & (wpr - 1)) == 0) return (((uint64_t)t.O + kFlagRows - 1) / kFlagRows) * ((wpr + 31) / 32);
    return (n_kernels + 31) / 32;
}

// How the rebuild stages a weight tensor in shared memory: a unit is a block of rows (filters) by a range of input
// channels that fits one stage buffer.  Row pieces are kept at or below kGatherPieceBytes so that a unit has at
// least eight rows for a thread to walk down; a row is cut at multiples of 8 channels, which is a multiple of 16
// bytes for either element width (bulk copies).  ru stays 0 when the tensor cannot be staged: rows that are not
// multiples of 16 bytes, 2-D kernels so large that eight of them exceed a stage buffer.
void stage_plan(ItemDesc* it) {
    const uint64_t cell = (uint64_t)it->blk * it->elem_bytes, row_bytes = cell * it->Cin;
    if (row_bytes % 16 != 0 || (uint64_t)it->Cin * it->blk >= (1ull << 31)) return;
    auto shape = [&](uint64_t longest_piece, int32_t* ru, int32_t* ch, int32_t* nch) {
        uint64_t piece = row_bytes;
        if (row_bytes <= longest_piece) {
            *ch = it->Cin, *nch = 1;
        } else {
            uint64_t c = (longest_piece / cell) & ~7ull;
            if (c == 0) c = 8;
            piece = c * cell;
            if (piece > kGatherStageBytes) return false;
            *ch = (int32_t)c, *nch = (int32_t)((it->Cin + c - 1) / c);
        }
        *ru = (int32_t)std::min<uint64_t>(256, kGatherStageBytes / piece);
        return true;
    };
    int32_t ru, ch, nch;
    if (!shape(kGatherPieceBytes, &ru, &ch, &nch) || !shape(kGatherStageBytes, &it->ru_c, &it->ch_c, &it->nch_c)) return;
    it->ru = ru, it->ch = ch, it->nch = nch;
    it->kind = kItemStaged;
    it->magic = it->blk > 1 ? (uint32_t)((1ull << 32) / (uint32_t)it->blk) + 1u : 0u;
}

bool tensor_extents_ok(const dnns_tensor& t) {
    return t.O > 0 && t.I > 0 && t.KH > 0 && t.KW > 0 && t.in_spatial > 0;
}

// Shape-level validation and counting; no device access.
dnns_status inspect(const dnns_model* m, dnns_scope scope, int32_t maxv, Counts* c) {
    if (!m || !m->tensors || !m->groups || m->n_tensors <= 0 || m->n_groups <= 0 || m->n_bn < 0) return DNNS_ERR_INVALID_ARG;
    if (m->n_bn > 0 && !m->bns) return DNNS_ERR_INVALID_ARG;
    if (scope != DNNS_SCOPE_GLOBAL && scope != DNNS_SCOPE_PER_TENSOR) return DNNS_ERR_INVALID_ARG;
    if (maxv < 1 || maxv > kMaxVariants) return DNNS_ERR_UNSUPPORTED;
    c->T = m->n_tensors, c->G = m->n_groups, c->B = m->n_bn;
    c->dtype = m->tensors[0].dtype;
    if (c->dtype != DNNS_F32 && c->dtype != DNNS_BF16) return DNNS_ERR_UNSUPPORTED;
    c->elem_bytes = c->dtype == DNNS_F32 ? 4 : 2;
    for (int g = 0; g < m->n_groups; ++g) {
        if (m->groups[g].C <= 0) return DNNS_ERR_INVALID_ARG;
        if (m->groups[g].C > 65536) return DNNS_ERR_UNSUPPORTED;
        c->keep_words += ((uint64_t)m->groups[g].C + 31) / 32;
    }
    uint64_t n_prunable = 0, seg_count = 0;
    for (int i = 0; i < m->n_tensors; ++i) {
        const dnns_tensor& t = m->tensors[i];
        if (!t.data || !tensor_extents_ok(t)) return DNNS_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(t.data) & 15) return DNNS_ERR_INVALID_ARG;
        if (t.dtype != c->dtype) return DNNS_ERR_UNSUPPORTED;
        if (t.out_group < 0 || t.out_group >= m->n_groups || t.in_group < 0 || t.in_group >= m->n_groups)
            return DNNS_ERR_BAD_GRAPH;
        if (t.O != m->groups[t.out_group].C) return DNNS_ERR_BAD_GRAPH;
        if ((int64_t)t.I != (int64_t)m->groups[t.in_group].C * t.in_spatial) return DNNS_ERR_BAD_GRAPH;
        const uint64_t numel = (uint64_t)t.O * t.I * t.KH * t.KW;
        if (numel >= (1ull << 31)) return DNNS_ERR_UNSUPPORTED;
        c->tiles += (uint32_t)((numel * c->elem_bytes + kTileBytes - 1) / kTileBytes);
        c->mask_words += (numel + 31) / 32;
        c->out_words += ((uint64_t)t.O + 31) / 32;
        c->sum_O += t.O, c->sum_I += t.I;
        c->in_words += ((uint64_t)t.I + 31) / 32;
        c->flag_units += flag_units_of(t);
        if (t.bias) ++c->n_bias;
        {
            uint32_t chunks, rows;
            if (extrema_by_rows(t.O, (uint64_t)t.I * t.KH * t.KW, c->elem_bytes, &chunks, &rows))
                c->extrema_units += chunks * (((uint32_t)t.O + rows - 1) / rows);
        }
        {   // tensors the rebuild cannot stage take its element path: 16 KB units, at most the whole tensor
            ItemDesc probe{};
            probe.Cin = t.I / t.in_spatial, probe.blk = t.KH * t.KW * t.in_spatial, probe.elem_bytes = c->elem_bytes;
            stage_plan(&probe);
            if (probe.kind != kItemStaged) c->element_units += (uint32_t)((numel * c->elem_bytes + 16383) / 16384);
        }
        if (t.prunable) {
            n_prunable += numel;
            ++seg_count;
        }
    }
    if (scope == DNNS_SCOPE_GLOBAL) {
        if (n_prunable >= (1ull << 32)) return DNNS_ERR_UNSUPPORTED;
        c->S = n_prunable ? 1 : 0;
    } else {
        c->S = (uint32_t)seg_count;
    }
    // 31-bit keys: the second ranking sweep keeps a list of the keys it counts (the tie split then needs no sweep of
    // its own) where segment and slot fit its entries and the (variant, segment) pairs fit shared memory
    if (c->dtype == DNNS_F32 && c->S >= 1 && c->S <= kTieListMaxSegs && (uint64_t)maxv * c->S <= kTieListMaxPairs &&
        c->tiles < (1u << 20))
        c->tie_list_entries = std::max<uint64_t>(65536, n_prunable / 16);
    std::vector<char> has_bn(m->n_tensors, 0);
    for (int b = 0; b < m->n_bn; ++b) {
        const dnns_bn& bn = m->bns[b];
        if (!bn.gamma || !bn.beta || !bn.mean || !bn.var) return DNNS_ERR_INVALID_ARG;
        if (bn.tensor < 0 || bn.tensor >= m->n_tensors) return DNNS_ERR_BAD_GRAPH;
        if (bn.C != m->tensors[bn.tensor].O) return DNNS_ERR_BAD_GRAPH;
        if (has_bn[bn.tensor]) return DNNS_ERR_BAD_GRAPH;
        has_bn[bn.tensor] = 1;
    }
    c->items = c->T + 4 * c->B + c->n_bias;
    // vector items are dealt out in pieces of kVecPiece rows
    c->n_vec = 0;
    for (int b = 0; b < m->n_bn; ++b) c->n_vec += 4 * (((uint32_t)m->bns[b].C + kVecPiece - 1) / kVecPiece);
    for (int i = 0; i < m->n_tensors; ++i)
        if (m->tensors[i].bias) c->n_vec += ((uint32_t)m->tensors[i].O + kVecPiece - 1) / kVecPiece;
    return DNNS_OK;
}

// Prepared layouts of the rebuild (one per set of keep counts in use): header, item table, block starts, unit -> item.
constexpr uint32_t kMaxGatherBlocks = 1024;
constexpr uint32_t kMaxSweepBlocks = 4096;  // blocks of the extrema sweep (three per SM)
uint64_t layout_slot_bytes(const Counts& c) {
    return align_up(sizeof(RebuildHeader)) + align_up(sizeof(RebuildItem) * (uint64_t)c.items) + align_up(4ull * rebuild_ranges(kMaxGatherBlocks)) +
           align_up(4ull * (c.element_units + 1));
}
uint32_t layout_slots(int32_t maxv) { return (uint32_t)std::max(maxv, (int32_t)DNNS_MULTI_MAX) + 1; }

WsMap map_workspace(const Counts& c, int32_t maxv) {
    WsMap w{};
    uint64_t o = 0;
    auto take = [&](uint64_t bytes) {
        const uint64_t at = o;
        o = align_up(o + bytes);
        return at;
    };
    w.tensors = take(sizeof(TensorDesc) * c.T);
    w.groups = take(sizeof(GroupDesc) * c.G);
    w.bns = take(sizeof(BnDesc) * (c.B ? c.B : 1));
    w.segs = take(sizeof(SegDesc) * (c.S ? c.S : 1));
    w.items = take(sizeof(ItemDesc) * c.items);
    w.tile_tensor = take(4ull * c.tiles);
    w.prod_list = take(4ull * c.T);
    w.cons_list = take(4ull * c.T);
    w.producers = take(sizeof(ProducerDesc) * c.T);
    w.consumers = take(sizeof(ConsumerDesc) * c.T);
    w.flag_prefix = take(4ull * (c.T + 1));
    w.flag_unit_tensor = take(4ull * (c.flag_units + 1));
    w.vec_items = take(8ull * (c.n_vec + 1));
    w.extrema_bounds = take(4ull * (kMaxSweepBlocks + 1));
    w.extrema_units = take(sizeof(ExtremaUnit) * (uint64_t)(c.extrema_units + 1));
    w.status = take(4);
    w.tables_end = o;
    const uint64_t vs = (uint64_t)maxv * (c.S ? c.S : 1);
    w.k_dev = take(8 * vs);
    w.bitmap = take(4ull * kBitmapWords * (c.S ? c.S : 1));
    w.sel = take(sizeof(SelectState) * vs);
    w.tie_prefix = take(4ull * maxv * c.tiles);
    w.tie_split = take(sizeof(TieSplit) * vs);
    w.layouts = take(layout_slot_bytes(c) * layout_slots(maxv));
    w.ebits = take(4ull * c.mask_words * kMultiMax);  // one buffer per slot of the multi-variant sweep
    w.rowmax = take(4ull * c.sum_O);   // largest key per filter and per input column (portfolio-wide zero structures);
    w.colmax = take(4ull * c.sum_I);   // contiguous, cleared together
    w.casc_rem0 = take(4ull * c.keep_words);
    w.casc_rem1 = take(4ull * c.keep_words);
    w.casc_lost = take(4ull * c.keep_words);
    w.casc_live = take(4ull * (c.out_words + c.in_words));
    w.casc_changed = take(4ull * (kMaxCascadePasses + 1));
    w.shift_zero = take(4ull * (c.out_words + 1));
    w.fold_count = take(4);
    w.fold_jobs = take(sizeof(FoldJob) * (uint64_t)c.tiles);
    w.tie_list = take(8ull * c.tie_list_entries);
    w.tie_match = take(c.tie_list_entries ? 4ull * kTieMatchCap * vs : 0);
    w.clear_begin = o;
    w.any_need = take(4);
    w.hist_done = take(4);
    w.tie_list_n = take(4);
    w.tie_fallback = take(4);
    w.tie_match_n = take(4 * vs);
    w.need = take(4 * vs);
    w.tie_bitmap = take(4ull * kBitmapWords * (c.S ? c.S : 1));
    w.tile_ties = take(4ull * maxv * c.tiles);
    w.hist1 = take(4ull * kHistBins * (c.S ? c.S : 1));
    w.hist2 = take(c.dtype == DNNS_F32 ? 4ull * kLowBins * vs : 0);
    w.total = o;
    return w;
}

}  // namespace

struct dnns_plan {
    Counts c;
    WsMap map;
    dnns_scope scope;
    int32_t maxv;
    int n_sm;
    char* ws;
    Tables tb;
    ThresholdWs tws;
    bool tie_tables_valid = false;  // the per-tile tables of the weights equal to tau belong to the latest threshold call
    uint32_t n_extrema_units = 0;
    // Layouts of the rebuild prepared for sets of keep counts: the device array a dnns_propagate_keep* call wrote
    // its counts to names the slot its layout went to; dnns_compact looks its keep_count argument up here.
    std::vector<const int32_t*> layout_owner;
    uint32_t layout_next;
    // The sweep for the per-filter / per-column maxima runs beside the ranking kernels of a threshold call: a second
    // stream forked from the caller's and joined again before the call returns (host objects, no device memory).
    cudaStream_t side = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    CascadeWs kws;
    uint64_t launches;
    int last_n_k;
    KernelTimer timer;
    // host-side layout, handed out by dnns_plan_layout
    std::vector<uint64_t> arena_off, mask_off, nzmap_off, outnz_off, innz_off, keep_off, keepidx_off, seg_size;
    std::vector<int32_t> seg_of_tensor;
    dnns_layout layout;
};

namespace {
struct ProfileScope {  // makes the plan's profile the active one for the launches of one call
    explicit ProfileScope(dnns_plan* p) { dnns::g_timer = p ? &p->timer : nullptr; }
    ~ProfileScope() { dnns::g_timer = nullptr; }
};
struct Range {  // an NVTX range around the host side of one entry point, named after the step it enqueues
    explicit Range(const char* name) { nvtxRangePushA(name); }
    ~Range() { nvtxRangePop(); }
};
}  // namespace

namespace {

RebuildSlot layout_slot(const dnns_plan* p, uint32_t index) {
    char* base = p->ws + p->map.layouts + (uint64_t)index * layout_slot_bytes(p->c);
    RebuildSlot r;
    r.header = reinterpret_cast<RebuildHeader*>(base);
    base += align_up(sizeof(RebuildHeader));
    r.items = reinterpret_cast<RebuildItem*>(base);
    base += align_up(sizeof(RebuildItem) * (uint64_t)p->c.items);
    r.range_item = reinterpret_cast<uint32_t*>(base);
    base += align_up(4ull * rebuild_ranges(kMaxGatherBlocks));
    r.unit_item = reinterpret_cast<uint32_t*>(base);
    return r;
}

int find_layout(const dnns_plan* p, const int32_t* keep_count) {
    for (size_t s = 0; s < p->layout_owner.size(); ++s)
        if (p->layout_owner[s] == keep_count) return (int)s;
    return -1;
}

// Enqueue the layout kernel for n arrays of keep counts (device) and remember which slot belongs to which array.
// Returns the number of launches, -1 on a CUDA error.
int prepare_layouts(dnns_plan* p, const int32_t* const* keep_count, int n, cudaStream_t st) {
    int launches = 0;
    for (int first = 0; first < n; first += kLayoutBatch) {
        const int nb = std::min(kLayoutBatch, n - first);
        LayoutBatch lb{};
        std::vector<int> used;
        for (int i = 0; i < nb; ++i) {
            const int32_t* kc = keep_count[first + i];
            int s = find_layout(p, kc);
            if (s >= 0 && std::find(used.begin(), used.end(), s) != used.end()) s = -1;  // the same array twice in one batch
            while (s < 0) {   // the next slot in turn that this batch has not taken yet
                const int cand = (int)(p->layout_next++ % p->layout_owner.size());
                if (std::find(used.begin(), used.end(), cand) == used.end()) s = cand;
            }
            for (auto& o : p->layout_owner)
                if (o == kc) o = nullptr;
            p->layout_owner[s] = kc;
            used.push_back(s);
            lb.keep_count[i] = kc;
            lb.slot[i] = layout_slot(p, (uint32_t)s);
        }
        if (launch_rebuild_layout(p->tb, lb, nb, p->n_sm, st) < 0) return -1;
        ++launches;
    }
    return launches;
}

// The sweeps that mask tile by tile read per-tile tables of the weights equal to tau.  A threshold call that finds the
// tie split in the lists of its second sweep does not make them: the first such sweep after it enqueues them (one
// more read of the weights).
bool ensure_tie_tables(dnns_plan* p, const dnns_threshold* thr_dev, cudaStream_t st) {
    if (p->tie_tables_valid) return true;
    const int n = launch_tie_tables(p->tb, p->tws, p->last_n_k, thr_dev, p->n_sm, st);
    if (n < 0) return false;
    p->launches += n;
    p->tie_tables_valid = true;
    return true;
}

}  // namespace

extern "C" {

const char* dnns_status_string(dnns_status s) {
    switch (s) {
        case DNNS_OK: return "ok";
        case DNNS_ERR_INVALID_ARG: return "invalid argument";
        case DNNS_ERR_BAD_GRAPH: return "inconsistent model graph";
        case DNNS_ERR_WORKSPACE: return "workspace or destination arena too small";
        case DNNS_ERR_UNSUPPORTED: return "unsupported dtype or extent";
        case DNNS_ERR_CUDA: return "CUDA runtime error";
        case DNNS_ERR_TIMEOUT: return "device-side wait expired";
        case DNNS_ERR_STATIC_LIMIT: return "input exceeds the size limit of the built-in scratch (DNNS_STATIC_MAX_NUMEL)";
    }
    return "unknown status";
}

size_t dnns_workspace_bytes(const dnns_model* model, dnns_scope scope, int32_t max_variants) {
    Counts c;
    if (inspect(model, scope, max_variants, &c) != DNNS_OK) return 0;
    return (size_t)map_workspace(c, max_variants).total;
}

dnns_status dnns_plan_create(const dnns_model* m, dnns_scope scope, int32_t maxv, void* ws_dev, size_t ws_bytes,
                             void* stream, dnns_plan** plan_out) {
    if (!plan_out) return DNNS_ERR_INVALID_ARG;
    *plan_out = nullptr;
    Counts c;
    dnns_status s = inspect(m, scope, maxv, &c);
    if (s != DNNS_OK) return s;
    if (!ws_dev || (reinterpret_cast<uintptr_t>(ws_dev) & (kAlign - 1))) return DNNS_ERR_INVALID_ARG;
    const WsMap map = map_workspace(c, maxv);
    if (ws_bytes < map.total) return DNNS_ERR_WORKSPACE;

    dnns_plan* p = new (std::nothrow) dnns_plan();
    if (!p) return DNNS_ERR_INVALID_ARG;
    p->c = c, p->map = map, p->scope = scope, p->maxv = maxv, p->ws = static_cast<char*>(ws_dev);
    p->launches = 0, p->last_n_k = 0;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&p->n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        init_kernel_attributes() != cudaSuccess || init_compact_attributes() != cudaSuccess) {
        delete p;
        return DNNS_ERR_CUDA;
    }

    // ---- build the tables on the host
    std::vector<char> host(map.tables_end, 0);
    auto* td = reinterpret_cast<TensorDesc*>(host.data() + map.tensors);
    auto* gd = reinterpret_cast<GroupDesc*>(host.data() + map.groups);
    auto* bd = reinterpret_cast<BnDesc*>(host.data() + map.bns);
    auto* sd = reinterpret_cast<SegDesc*>(host.data() + map.segs);
    auto* id = reinterpret_cast<ItemDesc*>(host.data() + map.items);
    auto* tile_tensor = reinterpret_cast<uint32_t*>(host.data() + map.tile_tensor);
    auto* prod_list = reinterpret_cast<int32_t*>(host.data() + map.prod_list);
    auto* cons_list = reinterpret_cast<int32_t*>(host.data() + map.cons_list);
    auto* flag_prefix = reinterpret_cast<uint32_t*>(host.data() + map.flag_prefix);
    auto* flag_unit_tensor = reinterpret_cast<uint32_t*>(host.data() + map.flag_unit_tensor);
    auto* producers = reinterpret_cast<ProducerDesc*>(host.data() + map.producers);
    auto* consumers = reinterpret_cast<ConsumerDesc*>(host.data() + map.consumers);

    p->arena_off.resize(c.T), p->mask_off.resize(c.T), p->nzmap_off.resize(c.T), p->outnz_off.resize(c.T);
    p->innz_off.resize(c.T), p->seg_of_tensor.assign(c.T, -1), p->keep_off.resize(c.G), p->keepidx_off.resize(c.G);
    p->seg_size.assign(c.S ? c.S : 1, 0);
    uint64_t arena = 0, mask_w = 0, map_w = 0, out_w = 0, in_w = 0, compact_bytes = 0, n_prunable = 0, flag_units = 0;
    uint64_t row_e = 0, col_e = 0;
    uint32_t tb_extrema_blocks = 1;
    uint32_t tile = 0, seg = 0;
    for (uint32_t S = 0; S < c.S; ++S) sd[S] = SegDesc{0xFFFFFFFFu, 0, 0};
    for (uint32_t i = 0; i < c.T; ++i) {
        const dnns_tensor& t = m->tensors[i];
        TensorDesc& d = td[i];
        d.src = t.data, d.bias = t.bias;
        d.numel = (uint32_t)((uint64_t)t.O * t.I * t.KH * t.KW);
        d.O = t.O, d.I = t.I, d.KK = t.KH * t.KW, d.S = t.in_spatial;
        d.out_group = t.out_group, d.in_group = t.in_group;
        d.bn = -1;
        d.arena_off = arena, p->arena_off[i] = arena;
        arena = align_up(arena + (uint64_t)d.numel * c.elem_bytes);
        d.tile0 = tile;
        d.n_tiles = (uint32_t)(((uint64_t)d.numel * c.elem_bytes + kTileBytes - 1) / kTileBytes);
        for (uint32_t k = 0; k < d.n_tiles; ++k) tile_tensor[tile + k] = i;
        d.off_mask = (uint32_t)mask_w, p->mask_off[i] = mask_w, mask_w += ((uint64_t)d.numel + 31) / 32;
        d.off_nzmap = (uint32_t)map_w, p->nzmap_off[i] = map_w, map_w += ((uint64_t)t.O * t.I + 31) / 32;
        d.off_outnz = (uint32_t)out_w, p->outnz_off[i] = out_w, out_w += ((uint64_t)t.O + 31) / 32;
        d.off_innz = (uint32_t)in_w, p->innz_off[i] = in_w, in_w += ((uint64_t)t.I + 31) / 32;
        d.off_row = (uint32_t)row_e, row_e += t.O;
        d.off_col = (uint32_t)col_e, col_e += t.I;
        d.seg = -1;
        if (t.prunable) {
            const uint32_t sgi = scope == DNNS_SCOPE_GLOBAL ? 0 : seg++;
            d.seg = (int32_t)sgi;
            p->seg_of_tensor[i] = (int32_t)sgi;
            if (sd[sgi].tile_begin == 0xFFFFFFFFu) sd[sgi].tile_begin = tile;
            sd[sgi].tile_end = tile + d.n_tiles;
            sd[sgi].size += d.numel;
            p->seg_size[sgi] += d.numel;
            n_prunable += d.numel;
        }
        tile += d.n_tiles;
        flag_prefix[i] = (uint32_t)flag_units;
        const uint64_t n_units = flag_units_of(t);
        if (flag_units + n_units < (1ull << 32))
            for (uint64_t k = 0; k < n_units; ++k) flag_unit_tensor[flag_units + k] = (uint32_t)i;  // unit -> its tensor
        flag_units += n_units;
    }
    flag_prefix[c.T] = (uint32_t)flag_units;
    if (flag_units >= (1ull << 32)) {
        delete p;
        return DNNS_ERR_UNSUPPORTED;
    }
    if (mask_w >= (1ull << 32) || map_w >= (1ull << 32) || row_e >= (1ull << 32) || col_e >= (1ull << 32)) {
        delete p;
        return DNNS_ERR_UNSUPPORTED;
    }
    for (uint32_t S = 0; S < c.S; ++S)
        if (p->seg_size[S] >= (1ull << 32)) {
            delete p;
            return DNNS_ERR_UNSUPPORTED;
        }
    uint64_t keep_w = 0, keep_i = 0;
    int np = 0, nc = 0;
    for (uint32_t g = 0; g < c.G; ++g) {
        GroupDesc& G = gd[g];
        G.C = m->groups[g].C, G.flags = m->groups[g].flags;
        G.off_bits = (uint32_t)keep_w, p->keep_off[g] = keep_w, keep_w += ((uint64_t)G.C + 31) / 32;
        G.off_idx = (uint32_t)keep_i, p->keepidx_off[g] = keep_i, keep_i += G.C;
        G.prod_begin = np;
        for (uint32_t i = 0; i < c.T; ++i)
            if (m->tensors[i].out_group == (int)g) prod_list[np++] = (int32_t)i;
        G.prod_end = np;
        G.cons_begin = nc;
        for (uint32_t i = 0; i < c.T; ++i)
            if (m->tensors[i].in_group == (int)g) cons_list[nc++] = (int32_t)i;
        G.cons_end = nc;
    }
    for (uint32_t b = 0; b < c.B; ++b) {
        const dnns_bn& bn = m->bns[b];
        bd[b] = BnDesc{bn.gamma, bn.beta, bn.mean, bn.var, bn.C, bn.tensor, -1, bn.eps};
        td[bn.tensor].bn = (int32_t)b;
    }
    for (int i = 0; i < np; ++i) {
        const TensorDesc& d = td[prod_list[i]];
        ProducerDesc pd{nullptr, nullptr, nullptr, d.bias, d.off_outnz, 0};
        if (d.bn >= 0) pd.beta = bd[d.bn].beta, pd.gamma = bd[d.bn].gamma, pd.mean = bd[d.bn].mean;
        producers[i] = pd;
    }
    for (int i = 0; i < nc; ++i) consumers[i] = ConsumerDesc{td[cons_list[i]].off_innz, td[cons_list[i]].S};
    {   // the row-walking sweep for the largest keys: its tensors and their units
        auto* units = reinterpret_cast<ExtremaUnit*>(host.data() + map.extrema_units);
        uint32_t n_units = 0;
        for (uint32_t i = 0; i < c.T; ++i) {
            uint32_t chunks, rows;
            const uint64_t L = (uint64_t)td[i].I * td[i].KK;
            td[i].by_rows = extrema_by_rows(td[i].O, L, c.elem_bytes, &chunks, &rows) ? 1u : 0u;
            if (!td[i].by_rows) continue;
            const uint32_t nv = (uint32_t)(L * c.elem_bytes / 16);
            for (uint32_t r0 = 0; r0 < (uint32_t)td[i].O; r0 += rows)
                for (uint32_t ch = 0; ch < chunks; ++ch) {
                    const uint32_t v0 = ch * kExtremaChunkVecs;
                    units[n_units++] = ExtremaUnit{i, r0, std::min(rows, (uint32_t)td[i].O - r0), v0, std::min(kExtremaChunkVecs, nv - v0), {0, 0, 0}};
                }
        }
        p->n_extrema_units = n_units;
    }
    {   // tile ranges of the extrema sweep: about equal cost per block; a tile whose column maxima stay in registers
        // (rows that divide the tile) counts 2, any other tile 3
        auto* bounds = reinterpret_cast<uint32_t*>(host.data() + map.extrema_bounds);
        const uint32_t blocks = std::max(1u, std::min({(uint32_t)p->n_sm * 3u, kMaxSweepBlocks, c.tiles}));
        const uint32_t tile_elems = kTileBytes / c.elem_bytes, vec = 16 / c.elem_bytes;
        std::vector<uint64_t> cost_before(c.tiles + 1, 0);
        for (uint32_t i = 0; i < c.T; ++i) {
            const uint64_t L = (uint64_t)td[i].I * td[i].KK;
            const bool cheap = L <= tile_elems && tile_elems % L == 0 && L % vec == 0 && (uint32_t)td[i].I <= 8192u;
            // (the tiles of a tensor that the row-walking sweep takes cost this one nothing)
            for (uint32_t k = 0; k < td[i].n_tiles; ++k) cost_before[td[i].tile0 + k + 1] = td[i].by_rows ? 0 : (cheap ? 2 : 3);
        }
        for (uint32_t t = 0; t < c.tiles; ++t) cost_before[t + 1] += cost_before[t];
        uint32_t t = 0;
        for (uint32_t b = 0; b <= blocks; ++b) {
            const uint64_t want = cost_before[c.tiles] * b / blocks;
            while (t < c.tiles && cost_before[t] < want) ++t;
            bounds[b] = b == blocks ? c.tiles : t;
        }
        tb_extrema_blocks = blocks;
    }
    // gather items: weights, then BN vectors, then biases
    auto* vec_items = reinterpret_cast<uint32_t*>(host.data() + map.vec_items);
    uint32_t n_it = 0, n_vec = 0;
    for (uint32_t i = 0; i < c.T; ++i) {
        const dnns_tensor& t = m->tensors[i];
        ItemDesc w_it{};
        w_it.src = t.data, w_it.arena_off = td[i].arena_off, w_it.tensor = (int32_t)i;
        w_it.O = t.O, w_it.Cin = t.I / t.in_spatial, w_it.blk = t.KH * t.KW * t.in_spatial;
        w_it.out_group = t.out_group, w_it.in_group = t.in_group, w_it.elem_bytes = c.elem_bytes;
        w_it.ko_off = gd[t.out_group].off_idx, w_it.ki_off = gd[t.in_group].off_idx;
        w_it.seg = td[i].seg, w_it.off_mask = td[i].off_mask, w_it.numel = td[i].numel, w_it.S = t.in_spatial;
        w_it.kind = kItemElement, w_it.vec_rank = -1;
        stage_plan(&w_it);
        id[n_it++] = w_it;
        compact_bytes += align_up((uint64_t)td[i].numel * c.elem_bytes);
    }
    auto vector_item = [&](const float* v, int32_t C, int32_t group) {
        ItemDesc it{};
        it.src = v, it.tensor = -1, it.O = C, it.Cin = 1, it.blk = 1, it.out_group = group, it.in_group = -1, it.elem_bytes = 4;
        it.ko_off = gd[group].off_idx, it.seg = -1, it.S = 1, it.kind = kItemVector, it.vec_rank = (int32_t)n_vec;  // (rank of its first piece)
        for (uint32_t piece = 0; piece * kVecPiece < (uint32_t)C; ++piece) vec_items[2 * n_vec] = n_it, vec_items[2 * n_vec + 1] = piece, ++n_vec;
        id[n_it++] = it;
        compact_bytes += align_up(4ull * C);
    };
    for (uint32_t b = 0; b < c.B; ++b) {
        const dnns_bn& bn = m->bns[b];
        const float* vec[4] = {bn.gamma, bn.beta, bn.mean, bn.var};
        for (int k = 0; k < 4; ++k) vector_item(vec[k], bn.C, m->tensors[bn.tensor].out_group);
    }
    for (uint32_t i = 0; i < c.T; ++i)
        if (m->tensors[i].bias) {
            if (td[i].bn >= 0) bd[td[i].bn].bias_item = (int32_t)n_it;
            vector_item(m->tensors[i].bias, m->tensors[i].O, m->tensors[i].out_group);
        }

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(p->ws, host.data(), map.tables_end, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        delete p;
        return DNNS_ERR_CUDA;
    }

    char* w = p->ws;
    Tables& tb = p->tb;
    tb.tensors = reinterpret_cast<TensorDesc*>(w + map.tensors);
    tb.groups = reinterpret_cast<GroupDesc*>(w + map.groups);
    tb.bns = reinterpret_cast<BnDesc*>(w + map.bns);
    tb.segs = reinterpret_cast<SegDesc*>(w + map.segs);
    tb.items = reinterpret_cast<ItemDesc*>(w + map.items);
    tb.tile_tensor = reinterpret_cast<uint32_t*>(w + map.tile_tensor);
    tb.prod_list = reinterpret_cast<int32_t*>(w + map.prod_list);
    tb.cons_list = reinterpret_cast<int32_t*>(w + map.cons_list);
    tb.producers = reinterpret_cast<ProducerDesc*>(w + map.producers);
    tb.consumers = reinterpret_cast<ConsumerDesc*>(w + map.consumers);
    tb.status = reinterpret_cast<uint32_t*>(w + map.status);
    tb.shift_zero = reinterpret_cast<uint32_t*>(w + map.shift_zero);
    tb.flag_prefix = reinterpret_cast<uint32_t*>(w + map.flag_prefix);
    tb.flag_unit_tensor = reinterpret_cast<uint32_t*>(w + map.flag_unit_tensor);
    tb.ebits = reinterpret_cast<uint32_t*>(w + map.ebits);
    tb.n_flag_units = (uint32_t)flag_units;
    tb.n_tensors = c.T, tb.n_groups = c.G, tb.n_bn = c.B, tb.n_segs = c.S, tb.n_items = c.items, tb.n_tiles = c.tiles;
    tb.tile_elems = kTileBytes / c.elem_bytes;
    tb.dtype = c.dtype;
    ThresholdWs& t = p->tws;
    t.k_dev = reinterpret_cast<uint64_t*>(w + map.k_dev);
    t.hist1 = reinterpret_cast<uint32_t*>(w + map.hist1);
    t.hist2 = reinterpret_cast<uint32_t*>(w + map.hist2);
    t.bitmap = reinterpret_cast<uint32_t*>(w + map.bitmap);
    t.tie_bitmap = reinterpret_cast<uint32_t*>(w + map.tie_bitmap);
    t.sel = reinterpret_cast<SelectState*>(w + map.sel);
    t.need = reinterpret_cast<uint32_t*>(w + map.need);
    t.any_need = reinterpret_cast<uint32_t*>(w + map.any_need);
    t.hist_done = reinterpret_cast<uint32_t*>(w + map.hist_done);
    t.tie_list = c.tie_list_entries ? reinterpret_cast<unsigned long long*>(w + map.tie_list) : nullptr;
    t.tie_list_cap = (uint32_t)c.tie_list_entries;
    t.tie_list_n = reinterpret_cast<uint32_t*>(w + map.tie_list_n);
    t.tie_match = reinterpret_cast<uint32_t*>(w + map.tie_match);
    t.tie_match_n = reinterpret_cast<uint32_t*>(w + map.tie_match_n);
    t.tie_fallback = reinterpret_cast<uint32_t*>(w + map.tie_fallback);
    t.ties_if = nullptr;
    t.tile_ties = reinterpret_cast<uint32_t*>(w + map.tile_ties);
    t.tie_prefix = reinterpret_cast<uint32_t*>(w + map.tie_prefix);
    t.split = reinterpret_cast<TieSplit*>(w + map.tie_split);
    tb.vec_items = reinterpret_cast<uint32_t*>(w + map.vec_items);
    tb.n_vec_items = c.n_vec;
    tb.extrema_bounds = reinterpret_cast<uint32_t*>(w + map.extrema_bounds);
    tb.extrema_blocks = tb_extrema_blocks;
    tb.extrema_units = reinterpret_cast<ExtremaUnit*>(w + map.extrema_units);
    tb.n_extrema_units = p->n_extrema_units;
    p->layout_owner.assign(layout_slots(maxv), nullptr);
    p->layout_next = 0;
    if (cudaStreamCreateWithFlags(&p->side, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&p->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&p->ev_join, cudaEventDisableTiming) != cudaSuccess) {
        dnns_plan_destroy(p);
        return DNNS_ERR_CUDA;
    }
    p->kws.rem[0] = reinterpret_cast<uint32_t*>(w + map.casc_rem0);
    p->kws.rem[1] = reinterpret_cast<uint32_t*>(w + map.casc_rem1);
    p->kws.lost = reinterpret_cast<uint32_t*>(w + map.casc_lost);
    p->kws.live = reinterpret_cast<uint32_t*>(w + map.casc_live);
    p->kws.live_in_offset = (uint32_t)c.out_words;
    p->kws.changed = reinterpret_cast<uint32_t*>(w + map.casc_changed);

    dnns_layout& L = p->layout;
    L.n_tensors = c.T, L.n_bn = c.B, L.n_groups = c.G, L.n_segments = c.S, L.n_bias = c.n_bias;
    L.elem_bytes = c.elem_bytes;
    L.n_prunable = n_prunable;
    L.masked_arena_bytes = arena;
    L.mask_words = mask_w, L.nz_map_words = map_w, L.out_nz_words = out_w, L.in_nz_words = in_w;
    L.keep_words = keep_w, L.keep_idx_len = keep_i;
    L.compact_arena_bytes = compact_bytes;
    L.n_compact_items = (int32_t)c.items;
    L.arena_offset = p->arena_off.data(), L.mask_offset = p->mask_off.data(), L.nz_map_offset = p->nzmap_off.data();
    L.out_nz_offset = p->outnz_off.data(), L.in_nz_offset = p->innz_off.data();
    L.keep_offset = p->keep_off.data(), L.keep_idx_offset = p->keepidx_off.data();
    L.segment_size = p->seg_size.data(), L.segment_of_tensor = p->seg_of_tensor.data();
    *plan_out = p;
    return DNNS_OK;
}

void dnns_plan_destroy(dnns_plan* plan) {
    if (!plan) return;
    cudaDeviceSynchronize();
    plan->timer.clear();
    if (plan->ev_fork) cudaEventDestroy(plan->ev_fork);
    if (plan->ev_join) cudaEventDestroy(plan->ev_join);
    if (plan->side) cudaStreamDestroy(plan->side);
    delete plan;
}

dnns_status dnns_plan_layout(const dnns_plan* plan, dnns_layout* out) {
    if (!plan || !out) return DNNS_ERR_INVALID_ARG;
    *out = plan->layout;
    return DNNS_OK;
}

uint64_t dnns_plan_launch_count(const dnns_plan* plan) { return plan ? plan->launches : 0; }

dnns_status dnns_magnitude_threshold(dnns_plan* p, const uint64_t* k, int32_t n_k, dnns_threshold* thr_dev,
                                     void* stream) {
    Range nvtx_range("dnns: step 1 threshold");
    if (!p || !k || !thr_dev || n_k < 1 || n_k > p->maxv) return DNNS_ERR_INVALID_ARG;
    const uint32_t S = p->c.S;
    if (S == 0) return DNNS_OK;
    for (int v = 0; v < n_k; ++v)
        for (uint32_t s = 0; s < S; ++s)
            if (k[(size_t)v * S + s] > p->seg_size[s]) return DNNS_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint64_t clear_end = p->map.hist2 + (p->c.dtype == DNNS_F32 ? 4ull * kLowBins * S * n_k : 0);
    if (cudaMemsetAsync(p->ws + p->map.clear_begin, 0, clear_end - p->map.clear_begin, st) != cudaSuccess)
        return DNNS_ERR_CUDA;
    ProfileScope profile_scope(p);
    // beside the ranking: the largest key of every filter and every input column, for dnns_zero_structures_portfolio
    uint32_t* rowmax = reinterpret_cast<uint32_t*>(p->ws + p->map.rowmax);
    const uint64_t clear_bytes = p->map.colmax + 4ull * p->c.sum_I - p->map.rowmax;  // both tables: the maxima start at zero
    if (cudaEventRecord(p->ev_fork, st) != cudaSuccess || cudaStreamWaitEvent(p->side, p->ev_fork, 0) != cudaSuccess ||
        cudaMemsetAsync(rowmax, 0, clear_bytes, p->side) != cudaSuccess)
        return DNNS_ERR_CUDA;
    const int n_side = launch_extrema(p->tb, rowmax, reinterpret_cast<uint32_t*>(p->ws + p->map.colmax), p->n_sm, p->side);
    const bool joined = cudaEventRecord(p->ev_join, p->side) == cudaSuccess;
    const int n = launch_threshold(p->tb, p->tws, n_k, k, thr_dev, p->n_sm, st);
    if (!joined || cudaStreamWaitEvent(st, p->ev_join, 0) != cudaSuccess || n < 0 || n_side < 0) return DNNS_ERR_CUDA;
    p->launches += n + n_side;
    p->last_n_k = n_k;
    p->tie_tables_valid = p->tws.tie_list == nullptr;  // (a call that found the tie split in its lists may have left them out)
    return DNNS_OK;
}

dnns_status dnns_apply_mask(dnns_plan* p, const dnns_threshold* thr_dev, int32_t variant, void* masked_arena,
                            uint32_t* mask_bits, void* stream) {
    Range nvtx_range("dnns: step 2 mask");
    if (!p || !thr_dev || variant < 0 || variant >= p->last_n_k) return DNNS_ERR_INVALID_ARG;  // a variant of the latest threshold call
    if (masked_arena && (reinterpret_cast<uintptr_t>(masked_arena) & 15)) return DNNS_ERR_INVALID_ARG;
    ProfileScope profile_scope(p);
    if (!ensure_tie_tables(p, thr_dev, static_cast<cudaStream_t>(stream))) return DNNS_ERR_CUDA;
    const int n = launch_tile_sweep(p->tb, p->tws, true, false, thr_dev, variant, nullptr, masked_arena, mask_bits,
                                    nullptr, nullptr, nullptr, 0, 0, p->n_sm, static_cast<cudaStream_t>(stream));
    if (n < 0) return DNNS_ERR_CUDA;
    p->launches += n;
    return DNNS_OK;
}

dnns_status dnns_zero_structures(dnns_plan* p, const void* masked_arena, uint32_t* nz_map, uint32_t* out_nz,
                                 uint32_t* in_nz, void* stream) {
    Range nvtx_range("dnns: step 3 zero structures");
    if (!p || !out_nz || !in_nz) return DNNS_ERR_INVALID_ARG;
    if (masked_arena && (reinterpret_cast<uintptr_t>(masked_arena) & 15)) return DNNS_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const dnns_layout& L = p->layout;
    // (the sweep clears the flag words before the flag kernel ORs into them)
    ProfileScope profile_scope(p);
    const int n = launch_tile_sweep(p->tb, p->tws, false, true, nullptr, 0, masked_arena, nullptr, nullptr, nz_map,
                                    out_nz, in_nz, (uint32_t)L.out_nz_words, (uint32_t)L.in_nz_words, p->n_sm, st);
    if (n < 0) return DNNS_ERR_CUDA;
    p->launches += n;
    return DNNS_OK;
}

dnns_status dnns_mask_and_structures(dnns_plan* p, const dnns_threshold* thr_dev, int32_t variant, void* masked_arena,
                                     uint32_t* mask_bits, uint32_t* nz_map, uint32_t* out_nz, uint32_t* in_nz,
                                     void* stream) {
    Range nvtx_range("dnns: steps 2+3");
    if (!p || !thr_dev || !out_nz || !in_nz || variant < 0 || variant >= p->last_n_k) return DNNS_ERR_INVALID_ARG;
    if (masked_arena && (reinterpret_cast<uintptr_t>(masked_arena) & 15)) return DNNS_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const dnns_layout& L = p->layout;
    // the flag words are OR-ed into; the kernel map is stored word by word and needs no clearing
    ProfileScope profile_scope(p);
    if (!ensure_tie_tables(p, thr_dev, st)) return DNNS_ERR_CUDA;
    const int n = launch_tile_sweep(p->tb, p->tws, true, true, thr_dev, variant, nullptr, masked_arena, mask_bits,
                                    nz_map, out_nz, in_nz, (uint32_t)L.out_nz_words, (uint32_t)L.in_nz_words, p->n_sm, st);
    if (n < 0) return DNNS_ERR_CUDA;
    p->launches += n;
    return DNNS_OK;
}

dnns_status dnns_mask_and_structures_multi(dnns_plan* p, const dnns_threshold* thr_dev, int32_t first_variant,
                                           int32_t n_variants, void* const* masked_arenas, uint32_t* const* mask_bits,
                                           uint32_t* const* nz_map, uint32_t* const* out_nz, uint32_t* const* in_nz,
                                           void* stream) {
    Range nvtx_range("dnns: steps 2+3, several variants");
    if (!p || !thr_dev || !masked_arenas || !out_nz || !in_nz || n_variants < 1 || n_variants > kMultiMax ||
        first_variant < 0 || first_variant + n_variants > p->last_n_k)
        return DNNS_ERR_INVALID_ARG;
    // masked_arenas all NULL: the masked weights are not written (see dnns_compact_masked); mask bits are then required
    bool no_store = true;
    for (int g = 0; g < n_variants; ++g) no_store = no_store && masked_arenas[g] == nullptr;
    if (no_store && !mask_bits) return DNNS_ERR_INVALID_ARG;
    MultiSweepArgs ma;
    for (int g = 0; g < kMultiMax; ++g) {
        const int s = g < n_variants ? g : 0;
        if (!out_nz[s] || !in_nz[s]) return DNNS_ERR_INVALID_ARG;
        if (no_store) {
            if (!mask_bits[s]) return DNNS_ERR_INVALID_ARG;
        } else if (!masked_arenas[s] || (reinterpret_cast<uintptr_t>(masked_arenas[s]) & 15)) {
            return DNNS_ERR_INVALID_ARG;
        }
        for (int h = 0; h < s; ++h) {  // every variant needs buffers of its own
            if ((!no_store && masked_arenas[h] == masked_arenas[s]) || out_nz[h] == out_nz[s] || in_nz[h] == in_nz[s])
                return DNNS_ERR_INVALID_ARG;
            if (mask_bits && mask_bits[s] && mask_bits[h] == mask_bits[s]) return DNNS_ERR_INVALID_ARG;
        }
        ma.variant[g] = first_variant + s;
        ma.dst[g] = no_store ? nullptr : static_cast<char*>(masked_arenas[s]);
        ma.mask_bits[g] = mask_bits ? mask_bits[s] : nullptr;
        ma.ebits[g] = p->tb.ebits + (size_t)s * p->c.mask_words;
        ma.clear_a[g] = out_nz[s];
        ma.clear_b[g] = in_nz[s];
    }
    const dnns_layout& L = p->layout;
    ProfileScope profile_scope(p);
    if (!ensure_tie_tables(p, thr_dev, static_cast<cudaStream_t>(stream))) return DNNS_ERR_CUDA;
    const int n = launch_multi_sweep(p->tb, p->tws, thr_dev, ma, n_variants, nz_map, (uint32_t)L.out_nz_words,
                                     (uint32_t)L.in_nz_words, p->n_sm, static_cast<cudaStream_t>(stream));
    if (n < 0) return DNNS_ERR_CUDA;
    p->launches += n;
    return DNNS_OK;
}

dnns_status dnns_zero_structures_portfolio(dnns_plan* p, const dnns_threshold* thr_dev, int32_t first_variant,
                                           int32_t n_variants, uint32_t* const* out_nz, uint32_t* const* in_nz,
                                           void* stream) {
    Range nvtx_range("dnns: step 3, portfolio");
    if (!p || !thr_dev || !out_nz || !in_nz || n_variants < 1 || n_variants > kPortfolioMax || first_variant < 0 ||
        first_variant + n_variants > p->last_n_k)
        return DNNS_ERR_INVALID_ARG;
    for (int v = 0; v < n_variants; ++v) {
        if (!out_nz[v] || !in_nz[v]) return DNNS_ERR_INVALID_ARG;
        for (int u = 0; u < v; ++u)  // every variant writes flags of its own
            if (out_nz[u] == out_nz[v] || in_nz[u] == in_nz[v]) return DNNS_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    ProfileScope profile_scope(p);
    const int n2 = launch_extrema_flags(p->tb, reinterpret_cast<uint32_t*>(p->ws + p->map.rowmax),
                                        reinterpret_cast<uint32_t*>(p->ws + p->map.colmax), thr_dev, p->tws.split,
                                        first_variant, n_variants, out_nz, in_nz, st);
    if (n2 < 0) return DNNS_ERR_CUDA;
    const int n1 = 0;
    p->launches += n1 + n2;
    return DNNS_OK;
}

dnns_status dnns_propagate_keep(dnns_plan* p, const uint32_t* out_nz, const uint32_t* in_nz, uint32_t policy,
                                int32_t min_keep, uint32_t* keep_bits, int32_t* keep_idx, int32_t* keep_count,
                                uint64_t* stats, void* stream) {
    Range nvtx_range("dnns: step 4 keep sets");
    if (!p || !out_nz || !in_nz || !keep_bits || !keep_idx || !keep_count) return DNNS_ERR_INVALID_ARG;
    if (policy & ~(uint32_t)(DNNS_RULE_PRODUCER | DNNS_RULE_CONSUMER | DNNS_SHIFT_STRICT)) return DNNS_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (stats && cudaMemsetAsync(stats, 0, 32, st) != cudaSuccess) return DNNS_ERR_CUDA;
    ProfileScope profile_scope(p);
    const int n = launch_propagate(p->tb, out_nz, in_nz, policy, min_keep, keep_bits, keep_idx, keep_count, stats, st);
    if (n < 0) return DNNS_ERR_CUDA;
    const int32_t* kc[1] = {keep_count};
    const int nl = prepare_layouts(p, kc, 1, st);  // the rebuild's layout for these counts, while they are hot
    if (nl < 0) return DNNS_ERR_CUDA;
    p->launches += n + nl;
    return DNNS_OK;
}

dnns_status dnns_propagate_keep_multi(dnns_plan* p, int32_t n_variants, const uint32_t* const* out_nz,
                                      const uint32_t* const* in_nz, uint32_t policy, int32_t min_keep,
                                      uint32_t* const* keep_bits, int32_t* const* keep_idx, int32_t* const* keep_count,
                                      uint64_t* stats, void* stream) {
    Range nvtx_range("dnns: step 4, several variants");
    if (!p || !out_nz || !in_nz || !keep_bits || !keep_idx || !keep_count || n_variants < 1 || n_variants > kPortfolioMax)
        return DNNS_ERR_INVALID_ARG;
    if (policy & ~(uint32_t)(DNNS_RULE_PRODUCER | DNNS_RULE_CONSUMER | DNNS_SHIFT_STRICT)) return DNNS_ERR_INVALID_ARG;
    for (int v = 0; v < n_variants; ++v) {
        if (!out_nz[v] || !in_nz[v] || !keep_bits[v] || !keep_idx[v] || !keep_count[v]) return DNNS_ERR_INVALID_ARG;
        for (int u = 0; u < v; ++u)  // every variant writes buffers of its own
            if (keep_bits[u] == keep_bits[v] || keep_idx[u] == keep_idx[v] || keep_count[u] == keep_count[v])
                return DNNS_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // (the statistics are cleared by the kernel that prepares their bit words, ahead of the propagation)
    ProfileScope profile_scope(p);
    const int n = launch_propagate_multi(p->tb, n_variants, out_nz, in_nz, policy, min_keep, keep_bits, keep_idx, keep_count,
                                         stats, st);
    if (n < 0) return DNNS_ERR_CUDA;
    const int nl = prepare_layouts(p, keep_count, n_variants, st);
    if (nl < 0) return DNNS_ERR_CUDA;
    p->launches += n + nl;
    return DNNS_OK;
}

dnns_status dnns_propagate_keep_cascade(dnns_plan* p, const uint32_t* nz_map, uint32_t policy, int32_t min_keep,
                                        int32_t max_passes, uint32_t* keep_bits, int32_t* keep_idx, int32_t* keep_count,
                                        uint64_t* stats, void* stream) {
    Range nvtx_range("dnns: step 4 to a fixed point");
    if (!p || !nz_map || !keep_bits || !keep_idx || !keep_count) return DNNS_ERR_INVALID_ARG;
    if (policy & ~(uint32_t)(DNNS_RULE_PRODUCER | DNNS_RULE_CONSUMER | DNNS_SHIFT_STRICT)) return DNNS_ERR_INVALID_ARG;
    if (max_passes < 1 || max_passes > kMaxCascadePasses) return DNNS_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (stats && cudaMemsetAsync(stats, 0, 32, st) != cudaSuccess) return DNNS_ERR_CUDA;
    const dnns_layout& L = p->layout;
    ProfileScope profile_scope(p);
    const int n = launch_propagate_cascade(p->tb, p->kws, nz_map, policy, min_keep, max_passes, keep_bits, keep_idx,
                                           keep_count, stats, (uint32_t)L.keep_words,
                                           (uint32_t)(L.out_nz_words + L.in_nz_words), p->n_sm, st);
    if (n < 0) return DNNS_ERR_CUDA;
    const int32_t* kc[1] = {keep_count};
    const int nl = prepare_layouts(p, kc, 1, st);
    if (nl < 0) return DNNS_ERR_CUDA;
    p->launches += n + nl;
    return DNNS_OK;
}

// The rebuild of n variants in one launch.  masked_arenas NULL: from the dense model, masking on the way (thr_dev set).
static dnns_status rebuild_variants(dnns_plan* p, int n, const void* const* masked_arenas, const dnns_threshold* thr_dev,
                                    int32_t first_variant, const int32_t* const* keep_idx, const int32_t* const* keep_count,
                                    void* const* dst_arena, size_t dst_bytes, uint64_t* const* dst_offsets,
                                    int32_t* const* dst_shapes, void* stream) {
    for (int i = 0; i < n; ++i) {
        if (!keep_idx[i] || !keep_count[i] || !dst_arena[i] || !dst_offsets[i] || !dst_shapes[i]) return DNNS_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(dst_arena[i]) & (kAlign - 1)) return DNNS_ERR_INVALID_ARG;
        if (masked_arenas && masked_arenas[i] && (reinterpret_cast<uintptr_t>(masked_arenas[i]) & 15)) return DNNS_ERR_INVALID_ARG;
        for (int j = 0; j < i; ++j)  // every variant has outputs of its own
            if (dst_arena[j] == dst_arena[i] || dst_offsets[j] == dst_offsets[i] || dst_shapes[j] == dst_shapes[i] ||
                keep_count[j] == keep_count[i])
                return DNNS_ERR_INVALID_ARG;
    }
    ProfileScope profile_scope(p);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // counts that no dnns_propagate_keep* call of this plan wrote are laid out now
    std::vector<const int32_t*> missing;
    for (int i = 0; i < n; ++i)
        if (find_layout(p, keep_count[i]) < 0) missing.push_back(keep_count[i]);
    int nl = 0;
    if (!missing.empty() && (nl = prepare_layouts(p, missing.data(), (int)missing.size(), st)) < 0) return DNNS_ERR_CUDA;
    GatherBatch gb{};
    gb.n = n;
    for (int i = 0; i < n; ++i) {
        const int slot = find_layout(p, keep_count[i]);
        if (slot < 0) return DNNS_ERR_INVALID_ARG;  // more distinct count arrays in one call than layouts can be held
        GatherJob& job = gb.job[i];
        job.lay = layout_slot(p, (uint32_t)slot);
        job.src_arena = masked_arenas ? static_cast<const char*>(masked_arenas[i]) : nullptr;
        job.keep_idx = keep_idx[i];
        job.dst_arena = static_cast<char*>(dst_arena[i]);
        job.dst_bytes = dst_bytes;
        job.dst_offsets = dst_offsets[i];
        job.dst_shapes = dst_shapes[i];
        job.variant = first_variant + i;
    }
    const int k = launch_compact(p->tb, gb, p->n_sm, st, thr_dev, thr_dev ? p->tws.split : nullptr);
    if (k < 0) return DNNS_ERR_CUDA;
    p->launches += k + nl;
    return DNNS_OK;
}

dnns_status dnns_compact(dnns_plan* p, const void* masked_arena, const int32_t* keep_idx, const int32_t* keep_count,
                         void* dst_arena, size_t dst_bytes, uint64_t* dst_offsets_dev, int32_t* dst_shapes_dev,
                         void* stream) {
    Range nvtx_range("dnns: step 5 rebuild");
    if (!p || !keep_idx || !keep_count || !dst_arena || !dst_offsets_dev || !dst_shapes_dev) return DNNS_ERR_INVALID_ARG;
    const void* arenas[1] = {masked_arena};
    return rebuild_variants(p, 1, arenas, nullptr, 0, &keep_idx, &keep_count, &dst_arena, dst_bytes, &dst_offsets_dev,
                            &dst_shapes_dev, stream);
}

dnns_status dnns_compact_masked(dnns_plan* p, const dnns_threshold* thr_dev, int32_t variant,
                                const int32_t* keep_idx, const int32_t* keep_count, void* dst_arena, size_t dst_bytes,
                                uint64_t* dst_offsets_dev, int32_t* dst_shapes_dev, void* stream) {
    Range nvtx_range("dnns: steps 2+5 rebuild from the dense model");
    if (!p || !thr_dev || !keep_idx || !keep_count || !dst_arena || !dst_offsets_dev || !dst_shapes_dev ||
        variant < 0 || variant >= p->last_n_k)
        return DNNS_ERR_INVALID_ARG;
    return rebuild_variants(p, 1, nullptr, thr_dev, variant, &keep_idx, &keep_count, &dst_arena, dst_bytes,
                            &dst_offsets_dev, &dst_shapes_dev, stream);
}

dnns_status dnns_compact_masked_multi(dnns_plan* p, const dnns_threshold* thr_dev, int32_t first_variant,
                                      int32_t n_variants, const int32_t* const* keep_idx,
                                      const int32_t* const* keep_count, void* const* dst_arenas, size_t dst_bytes,
                                      uint64_t* const* dst_offsets_dev, int32_t* const* dst_shapes_dev, void* stream) {
    Range nvtx_range("dnns: steps 2+5 rebuild from the dense model, several variants");
    if (!p || !thr_dev || !keep_idx || !keep_count || !dst_arenas || !dst_offsets_dev || !dst_shapes_dev || n_variants < 1 ||
        n_variants > kPortfolioMax || first_variant < 0 || first_variant + n_variants > p->last_n_k)
        return DNNS_ERR_INVALID_ARG;
    return rebuild_variants(p, n_variants, nullptr, thr_dev, first_variant, keep_idx, keep_count, dst_arenas, dst_bytes,
                            dst_offsets_dev, dst_shapes_dev, stream);
}

dnns_status dnns_fold_batchnorm(dnns_plan* p, void* dst_arena, const uint64_t* dst_offsets_dev,
                                const int32_t* dst_shapes_dev, void* stream) {
    Range nvtx_range("dnns: conv+BN fusion");
    if (!p || !dst_arena || !dst_offsets_dev || !dst_shapes_dev) return DNNS_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(dst_arena) & (kAlign - 1)) return DNNS_ERR_INVALID_ARG;
    ProfileScope profile_scope(p);
    const int n = launch_fold(p->tb, dst_arena, dst_offsets_dev, dst_shapes_dev, reinterpret_cast<uint32_t*>(p->ws + p->map.fold_count),
                              reinterpret_cast<FoldJob*>(p->ws + p->map.fold_jobs), p->n_sm, static_cast<cudaStream_t>(stream));
    if (n < 0) return DNNS_ERR_CUDA;
    p->launches += n;
    return DNNS_OK;
}

dnns_status dnns_plan_profile(dnns_plan* p, int32_t enable) {
    if (!p) return DNNS_ERR_INVALID_ARG;
    if (enable) {
        if (cudaDeviceSynchronize() != cudaSuccess) return DNNS_ERR_CUDA;
        p->timer.clear();
    }
    p->timer.on = enable != 0;
    return DNNS_OK;
}

dnns_status dnns_plan_tie_sweep(dnns_plan* p, int32_t* swept) {
    if (!p || !swept) return DNNS_ERR_INVALID_ARG;
    uint32_t any_need = 0, fallback = 0;
    if (cudaDeviceSynchronize() != cudaSuccess ||
        cudaMemcpy(&any_need, p->tws.any_need, sizeof(any_need), cudaMemcpyDeviceToHost) != cudaSuccess ||
        cudaMemcpy(&fallback, p->tws.tie_fallback, sizeof(fallback), cudaMemcpyDeviceToHost) != cudaSuccess)
        return DNNS_ERR_CUDA;
    const bool lists = p->tws.tie_list != nullptr;
    *swept = any_need && (!lists || fallback || p->tie_tables_valid) ? 1 : 0;
    return DNNS_OK;
}

dnns_status dnns_plan_profile_read(dnns_plan* p, const char* kernel, double* total_ms, uint64_t* launches) {
    if (!p || !kernel || !total_ms || !launches) return DNNS_ERR_INVALID_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return DNNS_ERR_CUDA;
    const size_t n = strlen(kernel);
    double sum = 0;
    uint64_t cnt = 0;
    for (const KernelTimer::Rec& r : p->timer.recs) {
        if (strncmp(r.name, kernel, n) != 0) continue;
        float ms = 0;
        if (cudaEventElapsedTime(&ms, r.start, r.stop) != cudaSuccess) return DNNS_ERR_CUDA;
        sum += ms;
        ++cnt;
    }
    *total_ms = sum;
    *launches = cnt;
    return DNNS_OK;
}

dnns_status dnns_last_device_status(dnns_plan* p, void* stream) {
    if (!p) return DNNS_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t s = 0;
    if (cudaMemcpyAsync(&s, p->tb.status, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemsetAsync(p->tb.status, 0, 4, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess)
        return DNNS_ERR_CUDA;
    return static_cast<dnns_status>(s);
}

}  // extern "C"
