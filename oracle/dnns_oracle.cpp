// CPU oracle for the sparse-to-pruned conversion path (TEST INFRASTRUCTURE).
//
// This file is test infrastructure, not part of the product: it is only used
// by the test-suite, by the smoke check and by the benchmark's CPU-baseline leg.
// It is a plain, single-threaded, deliberately slow restatement of what the
// method defines, written from the paper and sharing nothing with the CUDA
// library (no header, no helper, no table).  Every function is the textbook
// definition of its step: a full sort for the threshold, one walk for the mask,
// triple loops for the zero-structure flags, per-channel loops for the plan and
// nested loops for the rebuild.
//
// Steps and the passages they restate:
//   O1 orc_threshold       - magnitude ranking: the k weights of least magnitude
//                            are the ones to mask (Section III-C; Section IV-B,
//                            "compression ratio C": C-1 of every C weights zero).
//   O2 orc_apply_mask      - masking sets the selected weights to zero; the sparse
//                            model keeps its size (Section III-C).
//   O3 orc_zero_structures - Module 2 (Sparsity Analyser): all-zero 2-D kernels,
//                            then channels all of whose kernels are zero.
//   O4 orc_propagate_keep  - Module 3 (Prune Planner, Algorithm 1): C_out of a
//                            layer = its zero channels, C_in = those of the layer
//                            before it; generalised from a chain to channel groups
//                            (see the comment on the function).
//   O5 orc_compact         - Module 4 (Model Pruner, Algorithm 2): rebuild each
//                            layer with |C'_in| x |C'_out| channels and move the
//                            surviving out-channels, biases and in-channels over.
//   O8 orc_propagate_keep_cascade - Algorithm 1 applied again and again: once channels
//                            are gone, filters that only read removed channels (and input
//                            columns only read by removed filters) are zero channels too.
//   O7 orc_fold_batchnorm  - Module 1 (Model Pre-Processor): fuse each convolution
//                            with the batch normalisation that follows it.
//
// Parity against numbers printed in the paper: unpinned (every number the paper
// prints depends on trained weights).  The functions are pinned instead by brute
// force, closed forms, hand-built cases and invariants in the CPU test-suite.
//
// Layout: weights are OIHW, contiguous; filter o is I*KH*KW consecutive elements,
// the 2-D kernel (o,i) is KH*KW consecutive elements.  A fully-connected layer is
// [O][I] with KH=KW=1 and I = C_in*in_spatial, the columns of input channel c
// being c*in_spatial .. (c+1)*in_spatial-1.  Bit sets are uint32 words, bit b of
// the set stored at word b/32, position b%32.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

extern "C" {

enum { ORC_F32 = 0, ORC_BF16 = 1 };
enum { ORC_SCOPE_GLOBAL = 0, ORC_SCOPE_PER_TENSOR = 1 };
enum { ORC_RULE_PRODUCER = 1, ORC_RULE_CONSUMER = 2, ORC_SHIFT_STRICT = 4 };
enum { ORC_GROUP_FROZEN = 1 };

typedef struct {
    void* data;
    int32_t dtype;
    int32_t O, I, KH, KW;
    int32_t in_spatial;
    int32_t prunable;
    int32_t out_group, in_group;
    float* bias;  // nullable, length O
} orc_tensor;

typedef struct {
    float *gamma, *beta, *mean, *var;
    int32_t C;
    int32_t tensor;  // the conv this BN follows
    float eps;
} orc_bn;

typedef struct {
    int32_t C;
    uint32_t flags;
} orc_group;

typedef struct {
    int32_t n_tensors;
    const orc_tensor* tensors;
    int32_t n_bn;
    const orc_bn* bns;
    int32_t n_groups;
    const orc_group* groups;
} orc_model;

typedef struct {
    uint32_t tau_bits;  // magnitude bit pattern of the k-th smallest weight
    uint32_t pad;
    uint64_t n_below;   // weights with magnitude strictly below tau
    uint64_t n_tie;     // k - n_below: how many weights equal to tau are masked
    uint64_t n_equal;   // weights with magnitude exactly tau
} orc_threshold_rec;

}  // extern "C"

namespace {

inline int64_t numel(const orc_tensor& t) { return (int64_t)t.O * t.I * t.KH * t.KW; }

// Magnitude key of element e: the stored word with the sign bit cleared.  As an
// unsigned integer it orders finite values by |w|, puts -0 with +0, infinities
// above every finite value and NaNs above those.
inline uint32_t key_of(const orc_tensor& t, int64_t e) {
    if (t.dtype == ORC_F32) {
        uint32_t u;
        std::memcpy(&u, (const char*)t.data + 4 * e, 4);
        return u & 0x7FFFFFFFu;
    }
    uint16_t h;
    std::memcpy(&h, (const char*)t.data + 2 * e, 2);
    return (uint32_t)(h & 0x7FFFu);
}

inline void copy_elem(const orc_tensor& s, int64_t es, const orc_tensor& d, int64_t ed) {
    const int b = s.dtype == ORC_F32 ? 4 : 2;
    std::memcpy((char*)d.data + b * ed, (const char*)s.data + b * es, b);
}

inline void zero_elem(const orc_tensor& d, int64_t e) {
    const int b = d.dtype == ORC_F32 ? 4 : 2;
    std::memset((char*)d.data + b * e, 0, b);
}

// Ranking segments: the whole model, or one per prunable tensor.
std::vector<std::vector<int>> segments_of(const orc_model* m, int scope) {
    std::vector<std::vector<int>> segs;
    if (scope == ORC_SCOPE_GLOBAL) segs.emplace_back();
    for (int t = 0; t < m->n_tensors; ++t) {
        if (!m->tensors[t].prunable) continue;
        if (scope == ORC_SCOPE_GLOBAL) segs[0].push_back(t);
        else segs.push_back({t});
    }
    return segs;
}

inline bool get_bit(const uint32_t* w, int64_t b) { return (w[b >> 5] >> (b & 31)) & 1u; }
inline void set_bit(uint32_t* w, int64_t b) { w[b >> 5] |= 1u << (b & 31); }

}  // namespace

extern "C" {

int orc_num_segments(const orc_model* m, int scope) { return (int)segments_of(m, scope).size(); }

// O1.  For each segment and each k: sort the magnitude keys of the segment (in
// global index order: tensors in descriptor order, row-major inside each), take
// the k-th smallest as tau, count the keys below and equal to it.
// k[v*S + s] is the count for variant v, segment s; rec likewise.  k == 0 gives
// an all-zero record.  Returns 0, or 1 when some k exceeds its segment's size.
int orc_threshold(const orc_model* m, int scope, const uint64_t* k, int n_k, orc_threshold_rec* rec) {
    auto segs = segments_of(m, scope);
    const int S = (int)segs.size();
    for (int s = 0; s < S; ++s) {
        std::vector<uint32_t> keys;
        for (int t : segs[s]) {
            const orc_tensor& T = m->tensors[t];
            for (int64_t e = 0; e < numel(T); ++e) keys.push_back(key_of(T, e));
        }
        std::sort(keys.begin(), keys.end());
        for (int v = 0; v < n_k; ++v) {
            const uint64_t kk = k[(size_t)v * S + s];
            orc_threshold_rec& r = rec[(size_t)v * S + s];
            r.tau_bits = 0; r.pad = 0; r.n_below = 0; r.n_tie = 0; r.n_equal = 0;
            if (kk == 0) continue;
            if (kk > keys.size()) return 1;
            const uint32_t tau = keys[kk - 1];
            uint64_t below = 0, equal = 0;
            for (uint32_t x : keys) { below += x < tau; equal += x == tau; }
            r.tau_bits = tau;
            r.n_below = below;
            r.n_tie = kk - below;
            r.n_equal = equal;
        }
    }
    return 0;
}

// O2.  Walk each segment in global index order.  A weight is masked when its key
// is below tau, or equals tau while fewer than n_tie ties have been seen so far.
// Masked weights become +0 (all bits clear); kept weights are copied bit for bit.
// The all-zero record (k = 0) masks nothing.  Tensors that are not prunable are
// copied.  rec holds one record per segment.  mask_bits[t]
// (nullable, per tensor, numel bits) gets 1 for kept elements; for tensors that
// are not prunable every bit is 1.
void orc_apply_mask(const orc_model* src, const orc_model* dst, int scope, const orc_threshold_rec* rec,
                    uint32_t* const* mask_bits) {
    auto segs = segments_of(src, scope);
    for (int t = 0; t < src->n_tensors; ++t) {
        const orc_tensor& T = src->tensors[t];
        if (mask_bits && mask_bits[t]) std::memset(mask_bits[t], 0, (size_t)((numel(T) + 31) / 32) * 4);
        if (T.prunable) continue;
        for (int64_t e = 0; e < numel(T); ++e) {
            copy_elem(T, e, dst->tensors[t], e);
            if (mask_bits && mask_bits[t]) set_bit(mask_bits[t], e);
        }
    }
    for (size_t s = 0; s < segs.size(); ++s) {
        const orc_threshold_rec& r = rec[s];
        uint64_t seen_ties = 0;
        for (int t : segs[s]) {
            const orc_tensor& T = src->tensors[t];
            for (int64_t e = 0; e < numel(T); ++e) {
                const uint32_t key = key_of(T, e);
                bool prune = false;
                if (key < r.tau_bits) prune = true;
                else if (key == r.tau_bits) { prune = seen_ties < r.n_tie; ++seen_ties; }
                if (prune) zero_elem(dst->tensors[t], e);
                else {
                    copy_elem(T, e, dst->tensors[t], e);
                    if (mask_bits && mask_bits[t]) set_bit(mask_bits[t], e);
                }
            }
        }
    }
}

// O3.  An element is zero when its magnitude key is 0.  NZ[o][i] says whether the
// 2-D kernel (o,i) has a non-zero element; out_nz[o] ORs NZ over i (filter o is
// not all zero), in_nz[i] ORs NZ over o (some filter reads input column i).
// nz_map[t] (nullable): O*I bits, bit o*I+i.  out_nz[t]: O bits.  in_nz[t]: I bits.
void orc_zero_structures(const orc_model* m, uint32_t* const* nz_map, uint32_t* const* out_nz,
                         uint32_t* const* in_nz) {
    for (int t = 0; t < m->n_tensors; ++t) {
        const orc_tensor& T = m->tensors[t];
        const int64_t kk = (int64_t)T.KH * T.KW;
        if (nz_map && nz_map[t]) std::memset(nz_map[t], 0, (size_t)(((int64_t)T.O * T.I + 31) / 32) * 4);
        std::memset(out_nz[t], 0, (size_t)((T.O + 31) / 32) * 4);
        std::memset(in_nz[t], 0, (size_t)((T.I + 31) / 32) * 4);
        for (int64_t o = 0; o < T.O; ++o)
            for (int64_t i = 0; i < T.I; ++i) {
                bool nz = false;
                for (int64_t r = 0; r < kk; ++r)
                    if (key_of(T, (o * T.I + i) * kk + r) != 0) nz = true;
                if (nz) {
                    if (nz_map && nz_map[t]) set_bit(nz_map[t], o * T.I + i);
                    set_bit(out_nz[t], o);
                    set_bit(in_nz[t], i);
                }
            }
    }
}

// O4.  Algorithm 1 gives every conv layer L_n the pair (C_in, C_out): C_out are
// the zero channels (all-zero filters) of L_n, C_in those of L_{n-1}.  In a chain
// the out-axis of L_{n-1} and the in-axis of L_n are the same set of channels; a
// channel group is that set, and with residual adds a group has several
// producers (out-axes) and several consumers (in-axes).  Per channel j of group g:
//   prod_dead  - g has producers and filter j of every producer is all zero
//                (Algorithm 1's rule, needing *all* tensors that write channel j);
//   cons_dead  - g has consumers and no consumer has a non-zero weight in the
//                columns of channel j;
//   shift_zero(p, j) - the constant that producer p's zero filter still emits
//                after its BatchNorm, beta + gamma*(bias-mean)/sqrt(var+eps), is
//                zero, tested structurally: beta == 0 and (gamma == 0 or
//                mean == bias); without BN: bias == 0 (absent bias counts as 0);
//   remove     = (RULE_PRODUCER and prod_dead and shift_ok) or (RULE_CONSUMER and cons_dead),
//                shift_ok being true unless SHIFT_STRICT, which wants shift_zero for every producer.
// Frozen groups keep everything.  If fewer than min(min_keep, C) channels stay,
// removed channels are taken back in ascending order.  Single pass: nothing is
// re-evaluated after removal.
// Outputs per group: keep_bits (C bits), keep_idx (kept channels ascending, room for C),
// keep_count.  stats (nullable, 4 words): [0] removed (producer, channel) pairs whose
// constant is dropped although somebody still reads it (prod_dead, not cons_dead, not
// shift_zero): while this is 0 the rebuilt model computes exactly what the sparse model
// does; [1] channels removed, [2] channels taken back by min_keep, [3] 0.
void orc_propagate_keep(const orc_model* m, uint32_t* const* out_nz, uint32_t* const* in_nz, uint32_t policy,
                        int32_t min_keep, uint32_t* const* keep_bits, int32_t* const* keep_idx,
                        int32_t* keep_count, uint64_t* stats) {
    if (stats) stats[0] = stats[1] = stats[2] = stats[3] = 0;
    for (int g = 0; g < m->n_groups; ++g) {
        const int C = m->groups[g].C;
        std::vector<int> producers, consumers;
        for (int t = 0; t < m->n_tensors; ++t) {
            if (m->tensors[t].out_group == g) producers.push_back(t);
            if (m->tensors[t].in_group == g) consumers.push_back(t);
        }
        auto shift_zero = [&](int p, int j) {
            const orc_tensor& T = m->tensors[p];
            const float bias = T.bias ? T.bias[j] : 0.0f;
            for (int b = 0; b < m->n_bn; ++b)
                if (m->bns[b].tensor == p) {
                    const orc_bn& B = m->bns[b];
                    return B.beta[j] == 0.0f && (B.gamma[j] == 0.0f || B.mean[j] == bias);
                }
            return bias == 0.0f;
        };
        std::vector<char> remove(C, 0), prod_dead_v(C, 0), cons_dead_v(C, 0);
        for (int j = 0; j < C; ++j) {
            bool prod_dead = !producers.empty();
            for (int p : producers)
                if (get_bit(out_nz[p], j)) prod_dead = false;
            bool cons_dead = !consumers.empty();
            for (int q : consumers) {
                const int S = m->tensors[q].in_spatial;
                for (int s = 0; s < S; ++s)
                    if (get_bit(in_nz[q], (int64_t)j * S + s)) cons_dead = false;
            }
            bool shift_ok = true;
            if (policy & ORC_SHIFT_STRICT)
                for (int p : producers)
                    if (!shift_zero(p, j)) shift_ok = false;
            prod_dead_v[j] = prod_dead;
            cons_dead_v[j] = cons_dead;
            remove[j] = ((policy & ORC_RULE_PRODUCER) && prod_dead && shift_ok) ||
                        ((policy & ORC_RULE_CONSUMER) && cons_dead);
            if (m->groups[g].flags & ORC_GROUP_FROZEN) remove[j] = 0;
        }
        int kept = 0;
        for (int j = 0; j < C; ++j) kept += !remove[j];
        const int floor_keep = std::min<int>(std::max<int>(min_keep, 0), C);
        for (int j = 0; j < C && kept < floor_keep; ++j)
            if (remove[j]) { remove[j] = 0; ++kept; if (stats) ++stats[2]; }
        std::memset(keep_bits[g], 0, (size_t)((C + 31) / 32) * 4);
        int n = 0;
        for (int j = 0; j < C; ++j) {
            if (!remove[j]) { set_bit(keep_bits[g], j); keep_idx[g][n++] = j; continue; }
            if (stats) {
                ++stats[1];
                if (prod_dead_v[j] && !cons_dead_v[j])
                    for (int p : producers)
                        if (!shift_zero(p, j)) ++stats[0];
            }
        }
        keep_count[g] = n;
    }
}

// O5.  Algorithm 2: the rebuilt layer has O' = |keep(out_group)| filters and
// C'_in = |keep(in_group)| input channels; element (a, c, s, y, x) of the new
// layer is element (keep_out[a], keep_in[c], s, y, x) of the old one, keep lists
// ascending so the surviving channels stay in their original order.  BN vectors
// and biases follow the out-axis of their tensor.  dst_w[t] needs room for
// O'*C'_in*in_spatial*KH*KW elements; dst_bn[4*b+{0,1,2,3}] = gamma, beta, mean,
// var of BN b (room for C'); dst_bias[t] nullable where the tensor has no bias.
// shapes[2*t], shapes[2*t+1] = O', I' (I' = C'_in*in_spatial).
void orc_compact(const orc_model* m, int32_t* const* keep_idx, const int32_t* keep_count, void* const* dst_w,
                 float* const* dst_bn, float* const* dst_bias, int32_t* shapes) {
    for (int t = 0; t < m->n_tensors; ++t) {
        const orc_tensor& T = m->tensors[t];
        const int32_t* ko = keep_idx[T.out_group];
        const int32_t* ki = keep_idx[T.in_group];
        const int On = keep_count[T.out_group], Cn = keep_count[T.in_group];
        const int64_t blk = (int64_t)T.in_spatial * T.KH * T.KW;  // elements per (filter, input channel)
        const int64_t C_in = T.I / T.in_spatial;
        orc_tensor D = T;
        D.data = dst_w[t];
        for (int64_t a = 0; a < On; ++a)
            for (int64_t c = 0; c < Cn; ++c)
                for (int64_t r = 0; r < blk; ++r)
                    copy_elem(T, ((int64_t)ko[a] * C_in + ki[c]) * blk + r, D, (a * Cn + c) * blk + r);
        shapes[2 * t] = On;
        shapes[2 * t + 1] = Cn * T.in_spatial;
        if (T.bias && dst_bias && dst_bias[t])
            for (int a = 0; a < On; ++a) dst_bias[t][a] = T.bias[ko[a]];
    }
    for (int b = 0; b < m->n_bn; ++b) {
        const orc_bn& B = m->bns[b];
        const int g = m->tensors[B.tensor].out_group;
        const float* src[4] = {B.gamma, B.beta, B.mean, B.var};
        for (int v = 0; v < 4; ++v)
            for (int a = 0; a < keep_count[g]; ++a) dst_bn[4 * b + v][a] = src[v][keep_idx[g][a]];
    }
}

// O8.  Fixed point of the plan.  Algorithm 1 looks at the zero channels once; but a filter whose
// only non-zero 2-D kernels sit in input channels that are being removed is as good as zero, and
// an input column that only removed filters read is as good as unread.  Pass p evaluates the rule of
// O4 for every channel with "zero" judged on the kernel maps restricted to what pass p-1 kept:
//   prod_dead  - every producer's filter j has no non-zero kernel in a kept input channel,
//   cons_dead  - no kept filter of any consumer has a non-zero kernel in the columns of channel j,
// all channels judged against the same previous sets (simultaneous update), removed channels stay
// removed.  Passes stop when nothing changes or after max_passes.  Pass 1 is O4's single pass.
// min_keep is applied once, at the end.  nz_map[t]: O*I bits as written by orc_zero_structures.
// stats: [0] as in O4, judged in the last pass, [1] channels removed, [2] taken back by min_keep,
// [3] passes that removed something.
void orc_propagate_keep_cascade(const orc_model* m, uint32_t* const* nz_map, uint32_t policy, int32_t min_keep,
                                int32_t max_passes, uint32_t* const* keep_bits, int32_t* const* keep_idx,
                                int32_t* keep_count, uint64_t* stats) {
    const int G = m->n_groups;
    std::vector<std::vector<char>> removed(G), lost(G);
    for (int g = 0; g < G; ++g) removed[g].assign(m->groups[g].C, 0), lost[g].assign(m->groups[g].C, 0);
    auto shift_zero = [&](int p, int j) {
        const orc_tensor& T = m->tensors[p];
        const float bias = T.bias ? T.bias[j] : 0.0f;
        for (int b = 0; b < m->n_bn; ++b)
            if (m->bns[b].tensor == p) {
                const orc_bn& B = m->bns[b];
                return B.beta[j] == 0.0f && (B.gamma[j] == 0.0f || B.mean[j] == bias);
            }
        return bias == 0.0f;
    };
    uint64_t passes = 0;
    for (int pass = 0; pass < max_passes; ++pass) {
        std::vector<std::vector<char>> next = removed;
        bool changed = false;
        for (int g = 0; g < G; ++g) {
            if (m->groups[g].flags & ORC_GROUP_FROZEN) continue;
            std::vector<int> producers, consumers;
            for (int t = 0; t < m->n_tensors; ++t) {
                if (m->tensors[t].out_group == g) producers.push_back(t);
                if (m->tensors[t].in_group == g) consumers.push_back(t);
            }
            for (int j = 0; j < m->groups[g].C; ++j) {
                bool prod_dead = !producers.empty();
                for (int p : producers) {
                    const orc_tensor& T = m->tensors[p];
                    for (int i = 0; i < T.I; ++i)
                        if (!removed[T.in_group][i / T.in_spatial] && get_bit(nz_map[p], (int64_t)j * T.I + i)) prod_dead = false;
                }
                bool cons_dead = !consumers.empty();
                for (int q : consumers) {
                    const orc_tensor& T = m->tensors[q];
                    for (int o = 0; o < T.O; ++o)
                        for (int s2 = 0; s2 < T.in_spatial; ++s2)
                            if (!removed[T.out_group][o] && get_bit(nz_map[q], (int64_t)o * T.I + (int64_t)j * T.in_spatial + s2))
                                cons_dead = false;
                }
                bool shift_ok = true;
                if (policy & ORC_SHIFT_STRICT)
                    for (int p : producers)
                        if (!shift_zero(p, j)) shift_ok = false;
                const bool rule = ((policy & ORC_RULE_PRODUCER) && prod_dead && shift_ok) ||
                                  ((policy & ORC_RULE_CONSUMER) && cons_dead);
                lost[g][j] = prod_dead && !cons_dead;
                if (rule && !removed[g][j]) next[g][j] = 1, changed = true;
            }
        }
        removed.swap(next);
        if (!changed) break;
        ++passes;
    }
    if (stats) stats[0] = stats[1] = stats[2] = 0, stats[3] = passes;
    for (int g = 0; g < G; ++g) {
        const int C = m->groups[g].C;
        int kept = 0;
        for (int j = 0; j < C; ++j) kept += !removed[g][j];
        const int floor_keep = std::min<int>(std::max<int>(min_keep, 0), C);
        for (int j = 0; j < C && kept < floor_keep; ++j)
            if (removed[g][j]) { removed[g][j] = 0; ++kept; if (stats) ++stats[2]; }
        std::memset(keep_bits[g], 0, (size_t)((C + 31) / 32) * 4);
        int n = 0;
        for (int j = 0; j < C; ++j) {
            if (!removed[g][j]) { set_bit(keep_bits[g], j); keep_idx[g][n++] = j; continue; }
            if (stats) {
                ++stats[1];
                if (lost[g][j])
                    for (int t = 0; t < m->n_tensors; ++t)
                        if (m->tensors[t].out_group == g && !shift_zero(t, j)) ++stats[0];
            }
        }
        keep_count[g] = n;
    }
}

// O7.  Module 1 fuses a convolution with the batch normalisation behind it.  BN maps the
// conv output y_o (plus the conv bias) to gamma_o * (y_o + bias_o - mean_o) / sqrt(var_o + eps) +
// beta_o, which is a convolution again with
//   scale_o = gamma_o / sqrt(var_o + eps),  W_f[o] = W[o] * scale_o,
//   b_f[o]  = beta_o + (bias_o - mean_o) * scale_o        (bias_o = 0 without a bias),
// evaluated here in double precision.  folded_w[t] (numel doubles) is filled for tensors that
// have a BN and may be null for the others; scale[b], folded_bias[b] hold C doubles per BN.
void orc_fold_batchnorm(const orc_model* m, double* const* folded_w, double* const* scale, double* const* folded_bias) {
    for (int b = 0; b < m->n_bn; ++b) {
        const orc_bn& B = m->bns[b];
        const orc_tensor& T = m->tensors[B.tensor];
        const int64_t row = (int64_t)T.I * T.KH * T.KW;
        for (int64_t o = 0; o < T.O; ++o) {
            const double s = (double)B.gamma[o] / std::sqrt((double)B.var[o] + (double)B.eps);
            const double bias = T.bias ? (double)T.bias[o] : 0.0;
            scale[b][o] = s;
            folded_bias[b][o] = (double)B.beta[o] + (bias - (double)B.mean[o]) * s;
            for (int64_t r = 0; r < row; ++r) {
                double w;
                if (T.dtype == ORC_F32) {
                    float f;
                    std::memcpy(&f, (const char*)T.data + 4 * (o * row + r), 4);
                    w = f;
                } else {
                    uint16_t h;
                    std::memcpy(&h, (const char*)T.data + 2 * (o * row + r), 2);
                    const uint32_t u = (uint32_t)h << 16;
                    float f;
                    std::memcpy(&f, &u, 4);
                    w = f;
                }
                folded_w[B.tensor][o * row + r] = w * s;
            }
        }
    }
}

}  // extern "C"
