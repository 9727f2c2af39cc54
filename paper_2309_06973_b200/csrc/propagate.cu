// Step 4: keep sets per channel group - Module 3, the Prune Planner (Algorithm 1), for every
// group of the model in one launch.  Algorithm 1 hands layer L_n the zero channels of L_n as
// C_out and those of L_{n-1} as C_in; the two are one set of channels, a "group", which with
// residual adds has several producers and consumers.  One block per group.  The data are a few
// kilobytes of flag bits, so the launch is latency-bound: the flag words of all producers and
// consumers are fetched as independent loads (one (tensor, word) pair per thread and step) and
// OR-ed in shared memory, instead of walking the tensors channel by channel.
#include "dnns_internal.cuh"

namespace dnns {

namespace {

constexpr int kThreads = 256;
constexpr int kMaxGroupWords = 65536 / 32;
DNNS_BOUNDS_COUNTER  // (checked build: index violations counted in this file)

__device__ __forceinline__ bool get_bit(const uint32_t* w, uint32_t b) { return (w[b >> 5] >> (b & 31)) & 1u; }

// The constant a zero filter of producer p (an index into the producer list) still emits on channel
// j is structurally zero.
__device__ __forceinline__ bool shift_zero(const Tables& tb, int p, int j) {
    const ProducerDesc d = tb.producers[p];
    const float bias = d.bias ? d.bias[j] : 0.0f;
    if (d.beta) return d.beta[j] == 0.0f && (d.gamma[j] == 0.0f || d.mean[j] == bias);
    return bias == 0.0f;
}

// The rule of Algorithm 1 for one group: from the flag words of its producers and consumers to the
// words of removed channels (s_rem) and of dead channels that somebody still reads (s_lost).
// Returns the number of removed channels counted by this thread.
__device__ __forceinline__ uint32_t eval_group(const Tables& tb, const GroupDesc& gd, const uint32_t* __restrict__ out_nz,
                                               const uint32_t* __restrict__ in_nz, uint32_t policy, uint32_t* s_prod,
                                               uint32_t* s_cons, uint32_t* s_rem) {
    const int C = gd.C;
    const int n_words = (C + 31) / 32;
    const bool frozen = gd.flags & DNNS_GROUP_FROZEN;
    const int n_prod = gd.prod_end - gd.prod_begin, n_cons = gd.cons_end - gd.cons_begin;
    for (int w = threadIdx.x; w < n_words; w += kThreads) s_prod[w] = s_cons[w] = 0;
    __syncthreads();
    if (!frozen) {
        // One (tensor, word) pair per thread and step, producers first, then consumers: all flag
        // words of the group are requested in one go.  Producers OR their filter flags; consumers OR
        // their input-column flags (with S columns per channel the S bits are folded).
        const int n_pw = n_prod * n_words, n_all = n_pw + n_cons * n_words;
        constexpr int kBatch = 4;  // pairs per thread and round: their loads are all issued before the first one is used
        for (int base = threadIdx.x; base < n_all; base += kThreads * kBatch) {
            uint32_t off[kBatch], x[kBatch];
            int S[kBatch], w[kBatch];
            bool prod[kBatch], ok[kBatch];
#pragma unroll
            for (int b = 0; b < kBatch; ++b) {
                const int it = base + b * kThreads;
                ok[b] = it < n_all;
                prod[b] = it < n_pw;
                off[b] = 0, S[b] = 1, w[b] = 0;
                if (!ok[b]) continue;
                if (prod[b]) {
                    const int p = it / n_words;
                    w[b] = it - p * n_words;
                    off[b] = tb.producers[gd.prod_begin + p].off_outnz;
                } else {
                    const int q = (it - n_pw) / n_words;
                    w[b] = (it - n_pw) - q * n_words;
                    const ConsumerDesc d = tb.consumers[gd.cons_begin + q];
                    off[b] = d.off_innz, S[b] = d.S;
                }
            }
#pragma unroll
            for (int b = 0; b < kBatch; ++b) {
                x[b] = 0;
                if (!ok[b]) continue;
                if (prod[b]) {
                    x[b] = out_nz[off[b] + w[b]];
                } else if (S[b] == 1) {
                    x[b] = in_nz[off[b] + w[b]];
                } else {  // S columns per channel: the S bits of a channel are folded
                    for (int bit = 0; bit < 32 && w[b] * 32 + bit < C; ++bit)
                        for (int sc = 0; sc < S[b]; ++sc)
                            if (get_bit(in_nz + off[b], (uint32_t)(w[b] * 32 + bit) * S[b] + sc)) x[b] |= 1u << bit;
                }
            }
#pragma unroll
            for (int b = 0; b < kBatch; ++b)
                if (ok[b] && x[b]) atomicOr(prod[b] ? &s_prod[w[b]] : &s_cons[w[b]], x[b]);
        }
    }
    __syncthreads();
    uint32_t removed_local = 0;
    for (int w = threadIdx.x; w < n_words; w += kThreads) {
        const uint32_t valid = (w == n_words - 1 && (C & 31)) ? ((1u << (C & 31)) - 1u) : 0xffffffffu;
        uint32_t prod_dead = (n_prod > 0 && !frozen) ? ~s_prod[w] & valid : 0u;
        const uint32_t cons_dead = (n_cons > 0 && !frozen) ? ~s_cons[w] & valid : 0u;
        uint32_t shift_bad = 0;
        if ((policy & DNNS_SHIFT_STRICT) && prod_dead) {
            for (uint32_t m = prod_dead; m; m &= m - 1) {
                const int j = w * 32 + __ffs(m) - 1;
                for (int p = gd.prod_begin; p < gd.prod_end; ++p)
                    if (!shift_zero(tb, p, j)) shift_bad |= 1u << (j & 31);
            }
        }
        const uint32_t rem = ((policy & DNNS_RULE_PRODUCER) ? prod_dead & ~shift_bad : 0u) |
                             ((policy & DNNS_RULE_CONSUMER) ? cons_dead : 0u);
        s_rem[w] = rem;
        s_prod[w] = prod_dead & ~cons_dead;  // from here on: dead channel that somebody still reads
        removed_local += __popc(rem);
    }
    return removed_local;
}

// From the removal words of a group to its outputs: layer-collapse guard, keep bits, ascending index
// list, count, statistics.  removed_local: this thread's share of the removed-channel count.
__device__ __forceinline__ void finalize_group(const Tables& tb, const GroupDesc& gd, int g, int32_t min_keep,
                                               uint32_t removed_local, uint32_t* s_rem, const uint32_t* s_lost,
                                               uint32_t* s_pre, uint32_t* scratch, uint32_t* s_rekept,
                                               uint32_t* keep_bits, int32_t* keep_idx, int32_t* keep_count,
                                               unsigned long long* stats, const uint32_t* __restrict__ shift_bits = nullptr) {
    const int C = gd.C;
    const int n_words = (C + 31) / 32;
    uint32_t removed;
    block_exclusive_scan<uint32_t>(removed_local, scratch, &removed);

    // layer collapse guard: take removed channels back, lowest index first
    const int floor_keep = min(max(min_keep, 0), C);
    if (threadIdx.x == 0) {
        int need = floor_keep - (C - (int)removed);
        uint32_t rekept = 0;
        for (int w = 0; need > 0 && w < n_words; ++w) {
            while (need > 0 && s_rem[w]) {
                s_rem[w] &= s_rem[w] - 1;  // clear the lowest set bit
                --need;
                ++rekept;
            }
        }
        *s_rekept = rekept;
    }
    __syncthreads();

    // kept channels before each word, then the ascending index list
    uint32_t carry = 0;
    for (int base = 0; base < n_words; base += kThreads) {
        const int w = base + threadIdx.x;
        uint32_t keep_w = 0;
        if (w < n_words) {
            const uint32_t valid = (w == n_words - 1 && (C & 31)) ? ((1u << (C & 31)) - 1u) : 0xffffffffu;
            keep_w = ~s_rem[w] & valid;
            keep_bits[gd.off_bits + w] = keep_w;
        }
        uint32_t total;
        const uint32_t ex = block_exclusive_scan<uint32_t>(__popc(keep_w), scratch, &total);
        if (w < n_words) s_pre[w] = carry + ex;
        carry += total;
    }
    __syncthreads();
    unsigned long long lost_pairs = 0;
    for (int j = threadIdx.x; j < C; j += kThreads) {
        const uint32_t rem = s_rem[j >> 5], bit = 1u << (j & 31);
        if (!(rem & bit)) {
            keep_idx[gd.off_idx + s_pre[j >> 5] + __popc(~rem & (bit - 1u))] = j;
        } else if (stats && !shift_bits && (s_lost[j >> 5] & bit)) {
            for (int p = gd.prod_begin; p < gd.prod_end; ++p)
                if (!shift_zero(tb, p, j)) ++lost_pairs;
        }
    }
    if (stats && shift_bits) {
        // the same count word by word from the prepared bits: removed channels that somebody still reads, against
        // every producer's "constant is zero" word (eight producers' words requested together)
        constexpr int kProd = 8;
        for (int w = threadIdx.x; w < n_words; w += kThreads) {
            const uint32_t lost = s_rem[w] & s_lost[w];
            if (!lost) continue;
            for (int p0 = gd.prod_begin; p0 < gd.prod_end; p0 += kProd) {
                uint32_t z[kProd];
#pragma unroll
                for (int t = 0; t < kProd; ++t)
                    z[t] = p0 + t < gd.prod_end ? shift_bits[tb.producers[p0 + t].off_outnz + w] : 0xffffffffu;
#pragma unroll
                for (int t = 0; t < kProd; ++t) lost_pairs += __popc(lost & ~z[t]);
            }
        }
    }
    if (threadIdx.x == 0) keep_count[g] = (int32_t)carry;
    if (stats) {  // cleared by the entry point before the launch
        if (lost_pairs) atomicAdd(&stats[0], lost_pairs);
        if (threadIdx.x == 0) {
            if (C - (int)carry) atomicAdd(&stats[1], (unsigned long long)(C - (int)carry));
            if (*s_rekept) atomicAdd(&stats[2], (unsigned long long)*s_rekept);
        }
    }
}

__global__ void __launch_bounds__(kThreads) k_propagate(Tables tb, const uint32_t* __restrict__ out_nz,
                                                        const uint32_t* __restrict__ in_nz, uint32_t policy,
                                                        int32_t min_keep, uint32_t* keep_bits, int32_t* keep_idx,
                                                        int32_t* keep_count, unsigned long long* stats) {
    __shared__ uint32_t s_prod[kMaxGroupWords];  // some producer's filter j is alive; later: lost channels
    __shared__ uint32_t s_cons[kMaxGroupWords];  // some consumer reads channel j
    __shared__ uint32_t s_rem[kMaxGroupWords];   // channel j is removed
    __shared__ uint32_t s_pre[kMaxGroupWords];   // kept channels in earlier words
    __shared__ uint32_t scratch[33];
    __shared__ uint32_t s_rekept;
    const int g = blockIdx.x;
    const GroupDesc gd = tb.groups[g];
    const uint32_t removed_local = eval_group(tb, gd, out_nz, in_nz, policy, s_prod, s_cons, s_rem);
    finalize_group(tb, gd, g, min_keep, removed_local, s_rem, s_prod, s_pre, scratch, &s_rekept, keep_bits, keep_idx,
                   keep_count, stats);
}

// For the statistics: per producer (an entry of the producer list) and channel, whether the constant a zero filter
// still emits is structurally zero - the same for every variant of a call, so it is worked out once, a block per
// producer, a warp per word.
__global__ void __launch_bounds__(kThreads) k_shift_zero(Tables tb, unsigned long long* __restrict__ stats, int n_stats) {
    const int p = blockIdx.x;
    if (p == 0)  // the statistics of the propagation that follows start at zero
        for (int i = threadIdx.x; i < n_stats; i += kThreads) stats[i] = 0;
    const int C = tb.tensors[tb.prod_list[p]].O;
    const int n_words = (C + 31) / 32, lane = threadIdx.x & 31;
    uint32_t* out = tb.shift_zero + tb.producers[p].off_outnz;
    for (int w = threadIdx.x >> 5; w < n_words; w += kThreads / 32) {
        const int j = w * 32 + lane;
        const bool zero = j < C ? shift_zero(tb, p, j) : true;
        const uint32_t word = __ballot_sync(0xffffffffu, zero);
        if (lane == 0) out[w] = word;
    }
}

// The same for the variants of one multi-variant sweep in one launch: blockIdx.y picks the variant's buffers.
struct PropagateMultiArgs {
    const uint32_t* out_nz[kPortfolioMax];
    const uint32_t* in_nz[kPortfolioMax];
    uint32_t* keep_bits[kPortfolioMax];
    int32_t* keep_idx[kPortfolioMax];
    int32_t* keep_count[kPortfolioMax];
};

__global__ void __launch_bounds__(kThreads) k_propagate_multi(Tables tb, PropagateMultiArgs pa, uint32_t policy,
                                                              int32_t min_keep, unsigned long long* stats) {
    __shared__ uint32_t s_prod[kMaxGroupWords];
    __shared__ uint32_t s_cons[kMaxGroupWords];
    __shared__ uint32_t s_rem[kMaxGroupWords];
    __shared__ uint32_t s_pre[kMaxGroupWords];
    __shared__ uint32_t scratch[33];
    __shared__ uint32_t s_rekept;
    const int g = blockIdx.x, v = blockIdx.y;
    const GroupDesc gd = tb.groups[g];
    const uint32_t removed_local = eval_group(tb, gd, pa.out_nz[v], pa.in_nz[v], policy, s_prod, s_cons, s_rem);
    finalize_group(tb, gd, g, min_keep, removed_local, s_rem, s_prod, s_pre, scratch, &s_rekept, pa.keep_bits[v],
                   pa.keep_idx[v], pa.keep_count[v], stats ? stats + 4 * v : nullptr, tb.shift_zero);
}

// ---- fixed point: the rule applied pass after pass on kernel maps restricted to what is still kept
//
// Pass p: k_live recomputes the filter / input-column flags from the kernel maps, ignoring input
// channels and filters that pass p-1 removed; k_cascade_eval applies the rule to those flags and
// notes whether anything changed.  Removal only grows, so the passes after the one that changed
// nothing return at once; k_cascade_finish turns the final removal words into the outputs.

// Same units as the flag kernel of step 3 (see there), reading kernel-map words instead of building them.
__global__ void __launch_bounds__(256) k_live(Tables tb, const uint32_t* __restrict__ nz_map,
                                              const uint32_t* __restrict__ rem, uint32_t* live_out, uint32_t* live_in,
                                              const uint32_t* __restrict__ changed_before) {
    if (changed_before && *changed_before == 0) return;
    const int lane = threadIdx.x & 31;
    const uint32_t n_warps = gridDim.x * (blockDim.x >> 5), warp = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const uint32_t per = (tb.n_flag_units + n_warps - 1) / n_warps;
    const uint32_t lo = min(tb.n_flag_units, warp * per), hi = min(tb.n_flag_units, lo + per);
    if (lo >= hi) return;
    uint32_t t = tb.flag_unit_tensor[lo];  // the tensor holding unit lo
    uint32_t unit = lo;
    while (unit < hi) {
        const uint32_t t_begin = tb.flag_prefix[t], t_end = tb.flag_prefix[t + 1];
        if (unit >= t_end) {
            ++t;
            continue;
        }
        const TensorDesc& d = tb.tensors[t];
        const uint32_t I = d.I, O = d.O, n_kernels = O * I, S = d.S;
        const uint32_t* map = nz_map + d.off_nzmap;
        const uint32_t* rem_in = rem + tb.groups[d.in_group].off_bits;    // removed input channels
        const uint32_t* rem_out = rem + tb.groups[d.out_group].off_bits;  // removed filters
        uint32_t* g_in = live_in + d.off_innz;
        uint32_t* g_out = live_out + d.off_outnz;
        const uint32_t wpr = (S == 1 && I % 32 == 0 && ((I / 32) & (I / 32 - 1)) == 0) ? I / 32 : 0;
        const bool by_blocks = (I % 32 == 0 && ((I / 32) & (I / 32 - 1)) == 0);  // how the plan cut this tensor into units
        const uint32_t run_end = min(hi, t_end);
        if (wpr) {
            const uint32_t n_chunks = (wpr + 31) / 32, cw = min(wpr, 32u);
            const int cw_shift = __ffs(cw) - 1;
            for (; unit < run_end; ++unit) {
                const uint32_t local = unit - t_begin, rb = local / n_chunks, cc = local - rb * n_chunks;
                const uint32_t row0 = rb * kFlagRows, iw = cc * 32 + (lane & (cw - 1));
                const uint32_t kept_cols = ~rem_in[DNNS_IDX(iw, (I / S + 31) / 32)];
                uint32_t acc = 0, rows = 0;
                const uint32_t n_steps = (kFlagRows * cw + 31) / 32;
                const uint32_t group_mask = cw == 32 ? 0xffffffffu : ((1u << cw) - 1u);
                for (uint32_t step = 0; step < n_steps; ++step) {  // same trip count in every lane
                    const uint32_t k = step * 32 + lane;
                    const uint32_t o = row0 + (k >> cw_shift);
                    uint32_t word = 0;
                    bool row_kept = false;
                    if (k < kFlagRows * cw && o < O) {
                        word = __ldg(map + o * wpr + iw);
                        row_kept = !((rem_out[o >> 5] >> (o & 31)) & 1u);
                    }
                    if (row_kept) acc |= word;                       // columns some kept filter reads
                    const uint32_t nzl = __ballot_sync(0xffffffffu, (word & kept_cols) != 0);  // filters alive in kept columns
                    for (uint32_t g = 0; g < min(32u >> cw_shift, kFlagRows); ++g)
                        if ((nzl >> (g << cw_shift)) & group_mask) rows |= 1u << (((step * 32) >> cw_shift) + g);
                }
                if (lane == 0 && rows) atomicOr(&g_out[row0 >> 5], rows << (row0 & 31));
                for (uint32_t sft = cw; sft < 32; sft <<= 1) acc |= __shfl_xor_sync(0xffffffffu, acc, sft);
                if ((uint32_t)lane < cw && acc) atomicOr(&g_in[iw], acc);
            }
        } else {
            // one kernel per lane; a tensor the plan cut into filter blocks is walked kernel by kernel
            const uint32_t n_units_here = t_end - t_begin;
            for (; unit < run_end; ++unit) {
                // spread the tensor's kernels over its units, 32 per step
                const uint32_t per_unit = by_blocks ? ((n_kernels + n_units_here - 1) / n_units_here + 31) / 32 * 32 : 32;
                const uint32_t q_begin = (unit - t_begin) * per_unit, q_end = min(n_kernels, q_begin + per_unit);
                for (uint32_t qb = q_begin; qb < q_end; qb += 32) {
                    const uint32_t q = qb + lane;
                    if (q < q_end && ((map[DNNS_IDX(q >> 5, (n_kernels + 31) / 32)] >> (q & 31)) & 1u)) {
                        const uint32_t o = q / I, i = q - o * I, c = i / S;
                        if (!((rem_in[c >> 5] >> (c & 31)) & 1u)) atomicOr(&g_out[o >> 5], 1u << (o & 31));
                        if (!((rem_out[o >> 5] >> (o & 31)) & 1u)) atomicOr(&g_in[i >> 5], 1u << (i & 31));
                    }
                }
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads) k_cascade_eval(Tables tb, const uint32_t* __restrict__ live_out,
                                                           const uint32_t* __restrict__ live_in, uint32_t policy,
                                                           const uint32_t* __restrict__ rem_prev, uint32_t* rem_next,
                                                           uint32_t* lost, const uint32_t* __restrict__ changed_before,
                                                           uint32_t* changed_now) {
    if (changed_before && *changed_before == 0) return;
    __shared__ uint32_t s_prod[kMaxGroupWords], s_cons[kMaxGroupWords], s_rem[kMaxGroupWords];
    const int g = blockIdx.x;
    const GroupDesc gd = tb.groups[g];
    eval_group(tb, gd, live_out, live_in, policy, s_prod, s_cons, s_rem);
    __syncthreads();
    const int n_words = (gd.C + 31) / 32;
    bool differs = false;
    for (int w = threadIdx.x; w < n_words; w += kThreads) {
        const uint32_t r = s_rem[w] | rem_prev[gd.off_bits + w];  // removal only grows
        differs |= r != rem_prev[gd.off_bits + w];
        rem_next[gd.off_bits + w] = r;
        lost[gd.off_bits + w] = s_prod[w];
    }
    if (differs) atomicOr(changed_now, 1u);
}

__global__ void __launch_bounds__(kThreads) k_cascade_finish(Tables tb, const uint32_t* __restrict__ rem,
                                                             const uint32_t* __restrict__ lost, int32_t min_keep,
                                                             const uint32_t* __restrict__ changed, int n_passes,
                                                             uint32_t* keep_bits, int32_t* keep_idx, int32_t* keep_count,
                                                             unsigned long long* stats) {
    __shared__ uint32_t s_rem[kMaxGroupWords], s_lost[kMaxGroupWords], s_pre[kMaxGroupWords];
    __shared__ uint32_t scratch[33];
    __shared__ uint32_t s_rekept;
    const int g = blockIdx.x;
    const GroupDesc gd = tb.groups[g];
    const int n_words = (gd.C + 31) / 32;
    uint32_t removed_local = 0;
    for (int w = threadIdx.x; w < n_words; w += kThreads) {
        s_rem[w] = rem[gd.off_bits + w];
        s_lost[w] = lost[gd.off_bits + w];
        removed_local += __popc(s_rem[w]);
    }
    __syncthreads();
    finalize_group(tb, gd, g, min_keep, removed_local, s_rem, s_lost, s_pre, scratch, &s_rekept, keep_bits, keep_idx,
                   keep_count, stats);
    if (stats && g == 0 && threadIdx.x == 0) {
        unsigned long long passes = 0;
        for (int p = 1; p <= n_passes; ++p) passes += changed[p];
        stats[3] = passes;
    }
}

}  // namespace

int launch_propagate(const Tables& tb, const uint32_t* out_nz, const uint32_t* in_nz, uint32_t policy,
                     int32_t min_keep, uint32_t* keep_bits, int32_t* keep_idx, int32_t* keep_count, uint64_t* stats,
                     cudaStream_t st) {
    ScopedKernel timed("k_propagate", st);
    k_propagate<<<tb.n_groups, kThreads, 0, st>>>(tb, out_nz, in_nz, policy, min_keep, keep_bits, keep_idx,
                                                  keep_count, reinterpret_cast<unsigned long long*>(stats));
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_propagate_multi(const Tables& tb, int n_variants, const uint32_t* const* out_nz, const uint32_t* const* in_nz,
                           uint32_t policy, int32_t min_keep, uint32_t* const* keep_bits, int32_t* const* keep_idx,
                           int32_t* const* keep_count, uint64_t* stats, cudaStream_t st) {
    PropagateMultiArgs pa{};
    for (int v = 0; v < n_variants; ++v) {
        pa.out_nz[v] = out_nz[v], pa.in_nz[v] = in_nz[v];
        pa.keep_bits[v] = keep_bits[v], pa.keep_idx[v] = keep_idx[v], pa.keep_count[v] = keep_count[v];
    }
    int launches = 1;
    if (stats) {
        ScopedKernel timed("k_shift_zero", st);
        k_shift_zero<<<tb.n_tensors, kThreads, 0, st>>>(tb, reinterpret_cast<unsigned long long*>(stats), 4 * n_variants);  // the producer list has an entry per tensor
        ++launches;
    }
    ScopedKernel timed("k_propagate", st);
    k_propagate_multi<<<dim3(tb.n_groups, n_variants), kThreads, 0, st>>>(tb, pa, policy, min_keep,
                                                                        reinterpret_cast<unsigned long long*>(stats));
    return cudaGetLastError() == cudaSuccess ? launches : -1;
}

int launch_propagate_cascade(const Tables& tb, const CascadeWs& cw, const uint32_t* nz_map, uint32_t policy,
                             int32_t min_keep, int32_t max_passes, uint32_t* keep_bits, int32_t* keep_idx,
                             int32_t* keep_count, uint64_t* stats, uint32_t n_keep_words, uint32_t n_live_words, int n_sm,
                             cudaStream_t st) {
    // changed[0] = 1 (there is always a first pass), changed[p] is set by pass p; removal words start at zero
    if (cudaMemsetAsync(cw.changed, 0, 4 * (size_t)(max_passes + 1), st) != cudaSuccess ||
        cudaMemsetAsync(cw.rem[0], 0, 4 * (size_t)n_keep_words, st) != cudaSuccess)
        return -1;
    const uint32_t live_blocks = min((uint32_t)n_sm * 64u, (tb.n_flag_units + 7) / 8);
    int launches = 0;
    for (int p = 1; p <= max_passes; ++p) {
        const uint32_t* before = p == 1 ? nullptr : cw.changed + (p - 1);
        if (cudaMemsetAsync(cw.live, 0, 4 * (size_t)n_live_words, st) != cudaSuccess) return -1;
        k_live<<<max(live_blocks, 1u), 256, 0, st>>>(tb, nz_map, cw.rem[(p - 1) & 1], cw.live, cw.live + cw.live_in_offset,
                                                     before);
        k_cascade_eval<<<tb.n_groups, kThreads, 0, st>>>(tb, cw.live, cw.live + cw.live_in_offset, policy,
                                                         cw.rem[(p - 1) & 1], cw.rem[p & 1], cw.lost, before, cw.changed + p);
        launches += 2;
    }
    k_cascade_finish<<<tb.n_groups, kThreads, 0, st>>>(tb, cw.rem[max_passes & 1], cw.lost, min_keep, cw.changed, max_passes,
                                                       keep_bits, keep_idx, keep_count,
                                                       reinterpret_cast<unsigned long long*>(stats));
    return cudaGetLastError() == cudaSuccess ? launches + 1 : -1;
}

#ifdef DNNS_BOUNDS_CHECK
unsigned int bounds_violations_propagate(bool reset) {
    unsigned int n = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&n, g_bounds_violations, sizeof(n)) != cudaSuccess) return 0xFFFFFFFFu;
    if (reset) cudaMemcpyToSymbol(g_bounds_violations, &zero, sizeof(zero));
    return n;
}
#endif

}  // namespace dnns
