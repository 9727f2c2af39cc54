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

__device__ __forceinline__ bool get_bit(const uint32_t* w, uint32_t b) { return (w[b >> 5] >> (b & 31)) & 1u; }

// The constant a zero filter of producer p (an index into the producer list) still emits on channel
// j is structurally zero.
__device__ __forceinline__ bool shift_zero(const Tables& tb, int p, int j) {
    const ProducerDesc d = tb.producers[p];
    const float bias = d.bias ? d.bias[j] : 0.0f;
    if (d.beta) return d.beta[j] == 0.0f && (d.gamma[j] == 0.0f || d.mean[j] == bias);
    return bias == 0.0f;
}

__global__ void __launch_bounds__(kThreads) k_propagate(Tables tb, const uint32_t* __restrict__ out_nz,
                                                        const uint32_t* __restrict__ in_nz, uint32_t policy,
                                                        int32_t min_keep, uint32_t* keep_bits, int32_t* keep_idx,
                                                        int32_t* keep_count, unsigned long long* stats) {
    __shared__ uint32_t s_prod[kMaxGroupWords];  // some producer's filter j is alive
    __shared__ uint32_t s_cons[kMaxGroupWords];  // some consumer reads channel j
    __shared__ uint32_t s_rem[kMaxGroupWords];   // channel j is removed
    __shared__ uint32_t s_pre[kMaxGroupWords];   // kept channels in earlier words
    __shared__ uint32_t scratch[33];
    __shared__ uint32_t s_rekept;
    const int g = blockIdx.x;
    const GroupDesc gd = tb.groups[g];
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
        const int n_pw = n_prod * n_words;
        for (int it = threadIdx.x; it < n_pw + n_cons * n_words; it += kThreads) {
            if (it < n_pw) {
                const int p = it / n_words, w = it - p * n_words;
                const uint32_t x = out_nz[tb.producers[gd.prod_begin + p].off_outnz + w];
                if (x) atomicOr(&s_prod[w], x);
                continue;
            }
            const int q = (it - n_pw) / n_words, w = (it - n_pw) - q * n_words;
            const ConsumerDesc d = tb.consumers[gd.cons_begin + q];
            uint32_t x = 0;
            if (d.S == 1) {
                x = in_nz[d.off_innz + w];
            } else {
                for (int b = 0; b < 32 && w * 32 + b < C; ++b)
                    for (int s = 0; s < d.S; ++s)
                        if (get_bit(in_nz + d.off_innz, (uint32_t)(w * 32 + b) * d.S + s)) x |= 1u << b;
            }
            if (x) atomicOr(&s_cons[w], x);
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
        s_rekept = rekept;
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
        } else if (stats && (s_prod[j >> 5] & bit)) {
            for (int p = gd.prod_begin; p < gd.prod_end; ++p)
                if (!shift_zero(tb, p, j)) ++lost_pairs;
        }
    }
    if (threadIdx.x == 0) keep_count[g] = (int32_t)carry;
    if (stats) {  // cleared by the entry point before the launch
        if (lost_pairs) atomicAdd(&stats[0], lost_pairs);
        if (threadIdx.x == 0) {
            if (C - (int)carry) atomicAdd(&stats[1], (unsigned long long)(C - (int)carry));
            if (s_rekept) atomicAdd(&stats[2], (unsigned long long)s_rekept);
        }
    }
}

}  // namespace

int launch_propagate(const Tables& tb, const uint32_t* out_nz, const uint32_t* in_nz, uint32_t policy,
                     int32_t min_keep, uint32_t* keep_bits, int32_t* keep_idx, int32_t* keep_count, uint64_t* stats,
                     cudaStream_t st) {
    k_propagate<<<tb.n_groups, kThreads, 0, st>>>(tb, out_nz, in_nz, policy, min_keep, keep_bits, keep_idx,
                                                  keep_count, reinterpret_cast<unsigned long long*>(stats));
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace dnns
