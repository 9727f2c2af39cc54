// Step 4: keep sets per channel group - Module 3, the Prune Planner (Algorithm 1), for every
// group of the model in one launch.  Algorithm 1 hands layer L_n the zero channels of L_n as
// C_out and those of L_{n-1} as C_in; the two are one set of channels, a "group", which with
// residual adds has several producers and consumers.  One block per group; the data are a few
// kilobytes of flag bits, so the launch is latency-bound by design.
#include "dnns_internal.cuh"

namespace dnns {

namespace {

constexpr int kThreads = 256;
constexpr int kMaxGroupWords = 65536 / 32;

__device__ __forceinline__ bool get_bit(const uint32_t* w, uint32_t b) { return (w[b >> 5] >> (b & 31)) & 1u; }

// The constant a zero filter of producer `t` still emits on channel j is structurally zero.
__device__ __forceinline__ bool shift_zero(const Tables& tb, int t, int j) {
    const TensorDesc& d = tb.tensors[t];
    const float bias = d.bias ? d.bias[j] : 0.0f;
    if (d.bn >= 0) {
        const BnDesc& b = tb.bns[d.bn];
        return b.beta[j] == 0.0f && (b.gamma[j] == 0.0f || b.mean[j] == bias);
    }
    return bias == 0.0f;
}

__global__ void __launch_bounds__(kThreads) k_propagate(Tables tb, const uint32_t* __restrict__ out_nz,
                                                        const uint32_t* __restrict__ in_nz, uint32_t policy,
                                                        int32_t min_keep, uint32_t* keep_bits, int32_t* keep_idx,
                                                        int32_t* keep_count, unsigned long long* stats) {
    __shared__ uint32_t s_rem[kMaxGroupWords];   // channel is removed
    __shared__ uint32_t s_lost[kMaxGroupWords];  // all producers dead while some consumer still reads it
    __shared__ uint32_t scratch[33];
    __shared__ uint32_t s_rekept;
    const int g = blockIdx.x;
    const GroupDesc gd = tb.groups[g];
    const int C = gd.C;
    const int lane = threadIdx.x & 31;
    const bool frozen = gd.flags & DNNS_GROUP_FROZEN;
    const int n_prod = gd.prod_end - gd.prod_begin, n_cons = gd.cons_end - gd.cons_begin;

    uint32_t removed_local = 0;
    for (int base = 0; base < C; base += kThreads) {
        const int j = base + threadIdx.x;
        bool remove = false, lost = false;
        if (j < C && !frozen) {
            bool prod_dead = n_prod > 0;
            for (int p = gd.prod_begin; p < gd.prod_end; ++p) {
                const TensorDesc& d = tb.tensors[tb.prod_list[p]];
                if (get_bit(out_nz + d.off_outnz, j)) prod_dead = false;
            }
            bool cons_dead = n_cons > 0;
            for (int q = gd.cons_begin; q < gd.cons_end; ++q) {
                const TensorDesc& d = tb.tensors[tb.cons_list[q]];
                for (int s = 0; s < d.S; ++s)
                    if (get_bit(in_nz + d.off_innz, (uint32_t)j * d.S + s)) cons_dead = false;
            }
            bool shift_ok = true;
            if ((policy & DNNS_SHIFT_STRICT) && prod_dead)
                for (int p = gd.prod_begin; p < gd.prod_end; ++p)
                    if (!shift_zero(tb, tb.prod_list[p], j)) shift_ok = false;
            remove = ((policy & DNNS_RULE_PRODUCER) && prod_dead && shift_ok) ||
                     ((policy & DNNS_RULE_CONSUMER) && cons_dead);
            lost = prod_dead && !cons_dead;
        }
        const uint32_t rw = __ballot_sync(0xffffffffu, remove), lw = __ballot_sync(0xffffffffu, lost);
        if (lane == 0 && base + (int)(threadIdx.x & ~31u) < C) {
            s_rem[j >> 5] = rw;
            s_lost[j >> 5] = lw;
            removed_local += __popc(rw);
        }
    }
    uint32_t removed;
    block_exclusive_scan<uint32_t>(removed_local, scratch, &removed);

    // layer collapse guard: take removed channels back, lowest index first
    const int floor_keep = min(max(min_keep, 0), C);
    if (threadIdx.x == 0) {
        int need = floor_keep - (C - (int)removed);
        uint32_t rekept = 0;
        for (int w = 0; need > 0 && w < (C + 31) / 32; ++w) {
            while (need > 0 && s_rem[w]) {
                s_rem[w] &= s_rem[w] - 1;  // clear the lowest set bit
                --need;
                ++rekept;
            }
        }
        s_rekept = rekept;
    }
    __syncthreads();

    uint32_t carry = 0;
    unsigned long long lost_pairs = 0;
    for (int base = 0; base < C; base += kThreads) {
        const int j = base + threadIdx.x;
        const bool valid = j < C;
        const bool keep = valid && !get_bit(s_rem, j);
        uint32_t total;
        const uint32_t ex = block_exclusive_scan<uint32_t>(keep, scratch, &total);
        if (keep) keep_idx[gd.off_idx + carry + ex] = j;
        carry += total;
        const uint32_t kw = __ballot_sync(0xffffffffu, keep);
        if (lane == 0 && base + (int)(threadIdx.x & ~31u) < C) keep_bits[gd.off_bits + (j >> 5)] = kw;
        if (stats && valid && !keep && get_bit(s_lost, j))
            for (int p = gd.prod_begin; p < gd.prod_end; ++p)
                if (!shift_zero(tb, tb.prod_list[p], j)) ++lost_pairs;
    }
    if (threadIdx.x == 0) keep_count[g] = (int32_t)carry;
    if (stats) {
        if (lost_pairs) atomicAdd(&stats[0], lost_pairs);
        if (threadIdx.x == 0) {
            atomicAdd(&stats[1], (unsigned long long)(C - (int)carry));
            atomicAdd(&stats[2], (unsigned long long)s_rekept);
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
